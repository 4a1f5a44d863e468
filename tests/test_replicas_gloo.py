"""The benchmark's multi-GPU mode is "replicas only": N independent searches, no collective on
the data path.  The only cross-rank step is the combination of the ranks' measurements (slowest
replica for times, sum for throughput); it is exercised here with two gloo ranks on the CPU."""
import os
import socket
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out_dir: str):
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    torch.distributed.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # rank r measured: step time 10 + r, search 4 + 0.5 r, end-to-end 5 - r, 100 (r + 1) tokens/s
        got = bench.combine_replicas(10.0 + rank, 4.0 + 0.5 * rank, 5.0 - rank, 100.0 * (rank + 1), world,
                                     torch.device("cpu"))
        torch.save(got, os.path.join(out_dir, f"r{rank}.pt"))
    finally:
        torch.distributed.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_summed_throughput(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        total_ms, dp_ms, e2e_ms, tok_s = torch.load(os.path.join(str(tmp_path), f"r{r}.pt"))
        assert (total_ms, dp_ms, e2e_ms, tok_s) == (11.0, 4.5, 5.0, 300.0)


def test_single_replica_is_passed_through():
    import bench
    assert bench.combine_replicas(1.0, 2.0, 3.0, 4.0, 1, torch.device("cpu")) == (1.0, 2.0, 3.0, 4.0)


def test_plain_invocation_with_gpus_2_starts_two_ranks_itself():
    """`python bench.py --gpus 2` without torchrun launches the two ranks on 127.0.0.1 and reports
    n_gpus = 2 (checked with the GPU-free combine-check mode: gloo, made-up measurements)."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--mode", "combine-check"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                       # rank 0 alone prints
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2
    assert (out["ms_per_step"], out["value"], out["e2e"], out["decode_tokens_per_s"]) == (11.0, 4.5, 5.0, 300.0)
