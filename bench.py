#!/usr/bin/env python
"""Benchmark of the layer-skip search hot path on a B200.

A "step" is one round of the self-speculative loop on the LLaMA3-8B shape with a
512-token verified context: K draft tokens through the layer-skipped model, one
full-model verification pass over K+1 tokens, greedy acceptance, and the dynamic-
programming layer search (M = 12) on the last accepted token.  The headline value is
the search's latency per verification, measured with CUDA events inside the timed steps.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 runs N independent replicas, one per GPU: the path is a single sequence and does not
shard, so there is no collective on the data path.  Under torchrun the ranks are the
replicas; a plain `python bench.py --gpus N` starts the N ranks itself (one torchrun-style
launch on 127.0.0.1).
--impl reference times the CPU oracle (a deliberately plain program) on a bounded
sample of the same workload.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import socket
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import datagen  # noqa: E402

WORKLOADS = {
    # the headline workload: LLaMA3-8B shape, 512-token context, M = 12, one objective token
    "8b-c512-M12": dict(model="8b", ctx=512, M=12, T=1, K=4),
    # small stand-ins for quick checks and profiler captures (not bench lines)
    "8b-l6-c512-M3": dict(model="8b-l6", ctx=512, M=3, T=1, K=4),
    "mini8b-c128-M2": dict(model="mini8b", ctx=128, M=2, T=1, K=3),
    "tiny-c64-M2": dict(model="tiny", ctx=64, M=2, T=1, K=4),
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.rows = []
        self.proc = None

    def start(self):
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def workload_config(name: str, world: int) -> dict:
    """The `config` object of the JSON line: the same for the CUDA arm and the oracle arm."""
    wl = WORKLOADS[name]
    cfg = datagen.CONFIGS[wl["model"]]
    return {"workload": name, "model_shape": cfg.name, "L": cfg.L, "M": wl["M"], "T": wl["T"],
            "draft_len": wl["K"], "ctx_len": wl["ctx"], "replicas": world,
            "l2": "inputs larger than L2 (every layer's matrices are streamed once per search)"}


KERNEL_SOURCES = ["engine2.cuh", "gemm_tc.cuh", "kernels.cuh", "clasp_api.cu"]


def kernel_sources_digest() -> str:
    """Digest of the CUDA sources: ties a stored profiler figure to the kernel it was taken from."""
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2505_24196_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(workload: str):
    """DRAM bytes (read + write) of one launch of the dominant kernel from the committed ncu summary of
    this workload -- or None when the CUDA sources have changed since that capture (the summary names
    the digest of the sources it was taken from)."""
    path = os.path.join(ROOT, "profiles", "engine_kernel_8b_l6_c512_M3_ncu.md")
    if workload != "8b-c512-M12" or not os.path.exists(path):
        return None, "no capture for this workload"
    text = open(path).read()
    m = re.search(r"traffic_bytes_per_search_launch:\s*(\d+)", text)
    g = re.search(r"kernel_sources_digest:\s*([0-9a-f]+)", text)
    if not m or not g:
        return None, "summary holds no machine-readable figure"
    if g.group(1) != kernel_sources_digest():
        return None, "kernel sources changed since the capture in profiles/engine_kernel_8b_l6_c512_M3_ncu.md"
    return int(m.group(1)), "profiles/engine_kernel_8b_l6_c512_M3_ncu.md (6-layer capture x 31 / 5 applied layers)"


def dp_algorithmic_bytes(cfg, ctx_len: int) -> int:
    """Bytes the search must move: the matrices of layers 1..L-1 once, plus the visible
    K/V of those layers once."""
    esz = 2 if cfg.dtype == "bf16" else 4
    kv = 2 * ctx_len * cfg.n_kv_heads * cfg.head_dim * esz
    return (cfg.L - 1) * (cfg.layer_matrix_bytes() + kv)


# --------------------------------------------------------------------------- ours

def run_ours(args, rank, world):
    import paper_2505_24196_b200 as clasp
    from paper_2505_24196_b200.binding import _check
    wl = WORKLOADS[args.workload]
    cfg = datagen.CONFIGS[wl["model"]]
    M, T, K, C0 = wl["M"], wl["T"], wl["K"], wl["ctx"]
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    steps, warmup = args.steps, max(args.warmup, 3)
    max_ctx = C0 + (steps + warmup + 4) * (K + 1) * 2 + 64
    ccfg = clasp.make_config(cfg, max_ctx=max_ctx, max_rows=128, max_M=max(M, 1), max_T=T,
                             max_head_rows=K + 1)
    eng = clasp.Clasp(ccfg, device=dev)
    t0 = time.time()
    layers = [datagen.layer_weights(cfg, l, dev) for l in range(cfg.L)]
    head = datagen.head_weights(cfg, dev)
    eng.load_layers(0, layers)
    eng.load_head(head)
    torch.cuda.synchronize()
    t_gen = time.time() - t0
    kv = clasp.KVCache(ccfg, device=dev)
    prompt = datagen.token_ids(cfg, C0, stream=rank).tolist()
    dec = clasp.SelfSpeculativeDecoder(eng, kv, M=M, K=K, time_stages=True)
    dec.prefill(prompt)
    torch.cuda.synchronize()
    if args.mode == "dp-only":
        return dp_only(args, eng, dec, kv, cfg, wl)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        dec.round()
    for k in dec.stage_ms:
        dec.stage_ms[k] = 0.0
    n_rounds0 = len(dec.rounds)
    launches0 = eng.launch_count()
    sampler = ClockSampler(local)
    sampler.start()
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.profiler.start()   # lets `ncu --profile-from-start off` list only the timed region's launches
    ev0.record(eng.stream)
    new_tokens = 0
    for _ in range(steps):
        new_tokens += len(dec.round())
    ev1.record(eng.stream)
    barrier()
    torch.cuda.profiler.stop()
    total_ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop()
    launches = eng.launch_count() - launches0
    stage = {k: v / steps for k, v in dec.stage_ms.items()}
    dp_ms = stage["dp"]
    accepted = [r["accepted"] for r in dec.rounds[n_rounds0:]]
    ctx_now = dec.n_valid

    # ---- end to end through the C ABI with host buffers: the objective's hidden states come
    # from pinned host memory each step and the mask and score table go back to the host.
    L, d = cfg.L, cfg.d_model
    hid_host = dec.hidden[0].cpu().pin_memory()
    hid_dev = torch.empty_like(dec.hidden[0])
    mask_host = torch.empty(L, dtype=torch.uint8).pin_memory()
    score_host = torch.empty((L + 1, M + 1), dtype=torch.float32).pin_memory()
    obj = ctx_now - 1
    e2e_ms = []
    for it in range(3 + steps):
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(eng.stream)
        hid_dev.copy_(hid_host, non_blocking=True)
        r = eng.dp_search(hid_dev, d, 0, kv, obj, obj, T, M, want_margins=False, want_g=False)
        mask_host.copy_(r["S"], non_blocking=True)
        score_host.copy_(r["D"], non_blocking=True)
        b.record(eng.stream)
        b.synchronize()
        if it >= 3:
            e2e_ms.append(a.elapsed_time(b))
    e2e_val = sum(e2e_ms) / len(e2e_ms)
    h2d = hid_host.numel() * 4
    d2h = mask_host.numel() + score_host.numel() * 4

    # ---- per-launch timing of the dominant kernel (the persistent layer kernel: one launch is a
    # whole search): the library brackets each launch with CUDA events on its own stream.
    roof = None
    if hasattr(eng.lib, "clasp_profile_gemm"):
        roof = gemm_roofline(eng, dec, kv, hid_dev, obj, T, M, d)
        roof["traffic"], roof["traffic_source"] = ncu_traffic(args.workload)
        roof["traffic_unit"] = "bytes per launch (ncu dram__bytes_read.sum + dram__bytes_write.sum)"
    peak, which = measured_peaks()
    alg_bytes = dp_algorithmic_bytes(cfg, obj)
    dp_gbs = alg_bytes / (dp_ms * 1e-3) / 1e9

    status = eng.device_status()
    if status != 0:
        raise RuntimeError(f"device status {status}")

    # max over ranks of the time-like numbers, sum of the throughput
    tok_s = new_tokens / (total_ms * 1e-3)
    total_ms, dp_ms, e2e_val, tok_s = combine_replicas(total_ms, dp_ms, e2e_val, tok_s, world, dev)
    out = {
        "metric": "dp_search_ms_per_verify", "value": round(dp_ms, 4), "unit": "ms",
        "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": round(total_ms / steps, 4),
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if cfg.dtype == "bf16" else "f32",
        "data": "synthetic (seeded random-init weights, uniform random token ids)",
        "config": workload_config(args.workload, world),
        "run": {"ctx_len_after_timed_rounds": ctx_now, "kernel_sources_digest": kernel_sources_digest()},
        "stage_ms": {k: round(v, 4) for k, v in stage.items()},
        "decode_tokens_per_s": round(tok_s, 2),
        "mean_accepted": round(sum(accepted) / max(len(accepted), 1), 3),
        "dp_hbm": {"algorithmic_bytes": alg_bytes, "achieved_gbs": round(dp_gbs, 1),
                   "frac_of_measured_copy": round(dp_gbs / peak, 4), "frac_of_8tbs_nominal": round(dp_gbs / 8000.0, 4),
                   "peak_source": which},
        "e2e": {"value": round(e2e_val, 4), "unit": "ms", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "setup_s": {"weights": round(t_gen, 1)},
    }
    if roof is not None:
        out["roofline"] = roof
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(cfg, wl, layers=layers, head=head)
    if rank == 0:
        print(json.dumps(out), flush=True)


def combine_replicas(total_ms, dp_ms, e2e_ms, tok_s, world, device):
    """Replicas only: every rank runs the same independent job.  Time-like numbers are the maximum
    over the ranks (the slowest replica), throughput is the sum.  No data crosses between replicas."""
    if world > 1:
        t = torch.tensor([total_ms, dp_ms, e2e_ms], device=device, dtype=torch.float64)
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
        total_ms, dp_ms, e2e_ms = t.tolist()
        s = torch.tensor([tok_s], device=device, dtype=torch.float64)
        torch.distributed.all_reduce(s, op=torch.distributed.ReduceOp.SUM)
        tok_s = float(s[0])
    return total_ms, dp_ms, e2e_ms, tok_s


def dp_only(args, eng, dec, kv, cfg, wl):
    """Profiling aid: after the prefill, run only the layer search `steps` times inside a
    cudaProfilerStart/Stop range (for `ncu --profile-from-start off`) and print its latency."""
    M, T, C0 = wl["M"], wl["T"], wl["ctx"]
    d = cfg.d_model
    toks = torch.as_tensor(datagen.token_ids(cfg, 1, stream=9).tolist(), dtype=torch.int32).cuda()
    _, hid = eng.verify(toks, C0, kv, 1)
    for _ in range(max(args.warmup, 1)):
        eng.dp_search(hid[0], d, 0, kv, C0, C0, T, M, want_margins=False, want_g=False)
    torch.cuda.synchronize()
    torch.cuda.profiler.start()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n0 = eng.launch_count()
    a.record(eng.stream)
    for _ in range(args.steps):
        eng.dp_search(hid[0], d, 0, kv, C0, C0, T, M, want_margins=False, want_g=False)
    b.record(eng.stream)
    torch.cuda.synchronize()
    torch.cuda.profiler.stop()
    ms = a.elapsed_time(b) / args.steps
    byts = dp_algorithmic_bytes(cfg, C0)
    print(json.dumps({"mode": "dp-only", "workload": args.workload, "dp_ms": round(ms, 4),
                      "gbs": round(byts / ms / 1e6, 1), "launches_per_search": (eng.launch_count() - n0) // args.steps,
                      "device_status": eng.device_status()}), flush=True)


def gemm_roofline(eng, dec, kv, hid_dev, obj, T, M, d):
    import ctypes as C
    lib = eng.lib
    lib.clasp_profile_gemm.restype = C.c_int
    lib.clasp_profile_gemm.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_double),
                                       C.POINTER(C.c_double)]
    n, ms, byts = C.c_int64(), C.c_double(), C.c_double()
    lib.clasp_profile_gemm(eng.handle, 1, None, None, None)
    for _ in range(3):
        eng.dp_search(hid_dev, d, 0, kv, obj, obj, T, M, want_margins=False, want_g=False)
    lib.clasp_profile_gemm(eng.handle, 0, C.byref(n), C.byref(ms), C.byref(byts))
    peak, which = measured_peaks()
    achieved = byts.value / (ms.value * 1e-3) / 1e9 if ms.value > 0 else 0.0
    return {"bound": "hbm", "kernel": "pk::engine_kernel (one launch = one whole search)", "achieved": round(achieved, 1), "peak": peak,
            "unit": "GB/s", "frac": round(achieved / peak, 4), "peak_source": which + " copy bandwidth",
            "launches_timed": int(n.value), "avg_launch_us": round(ms.value * 1e3 / max(n.value, 1), 2),
            "traffic": None}


# --------------------------------------------------------------------------- CPU oracle legs

def oracle_sample(cfg, wl, layers=None, head=None, n_steps=5, repeats=1):
    """Times the oracle's search on a bounded sample: the first n_steps DP steps (layers
    1..n_steps-1 applied) on the same seeded workload.  The full-model states and the cache
    those steps need come from the oracle's own prefill of the first n_steps layers."""
    import numpy as np
    from oracle import clasp_oracle as orc
    from oracle import from_torch
    import dataclasses
    sub = dataclasses.replace(cfg, L=n_steps)            # same layer stream, first n_steps layers
    if layers is None:
        # seeded inputs only: the generator is plain torch arithmetic, run where it is fastest
        gen_dev = "cuda" if torch.cuda.is_available() else "cpu"
        lay = lambda l: {k: v.cpu() for k, v in datagen.layer_weights(cfg, l, gen_dev).items()}
        hd = {"embed": datagen.make_tensor(cfg, 1 << 20, "embed", 0, gen_dev).cpu()}
    else:
        lay = lambda l: layers[l]
        hd = {"embed": head["embed"]}
    # float64 copies of the sampled layers are made before the clock starts: the timed region is the
    # oracle's arithmetic, not the conversion of its inputs
    model = from_torch.model_from_tensors(sub, lay, None, resident=True)
    C0, M = wl["ctx"], wl["M"]
    toks = datagen.token_ids(cfg, C0, stream=0).numpy().astype(np.int64)
    emb = from_torch.to_f64(hd["embed"][torch.as_tensor(toks).to(hd["embed"].device)])
    cache = orc.KVCache(sub, C0)
    t0 = time.time()
    hidden = orc.forward_hidden(model, emb, cache, 0)
    t_prefill = time.time() - t0
    x = hidden[C0 - 1][:, None, :]
    times = []
    res = None
    for _ in range(repeats):
        t0 = time.time()
        res = orc.dp_search(model, x, cache, C0 - 1, C0 - 1, min(M, n_steps))
        times.append(time.time() - t0)
    return times, t_prefill, res


def layer_row_applications(L, M, n_steps=None):
    """Decoder-layer passes over one candidate state that Algorithm 1 makes in its first n_steps steps
    (all L when None): sum over i of min(i - 1, M).  The oracle's cost is proportional to it."""
    n = L if n_steps is None else n_steps
    return sum(min(i - 1, M) for i in range(1, n + 1))


def cpu_baseline(cfg, wl, layers=None, head=None):
    n_steps = min(8, cfg.L)
    times, t_prefill, _ = oracle_sample(cfg, wl, layers, head, n_steps)
    t_dp = times[0]
    full, part = layer_row_applications(cfg.L, wl["M"]), layer_row_applications(cfg.L, wl["M"], n_steps)
    scale = full / part
    return {"value": round(t_dp * 1e3 * scale, 1), "unit": "ms", "cores": torch.get_num_threads(),
            "kind": "oracle",
            "sample": (f"DP steps i=1..{n_steps} of {cfg.L} on the same workload ({part} of the search's {full} "
                       f"layer passes over one state, {t_dp:.2f} s measured), scaled by {full}/{part}; the oracle's "
                       f"prefill of those layers ({t_prefill:.1f} s) and the float64 copies of its inputs not counted")}


def run_reference(args, rank, world):
    if rank != 0:
        return
    wl = WORKLOADS[args.workload]
    cfg = datagen.CONFIGS[wl["model"]]
    n_steps = min(4, cfg.L)
    steps, warmup = args.steps, args.warmup
    times, _, _ = oracle_sample(cfg, wl, n_steps=n_steps, repeats=warmup + steps)
    times = times[warmup:]
    full, part = layer_row_applications(cfg.L, wl["M"]), layer_row_applications(cfg.L, wl["M"], n_steps)
    scale = full / part
    val = sum(times) / len(times) * 1e3 * scale
    sample = (f"per step: oracle DP steps i=1..{n_steps} of {cfg.L} ({part} of the search's {full} layer passes "
              f"over one state), scaled by {full}/{part}")
    out = {"impl": "reference", "metric": "dp_search_ms_per_verify", "value": round(val, 1), "unit": "ms",
           "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": round(val, 1),
           "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
           "data": "synthetic (seeded random-init weights, uniform random token ids)",
           "config": workload_config(args.workload, world),
           "cpu_baseline": {"value": round(val, 1), "unit": "ms", "cores": torch.get_num_threads(),
                            "kind": "oracle", "sample": sample},
           "e2e": {"value": round(val, 1), "unit": "ms", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


# --------------------------------------------------------------------------- replicas

def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch_replicas(n: int, argv) -> int:
    """`python bench.py --gpus N` outside torchrun: start the N ranks (one replica per GPU) the way
    torchrun would, on 127.0.0.1, and pass their output through (rank 0 prints the JSON line)."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def combine_check(rank, world):
    """Replica plumbing without a GPU: every rank contributes made-up measurements, rank 0 prints what
    the benchmark would report for them (slowest time, summed throughput, n_gpus = ranks)."""
    total_ms, dp_ms, e2e_ms, tok_s = combine_replicas(10.0 + rank, 4.0 + 0.5 * rank, 5.0 - rank, 100.0 * (rank + 1),
                                                      world, torch.device("cpu"))
    if rank == 0:
        print(json.dumps({"mode": "combine-check", "n_gpus": world, "ms_per_step": total_ms, "value": dp_ms,
                          "e2e": e2e_ms, "decode_tokens_per_s": tok_s}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="8b-c512-M12", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--mode", default="round", choices=["round", "dp-only", "combine-check"],
                    help="dp-only: profiling aid, runs just the layer search inside a profiler range; "
                         "combine-check: the replicas' cross-rank step on made-up numbers over gloo (no GPU)")
    args = ap.parse_args()
    if "WORLD_SIZE" not in os.environ and args.gpus > 1 and args.impl == "ours":
        sys.exit(launch_replicas(args.gpus, sys.argv[1:]))
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if args.mode == "combine-check":
        if world > 1:
            torch.distributed.init_process_group("gloo")
        try:
            combine_check(rank, world)
        finally:
            if world > 1:
                torch.distributed.destroy_process_group()
        return
    if world > 1:
        torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", 0)))
        torch.distributed.init_process_group("nccl")
    try:
        run_ours(args, rank, world)
    finally:
        if world > 1:
            torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
