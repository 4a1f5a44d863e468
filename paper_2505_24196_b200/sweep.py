#!/usr/bin/env python
"""Measurements beside the headline benchmark: the layer search over context lengths, numbers of
skipped layers and objective rows, on the 8B and 70B shapes, and the end-to-end greedy
self-speculative loop.  One JSON line per measurement.

    python -m paper_2505_24196_b200.sweep dp     --model 8b  --ctx 512 2048 8192 --M 8 12 16 --T 1
    python -m paper_2505_24196_b200.sweep dp     --model 70b --ctx 1024 --M 32 40
    python -m paper_2505_24196_b200.sweep decode --model 8b  --prompt 512 --new 256 --K 4 8 --M 12
    python -m paper_2505_24196_b200.sweep trace  --model 8b  --ctx 512 --M 12 --job 20

Weights are seeded random-init tensors and the prompts uniform random token ids (see `datagen`).
Times come from CUDA events on the library's stream; the per-layer split comes from the
persistent kernel's own step tracing (median over CTAs, mean over the layers of one search).
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import datagen  # noqa: E402
import paper_2505_24196_b200 as clasp  # noqa: E402
from paper_2505_24196_b200.decode import greedy_autoregressive  # noqa: E402

TRACE_SLOTS = 64
SLOT = {"start": 0, "qkv": 1, "att_ready": 2, "att_pub": 5, "merge": 6, "o": 7, "gu": 8, "down": 9, "dp_done": 13,
        "mma_first_qkv": 16, "mma_first_o": 17, "mma_first_gu": 18, "mma_first_down": 19,
        "mma_last_qkv": 20, "mma_last_o": 21, "mma_last_gu": 22, "mma_last_down": 23}


def build_engine(name, max_ctx, max_M, max_T, max_head_rows=8, flags=0):
    cfg = datagen.CONFIGS[name]
    dev = torch.device("cuda", 0)
    ccfg = clasp.make_config(cfg, max_ctx=max_ctx, max_rows=128, max_M=max_M, max_T=max_T,
                             max_head_rows=max_head_rows, flags=flags)
    eng = clasp.Clasp(ccfg, device=dev)
    layers = [datagen.layer_weights(cfg, l, dev) for l in range(cfg.L)]
    head = datagen.head_weights(cfg, dev)
    eng.load_layers(0, layers)
    eng.load_head(head)
    torch.cuda.synchronize()
    return cfg, ccfg, eng, (layers, head)


def prefill_to(eng, kv, toks, done, upto, want_rows):
    """Continue the chunked prefill from position `done` to `upto`; the last chunk holds exactly the
    last `want_rows` positions, whose hidden states are returned."""
    s = done
    while s < upto - want_rows:
        n = min(128, upto - want_rows - s)
        eng.verify(toks[s:s + n], s, kv, 0, want_hidden=False)
        s += n
    _, hid = eng.verify(toks[s:upto], s, kv, 1, want_hidden=True)
    return hid


def layer_split(eng, run, n_jobs):
    """Per-layer medians (us) of the persistent kernel's step stamps for one search."""
    import numpy as np
    G = eng.engine_ctas()
    cap = (n_jobs + 4) * TRACE_SLOTS
    st = torch.zeros((G, cap), dtype=torch.int64, device=eng.device)
    eng.set_trace(st, cap)
    run()
    torch.cuda.synchronize()
    eng.set_trace(None, 0)
    s = st.cpu().numpy().astype(np.float64)
    att, mlp, gemm = [], [], []
    for jb in range(3, n_jobs):
        blk = s[:, jb * TRACE_SLOTS:(jb + 1) * TRACE_SLOTS]

        def med(name):
            col = blk[:, SLOT[name]]
            col = col[col > 0]
            return float(np.median(col)) if len(col) else float("nan")
        att.append((med("mma_first_o") - med("qkv")) / 1e3)
        mlp.append((med("down") - med("mma_first_gu")) / 1e3)
        gemm.append(sum(med("mma_last_" + k) - med("mma_first_" + k) for k in ("qkv", "o", "gu", "down")) / 1e3)
    f = lambda v: round(float(np.nanmean(v)), 2) if len(v) else None
    return {"attention_us_per_layer": f(att), "mlp_us_per_layer": f(mlp), "weight_products_us_per_layer": f(gemm)}


def cmd_dp(args):
    cfg0 = datagen.CONFIGS[args.model]
    max_ctx = max(args.ctx) + 64
    cfg, ccfg, eng, keep = build_engine(args.model, max_ctx, max(args.M), max(args.T), flags=args.flags)
    kv = clasp.KVCache(ccfg, device=eng.device)
    toks = datagen.token_ids(cfg, max(args.ctx)).to(eng.device)
    d, L = cfg.d_model, cfg.L
    esz = 2
    done = 0
    for C in sorted(args.ctx):
        hid_all = prefill_to(eng, kv, toks, done, C, max(args.T))
        done = C
        for T in args.T:
            hid = hid_all[-T:].contiguous()
            for M in args.M:
                if M * T > 128:
                    continue
                p0 = C - T
                run = lambda: eng.dp_search(hid, d, (L + 1) * d, kv, p0, p0, T, M, want_margins=False, want_g=False)
                for _ in range(3):
                    run()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(eng.stream)
                for _ in range(args.reps):
                    r = run()
                b.record(eng.stream)
                torch.cuda.synchronize()
                ms = a.elapsed_time(b) / args.reps
                byts = (L - 1) * (cfg.layer_matrix_bytes() + 2 * p0 * cfg.n_kv_heads * cfg.head_dim * esz)
                out = {"what": "dp_search", "model": cfg.name, "flags": args.flags, "ctx": C, "M": M, "T": T,
                       "dp_ms": round(ms, 4),
                       "algorithmic_gb": round(byts / 1e9, 3), "gbs": round(byts / ms / 1e6, 1),
                       "skipped": int(r["S"].sum()), "device_status": eng.device_status()}
                out.update(layer_split(eng, run, L))
                print(json.dumps(out), flush=True)
    eng.close()


STAMP_NAMES = (["job_start", "qkv_epilogue_done", "attention_ready", "attention_q_loaded", "attention_tiles_done",
                "attention_published", "attention_merged", "o_epilogue_done", "gate_up_epilogue_done",
                "down_epilogue_done", "eq2_sums_published", "eq2_sums_complete", "eq2_decided", "eq2_step_done",
                "head_done", "-"]
               + [f"{a}_{b}" for a in ("mma_first", "mma_last", "accumulator_ready") for b in ("qkv", "o", "gate_up", "down")]
               + ["eq2_next_operand_point", "operand_ready_qkv", "operand_ready_o", "operand_ready_gate_up"]
               + [f"fine_{n:02d}" for n in range(32)])


def cmd_trace(args):
    """Time line of one job of a search: per stamp the min / median / max over the CTAs, in
    microseconds after the job's first stamp."""
    import numpy as np
    C, M, T = args.ctx[0], args.M[0], args.T[0]
    cfg, ccfg, eng, keep = build_engine(args.model, C + 64, M, T, flags=args.flags)
    kv = clasp.KVCache(ccfg, device=eng.device)
    toks = datagen.token_ids(cfg, C).to(eng.device)
    hid = prefill_to(eng, kv, toks, 0, C, T)[-T:].contiguous()
    d, L = cfg.d_model, cfg.L
    p0 = C - T
    run = lambda: eng.dp_search(hid, d, (L + 1) * d, kv, p0, p0, T, M, want_margins=False, want_g=False)
    for _ in range(3):
        run()
    G = eng.engine_ctas()
    cap = (L + 4) * TRACE_SLOTS
    st = torch.zeros((G, cap), dtype=torch.int64, device=eng.device)
    eng.set_trace(st, cap)
    run()
    torch.cuda.synchronize()
    eng.set_trace(None, 0)
    s = st.cpu().numpy().astype(np.float64)
    jb = args.job
    blk = s[:, jb * TRACE_SLOTS:(jb + 1) * TRACE_SLOTS]
    base = blk[blk > 0].min()
    rows = []
    for k, name in enumerate(STAMP_NAMES):
        col = blk[:, k]
        col = col[col > 0]
        if len(col):
            col = (col - base) / 1e3
            rows.append((float(np.median(col)), name, float(col.min()), float(col.max())))
    print(f"# job {jb} (DP step {jb + 1}, layer {jb}) of a search: model {cfg.name}, ctx {C}, M {M}, T {T}; us after the job's first stamp")
    for med, name, lo, hi in sorted(rows):
        print(f"{name:28s} min {lo:8.2f}  median {med:8.2f}  max {hi:8.2f}")
    starts = [s[:, j * TRACE_SLOTS][s[:, j * TRACE_SLOTS] > 0].min() for j in range(L) if (s[:, j * TRACE_SLOTS] > 0).any()]
    print("job durations (us):", " ".join(f"{(starts[i + 1] - starts[i]) / 1e3:.0f}" for i in range(len(starts) - 1)))
    eng.close()


def cmd_decode(args):
    max_ctx = args.prompt + args.new + 4 * (max(args.K) + 1) + 64
    cfg, ccfg, eng, keep = build_engine(args.model, max_ctx, max(args.M), 1, max_head_rows=max(args.K) + 1)
    prompt = datagen.token_ids(cfg, args.prompt, stream=7).tolist()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    kv = clasp.KVCache(ccfg, device=eng.device)
    torch.cuda.synchronize()
    a.record(eng.stream)
    ar = greedy_autoregressive(eng, kv, prompt, args.new)
    b.record(eng.stream)
    torch.cuda.synchronize()
    ar_ms = a.elapsed_time(b)
    print(json.dumps({"what": "autoregressive", "model": cfg.name, "prompt": args.prompt, "new": args.new,
                      "total_ms_incl_prefill": round(ar_ms, 2)}), flush=True)
    for M in args.M:
        for K in args.K:
            kv = clasp.KVCache(ccfg, device=eng.device)
            dec = clasp.SelfSpeculativeDecoder(eng, kv, M=M, K=K, dp_interval=args.dp_interval, time_stages=True)
            torch.cuda.synchronize()
            a.record(eng.stream)
            first = dec.prefill(prompt)
            b.record(eng.stream)
            torch.cuda.synchronize()
            prefill_ms = a.elapsed_time(b)
            for k in dec.stage_ms:
                dec.stage_ms[k] = 0.0
            out = [first]
            a.record(eng.stream)
            while len(out) < args.new:
                out.extend(dec.round())
            b.record(eng.stream)
            torch.cuda.synchronize()
            ms = a.elapsed_time(b)
            out = out[:args.new]
            acc = [r["accepted"] for r in dec.rounds]
            # Sparse Persistence (Sec. 3.7): Jaccard similarity of the skip sets of consecutive searches
            sets = [frozenset(i for i, b in enumerate(r["S"]) if b) for r in dec.rounds[::args.dp_interval]]
            jac = [len(x & y) / max(len(x | y), 1) for x, y in zip(sets, sets[1:])]
            print(json.dumps({"what": "self_speculative", "model": cfg.name, "prompt": args.prompt, "new": args.new,
                              "M": M, "K": K, "dp_interval": args.dp_interval, "identical_to_autoregressive": out == ar,
                              "decode_ms": round(ms, 2), "prefill_and_first_search_ms": round(prefill_ms, 2),
                              "tokens_per_s": round((args.new - 1) / ms * 1e3, 2), "rounds": len(dec.rounds),
                              "mean_accepted_drafts": round(sum(acc) / max(len(acc), 1), 3),
                              "mean_jaccard_of_consecutive_skip_sets": round(sum(jac) / max(len(jac), 1), 3),
                              "stage_ms_total": {k: round(v, 2) for k, v in dec.stage_ms.items()},
                              "device_status": eng.device_status()}), flush=True)
    eng.close()


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="cmd", required=True)
    p = sub.add_parser("dp")
    p.add_argument("--model", default="8b")
    p.add_argument("--ctx", type=int, nargs="+", default=[512])
    p.add_argument("--M", type=int, nargs="+", default=[12])
    p.add_argument("--T", type=int, nargs="+", default=[1])
    p.add_argument("--reps", type=int, default=10)
    p.add_argument("--flags", type=int, default=0, help="library flags (8: leave out unreachable states)")
    p = sub.add_parser("trace")
    p.add_argument("--model", default="8b")
    p.add_argument("--ctx", type=int, nargs="+", default=[512])
    p.add_argument("--M", type=int, nargs="+", default=[12])
    p.add_argument("--T", type=int, nargs="+", default=[1])
    p.add_argument("--job", type=int, default=20)
    p.add_argument("--flags", type=int, default=0, help="library flags (16: no tensor-core attention)")
    p = sub.add_parser("decode")
    p.add_argument("--model", default="8b")
    p.add_argument("--prompt", type=int, default=512)
    p.add_argument("--new", type=int, default=256)
    p.add_argument("--K", type=int, nargs="+", default=[4])
    p.add_argument("--M", type=int, nargs="+", default=[12])
    p.add_argument("--dp-interval", type=int, default=1)
    args = ap.parse_args()
    {"dp": cmd_dp, "decode": cmd_decode, "trace": cmd_trace}[args.cmd](args)


if __name__ == "__main__":
    main()
