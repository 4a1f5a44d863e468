"""Shared test plumbing: builds the same seeded model for the oracle (float64 numpy)
and for the CUDA library (device tensors).  No arithmetic of the method lives here."""
from __future__ import annotations

import numpy as np
import torch

import datagen
from oracle import clasp_oracle as orc
from oracle import from_torch


class Pair:
    """One seeded model, seen by both sides."""

    def __init__(self, cfg, max_ctx, max_rows, max_M, max_T=1, max_head_rows=16, flags=0, gen_device="cpu"):
        import paper_2505_24196_b200 as clasp
        self.cfg = cfg
        self.layers_src = [datagen.layer_weights(cfg, l, gen_device) for l in range(cfg.L)]
        self.head_src = datagen.head_weights(cfg, gen_device)
        self.oracle = from_torch.model_from_tensors(cfg, self.layers_src, self.head_src, resident=True)
        self.ccfg = clasp.make_config(cfg, max_ctx, max_rows, max_M, max_T, max_head_rows, flags)
        self.engine = clasp.Clasp(self.ccfg)
        self.layers_dev = [{k: v.cuda().contiguous() for k, v in lw.items()} for lw in self.layers_src]
        self.head_dev = {k: v.cuda().contiguous() for k, v in self.head_src.items()}
        self.engine.load_layers(0, self.layers_dev)
        self.engine.load_head(self.head_dev)
        self.max_ctx = max_ctx

    def new_kv(self):
        import paper_2505_24196_b200 as clasp
        return clasp.KVCache(self.ccfg)

    def new_oracle_cache(self):
        return orc.KVCache(self.cfg, self.max_ctx)


def rel_l2(a: np.ndarray, b: np.ndarray) -> float:
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def tol_hidden(cfg) -> float:
    """Relative-L2 bound on hidden states: 1e-4 for fp32 models, 2e-2 for bf16 models."""
    return 1e-4 if cfg.dtype == "fp32" else 2e-2


def kv_to_oracle(kv, n: int, ocache: "orc.KVCache"):
    """Copy the first n positions of a device cache into an oracle cache (used only to
    hand the SAME seeded cache contents to both sides in single-layer tests)."""
    ocache.k[:, :n] = kv.k[:, :n].double().cpu().numpy()
    ocache.v[:, :n] = kv.v[:, :n].double().cpu().numpy()
