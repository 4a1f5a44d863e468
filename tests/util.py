"""Shared test plumbing: builds the same seeded model for the oracle (float64 numpy)
and for the CUDA library (device tensors).  No arithmetic of the method lives here."""
from __future__ import annotations

import contextlib

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

    def engine_with_flags(self, flags: int, **kw):
        """A second context over the same device weights with other library flags."""
        import paper_2505_24196_b200 as clasp
        ccfg = clasp.make_config(self.cfg, kw.get("max_ctx", self.max_ctx), kw.get("max_rows", self.ccfg.max_rows),
                                 kw.get("max_M", self.ccfg.max_M), kw.get("max_T", self.ccfg.max_T),
                                 kw.get("max_head_rows", self.ccfg.max_head_rows), flags)
        eng = clasp.Clasp(ccfg)
        eng.load_layers(0, self.layers_dev)
        eng.load_head(self.head_dev)
        return eng

    def new_kv(self):
        import paper_2505_24196_b200 as clasp
        return clasp.KVCache(self.ccfg)

    def new_oracle_cache(self):
        return orc.KVCache(self.cfg, self.max_ctx)


def rel_l2(a: np.ndarray, b: np.ndarray) -> float:
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def max_abs_ok(a: np.ndarray, b: np.ndarray, tol: float) -> bool:
    """Guard beside a relative-L2 bound: no single element may be off by more than 8 * tol times
    the root mean square of the reference (a relative-L2 bound alone lets one bad feature of a wide
    row pass; errors that are spread like rounding noise stay far below this)."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    rms = float(np.sqrt(np.mean(b * b)))
    return float(np.max(np.abs(a - b))) <= 8.0 * tol * max(rms, 1e-300)


def close_hidden(a: np.ndarray, b: np.ndarray, tol: float) -> bool:
    return rel_l2(a, b) < tol and max_abs_ok(a, b, tol)


def tol_hidden(cfg) -> float:
    """Relative-L2 bound on hidden states: 1e-4 for fp32 models, 2e-2 for bf16 models."""
    return 1e-4 if cfg.dtype == "fp32" else 2e-2


def kv_to_oracle(kv, n: int, ocache: "orc.KVCache"):
    """Copy the first n positions of a device cache into an oracle cache (used only to
    hand the SAME seeded cache contents to both sides in single-layer tests)."""
    ocache.k[:, :n] = kv.k[:, :n].double().cpu().numpy()
    ocache.v[:, :n] = kv.v[:, :n].double().cpu().numpy()


def device_choices(margin: np.ndarray, L: int, M: int) -> np.ndarray:
    """The decisions a search took, read off its margins (strict '>' takes APPLY; the diagonal is a
    forced SKIP) -- the choice table itself stays in the library's workspace."""
    ch = np.full((L + 1, M + 1), 255, dtype=np.uint8)
    for i in range(1, L + 1):
        ch[i, 0] = orc.APPLY
        for j in range(1, min(i, M) + 1):
            ch[i, j] = orc.SKIP if (j == i or not margin[i, j] > 0.0) else orc.APPLY
    return ch


def path_cells(choice: np.ndarray, L: int, M: int):
    """Cells the backtrack of Algorithm 1 visits from (L, M)."""
    cells, i, j = [], L, M
    while i > 0 and j > 0:
        cells.append((i, j))
        if choice[i, j] == orc.SKIP:
            j -= 1
        i -= 1
    return cells


def check_search_against_oracle(D, margin, S, g_final, ref, L: int, M: int, tol: float) -> int:
    """Eq. 2 decisions of an unforced device search against the oracle's, cell by cell: wherever the
    oracle's margin is decisive (> 1e-3) and the walk so far agreed (both parents of the cell are the
    same states on both sides), the device takes the same branch and reports the same score and
    margin.  A near-tie only excuses the cells that descend from it.  The skip set and g[L][M] are
    compared when every cell on the oracle's backtracked path agreed.  Returns the number of decisive
    cells that were compared."""
    choice_g = device_choices(margin, L, M)
    agree = np.zeros((L + 1, M + 1), dtype=bool)
    agree[:, 0] = True
    n_checked = 0
    for i in range(1, L + 1):
        for j in range(1, min(i, M) + 1):
            if not (agree[i - 1, j - 1] and (j == i or agree[i - 1, j])):
                continue
            if j == i:                                   # diagonal: forced skip, score only
                assert abs(D[i, j] - ref["D"][i, j]) < 1e-3, (i, j)
                agree[i, j] = True
                continue
            assert abs(margin[i, j] - ref["margin"][i, j]) < 2e-3, (i, j)
            if abs(ref["margin"][i, j]) > 1e-3:
                assert choice_g[i, j] == ref["choice"][i, j], (i, j)
                assert abs(D[i, j] - ref["D"][i, j]) < 1e-3, (i, j)
                agree[i, j] = True
                n_checked += 1
            else:
                agree[i, j] = choice_g[i, j] == ref["choice"][i, j]
    if all(agree[i, j] for i, j in path_cells(ref["choice"], L, M)):
        np.testing.assert_array_equal(S, ref["S"])
        if g_final is not None:
            assert close_hidden(g_final, ref["g"][L, M], tol)
    return n_checked


def search_that_applies_layer_1(m, C0, T, seed):
    """Hidden states x[0..2] such that the best state with one skipped layer is f_1(x_0): the search
    must compute it (rows attend to the cache and to the rows before them) and return it as g[L][M]."""
    cfg, eng = m.cfg, m.engine
    L, d, M = cfg.L, cfg.d_model, 1
    p0 = C0 - T
    x0 = datagen.normal_rows(seed, 0, (T, d)).to(torch.float32)
    w = m.oracle.layer(1)
    f1, _, _ = orc.decoder_layer(x0.double().numpy(), w, m.ocache.k[1], m.ocache.v[1], p0, p0, cfg)
    x1 = x0 + datagen.normal_rows(seed, 1, (T, d)).to(torch.float32)          # far from everything
    x2 = torch.from_numpy(f1).to(torch.float32)
    x = torch.stack([x0, x1, x2])
    ref = orc.dp_search(m.oracle, x.double().numpy(), m.ocache, p0, p0, M)
    assert list(ref["S"]) == [1, 0]                # layer 0 skipped, layer 1 applied by the search
    res = eng.dp_search(x.cuda(), T * d, d, m.kv, p0, p0, T, M)
    torch.cuda.synchronize()
    assert eng.device_status() == 0
    np.testing.assert_array_equal(res["S"].cpu().numpy(), ref["S"])
    got = res["g_final"].cpu().numpy().reshape(T, d)
    for r in range(T):                             # row by row: a wrong row must not hide among good ones
        assert rel_l2(got[r:r + 1], f1[r:r + 1]) < 2e-2, r
    D = res["D"].cpu().numpy()
    np.testing.assert_allclose(D[~np.isnan(D)], ref["D"][~np.isnan(D)], atol=1e-3)


@contextlib.contextmanager
def scaled_keys(m, first, factor):
    """Layer 1's cached keys from position `first` on times a power of two (exact in bf16 and float64), on
    both sides.  With unit-variance keys a row's weights spread evenly over thousands of positions and the attention
    output nearly vanishes in the layer output; larger keys concentrate them on a few positions, so that a
    mistake in any tile of keys or values moves some row by far more than the tolerance."""
    m.kv.k[1, first:] *= factor
    m.ocache.k[1][first:] *= float(factor)
    try:
        yield
    finally:
        m.kv.k[1, first:] /= factor
        m.ocache.k[1][first:] /= float(factor)
