"""Parity at a long context: the LLaMA3-8B layer shape (d = 4096, 32 / 8 heads of 128, FFN 14336, bf16)
over an 8192-position cache (every run of cache keys spans several tiles), on a two-layer model so that
the oracle can hold a layer in float64: sampled rows of one decoder layer, one search with T = 4
objective rows per state (M = 2) compared cell by cell, and searches built so that the chosen state is
a layer output the search itself computed (M = 1): its rows are compared with the oracle's, for row
counts that take the 64-row and the 128-row shape of the tensor-core attention, two blocks of
(row, head) pairs, and keys that grow along the context so that the running maximum moves late.

Inputs are seeded and synthetic, the same bytes on both sides (weights created on the device and copied
to the host for the oracle; cache contents and states from seeded normal streams).  Tolerances: hidden
states relative L2 <= 2e-2 (bf16 model), scores 1e-3."""
import dataclasses

import numpy as np
import pytest
import torch

import datagen
from oracle import clasp_oracle as orc
from oracle import from_torch
from tests.util import rel_l2, scaled_keys, search_that_applies_layer_1

pytestmark = pytest.mark.gpu

C0 = 8192


class LongContext8B:
    def __init__(self):
        import paper_2505_24196_b200 as clasp
        self.cfg = cfg = dataclasses.replace(datagen.CONFIGS["8b"], name="8b-l2", L=2, vocab=8192)
        dev = torch.device("cuda", 0)
        self.ccfg = clasp.make_config(cfg, max_ctx=C0 + 64, max_rows=128, max_M=2, max_T=40, max_head_rows=8)
        self.engine = clasp.Clasp(self.ccfg, device=dev)
        self.layers = [datagen.layer_weights(cfg, l, dev) for l in range(cfg.L)]
        self.head = datagen.head_weights(cfg, dev)
        self.engine.load_layers(0, self.layers)
        self.engine.load_head(self.head)
        self.kv = clasp.KVCache(self.ccfg, device=dev)
        shp = tuple(self.kv.k.shape)
        ck = datagen.normal_rows(71, 0, shp).to(cfg.torch_dtype)
        cv = datagen.normal_rows(71, 1, shp).to(cfg.torch_dtype)
        self.kv.k.copy_(ck)
        self.kv.v.copy_(cv)
        self.ocache = orc.KVCache(cfg, C0 + 64)
        self.ocache.k[:] = ck.double().numpy()
        self.ocache.v[:] = cv.double().numpy()
        # the oracle converts a layer to float64 when it asks for it (only layer 1 is ever applied)
        self.oracle = from_torch.model_from_tensors(cfg, self.layers, None, resident=False)


@pytest.fixture(scope="module")
def mlong():
    m = LongContext8B()
    yield m
    assert m.engine.device_status() == 0
    m.engine.close()


def test_layer_rows_over_a_long_context(mlong):
    cfg = mlong.cfg
    assert mlong.engine.engine_active()
    x = datagen.normal_rows(72, 0, (12, cfg.d_model)).to(torch.float32)
    out = mlong.engine.layer_forward(1, x.cuda(), 12, 1, C0, C0, mlong.kv).cpu().numpy()
    w = mlong.oracle.layer(1)
    for r in (0, 7, 11):
        ref, _, _ = orc.decoder_layer(x[r:r + 1].double().numpy(), w, mlong.ocache.k[1], mlong.ocache.v[1], C0, C0, cfg)
        assert rel_l2(out[r:r + 1], ref) < 2e-2, r
    assert mlong.engine.device_status() == 0


def test_search_over_a_long_context(mlong):
    """L = 2, M = 2, T = 4: step 2 pushes one state of 4 rows through layer 1 (each row sees the cache
    and the rows before it in its state); the whole table is compared with the oracle's."""
    cfg, eng = mlong.cfg, mlong.engine
    L, d, T, M = cfg.L, cfg.d_model, 4, 2
    steps = datagen.normal_rows(73, 0, (L + 1, T, d))
    steps[1:] *= 0.2
    x = torch.cumsum(steps, dim=0).to(torch.float32)          # [L+1, T, d]
    p0 = C0 - T
    ref = orc.dp_search(mlong.oracle, x.double().numpy(), mlong.ocache, p0, p0, M)
    res = eng.dp_search(x.cuda(), T * d, d, mlong.kv, p0, p0, T, M)
    torch.cuda.synchronize()
    assert eng.device_status() == 0
    D = res["D"].cpu().numpy()
    assert np.array_equal(np.isnan(D), np.isnan(ref["D"]))
    np.testing.assert_allclose(D[~np.isnan(D)], ref["D"][~np.isnan(D)], atol=1e-3)
    m = ~np.isnan(ref["margin"])
    np.testing.assert_allclose(res["margin"].cpu().numpy()[m], ref["margin"][m], atol=2e-3)
    if np.nanmin(np.abs(ref["margin"])) > 1e-3:
        np.testing.assert_array_equal(res["S"].cpu().numpy(), ref["S"])
        assert rel_l2(res["g_final"].cpu().numpy(), ref["g"][L, M]) < 2e-2
    assert int(res["S"].sum()) == M


@pytest.mark.parametrize("T", [12, 40])
def test_search_returns_the_layer_output_it_computed(mlong, T):
    """T = 12: 48 (row, head) pairs per kv head, one 64-row item; T = 40: 160 pairs, a full 128-row
    block and a second one with 32 rows."""
    with scaled_keys(mlong, 0, 4):
        search_that_applies_layer_1(mlong, C0, T, 74 + T)


@pytest.mark.parametrize("lo_scale", [1, 2])
def test_search_with_keys_that_grow_along_the_context(mlong, lo_scale):
    """Keys from the middle of the cache on 4 times those before: the scores of the later tiles
    exceed the maximum the first tile fixed by more than 2^8, so the rows' running maxima move
    and the accumulated output is rescaled.  (Much larger keys would test bf16's rounding of q instead:
    a score of several hundred carries an absolute error near 1.)"""
    # (the step sits inside a run of keys, past its first 64-key tile: a run is one item's share of the context)
    with scaled_keys(mlong, 0, lo_scale), scaled_keys(mlong, C0 // 2 + 100, 4):
        search_that_applies_layer_1(mlong, C0, 12, 91)
