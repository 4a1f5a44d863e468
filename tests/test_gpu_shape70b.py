"""Parity on the LLaMA3-70B layer shape (d = 8192, 64 / 8 heads of 128, FFN 28672, bf16) with the row
counts of the 70B searches (40 candidate rows, a 1024-position cache), on a two-layer model so that the
oracle can hold a layer in float64: sampled rows of one decoder layer, and one search whose single
layer pass carries 40 rows (M = 2 states of T = 20 objective rows) compared cell by cell; and a search
over a 4096-position context (160 (row, head) pairs per kv head, eight query heads per kv head: two
128-row blocks of the tensor-core attention) whose result is a layer output it computed itself.

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

C0 = 1024
C_LONG = 4096     # a context long enough for the search's tensor-core attention


class Shape70B:
    def __init__(self):
        import paper_2505_24196_b200 as clasp
        self.cfg = cfg = dataclasses.replace(datagen.CONFIGS["70b"], name="70b-l2", L=2, vocab=8192)
        dev = torch.device("cuda", 0)
        self.ccfg = clasp.make_config(cfg, max_ctx=C_LONG + 64, max_rows=128, max_M=2, max_T=20, max_head_rows=8)
        self.engine = clasp.Clasp(self.ccfg, device=dev)
        self.layers = [datagen.layer_weights(cfg, l, dev) for l in range(cfg.L)]
        self.head = datagen.head_weights(cfg, dev)
        self.engine.load_layers(0, self.layers)
        self.engine.load_head(self.head)
        self.kv = clasp.KVCache(self.ccfg, device=dev)
        shp = tuple(self.kv.k.shape)
        ck = datagen.normal_rows(61, 0, shp).to(cfg.torch_dtype)
        cv = datagen.normal_rows(61, 1, shp).to(cfg.torch_dtype)
        self.kv.k.copy_(ck)
        self.kv.v.copy_(cv)
        self.ocache = orc.KVCache(cfg, C_LONG + 64)
        self.ocache.k[:] = ck.double().numpy()
        self.ocache.v[:] = cv.double().numpy()
        # the oracle converts a layer to float64 when it asks for it (only layer 1 is ever applied)
        self.oracle = from_torch.model_from_tensors(cfg, self.layers, None, resident=False)


@pytest.fixture(scope="module")
def m70():
    m = Shape70B()
    yield m
    assert m.engine.device_status() == 0
    m.engine.close()


def test_layer_rows_on_the_70b_shape(m70):
    cfg = m70.cfg
    assert m70.engine.engine_active()      # this shape runs in the one-launch-per-call kernel, not its fall-back
    x = datagen.normal_rows(62, 0, (40, cfg.d_model)).to(torch.float32)
    out = m70.engine.layer_forward(1, x.cuda(), 40, 1, C0, C0, m70.kv).cpu().numpy()
    w = m70.oracle.layer(1)
    for r in (0, 17, 39):
        ref, _, _ = orc.decoder_layer(x[r:r + 1].double().numpy(), w, m70.ocache.k[1], m70.ocache.v[1], C0, C0, cfg)
        assert rel_l2(out[r:r + 1], ref) < 2e-2, r
    assert m70.engine.device_status() == 0


def test_search_with_forty_rows_on_the_70b_shape(m70):
    """L = 2, M = 2, T = 20: step 2 pushes one state of 20 rows through layer 1 and the diagonal adds
    another 20 candidate rows; the whole table is compared with the oracle's."""
    cfg, eng = m70.cfg, m70.engine
    L, d, T, M = cfg.L, cfg.d_model, 20, 2
    steps = datagen.normal_rows(63, 0, (L + 1, T, d))
    steps[1:] *= 0.2
    x = torch.cumsum(steps, dim=0).to(torch.float32)          # [L+1, T, d]
    p0 = C0 - T
    ref = orc.dp_search(m70.oracle, x.double().numpy(), m70.ocache, p0, p0, M)
    res = eng.dp_search(x.cuda(), T * d, d, m70.kv, p0, p0, T, M)
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


def test_search_over_a_long_context_on_the_70b_shape(m70):
    """M = 1, T = 20, 4076 visible positions: g[L][M] is f_1(x_0), computed by the search over the cache
    (keys scaled by 4 so that the attention carries weight in the layer output) and its own rows."""
    with scaled_keys(m70, 0, 4):
        search_that_applies_layer_1(m70, C_LONG, 20, 64)

