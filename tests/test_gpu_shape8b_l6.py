"""The whole Eq. 2 table at the 8B layer shape over many steps: a 6-layer model of the LLaMA3-8B
layer shape (d = 4096, 32 / 8 heads of 128, FFN 14336, bf16), a 512-position cache, M = 3, T = 1 --
small enough for the oracle to run the complete search, large enough that the steps with 2 and 3
candidate rows, the q/k/v product over both Eq. 2 candidates and the chain of deferred decisions run
at the shape bench.py times.  The oracle's own prefill supplies the objective states; its cache,
rounded to the cache dtype, is handed to the device byte for byte.

Tolerances: scores 1e-3, margins 2e-3, decisions identical wherever the oracle's margin exceeds 1e-3
(cell by cell), hidden states relative L2 <= 2e-2 plus the max-abs guard."""
import numpy as np
import pytest
import torch

import datagen
from oracle import clasp_oracle as orc
from oracle import from_torch
from tests.util import check_search_against_oracle, close_hidden

pytestmark = pytest.mark.gpu

C0, M = 512, 3
FLAG_NO_DEFER = 2


class Shape8bL6:
    def __init__(self):
        import paper_2505_24196_b200 as clasp
        self.clasp = clasp
        self.cfg = cfg = datagen.CONFIGS["8b-l6"]
        dev = torch.device("cuda", 0)
        self.layers = [datagen.layer_weights(cfg, l, dev) for l in range(cfg.L)]
        self.head = datagen.head_weights(cfg, dev)
        layers_host = [{k: v.cpu() for k, v in lw.items()} for lw in self.layers]
        head_host = {k: v.cpu() for k, v in self.head.items()}
        # float64 copies are made one layer at a time
        self.oracle = from_torch.model_from_tensors(cfg, layers_host, head_host, resident=False)
        toks = datagen.token_ids(cfg, C0).numpy()
        self.ocache = orc.KVCache(cfg, C0 + 64)
        _, hid_o, _ = orc.verify_forward(self.oracle, toks, self.ocache, 0)
        self.x_o = hid_o[C0 - 1]                                         # [L+1, d] states of the last token
        # the cache both sides read: the oracle's keys / values rounded to the cache dtype
        k16 = torch.from_numpy(self.ocache.k).to(cfg.torch_dtype)
        v16 = torch.from_numpy(self.ocache.v).to(cfg.torch_dtype)
        self.ocache.k[:] = k16.double().numpy()
        self.ocache.v[:] = v16.double().numpy()
        self.k16, self.v16 = k16, v16
        self.ref = orc.dp_search(self.oracle, self.x_o[:, None, :], self.ocache, C0 - 1, C0 - 1, M)

    def engine(self, flags=0):
        clasp = self.clasp
        ccfg = clasp.make_config(self.cfg, max_ctx=C0 + 64, max_rows=64, max_M=M, max_T=1, max_head_rows=4,
                                 flags=flags)
        eng = clasp.Clasp(ccfg)
        eng.load_layers(0, self.layers)
        eng.load_head(self.head)
        kv = clasp.KVCache(ccfg)
        kv.k.copy_(self.k16)
        kv.v.copy_(self.v16)
        return eng, kv


@pytest.fixture(scope="module")
def shape():
    return Shape8bL6()


@pytest.mark.parametrize("flags", [0, FLAG_NO_DEFER], ids=["deferred", "no-defer"])
def test_whole_table_against_oracle(shape, flags):
    cfg, ref = shape.cfg, shape.ref
    L, d = cfg.L, cfg.d_model
    eng, kv = shape.engine(flags)
    try:
        assert eng.engine_active()
        x = torch.from_numpy(shape.x_o).to(torch.float32).cuda()
        p0 = C0 - 1
        res = eng.dp_search(x, d, 0, kv, p0, p0, 1, M)
        torch.cuda.synchronize()
        assert eng.device_status() == 0
        D, margin = res["D"].cpu().numpy(), res["margin"].cpu().numpy()
        S = res["S"].cpu().numpy()
        assert np.array_equal(np.isnan(D), np.isnan(ref["D"]))
        assert int(S.sum()) == M
        n = check_search_against_oracle(D, margin, S, res["g_final"].cpu().numpy(), ref, L, M, 2e-2)
        assert n >= 1                                    # the comparison was not vacuous
        # with the oracle's decisions forced, every cell and the final state are compared
        forced = torch.from_numpy(ref["choice"].copy()).cuda()
        rf = eng.dp_search(x, d, 0, kv, p0, p0, 1, M, forced_choice=forced)
        torch.cuda.synchronize()
        Df, mf = rf["D"].cpu().numpy(), rf["margin"].cpu().numpy()
        ok = ~np.isnan(ref["D"])
        np.testing.assert_allclose(Df[ok], ref["D"][ok], atol=1e-3)
        mk = ~np.isnan(ref["margin"])
        np.testing.assert_allclose(mf[mk], ref["margin"][mk], atol=2e-3)
        np.testing.assert_array_equal(rf["S"].cpu().numpy(), ref["S"])
        assert close_hidden(rf["g_final"].cpu().numpy(), ref["g"][L, M], 2e-2)
        assert eng.device_status() == 0
    finally:
        eng.close()
