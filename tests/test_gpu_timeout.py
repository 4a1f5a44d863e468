"""The wind-down path of the kernels' bounded waits, reached without a kernel that would wait
forever: the context's wait limit is set to one poll, so the first wait of a healthy launch that is
not satisfied at once (a copy still in flight) gives up.  The kernel must then end by itself (copies
in flight awaited, tensor memory freed), the status call must report CLASP_ERR_TIMEOUT once, and the
context must work again after the limit is restored."""
import pytest
import torch

import datagen
from oracle import clasp_oracle as orc
from tests.util import Pair, close_hidden, kv_to_oracle, tol_hidden

pytestmark = pytest.mark.gpu

TIMEOUT = -6


@pytest.fixture(scope="module")
def pair():
    cfg = datagen.CONFIGS["small"]
    p = Pair(cfg, max_ctx=96, max_rows=32, max_M=2, max_T=1, max_head_rows=4)
    yield p
    p.engine.close()


def _layer_inputs(pair):
    cfg = pair.cfg
    kv = pair.new_kv()
    kv.k.copy_(datagen.normal_rows(81, 0, tuple(kv.k.shape)).to(cfg.torch_dtype))
    kv.v.copy_(datagen.normal_rows(81, 1, tuple(kv.v.shape)).to(cfg.torch_dtype))
    x = datagen.normal_rows(82, 0, (4, cfg.d_model)).to(torch.float32)
    return kv, x


def test_gemm_wait_that_runs_out_is_reported_and_the_context_recovers(pair):
    eng = pair.engine
    x = datagen.normal_rows(83, 0, (5, 1376)).to(torch.bfloat16).cuda()
    w = datagen.normal_rows(83, 1, (1000, 1376), 0.05).to(torch.bfloat16).cuda()
    good = eng.gemm_xwT(x, w)
    assert eng.device_status() == 0
    eng.set_wait_limit(1)
    eng.gemm_xwT(x, w)
    assert eng.device_status() == TIMEOUT
    assert eng.device_status() == 0            # reported once, then cleared
    eng.set_wait_limit(0)
    again = eng.gemm_xwT(x, w)
    assert eng.device_status() == 0
    assert torch.equal(again, good)


def test_layer_kernel_wait_that_runs_out_is_reported_and_the_context_recovers(pair):
    cfg, eng = pair.cfg, pair.engine
    assert eng.engine_active()
    kv, x = _layer_inputs(pair)
    good = eng.layer_forward(2, x.cuda(), 4, 1, 40, 40, kv)
    assert eng.device_status() == 0
    eng.set_wait_limit(1)
    eng.layer_forward(2, x.cuda(), 4, 1, 40, 40, kv)
    assert eng.device_status() == TIMEOUT
    assert eng.device_status() == 0
    eng.set_wait_limit(0)
    again = eng.layer_forward(2, x.cuda(), 4, 1, 40, 40, kv)
    assert eng.device_status() == 0
    assert torch.equal(again, good)
    # and the recovered context still computes the layer: one state against the oracle
    ocache = pair.new_oracle_cache()
    kv_to_oracle(kv, pair.max_ctx, ocache)
    ref, _, _ = orc.decoder_layer(x[:1].double().numpy(), pair.oracle.layer(2), ocache.k[2], ocache.v[2], 40, 40, cfg)
    assert close_hidden(again[:1].cpu().numpy(), ref, tol_hidden(cfg))
