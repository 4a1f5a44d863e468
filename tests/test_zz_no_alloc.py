"""The allocation-free GEMM entry point against the context-based one.

Some callers may not allocate device memory at all (a plug-in's enqueue hook, a server
whose memory pool owns the whole GPU), so clasp_gemm_xwT_noalloc keeps its split-K
scratch in an array built into the library.  This file is collected last on purpose:
a run that stops at the first failure has then already run every other test.
"""
import pytest
import torch

import datagen

pytestmark = pytest.mark.gpu


def test_noalloc_gemm_matches_context_gemm_twice_in_a_row():
    import paper_2505_24196_b200 as clasp
    cfg = datagen.CONFIGS["small"]
    eng = clasp.Clasp(clasp.make_config(cfg, max_ctx=64, max_rows=64, max_M=1))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # two different shapes back to back: the second call inherits the first one's scratch
    # contents (partial sums of another shape, used counters) and must not be disturbed
    for call, (R, N, K) in enumerate([(12, 1000, 2048), (5, 384, 4096), (12, 1000, 2048)]):
        x = datagen.normal_rows(71, call, (R, K)).to(torch.bfloat16).cuda()
        w = datagen.normal_rows(72, call, (N, K), 0.05).to(torch.bfloat16).cuda()
        ref = eng.gemm_xwT(x, w)
        y = torch.full((R, N), float("nan"), dtype=torch.float32, device="cuda")
        clasp.gemm_xwT_noalloc(x, w, y, status_out=status)
        torch.cuda.synchronize()
        assert int(status[0]) == 0
        err = float(torch.linalg.norm(y.double() - ref.double()) / torch.linalg.norm(ref.double()))
        assert err < 2e-6, (call, err)
        # same kernel, same split-K schedule: the two entry points agree exactly
        assert torch.equal(y, ref)
        exact = x.double() @ w.double().T
        assert float(torch.linalg.norm(y.double() - exact) / torch.linalg.norm(exact)) < 2e-6
    assert eng.device_status() == 0
    eng.close()


@pytest.mark.parametrize("R,N,K", [(200, 256, 512), (256, 130, 72), (33, 128, 64), (16, 384, 4096)])
def test_noalloc_gemm_wide_ragged_and_unsplit_shapes(R, N, K):
    """The entry point's whole range: up to 256 rows (256 accumulator columns, 48 KB stages), a row
    count that is not a multiple of 16, a ragged N and K, a single-split product that uses no scratch;
    with and without a status word (without one a wait that gave up would go unreported, the product
    itself is the same)."""
    import paper_2505_24196_b200 as clasp
    cfg = datagen.CONFIGS["small"]
    eng = clasp.Clasp(clasp.make_config(cfg, max_ctx=64, max_rows=64, max_M=1))
    x = datagen.normal_rows(73, R + N, (R, K)).to(torch.bfloat16).cuda()
    w = datagen.normal_rows(74, N + K, (N, K), 0.05).to(torch.bfloat16).cuda()
    ref = eng.gemm_xwT(x, w)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    y1 = torch.full((R, N), float("nan"), dtype=torch.float32, device="cuda")
    y2 = torch.full((R, N), float("nan"), dtype=torch.float32, device="cuda")
    clasp.gemm_xwT_noalloc(x, w, y1, status_out=status)
    clasp.gemm_xwT_noalloc(x, w, y2)                       # status_out == NULL
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    assert torch.equal(y1, ref) and torch.equal(y2, ref)
    exact = x.double() @ w.double().T
    assert float(torch.linalg.norm(y1.double() - exact) / torch.linalg.norm(exact)) < 2e-6
    assert eng.device_status() == 0
    eng.close()


def test_noalloc_gemm_refuses_what_does_not_fit():
    import paper_2505_24196_b200 as clasp
    x = torch.zeros((257, 64), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((128, 64), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((257, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(clasp.ClaspError) as e:
        clasp.gemm_xwT_noalloc(x, w, y)                       # more rows than the entry point takes
    assert e.value.code == -3
    # split-K partial sums of 6 splits x 256 rows x 6144 columns exceed the built-in array
    x = torch.zeros((256, 4096), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((6144, 4096), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((256, 6144), dtype=torch.float32, device="cuda")
    with pytest.raises(clasp.ClaspError) as e:
        clasp.gemm_xwT_noalloc(x, w, y)
    assert e.value.code == -3
