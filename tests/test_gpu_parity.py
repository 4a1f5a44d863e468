"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same
seeded inputs.  Tolerances: hidden states relative L2 <= 1e-4 (fp32 model) or
<= 2e-2 (bf16 model); cosine scores within 1e-3; skip masks identical wherever the
oracle's decision margins exceed 1e-3; tokens identical."""
import dataclasses

import numpy as np
import pytest
import torch

import datagen
from oracle import clasp_oracle as orc
from tests.util import Pair, check_search_against_oracle, close_hidden, kv_to_oracle, rel_l2, tol_hidden

pytestmark = pytest.mark.gpu

FLAG_FORCE_SIMT, FLAG_NO_DEFER, FLAG_MULTI_KERNEL, FLAG_PRUNE = 1, 2, 4, 8
# (config name, library flags): the fp32 model runs the CUDA-core GEMM; the bf16 models run
# the tcgen05 GEMM, and once more with the CUDA-core GEMM as a cross-check of the rest.
ENGINES = [("tiny", 0), ("small", 0), ("mini8b", 0), ("small", FLAG_FORCE_SIMT)]


@pytest.fixture(scope="module", params=ENGINES, ids=lambda p: f"{p[0]}-flags{p[1]}")
def pair(request):
    name, flags = request.param
    cfg = datagen.CONFIGS[name]
    p = Pair(cfg, max_ctx=192, max_rows=96, max_M=cfg.L, max_T=4, max_head_rows=16, flags=flags)
    yield p
    assert p.engine.device_status() == 0
    p.engine.close()


def _prefill_both(p, n_tok):
    toks = datagen.token_ids(p.cfg, n_tok)
    ocache = p.new_oracle_cache()
    am_o, hid_o, logits_o = orc.verify_forward(p.oracle, toks.numpy(), ocache, 0)
    kv = p.new_kv()
    am_g, hid_g = p.engine.verify(toks.cuda(), 0, kv, min(n_tok, 16))
    torch.cuda.synchronize()
    return toks, ocache, am_o, hid_o, logits_o, kv, am_g, hid_g


@pytest.mark.parametrize("R,N,K", [(1, 256, 512), (5, 1000, 1376), (17, 384, 64), (40, 128, 4096), (3, 130, 72),
                                   (200, 256, 512), (256, 130, 72), (33, 128, 64)])
def test_gemm_against_definition(pair, R, N, K):
    """y = x w^T against the float64 product of the same rounded operands; ragged N and K."""
    cfg = pair.cfg
    dt = cfg.torch_dtype
    x = datagen.normal_rows(31, R * 7 + N, (R, K)).to(dt)
    w = datagen.normal_rows(32, N + K, (N, K), 0.05).to(dt)
    y = pair.engine.gemm_xwT(x.cuda(), w.cuda()).cpu().double().numpy()
    ref = x.double().numpy() @ w.double().numpy().T
    assert rel_l2(y, ref) < 2e-6
    assert pair.engine.device_status() == 0


def test_gemm_rows_are_batch_invariant(pair):
    """A row's result must not depend on how many other rows share the launch."""
    dt = pair.cfg.torch_dtype
    K, N = 1376, 520
    x = datagen.normal_rows(33, 0, (37, K)).to(dt).cuda()
    w = datagen.normal_rows(33, 1, (N, K), 0.05).to(dt).cuda()
    y_all = pair.engine.gemm_xwT(x, w)
    for r in (0, 16, 36):
        y_one = pair.engine.gemm_xwT(x[r:r + 1].contiguous(), w)
        assert torch.equal(y_one[0], y_all[r])


@pytest.mark.parametrize("S,T,C", [(1, 1, 0), (3, 1, 40), (2, 4, 33), (5, 2, 150)])
def test_layer_forward(pair, S, T, C):
    """One decoder layer over S independent states of T rows, cache of C positions."""
    cfg = pair.cfg
    kv = pair.new_kv()
    # seeded cache contents and inputs, identical on both sides
    ck = datagen.normal_rows(41, 0, (cfg.L, pair.max_ctx, cfg.n_kv_heads, cfg.head_dim)).to(cfg.torch_dtype)
    cv = datagen.normal_rows(41, 1, (cfg.L, pair.max_ctx, cfg.n_kv_heads, cfg.head_dim)).to(cfg.torch_dtype)
    kv.k.copy_(ck)
    kv.v.copy_(cv)
    ocache = pair.new_oracle_cache()
    kv_to_oracle(kv, pair.max_ctx, ocache)
    x = datagen.normal_rows(42, S * 100 + T, (S * T, cfg.d_model)).to(torch.float32)
    layer = min(2, cfg.L - 1)
    out = pair.engine.layer_forward(layer, x.cuda(), S, T, C, C, kv).cpu().numpy()
    xs = x.double().numpy().reshape(S, T, cfg.d_model)
    for s in range(S):
        ref, _, _ = orc.decoder_layer(xs[s], pair.oracle.layer(layer), ocache.k[layer], ocache.v[layer], C, C, cfg)
        assert close_hidden(out[s * T:(s + 1) * T], ref, tol_hidden(cfg))
    # the search never writes the cache
    assert torch.equal(kv.k.cpu(), ck) and torch.equal(kv.v.cpu(), cv)


def test_verify_forward_hidden_states_and_cache(pair):
    cfg = pair.cfg
    n = 70
    toks, ocache, am_o, hid_o, logits_o, kv, am_g, hid_g = _prefill_both(pair, n)
    hid_g = hid_g.cpu().numpy()
    tol = tol_hidden(cfg)
    for l in range(cfg.L + 1):
        assert close_hidden(hid_g[:, l], hid_o[:, l], tol), l
    assert rel_l2(kv.k[:, :n].float().cpu().numpy(), ocache.k[:, :n]) < max(tol, 5e-3)
    assert rel_l2(kv.v[:, :n].float().cpu().numpy(), ocache.v[:, :n]) < max(tol, 5e-3)
    # greedy tokens of the last rows: identical wherever the oracle's top-2 gap is not a near-tie
    srt = np.sort(logits_o[-16:], axis=-1)
    gap = srt[:, -1] - srt[:, -2]
    scale = np.abs(logits_o).max()
    am_g = am_g.cpu().numpy()
    for r in range(16):
        if gap[r] > 2 * tol * scale:
            assert am_g[r] == am_o[n - 16 + r]
    # chunked prefill continues a cache exactly like the one-shot pass does
    kv2 = pair.new_kv()
    pair.engine.verify(toks[:33].cuda(), 0, kv2, 0, want_hidden=False)
    _, hid2 = pair.engine.verify(toks[33:].cuda(), 33, kv2, 1)
    assert rel_l2(hid2.cpu().numpy(), hid_o[33:]) < tol


@pytest.mark.parametrize("M,T", [(2, 1), (3, 1), (1, 1), (2, 3), (5, 4)])
def test_dp_search_against_oracle(pair, M, T):
    cfg = pair.cfg
    if M > cfg.L:
        pytest.skip("more skipped layers than the model has")   # (5, 4): 20 candidate rows, three row blocks
    n = 64
    toks, ocache, am_o, hid_o, _, kv, am_g, hid_g = _prefill_both(pair, n)
    p0 = n - T                                           # first objective position
    L, d = cfg.L, cfg.d_model
    x_o = np.transpose(hid_o[p0:n], (1, 0, 2))           # [L+1, T, d]
    ref = orc.dp_search(pair.oracle, x_o, ocache, p0, p0, M)
    res = pair.engine.dp_search(hid_g[p0], d, (L + 1) * d, kv, p0, p0, T, M)
    torch.cuda.synchronize()
    assert pair.engine.device_status() == 0
    D = res["D"].cpu().numpy()
    margin = res["margin"].cpu().numpy()
    S = res["S"].cpu().numpy()
    # table shape: NaN exactly where j > i
    assert np.array_equal(np.isnan(D), np.isnan(ref["D"]))
    assert int(S.sum()) == M
    # Eq. 2 decisions cell by cell (a near-tie only excuses the cells that descend from it)
    check_search_against_oracle(D, margin, S, res["g_final"].cpu().numpy(), ref, L, M, tol_hidden(cfg))
    # in every case: follow the oracle's decisions and compare states and scores
    forced = torch.from_numpy(ref["choice"].copy()).cuda()
    res_f = pair.engine.dp_search(hid_g[p0], d, (L + 1) * d, kv, p0, p0, T, M, forced_choice=forced)
    np.testing.assert_array_equal(res_f["S"].cpu().numpy(), ref["S"])
    Df = res_f["D"].cpu().numpy()
    np.testing.assert_allclose(Df[~np.isnan(Df)], ref["D"][~np.isnan(Df)], atol=1e-3)
    assert close_hidden(res_f["g_final"].cpu().numpy(), ref["g"][L, M], tol_hidden(cfg))


def test_dp_search_edge_cases(pair):
    cfg = pair.cfg
    L, d = cfg.L, cfg.d_model
    n = 20
    toks, ocache, am_o, hid_o, _, kv, am_g, hid_g = _prefill_both(pair, n)
    p0 = n - 1
    # M = 0: nothing skipped, D(i, 0) = 1
    r0 = pair.engine.dp_search(hid_g[p0], d, 0, kv, p0, p0, 1, 0)
    assert int(r0["S"].sum()) == 0 and torch.all(r0["D"] == 1.0)
    # M = L: everything skipped, g[L][L] = x_0 exactly
    rL = pair.engine.dp_search(hid_g[p0], d, 0, kv, p0, p0, 1, L)
    assert int(rL["S"].sum()) == L
    assert torch.equal(rL["g_final"][0], hid_g[p0, 0])
    ref = orc.dp_search(pair.oracle, hid_o[p0][:, None, :], ocache, p0, p0, L)
    assert abs(float(rL["D"][L, L]) - ref["D"][L, L]) < 1e-3
    # empty visible cache (objective token at position 0)
    kv1 = pair.new_kv()
    _, hid1 = pair.engine.verify(toks[:1].cuda(), 0, kv1, 1)
    oc1 = pair.new_oracle_cache()
    _, hid1_o, _ = orc.verify_forward(pair.oracle, toks[:1].numpy(), oc1, 0)
    ref1 = orc.dp_search(pair.oracle, hid1_o[0][:, None, :], oc1, 0, 0, 2)
    forced = torch.from_numpy(ref1["choice"].copy()).cuda()
    r1 = pair.engine.dp_search(hid1[0], d, 0, kv1, 0, 0, 1, 2, forced_choice=forced)
    D1 = r1["D"].cpu().numpy()
    np.testing.assert_allclose(D1[~np.isnan(D1)], ref1["D"][~np.isnan(D1)], atol=1e-3)
    # two runs in a row give bit-identical tables (fixed reduction orders; the sums that cross CTAs
    # are exact integer atomics on fixed-point values, so arrival order cannot change them)
    ra = pair.engine.dp_search(hid_g[p0], d, 0, kv, p0, p0, 1, 2)
    rb = pair.engine.dp_search(hid_g[p0], d, 0, kv, p0, p0, 1, 2)
    assert torch.equal(ra["D"].nan_to_num(7.0), rb["D"].nan_to_num(7.0)) and torch.equal(ra["S"], rb["S"])


def test_search_with_and_without_deferred_decision(pair):
    """The persistent kernel normally starts a layer's q/k/v product on both Eq. 2 candidates of every
    state before the decision exists; CLASP_FLAG_NO_DEFER makes it wait for the decision instead.  Both
    orders multiply the same operand bytes, so tables, mask and final state agree."""
    cfg = pair.cfg
    L, d = cfg.L, cfg.d_model
    toks, ocache, am_o, hid_o, _, kv, am_g, hid_g = _prefill_both(pair, 48)
    p0 = 47
    M = min(3, L)
    a = pair.engine.dp_search(hid_g[p0], d, 0, kv, p0, p0, 1, M)
    eng2 = pair.engine_with_flags(pair.ccfg.flags | FLAG_NO_DEFER)
    try:
        b = eng2.dp_search(hid_g[p0], d, 0, kv, p0, p0, 1, M)
        torch.cuda.synchronize()
        assert pair.engine.device_status() == 0 and eng2.device_status() == 0
        assert eng2.engine_active() == pair.engine.engine_active()
        assert torch.equal(a["S"], b["S"])
        np.testing.assert_allclose(a["D"].nan_to_num(7.0).cpu().numpy(), b["D"].nan_to_num(7.0).cpu().numpy(), atol=1e-6)
        assert rel_l2(a["g_final"].cpu().numpy(), b["g_final"].cpu().numpy()) < 1e-6
        ref = orc.dp_search(pair.oracle, hid_o[p0][:, None, :], ocache, p0, p0, M)
        forced = torch.from_numpy(ref["choice"].copy()).cuda()
        c = eng2.dp_search(hid_g[p0], d, 0, kv, p0, p0, 1, M, forced_choice=forced)
        Dc = c["D"].cpu().numpy()
        np.testing.assert_allclose(Dc[~np.isnan(Dc)], ref["D"][~np.isnan(Dc)], atol=1e-3)
        assert close_hidden(c["g_final"].cpu().numpy(), ref["g"][L, M], tol_hidden(cfg))
        assert eng2.device_status() == 0
    finally:
        eng2.close()


@pytest.mark.parametrize("M,T,extra", [(2, 1, 0), (3, 1, 0), (3, 2, 0), (4, 1, 0), (3, 1, FLAG_NO_DEFER)])
def test_search_without_the_unreachable_states(pair, M, T, extra):
    """CLASP_FLAG_PRUNE leaves out the states from which (L, M) cannot be reached (j < M - (L - i)).
    Result-neutral: the skip set, g[L][M] and every reachable cell equal the unpruned search's (a row's
    arithmetic does not depend on which other rows share its launch); the cells left out read NaN,
    exactly where the oracle's pruned table has none either."""
    cfg = pair.cfg
    L, d = cfg.L, cfg.d_model
    M = min(M, L)
    n = 40
    toks, ocache, am_o, hid_o, _, kv, am_g, hid_g = _prefill_both(pair, n)
    p0 = n - T
    full = pair.engine.dp_search(hid_g[p0], d, (L + 1) * d, kv, p0, p0, T, M)
    eng2 = pair.engine_with_flags(pair.ccfg.flags | FLAG_PRUNE | extra)
    try:
        pr = eng2.dp_search(hid_g[p0], d, (L + 1) * d, kv, p0, p0, T, M)
        torch.cuda.synchronize()
        assert eng2.device_status() == 0 and pair.engine.device_status() == 0
        Df, Dp = full["D"].cpu().numpy(), pr["D"].cpu().numpy()
        mf, mp = full["margin"].cpu().numpy(), pr["margin"].cpu().numpy()
        x_o = np.transpose(hid_o[p0:n], (1, 0, 2))
        ref = orc.dp_search(pair.oracle, x_o, ocache, p0, p0, M, prune=True)
        assert np.array_equal(np.isnan(Dp), np.isnan(ref["D"]))
        assert np.array_equal(np.isnan(mp), np.isnan(ref["margin"]))
        keep = ~np.isnan(Dp)
        assert np.isnan(Dp).sum() > np.isnan(Df).sum() or M == 1      # something was left out
        np.testing.assert_allclose(Dp[keep], Df[keep], rtol=0, atol=1e-6)
        km = ~np.isnan(mp)
        np.testing.assert_allclose(mp[km], mf[km], rtol=0, atol=2e-6)
        assert torch.equal(pr["S"], full["S"])
        assert rel_l2(pr["g_final"].cpu().numpy(), full["g_final"].cpu().numpy()) < 1e-6
        # and against the oracle's pruned search with its decisions forced
        forced = torch.from_numpy(ref["choice"].copy()).cuda()
        pf = eng2.dp_search(hid_g[p0], d, (L + 1) * d, kv, p0, p0, T, M, forced_choice=forced)
        Dq = pf["D"].cpu().numpy()
        assert np.array_equal(np.isnan(Dq), np.isnan(ref["D"]))
        np.testing.assert_allclose(Dq[keep], ref["D"][keep], atol=1e-3)
        np.testing.assert_array_equal(pf["S"].cpu().numpy(), ref["S"])
        assert close_hidden(pf["g_final"].cpu().numpy(), ref["g"][L, M], tol_hidden(cfg))
        assert eng2.device_status() == 0
    finally:
        eng2.close()


def test_persistent_kernel_serves_the_bf16_models(pair):
    """The one-launch-per-call kernel is what a bf16 context runs (a silent fall-back to one kernel per
    step would be several times slower); the fp32 model and the diagnostic flags use the other path."""
    expect = pair.cfg.dtype == "bf16" and not (pair.ccfg.flags & (FLAG_FORCE_SIMT | FLAG_MULTI_KERNEL))
    assert pair.engine.engine_active() == expect
    assert (pair.engine.engine_ctas() > 0) == expect
    if pair.cfg.dtype == "bf16" and not pair.ccfg.flags:
        eng2 = pair.engine_with_flags(FLAG_MULTI_KERNEL)
        try:
            assert not eng2.engine_active()
            # same arithmetic through the other path: one layer, same input
            kv = pair.new_kv()
            x = datagen.normal_rows(43, 1, (6, pair.cfg.d_model)).to(torch.float32).cuda()
            a = pair.engine.layer_forward(1, x, 3, 2, 0, 0, kv).cpu().numpy()
            b = eng2.layer_forward(1, x, 3, 2, 0, 0, kv).cpu().numpy()
            assert close_hidden(a, b, 5e-3)
            assert eng2.device_status() == 0
        finally:
            eng2.close()


def test_argument_errors(pair):
    import paper_2505_24196_b200 as clasp
    cfg = pair.cfg
    kv = pair.new_kv()
    hid = torch.zeros((cfg.L + 1, cfg.d_model), device="cuda")
    with pytest.raises(clasp.ClaspError) as e:
        pair.engine.dp_search(hid, cfg.d_model, 0, kv, 4, 4, 1, cfg.L + 1)
    assert e.value.code == -1
    with pytest.raises(clasp.ClaspError) as e:
        pair.engine.dp_search(hid, cfg.d_model, 0, kv, pair.max_ctx, pair.max_ctx, 1, 1)
    assert e.value.code == -3
    with pytest.raises(clasp.ClaspError) as e:
        pair.engine.verify(torch.zeros(97, dtype=torch.int32, device="cuda"), 0, kv, 1)
    assert e.value.code == -3
    # float buffers must be 16-byte aligned and strides multiples of 4 elements: refused on the host,
    # nothing is launched
    n0 = pair.engine.launch_count()
    wide = torch.zeros((cfg.L + 1) * (cfg.d_model + 4) + 8, device="cuda")
    with pytest.raises(clasp.ClaspError) as e:
        pair.engine.dp_search(wide[1:], cfg.d_model, 0, kv, 4, 4, 1, 1)          # misaligned base
    assert e.value.code == -1
    with pytest.raises(clasp.ClaspError) as e:
        pair.engine.dp_search(wide, cfg.d_model + 2, 0, kv, 4, 4, 1, 1)          # stride not a multiple of 4
    assert e.value.code == -1
    lib, h = pair.engine.lib, pair.engine.handle
    x = torch.zeros(2 * cfg.d_model + 8, device="cuda")
    kvl = clasp.binding.ClaspKvLayer(kv.array[0].k, kv.array[0].v)
    import ctypes
    rc = lib.clasp_layer_forward(h, 0, x.data_ptr() + 4, cfg.d_model, 1, 1, 0, 0, ctypes.byref(kvl), 0,
                                 x.data_ptr(), cfg.d_model)
    assert rc == -1
    bad = clasp.binding.ClaspKvLayer(kv.array[0].k + 2, kv.array[0].v)
    rc = lib.clasp_layer_forward(h, 0, x.data_ptr(), cfg.d_model, 1, 1, 0, 0, ctypes.byref(bad), 0,
                                 x.data_ptr(), cfg.d_model)
    assert rc == -1
    assert pair.engine.launch_count() == n0
    assert pair.engine.device_status() == 0


def test_draft_with_empty_mask_is_the_full_model(pair):
    cfg = pair.cfg
    n = 12
    toks = datagen.token_ids(cfg, n)
    kv_a, kv_b = pair.new_kv(), pair.new_kv()
    pair.engine.verify(toks[:n - 1].cuda(), 0, kv_a, 0, want_hidden=False)
    pair.engine.verify(toks[:n - 1].cuda(), 0, kv_b, 0, want_hidden=False)
    am, _ = pair.engine.verify(toks[n - 1:].cuda(), n - 1, kv_a, 1, want_hidden=False)
    out = torch.zeros(1, dtype=torch.int32, device="cuda")
    prob = torch.zeros(1, dtype=torch.float32, device="cuda")
    pair.engine.draft_forward(bytes(cfg.L), toks[n - 1:].cuda(), n - 1, kv_b, out, prob)
    assert int(out[0]) == int(am[0])
    assert 0.0 < float(prob[0]) <= 1.0
    assert torch.equal(kv_a.k[:, :n], kv_b.k[:, :n])


def test_decode_is_lossless_and_matches_oracle(pair):
    """Greedy self-speculative tokens == greedy autoregressive tokens of the same CUDA
    model (Sec. 3.1: lossless), and both equal the oracle's as long as the oracle's top-2
    logit gap is not a near-tie."""
    import paper_2505_24196_b200 as clasp
    from paper_2505_24196_b200.decode import greedy_autoregressive
    cfg = pair.cfg
    prompt = datagen.token_ids(cfg, 24, stream=3).tolist()
    n_new = 24
    ar = greedy_autoregressive(pair.engine, pair.new_kv(), prompt, n_new)
    for K, M in [(4, 2), (3, 1)]:
        dec = clasp.SelfSpeculativeDecoder(pair.engine, pair.new_kv(), M=M, K=K)
        sd = dec.generate(prompt, n_new)
        assert sd == ar, (K, M)
        assert all(sum(r["S"]) == M for r in dec.rounds)
    # against the oracle: walk its own greedy path and stop comparing at the first near-tie
    ocache = orc.KVCache(cfg, 96)
    am, _, logits = orc.verify_forward(pair.oracle, prompt, ocache, 0)
    tol = 2 * tol_hidden(cfg)
    pos, tok = len(prompt), int(am[-1])
    row = logits[-1]
    for k in range(n_new):
        srt = np.sort(row)
        if srt[-1] - srt[-2] <= tol * np.abs(row).max():
            break
        assert ar[k] == tok, k
        am, _, lg = orc.verify_forward(pair.oracle, [tok], ocache, pos)
        pos, tok, row = pos + 1, int(am[0]), lg[0]
