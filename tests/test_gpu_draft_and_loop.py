"""The layer-skipped draft forward (Sec. 3.1 drafting stage, Sec. 3.3) and the two loop controls of
Sec. 3.7 / Sec. 5.3.3 (optimisation interval, draft-exiting threshold) against the CPU oracle,
through the C ABI.  Tolerances as in test_gpu_parity: hidden states / K/V relative L2 <= 1e-4
(fp32 model) or 2e-2 (bf16) plus a max-abs guard, probabilities within 1e-3, tokens identical
unless the oracle's top-2 logits are a near-tie."""
import numpy as np
import pytest
import torch

import datagen
from oracle import clasp_oracle as orc
from tests.util import Pair, close_hidden, kv_to_oracle, tol_hidden

pytestmark = pytest.mark.gpu

ENGINES = [("tiny", 0), ("small", 0), ("mini8b", 0)]


@pytest.fixture(scope="module", params=ENGINES, ids=lambda p: f"{p[0]}-flags{p[1]}")
def pair(request):
    name, flags = request.param
    cfg = datagen.CONFIGS[name]
    p = Pair(cfg, max_ctx=160, max_rows=64, max_M=cfg.L, max_T=1, max_head_rows=8, flags=flags)
    yield p
    assert p.engine.device_status() == 0
    p.engine.close()


def _masks(pair, hid_last, kv, n):
    """A searched skip set (M = 2) and hand-made ones that skip the first / the last layer."""
    L = pair.cfg.L
    res = pair.engine.dp_search(hid_last, pair.cfg.d_model, 0, kv, n - 1, n - 1, 1, 2)
    searched = res["S"].cpu().numpy().astype(np.uint8)
    first = np.zeros(L, dtype=np.uint8)
    first[0] = 1
    first[L // 2] = 1
    last = np.zeros(L, dtype=np.uint8)
    last[L - 1] = 1
    last[1] = 1
    alternate = np.array([l % 2 for l in range(L)], dtype=np.uint8)
    return [("searched", searched), ("first+middle", first), ("second+last", last), ("every other", alternate)]


def test_draft_with_skipped_layers_against_oracle(pair):
    """One drafted token with a non-empty skip set: token, confidence, the K/V the kept layers write
    at the draft position, and nothing written by the skipped layers."""
    cfg, eng = pair.cfg, pair.engine
    n = 24
    toks = datagen.token_ids(cfg, n, stream=11)
    kv = pair.new_kv()
    am, hid = eng.verify(toks.cuda(), 0, kv, 1)
    torch.cuda.synchronize()
    tok_in = torch.tensor([int(am[0])], dtype=torch.int32, device="cuda")
    tol = tol_hidden(cfg)
    for name, S in _masks(pair, hid[n - 1], kv, n):
        snap_k, snap_v = kv.k.clone(), kv.v.clone()
        # the oracle reads the very cache the device reads
        ocache = pair.new_oracle_cache()
        kv_to_oracle(kv, n, ocache)
        out = torch.zeros(1, dtype=torch.int32, device="cuda")
        prob = torch.zeros(1, dtype=torch.float32, device="cuda")
        eng.draft_forward(bytes(S.tolist()), tok_in, n, kv, out, prob)
        torch.cuda.synchronize()
        assert eng.device_status() == 0
        am_o, hid_o, lg_o = orc.verify_forward(pair.oracle, [int(tok_in[0])], ocache, n, skip=S)
        # confidence = softmax probability of the greedy token
        p_o = float(orc.top1_probability(lg_o)[0])
        assert abs(float(prob[0]) - p_o) < 1e-3 and abs(float(prob[0]) - p_o) < 0.05 * p_o, name
        # the token, unless the oracle's two best logits are a near-tie
        srt = np.sort(lg_o[0])
        if srt[-1] - srt[-2] > 2 * tol * np.abs(lg_o).max():
            assert int(out[0]) == int(am_o[0]), name
        for l in range(cfg.L):
            k_new, v_new = kv.k[l, n].float().cpu().numpy(), kv.v[l, n].float().cpu().numpy()
            if S[l]:
                # a skipped layer reads and writes nothing
                assert torch.equal(kv.k[l], snap_k[l]) and torch.equal(kv.v[l], snap_v[l]), (name, l)
            else:
                assert close_hidden(k_new, ocache.k[l, n], max(tol, 5e-3)), (name, l)
                assert close_hidden(v_new, ocache.v[l, n], max(tol, 5e-3)), (name, l)
                # ... and only at the draft position
                assert torch.equal(kv.k[l, :n], snap_k[l, :n]) and torch.equal(kv.k[l, n + 1:], snap_k[l, n + 1:])
                assert torch.equal(kv.v[l, :n], snap_v[l, :n]) and torch.equal(kv.v[l, n + 1:], snap_v[l, n + 1:])
        # put the draft position back for the next skip set
        kv.k.copy_(snap_k)
        kv.v.copy_(snap_v)


def test_draft_chain_against_oracle(pair):
    """K drafted tokens in a row, each fed the one before (kept layers read the K/V the earlier
    drafts wrote): tokens and confidences follow the oracle's layer-skipped model."""
    cfg, eng = pair.cfg, pair.engine
    n, K = 20, 4
    toks = datagen.token_ids(cfg, n, stream=12)
    kv = pair.new_kv()
    am, hid = eng.verify(toks.cuda(), 0, kv, 1)
    torch.cuda.synchronize()
    S = np.array([1 if l in (1, cfg.L - 2) else 0 for l in range(cfg.L)], dtype=np.uint8)
    ocache = pair.new_oracle_cache()
    kv_to_oracle(kv, n, ocache)
    chain = torch.zeros(K + 1, dtype=torch.int32, device="cuda")
    chain[0] = am[0]
    prob = torch.zeros(K, dtype=torch.float32, device="cuda")
    for k in range(K):
        eng.draft_forward(bytes(S.tolist()), chain[k:k + 1], n + k, kv, chain[k + 1:k + 2], prob[k:k + 1])
    torch.cuda.synchronize()
    assert eng.device_status() == 0
    tol = tol_hidden(cfg)
    tok = int(chain[0])
    for k in range(K):
        am_o, _, lg_o = orc.verify_forward(pair.oracle, [tok], ocache, n + k, skip=S)
        p_o = float(orc.top1_probability(lg_o)[0])
        assert abs(float(prob[k]) - p_o) < 1e-3 and abs(float(prob[k]) - p_o) < 0.05 * p_o, k
        srt = np.sort(lg_o[0])
        if srt[-1] - srt[-2] <= 2 * tol * np.abs(lg_o).max():
            break                                   # near-tie: the two sides may part ways here
        assert int(chain[k + 1]) == int(am_o[0]), k
        tok = int(am_o[0])


@pytest.mark.parametrize("N", [2, 3])
def test_optimisation_interval(pair, N):
    """Sec. 3.7: with interval N the skip set is searched after every N-th verification and kept in
    between; the output stays the full model's greedy output."""
    import paper_2505_24196_b200 as clasp
    from paper_2505_24196_b200.decode import greedy_autoregressive
    cfg = pair.cfg
    prompt = datagen.token_ids(cfg, 24, stream=3).tolist()
    n_new, M, K = 20, 2, 3
    ar = greedy_autoregressive(pair.engine, pair.new_kv(), prompt, n_new)
    dec = clasp.SelfSpeculativeDecoder(pair.engine, pair.new_kv(), M=M, K=K, dp_interval=N)
    sd = dec.generate(prompt, n_new)
    assert sd == ar
    assert len(dec.rounds) >= 2 * N
    for k, r in enumerate(dec.rounds):
        assert r["S"] == dec.rounds[(k // N) * N]["S"], k          # kept between searches
        assert sum(r["S"]) == M
    if cfg.dtype == "fp32":
        # the fp32 model follows the oracle's loop round for round: same tokens, same accepted
        # counts, and the same skip sets wherever the oracle's search was decisive
        sd_o, rounds_o = orc.greedy_self_speculative(pair.oracle, prompt, n_new, 160, M=M, K=K, dp_interval=N)
        assert sd == sd_o
        assert [r["accepted"] for r in dec.rounds] == [r["accepted"] for r in rounds_o]
        same = sum(bytes(ro["S"].tolist()) == rg["S"] for ro, rg in zip(rounds_o, dec.rounds))
        assert same >= len(rounds_o) - N          # at most one search may sit on a near-tie


def test_draft_exit_threshold(pair):
    """Sec. 5.3.3: a draft whose confidence is below the threshold ends the round's drafting; it is
    still verified, and the output stays lossless.  The rounds stop where the oracle's do, up to the
    first round whose deciding confidence lies within the tolerance of the threshold."""
    import paper_2505_24196_b200 as clasp
    from paper_2505_24196_b200.decode import greedy_autoregressive
    cfg = pair.cfg
    prompt = datagen.token_ids(cfg, 24, stream=4).tolist()
    n_new, M, K = 16, 2, 4
    _, r0 = orc.greedy_self_speculative(pair.oracle, prompt, n_new, 160, M=M, K=K)
    # threshold in the widest gap between the rounds' first-draft confidences (a random-init model is
    # least sure of a round's first draft), so that the decisions are as far from ties as they can be
    first = sorted(r["confidence"][0] for r in r0)
    gaps = [(first[k + 1] - first[k], k) for k in range(1, len(first) - 2)]
    k = max(gaps)[1]
    thr = 0.5 * (first[k] + first[k + 1])
    sd_o, rounds_o = orc.greedy_self_speculative(pair.oracle, prompt, n_new, 160, M=M, K=K, exit_threshold=thr)
    ar = greedy_autoregressive(pair.engine, pair.new_kv(), prompt, n_new)
    dec = clasp.SelfSpeculativeDecoder(pair.engine, pair.new_kv(), M=M, K=K, exit_threshold=thr)
    sd = dec.generate(prompt, n_new)
    assert sd == ar
    for r in dec.rounds:
        c = r["confidence"]
        assert len(c) == r["drafted"] <= K and 0 <= r["accepted"] <= r["drafted"]
        assert all(x >= thr for x in c[:-1])
        assert c[-1] < thr or r["drafted"] == K
    rel = 1e-5 if cfg.dtype == "fp32" else 2e-3
    for ro, rg in zip(rounds_o, dec.rounds):
        if bytes(ro["S"].tolist()) != rg["S"]:
            break                                   # a near-tie in a search: different draft models from here on
        if any(abs(c - thr) <= rel * thr for c in ro["confidence"]):
            break                                   # the decision itself is a near-tie
        assert rg["drafted"] == ro["drafted"]
        np.testing.assert_allclose(rg["confidence"], ro["confidence"], rtol=50 * rel, atol=1e-3)
        if rg["accepted"] != ro["accepted"]:
            break                                   # a near-tie between tokens: the loops part ways
