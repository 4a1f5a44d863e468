"""Non-greedy path on the device (Sec. 4 / Table 1, temperature 1) through the C ABI: draws, the accept /
resample rule and the sampling loop against the oracle, and the losslessness of the rule as a
distribution test (the committed token is distributed as the full model's distribution, chi-square
within five standard deviations; acceptance rate = sum_v min(p, q) within five binomial deviations)."""
import math

import numpy as np
import pytest
import torch

import datagen
from oracle import clasp_oracle as orc
from tests.util import Pair

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


def _one_round(pair, kv, pending, n_valid, mask, K, T, seed, rnd, bufs):
    eng = pair.engine
    tok, q, p, n_acc, committed = bufs
    tok[:1] = pending
    for k in range(K):
        eng.draft_sample(bytes(mask), tok[k:k + 1], n_valid + k, kv, T, seed, rnd, tok[k + 1:k + 2], q[k])
    eng.verify_sample(tok, n_valid, kv, K, q, T, seed, rnd, p, n_acc, committed)
    torch.cuda.synchronize()
    a = int(n_acc[0])
    return tok[1:].cpu().tolist(), a, committed[:a + 1].cpu().tolist()


def _buffers(cfg, K):
    V = cfg.vocab
    return (torch.zeros(K + 1, dtype=torch.int32, device="cuda"), torch.empty((K, V), dtype=torch.float32, device="cuda"),
            torch.empty((K + 1, V), dtype=torch.float32, device="cuda"), torch.zeros(1, dtype=torch.int32, device="cuda"),
            torch.zeros(K + 1, dtype=torch.int32, device="cuda"))


@pytest.mark.parametrize("T", [1.0, 0.3])
def test_draws_and_rule_against_oracle_on_the_devices_own_logits(pair, T):
    """Same logits on both sides (the device's, read back), so only the random draws and the rule are
    compared: drafts are the oracle's Gumbel-max draws of the draft logits, the accepted count and the
    committed tokens are the oracle's for the full model's logits.  (A float near-tie may flip one
    decision in a few hundred; one mismatch is tolerated.)"""
    cfg, eng = pair.cfg, pair.engine
    n, K = 20, 3
    toks = datagen.token_ids(cfg, n, stream=21)
    kv = pair.new_kv()
    am, _ = eng.verify(toks.cuda(), 0, kv, 1, want_hidden=False)
    pending = int(am[0])
    mask = [1 if l in (1, cfg.L - 1) else 0 for l in range(cfg.L)]
    bufs = _buffers(cfg, K)
    mismatches, rejections = 0, 0
    for trial in range(24):
        seed, rnd = 5000 + 17 * trial + (trial << 33), 1 + trial % 3
        drafts, a, committed = _one_round(pair, kv, pending, n, mask, K, T, seed, rnd, bufs)
        q64, p64 = bufs[1].double().cpu().numpy(), bufs[2].double().cpu().numpy()
        want_d = [orc.gumbel_max_sample(q64[k], T, seed, n + k + 1, orc.DRAW_DRAFT, rnd) for k in range(K)]
        # (draft k + 1 is conditioned on draft k: compare position by position)
        mismatches += sum(int(x != y) for x, y in zip(drafts, want_d))
        a_o, new_o = orc.speculative_accept(p64, q64, drafts, T, seed, n + 1, rnd)
        mismatches += int((a, committed) != (a_o, new_o))
        rejections += int(a < K)
        assert len(committed) == a + 1 and committed[:a] == drafts[:a]
    assert mismatches <= 1
    assert eng.device_status() == 0


def test_sampling_without_drafts_is_a_draw_of_the_full_model(pair):
    """n_drafts = 0 (prompt prefill, plain ancestral sampling): the token after the rows is the oracle's
    draw for the device's logits."""
    cfg, eng = pair.cfg, pair.engine
    toks = datagen.token_ids(cfg, 9, stream=22)
    kv = pair.new_kv()
    p = torch.empty((1, cfg.vocab), dtype=torch.float32, device="cuda")
    n_acc = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.zeros(1, dtype=torch.int32, device="cuda")
    for seed in (1, 2, 3 + (7 << 32)):
        eng.verify_sample(toks.cuda(), 0, kv, 0, None, 0.8, seed, 0, p, n_acc, out)
        torch.cuda.synchronize()
        assert int(n_acc[0]) == 0
        assert int(out[0]) == orc.gumbel_max_sample(p[0].double().cpu().numpy(), 0.8, seed, 9, orc.DRAW_TARGET, 0)


def test_sampling_loop_follows_the_oracle_loop(pair):
    """The fp32 model follows the oracle's sampling loop token for token (same seed, same skip set);
    every model's loop is reproducible and seed-dependent."""
    import paper_2505_24196_b200 as clasp
    cfg = pair.cfg
    prompt = datagen.token_ids(cfg, 16, stream=23).tolist()
    mask = bytes([1 if l % 3 == 1 else 0 for l in range(cfg.L)])
    n_new, K, T, seed = 12, 3, 1.0, 4242
    s1 = clasp.SpeculativeSampler(pair.engine, pair.new_kv(), M=0, K=K, temperature=T, seed=seed, fixed_mask=mask)
    out1 = s1.generate(prompt, n_new)
    s2 = clasp.SpeculativeSampler(pair.engine, pair.new_kv(), M=0, K=K, temperature=T, seed=seed, fixed_mask=mask)
    assert s2.generate(prompt, n_new) == out1
    s3 = clasp.SpeculativeSampler(pair.engine, pair.new_kv(), M=0, K=K, temperature=T, seed=seed + 1, fixed_mask=mask)
    assert s3.generate(prompt, n_new) != out1
    assert all(0 <= r["accepted"] <= K and len(r["committed"]) == r["accepted"] + 1 for r in s1.rounds)
    if cfg.dtype == "fp32":
        out_o, rounds_o = orc.sampling_self_speculative(pair.oracle, prompt, n_new, 160, M=0, K=K, temperature=T,
                                                        seed=seed, fixed_mask=list(mask))
        assert out1 == out_o
        assert [r["accepted"] for r in s1.rounds] == [r["accepted"] for r in rounds_o]
    # with the search in the loop: runs, stays reproducible
    s4 = clasp.SpeculativeSampler(pair.engine, pair.new_kv(), M=2, K=K, temperature=T, seed=seed)
    s5 = clasp.SpeculativeSampler(pair.engine, pair.new_kv(), M=2, K=K, temperature=T, seed=seed)
    assert s4.generate(prompt, 8) == s5.generate(prompt, 8)
    assert all(sum(r["S"]) == 2 for r in s4.rounds)


def _chi2_ok(counts, probs, z=5.0):
    counts, probs = np.asarray(counts, float), np.asarray(probs, float)
    n = counts.sum()
    stat = float(((counts - n * probs) ** 2 / (n * probs)).sum())
    dof = len(probs) - 1
    return stat < dof + z * math.sqrt(2.0 * dof), stat


@pytest.mark.parametrize("T", [1.0, 0.05])
def test_committed_token_is_distributed_as_the_full_model(pair, T):
    """Losslessness on the device: over many seeds at one fixed context, the first committed token
    follows softmax(p / T) of the full model's logits there, although the drafts come from a model with
    half of its layers skipped; the share of accepted first drafts is sum_v min(p, q)."""
    cfg, eng = pair.cfg, pair.engine
    if cfg.name != "tiny":
        pytest.skip("statistics on the small vocabulary only (the rule's code is the same for every model)")
    n, K, N = 12, 1, 4000
    toks = datagen.token_ids(cfg, n, stream=24)
    kv = pair.new_kv()
    am, _ = eng.verify(toks.cuda(), 0, kv, 1, want_hidden=False)
    pending = int(am[0])
    mask = [l % 2 for l in range(cfg.L)]
    bufs = _buffers(cfg, K)
    first = np.zeros(cfg.vocab)
    accepted = 0
    for s in range(N):
        drafts, a, committed = _one_round(pair, kv, pending, n, mask, K, T, 900000 + s, 1, bufs)
        first[committed[0]] += 1
        accepted += a
    p0 = np.exp(orc.log_softmax(bufs[2][0].double().cpu().numpy() / T))
    q0 = np.exp(orc.log_softmax(bufs[1][0].double().cpu().numpy() / T))
    # buckets: the likeliest tokens one by one while each expects >= 20 draws, the rest by token id mod 8
    order = np.argsort(-p0)
    single = [v for v in order[:24] if p0[v] * N >= 20]
    rest = np.setdiff1d(np.arange(cfg.vocab), single)
    counts = [first[v] for v in single] + [first[rest[rest % 8 == b]].sum() for b in range(8)]
    probs = [p0[v] for v in single] + [p0[rest[rest % 8 == b]].sum() for b in range(8)]
    keep = [i for i, pr in enumerate(probs) if pr * N >= 5]
    counts, probs = np.array(counts)[keep], np.array(probs)[keep]
    ok, stat = _chi2_ok(counts, probs / probs.sum())      # (conditioned on the buckets that were kept)
    assert ok, stat
    rate = float(np.minimum(p0, q0).sum())
    assert abs(accepted / N - rate) < 5 * math.sqrt(max(rate * (1 - rate), 1e-4) / N) + 1e-3
