"""Pins of the oracle's non-greedy path (speculative sampling, Sec. 4 / Table 1 temperature 1) against
what the mathematics fixes: the generator's published known answers, the distribution a Gumbel-max
draw must have, and the losslessness of the accept / resample rule (the committed token is
distributed as the full model's distribution, whatever the draft's; Leviathan et al. 2023, cited by
the paper for that property)."""
import math
import os

import numpy as np
import pytest

import datagen
from oracle import clasp_oracle as orc
from oracle import from_torch

TINY = datagen.CONFIGS["tiny"]
HERE = os.path.dirname(os.path.abspath(__file__))


def chi2_ok(counts, probs, z=5.0):
    """Pearson statistic within mean + z standard deviations of its chi-square law."""
    counts, probs = np.asarray(counts, float), np.asarray(probs, float)
    n = counts.sum()
    stat = float(((counts - n * probs) ** 2 / (n * probs)).sum())
    dof = len(probs) - 1
    return stat < dof + z * math.sqrt(2.0 * dof), stat


def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(HERE, "golden", "philox4x32_10_kat.txt")) if not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        out = orc.philox4x32_10(v[0], v[1], v[2], v[3], v[4], v[5])
        assert [int(x) for x in out] == v[6:10]


def test_uniform_draws_are_uniform_and_differ_by_counter_field():
    idx = np.arange(200000)
    u = orc.uniform_draws(1234, idx, 7, orc.DRAW_DRAFT, 1)
    assert u.min() > 0.0 and u.max() < 1.0
    assert np.all(u * 16777216.0 - 0.5 == np.round(u * 16777216.0 - 0.5))      # on the 2^-24 grid
    ok, stat = chi2_ok(np.bincount((u * 64).astype(int), minlength=64), np.full(64, 1 / 64))
    assert ok, stat
    # every counter field and the seed select another stream: no correlation with the first
    for other in (orc.uniform_draws(1234, idx, 8, orc.DRAW_DRAFT, 1), orc.uniform_draws(1234, idx, 7, orc.DRAW_ACCEPT, 1),
                  orc.uniform_draws(1234, idx, 7, orc.DRAW_DRAFT, 2), orc.uniform_draws(1235, idx, 7, orc.DRAW_DRAFT, 1),
                  orc.uniform_draws(1234 + (1 << 32), idx, 7, orc.DRAW_DRAFT, 1)):
        assert abs(np.corrcoef(u, other)[0, 1]) < 0.01
    assert abs(np.corrcoef(u[:-1], u[1:])[0, 1]) < 0.01


@pytest.mark.parametrize("T", [1.0, 0.5, 2.0])
def test_gumbel_max_draw_has_the_softmax_distribution(T):
    logits = np.array([1.0, -0.5, 2.0, 0.0, -np.inf, 0.7])
    p = np.exp(orc.log_softmax(logits / T))
    n = 30000
    cnt = np.zeros(6)
    for s in range(n):
        cnt[orc.gumbel_max_sample(logits, T, 1000 + s, 3, orc.DRAW_TARGET, 0)] += 1
    assert cnt[4] == 0                                   # probability zero is never drawn
    keep = p > 0
    ok, stat = chi2_ok(cnt[keep], p[keep])
    assert ok, stat


def _rule_trials(p_logits, q_logits, n, T=1.0):
    """n independent rounds of (draft from q, accept / resample against p) on fixed distributions."""
    K, V = q_logits.shape
    first, second, n_acc = np.zeros(V), np.zeros(V), np.zeros(K + 1)
    for s in range(n):
        seed = 77000 + s
        drafts = [orc.gumbel_max_sample(q_logits[k], T, seed, 10 + k, orc.DRAW_DRAFT, 1) for k in range(K)]
        a, new = orc.speculative_accept(p_logits, q_logits, drafts, T, seed, 10, 1)
        assert len(new) == a + 1 and new[:a] == drafts[:a]
        first[new[0]] += 1
        if len(new) > 1:
            second[new[1]] += 1
        n_acc[a] += 1
    return first, second, n_acc


def test_accept_resample_rule_is_lossless():
    """Whatever the draft distribution, the token committed at a position is distributed as the full
    model's distribution there; the acceptance rate is sum_v min(p, q)."""
    rng = np.random.default_rng(5)
    V, K, n = 7, 2, 30000
    p_logits = rng.normal(size=(K + 1, V)) * 1.5
    q_logits = p_logits[:K] + rng.normal(size=(K, V)) * 1.0      # a draft that is off, not unrelated
    q_logits[0, 3] = -np.inf                                       # a token the draft can never propose
    for T in (1.0, 0.7):
        first, second, n_acc = _rule_trials(p_logits, q_logits, n, T)
        p0 = np.exp(orc.log_softmax(p_logits[0] / T))
        q0 = np.exp(orc.log_softmax(q_logits[0] / T))
        ok, stat = chi2_ok(first, p0)
        assert ok, (T, stat)
        rate = np.minimum(p0, q0).sum()
        acc0 = 1.0 - n_acc[0] / n
        assert abs(acc0 - rate) < 5 * math.sqrt(rate * (1 - rate) / n)
        # the second position is reached only after an acceptance and is again distributed as p_1
        p1 = np.exp(orc.log_softmax(p_logits[1] / T))
        ok, stat = chi2_ok(second, p1)
        assert ok, (T, stat)


def test_accept_rule_limits():
    V = 5
    p = np.array([[0.0, 1.0, 2.0, -1.0, 0.5], [1.0, 0.0, 0.0, 0.0, 0.0]])
    # the draft IS the full model: always accepted, then a draw of the next position's distribution
    for s in range(200):
        x = orc.gumbel_max_sample(p[0], 1.0, s, 10, orc.DRAW_DRAFT, 1)
        a, new = orc.speculative_accept(p, p[:1], [x], 1.0, s, 10, 1)
        assert a == 1 and new[0] == x
        assert new[1] == orc.gumbel_max_sample(p[1], 1.0, s, 11, orc.DRAW_TARGET, 1)
    # disjoint supports: always rejected, the replacement is a draw of p itself
    ninf = -np.inf
    pd = np.array([[0.0, 1.0, ninf, ninf, ninf], [0.0] * 5])
    qd = np.array([[ninf, ninf, 0.0, 1.0, 0.5]])
    cnt = np.zeros(V)
    for s in range(4000):
        x = orc.gumbel_max_sample(qd[0], 1.0, s, 10, orc.DRAW_DRAFT, 1)
        a, new = orc.speculative_accept(pd, qd, [x], 1.0, s, 10, 1)
        assert a == 0 and len(new) == 1
        cnt[new[0]] += 1
    assert cnt[2:].sum() == 0
    ok, stat = chi2_ok(cnt[:2], np.exp(orc.log_softmax(pd[0]))[:2])
    assert ok, stat


def test_sampling_loop_alignment_of_positions_and_rows():
    """The loop hands the rule the right rows: with a draft that skips nothing every draft is accepted
    and each committed token is the draw its position's full-model logits give; with a draft that
    skips every layer the replacement at a rejected position is the draw of max(0, p - q) there."""
    model = from_torch.model_from_datagen(TINY)
    prompt = datagen.token_ids(TINY, 12).numpy()
    seed, T, K = 99, 1.0, 3
    toks, rounds = orc.sampling_self_speculative(model, prompt, 9, 64, M=0, K=K, temperature=T, seed=seed,
                                                 fixed_mask=[0] * TINY.L)
    assert all(r["accepted"] == K for r in rounds)
    seq = list(prompt) + toks
    cache = orc.KVCache(TINY, 64)
    _, _, lg = orc.verify_forward(model, seq[:-1], cache, 0)
    P = len(prompt)
    assert toks[0] == orc.gumbel_max_sample(lg[P - 1], T, seed, P, orc.DRAW_TARGET, 0)
    pos = P + 1
    for rnd, r in enumerate(rounds, start=1):
        for k, t in enumerate(r["committed"]):
            if pos - P >= len(toks):
                break
            purpose = orc.DRAW_DRAFT if k < K else orc.DRAW_TARGET
            assert seq[pos] == t == orc.gumbel_max_sample(lg[pos - 1], T, seed, pos, purpose, rnd), (rnd, k)
            pos += 1
    # a draft that skips every layer, at a low temperature (sharp distributions: the two models disagree
    # often enough for rejections to occur within a few rounds)
    T2 = 0.05
    toks2, rounds2 = orc.sampling_self_speculative(model, prompt, 12, 64, M=TINY.L, K=2, temperature=T2, seed=seed,
                                                   fixed_mask=[1] * TINY.L)
    seq2 = list(prompt) + toks2
    cache2 = orc.KVCache(TINY, 64)
    _, _, lp = orc.verify_forward(model, seq2[:-1], cache2, 0)
    pos = P + 1
    checked = 0
    for rnd, r in enumerate(rounds2, start=1):
        a = r["accepted"]
        if a < 2 and pos + a - P < len(toks2):
            # q at the rejected position: the all-skipped model reads only the previous token
            _, _, lq = orc.verify_forward(model, [seq2[pos + a - 1]], orc.KVCache(TINY, 64), pos + a - 1, skip=[1] * TINY.L)
            resid = np.maximum(np.exp(orc.log_softmax(lp[pos + a - 1] / T2)) - np.exp(orc.log_softmax(lq[0] / T2)), 0.0)
            with np.errstate(divide="ignore"):
                want = orc.gumbel_max_sample(np.log(resid), 1.0, seed, pos + a, orc.DRAW_RESIDUAL, rnd)
            assert seq2[pos + a] == want
            checked += 1
        pos += a + 1
    assert checked >= 1
    # same seed, same tokens; another seed, other tokens
    again, _ = orc.sampling_self_speculative(model, prompt, 9, 64, M=0, K=K, temperature=T, seed=seed, fixed_mask=[0] * TINY.L)
    other, _ = orc.sampling_self_speculative(model, prompt, 9, 64, M=0, K=K, temperature=T, seed=seed + 1, fixed_mask=[0] * TINY.L)
    assert again == toks and other != toks
