"""Pins of the CPU oracle against what the paper and the mathematics fix.

Each test is chosen so that a plausible slip in the oracle (dropped term, wrong
sign or index, transposed operand, off-by-one in the table) breaks it.
"""
import dataclasses
import itertools
import math

import numpy as np
import pytest
import torch

import datagen
from oracle import clasp_oracle as orc
from oracle import from_torch

TINY = datagen.CONFIGS["tiny"]


@pytest.fixture(scope="module")
def tiny():
    model = from_torch.model_from_datagen(TINY)
    toks = datagen.token_ids(TINY, 64).numpy()
    cache = orc.KVCache(TINY, 128)
    am, hid, logits = orc.verify_forward(model, toks, cache, 0)
    return model, toks, cache, am, hid, logits


# ---------------- elementary pieces: closed forms ----------------

def test_rmsnorm_closed_form():
    x = np.full((1, 8), 3.0)
    w = np.arange(1, 9, dtype=np.float64)
    # mean square is 9, so x / sqrt(9 + eps) is 1 up to eps
    np.testing.assert_allclose(orc.rmsnorm(x, w, 0.0)[0], w, rtol=1e-15)
    y = orc.rmsnorm(np.array([[3.0, 4.0]]), np.ones(2), 0.0)
    np.testing.assert_allclose(y[0], [3 / math.sqrt(12.5), 4 / math.sqrt(12.5)], rtol=1e-15)
    # eps is added to the mean square, under the root
    y = orc.rmsnorm(np.array([[0.0, 0.0]]), np.ones(2), 1e-5)
    assert np.all(y == 0)
    y = orc.rmsnorm(np.array([[2.0, 2.0]]), np.ones(2), 5.0)
    np.testing.assert_allclose(y[0], [2 / 3, 2 / 3], rtol=1e-15)


def test_rope_is_a_rotation_of_pairs_i_and_i_plus_half():
    hd, theta = 8, 10000.0
    x = datagen.normal_rows(11, 0, (3, 2, hd)).numpy()
    pos = np.array([0, 1, 7])
    y = orc.rope(x, pos, theta)
    np.testing.assert_array_equal(y[0], x[0])                    # position 0: identity
    np.testing.assert_allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-14)
    # pair (i, i + hd/2) turns by pos * theta^(-2i/hd), counter-clockwise
    for i in range(hd // 2):
        ang = 7 * theta ** (-2.0 * i / hd)
        a, b = x[2, 1, i], x[2, 1, i + hd // 2]
        np.testing.assert_allclose(y[2, 1, i], a * math.cos(ang) - b * math.sin(ang), rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(y[2, 1, i + hd // 2], b * math.cos(ang) + a * math.sin(ang), rtol=1e-12, atol=1e-14)
    # relative-position property: <rope(q,m), rope(k,n)> depends on m-n only
    q = datagen.normal_rows(11, 1, (1, 1, hd)).numpy()
    k = datagen.normal_rows(11, 2, (1, 1, hd)).numpy()
    d1 = np.sum(orc.rope(q, np.array([5]), theta) * orc.rope(k, np.array([2]), theta))
    d2 = np.sum(orc.rope(q, np.array([13]), theta) * orc.rope(k, np.array([10]), theta))
    np.testing.assert_allclose(d1, d2, rtol=1e-12)


def test_cosine_score_closed_forms():
    a = np.array([[1.0, 0.0], [0.0, 2.0]])
    b = np.array([[0.0, 5.0], [0.0, 3.0]])
    assert orc.cosine_score(a[:1], b[:1]) == 0.0
    assert orc.cosine_score(a[1:], b[1:]) == 1.0
    assert orc.cosine_score(a, b) == 0.5                         # mean over the T rows
    assert orc.cosine_score(a[:1], -3 * a[:1]) == -1.0
    assert orc.cosine_score(np.zeros((1, 2)), a[:1]) == 0.0      # zero vector: eps guard, no NaN


def _layer_by_loops(X, w, ck, cv, C, pos0, cfg):
    """The decoder layer written out with scalar loops (tiny sizes only)."""
    T, d = X.shape
    nq, nkv, hd = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    half = hd // 2

    def norm(row, wt):
        ms = sum(v * v for v in row) / len(row)
        return [v / math.sqrt(ms + cfg.rms_eps) * g for v, g in zip(row, wt)]

    def matvec(Wm, vec):
        return [sum(Wm[o][i] * vec[i] for i in range(len(vec))) for o in range(len(Wm))]

    def rot(vec, p):
        out = list(vec)
        for i in range(half):
            ang = p * cfg.rope_theta ** (-2.0 * i / hd)
            out[i] = vec[i] * math.cos(ang) - vec[i + half] * math.sin(ang)
            out[i + half] = vec[i + half] * math.cos(ang) + vec[i] * math.sin(ang)
        return out

    ks, vs, outs = [], [], []
    for t in range(T):
        a = norm(list(X[t]), w["attn_norm"])
        q, k, v = matvec(w["wq"], a), matvec(w["wk"], a), matvec(w["wv"], a)
        q = [rot(q[h * hd:(h + 1) * hd], pos0 + t) for h in range(nq)]
        k = [rot(k[h * hd:(h + 1) * hd], pos0 + t) for h in range(nkv)]
        v = [v[h * hd:(h + 1) * hd] for h in range(nkv)]
        ks.append(k)
        vs.append(v)
        att = []
        for h in range(nq):
            kh = h // (nq // nkv)
            keys = [list(ck[c, kh]) for c in range(C)] + [ks[u][kh] for u in range(t + 1)]
            vals = [list(cv[c, kh]) for c in range(C)] + [vs[u][kh] for u in range(t + 1)]
            sc = [sum(a_ * b_ for a_, b_ in zip(q[h], key)) / math.sqrt(hd) for key in keys]
            mx = max(sc)
            e = [math.exp(s - mx) for s in sc]
            z = sum(e)
            att += [sum(e[n] / z * vals[n][c] for n in range(len(vals))) for c in range(hd)]
        o = matvec(w["wo"], att)
        x1 = [X[t][i] + o[i] for i in range(d)]
        m = norm(x1, w["mlp_norm"])
        gt, up = matvec(w["w_gate"], m), matvec(w["w_up"], m)
        act = [g_ / (1.0 + math.exp(-g_)) * u_ for g_, u_ in zip(gt, up)]
        dn = matvec(w["w_down"], act)
        outs.append([x1[i] + dn[i] for i in range(d)])
    return np.array(outs)


def test_decoder_layer_against_scalar_loops():
    cfg = dataclasses.replace(TINY, d_model=16, n_q_heads=4, n_kv_heads=2, head_dim=4, d_ffn=24, L=1)
    rng = lambda s, shape, std=1.0: datagen.normal_rows(21, s, shape, std).numpy()
    w = {"attn_norm": 1 + 0.2 * rng(0, (16,)), "mlp_norm": 1 + 0.2 * rng(1, (16,)),
         "wq": rng(2, (16, 16), 0.3), "wk": rng(3, (8, 16), 0.3), "wv": rng(4, (8, 16), 0.3),
         "wo": rng(5, (16, 16), 0.3), "w_gate": rng(6, (24, 16), 0.3), "w_up": rng(7, (24, 16), 0.3),
         "w_down": rng(8, (16, 24), 0.3)}
    C, T, pos0 = 5, 3, 9
    ck, cv = rng(9, (C, 2, 4)), rng(10, (C, 2, 4))
    X = rng(11, (T, 16))
    out, k, v = orc.decoder_layer(X, w, ck, cv, C, pos0, cfg)
    ref = _layer_by_loops(X, w, ck, cv, C, pos0, cfg)
    np.testing.assert_allclose(out, ref, rtol=1e-11, atol=1e-12)


def test_full_forward_against_transformers_llama():
    """Library-routine pin: the same tensors loaded into the `transformers`
    LLaMA model give the same per-layer hidden states and logits (float64)."""
    transformers = pytest.importorskip("transformers")
    cfg = dataclasses.replace(TINY, L=3, norm_std=0.1, name="tiny3")
    layers = [datagen.layer_weights(cfg, l) for l in range(cfg.L)]
    head = datagen.head_weights(cfg)
    model = from_torch.model_from_tensors(cfg, layers, head)
    toks = datagen.token_ids(cfg, 12).numpy()
    cache = orc.KVCache(cfg, 16)
    am, hid, logits = orc.verify_forward(model, toks, cache, 0)

    hf_cfg = transformers.LlamaConfig(
        vocab_size=cfg.vocab, hidden_size=cfg.d_model, intermediate_size=cfg.d_ffn,
        num_hidden_layers=cfg.L, num_attention_heads=cfg.n_q_heads, num_key_value_heads=cfg.n_kv_heads,
        head_dim=cfg.head_dim, rms_norm_eps=cfg.rms_eps, rope_theta=cfg.rope_theta,
        max_position_embeddings=64, attention_bias=False, mlp_bias=False, tie_word_embeddings=False,
        attn_implementation="eager")
    try:
        hf_cfg.rope_parameters = {"rope_type": "default", "rope_theta": cfg.rope_theta}
    except Exception:
        pass
    hf = transformers.LlamaForCausalLM(hf_cfg).to(torch.float64).eval()
    sd = {"model.embed_tokens.weight": head["embed"], "model.norm.weight": head["final_norm"],
          "lm_head.weight": head["lm_head"]}
    names = {"attn_norm": "input_layernorm.weight", "mlp_norm": "post_attention_layernorm.weight",
             "wq": "self_attn.q_proj.weight", "wk": "self_attn.k_proj.weight", "wv": "self_attn.v_proj.weight",
             "wo": "self_attn.o_proj.weight", "w_gate": "mlp.gate_proj.weight", "w_up": "mlp.up_proj.weight",
             "w_down": "mlp.down_proj.weight"}
    for l, lw in enumerate(layers):
        for k, v in lw.items():
            sd[f"model.layers.{l}.{names[k]}"] = v
    missing = hf.load_state_dict({k: v.to(torch.float64) for k, v in sd.items()}, strict=False)
    assert not [m for m in missing.missing_keys if "rotary" not in m]
    with torch.no_grad():
        out = hf(torch.from_numpy(toks.astype(np.int64))[None], output_hidden_states=True)
    # transformers' hidden_states[l] for l < L is the residual stream entering layer l;
    # its last entry is AFTER the final norm, so compare that one through the logits.
    # The library evaluates the rotary angles in float32 whatever the model dtype,
    # which bounds the agreement near 1e-7; a wrong convention (pairing, sign,
    # GQA mapping, norm placement) shows up at order 1.
    for l in range(cfg.L):
        np.testing.assert_allclose(hid[:, l], out.hidden_states[l][0].numpy(), rtol=1e-5, atol=1e-6)
    np.testing.assert_allclose(logits, out.logits[0].numpy(), rtol=1e-5, atol=1e-6)
    # incremental decoding through the cache equals the one-shot forward
    cache2 = orc.KVCache(cfg, 16)
    orc.verify_forward(model, toks[:7], cache2, 0)
    _, hid2, _ = orc.verify_forward(model, toks[7:], cache2, 7)
    np.testing.assert_allclose(hid2, hid[7:], rtol=1e-10, atol=1e-12)


# ---------------- the dynamic programme ----------------

def test_column_zero_is_the_full_model(tiny):
    """Applying layer i-1 to g[i-1, 0] = x_{i-1} under the search's attention
    rule (cache before the token + the state's own key) gives x_i: cosine 1."""
    model, toks, cache, am, hid, _ = tiny
    p = 63
    x = hid[p]
    for i in range(1, TINY.L + 1):
        G, _, _ = orc.decoder_layer(x[i - 1][None], model.layer(i - 1), cache.k[i - 1], cache.v[i - 1], p, p, TINY)
        np.testing.assert_allclose(G[0], x[i], rtol=1e-12, atol=1e-13)
        assert abs(orc.cosine_score(x[i][None], G) - 1.0) < 1e-14
    r = orc.dp_search(model, x[:, None, :], cache, p, p, 0)
    assert r["S"].sum() == 0 and np.all(r["D"][:, 0] == 1.0)


@pytest.mark.parametrize("M", [1, 2, 3, 8])
def test_backtracked_set_has_M_layers_and_replays_to_g(tiny, M):
    model, toks, cache, am, hid, _ = tiny
    p = 63
    x = hid[p][:, None, :]
    r = orc.dp_search(model, x, cache, p, p, M)
    assert int(r["S"].sum()) == M
    rp = orc.replay(model, x[0], r["S"], cache, p, p)
    # (column 0 of the table holds the full model's x_i from the batched prefill while the
    # replay recomputes them row by row: equal up to the matmul's summation order)
    np.testing.assert_allclose(rp, r["g"][TINY.L, M], rtol=1e-11, atol=1e-13)
    assert abs(orc.cosine_score(x[TINY.L], rp) - r["D"][TINY.L, M]) < 1e-13
    # table shape invariants: defined exactly where j <= i; D is the larger candidate
    for i in range(TINY.L + 1):
        for j in range(M + 1):
            assert np.isnan(r["D"][i, j]) == (j > i)
    if M == 8:                                     # everything skipped: g = x_0
        np.testing.assert_array_equal(r["g"][8, 8], x[0])


def test_dp_step_is_eq2(tiny):
    """Recompute one interior cell by hand from row i-1 of the table."""
    model, toks, cache, am, hid, _ = tiny
    p, M = 63, 3
    x = hid[p][:, None, :]
    r = orc.dp_search(model, x, cache, p, p, M)
    for (i, j) in [(2, 1), (5, 2), (8, 3), (4, 3)]:
        G, _, _ = orc.decoder_layer(r["g"][i - 1, j], model.layer(i - 1), cache.k[i - 1], cache.v[i - 1], p, p, TINY)
        ca = orc.cosine_score(x[i], G)
        cs = orc.cosine_score(x[i], r["g"][i - 1, j - 1])
        assert r["D"][i, j] == max(ca, cs)
        np.testing.assert_array_equal(r["g"][i, j], G if ca > cs else r["g"][i - 1, j - 1])
        assert r["margin"][i, j] == ca - cs


def test_exhaustive_search_bounds_the_dp(tiny):
    """All C(8,2) = 28 skip sets: the best is at least the DP's objective, and
    the DP's own set scores exactly D[L, M] in the enumeration."""
    model, toks, cache, am, hid, _ = tiny
    p, M = 63, 2
    x = hid[p][:, None, :]
    r = orc.dp_search(model, x, cache, p, p, M)
    bf = orc.brute_force(model, x, cache, p, p, M)
    assert len(bf) == 28
    assert bf[0][0] >= r["D"][TINY.L, M] - 1e-13
    mine = [s for s, S in bf if np.array_equal(S, r["S"])]
    assert len(mine) == 1 and abs(mine[0] - r["D"][TINY.L, M]) < 1e-13


def test_L2_M1_dp_equals_exhaustive():
    """With two layers and one skip the last step compares both subsets directly."""
    cfg = dataclasses.replace(TINY, L=2, name="tiny2")
    model = from_torch.model_from_datagen(cfg)
    toks = datagen.token_ids(cfg, 10).numpy()
    cache = orc.KVCache(cfg, 16)
    _, hid, _ = orc.verify_forward(model, toks, cache, 0)
    x = hid[9][:, None, :]
    r = orc.dp_search(model, x, cache, 9, 9, 1)
    bf = orc.brute_force(model, x, cache, 9, 9, 1)
    assert abs(bf[0][0] - r["D"][2, 1]) < 1e-13
    np.testing.assert_array_equal(bf[0][1], r["S"])


def test_L1_M1():
    cfg = dataclasses.replace(TINY, L=1, name="tiny1")
    model = from_torch.model_from_datagen(cfg)
    toks = datagen.token_ids(cfg, 6).numpy()
    cache = orc.KVCache(cfg, 8)
    _, hid, _ = orc.verify_forward(model, toks, cache, 0)
    x = hid[5][:, None, :]
    r = orc.dp_search(model, x, cache, 5, 5, 1)
    np.testing.assert_array_equal(r["S"], [1])
    assert r["D"][1, 1] == orc.cosine_score(x[1], x[0])


def test_identity_layers_skip_the_last_M():
    """W_o = W_down = 0 makes every layer the identity: all cosines are exactly 1,
    every tie keeps the skip candidate, so the walk marks the LAST M layers.
    Pins the strict '>' and the start and direction of the backtrack."""
    cfg = dataclasses.replace(TINY, L=6, name="tiny6")
    layers = [datagen.layer_weights(cfg, l) for l in range(cfg.L)]
    for lw in layers:
        lw["wo"].zero_()
        lw["w_down"].zero_()
    model = from_torch.model_from_tensors(cfg, layers, datagen.head_weights(cfg))
    toks = datagen.token_ids(cfg, 9).numpy()
    cache = orc.KVCache(cfg, 16)
    _, hid, _ = orc.verify_forward(model, toks, cache, 0)
    x = hid[8][:, None, :]
    for M in (1, 2, 4):
        r = orc.dp_search(model, x, cache, 8, 8, M)
        np.testing.assert_array_equal(r["S"], [0] * (cfg.L - M) + [1] * M)
        assert abs(np.nanmin(r["D"]) - 1.0) < 1e-15 and np.nanmax(np.abs(r["margin"])) == 0.0


def test_backtrack_walk_by_hand():
    # L=4, M=2; choices written so the walk goes (4,2) apply -> (3,2) skip -> (2,1) apply -> (1,1) skip
    ch = np.full((5, 3), 255, dtype=np.uint8)
    ch[4, 2], ch[3, 2], ch[2, 1], ch[1, 1] = orc.APPLY, orc.SKIP, orc.APPLY, orc.SKIP
    np.testing.assert_array_equal(orc.backtrack(ch, 4, 2), [1, 0, 1, 0])
    # exits at j = 0 with i > 0: the lower layers are all kept
    ch = np.full((5, 2), 255, dtype=np.uint8)
    ch[4, 1] = orc.SKIP
    np.testing.assert_array_equal(orc.backtrack(ch, 4, 1), [0, 0, 0, 1])


def test_forced_choice_replays_any_subset(tiny):
    """Forcing the decisions along a chosen path makes g[L, M] the replay of that set."""
    model, toks, cache, am, hid, _ = tiny
    p, M, L = 63, 2, TINY.L
    x = hid[p][:, None, :]
    S = np.array([0, 1, 0, 0, 1, 0, 0, 0], dtype=np.uint8)
    forced = np.full((L + 1, M + 1), 255, dtype=np.uint8)
    j = 0
    for i in range(1, L + 1):                       # path from (0,0) upward
        if S[i - 1]:
            j += 1
            forced[i, j] = orc.SKIP
        else:
            forced[i, j] = orc.APPLY
    r = orc.dp_search(model, x, cache, p, p, M, forced_choice=forced)
    np.testing.assert_array_equal(r["S"], S)
    np.testing.assert_allclose(r["g"][L, M], orc.replay(model, x[0], S, cache, p, p), rtol=1e-11, atol=1e-13)


def test_T_gt_1_reduces_to_T1_on_its_first_row(tiny):
    """With T rows the first row of every state sees exactly what a T = 1 search
    at that position sees (causality inside a state)."""
    model, toks, cache, am, hid, _ = tiny
    p = 60
    xT = np.transpose(hid[p:p + 3], (1, 0, 2))          # [L+1, 3, d]
    forced = orc.dp_search(model, xT[:, :1], cache, p, p, 2)["choice"]
    rT = orc.dp_search(model, xT, cache, p, p, 2, forced_choice=forced)
    r1 = orc.dp_search(model, xT[:, :1], cache, p, p, 2)
    np.testing.assert_allclose(rT["g"][TINY.L, 2][0], r1["g"][TINY.L, 2][0], rtol=1e-12)


# ---------------- the decoding loop: losslessness ----------------

@pytest.mark.parametrize("K,M,mask", [(4, 2, None), (3, 3, None), (5, 0, [0, 1, 1, 0, 1, 0, 1, 1]), (1, 1, None)])
def test_self_speculative_is_lossless(K, M, mask):
    """Greedy self-speculative output is token-identical to plain greedy decoding
    of the full model, whatever the skip set and draft length (Sec. 3.1, Sec. 4)."""
    model = from_torch.model_from_datagen(TINY)
    prompt = datagen.token_ids(TINY, 24).numpy()
    n_new = 20
    ar = orc.greedy_autoregressive(model, prompt, n_new, 80)
    sd, rounds = orc.greedy_self_speculative(model, prompt, n_new, 80, M=M, K=K, fixed_mask=mask)
    assert sd == ar
    assert all(0 <= r["accepted"] <= K for r in rounds)
    if mask is None:
        assert all(int(r["S"].sum()) == M for r in rounds)


def test_full_mask_draft_accepts_everything():
    """A draft that skips nothing IS the full model: every draft token is accepted."""
    model = from_torch.model_from_datagen(TINY)
    prompt = datagen.token_ids(TINY, 16).numpy()
    sd, rounds = orc.greedy_self_speculative(model, prompt, 12, 64, M=0, K=3, fixed_mask=[0] * 8)
    assert all(r["accepted"] == 3 for r in rounds)
    assert sd == orc.greedy_autoregressive(model, prompt, 12, 64)


def test_argmax_takes_the_lowest_index_on_an_exact_tie():
    """Greedy accept rule: ties between logits go to the lowest token id."""
    lg = np.array([[0.0, 3.0, 3.0, 1.0], [2.0, 2.0, 2.0, 2.0], [-1.0, -5.0, -1.0, -1.0]])
    np.testing.assert_array_equal(orc.argmax_lowest(lg), [1, 0, 0])


def test_top1_probability_closed_forms():
    # uniform logits: 1 / vocab; one logit ahead by ln(3) among 4: 3 / (3 + 3) = 1/2
    np.testing.assert_allclose(orc.top1_probability(np.zeros((1, 8))), [0.125], rtol=1e-15)
    np.testing.assert_allclose(orc.top1_probability(np.array([[math.log(3.0), 0.0, 0.0, 0.0]])), [0.5], rtol=1e-15)
    # invariant under a shift of all logits, also a large one
    np.testing.assert_allclose(orc.top1_probability(np.array([[1000.0 + math.log(3.0), 1000.0, 1000.0, 1000.0]])),
                               [0.5], rtol=1e-12)


# ---------------- lower optimisation frequency (Sec. 3.7) ----------------

@pytest.mark.parametrize("N", [2, 3])
def test_optimisation_interval_keeps_the_skip_set_between_searches(N):
    """With interval N the skip set changes only after every N-th verification; the output
    stays lossless, and the searches that do run see the same inputs as in the interval-1
    loop as long as the committed tokens agree (they do: both are lossless)."""
    model = from_torch.model_from_datagen(TINY)
    prompt = datagen.token_ids(TINY, 24).numpy()
    n_new = 18
    ar = orc.greedy_autoregressive(model, prompt, n_new, 96)
    sd, rounds = orc.greedy_self_speculative(model, prompt, n_new, 96, M=2, K=3, dp_interval=N)
    assert sd == ar
    assert len(rounds) >= 2 * N
    for k in range(len(rounds)):
        first_of_block = (k // N) * N
        np.testing.assert_array_equal(rounds[k]["S"], rounds[first_of_block]["S"])
    assert all(int(r["S"].sum()) == 2 for r in rounds)


def test_an_interval_beyond_the_run_is_the_fixed_first_skip_set():
    """Limit of Sec. 3.7: if the search never runs again, every round drafts with the set found
    after the prefill -- the loop with that set given as a fixed mask, round for round."""
    model = from_torch.model_from_datagen(TINY)
    prompt = datagen.token_ids(TINY, 24).numpy()
    n_new = 14
    sd, rounds = orc.greedy_self_speculative(model, prompt, n_new, 96, M=2, K=3, dp_interval=10 ** 6)
    S0 = rounds[0]["S"]
    sd_f, rounds_f = orc.greedy_self_speculative(model, prompt, n_new, 96, M=2, K=3, fixed_mask=S0)
    assert sd == sd_f
    assert [r["accepted"] for r in rounds] == [r["accepted"] for r in rounds_f]
    assert all(np.array_equal(r["S"], S0) for r in rounds)
    # and the first set is the search on the last prompt token (reading 12)
    cache = orc.KVCache(TINY, 96)
    _, hid, _ = orc.verify_forward(model, prompt, cache, 0)
    ref = orc.dp_search(model, hid[len(prompt) - 1][:, None, :], cache, len(prompt) - 1, len(prompt) - 1, 2)
    np.testing.assert_array_equal(S0, ref["S"])


# ---------------- draft-exiting threshold (Sec. 5.3.3) ----------------

def test_exit_threshold_limits():
    """Threshold 0 never stops a round early (the fixed-length loop, round for round); a threshold
    above 1 stops every round after its first draft (the K = 1 loop, round for round)."""
    model = from_torch.model_from_datagen(TINY)
    prompt = datagen.token_ids(TINY, 24).numpy()
    n_new = 14
    base, r_base = orc.greedy_self_speculative(model, prompt, n_new, 96, M=2, K=3)
    zero, r_zero = orc.greedy_self_speculative(model, prompt, n_new, 96, M=2, K=3, exit_threshold=0.0)
    assert zero == base and [r["drafted"] for r in r_zero] == [3] * len(r_base)
    one, r_one = orc.greedy_self_speculative(model, prompt, n_new, 96, M=2, K=3, exit_threshold=1.5)
    k1, r_k1 = orc.greedy_self_speculative(model, prompt, n_new, 96, M=2, K=1)
    assert one == k1
    assert [r["drafted"] for r in r_one] == [1] * len(r_k1)
    assert [r["accepted"] for r in r_one] == [r["accepted"] for r in r_k1]


def test_exit_threshold_stops_at_the_first_low_confidence_draft_and_stays_lossless():
    model = from_torch.model_from_datagen(TINY)
    prompt = datagen.token_ids(TINY, 24).numpy()
    n_new = 16
    ar = orc.greedy_autoregressive(model, prompt, n_new, 96)
    _, r0 = orc.greedy_self_speculative(model, prompt, n_new, 96, M=2, K=4)
    # (a random-init model is least sure of a round's first draft: put the threshold among those, so
    # that some rounds stop after one draft and the others run to the cap)
    first = sorted(r["confidence"][0] for r in r0)
    thr = first[len(first) // 2]
    sd, rounds = orc.greedy_self_speculative(model, prompt, n_new, 96, M=2, K=4, exit_threshold=thr)
    assert sd == ar
    assert any(r["drafted"] < 4 for r in rounds) and any(r["drafted"] > 1 for r in rounds)
    for r in rounds:
        c = r["confidence"]
        assert len(c) == r["drafted"] and 0 <= r["accepted"] <= r["drafted"]
        assert all(x >= thr for x in c[:-1])        # every draft before the last was confident
        assert c[-1] < thr or r["drafted"] == 4     # the last one was not, or the cap ended the round
        # the confidence is the softmax probability of the greedy token: between 1/vocab and 1
        assert all(1.0 / TINY.vocab <= x <= 1.0 for x in c)


# ---------------- reachability pruning (result-neutral) ----------------

@pytest.mark.parametrize("M", [1, 2, 3, 5, 8])
def test_pruning_unreachable_states_changes_nothing_reachable(tiny, M):
    """States with j < M - (L - i) cannot lie on a path to (L, M).  Leaving them out must not change
    the skip set, any reachable score, margin, decision or state; the cells left out are exactly
    those, and the number of layer applications drops by the count of the pruned apply-cells."""
    model, toks, cache, am, hid, logits = tiny
    L = TINY.L
    p = 40
    x = hid[p][:, None, :]
    full = orc.dp_search(model, x, cache, p, p, M)
    pr = orc.dp_search(model, x, cache, p, p, M, prune=True)
    np.testing.assert_array_equal(pr["S"], full["S"])
    n_pruned_apply = 0
    for i in range(L + 1):
        for j in range(M + 1):
            exists = j <= min(i, M)
            reach = exists and j >= M - (L - i)
            if j == 0:
                assert pr["D"][i, 0] == 1.0          # column 0 is the given full-model state: always there
                continue
            if reach:
                assert pr["D"][i, j] == full["D"][i, j] and pr["choice"][i, j] == full["choice"][i, j]
                np.testing.assert_array_equal(pr["g"][i, j], full["g"][i, j])
                if not np.isnan(full["margin"][i, j]):
                    assert pr["margin"][i, j] == full["margin"][i, j]
            else:
                assert np.isnan(pr["D"][i, j]) and pr["choice"][i, j] == 255
                if exists and j <= i - 1:
                    n_pruned_apply += 1
    assert full["applied"] - pr["applied"] == n_pruned_apply
    # every cell the backtrack visits is reachable (so pruning can never be seen by it)
    i, j = L, M
    while i > 0 and j > 0:
        assert orc.reachable(i, j, L, M)
        if full["choice"][i, j] == orc.SKIP:
            j -= 1
        i -= 1


def test_reachability_by_brute_force():
    """reachable(i, j) against its definition: some sequence of L - i further steps, each keeping j
    or raising it by one (a skip), ends at M."""
    L, M = 7, 3
    for i in range(L + 1):
        for j in range(M + 1):
            if j > min(i, M):
                continue
            ends = {j}
            for _ in range(L - i):
                ends = ends | {e + 1 for e in ends}
            assert orc.reachable(i, j, L, M) == (M in ends), (i, j)
