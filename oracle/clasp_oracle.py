"""CPU oracle for the layer-skip search of CLaSp -- TEST INFRASTRUCTURE ONLY.

A plain, slow, float64 numpy statement of what the GPU library computes: the
LLaMA-style decoder layer, the dynamic programme of Algorithm 1 with its
backtrack, replay of a skip set, exhaustive search over skip sets, and the
greedy autoregressive / self-speculative decoding loops of Sec. 3.1.  It shares
no code with the CUDA path and must never be imported by the product package:
only the tests, the smoke check and the benchmark's CPU-baseline leg use it.

Everything is float64.  For a bf16 model the caller passes the bf16-rounded
weight VALUES converted to float64; nothing else is rounded here.

Conventions fixed where the paper is silent (each pinned by a test unless noted):
  * layers are f_0..f_{L-1};  h_0 = embedding,  h_{l+1} = f_l(h_l)   (Sec. 3.4)
  * x_L is the residual stream BEFORE the final RMSNorm
  * RoPE pairs element i with i + head_dim/2 ("rotate half"), inv_freq_i =
    theta^(-2i/head_dim), no frequency rescaling   (pinned against the
    `transformers` LLaMA implementation)
  * a DP state attends to the verified cache positions [0, C) plus its own
    freshly computed keys/values, causally among its T rows; states never see
    each other and the cache is never written by the search (Sec. 3.6)
  * cosine(a, b) = a.b / (max(|a|, 1e-12) * max(|b|, 1e-12))
  * T > 1 objective positions: the score of a state is the arithmetic mean of
    the T per-position cosines.  PARITY UNPINNED by the paper for T > 1 (the
    paper uses the single last accepted token); pinned only by its T = 1
    reduction.
  * a strict '>' decides for "apply the layer"; an exact tie keeps the skip
    candidate (Algorithm 1, the if/else on sigma)
  * the search after the prompt's prefill (first draft round) uses the last
    prompt token as objective.  PARITY UNPINNED by the paper (it does not say
    where the first skip set comes from); it cannot affect losslessness.
  * lower optimisation frequency (Sec. 3.7, Sec. 5.3.2): with interval N the
    search runs after every N-th verification; the rounds in between keep the
    last skip set.
  * draft-exiting threshold (Sec. 5.3.3): the confidence of a drafted token is
    the draft model's softmax probability of that (greedy) token; a token whose
    confidence is below the threshold is still handed to the verification (it
    has been computed) but ends the drafting of that round.  The paper names
    the mechanism and its best value (about 0.7) only; this reading is pinned by
    its two limits (threshold 0 = fixed draft length, threshold > 1 = one draft
    per round) and by losslessness.
"""
from __future__ import annotations

import itertools
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import numpy as np

COS_EPS = 1e-12


# --------------------------------------------------------------------------
# decoder layer (LLaMA family named in Sec. 4; shapes from the configs)
# --------------------------------------------------------------------------

def rmsnorm(x: np.ndarray, w: np.ndarray, eps: float) -> np.ndarray:
    """y = x / sqrt(mean(x^2) + eps) * w, row-wise over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * w


def rope(x: np.ndarray, positions: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding of x[T, n_heads, head_dim] at absolute positions[T]."""
    hd = x.shape[-1]
    half = hd // 2
    inv_freq = theta ** (-np.arange(half, dtype=np.float64) * 2.0 / hd)
    ang = positions.astype(np.float64)[:, None] * inv_freq[None, :]      # [T, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def decoder_layer(X: np.ndarray, w: Dict[str, np.ndarray], cache_k: np.ndarray,
                  cache_v: np.ndarray, C: int, pos0: int, cfg) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """f_l(X) for the T rows X[T, d] sitting at positions pos0..pos0+T-1.

    Row t attends to cache_k/cache_v[0:C] (keys stored after RoPE) and to the
    rows 0..t of X itself.  Returns (out[T, d], k_new[T, n_kv, hd], v_new[...]);
    the cache arrays are not modified.
    """
    T, d = X.shape
    nq, nkv, hd = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    group = nq // nkv
    pos = pos0 + np.arange(T)

    a = rmsnorm(X, w["attn_norm"], cfg.rms_eps)
    q = (a @ w["wq"].T).reshape(T, nq, hd)
    k = (a @ w["wk"].T).reshape(T, nkv, hd)
    v = (a @ w["wv"].T).reshape(T, nkv, hd)
    q = rope(q, pos, cfg.rope_theta)
    k = rope(k, pos, cfg.rope_theta)

    attn = np.zeros((T, nq, hd))
    for t in range(T):
        keys = np.concatenate([cache_k[:C], k[:t + 1]], axis=0)          # [C+t+1, nkv, hd]
        vals = np.concatenate([cache_v[:C], v[:t + 1]], axis=0)
        for h in range(nq):
            kh = h // group
            s = keys[:, kh, :] @ q[t, h] / np.sqrt(hd)
            p = np.exp(s - s.max())
            p /= p.sum()
            attn[t, h] = p @ vals[:, kh, :]
    x1 = X + attn.reshape(T, nq * hd) @ w["wo"].T
    m = rmsnorm(x1, w["mlp_norm"], cfg.rms_eps)
    out = x1 + (silu(m @ w["w_gate"].T) * (m @ w["w_up"].T)) @ w["w_down"].T
    return out, k, v


# --------------------------------------------------------------------------
# model container and full forward (the verify model of Sec. 3.1)
# --------------------------------------------------------------------------

class Model:
    """Weights as float64 arrays; `layer_fn(l)` may build them lazily."""

    def __init__(self, cfg, layer_fn: Callable[[int], Dict[str, np.ndarray]],
                 head: Optional[Dict[str, np.ndarray]] = None):
        self.cfg = cfg
        self.layer = layer_fn
        self.head = head


class KVCache:
    def __init__(self, cfg, max_ctx: int):
        shape = (cfg.L, max_ctx, cfg.n_kv_heads, cfg.head_dim)
        self.k = np.zeros(shape)
        self.v = np.zeros(shape)


def forward_hidden(model: Model, h0: np.ndarray, cache: KVCache, pos0: int,
                   skip: Optional[Sequence[int]] = None, write_cache: bool = True) -> np.ndarray:
    """Run rows h0[n, d] at positions pos0.. through the layers not in `skip`.

    Returns hidden[n, L+1, d] with hidden[:, l] the residual stream entering
    layer l (hidden[:, L] = output of the last layer, before the final norm).
    Layers that run write their K/V at pos0..pos0+n-1; skipped layers pass the
    state through and write nothing.
    """
    cfg = model.cfg
    n, d = h0.shape
    hidden = np.zeros((n, cfg.L + 1, d))
    hidden[:, 0] = h0
    x = h0
    for l in range(cfg.L):
        if skip is not None and skip[l]:
            hidden[:, l + 1] = x
            continue
        x, k, v = decoder_layer(x, model.layer(l), cache.k[l], cache.v[l], pos0, pos0, cfg)
        if write_cache:
            cache.k[l, pos0:pos0 + n] = k
            cache.v[l, pos0:pos0 + n] = v
        hidden[:, l + 1] = x
    return hidden


def logits_from_hidden(model: Model, x_top: np.ndarray) -> np.ndarray:
    h = rmsnorm(x_top, model.head["final_norm"], model.cfg.rms_eps)
    return h @ model.head["lm_head"].T


def argmax_lowest(logits: np.ndarray) -> np.ndarray:
    """Row-wise argmax; ties go to the lowest index (np.argmax does that)."""
    return np.argmax(logits, axis=-1)


def top1_probability(logits: np.ndarray) -> np.ndarray:
    """Softmax probability of the greedy token of each row of logits[n, vocab]."""
    z = logits - logits.max(axis=-1, keepdims=True)
    return 1.0 / np.exp(z).sum(axis=-1)


def verify_forward(model: Model, tokens: Sequence[int], cache: KVCache, pos0: int,
                   skip: Optional[Sequence[int]] = None):
    """Embed tokens, run the (possibly layer-skipped) model, return
    (argmax[n], hidden[n, L+1, d], logits[n, vocab])."""
    h0 = model.head["embed"][np.asarray(tokens, dtype=np.int64)]
    hidden = forward_hidden(model, h0, cache, pos0, skip)
    logits = logits_from_hidden(model, hidden[:, model.cfg.L])
    return argmax_lowest(logits), hidden, logits


# --------------------------------------------------------------------------
# the dynamic programme (Eq. 2, Algorithm 1)
# --------------------------------------------------------------------------

def cosine_score(x: np.ndarray, y: np.ndarray) -> float:
    """Mean over the T rows of cosine(x[t], y[t]);  x, y: [T, d]."""
    num = np.sum(x * y, axis=-1)
    den = np.maximum(np.linalg.norm(x, axis=-1), COS_EPS) * np.maximum(np.linalg.norm(y, axis=-1), COS_EPS)
    return float(np.mean(num / den))


APPLY, SKIP = 0, 1


def reachable(i: int, j: int, L: int, M: int) -> bool:
    """Can the backtrack from (L, M) pass through cell (i, j)?  Each remaining step removes at most
    one skip, so it needs j >= M - (L - i) (and j <= min(i, M) for the cell to exist)."""
    return M - (L - i) <= j <= min(i, M)


def dp_search(model: Model, x: np.ndarray, cache: KVCache, C: int, pos0: int, M: int,
              forced_choice: Optional[np.ndarray] = None, prune: bool = False):
    """Algorithm 1.  x[L+1, T, d] are the full model's states of the T objective
    rows; the search reads cache positions [0, C) and never writes the cache.

    Returns a dict with
      g      [L+1, M+1, T, d]  best state after i layers with j skipped (NaN where j > i)
      D      [L+1, M+1]        its score (Eq. 2);  NaN where j > i
      margin [L+1, M+1]        score(apply) - score(skip) where both exist, else NaN
      choice [L+1, M+1] uint8  SKIP (1) / APPLY (0) taken at (i, j); 255 where undefined
      S      [L] uint8         backtracked skip set, 1 = skipped
    prune=True leaves out the states from which (L, M) cannot be reached (the paper's Algorithm 1
    computes them; they can never influence S): their cells stay NaN / 255 and `applied` counts the
    decoder-layer applications that were made.
    """
    cfg = model.cfg
    L = cfg.L
    Lp1, T, d = x.shape
    assert Lp1 == L + 1 and 0 <= M <= L
    g = np.full((L + 1, M + 1, T, d), np.nan)
    D = np.full((L + 1, M + 1), np.nan)
    margin = np.full((L + 1, M + 1), np.nan)
    choice = np.full((L + 1, M + 1), 255, dtype=np.uint8)
    g[0, 0] = x[0]
    D[0, 0] = 1.0
    applied = 0
    for i in range(1, L + 1):
        g[i, 0] = x[i]                      # column 0: nothing skipped = the full model
        D[i, 0] = 1.0
        choice[i, 0] = APPLY
        ell = min(i - 1, M)
        w = model.layer(i - 1) if ell > 0 else None
        for j in range(1, ell + 1):
            if prune and not reachable(i, j, L, M):
                continue
            G, _, _ = decoder_layer(g[i - 1, j], w, cache.k[i - 1], cache.v[i - 1], C, pos0, cfg)
            applied += 1
            s_app = cosine_score(x[i], G)
            s_skip = cosine_score(x[i], g[i - 1, j - 1])
            margin[i, j] = s_app - s_skip
            take_apply = s_app > s_skip
            if forced_choice is not None and forced_choice[i, j] != 255:
                take_apply = forced_choice[i, j] == APPLY
            if take_apply:
                g[i, j], D[i, j], choice[i, j] = G, s_app, APPLY
            else:
                g[i, j], D[i, j], choice[i, j] = g[i - 1, j - 1], s_skip, SKIP
        if i <= M and not (prune and not reachable(i, i, L, M)):   # diagonal: the first i layers all skipped
            g[i, i] = g[i - 1, i - 1]
            D[i, i] = cosine_score(x[i], g[i, i])
            choice[i, i] = SKIP
    return {"g": g, "D": D, "margin": margin, "choice": choice, "S": backtrack(choice, L, M), "applied": applied}


def backtrack(choice: np.ndarray, L: int, M: int) -> np.ndarray:
    """Walk from (L, M) down; a SKIP at (i, j) marks layer i-1 and moves to
    (i-1, j-1), an APPLY moves to (i-1, j).  Stops when no skips remain: all
    lower layers are kept."""
    S = np.zeros(L, dtype=np.uint8)
    i, j = L, M
    while i > 0 and j > 0:
        if choice[i, j] == SKIP:
            S[i - 1] = 1
            j -= 1
        i -= 1
    return S


def replay(model: Model, x0: np.ndarray, S: Sequence[int], cache: KVCache, C: int, pos0: int) -> np.ndarray:
    """Push x0[T, d] through the layers not in S, reading cache [0, C) only."""
    r = x0
    for l in range(model.cfg.L):
        if not S[l]:
            r, _, _ = decoder_layer(r, model.layer(l), cache.k[l], cache.v[l], C, pos0, model.cfg)
    return r


def brute_force(model: Model, x: np.ndarray, cache: KVCache, C: int, pos0: int, M: int):
    """Score every skip set of size M: list of (score, S) sorted best first."""
    L = model.cfg.L
    out = []
    for comb in itertools.combinations(range(L), M):
        S = np.zeros(L, dtype=np.uint8)
        S[list(comb)] = 1
        r = replay(model, x[0], S, cache, C, pos0)
        out.append((cosine_score(x[L], r), S))
    out.sort(key=lambda e: -e[0])
    return out


# --------------------------------------------------------------------------
# decoding loops (Sec. 3.1: draft, verify, layer optimisation)
# --------------------------------------------------------------------------

def greedy_autoregressive(model: Model, prompt: Sequence[int], n_new: int, max_ctx: int) -> List[int]:
    cache = KVCache(model.cfg, max_ctx)
    am, _, _ = verify_forward(model, prompt, cache, 0)
    out = [int(am[-1])]
    pos = len(prompt)
    while len(out) < n_new:
        am, _, _ = verify_forward(model, [out[-1]], cache, pos)
        out.append(int(am[0]))
        pos += 1
    return out


def greedy_self_speculative(model: Model, prompt: Sequence[int], n_new: int, max_ctx: int,
                            M: int, K: int, fixed_mask: Optional[Sequence[int]] = None,
                            dp_interval: int = 1, exit_threshold: float = 0.0):
    """Draft up to K tokens with the layer-skipped model, verify them with the
    full model in one pass, accept the longest matching prefix plus the full
    model's own next token, then re-run the layer search on the last accepted
    token (after every dp_interval-th verification, Sec. 3.7).  A drafted token
    whose softmax probability is below exit_threshold ends the round's drafting
    (Sec. 5.3.3); it is still verified.

    Returns (tokens, stats) where stats lists per round the accepted count, the
    skip set used, the number of drafted tokens and their confidences.
    """
    cfg = model.cfg
    cache = KVCache(cfg, max_ctx)
    P = len(prompt)
    am, hidden, _ = verify_forward(model, prompt, cache, 0)
    out = [int(am[-1])]
    pending = out[0]              # committed token whose K/V is not in the cache yet
    n_valid = P                   # cache positions [0, n_valid) hold full-model K/V

    def search(hid_row, obj_pos):
        if fixed_mask is not None:
            return np.asarray(fixed_mask, dtype=np.uint8)
        xs = hid_row[:, None, :]                                   # [L+1, 1, d]
        return dp_search(model, xs, cache, obj_pos, obj_pos, M)["S"]

    S = search(hidden[P - 1], P - 1)
    rounds = []
    n_verify = 0
    while len(out) < n_new:
        # draft: K single-token passes of the layer-skipped model
        drafts, conf, tok = [], [], pending
        for k in range(K):
            a, _, lg = verify_forward(model, [tok], cache, n_valid + k, skip=S)
            tok = int(a[0])
            drafts.append(tok)
            conf.append(float(top1_probability(lg)[0]))
            if conf[-1] < exit_threshold:
                break
        n_d = len(drafts)
        # verify: one full-model pass over [pending, d_1..d_n]
        am, hidden, _ = verify_forward(model, [pending] + drafts, cache, n_valid)
        a = 0
        while a < n_d and drafts[a] == int(am[a]):
            a += 1
        new = drafts[:a] + [int(am[a])]
        out.extend(new)
        rounds.append({"accepted": a, "S": S.copy(), "drafted": n_d, "confidence": conf})
        obj_row = hidden[a]                        # last position whose K/V is now valid
        obj_pos = n_valid + a
        n_valid += a + 1
        pending = new[-1]
        n_verify += 1
        if n_verify % dp_interval == 0:
            S = search(obj_row, obj_pos)
    return out[:n_new], rounds


# --------------------------------------------------------------------------
# non-greedy decoding: speculative sampling (Sec. 4, Table 1 "Temperature = 1";
# the accept / resample rule is the one of Leviathan et al. 2023, which the
# paper cites for losslessness)
# --------------------------------------------------------------------------
# Random numbers come from one counter-based generator, Philox4x32-10 (Salmon
# et al., "Parallel random numbers: as easy as 1, 2, 3", SC'11), keyed by the
# seed and counted by (index, position, purpose, round), so that every draw is
# a pure function of where it is used.  The CUDA side implements the same
# published definition on its own.

PHILOX_M0, PHILOX_M1 = 0xD2511F53, 0xCD9E8D57
PHILOX_W0, PHILOX_W1 = 0x9E3779B9, 0xBB67AE85
DRAW_DRAFT, DRAW_ACCEPT, DRAW_RESIDUAL, DRAW_TARGET = 0, 1, 2, 3


def philox4x32_10(c0, c1, c2, c3, k0: int, k1: int):
    """Ten rounds of Philox-4x32 on uint32 arrays c0..c3 (broadcast together) with key (k0, k1)."""
    c0, c1, c2, c3 = np.broadcast_arrays(*[np.asarray(c, dtype=np.uint64) for c in (c0, c1, c2, c3)])
    mask = np.uint64(0xFFFFFFFF)
    for r in range(10):
        p0 = np.uint64(PHILOX_M0) * c0                      # 64-bit products of 32-bit factors
        p1 = np.uint64(PHILOX_M1) * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & mask
        hi1, lo1 = p1 >> np.uint64(32), p1 & mask
        c0, c1, c2, c3 = hi1 ^ c1 ^ np.uint64(k0), lo1, hi0 ^ c3 ^ np.uint64(k1), lo0
        k0 = (k0 + PHILOX_W0) & 0xFFFFFFFF
        k1 = (k1 + PHILOX_W1) & 0xFFFFFFFF
    return [c.astype(np.uint32) for c in (c0, c1, c2, c3)]


def uniform_draws(seed: int, index, position: int, purpose: int, rnd: int) -> np.ndarray:
    """Uniforms in (0, 1) on a 2^-24 grid (exact in float and double): ((x >> 8) + 0.5) / 2^24 of
    the first Philox word for counter (index, position, purpose, round) and key = the 64-bit seed."""
    x = philox4x32_10(index, position, purpose, rnd, seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)[0]
    return ((x >> np.uint32(8)).astype(np.float64) + 0.5) * (1.0 / 16777216.0)


def gumbel_max_sample(logits: np.ndarray, temperature: float, seed: int, position: int, purpose: int,
                      rnd: int) -> int:
    """A sample of softmax(logits / temperature): argmax of logits / temperature + Gumbel noise
    (noise of entry v from draw v); entries at -inf can never win; lowest index on exact ties."""
    u = uniform_draws(seed, np.arange(logits.shape[0]), position, purpose, rnd)
    return int(np.argmax(logits / temperature - np.log(-np.log(u))))


def log_softmax(z: np.ndarray) -> np.ndarray:
    z = z - z.max()
    return z - np.log(np.exp(z).sum())


def speculative_accept(p_logits: np.ndarray, q_logits: np.ndarray, drafts: Sequence[int], temperature: float,
                       seed: int, pos0: int, rnd: int):
    """The accept / resample rule.  drafts[k] was sampled from q_k = softmax(q_logits[k] / T) and
    would sit at position pos0 + k; p_k = softmax(p_logits[k] / T) is the full model's distribution
    there (p_logits has one more row: the position after the last draft).  Draft k is accepted with
    probability min(1, p_k(x) / q_k(x)); the first rejected position gets a sample of
    norm(max(0, p_k - q_k)) instead and ends the round; if every draft is accepted the next position
    gets a sample of p_K.  Returns (accepted, committed tokens) -- accepted + 1 tokens."""
    K = len(drafts)
    out = []
    for k in range(K):
        lp, lq = log_softmax(p_logits[k] / temperature), log_softmax(q_logits[k] / temperature)
        x = int(drafts[k])
        u = float(uniform_draws(seed, 0, pos0 + k, DRAW_ACCEPT, rnd))
        if u < np.exp(min(0.0, lp[x] - lq[x])):
            out.append(x)
            continue
        resid = np.maximum(np.exp(lp) - np.exp(lq), 0.0)
        with np.errstate(divide="ignore"):
            lr = np.log(resid)                              # -inf where p <= q
        out.append(gumbel_max_sample(lr, 1.0, seed, pos0 + k, DRAW_RESIDUAL, rnd))
        return k, out
    out.append(gumbel_max_sample(p_logits[K], temperature, seed, pos0 + K, DRAW_TARGET, rnd))
    return K, out


def sampling_autoregressive(model: Model, prompt: Sequence[int], n_new: int, max_ctx: int, temperature: float,
                            seed: int) -> List[int]:
    """Plain ancestral sampling of the full model (the distribution speculative sampling preserves)."""
    cache = KVCache(model.cfg, max_ctx)
    _, _, lg = verify_forward(model, prompt, cache, 0)
    pos = len(prompt)
    out = [gumbel_max_sample(lg[-1], temperature, seed, pos, DRAW_TARGET, 0)]
    while len(out) < n_new:
        _, _, lg = verify_forward(model, [out[-1]], cache, pos)
        pos += 1
        out.append(gumbel_max_sample(lg[0], temperature, seed, pos, DRAW_TARGET, 0))
    return out


def sampling_self_speculative(model: Model, prompt: Sequence[int], n_new: int, max_ctx: int, M: int, K: int,
                              temperature: float, seed: int, fixed_mask: Optional[Sequence[int]] = None,
                              dp_interval: int = 1):
    """The three-stage loop of Sec. 3.1 with sampling instead of arg-max: drafts are samples of the
    layer-skipped model, the verification applies the accept / resample rule, the layer search runs on
    the last accepted position as in the greedy loop.  Returns (tokens, per-round stats)."""
    cfg = model.cfg
    cache = KVCache(cfg, max_ctx)
    P = len(prompt)
    _, hidden, lg = verify_forward(model, prompt, cache, 0)
    out = [gumbel_max_sample(lg[-1], temperature, seed, P, DRAW_TARGET, 0)]
    pending, n_valid = out[0], P

    def search(hid_row, obj_pos):
        if fixed_mask is not None:
            return np.asarray(fixed_mask, dtype=np.uint8)
        return dp_search(model, hid_row[:, None, :], cache, obj_pos, obj_pos, M)["S"]

    S = search(hidden[P - 1], P - 1)
    rounds = []
    rnd = 0
    while len(out) < n_new:
        rnd += 1
        drafts, q_rows, tok = [], [], pending
        for k in range(K):
            _, _, lq = verify_forward(model, [tok], cache, n_valid + k, skip=S)
            # draft k is the token that would sit at position n_valid + k + 1
            tok = gumbel_max_sample(lq[0], temperature, seed, n_valid + k + 1, DRAW_DRAFT, rnd)
            drafts.append(tok)
            q_rows.append(lq[0])
        _, hidden, lp = verify_forward(model, [pending] + drafts, cache, n_valid)
        a, new = speculative_accept(lp, np.stack(q_rows), drafts, temperature, seed, n_valid + 1, rnd)
        out.extend(new)
        rounds.append({"accepted": a, "S": S.copy(), "drafts": drafts, "committed": new})
        obj_row, obj_pos = hidden[a], n_valid + a
        n_valid += a + 1
        pending = new[-1]
        if rnd % dp_interval == 0:
            S = search(obj_row, obj_pos)
    return out[:n_new], rounds
