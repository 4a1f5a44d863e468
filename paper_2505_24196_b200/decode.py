"""Host-side driver of the three-stage loop (draft, verify, layer optimisation; Sec. 3.1).

Control flow and argument marshalling only: every forward pass, the search and the
acceptance rule run inside libclasp.so.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import torch

from .binding import Clasp, KVCache


class SelfSpeculativeDecoder:
    """Greedy self-speculative decoding with the skip set re-optimised after verification.

    M: layers the draft model skips; K: most drafts per round; dp_interval: run the layer
    search every that many verifications (1 = after each, the paper's default
    before its lower-frequency optimisation of Sec. 3.7); exit_threshold: a drafted token
    whose softmax probability (returned by the draft call) is below it ends the round's
    drafting (Sec. 5.3.3; 0 = always draft K tokens).  The comparison is the only step taken
    here, on one float per draft read back from the device.
    """

    def __init__(self, engine: Clasp, kv: KVCache, M: int, K: int, dp_interval: int = 1, T: int = 1,
                 time_stages: bool = False, exit_threshold: float = 0.0):
        self.e, self.kv, self.M, self.K, self.T = engine, kv, M, K, T
        self.dp_interval = dp_interval
        self.exit_threshold = float(exit_threshold)
        self.time_stages = time_stages
        dev = engine.device
        L, d = engine.cfg.L, engine.cfg.d_model
        self.draft_tok = torch.zeros(K + 1, dtype=torch.int32, device=dev)   # [pending, d_1..d_K]
        self.argmax = torch.zeros(K + 1, dtype=torch.int32, device=dev)
        self.hidden = torch.empty((K + 1, L + 1, d), dtype=torch.float32, device=dev)
        self.pinned_in = torch.zeros(K + 1, dtype=torch.int32).pin_memory()
        self.pinned_out = torch.zeros(2 * (K + 1), dtype=torch.int32).pin_memory()
        self.conf = torch.zeros(K, dtype=torch.float32, device=dev)          # confidence of d_1..d_K
        self.pinned_conf = torch.zeros(K, dtype=torch.float32).pin_memory()
        self.mask_host = bytes(L)
        self.stage_ms = {"dp": 0.0, "draft": 0.0, "verify": 0.0}
        self.rounds: List[Dict] = []
        self.n_valid = 0
        self.pending: Optional[int] = None

    # ---- helpers
    def _timed(self, name, fn):
        if not self.time_stages:
            return fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(self.e.stream)
        out = fn()
        b.record(self.e.stream)
        b.synchronize()
        self.stage_ms[name] += a.elapsed_time(b)
        return out

    def _search(self, hidden_row: torch.Tensor, obj_pos: int):
        """hidden_row: view [L+1, d] of the objective token's states (T = 1)."""
        if self.M == 0:
            self.mask_host = bytes(self.e.cfg.L)
            return
        d = self.e.cfg.d_model
        r = self.e.dp_search(hidden_row, d, 0, self.kv, obj_pos, obj_pos, 1, self.M,
                             want_margins=False, want_g=False)
        self.mask_host = bytes(r["S"].cpu().tolist())
        self.last_search = r

    def prefill(self, prompt: Sequence[int]) -> int:
        """Full-model pass over the prompt (in chunks of max_rows); returns the first new token
        and runs the first layer search on the last prompt token."""
        e = self.e
        toks = torch.as_tensor(list(prompt), dtype=torch.int32).to(e.device)
        P, step = toks.numel(), e.cfg.max_rows
        am = hid = None
        for s in range(0, P, step):
            chunk = toks[s:s + step]
            last = s + step >= P
            am, hid = e.verify(chunk, s, self.kv, 1 if last else 0, want_hidden=last)
        first = int(am.cpu()[0])
        self.n_valid, self.pending = P, first
        self._timed("dp", lambda: self._search(hid[-1], P - 1))
        return first

    def round(self) -> List[int]:
        """One draft / verify / layer-optimisation round; returns the committed tokens."""
        e, K = self.e, self.K
        self.pinned_in[0] = self.pending
        self.draft_tok[:1].copy_(self.pinned_in[:1], non_blocking=True)

        thr = self.exit_threshold
        conf: List[float] = []

        def draft():
            for k in range(K):
                e.draft_forward(self.mask_host, self.draft_tok[k:k + 1], self.n_valid + k, self.kv,
                                self.draft_tok[k + 1:k + 2], self.conf[k:k + 1] if thr > 0.0 else None)
                if thr > 0.0:
                    self.pinned_conf[k:k + 1].copy_(self.conf[k:k + 1], non_blocking=True)
                    e.stream.synchronize()
                    conf.append(float(self.pinned_conf[k]))
                    if conf[-1] < thr:
                        return k + 1
            return K
        n_d = self._timed("draft", draft)
        self._timed("verify", lambda: e.verify(self.draft_tok[:n_d + 1], self.n_valid, self.kv, n_d + 1,
                                               hidden_out=self.hidden, argmax_out=self.argmax))
        self.pinned_out[:K + 1].copy_(self.draft_tok, non_blocking=True)
        self.pinned_out[K + 1:].copy_(self.argmax, non_blocking=True)
        e.stream.synchronize()
        host = self.pinned_out.tolist()
        a, committed = e.accept(host[1:n_d + 1], host[K + 1:K + 2 + n_d])
        obj_pos = self.n_valid + a
        self.n_valid += a + 1
        self.pending = committed[-1]
        self.rounds.append({"accepted": a, "S": self.mask_host, "drafted": n_d, "confidence": conf})
        if len(self.rounds) % self.dp_interval == 0:
            self._timed("dp", lambda: self._search(self.hidden[a], obj_pos))
        return committed

    def generate(self, prompt: Sequence[int], n_new: int) -> List[int]:
        out = [self.prefill(prompt)]
        while len(out) < n_new:
            out.extend(self.round())
        return out[:n_new]


def greedy_autoregressive(engine: Clasp, kv: KVCache, prompt: Sequence[int], n_new: int) -> List[int]:
    """Plain greedy decoding of the full model, one token per pass (the lossless reference
    the self-speculative output must equal)."""
    toks = torch.as_tensor(list(prompt), dtype=torch.int32).to(engine.device)
    P, step = toks.numel(), engine.cfg.max_rows
    am = None
    for s in range(0, P, step):
        last = s + step >= P
        am, _ = engine.verify(toks[s:s + step], s, kv, 1 if last else 0, want_hidden=False)
    cur = am.clone()
    out = [int(cur.cpu()[0])]
    pos = P
    nxt = torch.empty(1, dtype=torch.int32, device=engine.device)
    while len(out) < n_new:
        engine.verify(cur, pos, kv, 1, want_hidden=False, argmax_out=nxt)
        cur, nxt = nxt, cur
        out.append(int(cur.cpu()[0]))
        pos += 1
    return out


class SpeculativeSampler:
    """Non-greedy self-speculative decoding (Table 1, temperature 1): drafts are draws of the
    layer-skipped model, the verification accepts or replaces them by the rule of speculative
    sampling (inside the library), the layer search runs on the last accepted position as in the
    greedy loop.  Control flow only; all arithmetic and every random draw happen in libclasp.so."""

    def __init__(self, engine: Clasp, kv: KVCache, M: int, K: int, temperature: float, seed: int, dp_interval: int = 1,
                 fixed_mask: Optional[bytes] = None):
        self.e, self.kv, self.M, self.K = engine, kv, M, K
        self.temperature, self.seed, self.dp_interval, self.fixed_mask = float(temperature), int(seed), dp_interval, fixed_mask
        dev = engine.device
        L, d, V = engine.cfg.L, engine.cfg.d_model, engine.cfg.vocab
        self.tok = torch.zeros(K + 1, dtype=torch.int32, device=dev)        # [pending, d_1..d_K]
        self.q_logits = torch.empty((K, V), dtype=torch.float32, device=dev)
        self.p_logits = torch.empty((K + 1, V), dtype=torch.float32, device=dev)
        self.n_acc = torch.zeros(1, dtype=torch.int32, device=dev)
        self.committed = torch.zeros(K + 1, dtype=torch.int32, device=dev)
        self.hidden = torch.empty((K + 1, L + 1, d), dtype=torch.float32, device=dev)
        self.mask_host = bytes(L) if fixed_mask is None else bytes(fixed_mask)
        self.rounds: List[Dict] = []
        self.n_valid, self.pending, self.rnd = 0, None, 0

    def _search(self, hidden_row: torch.Tensor, obj_pos: int):
        if self.fixed_mask is not None or self.M == 0:
            return
        r = self.e.dp_search(hidden_row, self.e.cfg.d_model, 0, self.kv, obj_pos, obj_pos, 1, self.M,
                             want_margins=False, want_g=False)
        self.mask_host = bytes(r["S"].cpu().tolist())

    def prefill(self, prompt: Sequence[int]) -> int:
        e = self.e
        toks = torch.as_tensor(list(prompt), dtype=torch.int32).to(e.device)
        P, step = toks.numel(), e.cfg.max_rows
        hid = None
        for s in range(0, P, step):
            chunk = toks[s:s + step]
            if s + step >= P:
                hid = torch.empty((chunk.numel(), e.cfg.L + 1, e.cfg.d_model), dtype=torch.float32, device=e.device)
                e.verify_sample(chunk, s, self.kv, 0, None, self.temperature, self.seed, 0, self.p_logits, self.n_acc,
                                self.committed, hid)
            else:
                e.verify(chunk, s, self.kv, 0, want_hidden=False)
        first = int(self.committed.cpu()[0])
        self.n_valid, self.pending = P, first
        self._search(hid[-1], P - 1)
        return first

    def round(self) -> List[int]:
        e, K = self.e, self.K
        self.rnd += 1
        self.tok[:1] = self.pending
        for k in range(K):
            e.draft_sample(self.mask_host, self.tok[k:k + 1], self.n_valid + k, self.kv, self.temperature, self.seed,
                           self.rnd, self.tok[k + 1:k + 2], self.q_logits[k])
        e.verify_sample(self.tok, self.n_valid, self.kv, K, self.q_logits, self.temperature, self.seed, self.rnd,
                        self.p_logits, self.n_acc, self.committed, self.hidden)
        a = int(self.n_acc.cpu()[0])
        new = self.committed[:a + 1].cpu().tolist()
        self.rounds.append({"accepted": a, "S": self.mask_host, "drafts": self.tok[1:].cpu().tolist(), "committed": new})
        obj_pos = self.n_valid + a
        self.n_valid += a + 1
        self.pending = new[-1]
        if self.rnd % self.dp_interval == 0:
            self._search(self.hidden[a], obj_pos)
        return new

    def generate(self, prompt: Sequence[int], n_new: int) -> List[int]:
        out = [self.prefill(prompt)]
        while len(out) < n_new:
            out.extend(self.round())
        return out[:n_new]
