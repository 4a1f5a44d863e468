"""Thin ctypes binding of libclasp.so: argument marshalling only.

PyTorch is used for device memory and the stream; every arithmetic step runs in
the library's CUDA kernels.  There is no CPU fallback: importing works without a
GPU (so that the exported symbols can be checked), but creating a context
without the library or without a CUDA device raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import torch

from . import build as _build

CLASP_FP32, CLASP_BF16 = 0, 1
CHOICE_APPLY, CHOICE_SKIP, CHOICE_NONE = 0, 1, 255
FLAG_FORCE_SIMT, FLAG_NO_DEFER, FLAG_MULTI_KERNEL, FLAG_PRUNE, FLAG_NO_ATT_TC = 1, 2, 4, 8, 16

SYMBOLS = ["clasp_workspace_bytes", "clasp_create", "clasp_destroy", "clasp_load_layers", "clasp_load_head",
           "clasp_dp_search", "clasp_verify", "clasp_draft_forward", "clasp_accept", "clasp_layer_forward",
           "clasp_gemm_xwT", "clasp_gemm_xwT_noalloc", "clasp_profile_gemm", "clasp_last_device_status", "clasp_launch_count", "clasp_engine_trace", "clasp_strerror",
           "clasp_engine_active", "clasp_set_wait_limit", "clasp_draft_sample", "clasp_verify_sample"]


class ClaspConfig(C.Structure):
    _fields_ = [("L", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("d_ffn", C.c_int32), ("vocab", C.c_int32), ("dtype", C.c_int32),
                ("rms_eps", C.c_float), ("rope_theta", C.c_float), ("max_ctx", C.c_int32),
                ("max_rows", C.c_int32), ("max_M", C.c_int32), ("max_T", C.c_int32),
                ("max_head_rows", C.c_int32), ("flags", C.c_int32)]


class ClaspLayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down")]


class ClaspKvLayer(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p)]


class ClaspError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {strerror(code)} ({code})")
        self.code = code


_lib = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """Load libclasp.so (building it with nvcc first when it is missing or stale)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    if path is None:
        path = _build.LIB
        if not os.path.exists(path) or _build.is_stale():
            path = _build.build()
    lib = C.CDLL(path)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    lib.clasp_workspace_bytes.restype = C.c_size_t
    lib.clasp_workspace_bytes.argtypes = [C.POINTER(ClaspConfig)]
    lib.clasp_create.restype = C.c_int
    lib.clasp_create.argtypes = [C.POINTER(ClaspConfig), vp, C.c_size_t, vp, C.POINTER(vp)]
    lib.clasp_destroy.restype = None
    lib.clasp_destroy.argtypes = [vp]
    lib.clasp_load_layers.restype = C.c_int
    lib.clasp_load_layers.argtypes = [vp, i32, i32, C.POINTER(ClaspLayerWeights)]
    lib.clasp_load_head.restype = C.c_int
    lib.clasp_load_head.argtypes = [vp, vp, vp, vp]
    lib.clasp_dp_search.restype = C.c_int
    lib.clasp_dp_search.argtypes = [vp, vp, i64, i64, C.POINTER(ClaspKvLayer), i32, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.clasp_verify.restype = C.c_int
    lib.clasp_verify.argtypes = [vp, vp, i32, i32, C.POINTER(ClaspKvLayer), i32, vp, vp]
    lib.clasp_draft_forward.restype = C.c_int
    lib.clasp_draft_forward.argtypes = [vp, C.c_char_p, vp, i32, C.POINTER(ClaspKvLayer), vp, vp]
    lib.clasp_draft_sample.restype = C.c_int
    lib.clasp_draft_sample.argtypes = [vp, C.c_char_p, vp, i32, C.POINTER(ClaspKvLayer), C.c_float, C.c_uint64, i32, vp, vp]
    lib.clasp_verify_sample.restype = C.c_int
    lib.clasp_verify_sample.argtypes = [vp, vp, i32, i32, C.POINTER(ClaspKvLayer), i32, vp, C.c_float, C.c_uint64, i32,
                                        vp, vp, vp, vp]
    lib.clasp_accept.restype = C.c_int
    lib.clasp_accept.argtypes = [C.POINTER(i32), C.POINTER(i32), i32, C.POINTER(i32), C.POINTER(i32)]
    lib.clasp_layer_forward.restype = C.c_int
    lib.clasp_layer_forward.argtypes = [vp, i32, vp, i64, i32, i32, i32, i32, C.POINTER(ClaspKvLayer), i32, vp, i64]
    lib.clasp_gemm_xwT.restype = C.c_int
    lib.clasp_gemm_xwT.argtypes = [vp, vp, vp, i32, i32, i32, vp]
    lib.clasp_gemm_xwT_noalloc.restype = C.c_int
    lib.clasp_gemm_xwT_noalloc.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp]
    lib.clasp_profile_gemm.restype = C.c_int
    lib.clasp_profile_gemm.argtypes = [vp, i32, C.POINTER(i64), C.POINTER(C.c_double), C.POINTER(C.c_double)]
    lib.clasp_last_device_status.restype = C.c_int
    lib.clasp_last_device_status.argtypes = [vp]
    lib.clasp_launch_count.restype = C.c_int64
    lib.clasp_launch_count.argtypes = [vp]
    lib.clasp_engine_trace.restype = C.c_int
    lib.clasp_engine_trace.argtypes = [vp, vp, i32, C.POINTER(i32)]
    lib.clasp_engine_active.restype = C.c_int
    lib.clasp_engine_active.argtypes = [vp]
    lib.clasp_set_wait_limit.restype = C.c_int
    lib.clasp_set_wait_limit.argtypes = [vp, C.c_uint32]
    lib.clasp_strerror.restype = C.c_char_p
    lib.clasp_strerror.argtypes = [C.c_int]
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load_library().clasp_strerror(code).decode()


def _check(code: int, what: str):
    if code != 0:
        raise ClaspError(code, what)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def gemm_xwT_noalloc(x: torch.Tensor, w: torch.Tensor, y: torch.Tensor,
                     status_out: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """y = x w^T (bf16 in, float out) through the allocation-free entry point: no context,
    no workspace; the library's built-in scratch array is used.  The caller owns x, w, y."""
    R, K = x.shape
    N = w.shape[0]
    assert x.dtype == torch.bfloat16 and w.dtype == torch.bfloat16 and y.dtype == torch.float32
    assert x.is_contiguous() and w.is_contiguous() and y.is_contiguous() and y.shape == (R, N)
    st = stream if stream is not None else torch.cuda.current_stream(x.device)
    with torch.cuda.device(x.device):
        _check(load_library().clasp_gemm_xwT_noalloc(x.data_ptr(), w.data_ptr(), R, N, K, y.data_ptr(),
                                                     st.cuda_stream, _ptr(status_out)), "clasp_gemm_xwT_noalloc")


def make_config(model_cfg, max_ctx: int, max_rows: int, max_M: int, max_T: int = 1,
                max_head_rows: int = 16, flags: int = 0) -> ClaspConfig:
    """ClaspConfig from a shape description with the field names of datagen.ModelConfig."""
    return ClaspConfig(L=model_cfg.L, d_model=model_cfg.d_model, n_q_heads=model_cfg.n_q_heads,
                       n_kv_heads=model_cfg.n_kv_heads, head_dim=model_cfg.head_dim, d_ffn=model_cfg.d_ffn,
                       vocab=model_cfg.vocab, dtype=CLASP_BF16 if model_cfg.dtype == "bf16" else CLASP_FP32,
                       rms_eps=model_cfg.rms_eps, rope_theta=model_cfg.rope_theta, max_ctx=max_ctx,
                       max_rows=max_rows, max_M=max_M, max_T=max_T, max_head_rows=max_head_rows, flags=flags)


class KVCache:
    """Device KV cache: per layer K and V of shape [max_ctx, n_kv_heads, head_dim]."""

    def __init__(self, cfg: ClaspConfig, device="cuda"):
        dt = torch.bfloat16 if cfg.dtype == CLASP_BF16 else torch.float32
        shape = (cfg.L, cfg.max_ctx, cfg.n_kv_heads, cfg.head_dim)
        self.k = torch.zeros(shape, dtype=dt, device=device)
        self.v = torch.zeros(shape, dtype=dt, device=device)
        self.array = (ClaspKvLayer * cfg.L)()
        for l in range(cfg.L):
            self.array[l].k = self.k[l].data_ptr()
            self.array[l].v = self.v[l].data_ptr()


class Clasp:
    """Owns a clasp_ctx, its workspace and references to the borrowed weights."""

    def __init__(self, cfg: ClaspConfig, device="cuda", stream: Optional[torch.cuda.Stream] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2505_24196_b200 needs a CUDA device: there is no CPU path")
        self.lib = load_library()
        self.cfg = cfg
        self.device = torch.device(device)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        nbytes = self.lib.clasp_workspace_bytes(C.byref(cfg))
        if nbytes == 0:
            raise ClaspError(-2, "clasp_workspace_bytes")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        handle = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(self.lib.clasp_create(C.byref(cfg), self.workspace.data_ptr(), nbytes,
                                         self.stream.cuda_stream, C.byref(handle)), "clasp_create")
        self.handle = handle
        self._keep: List[object] = []

    def close(self):
        if getattr(self, "handle", None):
            self.lib.clasp_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- weights
    def load_layers(self, first: int, layers: Sequence[Dict[str, torch.Tensor]]):
        arr = (ClaspLayerWeights * len(layers))()
        for i, lw in enumerate(layers):
            for name, _ in ClaspLayerWeights._fields_:
                t = lw[name]
                assert t.is_cuda and t.is_contiguous()
                setattr(arr[i], name, t.data_ptr())
        self._keep.append(list(layers))
        _check(self.lib.clasp_load_layers(self.handle, first, len(layers), arr), "clasp_load_layers")

    def load_head(self, head: Dict[str, torch.Tensor]):
        self._keep.append(head)
        _check(self.lib.clasp_load_head(self.handle, head["embed"].data_ptr(), head["final_norm"].data_ptr(),
                                        head["lm_head"].data_ptr()), "clasp_load_head")

    # ---- the calls of the hot path
    def dp_search(self, hidden_states: torch.Tensor, layer_stride: int, token_stride: int, kv: KVCache,
                  ctx_len: int, pos0: int, T: int, M: int, want_margins=True, want_g=True,
                  forced_choice: Optional[torch.Tensor] = None):
        """hidden_states: float32 device tensor; element (l, t, c) at l*layer_stride + t*token_stride + c
        (strides in elements from hidden_states' first element).  Returns a dict of device tensors."""
        L, d = self.cfg.L, self.cfg.d_model
        dev = self.device
        mask = torch.empty(L, dtype=torch.uint8, device=dev)
        scores = torch.empty((L + 1, M + 1), dtype=torch.float32, device=dev)
        margins = torch.empty((L + 1, M + 1), dtype=torch.float32, device=dev) if want_margins else None
        g = torch.empty((T, d), dtype=torch.float32, device=dev) if want_g else None
        _check(self.lib.clasp_dp_search(self.handle, hidden_states.data_ptr(), layer_stride, token_stride,
                                        kv.array, ctx_len, pos0, T, M, mask.data_ptr(), scores.data_ptr(),
                                        _ptr(margins), _ptr(g), _ptr(forced_choice)), "clasp_dp_search")
        return {"S": mask, "D": scores, "margin": margins, "g_final": g}

    def verify(self, tokens: torch.Tensor, pos0: int, kv: KVCache, n_head_rows: int,
               want_hidden: bool = True, hidden_out: Optional[torch.Tensor] = None,
               argmax_out: Optional[torch.Tensor] = None):
        n = tokens.numel()
        L, d = self.cfg.L, self.cfg.d_model
        if argmax_out is None:
            argmax_out = torch.empty(max(n_head_rows, 1), dtype=torch.int32, device=self.device)
        if want_hidden and hidden_out is None:
            hidden_out = torch.empty((n, L + 1, d), dtype=torch.float32, device=self.device)
        _check(self.lib.clasp_verify(self.handle, tokens.data_ptr(), n, pos0, kv.array, n_head_rows,
                                     argmax_out.data_ptr(), _ptr(hidden_out) if want_hidden else None),
               "clasp_verify")
        return argmax_out[:n_head_rows], hidden_out

    def draft_forward(self, skip_mask_host: bytes, token_in: torch.Tensor, pos: int, kv: KVCache,
                      token_out: torch.Tensor, top1_prob_out: Optional[torch.Tensor] = None):
        _check(self.lib.clasp_draft_forward(self.handle, skip_mask_host, token_in.data_ptr(), pos, kv.array,
                                            token_out.data_ptr(), _ptr(top1_prob_out)), "clasp_draft_forward")

    def draft_sample(self, skip_mask_host: bytes, token_in: torch.Tensor, pos: int, kv: KVCache, temperature: float,
                     seed: int, rnd: int, token_out: torch.Tensor, logits_out: torch.Tensor):
        _check(self.lib.clasp_draft_sample(self.handle, skip_mask_host, token_in.data_ptr(), pos, kv.array, temperature,
                                           seed, rnd, token_out.data_ptr(), logits_out.data_ptr()), "clasp_draft_sample")

    def verify_sample(self, tokens: torch.Tensor, pos0: int, kv: KVCache, n_drafts: int,
                      draft_logits: Optional[torch.Tensor], temperature: float, seed: int, rnd: int,
                      logits_ws: torch.Tensor, n_accepted_out: torch.Tensor, committed_out: torch.Tensor,
                      hidden_out: Optional[torch.Tensor] = None):
        _check(self.lib.clasp_verify_sample(self.handle, tokens.data_ptr(), tokens.numel(), pos0, kv.array, n_drafts,
                                            _ptr(draft_logits), temperature, seed, rnd, logits_ws.data_ptr(),
                                            n_accepted_out.data_ptr(), committed_out.data_ptr(), _ptr(hidden_out)),
               "clasp_verify_sample")

    def accept(self, draft: Sequence[int], full_argmax: Sequence[int]):
        K = len(draft)
        d = (C.c_int32 * max(K, 1))(*draft)
        f = (C.c_int32 * (K + 1))(*full_argmax)
        a = C.c_int32()
        out = (C.c_int32 * (K + 1))()
        _check(self.lib.clasp_accept(d, f, K, C.byref(a), out), "clasp_accept")
        return a.value, list(out[:a.value + 1])

    def layer_forward(self, layer: int, x_in: torch.Tensor, S: int, T: int, ctx_len: int, pos0: int,
                      kv: KVCache, write_kv: bool = False) -> torch.Tensor:
        assert x_in.dtype == torch.float32 and x_in.is_contiguous() and x_in.shape == (S * T, self.cfg.d_model)
        out = torch.empty_like(x_in)
        kvl = ClaspKvLayer(kv.array[layer].k, kv.array[layer].v)
        _check(self.lib.clasp_layer_forward(self.handle, layer, x_in.data_ptr(), x_in.shape[1], S, T, ctx_len,
                                            pos0, C.byref(kvl), int(write_kv), out.data_ptr(), out.shape[1]),
               "clasp_layer_forward")
        return out

    def gemm_xwT(self, x: torch.Tensor, w: torch.Tensor) -> torch.Tensor:
        R, K = x.shape
        N = w.shape[0]
        y = torch.empty((R, N), dtype=torch.float32, device=self.device)
        _check(self.lib.clasp_gemm_xwT(self.handle, x.data_ptr(), w.data_ptr(), R, N, K, y.data_ptr()),
               "clasp_gemm_xwT")
        return y

    def device_status(self) -> int:
        return self.lib.clasp_last_device_status(self.handle)

    def launch_count(self) -> int:
        return self.lib.clasp_launch_count(self.handle)

    def engine_ctas(self) -> int:
        """Grid size of the persistent kernel (0 when the context does not use it); query only."""
        n = C.c_int32()
        _check(self.lib.clasp_engine_trace(self.handle, None, -1, C.byref(n)), "clasp_engine_trace")
        return n.value

    def engine_active(self) -> bool:
        r = self.lib.clasp_engine_active(self.handle)
        if r < 0:
            raise ClaspError(r, "clasp_engine_active")
        return r == 1

    def set_wait_limit(self, polls: int):
        _check(self.lib.clasp_set_wait_limit(self.handle, polls), "clasp_set_wait_limit")

    def set_trace(self, stamps: Optional[torch.Tensor], cap_per_cta: int = 0):
        """stamps: int64 device tensor [n_ctas, cap_per_cta] or None to stop tracing."""
        self._trace = stamps
        _check(self.lib.clasp_engine_trace(self.handle, _ptr(stamps), cap_per_cta, None), "clasp_engine_trace")
