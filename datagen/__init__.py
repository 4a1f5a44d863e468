"""Seeded synthetic inputs: model shapes, random-init weights, token ids.

This module serves both the CPU oracle's tests and the CUDA path's tests and
benchmark.  It contains no arithmetic of the layer-skip method itself (no
decoder layer, no cosine, no dynamic programme): only shapes and a
counter-based random number generator.

Weights are a pure function of (seed, layer, tensor id, flat index): a
SplitMix64-style integer hash gives two uniforms per element and Box-Muller
turns them into a normal deviate in float64, which is scaled by the tensor's
standard deviation and rounded to the model dtype.  The integer part is exact
on every device; the transcendental part is evaluated by whatever device the
tensors are created on, so a test that needs the very same bytes on the CPU
and on the GPU creates them once and copies them.

Random-init LLaMA-3-shaped decoders stand in for the trained checkpoints and
the uniform random token ids stand in for the benchmark prompts the paper
measured on (Sec. 4, experimental setup); neither is available offline.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict

import torch

_MASK64 = (1 << 64) - 1


@dataclasses.dataclass(frozen=True)
class ModelConfig:
    """Shape of a LLaMA-style decoder (the model family of Sec. 4)."""

    name: str
    L: int                 # decoder layers
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    dtype: str             # "fp32" | "bf16": storage type of weights and KV cache
    rms_eps: float = 1e-5
    rope_theta: float = 500000.0
    init_std: float = 0.02
    scale_out_proj: bool = False   # std of W_o and W_down = init_std / sqrt(2 L)
    norm_std: float = 0.0          # norm weights = 1 + norm_std * N(0,1)
    seed: int = 1

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def torch_dtype(self) -> torch.dtype:
        return {"fp32": torch.float32, "bf16": torch.bfloat16}[self.dtype]

    def layer_params(self) -> int:
        d = self.d_model
        return (d * (self.q_dim + 2 * self.kv_dim) + self.q_dim * d
                + 3 * d * self.d_ffn + 2 * d)

    def layer_matrix_bytes(self) -> int:
        """Bytes of the seven projection matrices of one layer."""
        esz = 4 if self.dtype == "fp32" else 2
        return (self.layer_params() - 2 * self.d_model) * esz


CONFIGS: Dict[str, ModelConfig] = {
    # the small fp32 case the oracle finishes in seconds
    "tiny": ModelConfig("tiny", L=8, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64,
                        d_ffn=688, vocab=1024, dtype="fp32", seed=1),
    # a bf16 case small enough for the oracle that still spans several GEMM
    # tiles with ragged tails (d_ffn and vocab are not multiples of 128)
    "small": ModelConfig("small", L=6, d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=64,
                         d_ffn=1376, vocab=2000, dtype="bf16", norm_std=0.1, seed=5),
    # head_dim 128 and GQA group 4 as in the 8B shape, few layers
    "mini8b": ModelConfig("mini8b", L=4, d_model=1024, n_q_heads=8, n_kv_heads=2, head_dim=128,
                          d_ffn=3584, vocab=4096, dtype="bf16", scale_out_proj=True,
                          norm_std=0.1, seed=6),
    # LLaMA3-8B shape (headline search, context sweep, decode loop)
    "8b": ModelConfig("8b", L=32, d_model=4096, n_q_heads=32, n_kv_heads=8, head_dim=128,
                      d_ffn=14336, vocab=128256, dtype="bf16", scale_out_proj=True, seed=2),
    # the 8B layer shape with few layers and a small vocabulary: a profiler capture saves and
    # restores device memory per pass, so it runs on ~3 GB of weights instead of 16 GB
    "8b-l6": ModelConfig("8b-l6", L=6, d_model=4096, n_q_heads=32, n_kv_heads=8, head_dim=128,
                         d_ffn=14336, vocab=16384, dtype="bf16", scale_out_proj=True, seed=2),
    # LLaMA3-70B shape
    "70b": ModelConfig("70b", L=80, d_model=8192, n_q_heads=64, n_kv_heads=8, head_dim=128,
                       d_ffn=28672, vocab=128256, dtype="bf16", scale_out_proj=True, seed=3),
}

# tensor ids inside a layer (part of the random stream key)
LAYER_TENSORS = ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down")
HEAD_TENSORS = ("embed", "final_norm", "lm_head")
_HEAD_LAYER_KEY = 1 << 20      # "layer" key used for the embedding / head tensors
_TOKEN_LAYER_KEY = (1 << 20) + 1


def _to_i64(v: int) -> int:
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor holding uint64 bit patterns."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64(x: torch.Tensor) -> torch.Tensor:
    """SplitMix64 finaliser on int64 tensors (wrap-around arithmetic)."""
    x = (x ^ _lsr(x, 30)) * _to_i64(0xBF58476D1CE4E5B9)
    x = (x ^ _lsr(x, 27)) * _to_i64(0x94D049BB133111EB)
    return x ^ _lsr(x, 31)


def _mix64_int(v: int) -> int:
    v &= _MASK64
    v = ((v ^ (v >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    v = ((v ^ (v >> 27)) * 0x94D049BB133111EB) & _MASK64
    return v ^ (v >> 31)


def stream_key(seed: int, layer: int, tensor_id: int) -> int:
    """64-bit key of one tensor's random stream."""
    k = _mix64_int(seed * 0x9E3779B97F4A7C15 + 0x1234567)
    k = _mix64_int(k ^ (layer * 0xD1B54A32D192ED03 + 0x51))
    k = _mix64_int(k ^ (tensor_id * 0x8CB92BA72F3D8DD7 + 0x77))
    return k


def raw_bits(key: int, n: int, lane: int, device="cpu", start: int = 0) -> torch.Tensor:
    """n 64-bit hash values (as int64 bit patterns) for counters start..start+n-1."""
    idx = torch.arange(start, start + n, dtype=torch.int64, device=device)
    x = idx * 2 + lane
    x = x * _to_i64(0x9E3779B97F4A7C15) + _to_i64(key)
    return _mix64(_mix64(x) ^ _to_i64(key >> 1))


def uniform01(key: int, n: int, lane: int, device="cpu", start: int = 0) -> torch.Tensor:
    """float64 uniforms in the open interval (0, 1)."""
    bits = _lsr(raw_bits(key, n, lane, device, start), 11)          # 53 bits
    return (bits.to(torch.float64) + 0.5) * (1.0 / 9007199254740992.0)


def standard_normal(key: int, n: int, device="cpu", chunk: int = 1 << 24) -> torch.Tensor:
    """n float64 standard normal deviates (Box-Muller, one per counter)."""
    out = torch.empty(n, dtype=torch.float64, device=device)
    for s in range(0, n, chunk):
        m = min(chunk, n - s)
        u1 = uniform01(key, m, 0, device, s)
        u2 = uniform01(key, m, 1, device, s)
        out[s:s + m] = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
    return out


def _tensor_spec(cfg: ModelConfig, name: str):
    """(shape, std, is_norm) of a named tensor; matrices are row-major [out, in]."""
    d, f = cfg.d_model, cfg.d_ffn
    out_std = cfg.init_std / math.sqrt(2.0 * cfg.L) if cfg.scale_out_proj else cfg.init_std
    table = {
        "attn_norm": ((d,), cfg.norm_std, True),
        "mlp_norm": ((d,), cfg.norm_std, True),
        "final_norm": ((d,), cfg.norm_std, True),
        "wq": ((cfg.q_dim, d), cfg.init_std, False),
        "wk": ((cfg.kv_dim, d), cfg.init_std, False),
        "wv": ((cfg.kv_dim, d), cfg.init_std, False),
        "wo": ((d, cfg.q_dim), out_std, False),
        "w_gate": ((f, d), cfg.init_std, False),
        "w_up": ((f, d), cfg.init_std, False),
        "w_down": ((d, f), out_std, False),
        "embed": ((cfg.vocab, d), cfg.init_std, False),
        "lm_head": ((cfg.vocab, d), cfg.init_std, False),
    }
    return table[name]


def make_tensor(cfg: ModelConfig, layer_key: int, name: str, tensor_id: int, device="cpu",
                seed=None) -> torch.Tensor:
    shape, std, is_norm = _tensor_spec(cfg, name)
    n = 1
    for s in shape:
        n *= s
    seed = cfg.seed if seed is None else seed
    if is_norm and std == 0.0:
        return torch.ones(shape, dtype=torch.float32, device=device)
    z = standard_normal(stream_key(seed, layer_key, tensor_id), n, device)
    if is_norm:
        return (1.0 + std * z).to(torch.float32).reshape(shape)   # norm weights stay fp32
    return (std * z).to(cfg.torch_dtype).reshape(shape)


def layer_weights(cfg: ModelConfig, layer: int, device="cpu", seed=None) -> Dict[str, torch.Tensor]:
    """The nine tensors of decoder layer `layer` (0-based), in the model dtype."""
    return {name: make_tensor(cfg, layer, name, tid, device, seed)
            for tid, name in enumerate(LAYER_TENSORS)}


def head_weights(cfg: ModelConfig, device="cpu", seed=None) -> Dict[str, torch.Tensor]:
    """Token embedding, final norm weight and (untied) LM head."""
    return {name: make_tensor(cfg, _HEAD_LAYER_KEY, name, tid, device, seed)
            for tid, name in enumerate(HEAD_TENSORS)}


def token_ids(cfg: ModelConfig, n: int, seed=None, stream: int = 0) -> torch.Tensor:
    """n uniform random token ids in [0, vocab), int32, on the CPU."""
    seed = cfg.seed if seed is None else seed
    u = uniform01(stream_key(seed, _TOKEN_LAYER_KEY, stream), n, 0)
    return torch.clamp((u * cfg.vocab).to(torch.int64), max=cfg.vocab - 1).to(torch.int32)


def normal_rows(seed: int, stream: int, shape, std: float = 1.0) -> torch.Tensor:
    """Generic float64 normal tensor on the CPU (unit-test inputs)."""
    n = 1
    for s in shape:
        n *= s
    return (std * standard_normal(stream_key(seed, (1 << 20) + 2, stream), n)).reshape(shape)
