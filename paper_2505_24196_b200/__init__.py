"""B200-native (sm_100a) layer-skip search for self-speculative decoding.

The product is libclasp.so (CUDA kernels behind the C ABI of include/clasp.h);
this package is its thin ctypes binding.
"""
from .binding import (gemm_xwT_noalloc, CLASP_BF16, CLASP_FP32, CHOICE_APPLY, CHOICE_NONE, CHOICE_SKIP, FLAG_FORCE_SIMT, FLAG_MULTI_KERNEL, FLAG_NO_ATT_TC, FLAG_NO_DEFER, FLAG_PRUNE, Clasp,
                      ClaspConfig, ClaspError, ClaspKvLayer, ClaspLayerWeights, KVCache, SYMBOLS, load_library,
                      make_config, strerror)
from .decode import SelfSpeculativeDecoder, SpeculativeSampler

__all__ = ["Clasp", "ClaspConfig", "ClaspError", "KVCache", "SelfSpeculativeDecoder", "SpeculativeSampler", "load_library",
           "make_config", "strerror", "SYMBOLS"]
