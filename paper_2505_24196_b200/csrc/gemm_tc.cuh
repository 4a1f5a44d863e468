// Weight-streaming skinny GEMM on the sm_100a tensor cores.
//
//   y[r, n] = sum_k x[r, k] * w[n, k]      x: [R, K] bf16 (R small), w: [N, K] bf16
//
// At DP step i (Algorithm 1) all min(i-1, M) candidate states go through layer i-1
// together (Sec. 3.6), so each weight matrix is read from HBM exactly once per step
// and the work is bandwidth-bound.  The weight's output dimension sits on the MMA's
// M axis (128 rows per CTA), the R activation rows on its N axis (padded to a
// multiple of 16, at most 256), accumulators live in tensor memory:
//
//   warp 0   : one lane issues TMA loads (128B-swizzled [128 x 64] weight tiles and
//              [BN x 64] activation tiles) into a ring of shared-memory stages
//   warp 1   : allocates tensor memory; one lane issues tcgen05.mma (M=128, N=BN, K=16)
//              and commits each stage back to the producer
//   warps 2-5: read the accumulators with tcgen05.ld (one lane quarter per warp) and
//              run the epilogue: plain store, residual add, or SwiGLU of a gate/up pair
//
// Split-K: blockIdx.y selects a K range; partial sums go to a workspace and the CTA
// that arrives last at the tile's counter adds them in split-index order, so the
// result is a fixed function of (N, K, splits) and never of R or of arrival order.
// Every wait is bounded; one that runs out sets *status and the CTA winds down.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace clasp {
namespace tc {

constexpr int BM = 128;       // weight rows (output features) per CTA
constexpr int BK = 64;        // K elements per stage: 128 bytes of bf16 = one swizzle row
constexpr int THREADS = 192;  // producer warp, MMA warp, four epilogue warps
constexpr int A_TILE_BYTES = BM * BK * 2;
constexpr uint32_t SPIN_FAST = 1u << 14;
constexpr uint32_t SPIN_SLOW = 1u << 21;  // x ~128 ns sleeps: gives up after roughly 0.3 s

struct Params {
  int R;        // valid activation rows
  int BN;       // rows padded to a multiple of 16 (the MMA's N)
  int K;        // reduction length
  int k_chunks; // ceil(K / 64)
  int splits;   // gridDim.y
  int stages;
  int dual;     // 1: SwiGLU, second weight matrix through map A1 into a second accumulator
  int n_mats;   // 1..3 weight matrices stacked along N (fused q/k/v projection)
  int N[3];
  int tiles[3];    // ceil(N[m] / 128)
  int col_off[3];  // output column of matrix m's first feature
  int epi;         // 0 store float, 1 residual add (float), 2 SwiGLU (bf16 out)
  int n_total;     // sum of N[m]: row length of the partial-sum workspace
  float* yf;
  long long ldy;
  const float* resid;
  long long ldr;
  __nv_bfloat16* yo;
  long long ldo;
  float* partial;  // [splits][dual+1][R][n_total]
  int* counters;   // one per tile, zero on entry, zero again on exit
  int* status;     // set to 1 when a bounded wait gives up
  uint32_t spin_fast, spin_slow;  // polls without / with a ~128 ns sleep before a wait gives up
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false (and *status = 1) if the phase never completes.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int* status, uint32_t n_fast = SPIN_FAST,
                                          uint32_t n_slow = SPIN_SLOW) {
  for (uint32_t it = 0; it < n_fast; ++it)
    if (mbar_test(bar, parity)) return true;
  for (uint32_t it = 0; it < n_slow; ++it) {
    if (mbar_test(bar, parity)) return true;
    __nanosleep(128);
  }
  atomicExch(status, 1);
  return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x,
                                            int y, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%3, %4}], [%2], %5;"
      :
      : "r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "l"(policy)
      : "memory");
}
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr) {
  // K-major operand, 128-byte swizzle: rows of 128 B, 8-row groups 1024 B apart.
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                         uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      :
      : "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32"
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ float silu(float g) { return g / (1.0f + __expf(-g)); }

__global__ void __launch_bounds__(THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap mapA0, const __grid_constant__ CUtensorMap mapA1,
               const __grid_constant__ CUtensorMap mapA2, const __grid_constant__ CUtensorMap mapB,
               const Params p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[8], bar_empty[8], bar_accum;
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort, s_is_last;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int a_bytes = A_TILE_BYTES * (p.dual ? 2 : 1);
  const int b_bytes = p.BN * BK * 2;
  const int stage_bytes = a_bytes + b_bytes;  // multiples of 2048: every tile stays 1024-aligned

  // which weight matrix and which 128 features this CTA owns
  int tile = blockIdx.x, mat = 0;
  while (mat + 1 < p.n_mats && tile >= p.tiles[mat]) { tile -= p.tiles[mat]; ++mat; }
  const int n0 = tile * BM;
  const CUtensorMap* mapA = mat == 0 ? &mapA0 : (mat == 1 ? &mapA1 : &mapA2);
  const int kc_begin = (int)((long long)p.k_chunks * blockIdx.y / p.splits);
  const int kc_end = (int)((long long)p.k_chunks * (blockIdx.y + 1) / p.splits);
  const int n_iter = kc_end - kc_begin;

  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < p.BN * (p.dual ? 2 : 1)) tmem_cols <<= 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    mbar_init(smem_u32(&bar_accum), 1);
    s_abort = 0;
    s_is_last = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)),
                 "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = s_tmem_base;

  if (warp == 0) {
    // ------------------------------------------------ TMA producer
    if (lane == 0) {
      uint64_t pol_stream, pol_keep;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
      for (int it = 0; it < n_iter; ++it) {
        const int s = it % p.stages;
        const uint32_t phase = (uint32_t)(it / p.stages) & 1u;
        if (!mbar_wait(smem_u32(&bar_empty[s]), phase ^ 1u, p.status, p.spin_fast, p.spin_slow)) { s_abort = 1; break; }
        const uint32_t full = smem_u32(&bar_full[s]);
        const uint32_t sa = smem_base + s * stage_bytes;
        const int kx = (kc_begin + it) * BK;
        mbar_expect_tx(full, (uint32_t)stage_bytes);
        if (p.dual) {
          tma_load_2d(sa, &mapA0, full, kx, n0, pol_stream);
          tma_load_2d(sa + A_TILE_BYTES, &mapA1, full, kx, n0, pol_stream);
        } else {
          tma_load_2d(sa, mapA, full, kx, n0, pol_stream);
        }
        tma_load_2d(sa + a_bytes, &mapB, full, kx, 0, pol_keep);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.BN >> 3) << 17) | (8u << 24);
      bool ok = true;
      for (int it = 0; it < n_iter && ok; ++it) {
        const int s = it % p.stages;
        const uint32_t phase = (uint32_t)(it / p.stages) & 1u;
        if (!mbar_wait(smem_u32(&bar_full[s]), phase, p.status, p.spin_fast, p.spin_slow)) { s_abort = 1; ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t sa = smem_base + s * stage_bytes;
        const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sa + a_bytes);
#pragma unroll
        for (int kk = 0; kk < BK / 16; ++kk) {
          const uint32_t acc = (it > 0 || kk > 0) ? 1u : 0u;
          mma_bf16(tmem_base, da + 2 * kk, db + 2 * kk, idesc, acc);
          if (p.dual) {
            const uint64_t da2 = make_smem_desc(sa + A_TILE_BYTES);
            mma_bf16(tmem_base + p.BN, da2 + 2 * kk, db + 2 * kk, idesc, acc);
          }
        }
        mma_commit(smem_u32(&bar_empty[s]));  // stage reusable once these MMAs have read it
      }
      if (ok) mma_commit(smem_u32(&bar_accum));
    }
  } else {
    // ------------------------------------------------ epilogue (4 warps, 128 threads)
    const int q = warp & 3;  // tensor-memory lane quarter this warp may read
    const int n_local = n0 + q * 32 + lane;
    const bool n_ok = n_local < p.N[mat];
    const int col = p.col_off[mat] + n_local;
    const bool have_acc = n_iter > 0;
    bool ok = true;
    if (have_acc) ok = mbar_wait(smem_u32(&bar_accum), 0, p.status, p.spin_fast, p.spin_slow);
    ok = __all_sync(0xffffffffu, ok);  // tcgen05.ld below needs the whole warp
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
    const int planes = p.dual ? 2 : 1;
    if (ok) {
      for (int c0 = 0; c0 < p.R; c0 += 16) {
        float g[16], u[16];
        if (have_acc) {
          tmem_ld16(t_lane + c0, g);
          if (p.dual) tmem_ld16(t_lane + p.BN + c0, u);
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) { g[i] = 0.f; u[i] = 0.f; }
        }
        if (p.splits == 1) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int r = c0 + i;
            if (r < p.R && n_ok) {
              if (p.epi == 0) p.yf[r * p.ldy + col] = g[i];
              else if (p.epi == 1) p.yf[r * p.ldy + col] = p.resid[r * p.ldr + col] + g[i];
              else p.yo[r * p.ldo + col] = __float2bfloat16_rn(silu(g[i]) * u[i]);
            }
          }
        } else {
          float* part = p.partial + (long long)blockIdx.y * planes * p.R * p.n_total;
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int r = c0 + i;
            if (r < p.R && n_ok) {
              part[(long long)r * p.n_total + col] = g[i];
              if (p.dual) part[((long long)p.R + r) * p.n_total + col] = u[i];
            }
          }
        }
      }
    }
    if (p.splits > 1) {
      // last CTA of this tile (by arrival) adds the partial sums in split order
      __threadfence();
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (threadIdx.x == 64) {
        const int prev = atomicAdd(&p.counters[blockIdx.x], 1);
        s_is_last = (prev == p.splits - 1);
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (s_is_last) {
        __threadfence();
        if (n_ok) {
          const long long plane = (long long)p.R * p.n_total;
          for (int r = 0; r < p.R; ++r) {
            float g = 0.f, u = 0.f;
            for (int s = 0; s < p.splits; ++s) {
              const float* part = p.partial + (long long)s * planes * plane;
              g += __ldcg(part + (long long)r * p.n_total + col);
              if (p.dual) u += __ldcg(part + plane + (long long)r * p.n_total + col);
            }
            if (p.epi == 0) p.yf[r * p.ldy + col] = g;
            else if (p.epi == 1) p.yf[r * p.ldy + col] = p.resid[r * p.ldr + col] + g;
            else p.yo[r * p.ldo + col] = __float2bfloat16_rn(silu(g) * u);
          }
        }
        if (threadIdx.x == 64) p.counters[blockIdx.x] = 0;
      }
    }
  }

  // ---------------------------------------------------- wind down
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (s_abort) {
    // a wait gave up: let copies and MMAs still in flight drain before the CTA's
    // shared and tensor memory are released
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols)
                 : "memory");
  }
}

}  // namespace tc
}  // namespace clasp
