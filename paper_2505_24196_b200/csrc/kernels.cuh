// CUDA-core kernels of the layer-skip search: everything of a decoder layer that
// is not a weight-streaming GEMM on the tensor cores (RMSNorm, rotary embedding,
// attention over the verified cache plus a state's own rows, the cosine / select /
// write-back step of Eq. 2, the backtrack of Algorithm 1, embedding gather, argmax),
// plus a CUDA-core GEMM used by the fp32 model (whose tolerance rules out bf16
// tensor-core products).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace clasp {

// ---------------------------------------------------------------- helpers

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// 8 consecutive elements of the model dtype as floats (16-byte aligned for bf16,
// 32-byte aligned for float).
__device__ __forceinline__ void load8(const float* p, float (&f)[8]) {
  float4 a = *reinterpret_cast<const float4*>(p);
  float4 b = *reinterpret_cast<const float4*>(p + 4);
  f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w;
  f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&f)[8]) {
  uint4 u = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float v) {
  return __float2bfloat16_rn(v);
}

__device__ __forceinline__ float silu_f(float g) { return g / (1.0f + __expf(-g)); }

// ---------------------------------------------------------------- RMSNorm
// y[r, :] = x[r, :] * rsqrt(mean(x^2) + eps) * w, rounded to the GEMM operand type.
// One block per row; the sum of squares is reduced in a fixed order.
template <typename TO>
__global__ void rmsnorm_kernel(const float* __restrict__ x, int64_t ldx, const float* __restrict__ w,
                               int d, float eps, TO* __restrict__ y) {
  const int r = blockIdx.x;
  const float* xr = x + (int64_t)r * ldx;
  float ss = 0.f;
  for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4) {
    float4 v = *reinterpret_cast<const float4*>(xr + c);
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  __shared__ float red[32];
  __shared__ float s_scale;
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x < 32) {
    float v = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.f;
    v = warp_sum(v);
    if (threadIdx.x == 0) s_scale = rsqrtf(v / (float)d + eps);
  }
  __syncthreads();
  const float sc = s_scale;
  TO* yr = y + (int64_t)r * d;
  for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4) {
    float4 v = *reinterpret_cast<const float4*>(xr + c);
    float4 g = *reinterpret_cast<const float4*>(w + c);
    yr[c] = from_float<TO>(v.x * sc * g.x);
    yr[c + 1] = from_float<TO>(v.y * sc * g.y);
    yr[c + 2] = from_float<TO>(v.z * sc * g.z);
    yr[c + 3] = from_float<TO>(v.w * sc * g.w);
  }
}

// ---------------------------------------------------------------- CUDA-core GEMM
// y[r, n] = sum_k x[r, k] * w[n, k]; one warp per output column n, lanes stride
// over k with 8-element vector loads, rows in blocks of RB.  The summation order
// depends on K only, never on the number of rows.
enum { EPI_STORE = 0, EPI_RESID = 1, EPI_SWIGLU = 2 };

template <typename TW, int EPI, int RB>
__global__ void gemm_simt_kernel(const TW* __restrict__ x, int64_t ldx, const TW* __restrict__ w,
                                 const TW* __restrict__ w2, int R, int N, int K,
                                 float* __restrict__ yf, int64_t ldy, const float* __restrict__ resid,
                                 int64_t ldr, TW* __restrict__ yo, int64_t ldo) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n = blockIdx.x * (blockDim.x >> 5) + warp;
  if (n >= N) return;
  const TW* wr = w + (int64_t)n * K;
  const TW* w2r = (EPI == EPI_SWIGLU) ? w2 + (int64_t)n * K : nullptr;
  for (int r0 = 0; r0 < R; r0 += RB) {
    float acc[RB], acc2[RB];
#pragma unroll
    for (int i = 0; i < RB; ++i) { acc[i] = 0.f; acc2[i] = 0.f; }
    for (int k = lane * 8; k < K; k += 256) {
      float wv[8], w2v[8];
      load8(wr + k, wv);
      if (EPI == EPI_SWIGLU) load8(w2r + k, w2v);
#pragma unroll
      for (int i = 0; i < RB; ++i) {
        if (r0 + i < R) {
          float xv[8];
          load8(x + (int64_t)(r0 + i) * ldx + k, xv);
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            acc[i] = fmaf(xv[e], wv[e], acc[i]);
            if (EPI == EPI_SWIGLU) acc2[i] = fmaf(xv[e], w2v[e], acc2[i]);
          }
        }
      }
    }
#pragma unroll
    for (int i = 0; i < RB; ++i) {
      float a = warp_sum(acc[i]);
      float b = (EPI == EPI_SWIGLU) ? warp_sum(acc2[i]) : 0.f;
      if (lane == 0 && r0 + i < R) {
        const int r = r0 + i;
        if (EPI == EPI_STORE) yf[(int64_t)r * ldy + n] = a;
        if (EPI == EPI_RESID) yf[(int64_t)r * ldy + n] = resid[(int64_t)r * ldr + n] + a;
        if (EPI == EPI_SWIGLU) yo[(int64_t)r * ldo + n] = from_float<TW>(silu_f(a) * b);
      }
    }
  }
}

// ---------------------------------------------------------------- rotary table
// cs[t, i] = (cos, sin) of (pos0 + t) * theta^(-2i/hd), evaluated in double so
// that long contexts do not lose the angle's low bits.
__global__ void rope_table_kernel(float2* __restrict__ cs, int T, int half, int pos0, double theta) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= T * half) return;
  const int t = idx / half, i = idx % half;
  const double inv = exp2(-(2.0 * i / (2.0 * half)) * log2(theta));
  double s, c;
  sincos((double)(pos0 + t) * inv, &s, &c);
  cs[idx] = make_float2((float)c, (float)s);
}

// K/V of the rows: rotate k, round k and v to the cache dtype and store them at row
// (own_base + r) of own_k / own_v ([rows, n_kv, hd]).  q stays un-rotated in qkv; the
// attention kernel rotates it while loading.  One block per row.
template <typename TW>
__global__ void kv_store_kernel(const float* __restrict__ qkv, int64_t ld, const float2* __restrict__ cs,
                                int T, int nq, int nkv, int hd, TW* __restrict__ own_k,
                                TW* __restrict__ own_v, int64_t own_base) {
  const int r = blockIdx.x, t = r % T, half = hd >> 1;
  const float* row = qkv + (int64_t)r * ld;
  const float2* c = cs + (int64_t)t * half;
  const float* kr = row + nq * hd;
  const float* vr = kr + nkv * hd;
  TW* ko = own_k + (own_base + r) * (int64_t)(nkv * hd);
  TW* vo = own_v + (own_base + r) * (int64_t)(nkv * hd);
  for (int idx = threadIdx.x; idx < nkv * half; idx += blockDim.x) {
    const int h = idx / half, i = idx % half;
    const float a = kr[h * hd + i], b = kr[h * hd + i + half];
    ko[h * hd + i] = from_float<TW>(a * c[i].x - b * c[i].y);
    ko[h * hd + i + half] = from_float<TW>(b * c[i].x + a * c[i].y);
  }
  for (int idx = threadIdx.x; idx < nkv * hd; idx += blockDim.x) vo[idx] = from_float<TW>(vr[idx]);
}

// ---------------------------------------------------------------- attention
// Grid (key chunk, kv head, pair block).  A CTA stages 64-key tiles of one kv head's K
// and V in shared memory and runs every (row, query head) pair of that kv head against
// them, so the cache is read from HBM/L2 once per pair block instead of once per pair.
// Chunks [0, n_cache_chunks) cover the verified cache, nsub tiles of 64 keys each with an
// online softmax across the tiles; the remaining chunks cover the rows' own keys, 64
// flattened rows per chunk, masked so that row (s, t) sees rows (s, t' <= t) only
// (Sec. 3.6: states share the cache and never see each other).  q is rotated (RoPE) while
// it is loaded.  Each (pair, chunk) leaves an un-normalised partial (acc[hd], max, sum);
// attn_merge_kernel adds the chunks in index order, so the result depends on (C, R) only
// through the fixed chunking and never on timing.
constexpr int ATT_KEYS = 64;
constexpr int ATT_WARPS = 8;
constexpr int ATT_PPW = 8;
constexpr int ATT_PAIRS = ATT_WARPS * ATT_PPW;
constexpr int ATT_MAX_CACHE_CHUNKS = 16;

template <typename TW, int HD>
constexpr int att_smem_bytes() {
  return ATT_KEYS * (HD + 16 / (int)sizeof(TW)) * (int)sizeof(TW) + ATT_KEYS * HD * (int)sizeof(TW) +
         ATT_PAIRS * HD * 4 + ATT_WARPS * ATT_KEYS * 4;
}

template <int DPL> __device__ __forceinline__ void load_dpl(const float* p, float (&f)[DPL]) {
  if (DPL == 4) { float4 v = *reinterpret_cast<const float4*>(p); f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w; }
  else { float2 v = *reinterpret_cast<const float2*>(p); f[0] = v.x; f[1] = v.y; }
}
template <int DPL> __device__ __forceinline__ void load_dpl(const __nv_bfloat16* p, float (&f)[DPL]) {
  if (DPL == 4) {
    uint2 u = *reinterpret_cast<const uint2*>(p);
    f[0] = __uint_as_float(u.x << 16); f[1] = __uint_as_float(u.x & 0xffff0000u);
    f[2] = __uint_as_float(u.y << 16); f[3] = __uint_as_float(u.y & 0xffff0000u);
  } else {
    uint32_t u = *reinterpret_cast<const uint32_t*>(p);
    f[0] = __uint_as_float(u << 16); f[1] = __uint_as_float(u & 0xffff0000u);
  }
}

template <typename TW, int HD>
__global__ void __launch_bounds__(ATT_WARPS * 32)
attn_tile_kernel(const float* __restrict__ qkv, int64_t ldq, const float2* __restrict__ cs,
                 const TW* __restrict__ ck, const TW* __restrict__ cv, int C,
                 const TW* __restrict__ own_k, const TW* __restrict__ own_v, int64_t own_base,
                 int R, int T, int nq, int nkv, int n_cache_chunks, int nsub, int n_chunks,
                 float* __restrict__ part_acc, float2* __restrict__ part_ml) {
  constexpr int DPL = HD / 32;
  constexpr int KLD = HD + 16 / (int)sizeof(TW);       // padded K row: conflict-free 16-byte reads
  constexpr int VEC = 16 / (int)sizeof(TW);            // elements per 16-byte vector
  constexpr int VPR = HD / VEC;                        // vectors per row
  extern __shared__ __align__(16) unsigned char att_smem[];
  TW* k_s = reinterpret_cast<TW*>(att_smem);
  TW* v_s = k_s + ATT_KEYS * KLD;
  float* q_s = reinterpret_cast<float*>(v_s + ATT_KEYS * HD);
  float* p_s = q_s + ATT_PAIRS * HD;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunk = blockIdx.x, kvh = blockIdx.y, pb = blockIdx.z;
  const int G = nq / nkv, n_pairs = R * G, half = HD / 2;
  const bool own_chunk = chunk >= n_cache_chunks;
  const int64_t kvld = (int64_t)nkv * HD;
  const float scale = rsqrtf((float)HD) * 1.4426950408889634f;  // 1/sqrt(hd) * log2(e)

  // this warp's pairs: p = pb*ATT_PAIRS + pi*ATT_WARPS + warp
  float m[ATT_PPW], l[ATT_PPW], acc[ATT_PPW][DPL];
#pragma unroll
  for (int pi = 0; pi < ATT_PPW; ++pi) {
    m[pi] = -INFINITY; l[pi] = 0.f;
#pragma unroll
    for (int i = 0; i < DPL; ++i) acc[pi][i] = 0.f;
    const int p = pb * ATT_PAIRS + pi * ATT_WARPS + warp;
    if (p < n_pairs) {
      const int r = p / G, hq = kvh * G + p % G, t = r % T;
      const float* qr = qkv + (int64_t)r * ldq + hq * HD;
      float* qd = q_s + (warp * ATT_PPW + pi) * HD;
      for (int c = lane; c < half; c += 32) {
        const float a = qr[c], b = qr[c + half];
        const float2 w = cs[(int64_t)t * half + c];
        qd[c] = (a * w.x - b * w.y) * scale;
        qd[c + half] = (b * w.x + a * w.y) * scale;
      }
    }
  }
  __syncwarp();

  const int n_tiles = own_chunk ? 1 : nsub;
  for (int st = 0; st < n_tiles; ++st) {
    int key0, nkeys;
    const TW *src_k, *src_v;
    if (!own_chunk) {
      key0 = (chunk * nsub + st) * ATT_KEYS;
      nkeys = min(ATT_KEYS, C - key0);
      src_k = ck + (int64_t)key0 * kvld + kvh * HD;
      src_v = cv + (int64_t)key0 * kvld + kvh * HD;
    } else {
      key0 = (chunk - n_cache_chunks) * ATT_KEYS;       // first flattened own row of this chunk
      nkeys = min(ATT_KEYS, R - key0);
      src_k = own_k + (own_base + key0) * kvld + kvh * HD;
      src_v = own_v + (own_base + key0) * kvld + kvh * HD;
    }
    if (nkeys <= 0) break;                               // uniform across the CTA
    __syncthreads();                                     // previous tile fully consumed
    for (int v = threadIdx.x; v < ATT_KEYS * VPR; v += blockDim.x) {
      const int row = v / VPR, cv16 = v % VPR;
      uint4 kk = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
      if (row < nkeys) {
        kk = *reinterpret_cast<const uint4*>(src_k + (int64_t)row * kvld + cv16 * VEC);
        vv = *reinterpret_cast<const uint4*>(src_v + (int64_t)row * kvld + cv16 * VEC);
      }
      *reinterpret_cast<uint4*>(k_s + row * KLD + cv16 * VEC) = kk;
      *reinterpret_cast<uint4*>(v_s + row * HD + cv16 * VEC) = vv;
    }
    __syncthreads();

#pragma unroll
    for (int pi = 0; pi < ATT_PPW; ++pi) {
      const int p = pb * ATT_PAIRS + pi * ATT_WARPS + warp;
      if (p >= n_pairs) continue;                        // warp-uniform
      const int r = p / G;
      bool ok0 = lane < nkeys, ok1 = lane + 32 < nkeys;
      if (own_chunk) {
        const int r0 = key0 + lane, r1 = key0 + lane + 32;
        ok0 = ok0 && (r0 / T == r / T) && (r0 <= r);
        ok1 = ok1 && (r1 / T == r / T) && (r1 <= r);
      }
      if (!__any_sync(0xffffffffu, ok0 || ok1)) continue;
      const float* qd = q_s + (warp * ATT_PPW + pi) * HD;
      const TW* k0 = k_s + lane * KLD;
      const TW* k1 = k_s + (lane + 32) * KLD;
      float s0 = 0.f, s1 = 0.f;
#pragma unroll 4
      for (int c = 0; c < HD; c += 8) {
        float a[8], b[8];
        load8(k0 + c, a);
        load8(k1 + c, b);
        const float4 q0 = *reinterpret_cast<const float4*>(qd + c);
        const float4 q1 = *reinterpret_cast<const float4*>(qd + c + 4);
        s0 = fmaf(a[0], q0.x, s0); s0 = fmaf(a[1], q0.y, s0); s0 = fmaf(a[2], q0.z, s0); s0 = fmaf(a[3], q0.w, s0);
        s0 = fmaf(a[4], q1.x, s0); s0 = fmaf(a[5], q1.y, s0); s0 = fmaf(a[6], q1.z, s0); s0 = fmaf(a[7], q1.w, s0);
        s1 = fmaf(b[0], q0.x, s1); s1 = fmaf(b[1], q0.y, s1); s1 = fmaf(b[2], q0.z, s1); s1 = fmaf(b[3], q0.w, s1);
        s1 = fmaf(b[4], q1.x, s1); s1 = fmaf(b[5], q1.y, s1); s1 = fmaf(b[6], q1.z, s1); s1 = fmaf(b[7], q1.w, s1);
      }
      if (!ok0) s0 = -INFINITY;
      if (!ok1) s1 = -INFINITY;
      const float m_new = fmaxf(m[pi], warp_max(fmaxf(s0, s1)));
      const float corr = exp2f(m[pi] - m_new);          // m = -inf on the first tile: exp2(-inf) = 0
      const float p0 = ok0 ? exp2f(s0 - m_new) : 0.f;
      const float p1 = ok1 ? exp2f(s1 - m_new) : 0.f;
      l[pi] = l[pi] * corr + warp_sum(p0 + p1);
      m[pi] = m_new;
      float* pw = p_s + warp * ATT_KEYS;
      __syncwarp();
      pw[lane] = p0;
      pw[lane + 32] = p1;
      __syncwarp();
      float o[DPL];
#pragma unroll
      for (int i = 0; i < DPL; ++i) o[i] = acc[pi][i] * corr;
      const TW* vcol = v_s + lane * DPL;
#pragma unroll 8
      for (int k = 0; k < ATT_KEYS; ++k) {
        float vv[DPL];
        load_dpl<DPL>(vcol + k * HD, vv);
        const float pk = pw[k];
#pragma unroll
        for (int i = 0; i < DPL; ++i) o[i] = fmaf(pk, vv[i], o[i]);
      }
#pragma unroll
      for (int i = 0; i < DPL; ++i) acc[pi][i] = o[i];
    }
  }

#pragma unroll
  for (int pi = 0; pi < ATT_PPW; ++pi) {
    const int p = pb * ATT_PAIRS + pi * ATT_WARPS + warp;
    if (p >= n_pairs) continue;
    const int r = p / G, hq = kvh * G + p % G;
    const int64_t idx = ((int64_t)r * nq + hq) * n_chunks + chunk;
    float* pa = part_acc + idx * HD + lane * DPL;
#pragma unroll
    for (int i = 0; i < DPL; ++i) pa[i] = acc[pi][i];
    if (lane == 0) part_ml[idx] = make_float2(m[pi], l[pi]);
  }
}

// Merge the chunks of one (row, head) in index order and round to the operand type.
// A chunk that held no visible key has max = -inf and weight 0.
template <typename TO, int HD>
__global__ void attn_merge_kernel(const float* __restrict__ part_acc, const float2* __restrict__ part_ml,
                                  int R, int nq, int nsplit, TO* __restrict__ out) {
  const int64_t rh = blockIdx.x;  // r * nq + h
  const int c = threadIdx.x;      // HD threads
  float mx = -INFINITY;
  for (int sp = 0; sp < nsplit; ++sp) mx = fmaxf(mx, part_ml[rh * nsplit + sp].x);
  float num = 0.f, den = 0.f;
  for (int sp = 0; sp < nsplit; ++sp) {
    const float2 ml = part_ml[rh * nsplit + sp];
    if (ml.x == -INFINITY) continue;
    const float wgt = exp2f(ml.x - mx);
    num = fmaf(wgt, part_acc[(rh * nsplit + sp) * HD + c], num);
    den = fmaf(wgt, ml.y, den);
  }
  out[rh * HD + c] = from_float<TO>(num / den);
}

// ---------------------------------------------------------------- Eq. 2 step
// Block b of DP step i:
//   b == 0            : g_next[0] = x_i,  D[i][0] = 1
//   1 <= b <= ell     : j = b.  sigma_app = cos(x_i, G[j-1]), sigma_skip = cos(x_i, g_prev[j-1]);
//                       APPLY iff sigma_app > sigma_skip (strict), unless forced.
//   b == ell + 1      : (only when i <= M) diagonal j = i: g_next[i] = g_prev[i-1].
// A state's score is the mean over its T rows of the per-row cosine.
struct DpStepArgs {
  const float* x_i;       // row t at x_i + t * x_tok_stride
  int64_t x_tok_stride;
  const float* G;         // [ell*T, d] layer outputs of the ell states j = j_lo .. j_lo + ell - 1
  const float* g_prev;    // [(M+1)*T, d]
  float* g_next;          // [(M+1)*T, d]
  float* D;               // row i of the tables: [M+1]
  float* margin;          // may be null
  uint8_t* choice;        // row i of the choice table (always present: workspace)
  const uint8_t* forced;  // row i or null
  int T, d, ell, i, M;
  int j_lo;               // first state the step carries (1, or later when unreachable states are left out)
};

__device__ __forceinline__ void block_sum3(double (&v)[3], double* sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
  for (int k = 0; k < 3; ++k) v[k] = warp_sum_d(v[k]);
  __syncthreads();
  if (lane == 0) { sh[warp * 3] = v[0]; sh[warp * 3 + 1] = v[1]; sh[warp * 3 + 2] = v[2]; }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < 3; ++k) {
    double s = 0.0;
    for (int w2 = 0; w2 < nw; ++w2) s += sh[w2 * 3 + k];
    v[k] = s;
  }
}

// mean over T rows of cos(x_i[t], y[t])
__device__ float mean_cosine(const DpStepArgs& a, const float* y, double* sh) {
  double total = 0.0;
  for (int t = 0; t < a.T; ++t) {
    const float* xr = a.x_i + t * a.x_tok_stride;
    const float* yr = y + (int64_t)t * a.d;
    float xx = 0.f, yy = 0.f, xy = 0.f;
    for (int c = threadIdx.x * 4; c < a.d; c += blockDim.x * 4) {
      const float4 u = *reinterpret_cast<const float4*>(xr + c);
      const float4 v = *reinterpret_cast<const float4*>(yr + c);
      xx += u.x * u.x + u.y * u.y + u.z * u.z + u.w * u.w;
      yy += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
      xy += u.x * v.x + u.y * v.y + u.z * v.z + u.w * v.w;
    }
    double v3[3] = {(double)xx, (double)yy, (double)xy};
    block_sum3(v3, sh);
    const double nx = fmax(sqrt(v3[0]), 1e-12), ny = fmax(sqrt(v3[1]), 1e-12);
    total += v3[2] / (nx * ny);
  }
  return (float)(total / a.T);
}

__global__ void dp_step_kernel(DpStepArgs a) {
  __shared__ double sh[32 * 3];
  __shared__ int s_take_apply;
  const int b = blockIdx.x;
  const int64_t Td = (int64_t)a.T * a.d;
  if (b == 0) {
    for (int t = 0; t < a.T; ++t)
      for (int c = threadIdx.x * 4; c < a.d; c += blockDim.x * 4)
        *reinterpret_cast<float4*>(a.g_next + (int64_t)t * a.d + c) =
            *reinterpret_cast<const float4*>(a.x_i + t * a.x_tok_stride + c);
    if (threadIdx.x == 0) {
      a.D[0] = 1.0f;
      a.choice[0] = 0;
    }
    return;
  }
  if (b == a.ell + 1) {  // (only launched while i <= M) diagonal j = i: all of the first i layers skipped
    const int j = a.i;
    const float* src = a.g_prev + (int64_t)(j - 1) * Td;
    const float sc = mean_cosine(a, src, sh);
    for (int64_t c = threadIdx.x * 4; c < Td; c += blockDim.x * 4)
      *reinterpret_cast<float4*>(a.g_next + (int64_t)j * Td + c) = *reinterpret_cast<const float4*>(src + c);
    if (threadIdx.x == 0) {
      a.D[j] = sc;
      a.choice[j] = 1;
    }
    return;
  }
  const int j = a.j_lo + b - 1;
  const float* app = a.G + (int64_t)(b - 1) * Td;
  const float* skp = a.g_prev + (int64_t)(j - 1) * Td;
  const float s_app = mean_cosine(a, app, sh);
  const float s_skip = mean_cosine(a, skp, sh);
  if (threadIdx.x == 0) {
    int take = s_app > s_skip;
    if (a.forced && a.forced[j] != 255) take = (a.forced[j] == 0);
    s_take_apply = take;
    a.D[j] = take ? s_app : s_skip;
    if (a.margin) a.margin[j] = s_app - s_skip;
    a.choice[j] = take ? 0 : 1;
  }
  __syncthreads();
  const float* src = s_take_apply ? app : skp;
  for (int64_t c = threadIdx.x * 4; c < Td; c += blockDim.x * 4)
    *reinterpret_cast<float4*>(a.g_next + (int64_t)j * Td + c) = *reinterpret_cast<const float4*>(src + c);
}

// Backtrack of Algorithm 1 on the choice table [(L+1) x (M+1)]: one thread.
__global__ void backtrack_kernel(const uint8_t* __restrict__ choice, int L, int M, uint8_t* __restrict__ S) {
  if (blockIdx.x != 0 || threadIdx.x != 0) return;
  for (int l = 0; l < L; ++l) S[l] = 0;
  int i = L, j = M;
  while (i > 0 && j > 0) {
    if (choice[i * (M + 1) + j] == 1) {
      S[i - 1] = 1;
      --j;
    }
    --i;
  }
}

__global__ void fill_tables_kernel(float* D, float* margin, uint8_t* choice, int n) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n) return;
  D[idx] = __int_as_float(0x7fc00000);
  if (margin) margin[idx] = __int_as_float(0x7fc00000);
  choice[idx] = 255;
}

// D(0, 0) = 1 and its choice entry: the origin of the table (g[0][0] = x_0)
__global__ void dp_origin_kernel(float* D, uint8_t* choice) {
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    D[0] = 1.0f;
    choice[0] = 0;
  }
}

// rows of floats: dst[r, :] = src[r, :] (strided)
__global__ void copy_rows_kernel(const float* __restrict__ src, int64_t lds, float* __restrict__ dst,
                                 int64_t ldd, int d) {
  const int r = blockIdx.x;
  for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4)
    *reinterpret_cast<float4*>(dst + r * ldd + c) = *reinterpret_cast<const float4*>(src + r * lds + c);
}

// ---------------------------------------------------------------- embedding, argmax
template <typename TW>
__global__ void embed_kernel(const int32_t* __restrict__ tokens, const TW* __restrict__ table, int d,
                             int vocab, float* __restrict__ out, int64_t ldo) {
  const int r = blockIdx.x;
  int tok = tokens[r];
  tok = tok < 0 ? 0 : (tok >= vocab ? vocab - 1 : tok);
  const TW* src = table + (int64_t)tok * d;
  for (int c = threadIdx.x; c < d; c += blockDim.x) out[r * ldo + c] = to_float(src[c]);
}

// Greedy token of each logits row: largest value, lowest index on ties; also the
// softmax probability of that token when asked for.
__global__ void argmax_kernel(const float* __restrict__ logits, int vocab, int32_t* __restrict__ out,
                              float* __restrict__ top1_prob) {
  const int r = blockIdx.x;
  const float* row = logits + (int64_t)r * vocab;
  float best = -INFINITY;
  int bi = 0x7fffffff;
  for (int c = threadIdx.x; c < vocab; c += blockDim.x) {
    const float v = row[c];
    if (v > best || (v == best && c < bi)) { best = v; bi = c; }
  }
  __shared__ float sv[32];
  __shared__ int si[32];
  __shared__ float s_best;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  if (lane == 0) { sv[warp] = best; si[warp] = bi; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w2 = 0; w2 < nw; ++w2)
      if (sv[w2] > best || (sv[w2] == best && si[w2] < bi)) { best = sv[w2]; bi = si[w2]; }
    out[r] = bi;
    s_best = best;
  }
  if (top1_prob == nullptr) return;
  __syncthreads();
  const float mx = s_best;
  float sum = 0.f;
  for (int c = threadIdx.x; c < vocab; c += blockDim.x) sum += __expf(row[c] - mx);
  sum = warp_sum(sum);
  __syncthreads();
  if (lane == 0) sv[warp] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f;
    for (int w2 = 0; w2 < nw; ++w2) tot += sv[w2];
    top1_prob[r] = 1.0f / tot;
  }
}

}  // namespace clasp
