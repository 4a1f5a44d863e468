// Non-greedy decoding (Sec. 4, Table 1 "Temperature = 1"): draws of softmax(logits / T) by the
// Gumbel-max rule and the accept / resample rule of speculative sampling (Leviathan et al. 2023,
// which the paper cites for losslessness), on full rows of logits the forwards leave in global memory.
//
// Random numbers: Philox4x32-10 (Salmon et al., SC'11), key = the caller's 64-bit seed, counter =
// (index, position, purpose, round).  A uniform is ((x >> 8) + 0.5) / 2^24 of the first output word:
// exact in float, never 0 or 1.  Every draw is a pure function of where it is used, so no generator
// state lives anywhere and a round can be replayed.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace clasp {
namespace smp {

enum { DRAW_DRAFT = 0, DRAW_ACCEPT = 1, DRAW_RESIDUAL = 2, DRAW_TARGET = 3 };
constexpr int THREADS = 1024;
constexpr int MAX_DRAFTS = 63;

__device__ __forceinline__ uint32_t philox_first_word(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                                      uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return c0;
}
__device__ __forceinline__ float uniform24(unsigned long long seed, uint32_t index, uint32_t pos, uint32_t purpose,
                                           uint32_t rnd) {
  const uint32_t x = philox_first_word(index, pos, purpose, rnd, (uint32_t)seed, (uint32_t)(seed >> 32));
  return ((float)(x >> 8) + 0.5f) * (1.0f / 16777216.0f);
}
__device__ __forceinline__ float gumbel(unsigned long long seed, uint32_t index, uint32_t pos, uint32_t purpose,
                                        uint32_t rnd) {
  return -logf(-logf(uniform24(seed, index, pos, purpose, rnd)));
}

// (value, index) maximum over the block, lowest index on ties; result valid in thread 0
struct Best { float v; int i; };
__device__ __forceinline__ Best better(Best a, Best b) { return (b.v > a.v || (b.v == a.v && b.i < a.i)) ? b : a; }
__device__ Best block_argmax(Best mine, float* sv, int* si) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Best other{__shfl_xor_sync(0xffffffffu, mine.v, o), __shfl_xor_sync(0xffffffffu, mine.i, o)};
    mine = better(mine, other);
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  __syncthreads();
  if (lane == 0) { sv[warp] = mine.v; si[warp] = mine.i; }
  __syncthreads();
  if (threadIdx.x == 0)
    for (int w = 0; w < nw; ++w) mine = better(mine, Best{sv[w], si[w]});
  return mine;
}
// (max, sum of exp(x - max)) of a row scaled by inv_t, as the log normaliser; valid in every thread
__device__ float block_log_norm(const float* row, int n, float inv_t, float* sv) {
  float mx = -INFINITY;
  for (int c = threadIdx.x; c < n; c += blockDim.x) mx = fmaxf(mx, row[c] * inv_t);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  __syncthreads();
  if (lane == 0) sv[warp] = mx;
  __syncthreads();
  mx = sv[0];
  for (int w = 1; w < nw; ++w) mx = fmaxf(mx, sv[w]);
  float sum = 0.f;
  for (int c = threadIdx.x; c < n; c += blockDim.x) sum += expf(row[c] * inv_t - mx);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  __syncthreads();
  if (lane == 0) sv[warp] = sum;
  __syncthreads();
  float tot = 0.f;
  for (int w = 0; w < nw; ++w) tot += sv[w];   // fixed order
  return mx + logf(tot);
}

// token_out[0] = a draw of softmax(logits / T): arg-max of logits / T + Gumbel noise, lowest index on ties
__global__ void __launch_bounds__(THREADS)
gumbel_argmax_kernel(const float* __restrict__ logits, int vocab, float inv_t, unsigned long long seed, int pos,
                     int purpose, int rnd, int32_t* __restrict__ token_out) {
  __shared__ float sv[32];
  __shared__ int si[32];
  Best mine{-INFINITY, 0x7fffffff};
  for (int c = threadIdx.x; c < vocab; c += blockDim.x) {
    const float l = logits[c];
    if (l == -INFINITY) continue;
    mine = better(mine, Best{l * inv_t + gumbel(seed, (uint32_t)c, (uint32_t)pos, (uint32_t)purpose, (uint32_t)rnd), c});
  }
  mine = block_argmax(mine, sv, si);
  if (threadIdx.x == 0) token_out[0] = mine.i;
}

struct AcceptScratch {
  float acc_prob[MAX_DRAFTS + 1];   // min(1, p_k(x_k) / q_k(x_k))
  int32_t repl[MAX_DRAFTS + 1];     // draw of norm(max(0, p_k - q_k)); entry n_drafts: draw of p at the next position
};

// Block k < n_drafts: acceptance probability of draft k and its replacement token; block n_drafts: the
// token of the position after the last draft.  p: full model's logits [n_drafts + 1, vocab], q: the draft
// model's [n_drafts, vocab]; draft k sits at position pos0 + k.
__global__ void __launch_bounds__(THREADS)
spec_rows_kernel(const float* __restrict__ p, const float* __restrict__ q, const int32_t* __restrict__ drafts, int n_drafts,
                 int vocab, float inv_t, unsigned long long seed, int pos0, int rnd, AcceptScratch* __restrict__ out) {
  __shared__ float sv[32];
  __shared__ int si[32];
  const int k = blockIdx.x;
  const float* pr = p + (long long)k * vocab;
  const int pos = pos0 + k;
  Best mine{-INFINITY, 0x7fffffff};
  if (k == n_drafts) {
    for (int c = threadIdx.x; c < vocab; c += blockDim.x) {
      const float l = pr[c];
      if (l == -INFINITY) continue;
      mine = better(mine, Best{l * inv_t + gumbel(seed, (uint32_t)c, (uint32_t)pos, DRAW_TARGET, (uint32_t)rnd), c});
    }
    mine = block_argmax(mine, sv, si);
    if (threadIdx.x == 0) out->repl[k] = mine.i;
    return;
  }
  const float* qr = q + (long long)k * vocab;
  const float zp = block_log_norm(pr, vocab, inv_t, sv);
  const float zq = block_log_norm(qr, vocab, inv_t, sv);
  for (int c = threadIdx.x; c < vocab; c += blockDim.x) {
    const float resid = expf(pr[c] * inv_t - zp) - expf(qr[c] * inv_t - zq);
    if (resid > 0.f)
      mine = better(mine, Best{logf(resid) + gumbel(seed, (uint32_t)c, (uint32_t)pos, DRAW_RESIDUAL, (uint32_t)rnd), c});
  }
  mine = block_argmax(mine, sv, si);
  if (threadIdx.x == 0) {
    const int x = drafts[k];
    const float lr = (pr[x] * inv_t - zp) - (qr[x] * inv_t - zq);
    out->acc_prob[k] = expf(fminf(lr, 0.f));
    out->repl[k] = mine.i < vocab ? mine.i : x;   // (no positive residual: p == q, the draft cannot be rejected)
  }
}

// One thread: walk the drafts, accept while u_k < acc_prob[k], then commit the replacement.
__global__ void spec_commit_kernel(const AcceptScratch* __restrict__ in, const int32_t* __restrict__ drafts, int n_drafts,
                                   unsigned long long seed, int pos0, int rnd, int32_t* __restrict__ n_accepted,
                                   int32_t* __restrict__ committed) {
  if (blockIdx.x != 0 || threadIdx.x != 0) return;
  int a = 0;
  while (a < n_drafts && uniform24(seed, 0u, (uint32_t)(pos0 + a), DRAW_ACCEPT, (uint32_t)rnd) < in->acc_prob[a]) {
    committed[a] = drafts[a];
    ++a;
  }
  committed[a] = in->repl[a];
  n_accepted[0] = a;
}

}  // namespace smp
}  // namespace clasp
