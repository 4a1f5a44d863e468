// Measurement aid (not part of libclasp.so): cycles per tcgen05.mma (kind::f16, cta_group::1, K = 16) with
// both operands resident in shared memory, for the two ways of issuing it -- one lane that runs the whole
// issue loop (mode 0) against a converged warp in which an elected lane issues (mode 1) -- over the
// instruction shapes the layer kernel uses (M = 64 / 128 weight rows, N = 16 .. 256 activation rows), with
// 1, 2 or 4 independent accumulators and one or two issuing warps, on one CTA and on 148.
//
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -o mma_issue_bench \
//        paper_2505_24196_b200/csrc/mma_issue_bench.cu && ./mma_issue_bench
//
// Every wait is bounded; operands are zeros (the multiply's timing does not depend on the data).
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
constexpr uint32_t DESC_HI = 64u | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t desc_lo(uint32_t a) { return ((a & 0x3FFFFu) >> 4) | (1u << 16); }

// divergent form (one lane runs the loop): descriptors from two 32-bit halves
template <bool ACC>
__device__ __forceinline__ void mma_lo(uint32_t d, uint32_t a_lo, uint32_t b_lo, uint32_t idesc) {
  if (ACC)
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.eq.u32 p, 1, 1;\n\tmov.b64 da, {%1, %4};\n\tmov.b64 db, {%2, %4};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t}" ::"r"(d), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(DESC_HI));
  else
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.eq.u32 p, 1, 0;\n\tmov.b64 da, {%1, %4};\n\tmov.b64 db, {%2, %4};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t}" ::"r"(d), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(DESC_HI));
}
// converged form: the whole warp runs the loop, `pred` (one elected lane) issues
__device__ __forceinline__ void mma_el(uint32_t d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc, uint32_t pred) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %4, 0;\n\tsetp.ne.u32 q, %5, 0;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d), "l"(da), "l"(db), "r"(idesc), "r"(acc), "r"(pred));
}
__device__ __forceinline__ uint32_t elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
  return pred;
}
__device__ __forceinline__ void commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}

// MODE 0: lane 0 only (divergent), MODE 1: converged warp + elected lane
template <int M, int N, int NACC, int MODE>
__global__ void __launch_bounds__(128, 1) bench(int groups, int issuers, long long* out, int* err) {
  extern __shared__ uint8_t raw[];
  __shared__ uint64_t bar[2];
  __shared__ uint32_t tmem_base_s;
  uint8_t* base = (uint8_t*)(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
  for (int i = threadIdx.x; i < 160 * 1024 / 16; i += blockDim.x) reinterpret_cast<uint4*>(base)[i] = make_uint4(0, 0, 0, 0);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar[0])));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar[1])));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = tmem_base_s;
  const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
  const uint32_t a0 = desc_lo(smem_u32(base));
  const uint32_t b0 = desc_lo(smem_u32(base + 128 * 1024));
  constexpr uint32_t CH = M * 128 / 16;   // descriptor step of one 64-column chunk of M rows
  constexpr int WRAP = (128 * 1024) / (M * 128) / 4;   // groups of 4 chunks inside 128 KB
  if (warp >= 1 && warp <= issuers && (MODE == 1 || lane == 0)) {
    const int w = warp - 1;
    const uint32_t mybar = smem_u32(&bar[w]);
    const uint32_t d0 = tmem + (uint32_t)(w * (NACC * N <= 256 ? 256 : 0));
    long long t0 = clock64();
    if (MODE == 0) {
      int gw = 0;
      uint32_t a_lo = a0;
      for (int g = 0; g < groups; ++g) {
#pragma unroll
        for (int s = 0; s < 16; ++s) {
          const uint32_t d = d0 + (uint32_t)((s % NACC) * N);
          const uint32_t a = a_lo + (uint32_t)((s >> 2) * CH + (s & 3) * 2);
          const uint32_t b = b0 + (uint32_t)((s & 3) * 2);
          if (s < NACC) { if (g == 0) mma_lo<false>(d, a, b, idesc); else mma_lo<true>(d, a, b, idesc); }
          else mma_lo<true>(d, a, b, idesc);
        }
        a_lo += 4 * CH;
        if (++gw == WRAP) { gw = 0; a_lo = a0; }
      }
    } else {
      const uint32_t el = elect_one();
      int gw = 0;
      uint64_t da = ((uint64_t)DESC_HI << 32) | a0;
      const uint64_t da0 = da;
      const uint64_t db = ((uint64_t)DESC_HI << 32) | b0;
      for (int g = 0; g < groups; ++g) {
#pragma unroll
        for (int s = 0; s < 16; ++s) {
          const uint32_t d = d0 + (uint32_t)((s % NACC) * N);
          mma_el(d, da + (uint64_t)((s >> 2) * CH + (s & 3) * 2), db + (uint64_t)((s & 3) * 2), idesc,
                 (s < NACC && g == 0) ? 0u : 1u, el);
        }
        da += 4 * CH;
        if (++gw == WRAP) { gw = 0; da = da0; }
      }
    }
    long long t1 = clock64();
    bool done = true;
    if (MODE == 0 || elect_one()) {
      commit(mybar);
      done = false;
      for (int s = 0; s < (1 << 24); ++s) if (mbar_test(mybar, 0)) { done = true; break; }
      if (!done) atomicExch(err, 1);
    }
    if (MODE == 1) __syncwarp();
    long long t2 = clock64();
    if (lane == 0) {
      out[(blockIdx.x * 2 + w) * 2 + 0] = t1 - t0;
      out[(blockIdx.x * 2 + w) * 2 + 1] = t2 - t0;
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (*err) for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  if (warp == 0) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

long long* out; int* err;
template <int M, int N, int NACC, int MODE>
int run(int grid, int issuers) {
  const int groups = 256;
  cudaFuncSetAttribute(bench<M, N, NACC, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 162 * 1024);
  cudaMemset(out, 0, 148 * 4 * sizeof(long long));
  bench<M, N, NACC, MODE><<<grid, 128, 162 * 1024>>>(groups, issuers, out, err);
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) { printf("CUDA error %s\n", cudaGetErrorString(e)); exit(1); }
  long long h[4]; int herr = 0;
  cudaMemcpy(h, out, sizeof(h), cudaMemcpyDeviceToHost);
  cudaMemcpy(&herr, err, 4, cudaMemcpyDeviceToHost);
  if (herr) { printf("timeout flag set\n"); exit(2); }
  const double n = groups * 16.0;
  printf("%3d %3d nacc %d mode %d issuers %d grid %3d | issue %6.1f total %6.1f", M, N, NACC, MODE, issuers, grid, h[0] / n, h[1] / n);
  if (issuers == 2) printf("  [%6.1f %6.1f]", h[2] / n, h[3] / n);
  printf("\n");
  return 0;
}
template <int M, int N>
void sweep() {
  for (int grid : {1, 148}) {
    run<M, N, 1, 0>(grid, 1); run<M, N, 1, 1>(grid, 1);
    run<M, N, 2, 0>(grid, 1); run<M, N, 2, 1>(grid, 1);
    if (N * 4 <= 256) { run<M, N, 4, 0>(grid, 1); run<M, N, 4, 1>(grid, 1); }
    if (N <= 128) { run<M, N, 2, 0>(grid, 2); run<M, N, 2, 1>(grid, 2); }
  }
}
int main() {
  cudaMalloc(&out, 148 * 4 * sizeof(long long));
  cudaMalloc(&err, 4);
  cudaMemset(err, 0, 4);
  printf("cycles per MMA (K = 16); mode 0 = one lane runs the loop, mode 1 = converged warp + elected lane\n");
  sweep<64, 16>(); sweep<64, 32>(); sweep<64, 64>(); sweep<64, 128>(); sweep<64, 256>();
  sweep<128, 16>(); sweep<128, 32>(); sweep<128, 64>(); sweep<128, 128>(); sweep<128, 256>();
  return 0;
}
