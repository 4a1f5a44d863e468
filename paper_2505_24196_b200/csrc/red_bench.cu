// Measurement aid (not part of libclasp.so): what it costs to sum per-CTA partial outputs of a product
// through global memory, the step a split of a product over K (every CTA owning a slice of d_ffn for
// gate/up AND down, so that down needs no operand from other CTAs) would add to each layer: G CTAs each
// add an [R, d] block of partial sums into one [R, d] result.
//   mode 0: 64-bit fixed-point `red.global.add.u64` per value (exact, order-independent: the form the
//           library's other cross-CTA sums use)
//   mode 1: `red.global.add.f32` per value (order-dependent rounding)
//   mode 2: `red.global.add.v4.f32` (four values per instruction)
// Timed with CUDA events around `reps` launches after one warm-up launch; the result buffer is cleared
// before each launch outside the timed region.
//
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -o red_bench \
//        paper_2505_24196_b200/csrc/red_bench.cu && ./red_bench
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#define CK(x)                                                                      \
  do {                                                                             \
    cudaError_t e_ = (x);                                                          \
    if (e_ != cudaSuccess) {                                                       \
      printf("CUDA error %s at %s:%d\n", cudaGetErrorString(e_), __FILE__, __LINE__); \
      exit(1);                                                                     \
    }                                                                              \
  } while (0)

template <int MODE>
__global__ void __launch_bounds__(256) add_partials(unsigned long long* out64, float* out32, int n, float v) {
  // every CTA walks the whole result, starting at its own offset so that the CTAs do not march in step
  const int start = (int)(((long long)blockIdx.x * n / gridDim.x) & ~3ll);
  if (MODE == 2) {
    for (int i = threadIdx.x * 4; i < n; i += blockDim.x * 4) {
      int k = start + i;
      if (k >= n) k -= n;
      asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(out32 + k), "f"(v), "f"(v), "f"(v), "f"(v)
                   : "memory");
    }
  } else {
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
      int k = start + i;
      if (k >= n) k -= n;
      if (MODE == 0) {
        const long long q = __double2ll_rn((double)v * 268435456.0);
        asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(out64 + k), "l"(q) : "memory");
      } else {
        asm volatile("red.relaxed.gpu.global.add.f32 [%0], %1;" ::"l"(out32 + k), "f"(v) : "memory");
      }
    }
  }
}

template <int MODE>
static void run(int G, int R, int d, unsigned long long* out64, float* out32) {
  const int n = R * d, reps = 20;
  cudaEvent_t a, b;
  CK(cudaEventCreate(&a));
  CK(cudaEventCreate(&b));
  float total = 0.f;
  for (int r = 0; r <= reps; ++r) {
    CK(cudaMemset(out64, 0, (size_t)n * 8));
    CK(cudaMemset(out32, 0, (size_t)n * 4));
    CK(cudaEventRecord(a));
    add_partials<MODE><<<G, 256>>>(out64, out32, n, 1.0f);
    CK(cudaEventRecord(b));
    CK(cudaEventSynchronize(b));
    float ms;
    CK(cudaEventElapsedTime(&ms, a, b));
    if (r > 0) total += ms;
  }
  // check: every value was added G times
  double got = 0;
  if (MODE == 0) {
    unsigned long long h;
    CK(cudaMemcpy(&h, out64 + n / 2, 8, cudaMemcpyDeviceToHost));
    got = (double)(long long)h / 268435456.0;
  } else {
    float h;
    CK(cudaMemcpy(&h, out32 + n / 2, 4, cudaMemcpyDeviceToHost));
    got = h;
  }
  printf("G %3d  R %3d  d %5d  mode %d : %7.2f us per launch (%.1f M values, sum check %.0f)\n", G, R, d, MODE,
         total / reps * 1e3, (double)G * n / 1e6, got);
}

int main() {
  unsigned long long* out64;
  float* out32;
  const int max_n = 128 * 8192;
  CK(cudaMalloc(&out64, (size_t)max_n * 8));
  CK(cudaMalloc(&out32, (size_t)max_n * 4));
  const int G = 148;
  for (int R : {12, 16, 96}) {
    run<0>(G, R, 4096, out64, out32);
    run<1>(G, R, 4096, out64, out32);
    run<2>(G, R, 4096, out64, out32);
  }
  run<0>(G, 32, 8192, out64, out32);
  run<2>(G, 32, 8192, out64, out32);
  return 0;
}
