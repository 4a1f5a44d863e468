// Persistent layer engine: one cooperative kernel runs a whole list of jobs (decoder
// layers, Eq. 2 steps, the LM head) so that the weights of consecutive products stream
// from HBM without a gap.
//
// One CTA per SM, twelve warps:
//   warp 0      lane 0 issues the TMA loads of weight tiles ([128 x 64] bf16, 128B swizzle)
//               into a ring of shared-memory slots.  Weight addresses never depend on
//               activations, so this warp runs ahead across products, layers and jobs and
//               only ever waits for a free slot.
//   warp 1      lane 0 issues the TMA loads of the activation operand ([BN x 64] bf16) into
//               the same slots; it waits until the product's operand has been written.
//   warp 2      lane 0 issues tcgen05.mma (M = 128 weight rows, N = BN activation rows,
//               K = 16) into one of two accumulators in tensor memory.
//   warp 3      allocates / frees tensor memory.
//   warps 4-11  "workers": read accumulators (tcgen05.ld), write split-K partial sums, and
//               run everything that is not a product: finishing a tile (sum of partials,
//               residual, norm operand, RoPE, SwiGLU, arg-max), attention over the cache,
//               and the cosine / select / write-back step of Eq. 2.
//
// Work split of a product: its (tile, k-chunk) units are numbered tile-major and CTA c takes
// the contiguous range [c U / G, (c+1) U / G)  ("stream-K"), so every CTA streams the same
// number of bytes.  A CTA writes one partial tile per tile it touches; the CTA that arrives
// last at a tile's counter adds the partials in CTA order and finishes the tile.  The split
// and every reduction order are functions of the shapes and the grid size only, never of
// the number of rows or of timing.
//
// RMSNorm is applied as  (x * w) W^T * rsqrt(mean(x^2) + eps):  the operand is x * w rounded
// to bf16, the per-row factor multiplies the product when a tile is finished.
//
// Steps that need the whole previous step are separated by a grid barrier (a counter in
// global memory).  Every wait (mbarrier, grid barrier) is bounded: when one runs out the
// CTA raises an abort flag that all other waits observe, drains and frees its tensor
// memory; the host then reports CLASP_ERR_TIMEOUT.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gemm_tc.cuh"
#include "kernels.cuh"

namespace clasp {
namespace pk {

using bf16 = __nv_bfloat16;

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int A_TILE_BYTES = BM * BK * 2;
constexpr int THREADS = 384;
constexpr int WORKERS = 256;
constexpr int WORKER_T0 = 128;  // first worker thread
constexpr int MAX_SLOTS = 12;
constexpr int ATT_KEYS = 32;
constexpr int ATT_LD = 136;     // padded row of a 128-wide K/V tile in elements (272 B)
constexpr int SCRATCH_BYTES = 2 * ATT_KEYS * ATT_LD * 2 + 2048;
constexpr int MAX_SEGS = 256;
constexpr int MAX_ROWS = 128;   // rows one launch may push through a layer

enum { JOB_LAYER = 0, JOB_HEAD = 1, JOB_SELECT = 2 };
enum { G_QKV = 0, G_O = 1, G_GU = 2, G_DOWN = 3, G_HEAD = 4 };

struct Cfg {
  int L, d, qd, kvd, hd, nq, nkv, dffn, vocab;
  float eps;
  int G;           // CTAs
  int Rcap;        // row capacity of the per-row tables (ss, cosp)
  int n_dt;        // ceil(d / 128)
  int run_len;     // cache keys per attention run (multiple of ATT_KEYS)
  int chunk_cap;   // attention partials per (row, head)
  int cnt_base[5]; // first tile counter of each product kind
  int BN;          // activation rows padded to a multiple of 16 (MMA N)
  int n_slots;
  int slot_bytes;
  int pf_max;      // weight tiles a CTA may prefetch into L2 beyond its ring while the ring is full
  // stream-K tables (ints in Params::tabs), one set per product kind
  int tab_lo[5];    // [G + 1] first unit of each CTA
  int tab_seg0[5];  // [tiles + 1] first entry of each tile in the segment list
  int tab_segc[5];  // segment list: CTA of every partial tile, tile-major, CTA order
  int segmax[5];    // partial-tile slots per CTA
};

struct Bufs {
  bf16* xn_a;      // [Rcap, d]   operand of the q/k/v product and of the LM head
  bf16* xn_m;      // [Rcap, d]   operand of the gate/up product
  bf16* attn;      // [Rcap, qd]  operand of the o product
  bf16* act;       // [Rcap, dffn] operand of the down product
  float* q;        // [Rcap, qd]  rotated, pre-scaled queries
  float* x1;       // [Rcap, d]   residual stream after attention
  float* Gbuf;     // [Rcap, d]   layer outputs of the candidate states (Eq. 2)
  float* part;     // split-K partial tiles
  float* att_acc;  // [Rcap*nq, chunk_cap, hd]
  float2* att_ml;  // [Rcap*nq, chunk_cap]
  float* ss_a;     // [n_dt, Rcap] sums of squares per column tile (attention norm / head norm)
  float* ss_m;     // [n_dt, Rcap] (MLP norm)
  float* cosp;     // [n_dt, Rcap + T, 5] partial dot products of Eq. 2
  float4* tile_best; // [head tiles, head rows] (max, index bits, sum exp, -)
  int* counters;
  const float2* rope;  // [T, hd/2] (cos, sin) of the rows' positions
};

struct Ctl {
  unsigned int bar;
  int abort;
  int status;
  int pad;
};

struct Job {
  int type, layer;
  int S, T, R;
  int C;         // cache positions visible to every row (separate own rows), or, when
                 // `uniform`, the position of the first row
  int uniform;   // 1: the rows' K/V are written into the cache and attention is causal by position
  int prep;      // 1: build the first operand from x_in when the job starts
  int dp;        // 1: the layer output feeds the Eq. 2 step below
  int row_off;   // JOB_HEAD: first row (of the previous job's rows) that goes through the head
  const float* x_in;
  long long ldx;
  float* x_out;
  long long ldo;
  const float* norm_in;    // norm weight used by `prep`
  const float* norm_mlp;
  const float* norm_next;  // norm weight of the next product's operand, or null
  const bf16* ck;
  const bf16* cv;
  bf16* ok;
  bf16* ov;
  long long own_base;
  // Eq. 2 step i
  int i, ell, diag, M;
  const float* x_i;
  const float* x_im1;
  long long x_tok_stride;
  const float* g_prev;
  float* g_next;
  float* D;
  float* margin;
  uint8_t* choice;
  const uint8_t* forced;
  float* g_final;  // written with g_next[M] when not null
  // head
  int32_t* argmax_out;
  float* top1_out;
};

struct Params {
  Cfg c;
  Bufs b;
  const Job* jobs;
  int n_jobs;
  const CUtensorMap* wmaps;  // [L*7 + 1]
  const int* tabs;
  Ctl* ctl;
  unsigned long long* trace;  // optional [G, trace_cap] time stamps (ns) of the workers' steps
  int trace_cap;
};

struct GemmDesc {
  int kind;
  int tiles, kc, dual, n_mats, K;
  int mat_tiles[3], mat_N[3];
  int map_base, bmap, cnt_base;
};

__device__ __forceinline__ GemmDesc make_desc(const Cfg& c, int kind, int layer) {
  GemmDesc g;
  g.kind = kind;
  g.dual = 0; g.n_mats = 1;
  g.mat_N[0] = g.mat_N[1] = g.mat_N[2] = 0;
  if (kind == G_QKV) {
    g.n_mats = 3; g.mat_N[0] = c.qd; g.mat_N[1] = c.kvd; g.mat_N[2] = c.kvd; g.K = c.d;
    g.map_base = layer * 7; g.bmap = 0;
  } else if (kind == G_O) {
    g.mat_N[0] = c.d; g.K = c.qd; g.map_base = layer * 7 + 3; g.bmap = 1;
  } else if (kind == G_GU) {
    g.dual = 1; g.mat_N[0] = c.dffn; g.K = c.d; g.map_base = layer * 7 + 4; g.bmap = 2;
  } else if (kind == G_DOWN) {
    g.mat_N[0] = c.d; g.K = c.dffn; g.map_base = layer * 7 + 6; g.bmap = 3;
  } else {
    g.mat_N[0] = c.vocab; g.K = c.d; g.map_base = c.L * 7; g.bmap = 4;
  }
  g.tiles = 0;
  for (int m = 0; m < 3; ++m) {
    g.mat_tiles[m] = (g.mat_N[m] + BM - 1) / BM;
    g.tiles += g.mat_tiles[m];
  }
  g.kc = (g.K + BK - 1) / BK;
  g.cnt_base = c.cnt_base[kind];
  return g;
}

// units [lo, hi) of CTA c (host-built table: lo(c) = floor(c U / G))
__device__ __forceinline__ void sk_range(const Params& p, const GemmDesc& g, int c, int& lo, int& hi) {
  const int* t = p.tabs + p.c.tab_lo[g.kind];
  lo = __ldg(t + c);
  hi = __ldg(t + c + 1);
}
// most tiles one CTA can touch in a product (bounds the partial-tile slots per CTA)
__host__ __device__ inline int sk_max_segs(long long tiles, long long kc, int G) {
  const long long U = tiles * kc;
  const long long per = (U + G - 1) / G;
  return (int)((per + kc - 1) / kc + 1);
}

// ------------------------------------------------------------------ small PTX helpers
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ int ld_volatile_i32(const int* p) {
  int v;
  asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ void worker_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ bool worker_and(bool ok) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 q, %1, 0;\n\t"
      "barrier.cta.red.and.pred p, 1, 256, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)ok)
      : "memory");
  return r != 0;
}
__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                                  uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
// x = hi + lo with hi, lo bf16: two values packed per register (first value in the low half)
__device__ __forceinline__ void split2(float x, float y, uint32_t& hi, uint32_t& lo) {
  const bf16 xh = __float2bfloat16_rn(x), yh = __float2bfloat16_rn(y);
  const bf16 xl = __float2bfloat16_rn(x - __bfloat162float(xh));
  const bf16 yl = __float2bfloat16_rn(y - __bfloat162float(yh));
  hi = (uint32_t)__bfloat16_as_ushort(xh) | ((uint32_t)__bfloat16_as_ushort(yh) << 16);
  lo = (uint32_t)__bfloat16_as_ushort(xl) | ((uint32_t)__bfloat16_as_ushort(yl) << 16);
}

// ------------------------------------------------------------------ shared state
struct Shared {
  uint64_t full[MAX_SLOTS], empty[MAX_SLOTS];
  uint64_t acc_full[2], acc_empty[2];
  uint64_t dep;
  uint32_t tmem_base;
  volatile int abort;
  int flag;                 // broadcast of a one-thread decision to the workers
  int n_seg;
  long long seg_off[MAX_SEGS];
  float rs_a[MAX_ROWS], rs_m[MAX_ROWS];
  double cosv[MAX_ROWS + 16][5];
  int choice[MAX_ROWS + 2];
};

constexpr uint32_t WAIT_FAST = 1u << 12;
constexpr uint32_t WAIT_SLOW = 1u << 22;  // x ~100 ns: gives up after roughly half a second

// Bounded mbarrier wait that also ends when any CTA raised the abort flag.
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, Ctl* ctl, Shared* sh) {
  const uint32_t b = tc::smem_u32(bar);
  for (uint32_t it = 0; it < WAIT_FAST; ++it)
    if (tc::mbar_test(b, parity)) return true;
  for (uint32_t it = 0; it < WAIT_SLOW; ++it) {
    if (tc::mbar_test(b, parity)) return true;
    if (sh->abort || ld_volatile_i32(&ctl->abort)) { sh->abort = 1; return false; }
    __nanosleep(100);
  }
  atomicExch(&ctl->status, 1);
  atomicExch(&ctl->abort, 1);
  sh->abort = 1;
  return false;
}

// Grid barrier of the worker threads (all 256 call it).  `epoch` counts barriers.  Only one
// thread fences and signals: the CTA barrier before it orders the other workers' writes first.
__device__ __forceinline__ bool grid_barrier(const Params& p, Shared* sh, unsigned& epoch, int wtid) {
  ++epoch;
  worker_sync();
  if (wtid == 0) {
    const unsigned target = epoch * (unsigned)p.c.G;
    __threadfence();
    atomicAdd(&p.ctl->bar, 1u);
    bool ok = false;
    for (uint32_t it = 0; it < (1u << 24); ++it) {
      if (ld_acquire_u32(&p.ctl->bar) >= target) { ok = true; break; }
      if ((it & 63u) == 63u) {
        if (sh->abort || ld_volatile_i32(&p.ctl->abort)) break;
        if (it > 8192u) __nanosleep(64);
      }
    }
    if (!ok) {
      if (!ld_volatile_i32(&p.ctl->abort)) atomicExch(&p.ctl->status, 1);
      atomicExch(&p.ctl->abort, 1);
      sh->abort = 1;
    }
    __threadfence();
    sh->flag = ok ? 1 : 0;
  }
  worker_sync();
  return sh->flag != 0;
}

// ------------------------------------------------------------------ producers and MMA issuer
__device__ __forceinline__ int n_gemm_phases(const Job& J) {
  return J.type == JOB_LAYER ? 4 : (J.type == JOB_HEAD ? 1 : 0);
}
__device__ __forceinline__ int gemm_kind(const Job& J, int ph) { return J.type == JOB_HEAD ? G_HEAD : ph; }

struct Ring {
  int slot;
  uint32_t round;  // how many times the ring wrapped
  __device__ __forceinline__ void advance(int n_slots) {
    if (++slot == n_slots) { slot = 0; ++round; }
  }
};

// Walks the weight tiles of this CTA in the order they are consumed: products of a job,
// jobs of the list.  Used twice by the weight producer: once for the loads into the ring
// and once, running ahead, for L2 prefetches.
struct TileIter {
  int jb, ph, q, hi, half;
  GemmDesc g;
  __device__ void reset() { jb = 0; ph = -1; q = 0; hi = 0; half = 0; }
  __device__ bool next(const Params& p, int& map_idx, int& x, int& y) {
    for (;;) {
      if (ph >= 0 && q < hi) {
        int tile = q / g.kc;
        x = (q - tile * g.kc) * BK;
        int mat = 0;
        while (mat + 1 < g.n_mats && tile >= g.mat_tiles[mat]) { tile -= g.mat_tiles[mat]; ++mat; }
        map_idx = g.map_base + mat + half;
        y = tile * BM;
        if (g.dual && half == 0) half = 1;
        else { half = 0; ++q; }
        return true;
      }
      if (jb >= p.n_jobs) return false;
      const Job& J = p.jobs[jb];
      ++ph;
      if (ph >= n_gemm_phases(J)) { ++jb; ph = -1; hi = 0; q = 0; continue; }
      g = make_desc(p.c, gemm_kind(J, ph), J.layer);
      sk_range(p, g, blockIdx.x, q, hi);
      half = 0;
    }
  }
};

__device__ void producer_a(const Params& p, Shared* sh, uint32_t ring_base) {
  const Cfg& c = p.c;
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  Ring rg{0, 0};
  TileIter ld, pf;
  ld.reset();
  pf.reset();
  int ahead = 0;        // tiles the prefetch iterator is ahead of the load iterator
  bool pf_live = c.pf_max > 0;
  int mi, x, y;
  while (ld.next(p, mi, x, y)) {
    if (ahead > 0) --ahead;
    else if (pf_live) { int a, b2, c2; pf_live = pf.next(p, a, b2, c2); }  // keep pf >= ld
    // wait for the slot; while the ring is full, keep HBM busy by prefetching later tiles into L2
    const uint32_t eb = tc::smem_u32(&sh->empty[rg.slot]);
    const uint32_t par = (rg.round & 1u) ^ 1u;
    bool ok = false;
    for (uint32_t it = 0; it < WAIT_SLOW; ++it) {
      if (tc::mbar_test(eb, par)) { ok = true; break; }
      if (pf_live && ahead < c.pf_max) {
        int pm, px, py;
        pf_live = pf.next(p, pm, px, py);
        if (pf_live) {
          asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(p.wmaps + pm),
                       "r"(px), "r"(py)
                       : "memory");
          ++ahead;
        }
        continue;
      }
      if (it > WAIT_FAST) {
        if (sh->abort || ld_volatile_i32(&p.ctl->abort)) { sh->abort = 1; return; }
        __nanosleep(100);
      }
    }
    if (!ok) {
      atomicExch(&p.ctl->status, 1);
      atomicExch(&p.ctl->abort, 1);
      sh->abort = 1;
      return;
    }
    const uint32_t full = tc::smem_u32(&sh->full[rg.slot]);
    tc::mbar_expect_tx(full, A_TILE_BYTES);
    tc::tma_load_2d(ring_base + rg.slot * c.slot_bytes, p.wmaps + mi, full, x, y, pol);
    rg.advance(c.n_slots);
  }
}

__device__ void producer_b(const Params& p, Shared* sh, uint32_t ring_base, const CUtensorMap* const* bmaps) {
  const Cfg& c = p.c;
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  Ring rg{0, 0};
  uint32_t seq = 0;
  const uint32_t b_bytes = (uint32_t)c.BN * BK * 2;
  for (int jb = 0; jb < p.n_jobs; ++jb) {
    const Job& J = p.jobs[jb];
    const int nph = n_gemm_phases(J);
    for (int ph = 0; ph < nph; ++ph, ++seq) {
      const GemmDesc g = make_desc(c, gemm_kind(J, ph), J.layer);
      // the operand of this product exists once the workers passed the barrier before it
      if (!wait_bar(&sh->dep, seq & 1u, p.ctl, sh)) return;
      fence_proxy_async();
      int lo, hi;
      sk_range(p, g, blockIdx.x, lo, hi);
      int kcx = lo % g.kc;
      for (int q = lo; q < hi; ++q) {
        if (!wait_bar(&sh->empty[rg.slot], (rg.round & 1u) ^ 1u, p.ctl, sh)) return;
        const uint32_t full = tc::smem_u32(&sh->full[rg.slot]);
        tc::mbar_expect_tx(full, b_bytes);
        tc::tma_load_2d(ring_base + rg.slot * c.slot_bytes + A_TILE_BYTES, bmaps[g.bmap], full, kcx * BK, 0, pol);
        rg.advance(c.n_slots);
        if (g.dual) {  // the "up" slot reuses the operand tile of the "gate" slot before it
          if (!wait_bar(&sh->empty[rg.slot], (rg.round & 1u) ^ 1u, p.ctl, sh)) return;
          mbar_arrive(tc::smem_u32(&sh->full[rg.slot]));
          rg.advance(c.n_slots);
        }
        if (++kcx == g.kc) kcx = 0;
      }
    }
  }
}

__device__ void mma_issuer(const Params& p, Shared* sh, uint32_t ring_base, uint32_t tmem_base) {
  const Cfg& c = p.c;
  const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(c.BN >> 3) << 17) | (8u << 24);
  Ring rg{0, 0};
  uint32_t n_acc = 0;  // accumulators handed to the workers so far
  for (int jb = 0; jb < p.n_jobs; ++jb) {
    const Job& J = p.jobs[jb];
    const int nph = n_gemm_phases(J);
    for (int ph = 0; ph < nph; ++ph) {
      const GemmDesc g = make_desc(c, gemm_kind(J, ph), J.layer);
      int lo, hi;
      sk_range(p, g, blockIdx.x, lo, hi);
      int q = lo;
      while (q < hi) {
        const int seg_end = min(hi, (q / g.kc + 1) * g.kc);
        const uint32_t buf = n_acc & 1u;
        if (!wait_bar(&sh->acc_empty[buf], ((n_acc >> 1) & 1u) ^ 1u, p.ctl, sh)) return;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t acc = tmem_base + buf * 256u;
        bool first = true;
        for (; q < seg_end; ++q) {
          if (!wait_bar(&sh->full[rg.slot], rg.round & 1u, p.ctl, sh)) return;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t sa = ring_base + rg.slot * c.slot_bytes;
          const uint64_t da = tc::make_smem_desc(sa), db = tc::make_smem_desc(sa + A_TILE_BYTES);
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk)
            tc::mma_bf16(acc, da + 2 * kk, db + 2 * kk, idesc, (first && kk == 0) ? 0u : 1u);
          const uint32_t e0 = tc::smem_u32(&sh->empty[rg.slot]);
          rg.advance(c.n_slots);
          if (g.dual) {
            if (!wait_bar(&sh->full[rg.slot], rg.round & 1u, p.ctl, sh)) return;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t da2 = tc::make_smem_desc(ring_base + rg.slot * c.slot_bytes);
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk)
              tc::mma_bf16(acc + (uint32_t)c.BN, da2 + 2 * kk, db + 2 * kk, idesc, (first && kk == 0) ? 0u : 1u);
            tc::mma_commit(e0);
            tc::mma_commit(tc::smem_u32(&sh->empty[rg.slot]));
            rg.advance(c.n_slots);
          } else {
            tc::mma_commit(e0);
          }
          first = false;
        }
        tc::mma_commit(tc::smem_u32(&sh->acc_full[buf]));
        ++n_acc;
      }
    }
  }
}

// ------------------------------------------------------------------ worker steps
struct Worker {
  const Params& p;
  Shared* sh;
  uint8_t* scratch;
  uint32_t tmem_base;
  int wtid, ww, lane;  // worker thread, worker warp (0..7), lane
  unsigned epoch;
  uint32_t n_acc;
  uint32_t n_dep;

  int n_mark;
  // time stamp of a step boundary (tracing aid; one thread per CTA)
  __device__ __forceinline__ void mark() {
    if (p.trace != nullptr && wtid == 0 && n_mark < p.trace_cap) {
      unsigned long long t;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
      p.trace[(long long)blockIdx.x * p.trace_cap + n_mark] = t;
    }
    ++n_mark;
  }
  __device__ __forceinline__ bool barrier() {
    mark();
    const bool ok = grid_barrier(p, sh, epoch, wtid);
    mark();
    return ok;
  }
  __device__ __forceinline__ void release_operand() {  // lets warp 1 load the next product's operand
    if (wtid == 0) mbar_arrive(tc::smem_u32(&sh->dep));
    ++n_dep;
  }

  // per-row factors rsqrt(mean(x^2) + eps) from the per-tile sums of squares
  __device__ void row_scales(const float* ss, int R, int row_off, float* out) {
    const Cfg& c = p.c;
    for (int r = wtid; r < R; r += WORKERS) {
      float s = 0.f;
      for (int t = 0; t < c.n_dt; ++t) s += __ldcg(ss + (long long)t * c.Rcap + row_off + r);
      out[r] = rsqrtf(s / (float)c.d + c.eps);
    }
    worker_sync();
  }

  // operand of the first product from rows the engine did not produce itself
  __device__ void prep(const Job& J) {
    const Cfg& c = p.c;
    for (int t = blockIdx.x; t < c.n_dt; t += c.G) {
      const int col = t * BM + lane * 4;
      for (int r = ww; r < J.R; r += 8) {
        float ssq = 0.f;
        if (col < c.d) {
          const float4 v = *reinterpret_cast<const float4*>(J.x_in + r * J.ldx + col);
          const float4 w = *reinterpret_cast<const float4*>(J.norm_in + col);
          ssq = v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
          __nv_bfloat162 a = __floats2bfloat162_rn(v.x * w.x, v.y * w.y);
          __nv_bfloat162 b = __floats2bfloat162_rn(v.z * w.z, v.w * w.w);
          uint2 u;
          u.x = *reinterpret_cast<uint32_t*>(&a);
          u.y = *reinterpret_cast<uint32_t*>(&b);
          *reinterpret_cast<uint2*>(p.b.xn_a + (long long)r * c.d + col) = u;
        }
        ssq = warp_sum(ssq);
        if (lane == 0) p.b.ss_a[(long long)t * c.Rcap + r] = ssq;
      }
    }
    fence_proxy_async();
  }

  // number of partial tiles of `tile` (host-built table)
  __device__ __forceinline__ int count_segments(const GemmDesc& g, int tile) const {
    const int* t = p.tabs + p.c.tab_seg0[g.kind] + tile;
    return __ldg(t + 1) - __ldg(t);
  }
  // offsets of the partial tiles of `tile`, in CTA order -> sh->seg_off (threads s < n_seg)
  __device__ void list_segments(const GemmDesc& g, int tile, int R) {
    const Cfg& c = p.c;
    const int s0 = __ldg(p.tabs + c.tab_seg0[g.kind] + tile);
    const int n = min(__ldg(p.tabs + c.tab_seg0[g.kind] + tile + 1) - s0, MAX_SEGS);
    const long long stride = (long long)(g.dual + 1) * R * BM;
    if (wtid < n) {
      const int cc = __ldg(p.tabs + c.tab_segc[g.kind] + s0 + wtid);
      const int lo = __ldg(p.tabs + c.tab_lo[g.kind] + cc);
      sh->seg_off[wtid] = ((long long)cc * c.segmax[g.kind] + (tile - lo / g.kc)) * stride;
    }
    if (wtid == 0) sh->n_seg = n;
    worker_sync();
  }

  // sum over the partial tiles (CTA order) of 4 consecutive features of two rows at once;
  // all loads of a batch are issued before the first add
  __device__ __forceinline__ void sum4x2(int plane, int r0, int r1, bool two, int R, float4& a0, float4& a1) const {
    a0 = make_float4(0.f, 0.f, 0.f, 0.f);
    a1 = a0;
    const int n = sh->n_seg;
    const float* base = p.b.part + ((long long)plane * R) * BM + lane * 4;
    for (int s0 = 0; s0 < n; s0 += 4) {
      float4 v[4], w[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        w[k] = v[k];
        if (s0 + k < n) {
          const float* q = base + sh->seg_off[s0 + k];
          v[k] = __ldcg(reinterpret_cast<const float4*>(q + (long long)r0 * BM));
          if (two) w[k] = __ldcg(reinterpret_cast<const float4*>(q + (long long)r1 * BM));
        }
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        a0.x += v[k].x; a0.y += v[k].y; a0.z += v[k].z; a0.w += v[k].w;
        a1.x += w[k].x; a1.y += w[k].y; a1.z += w[k].z; a1.w += w[k].w;
      }
    }
  }
  __device__ __forceinline__ void sum1x2(int r, int R, int f0, int f1, float& a, float& b) const {
    a = 0.f;
    b = 0.f;
    const int n = sh->n_seg;
    for (int s0 = 0; s0 < n; s0 += 4) {
      float v[4], w[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        v[k] = 0.f;
        w[k] = 0.f;
        if (s0 + k < n) {
          const float* q = p.b.part + sh->seg_off[s0 + k] + (long long)r * BM;
          v[k] = __ldcg(q + f0);
          w[k] = __ldcg(q + f1);
        }
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) { a += v[k]; b += w[k]; }
    }
  }

  // ---- finishing a tile of each product kind (all 256 workers; seg list already in shared).
  // Rows are taken two at a time per warp so that all loads of both rows are in flight together.
  __device__ __forceinline__ static uint2 pack4(float a, float b, float c2, float d2) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c2, d2);
    uint2 u;
    u.x = *reinterpret_cast<uint32_t*>(&lo);
    u.y = *reinterpret_cast<uint32_t*>(&hi);
    return u;
  }

  __device__ void finish_qkv(const Job& J, const GemmDesc& g, int tile) {
    const Cfg& c = p.c;
    int mat = 0, trow = tile;
    while (mat + 1 < g.n_mats && trow >= g.mat_tiles[mat]) { trow -= g.mat_tiles[mat]; ++mat; }
    const int half = c.hd >> 1;
    const int pidx = wtid & 63;
    const int hh = pidx / half, i = pidx % half;
    const int f0 = hh * c.hd + i, f1 = f0 + half;
    const int n0 = trow * BM + f0;  // feature inside the matrix
    if (n0 >= g.mat_N[mat]) return;
    const int head = n0 / c.hd;
    const float qscale = rsqrtf((float)c.hd) * 1.4426950408889634f;
    for (int r = wtid >> 6; r < J.R; r += 4) {
      const float rs = sh->rs_a[r];
      float2 cs = make_float2(1.f, 0.f);
      if (mat < 2) cs = p.b.rope[(long long)(r % J.T) * half + i];
      float a, b;
      sum1x2(r, J.R, f0, f1, a, b);
      a *= rs;
      b *= rs;
      const float ra = a * cs.x - b * cs.y, rb = b * cs.x + a * cs.y;
      if (mat == 0) {
        float* qr = p.b.q + (long long)r * c.qd + head * c.hd;
        qr[i] = ra * qscale;
        qr[i + half] = rb * qscale;
      } else {
        bf16* dst = (mat == 1 ? J.ok : J.ov) + (J.own_base + r) * (long long)c.kvd + head * c.hd;
        dst[i] = __float2bfloat16_rn(ra);
        dst[i + half] = __float2bfloat16_rn(rb);
      }
    }
  }

  __device__ void finish_o(const Job& J, int tile) {
    const Cfg& c = p.c;
    const int col = tile * BM + lane * 4;
    const bool cv = col < c.d;
    float4 w = make_float4(0.f, 0.f, 0.f, 0.f);
    if (cv) w = *reinterpret_cast<const float4*>(J.norm_mlp + col);
    for (int r0 = ww; r0 < J.R; r0 += 16) {
      const int r1 = r0 + 8;
      const bool two = r1 < J.R;
      float4 x0 = make_float4(0.f, 0.f, 0.f, 0.f), x1v = x0, s0, s1;
      if (cv) {
        x0 = *reinterpret_cast<const float4*>(J.x_in + r0 * J.ldx + col);
        if (two) x1v = *reinterpret_cast<const float4*>(J.x_in + r1 * J.ldx + col);
      }
      sum4x2(0, r0, r1, two, J.R, s0, s1);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (h == 1 && !two) break;
        const int r = h ? r1 : r0;
        const float4 x = h ? x1v : x0, sv = h ? s1 : s0;
        const float4 y = make_float4(x.x + sv.x, x.y + sv.y, x.z + sv.z, x.w + sv.w);
        float ssq = 0.f;
        if (cv) {
          *reinterpret_cast<float4*>(p.b.x1 + (long long)r * c.d + col) = y;
          ssq = y.x * y.x + y.y * y.y + y.z * y.z + y.w * y.w;
          *reinterpret_cast<uint2*>(p.b.xn_m + (long long)r * c.d + col) = pack4(y.x * w.x, y.y * w.y, y.z * w.z, y.w * w.w);
        }
        ssq = warp_sum(ssq);
        if (lane == 0) p.b.ss_m[(long long)tile * c.Rcap + r] = ssq;
      }
    }
    fence_proxy_async();
  }

  __device__ void finish_gu(const Job& J, int tile) {
    const Cfg& c = p.c;
    const int col = tile * BM + lane * 4;
    if (col >= c.dffn) return;
    for (int r0 = ww; r0 < J.R; r0 += 16) {
      const int r1 = r0 + 8;
      const bool two = r1 < J.R;
      float4 g0, g1, u0, u1;
      sum4x2(0, r0, r1, two, J.R, g0, g1);
      sum4x2(1, r0, r1, two, J.R, u0, u1);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (h == 1 && !two) break;
        const int r = h ? r1 : r0;
        const float rs = sh->rs_m[r];
        const float4 gg = h ? g1 : g0, uu = h ? u1 : u0;
        *reinterpret_cast<uint2*>(p.b.act + (long long)r * c.dffn + col) =
            pack4(silu_f(rs * gg.x) * (rs * uu.x), silu_f(rs * gg.y) * (rs * uu.y), silu_f(rs * gg.z) * (rs * uu.z),
                  silu_f(rs * gg.w) * (rs * uu.w));
      }
    }
    fence_proxy_async();
  }

  // skip candidate of state j (1-based) at row t: g[i-1][j-1]
  __device__ __forceinline__ const float* skip_src(const Job& J, int j, int t) const {
    return j == 1 ? J.x_im1 + t * J.x_tok_stride : J.g_prev + ((long long)(j - 1) * J.T + t) * p.c.d;
  }

  // partial dot products of Eq. 2 over the 128 columns of `tile` for row r: apply candidate y
  // (when have_apply) and skip candidate s against x_i
  __device__ __forceinline__ void cos_partials(int tile, int r, bool cv, bool have_apply, const float4& x,
                                               const float4& sk, const float4& y) {
    const Cfg& c = p.c;
    float v[5] = {0.f, 0.f, 0.f, 0.f, 0.f};
    if (cv) {
      if (have_apply) {
        v[0] = x.x * y.x + x.y * y.y + x.z * y.z + x.w * y.w;
        v[1] = y.x * y.x + y.y * y.y + y.z * y.z + y.w * y.w;
      }
      v[2] = x.x * sk.x + x.y * sk.y + x.z * sk.z + x.w * sk.w;
      v[3] = sk.x * sk.x + sk.y * sk.y + sk.z * sk.z + sk.w * sk.w;
      v[4] = x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
    }
#pragma unroll
    for (int k = 0; k < 5; ++k) v[k] = warp_sum(v[k]);
    if (lane == 0) {
      float* dst = p.b.cosp + ((long long)tile * (c.Rcap + MAX_ROWS) + r) * 5;
#pragma unroll
      for (int k = 0; k < 5; ++k) dst[k] = v[k];
    }
  }

  __device__ void finish_down(const Job& J, int tile) {
    const Cfg& c = p.c;
    const int col = tile * BM + lane * 4;
    const bool cv = col < c.d;
    const int rows = J.R + ((J.dp && J.diag) ? J.T : 0);
    const float4 z4 = make_float4(0.f, 0.f, 0.f, 0.f);
    float4 w = z4;
    if (cv && !J.dp && J.norm_next) w = *reinterpret_cast<const float4*>(J.norm_next + col);
    for (int r0 = ww; r0 < rows; r0 += 16) {
      const int r1 = r0 + 8;
      const bool two = r1 < rows;
      float4 xa[2] = {z4, z4}, xi[2] = {z4, z4}, sk[2] = {z4, z4}, sv[2];
      // residual, objective and skip-candidate rows first, then the partial tiles
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int r = h ? r1 : r0;
        if ((h == 1 && !two) || !cv) continue;
        if (r < J.R) xa[h] = *reinterpret_cast<const float4*>(p.b.x1 + (long long)r * c.d + col);
        if (J.dp) {
          const int t = r % J.T, j = r / J.T + 1;
          xi[h] = *reinterpret_cast<const float4*>(J.x_i + t * J.x_tok_stride + col);
          sk[h] = *reinterpret_cast<const float4*>(skip_src(J, j, t) + col);
        }
      }
      sum4x2(0, r0 < J.R ? r0 : 0, r1 < J.R ? r1 : 0, two, J.R, sv[0], sv[1]);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (h == 1 && !two) break;
        const int r = h ? r1 : r0;
        const bool real = r < J.R;
        const float4 y = make_float4(xa[h].x + sv[h].x, xa[h].y + sv[h].y, xa[h].z + sv[h].z, xa[h].w + sv[h].w);
        if (J.dp) {
          if (real && cv) *reinterpret_cast<float4*>(p.b.Gbuf + (long long)r * c.d + col) = y;
          cos_partials(tile, r, cv, real, xi[h], sk[h], y);
        } else {
          float ssq = 0.f;
          if (cv) {
            *reinterpret_cast<float4*>(J.x_out + r * J.ldo + col) = y;
            if (J.norm_next) {
              ssq = y.x * y.x + y.y * y.y + y.z * y.z + y.w * y.w;
              *reinterpret_cast<uint2*>(p.b.xn_a + (long long)r * c.d + col) =
                  pack4(y.x * w.x, y.y * w.y, y.z * w.z, y.w * w.w);
            }
          }
          if (J.norm_next) {
            ssq = warp_sum(ssq);
            if (lane == 0) p.b.ss_a[(long long)tile * c.Rcap + r] = ssq;
          }
        }
      }
    }
    fence_proxy_async();
  }

  // logits of one vocabulary tile: greedy token (lowest index on ties) and sum of exp
  __device__ void finish_head(const Job& J, int tile) {
    const Cfg& c = p.c;
    const int col = tile * BM + lane * 4;
    for (int r0 = ww; r0 < J.R; r0 += 16) {
      const int r1 = r0 + 8;
      const bool two = r1 < J.R;
      float4 s0, s1;
      sum4x2(0, r0, r1, two, J.R, s0, s1);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (h == 1 && !two) break;
        const int r = h ? r1 : r0;
        const float4 sv = h ? s1 : s0;
        const float rs = sh->rs_a[r];
        float v[4] = {rs * sv.x, rs * sv.y, rs * sv.z, rs * sv.w};
        float best = -INFINITY;
        int bi = 0x7fffffff;
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if (col + k < c.vocab && v[k] > best) { best = v[k]; bi = col + k; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float ov = __shfl_xor_sync(0xffffffffu, best, o);
          const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
          if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
        }
        float se = 0.f;
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if (col + k < c.vocab) se += __expf(v[k] - best);
        se = warp_sum(se);
        if (lane == 0)
          p.b.tile_best[(long long)tile * MAX_ROWS + r] = make_float4(best, __int_as_float(bi), se, 0.f);
      }
    }
  }

  // ---- accumulators of one product: partial tiles out, last arriver finishes the tile
  __device__ bool gemm_epilogue(const Job& J, int kind) {
    const Cfg& c = p.c;
    const GemmDesc g = make_desc(c, kind, J.layer);
    int lo, hi;
    sk_range(p, g, blockIdx.x, lo, hi);
    const int segmax = c.segmax[kind];
    const int planes = g.dual + 1;
    const long long stride = (long long)planes * J.R * BM;
    const int quarter = ww & 3, group = ww >> 2;
    const int ncb = (J.R + 15) >> 4;
    int q = lo;
    while (q < hi) {
      const int tile = q / g.kc;
      const int seg_end = min(hi, (tile + 1) * g.kc);
      const int seg = tile - lo / g.kc;
      const uint32_t buf = n_acc & 1u;
      bool ok = wait_bar(&sh->acc_full[buf], (n_acc >> 1) & 1u, p.ctl, sh);
      ok = worker_and(ok);
      if (!ok) return false;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      float* part = p.b.part + ((long long)blockIdx.x * segmax + seg) * stride;
      const uint32_t t_lane = tmem_base + buf * 256u + ((uint32_t)(quarter * 32) << 16);
      for (int item = group; item < planes * ncb; item += 2) {
        const int plane = item / ncb, cb = item % ncb;
        float v[16];
        tc::tmem_ld16(t_lane + (uint32_t)(plane * c.BN + cb * 16), v);
        float* dst = part + ((long long)plane * J.R + cb * 16) * BM + quarter * 32 + lane;
#pragma unroll
        for (int k = 0; k < 16; ++k)
          if (cb * 16 + k < J.R) __stcg(dst + k * BM, v[k]);
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      worker_sync();
      if (wtid == 0) {
        mbar_arrive(tc::smem_u32(&sh->acc_empty[buf]));
        const int nseg = count_segments(g, tile);
        __threadfence();  // the workers' partial tiles (ordered by the CTA barrier) before the count
        const int prev = atomicAdd(&p.b.counters[g.cnt_base + tile], 1);
        const int last = ((prev + 1) % nseg) == 0;
        if (last) __threadfence();
        sh->flag = last;
      }
      worker_sync();
      if (sh->flag) {
        list_segments(g, tile, J.R);
        if (kind == G_QKV) finish_qkv(J, g, tile);
        else if (kind == G_O) finish_o(J, tile);
        else if (kind == G_GU) finish_gu(J, tile);
        else if (kind == G_DOWN) finish_down(J, tile);
        else finish_head(J, tile);
        worker_sync();  // seg list and flag are reused by the next segment
      }
      ++n_acc;
      q = seg_end;
    }
    return true;
  }

  // ---- attention: partial softmax over one run of cache keys or one chunk of own rows
  template <int HD>
  __device__ void attention_partials(const Job& J) {
    const Cfg& c = p.c;
    constexpr int KS = HD / 16;   // k-steps of q.k
    constexpr int NB = HD / 8;    // 8-wide output blocks of p.v
    constexpr int LD = HD + 8;    // padded smem row (elements)
    bf16* k_s = reinterpret_cast<bf16*>(scratch);
    bf16* v_s = k_s + ATT_KEYS * LD;
    const int Gq = c.nq / c.nkv;
    const int P = J.R * Gq;                      // (row, query head) pairs per kv head
    const int n_pbg = (P + 127) / 128;
    const int k_tot = J.uniform ? J.C + J.T : J.C;
    const int n_runs = (k_tot + c.run_len - 1) / c.run_len;
    const int n_own = J.uniform ? 0 : (J.R + ATT_KEYS - 1) / ATT_KEYS;
    const int n_chunks = n_runs + n_own;
    const int n_items = c.nkv * n_chunks * n_pbg;
    const int g8 = lane >> 2, c4 = lane & 3;
    const long long kvld = c.kvd;
    for (int it = blockIdx.x; it < n_items; it += c.G) {
      const int pbg = it % n_pbg;
      const int chunk = (it / n_pbg) % n_chunks;
      const int kvh = it / (n_pbg * n_chunks);
      const bool own = chunk >= n_runs;
      const int p0 = (pbg * 8 + ww) * 16;        // first pair of this warp
      const bool active = p0 < P;
      // pairs of this thread: rows g8 and g8 + 8 of the warp's 16-pair block
      int rr[2], hq[2];
      bool pv[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int pp = p0 + g8 + h * 8;
        pv[h] = pp < P;
        rr[h] = pv[h] ? pp / Gq : 0;
        hq[h] = kvh * Gq + (pv[h] ? pp % Gq : 0);
      }
      uint32_t qh[KS][4], ql[KS][4];
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
#pragma unroll
          for (int kh = 0; kh < 2; ++kh) {
            float2 v = make_float2(0.f, 0.f);
            if (active && pv[h])
              v = __ldcg(reinterpret_cast<const float2*>(p.b.q + (long long)rr[h] * c.qd + hq[h] * HD + ks * 16 +
                                                          kh * 8 + c4 * 2));
            split2(v.x, v.y, qh[ks][h + kh * 2], ql[ks][h + kh * 2]);
          }
        }
      }
      float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
      float o[NB][4];
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) { o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f; }

      int key_lo, key_hi;
      const bf16 *src_k, *src_v;
      if (!own) {
        key_lo = chunk * c.run_len;
        key_hi = min(k_tot, key_lo + c.run_len);
        src_k = J.ck + kvh * HD;
        src_v = J.cv + kvh * HD;
      } else {
        key_lo = (chunk - n_runs) * ATT_KEYS;
        key_hi = min(J.R, key_lo + ATT_KEYS);
        src_k = J.ok + J.own_base * kvld + kvh * HD;
        src_v = J.ov + J.own_base * kvld + kvh * HD;
      }
      for (int key0 = key_lo; key0 < key_hi; key0 += ATT_KEYS) {
        const int nkeys = min(ATT_KEYS, key_hi - key0);
        worker_sync();  // previous tile consumed
        for (int v = wtid; v < ATT_KEYS * (HD / 8); v += WORKERS) {
          const int row = v / (HD / 8), cv = v % (HD / 8);
          uint4 kk = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
          if (row < nkeys) {
            kk = __ldcg(reinterpret_cast<const uint4*>(src_k + (long long)(key0 + row) * kvld + cv * 8));
            vv = __ldcg(reinterpret_cast<const uint4*>(src_v + (long long)(key0 + row) * kvld + cv * 8));
          }
          *reinterpret_cast<uint4*>(k_s + row * LD + cv * 8) = kk;
          *reinterpret_cast<uint4*>(v_s + row * LD + cv * 8) = vv;
        }
        worker_sync();
        if (!active) continue;
        // scores of 16 pairs x 32 keys
        float s[4][4];
#pragma unroll
        for (int nb = 0; nb < 4; ++nb) {
          s[nb][0] = s[nb][1] = s[nb][2] = s[nb][3] = 0.f;
          const bf16* kr = k_s + (nb * 8 + g8) * LD + c4 * 2;
#pragma unroll
          for (int ks = 0; ks < KS; ++ks) {
            const uint32_t b0 = *reinterpret_cast<const uint32_t*>(kr + ks * 16);
            const uint32_t b1 = *reinterpret_cast<const uint32_t*>(kr + ks * 16 + 8);
            mma_16816(s[nb], qh[ks], b0, b1);
            mma_16816(s[nb], ql[ks], b0, b1);
          }
        }
        // visibility
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nb = 0; nb < 4; ++nb) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int h = e >> 1;
            const int key = key0 + nb * 8 + c4 * 2 + (e & 1);
            bool vis = pv[h] && key < key_hi;
            if (own) vis = vis && (key / J.T == rr[h] / J.T) && key <= rr[h];
            else if (J.uniform) vis = vis && key <= J.C + rr[h];
            if (!vis) s[nb][e] = -INFINITY;
            mx[h] = fmaxf(mx[h], s[nb][e]);
          }
        }
        float corr[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
          mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
          const float m_new = fmaxf(m[h], mx[h]);
          corr[h] = (m_new == -INFINITY) ? 1.f : exp2f(m[h] - m_new);
          m[h] = m_new;
        }
        float rs[2] = {0.f, 0.f};
#pragma unroll
        for (int nb = 0; nb < 4; ++nb) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int h = e >> 1;
            const float pe = (s[nb][e] == -INFINITY) ? 0.f : exp2f(s[nb][e] - m[h]);
            s[nb][e] = pe;
            rs[h] += pe;
          }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          rs[h] += __shfl_xor_sync(0xffffffffu, rs[h], 1);
          rs[h] += __shfl_xor_sync(0xffffffffu, rs[h], 2);
          l[h] = l[h] * corr[h] + rs[h];
        }
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
          o[nb][0] *= corr[0]; o[nb][1] *= corr[0];
          o[nb][2] *= corr[1]; o[nb][3] *= corr[1];
        }
        // p.v: two k-steps of 16 keys
#pragma unroll
        for (int k2 = 0; k2 < 2; ++k2) {
          uint32_t ph[4], pl[4];
          split2(s[2 * k2][0], s[2 * k2][1], ph[0], pl[0]);
          split2(s[2 * k2][2], s[2 * k2][3], ph[1], pl[1]);
          split2(s[2 * k2 + 1][0], s[2 * k2 + 1][1], ph[2], pl[2]);
          split2(s[2 * k2 + 1][2], s[2 * k2 + 1][3], ph[3], pl[3]);
          const int mrow = k2 * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
          const int mcol = (lane >> 4) * 8;
#pragma unroll
          for (int nb = 0; nb < NB; nb += 2) {
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4_trans(tc::smem_u32(v_s + mrow * LD + nb * 8 + mcol), b0, b1, b2, b3);
            mma_16816(o[nb], ph, b0, b1);
            mma_16816(o[nb], pl, b0, b1);
            mma_16816(o[nb + 1], ph, b2, b3);
            mma_16816(o[nb + 1], pl, b2, b3);
          }
        }
      }
      if (active) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (!pv[h]) continue;
          const long long idx = ((long long)rr[h] * c.nq + hq[h]) * c.chunk_cap + chunk;
          float* pa = p.b.att_acc + idx * HD + c4 * 2;
#pragma unroll
          for (int nb = 0; nb < NB; ++nb)
            *reinterpret_cast<float2*>(pa + nb * 8) = make_float2(o[nb][2 * h], o[nb][2 * h + 1]);
          if (c4 == 0) p.b.att_ml[idx] = make_float2(m[h], l[h]);
        }
      }
    }
  }

  // chunks of one (row, head) merged; one warp per pair.  The chunk weights come from one
  // load per lane, the accumulators are fetched eight chunks at a time.
  template <int DPL>
  __device__ void attention_merge_t(const Job& J) {
    const Cfg& c = p.c;
    const int k_tot = J.uniform ? J.C + J.T : J.C;
    const int n_runs = (k_tot + c.run_len - 1) / c.run_len;
    const int n_chunks = n_runs + (J.uniform ? 0 : (J.R + ATT_KEYS - 1) / ATT_KEYS);
    const int n_pairs = J.R * c.nq;
    for (int pr = blockIdx.x * 8 + ww; pr < n_pairs; pr += c.G * 8) {
      const float2* ml = p.b.att_ml + (long long)pr * c.chunk_cap;
      float2 v0 = make_float2(-INFINITY, 0.f), v1 = v0;
      if (lane < n_chunks) v0 = __ldcg(ml + lane);
      if (lane + 32 < n_chunks) v1 = __ldcg(ml + lane + 32);
      const float mx = warp_max(fmaxf(v0.x, v1.x));
      const float w0 = v0.x == -INFINITY ? 0.f : exp2f(v0.x - mx);
      const float w1 = v1.x == -INFINITY ? 0.f : exp2f(v1.x - mx);
      const float den = warp_sum(w0 * v0.y + w1 * v1.y);
      float num[DPL];
#pragma unroll
      for (int k = 0; k < DPL; ++k) num[k] = 0.f;
      const float* acc = p.b.att_acc + (long long)pr * c.chunk_cap * c.hd + lane * DPL;
      for (int ch0 = 0; ch0 < n_chunks; ch0 += 8) {
        float a[8][DPL];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
#pragma unroll
          for (int k = 0; k < DPL; ++k) a[e][k] = 0.f;
          if (ch0 + e < n_chunks) {
            if (DPL == 4) {
              const float4 t = __ldcg(reinterpret_cast<const float4*>(acc + (long long)(ch0 + e) * c.hd));
              a[e][0] = t.x; a[e][1] = t.y; a[e][2] = t.z; a[e][3] = t.w;
            } else {
              const float2 t = __ldcg(reinterpret_cast<const float2*>(acc + (long long)(ch0 + e) * c.hd));
              a[e][0] = t.x; a[e][1] = t.y;
            }
          }
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const int ch = ch0 + e;
          const float wa = __shfl_sync(0xffffffffu, w0, ch & 31), wb = __shfl_sync(0xffffffffu, w1, ch & 31);
          const float w = ch < 32 ? wa : wb;
#pragma unroll
          for (int k = 0; k < DPL; ++k) num[k] = fmaf(w, a[e][k], num[k]);
        }
      }
      bf16* dst = p.b.attn + (long long)pr * c.hd + lane * DPL;
      const float inv = 1.0f / den;
      if (DPL == 4) {
        *reinterpret_cast<uint2*>(dst) = pack4(num[0] * inv, num[1] * inv, num[2] * inv, num[DPL - 1] * inv);
      } else {
        __nv_bfloat162 t = __floats2bfloat162_rn(num[0] * inv, num[1] * inv);
        *reinterpret_cast<__nv_bfloat162*>(dst) = t;
      }
    }
    fence_proxy_async();
  }
  __device__ void attention_merge(const Job& J) {
    if (p.c.hd == 128) attention_merge_t<4>(J);
    else attention_merge_t<2>(J);
  }

  // L2 prefetch of the cache lines this CTA's attention items will read (issued when the
  // job starts, long before the queries exist)
  __device__ void attention_prefetch(const Job& J) {
    const Cfg& c = p.c;
    const int Gq = c.nq / c.nkv;
    const int n_pbg = (J.R * Gq + 127) / 128;
    const int k_tot = J.uniform ? J.C : J.C;  // keys already in the cache
    const int n_runs_all = ((J.uniform ? J.C + J.T : J.C) + c.run_len - 1) / c.run_len;
    const int n_own = J.uniform ? 0 : (J.R + ATT_KEYS - 1) / ATT_KEYS;
    const int n_chunks = n_runs_all + n_own;
    const int n_items = c.nkv * n_chunks * n_pbg;
    const int lpr = (c.hd * 2 + 127) / 128;  // 128-byte lines per key row of one head
    for (int it = blockIdx.x; it < n_items; it += c.G) {
      const int chunk = (it / n_pbg) % n_chunks;
      const int kvh = it / (n_pbg * n_chunks);
      if (chunk >= n_runs_all) continue;
      const int key_lo = chunk * c.run_len, key_hi = min(k_tot, key_lo + c.run_len);
      const int n_lines = (key_hi - key_lo) * lpr * 2;
      for (int v = wtid; v < n_lines; v += WORKERS) {
        const int which = v & 1, ln = (v >> 1) % lpr, key = key_lo + (v >> 1) / lpr;
        const bf16* base = which ? J.cv : J.ck;
        const bf16* addr = base + (long long)key * c.kvd + kvh * c.hd + ln * 64;
        asm volatile("prefetch.global.L2 [%0];" ::"l"(addr));
      }
    }
  }

  // ---- Eq. 2 step i: decisions from the per-tile partial dot products, then write-back
  __device__ void dp_select(const Job& J) {
    const Cfg& c = p.c;
    const int rows = J.ell * J.T + (J.diag ? J.T : 0);
    const long long rstride = (long long)(c.Rcap + MAX_ROWS) * 5;
    // one warp per row: lanes take column tiles, then a fixed shuffle tree adds them up
    for (int r = ww; r < rows; r += 8) {
      double v[5] = {0.0, 0.0, 0.0, 0.0, 0.0};
      for (int t = lane; t < c.n_dt; t += 32) {
        const float* src = p.b.cosp + t * rstride + (long long)r * 5;
        float f[5];
#pragma unroll
        for (int k = 0; k < 5; ++k) f[k] = __ldcg(src + k);
#pragma unroll
        for (int k = 0; k < 5; ++k) v[k] += (double)f[k];
      }
#pragma unroll
      for (int k = 0; k < 5; ++k) {
        v[k] = warp_sum_d(v[k]);
        if (lane == 0) sh->cosv[r][k] = v[k];
      }
    }
    worker_sync();
    const int n_states = J.ell + (J.diag ? 1 : 0);
    if (wtid < n_states) {
      const int j = wtid + 1;
      double app = 0.0, skp = 0.0;
      for (int t = 0; t < J.T; ++t) {
        const double* v = sh->cosv[(j - 1) * J.T + t];
        const double nx = fmax(sqrt(v[4]), 1e-12);
        app += v[0] / (nx * fmax(sqrt(v[1]), 1e-12));
        skp += v[2] / (nx * fmax(sqrt(v[3]), 1e-12));
      }
      const float s_app = (float)(app / J.T), s_skip = (float)(skp / J.T);
      int take = 0;
      if (j <= J.ell) {
        take = s_app > s_skip;
        if (J.forced && J.forced[j] != 255) take = (J.forced[j] == 0);
      }
      sh->choice[j] = take;
      if (blockIdx.x == 0) {
        J.D[j] = take ? s_app : s_skip;
        J.choice[j] = take ? 0 : 1;
        if (J.margin && j <= J.ell) J.margin[j] = s_app - s_skip;
      }
    }
    if (blockIdx.x == 0 && wtid == 0) {
      J.D[0] = 1.0f;
      J.choice[0] = 0;
    }
    worker_sync();
    // write-back of g[i][1..n_states] and the next step's operand: one (column tile, row) per warp
    const int n_units = c.n_dt * n_states * J.T;
    for (int u = blockIdx.x * 8 + ww; u < n_units; u += c.G * 8) {
      const int tile = u % c.n_dt, r = u / c.n_dt;
      const int col = tile * BM + lane * 4;
      const int j = r / J.T + 1, t = r % J.T;
      float ssq = 0.f;
      if (col < c.d) {
        const float* src = sh->choice[j] ? p.b.Gbuf + (long long)r * c.d : skip_src(J, j, t);
        const float4 y = __ldcg(reinterpret_cast<const float4*>(src + col));
        *reinterpret_cast<float4*>(J.g_next + ((long long)j * J.T + t) * c.d + col) = y;
        if (J.g_final && j == J.M) *reinterpret_cast<float4*>(J.g_final + (long long)t * c.d + col) = y;
        if (J.norm_next) {
          const float4 w = *reinterpret_cast<const float4*>(J.norm_next + col);
          ssq = y.x * y.x + y.y * y.y + y.z * y.z + y.w * y.w;
          *reinterpret_cast<uint2*>(p.b.xn_a + (long long)r * c.d + col) = pack4(y.x * w.x, y.y * w.y, y.z * w.z, y.w * w.w);
        }
      }
      if (J.norm_next) {
        ssq = warp_sum(ssq);
        if (lane == 0) p.b.ss_a[(long long)tile * c.Rcap + r] = ssq;
      }
    }
    fence_proxy_async();
  }

  // greedy token of each head row from the per-tile results (CTA 0, one warp per row)
  __device__ void head_merge(const Job& J) {
    const Cfg& c = p.c;
    if (blockIdx.x != 0) return;
    const int n_tiles = (c.vocab + BM - 1) / BM;
    for (int r = ww; r < J.R; r += 8) {
      float best = -INFINITY;
      int bi = 0x7fffffff;
      for (int t = lane; t < n_tiles; t += 32) {
        const float4 v = __ldcg(p.b.tile_best + (long long)t * MAX_ROWS + r);
        const int vi = __float_as_int(v.y);
        if (v.x > best || (v.x == best && vi < bi)) { best = v.x; bi = vi; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
      }
      float se = 0.f;
      for (int t = lane; t < n_tiles; t += 32) {
        const float4 v = __ldcg(p.b.tile_best + (long long)t * MAX_ROWS + r);
        se += v.z * __expf(v.x - best);
      }
      se = warp_sum(se);
      if (lane == 0) {
        J.argmax_out[r] = bi;
        if (J.top1_out) J.top1_out[r] = 1.0f / se;
      }
    }
  }

  // ---- the job list
  __device__ bool run() {
    const Cfg& c = p.c;
    for (int jb = 0; jb < p.n_jobs; ++jb) {
      const Job& J = p.jobs[jb];
      if (J.type == JOB_SELECT) {
        // step with no candidate that goes through a layer (i = 1): only the diagonal state
        for (int tile = blockIdx.x; tile < c.n_dt; tile += c.G) {
          const int col = tile * BM + lane * 4;
          const bool cv = col < c.d;
          for (int r = ww; r < J.T; r += 8) {
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f), sk = x;
            if (cv) {
              x = *reinterpret_cast<const float4*>(J.x_i + r * J.x_tok_stride + col);
              sk = *reinterpret_cast<const float4*>(skip_src(J, 1, r) + col);
            }
            cos_partials(tile, r, cv, false, x, sk, x);
          }
        }
        if (!barrier()) return false;
        dp_select(J);
        if (!barrier()) return false;
        continue;
      }
      if (J.type == JOB_HEAD) {
        row_scales(p.b.ss_a, J.R, J.row_off, sh->rs_a);
        release_operand();
        if (!gemm_epilogue(J, G_HEAD)) return false;
        if (!barrier()) return false;
        head_merge(J);
        if (!barrier()) return false;
        continue;
      }
      attention_prefetch(J);
      if (J.prep) {
        prep(J);
        if (!barrier()) return false;
      }
      row_scales(p.b.ss_a, J.R, 0, sh->rs_a);
      release_operand();
      if (!gemm_epilogue(J, G_QKV)) return false;
      if (!barrier()) return false;
      if (c.hd == 128) attention_partials<128>(J);
      else attention_partials<64>(J);
      if (!barrier()) return false;
      attention_merge(J);
      if (!barrier()) return false;
      release_operand();
      if (!gemm_epilogue(J, G_O)) return false;
      if (!barrier()) return false;
      row_scales(p.b.ss_m, J.R, 0, sh->rs_m);
      release_operand();
      if (!gemm_epilogue(J, G_GU)) return false;
      if (!barrier()) return false;
      release_operand();
      if (!gemm_epilogue(J, G_DOWN)) return false;
      if (!barrier()) return false;
      if (J.dp) {
        dp_select(J);
        if (!barrier()) return false;
      }
    }
    return true;
  }
};

// ------------------------------------------------------------------ the kernel
__global__ void __launch_bounds__(THREADS, 1)
engine_kernel(const __grid_constant__ CUtensorMap map_xn_a, const __grid_constant__ CUtensorMap map_attn,
              const __grid_constant__ CUtensorMap map_xn_m, const __grid_constant__ CUtensorMap map_act,
              const __grid_constant__ CUtensorMap map_head, const __grid_constant__ Params p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ Shared sh;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint8_t* ring = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t ring_base = tc::smem_u32(ring);
  uint8_t* scratch = ring + (size_t)p.c.n_slots * p.c.slot_bytes;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.c.n_slots; ++s) {
      tc::mbar_init(tc::smem_u32(&sh.full[s]), 2);   // weight tile + operand tile
      tc::mbar_init(tc::smem_u32(&sh.empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      tc::mbar_init(tc::smem_u32(&sh.acc_full[b]), 1);
      tc::mbar_init(tc::smem_u32(&sh.acc_empty[b]), 1);
    }
    tc::mbar_init(tc::smem_u32(&sh.dep), 1);
    sh.abort = 0;
    sh.flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 3) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc::smem_u32(&sh.tmem_base)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = sh.tmem_base;

  if (warp == 0) {
    if (lane == 0) producer_a(p, &sh, ring_base);
  } else if (warp == 1) {
    if (lane == 0) {
      const CUtensorMap* bmaps[5] = {&map_xn_a, &map_attn, &map_xn_m, &map_act, &map_head};
      producer_b(p, &sh, ring_base, bmaps);
    }
  } else if (warp == 2) {
    if (lane == 0) mma_issuer(p, &sh, ring_base, tmem_base);
  } else if (warp >= 4) {
    Worker w{p, &sh, scratch, tmem_base, (int)threadIdx.x - WORKER_T0, warp - 4, lane, 0u, 0u, 0u, 0};
    w.run();
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (sh.abort) {
    // a wait gave up somewhere: let copies and MMAs still in flight land before the CTA's
    // shared and tensor memory are released
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  if (warp == 3) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

}  // namespace pk
}  // namespace clasp
