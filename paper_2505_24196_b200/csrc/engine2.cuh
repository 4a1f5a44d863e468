// Persistent layer engine: one cooperative kernel runs a whole list of jobs (decoder layers,
// Eq. 2 steps, the LM head), streaming every weight matrix from HBM exactly once and without
// a gap between consecutive products.
//
// Work split of a product y = x W^T: the output features are dealt out to the CTAs in
// contiguous ranges of 8-feature units and every CTA runs the whole reduction for its range.
// There is no split-K, so no partial sums are exchanged: the CTA that owns a feature finishes
// it (residual, norm operand, SwiGLU, cosine partials, arg-max) straight from its accumulator.
// The split and all reduction orders depend on shapes and grid size only, never on the number
// of rows or on timing.
//
// One CTA per SM, twelve warps:
//   warp 0      lane 0 issues the TMA loads of weight rows (boxes of 8..128 rows x 64 columns,
//               128B swizzle) into a ring of 1 KB shared-memory pages.  Weight addresses never
//               depend on activations: this warp runs ahead across products, layers and jobs.
//   warp 1      lane 0 loads the activation operand ([BN x 64] bf16 per 64-column chunk) next to
//               the weight rows once the CTAs that produce those columns have published them.
//   warp 2      issues tcgen05.mma: M = 128 weight rows (rows beyond the CTA's range are whatever
//               bytes follow in the ring; their accumulator lanes are never read; tiles of at most
//               64 rows use M = 64), N = BN activation rows, K = 16.  All 32 lanes walk the schedule
//               and one elected lane issues, which keeps the descriptor arithmetic warp-uniform:
//               the warp then issues as fast as the tensor pipe multiplies (23 cycles per M = 64,
//               39 per M = 128 instruction at these N).
//   warp 3      allocates / frees tensor memory.
//   warps 4-11  "workers": epilogues, attention, Eq. 2 select, arg-max.
//
// Synchronisation between CTAs is through global memory: after finishing step s of job j a
// CTA stores j+1 to flag[s][cta] (release) and adds one to the arrival counter of step s.  A
// consumer that needs a few specific producers (attention) polls their flags; one that needs
// all of them (the operand of a product, the Eq. 2 decision) polls the counter once.  RMSNorm is applied as (x * w) W^T * rsqrt(mean(x^2) +
// eps): the operand is x * w rounded to bf16, the per-row factor multiplies the product later.
//
// Every wait (mbarrier, flag) is bounded: when one runs out the CTA raises an abort flag that
// all other waits observe, drains, frees its tensor memory and returns; the host then reports
// CLASP_ERR_TIMEOUT.
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

constexpr int BK = 64;
constexpr int PAGE = 1024;            // ring granule: 8 rows x 128 B, one swizzle atom
constexpr int THREADS = 384;
constexpr int WORKERS = 256;
constexpr int WORKER_T0 = 128;
constexpr int NB = 32;                // items in flight (mbarrier pairs)
constexpr int ATT_KEYS = 32;
constexpr int SCRATCH_BYTES = 2 * ATT_KEYS * 136 * 2 + 2048;  // two padded K/V tiles + slack (>= 16 KB guard)
constexpr int TC_MIN_CTX = 4000;              // search contexts from here on take the tensor-core attention
constexpr int TC_MIN_CTX_WIDE = 1000;         // ... with 256 or more (row, query head) pairs per kv head: from here on
constexpr int TC_MIN_CTX_NARROW = 2500;       // ... with at most 64 pairs per kv head (one 64-row item): from here on
constexpr int TC_ROWS = 128;                  // (row, query head) pairs of one tensor-core attention item
constexpr int SCRATCH_TC64_BYTES = 57 * 1024; // the same with 64 rows per item: q tile 16 KB, P tile 8 KB
constexpr int SCRATCH_TC_BYTES = 81 * 1024;   // q tile 32 KB, K, V and P tiles 16 KB each (1024-aligned), 1 KB of per-row words
constexpr int MAX_ROWS = 128;         // rows one launch may push through a layer
// Rows (accumulator columns) a worker group finishes per pass; the two groups of four warps take alternate
// blocks.  4 or 8: with 4 the unrolled per-row code is half as long and 5 to 8 rows already keep both groups
// busy (measured against 8: 8B search -0.5 %, forward passes -1.7 %, 8192-key contexts -3 %; launches with
// many rows make more passes: 70B search with 32 rows +0.6 %, 128-row prefill +3 %).
constexpr int RB = 4;
constexpr int N_HEIGHTS = 4;          // distinct tile heights (TMA box heights) per weight matrix
constexpr int MAX_CTAS = 192;

enum { JOB_LAYER = 0, JOB_HEAD = 1, JOB_SELECT = 2 };
enum { G_QKV = 0, G_O = 1, G_GU = 2, G_DOWN = 3, G_HEAD = 4 };
// feature splits: which CTA owns which output features
enum { S_QKV = 0, S_D = 1, S_F = 2, S_V = 3, N_SPLITS = 4 };
// flag kinds
enum { F_PREP = 0, F_QKV, F_ATTN, F_MERGE, F_O, F_GU, F_DOWN, F_SELECT, F_HEAD, N_FLAGS };
// trace slots of a job (time stamps of the workers' step boundaries)
enum { T_START = 0, T_QKV, T_ATT_READY, T_ATT_Q, T_ATT_TILES, T_ATT_PUB, T_MERGE, T_O, T_GU, T_DOWN, T_DP_PUB,
       T_DP_ALL, T_DP_DECIDED, T_DP_DONE, T_HEAD,
       // per product ph = 0..3 (q/k/v, o, gate/up, down): first ring item of the product ready for the MMA issuer,
       // its last MMA issued, and the product's first accumulator complete (seen by the workers)
       T_MMA_FIRST = 16, T_MMA_LAST = 20, T_ACC = 24,
       // the Eq. 2 step has published the next layer's operand; the operand producer has seen the operands
       // of the q/k/v, o and gate/up products complete
       T_SEL_PUB = 28, T_B_READY = 29,
       // finer stamps inside a step while looking for a delay (workers): T_FINE + n, n < 32
       T_FINE = 32 };
constexpr int TRACE_SLOTS = 64;  // time stamps per job

struct TileDesc {      // one accumulator's worth of a CTA's feature range: rows y0.. of one weight matrix
  int f0;              // first feature in the product's feature space
  short n_rows;        // features (multiple of 8, <= 128) = height of the TMA box
  short map_local;     // matrix * N_HEIGHTS + height index
  int y0;              // first row in the matrix
};

struct Cfg {
  int L, d, qd, kvd, hd, nq, nkv, dffn, vocab;
  float eps;
  int G;
  int Rcap;            // row capacity of the per-row tables
  int run_len, chunk_cap;
  int BN;              // activation rows padded to a multiple of 16 (MMA N)
  int ring_pages;
  int att_rows;        // tensor-core attention: (row, query head) pairs per item, 64 or 128
  int att_tc;          // 1: search jobs run the attention over their cache keys on tcgen05 (kernel instantiation with
                       // TC set; the launch carries SCRATCH_TC_BYTES of worker scratch instead of SCRATCH_BYTES)
  // tables (ints / structs in Params::tabs, offsets in ints)
  int split_lo[N_SPLITS];    // [G + 1] first feature of each CTA: lo(c) = 8 floor(c units / G)
  int split_units[N_SPLITS]; // 8-feature units of each split
  int tile_idx[5];           // per product kind: [G + 1] first TileDesc of each CTA
  int tiles_off;             // TileDesc array
  int kpi[5];                // 64-column chunks per ring item
  int use3d[5];              // 1: one 3-D box {64 columns, rows, kpi chunks} per item and matrix (needs K % 64 == 0),
                             // 0: one 2-D box per chunk
  int map3d_off;             // index of the first 3-D weight map in Params::wmaps
};

struct Bufs {
  bf16* xn_a;      // [rows, d]    operand of the q/k/v product and of the LM head
  bf16* xn_m;      // [rows, d]    operand of the gate/up product
  bf16* attn;      // [rows, qd]   operand of the o product
  bf16* act;       // [rows, dffn] operand of the down product
  float* qkv;      // [rows, qd + 2 kvd] projections (norm factor applied, not rotated)
  float* x1;       // [rows, d]    residual stream after attention
  float* Gbuf;     // [rows, d]    layer outputs of the candidate states (Eq. 2)
  uint2* att_acc;  // [rows*nq, chunk_cap, hd / 2] partial attention outputs: (two bf16 values, tag) per 8 bytes
  uint4* att_ml;   // [rows*nq, chunk_cap] (running maximum, tag, sum, tag)
  long long* ss_a; // [jobs, Rcap] row sums of squares of the operand of job j's first product (attention
                   // norm / head norm), summed over the CTAs in fixed point; zero at launch
  long long* ss_m; // [jobs, Rcap] same for the operand of job j's gate/up product (MLP norm)
  long long* cosacc;  // [jobs, Rcap + MAX_ROWS, 5] dot products of Eq. 2 summed over the CTAs in fixed point
                   // (integer atomics: the sum does not depend on arrival order); zero at launch
  float4* head_best;  // [G, MAX_ROWS] (max, index bits, sum exp, -)
  int* flags;      // [N_FLAGS, G] epoch flags, followed by N_FLAGS arrival counters 32 ints apart
  const float2* rope;  // [T, hd/2] (cos, sin) of the rows' positions
};

struct Ctl {
  int abort;
  int status;
  int pad[2];
};

struct Job {
  int type, layer;
  int S, T, R;
  int C;         // cache positions visible to every row (own rows separate), or, when `uniform`,
                 // the position of the first row
  int uniform;   // 1: the rows' K/V go into the cache and attention is causal by position
  int prep;      // 1: build the first operand from x_in when the job starts
  int dp;        // 1: the layer output feeds the Eq. 2 step below
  int defer;     // 1 (with dp): the next layer does not wait for the Eq. 2 decision.  Its q/k/v product takes
                 // both candidates of every state -- operand rows [0, BN) the layer outputs (written by the
                 // down epilogue), rows [BN, 2 BN) the skip candidates -- and its epilogue keeps the chosen one
  int dual_src;  // 1: this job's q/k/v operand has those two row blocks (the previous job has `defer`)
  int row_off;   // JOB_HEAD: first row (of the previous job's rows) that goes through the head
  int kvmap;     // tensor-core attention: index in Params::kvmaps of the tensor map of this layer's key cache (values: + 1)
  int in_shift;  // first row of the previous job's operand rows / decisions that is this job's row 0 (a search that
                 // leaves out unreachable states drops leading states from one step to the next)
  int src_flag;  // step kind that publishes this job's first operand (F_PREP / F_DOWN / F_SELECT)
  int src_tgt;   // how often every CTA has published that step once the operand is complete
  int tgt[N_FLAGS];  // how often every CTA has published each step kind when this job's step is done
  const float* x_in;
  long long ldx;
  float* x_out;
  long long ldo;
  const float* norm_in;    // norm weight used by `prep`
  const float* norm_mlp;
  const float* norm_next;  // norm weight of the next product's operand, or null
  bf16* ck;                // cache of this layer (written when `uniform`)
  bf16* cv;
  // Eq. 2 step i
  int i, ell, diag, M;
  const float* x_i;
  const float* x_im1;
  long long x_tok_stride;
  long long x_im1_stride;  // row stride of x_im1 (the objective rows' stride, or d_model when x_im1 points into g)
  const float* g_prev;
  float* g_next;
  float* D;        // D, margin, choice, forced: row i of the tables, offset so that local state 1 is entry [1]
  float* margin;
  uint8_t* choice;
  float* D0;       // entry (i, 0) of the score table and of the choice table
  uint8_t* choice0;
  const uint8_t* forced;
  float* g_final;  // written with g_next[M] when not null
  // head
  int32_t* argmax_out;
  float* top1_out;
  float* logits_out;  // optional [R, vocab]: the head rows' logits (for sampling instead of arg-max)
};

struct Params {
  Cfg c;
  Bufs b;
  const Job* jobs;
  int n_jobs;
  const CUtensorMap* wmaps;  // [(L*7 + 1) * N_HEIGHTS] 2-D maps, then as many 3-D maps
  const CUtensorMap* kvmaps; // tensor-core attention: per layer job, 2-D maps {kv width, context rows} of the key and value cache
  const int* tabs;
  Ctl* ctl;
  unsigned long long* trace;  // optional [G, trace_cap] time stamps (ns)
  int trace_cap;
  uint32_t launch_tag;        // (launch number << 7): with the job number, the tag that marks a partial attention result
                              // as written by this job of this launch (never repeated over a context's life)
  uint32_t wait_fast;         // polls of a wait before it starts to sleep between polls
  uint32_t wait_slow;         // further polls (about 100 ns apart) before the wait gives up
};

// ------------------------------------------------------------------ small PTX helpers
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ int ld_acquire_i32(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_i32(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
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
__device__ __forceinline__ bool worker_or(bool v) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 q, %1, 0;\n\t"
      "barrier.cta.red.or.pred p, 1, 256, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)v)
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
// two values rounded to bf16, packed into one register (first value in the low half)
__device__ __forceinline__ uint32_t pack2(float x, float y) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
  return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ uint2 pack4(float a, float b, float c2, float d2) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c2, d2);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&lo);
  u.y = *reinterpret_cast<uint32_t*>(&hi);
  return u;
}

// r / T and r % T for the small row counts of a job (r * T < 65536) without the integer-division sequence
struct RowDiv {
  unsigned inv;
  int T;
  __device__ __forceinline__ explicit RowDiv(int t) : inv((65536u + (unsigned)t - 1u) / (unsigned)t), T(t) {}
  __device__ __forceinline__ int div(int r) const { return (int)(((unsigned)r * inv) >> 16); }
  __device__ __forceinline__ int mod(int r) const { return r - div(r) * T; }
};

// tcgen05.mma issued by the elected lane of a converged warp.  The whole warp walks the schedule, so the
// descriptor arithmetic stays warp-uniform (a loop that only one lane runs pays ~60 cycles per instruction
// for moving its operands to the uniform registers the instruction reads; measured with resident operands:
// 23 cycles per M = 64, N <= 32 multiply and 39 per M = 128 one in this form, the tensor pipe's own rate).
// Descriptor: start address and leading byte offset in the low word; 1024-byte group stride, version and
// 128B swizzle in the high word, the same for every tile.
constexpr uint32_t DESC_HI = 64u | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr) {
  return ((uint64_t)DESC_HI << 32) | (uint64_t)(((smem_addr & 0x3FFFFu) >> 4) | (1u << 16));
}
__device__ __forceinline__ uint32_t elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
  return pred;
}
template <bool ACC>
__device__ __forceinline__ void mma_el(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t el) {
  if (ACC) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.eq.u32 p, 1, 1;\n\t"
        "setp.ne.u32 q, %4, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(da), "l"(db), "r"(idesc), "r"(el));
  } else {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.eq.u32 p, 1, 0;\n\t"
        "setp.ne.u32 q, %4, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(da), "l"(db), "r"(idesc), "r"(el));
  }
}
// the four K = 16 steps of one 64-column chunk
template <bool FIRST>
__device__ __forceinline__ void mma_chunk(uint32_t acc, uint64_t da, uint64_t db, uint32_t idesc, uint32_t el) {
  mma_el<!FIRST>(acc, da, db, idesc, el);
  mma_el<true>(acc, da + 2, db + 2, idesc, el);
  mma_el<true>(acc, da + 4, db + 4, idesc, el);
  mma_el<true>(acc, da + 6, db + 6, idesc, el);
}
__device__ __forceinline__ void mma_commit_el(uint32_t bar, uint32_t el) {
  asm volatile(
      "{\n\t.reg .pred q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(bar), "r"(el)
      : "memory");
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%3, %4, %5}], [%2], %6;"
      :
      : "r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z), "l"(policy)
      : "memory");
}

// ------------------------------------------------------------------ shared state
struct Shared {
  uint64_t full[NB], empty[NB];
  uint64_t acc_full[2], acc_empty[2];
  uint64_t att_bar;         // completion of the attention's own tcgen05 multiplies
  uint64_t att_k_bar, att_v_bar;   // arrival of the attention's K / V tile
  uint32_t tmem_base;
  volatile int abort;
  uint32_t wait_fast, wait_slow;   // the launch's wait limits
  volatile int a_issued;    // ring items whose weight loads have been issued (warp 0 -> warp 1)
  int flag;                 // broadcast of a one-thread decision to the workers
  float rs[MAX_ROWS];       // per-row norm factors of the current product
  float rs_next[MAX_ROWS];  // Eq. 2 step: norm factors of the rows it hands to the next layer
  int choice[MAX_ROWS + 2];   // Eq. 2 decision per state (1: the layer output was taken)
  int choice_row[MAX_ROWS + 16];  // the same per candidate row
  int foot[NB];             // warp 0: ring pages each item in flight gives back when it retires
  alignas(16) int job_words[(sizeof(Job) + 3) / 4];  // the workers' copy of the current job descriptor (read back as a
                                                     // Job: its pointer fields need 8-byte alignment)
};
// The workers' scratch area holds either the attention K/V tiles or, during epilogues and the
// Eq. 2 step, the cross-warp reduction tables below (the two uses never overlap in time).
constexpr int RED_ROWS = MAX_ROWS + 16;
struct RedTables {
  float red[4][RED_ROWS][5];   // [lane quarter][row][value]: per-row sums of one warp
  double cosv[RED_ROWS][5];
};
static_assert(sizeof(RedTables) <= SCRATCH_BYTES, "reduction tables must fit the scratch area");

constexpr uint32_t POLL_NS = 100;      // pause between two polls of a flag or counter in global memory: the line is polled
                                       // by every CTA while the last ones still add to it (no pause: +0.7 % on the 8B search)
constexpr uint32_t WAIT_FAST = 1u << 12;
constexpr uint32_t WAIT_SLOW = 1u << 22;  // x ~100 ns: gives up after roughly half a second (the defaults of
                                          // Params::wait_fast / wait_slow)

__device__ __forceinline__ void raise_abort(Ctl* ctl, Shared* sh, bool timed_out) {
  if (timed_out && !ld_volatile_i32(&ctl->abort)) atomicExch(&ctl->status, 1);
  atomicExch(&ctl->abort, 1);
  sh->abort = 1;
}
__device__ __forceinline__ bool aborted(Ctl* ctl, Shared* sh) {
  if (sh->abort) return true;
  if (ld_volatile_i32(&ctl->abort)) { sh->abort = 1; return true; }
  return false;
}

// Bounded mbarrier wait that also ends when any CTA raised the abort flag.
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, Ctl* ctl, Shared* sh) {
  const uint32_t b = tc::smem_u32(bar);
  const uint32_t n_fast = sh->wait_fast, n_slow = sh->wait_slow;
  for (uint32_t it = 0; it < n_fast; ++it)
    if (tc::mbar_test(b, parity)) return true;
  for (uint32_t it = 0; it < n_slow; ++it) {
    if (tc::mbar_test(b, parity)) return true;
    if (aborted(ctl, sh)) return false;
    __nanosleep(100);
  }
  raise_abort(ctl, sh, true);
  return false;
}

// Bounded wait until flag >= epoch.
__device__ __forceinline__ bool wait_flag(const int* flag, int epoch, Ctl* ctl, Shared* sh) {
  const uint32_t n = 2u * sh->wait_slow;
  for (uint32_t it = 0; it < n; ++it) {
    if (ld_acquire_i32(flag) >= epoch) return true;
    __nanosleep(POLL_NS);
    if ((it & 15u) == 15u) {
      if (aborted(ctl, sh)) return false;
    }
  }
  raise_abort(ctl, sh, true);
  return false;
}

// Bounded wait until all G CTAs have published step `kind` `tgt` times.
__device__ __forceinline__ bool wait_count(const Params& p, int kind, int tgt, Shared* sh) {
  const int* cnt = p.b.flags + N_FLAGS * p.c.G + kind * 32;
  return wait_flag(cnt, tgt * p.c.G, p.ctl, sh);
}

// ------------------------------------------------------------------ the schedule every role walks
__device__ __forceinline__ int n_gemm_phases(const Job& J) {
  return J.type == JOB_LAYER ? 4 : (J.type == JOB_HEAD ? 1 : 0);
}
__device__ __forceinline__ int gemm_kind(const Job& J, int ph) { return J.type == JOB_HEAD ? G_HEAD : ph; }
__device__ __forceinline__ int kind_K(const Cfg& c, int kind) {
  return kind == G_O ? c.qd : (kind == G_DOWN ? c.dffn : c.d);
}
__device__ __forceinline__ int kind_map_base(const Cfg& c, int kind, int layer) {
  const int m = kind == G_QKV ? 0 : (kind == G_O ? 3 : (kind == G_GU ? 4 : (kind == G_DOWN ? 6 : 0)));
  return ((kind == G_HEAD ? c.L * 7 : layer * 7) + m) * N_HEIGHTS;
}

struct Phase {   // one product of one job, as seen by this CTA
  int kind, dual, kc, kpi, n_groups;  // chunks, chunks per item, items per tile
  int bmul;                           // operand row blocks of BN rows (2 for a q/k/v product over both candidates)
  int tile0, n_tiles;                 // this CTA's TileDesc range
  int map_base;
  int g0;                             // chunk group this CTA starts its reduction at: CTAs walk the
                                      // columns of their weight rows at staggered offsets so that the
                                      // grid's reads spread over all HBM channels at any moment
  __device__ __forceinline__ void init(const Params& p, const Job& J, int ph) {
    const Cfg& c = p.c;
    kind = gemm_kind(J, ph);
    dual = kind == G_GU;
    kc = (kind_K(c, kind) + BK - 1) / BK;
    kpi = c.kpi[kind];
    n_groups = (kc + kpi - 1) / kpi;
    bmul = (kind == G_QKV && J.dual_src) ? 2 : 1;
    const int* ti = p.tabs + c.tile_idx[kind] + blockIdx.x;
    tile0 = __ldg(ti);
    n_tiles = __ldg(ti + 1) - tile0;
    map_base = kind_map_base(c, kind, J.layer);
    g0 = (int)(((long long)blockIdx.x * n_groups) / c.G);
  }
  __device__ __forceinline__ int group_at(int gi) const {
    const int g = g0 + gi;
    return g >= n_groups ? g - n_groups : g;
  }
};

// ring placement of items: identical arithmetic in the three pipeline roles
struct RingPos {
  int pos;        // next free page
  uint32_t item;  // items placed so far
  // returns the page the item starts at and, through `footprint`, the pages it takes out of the ring
  // (its own plus the unused tail when it wraps)
  __device__ __forceinline__ int place(int pages, int ring_pages, int& footprint) {
    footprint = pages;
    if (pos + pages > ring_pages) { footprint += ring_pages - pos; pos = 0; }
    const int at = pos;
    pos += pages;
    ++item;
    return at;
  }
};

// Position in the sequence of ring items of a launch: (job, product, tile, chunk group).
struct ItemCursor {
  int jb, ph, nph, t, gi;
  bool valid;
  Phase P;
  TileDesc td;
  __device__ __forceinline__ void settle(const Params& p, const TileDesc* tiles, bool new_tile) {
    for (;;) {
      if (jb >= p.n_jobs) { valid = false; return; }
      if (ph >= nph) {
        ++jb; ph = 0; t = 0; gi = 0; new_tile = true;
        if (jb < p.n_jobs) {
          nph = n_gemm_phases(p.jobs[jb]);
          if (nph > 0) P.init(p, p.jobs[jb], 0);
        }
        continue;
      }
      if (t >= P.n_tiles) {
        ++ph; t = 0; gi = 0; new_tile = true;
        if (ph < nph) P.init(p, p.jobs[jb], ph);
        continue;
      }
      if (gi >= P.n_groups) { ++t; gi = 0; new_tile = true; continue; }
      if (new_tile) td = tiles[P.tile0 + t];
      return;
    }
  }
  __device__ __forceinline__ void first(const Params& p, const TileDesc* tiles) {
    jb = 0; ph = 0; t = 0; gi = 0; valid = true;
    nph = n_gemm_phases(p.jobs[0]);
    if (nph > 0) P.init(p, p.jobs[0], 0);
    settle(p, tiles, true);
  }
  __device__ __forceinline__ int a_pages() const { return td.n_rows >> 3; }
  __device__ __forceinline__ int w_pages() const { return (P.dual + 1) * (td.n_rows >> 3); }  // weight pages of one chunk
  __device__ __forceinline__ int k0() const { return P.group_at(gi) * P.kpi; }
  __device__ __forceinline__ int nk() const { return min(P.kc, k0() + P.kpi) - k0(); }
  __device__ __forceinline__ void next(const Params& p, const TileDesc* tiles) {
    ++gi;
    settle(p, tiles, false);
  }
};

// Ring item of tile (rows n) of a product: kpi chunks of weight rows, then kpi operand tiles:
//   [W chunk 0 | W chunk 1 | ...]  each (dual + 1) * n / 8 pages (gate rows, then up rows)
//   [X chunk 0 | X chunk 1 | ...]  each BN / 8 pages
// Warp 0, all lanes: every lane walks the schedule; lane 0 does the ring bookkeeping.  With 3-D
// maps one box brings all chunks of an item (a thread can issue a TMA only every ~150 cycles, so
// the number of boxes, not their size, bounds the rate); otherwise lane k issues chunk k.
__device__ void producer_a(const Params& p, Shared* sh, uint32_t ring_base, int lane) {
  const Cfg& c = p.c;
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  const TileDesc* tiles = reinterpret_cast<const TileDesc*>(p.tabs + c.tiles_off);
  RingPos rp{0, 0};
  int used = 0;
  uint32_t tail = 0;
  int* foot = sh->foot;
  const int b_pages = (c.BN * BK * 2) / PAGE;
  ItemCursor L;
  L.first(p, tiles);
  while (L.valid) {
    const Phase& P = L.P;
    const TileDesc& td = L.td;
    const bool d3 = c.use3d[P.kind] != 0;
    const int a_pages = L.a_pages(), w_pages = L.w_pages();
    const int pages = P.kpi * (w_pages + P.bmul * b_pages);
    // make room: items leave the ring in the order they entered it
    int fp;
    RingPos probe = rp;
    probe.place(pages, c.ring_pages, fp);
    while (used + fp > c.ring_pages || rp.item - tail >= (uint32_t)NB) {
      const bool ok = wait_bar(&sh->empty[tail % NB], (tail / NB) & 1u, p.ctl, sh);
      if (!__all_sync(0xffffffffu, ok)) return;
      used -= foot[tail % NB];
      ++tail;
    }
    const uint32_t it = rp.item;
    const int at = rp.place(pages, c.ring_pages, fp);
    __syncwarp();
    if (lane == 0) foot[it % NB] = fp;
    used += fp;
    const int k0 = L.k0(), nk = L.nk();
    const uint32_t full = tc::smem_u32(&sh->full[it % NB]);
    const uint32_t dst = ring_base + (uint32_t)at * PAGE;
    const CUtensorMap* map2 = p.wmaps + P.map_base + td.map_local;
    if (d3) {  // boxes always span kpi chunks; chunks beyond K arrive as zeros
      if (lane == 0) {
        tc::mbar_expect_tx(full, (uint32_t)(P.kpi * w_pages * PAGE));
        tma_load_3d(dst, map2 + c.map3d_off, full, 0, td.y0, k0, pol);
      }
    } else {
      if (lane == 0) tc::mbar_expect_tx(full, (uint32_t)(nk * w_pages * PAGE));
      __syncwarp();
      const int kk = lane >> 1, half = lane & 1;     // lane -> (chunk, gate / up)
      if (kk < nk && half <= P.dual)
        tc::tma_load_2d(dst + (uint32_t)((kk * w_pages + half * a_pages) * PAGE), map2 + half * N_HEIGHTS, full,
                        (k0 + kk) * BK, td.y0, pol);
    }
    __syncwarp();
    if (lane == 0) sh->a_issued = (int)(it + 1);
    L.next(p, tiles);
  }
}

template <bool TR>
__device__ __forceinline__ void issuer_mark(const Params& p, int jb, int slot) {
  if (!TR) return;
  const int idx = jb * TRACE_SLOTS + slot;
  if (p.trace != nullptr && idx < p.trace_cap) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    p.trace[(long long)blockIdx.x * p.trace_cap + idx] = t;
  }
}

// Warp 1, all lanes: lane k issues the operand tile of an item's chunk k.
template <bool TR>
__device__ void producer_b(const Params& p, Shared* sh, uint32_t ring_base, const CUtensorMap* const* bmaps,
                           const CUtensorMap* const* bmaps3, int lane) {
  const Cfg& c = p.c;
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  const TileDesc* tiles = reinterpret_cast<const TileDesc*>(p.tabs + c.tiles_off);
  RingPos rp{0, 0};
  const int b_pages = (c.BN * BK * 2) / PAGE;
  const uint32_t b_bytes = (uint32_t)c.BN * BK * 2;
  for (int jb = 0; jb < p.n_jobs; ++jb) {
    const Job& J = p.jobs[jb];
    const int nph = n_gemm_phases(J);
    for (int ph = 0; ph < nph; ++ph) {
      Phase P;
      P.init(p, J, ph);
      if (P.n_tiles == 0) continue;
      // the operand exists once every CTA has published the step that writes it
      int fkind, tgt, bmap;
      const int row0 = P.kind == G_QKV ? J.in_shift : 0;   // first operand row of this job in the rows' buffer
      if (P.kind == G_QKV) { fkind = J.src_flag; tgt = J.src_tgt; bmap = J.dual_src ? 5 : 0; }
      else if (P.kind == G_O) { fkind = F_MERGE; tgt = J.tgt[F_MERGE]; bmap = 1; }
      else if (P.kind == G_GU) { fkind = F_O; tgt = J.tgt[F_O]; bmap = 2; }
      else if (P.kind == G_DOWN) { fkind = F_GU; tgt = J.tgt[F_GU]; bmap = 3; }
      else { fkind = J.src_flag; tgt = J.src_tgt; bmap = 4; }
      {
        bool ok = true;
        if (lane == 0) ok = wait_count(p, fkind, tgt, sh);
        if (!__all_sync(0xffffffffu, ok)) return;
        if (lane == 0 && P.kind < 3) issuer_mark<TR>(p, jb, T_B_READY + P.kind);
      }
      fence_proxy_async();  // the producers' ordinary stores before this warp's TMA reads
      const bool d3 = c.use3d[P.kind] != 0;
      for (int t = 0; t < P.n_tiles; ++t) {
        const TileDesc td = tiles[P.tile0 + t];
        const int w_pages = (P.dual + 1) * (td.n_rows >> 3);
        const int pages = P.kpi * (w_pages + P.bmul * b_pages);
        const uint32_t pb_bytes = (uint32_t)P.bmul * b_bytes;   // operand tile of one chunk
        for (int gi = 0; gi < P.n_groups; ++gi) {
          int fp;
          const uint32_t it = rp.item;
          const int at = rp.place(pages, c.ring_pages, fp);
          // the weight producer has made room for this item
          bool ok = false;
          const uint32_t n_fast = sh->wait_fast, n_slow = sh->wait_slow;
          for (uint32_t w = 0; w < n_slow; ++w) {
            if ((uint32_t)sh->a_issued > it) { ok = true; break; }
            if (w > n_fast) {
              if (aborted(p.ctl, sh)) break;
              __nanosleep(100);
            }
          }
          if (!ok && !aborted(p.ctl, sh)) raise_abort(p.ctl, sh, true);
          if (!__all_sync(0xffffffffu, ok)) return;
          const int k0 = P.group_at(gi) * P.kpi, nk = min(P.kc, k0 + P.kpi) - k0;
          const uint32_t full = tc::smem_u32(&sh->full[it % NB]);
          const uint32_t dst = ring_base + (uint32_t)(at + P.kpi * w_pages) * PAGE;
          if (d3) {
            if (lane == 0) {
              tc::mbar_expect_tx(full, (uint32_t)P.kpi * pb_bytes);
              tma_load_3d(dst, bmaps3[bmap], full, 0, row0, k0, pol);
            }
          } else {
            if (lane == 0) tc::mbar_expect_tx(full, (uint32_t)nk * pb_bytes);
            __syncwarp();
            if (lane < nk) tc::tma_load_2d(dst + (uint32_t)lane * pb_bytes, bmaps[bmap], full, (k0 + lane) * BK, row0, pol);
          }
          __syncwarp();
        }
      }
    }
  }
}

// MMA issuer (warp 2, all lanes converged, one elected lane issues): adds the ring items of each tile up in
// the tile's accumulator; buffer b holds it at column b * 256 (gate at +0, up at +BN).
template <bool TR>
__device__ void mma_issuer(const Params& p, Shared* sh, uint32_t ring_base, uint32_t tmem_base, int lane) {
  const Cfg& c = p.c;
  const uint32_t idesc0 = (1u << 4) | (1u << 7) | (1u << 10);
  const TileDesc* tiles = reinterpret_cast<const TileDesc*>(p.tabs + c.tiles_off);
  RingPos rp{0, 0};
  const int b_pages = (c.BN * BK * 2) / PAGE;
  uint32_t n_acc = 0;
  const uint32_t el = elect_one();
  for (int jb = 0; jb < p.n_jobs; ++jb) {
    const Job& J = p.jobs[jb];
    const int nph = n_gemm_phases(J);
    for (int ph = 0; ph < nph; ++ph) {
      Phase P;
      P.init(p, J, ph);
      for (int t = 0; t < P.n_tiles; ++t) {
        const TileDesc td = tiles[P.tile0 + t];
        const int a_pages = td.n_rows >> 3;
        const int w_pages = (P.dual + 1) * a_pages;
        const int pages = P.kpi * (w_pages + P.bmul * b_pages);
        // tiles of at most 64 weight rows take the M = 64 shape: the multiply reads half the operand
        // rows from shared memory (row r of its accumulator sits in lane 32 (r / 16) + r % 16)
        const uint32_t idesc = idesc0 | ((uint32_t)((P.bmul * c.BN) >> 3) << 17) | ((td.n_rows <= 64 ? 4u : 8u) << 24);
        const uint32_t buf = n_acc & 1u;
        if (!__all_sync(0xffffffffu, wait_bar(&sh->acc_empty[buf], ((n_acc >> 1) & 1u) ^ 1u, p.ctl, sh))) return;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t acc = tmem_base + buf * 256u;
        const uint32_t acc2 = acc + (uint32_t)c.BN;
        const uint64_t up_lo = (uint64_t)(a_pages * (PAGE / 16));              // gate rows -> up rows
        const uint64_t w_lo = (uint64_t)(w_pages * (PAGE / 16));               // weights of one chunk
        const uint64_t x_lo = (uint64_t)(P.bmul * b_pages * (PAGE / 16));      // operand tile of one chunk
        const uint64_t x0_lo = (uint64_t)P.kpi * w_lo;                         // first weight chunk -> first operand tile
        for (int gi = 0; gi < P.n_groups; ++gi) {
          int fp;
          const uint32_t it = rp.item;
          const int at = rp.place(pages, c.ring_pages, fp);
          if (!__all_sync(0xffffffffu, wait_bar(&sh->full[it % NB], (it / NB) & 1u, p.ctl, sh))) return;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          if (t == 0 && gi == 0 && lane == 0) issuer_mark<TR>(p, jb, T_MMA_FIRST + ph);
          const int k0 = P.group_at(gi) * P.kpi;
          const int nk = min(P.kc, k0 + P.kpi) - k0;
          uint64_t da = make_desc(ring_base + (uint32_t)at * PAGE);
          uint64_t db = da + x0_lo;
          int k = 0;
          if (gi == 0) {  // the first item of the tile overwrites the accumulator
            mma_chunk<true>(acc, da, db, idesc, el);
            if (P.dual) mma_chunk<true>(acc2, da + up_lo, db, idesc, el);
            da += w_lo;
            db += x_lo;
            k = 1;
          }
          if (P.dual) {
            for (; k < nk; ++k) {
              mma_chunk<false>(acc, da, db, idesc, el);
              mma_chunk<false>(acc2, da + up_lo, db, idesc, el);
              da += w_lo;
              db += x_lo;
            }
          } else {
            for (; k < nk; ++k) {
              mma_chunk<false>(acc, da, db, idesc, el);
              da += w_lo;
              db += x_lo;
            }
          }
          mma_commit_el(tc::smem_u32(&sh->empty[it % NB]), el);
        }
        mma_commit_el(tc::smem_u32(&sh->acc_full[buf]), el);
        if (lane == 0 && t == P.n_tiles - 1) issuer_mark<TR>(p, jb, T_MMA_LAST + ph);
        ++n_acc;
      }
    }
  }
}

// ------------------------------------------------------------------ worker steps
// TR: the step stamps are compiled in; HD: the model's head dimension (64 or 128).  The kernel is
// sensitive to its code size, so an instantiation carries neither stamps it does not take nor the
// attention code of the other head dimension; TC: the instantiation for searches over long contexts (tensor-core
// attention over the cache keys, Eq. 2 write-back dealt to all threads); it is launched for nothing else.
template <bool TR, int HD, bool TC>
struct Worker {
  const Params& p;
  Shared* sh;
  uint8_t* scratch;
  uint32_t tmem_base;
  int wtid, ww, lane;
  uint32_t n_acc;
  int n_mark;
  uint32_t att_phase = 0;   // parity of att_bar's next completion
  uint32_t att_kph = 0, att_vph = 0;   // the same for the K / V tile barriers (worker warp 4)

  // time stamp of step `slot` (one of the T_* above) of the current job
  __device__ __forceinline__ void mark(int slot) {
    if (!TR) return;
    const int idx = n_mark * TRACE_SLOTS + slot;
    if (p.trace != nullptr && wtid == 0 && idx < p.trace_cap) {
      unsigned long long t;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
      p.trace[(long long)blockIdx.x * p.trace_cap + idx] = t;
    }
  }

  // all workers' stores of this step become visible, then the CTA's flag of `kind` says so
  __device__ __forceinline__ void publish(int kind, int epoch) {
    worker_sync();
    if (wtid == 0) {
      __threadfence();  // the workers' stores (ordered before this thread by the CTA barrier) first
      int* flag = p.b.flags + kind * p.c.G + blockIdx.x;
      int* cnt = p.b.flags + N_FLAGS * p.c.G + kind * 32;
      asm volatile("st.relaxed.gpu.global.s32 [%0], %1;" ::"l"(flag), "r"(epoch) : "memory");
      asm volatile("red.relaxed.gpu.global.add.s32 [%0], 1;" ::"l"(cnt) : "memory");
    }
  }
  // every CTA has published step `kind` tgt times: one thread polls, the others wait for it
  __device__ bool wait_all(int kind, int tgt) {
    bool ok = true;
    if (wtid == 0) ok = wait_count(p, kind, tgt, sh);
    return worker_and(ok);
  }
  // wait for flags [first, first + n) of `kind`: one flag per thread
  __device__ bool wait_flags(int kind, int first, int n, int epoch) {
    bool ok = true;
    for (int k = wtid; k < n; k += WORKERS) ok = wait_flag(p.b.flags + kind * p.c.G + first + k, epoch, p.ctl, sh) && ok;
    return worker_and(ok);
  }

  // Feature (row of an accumulator of n rows) that thread `lane` of lane quarter `quarter` owns, or -1:
  // an M = 128 accumulator has row r in lane r, an M = 64 one (n <= 64) in lane 32 (r / 16) + r % 16.
  __device__ __forceinline__ static int feat_local(int n, int quarter, int lane) {
    const int fl = n <= 64 ? (lane < 16 ? quarter * 16 + lane : n) : quarter * 32 + lane;
    return fl < n ? fl : -1;
  }
  __device__ __forceinline__ const int* split_lo(int split) const { return p.tabs + p.c.split_lo[split]; }
  __device__ __forceinline__ RedTables* tables() const { return reinterpret_cast<RedTables*>(scratch); }

  // fixed-point scale of the sums of squares (2^24: sums up to 5e11, resolution 6e-8)
  static constexpr double SS_FIX = 16777216.0;
  __device__ __forceinline__ static void ss_add(long long* dst, float v) {
    const long long q = __double2ll_rn((double)v * SS_FIX);
    asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(dst), "l"(q) : "memory");
  }
  // Sums of several values over the warp with N - 1 + log2(32 / N) shuffles, independent within a stage,
  // instead of N five-step butterflies.
  // Same for N = 4, 8 or 16 values: every lane l returns the total of v[l & (N - 1)].
  template <int N>
  __device__ __forceinline__ static float warp_reduce(float (&v)[N], int lane) {
#pragma unroll
    for (int w = N / 2; w >= 1; w >>= 1) {
      const bool up = (lane & w) != 0;
#pragma unroll
      for (int i = 0; i < w; ++i) {
        const float send = up ? v[i] : v[i + w];
        const float keep = up ? v[i + w] : v[i];
        v[i] = keep + __shfl_xor_sync(0xffffffffu, send, w);
      }
    }
    float t = v[0];
#pragma unroll
    for (int o = N; o < 32; o <<= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    return t;
  }
  // RB accumulator columns of this thread's lane
  __device__ __forceinline__ static void tmem_ld_rb(uint32_t taddr, float (&v)[RB]) {
    uint32_t r[RB];
    if constexpr (RB == 8) {
      asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                   : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                   : "r"(taddr));
    } else {
      static_assert(RB == 4 || RB == 8, "row block of 4 or 8 accumulator columns");
      asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
                   : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                   : "r"(taddr));
    }
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < RB; ++i) v[i] = __uint_as_float(r[i]);
  }

  // per-row factors rsqrt(mean(x^2) + eps) from the accumulated sums of squares
  __device__ void row_scales(const long long* ss, int R, int row_off) {
    const Cfg& c = p.c;
    for (int r = wtid; r < R; r += WORKERS) {
      const double s = (double)__ldcg(ss + row_off + r) * (1.0 / SS_FIX);
      sh->rs[r] = rsqrtf((float)s / (float)c.d + c.eps);
    }
    worker_sync();
  }

  // operand of the first product from rows the engine did not produce itself: this CTA's
  // slice of the d features
  __device__ void prep(const Job& J, int epoch) {
    const Cfg& c = p.c;
    const int f_lo = __ldg(split_lo(S_D) + blockIdx.x), f_hi = __ldg(split_lo(S_D) + blockIdx.x + 1);
    const int n4 = (f_hi - f_lo) >> 2;
    for (int r = ww; r < J.R; r += 8) {
      float ssq = 0.f;
      for (int q = lane; q < n4; q += 32) {
        const int col = f_lo + q * 4;
        const float4 v = *reinterpret_cast<const float4*>(J.x_in + r * J.ldx + col);
        const float4 w = *reinterpret_cast<const float4*>(J.norm_in + col);
        ssq += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        *reinterpret_cast<uint2*>(p.b.xn_a + (long long)r * c.d + col) = pack4(v.x * w.x, v.y * w.y, v.z * w.z, v.w * w.w);
      }
      ssq = warp_sum(ssq);
      if (lane == 0 && n4 > 0) ss_add(p.b.ss_a + (long long)(epoch - 1) * c.Rcap + r, ssq);
    }
    publish(F_PREP, epoch);
  }

  // ---- epilogue of one accumulator: tile td of product P.kind.
  // Thread (quarter q, lane) owns feature td.f0 + 32 q + lane; the two warps of a quarter take
  // alternating blocks of RB rows (accumulator columns).  Per-row sums over the CTA's features
  // (sums of squares, cosine partials, arg-max) go through RedTables: one entry per (quarter, row).
  // For the down product of an Eq. 2 job the thread's layer outputs (keep_y) and skip candidates
  // (keep_s) of its first block of RB rows stay in registers for dp_step.
  __device__ bool epilogue(const Job& J, int jb, const Phase& P, const TileDesc& td, int tile_no, float (&keep_y)[RB],
                           float (&keep_s)[RB]) {
    const Cfg& c = p.c;
    RedTables* T = tables();
    const int quarter = ww & 3, group = ww >> 2;
    const int fl = feat_local(td.n_rows, quarter, lane);
    const bool fv = fl >= 0;
    const int f = td.f0 + fl;
    const bool dpd = P.kind == G_DOWN && J.dp;
    const int rows_all = J.R + ((dpd && J.diag) ? J.T : 0);   // Eq. 2: plus the rows of the diagonal state
    const int ncb = (J.R + RB - 1) / RB;
    const bool resid = P.kind == G_O || P.kind == G_DOWN;
    const RowDiv rd(J.T);
    // Eq. 2: objective row and skip candidate of every row of the first block, fetched early
    float xi[RB];
    if (dpd) {
#pragma unroll
      for (int k = 0; k < RB; ++k) {
        const int r = group * RB + k;
        xi[k] = 0.f;
        keep_s[k] = 0.f;
        keep_y[k] = 0.f;
        if (fv && r < rows_all) {
          xi[k] = __ldg(J.x_i + rd.mod(r) * J.x_tok_stride + f);
          keep_s[k] = __ldcg(skip_row(J, r) + f);
        }
      }
      if (J.defer && fv) {   // the skip candidates' rows of the next layer's operand
        const float wq = __ldg(J.norm_next + f);
#pragma unroll
        for (int k = 0; k < RB; ++k) {
          const int r = group * RB + k;
          if (r < rows_all) p.b.xn_a[(long long)(c.BN + r) * c.d + f] = __float2bfloat16_rn(keep_s[k] * wq);
        }
        for (int cb = group + 2; cb * RB < rows_all; cb += 2) {
#pragma unroll
          for (int k = 0; k < RB; ++k) {
            const int r = cb * RB + k;
            if (r < rows_all)
              p.b.xn_a[(long long)(c.BN + r) * c.d + f] =
                  __float2bfloat16_rn(__ldcg(skip_row(J, r) + f) * wq);
          }
        }
      }
    }
    // residual rows of this thread's first two blocks are fetched before the accumulator is ready (a load
    // from L2 costs 1 - 2 us here; with twelve rows no block is left that would wait for one)
    float res[RB], res_n[RB];
#pragma unroll
    for (int k = 0; k < RB; ++k) { res[k] = 0.f; res_n[k] = 0.f; }
    if (resid && fv) {
#pragma unroll
      for (int k = 0; k < RB; ++k) {
        const int r = group * RB + k, r2 = r + 2 * RB;
        if (r < J.R) res[k] = P.kind == G_O ? __ldcg(J.x_in + r * J.ldx + f) : __ldcg(p.b.x1 + (long long)r * c.d + f);
        if (r2 < J.R) res_n[k] = P.kind == G_O ? __ldcg(J.x_in + r2 * J.ldx + f) : __ldcg(p.b.x1 + (long long)r2 * c.d + f);
      }
    }
    float wn = 0.f;
    if (fv) {
      if (P.kind == G_O) wn = __ldg(J.norm_mlp + f);
      else if (P.kind == G_DOWN && (!J.dp || J.defer) && J.norm_next) wn = __ldg(J.norm_next + f);
    }
    const uint32_t buf = n_acc & 1u;
    // one thread polls the barrier, the others sleep in the hardware barrier behind it
    bool ok = true;
    if (wtid == 0) ok = wait_bar(&sh->acc_full[buf], (n_acc >> 1) & 1u, p.ctl, sh);
    ok = worker_and(ok);
    if (!ok) return false;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (tile_no == 0 && P.kind < 4) mark(T_ACC + P.kind);
    if (P.kind == G_QKV && tile_no == 0 && (J.src_flag == F_SELECT || J.dual_src)) {
      // the rows come from an Eq. 2 step: it left their factors in shared memory
      for (int r = wtid; r < J.R; r += WORKERS) sh->rs[r] = sh->rs_next[r + J.in_shift];
      worker_sync();
    } else if ((P.kind == G_QKV || P.kind == G_GU || P.kind == G_HEAD) && tile_no == 0) {
      // the reduction consumed every operand column, so every CTA's sums of squares are published
      row_scales((P.kind == G_GU ? p.b.ss_m : p.b.ss_a) + (long long)jb * c.Rcap, J.R, P.kind == G_HEAD ? J.row_off : 0);
    }
    const uint32_t t_lane = tmem_base + buf * 256u + ((uint32_t)(quarter * 32) << 16);
    for (int cb = group; cb < ncb; cb += 2) {
      float v[RB], u[RB];
      tmem_ld_rb(t_lane + (uint32_t)(cb * RB), v);
      if (P.dual || P.bmul == 2) tmem_ld_rb(t_lane + (uint32_t)(c.BN + cb * RB), u);
      if (P.bmul == 2) {
        // both candidates of every state went through the product (v: layer output, u: skip candidate):
        // keep the one the Eq. 2 step chose
#pragma unroll
        for (int k = 0; k < RB; ++k) {
          const int r = cb * RB + k;
          if (r < J.R && !sh->choice_row[r + J.in_shift]) v[k] = u[k];
        }
      }
      if (cb == group + 2) {
#pragma unroll
        for (int k = 0; k < RB; ++k) res[k] = res_n[k];
      } else if (cb != group && resid && fv) {
#pragma unroll
        for (int k = 0; k < RB; ++k) {
          const int r = cb * RB + k;
          res[k] = 0.f;
          if (r < J.R) res[k] = P.kind == G_O ? __ldcg(J.x_in + r * J.ldx + f) : __ldcg(p.b.x1 + (long long)r * c.d + f);
        }
      }
      if (P.kind == G_QKV) {
        if (fv) {
#pragma unroll
          for (int k = 0; k < RB; ++k) {
            const int r = cb * RB + k;
            if (r < J.R) __stcg(p.b.qkv + (long long)r * (c.qd + 2 * c.kvd) + f, v[k] * sh->rs[r]);
          }
        }
      } else if (P.kind == G_O) {
        float sq[RB];
#pragma unroll
        for (int k = 0; k < RB; ++k) {
          const int r = cb * RB + k;
          const float y = (fv && r < J.R) ? res[k] + v[k] : 0.f;
          if (fv && r < J.R) {
            __stcg(p.b.x1 + (long long)r * c.d + f, y);
            p.b.xn_m[(long long)r * c.d + f] = __float2bfloat16_rn(y * wn);
          }
          sq[k] = y * y;
        }
        const float tot = warp_reduce<RB>(sq, lane);
        if (lane < RB && cb * RB + lane < J.R) T->red[quarter][cb * RB + lane][0] = tot;
      } else if (P.kind == G_GU) {
        if (fv) {
#pragma unroll
          for (int k = 0; k < RB; ++k) {
            const int r = cb * RB + k;
            if (r < J.R) {
              const float rs = sh->rs[r];
              p.b.act[(long long)r * c.dffn + f] = __float2bfloat16_rn(silu_f(rs * v[k]) * (rs * u[k]));
            }
          }
        }
      } else if (dpd) {
        // layer outputs of the candidate states; per row the two sums of Eq. 2 that involve them
        // (x.y and y.y; the sums over the skip candidates were added when those were written)
        if (cb != group) {
#pragma unroll
          for (int k = 0; k < RB; ++k) {
            const int r = cb * RB + k;
            xi[k] = (fv && r < J.R) ? __ldg(J.x_i + rd.mod(r) * J.x_tok_stride + f) : 0.f;
          }
        }
        float pr[2 * RB];
#pragma unroll
        for (int k = 0; k < RB; ++k) {
          const int r = cb * RB + k;
          const float y = (fv && r < J.R) ? res[k] + v[k] : 0.f;
          if (fv && r < J.R && ncb > 2) __stcg(p.b.Gbuf + (long long)r * c.d + f, y);
          if (J.defer && fv && r < J.R) p.b.xn_a[(long long)r * c.d + f] = __float2bfloat16_rn(y * wn);
          if (cb == group) keep_y[k] = y;
          pr[k] = xi[k] * y;
          pr[RB + k] = y * y;
        }
        const float tot = warp_reduce<2 * RB>(pr, lane);
        if (lane < 2 * RB && cb * RB + (lane & (RB - 1)) < J.R) T->red[quarter][cb * RB + (lane & (RB - 1))][lane / RB] = tot;
      } else if (P.kind == G_DOWN) {
        float sq[RB];
#pragma unroll
        for (int k = 0; k < RB; ++k) {
          const int r = cb * RB + k;
          const float y = (fv && r < J.R) ? res[k] + v[k] : 0.f;
          if (fv && r < J.R) {
            __stcg(J.x_out + r * J.ldo + f, y);
            if (J.norm_next) p.b.xn_a[(long long)r * c.d + f] = __float2bfloat16_rn(y * wn);
          }
          sq[k] = y * y;
        }
        if (J.norm_next) {
          const float tot = warp_reduce<RB>(sq, lane);
          if (lane < RB && cb * RB + lane < J.R) T->red[quarter][cb * RB + lane][0] = tot;
        }
      } else {  // G_HEAD: best logit of this tile per row (lowest index on ties) and sum of exp
#pragma unroll
        for (int k = 0; k < RB; ++k) {
          const int r = cb * RB + k;
          if (r >= J.R) break;
          const float mine = fv ? v[k] * sh->rs[r] : -INFINITY;
          if (J.logits_out && fv) __stcg(J.logits_out + (long long)r * c.vocab + f, mine);
          float best = mine;
          int bi = fv ? f : 0x7fffffff;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, best, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
          }
          const float se = warp_sum(fv ? __expf(mine - best) : 0.f);
          if (lane == 0) {
            T->red[quarter][r][0] = best;
            T->red[quarter][r][1] = __int_as_float(bi);
            T->red[quarter][r][2] = se;
          }
        }
      }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    worker_sync();
    if (wtid == 0) mbar_arrive(tc::smem_u32(&sh->acc_empty[buf]));
    ++n_acc;
    // cross-warp part of the per-row sums: add the four quarters in a fixed order
    if (P.kind == G_O || (P.kind == G_DOWN && !J.dp && J.norm_next)) {
      // o product: MLP norm of this job; down product: the next job's first operand
      long long* ss = P.kind == G_O ? p.b.ss_m + (long long)jb * c.Rcap : p.b.ss_a + (long long)(jb + 1) * c.Rcap;
      for (int r = wtid; r < J.R; r += WORKERS)
        ss_add(ss + r, T->red[0][r][0] + T->red[1][r][0] + T->red[2][r][0] + T->red[3][r][0]);
    } else if (P.kind == G_HEAD) {
      for (int r = wtid; r < J.R; r += WORKERS) {
        float best = -INFINITY, se = 0.f;
        int bi = 0x7fffffff;
        for (int q4 = 0; q4 < 4; ++q4) {
          const float ov = T->red[q4][r][0];
          const int oi = __float_as_int(T->red[q4][r][1]);
          if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
        }
        for (int q4 = 0; q4 < 4; ++q4) {
          const float ov = T->red[q4][r][0];
          if (ov != -INFINITY) se += T->red[q4][r][2] * __expf(ov - best);
        }
        float4* dst = p.b.head_best + (long long)blockIdx.x * MAX_ROWS + r;
        if (tile_no > 0) {
          const float4 o = *dst;
          const int oi = __float_as_int(o.y);
          const float nb = fmaxf(o.x, best);
          se = se * __expf(best - nb) + o.z * __expf(o.x - nb);
          if (o.x > best || (o.x == best && oi < bi)) { best = o.x; bi = oi; }
        }
        *dst = make_float4(best, __int_as_float(bi), se, 0.f);
      }
    }
    if (P.kind == G_HEAD || P.kind == G_O || (P.kind == G_DOWN && !J.dp)) worker_sync();  // tables reused by the next tile
    return true;
  }

  // skip candidate of state j (1-based) at row t: g[i-1][j-1]
  // the same by row r = (j - 1) T + t of the step: state 1's candidates are the objective rows of the step
  // before, the others row r - T ... of g, i.e. row r of the array that starts at g[i-1][0]
  __device__ __forceinline__ const float* skip_row(const Job& J, int r) const {
    return r < J.T ? J.x_im1 + r * J.x_im1_stride : J.g_prev + (long long)r * p.c.d;
  }
  __device__ __forceinline__ const float* skip_src(const Job& J, int j, int t) const {
    return j == 1 ? J.x_im1 + t * J.x_im1_stride : J.g_prev + ((long long)(j - 1) * J.T + t) * p.c.d;
  }

  static constexpr double COS_FIX = 268435456.0;  // 2^28: sums up to 3e10 with 4e-9 resolution
  __device__ __forceinline__ static void cos_add(unsigned long long* dst, float part) {
    const long long q = __double2ll_rn((double)part * COS_FIX);
    asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(dst), "l"(q) : "memory");
  }

  // This CTA's share of the three sums of Eq. 2 that do not involve a layer output, for the step of
  // job `tgt` with `rows` candidate rows: x.s, s.s and x.x, where x = x_new[t] is that step's objective
  // row and s the skip candidate of state j: x_old[t] for j = 1, else g[j - 1][t].  They are added
  // to the job's accumulators as soon as the candidates exist, off the step's critical path.
  __device__ void pre_sums(int tgt, int rows, int Tn, const float* x_new, const float* x_old, long long xs,
                           long long xs_old, const float* g, bool fv, int f) {
    const Cfg& c = p.c;
    RedTables* T = tables();
    const int quarter = ww & 3, group = ww >> 2;
    const int ncb = (rows + RB - 1) / RB;
    const RowDiv rd(Tn);
    for (int cb = group; cb < ncb; cb += 2) {
      float pa[2 * RB], pb[RB];
#pragma unroll
      for (int k = 0; k < RB; ++k) {
        const int r = cb * RB + k;
        float xv = 0.f, sv = 0.f;
        if (fv && r < rows) {
          const int j = rd.div(r) + 1, t = rd.mod(r);
          xv = __ldg(x_new + t * xs + f);
          sv = __ldcg((j == 1 ? x_old + t * xs_old : g + ((long long)(j - 1) * Tn + t) * c.d) + f);
        }
        pa[k] = xv * sv;
        pa[RB + k] = sv * sv;
        pb[k] = xv * xv;
      }
      const float ta = warp_reduce<2 * RB>(pa, lane);
      const float tb = warp_reduce<RB>(pb, lane);
      const int r = cb * RB + (lane & (RB - 1));
      if (lane < 2 * RB && r < rows) {
        T->red[quarter][r][2 + lane / RB] = ta;
        if (lane < RB) T->red[quarter][r][4] = tb;
      }
    }
    worker_sync();
    unsigned long long* acc =
        reinterpret_cast<unsigned long long*>(p.b.cosacc) + (long long)tgt * ((long long)(c.Rcap + MAX_ROWS) * 5);
    for (int idx = wtid; idx < rows * 3; idx += WORKERS) {
      const int r = idx / 3, k = 2 + idx % 3;
      cos_add(acc + r * 5 + k, T->red[0][r][k] + T->red[1][r][k] + T->red[2][r][k] + T->red[3][r][k]);
    }
    worker_sync();  // the tables are reused
  }

  // ---- Eq. 2 step i over this CTA's slice of the d features (thread <-> feature as in the
  // epilogue):
  //   (1) this CTA's share of x.y and y.y goes to the job's fixed-point accumulators, publish;
  //   (2) wait for every CTA, read the totals, decide (every CTA decides alike); the chosen row's
  //       sum of squares is also the next layer's norm factor;
  //   (3) write this CTA's slice of the next layer's operand, publish;
  //   (4) this CTA's slice of g[i][.].
  // The sums over the skip candidates (x.s, s.s, x.x) were added earlier: by a layer job while it waited
  // for its o product, by a select-only job at its start.
  // from_epilogue: the down product's epilogue left the partials of this CTA in the tables and
  // the thread's layer outputs / skip candidates of its first row block in keep_y / keep_s.
  // Eq. 2 step, rows past the two worker groups' first blocks: they come from global memory, and their
  // (row, feature) pairs are dealt to all worker threads -- with many rows (several objective rows per state) a
  // thread per feature would walk its row blocks one dependent load after the other.  to_operand: the chosen
  // rows, normed, as the next layer's operand; else as g[i][.] for the next step (row r of the step is
  // g[i][j][t] with j T + t = r + T).  Only in the instantiation for long contexts and many rows.
  __device__ __forceinline__ void spread_rows(const Job& J, int f_lo, int nf, int rows, bool to_operand) const {
    const int d = p.c.d, r_rest = 2 * RB, n_rest = max(rows - r_rest, 0) * nf;
    float* const g_out = J.g_next + (long long)J.T * d;
    const int gf_lo = (J.M - 1) * J.T;                              // first row of state M, if the step has it
    float* const gf_out = (J.g_final && rows > gf_lo) ? J.g_final : nullptr;
#pragma unroll 4
    for (int idx = wtid; idx < n_rest; idx += WORKERS) {
      const int rq = idx / nf;
      const int r = r_rest + rq, ff = f_lo + (idx - rq * nf);
      const float y = sh->choice_row[r] ? __ldcg(p.b.Gbuf + (long long)r * d + ff) : __ldcg(skip_row(J, r) + ff);
      if (to_operand) {
        p.b.xn_a[(long long)r * d + ff] = __float2bfloat16_rn(y * __ldg(J.norm_next + ff));
      } else {
        __stcg(g_out + (long long)r * d + ff, y);
        if (gf_out && r >= gf_lo) gf_out[(long long)(r - gf_lo) * d + ff] = y;
      }
    }
  }

  __device__ bool dp_step(const Job& J, int jb, bool from_epilogue, float (&keep_y)[RB], float (&keep_s)[RB]) {
    const Cfg& c = p.c;
    RedTables* T = tables();
    const int f_lo = __ldg(split_lo(S_D) + blockIdx.x), f_hi = __ldg(split_lo(S_D) + blockIdx.x + 1);
    const int quarter = ww & 3, group = ww >> 2;
    const int fl = feat_local(f_hi - f_lo, quarter, lane);   // a slice has at most 128 features (checked on the host)
    const bool fv = fl >= 0;
    const int f = f_lo + fl;
    const int n_states = J.ell + (J.diag ? 1 : 0);
    const int rows = n_states * J.T;
    const int ncb = (rows + RB - 1) / RB;
    unsigned long long* acc =
        reinterpret_cast<unsigned long long*>(p.b.cosacc) + (long long)jb * ((long long)(c.Rcap + MAX_ROWS) * 5);
    const RowDiv rd(J.T);
    const float wn = (fv && J.norm_next) ? __ldg(J.norm_next + f) : 0.f;   // needed right after the decision
    // (a layer job adds its sums over the skip candidates while it waits for its o product)
    if (J.type == JOB_SELECT) pre_sums(jb, rows, J.T, J.x_i, J.x_im1, J.x_tok_stride, J.x_im1_stride, J.g_prev, fv, f);
    if (!from_epilogue) {
      // no layer ran for this CTA's features: only skip candidates exist
#pragma unroll
      for (int k = 0; k < RB; ++k) {
        const int r = group * RB + k;
        keep_y[k] = 0.f;
        keep_s[k] = (fv && r < rows) ? __ldcg(skip_row(J, r) + f) : 0.f;
      }
    } else {
      for (int idx = wtid; idx < J.R * 2; idx += WORKERS) {
        const int r = idx >> 1, k = idx & 1;
        cos_add(acc + r * 5 + k, T->red[0][r][k] + T->red[1][r][k] + T->red[2][r][k] + T->red[3][r][k]);
      }
    }
    publish(F_DOWN, jb + 1);
    mark(T_DP_PUB);
    // (2) once every CTA has added its share: read the totals, decide
    if (!wait_all(F_DOWN, J.tgt[F_DOWN])) return false;
    mark(T_DP_ALL);
    for (int idx = wtid; idx < rows * 5; idx += WORKERS)
      T->cosv[idx / 5][idx % 5] = (double)(long long)__ldcg(acc + idx) * (1.0 / COS_FIX);
    worker_sync();
    if (wtid < n_states) {
      const int j = wtid + 1;
      // the sums are exact to the fixed-point step; the few operations on them run in float
      float app = 0.f, skp = 0.f;
      for (int t = 0; t < J.T; ++t) {
        const double* v = T->cosv[(j - 1) * J.T + t];
        const float nx = fmaxf(sqrtf((float)v[4]), 1e-12f);
        app += (float)v[0] / (nx * fmaxf(sqrtf((float)v[1]), 1e-12f));
        skp += (float)v[2] / (nx * fmaxf(sqrtf((float)v[3]), 1e-12f));
      }
      const float s_app = app / (float)J.T, s_skip = skp / (float)J.T;
      int take = 0;
      if (j <= J.ell) {
        take = s_app > s_skip;
        if (J.forced && J.forced[j] != 255) take = (J.forced[j] == 0);
      }
      sh->choice[j] = take;
      for (int t = 0; t < J.T; ++t) sh->choice_row[(j - 1) * J.T + t] = take;
      for (int t = 0; t < J.T; ++t) {
        const double* v = T->cosv[(j - 1) * J.T + t];
        sh->rs_next[(j - 1) * J.T + t] = rsqrtf((float)(take ? v[1] : v[3]) / (float)c.d + c.eps);
      }
      if (blockIdx.x == 0) {
        J.D[j] = take ? s_app : s_skip;
        J.choice[j] = take ? 0 : 1;
        if (J.margin && j <= J.ell) J.margin[j] = s_app - s_skip;
      }
    }
    if (blockIdx.x == 0 && wtid == 0) {
      J.D0[0] = 1.0f;
      J.choice0[0] = 0;
    }
    worker_sync();
    mark(T_DP_DECIDED);
    // (3) the next layer's operand: the first block of rows comes from registers
    float y16[RB];
#pragma unroll
    for (int k = 0; k < RB; ++k) {
      const int r = group * RB + k;
      y16[k] = 0.f;
      if (fv && r < rows) y16[k] = sh->choice_row[r] ? keep_y[k] : keep_s[k];
    }
    if constexpr (TC) {
      // (the instantiation for long contexts and many rows deals the rows past the first blocks to all threads)
      if (J.norm_next && !J.defer) {
        if (fv) {
#pragma unroll
          for (int k = 0; k < RB; ++k) {
            const int r = group * RB + k;
            if (r < rows) p.b.xn_a[(long long)r * c.d + f] = __float2bfloat16_rn(y16[k] * wn);
          }
        }
        spread_rows(J, f_lo, f_hi - f_lo, rows, true);
      }
    } else if (J.norm_next && fv && !J.defer) {
      for (int cb = group; cb < ncb; cb += 2) {
#pragma unroll
        for (int k = 0; k < RB; ++k) {
          const int r = cb * RB + k;
          if (r < rows) {
            const float y = cb == group ? y16[k]
                                        : (sh->choice_row[r] ? __ldcg(p.b.Gbuf + (long long)r * c.d + f) : __ldcg(skip_row(J, r) + f));
            p.b.xn_a[(long long)r * c.d + f] = __float2bfloat16_rn(y * wn);
          }
        }
      }
    }
    if (!J.defer) publish(F_SELECT, jb + 1);   // (a deferred step's successor reads both candidates: nobody waits)
    mark(T_SEL_PUB);
    // (4) g[i][.] for the next step (read back only by this thread: same feature in every step)
    float* const g_out = J.g_next + (long long)J.T * c.d + f;
    const int gf_lo = (J.M - 1) * J.T;                              // first row of state M, if the step has it
    float* const gf_out = (J.g_final && rows > gf_lo) ? J.g_final + f : nullptr;
    if constexpr (TC) {
      if (fv) {
#pragma unroll
        for (int k = 0; k < RB; ++k) {
          const int r = group * RB + k;
          if (r < rows) {
            __stcg(g_out + (long long)r * c.d, y16[k]);
            if (gf_out && r >= gf_lo) gf_out[(long long)(r - gf_lo) * c.d] = y16[k];
          }
        }
      }
      spread_rows(J, f_lo, f_hi - f_lo, rows, false);
    } else if (fv) {
      for (int cb = group; cb < ncb; cb += 2) {
#pragma unroll
        for (int k = 0; k < RB; ++k) {
          const int r = cb * RB + k;
          if (r < rows) {   // row r of the step is g[i][j][t] with j T + t = r + T
            const float y = cb == group ? y16[k]
                                        : (sh->choice_row[r] ? __ldcg(p.b.Gbuf + (long long)r * c.d + f) : __ldcg(skip_row(J, r) + f));
            __stcg(g_out + (long long)r * c.d, y);
            if (gf_out && r >= gf_lo) gf_out[(long long)(r - gf_lo) * c.d] = y;
          }
        }
      }
    }
    return true;
  }

  // ---- attention: partial softmax over one run of cache keys or one chunk of own rows.
  // q, k, v of the rows come from the projection buffer (norm factor applied, not rotated): they
  // are rotated here; new keys / values are rounded to the cache type before use.
  // OWN_ONLY: the caller has already dealt with the runs of cache keys (attention_tc) and waited for the
  // projections; only the chunks of the rows' own keys are left, dealt out from the last CTA downwards.
  template <bool OWN_ONLY = false>
  __device__ bool attention_partials(const Job& J, int jb) {
    const Cfg& c = p.c;
    constexpr int KS = HD / 16;
    constexpr int NBLK = HD / 8;
    constexpr int LD = HD + 8;
    constexpr int HALF = HD / 2;
    bf16* k_s = reinterpret_cast<bf16*>(scratch);
    bf16* v_s = k_s + ATT_KEYS * LD;
    const int Gq = c.nq / c.nkv;
    const int Pn = J.R * Gq;
    const int n_pbg = (Pn + 127) / 128;
    const int k_tot = J.uniform ? J.C + J.T : J.C;
    const int n_runs = (k_tot + c.run_len - 1) / c.run_len;
    const int n_own = J.uniform ? 0 : (J.R + ATT_KEYS - 1) / ATT_KEYS;
    const int n_chunks = n_runs + n_own;
    const int n_ch = OWN_ONLY ? n_own : n_chunks;   // chunks this call deals out
    const int n_items = c.nkv * n_ch * n_pbg;
    const int g8 = lane >> 2, c4 = lane & 3;
    const long long kvld = c.kvd;
    const int qkvd = c.qd + 2 * c.kvd;
    const float qscale = rsqrtf((float)HD) * 1.4426950408889634f;
    const RowDiv rdT(J.T);
    const uint32_t tag = p.launch_tag | (uint32_t)(jb + 1);
    // The cache does not depend on this layer's projections: the first K/V tile of this CTA's first
    // item is on its way from HBM while the CTA waits for them.
    constexpr int FILL = ATT_KEYS * (HD / 8) / WORKERS;   // 16-byte pieces of a tile per thread
    static_assert(FILL * WORKERS == ATT_KEYS * (HD / 8), "tile pieces must divide among the workers");
    uint4 pre_k[FILL], pre_v[FILL];
    bool pre_ok = false;
    if (!OWN_ONLY && (int)blockIdx.x < n_items) {
      const int chunk = ((int)blockIdx.x / n_pbg) % n_chunks;
      const int kvh = (int)blockIdx.x / (n_pbg * n_chunks);
      if (chunk < n_runs) {
        const int key_lo = chunk * c.run_len;
        pre_ok = true;
#pragma unroll
        for (int e = 0; e < FILL; ++e) {
          const int vv = wtid + e * WORKERS;
          const int key = key_lo + vv / (HD / 8), cv8 = vv % (HD / 8);
          pre_k[e] = make_uint4(0, 0, 0, 0);
          pre_v[e] = make_uint4(0, 0, 0, 0);
          if (key < J.C) {   // positions this launch never writes
            pre_k[e] = __ldcg(reinterpret_cast<const uint4*>(J.ck + (long long)key * kvld + kvh * HD + cv8 * 8));
            pre_v[e] = __ldcg(reinterpret_cast<const uint4*>(J.cv + (long long)key * kvld + kvh * HD + cv8 * 8));
          }
        }
      }
    }
    // every row's q, k, v exist once all CTAs have published their slice of the projections
    if (!OWN_ONLY) {
      if (!wait_all(F_QKV, J.tgt[F_QKV])) return false;
      mark(T_ATT_READY);
    }
    for (int it = OWN_ONLY ? c.G - 1 - (int)blockIdx.x : (int)blockIdx.x; it < n_items; it += c.G) {
      const int pbg = it % n_pbg;
      const int chunk = (OWN_ONLY ? n_runs : 0) + (it / n_pbg) % n_ch;
      const int kvh = it / (n_pbg * n_ch);
      const bool own = chunk >= n_runs;
      const int p0 = (pbg * 8 + ww) * 16;
      const bool active = p0 < Pn;
      int rr[2], hq[2], tq[2], sq[2];   // row, query head, position and state of the row
      bool pv[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int pp = p0 + g8 + h * 8;
        pv[h] = pp < Pn;
        rr[h] = pv[h] ? pp / Gq : 0;
        hq[h] = kvh * Gq + (pv[h] ? pp % Gq : 0);
        sq[h] = rdT.div(rr[h]);
        tq[h] = rr[h] - sq[h] * J.T;
      }
      // q fragments, rotated.  Element i of the first half pairs with element i + HD/2: one load
      // of each gives the rotated values of both, i.e. the fragments of k-steps ks and ks + KS/2.
      uint32_t qh[KS][4];
      {
        // all loads first (one trip to L2), then the rotation
        float2 raw_lo[KS / 2][4], raw_hi[KS / 2][4];
#pragma unroll
        for (int ks = 0; ks < KS / 2; ++ks) {
#pragma unroll
          for (int h = 0; h < 2; ++h) {
#pragma unroll
            for (int kh = 0; kh < 2; ++kh) {
              raw_lo[ks][h + kh * 2] = make_float2(0.f, 0.f);
              raw_hi[ks][h + kh * 2] = make_float2(0.f, 0.f);
              if (active && pv[h]) {
                const int i = ks * 16 + kh * 8 + c4 * 2;           // dims i, i + 1 of the first half
                const float* qr = p.b.qkv + (long long)rr[h] * qkvd + hq[h] * HD;
                raw_lo[ks][h + kh * 2] = __ldcg(reinterpret_cast<const float2*>(qr + i));
                raw_hi[ks][h + kh * 2] = __ldcg(reinterpret_cast<const float2*>(qr + i + HALF));
              }
            }
          }
        }
#pragma unroll
        for (int ks = 0; ks < KS / 2; ++ks) {
#pragma unroll
          for (int h = 0; h < 2; ++h) {
#pragma unroll
            for (int kh = 0; kh < 2; ++kh) {
              const int i = ks * 16 + kh * 8 + c4 * 2;
              const float2 lo2 = raw_lo[ks][h + kh * 2], hi2 = raw_hi[ks][h + kh * 2];
              const float4 cs = *reinterpret_cast<const float4*>(p.b.rope + (long long)tq[h] * HALF + i);
              const float2 v0 = make_float2((lo2.x * cs.x - hi2.x * cs.y) * qscale, (lo2.y * cs.z - hi2.y * cs.w) * qscale);
              const float2 v1 = make_float2((hi2.x * cs.x + lo2.x * cs.y) * qscale, (hi2.y * cs.z + lo2.y * cs.w) * qscale);
              qh[ks][h + kh * 2] = pack2(v0.x, v0.y);
              qh[ks + KS / 2][h + kh * 2] = pack2(v1.x, v1.y);
            }
          }
        }
      }
      mark(T_ATT_Q);
      float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
      float o[NBLK][4];
#pragma unroll
      for (int nb = 0; nb < NBLK; ++nb) { o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f; }

      int key_lo, key_hi;
      if (!own) { key_lo = chunk * c.run_len; key_hi = min(k_tot, key_lo + c.run_len); }
      else { key_lo = (chunk - n_runs) * ATT_KEYS; key_hi = min(J.R, key_lo + ATT_KEYS); }
      // cache pieces of the tile at k0 into the rolling registers (issued one tile ahead of their use)
      auto load_cache_tile = [&](int k0) {
#pragma unroll
        for (int e = 0; e < FILL; ++e) {
          const int vv = wtid + e * WORKERS;
          const int key = k0 + vv / (HD / 8), cv8 = vv % (HD / 8);
          pre_k[e] = make_uint4(0, 0, 0, 0);
          pre_v[e] = make_uint4(0, 0, 0, 0);
          if (key < key_hi && key < J.C) {
            pre_k[e] = __ldcg(reinterpret_cast<const uint4*>(J.ck + (long long)key * kvld + kvh * HD + cv8 * 8));
            pre_v[e] = __ldcg(reinterpret_cast<const uint4*>(J.cv + (long long)key * kvld + kvh * HD + cv8 * 8));
          }
        }
      };
      if (!own && !(pre_ok && it == (int)blockIdx.x)) load_cache_tile(key_lo);
      for (int key0 = key_lo; key0 < key_hi; key0 += ATT_KEYS) {
        const int nkeys = min(ATT_KEYS, key_hi - key0);
        worker_sync();  // previous tile consumed
        // K/V tile: cache rows as they are; rows of this call rotated / rounded from the projections
#pragma unroll
        for (int e = 0; e < FILL; ++e) {
          const int vv = wtid + e * WORKERS;
          const int row = vv / (HD / 8), cv8 = vv % (HD / 8);
          uint4 kk = make_uint4(0, 0, 0, 0), vq = make_uint4(0, 0, 0, 0);
          if (row < nkeys) {
            const int key = key0 + row;
            const int new_row = own ? key : (J.uniform ? key - J.C : -1);
            if (new_row < 0) {
              kk = pre_k[e];
              vq = pre_v[e];
            } else {
              const float* kr = p.b.qkv + (long long)new_row * qkvd + c.qd + kvh * HD;
              const float* vr = kr + c.kvd;
              const int d0 = cv8 * 8, i0 = d0 % HALF;
              float ka[8], kb[8], vf[8];
#pragma unroll
              for (int e = 0; e < 8; e += 4) {
                const float4 a4 = __ldcg(reinterpret_cast<const float4*>(kr + i0 + e));
                const float4 b4 = __ldcg(reinterpret_cast<const float4*>(kr + i0 + HALF + e));
                const float4 v4 = __ldcg(reinterpret_cast<const float4*>(vr + d0 + e));
                ka[e] = a4.x; ka[e + 1] = a4.y; ka[e + 2] = a4.z; ka[e + 3] = a4.w;
                kb[e] = b4.x; kb[e + 1] = b4.y; kb[e + 2] = b4.z; kb[e + 3] = b4.w;
                vf[e] = v4.x; vf[e + 1] = v4.y; vf[e + 2] = v4.z; vf[e + 3] = v4.w;
              }
              float kro[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const float2 cs = p.b.rope[(long long)rdT.mod(new_row) * HALF + i0 + e];
                kro[e] = d0 < HALF ? ka[e] * cs.x - kb[e] * cs.y : kb[e] * cs.x + ka[e] * cs.y;
              }
              const uint2 k01 = pack4(kro[0], kro[1], kro[2], kro[3]), k23 = pack4(kro[4], kro[5], kro[6], kro[7]);
              const uint2 v01 = pack4(vf[0], vf[1], vf[2], vf[3]), v23 = pack4(vf[4], vf[5], vf[6], vf[7]);
              kk = make_uint4(k01.x, k01.y, k23.x, k23.y);
              vq = make_uint4(v01.x, v01.y, v23.x, v23.y);
              if (J.uniform && pbg == 0) {  // this item owns the cache rows of its keys
                *reinterpret_cast<uint4*>(J.ck + (long long)key * kvld + kvh * HD + cv8 * 8) = kk;
                *reinterpret_cast<uint4*>(J.cv + (long long)key * kvld + kvh * HD + cv8 * 8) = vq;
              }
            }
          }
          *reinterpret_cast<uint4*>(k_s + row * LD + cv8 * 8) = kk;
          *reinterpret_cast<uint4*>(v_s + row * LD + cv8 * 8) = vq;
        }
        if (!own && key0 + ATT_KEYS < key_hi) load_cache_tile(key0 + ATT_KEYS);   // in flight during the tile's math
        worker_sync();
        if (!active) continue;
        // S = Q K^T.  The multiplies are issued in program order (volatile asm): the k-step is the outer loop,
        // so that four independent accumulators alternate instead of eight dependent multiplies in a row.
        float s[4][4];
#pragma unroll
        for (int nb = 0; nb < 4; ++nb) s[nb][0] = s[nb][1] = s[nb][2] = s[nb][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
          uint32_t b0[4], b1[4];
#pragma unroll
          for (int nb = 0; nb < 4; ++nb) {
            const bf16* kr = k_s + (nb * 8 + g8) * LD + c4 * 2 + ks * 16;
            b0[nb] = *reinterpret_cast<const uint32_t*>(kr);
            b1[nb] = *reinterpret_cast<const uint32_t*>(kr + 8);
          }
#pragma unroll
          for (int nb = 0; nb < 4; ++nb) mma_16816(s[nb], qh[ks], b0[nb], b1[nb]);
        }
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nb = 0; nb < 4; ++nb) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int h = e >> 1;
            const int key = key0 + nb * 8 + c4 * 2 + (e & 1);
            bool vis = pv[h] && key < key_hi;
            if (own) vis = vis && (rdT.div(key) == sq[h]) && key <= rr[h];
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
        float rsum[2] = {0.f, 0.f};
#pragma unroll
        for (int nb = 0; nb < 4; ++nb) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int h = e >> 1;
            const float pe = (s[nb][e] == -INFINITY) ? 0.f : exp2f(s[nb][e] - m[h]);
            s[nb][e] = pe;
            rsum[h] += pe;
          }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          rsum[h] += __shfl_xor_sync(0xffffffffu, rsum[h], 1);
          rsum[h] += __shfl_xor_sync(0xffffffffu, rsum[h], 2);
          l[h] = l[h] * corr[h] + rsum[h];
        }
#pragma unroll
        for (int nb = 0; nb < NBLK; ++nb) {
          o[nb][0] *= corr[0]; o[nb][1] *= corr[0];
          o[nb][2] *= corr[1]; o[nb][3] *= corr[1];
        }
#pragma unroll
        for (int k2 = 0; k2 < 2; ++k2) {
          uint32_t ph[4];
          ph[0] = pack2(s[2 * k2][0], s[2 * k2][1]);
          ph[1] = pack2(s[2 * k2][2], s[2 * k2][3]);
          ph[2] = pack2(s[2 * k2 + 1][0], s[2 * k2 + 1][1]);
          ph[3] = pack2(s[2 * k2 + 1][2], s[2 * k2 + 1][3]);
          const int mrow = k2 * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
          const int mcol = (lane >> 4) * 8;
#pragma unroll
          for (int nb = 0; nb < NBLK; nb += 8) {   // four fragment loads in flight, then their eight multiplies
            uint32_t vb[4][4];
#pragma unroll
            for (int q = 0; q < 4; ++q)
              ldmatrix_x4_trans(tc::smem_u32(v_s + mrow * LD + (nb + 2 * q) * 8 + mcol), vb[q][0], vb[q][1], vb[q][2], vb[q][3]);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              mma_16816(o[nb + 2 * q], ph, vb[q][0], vb[q][1]);
              mma_16816(o[nb + 2 * q + 1], ph, vb[q][2], vb[q][3]);
            }
          }
        }
      }
      mark(T_ATT_TILES);
      if (active) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (!pv[h]) continue;
          // Every 8-byte store carries its own tag, so the merge needs no flag and no fence: it reads the
          // partial results themselves until every piece shows this job's tag (8-byte accesses are single
          // copies).  Values as bf16: the merged row is rounded to bf16 for the o product anyway.
          const long long idx = ((long long)rr[h] * c.nq + hq[h]) * c.chunk_cap + chunk;
          uint2* pa = p.b.att_acc + idx * (HD / 2) + c4;
#pragma unroll
          for (int nb = 0; nb < NBLK; ++nb) __stcg(pa + nb * 4, make_uint2(pack2(o[nb][2 * h], o[nb][2 * h + 1]), tag));
          if (c4 == 0) __stcg(p.b.att_ml + idx, make_uint4(__float_as_uint(m[h]), tag, __float_as_uint(l[h]), tag));
        }
      }
    }
    return true;
  }

  // 16 accumulator columns of this thread's lane: write (the read is tc::tmem_ld16)
  __device__ __forceinline__ static void tmem_st16(uint32_t taddr, const float (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
        "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
        "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
        "r"(__float_as_uint(v[15]))
        : "memory");
  }

  // 32 accumulator columns of this thread's lane
  __device__ __forceinline__ static void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
  }

  // ---- pieces of the tensor-core attention
  // scratch: Q tile [2 halves][AM rows][128 B], K and V tiles [2 halves][64 keys][128 B], P tile [AM rows][128 B],
  // then two floats per row (what the halves of a row tell each other); AM = 64 or 128 rows per item
  static constexpr int TK = 64;
  static constexpr uint32_t Q_OFF = 0;
  __device__ __forceinline__ static uint32_t k_off(int AM) { return (uint32_t)AM * 256u; }
  __device__ __forceinline__ static uint32_t v_off(int AM) { return k_off(AM) + TK * 256; }
  __device__ __forceinline__ static uint32_t p_off(int AM) { return v_off(AM) + TK * 256; }
  __device__ __forceinline__ static uint32_t x_off(int AM) { return p_off(AM) + (uint32_t)AM * 128u; }
  static constexpr uint32_t S_COL = 0, O_COL = 128;
  // worker warp 4, one lane: the 64-key tile at key0 of one kv head, two 64-dim halves of [64 keys][128 bytes]
  // as the tensor map's 128-byte swizzle lays them out (rows past the context read as zeros)
  __device__ __forceinline__ void tc_fetch(const CUtensorMap* map, uint32_t dst, uint64_t* bar, int kvh, int key0,
                                           uint64_t policy, uint32_t el) const {
    if (ww != 4 || !el) return;
    const uint32_t b = tc::smem_u32(bar);
    tc::mbar_expect_tx(b, (uint32_t)(TK * HD * 2));
    tc::tma_load_2d(dst, map, b, kvh * HD, key0, policy);
    tc::tma_load_2d(dst + TK * 128, map, b, kvh * HD + 64, key0, policy);
  }
  // worker warp 4: the multiplies of one step, then one commit on the attention's barrier
  // (it first waits for the tiles the multiplies read; a wait that runs out raises the abort flag, which ends tc_wait)
  __device__ __forceinline__ void tc_issue(uint32_t s_base, int AM, bool pv, bool pv_acc, bool qk) {
    if (ww != 4) return;
    if (pv) {
      if (!wait_bar(&sh->att_v_bar, att_vph & 1u, p.ctl, sh)) return;
      att_vph ^= 1u;
    }
    if (qk) {
      if (!wait_bar(&sh->att_k_bar, att_kph & 1u, p.ctl, sh)) return;
      att_kph ^= 1u;
    }
    const uint32_t idesc_qk = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TK >> 3) << 17) | ((uint32_t)(AM >> 4) << 24);
    const uint32_t idesc_pv = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(HD >> 3) << 17) | ((uint32_t)(AM >> 4) << 24);
    const uint32_t K_OFF = k_off(AM), V_OFF = v_off(AM), P_OFF = p_off(AM);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t el = elect_one();
    if (pv) {
      const uint64_t da = make_desc(s_base + P_OFF);
      // V: 8-key groups 1024 bytes apart (stride offset), 64-dim halves TK * 128 bytes apart (leading offset)
      const uint64_t db = ((uint64_t)DESC_HI << 32) | (uint64_t)((((s_base + V_OFF) & 0x3FFFFu) >> 4) | ((uint32_t)(TK * 128 / 16) << 16));
      if (pv_acc) mma_el<true>(tmem_base + O_COL, da, db, idesc_pv, el);
      else mma_el<false>(tmem_base + O_COL, da, db, idesc_pv, el);
#pragma unroll
      for (int s4 = 1; s4 < TK / 16; ++s4)
        mma_el<true>(tmem_base + O_COL, da + (uint64_t)(2 * s4), db + (uint64_t)(s4 * (16 * 128 / 16)), idesc_pv, el);
    }
    if (qk) {
#pragma unroll
      for (int s8 = 0; s8 < HD / 16; ++s8) {
        const uint64_t da = make_desc(s_base + Q_OFF + (s8 >> 2) * (AM * 128)) + (uint64_t)((s8 & 3) * 2);
        const uint64_t db = make_desc(s_base + K_OFF + (s8 >> 2) * (TK * 128)) + (uint64_t)((s8 & 3) * 2);
        if (s8 == 0) mma_el<false>(tmem_base + S_COL, da, db, idesc_qk, el);
        else mma_el<true>(tmem_base + S_COL, da, db, idesc_qk, el);
      }
    }
    mma_commit_el(tc::smem_u32(&sh->att_bar), el);
  }
  // one thread polls the barrier, the others sleep in the hardware barrier behind it (one decision for all)
  __device__ __forceinline__ bool tc_wait() {
    bool ok = true;
    if (wtid == 0) ok = wait_bar(&sh->att_bar, att_phase & 1u, p.ctl, sh);
    att_phase ^= 1u;
    ok = worker_and(ok);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    return ok;
  }
  // Every thread polls the barrier itself: no CTA barrier behind the wait.  A thread whose wait ran out carries
  // on (it touches shared and tensor memory only) and reports it at the next reducing barrier, where all decide together.
  __device__ __forceinline__ bool tc_poll() {
    const bool ok = wait_bar(&sh->att_bar, att_phase & 1u, p.ctl, sh);
    att_phase ^= 1u;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    return ok;
  }
  // generic-proxy writes of the tiles before the tensor core reads them; tensor-memory accesses before the barrier
  __device__ __forceinline__ static void tc_fences() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  }
  __device__ __forceinline__ static float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
  }
  // weights of 32 columns of a row under the maximum m: bf16 into the row of the P tile (pieces 4 half ..) if `wr`,
  // their sum back; columns from nv on are not keys of the run and weigh nothing
  template <bool MASKED>
  __device__ __forceinline__ static float tc_weights(const float (&s)[32], int nv, float m, uint8_t* p_row, int swz, int half,
                                                     bool wr) {
    float r4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float w[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        w[k] = ex2(s[j * 8 + k] - m);
        if (MASKED && j * 8 + k >= nv) w[k] = 0.f;
        r4[k & 3] += w[k];
      }
      const uint2 p01 = pack4(w[0], w[1], w[2], w[3]), p23 = pack4(w[4], w[5], w[6], w[7]);
      if (wr) *reinterpret_cast<uint4*>(p_row + (((half * 4 + j) ^ swz) << 4)) = make_uint4(p01.x, p01.y, p23.x, p23.y);
    }
    return (r4[0] + r4[1]) + (r4[2] + r4[3]);
  }

  // ---- attention of a search job over its cache keys on the tensor cores (head dimension 128).
  // Item = (kv head, run of cache keys, block of 64 or 128 (row, query head) pairs).  Per 64-key tile:
  //   S = Q K^T   (M = the block's pairs, N = 64 keys, K = 128 dims; Q and K tiles K-major, 128-byte swizzle)
  //   P = exp2(S - m) as bf16 into shared memory, row sums in registers
  //   O += P V    (N = 128 dims, K = 64 keys; the V tile stays as the cache has it, key rows of 128 dims,
  //                i.e. the MN-major form of the B operand)
  // S and O live in tensor memory, which no product uses while the attention runs (the o projection
  // waits for the merged rows of every CTA).  A row of S sits in one lane: worker warps w and w + 4 share
  // lane quarter w & 3 and take 32 of the row's 64 columns each.  The row's maximum m is fixed by the
  // first tile and only moves when a later tile exceeds it by more than 2^8 (the whole CTA then takes a
  // slow path that rescales O and the sums), so a tile is normally one trip over S.  K and V tiles come
  // by TMA through the layer's tensor maps, each as soon as the multiplies that read its predecessor are done.  The partial result of an item has the format of
  // attention_partials, which still computes the chunks of the rows' own keys.
  __device__ bool attention_tc(const Job& J, int jb) {
    if constexpr (HD != 128 || !TC) {
      return false;
    } else {
      const Cfg& c = p.c;
      static_assert(256 * TC_ROWS + 2 * TK * 256 + 128 * TC_ROWS + 2 * TC_ROWS * 4 <= SCRATCH_TC_BYTES, "attention tiles must fit the scratch area");
      const int AM = c.att_rows;   // 64: an M = 64 accumulator keeps row r in lane 32 (r / 16) + r % 16; 128: row r in lane r
      const uint32_t K_OFF = k_off(AM), V_OFF = v_off(AM), P_OFF = p_off(AM);
      const uint32_t s_base = tc::smem_u32(scratch);
      float* xch = reinterpret_cast<float*>(scratch + x_off(AM));
      const int Gq = c.nq / c.nkv;
      const int Pn = J.R * Gq;
      const int n_pb = (Pn + AM - 1) / AM;
      const int n_runs = (J.C + c.run_len - 1) / c.run_len;
      const int n_items = c.nkv * n_runs * n_pb;
      const int qkvd = c.qd + 2 * c.kvd;
      const float qscale = rsqrtf((float)HD) * 1.4426950408889634f;
      const RowDiv rdT(J.T), rdG(Gq);
      const uint32_t tag = p.launch_tag | (uint32_t)(jb + 1);
      const int quarter = ww & 3, half = ww >> 2;
      const int qrows = AM >> 2;                       // rows of a lane quarter
      const bool lane_ok = lane < qrows;
      const int row = quarter * qrows + (lane_ok ? lane : 0);
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16);
      const CUtensorMap* kmap = p.kvmaps + J.kvmap;
      const CUtensorMap* vmap = kmap + 1;
      const uint32_t el = elect_one();
      uint64_t pol;
      asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
      if (ww == 4 && el) {
        // the maps were written by a copy on the stream before this launch, at addresses earlier launches also used:
        // the copies of them this SM may still hold are dropped
        asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(kmap) : "memory");
        asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(vmap) : "memory");
      }
      int it = blockIdx.x;
      if (it < n_items) {   // the cache does not depend on this layer's projections
        const int run = (it / n_pb) % n_runs, kvh = it / (n_pb * n_runs);
        tc_fetch(kmap, s_base + K_OFF, &sh->att_k_bar, kvh, run * c.run_len, pol, el);
        tc_fetch(vmap, s_base + V_OFF, &sh->att_v_bar, kvh, run * c.run_len, pol, el);
      }
      if (!wait_all(F_QKV, J.tgt[F_QKV])) return false;
      mark(T_ATT_READY);
      for (; it < n_items; it += c.G) {
        const int pb = it % n_pb;
        const int run = (it / n_pb) % n_runs;
        const int kvh = it / (n_pb * n_runs);
        const int key_lo = run * c.run_len, key_hi = min(J.C, key_lo + c.run_len);
        const int nt = (key_hi - key_lo + TK - 1) / TK;
        if (it != (int)blockIdx.x) {   // (the last item's multiplies are done: both tiles are free)
          tc_fetch(kmap, s_base + K_OFF, &sh->att_k_bar, kvh, key_lo, pol, el);
          tc_fetch(vmap, s_base + V_OFF, &sh->att_v_bar, kvh, key_lo, pol, el);
        }
        // Q tile: rows rotated and scaled; dims i and i + 64 of a row share a rotation, so one thread
        // makes the pieces (row, j) and (row, j + 8) from the same loads
#pragma unroll 2
        for (int e = 0; e < AM * 8 / WORKERS; ++e) {   // (two tasks' loads in flight)
          const int task = wtid + e * WORKERS;
          const int qrow = task >> 3, j = task & 7;
          const int pp = pb * AM + qrow;
          uint4 lo_p = make_uint4(0, 0, 0, 0), hi_p = make_uint4(0, 0, 0, 0);
          if (pp < Pn) {
            const int rr = rdG.div(pp);
            const int hq = kvh * Gq + (pp - rr * Gq);
            const float* qr = p.b.qkv + (long long)rr * qkvd + hq * HD + j * 8;
            const float4 a0 = __ldcg(reinterpret_cast<const float4*>(qr)), a1 = __ldcg(reinterpret_cast<const float4*>(qr + 4));
            const float4 b0 = __ldcg(reinterpret_cast<const float4*>(qr + HD / 2)), b1 = __ldcg(reinterpret_cast<const float4*>(qr + HD / 2 + 4));
            const float4* cs4 = reinterpret_cast<const float4*>(p.b.rope + (long long)rdT.mod(rr) * (HD / 2) + j * 8);
            const float lo[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float hi[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
            float v0[8], v1[8];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const float4 cs = cs4[q];   // (cos, sin) of dims 2q and 2q + 1
              v0[2 * q] = (lo[2 * q] * cs.x - hi[2 * q] * cs.y) * qscale;
              v1[2 * q] = (hi[2 * q] * cs.x + lo[2 * q] * cs.y) * qscale;
              v0[2 * q + 1] = (lo[2 * q + 1] * cs.z - hi[2 * q + 1] * cs.w) * qscale;
              v1[2 * q + 1] = (hi[2 * q + 1] * cs.z + lo[2 * q + 1] * cs.w) * qscale;
            }
            const uint2 l01 = pack4(v0[0], v0[1], v0[2], v0[3]), l23 = pack4(v0[4], v0[5], v0[6], v0[7]);
            const uint2 h01 = pack4(v1[0], v1[1], v1[2], v1[3]), h23 = pack4(v1[4], v1[5], v1[6], v1[7]);
            lo_p = make_uint4(l01.x, l01.y, l23.x, l23.y);
            hi_p = make_uint4(h01.x, h01.y, h23.x, h23.y);
          }
          uint8_t* dst = scratch + Q_OFF + qrow * 128 + ((j ^ (qrow & 7)) << 4);
          *reinterpret_cast<uint4*>(dst) = lo_p;
          *reinterpret_cast<uint4*>(dst + AM * 128) = hi_p;
        }
        mark(T_ATT_Q);
        tc_fences();
        worker_sync();
        tc_issue(s_base, AM, false, false, true);
        if (!tc_wait()) return false;
        if (nt > 1) tc_fetch(kmap, s_base + K_OFF, &sh->att_k_bar, kvh, key_lo + TK, pol, el);   // S of tile 0 exists: K is free

        const bool rows_here = pb * AM + quarter * qrows < Pn;
        float m_used = -INFINITY, l_part = 0.f;
        bool failed = false;   // this thread's last wait for the multiplies ran out
        for (int t = 0; t < nt; ++t) {
          const int nv = key_hi - (key_lo + t * TK) - half * 32;   // columns of this half that are keys of the run
          float s[32];
          float mx = -INFINITY;
          if (rows_here) {
            tmem_ld32(t_row + S_COL + half * 32, s);
            float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int k = 0; k < 32; ++k)
              if (k < nv) m4[k & 3] = fmaxf(m4[k & 3], s[k]);
            mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
          }
          if (t == 0) {   // the row's maximum over both halves of the first tile
            if (lane_ok) xch[half * TC_ROWS + row] = mx;
            worker_sync();
            m_used = fmaxf(mx, xch[(half ^ 1) * TC_ROWS + row]);
          }
          float rs = 0.f;
          if (rows_here) {
            if (nv >= 32) rs = tc_weights<false>(s, nv, m_used, scratch + P_OFF + row * 128, row & 7, half, lane_ok);
            else rs = tc_weights<true>(s, nv, m_used, scratch + P_OFF + row * 128, row & 7, half, lane_ok);
          }
          tc_fences();
          if (worker_or(failed || (rows_here && lane_ok && t > 0 && mx > m_used + 8.f))) {
            if (!worker_and(!failed)) return false;
            // some row of this CTA outgrew its maximum: every row looks at both halves again
            if (lane_ok) xch[half * TC_ROWS + row] = mx;
            worker_sync();
            const float m_new = fmaxf(m_used, fmaxf(mx, xch[(half ^ 1) * TC_ROWS + row]));
            const bool moved = m_new > m_used + 8.f;   // the same answer in both halves of the row
            if (rows_here && __any_sync(0xffffffffu, moved)) {
              const float corr = moved ? exp2f(m_used - m_new) : 1.f;
              if (moved) { l_part *= corr; m_used = m_new; }
#pragma unroll
              for (int q = 0; q < HD / 32; ++q) {   // this half's 64 columns of O
                float o[16];
                tc::tmem_ld16(t_row + O_COL + half * (HD / 2) + q * 16, o);
#pragma unroll
                for (int k = 0; k < 16; ++k) o[k] *= corr;
                tmem_st16(t_row + O_COL + half * (HD / 2) + q * 16, o);
              }
              asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
              rs = tc_weights<true>(s, nv, m_used, scratch + P_OFF + row * 128, row & 7, half, lane_ok);
            }
            tc_fences();
            worker_sync();
          }
          l_part += rs;
          tc_issue(s_base, AM, true, t > 0, t + 1 < nt);
          failed = !tc_poll();
          // the multiplies just waited for were the last readers of V (t) and K (t + 1)
          if (t + 1 < nt) tc_fetch(vmap, s_base + V_OFF, &sh->att_v_bar, kvh, key_lo + (t + 1) * TK, pol, el);
          if (t + 2 < nt) tc_fetch(kmap, s_base + K_OFF, &sh->att_k_bar, kvh, key_lo + (t + 2) * TK, pol, el);
        }
        mark(T_ATT_TILES);
        if (lane_ok) xch[half * TC_ROWS + row] = l_part;
        if (!worker_and(!failed)) return false;
        if (rows_here) {
          const float l_sum = l_part + xch[(half ^ 1) * TC_ROWS + row];
          const int pp = pb * AM + row;
          const int rr = rdG.div(min(pp, Pn - 1));
          const int hq = kvh * Gq + (min(pp, Pn - 1) - rr * Gq);
          const long long idx = ((long long)rr * c.nq + hq) * c.chunk_cap + run;
          uint4* pa = reinterpret_cast<uint4*>(p.b.att_acc + idx * (HD / 2)) + half * (HD / 8);
#pragma unroll
          for (int q = 0; q < HD / 32; ++q) {
            float o[16];
            tc::tmem_ld16(t_row + O_COL + half * (HD / 2) + q * 16, o);
            if (pp < Pn && lane_ok) {
#pragma unroll
              for (int k = 0; k < 4; ++k)
                __stcg(pa + q * 4 + k, make_uint4(pack2(o[4 * k], o[4 * k + 1]), tag, pack2(o[4 * k + 2], o[4 * k + 3]), tag));
            }
          }
          if (pp < Pn && lane_ok && half == 0) __stcg(p.b.att_ml + idx, make_uint4(__float_as_uint(m_used), tag, __float_as_uint(l_sum), tag));
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      worker_sync();
      return true;
    }
  }

  // All chunks of a (row, query head) pair merged by one warp; the pairs are dealt out to all CTAs and,
  // inside a CTA, to its warps.  There is no flag to wait for: the warp reads the partial results until
  // every piece carries this job's tag (see attention_partials), one trip to L2 when they are there.
  __device__ bool attention_merge(const Job& J, int jb) {
    constexpr int LANES = HD / 4;    // lanes that hold four head dimensions each
    constexpr int MB = 17;           // partials fetched per trip to L2 (a 512-key context has 17)
    const Cfg& c = p.c;
    const int k_tot = J.uniform ? J.C + J.T : J.C;
    const int n_runs = (k_tot + c.run_len - 1) / c.run_len;
    const int n_chunks = n_runs + (J.uniform ? 0 : (J.R + ATT_KEYS - 1) / ATT_KEYS);
    const uint32_t tag = p.launch_tag | (uint32_t)(jb + 1);
    const uint32_t n_poll = 2u * sh->wait_slow;
    bool all_ok = true;
    for (int u = (int)blockIdx.x + c.G * ww; u < J.R * c.nq; u += c.G * 8) {
      const long long pr = u;        // = row * nq + query head
      const uint4* ml = p.b.att_ml + pr * c.chunk_cap;
      const uint4* acc = reinterpret_cast<const uint4*>(p.b.att_acc + pr * c.chunk_cap * (HD / 2)) + lane;
      uint4 v0, v1, a[MB];
      // one trip: maxima / sums of all chunks and the first MB partial outputs; repeated until all are tagged
      auto load_trip = [&](int ch0, bool with_ml) -> bool {
        bool ok = true;
        if (with_ml) {
          v0 = v1 = make_uint4(0xff800000u, tag, 0u, tag);   // (-inf, 0)
          if (lane < n_chunks) v0 = __ldcg(ml + lane);
          if (lane + 32 < n_chunks) v1 = __ldcg(ml + lane + 32);
        }
#pragma unroll
        for (int e = 0; e < MB; ++e) {
          a[e] = make_uint4(0u, tag, 0u, tag);
          if (ch0 + e < n_chunks && lane < LANES) a[e] = __ldcg(acc + (long long)(ch0 + e) * LANES);
        }
        if (with_ml) ok = v0.y == tag && v0.w == tag && v1.y == tag && v1.w == tag;
#pragma unroll
        for (int e = 0; e < MB; ++e) ok = ok && a[e].y == tag && a[e].w == tag;
        return __all_sync(0xffffffffu, ok);
      };
      auto poll_trip = [&](int ch0, bool with_ml) -> bool {
        for (uint32_t it = 0; it < n_poll; ++it) {
          if (load_trip(ch0, with_ml)) return true;
          if ((it & 15u) == 15u && aborted(p.ctl, sh)) return false;
          __nanosleep(POLL_NS);
        }
        raise_abort(p.ctl, sh, true);
        return false;
      };
      if (!poll_trip(0, true)) { all_ok = false; break; }
      const float m0 = __uint_as_float(v0.x), m1 = __uint_as_float(v1.x);
      const float mx = warp_max(fmaxf(m0, m1));
      const float w0 = m0 == -INFINITY ? 0.f : exp2f(m0 - mx);
      const float w1 = m1 == -INFINITY ? 0.f : exp2f(m1 - mx);
      const float den = warp_sum(w0 * __uint_as_float(v0.z) + w1 * __uint_as_float(v1.z));
      float num[4] = {0.f, 0.f, 0.f, 0.f};
      bool ok = true;
      for (int ch0 = 0; ch0 < n_chunks; ch0 += MB) {
        if (ch0 > 0 && !poll_trip(ch0, false)) { ok = false; break; }
#pragma unroll
        for (int e = 0; e < MB; ++e) {
          const int ch = ch0 + e;
          const float wa = __shfl_sync(0xffffffffu, w0, ch & 31), wb = __shfl_sync(0xffffffffu, w1, ch & 31);
          const float w = ch < 32 ? wa : wb;
          const float2 d01 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&a[e].x));
          const float2 d23 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&a[e].z));
          num[0] = fmaf(w, d01.x, num[0]); num[1] = fmaf(w, d01.y, num[1]);
          num[2] = fmaf(w, d23.x, num[2]); num[3] = fmaf(w, d23.y, num[3]);
        }
      }
      if (!ok) { all_ok = false; break; }
      const float inv = 1.0f / den;
      if (lane < LANES)
        *reinterpret_cast<uint2*>(p.b.attn + pr * HD + lane * 4) = pack4(num[0] * inv, num[1] * inv, num[2] * inv, num[3] * inv);
    }
    if (!worker_and(all_ok)) return false;
    publish(F_MERGE, jb + 1);
    return true;
  }

  // greedy token of each head row from every CTA's best (CTA 0, one warp per row)
  __device__ bool head_merge(const Job& J, int jb) {
    const Cfg& c = p.c;
    publish(F_HEAD, jb + 1);
    if (blockIdx.x != 0) return true;
    if (!wait_all(F_HEAD, J.tgt[F_HEAD])) return false;
    const int* vlo = split_lo(S_V);
    for (int r = ww; r < J.R; r += 8) {
      float best = -INFINITY;
      int bi = 0x7fffffff;
      for (int cc = lane; cc < c.G; cc += 32) {
        if (__ldg(vlo + cc + 1) <= __ldg(vlo + cc)) continue;
        const float4 v = __ldcg(p.b.head_best + (long long)cc * MAX_ROWS + r);
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
      for (int cc = lane; cc < c.G; cc += 32) {
        if (__ldg(vlo + cc + 1) <= __ldg(vlo + cc)) continue;
        const float4 v = __ldcg(p.b.head_best + (long long)cc * MAX_ROWS + r);
        se += v.z * __expf(v.x - best);
      }
      se = warp_sum(se);
      if (lane == 0) {
        J.argmax_out[r] = bi;
        if (J.top1_out) J.top1_out[r] = 1.0f / se;
      }
    }
    return true;
  }

  // ---- the job list
  __device__ bool run() {
    const Cfg& c = p.c;
    const TileDesc* tiles = reinterpret_cast<const TileDesc*>(p.tabs + c.tiles_off);
    float keep_y[RB], keep_s[RB];
#pragma unroll
    for (int k = 0; k < RB; ++k) { keep_y[k] = 0.f; keep_s[k] = 0.f; }
    for (int jb = 0; jb < p.n_jobs; ++jb) {
      // the job descriptor goes to shared memory and from there into a local copy: its fields
      // must not look as if a store to global memory could change them
      worker_sync();
      {
        const int* src = reinterpret_cast<const int*>(p.jobs + jb);
        for (int k = wtid; k < (int)(sizeof(Job) / 4); k += WORKERS) sh->job_words[k] = __ldg(src + k);
      }
      worker_sync();
      const Job J = *reinterpret_cast<const Job*>(sh->job_words);
      n_mark = jb;
      mark(T_START);
      if (J.type == JOB_SELECT) {
        if (!dp_step(J, jb, false, keep_y, keep_s)) return false;
        continue;
      }
      if (J.type == JOB_HEAD) {
        Phase P;
        P.init(p, J, 0);
        for (int t = 0; t < P.n_tiles; ++t)
          if (!epilogue(J, jb, P, tiles[P.tile0 + t], t, keep_y, keep_s)) return false;
        if (!head_merge(J, jb)) return false;
        mark(T_HEAD);
        continue;
      }
      if (J.prep) prep(J, jb + 1);
      for (int ph = 0; ph < 4; ++ph) {
        Phase P;
        P.init(p, J, ph);
        if (ph == G_O && J.dp) {
          // idle time (the o product is being multiplied): this CTA's share of the sums of this job's
          // Eq. 2 step over the skip candidates, which the previous step left in g
          const int f_lo = __ldg(split_lo(S_D) + blockIdx.x), f_hi = __ldg(split_lo(S_D) + blockIdx.x + 1);
          const int fl = feat_local(f_hi - f_lo, ww & 3, lane);
          pre_sums(jb, (J.ell + (J.diag ? 1 : 0)) * J.T, J.T, J.x_i, J.x_im1, J.x_tok_stride, J.x_im1_stride, J.g_prev, fl >= 0,
                   f_lo + fl);
        }
        for (int t = 0; t < P.n_tiles; ++t)
          if (!epilogue(J, jb, P, tiles[P.tile0 + t], t, keep_y, keep_s)) return false;
        mark(ph == G_QKV ? T_QKV : (ph == G_O ? T_O : (ph == G_GU ? T_GU : T_DOWN)));
        if (ph == G_QKV) {
          publish(F_QKV, jb + 1);
          if constexpr (TC) {   // (only launched for searches over long contexts: no forward-pass jobs)
            if (!attention_tc(J, jb)) return false;
            if (!attention_partials<true>(J, jb)) return false;
          } else {
            if (!attention_partials(J, jb)) return false;
          }
          mark(T_ATT_PUB);
          if (!attention_merge(J, jb)) return false;
          mark(T_MERGE);
        } else if (ph == G_O) {
          publish(F_O, jb + 1);
        } else if (ph == G_GU) {
          publish(F_GU, jb + 1);
        } else {
          if (J.dp) {
            if (!dp_step(J, jb, P.n_tiles > 0, keep_y, keep_s)) return false;
          } else {
            publish(F_DOWN, jb + 1);
          }
          mark(T_DP_DONE);
        }
      }
    }
    return true;
  }
};

// ------------------------------------------------------------------ the kernel
constexpr int REGS_SPECIAL = 72;
constexpr int REGS_WORKER = (THREADS * 168 - 128 * REGS_SPECIAL) / 256 / 8 * 8;
static_assert(THREADS == 384 && WORKER_T0 == 128, "register split assumes one special and two worker warp groups");
static_assert(128 * REGS_SPECIAL + 256 * REGS_WORKER <= THREADS * 168, "register pool of the CTA");

template <bool TR, int HD, bool TC>
__global__ void __launch_bounds__(THREADS, 1)
engine_kernel(const __grid_constant__ CUtensorMap map_xn_a, const __grid_constant__ CUtensorMap map_attn,
              const __grid_constant__ CUtensorMap map_xn_m, const __grid_constant__ CUtensorMap map_act,
              const __grid_constant__ CUtensorMap map_head, const __grid_constant__ CUtensorMap map3_xn_a,
              const __grid_constant__ CUtensorMap map3_attn, const __grid_constant__ CUtensorMap map3_xn_m,
              const __grid_constant__ CUtensorMap map3_act, const __grid_constant__ CUtensorMap map3_head,
              const __grid_constant__ CUtensorMap map_xn_a2, const __grid_constant__ CUtensorMap map3_xn_a2,
              const __grid_constant__ Params p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ Shared sh;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint8_t* ring = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t ring_base = tc::smem_u32(ring);
  uint8_t* scratch = ring + (size_t)p.c.ring_pages * PAGE;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NB; ++s) {
      tc::mbar_init(tc::smem_u32(&sh.full[s]), 2);   // weight rows + operand tile
      tc::mbar_init(tc::smem_u32(&sh.empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      tc::mbar_init(tc::smem_u32(&sh.acc_full[b]), 1);
      tc::mbar_init(tc::smem_u32(&sh.acc_empty[b]), 1);
    }
    tc::mbar_init(tc::smem_u32(&sh.att_bar), 1);
    tc::mbar_init(tc::smem_u32(&sh.att_k_bar), 1);
    tc::mbar_init(tc::smem_u32(&sh.att_v_bar), 1);
    sh.abort = 0;
    sh.wait_fast = p.wait_fast;
    sh.wait_slow = p.wait_slow;
    sh.a_issued = 0;
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

  // The register file is re-divided between the warp groups: the four loader / issuer warps keep
  // REGS_SPECIAL registers per thread, the two worker groups take the rest
  // (128 * REGS_SPECIAL + 256 * REGS_WORKER = 384 * 168, the allocation the CTA was launched with).
  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_SPECIAL));
    if (warp == 0) {
      producer_a(p, &sh, ring_base, lane);
    } else if (warp == 1) {
      const CUtensorMap* bmaps[6] = {&map_xn_a, &map_attn, &map_xn_m, &map_act, &map_head, &map_xn_a2};
      const CUtensorMap* bmaps3[6] = {&map3_xn_a, &map3_attn, &map3_xn_m, &map3_act, &map3_head, &map3_xn_a2};
      producer_b<TR>(p, &sh, ring_base, bmaps, bmaps3, lane);
    } else if (warp == 2) {
      mma_issuer<TR>(p, &sh, ring_base, tmem_base, lane);
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_WORKER));
    Worker<TR, HD, TC> w{p, &sh, scratch, tmem_base, (int)threadIdx.x - WORKER_T0, warp - 4, lane, 0u, 0};
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
