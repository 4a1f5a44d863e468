// C ABI of the layer-skip search library: context, argument checks and the host-side
// launch sequences.  Every arithmetic step runs in the kernels of kernels.cuh and
// gemm_tc.cuh; this file only sequences launches on the caller's stream.
#include "../../include/clasp.h"

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <array>
#include <cstring>
#include <map>
#include <mutex>
#include <tuple>
#include <vector>

#include "gemm_tc.cuh"
#include "kernels.cuh"
#include "engine2.cuh"
#include "sampling.cuh"

namespace {

using bf16 = __nv_bfloat16;
constexpr int MAX_COUNTERS = 4096;   // tiles of one GEMM launch that may use split-K
constexpr size_t PARTIAL_FLOATS = (size_t)296 * 2 * 128 * 128 + (1 << 20);

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

struct LayerMaps {
  CUtensorMap wq, wk, wv, wo, w_gate, w_up, w_down;
};

struct Workspace {
  int* status;
  int* counters;
  void* xn;
  float* qkv;
  void* own_k;
  void* own_v;
  void* attn;
  float* x1;
  void* act;
  float* G;
  float* hping;
  float* hpong;
  float* grow[2];
  uint8_t* choice;
  float2* rope;
  float* att_acc;
  float2* att_ml;
  float* logits;
  float* partial;
  // persistent layer engine
  void* xn_m;
  uint2* e_att_acc;
  uint4* e_att_ml;
  size_t e_att_bytes;
  long long* ss_a;
  long long* ss_m;
  size_t acc_bytes;
  long long* cosacc;
  size_t cosacc_bytes;
  float4* head_best;
  int* flags;
  clasp::pk::Ctl* ctl;
  CUtensorMap* wmaps;
  CUtensorMap* kvmaps;   // tensor-core attention: key and value cache maps of each layer job of the launch
  clasp::pk::Job* jobs;
  int* tabs;
  clasp::smp::AcceptScratch* spec;
  int e_chunk_cap;
  int e_run_len;
  int e_rcap;
  size_t bytes;
};

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

bool config_ok(const clasp_config* c) {
  if (!c) return false;
  if (c->L < 1 || c->d_model < 8 || c->d_model % 8 || c->d_ffn < 8 || c->d_ffn % 8) return false;
  if (c->n_kv_heads < 1 || c->n_q_heads < c->n_kv_heads || c->n_q_heads % c->n_kv_heads) return false;
  if (c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->vocab < 1 || c->max_ctx < 1 || c->max_rows < 1 || c->max_head_rows < 1) return false;
  if (c->max_M < 0 || c->max_M > c->L || c->max_T < 1) return false;
  if (c->dtype != CLASP_FP32 && c->dtype != CLASP_BF16) return false;
  return true;
}

constexpr int ENGINE_MAX_CTAS = clasp::pk::MAX_CTAS;
constexpr size_t ENGINE_TAB_INTS = 96 * 1024;

// Lays the workspace out; with base == nullptr only the size is computed.
Workspace carve(const clasp_config& c, uint8_t* base) {
  Workspace w{};
  size_t off = 0;
  auto take = [&](size_t bytes) -> void* {
    void* p = base ? base + off : nullptr;
    off += align_up(bytes, 256);
    return p;
  };
  const size_t esz = c.dtype == CLASP_BF16 ? 2 : 4;
  const size_t R = c.max_rows, d = c.d_model;
  const size_t qd = (size_t)c.n_q_heads * c.head_dim, kvd = (size_t)c.n_kv_heads * c.head_dim;
  const size_t grows = (size_t)(c.max_M + 1) * c.max_T;
  w.status = (int*)take(256);
  w.counters = (int*)take(MAX_COUNTERS * sizeof(int));
  w.xn = take(R * d * esz);
  w.qkv = (float*)take(R * (qd + 2 * kvd) * 4);
  w.own_k = take(R * kvd * esz);
  w.own_v = take(R * kvd * esz);
  w.attn = take(R * qd * esz);
  w.x1 = (float*)take(R * d * 4);
  w.act = take(R * (size_t)c.d_ffn * esz);
  w.G = (float*)take(R * d * 4);
  w.hping = (float*)take(R * d * 4);
  w.hpong = (float*)take(R * d * 4);
  w.grow[0] = (float*)take(grows * d * 4);
  w.grow[1] = (float*)take(grows * d * 4);
  w.choice = (uint8_t*)take((size_t)(c.L + 1) * (c.max_M + 1));
  w.rope = (float2*)take(R * (c.head_dim / 2) * sizeof(float2));
  const size_t att_chunks = clasp::ATT_MAX_CACHE_CHUNKS + (R + clasp::ATT_KEYS - 1) / clasp::ATT_KEYS;
  w.att_acc = (float*)take(R * c.n_q_heads * att_chunks * (size_t)c.head_dim * 4);
  w.att_ml = (float2*)take(R * c.n_q_heads * att_chunks * sizeof(float2));
  w.logits = (float*)take((size_t)c.max_head_rows * c.vocab * 4);
  w.partial = (float*)take(PARTIAL_FLOATS * 4);
  w.spec = (clasp::smp::AcceptScratch*)take(sizeof(clasp::smp::AcceptScratch));
  if (c.dtype == CLASP_BF16) {
    // buffers of the persistent layer engine (per-CTA tables sized for ENGINE_MAX_CTAS)
    namespace pk = clasp::pk;
    const size_t Re = R < (size_t)pk::MAX_ROWS ? R : (size_t)pk::MAX_ROWS;
    const size_t rcap = align_up(Re, 16);
    const size_t G = ENGINE_MAX_CTAS;
    w.e_rcap = (int)rcap;
    w.xn_m = take(R * d * 2);
    w.e_run_len = pk::ATT_KEYS * ((c.max_ctx + pk::ATT_KEYS * 32 - 1) / (pk::ATT_KEYS * 32));
    w.e_chunk_cap = 32 + (int)((rcap + pk::ATT_KEYS - 1) / pk::ATT_KEYS);   // at most 32 runs of cache keys + own rows
    // partial attention outputs (two bf16 values + tag per 8 bytes) and their (maximum, tag, sum, tag): contiguous
    w.e_att_acc = (uint2*)take(rcap * c.n_q_heads * (size_t)w.e_chunk_cap * c.head_dim * 4);
    w.e_att_ml = (uint4*)take(rcap * c.n_q_heads * (size_t)w.e_chunk_cap * sizeof(uint4));
    w.e_att_bytes = (size_t)((uint8_t*)w.e_att_ml - (uint8_t*)w.e_att_acc) +
                    align_up(rcap * c.n_q_heads * (size_t)w.e_chunk_cap * sizeof(uint4), 256);
    // fixed-point accumulators, zeroed before every launch: ss_a, ss_m, cosacc are contiguous
    const size_t ss_bytes = align_up(((size_t)c.L + 5) * rcap * sizeof(long long), 256);
    w.ss_a = (long long*)take(ss_bytes);
    w.ss_m = (long long*)take(ss_bytes);
    w.cosacc_bytes = ((size_t)c.L + 4) * (rcap + pk::MAX_ROWS) * 5 * sizeof(long long);
    w.cosacc = (long long*)take(w.cosacc_bytes);
    w.acc_bytes = (size_t)((uint8_t*)w.cosacc - (uint8_t*)w.ss_a) + align_up(w.cosacc_bytes, 256);
    w.head_best = (float4*)take(G * pk::MAX_ROWS * sizeof(float4));
    w.flags = (int*)take(pk::N_FLAGS * (G + 32) * sizeof(int));
    w.ctl = (pk::Ctl*)take(256);
    w.wmaps = (CUtensorMap*)take(((size_t)c.L * 7 + 1) * pk::N_HEIGHTS * 2 * sizeof(CUtensorMap));
    w.kvmaps = (CUtensorMap*)take(((size_t)c.L + 4) * 2 * sizeof(CUtensorMap));
    w.jobs = (pk::Job*)take(((size_t)c.L + 4) * sizeof(pk::Job));
    w.tabs = (int*)take(ENGINE_TAB_INTS * sizeof(int));
  }
  w.bytes = off;
  return w;
}

}  // namespace

struct clasp_ctx {
  clasp_config cfg;
  cudaStream_t stream;
  Workspace ws;
  std::vector<clasp_layer_weights> layers;
  std::vector<uint8_t> loaded;
  std::vector<LayerMaps> maps;
  const void* embed = nullptr;
  const float* final_norm = nullptr;
  const void* lm_head = nullptr;
  CUtensorMap lm_head_map;
  bool use_tc = false;
  EncodeTiledFn encode = nullptr;
  std::map<std::tuple<const void*, int, int>, CUtensorMap> xmaps;
  int64_t launches = 0;
  bool profiling = false;
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> prof_events;
  double prof_bytes = 0.0;
  int cta_cap = 296;
  int smem_budget = 110 * 1024;
  int num_sms = 148;
  // persistent layer engine
  bool use_engine = false;
  int e_G = 0;              // CTAs of the cooperative grid (one per SM)
  int e_static_smem = 0;
  const void* e_kernel[4] = {nullptr, nullptr, nullptr, nullptr};   // the layer kernel for this head dimension: plain, with step
                                                                    // stamps; [2], [3]: the same with the tensor-core attention
  int e_split_lo[clasp::pk::N_SPLITS], e_split_units[clasp::pk::N_SPLITS], e_tile_idx[5], e_tiles_off = 0,
      e_kpi[5], e_use3d[5], e_wpages[5];
  int e_heights[8][clasp::pk::N_HEIGHTS];   // tile heights per matrix slot (wq wk wv wo gate up down head)
  std::vector<CUtensorMap> e_wmaps_host;
  std::vector<CUtensorMap> e_kvmaps_host;
  bool e_wmaps_dirty = true;
  std::map<int, std::array<CUtensorMap, 10>> e_bmaps;          // by BN: 2-D maps of the four operands, then 3-D, then xn with 2 BN rows (2-D, 3-D)
  std::map<std::pair<int, int>, std::array<CUtensorMap, 2>> e_headmaps;  // by (row offset, BN): 2-D, 3-D
  std::vector<clasp::pk::Job> e_jobs;
  unsigned long long* e_trace = nullptr;
  int e_trace_cap = 0;
  uint32_t wait_limit = 0;   // 0: the kernels' default wait limits
  uint32_t launch_seq = 0;   // launches of the persistent kernel so far (tags of the attention's partial results)
};

namespace {

#define CUDA_TRY(expr)                              \
  do {                                              \
    cudaError_t e__ = (expr);                       \
    if (e__ != cudaSuccess) return CLASP_ERR_CUDA;  \
  } while (0)

int launch_check(clasp_ctx* ctx, int n = 1) {
  ctx->launches += n;
  return cudaGetLastError() == cudaSuccess ? CLASP_OK : CLASP_ERR_CUDA;
}

// 2-D bf16 tensor map over a row-major [rows, cols] matrix, box [box_rows x 64 cols],
// 128-byte swizzle, zero fill outside the matrix.
int make_map(clasp_ctx* ctx, const void* ptr, int rows, int cols, int box_rows, CUtensorMap* out) {
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)clasp::tc::BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = ctx->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides,
                           box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? CLASP_OK : CLASP_ERR_CUDA;
}

// 3-D bf16 tensor map over the same matrix seen as {64 columns, rows, K/64 chunks} (strides
// {cols*2, 128} bytes): a box {64, box_rows, box_chunks} lands in shared memory as box_chunks
// consecutive [box_rows x 128 B] swizzled tiles.  Needs cols % 64 == 0.
int make_map3(clasp_ctx* ctx, const void* ptr, int rows, int cols, int box_rows, int box_chunks, CUtensorMap* out) {
  cuuint64_t dims[3] = {64, (cuuint64_t)rows, (cuuint64_t)(cols / 64)};
  cuuint64_t strides[2] = {(cuuint64_t)cols * 2, 128};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, (cuuint32_t)box_chunks};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = ctx->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? CLASP_OK : CLASP_ERR_CUDA;
}

struct GemmCall {
  const void* x = nullptr;  // [R, K] operand dtype, contiguous
  int R = 0, K = 0;
  int n_mats = 1;
  const void* w[3] = {nullptr, nullptr, nullptr};
  const CUtensorMap* wmap[3] = {nullptr, nullptr, nullptr};
  int N[3] = {0, 0, 0};
  int col_off[3] = {0, 0, 0};
  int epi = clasp::EPI_STORE;
  const void* w2 = nullptr;  // SwiGLU: the "up" matrix
  const CUtensorMap* w2map = nullptr;
  float* yf = nullptr;
  int64_t ldy = 0;
  const float* resid = nullptr;
  int64_t ldr = 0;
  void* yo = nullptr;
  int64_t ldo = 0;
};

template <typename TW, int EPI>
int gemm_simt_one(clasp_ctx* ctx, const GemmCall& g, int m) {
  constexpr int WARPS = 8, RB = 4;
  const int N = g.N[m];
  dim3 grid((N + WARPS - 1) / WARPS), block(WARPS * 32);
  clasp::gemm_simt_kernel<TW, EPI, RB><<<grid, block, 0, ctx->stream>>>(
      (const TW*)g.x, g.K, (const TW*)g.w[m], (const TW*)g.w2, g.R, N, g.K,
      g.yf ? g.yf + g.col_off[m] : nullptr, g.ldy, g.resid ? g.resid + g.col_off[m] : nullptr, g.ldr,
      g.yo ? (TW*)g.yo + g.col_off[m] : nullptr, g.ldo);
  return launch_check(ctx);
}

template <typename TW>
int gemm_simt(clasp_ctx* ctx, const GemmCall& g) {
  for (int m = 0; m < g.n_mats; ++m) {
    int rc;
    if (g.epi == clasp::EPI_STORE) rc = gemm_simt_one<TW, clasp::EPI_STORE>(ctx, g, m);
    else if (g.epi == clasp::EPI_RESID) rc = gemm_simt_one<TW, clasp::EPI_RESID>(ctx, g, m);
    else rc = gemm_simt_one<TW, clasp::EPI_SWIGLU>(ctx, g, m);
    if (rc) return rc;
  }
  return CLASP_OK;
}

int gemm_tc(clasp_ctx* ctx, const GemmCall& g) {
  using namespace clasp::tc;
  const int dual = g.epi == clasp::EPI_SWIGLU ? 1 : 0;
  const int rb_max = dual ? 128 : 256;
  int tiles_total = 0, n_total = 0;
  Params p{};
  for (int m = 0; m < 3; ++m) {
    p.N[m] = m < g.n_mats ? g.N[m] : 0;
    p.tiles[m] = (p.N[m] + BM - 1) / BM;
    p.col_off[m] = m < g.n_mats ? g.col_off[m] : 0;
    tiles_total += p.tiles[m];
    if (m < g.n_mats && g.col_off[m] + g.N[m] > n_total) n_total = g.col_off[m] + g.N[m];
  }
  p.K = g.K;
  p.k_chunks = (g.K + BK - 1) / BK;
  // splits: a function of (N, K) only, so a row's sum never depends on the batch
  int splits = ctx->cta_cap / tiles_total;
  const int max_splits = p.k_chunks / 4 > 1 ? p.k_chunks / 4 : 1;
  if (splits > max_splits) splits = max_splits;
  if (splits < 1) splits = 1;
  if (splits > 1 && tiles_total > MAX_COUNTERS) splits = 1;
  p.dual = dual;
  p.n_mats = g.n_mats;
  p.epi = g.epi;
  p.n_total = n_total;
  p.ldy = g.ldy;
  p.ldr = g.ldr;
  p.ldo = g.ldo;
  p.counters = ctx->ws.counters;
  p.status = ctx->ws.status;
  p.partial = ctx->ws.partial;
  p.spin_fast = ctx->wait_limit ? (ctx->wait_limit < SPIN_FAST ? ctx->wait_limit : SPIN_FAST) : SPIN_FAST;
  p.spin_slow = ctx->wait_limit ? ctx->wait_limit : SPIN_SLOW;
  for (int r0 = 0; r0 < g.R; r0 += rb_max) {
    const int Rb = g.R - r0 < rb_max ? g.R - r0 : rb_max;
    p.R = Rb;
    p.BN = Rb <= 16 ? 16 : (Rb + 15) / 16 * 16;
    p.splits = splits;
    if ((size_t)splits * (dual + 1) * Rb * n_total > PARTIAL_FLOATS) p.splits = 1;
    const int stage_bytes = A_TILE_BYTES * (dual + 1) + p.BN * BK * 2;
    int stages = ctx->smem_budget / stage_bytes;
    if (stages > 8) stages = 8;
    if (stages < 2) stages = 2;
    const int per_cta = (p.k_chunks + p.splits - 1) / p.splits;
    if (stages > per_cta) stages = per_cta < 1 ? 1 : per_cta;
    p.stages = stages;
    const size_t smem = (size_t)stages * stage_bytes + 1024;
    const bf16* xb = (const bf16*)g.x + (size_t)r0 * g.K;
    auto key = std::make_tuple((const void*)xb, g.K, Rb * 1024 + p.BN);
    auto it = ctx->xmaps.find(key);
    if (it == ctx->xmaps.end()) {
      CUtensorMap mp;
      if (make_map(ctx, xb, Rb, g.K, p.BN, &mp)) return CLASP_ERR_CUDA;
      it = ctx->xmaps.emplace(key, mp).first;
    }
    p.yf = g.yf ? g.yf + (size_t)r0 * g.ldy : nullptr;
    p.resid = g.resid ? g.resid + (size_t)r0 * g.ldr : nullptr;
    p.yo = g.yo ? (bf16*)g.yo + (size_t)r0 * g.ldo : nullptr;
    const CUtensorMap* a0 = g.wmap[0];
    const CUtensorMap* a1 = dual ? g.w2map : (g.n_mats > 1 ? g.wmap[1] : g.wmap[0]);
    const CUtensorMap* a2 = g.n_mats > 2 ? g.wmap[2] : g.wmap[0];
    dim3 grid(tiles_total, p.splits), block(THREADS);
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (ctx->profiling) {
      if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return CLASP_ERR_CUDA;
      cudaEventRecord(e0, ctx->stream);
    }
    gemm_tc_kernel<<<grid, block, smem, ctx->stream>>>(*a0, *a1, *a2, it->second, p);
    if (ctx->profiling) {
      cudaEventRecord(e1, ctx->stream);
      ctx->prof_events.emplace_back(e0, e1);
      double nk = 0.0;
      for (int m = 0; m < g.n_mats; ++m) nk += (double)g.N[m] * g.K;
      ctx->prof_bytes += nk * 2.0 * (dual + 1);
    }
    int rc = launch_check(ctx);
    if (rc) return rc;
  }
  return CLASP_OK;
}

int gemm(clasp_ctx* ctx, const GemmCall& g) {
  if (g.R <= 0) return CLASP_OK;
  if (ctx->cfg.dtype == CLASP_FP32) return gemm_simt<float>(ctx, g);
  if (ctx->use_tc) return gemm_tc(ctx, g);
  return gemm_simt<bf16>(ctx, g);
}

template <typename TW, int HD>
int attention(clasp_ctx* ctx, int R, int T, int C, const clasp_kv_layer& kv, const TW* own_k, const TW* own_v,
              int64_t own_base) {
  const clasp_config& c = ctx->cfg;
  Workspace& ws = ctx->ws;
  const int qkvd = (c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
  // chunking is a function of C (cache) and R (own rows) only
  const int n_sub = (C + clasp::ATT_KEYS - 1) / clasp::ATT_KEYS;
  const int nsub = n_sub > 0 ? (n_sub + clasp::ATT_MAX_CACHE_CHUNKS - 1) / clasp::ATT_MAX_CACHE_CHUNKS : 1;
  const int n_cache_chunks = (n_sub + nsub - 1) / nsub;
  const int n_chunks = n_cache_chunks + (R + clasp::ATT_KEYS - 1) / clasp::ATT_KEYS;
  const int G = c.n_q_heads / c.n_kv_heads;
  const int pair_blocks = (R * G + clasp::ATT_PAIRS - 1) / clasp::ATT_PAIRS;
  constexpr int smem = clasp::att_smem_bytes<TW, HD>();
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(clasp::attn_tile_kernel<TW, HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) !=
        cudaSuccess)
      return CLASP_ERR_CUDA;
    attr_set = true;
  }
  dim3 grid(n_chunks, c.n_kv_heads, pair_blocks);
  clasp::attn_tile_kernel<TW, HD><<<grid, clasp::ATT_WARPS * 32, smem, ctx->stream>>>(
      ws.qkv, qkvd, ws.rope, (const TW*)kv.k, (const TW*)kv.v, C, own_k, own_v, own_base, R, T, c.n_q_heads,
      c.n_kv_heads, n_cache_chunks, nsub, n_chunks, ws.att_acc, ws.att_ml);
  int rc = launch_check(ctx);
  if (rc) return rc;
  clasp::attn_merge_kernel<TW, HD><<<R * c.n_q_heads, HD, 0, ctx->stream>>>(ws.att_acc, ws.att_ml, R, c.n_q_heads,
                                                                          n_chunks, (TW*)ws.attn);
  return launch_check(ctx);
}

template <typename TW>
int rmsnorm(clasp_ctx* ctx, const float* x, int64_t ldx, const float* w, int R, void* y) {
  clasp::rmsnorm_kernel<TW><<<R, 256, 0, ctx->stream>>>(x, ldx, w, ctx->cfg.d_model, ctx->cfg.rms_eps, (TW*)y);
  return launch_check(ctx);
}

int rope_table(clasp_ctx* ctx, int T, int pos0) {
  const int half = ctx->cfg.head_dim / 2, n = T * half;
  clasp::rope_table_kernel<<<(n + 255) / 256, 256, 0, ctx->stream>>>(ctx->ws.rope, T, half, pos0,
                                                                     (double)ctx->cfg.rope_theta);
  return launch_check(ctx);
}

// One decoder layer over S states x T rows (rope table for (T, pos0) already built).
// own K/V of the rows go to the cache at pos0.. when write_kv, else to scratch.
template <typename TW>
int run_layer(clasp_ctx* ctx, int l, const float* x, int64_t ldx, int S, int T, int C, int pos0,
              const clasp_kv_layer& kv, bool write_kv, float* out, int64_t ldo) {
  const clasp_config& c = ctx->cfg;
  Workspace& ws = ctx->ws;
  const clasp_layer_weights& W = ctx->layers[l];
  const bool tc = ctx->use_tc && c.dtype == CLASP_BF16;
  const LayerMaps* mp = tc ? &ctx->maps[l] : nullptr;
  const int R = S * T, d = c.d_model, qd = c.n_q_heads * c.head_dim, kvd = c.n_kv_heads * c.head_dim;
  const int qkvd = qd + 2 * kvd;
  int rc;
  if ((rc = rmsnorm<TW>(ctx, x, ldx, W.attn_norm, R, ws.xn))) return rc;
  {
    GemmCall g;
    g.x = ws.xn; g.R = R; g.K = d; g.n_mats = 3;
    g.w[0] = W.wq; g.w[1] = W.wk; g.w[2] = W.wv;
    if (tc) { g.wmap[0] = &mp->wq; g.wmap[1] = &mp->wk; g.wmap[2] = &mp->wv; }
    g.N[0] = qd; g.N[1] = kvd; g.N[2] = kvd;
    g.col_off[0] = 0; g.col_off[1] = qd; g.col_off[2] = qd + kvd;
    g.epi = clasp::EPI_STORE; g.yf = ws.qkv; g.ldy = qkvd;
    if ((rc = gemm(ctx, g))) return rc;
  }
  TW* own_k = write_kv ? (TW*)kv.k : (TW*)ws.own_k;
  TW* own_v = write_kv ? (TW*)kv.v : (TW*)ws.own_v;
  const int64_t own_base = write_kv ? pos0 : 0;
  clasp::kv_store_kernel<TW><<<R, 256, 0, ctx->stream>>>(ws.qkv, qkvd, ws.rope, T, c.n_q_heads, c.n_kv_heads,
                                                         c.head_dim, own_k, own_v, own_base);
  if ((rc = launch_check(ctx))) return rc;
  if (c.head_dim == 128) rc = attention<TW, 128>(ctx, R, T, C, kv, own_k, own_v, own_base);
  else rc = attention<TW, 64>(ctx, R, T, C, kv, own_k, own_v, own_base);
  if (rc) return rc;
  {
    GemmCall g;
    g.x = ws.attn; g.R = R; g.K = qd; g.n_mats = 1; g.w[0] = W.wo;
    if (tc) g.wmap[0] = &mp->wo;
    g.N[0] = d; g.epi = clasp::EPI_RESID; g.yf = ws.x1; g.ldy = d; g.resid = x; g.ldr = ldx;
    if ((rc = gemm(ctx, g))) return rc;
  }
  if ((rc = rmsnorm<TW>(ctx, ws.x1, d, W.mlp_norm, R, ws.xn))) return rc;
  {
    GemmCall g;
    g.x = ws.xn; g.R = R; g.K = d; g.n_mats = 1; g.w[0] = W.w_gate; g.w2 = W.w_up;
    if (tc) { g.wmap[0] = &mp->w_gate; g.w2map = &mp->w_up; }
    g.N[0] = c.d_ffn; g.epi = clasp::EPI_SWIGLU; g.yo = ws.act; g.ldo = c.d_ffn;
    if ((rc = gemm(ctx, g))) return rc;
  }
  {
    GemmCall g;
    g.x = ws.act; g.R = R; g.K = c.d_ffn; g.n_mats = 1; g.w[0] = W.w_down;
    if (tc) g.wmap[0] = &mp->w_down;
    g.N[0] = d; g.epi = clasp::EPI_RESID; g.yf = out; g.ldy = ldo; g.resid = ws.x1; g.ldr = d;
    if ((rc = gemm(ctx, g))) return rc;
  }
  return CLASP_OK;
}

int run_layer_any(clasp_ctx* ctx, int l, const float* x, int64_t ldx, int S, int T, int C, int pos0,
                  const clasp_kv_layer& kv, bool write_kv, float* out, int64_t ldo) {
  if (ctx->cfg.dtype == CLASP_FP32)
    return run_layer<float>(ctx, l, x, ldx, S, T, C, pos0, kv, write_kv, out, ldo);
  return run_layer<bf16>(ctx, l, x, ldx, S, T, C, pos0, kv, write_kv, out, ldo);
}

// float buffers are read and written with 16-byte vector accesses, K/V rows with 16-byte pieces
bool al16(const void* p) { return ((uintptr_t)p & 15) == 0; }
bool kv_aligned(const clasp_kv_layer* kv, int n) {
  for (int l = 0; l < n; ++l)
    if (!al16(kv[l].k) || !al16(kv[l].v)) return false;
  return true;
}

bool layers_ready(const clasp_ctx* ctx) {
  for (uint8_t b : ctx->loaded)
    if (!b) return false;
  return true;
}

// final norm + LM head + argmax over `rows` rows of x (float, stride ldx)
int run_head(clasp_ctx* ctx, const float* x, int64_t ldx, int rows, int32_t* argmax_out, float* top1,
             float* logits_out = nullptr) {
  const clasp_config& c = ctx->cfg;
  int rc;
  if (c.dtype == CLASP_FP32) rc = rmsnorm<float>(ctx, x, ldx, ctx->final_norm, rows, ctx->ws.xn);
  else rc = rmsnorm<bf16>(ctx, x, ldx, ctx->final_norm, rows, ctx->ws.xn);
  if (rc) return rc;
  GemmCall g;
  g.x = ctx->ws.xn; g.R = rows; g.K = c.d_model; g.n_mats = 1; g.w[0] = ctx->lm_head;
  g.wmap[0] = &ctx->lm_head_map; g.N[0] = c.vocab; g.epi = clasp::EPI_STORE;
  g.yf = ctx->ws.logits; g.ldy = c.vocab;
  if ((rc = gemm(ctx, g))) return rc;
  clasp::argmax_kernel<<<rows, 1024, 0, ctx->stream>>>(ctx->ws.logits, c.vocab, argmax_out, top1);
  if ((rc = launch_check(ctx))) return rc;
  if (logits_out)
    CUDA_TRY(cudaMemcpyAsync(logits_out, ctx->ws.logits, (size_t)rows * c.vocab * sizeof(float), cudaMemcpyDeviceToDevice,
                             ctx->stream));
  return CLASP_OK;
}

int embed_rows(clasp_ctx* ctx, const int32_t* tokens, int n, float* out, int64_t ldo) {
  const clasp_config& c = ctx->cfg;
  if (c.dtype == CLASP_FP32)
    clasp::embed_kernel<float><<<n, 256, 0, ctx->stream>>>(tokens, (const float*)ctx->embed, c.d_model, c.vocab, out, ldo);
  else
    clasp::embed_kernel<bf16><<<n, 256, 0, ctx->stream>>>(tokens, (const bf16*)ctx->embed, c.d_model, c.vocab, out, ldo);
  return launch_check(ctx);
}


// ---------------------------------------------------------------- persistent layer engine
// Host side of engine2.cuh: builds the job list of a call and launches the cooperative
// kernel once.  Used by the bf16 tensor-core configuration; the per-kernel sequences
// above remain for the fp32 model, for CLASP_FLAG_FORCE_SIMT and for shapes the engine
// does not take (more than 128 rows).
namespace pk = clasp::pk;

int engine_setup(clasp_ctx* ctx) {
  const clasp_config& c = ctx->cfg;
  ctx->use_engine = false;
  if (!ctx->use_tc || (c.flags & CLASP_FLAG_MULTI_KERNEL)) return CLASP_OK;
  int dev = 0, coop = 0, optin = 0;
  CUDA_TRY(cudaGetDevice(&dev));
  CUDA_TRY(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
  CUDA_TRY(cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
  if (!coop) return CLASP_OK;
  const int d = c.d_model, qd = c.n_q_heads * c.head_dim, kvd = c.n_kv_heads * c.head_dim;
  if (d % 8 || c.d_ffn % 8 || c.vocab % 8) return CLASP_OK;
  // the instantiations for this model's head dimension, without and with step stamps
  ctx->e_kernel[0] = c.head_dim == 128 ? (const void*)pk::engine_kernel<false, 128, false> : (const void*)pk::engine_kernel<false, 64, false>;
  ctx->e_kernel[1] = c.head_dim == 128 ? (const void*)pk::engine_kernel<true, 128, false> : (const void*)pk::engine_kernel<true, 64, false>;
  ctx->e_kernel[2] = c.head_dim == 128 ? (const void*)pk::engine_kernel<false, 128, true> : nullptr;
  ctx->e_kernel[3] = c.head_dim == 128 ? (const void*)pk::engine_kernel<true, 128, true> : nullptr;
  const int n_kern = c.head_dim == 128 ? 4 : 2;
  ctx->e_static_smem = 0;
  for (int k = 0; k < n_kern; ++k) {  // one shared-memory budget for both
    cudaFuncAttributes fa;
    CUDA_TRY(cudaFuncGetAttributes(&fa, ctx->e_kernel[k]));
    if ((int)fa.sharedSizeBytes > ctx->e_static_smem) ctx->e_static_smem = (int)fa.sharedSizeBytes;
  }
  const int dyn_max = optin - ctx->e_static_smem;
  if (dyn_max < 1024 + 64 * pk::PAGE + pk::SCRATCH_BYTES) return CLASP_OK;
  for (int k = 0; k < n_kern; ++k)
    CUDA_TRY(cudaFuncSetAttribute(ctx->e_kernel[k], cudaFuncAttributeMaxDynamicSharedMemorySize, dyn_max));
  int G = ctx->num_sms;
  if (G > ENGINE_MAX_CTAS) G = ENGINE_MAX_CTAS;
  // ---- feature splits and per-CTA tiles.  A CTA's range never straddles two weight matrices:
  // the CTAs of the q/k/v product are dealt to the three matrices in proportion to their rows.
  const int split_n[pk::N_SPLITS] = {qd + 2 * kvd, d, c.d_ffn, c.vocab};
  const int kind_split[5] = {pk::S_QKV, pk::S_D, pk::S_F, pk::S_D, pk::S_V};
  const int kind_K[5] = {d, qd, d, c.d_ffn, d};
  const int kind_slot0[5] = {0, 3, 4, 6, 7};   // first matrix slot of the kind
  std::vector<int> tab;
  std::vector<std::vector<int>> lo(pk::N_SPLITS);
  for (int s = 0; s < pk::N_SPLITS; ++s) {
    lo[s].assign(G + 1, 0);
    if (s == pk::S_QKV) {
      const int mat_n[3] = {qd, kvd, kvd};
      int share[3], given = 0;
      for (int m = 0; m < 3; ++m) { share[m] = (int)((long long)G * mat_n[m] / split_n[s]); if (share[m] < 1) share[m] = 1; given += share[m]; }
      for (int m = 0; given < G; m = (m + 1) % 3) { ++share[m]; ++given; }
      while (given > G) { int m = share[0] >= share[1] && share[0] >= share[2] ? 0 : (share[1] >= share[2] ? 1 : 2); --share[m]; --given; }
      if (G < 3) return CLASP_OK;
      int cc = 0, base = 0;
      for (int m = 0; m < 3; ++m) {
        const long long units = mat_n[m] / 8;
        for (int k = 0; k < share[m]; ++k) lo[s][cc + k] = base + (int)(units * k / share[m]) * 8;
        cc += share[m];
        base += mat_n[m];
      }
      lo[s][G] = base;
    } else {
      const long long units = split_n[s] / 8;
      for (int cc = 0; cc <= G; ++cc) lo[s][cc] = (int)(units * cc / G) * 8;
    }
    ctx->e_split_lo[s] = (int)tab.size();
    ctx->e_split_units[s] = split_n[s] / 8;
    tab.insert(tab.end(), lo[s].begin(), lo[s].end());
  }
  for (int cc = 0; cc < G; ++cc)
    if (lo[pk::S_D][cc + 1] - lo[pk::S_D][cc] > 128) return CLASP_OK;  // the Eq. 2 step takes one feature per thread
  std::vector<pk::TileDesc> tiles;
  std::vector<std::vector<int>> tidx(5, std::vector<int>(G + 1, 0));
  for (int sl = 0; sl < 8; ++sl)
    for (int h = 0; h < pk::N_HEIGHTS; ++h) ctx->e_heights[sl][h] = 0;
  for (int k = 0; k < 5; ++k) {
    const int s = kind_split[k];
    int mat_n[3] = {split_n[s], 0, 0}, n_mats = 1;
    if (k == pk::G_QKV) { mat_n[0] = qd; mat_n[1] = kvd; mat_n[2] = kvd; n_mats = 3; }
    int max_rows = 8;
    for (int cc = 0; cc < G; ++cc) {
      tidx[k][cc] = (int)tiles.size();
      for (int f0 = lo[s][cc]; f0 < lo[s][cc + 1]; f0 += 128) {
        const int n = std::min(128, lo[s][cc + 1] - f0);
        int m = 0, base = 0;
        while (m + 1 < n_mats && f0 >= base + mat_n[m]) { base += mat_n[m]; ++m; }
        if (f0 + n > base + mat_n[m]) return CLASP_OK;  // cannot happen: ranges are aligned to the matrices
        int* hts = ctx->e_heights[kind_slot0[k] + m];
        int hi = 0;
        while (hi < pk::N_HEIGHTS && hts[hi] != n && hts[hi] != 0) ++hi;
        if (hi == pk::N_HEIGHTS) return CLASP_OK;       // more distinct tile heights than maps per matrix
        hts[hi] = n;
        pk::TileDesc td{};
        td.f0 = f0; td.n_rows = (short)n; td.map_local = (short)(m * pk::N_HEIGHTS + hi); td.y0 = f0 - base;
        if (n > max_rows) max_rows = n;
        tiles.push_back(td);
      }
    }
    tidx[k][G] = (int)tiles.size();
    if (k == pk::G_GU)  // the up matrix is loaded with the gate matrix's heights
      for (int h = 0; h < pk::N_HEIGHTS; ++h) ctx->e_heights[5][h] = ctx->e_heights[4][h];
    const int a_pages = (k == pk::G_GU ? 2 : 1) * (max_rows / 8);
    ctx->e_wpages[k] = a_pages;   // weight pages of one chunk of the kind's tallest tile
    // ring items of about 32 KB of weights: every item costs the MMA issuers a barrier round trip, so
    // small items waste issue time, while items beyond a sixth of the ring leave too few in flight
    const int kpi_budget = 32, kpi_max = 8;
    int kpi = kpi_budget / a_pages;
    ctx->e_kpi[k] = kpi < 1 ? 1 : (kpi > kpi_max ? kpi_max : kpi);
    // (the gate/up product interleaves two matrices per chunk, which one box cannot deliver)
    ctx->e_use3d[k] = (k != pk::G_GU && kind_K[k] % 64 == 0 && ctx->e_kpi[k] > 1) ? 1 : 0;
  }
  for (int k = 0; k < 5; ++k) {
    ctx->e_tile_idx[k] = (int)tab.size();
    tab.insert(tab.end(), tidx[k].begin(), tidx[k].end());
  }
  static_assert(sizeof(pk::TileDesc) == 12, "table records are three ints");
  ctx->e_tiles_off = (int)tab.size();
  tab.resize(tab.size() + tiles.size() * 3);
  memcpy(tab.data() + ctx->e_tiles_off, tiles.data(), tiles.size() * sizeof(pk::TileDesc));
  if (tab.size() > ENGINE_TAB_INTS) return CLASP_OK;
  CUDA_TRY(cudaMemcpyAsync(ctx->ws.tabs, tab.data(), tab.size() * sizeof(int), cudaMemcpyHostToDevice, ctx->stream));
  CUDA_TRY(cudaStreamSynchronize(ctx->stream));
  ctx->e_G = G;
  ctx->e_wmaps_host.assign(((size_t)c.L * 7 + 1) * pk::N_HEIGHTS * 2, CUtensorMap{});
  ctx->e_wmaps_dirty = true;
  ctx->use_engine = true;
  return CLASP_OK;
}

// tensor maps of one weight matrix for every tile height its product uses: 2-D (one chunk per box)
// and, where the product takes them, 3-D (all chunks of a ring item in one box)
int engine_maps(clasp_ctx* ctx, int slot, int kind_slot, int kind, const void* w, int rows, int cols) {
  const size_t n2 = ((size_t)ctx->cfg.L * 7 + 1) * pk::N_HEIGHTS;
  for (int hi = 0; hi < pk::N_HEIGHTS; ++hi) {
    const int h = ctx->e_heights[kind_slot][hi];
    if (h == 0) continue;
    if (make_map(ctx, w, rows, cols, h, &ctx->e_wmaps_host[(size_t)slot * pk::N_HEIGHTS + hi])) return CLASP_ERR_CUDA;
    if (ctx->e_use3d[kind] &&
        make_map3(ctx, w, rows, cols, h, ctx->e_kpi[kind], &ctx->e_wmaps_host[n2 + (size_t)slot * pk::N_HEIGHTS + hi]))
      return CLASP_ERR_CUDA;
  }
  ctx->e_wmaps_dirty = true;
  return CLASP_OK;
}

// weight + visible K/V bytes one job must move (for the per-launch bandwidth figure)
double job_bytes(const clasp_ctx* ctx, const pk::Job& J) {
  const clasp_config& c = ctx->cfg;
  const double d = c.d_model, qd = (double)c.n_q_heads * c.head_dim, kvd = (double)c.n_kv_heads * c.head_dim;
  if (J.type == pk::JOB_HEAD) return 2.0 * c.vocab * d;
  if (J.type != pk::JOB_LAYER) return 0.0;
  return 2.0 * (d * (qd + 2 * kvd) + qd * d + 3.0 * d * c.d_ffn) + 2.0 * (double)J.C * kvd * 2.0;
}

// Launch the engine over ctx->e_jobs.  Rmax: most rows of any job; head_off: first row of the
// previous job that the head job (if any) reads.
int engine_launch(clasp_ctx* ctx, int Rmax, int head_off, int search_ctx = -1) {
  const clasp_config& c = ctx->cfg;
  Workspace& ws = ctx->ws;
  if (ctx->e_jobs.empty()) return CLASP_OK;
  // (the job number is also the low 7 bits of the tags of the attention's partial results)
  if (Rmax > pk::MAX_ROWS || (int)ctx->e_jobs.size() > c.L + 4 || ctx->e_jobs.size() > 127) return CLASP_ERR_CAPACITY;
  const int d = c.d_model, qd = c.n_q_heads * c.head_dim;
  const int rows_cap = c.max_rows;
  const int BN = Rmax <= 16 ? 16 : (Rmax + 15) / 16 * 16;
  int dev = 0, optin = 0;
  CUDA_TRY(cudaGetDevice(&dev));
  CUDA_TRY(cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
  // Searches over a long context run the attention over the cache keys on the tensor cores: that needs a
  // larger scratch area (taken from the weight ring) and runs of whole 64-key tiles.
  // (measured on the 8B shape: it pays from about 4096 positions on, from about 2500 when a kv head's pairs fit one
  // 64-row item -- those launches give up less of the ring --, and from about 1024 when a kv head has 256 or more
  // (row, query head) pairs; below that the smaller ring costs the products more than the attention gains)
  const int att_pairs = Rmax * (c.n_q_heads / c.n_kv_heads);
  // (the 70B layer shape, whose products lose more to the smaller ring, breaks even at 2048 positions with 256 - 320 pairs)
  const int wide_min = c.d_model >= 8192 ? 2 * pk::TC_MIN_CTX_WIDE : pk::TC_MIN_CTX_WIDE;
  bool att_tc = c.head_dim == 128 && !(c.flags & CLASP_FLAG_NO_ATT_TC) &&
                (search_ctx >= pk::TC_MIN_CTX || (search_ctx >= wide_min && att_pairs >= 256) ||
                 (search_ctx >= pk::TC_MIN_CTX_NARROW && att_pairs <= 64));
  // (that instantiation carries search jobs only: layer jobs with an Eq. 2 step and select jobs)
  for (const pk::Job& J : ctx->e_jobs)
    att_tc = att_tc && J.type != pk::JOB_HEAD && !(J.type == pk::JOB_LAYER && (J.uniform || !J.dp));
  // (row, query head) pairs of a kv head: up to 64 of them fit an M = 64 accumulator, which leaves the ring 24 KB more
  const int att_rows = att_pairs <= 64 ? 64 : pk::TC_ROWS;
  const int scratch_bytes = !att_tc ? pk::SCRATCH_BYTES : (att_rows == 64 ? pk::SCRATCH_TC64_BYTES : pk::SCRATCH_TC_BYTES);
  const int ring_pages = (optin - ctx->e_static_smem - 1024 - scratch_bytes) / pk::PAGE;
  // an item (gate + up rows and the operand tiles of kpi chunks) must fit the ring twice over
  const int b_pages = BN * pk::BK * 2 / pk::PAGE;
  // chunks per ring item in this launch: the set-up value when two such items fit the ring, else fewer,
  // loaded chunk by chunk through the 2-D maps (the 3-D boxes are built for the set-up value)
  bool any_dual = false;
  for (const pk::Job& J : ctx->e_jobs) any_dual = any_dual || J.dual_src;
  int kpi[5], use3d[5];
  for (int k = 0; k < 5; ++k) {
    kpi[k] = ctx->e_kpi[k];
    use3d[k] = ctx->e_use3d[k];
    const int bp = (k == pk::G_QKV && any_dual ? 2 : 1) * b_pages;
    while (kpi[k] > 1 && kpi[k] * (ctx->e_wpages[k] + bp) * 2 > ring_pages) --kpi[k];
    if (kpi[k] * (ctx->e_wpages[k] + bp) * 2 > ring_pages) return CLASP_ERR_CAPACITY;
    if (kpi[k] != ctx->e_kpi[k]) use3d[k] = 0;
    if (!use3d[k] && kpi[k] > 16) kpi[k] = 16;   // one lane pair per chunk
  }
  const size_t dyn = 1024 + (size_t)ring_pages * pk::PAGE + scratch_bytes;

  const int qdim = qd;
  auto bm = ctx->e_bmaps.find(BN);
  if (bm == ctx->e_bmaps.end()) {
    std::array<CUtensorMap, 10> m{};
    int rc = 0;
    rc |= make_map(ctx, ws.xn, rows_cap, d, BN, &m[0]);
    rc |= make_map(ctx, ws.attn, rows_cap, qdim, BN, &m[1]);
    rc |= make_map(ctx, ws.xn_m, rows_cap, d, BN, &m[2]);
    rc |= make_map(ctx, ws.act, rows_cap, c.d_ffn, BN, &m[3]);
    if (ctx->e_use3d[pk::G_QKV]) rc |= make_map3(ctx, ws.xn, rows_cap, d, BN, ctx->e_kpi[pk::G_QKV], &m[4]);
    if (ctx->e_use3d[pk::G_O]) rc |= make_map3(ctx, ws.attn, rows_cap, qdim, BN, ctx->e_kpi[pk::G_O], &m[5]);
    if (ctx->e_use3d[pk::G_GU]) rc |= make_map3(ctx, ws.xn_m, rows_cap, d, BN, ctx->e_kpi[pk::G_GU], &m[6]);
    if (ctx->e_use3d[pk::G_DOWN]) rc |= make_map3(ctx, ws.act, rows_cap, c.d_ffn, BN, ctx->e_kpi[pk::G_DOWN], &m[7]);
    if (2 * BN <= 256) {
      rc |= make_map(ctx, ws.xn, rows_cap, d, 2 * BN, &m[8]);
      if (ctx->e_use3d[pk::G_QKV]) rc |= make_map3(ctx, ws.xn, rows_cap, d, 2 * BN, ctx->e_kpi[pk::G_QKV], &m[9]);
    }
    if (rc) return CLASP_ERR_CUDA;
    bm = ctx->e_bmaps.emplace(BN, m).first;
  }
  auto hk = std::make_pair(head_off, BN);
  auto hm = ctx->e_headmaps.find(hk);
  if (hm == ctx->e_headmaps.end()) {
    std::array<CUtensorMap, 2> m{};
    const bf16* base = (const bf16*)ws.xn + (size_t)head_off * d;
    int rc = make_map(ctx, base, rows_cap - head_off, d, BN, &m[0]);
    if (ctx->e_use3d[pk::G_HEAD]) rc |= make_map3(ctx, base, rows_cap - head_off, d, BN, ctx->e_kpi[pk::G_HEAD], &m[1]);
    if (rc) return CLASP_ERR_CUDA;
    hm = ctx->e_headmaps.emplace(hk, m).first;
  }
  if (ctx->e_wmaps_dirty) {
    CUDA_TRY(cudaMemcpyAsync(ws.wmaps, ctx->e_wmaps_host.data(), ctx->e_wmaps_host.size() * sizeof(CUtensorMap),
                             cudaMemcpyHostToDevice, ctx->stream));
    ctx->e_wmaps_dirty = false;
  }
  if (att_tc) {
    // the caches of this launch's layer jobs as 2-D maps {kv width, context rows}: 64 x 64 boxes, 128-byte swizzle,
    // rows past the context read as zeros
    ctx->e_kvmaps_host.assign(ctx->e_jobs.size() * 2, CUtensorMap{});
    for (size_t j = 0; j < ctx->e_jobs.size(); ++j) {
      pk::Job& J = ctx->e_jobs[j];
      if (J.type != pk::JOB_LAYER || J.uniform) continue;
      J.kvmap = (int)(2 * j);
      if (make_map(ctx, J.ck, J.C, c.n_kv_heads * c.head_dim, 64, &ctx->e_kvmaps_host[2 * j]) ||
          make_map(ctx, J.cv, J.C, c.n_kv_heads * c.head_dim, 64, &ctx->e_kvmaps_host[2 * j + 1]))
        return CLASP_ERR_CUDA;
    }
    CUDA_TRY(cudaMemcpyAsync(ws.kvmaps, ctx->e_kvmaps_host.data(), ctx->e_kvmaps_host.size() * sizeof(CUtensorMap),
                             cudaMemcpyHostToDevice, ctx->stream));
  }
  CUDA_TRY(cudaMemcpyAsync(ws.jobs, ctx->e_jobs.data(), ctx->e_jobs.size() * sizeof(pk::Job),
                           cudaMemcpyHostToDevice, ctx->stream));
  CUDA_TRY(cudaMemsetAsync(ws.ctl, 0, 4, ctx->stream));  // abort flag; the status word is sticky
  CUDA_TRY(cudaMemsetAsync(ws.ss_a, 0, ws.acc_bytes, ctx->stream));  // all fixed-point accumulators
  CUDA_TRY(cudaMemsetAsync(ws.flags, 0, (size_t)pk::N_FLAGS * (ctx->e_G + 32) * sizeof(int), ctx->stream));

  pk::Params P{};
  P.c.L = c.L; P.c.d = d; P.c.qd = qd; P.c.kvd = c.n_kv_heads * c.head_dim; P.c.hd = c.head_dim;
  P.c.nq = c.n_q_heads; P.c.nkv = c.n_kv_heads; P.c.dffn = c.d_ffn; P.c.vocab = c.vocab; P.c.eps = c.rms_eps;
  P.c.G = ctx->e_G; P.c.Rcap = ws.e_rcap; P.c.run_len = ws.e_run_len; P.c.chunk_cap = ws.e_chunk_cap;
  // The forward passes cut the cache into runs of a length fixed by the context capacity, so that a
  // position's attention is summed in the same order whichever call computes it (verification and
  // one-token decoding must agree bit for bit).  The search only has to agree with itself: it cuts
  // the keys it sees into at most 32 runs, which spreads a short context over many more CTAs.
  if (search_ctx >= 0) P.c.run_len = pk::ATT_KEYS * ((search_ctx + pk::ATT_KEYS * 32 - 1) / (pk::ATT_KEYS * 32) > 0
                                                       ? (search_ctx + pk::ATT_KEYS * 32 - 1) / (pk::ATT_KEYS * 32) : 1);
  if (att_tc) {
    // run length: whole 64-key tiles, at most 32 runs; the cut that needs the fewest tile steps when the
    // (kv head, run, pair block) items are dealt out to the CTAs (one more step per round for its set-up)
    const int n_pb = (Rmax * (c.n_q_heads / c.n_kv_heads) + att_rows - 1) / att_rows;
    int best_len = 0;
    long best_cost = 0;
    for (int n = 1; n <= 32; ++n) {
      const int len = 64 * (((search_ctx + n - 1) / n + 63) / 64);
      const int runs = (search_ctx + len - 1) / len;
      const long rounds = ((long)c.n_kv_heads * runs * n_pb + ctx->e_G - 1) / ctx->e_G;
      const long cost = rounds * (len / 64 + 1);
      if (best_len == 0 || cost < best_cost) { best_len = len; best_cost = cost; }
    }
    P.c.run_len = best_len;
  }
  P.c.BN = BN; P.c.ring_pages = ring_pages; P.c.att_tc = att_tc ? 1 : 0; P.c.att_rows = att_rows;

  for (int s = 0; s < pk::N_SPLITS; ++s) { P.c.split_lo[s] = ctx->e_split_lo[s]; P.c.split_units[s] = ctx->e_split_units[s]; }
  for (int k = 0; k < 5; ++k) { P.c.tile_idx[k] = ctx->e_tile_idx[k]; P.c.kpi[k] = kpi[k]; P.c.use3d[k] = use3d[k]; }
  P.c.tiles_off = ctx->e_tiles_off; P.c.map3d_off = (int)(((size_t)c.L * 7 + 1) * pk::N_HEIGHTS);
  P.b.xn_a = (bf16*)ws.xn; P.b.xn_m = (bf16*)ws.xn_m; P.b.attn = (bf16*)ws.attn; P.b.act = (bf16*)ws.act;
  P.b.qkv = ws.qkv; P.b.x1 = ws.x1; P.b.Gbuf = ws.G; P.b.att_acc = ws.e_att_acc; P.b.att_ml = ws.e_att_ml;
  P.b.ss_a = ws.ss_a; P.b.ss_m = ws.ss_m; P.b.cosacc = ws.cosacc; P.b.head_best = ws.head_best; P.b.flags = ws.flags;
  P.b.rope = ws.rope;
  P.jobs = ws.jobs; P.n_jobs = (int)ctx->e_jobs.size(); P.wmaps = ws.wmaps; P.kvmaps = ws.kvmaps; P.tabs = ws.tabs; P.ctl = ws.ctl;
  P.trace = ctx->e_trace; P.trace_cap = ctx->e_trace_cap;
  ctx->launch_seq = (ctx->launch_seq + 1) & 0x1ffffffu;
  if (ctx->launch_seq == 0) {   // the tags start over: no old tag may survive in the buffers
    CUDA_TRY(cudaMemsetAsync(ws.e_att_acc, 0, ws.e_att_bytes, ctx->stream));
    ctx->launch_seq = 1;
  }
  P.launch_tag = ctx->launch_seq << 7;
  P.wait_fast = ctx->wait_limit ? (ctx->wait_limit < pk::WAIT_FAST ? ctx->wait_limit : pk::WAIT_FAST) : pk::WAIT_FAST;
  P.wait_slow = ctx->wait_limit ? ctx->wait_limit : pk::WAIT_SLOW;

  cudaEvent_t e0 = nullptr, e1 = nullptr;
  if (ctx->profiling) {
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return CLASP_ERR_CUDA;
    cudaEventRecord(e0, ctx->stream);
  }
  void* args[] = {(void*)&bm->second[0], (void*)&bm->second[1], (void*)&bm->second[2], (void*)&bm->second[3],
                  (void*)&hm->second[0], (void*)&bm->second[4], (void*)&bm->second[5], (void*)&bm->second[6],
                  (void*)&bm->second[7], (void*)&hm->second[1], (void*)&bm->second[8], (void*)&bm->second[9], (void*)&P};
  const void* kern = ctx->e_kernel[(att_tc ? 2 : 0) + (ctx->e_trace ? 1 : 0)];
  cudaError_t err = cudaLaunchCooperativeKernel(kern, dim3(ctx->e_G), dim3(pk::THREADS),
                                                args, dyn, ctx->stream);
  if (ctx->profiling) {
    cudaEventRecord(e1, ctx->stream);
    ctx->prof_events.emplace_back(e0, e1);
    for (const pk::Job& J : ctx->e_jobs) ctx->prof_bytes += job_bytes(ctx, J);
  }
  ctx->launches += 1;
  return err == cudaSuccess ? CLASP_OK : CLASP_ERR_CUDA;
}

// a decoder-layer job with the fields every caller sets the same way
pk::Job layer_job(clasp_ctx* ctx, int l, int S, int T, int C, bool uniform, const clasp_kv_layer& kv) {
  pk::Job J{};
  J.type = pk::JOB_LAYER; J.layer = l; J.S = S; J.T = T; J.R = S * T; J.C = C; J.uniform = uniform ? 1 : 0;
  J.norm_in = ctx->layers[l].attn_norm; J.norm_mlp = ctx->layers[l].mlp_norm;
  J.ck = (bf16*)kv.k; J.cv = (bf16*)kv.v;
  return J;
}

// fills in, per job, how often each step kind has been published once the job's own step of
// that kind is done, and which step of the previous job publishes the job's first operand
void link_jobs(std::vector<pk::Job>& jobs) {
  int n_pub[pk::N_FLAGS] = {0};
  for (size_t k = 0; k < jobs.size(); ++k) {
    pk::Job& J = jobs[k];
    int src_tgt = 0, src_flag = pk::F_PREP;
    if (k > 0) {
      const pk::Job& prev = jobs[k - 1];
      const bool from_select = (prev.type == pk::JOB_SELECT || (prev.type == pk::JOB_LAYER && prev.dp)) && !prev.defer;
      src_flag = from_select ? pk::F_SELECT : pk::F_DOWN;
      src_tgt = n_pub[src_flag];
    }
    if (J.type == pk::JOB_LAYER) {
      if (J.prep) ++n_pub[pk::F_PREP];
      ++n_pub[pk::F_QKV]; ++n_pub[pk::F_ATTN]; ++n_pub[pk::F_MERGE]; ++n_pub[pk::F_O]; ++n_pub[pk::F_GU];
      ++n_pub[pk::F_DOWN];
      if (J.dp && !J.defer) ++n_pub[pk::F_SELECT];
      if (J.prep) { src_flag = pk::F_PREP; src_tgt = n_pub[pk::F_PREP]; }
    } else if (J.type == pk::JOB_SELECT) {
      ++n_pub[pk::F_DOWN]; ++n_pub[pk::F_SELECT];
    } else {
      ++n_pub[pk::F_HEAD];
    }
    J.src_flag = src_flag; J.src_tgt = src_tgt;
    for (int f = 0; f < pk::N_FLAGS; ++f) J.tgt[f] = n_pub[f];
  }
}

}  // namespace

// =============================================================== C ABI

extern "C" {

size_t clasp_workspace_bytes(const clasp_config* cfg) {
  if (!config_ok(cfg)) return 0;
  return carve(*cfg, nullptr).bytes;
}

int clasp_create(const clasp_config* cfg, void* workspace, size_t workspace_bytes, void* cuda_stream,
                 clasp_ctx** out) {
  if (!out) return CLASP_ERR_INVALID_ARG;
  *out = nullptr;
  if (!cfg || !workspace) return CLASP_ERR_INVALID_ARG;
  if (cfg->dtype != CLASP_FP32 && cfg->dtype != CLASP_BF16) return CLASP_ERR_DTYPE;
  if (!config_ok(cfg)) return CLASP_ERR_SHAPE;
  if (((uintptr_t)workspace & 255) != 0) return CLASP_ERR_INVALID_ARG;
  Workspace ws = carve(*cfg, (uint8_t*)workspace);
  if (workspace_bytes < ws.bytes) return CLASP_ERR_CAPACITY;
  int dev = 0, n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev < 1) return CLASP_ERR_CUDA;
  CUDA_TRY(cudaGetDevice(&dev));
  cudaDeviceProp prop;
  CUDA_TRY(cudaGetDeviceProperties(&prop, dev));
  clasp_ctx* ctx = new clasp_ctx();
  ctx->cfg = *cfg;
  ctx->stream = (cudaStream_t)cuda_stream;
  ctx->ws = ws;
  ctx->layers.resize(cfg->L);
  ctx->loaded.assign(cfg->L, 0);
  ctx->num_sms = prop.multiProcessorCount;
  ctx->use_tc = cfg->dtype == CLASP_BF16 && !(cfg->flags & CLASP_FLAG_FORCE_SIMT);
  if (ctx->use_tc) {
    if (prop.major != 10) {  // the tcgen05 kernel exists for sm_100a only
      delete ctx;
      return CLASP_ERR_CUDA;
    }
    ctx->maps.resize(cfg->L);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn) {
      delete ctx;
      return CLASP_ERR_CUDA;
    }
    ctx->encode = (EncodeTiledFn)fn;
    if (cudaFuncSetAttribute(clasp::tc::gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             220 * 1024) != cudaSuccess) {
      delete ctx;
      return CLASP_ERR_CUDA;
    }
    ctx->cta_cap = 2 * ctx->num_sms;
  }
  if (cudaMemsetAsync(ws.status, 0, 256, ctx->stream) != cudaSuccess ||
      cudaMemsetAsync(ws.counters, 0, MAX_COUNTERS * sizeof(int), ctx->stream) != cudaSuccess) {
    delete ctx;
    return CLASP_ERR_CUDA;
  }
  if (ctx->use_tc) {
    if (engine_setup(ctx) != CLASP_OK || cudaMemsetAsync(ws.ctl, 0, 256, ctx->stream) != cudaSuccess ||
        cudaMemsetAsync(ws.e_att_acc, 0, ws.e_att_bytes, ctx->stream) != cudaSuccess) {
      delete ctx;
      return CLASP_ERR_CUDA;
    }
  }
  *out = ctx;
  return CLASP_OK;
}

void clasp_destroy(clasp_ctx* ctx) { delete ctx; }

int clasp_load_layers(clasp_ctx* ctx, int32_t first, int32_t count, const clasp_layer_weights* w) {
  if (!ctx || !w || first < 0 || count < 0 || first + count > ctx->cfg.L) return CLASP_ERR_INVALID_ARG;
  const clasp_config& c = ctx->cfg;
  const int d = c.d_model, qd = c.n_q_heads * c.head_dim, kvd = c.n_kv_heads * c.head_dim;
  for (int k = 0; k < count; ++k) {
    const clasp_layer_weights& lw = w[k];
    const void* ptrs[9] = {lw.attn_norm, lw.wq, lw.wk, lw.wv, lw.wo, lw.mlp_norm, lw.w_gate, lw.w_up, lw.w_down};
    for (const void* p : ptrs)
      if (!p || ((uintptr_t)p & 15)) return CLASP_ERR_INVALID_ARG;
    ctx->layers[first + k] = lw;
    if (ctx->use_tc) {
      LayerMaps& m = ctx->maps[first + k];
      int rc = 0;
      rc |= make_map(ctx, lw.wq, qd, d, clasp::tc::BM, &m.wq);
      rc |= make_map(ctx, lw.wk, kvd, d, clasp::tc::BM, &m.wk);
      rc |= make_map(ctx, lw.wv, kvd, d, clasp::tc::BM, &m.wv);
      rc |= make_map(ctx, lw.wo, d, qd, clasp::tc::BM, &m.wo);
      rc |= make_map(ctx, lw.w_gate, c.d_ffn, d, clasp::tc::BM, &m.w_gate);
      rc |= make_map(ctx, lw.w_up, c.d_ffn, d, clasp::tc::BM, &m.w_up);
      rc |= make_map(ctx, lw.w_down, d, c.d_ffn, clasp::tc::BM, &m.w_down);
      if (rc) return CLASP_ERR_CUDA;
      if (ctx->use_engine) {
        const int b7 = (first + k) * 7;
        int erc = 0;
        erc |= engine_maps(ctx, b7 + 0, 0, pk::G_QKV, lw.wq, qd, d);
        erc |= engine_maps(ctx, b7 + 1, 1, pk::G_QKV, lw.wk, kvd, d);
        erc |= engine_maps(ctx, b7 + 2, 2, pk::G_QKV, lw.wv, kvd, d);
        erc |= engine_maps(ctx, b7 + 3, 3, pk::G_O, lw.wo, d, qd);
        erc |= engine_maps(ctx, b7 + 4, 4, pk::G_GU, lw.w_gate, c.d_ffn, d);
        erc |= engine_maps(ctx, b7 + 5, 5, pk::G_GU, lw.w_up, c.d_ffn, d);
        erc |= engine_maps(ctx, b7 + 6, 6, pk::G_DOWN, lw.w_down, d, c.d_ffn);
        if (erc) return CLASP_ERR_CUDA;
      }
    }
    ctx->loaded[first + k] = 1;
  }
  return CLASP_OK;
}

int clasp_load_head(clasp_ctx* ctx, const void* embed, const float* final_norm, const void* lm_head) {
  if (!ctx || !embed || !final_norm || !lm_head) return CLASP_ERR_INVALID_ARG;
  if (((uintptr_t)embed & 15) || ((uintptr_t)final_norm & 15) || ((uintptr_t)lm_head & 15))
    return CLASP_ERR_INVALID_ARG;
  ctx->embed = embed;
  ctx->final_norm = final_norm;
  ctx->lm_head = lm_head;
  if (ctx->use_tc && make_map(ctx, lm_head, ctx->cfg.vocab, ctx->cfg.d_model, clasp::tc::BM, &ctx->lm_head_map))
    return CLASP_ERR_CUDA;
  if (ctx->use_engine && engine_maps(ctx, ctx->cfg.L * 7, 7, pk::G_HEAD, lm_head, ctx->cfg.vocab, ctx->cfg.d_model))
    return CLASP_ERR_CUDA;
  return CLASP_OK;
}

int clasp_layer_forward(clasp_ctx* ctx, int32_t layer, const float* x_in, int64_t in_stride, int32_t S,
                        int32_t T, int32_t ctx_len, int32_t pos0, const clasp_kv_layer* kv_layer,
                        int32_t write_kv, float* x_out, int64_t out_stride) {
  if (!ctx || !x_in || !x_out || !kv_layer || !kv_layer->k || !kv_layer->v) return CLASP_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->cfg.L || S < 1 || T < 1 || ctx_len < 0 || pos0 < 0) return CLASP_ERR_INVALID_ARG;
  if (write_kv && S != 1) return CLASP_ERR_INVALID_ARG;
  if (in_stride < ctx->cfg.d_model || out_stride < ctx->cfg.d_model) return CLASP_ERR_INVALID_ARG;
  if (!al16(x_in) || !al16(x_out) || (in_stride & 3) || (out_stride & 3) || !kv_aligned(kv_layer, 1))
    return CLASP_ERR_INVALID_ARG;
  if ((int64_t)S * T > ctx->cfg.max_rows || ctx_len > ctx->cfg.max_ctx || pos0 + T > ctx->cfg.max_ctx)
    return CLASP_ERR_CAPACITY;
  if (!ctx->loaded[layer]) return CLASP_ERR_NOT_LOADED;
  int rc = rope_table(ctx, T, pos0);
  if (rc) return rc;
  if (ctx->use_engine && S * T <= pk::MAX_ROWS && (!write_kv || pos0 == ctx_len)) {
    pk::Job J = layer_job(ctx, layer, S, T, ctx_len, write_kv != 0, *kv_layer);
    J.prep = 1; J.x_in = x_in; J.ldx = in_stride; J.x_out = x_out; J.ldo = out_stride;
    ctx->e_jobs.assign(1, J);
    link_jobs(ctx->e_jobs);
    return engine_launch(ctx, S * T, 0);
  }
  return run_layer_any(ctx, layer, x_in, in_stride, S, T, ctx_len, pos0, *kv_layer, write_kv != 0, x_out,
                       out_stride);
}

int clasp_dp_search(clasp_ctx* ctx, const float* hidden_states, int64_t layer_stride, int64_t token_stride,
                    const clasp_kv_layer* kv, int32_t ctx_len, int32_t pos0, int32_t T, int32_t M,
                    uint8_t* skip_mask, float* scores, float* margins, float* g_final,
                    const uint8_t* forced_choice) {
  if (!ctx || !hidden_states || !kv || !skip_mask || !scores) return CLASP_ERR_INVALID_ARG;
  const clasp_config& c = ctx->cfg;
  const int L = c.L, d = c.d_model;
  if (M < 0 || M > L || T < 1 || ctx_len < 0 || pos0 < 0) return CLASP_ERR_INVALID_ARG;
  if (M > c.max_M || T > c.max_T || (int64_t)M * T > c.max_rows || ctx_len > c.max_ctx ||
      (int64_t)pos0 + T > c.max_ctx)
    return CLASP_ERR_CAPACITY;
  for (int l = 0; l < L; ++l)
    if (!kv[l].k || !kv[l].v) return CLASP_ERR_INVALID_ARG;
  if (!al16(hidden_states) || (layer_stride & 3) || (token_stride & 3) || !al16(g_final) || !kv_aligned(kv, L))
    return CLASP_ERR_INVALID_ARG;
  if (M > 0 && !layers_ready(ctx)) return CLASP_ERR_NOT_LOADED;
  Workspace& ws = ctx->ws;
  const int ncell = (L + 1) * (M + 1);
  clasp::fill_tables_kernel<<<(ncell + 255) / 256, 256, 0, ctx->stream>>>(scores, margins, ws.choice, ncell);
  int rc = launch_check(ctx);
  if (rc) return rc;
  if ((rc = rope_table(ctx, T, pos0))) return rc;
  const int64_t Td = (int64_t)T * d;
  const bool prune = (c.flags & CLASP_FLAG_PRUNE) != 0;
  if (ctx->use_engine && M > 0 && M * T <= pk::MAX_ROWS) {
    // one cooperative launch for the whole search: step i = (layer i-1 over the candidate
    // states) + (Eq. 2 select); row 0 of the g table is x_i itself and is never stored
    clasp::dp_origin_kernel<<<1, 32, 0, ctx->stream>>>(scores, ws.choice);
    if ((rc = launch_check(ctx))) return rc;
    ctx->e_jobs.clear();
    int cur = 0, prev_lo = 1;
    for (int i = 1; i <= L; ++i) {
      const int ell = (i - 1 < M) ? i - 1 : M;
      // states the step carries: j_lo..ell (plus the diagonal state i while i <= M).  With pruning the
      // states from which (L, M) cannot be reached any more, j < M - (L - i), are left out; the job
      // sees its states as 1..n through pointers offset by j_lo - 1 states.
      const int j_lo = (prune && M - (L - i) > 1) ? M - (L - i) : 1;
      const int n = ell - j_lo + 1 > 0 ? ell - j_lo + 1 : 0;
      const int64_t sh = j_lo - 1;
      pk::Job J{};
      if (n > 0) {
        J = layer_job(ctx, i - 1, n, T, ctx_len, false, kv[i - 1]);
        J.x_in = ws.grow[cur] + j_lo * Td; J.ldx = d; J.dp = 1;
      } else {
        J.type = pk::JOB_SELECT; J.T = T;
      }
      J.i = i; J.ell = n; J.diag = i <= M ? 1 : 0; J.M = M - (int)sh;
      J.x_i = hidden_states + (int64_t)i * layer_stride;
      J.x_tok_stride = token_stride;
      if (j_lo == 1) { J.x_im1 = hidden_states + (int64_t)(i - 1) * layer_stride; J.x_im1_stride = token_stride; }
      else { J.x_im1 = ws.grow[cur] + sh * Td; J.x_im1_stride = d; }
      J.in_shift = (j_lo - prev_lo) * T;
      prev_lo = j_lo;
      J.g_prev = ws.grow[cur] + sh * Td; J.g_next = ws.grow[cur ^ 1] + sh * Td;
      J.D0 = scores + (int64_t)i * (M + 1);
      J.choice0 = ws.choice + (int64_t)i * (M + 1);
      J.D = J.D0 + sh;
      J.margin = margins ? margins + (int64_t)i * (M + 1) + sh : nullptr;
      J.choice = J.choice0 + sh;
      J.forced = forced_choice ? forced_choice + (int64_t)i * (M + 1) + sh : nullptr;
      J.norm_next = i < L ? ctx->layers[i].attn_norm : nullptr;
      J.g_final = (i == L) ? g_final : nullptr;
      ctx->e_jobs.push_back(J);
      cur ^= 1;
    }
    // a layer job followed by another layer job hands over both candidates of every state instead of
    // making the next layer wait for the Eq. 2 decision (needs 2 BN operand rows and accumulator columns)
    const int BNs = M * T <= 16 ? 16 : (M * T + 15) / 16 * 16;
    if (2 * BNs <= c.max_rows && 2 * BNs <= 128 && !(c.flags & CLASP_FLAG_NO_DEFER))
      for (size_t k = 0; k + 1 < ctx->e_jobs.size(); ++k)
        if (ctx->e_jobs[k].type == pk::JOB_LAYER && ctx->e_jobs[k + 1].type == pk::JOB_LAYER) {
          ctx->e_jobs[k].defer = 1;
          ctx->e_jobs[k + 1].dual_src = 1;
        }
    link_jobs(ctx->e_jobs);
    if ((rc = engine_launch(ctx, M * T, 0, ctx_len))) return rc;
    clasp::backtrack_kernel<<<1, 32, 0, ctx->stream>>>(ws.choice, L, M, skip_mask);
    return launch_check(ctx);
  }
  {
    clasp::DpStepArgs a0{};  // g[0][0] = x_0, D[0][0] = 1: the b == 0 path of a step over x_0 itself
    a0.x_i = hidden_states; a0.x_tok_stride = token_stride; a0.G = ws.G; a0.g_prev = ws.grow[0];
    a0.g_next = ws.grow[0]; a0.D = scores; a0.margin = nullptr; a0.choice = ws.choice; a0.forced = nullptr;
    a0.T = T; a0.d = d; a0.ell = 0; a0.i = 0; a0.M = M; a0.j_lo = 1;
    clasp::dp_step_kernel<<<1, 256, 0, ctx->stream>>>(a0);
    if ((rc = launch_check(ctx))) return rc;
  }
  int cur = 0;
  for (int i = 1; i <= L; ++i) {
    const int ell = (i - 1 < M) ? i - 1 : M;
    const int j_lo = (prune && M - (L - i) > 1) ? M - (L - i) : 1;   // first state the step carries
    const int n = ell - j_lo + 1 > 0 ? ell - j_lo + 1 : 0;
    float* g_prev = ws.grow[cur];
    float* g_next = ws.grow[cur ^ 1];
    if (n > 0) {
      // the candidate states j = j_lo..ell through layer i-1 in one batch (Sec. 3.6)
      rc = run_layer_any(ctx, i - 1, g_prev + j_lo * Td, d, n, T, ctx_len, pos0, kv[i - 1], false, ws.G, d);
      if (rc) return rc;
    }
    clasp::DpStepArgs a{};
    a.x_i = hidden_states + (int64_t)i * layer_stride;
    a.x_tok_stride = token_stride;
    a.G = ws.G;
    a.g_prev = g_prev;
    a.g_next = g_next;
    a.D = scores + (int64_t)i * (M + 1);
    a.margin = margins ? margins + (int64_t)i * (M + 1) : nullptr;
    a.choice = ws.choice + (int64_t)i * (M + 1);
    a.forced = forced_choice ? forced_choice + (int64_t)i * (M + 1) : nullptr;
    a.T = T; a.d = d; a.ell = n; a.i = i; a.M = M; a.j_lo = j_lo;
    const int blocks = 1 + n + (i <= M ? 1 : 0);
    clasp::dp_step_kernel<<<blocks, 256, 0, ctx->stream>>>(a);
    if ((rc = launch_check(ctx))) return rc;
    cur ^= 1;
  }
  clasp::backtrack_kernel<<<1, 32, 0, ctx->stream>>>(ws.choice, L, M, skip_mask);
  if ((rc = launch_check(ctx))) return rc;
  if (g_final) {
    clasp::copy_rows_kernel<<<T, 256, 0, ctx->stream>>>(ws.grow[cur] + (int64_t)M * Td, d, g_final, d, d);
    if ((rc = launch_check(ctx))) return rc;
  }
  return CLASP_OK;
}

}  // extern "C"

namespace {
int verify_impl(clasp_ctx* ctx, const int32_t* tokens, int32_t n, int32_t pos0, const clasp_kv_layer* kv,
                int32_t n_head_rows, int32_t* argmax_out, float* hidden_out, float* logits_out) {
  if (!ctx || !tokens || !kv || n < 1 || pos0 < 0 || n_head_rows < 0 || n_head_rows > n)
    return CLASP_ERR_INVALID_ARG;
  if (n_head_rows > 0 && !argmax_out) return CLASP_ERR_INVALID_ARG;
  const clasp_config& c = ctx->cfg;
  if (n > c.max_rows || (int64_t)pos0 + n > c.max_ctx || n_head_rows > c.max_head_rows) return CLASP_ERR_CAPACITY;
  for (int l = 0; l < c.L; ++l)
    if (!kv[l].k || !kv[l].v) return CLASP_ERR_INVALID_ARG;
  if (!al16(hidden_out) || !kv_aligned(kv, c.L)) return CLASP_ERR_INVALID_ARG;
  if (!layers_ready(ctx) || !ctx->embed) return CLASP_ERR_NOT_LOADED;
  const int d = c.d_model, L = c.L;
  int rc;
  if ((rc = rope_table(ctx, n, pos0))) return rc;
  if (ctx->use_engine && n <= pk::MAX_ROWS) {
    // embedding gather, then every layer and the head in one cooperative launch
    float* h0 = hidden_out ? hidden_out : ctx->ws.hping;
    const int64_t ld = hidden_out ? (int64_t)(L + 1) * d : d;
    if ((rc = embed_rows(ctx, tokens, n, h0, ld))) return rc;
    ctx->e_jobs.clear();
    float* a = ctx->ws.hping;
    float* b = ctx->ws.hpong;
    for (int l = 0; l < L; ++l) {
      pk::Job J = layer_job(ctx, l, 1, n, pos0, true, kv[l]);
      J.prep = l == 0 ? 1 : 0;
      if (hidden_out) {
        J.x_in = hidden_out + (int64_t)l * d; J.x_out = hidden_out + (int64_t)(l + 1) * d;
      } else {
        J.x_in = a; J.x_out = b;
        float* t = a; a = b; b = t;
      }
      J.ldx = ld; J.ldo = ld;
      J.norm_next = l + 1 < L ? ctx->layers[l + 1].attn_norm : (n_head_rows > 0 ? ctx->final_norm : nullptr);
      ctx->e_jobs.push_back(J);
    }
    if (n_head_rows > 0) {
      pk::Job H{};
      H.type = pk::JOB_HEAD; H.R = n_head_rows; H.T = 1; H.row_off = n - n_head_rows;
      H.argmax_out = argmax_out; H.logits_out = logits_out;
      ctx->e_jobs.push_back(H);
    }
    link_jobs(ctx->e_jobs);
    return engine_launch(ctx, n, n_head_rows > 0 ? n - n_head_rows : 0);
  }
  const float* x;
  int64_t ldx;
  if (hidden_out) {
    const int64_t ld = (int64_t)(L + 1) * d;
    if ((rc = embed_rows(ctx, tokens, n, hidden_out, ld))) return rc;
    for (int l = 0; l < L; ++l) {
      rc = run_layer_any(ctx, l, hidden_out + (int64_t)l * d, ld, 1, n, pos0, pos0, kv[l], true,
                         hidden_out + (int64_t)(l + 1) * d, ld);
      if (rc) return rc;
    }
    x = hidden_out + (int64_t)L * d;
    ldx = ld;
  } else {
    float* a = ctx->ws.hping;
    float* b = ctx->ws.hpong;
    if ((rc = embed_rows(ctx, tokens, n, a, d))) return rc;
    for (int l = 0; l < L; ++l) {
      if ((rc = run_layer_any(ctx, l, a, d, 1, n, pos0, pos0, kv[l], true, b, d))) return rc;
      float* t = a; a = b; b = t;
    }
    x = a;
    ldx = d;
  }
  if (n_head_rows > 0)
    return run_head(ctx, x + (int64_t)(n - n_head_rows) * ldx, ldx, n_head_rows, argmax_out, nullptr, logits_out);
  return CLASP_OK;
}

int draft_impl(clasp_ctx* ctx, const uint8_t* skip_mask_host, const int32_t* token_in, int32_t pos,
               const clasp_kv_layer* kv, int32_t* token_out, float* top1_prob_out, float* logits_out) {
  if (!ctx || !skip_mask_host || !token_in || !kv || !token_out || pos < 0) return CLASP_ERR_INVALID_ARG;
  const clasp_config& c = ctx->cfg;
  if ((int64_t)pos + 1 > c.max_ctx) return CLASP_ERR_CAPACITY;
  if (!layers_ready(ctx) || !ctx->embed) return CLASP_ERR_NOT_LOADED;
  for (int l = 0; l < c.L; ++l)
    if (!skip_mask_host[l] && (!kv[l].k || !kv[l].v || !kv_aligned(kv + l, 1))) return CLASP_ERR_INVALID_ARG;
  const int d = c.d_model;
  int rc;
  if ((rc = rope_table(ctx, 1, pos))) return rc;
  float* a = ctx->ws.hping;
  float* b = ctx->ws.hpong;
  if ((rc = embed_rows(ctx, token_in, 1, a, d))) return rc;
  int n_kept = 0;
  for (int l = 0; l < c.L; ++l) n_kept += skip_mask_host[l] ? 0 : 1;
  if (ctx->use_engine && n_kept > 0) {
    ctx->e_jobs.clear();
    for (int l = 0; l < c.L; ++l) {
      if (skip_mask_host[l]) continue;  // skipped layer: nothing read, nothing written
      if (!kv[l].k || !kv[l].v) return CLASP_ERR_INVALID_ARG;
      pk::Job J = layer_job(ctx, l, 1, 1, pos, true, kv[l]);
      J.prep = ctx->e_jobs.empty() ? 1 : 0;
      J.x_in = a; J.ldx = d; J.x_out = b; J.ldo = d;
      float* t = a; a = b; b = t;
      ctx->e_jobs.push_back(J);
    }
    for (size_t k = 0; k + 1 < ctx->e_jobs.size(); ++k)
      ctx->e_jobs[k].norm_next = ctx->layers[ctx->e_jobs[k + 1].layer].attn_norm;
    ctx->e_jobs.back().norm_next = ctx->final_norm;
    pk::Job H{};
    H.type = pk::JOB_HEAD; H.R = 1; H.T = 1; H.row_off = 0; H.argmax_out = token_out; H.top1_out = top1_prob_out;
    H.logits_out = logits_out;
    ctx->e_jobs.push_back(H);
    link_jobs(ctx->e_jobs);
    return engine_launch(ctx, 1, 0);
  }
  for (int l = 0; l < c.L; ++l) {
    if (skip_mask_host[l]) continue;  // skipped layer: state passes through, nothing read or written
    if (!kv[l].k || !kv[l].v) return CLASP_ERR_INVALID_ARG;
    if ((rc = run_layer_any(ctx, l, a, d, 1, 1, pos, pos, kv[l], true, b, d))) return rc;
    float* t = a; a = b; b = t;
  }
  return run_head(ctx, a, d, 1, token_out, top1_prob_out, logits_out);
}
}  // namespace

extern "C" {

int clasp_verify(clasp_ctx* ctx, const int32_t* tokens, int32_t n, int32_t pos0, const clasp_kv_layer* kv,
                 int32_t n_head_rows, int32_t* argmax_out, float* hidden_out) {
  return verify_impl(ctx, tokens, n, pos0, kv, n_head_rows, argmax_out, hidden_out, nullptr);
}

int clasp_draft_forward(clasp_ctx* ctx, const uint8_t* skip_mask_host, const int32_t* token_in, int32_t pos,
                        const clasp_kv_layer* kv, int32_t* token_out, float* top1_prob_out) {
  return draft_impl(ctx, skip_mask_host, token_in, pos, kv, token_out, top1_prob_out, nullptr);
}

int clasp_draft_sample(clasp_ctx* ctx, const uint8_t* skip_mask_host, const int32_t* token_in, int32_t pos,
                       const clasp_kv_layer* kv, float temperature, uint64_t seed, int32_t round, int32_t* token_out,
                       float* logits_out) {
  if (!logits_out || !(temperature > 0.f) || round < 0 || !al16(logits_out)) return CLASP_ERR_INVALID_ARG;
  int rc = draft_impl(ctx, skip_mask_host, token_in, pos, kv, token_out, nullptr, logits_out);
  if (rc) return rc;
  // the drafted token will sit at position pos + 1
  clasp::smp::gumbel_argmax_kernel<<<1, clasp::smp::THREADS, 0, ctx->stream>>>(
      logits_out, ctx->cfg.vocab, 1.0f / temperature, (unsigned long long)seed, pos + 1, clasp::smp::DRAW_DRAFT, round,
      token_out);
  return launch_check(ctx);
}

int clasp_verify_sample(clasp_ctx* ctx, const int32_t* tokens, int32_t n, int32_t pos0, const clasp_kv_layer* kv,
                        int32_t n_drafts, const float* draft_logits, float temperature, uint64_t seed, int32_t round,
                        float* logits_ws, int32_t* n_accepted_out, int32_t* committed_out, float* hidden_out) {
  if (!ctx || !logits_ws || !n_accepted_out || !committed_out || n_drafts < 0 || n_drafts >= n || round < 0 ||
      !(temperature > 0.f) || (n_drafts > 0 && !draft_logits) || !al16(logits_ws))
    return CLASP_ERR_INVALID_ARG;
  if (n_drafts > clasp::smp::MAX_DRAFTS) return CLASP_ERR_CAPACITY;
  // the last n_drafts + 1 rows go through the head; their logits land in logits_ws
  int rc = verify_impl(ctx, tokens, n, pos0, kv, n_drafts + 1, committed_out, hidden_out, logits_ws);
  if (rc) return rc;
  const int first = pos0 + n - n_drafts;   // position of the first draft (of the sampled token when there is none)
  clasp::smp::spec_rows_kernel<<<n_drafts + 1, clasp::smp::THREADS, 0, ctx->stream>>>(
      logits_ws, draft_logits, tokens + (n - n_drafts), n_drafts, ctx->cfg.vocab, 1.0f / temperature,
      (unsigned long long)seed, first, round, ctx->ws.spec);
  if ((rc = launch_check(ctx))) return rc;
  clasp::smp::spec_commit_kernel<<<1, 32, 0, ctx->stream>>>(ctx->ws.spec, tokens + (n - n_drafts), n_drafts,
                                                            (unsigned long long)seed, first, round, n_accepted_out,
                                                            committed_out);
  return launch_check(ctx);
}

int clasp_accept(const int32_t* draft, const int32_t* full_argmax, int32_t K, int32_t* n_accepted,
                 int32_t* committed) {
  if (K < 0 || !full_argmax || !n_accepted || !committed || (K > 0 && !draft)) return CLASP_ERR_INVALID_ARG;
  int a = 0;
  while (a < K && draft[a] == full_argmax[a]) ++a;
  for (int k = 0; k < a; ++k) committed[k] = draft[k];
  committed[a] = full_argmax[a];
  *n_accepted = a;
  return CLASP_OK;
}

int clasp_gemm_xwT(clasp_ctx* ctx, const void* x, const void* w, int32_t R, int32_t N, int32_t K, float* y) {
  if (!ctx || !x || !w || !y || R < 1 || N < 1 || K < 8 || K % 8) return CLASP_ERR_INVALID_ARG;
  if (((uintptr_t)x & 15) || ((uintptr_t)w & 15)) return CLASP_ERR_INVALID_ARG;
  GemmCall g;
  g.x = x; g.R = R; g.K = K; g.n_mats = 1; g.w[0] = w; g.N[0] = N; g.epi = clasp::EPI_STORE;
  g.yf = y; g.ldy = N;
  CUtensorMap mp;
  if (ctx->use_tc) {
    if (make_map(ctx, w, N, K, clasp::tc::BM, &mp)) return CLASP_ERR_CUDA;
    g.wmap[0] = &mp;
    ctx->xmaps.clear();  // caller-owned operand buffers come and go: do not keep stale maps
  }
  return gemm(ctx, g);
}

}  // extern "C"

// ---------------------------------------------------------------- allocation-free GEMM
// Scratch of clasp_gemm_xwT_noalloc: [4 MiB split-K partial sums][4096 tile counters]
// [status word].  In host code the symbol below is only a stand-in: the device address
// comes from cudaGetSymbolAddress, once per device, with that device current.
static __device__ __align__(256) unsigned char g_noalloc_scratch[CLASP_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr size_t NOALLOC_PARTIAL_BYTES = 4u * 1024u * 1024u;
constexpr int NOALLOC_COUNTERS = 4096;
constexpr int NOALLOC_MAX_DEVICES = 64;
struct NoAllocDevice {
  bool ready = false;
  unsigned char* scratch = nullptr;
  EncodeTiledFn encode = nullptr;
  int cta_cap = 296;
};
NoAllocDevice g_noalloc_dev[NOALLOC_MAX_DEVICES];
std::mutex g_noalloc_mutex;  // guards the one-time set-up only

int noalloc_setup(int dev, NoAllocDevice** out) {
  if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return CLASP_ERR_CAPACITY;
  NoAllocDevice& nd = g_noalloc_dev[dev];
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (!nd.ready) {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return CLASP_ERR_CUDA;
    if (prop.major != 10) return CLASP_ERR_CUDA;
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return CLASP_ERR_CUDA;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn)
      return CLASP_ERR_CUDA;
    if (cudaFuncSetAttribute(clasp::tc::gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             220 * 1024) != cudaSuccess)
      return CLASP_ERR_CUDA;
    nd.scratch = (unsigned char*)ptr;
    nd.encode = (EncodeTiledFn)fn;
    nd.cta_cap = 2 * prop.multiProcessorCount;
    nd.ready = true;
  }
  *out = &nd;
  return CLASP_OK;
}

int noalloc_map(EncodeTiledFn encode, const void* ptr, int rows, int cols, int box_rows, CUtensorMap* out) {
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)clasp::tc::BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? CLASP_OK : CLASP_ERR_CUDA;
}
}  // namespace

extern "C" {

int clasp_gemm_xwT_noalloc(const void* x, const void* w, int32_t R, int32_t N, int32_t K, float* y,
                           void* cuda_stream, int32_t* status_out) {
  using namespace clasp::tc;
  if (!x || !w || !y || R < 1 || N < 1 || K < 8 || K % 8) return CLASP_ERR_INVALID_ARG;
  if (((uintptr_t)x & 15) || ((uintptr_t)w & 15)) return CLASP_ERR_INVALID_ARG;
  if (R > CLASP_NOALLOC_MAX_ROWS) return CLASP_ERR_CAPACITY;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return CLASP_ERR_CUDA;
  NoAllocDevice* nd = nullptr;
  int rc = noalloc_setup(dev, &nd);
  if (rc) return rc;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  Params p{};
  const int tiles = (N + BM - 1) / BM;
  p.N[0] = N; p.tiles[0] = tiles; p.col_off[0] = 0;
  p.K = K;
  p.k_chunks = (K + BK - 1) / BK;
  int splits = nd->cta_cap / tiles;  // the schedule of clasp_gemm_xwT: a function of (N, K) only
  const int max_splits = p.k_chunks / 4 > 1 ? p.k_chunks / 4 : 1;
  if (splits > max_splits) splits = max_splits;
  if (splits < 1) splits = 1;
  if (splits > 1 && tiles > MAX_COUNTERS) splits = 1;
  if (splits > 1) {
    if ((size_t)splits * R * N * sizeof(float) > NOALLOC_PARTIAL_BYTES || tiles > NOALLOC_COUNTERS)
      return CLASP_ERR_CAPACITY;
  }
  p.R = R;
  p.BN = R <= 16 ? 16 : (R + 15) / 16 * 16;
  p.splits = splits;
  p.dual = 0; p.n_mats = 1; p.epi = clasp::EPI_STORE; p.n_total = N;
  p.yf = y; p.ldy = N;
  p.partial = (float*)nd->scratch;
  p.counters = (int*)(nd->scratch + NOALLOC_PARTIAL_BYTES);
  int* scratch_status = (int*)(nd->scratch + NOALLOC_PARTIAL_BYTES + NOALLOC_COUNTERS * sizeof(int));
  p.status = status_out ? status_out : scratch_status;
  p.spin_fast = SPIN_FAST; p.spin_slow = SPIN_SLOW;
  const int stage_bytes = A_TILE_BYTES + p.BN * BK * 2;
  int stages = 110 * 1024 / stage_bytes;
  if (stages > 8) stages = 8;
  if (stages < 2) stages = 2;
  const int per_cta = (p.k_chunks + splits - 1) / splits;
  if (stages > per_cta) stages = per_cta < 1 ? 1 : per_cta;
  p.stages = stages;
  const size_t smem = (size_t)stages * stage_bytes + 1024;
  CUtensorMap map_w, map_x;
  if (noalloc_map(nd->encode, w, N, K, BM, &map_w) || noalloc_map(nd->encode, x, R, K, p.BN, &map_x))
    return CLASP_ERR_CUDA;
  // the array keeps whatever the previous call left: the counters must start at zero
  if (cudaMemsetAsync(p.counters, 0, (NOALLOC_COUNTERS + 64) * sizeof(int), stream) != cudaSuccess)
    return CLASP_ERR_CUDA;
  dim3 grid(tiles, splits), block(THREADS);
  gemm_tc_kernel<<<grid, block, smem, stream>>>(map_w, map_w, map_w, map_x, p);
  return cudaGetLastError() == cudaSuccess ? CLASP_OK : CLASP_ERR_CUDA;
}

int clasp_last_device_status(clasp_ctx* ctx) {
  if (!ctx) return CLASP_ERR_INVALID_ARG;
  int st = 0;
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return CLASP_ERR_CUDA;
  if (cudaMemcpy(&st, ctx->ws.status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return CLASP_ERR_CUDA;
  if (ctx->use_engine) {
    int est = 0;
    if (cudaMemcpy(&est, &ctx->ws.ctl->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
      return CLASP_ERR_CUDA;
    if (est != 0) {
      cudaMemset(ctx->ws.ctl, 0, sizeof(clasp::pk::Ctl));
      st = 1;
    }
  }
  if (st != 0) {
    cudaMemset(ctx->ws.status, 0, sizeof(int));
    cudaMemset(ctx->ws.counters, 0, MAX_COUNTERS * sizeof(int));
    return CLASP_ERR_TIMEOUT;
  }
  return CLASP_OK;
}

int clasp_profile_gemm(clasp_ctx* ctx, int32_t enable, int64_t* n_launches, double* total_ms,
                       double* weight_bytes) {
  if (!ctx) return CLASP_ERR_INVALID_ARG;
  if (enable) {
    ctx->profiling = true;
    return CLASP_OK;
  }
  ctx->profiling = false;
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return CLASP_ERR_CUDA;
  double ms = 0.0;
  int rc = CLASP_OK;
  for (auto& pr : ctx->prof_events) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, pr.first, pr.second) != cudaSuccess) rc = CLASP_ERR_CUDA;
    ms += t;
    cudaEventDestroy(pr.first);
    cudaEventDestroy(pr.second);
  }
  if (n_launches) *n_launches = (int64_t)ctx->prof_events.size();
  if (total_ms) *total_ms = ms;
  if (weight_bytes) *weight_bytes = ctx->prof_bytes;
  ctx->prof_events.clear();
  ctx->prof_bytes = 0.0;
  return rc;
}

int64_t clasp_launch_count(const clasp_ctx* ctx) { return ctx ? ctx->launches : 0; }

int clasp_engine_trace(clasp_ctx* ctx, uint64_t* stamps, int32_t cap_per_cta, int32_t* n_ctas) {
  if (!ctx) return CLASP_ERR_INVALID_ARG;
  if (n_ctas) *n_ctas = ctx->use_engine ? ctx->e_G : 0;
  if (cap_per_cta < 0) return CLASP_OK;   // query only: the trace buffer in use stays
  ctx->e_trace = (unsigned long long*)stamps;
  ctx->e_trace_cap = stamps ? cap_per_cta : 0;
  return CLASP_OK;
}

int clasp_engine_active(const clasp_ctx* ctx) {
  if (!ctx) return CLASP_ERR_INVALID_ARG;
  return ctx->use_engine ? 1 : 0;
}

int clasp_set_wait_limit(clasp_ctx* ctx, uint32_t polls) {
  if (!ctx) return CLASP_ERR_INVALID_ARG;
  ctx->wait_limit = polls;
  return CLASP_OK;
}

const char* clasp_strerror(int code) {
  switch (code) {
    case CLASP_OK: return "ok";
    case CLASP_ERR_INVALID_ARG: return "invalid argument";
    case CLASP_ERR_SHAPE: return "unsupported shape";
    case CLASP_ERR_CAPACITY: return "capacity exceeded";
    case CLASP_ERR_DTYPE: return "unsupported dtype";
    case CLASP_ERR_CUDA: return "CUDA error";
    case CLASP_ERR_TIMEOUT: return "device-side wait timed out";
    case CLASP_ERR_NOT_LOADED: return "weights not loaded";
    default: return "unknown error";
  }
}

}  // extern "C"
