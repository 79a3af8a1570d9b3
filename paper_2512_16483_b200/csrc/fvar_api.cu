// Host side of libfvar: the C ABI, workspace layout, TMA descriptors and the sequencing of one
// scale step over block groups.  See include/fvar.h for the contract of every entry point.
#include <stdio.h>
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <map>
#include <mutex>

#include <string>
#include <vector>

#include "../../include/fvar.h"
#include "internal.h"
#include "ptx.cuh"

namespace fvar {

// ------------------------------------------------------------------------------------------------
// Tensor maps (the driver entry point is fetched through the runtime: no link against libcuda).
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;

bool tmap_init_driver() {
  if (g_encode) return true;
  void *fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess) return false;
  if (qres != cudaDriverEntryPointSuccess || fn == nullptr) return false;
  g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  return true;
}

bool tmap_2d(CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows, uint64_t ld_elems, uint32_t box_rows) {
  if (!tmap_init_driver()) return false;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || (ld_elems * 2) % 16 || box_rows == 0 || box_rows > 256) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ld_elems * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tmap_3d(CUtensorMap *m, const void *base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t ld1_elems,
             uint64_t ld2_elems, uint32_t box0, uint32_t box1) {
  if (!tmap_init_driver()) return false;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || (ld1_elems * 2) % 16 || (ld2_elems * 2) % 16 || box1 == 0 ||
      box1 > 256)
    return false;
  cuuint64_t dims[3] = {d0, d1, d2};
  cuuint64_t strides[2] = {ld1_elems * 2, ld2_elems * 2};
  cuuint32_t box[3] = {box0, box1, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tmap_kblocks(CUtensorMap *m, const void *base, uint64_t rows, uint64_t kblocks, uint64_t ld_elems, uint32_t box_rows,
                  uint32_t box_kb) {
  if (!tmap_init_driver()) return false;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || (ld_elems * 2) % 16 || box_rows == 0 || box_rows > 256 || box_kb == 0 || box_kb > 256)
    return false;
  cuuint64_t dims[3] = {64, rows, kblocks};
  cuuint64_t strides[2] = {ld_elems * 2, 128};
  cuuint32_t box[3] = {64, box_rows, box_kb};
  cuuint32_t estr[3] = {1, 1, 1};
  return g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Status word used by the kernel-level entry points (contexts carry their own in the workspace).
__device__ unsigned g_kernel_status;

static std::string g_init_error;

// Address of the status word on the current device (resolved once per device ordinal).
static unsigned *kernel_status_ptr() {
  static std::mutex mu;
  static unsigned *cache[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!cache[dev]) {
    void *addr = nullptr;
    if (cudaGetSymbolAddress(&addr, g_kernel_status) != cudaSuccess) return nullptr;
    cache[dev] = static_cast<unsigned *>(addr);
  }
  return cache[dev];
}

void set_global_error(const char *msg) { g_init_error = msg ? msg : ""; }

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline int bn_index(int bn) { return bn == 64 ? 0 : (bn == 128 ? 1 : 2); }
static const int kBNs[3] = {64, 128, 256};
constexpr size_t kSplitScratchBytes = 64u << 20;   // split-K partial tiles
constexpr size_t kSplitCounters = 4096;            // one arrival counter per tile
constexpr int kMaxCodebook = 65536;                // largest codebook fvar_set_codebook takes

enum WeightId { W_QKV = 0, W_O, W_FC1, W_FC2, W_ADA, W_CQ, W_CKV, W_CO, W_COUNT };

}  // namespace fvar

using namespace fvar;

struct fvar_ctx {
  fvar_cfg cfg;
  std::vector<int> hw;                 // 2 * n_scales
  std::vector<int> Mk;                 // tokens per scale
  int G, C, F, H, D, Bmax, Mmax, L_cap, ctx_cap, num_sms;
  int max_clusters;                    // resident CTA pairs of the pair GEMM (0: pairs not used)
  cudaStream_t st;         // the caller's stream
  cudaStream_t launch_st;  // where launches go: st, or cap_st while a graph is being captured
  cudaStream_t cap_st;     // private stream used only for capture (the legacy default stream cannot be captured)
  cudaStream_t cap_st2;    // second capture stream: the selection / fill branch of a late group runs beside the blocks
  cudaEvent_t ev_fork, ev_join;
  std::string err;
  long long launches;
  // weights (device pointers per block)
  std::vector<const bf16 *> w[W_COUNT];
  std::vector<const bf16 *> b_qkv, b_o, b_fc1, b_fc2, b_ada, ln_c_gamma;
  std::vector<CUtensorMap> wmap;       // [blk][W_COUNT][3]
  // workspace regions
  uint8_t *ws;
  size_t ws_bytes;
  unsigned *status;
  bf16 *kc, *vt, *ckc, *cvt, *silu_c, *y, *q, *a, *hbuf, *qt_pool;
  bf16 *xsplit[2];                     // hi / lo bf16 split of a group's input rows, [E][2][Mk][C]; groups alternate
  float *ada, *gcache, *x0, *xs, *scores, *split_partial;
  // LLS restoration: upsampled cached group output (and its bf16 split), the two projections, G / G^-1, T and P
  float *cup, *lls_xhat, *lls_chat, *lls_G, *lls_Ginv, *lls_T, *lls_P;
  bf16 *csplit;
  std::vector<CUtensorMap> csplit_map; // [scale]
  int lls_rank_cap;                    // min(kLlsMaxRank, Mmax)
  bool last_lls;                       // the last step restored by LLS (no index sets)
  // transition between scale steps: codebook (caller's memory), half-norms, packed arg-max words, codes and
  // the accumulated feature map F_k at the last scale's resolution
  const bf16 *codebook;
  int codebook_V;
  float *tr_hn, *tr_F;
  unsigned long long *tr_best;
  int *tr_codes;
  int tr_scale;                        // last scale accumulated into tr_F (-1: none)
  int tr_B;
  // pipelined host entry point: two staging slots each way, one stream per copy direction
  bf16 *hin[2], *hout[2];
  cudaStream_t h2d_st, d2h_st;
  cudaEvent_t ev_in[2], ev_cmp[2], ev_out[2];
  long long host_calls;
  bool host_pipe_ok;
  int *idx, *inv, *split_counters;
  std::vector<size_t> qt_off;          // [scale][group] offset (elements) into qt_pool
  std::vector<int> qt_r;               // [scale][group] rank of the stored projection (0: none)
  std::vector<CUtensorMap> qt_map;     // [scale][group]
  std::vector<CUtensorMap> xsplit_map; // [scale][2 buffers]: rows = elements x (hi rows, lo rows), 64 x 64 boxes
  std::vector<CUtensorMap> kmap, vmap, ckmap, cvmap;   // per block
  // GEMM A operands: one map per box height (16, 32, 64, 128 rows); q_map feeds the attention kernel
  struct ActMaps {
    CUtensorMap m[4];
    const bf16 *base;                  // the buffer behind the maps: [rows][cols], for maps of other box heights
    uint64_t cols, rows;
  };
  ActMaps y_map, a_map, h_map, silu_map;
  CUtensorMap q_map;
  // state
  int B;                               // batch of the current generation (0: no cond set)
  std::vector<int> len;                // committed cache rows per block
  std::vector<int> staged;             // rows staged by the last step per block
  int staged_scale;                    // scale whose rows are staged (-1: none)
  int last_scale;                      // last stepped scale (-1: none)
  int cache_scale;                     // scale of the valid group cache (-1: none)
  int cache_slot;                      // slot holding it
  int null_only_seen;
  std::vector<int> last_rank;          // r per group of the last step
  int last_E, last_M;
  int loaded_len, loaded_cache_scale;  // state set by fvar_load_kv / fvar_load_group_cache (-1: none)
  // per-launch event timing (fvar_profile_*)
  struct ProfRec { int kclass; double flops, bytes; cudaEvent_t e0, e1; };
  // CUDA graphs of the step body, keyed by everything that is baked into the launches
  struct GraphEntry { cudaGraphExec_t exec; long long kernels; };
  std::map<std::string, GraphEntry> graphs;
  bool use_graphs;
  int max_splits;                      // largest split-K factor the tile picker may use (1, 2 or 4)
  long long wait_cycles;               // budget of the kernels' bounded waits (0: default)
  int skinny_max_rows;                 // GEMMs of at most this many rows take the weight-streaming form (0: never)
  void drop_graphs() {
    for (auto &kv : graphs) cudaGraphExecDestroy(kv.second.exec);
    graphs.clear();
  }
  bool prof_on;
  std::vector<ProfRec> prof;
  std::vector<cudaEvent_t> ev_pool;
  size_t ev_used;

  size_t kv_block_elems() const { return static_cast<size_t>(Bmax) * H * L_cap * D; }
  size_t ckv_block_elems() const { return static_cast<size_t>(Bmax) * H * ctx_cap * D; }
  // slots 0 and 1 alternate between scale steps; slot 2 holds what fvar_load_group_cache loaded
  float *gslot(int slot, int g) const {
    return gcache + (static_cast<size_t>(slot) * G + g) * Bmax * Mmax * C;
  }
  cudaEvent_t event() {
    if (ev_used == ev_pool.size()) {
      cudaEvent_t e = nullptr;
      cudaEventCreate(&e);
      ev_pool.push_back(e);
    }
    return ev_pool[ev_used++];
  }
  // While a graph is being captured an event becomes an event-record node of the graph (the "external"
  // flag), so that the profile pass times the kernels where the timed run executes them: inside the graph,
  // without the host between launches.  `s`: the stream of the launch (default: where launches go).
  void prof_record(cudaEvent_t e, cudaStream_t s) {
    if (launch_st == cap_st && cap_st != nullptr && launch_st != st)
      cudaEventRecordWithFlags(e, s, cudaEventRecordExternal);
    else
      cudaEventRecord(e, s);
  }
  void prof_begin(int kclass, double flops, double bytes, cudaStream_t s = nullptr) {
    if (!prof_on) return;
    ProfRec r{kclass, flops, bytes, event(), event()};
    prof_record(r.e0, s ? s : launch_st);
    prof.push_back(r);
  }
  void launched(cudaStream_t s = nullptr) {
    launches++;
    if (prof_on && !prof.empty()) prof_record(prof.back().e1, s ? s : launch_st);
  }
  std::vector<cudaGraphExec_t> prof_execs;   // graphs instantiated by the profile pass (one per step, not cached)
  void drop_prof_execs() {
    for (cudaGraphExec_t e : prof_execs) cudaGraphExecDestroy(e);
    prof_execs.clear();
  }
  const CUtensorMap &wm(int blk, int wid, int bn) const { return wmap[(blk * W_COUNT + wid) * 3 + bn_index(bn)]; }
};

namespace {

struct Layout {
  size_t status, split_partial, split_counters, kc, vt, ckc, cvt, ada, silu_c, gcache, x0, xs, y, q, a, hbuf, xsplit[2], scores, idx, inv, qt_pool, total;
  size_t cup, csplit, lls_xhat, lls_chat, lls_G, lls_Ginv, lls_T, lls_P;
  size_t tr_hn, tr_best, tr_codes, tr_F;
  size_t hin[2], hout[2];
  std::vector<size_t> qt_off;
};

bool shape_ok(const fvar_cfg *c, std::string *why) {
  auto bad = [&](const char *m) { if (why) *why = m; return false; };
  if (!c || !c->scale_hw) return bad("null cfg");
  if (c->n_blocks <= 0 || c->blocks_per_group <= 0 || c->n_blocks % c->blocks_per_group) return bad("block grouping");
  if (c->width <= 0 || c->width % 64 || c->width > 8192) return bad("width must be a multiple of 64, <= 8192");
  if (c->head_dim != 64 && c->head_dim != 128) return bad("head_dim must be 64 or 128");
  if (c->n_heads * c->head_dim != c->width) return bad("n_heads * head_dim != width");
  if (c->ffn_dim <= 0 || c->ffn_dim % 64) return bad("ffn_dim must be a multiple of 64");
  if (c->n_scales <= 0 || c->max_batch <= 0) return bad("n_scales / max_batch");
  for (int k = 0; k < c->n_scales; ++k)
    if (c->scale_hw[2 * k] <= 0 || c->scale_hw[2 * k + 1] <= 0) return bad("scale_hw");
  if (c->has_cross_attn && (c->ctx_len <= 0 || c->ctx_width <= 0 || c->ctx_width % 64)) return bad("context shape");
  if (!(c->ln_eps > 0.f)) return bad("ln_eps");
  return true;
}

Layout make_layout(const fvar_cfg *c) {
  Layout L;
  const size_t B = c->max_batch, C = c->width, F = c->ffn_dim, nb = c->n_blocks, G = nb / c->blocks_per_group;
  size_t Mmax = 0, Ltot = 0;
  for (int k = 0; k < c->n_scales; ++k) {
    const size_t m = static_cast<size_t>(c->scale_hw[2 * k]) * c->scale_hw[2 * k + 1];
    Mmax = m > Mmax ? m : Mmax;
    Ltot += m;
  }
  const size_t L_cap = align_up(Ltot, 128), ctx_cap = c->has_cross_attn ? align_up(c->ctx_len, 128) : 0;
  const size_t Mk = align_up(Mmax, 64);          // projection operands: [hi | lo] halves of Mk columns
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 1024); return o; };
  L.status = take(256);
  L.split_partial = take(kSplitScratchBytes);
  L.split_counters = take(kSplitCounters * 4);
  L.kc = take(nb * B * L_cap * C * 2);
  L.vt = take(nb * B * L_cap * C * 2);
  L.ckc = take(nb * B * ctx_cap * C * 2);
  L.cvt = take(nb * B * ctx_cap * C * 2);
  L.ada = take(nb * B * 6 * C * 4);
  L.silu_c = take(align_up(B, 128) * C * 2);
  L.gcache = take(3 * G * B * Mmax * C * 4);
  L.x0 = take(B * Mmax * C * 4);
  L.xs = take(B * Mmax * C * 4);
  L.y = take(B * Mmax * C * 2);
  L.q = take(B * Mmax * C * 2);
  L.a = take(B * Mmax * C * 2);
  L.hbuf = take(B * Mmax * F * 2);
  L.xsplit[0] = take(B * 2 * Mk * C * 2);
  L.xsplit[1] = take(B * 2 * Mk * C * 2);
  {
    const size_t R = Mmax < static_cast<size_t>(kLlsMaxRank) ? Mmax : static_cast<size_t>(kLlsMaxRank);
    L.cup = take(B * Mmax * C * 4);
    L.csplit = take(B * 2 * Mk * C * 2);
    L.lls_xhat = take(B * R * C * 4);
    L.lls_chat = take(B * R * C * 4);
    L.lls_G = take(2 * B * R * R * 4);
    L.lls_Ginv = take(2 * B * R * R * 4);
    L.lls_T = take(2 * B * R * C * 4);
    L.lls_P = take(2 * B * Mmax * R * 4);
  }
  L.scores = take(B * Mmax * 4);
  L.idx = take(G * B * Mmax * 4);
  L.inv = take(G * B * Mmax * 4);
  L.qt_pool = off;
  size_t pool = 0;
  L.qt_off.resize(static_cast<size_t>(c->n_scales) * G);
  for (int k = 0; k < c->n_scales; ++k) {
    const size_t m = static_cast<size_t>(c->scale_hw[2 * k]) * c->scale_hw[2 * k + 1];
    for (size_t g = 0; g < G; ++g) {
      L.qt_off[k * G + g] = pool;
      pool += align_up(m * 2 * align_up(m, 64), 512);  // elements; r <= M rows of [Q^T | Q^T]
    }
  }
  take(pool * 2);
  const size_t M_last = static_cast<size_t>(c->scale_hw[2 * (c->n_scales - 1)]) * c->scale_hw[2 * (c->n_scales - 1) + 1];
  L.tr_hn = take(static_cast<size_t>(kMaxCodebook) * 4);
  L.tr_best = take(B * Mmax * 8);
  L.tr_codes = take(B * Mmax * 4);
  L.tr_F = take(B * M_last * C * 4);
  for (int s2 = 0; s2 < 2; ++s2) {
    L.hin[s2] = take(B * Mmax * C * 2);
    L.hout[s2] = take(B * Mmax * C * 2);
  }
  L.total = off;
  return L;
}

fvar_status fail(fvar_ctx *ctx, fvar_status s, const std::string &msg) {
  if (ctx) ctx->err = msg; else g_init_error = msg;
  return s;
}

fvar_status cuda_fail(fvar_ctx *ctx, cudaError_t e, const char *what) {
  return fail(ctx, FVAR_ECUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

#define FV_CUDA(ctx, call, what)                                \
  do {                                                          \
    cudaError_t e__ = (call);                                   \
    if (e__ != cudaSuccess) return cuda_fail(ctx, e__, what);   \
  } while (0)

// out = A W^T (+ epilogue) on the context's stream; picks the tile width from the problem size.
fvar_status run_gemm_map(fvar_ctx *ctx, int epi, const CUtensorMap &tmA, int blk, int wid, GemmArgs &g, const char *what);

// A operand from one of the library's activation buffers: a single row tile takes the shortest box
// that covers its rows.
fvar_status run_gemm(fvar_ctx *ctx, int epi, const fvar_ctx::ActMaps &maps, int blk, int wid, GemmArgs &g, const char *what) {
  if (g.nbatch == 1 && g.R <= ctx->skinny_max_rows && g.R <= gemm_skinny_row_limit(g.N, g.K) && !gemm_ksplit_wins(g.R, g.N, g.K) &&
      gemm_skinny_supported(epi, g.R, g.N, g.K)) {
    // few rows: bound by streaming the weights once, so the weights take the M side of the MMA and the K range
    // of every 128-feature tile is spread over a cluster (gemm_skinny.cu)
    const int S = gemm_skinny_pick_splits(g.N, g.K, 0, 0, g.R <= 64);
    g.splits = S;
    gemm_skinny_shape(g);
    CUtensorMap tmA, tmW;
    if (S > 0 && g.sk_stages >= 1 && gemm_skinny_map(&tmA, maps.base, maps.rows, maps.cols, maps.cols, g.sk_rp, g.sk_nk) &&
        gemm_skinny_map(&tmW, ctx->w[wid][blk], g.N, g.K, g.K, 128, g.sk_nk)) {
      g.splits = S;
      g.status = ctx->status;
      g.wait_cycles = ctx->wait_cycles;
      ctx->prof_begin(FVAR_KCLASS_GEMM, 2.0 * g.R * g.N * g.K,
                      2.0 * (static_cast<double>(g.N) * g.K + static_cast<double>(g.R) * g.K) +
                          (epi == EPI_F32 || epi == EPI_RESID ? 4.0 : 2.0) * g.R * g.N);
      FV_CUDA(ctx, launch_gemm_skinny(epi, tmA, tmW, g, ctx->launch_st), what);
      ctx->launched();
      return FVAR_OK;
    }
    g.splits = 1;
  }
  g.pf_ptr = nullptr;
  if (g.nbatch == 1 && ctx->skinny_max_rows > 0 && gemm_ksplit_wins(g.R, g.N, g.K) && epi != EPI_ARGMAX && g.N % 8 == 0) {
    // a few hundred rows, narrow output: 128 x 128 tiles with the K range spread over a cluster (gemm_skinny.cu, ROWS)
    g.sk_tiles_m = (g.R + 127) / 128;
    const int S = gemm_skinny_pick_splits(g.N, g.K, 0, g.sk_tiles_m);
    g.splits = S;
    gemm_skinny_shape(g);
    CUtensorMap tmA, tmW;
    if (S > 0 && g.sk_stages >= 1 && gemm_skinny_map(&tmA, maps.base, maps.rows, maps.cols, maps.cols, 128, g.sk_nk) &&
        gemm_skinny_map(&tmW, ctx->w[wid][blk], g.N, g.K, g.K, 128, g.sk_nk)) {
      g.status = ctx->status;
      g.wait_cycles = ctx->wait_cycles;
      ctx->prof_begin(FVAR_KCLASS_GEMM, 2.0 * g.R * g.N * g.K,
                      2.0 * (static_cast<double>(g.N) * g.K + static_cast<double>(g.R) * g.K) +
                          (epi == EPI_F32 || epi == EPI_RESID ? 4.0 : 2.0) * g.R * g.N);
      FV_CUDA(ctx, launch_gemm_skinny(epi, tmA, tmW, g, ctx->launch_st), what);
      ctx->launched();
      return FVAR_OK;
    }
    g.sk_tiles_m = 0;
    g.splits = 1;
  }
  int t = 3;
  if (g.nbatch == 1 && g.R <= 64) t = g.R <= 16 ? 0 : (g.R <= 32 ? 1 : 2);
  g.a_box_rows = 16 << t;
  return run_gemm_map(ctx, epi, maps.m[t], blk, wid, g, what);
}

fvar_status run_gemm_map(fvar_ctx *ctx, int epi, const CUtensorMap &tmA, int blk, int wid, GemmArgs &g, const char *what) {
  // CTA pairs need the full 128-row A box (tmA is then the activation buffer's 128-row map)
  const GemmPlan plan = gemm_plan(g.R, g.nbatch, g.N, g.K, ctx->num_sms, (g.a_box_rows == 128 || g.a_box_rows == 0) ? ctx->max_clusters : 0,
                                  ctx->max_splits, kSplitScratchBytes);
  const int bn = plan.block_n;
  g.splits = plan.splits;
  g.partial = ctx->split_partial;
  g.counters = ctx->split_counters;
  g.status = ctx->status;
  g.wait_cycles = ctx->wait_cycles;
  ctx->prof_begin(FVAR_KCLASS_GEMM, 2.0 * g.R * g.N * g.K * g.nbatch,
                  2.0 * (static_cast<double>(g.N) * g.K + static_cast<double>(g.R) * g.K * g.nbatch) +
                      (epi == EPI_F32 || epi == EPI_RESID ? 4.0 : 2.0) * g.R * g.N * g.nbatch);
  if (plan.pair)
    FV_CUDA(ctx, launch_gemm_pair(epi, bn, tmA, ctx->wm(blk, wid, bn / 2), g, ctx->launch_st), what);
  else
    FV_CUDA(ctx, launch_gemm(epi, bn, tmA, ctx->wm(blk, wid, bn), g, ctx->num_sms, ctx->launch_st), what);
  ctx->launched();
  return FVAR_OK;
}

GemmArgs gemm_args(int R, int N, int K) {
  GemmArgs g;
  memset(&g, 0, sizeof(g));
  g.R = R; g.N = N; g.K = K;
  g.nbatch = 1;
  g.rows_per_batch = R > 0 ? R : 1;
  g.bmul = 1;
  g.rmap = RowMap{1, 0, R};
  g.omap = RowMap{1, 0, R};
  return g;
}

}  // namespace

// ================================================================================================
extern "C" {

size_t fvar_workspace_bytes(const fvar_cfg *cfg) {
  if (!shape_ok(cfg, nullptr)) return 0;
  return make_layout(cfg).total;
}

fvar_status fvar_init(const fvar_weights *weights, const fvar_cfg *cfg, void *workspace, size_t bytes,
                      void *cuda_stream, fvar_ctx **out) {
  if (!out) return fail(nullptr, FVAR_EINVAL, "out is NULL");
  *out = nullptr;
  std::string why;
  if (!shape_ok(cfg, &why)) return fail(nullptr, FVAR_EINVAL, "bad shape: " + why);
  if (!weights || !workspace) return fail(nullptr, FVAR_EINVAL, "weights / workspace is NULL");
  if (reinterpret_cast<uintptr_t>(workspace) & 1023) return fail(nullptr, FVAR_EINVAL, "workspace must be 1024-byte aligned");
  const Layout L = make_layout(cfg);
  if (bytes < L.total) return fail(nullptr, FVAR_ENOMEM, "workspace too small");

  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess)
    return fail(nullptr, FVAR_ECUDA, "no CUDA device");
  if (prop.major != 10) return fail(nullptr, FVAR_ECUDA, "libfvar needs an sm_100 device (B200)");
  if (!tmap_init_driver()) return fail(nullptr, FVAR_ECUDA, "cuTensorMapEncodeTiled is not available");

  fvar_ctx *c = new fvar_ctx();
  c->cfg = *cfg;
  c->hw.assign(cfg->scale_hw, cfg->scale_hw + 2 * cfg->n_scales);
  c->cfg.scale_hw = c->hw.data();
  c->G = cfg->n_blocks / cfg->blocks_per_group;
  c->C = cfg->width; c->F = cfg->ffn_dim; c->H = cfg->n_heads; c->D = cfg->head_dim; c->Bmax = cfg->max_batch;
  c->Mmax = 0;
  size_t Ltot = 0;
  for (int k = 0; k < cfg->n_scales; ++k) {
    const int m = c->hw[2 * k] * c->hw[2 * k + 1];
    c->Mk.push_back(m);
    c->Mmax = m > c->Mmax ? m : c->Mmax;
    Ltot += m;
  }
  c->L_cap = static_cast<int>(align_up(Ltot, 128));
  c->ctx_cap = cfg->has_cross_attn ? static_cast<int>(align_up(cfg->ctx_len, 128)) : 0;
  c->num_sms = prop.multiProcessorCount;
  c->st = static_cast<cudaStream_t>(cuda_stream);
  c->launch_st = c->st;
  c->cap_st = nullptr;
  c->cap_st2 = nullptr;
  c->ev_fork = c->ev_join = nullptr;
  c->launches = 0;
  c->ws = static_cast<uint8_t *>(workspace);
  c->ws_bytes = bytes;
  auto at = [&](size_t off) { return c->ws + off; };
  c->status = reinterpret_cast<unsigned *>(at(L.status));
  c->split_partial = reinterpret_cast<float *>(at(L.split_partial));
  c->split_counters = reinterpret_cast<int *>(at(L.split_counters));
  c->kc = reinterpret_cast<bf16 *>(at(L.kc)); c->vt = reinterpret_cast<bf16 *>(at(L.vt));
  c->ckc = reinterpret_cast<bf16 *>(at(L.ckc)); c->cvt = reinterpret_cast<bf16 *>(at(L.cvt));
  c->ada = reinterpret_cast<float *>(at(L.ada)); c->silu_c = reinterpret_cast<bf16 *>(at(L.silu_c));
  c->gcache = reinterpret_cast<float *>(at(L.gcache));
  c->x0 = reinterpret_cast<float *>(at(L.x0)); c->xs = reinterpret_cast<float *>(at(L.xs));
  c->y = reinterpret_cast<bf16 *>(at(L.y)); c->q = reinterpret_cast<bf16 *>(at(L.q));
  c->a = reinterpret_cast<bf16 *>(at(L.a)); c->hbuf = reinterpret_cast<bf16 *>(at(L.hbuf));
  c->xsplit[0] = reinterpret_cast<bf16 *>(at(L.xsplit[0])); c->xsplit[1] = reinterpret_cast<bf16 *>(at(L.xsplit[1]));
  c->scores = reinterpret_cast<float *>(at(L.scores));
  c->cup = reinterpret_cast<float *>(at(L.cup)); c->csplit = reinterpret_cast<bf16 *>(at(L.csplit));
  c->lls_xhat = reinterpret_cast<float *>(at(L.lls_xhat)); c->lls_chat = reinterpret_cast<float *>(at(L.lls_chat));
  c->lls_G = reinterpret_cast<float *>(at(L.lls_G)); c->lls_Ginv = reinterpret_cast<float *>(at(L.lls_Ginv));
  c->lls_T = reinterpret_cast<float *>(at(L.lls_T)); c->lls_P = reinterpret_cast<float *>(at(L.lls_P));
  c->lls_rank_cap = c->Mmax < kLlsMaxRank ? c->Mmax : kLlsMaxRank;
  c->last_lls = false;
  c->idx = reinterpret_cast<int *>(at(L.idx)); c->inv = reinterpret_cast<int *>(at(L.inv));
  c->qt_pool = reinterpret_cast<bf16 *>(at(L.qt_pool));
  c->tr_hn = reinterpret_cast<float *>(at(L.tr_hn)); c->tr_F = reinterpret_cast<float *>(at(L.tr_F));
  c->tr_best = reinterpret_cast<unsigned long long *>(at(L.tr_best)); c->tr_codes = reinterpret_cast<int *>(at(L.tr_codes));
  c->codebook = nullptr; c->codebook_V = 0; c->tr_scale = -1; c->tr_B = 0;
  for (int s2 = 0; s2 < 2; ++s2) {
    c->hin[s2] = reinterpret_cast<bf16 *>(at(L.hin[s2]));
    c->hout[s2] = reinterpret_cast<bf16 *>(at(L.hout[s2]));
    c->ev_in[s2] = c->ev_cmp[s2] = c->ev_out[s2] = nullptr;
  }
  c->h2d_st = c->d2h_st = nullptr;
  c->host_calls = 0;
  c->qt_off = L.qt_off;
  c->qt_r.assign(L.qt_off.size(), 0);
  c->qt_map.resize(L.qt_off.size());

  auto destroy_fail = [&](fvar_status s, const std::string &m) { delete c; return fail(nullptr, s, m); };

  const int nb = cfg->n_blocks;
  const void *const *srcs[W_COUNT] = {weights->w_qkv, weights->w_o, weights->w_fc1, weights->w_fc2,
                                      weights->w_ada, weights->w_cq, weights->w_ckv, weights->w_co};
  const int n_w = cfg->has_cross_attn ? W_COUNT : W_CQ;
  for (int i = 0; i < n_w; ++i) {
    if (!srcs[i]) return destroy_fail(FVAR_EINVAL, "a weight array is NULL");
    for (int b = 0; b < nb; ++b) {
      if (!srcs[i][b]) return destroy_fail(FVAR_EINVAL, "a weight pointer is NULL");
      c->w[i].push_back(static_cast<const bf16 *>(srcs[i][b]));
    }
  }
  const void *const *bsrc[6] = {weights->b_qkv, weights->b_o, weights->b_fc1, weights->b_fc2, weights->b_ada,
                                weights->ln_c_gamma};
  std::vector<const bf16 *> *bdst[6] = {&c->b_qkv, &c->b_o, &c->b_fc1, &c->b_fc2, &c->b_ada, &c->ln_c_gamma};
  for (int i = 0; i < (cfg->has_cross_attn ? 6 : 5); ++i) {
    if (!bsrc[i]) return destroy_fail(FVAR_EINVAL, "a bias array is NULL");
    for (int b = 0; b < nb; ++b) {
      if (!bsrc[i][b]) return destroy_fail(FVAR_EINVAL, "a bias pointer is NULL");
      bdst[i]->push_back(static_cast<const bf16 *>(bsrc[i][b]));
    }
  }

  // Tensor maps.  Weights: [out][in], one map per tile width.  Activations: full-capacity buffers.
  const int C = c->C, F = c->F;
  const int w_rows[W_COUNT] = {3 * C, C, F, C, 6 * C, C, 2 * C, C};
  const int w_cols[W_COUNT] = {C, C, C, F, C, C, cfg->ctx_width, C};
  c->wmap.resize(static_cast<size_t>(nb) * W_COUNT * 3);
  bool ok = true;
  for (int b = 0; b < nb && ok; ++b)
    for (int i = 0; i < n_w && ok; ++i)
      for (int t = 0; t < 3 && ok; ++t)
        ok = tmap_2d(&c->wmap[(b * W_COUNT + i) * 3 + t], c->w[i][b], w_cols[i], w_rows[i], w_cols[i], kBNs[t]);
  const size_t act_rows = static_cast<size_t>(c->Bmax) * c->Mmax;
  c->y_map.base = c->y; c->y_map.cols = C; c->y_map.rows = act_rows;
  c->a_map.base = c->a; c->a_map.cols = C; c->a_map.rows = act_rows;
  c->h_map.base = c->hbuf; c->h_map.cols = F; c->h_map.rows = act_rows;
  c->silu_map.base = c->silu_c; c->silu_map.cols = C; c->silu_map.rows = c->Bmax;
  for (int t = 0; t < 4 && ok; ++t) {
    const uint32_t box = 16u << t;
    ok = tmap_2d(&c->y_map.m[t], c->y, C, act_rows, C, box) && tmap_2d(&c->a_map.m[t], c->a, C, act_rows, C, box) &&
         tmap_2d(&c->h_map.m[t], c->hbuf, F, act_rows, F, box) && tmap_2d(&c->silu_map.m[t], c->silu_c, C, c->Bmax, C, box);
  }
  ok = ok && tmap_2d(&c->q_map, c->q, C, act_rows, C, 128);
  c->xsplit_map.resize(static_cast<size_t>(cfg->n_scales) * 2);
  for (int k = 0; k < cfg->n_scales && ok; ++k)
    for (int t = 0; t < 2 && ok; ++t)
      ok = tmap_2d(&c->xsplit_map[k * 2 + t], c->xsplit[t], C, static_cast<size_t>(c->Bmax) * 2 * align_up(c->Mk[k], 64), C, 64);
  c->csplit_map.resize(cfg->n_scales);
  for (int k = 0; k < cfg->n_scales && ok; ++k)
    ok = tmap_2d(&c->csplit_map[k], c->csplit, C, static_cast<size_t>(c->Bmax) * 2 * align_up(c->Mk[k], 64), C, 64);
  c->kmap.resize(nb); c->vmap.resize(nb); c->ckmap.resize(nb); c->cvmap.resize(nb);
  const int BH = c->Bmax * c->H, D = c->D;
  for (int b = 0; b < nb && ok; ++b) {
    ok = tmap_3d(&c->kmap[b], c->kc + b * c->kv_block_elems(), D, c->L_cap, BH, D, static_cast<uint64_t>(c->L_cap) * D, 64, 128) &&
         tmap_3d(&c->vmap[b], c->vt + b * c->kv_block_elems(), c->L_cap, D, BH, c->L_cap, static_cast<uint64_t>(c->L_cap) * D, 64, D);
    if (ok && cfg->has_cross_attn)
      ok = tmap_3d(&c->ckmap[b], c->ckc + b * c->ckv_block_elems(), D, c->ctx_cap, BH, D, static_cast<uint64_t>(c->ctx_cap) * D, 64, 128) &&
           tmap_3d(&c->cvmap[b], c->cvt + b * c->ckv_block_elems(), c->ctx_cap, D, BH, c->ctx_cap, static_cast<uint64_t>(c->ctx_cap) * D, 64, D);
  }
  if (!ok) return destroy_fail(FVAR_ECUDA, "tensor map encoding failed");

  cudaError_t e = cudaMemsetAsync(c->ws, 0, L.total, c->st);
  if (e != cudaSuccess) return destroy_fail(FVAR_ECUDA, std::string("workspace memset: ") + cudaGetErrorString(e));

  c->B = 0;
  c->len.assign(nb, 0);
  c->staged.assign(nb, 0);
  c->staged_scale = -1; c->last_scale = -1; c->cache_scale = -1; c->cache_slot = 0; c->null_only_seen = 0;
  c->last_rank.assign(c->G, 0);
  c->last_E = 0; c->last_M = 0;
  c->loaded_len = -1; c->loaded_cache_scale = -1;
  c->prof_on = false; c->ev_used = 0;
  c->max_splits = 1;
  c->skinny_max_rows = 512;
  c->wait_cycles = 0;
  c->use_graphs = cudaStreamCreateWithFlags(&c->cap_st, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&c->cap_st2, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) == cudaSuccess;
  c->host_pipe_ok = cudaStreamCreateWithFlags(&c->h2d_st, cudaStreamNonBlocking) == cudaSuccess &&
                    cudaStreamCreateWithFlags(&c->d2h_st, cudaStreamNonBlocking) == cudaSuccess;
  for (int s2 = 0; s2 < 2 && c->host_pipe_ok; ++s2)
    c->host_pipe_ok = cudaEventCreateWithFlags(&c->ev_in[s2], cudaEventDisableTiming) == cudaSuccess &&
                      cudaEventCreateWithFlags(&c->ev_cmp[s2], cudaEventDisableTiming) == cudaSuccess &&
                      cudaEventCreateWithFlags(&c->ev_out[s2], cudaEventDisableTiming) == cudaSuccess;
  if (lls_prepare() != cudaSuccess || gemm_prepare() != cudaSuccess || gemm_pair_prepare() != cudaSuccess || gemm_skinny_prepare() != cudaSuccess ||
      attention_prepare() != cudaSuccess)
    return destroy_fail(FVAR_ECUDA, "kernel attribute set-up failed");
  c->max_clusters = gemm_pair_max_clusters();
  *out = c;
  return FVAR_OK;
}

fvar_status fvar_reset(fvar_ctx *ctx) {
  if (!ctx) return FVAR_EINVAL;
  std::fill(ctx->len.begin(), ctx->len.end(), 0);
  std::fill(ctx->staged.begin(), ctx->staged.end(), 0);
  ctx->staged_scale = -1; ctx->last_scale = -1; ctx->cache_scale = -1; ctx->null_only_seen = 0;
  ctx->loaded_len = -1; ctx->loaded_cache_scale = -1;
  return FVAR_OK;
}

fvar_status fvar_restore_loaded(fvar_ctx *ctx) {
  if (!ctx) return FVAR_EINVAL;
  if (ctx->loaded_len < 0 || ctx->loaded_cache_scale < 0)
    return fail(ctx, FVAR_ESTATE, "restore_loaded: needs fvar_load_kv and fvar_load_group_cache first");
  std::fill(ctx->len.begin(), ctx->len.end(), ctx->loaded_len);
  std::fill(ctx->staged.begin(), ctx->staged.end(), 0);
  ctx->staged_scale = -1;
  ctx->last_scale = ctx->loaded_cache_scale;
  ctx->cache_scale = ctx->loaded_cache_scale;
  ctx->cache_slot = 2;
  ctx->null_only_seen = 0;
  return FVAR_OK;
}

fvar_status fvar_set_option(fvar_ctx *ctx, int option, int value) {
  if (!ctx) return FVAR_EINVAL;
  if (option == FVAR_OPT_CUDA_GRAPHS) {
    ctx->use_graphs = value != 0;
    if (!value) {
      FV_CUDA(ctx, cudaStreamSynchronize(ctx->st), "stream synchronize");
      ctx->drop_graphs();
    }
    return FVAR_OK;
  }
  if (option == FVAR_OPT_GEMM_MAX_SPLITS) {
    if (value != 1 && value != 2 && value != 4) return fail(ctx, FVAR_EINVAL, "set_option: max splits must be 1, 2 or 4");
    FV_CUDA(ctx, cudaStreamSynchronize(ctx->st), "stream synchronize");
    ctx->drop_graphs();
    ctx->max_splits = value;
    return FVAR_OK;
  }
  if (option == FVAR_OPT_WAIT_KCYCLES) {
    if (value < 0) return fail(ctx, FVAR_EINVAL, "set_option: the wait budget must not be negative");
    FV_CUDA(ctx, cudaStreamSynchronize(ctx->st), "stream synchronize");
    ctx->drop_graphs();
    ctx->wait_cycles = static_cast<long long>(value) * 1000;
    return FVAR_OK;
  }
  if (option == FVAR_OPT_SKINNY_MAX_ROWS) {
    if (value < 0 || value > 512) return fail(ctx, FVAR_EINVAL, "set_option: skinny rows must be in [0, 512]");
    FV_CUDA(ctx, cudaStreamSynchronize(ctx->st), "stream synchronize");
    ctx->drop_graphs();
    ctx->skinny_max_rows = value;
    return FVAR_OK;
  }
  return fail(ctx, FVAR_EINVAL, "set_option: unknown option");
}

fvar_status fvar_profile_enable(fvar_ctx *ctx, int on) {
  if (!ctx) return FVAR_EINVAL;
  FV_CUDA(ctx, cudaStreamSynchronize(ctx->st), "stream synchronize");
  ctx->drop_prof_execs();
  ctx->prof.clear();
  ctx->ev_used = 0;
  ctx->prof_on = on != 0;
  return FVAR_OK;
}

fvar_status fvar_profile_dump(fvar_ctx *ctx, int kclass, float *ms_host, int capacity, int *count_host) {
  if (!ctx || !ms_host || !count_host || capacity < 0) return FVAR_EINVAL;
  FV_CUDA(ctx, cudaStreamSynchronize(ctx->st), "stream synchronize");
  int n = 0;
  for (const auto &r : ctx->prof) {
    if (r.kclass != kclass) continue;
    if (n < capacity) FV_CUDA(ctx, cudaEventElapsedTime(&ms_host[n], r.e0, r.e1), "event elapsed");
    ++n;
  }
  *count_host = n;
  return FVAR_OK;
}

fvar_status fvar_profile_read(fvar_ctx *ctx, int kclass, double *total_ms, long long *launches, double *flops,
                              double *bytes) {
  if (!ctx || !total_ms || !launches || !flops || !bytes) return FVAR_EINVAL;
  FV_CUDA(ctx, cudaStreamSynchronize(ctx->st), "stream synchronize");
  *total_ms = 0; *launches = 0; *flops = 0; *bytes = 0;
  for (const auto &r : ctx->prof) {
    if (r.kclass != kclass) continue;
    float ms = 0.f;
    FV_CUDA(ctx, cudaEventElapsedTime(&ms, r.e0, r.e1), "event elapsed");
    *total_ms += ms; *launches += 1; *flops += r.flops; *bytes += r.bytes;
  }
  return FVAR_OK;
}

void fvar_destroy(fvar_ctx *ctx) {
  if (!ctx) return;
  for (cudaEvent_t e : ctx->ev_pool) cudaEventDestroy(e);
  ctx->drop_prof_execs();
  ctx->drop_graphs();
  if (ctx->h2d_st) cudaStreamDestroy(ctx->h2d_st);
  if (ctx->d2h_st) cudaStreamDestroy(ctx->d2h_st);
  for (int s2 = 0; s2 < 2; ++s2) {
    if (ctx->ev_in[s2]) cudaEventDestroy(ctx->ev_in[s2]);
    if (ctx->ev_cmp[s2]) cudaEventDestroy(ctx->ev_cmp[s2]);
    if (ctx->ev_out[s2]) cudaEventDestroy(ctx->ev_out[s2]);
  }
  if (ctx->cap_st) cudaStreamDestroy(ctx->cap_st);
  if (ctx->cap_st2) cudaStreamDestroy(ctx->cap_st2);
  if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
  if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
  delete ctx;
}

const char *fvar_last_error(const fvar_ctx *ctx) { return ctx ? ctx->err.c_str() : g_init_error.c_str(); }

int fvar_cache_len(const fvar_ctx *ctx, int block) {
  if (!ctx || block < 0 || block >= ctx->cfg.n_blocks) return -1;
  return ctx->len[block];
}

long long fvar_launch_count(const fvar_ctx *ctx) { return ctx ? ctx->launches : 0; }

fvar_status fvar_poll_status(fvar_ctx *ctx) {
  unsigned word = 0;
  if (ctx) {
    FV_CUDA(ctx, cudaStreamSynchronize(ctx->st), "stream synchronize");
    FV_CUDA(ctx, cudaMemcpy(&word, ctx->status, sizeof(word), cudaMemcpyDeviceToHost), "status read");
    if (word) FV_CUDA(ctx, cudaMemset(ctx->status, 0, sizeof(word)), "status clear");
    if (word & kStatusTimeout) {
      // a kernel that gave up may have left arrival counters of a split reduction half counted
      FV_CUDA(ctx, cudaMemset(ctx->split_counters, 0, kSplitCounters * sizeof(int)), "counters clear");
      ctx->drop_graphs();
    }
  } else {
    FV_CUDA(ctx, cudaDeviceSynchronize(), "device synchronize");
    unsigned *ks = kernel_status_ptr();
    if (!ks) return fail(ctx, FVAR_ECUDA, "status word");
    FV_CUDA(ctx, cudaMemcpy(&word, ks, sizeof(word), cudaMemcpyDeviceToHost), "status read");
    if (word) FV_CUDA(ctx, cudaMemset(ks, 0, sizeof(word)), "status clear");
  }
  if (word & kStatusTimeout) return fail(ctx, FVAR_ETIMEOUT, "a device-side wait ran out");
  if (word & kStatusBadIndex) return fail(ctx, FVAR_EINVAL, "forced_indices out of range or not ascending");
  return FVAR_OK;
}

fvar_status fvar_set_cond(fvar_ctx *ctx, int B, const void *cond, const void *context) {
  if (!ctx) return FVAR_EINVAL;
  if (B <= 0 || B > ctx->Bmax || !cond) return fail(ctx, FVAR_EINVAL, "set_cond: bad batch or NULL cond");
  if (ctx->cfg.has_cross_attn && !context) return fail(ctx, FVAR_EINVAL, "set_cond: context is NULL");
  const int C = ctx->C, nb = ctx->cfg.n_blocks;
  FV_CUDA(ctx, launch_silu_bf16(static_cast<const bf16 *>(cond), ctx->silu_c, static_cast<long long>(B) * C, ctx->st), "silu");
  ctx->launched();
  for (int blk = 0; blk < nb; ++blk) {
    GemmArgs g = gemm_args(B, 6 * C, C);
    g.bias = ctx->b_ada[blk];
    g.out_f32 = ctx->ada + static_cast<size_t>(blk) * ctx->Bmax * 6 * C;
    g.ld_out = 6 * C;
    fvar_status s = run_gemm(ctx, EPI_F32, ctx->silu_map, blk, W_ADA, g, "ada gemm");
    if (s != FVAR_OK) return s;
  }
  if (ctx->cfg.has_cross_attn) {
    CUtensorMap ctx_map;
    const int T = ctx->cfg.ctx_len, Wc = ctx->cfg.ctx_width;
    if (!tmap_2d(&ctx_map, context, Wc, static_cast<uint64_t>(B) * T, Wc, 128))
      return fail(ctx, FVAR_EINVAL, "set_cond: context must be 16-byte aligned");
    for (int blk = 0; blk < nb; ++blk) {
      GemmArgs g = gemm_args(B * T, 2 * C, Wc);
      g.rows_per_batch = T;
      g.kc = ctx->ckc + blk * ctx->ckv_block_elems();
      g.vt = ctx->cvt + blk * ctx->ckv_block_elems();
      g.C = C; g.H = ctx->H; g.D = ctx->D; g.L_cap = ctx->ctx_cap; g.L_prev = 0; g.col_base = C;
      g.out_bf16 = ctx->q; g.ld_out = C;           // unused: no column maps to the q part
      fvar_status s = run_gemm_map(ctx, EPI_QKV, ctx_map, blk, W_CKV, g, "context kv gemm");
      if (s != FVAR_OK) return s;
    }
  }
  ctx->B = B;
  return fvar_reset(ctx);
}

fvar_status fvar_set_projection(fvar_ctx *ctx, int scale_idx, int group, const void *Qt, int r) {
  if (!ctx) return FVAR_EINVAL;
  if (scale_idx < 0 || scale_idx >= ctx->cfg.n_scales || group < 0 || group >= ctx->G || !Qt)
    return fail(ctx, FVAR_EINVAL, "set_projection: bad scale / group / pointer");
  const int M = ctx->Mk[scale_idx];
  if (r <= 0 || r > M) return fail(ctx, FVAR_EINVAL, "set_projection: need 0 < r <= M");
  // Stored as [Q^T | Q^T] with each half padded to Mk columns: the projection GEMM multiplies it
  // with the [hi | lo] split of the token rows (the padding stays zero from fvar_init).
  const size_t Mk = align_up(M, 64), slot = static_cast<size_t>(scale_idx) * ctx->G + group;
  bf16 *dst = ctx->qt_pool + ctx->qt_off[slot];
  for (int half = 0; half < 2; ++half)
    FV_CUDA(ctx, cudaMemcpy2DAsync(dst + half * Mk, 2 * Mk * 2, Qt, static_cast<size_t>(M) * 2, static_cast<size_t>(M) * 2, r,
                                   cudaMemcpyDeviceToDevice, ctx->st), "projection copy");
  if (!tmap_2d(&ctx->qt_map[slot], dst, Mk + M, r, 2 * Mk, 128)) return fail(ctx, FVAR_ECUDA, "projection tensor map");
  ctx->qt_r[slot] = r;
  return FVAR_OK;
}

fvar_status fvar_generate_projection(fvar_ctx *ctx, int scale_idx, int group, int r, unsigned long long seed) {
  if (!ctx) return FVAR_EINVAL;
  if (scale_idx < 0 || scale_idx >= ctx->cfg.n_scales || group < 0 || group >= ctx->G)
    return fail(ctx, FVAR_EINVAL, "generate_projection: bad scale / group");
  const int M = ctx->Mk[scale_idx];
  if (r <= 0 || r > M) return fail(ctx, FVAR_EINVAL, "generate_projection: need 0 < r <= M");
  const size_t Mk = align_up(M, 64), slot = static_cast<size_t>(scale_idx) * ctx->G + group;
  bf16 *dst = ctx->qt_pool + ctx->qt_off[slot];
  // the padding columns [M, Mk) of both halves stay zero from fvar_init (nothing ever writes them)
  FV_CUDA(ctx, launch_generate_projection(dst, M, static_cast<int>(Mk), r, seed, group, scale_idx, ctx->st), "generate_projection");
  ctx->launched();
  if (!tmap_2d(&ctx->qt_map[slot], dst, Mk + M, r, 2 * Mk, 128)) return fail(ctx, FVAR_ECUDA, "projection tensor map");
  ctx->qt_r[slot] = r;
  return FVAR_OK;
}

fvar_status fvar_get_projection(fvar_ctx *ctx, int scale_idx, int group, void *Qt_out, int *r_host) {
  if (!ctx) return FVAR_EINVAL;
  if (scale_idx < 0 || scale_idx >= ctx->cfg.n_scales || group < 0 || group >= ctx->G || !Qt_out || !r_host)
    return fail(ctx, FVAR_EINVAL, "get_projection: bad arguments");
  const size_t slot = static_cast<size_t>(scale_idx) * ctx->G + group;
  const int r = ctx->qt_r[slot], M = ctx->Mk[scale_idx];
  if (r <= 0) return fail(ctx, FVAR_ESTATE, "get_projection: no projection stored for this scale and group");
  const size_t Mk = align_up(M, 64);
  FV_CUDA(ctx, cudaMemcpy2DAsync(Qt_out, static_cast<size_t>(M) * 2, ctx->qt_pool + ctx->qt_off[slot], 2 * Mk * 2,
                                 static_cast<size_t>(M) * 2, r, cudaMemcpyDeviceToDevice, ctx->st), "projection copy");
  *r_host = r;
  return FVAR_OK;
}

fvar_status fvar_set_codebook(fvar_ctx *ctx, const void *Z, int V) {
  if (!ctx) return FVAR_EINVAL;
  if (!Z || V <= 0) return fail(ctx, FVAR_EINVAL, "set_codebook: NULL codebook or V <= 0");
  if (V > kMaxCodebook) return fail(ctx, FVAR_EUNSUPPORTED, "set_codebook: more than 65536 codewords");
  if (reinterpret_cast<uintptr_t>(Z) & 15) return fail(ctx, FVAR_EINVAL, "set_codebook: codebook must be 16-byte aligned");
  FV_CUDA(ctx, launch_half_norms(static_cast<const bf16 *>(Z), V, ctx->C, ctx->tr_hn, ctx->st), "half_norms");
  ctx->launched();
  ctx->codebook = static_cast<const bf16 *>(Z);
  ctx->codebook_V = V;
  ctx->tr_scale = -1;
  return FVAR_OK;
}

static fvar_status transition_impl(fvar_ctx *ctx, const void *fo, int scale_idx, int B, int *codes, void *next_tokens, bool dup) {
  if (!ctx) return FVAR_EINVAL;
  if (!ctx->codebook) return fail(ctx, FVAR_ESTATE, "scale_transition before set_codebook");
  const int nS = ctx->cfg.n_scales;
  if (!fo || scale_idx < 0 || scale_idx >= nS || B <= 0 || B > ctx->Bmax)
    return fail(ctx, FVAR_EINVAL, "scale_transition: bad arguments");
  if (scale_idx == nS - 1 && next_tokens != nullptr)
    return fail(ctx, FVAR_EINVAL, "scale_transition: there is no next input after the last scale (next_tokens must be NULL)");
  if (scale_idx > 0 && (ctx->tr_scale != scale_idx - 1 || ctx->tr_B != B))
    return fail(ctx, FVAR_ESTATE, "scale_transition: scales must be accumulated in order, 0 first, with one batch size");
  const int C = ctx->C, V = ctx->codebook_V, M = ctx->Mk[scale_idx], R = B * M;
  const int hk = ctx->hw[2 * scale_idx], wk = ctx->hw[2 * scale_idx + 1];
  const int hK = ctx->hw[2 * (nS - 1)], wK = ctx->hw[2 * (nS - 1) + 1];
  cudaStream_t st = ctx->st;

  // R_k = Q(F_k^o): scores F_k^o Z^T - |Z|^2 / 2 on the tensor cores, arg-max in the epilogue
  const GemmPlan plan = gemm_plan(R, 1, V, C, ctx->num_sms, ctx->max_clusters, 1, 0);
  CUtensorMap ta, tw;
  if (!tmap_2d(&ta, fo, C, R, C, 128) || !tmap_2d(&tw, ctx->codebook, C, V, C, plan.pair ? plan.block_n / 2 : plan.block_n))
    return fail(ctx, FVAR_EINVAL, "scale_transition: fo must be 16-byte aligned");
  FV_CUDA(ctx, cudaMemsetAsync(ctx->tr_best, 0, static_cast<size_t>(R) * 8, st), "arg-max words clear");
  GemmArgs g = gemm_args(R, V, C);
  g.col_sub = ctx->tr_hn;
  g.best = ctx->tr_best;
  g.status = ctx->status;
  ctx->prof_begin(FVAR_KCLASS_GEMM, 2.0 * R * V * C, 2.0 * (static_cast<double>(V) * C + static_cast<double>(R) * C) + 8.0 * R);
  if (plan.pair)
    FV_CUDA(ctx, launch_gemm_pair(EPI_ARGMAX, plan.block_n, ta, tw, g, st), "codeword search");
  else
    FV_CUDA(ctx, launch_gemm(EPI_ARGMAX, plan.block_n, ta, tw, g, ctx->num_sms, st), "codeword search");
  ctx->launched();
  ctx->prof_begin(FVAR_KCLASS_CONVERT, 0.0, 12.0 * R);
  FV_CUDA(ctx, launch_unpack_codes(ctx->tr_best, R, V, ctx->tr_codes, ctx->status, st), "unpack codes");
  ctx->launched();
  if (codes) FV_CUDA(ctx, cudaMemcpyAsync(codes, ctx->tr_codes, static_cast<size_t>(R) * 4, cudaMemcpyDeviceToDevice, st), "codes copy");

  // F_k = F_{k-1} + Up(R_k, (h_K, w_K))
  ctx->prof_begin(FVAR_KCLASS_RTR_FILL, 0.0, (scale_idx == 0 ? 4.0 : 8.0) * B * hK * wK * C + 2.0 * R * C);
  FV_CUDA(ctx, launch_up_accumulate(ctx->codebook, ctx->tr_codes, B, hk, wk, hK, wK, C, scale_idx == 0, ctx->tr_F, st), "up_accumulate");
  ctx->launched();
  // next input = Down(F_k, (h_{k+1}, w_{k+1}))
  if (next_tokens) {
    const int hn = ctx->hw[2 * (scale_idx + 1)], wn = ctx->hw[2 * (scale_idx + 1) + 1];
    ctx->prof_begin(FVAR_KCLASS_CONVERT, 0.0, 4.0 * B * hK * wK * C + 2.0 * B * hn * wn * C);
    FV_CUDA(ctx, launch_down_area(ctx->tr_F, B, hK, wK, hn, wn, C, static_cast<bf16 *>(next_tokens), dup, st), "down_area");
    ctx->launched();
  }
  ctx->tr_scale = scale_idx;
  ctx->tr_B = B;
  return FVAR_OK;
}

fvar_status fvar_scale_transition(fvar_ctx *ctx, const void *fo, int scale_idx, int B, int *codes, void *next_tokens) {
  return transition_impl(ctx, fo, scale_idx, B, codes, next_tokens, false);
}

fvar_status fvar_scale_transition_pairs(fvar_ctx *ctx, const void *fo, int scale_idx, int B, int *codes, void *next_tokens_pairs) {
  return transition_impl(ctx, fo, scale_idx, B, codes, next_tokens_pairs, true);
}

fvar_status fvar_get_feature(fvar_ctx *ctx, float *F_out) {
  if (!ctx) return FVAR_EINVAL;
  if (!F_out) return fail(ctx, FVAR_EINVAL, "get_feature: NULL output");
  if (ctx->tr_scale < 0) return fail(ctx, FVAR_ESTATE, "get_feature: no scale accumulated yet");
  const int nS = ctx->cfg.n_scales;
  const size_t n = static_cast<size_t>(ctx->tr_B) * ctx->hw[2 * (nS - 1)] * ctx->hw[2 * (nS - 1) + 1] * ctx->C;
  FV_CUDA(ctx, cudaMemcpyAsync(F_out, ctx->tr_F, n * 4, cudaMemcpyDeviceToDevice, ctx->st), "feature copy");
  return FVAR_OK;
}

fvar_status fvar_load_kv(fvar_ctx *ctx, const void *K, const void *V, int L) {
  if (!ctx) return FVAR_EINVAL;
  if (ctx->B <= 0) return fail(ctx, FVAR_ESTATE, "load_kv before set_cond");
  if (!K || !V || L < 0 || L > ctx->L_cap) return fail(ctx, FVAR_EINVAL, "load_kv: bad arguments");
  const size_t per_blk = static_cast<size_t>(ctx->B) * L * ctx->C;
  for (int blk = 0; blk < ctx->cfg.n_blocks; ++blk) {
    FV_CUDA(ctx, launch_load_kv(static_cast<const bf16 *>(K) + blk * per_blk, static_cast<const bf16 *>(V) + blk * per_blk,
                                ctx->B, L, ctx->H, ctx->D, ctx->L_cap, ctx->kc + blk * ctx->kv_block_elems(),
                                ctx->vt + blk * ctx->kv_block_elems(), ctx->st), "load_kv");
    ctx->launched();
    ctx->len[blk] = L;
  }
  ctx->staged_scale = -1;
  ctx->loaded_len = L;
  return FVAR_OK;
}

fvar_status fvar_load_group_cache(fvar_ctx *ctx, int scale_idx, const float *cache) {
  if (!ctx) return FVAR_EINVAL;
  if (ctx->B <= 0) return fail(ctx, FVAR_ESTATE, "load_group_cache before set_cond");
  if (scale_idx < 0 || scale_idx >= ctx->cfg.n_scales || !cache) return fail(ctx, FVAR_EINVAL, "load_group_cache: bad arguments");
  const int M = ctx->Mk[scale_idx];
  const size_t per = static_cast<size_t>(ctx->B) * M * ctx->C;
  for (int g = 0; g < ctx->G; ++g)
    FV_CUDA(ctx, cudaMemcpyAsync(ctx->gslot(2, g), cache + g * per, per * 4, cudaMemcpyDeviceToDevice, ctx->st), "group cache copy");
  ctx->cache_scale = scale_idx;
  ctx->cache_slot = 2;
  ctx->last_scale = scale_idx;
  ctx->loaded_cache_scale = scale_idx;
  return FVAR_OK;
}

// tokens_compact: `tokens` holds only the E elements the step computes, [E][M][C] (the host entry points upload
// nothing else); otherwise all B elements, [B][M][C].
static fvar_status scale_step_impl(fvar_ctx *ctx, const void *tokens, bool tokens_compact, int scale_idx,
                                   const fvar_keep_policy *pol, void *out) {
  if (!ctx) return FVAR_EINVAL;
  if (!pol) return fail(ctx, FVAR_EINVAL, "scale_step: policy is NULL");
  if (pol->mode == FVAR_SKIP) return FVAR_OK;
  if (pol->mode != FVAR_DENSE && pol->mode != FVAR_LOWRANK_RTR) return fail(ctx, FVAR_EINVAL, "scale_step: bad mode");
  if (pol->cfg_mode != FVAR_CFG_PAIR && pol->cfg_mode != FVAR_CFG_NULL_ONLY) return fail(ctx, FVAR_EINVAL, "scale_step: bad cfg_mode");
  if (!tokens || !out) return fail(ctx, FVAR_EINVAL, "scale_step: NULL tokens / out");
  if (ctx->B <= 0) return fail(ctx, FVAR_ESTATE, "scale_step before set_cond");
  if (scale_idx < 0 || scale_idx >= ctx->cfg.n_scales) return fail(ctx, FVAR_EINVAL, "scale_step: bad scale_idx");
  if (scale_idx < ctx->last_scale) return fail(ctx, FVAR_ESTATE, "scale_step: scale_idx decreased");
  if (pol->select != FVAR_SELECT_TOPR && pol->select != FVAR_SELECT_SAMPLE) return fail(ctx, FVAR_EINVAL, "scale_step: bad select");
  const bool sampled = pol->select == FVAR_SELECT_SAMPLE;
  if (sampled && !pol->sample_noise) return fail(ctx, FVAR_EINVAL, "scale_step: sampled selection needs sample_noise");
  if (pol->restore != FVAR_RESTORE_RTR && pol->restore != FVAR_RESTORE_LLS) return fail(ctx, FVAR_EINVAL, "scale_step: bad restore");
  const bool lls = pol->mode == FVAR_LOWRANK_RTR && pol->restore == FVAR_RESTORE_LLS;
  const bool null_only = pol->cfg_mode == FVAR_CFG_NULL_ONLY;
  if (null_only && (ctx->B % 2)) return fail(ctx, FVAR_EINVAL, "scale_step: null-only needs an even batch");
  if (!null_only && ctx->null_only_seen) return fail(ctx, FVAR_ESTATE, "scale_step: pair step after a null-only step");

  const int C = ctx->C, F = ctx->F, H = ctx->H, D = ctx->D, G = ctx->G, bpg = ctx->cfg.blocks_per_group;
  const int M = ctx->Mk[scale_idx], B = ctx->B;
  const int E = null_only ? B / 2 : B, bmul = null_only ? 2 : 1, boff = null_only ? 1 : 0;
  std::vector<int> rank(G, M);
  if (pol->mode == FVAR_LOWRANK_RTR) {
    for (int g = 0; g < G; ++g) {
      const int r = pol->rank_per_group ? pol->rank_per_group[g] : fvar_rank_from_keep_ratio(M, pol->keep_ratio);
      if (r < 1 || r > M) return fail(ctx, FVAR_EINVAL, "scale_step: need 1 <= r <= M");
      rank[g] = r;
    }
  }
  int r_max = 0;
  bool any_late = false;
  for (int g = 0; g < G; ++g) {
    if (rank[g] < M) {
      any_late = true;
      r_max = rank[g] > r_max ? rank[g] : r_max;
      if (ctx->qt_r[static_cast<size_t>(scale_idx) * G + g] != rank[g])
        return fail(ctx, FVAR_ESTATE, "scale_step: no projection of this rank set for a group");
      if (lls && rank[g] > ctx->lls_rank_cap) return fail(ctx, FVAR_EUNSUPPORTED, "scale_step: LLS restoration takes ranks up to 192");
      if (lls && ctx->cache_scale >= 0 && rank[g] > ctx->Mk[ctx->cache_scale])
        return fail(ctx, FVAR_EINVAL, "scale_step: LLS restoration needs r <= the tokens of the cached scale (the upsampled cache has no higher rank)");
    }
    for (int blk = g * bpg; blk < (g + 1) * bpg; ++blk)
      if (ctx->len[blk] + rank[g] > ctx->L_cap) return fail(ctx, FVAR_ESTATE, "scale_step: KV cache is full");
  }
  if (any_late && (ctx->cache_scale < 0 || ctx->cache_scale > scale_idx))
    return fail(ctx, FVAR_ESTATE, "scale_step: low-rank step without the previous scale's group outputs");

  const int prev_slot = ctx->cache_slot, cur_slot = (ctx->cache_scale < 0 || ctx->cache_slot == 2) ? 0 : (ctx->cache_slot ^ 1);
  const int h0 = ctx->cache_scale >= 0 ? ctx->hw[2 * ctx->cache_scale] : 0;
  const int w0 = ctx->cache_scale >= 0 ? ctx->hw[2 * ctx->cache_scale + 1] : 0;
  const int h1 = ctx->hw[2 * scale_idx], w1 = ctx->hw[2 * scale_idx + 1];
  const float scale_log2 = 1.4426950408889634f / sqrtf(static_cast<float>(D));
  const size_t ada_blk = static_cast<size_t>(ctx->Bmax) * 6 * C;
  cudaStream_t st = ctx->st;

  ctx->prof_begin(FVAR_KCLASS_CONVERT, 0.0, 6.0 * E * M * C);
  const int Mk = static_cast<int>(align_up(M, 64));
  // the projection of a late group reads its input rows as a hi / lo bf16 split, written by whoever produces them
  FV_CUDA(ctx, launch_tokens_to_f32(static_cast<const bf16 *>(tokens), ctx->x0, E, M, C, rank[0] < M ? ctx->xsplit[0] : nullptr, Mk,
                                    tokens_compact ? 1 : bmul, tokens_compact ? 0 : boff, bmul, boff, st), "tokens_to_f32");
  ctx->launched();
  const float *X_in = ctx->x0;
  const RowMap bmap{bmul, boff, M};              // buffers indexed by the caller's batch element
  fvar_status s;

  // Everything between the input and output conversions touches workspace memory only, so for a
  // given (scale, ranks, cache lengths, slots) it is the same chain of launches every time: it is
  // captured into a CUDA graph on first use and replayed afterwards.
  auto body = [&]() -> fvar_status {
  for (int g = 0; g < G; ++g) {
    const int r = rank[g];
    const bool late = r < M;
    const int R = E * r;
    float *gout = ctx->gslot(cur_slot, g);
    int *idx_g = ctx->idx + static_cast<size_t>(g) * ctx->Bmax * ctx->Mmax;
    int *inv_g = ctx->inv + static_cast<size_t>(g) * ctx->Bmax * ctx->Mmax;
    const RowMap smap{1, 0, r};                  // the compact work stream of this group
    // the next group's projection, if it has one, reads this group's output as a hi / lo bf16 split
    bf16 *next_split = (g + 1 < G && rank[g + 1] < M) ? ctx->xsplit[(g + 1) & 1] : nullptr;

    // While a graph is being captured, the index selection and the restoration fill of a late group
    // go to a second stream: they depend only on the group's input and on the previous scale's
    // cache, so they run beside the projection and the blocks and join before the scatter.
    const bool forked = late && st == ctx->cap_st;
    if (late) {
      cudaStream_t side = st;
      if (forked) {
        FV_CUDA(ctx, cudaEventRecord(ctx->ev_fork, st), "fork record");
        FV_CUDA(ctx, cudaStreamWaitEvent(ctx->cap_st2, ctx->ev_fork, 0), "fork wait");
        side = ctx->cap_st2;
      }
      if (lls) {
        // LLS restoration: no index set; the whole upsampled cache (Eq. "upcache") and its bf16 split, for its own
        // projection and restoration matrix
        ctx->prof_begin(FVAR_KCLASS_RTR_FILL, 0.0, 4.0 * E * C * (static_cast<double>(M) + h0 * w0) + 4.0 * E * M * C, side);
        FV_CUDA(ctx, launch_rtr_fill(ctx->gslot(prev_slot, g), ctx->cup, E, bmul, boff, h0, w0, h1, w1, C, nullptr, ctx->csplit, Mk, side), "cache upsample");
        ctx->launched(side);
      } else if (pol->forced_indices) {
        ctx->prof_begin(FVAR_KCLASS_CONVERT, 0.0, 4.0 * E * (M + 2.0 * r), side);
        FV_CUDA(ctx, launch_copy_indices(pol->forced_indices + static_cast<size_t>(g) * E * r_max, E, M, r, r_max, idx_g,
                                         inv_g, ctx->status, side), "copy_indices");
        ctx->launched(side);
      } else {
        ctx->prof_begin(FVAR_KCLASS_SCORE, 2.0 * E * M * C, 4.0 * E * M * C + 4.0 * E * M, side);
        FV_CUDA(ctx, launch_row_scores(X_in, bmap, E, M, C,
                                       sampled ? pol->sample_noise + static_cast<size_t>(g) * E * M : nullptr, ctx->scores, side), "row_scores");
        ctx->launched(side);
        ctx->prof_begin(FVAR_KCLASS_SELECT, 0.0, 4.0 * E * (2.0 * M + r), side);
        FV_CUDA(ctx, launch_select_topr(ctx->scores, E, M, r, idx_g, inv_g, side), "select_topr");
        ctx->launched(side);
      }
      if (!lls) {
        // restoration fill: rows outside the index set, from the upsampled cache of the previous scale
        ctx->prof_begin(FVAR_KCLASS_RTR_FILL, 0.0, 4.0 * E * C * (static_cast<double>(M - r) + h0 * w0) + 4.0 * E * M, side);
        FV_CUDA(ctx, launch_rtr_fill(ctx->gslot(prev_slot, g), gout, E, bmul, boff, h0, w0, h1, w1, C, inv_g, next_split, Mk, side), "rtr_fill");
        ctx->launched(side);
      }
      if (forked) FV_CUDA(ctx, cudaEventRecord(ctx->ev_join, side), "join record");
      // random projection: xs[e] = Qt * X[e]  (r x M times M x C), batched over e.  The reduction runs over the hi
      // and lo bf16 parts of X ([Qt | Qt] against [hi ; lo]); X's rows are read in place as an MN-major operand.
      GemmArgs ga = gemm_args(r, C, Mk + M);
      ga.nbatch = E;
      ga.a_batch_rows = 0;
      ga.b_batch_rows = 2 * Mk;
      ga.w_mn_major = 1;
      ga.out_f32 = lls ? ctx->lls_xhat : ctx->xs;   // LLS keeps the projection: the blocks work on a copy of their own
      ga.ld_out = C;
      ga.status = ctx->status;
      ga.wait_cycles = ctx->wait_cycles;
      // few row tiles over a long reduction (2 M rows of [hi ; lo]): the deterministic split-K of the row-tiled kernel
      // puts more CTAs on it
      int bn = 64, sp = 1;
      gemm_pick_tile((r + 127) / 128 * E, C, Mk + M, ctx->num_sms, 4, kSplitScratchBytes, &bn, &sp);
      ga.splits = sp;
      ga.partial = ctx->split_partial;
      ga.counters = ctx->split_counters;
      ctx->prof_begin(FVAR_KCLASS_GEMM, 2.0 * r * C * M * E, 2.0 * (static_cast<double>(r) * M + 2.0 * E * M * C) + 4.0 * E * r * C);
      FV_CUDA(ctx, launch_gemm(EPI_F32, bn, ctx->qt_map[static_cast<size_t>(scale_idx) * G + g],
                               ctx->xsplit_map[scale_idx * 2 + (g & 1)], ga, ctx->num_sms, st), "projection gemm");
      ctx->launched();
    }

    for (int t = 0; t < bpg; ++t) {
      const int blk = g * bpg + t;
      const bool first_dense = (t == 0) && !late, last = (t == bpg - 1);
      const float *in_ptr = first_dense ? X_in : ((lls && late && t == 0) ? ctx->lls_xhat : ctx->xs);
      const RowMap in_map = first_dense ? bmap : smap;
      const float *ada = ctx->ada + blk * ada_blk;
      const int L_prev = ctx->len[blk];
      // the weights each GEMM's successor will stream (gemm_skinny.cu asks L2 for them ahead of time)
      const size_t w_bytes[W_COUNT] = {6ull * C * C, 2ull * C * C, 2ull * F * C, 2ull * C * F, 0, 2ull * C * C, 0, 2ull * C * C};
      auto prefetch_next = [&](GemmArgs &ga, int next_blk, int next_wid) {
        if (next_blk < ctx->cfg.n_blocks) { ga.pf_ptr = ctx->w[next_wid][next_blk]; ga.pf_bytes = w_bytes[next_wid]; }
      };

      ctx->prof_begin(FVAR_KCLASS_LN, 0.0, 6.0 * R * C);
      FV_CUDA(ctx, launch_ln_modulate(in_ptr, in_map, E, r, C, ada, ada + C, 6 * C, bmul, boff, nullptr,
                                      ctx->cfg.ln_eps, ctx->y, st), "ln_modulate 1");
      ctx->launched();
      {
        GemmArgs ga = gemm_args(R, 3 * C, C);
        ga.bias = ctx->b_qkv[blk];
        ga.rows_per_batch = r; ga.bmul = bmul; ga.boff = boff;
        ga.out_bf16 = ctx->q; ga.ld_out = C;
        ga.kc = ctx->kc + blk * ctx->kv_block_elems();
        ga.vt = ctx->vt + blk * ctx->kv_block_elems();
        ga.C = C; ga.H = H; ga.D = D; ga.L_cap = ctx->L_cap; ga.L_prev = L_prev; ga.col_base = 0;
        prefetch_next(ga, blk, W_O);
        if ((s = run_gemm(ctx, EPI_QKV, ctx->y_map, blk, W_QKV, ga, "qkv gemm")) != FVAR_OK) return s;
      }
      {
        AttnArgs aa{E, H, r, D, L_prev + r, ctx->L_cap, bmul, boff, ctx->a, scale_log2, ctx->status, 1};
        aa.wait_cycles = ctx->wait_cycles;
        attention_plan(E, H, r, L_prev + r, ctx->num_sms, &aa.tiles_per_cta, &aa.kv_splits);
        ctx->prof_begin(FVAR_KCLASS_ATTENTION, 4.0 * E * r * (L_prev + r) * C, 4.0 * E * (L_prev + r) * C + 4.0 * E * r * C);
        FV_CUDA(ctx, launch_attention(ctx->q_map, ctx->kmap[blk], ctx->vmap[blk], aa, st), "attention");
        ctx->launched();
      }
      {
        GemmArgs ga = gemm_args(R, C, C);
        ga.bias = ctx->b_o[blk];
        ga.rows_per_batch = r; ga.bmul = bmul; ga.boff = boff;
        ga.resid = in_ptr; ga.rmap = in_map;
        ga.out_f32 = ctx->xs; ga.omap = smap; ga.ld_out = C;
        ga.gate = ada + 2 * C; ga.gate_stride = 6 * C;
        prefetch_next(ga, blk, ctx->cfg.has_cross_attn ? W_CQ : W_FC1);
        if ((s = run_gemm(ctx, EPI_RESID, ctx->a_map, blk, W_O, ga, "out-proj gemm")) != FVAR_OK) return s;
      }
      if (ctx->cfg.has_cross_attn) {
        ctx->prof_begin(FVAR_KCLASS_LN, 0.0, 6.0 * R * C);
        FV_CUDA(ctx, launch_ln_modulate(ctx->xs, smap, E, r, C, nullptr, nullptr, 0, bmul, boff, ctx->ln_c_gamma[blk],
                                        ctx->cfg.ln_eps, ctx->y, st), "ln cross");
        ctx->launched();
        GemmArgs gq = gemm_args(R, C, C);
        gq.out_bf16 = ctx->q; gq.ld_out = C;
        prefetch_next(gq, blk, W_CO);
        if ((s = run_gemm(ctx, EPI_BF16, ctx->y_map, blk, W_CQ, gq, "cross q gemm")) != FVAR_OK) return s;
        AttnArgs aa{E, H, r, D, ctx->cfg.ctx_len, ctx->ctx_cap, bmul, boff, ctx->a, scale_log2, ctx->status, 1};
        aa.wait_cycles = ctx->wait_cycles;
        attention_plan(E, H, r, ctx->cfg.ctx_len, ctx->num_sms, &aa.tiles_per_cta, &aa.kv_splits);
        ctx->prof_begin(FVAR_KCLASS_ATTENTION, 4.0 * E * r * ctx->cfg.ctx_len * C, 4.0 * E * ctx->cfg.ctx_len * C + 4.0 * E * r * C);
        FV_CUDA(ctx, launch_attention(ctx->q_map, ctx->ckmap[blk], ctx->cvmap[blk], aa, st), "cross attention");
        ctx->launched();
        GemmArgs go = gemm_args(R, C, C);
        go.rows_per_batch = r; go.bmul = bmul; go.boff = boff;
        go.resid = ctx->xs; go.rmap = smap; go.out_f32 = ctx->xs; go.omap = smap; go.ld_out = C;
        prefetch_next(go, blk, W_FC1);
        if ((s = run_gemm(ctx, EPI_RESID, ctx->a_map, blk, W_CO, go, "cross out gemm")) != FVAR_OK) return s;
      }
      ctx->prof_begin(FVAR_KCLASS_LN, 0.0, 6.0 * R * C);
      FV_CUDA(ctx, launch_ln_modulate(ctx->xs, smap, E, r, C, ada + 3 * C, ada + 4 * C, 6 * C, bmul, boff, nullptr,
                                      ctx->cfg.ln_eps, ctx->y, st), "ln_modulate 2");
      ctx->launched();
      {
        GemmArgs ga = gemm_args(R, F, C);
        ga.bias = ctx->b_fc1[blk];
        ga.out_bf16 = ctx->hbuf; ga.ld_out = F;
        prefetch_next(ga, blk, W_FC2);
        if ((s = run_gemm(ctx, EPI_GELU_BF16, ctx->y_map, blk, W_FC1, ga, "fc1 gemm")) != FVAR_OK) return s;
      }
      {
        GemmArgs ga = gemm_args(R, C, F);
        ga.bias = ctx->b_fc2[blk];
        ga.rows_per_batch = r; ga.bmul = bmul; ga.boff = boff;
        ga.resid = ctx->xs; ga.rmap = smap; ga.ld_out = C;
        ga.gate = ada + 5 * C; ga.gate_stride = 6 * C;
        if (last && !(lls && late)) {
          if (forked) FV_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_join, 0), "join wait");
          ga.out_f32 = gout; ga.omap = bmap;
          ga.scatter = late ? idx_g : nullptr;
          ga.xsplit = next_split; ga.xsplit_mk = Mk;
        } else {
          ga.out_f32 = ctx->xs; ga.omap = smap;
        }
        prefetch_next(ga, blk + 1, W_QKV);
        if ((s = run_gemm(ctx, EPI_RESID, ctx->h_map, blk, W_FC2, ga, "fc2 gemm")) != FVAR_OK) return s;
      }
      ctx->staged[blk] = r;
    }
    if (lls && late) {
      // F_k^o = (W_hat + W^{o,cache}) F_r^o (Eq. "lstsq", App. A.3) as P1 (G1^-1 F_r^o) + P2 (G2^-1 F_r^o) with
      // G1 = F_hat F_hat^T, P1 = F F_hat^T for the group's input F and its projection F_hat, and G2, P2 the same for
      // the upsampled cached output and its projection.  fp32 throughout.
      if (forked) FV_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_join, 0), "join wait");
      {
        GemmArgs ga = gemm_args(r, C, Mk + M);               // projection of the upsampled cache by the same Q
        ga.nbatch = E; ga.b_batch_rows = 2 * Mk; ga.w_mn_major = 1;
        ga.out_f32 = ctx->lls_chat; ga.ld_out = C;
        ga.status = ctx->status; ga.wait_cycles = ctx->wait_cycles;
        const int bn = gemm_pick_block_n((r + 127) / 128 * E, C, Mk + M, ctx->num_sms);
        ctx->prof_begin(FVAR_KCLASS_GEMM, 2.0 * r * C * M * E, 2.0 * (static_cast<double>(r) * M + 2.0 * E * M * C) + 4.0 * E * r * C);
        FV_CUDA(ctx, launch_gemm(EPI_F32, bn, ctx->qt_map[static_cast<size_t>(scale_idx) * G + g], ctx->csplit_map[scale_idx], ga,
                                 ctx->num_sms, st), "cache projection gemm");
        ctx->launched();
      }
      const long long rc = static_cast<long long>(r) * C, rr = static_cast<long long>(r) * r, mc = static_cast<long long>(M) * C,
                      mr = static_cast<long long>(M) * r;
      auto sg = [&](bool tb, const float *A, const float *Bm, float *O, int m, int n, int k, long long lda, long long ldb, long long ldo,
                    long long ao, long long as, long long bo, long long bs, long long oo, long long os, bool acc, const char *what) -> fvar_status {
        // few output tiles over a long reduction (the Gram matrices, F F_hat^T): cut K so that about all SMs work; the
        // partial products go through the split-K scratch area and are added in a fixed order
        const long long tiles = static_cast<long long>((m + 127) / 128) * ((n + 63) / 64) * E;
        int ks = 1;
        if (!acc && k >= 256 && tiles * 2 <= ctx->num_sms) {
          ks = static_cast<int>(ctx->num_sms / tiles);
          if (ks > k / 64) ks = k / 64;
          while (ks > 1 && static_cast<size_t>(ks) * E * m * n * 4 > kSplitScratchBytes) --ks;
        }
        ctx->prof_begin(FVAR_KCLASS_GEMM, 2.0 * m * n * k * E, 4.0 * E * (static_cast<double>(m) * k + static_cast<double>(n) * k + static_cast<double>(m) * n));
        FV_CUDA(ctx, launch_sgemm(tb, A, Bm, O, m, n, k, lda, ldb, ldo, ao, as, bo, bs, oo, os, E, acc, st, ks, ctx->split_partial), what);
        ctx->launched();
        if (ks > 1) ctx->launched();
        return FVAR_OK;
      };
      float *G1 = ctx->lls_G, *G2 = ctx->lls_G + E * rr, *I1 = ctx->lls_Ginv, *I2 = ctx->lls_Ginv + E * rr;
      float *T1 = ctx->lls_T, *T2 = ctx->lls_T + E * rc, *P1 = ctx->lls_P, *P2 = ctx->lls_P + E * mr;
      if ((s = sg(true, ctx->lls_xhat, ctx->lls_xhat, G1, r, r, C, C, C, r, 0, rc, 0, rc, 0, rr, false, "gram 1")) != FVAR_OK) return s;
      if ((s = sg(true, ctx->lls_chat, ctx->lls_chat, G2, r, r, C, C, C, r, 0, rc, 0, rc, 0, rr, false, "gram 2")) != FVAR_OK) return s;
      ctx->prof_begin(FVAR_KCLASS_CONVERT, 2.0 * E * rr * r, 16.0 * E * rr);
      FV_CUDA(ctx, launch_chol_inverse(ctx->lls_G, ctx->lls_Ginv, r, 2 * E, ctx->status, st), "gram inverse");
      ctx->launched();
      if ((s = sg(false, I1, ctx->xs, T1, r, C, r, r, C, C, 0, rr, 0, rc, 0, rc, false, "T1")) != FVAR_OK) return s;
      if ((s = sg(false, I2, ctx->xs, T2, r, C, r, r, C, C, 0, rr, 0, rc, 0, rc, false, "T2")) != FVAR_OK) return s;
      if ((s = sg(true, X_in, ctx->lls_xhat, P1, M, r, C, C, C, r, boff * mc, bmul * mc, 0, rc, 0, mr, false, "P1")) != FVAR_OK) return s;
      if ((s = sg(true, ctx->cup, ctx->lls_chat, P2, M, r, C, C, C, r, boff * mc, bmul * mc, 0, rc, 0, mr, false, "P2")) != FVAR_OK) return s;
      if ((s = sg(false, P1, T1, gout, M, C, r, r, C, C, 0, mr, 0, rc, boff * mc, bmul * mc, false, "restore 1")) != FVAR_OK) return s;
      if ((s = sg(false, P2, T2, gout, M, C, r, r, C, C, 0, mr, 0, rc, boff * mc, bmul * mc, true, "restore 2")) != FVAR_OK) return s;
      if (next_split) {
        ctx->prof_begin(FVAR_KCLASS_CONVERT, 0.0, 8.0 * E * mc);
        FV_CUDA(ctx, launch_split_rows(gout, boff * mc, bmul * mc, E, M, C, next_split, Mk, st), "split rows");
        ctx->launched();
      }
    }
    X_in = gout;
    ctx->last_rank[g] = r;
  }
  return FVAR_OK;
  };

  if (ctx->use_graphs && ctx->prof_on && !pol->forced_indices) {
    // Profile pass: the same capture, instantiated afresh for this step so that every launch has event nodes of
    // its own; the executable graph lives until the profile is switched off or read out.
    const long long l0 = ctx->launches;
    FV_CUDA(ctx, cudaStreamBeginCapture(ctx->cap_st, cudaStreamCaptureModeThreadLocal), "begin capture");
    st = ctx->launch_st = ctx->cap_st;
    s = body();
    st = ctx->launch_st = ctx->st;
    cudaGraph_t graph = nullptr;
    cudaError_t ce = cudaStreamEndCapture(ctx->cap_st, &graph);
    if (s != FVAR_OK) {
      if (graph) cudaGraphDestroy(graph);
      return s;
    }
    if (ce != cudaSuccess) return cuda_fail(ctx, ce, "end capture");
    (void)l0;
    cudaGraphExec_t exec = nullptr;
    ce = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    if (ce != cudaSuccess) return cuda_fail(ctx, ce, "graph instantiate");
    ctx->prof_execs.push_back(exec);
    FV_CUDA(ctx, cudaGraphLaunch(exec, st), "graph launch");
  } else if (ctx->use_graphs && !ctx->prof_on && !pol->forced_indices) {
    std::string key;
    auto put = [&](long long v) { key.append(reinterpret_cast<const char *>(&v), sizeof(v)); };
    put(scale_idx); put(B); put(E); put(prev_slot); put(cur_slot); put(ctx->cache_scale); put(lls ? 1 : 0);
    put(sampled ? static_cast<long long>(reinterpret_cast<uintptr_t>(pol->sample_noise)) : 0);
    for (int g = 0; g < G; ++g) put(rank[g]);
    for (int blk = 0; blk < ctx->cfg.n_blocks; ++blk) put(ctx->len[blk]);
    auto it = ctx->graphs.find(key);
    if (it == ctx->graphs.end()) {
      if (ctx->graphs.size() >= 256) ctx->drop_graphs();
      const long long l0 = ctx->launches;
      FV_CUDA(ctx, cudaStreamBeginCapture(ctx->cap_st, cudaStreamCaptureModeThreadLocal), "begin capture");
      st = ctx->launch_st = ctx->cap_st;
      s = body();
      st = ctx->launch_st = ctx->st;
      cudaGraph_t graph = nullptr;
      cudaError_t ce = cudaStreamEndCapture(ctx->cap_st, &graph);
      if (s != FVAR_OK) {
        if (graph) cudaGraphDestroy(graph);
        return s;
      }
      if (ce != cudaSuccess) return cuda_fail(ctx, ce, "end capture");
      fvar_ctx::GraphEntry ge;
      ge.kernels = ctx->launches - l0;
      ctx->launches = l0;
      ce = cudaGraphInstantiate(&ge.exec, graph, 0);
      cudaGraphDestroy(graph);
      if (ce != cudaSuccess) return cuda_fail(ctx, ce, "graph instantiate");
      it = ctx->graphs.emplace(key, ge).first;
    } else {
      // host-side bookkeeping the body would have done
      for (int g = 0; g < G; ++g) {
        ctx->last_rank[g] = rank[g];
        for (int blk = g * bpg; blk < (g + 1) * bpg; ++blk) ctx->staged[blk] = rank[g];
      }
      X_in = ctx->gslot(cur_slot, G - 1);
    }
    FV_CUDA(ctx, cudaGraphLaunch(it->second.exec, st), "graph launch");
    ctx->launches += it->second.kernels;
  } else {
    if ((s = body()) != FVAR_OK) return s;
  }
  ctx->prof_begin(FVAR_KCLASS_CONVERT, 0.0, 6.0 * E * M * C);
  FV_CUDA(ctx, launch_out_to_bf16(X_in, bmap, E, M, C, static_cast<bf16 *>(out), st), "out_to_bf16");
  ctx->launched();

  ctx->cache_scale = scale_idx;
  ctx->cache_slot = cur_slot;
  ctx->staged_scale = scale_idx;
  ctx->last_scale = scale_idx;
  ctx->last_E = E; ctx->last_M = M;
  ctx->last_lls = lls;
  if (null_only) ctx->null_only_seen = 1;
  return FVAR_OK;
}

fvar_status fvar_scale_step(fvar_ctx *ctx, const void *tokens, int scale_idx, const fvar_keep_policy *pol, void *out) {
  return scale_step_impl(ctx, tokens, false, scale_idx, pol, out);
}

// Host -> device copy of the token rows a step reads: every element, or with the null-prompt branch alone only
// elements 2p + 1, packed [E][M][C] (one strided copy).
static cudaError_t upload_tokens(fvar_ctx *ctx, bf16 *dst, const void *tokens_host, size_t per_elem_bytes, bool null_only,
                                 cudaStream_t st) {
  if (!null_only) return cudaMemcpyAsync(dst, tokens_host, per_elem_bytes * ctx->B, cudaMemcpyHostToDevice, st);
  return cudaMemcpy2DAsync(dst, per_elem_bytes, static_cast<const uint8_t *>(tokens_host) + per_elem_bytes, 2 * per_elem_bytes,
                           per_elem_bytes, static_cast<size_t>(ctx->B / 2), cudaMemcpyHostToDevice, st);
}

fvar_status fvar_scale_step_host(fvar_ctx *ctx, const void *tokens_host, int scale_idx, const fvar_keep_policy *pol,
                                 void *out_host) {
  if (!ctx) return FVAR_EINVAL;
  if (!pol) return fail(ctx, FVAR_EINVAL, "scale_step_host: policy is NULL");
  if (pol->mode == FVAR_SKIP) return FVAR_OK;
  if (!tokens_host || !out_host) return fail(ctx, FVAR_EINVAL, "scale_step_host: NULL tokens / out");
  if (scale_idx < 0 || scale_idx >= ctx->cfg.n_scales || ctx->B <= 0) return fail(ctx, FVAR_EINVAL, "scale_step_host: bad scale_idx or no cond");
  // Staging: the bf16 tokens land in the hidden-activation buffer (free until the first fc1) and
  // the bf16 output in the attention-output buffer (free after the last out-proj).
  const size_t M = ctx->Mk[scale_idx];
  const bool null_only = pol->cfg_mode == FVAR_CFG_NULL_ONLY && ctx->B % 2 == 0;
  const int E = null_only ? ctx->B / 2 : ctx->B;
  FV_CUDA(ctx, upload_tokens(ctx, ctx->hbuf, tokens_host, M * ctx->C * 2, null_only, ctx->st), "tokens H2D");
  fvar_status s = scale_step_impl(ctx, ctx->hbuf, null_only, scale_idx, pol, ctx->a);
  if (s != FVAR_OK) return s;
  FV_CUDA(ctx, cudaMemcpyAsync(out_host, ctx->a, static_cast<size_t>(E) * M * ctx->C * 2, cudaMemcpyDeviceToHost, ctx->st), "out D2H");
  FV_CUDA(ctx, cudaStreamSynchronize(ctx->st), "stream synchronize");
  return FVAR_OK;
}

fvar_status fvar_scale_step_host_async(fvar_ctx *ctx, const void *tokens_host, int scale_idx, const fvar_keep_policy *pol,
                                       void *out_host) {
  if (!ctx) return FVAR_EINVAL;
  if (!pol) return fail(ctx, FVAR_EINVAL, "scale_step_host_async: policy is NULL");
  if (pol->mode == FVAR_SKIP) return FVAR_OK;
  if (!tokens_host || !out_host) return fail(ctx, FVAR_EINVAL, "scale_step_host_async: NULL tokens / out");
  if (scale_idx < 0 || scale_idx >= ctx->cfg.n_scales || ctx->B <= 0) return fail(ctx, FVAR_EINVAL, "scale_step_host_async: bad scale_idx or no cond");
  if (!ctx->host_pipe_ok) return fail(ctx, FVAR_ECUDA, "scale_step_host_async: copy streams unavailable");
  const size_t M = ctx->Mk[scale_idx];
  const bool null_only = pol->cfg_mode == FVAR_CFG_NULL_ONLY && ctx->B % 2 == 0;
  const int E = null_only ? ctx->B / 2 : ctx->B;
  const int s = static_cast<int>(ctx->host_calls & 1);
  const bool reuse = ctx->host_calls >= 2;     // the slot was used two calls ago
  // host -> device on the upload stream, once the step that last read this slot has finished
  if (reuse) FV_CUDA(ctx, cudaStreamWaitEvent(ctx->h2d_st, ctx->ev_cmp[s], 0), "upload wait");
  FV_CUDA(ctx, upload_tokens(ctx, ctx->hin[s], tokens_host, M * ctx->C * 2, null_only, ctx->h2d_st), "tokens H2D");
  FV_CUDA(ctx, cudaEventRecord(ctx->ev_in[s], ctx->h2d_st), "upload record");
  // the step on the caller's stream, once its tokens are there and the slot's previous result has left
  FV_CUDA(ctx, cudaStreamWaitEvent(ctx->st, ctx->ev_in[s], 0), "step wait");
  if (reuse) FV_CUDA(ctx, cudaStreamWaitEvent(ctx->st, ctx->ev_out[s], 0), "step wait");
  fvar_status rc = scale_step_impl(ctx, ctx->hin[s], null_only, scale_idx, pol, ctx->hout[s]);
  if (rc != FVAR_OK) return rc;
  FV_CUDA(ctx, cudaEventRecord(ctx->ev_cmp[s], ctx->st), "step record");
  // device -> host on the download stream
  FV_CUDA(ctx, cudaStreamWaitEvent(ctx->d2h_st, ctx->ev_cmp[s], 0), "download wait");
  FV_CUDA(ctx, cudaMemcpyAsync(out_host, ctx->hout[s], static_cast<size_t>(E) * M * ctx->C * 2, cudaMemcpyDeviceToHost, ctx->d2h_st), "out D2H");
  FV_CUDA(ctx, cudaEventRecord(ctx->ev_out[s], ctx->d2h_st), "download record");
  ctx->host_calls++;
  return FVAR_OK;
}

fvar_status fvar_host_sync(fvar_ctx *ctx) {
  if (!ctx) return FVAR_EINVAL;
  if (ctx->h2d_st) FV_CUDA(ctx, cudaStreamSynchronize(ctx->h2d_st), "upload synchronize");
  FV_CUDA(ctx, cudaStreamSynchronize(ctx->st), "stream synchronize");
  if (ctx->d2h_st) FV_CUDA(ctx, cudaStreamSynchronize(ctx->d2h_st), "download synchronize");
  return FVAR_OK;
}

fvar_status fvar_kv_append(fvar_ctx *ctx, int scale_idx) {
  if (!ctx) return FVAR_EINVAL;
  if (ctx->staged_scale < 0 || ctx->staged_scale != scale_idx) return fail(ctx, FVAR_ESTATE, "kv_append: nothing staged for this scale");
  for (int blk = 0; blk < ctx->cfg.n_blocks; ++blk) {
    ctx->len[blk] += ctx->staged[blk];
    ctx->staged[blk] = 0;
  }
  ctx->staged_scale = -1;
  return FVAR_OK;
}

fvar_status fvar_get_indices(fvar_ctx *ctx, int group, int *idx_dev, int *count_host) {
  if (!ctx) return FVAR_EINVAL;
  if (group < 0 || group >= ctx->G || !idx_dev || !count_host) return fail(ctx, FVAR_EINVAL, "get_indices: bad arguments");
  if (ctx->last_scale < 0 || ctx->last_lls || ctx->last_rank[group] <= 0 || ctx->last_rank[group] >= ctx->last_M)
    return fail(ctx, FVAR_ESTATE, "get_indices: the last step did not select rows for this group");
  const int r = ctx->last_rank[group];
  FV_CUDA(ctx, cudaMemcpyAsync(idx_dev, ctx->idx + static_cast<size_t>(group) * ctx->Bmax * ctx->Mmax,
                               static_cast<size_t>(ctx->last_E) * r * 4, cudaMemcpyDeviceToDevice, ctx->st), "indices copy");
  *count_host = r;
  return FVAR_OK;
}

fvar_status fvar_get_group_output(fvar_ctx *ctx, int group, float *out_dev) {
  if (!ctx) return FVAR_EINVAL;
  if (group < 0 || group >= ctx->G || !out_dev) return fail(ctx, FVAR_EINVAL, "get_group_output: bad arguments");
  if (ctx->cache_scale < 0) return fail(ctx, FVAR_ESTATE, "get_group_output: no scale stepped yet");
  const size_t n = static_cast<size_t>(ctx->B) * ctx->Mk[ctx->cache_scale] * ctx->C;
  FV_CUDA(ctx, cudaMemcpyAsync(out_dev, ctx->gslot(ctx->cache_slot, group), n * 4, cudaMemcpyDeviceToDevice, ctx->st), "group output copy");
  return FVAR_OK;
}

// ------------------------------------------------------------------------------------------------ kernel-level
static fvar_status kfail(fvar_status s, const char *m) { g_init_error = m; return s; }
#define FK_CUDA(call, what)                                                                          \
  do {                                                                                               \
    cudaError_t e__ = (call);                                                                        \
    if (e__ != cudaSuccess) return kfail(FVAR_ECUDA, (std::string(what) + ": " + cudaGetErrorString(e__)).c_str()); \
  } while (0)

fvar_status fvar_row_scores(const float *x, int B, int M, int C, float *scores, void *stream) {
  if (!x || !scores || B <= 0 || M <= 0 || C <= 0 || C % 4) return kfail(FVAR_EINVAL, "row_scores: bad arguments");
  FK_CUDA(launch_row_scores(x, RowMap{1, 0, M}, B, M, C, nullptr, scores, static_cast<cudaStream_t>(stream)), "row_scores");
  return FVAR_OK;
}

fvar_status fvar_row_keys(const float *x, const float *noise, int B, int M, int C, float *keys, void *stream) {
  if (!x || !noise || !keys || B <= 0 || M <= 0 || C <= 0 || C % 4) return kfail(FVAR_EINVAL, "row_keys: bad arguments");
  FK_CUDA(launch_row_scores(x, RowMap{1, 0, M}, B, M, C, noise, keys, static_cast<cudaStream_t>(stream)), "row_keys");
  return FVAR_OK;
}

fvar_status fvar_select_topr(const float *scores, int B, int M, int r, int *idx, int *inv, void *stream) {
  if (!scores || !idx || !inv || B <= 0 || M <= 0 || r <= 0 || r > M) return kfail(FVAR_EINVAL, "select_topr: bad arguments");
  FK_CUDA(launch_select_topr(scores, B, M, r, idx, inv, static_cast<cudaStream_t>(stream)), "select_topr");
  return FVAR_OK;
}

fvar_status fvar_ln_modulate(const float *x, int R, int C, int rows_per_batch, const float *shift, const float *scale,
                             long long vec_stride, float eps, void *y, void *stream) {
  if (!x || !y || !shift || !scale || R <= 0 || C <= 0 || C % 8 || C > 8192 || rows_per_batch <= 0 || R % rows_per_batch)
    return kfail(FVAR_EINVAL, "ln_modulate: bad arguments");
  FK_CUDA(launch_ln_modulate(x, RowMap{1, 0, rows_per_batch}, R / rows_per_batch, rows_per_batch, C, shift, scale,
                             vec_stride, 1, 0, nullptr, eps, static_cast<bf16 *>(y), static_cast<cudaStream_t>(stream)),
          "ln_modulate");
  return FVAR_OK;
}

fvar_status fvar_gemm_bf16_form(const void *A, const void *W, const void *bias, int R, int N, int K, int form,
                                int block_n, float *out, void *stream) {
  if (!A || !W || !out || R <= 0 || N <= 0 || K <= 0 || K % 8) return kfail(FVAR_EINVAL, "gemm: bad arguments");
  if (form != FVAR_GEMM_AUTO && form != FVAR_GEMM_SINGLE && form != FVAR_GEMM_PAIR && form != FVAR_GEMM_SKINNY && form != FVAR_GEMM_KSPLIT)
    return kfail(FVAR_EINVAL, "gemm: bad form");
  if (form == FVAR_GEMM_SKINNY || form == FVAR_GEMM_KSPLIT) {
    const int tiles_m = form == FVAR_GEMM_KSPLIT ? (R + 127) / 128 : 0;
    if (form == FVAR_GEMM_SKINNY && !gemm_skinny_supported(EPI_F32, R, N, K))
      return kfail(FVAR_EINVAL, "gemm: the weight-streaming form needs R <= 512, N % 8 == 0");
    if (N % 8) return kfail(FVAR_EINVAL, "gemm: the cluster-split forms need N % 8 == 0");
    if (block_n < 0 || block_n > 8) return kfail(FVAR_EINVAL, "gemm: the cluster-split forms take 0 .. 8 K ranges");
    const int S = gemm_skinny_pick_splits(N, K, block_n, tiles_m, tiles_m == 0 && R <= 64);
    if (S <= 0) return kfail(FVAR_EINVAL, "gemm: this number of K ranges is not launchable for the problem");
    GemmArgs g = gemm_args(R, N, K);
    g.sk_tiles_m = tiles_m;
    g.splits = S;
    gemm_skinny_shape(g);
    CUtensorMap ta, tw;
    if (g.sk_stages < 1 || !gemm_skinny_map(&ta, A, R, K, K, g.sk_rp, g.sk_nk) || !gemm_skinny_map(&tw, W, N, K, K, 128, g.sk_nk))
      return kfail(FVAR_EINVAL, "gemm: operands must be 16-byte aligned");
    g.bias = static_cast<const bf16 *>(bias);
    g.out_f32 = out;
    g.ld_out = N;
    g.splits = S;
    g.status = kernel_status_ptr();
    if (!g.status) return kfail(FVAR_ECUDA, "gemm: status word");
    FK_CUDA(launch_gemm_skinny(EPI_F32, ta, tw, g, static_cast<cudaStream_t>(stream)), "gemm");
    return FVAR_OK;
  }
  int dev = 0, sms = 0;
  FK_CUDA(cudaGetDevice(&dev), "get device");
  FK_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev), "device attribute");
  const int max_clusters = form == FVAR_GEMM_SINGLE ? 0 : gemm_pair_max_clusters();
  GemmPlan plan = gemm_plan(R, 1, N, K, sms, max_clusters, 1, 0);
  if (form == FVAR_GEMM_PAIR) {
    if (R <= 128 || max_clusters <= 0) return kfail(FVAR_EINVAL, "gemm: the pair form needs R > 128 and a device that runs CTA pairs");
    if (block_n != 0 && block_n != 128 && block_n != 256) return kfail(FVAR_EINVAL, "gemm: pair block_n must be 128 or 256");
    if (!plan.pair) plan = GemmPlan{true, (N > 128) ? 256 : 128, 1};
    if (block_n) plan.block_n = block_n;
  } else if (block_n != 0) {
    if (form == FVAR_GEMM_AUTO) return kfail(FVAR_EINVAL, "gemm: block_n needs an explicit form");
    if (block_n != 64 && block_n != 128 && block_n != 256) return kfail(FVAR_EINVAL, "gemm: block_n must be 64, 128 or 256");
    plan.block_n = block_n;
  }
  const int bn = plan.block_n;
  CUtensorMap ta, tw;
  if (!tmap_2d(&ta, A, K, R, K, 128) || !tmap_2d(&tw, W, K, N, K, plan.pair ? bn / 2 : bn))
    return kfail(FVAR_EINVAL, "gemm: operands must be 16-byte aligned");
  GemmArgs g = gemm_args(R, N, K);
  g.bias = static_cast<const bf16 *>(bias);
  g.out_f32 = out;
  g.ld_out = N;
  g.status = kernel_status_ptr();
  if (!g.status) return kfail(FVAR_ECUDA, "gemm: status word");
  if (plan.pair)
    FK_CUDA(launch_gemm_pair(EPI_F32, bn, ta, tw, g, static_cast<cudaStream_t>(stream)), "gemm");
  else
    FK_CUDA(launch_gemm(EPI_F32, bn, ta, tw, g, sms, static_cast<cudaStream_t>(stream)), "gemm");
  return FVAR_OK;
}

fvar_status fvar_gemm_bf16_wt(const void *A, const void *Wt, const void *bias, int R, int N, int K, int block_n, float *out,
                              void *stream) {
  if (!A || !Wt || !out || R <= 0 || N <= 0 || K <= 0 || K % 8 || N % 8) return kfail(FVAR_EINVAL, "gemm_wt: bad arguments");
  int dev = 0, sms = 0;
  FK_CUDA(cudaGetDevice(&dev), "get device");
  FK_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev), "device attribute");
  int bn = block_n ? block_n : gemm_pick_block_n((R + 127) / 128, N, K, sms);
  if (bn != 64 && bn != 128 && bn != 256) return kfail(FVAR_EINVAL, "gemm_wt: block_n must be 64, 128 or 256");
  CUtensorMap ta, tw;
  if (!tmap_2d(&ta, A, K, R, K, 128) || !tmap_2d(&tw, Wt, N, K, N, 64)) return kfail(FVAR_EINVAL, "gemm_wt: operands must be 16-byte aligned");
  GemmArgs g = gemm_args(R, N, K);
  g.bias = static_cast<const bf16 *>(bias);
  g.out_f32 = out;
  g.ld_out = N;
  g.w_mn_major = 1;
  g.status = kernel_status_ptr();
  if (!g.status) return kfail(FVAR_ECUDA, "gemm_wt: status word");
  FK_CUDA(launch_gemm(EPI_F32, bn, ta, tw, g, sms, static_cast<cudaStream_t>(stream)), "gemm_wt");
  return FVAR_OK;
}

fvar_status fvar_gemm_bf16(const void *A, const void *W, const void *bias, int R, int N, int K, float *out, void *stream) {
  return fvar_gemm_bf16_form(A, W, bias, R, N, K, FVAR_GEMM_AUTO, 0, out, stream);
}

fvar_status fvar_attention(const void *q, const void *Kc, const void *Vt, int B, int H, int r, int D, int L, int L_cap,
                           void *out, void *stream) {
  if (!q || !Kc || !Vt || !out || B <= 0 || H <= 0 || r <= 0 || (D != 64 && D != 128) || L <= 0 || L > L_cap || L_cap % 8)
    return kfail(FVAR_EINVAL, "attention: bad arguments");
  CUtensorMap tq, tk, tv;
  const uint64_t BH = static_cast<uint64_t>(B) * H;
  if (!tmap_2d(&tq, q, static_cast<uint64_t>(H) * D, static_cast<uint64_t>(B) * r, static_cast<uint64_t>(H) * D, 128) ||
      !tmap_3d(&tk, Kc, D, L_cap, BH, D, static_cast<uint64_t>(L_cap) * D, 64, 128) ||
      !tmap_3d(&tv, Vt, L_cap, D, BH, L_cap, static_cast<uint64_t>(L_cap) * D, 64, D))
    return kfail(FVAR_EINVAL, "attention: operands must be 16-byte aligned");
  AttnArgs a{B, H, r, D, L, L_cap, 1, 0, static_cast<bf16 *>(out), 1.4426950408889634f / sqrtf(static_cast<float>(D)),
             kernel_status_ptr(), 1};
  int dev = 0, sms = 0;
  FK_CUDA(cudaGetDevice(&dev), "get device");
  FK_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev), "device attribute");
  attention_plan(B, H, r, L, sms, &a.tiles_per_cta, &a.kv_splits);
  if (!a.status) return kfail(FVAR_ECUDA, "attention: status word");
  FK_CUDA(launch_attention(tq, tk, tv, a, static_cast<cudaStream_t>(stream)), "attention");
  return FVAR_OK;
}

fvar_status fvar_cfg_combine(const void *pair, int B, long long per_elem, float guidance, void *out, void *stream) {
  if (!pair || !out || B <= 0 || (B & 1) || per_elem <= 0 || per_elem % 8 || (reinterpret_cast<uintptr_t>(pair) & 15) ||
      (reinterpret_cast<uintptr_t>(out) & 15))
    return kfail(FVAR_EINVAL, "cfg_combine: bad arguments");
  FK_CUDA(launch_cfg_combine(static_cast<const bf16 *>(pair), B / 2, per_elem, guidance, static_cast<bf16 *>(out),
                             static_cast<cudaStream_t>(stream)), "cfg_combine");
  return FVAR_OK;
}

fvar_status fvar_selftest_wait_timeout(fvar_ctx *ctx, long long cycles, void *stream) {
  if (cycles <= 0) return ctx ? fail(ctx, FVAR_EINVAL, "selftest: cycles must be positive") : kfail(FVAR_EINVAL, "selftest: cycles must be positive");
  unsigned *status = ctx ? ctx->status : kernel_status_ptr();
  if (!status) return kfail(FVAR_ECUDA, "selftest: status word");
  cudaStream_t st = ctx ? ctx->st : static_cast<cudaStream_t>(stream);
  cudaError_t e = launch_wait_selftest(cycles, status, st);
  if (e != cudaSuccess) return ctx ? cuda_fail(ctx, e, "selftest") : kfail(FVAR_ECUDA, cudaGetErrorString(e));
  if (ctx) ctx->launched();
  return FVAR_OK;
}

fvar_status fvar_l2_prefetch(const void *ptr, size_t bytes, void *stream) {
  if (!ptr || (reinterpret_cast<uintptr_t>(ptr) & 15)) return kfail(FVAR_EINVAL, "l2_prefetch: NULL or unaligned pointer");
  FK_CUDA(launch_l2_prefetch(ptr, bytes, static_cast<cudaStream_t>(stream)), "l2_prefetch");
  return FVAR_OK;
}

fvar_status fvar_rtr_fill(const float *prev, int B, int h0, int w0, int h1, int w1, int C, const int *inv, float *out,
                          void *stream) {
  if (!prev || !out || B <= 0 || h0 <= 0 || w0 <= 0 || h1 <= 0 || w1 <= 0 || C <= 0 || C % 4)
    return kfail(FVAR_EINVAL, "rtr_fill: bad arguments");
  FK_CUDA(launch_rtr_fill(prev, out, B, 1, 0, h0, w0, h1, w1, C, inv, nullptr, 0, static_cast<cudaStream_t>(stream)), "rtr_fill");
  return FVAR_OK;
}

}  // extern "C"
