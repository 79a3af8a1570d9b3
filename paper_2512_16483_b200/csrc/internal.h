// Internal launch interfaces between the translation units of libfvar.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace fvar {

typedef __nv_bfloat16 bf16;

// Maps (computed element e, row j within it) to a row of a per-batch buffer:
// row = (e * bmul + boff) * rpb + j.  Compact buffers use {1, 0, r}; buffers indexed by the
// caller's batch element use {2, 1, M} when only the null-prompt half of each pair is computed.
struct RowMap {
  int bmul, boff, rpb;
};

// Bilinear upsampling (Eq. "upcache", Eq. "var_upf"): source cell and weights of target cell (y, x) on an (h1, w1) grid
// read from an (h0, w0) grid -- half-pixel centres, source coordinate clamped at 0, neighbours clamped at the edge.
struct BilinearTap {
  int y0, y1, x0, x1;
  float w00, w01, w10, w11;
};
__host__ __device__ inline BilinearTap bilinear_tap(int y, int x, int h0, int w0, int h1, int w1) {
  const float sy = fmaxf((y + 0.5f) * (static_cast<float>(h0) / h1) - 0.5f, 0.f);
  const float sx = fmaxf((x + 0.5f) * (static_cast<float>(w0) / w1) - 0.5f, 0.f);
  BilinearTap t;
  t.y0 = min(static_cast<int>(sy), h0 - 1); t.x0 = min(static_cast<int>(sx), w0 - 1);
  t.y1 = min(t.y0 + 1, h0 - 1); t.x1 = min(t.x0 + 1, w0 - 1);
  const float fy = sy - t.y0, fx = sx - t.x0;
  t.w00 = (1.f - fy) * (1.f - fx); t.w01 = (1.f - fy) * fx; t.w10 = fy * (1.f - fx); t.w11 = fy * fx;
  return t;
}

enum EpiMode { EPI_F32 = 0, EPI_BF16 = 1, EPI_GELU_BF16 = 2, EPI_QKV = 3, EPI_RESID = 4, EPI_ARGMAX = 5 };

struct GemmArgs {
  int R, N, K;            // out[R][N] = A[R][K] * W[N][K]^T, per batch
  int a_box_rows;         // rows of the A tensor map's box (0 = 128)
  int nbatch;             // number of independent problems sharing the launch
  int a_batch_rows;       // row offset of batch e in the A tensor map (0: A shared by all)
  int b_batch_rows;       // row offset of batch e in the W tensor map (0: W shared by all)
  const bf16 *bias;       // [N] or nullptr
  int rows_per_batch;     // rows of one computed element inside R (epilogues that need (e, j))
  int bmul, boff;         // caller batch element of computed element e: e * bmul + boff
  // EPI_F32 / EPI_RESID output, EPI_BF16 / EPI_GELU_BF16 / EPI_QKV (q part) output
  float *out_f32;
  bf16 *out_bf16;
  long long ld_out;
  // EPI_RESID: out[omap(e, j')] = resid[rmap(e, j)] + gate[b] * (acc + bias); j' = scatter ? scatter[e][j] : j
  const float *resid;
  RowMap rmap, omap;
  const float *gate;      // vector of caller batch element b at gate + b * gate_stride, or nullptr (gate = 1)
  long long gate_stride;
  const int *scatter;     // [E][rows_per_batch] or nullptr
  // EPI_RESID, optional: the result also goes out as its two-term bf16 split for the next group's projection,
  // xsplit[e][half][row j'][col] with half 0 = hi = bf16(x), half 1 = lo = bf16(x - hi); xsplit_mk rows per half
  bf16 *xsplit;
  int xsplit_mk;
  // EPI_QKV: virtual column = col + col_base; [0,C) -> q, [C,2C) -> K cache, [2C,3C) -> transposed V cache
  bf16 *kc, *vt;
  int C, H, D, L_cap, L_prev, col_base;
  // EPI_ARGMAX: per row, the column with the largest (acc - col_sub[col]), lowest column on ties, kept as one
  // 64-bit word per row: ordered score bits << 32 | ~column (so that an unsigned max picks it); best must be
  // zero before the launch
  const float *col_sub;
  unsigned long long *best;
  // W given MN-major: the tensor map describes W^T, a row-major [K][N] matrix (64-column boxes of 64 K rows), with
  // batch e at row offset e * b_batch_rows along K.  Single-CTA kernel only.
  int w_mn_major;
  // split-K (splits > 1): fp32 partial tiles [tile][split][128][BN] and one arrival counter per tile
  int splits;
  float *partial;
  int *counters;
  unsigned *status;
  // Weight-streaming form (gemm_skinny.cu; `splits` is then the cluster size): rows per column chunk, the padded
  // MMA width of a chunk, chunks (1 or 2) and pipeline stages -- filled by gemm_skinny_shape
  int sk_rows_chunk, sk_rp, sk_nchunks, sk_stages, sk_small, sk_nk;
  int sk_tiles_m;          // > 0: the 128 x 128-tile mode of that kernel with this many row tiles (rows on the M side)
  // optional: weights the next GEMM of the chain will stream; every CTA asks L2 to prefetch its share
  const void *pf_ptr;
  unsigned long long pf_bytes;
  long long wait_cycles;   // budget of every bounded wait (0: the default, about half a second)
};

// Tensor maps: bf16, 2-D {cols, rows} with a {64, box_rows} box and 128-byte swizzle, or the 3-D
// forms used for the KV cache.
bool tmap_init_driver();
bool tmap_2d(CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows, uint64_t ld_elems, uint32_t box_rows);
// {64 K elements, rows, K blocks} view of a K-major [rows][64 * kblocks] matrix (row pitch ld_elems): a box
// {64, box_rows, box_kb} lands as box_kb consecutive swizzled [box_rows][64] tiles.
bool tmap_kblocks(CUtensorMap *m, const void *base, uint64_t rows, uint64_t kblocks, uint64_t ld_elems, uint32_t box_rows,
                  uint32_t box_kb);
bool tmap_3d(CUtensorMap *m, const void *base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t ld1_elems,
             uint64_t ld2_elems, uint32_t box0, uint32_t box1);

int gemm_pick_block_n(int tiles_m_total, int N, int K, int num_sms);
void gemm_pick_tile(int tiles_m_total, int N, int K, int num_sms, int max_splits, size_t scratch_bytes, int *block_n,
                    int *splits);
// Launches the tensor-core GEMM.  block_n in {64, 128, 256}: the W map's box must have block_n rows.
cudaError_t launch_gemm(int epi, int block_n, const CUtensorMap &tmA, const CUtensorMap &tmW, const GemmArgs &a,
                        int num_sms, cudaStream_t st);

// CTA-pair form (gemm_pair.cu): 256 x block_n tiles, block_n in {128, 256}; the W map's box must have
// block_n / 2 rows, the A map's box 128 rows.  One problem per launch (nbatch == 1), no split-K.
cudaError_t launch_gemm_pair(int epi, int block_n, const CUtensorMap &tmA, const CUtensorMap &tmW, const GemmArgs &a,
                             cudaStream_t st);
// Largest number of CTA pairs of the pair kernel that can be resident at once (0: pairs unavailable).
int gemm_pair_max_clusters();
// How a GEMM is launched: by single CTAs (block_n in {64, 128, 256}, optional split-K) or by CTA pairs
// (block_n in {128, 256}).
struct GemmPlan {
  bool pair;
  int block_n, splits;
};
// Picks the launch form and tile width from the measured cost model.  tiles_m_total: 128-row tiles over
// all batches; pairs are considered only for a single problem with more than one row tile.
GemmPlan gemm_plan(int R, int nbatch, int N, int K, int num_sms, int max_clusters, int max_splits, size_t scratch_bytes);

// Weight-streaming form for R <= 512 rows (gemm_skinny.cu): the weights are the M side of the MMA, the K range of
// a 128-feature tile is split over a cluster of `splits` CTAs that reduce through distributed shared memory.
// tmA: box {64, a.sk_rp} over the activation rows; tmW: box {64, 128} over the weight rows.
bool gemm_skinny_supported(int epi, int R, int N, int K);
int gemm_skinny_row_limit(int N, int K);
bool gemm_ksplit_wins(int R, int N, int K);                   // the 128 x 128-tile cluster-split mode is the faster form                      // rows up to which this form is the faster one
int gemm_skinny_pick_splits(int N, int K, int forced, int row_tiles = 0, int small_form = 0);      // 0: not launchable on this device
void gemm_skinny_shape(GemmArgs &a);      // needs a.R, a.K and a.splits
bool gemm_skinny_map(CUtensorMap *m, const void *base, uint64_t rows, uint64_t K, uint64_t ld, uint32_t box_rows, int nk);
cudaError_t launch_gemm_skinny(int epi, const CUtensorMap &tmA, const CUtensorMap &tmW, const GemmArgs &a, cudaStream_t st);
cudaError_t gemm_skinny_prepare();

// Set the dynamic shared-memory attribute of every instantiation (once, outside any stream capture).
cudaError_t gemm_prepare();
cudaError_t gemm_pair_prepare();
cudaError_t attention_prepare();

struct AttnArgs {
  int B_eff, H, r, D, L, L_cap;
  int bmul, boff;          // caller batch element (cache slot) of computed element e
  bf16 *out;               // [B_eff * r][H * D]
  float scale_log2;        // log2(e) / sqrt(D)
  unsigned *status;
  // kv_splits > 1: the key range is split over a cluster of that many CTAs (at most 8 supported by the kernel; the planner uses up to 6), merged through
  // distributed shared memory
  int kv_splits;
  int tiles_per_cta;       // 1: one 128-row query tile per CTA; otherwise two
  long long wait_cycles;   // budget of every bounded wait (0: the default)
};
// Query tiles per CTA (1 or 2) and key ranges per launch (1 = no split; at most 6).
void attention_plan(int B_eff, int H, int r, int L, int num_sms, int *tiles_per_cta, int *kv_splits);
cudaError_t launch_attention(const CUtensorMap &tmQ, const CUtensorMap &tmK, const CUtensorMap &tmV,
                             const AttnArgs &a, cudaStream_t st);

// Launch with programmatic stream serialization (see pdl_wait in ptx.cuh).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// Records the message fvar_last_error(NULL) returns.
void set_global_error(const char *msg);

// Memory-bound kernels.
cudaError_t launch_row_scores(const float *x, RowMap xmap, int E, int M, int C, const float *noise, float *scores,
                              cudaStream_t st);
cudaError_t launch_select_topr(const float *scores, int B, int M, int r, int *idx, int *inv, cudaStream_t st);
cudaError_t launch_copy_indices(const int *forced, int B, int M, int r, int ld_forced, int *idx, int *inv,
                                unsigned *status, cudaStream_t st);
cudaError_t launch_ln_modulate(const float *x, RowMap xmap, int E, int rows, int C, const float *shift,
                               const float *scale, long long vec_stride, int bmul, int boff,
                               const bf16 *gamma, float eps, bf16 *y, cudaStream_t st);
// xsplit (optional): the filled rows also go out as their two-term bf16 split, [E][2][mk][C] (see GemmArgs::xsplit).
cudaError_t launch_rtr_fill(const float *prev, float *out, int E, int bmul, int boff, int h0, int w0, int h1,
                            int w1, int C, const int *inv, bf16 *xsplit, int mk, cudaStream_t st);
// The E computed elements only: element e is read at element e * smul + soff of `tok` and written at element
// e * bmul + boff of `x`.  xsplit (optional): the rows also go out as hi = token, lo = 0 in the [E][2][mk][C] split
// layout (tokens are bf16 already).
cudaError_t launch_tokens_to_f32(const bf16 *tok, float *x, int E, int M, int C, bf16 *xsplit, int mk, int smul, int soff,
                                 int bmul, int boff, cudaStream_t st);
cudaError_t launch_out_to_bf16(const float *x, RowMap xmap, int E, int M, int C, bf16 *out, cudaStream_t st);
cudaError_t launch_generate_projection(bf16 *qt, int M, int Mk, int r, unsigned long long seed, int group, int scale,
                                       cudaStream_t st);
// Between two scale steps: codeword half-norms, the packed argmax words, Up-accumulate and area Down.
cudaError_t launch_half_norms(const bf16 *Z, int V, int C, float *hn, cudaStream_t st);
cudaError_t launch_unpack_codes(const unsigned long long *best, long long n, int V, int *codes, unsigned *status,
                                cudaStream_t st);
cudaError_t launch_up_accumulate(const bf16 *Z, const int *codes, int B, int h0, int w0, int h1, int w1, int C,
                                 bool overwrite, float *F, cudaStream_t st);
cudaError_t launch_cfg_combine(const bf16 *pair, int pairs, long long per_elem, float s, bf16 *out, cudaStream_t st);
// dup: every element is written twice, [2B][h1 * w1][C] (the two branches of a CFG pair).
cudaError_t launch_down_area(const float *F, int B, int h0, int w0, int h1, int w1, int C, bf16 *tokens, bool dup, cudaStream_t st);
// LLS restoration (lls.cu): fp32 products, the inverse of an r x r Gram matrix through its Cholesky factor, and the
// two-term bf16 split of fp32 rows.  Ranks up to kLlsMaxRank (the factor lives in one CTA's shared memory).
constexpr int kLlsMaxRank = 192;
cudaError_t lls_prepare();
// out[z] (+)= A[z] B[z]^T (trans_b: B stored [n][k]) or A[z] B[z] (B stored [k][n]); pitches and batch strides in floats.
cudaError_t launch_sgemm(bool trans_b, const float *A, const float *B, float *out, int m, int n, int k, long long lda, long long ldb,
                         long long ldo, long long a_off, long long a_stride, long long b_off, long long b_stride, long long o_off,
                         long long o_stride, int batch, bool accumulate, cudaStream_t st, int ksplit = 1, float *scratch = nullptr);
cudaError_t launch_chol_inverse(const float *G, float *Ginv, int r, int count, unsigned *status, cudaStream_t st);
cudaError_t launch_split_rows(const float *x, long long x_off, long long x_stride, int E, int M, int C, bf16 *xsplit, int mk,
                              cudaStream_t st);

// Self-test of the bounded wait: one CTA waits on an mbarrier nobody signals with a budget of `cycles`, flags the
// status word and returns.
cudaError_t launch_wait_selftest(long long cycles, unsigned *status, cudaStream_t st);
cudaError_t launch_l2_prefetch(const void *ptr, unsigned long long bytes, cudaStream_t st);
cudaError_t launch_silu_bf16(const bf16 *in, bf16 *out, long long n, cudaStream_t st);
cudaError_t launch_load_kv(const bf16 *K, const bf16 *V, int B, int L, int H, int D, int L_cap, bf16 *kc, bf16 *vt,
                           cudaStream_t st);

}  // namespace fvar
