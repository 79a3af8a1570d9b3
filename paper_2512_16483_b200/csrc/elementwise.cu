// HBM-bound kernels of the path: row score, top-r selection with ballot prefix-sum compaction,
// LayerNorm + AdaLN modulation, restoration fill (bilinear Up of the cached group output), and
// the layout / type conversions between them.  All use 16-byte vector accesses.
#include "internal.h"
#include "ptx.cuh"

namespace fvar {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ------------------------------------------------------------------------------------------------
// Row score s_i = sum_c x[i][c]^2: one warp per row, float4 loads.  Row (e, i) of the compact
// score array reads row xmap(e, i) of x.
// With `noise` (Exp(1) variates, one per row) the value written is the sampling key s_i / E_i: the r
// largest keys are a draw without replacement with probability proportional to s_i.
__global__ void __launch_bounds__(256) row_scores_kernel(const float *__restrict__ x, RowMap xmap, int M,
                                                         long long rows, int C, const float *__restrict__ noise,
                                                         float *__restrict__ scores) {
  pdl_wait();
  pdl_launch_dependents();
  const long long row = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int lane = threadIdx.x & 31;
  const int e = static_cast<int>(row / M), i = static_cast<int>(row - static_cast<long long>(e) * M);
  const float4 *p = reinterpret_cast<const float4 *>(x + (static_cast<long long>(e * xmap.bmul + xmap.boff) * xmap.rpb + i) * C);
  float acc = 0.f;
  for (int c = lane; c < C / 4; c += 32) {
    float4 v = __ldg(p + c);
    acc = fmaf(v.x, v.x, acc);
    acc = fmaf(v.y, v.y, acc);
    acc = fmaf(v.z, v.z, acc);
    acc = fmaf(v.w, v.w, acc);
  }
  acc = warp_sum(acc);
  if (lane == 0) scores[row] = noise ? __fdiv_rn(acc, noise[row]) : acc;
}

cudaError_t launch_row_scores(const float *x, RowMap xmap, int E, int M, int C, const float *noise, float *scores,
                              cudaStream_t st) {
  const long long rows = static_cast<long long>(E) * M;
  if (rows <= 0) return cudaSuccess;
  return launch_pdl(row_scores_kernel, dim3(static_cast<unsigned>((rows + 7) / 8)), dim3(256), 0, st, x, xmap, M, rows, C, noise, scores);
}

// ------------------------------------------------------------------------------------------------
// Top-r selection.  One CTA per batch element.  The fp32 scores map to unsigned keys whose order
// is the float order (NaN -> +inf, -0 -> +0); a 4-pass, 8-bit radix select finds the key of the
// r-th largest; rows are then compacted in ascending index order: every key above the threshold,
// plus the first (r - #above) rows whose key equals it.  Prefix sums use warp ballots.
constexpr int kSelThreads = 1024;

__device__ __forceinline__ unsigned score_key(float s) {
  if (s != s) s = INFINITY;
  s += 0.0f;                                    // -0 -> +0
  const unsigned u = __float_as_uint(s);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__global__ void __launch_bounds__(kSelThreads) select_topr_kernel(const float *__restrict__ scores, int M, int r,
                                                                  int *__restrict__ idx, int *__restrict__ inv) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ unsigned hist[256];
  __shared__ unsigned s_prefix, s_need;
  __shared__ int warp_gt[32], warp_eq[32];
  __shared__ int base_gt, base_eq;
  const int b = blockIdx.x;
  const float *s = scores + static_cast<long long>(b) * M;
  int *idx_b = idx + static_cast<long long>(b) * r;
  int *inv_b = inv + static_cast<long long>(b) * M;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // radix select: after the loop, `prefix` is the key of the r-th largest and `need` is how many
  // rows with exactly that key are taken
  unsigned prefix = 0, mask = 0, need = static_cast<unsigned>(r);
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    for (int i = tid; i < M; i += kSelThreads) {
      const unsigned k = score_key(s[i]);
      if ((k & mask) == prefix) atomicAdd(&hist[(k >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (warp == 0) {
      // Find the digit d at which the count of keys with a larger digit first reaches `need`:
      // lane l owns the 8 bins 255 - 8l ... 248 - 8l; a warp scan gives the count above its range.
      unsigned cnt[8], tot = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        cnt[j] = hist[255 - 8 * lane - j];
        tot += cnt[j];
      }
      unsigned incl = tot;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      unsigned acc = incl - tot;
      if (acc < need && need <= incl) {          // exactly one lane: the matching set holds >= need keys
        int d = 255 - 8 * lane;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (acc + cnt[j] >= need) break;
          acc += cnt[j];
          --d;
        }
        s_prefix = prefix | (static_cast<unsigned>(d) << shift);
        s_need = need - acc;
      }
    }
    __syncthreads();
    prefix = s_prefix;
    need = s_need;
    mask |= 255u << shift;
    __syncthreads();
  }
  const unsigned thr = prefix;

  if (tid == 0) {
    base_gt = 0;
    base_eq = 0;
  }
  __syncthreads();
  for (int start = 0; start < M; start += kSelThreads) {
    const int i = start + tid;
    const unsigned k = (i < M) ? score_key(s[i]) : 0u;
    const bool gt = (i < M) && k > thr;
    const bool eq = (i < M) && k == thr;
    const unsigned bgt = __ballot_sync(0xffffffffu, gt), beq = __ballot_sync(0xffffffffu, eq);
    if (lane == 0) {
      warp_gt[warp] = __popc(bgt);
      warp_eq[warp] = __popc(beq);
    }
    __syncthreads();
    if (warp == 0) {                           // exclusive scan of the 32 per-warp counts
      int g = warp_gt[lane], q = warp_eq[lane];
      int gi = g, qi = q;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int tg = __shfl_up_sync(0xffffffffu, gi, o), tq = __shfl_up_sync(0xffffffffu, qi, o);
        if (lane >= o) {
          gi += tg;
          qi += tq;
        }
      }
      warp_gt[lane] = gi - g;
      warp_eq[lane] = qi - q;
    }
    __syncthreads();
    const unsigned below = (1u << lane) - 1u;
    const int n_gt = base_gt + warp_gt[warp] + __popc(bgt & below);   // rows above thr before i
    const int n_eq = base_eq + warp_eq[warp] + __popc(beq & below);   // rows equal to thr before i
    if (i < M) {
      const bool take = gt || (eq && n_eq < static_cast<int>(need));
      const int pos = n_gt + min(n_eq, static_cast<int>(need));
      if (take) idx_b[pos] = i;
      inv_b[i] = take ? pos : -1;
    }
    __syncthreads();
    if (tid == kSelThreads - 1) {
      base_gt = n_gt + (gt ? 1 : 0);
      base_eq = n_eq + (eq ? 1 : 0);
    }
    __syncthreads();
  }
}

cudaError_t launch_select_topr(const float *scores, int B, int M, int r, int *idx, int *inv, cudaStream_t st) {
  if (B <= 0) return cudaSuccess;
  return launch_pdl(select_topr_kernel, dim3(B), dim3(kSelThreads), 0, st, scores, M, r, idx, inv);
}

// Test hook: take the caller's index lists instead of selecting.  Checks range and strict ascent;
// a bad list sets a status bit and the offending entry is clamped into range.
__global__ void copy_indices_kernel(const int *__restrict__ forced, int M, int r, int ld_forced,
                                    int *__restrict__ idx, int *__restrict__ inv, unsigned *status) {
  pdl_wait();
  pdl_launch_dependents();
  const int b = blockIdx.x;
  const int *f = forced + static_cast<long long>(b) * ld_forced;
  int *idx_b = idx + static_cast<long long>(b) * r;
  int *inv_b = inv + static_cast<long long>(b) * M;
  for (int i = threadIdx.x; i < M; i += blockDim.x) inv_b[i] = -1;
  __syncthreads();
  for (int j = threadIdx.x; j < r; j += blockDim.x) {
    int v = f[j];
    const bool bad = v < 0 || v >= M || (j > 0 && f[j - 1] >= v);
    if (bad) atomicOr(status, kStatusBadIndex);
    v = min(max(v, 0), M - 1);
    idx_b[j] = v;
    inv_b[v] = j;
  }
}

cudaError_t launch_copy_indices(const int *forced, int B, int M, int r, int ld_forced, int *idx, int *inv,
                                unsigned *status, cudaStream_t st) {
  return launch_pdl(copy_indices_kernel, dim3(B), dim3(256), 0, st, forced, M, r, ld_forced, idx, inv, status);
}

// ------------------------------------------------------------------------------------------------
// y = LN(x) * (1 + scale) + shift  (or LN(x) * gamma): one CTA of 128 threads per row, the row
// held in registers (two-pass mean / variance), bf16 output, 16-byte accesses.
constexpr int kLnThreads = 128;
constexpr int kLnMaxVec = 8;                    // 8 x (8 elements) x 128 threads = 8192 columns

// Normalises, modulates (or scales by gamma) and stores one group of 8 consecutive elements of a row: group g of
// the row whose values are in v, statistics mean / rstd; shift and scale at float offset voff, y row at yr.
__device__ __forceinline__ void ln_store_group(const float (&v)[8], float mean, float rstd, const bf16 *__restrict__ gamma,
                                               const float *__restrict__ scale, const float *__restrict__ shift, long long voff,
                                               int g, bf16 *__restrict__ yr) {
  float o[8];
  if (gamma != nullptr) {
    const uint4 gu = __ldg(reinterpret_cast<const uint4 *>(gamma) + g);
    const __nv_bfloat162 *gh = reinterpret_cast<const __nv_bfloat162 *>(&gu);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 gf = __bfloat1622float2(gh[i]);
      o[2 * i] = (v[2 * i] - mean) * rstd * gf.x;
      o[2 * i + 1] = (v[2 * i + 1] - mean) * rstd * gf.y;
    }
  } else {
    const float4 *sc = reinterpret_cast<const float4 *>(scale + voff) + 2 * g;
    const float4 *sh = reinterpret_cast<const float4 *>(shift + voff) + 2 * g;
    const float4 s0 = __ldg(sc), s1 = __ldg(sc + 1), h0 = __ldg(sh), h1 = __ldg(sh + 1);
    const float scv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
    const float shv[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i] = fmaf((v[i] - mean) * rstd, 1.0f + scv[i], shv[i]);
  }
  uint32_t w[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 h2 = __floats2bfloat162_rn(o[2 * i], o[2 * i + 1]);
    w[i] = *reinterpret_cast<uint32_t *>(&h2);
  }
  reinterpret_cast<uint4 *>(yr)[g] = make_uint4(w[0], w[1], w[2], w[3]);
}

__global__ void __launch_bounds__(kLnThreads) ln_modulate_kernel(const float *__restrict__ x, RowMap xmap, int rows,
                                                                 int C, const float *__restrict__ shift,
                                                                 const float *__restrict__ scale,
                                                                 long long vec_stride, int bmul, int boff,
                                                                 const bf16 *__restrict__ gamma, float eps,
                                                                 bf16 *__restrict__ y) {
  pdl_launch_dependents();      // nothing precedes the wait: the successor may start its own prologue right away
  pdl_wait();
  __shared__ float red[kLnThreads / 32];
  const int e = blockIdx.x / rows, j = blockIdx.x - e * rows;
  const float *xr = x + (static_cast<long long>(e * xmap.bmul + xmap.boff) * xmap.rpb + j) * C;
  bf16 *yr = y + static_cast<long long>(blockIdx.x) * C;
  const int nvec = C / 8;                       // 8-element groups in the row
  float v[kLnMaxVec][8];
  float sum = 0.f;
#pragma unroll
  for (int t = 0; t < kLnMaxVec; ++t) {
    const int g = threadIdx.x + t * kLnThreads;
    if (g < nvec) {
      const float4 a = reinterpret_cast<const float4 *>(xr)[2 * g], c = reinterpret_cast<const float4 *>(xr)[2 * g + 1];
      v[t][0] = a.x; v[t][1] = a.y; v[t][2] = a.z; v[t][3] = a.w;
      v[t][4] = c.x; v[t][5] = c.y; v[t][6] = c.z; v[t][7] = c.w;
#pragma unroll
      for (int i = 0; i < 8; ++i) sum += v[t][i];
    }
  }
  auto block_sum = [&](float val) {
    val = warp_sum(val);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = val;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kLnThreads / 32; ++w) tot += red[w];
    return tot;
  };
  const float mean = block_sum(sum) / C;
  float sq = 0.f;
#pragma unroll
  for (int t = 0; t < kLnMaxVec; ++t) {
    const int g = threadIdx.x + t * kLnThreads;
    if (g < nvec) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float d = v[t][i] - mean;
        sq = fmaf(d, d, sq);
      }
    }
  }
  const float rstd = rsqrtf(block_sum(sq) / C + eps);
  const long long voff = static_cast<long long>(e * bmul + boff) * vec_stride;
#pragma unroll
  for (int t = 0; t < kLnMaxVec; ++t) {
    const int g = threadIdx.x + t * kLnThreads;
    if (g < nvec) {
      ln_store_group(v[t], mean, rstd, gamma, scale, shift, voff, g, yr);
    }
  }
}

// Warp-per-row variant for C <= 256 * T: the row lives in the registers of one warp (T groups of 8
// elements per lane), statistics by shuffles only, no block-wide barrier; 8 rows per CTA.
template <int T>
__global__ void __launch_bounds__(256) ln_modulate_warp_kernel(const float *__restrict__ x, RowMap xmap, int rows, int total_rows,
                                                               int C, const float *__restrict__ shift,
                                                               const float *__restrict__ scale, long long vec_stride,
                                                               int bmul, int boff, const bf16 *__restrict__ gamma, float eps,
                                                               bf16 *__restrict__ y) {
  pdl_launch_dependents();      // nothing precedes the wait: the successor may start its own prologue right away
  pdl_wait();
  const int grow = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (grow >= total_rows) return;
  const int lane = threadIdx.x & 31;
  const int e = grow / rows, j = grow - e * rows;
  const float *xr = x + (static_cast<long long>(e * xmap.bmul + xmap.boff) * xmap.rpb + j) * C;
  bf16 *yr = y + static_cast<long long>(grow) * C;
  const int nvec = C / 8;
  float v[T][8];
  float sum = 0.f;
#pragma unroll
  for (int t = 0; t < T; ++t) {
    const int g = lane + t * 32;
    if (g < nvec) {
      const float4 a = __ldg(reinterpret_cast<const float4 *>(xr) + 2 * g), c = __ldg(reinterpret_cast<const float4 *>(xr) + 2 * g + 1);
      v[t][0] = a.x; v[t][1] = a.y; v[t][2] = a.z; v[t][3] = a.w;
      v[t][4] = c.x; v[t][5] = c.y; v[t][6] = c.z; v[t][7] = c.w;
#pragma unroll
      for (int i = 0; i < 8; ++i) sum += v[t][i];
    }
  }
  const float mean = warp_sum(sum) / C;
  float sq = 0.f;
#pragma unroll
  for (int t = 0; t < T; ++t)
    if (lane + t * 32 < nvec) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float d = v[t][i] - mean;
        sq = fmaf(d, d, sq);
      }
    }
  const float rstd = rsqrtf(warp_sum(sq) / C + eps);
  const long long voff = static_cast<long long>(e * bmul + boff) * vec_stride;
#pragma unroll
  for (int t = 0; t < T; ++t) {
    const int g = lane + t * 32;
    if (g < nvec) {
      ln_store_group(v[t], mean, rstd, gamma, scale, shift, voff, g, yr);
    }
  }
}

cudaError_t launch_ln_modulate(const float *x, RowMap xmap, int E, int rows, int C, const float *shift,
                               const float *scale, long long vec_stride, int bmul, int boff, const bf16 *gamma,
                               float eps, bf16 *y, cudaStream_t st) {
  if (E * rows <= 0) return cudaSuccess;
  if (C % 8 != 0 || C > 8 * kLnThreads * kLnMaxVec) return cudaErrorInvalidValue;
  const int total = E * rows;
  // few rows: a CTA per row finishes sooner (more threads per row); many rows: a warp per row streams better
  if (total >= 4096 && C <= 1024)
    return launch_pdl(ln_modulate_warp_kernel<4>, dim3((total + 7) / 8), dim3(256), 0, st, x, xmap, rows, total, C, shift, scale,
                      vec_stride, bmul, boff, gamma, eps, y);
  if (total >= 4096 && C <= 2048)
    return launch_pdl(ln_modulate_warp_kernel<8>, dim3((total + 7) / 8), dim3(256), 0, st, x, xmap, rows, total, C, shift, scale,
                      vec_stride, bmul, boff, gamma, eps, y);
  return launch_pdl(ln_modulate_kernel, dim3(E * rows), dim3(kLnThreads), 0, st, x, xmap, rows, C, shift, scale, vec_stride, bmul, boff, gamma,
                                                      eps, y);
}

// ------------------------------------------------------------------------------------------------
// Restoration fill: rows outside the index set take the bilinearly upsampled cached row
// (half-pixel centres, source coordinate clamped at 0, neighbours clamped at the edge).
// One warp per output row; rows inside the index set are skipped.
__global__ void __launch_bounds__(256) rtr_fill_kernel(const float *__restrict__ prev, float *__restrict__ out, int E,
                                                       int bmul, int boff, int h0, int w0, int h1, int w1, int C,
                                                       const int *__restrict__ inv, bf16 *__restrict__ xsplit, int mk) {
  pdl_wait();
  pdl_launch_dependents();
  const int M1 = h1 * w1;
  const long long gw = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  if (gw >= static_cast<long long>(E) * M1) return;
  const int e = static_cast<int>(gw / M1), i = static_cast<int>(gw - static_cast<long long>(e) * M1);
  if (inv != nullptr && inv[static_cast<long long>(e) * M1 + i] >= 0) return;
  const int b = e * bmul + boff;
  const int y = i / w1, xq = i - y * w1;
  const BilinearTap tap = bilinear_tap(y, xq, h0, w0, h1, w1);
  const int y0 = tap.y0, y1 = tap.y1, x0 = tap.x0, x1 = tap.x1;
  const float *src = prev + static_cast<long long>(b) * h0 * w0 * C;
  const float4 *p00 = reinterpret_cast<const float4 *>(src + (static_cast<long long>(y0) * w0 + x0) * C);
  const float4 *p01 = reinterpret_cast<const float4 *>(src + (static_cast<long long>(y0) * w0 + x1) * C);
  const float4 *p10 = reinterpret_cast<const float4 *>(src + (static_cast<long long>(y1) * w0 + x0) * C);
  const float4 *p11 = reinterpret_cast<const float4 *>(src + (static_cast<long long>(y1) * w0 + x1) * C);
  float4 *dst = reinterpret_cast<float4 *>(out + (static_cast<long long>(b) * M1 + i) * C);
  uint2 *hi_dst = xsplit ? reinterpret_cast<uint2 *>(xsplit + (static_cast<long long>(e) * 2 * mk + i) * C) : nullptr;
  const long long lo_off = static_cast<long long>(mk) * C / 4;      // in 4-element groups
  const float w00 = tap.w00, w01 = tap.w01, w10 = tap.w10, w11 = tap.w11;
#pragma unroll 4
  for (int c = threadIdx.x & 31; c < C / 4; c += 32) {
    const float4 a = __ldg(p00 + c), bq = __ldg(p01 + c), cq = __ldg(p10 + c), d = __ldg(p11 + c);
    float4 o;
    o.x = w00 * a.x + w01 * bq.x + w10 * cq.x + w11 * d.x;
    o.y = w00 * a.y + w01 * bq.y + w10 * cq.y + w11 * d.y;
    o.z = w00 * a.z + w01 * bq.z + w10 * cq.z + w11 * d.z;
    o.w = w00 * a.w + w01 * bq.w + w10 * cq.w + w11 * d.w;
    __stcs(dst + c, o);                          // written once, read by a later kernel: stream it
    if (hi_dst != nullptr) {
      const __nv_bfloat162 h0 = __floats2bfloat162_rn(o.x, o.y), h1 = __floats2bfloat162_rn(o.z, o.w);
      const float2 f0 = __bfloat1622float2(h0), f1 = __bfloat1622float2(h1);
      const __nv_bfloat162 l0 = __floats2bfloat162_rn(o.x - f0.x, o.y - f0.y), l1 = __floats2bfloat162_rn(o.z - f1.x, o.w - f1.y);
      hi_dst[c] = make_uint2(*reinterpret_cast<const uint32_t *>(&h0), *reinterpret_cast<const uint32_t *>(&h1));
      hi_dst[lo_off + c] = make_uint2(*reinterpret_cast<const uint32_t *>(&l0), *reinterpret_cast<const uint32_t *>(&l1));
    }
  }
}

cudaError_t launch_rtr_fill(const float *prev, float *out, int E, int bmul, int boff, int h0, int w0, int h1, int w1,
                            int C, const int *inv, bf16 *xsplit, int mk, cudaStream_t st) {
  const long long warps = static_cast<long long>(E) * h1 * w1;
  if (warps <= 0) return cudaSuccess;
  return launch_pdl(rtr_fill_kernel, dim3(static_cast<unsigned>((warps + 7) / 8)), dim3(256), 0, st, prev, out, E, bmul, boff, h0, w0, h1, w1, C,
                                                                         inv, xsplit, mk);
}

// ------------------------------------------------------------------------------------------------
// Projection drawn from a seed (Q_ij ~ N(0, 1/r), Sec. 3.3 RP of the paper).  Philox4x32-10 (Salmon et
// al., SC'11): call t, counter (t, group, scale, 0) under key (seed low, seed high), gives elements
// 4t .. 4t + 3 of Q^T flattened row-major (element n = j * M + i is Q_ij).  Uniforms u = (x + 0.5) 2^-32,
// Box-Muller on the word pairs (0, 1) and (2, 3) in fp64, one rounding to bf16.  Each value is written
// to both halves of the stored [Q^T | Q^T] row (row stride 2 * Mk).
__device__ __forceinline__ void philox_round(uint32_t (&c)[4], uint32_t k0, uint32_t k1) {
  const uint32_t hi0 = __umulhi(0xD2511F53u, c[0]), lo0 = 0xD2511F53u * c[0];
  const uint32_t hi1 = __umulhi(0xCD9E8D57u, c[2]), lo1 = 0xCD9E8D57u * c[2];
  const uint32_t n0 = hi1 ^ c[1] ^ k0, n2 = hi0 ^ c[3] ^ k1;
  c[0] = n0; c[1] = lo1; c[2] = n2; c[3] = lo0;
}

__global__ void __launch_bounds__(256) generate_projection_kernel(bf16 *__restrict__ qt, int M, int Mk, int r,
                                                                  uint32_t key0, uint32_t key1, uint32_t group,
                                                                  uint32_t scale) {
  const long long n_total = static_cast<long long>(M) * r;
  const long long t = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (4 * t >= n_total) return;
  uint32_t c[4] = {static_cast<uint32_t>(t), group, scale, 0u};
  uint32_t k0 = key0, k1 = key1;
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    philox_round(c, k0, k1);
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  const double sqrt_r = sqrt(static_cast<double>(r));
  double z[4];
#pragma unroll
  for (int a = 0; a < 4; a += 2) {
    const double u0 = (static_cast<double>(c[a]) + 0.5) * 0x1p-32, u1 = (static_cast<double>(c[a + 1]) + 0.5) * 0x1p-32;
    const double rad = sqrt(-2.0 * log(u0)), ang = (2.0 * 3.141592653589793) * u1;
    z[a] = rad * cos(ang);
    z[a + 1] = rad * sin(ang);
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const long long n = 4 * t + q;
    if (n < n_total) {
      const int j = static_cast<int>(n / M), i = static_cast<int>(n - static_cast<long long>(j) * M);
      const bf16 v = __double2bfloat16(z[q] / sqrt_r);
      qt[static_cast<long long>(j) * 2 * Mk + i] = v;
      qt[static_cast<long long>(j) * 2 * Mk + Mk + i] = v;
    }
  }
}

cudaError_t launch_generate_projection(bf16 *qt, int M, int Mk, int r, unsigned long long seed, int group, int scale,
                                       cudaStream_t st) {
  const long long calls = (static_cast<long long>(M) * r + 3) / 4;
  if (calls <= 0) return cudaSuccess;
  generate_projection_kernel<<<static_cast<unsigned>((calls + 255) / 256), 256, 0, st>>>(
      qt, M, Mk, r, static_cast<uint32_t>(seed & 0xFFFFFFFFull), static_cast<uint32_t>(seed >> 32),
      static_cast<uint32_t>(group), static_cast<uint32_t>(scale));
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// bf16 tokens -> the fp32 work stream, for the E batch elements the step computes only: computed element e is read
// at element e * smul + soff of `tok` and written at element e * bmul + boff of `x`.
__global__ void tokens_to_f32_kernel(const bf16 *__restrict__ tok, float *__restrict__ x, long long n8, long long per8,
                                     bf16 *__restrict__ xsplit, long long half8, int smul, int soff, int bmul, int boff) {
  pdl_wait();
  pdl_launch_dependents();
  const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n8) return;
  const long long e = i / per8, off = i - e * per8;
  const uint4 u = __ldg(reinterpret_cast<const uint4 *>(tok) + (e * smul + soff) * per8 + off);
  if (xsplit != nullptr) {                       // hi = the token itself, lo = 0
    uint4 *dst = reinterpret_cast<uint4 *>(xsplit) + e * 2 * half8 + off;
    dst[0] = u;
    dst[half8] = make_uint4(0u, 0u, 0u, 0u);
  }
  const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&u);
  const float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]), c = __bfloat1622float2(h[2]),
               d = __bfloat1622float2(h[3]);
  float4 *dst = reinterpret_cast<float4 *>(x) + 2 * ((e * bmul + boff) * per8 + off);
  dst[0] = make_float4(a.x, a.y, b.x, b.y);
  dst[1] = make_float4(c.x, c.y, d.x, d.y);
}

cudaError_t launch_tokens_to_f32(const bf16 *tok, float *x, int E, int M, int C, bf16 *xsplit, int mk, int smul, int soff,
                                 int bmul, int boff, cudaStream_t st) {
  const long long per8 = static_cast<long long>(M) * C / 8, n8 = static_cast<long long>(E) * per8;
  if (n8 <= 0) return cudaSuccess;
  return launch_pdl(tokens_to_f32_kernel, dim3(static_cast<unsigned>((n8 + 255) / 256)), dim3(256), 0, st, tok, x, n8, per8, xsplit,
                    static_cast<long long>(mk) * C / 8, smul, soff, bmul, boff);
}

__global__ void out_to_bf16_kernel(const float *__restrict__ x, RowMap xmap, int M, int C, bf16 *__restrict__ out) {
  pdl_wait();
  pdl_launch_dependents();
  const int e = blockIdx.y;
  const long long per = static_cast<long long>(M) * C / 8;
  const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= per) return;
  const float4 *src = reinterpret_cast<const float4 *>(x + static_cast<long long>(e * xmap.bmul + xmap.boff) * xmap.rpb * C);
  const float4 a = src[2 * i], b = src[2 * i + 1];
  __nv_bfloat162 h0 = __floats2bfloat162_rn(a.x, a.y), h1 = __floats2bfloat162_rn(a.z, a.w),
                 h2 = __floats2bfloat162_rn(b.x, b.y), h3 = __floats2bfloat162_rn(b.z, b.w);
  uint4 u = make_uint4(*reinterpret_cast<uint32_t *>(&h0), *reinterpret_cast<uint32_t *>(&h1),
                       *reinterpret_cast<uint32_t *>(&h2), *reinterpret_cast<uint32_t *>(&h3));
  reinterpret_cast<uint4 *>(out + static_cast<long long>(e) * M * C)[i] = u;
}

cudaError_t launch_out_to_bf16(const float *x, RowMap xmap, int E, int M, int C, bf16 *out, cudaStream_t st) {
  const long long per = static_cast<long long>(M) * C / 8;
  dim3 grid(static_cast<unsigned>((per + 255) / 256), E);
  return launch_pdl(out_to_bf16_kernel, dim3(grid), dim3(256), 0, st, x, xmap, M, C, out);
}

__global__ void silu_bf16_kernel(const bf16 *__restrict__ in, bf16 *__restrict__ out, long long n) {
  pdl_wait();
  pdl_launch_dependents();
  const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const float v = __bfloat162float(in[i]);
  out[i] = __float2bfloat16_rn(v / (1.0f + __expf(-v)));
}

cudaError_t launch_silu_bf16(const bf16 *in, bf16 *out, long long n, cudaStream_t st) {
  if (n <= 0) return cudaSuccess;
  return launch_pdl(silu_bf16_kernel, dim3(static_cast<unsigned>((n + 255) / 256)), dim3(256), 0, st, in, out, n);
}

// Self-test of the bounded wait every kernel of the library relies on: one thread initialises an mbarrier that
// nothing will ever signal and waits on it with the given budget.  The wait gives up, flags the status word
// (kStatusTimeout) and the kernel returns normally: no trap, no fault, the context stays usable.
__global__ void wait_selftest_kernel(long long cycles, unsigned *status) {
  __shared__ unsigned long long bar;
  __shared__ volatile int abort_flag;
  pdl_wait();
  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    mbar_fence_init();
    mbar_wait(smem_u32(&bar), 0, status, &abort_flag, wait_budget(cycles));
  }
}

cudaError_t launch_wait_selftest(long long cycles, unsigned *status, cudaStream_t st) {
  return launch_pdl(wait_selftest_kernel, dim3(1), dim3(32), 0, st, cycles, status);
}

// Asks L2 to fetch [ptr, ptr + bytes): one bulk prefetch of up to 16 KiB per thread.  The range must hold data that no
// kernel in flight writes (weights), so the requests go out before the wait that keeps stream order transitive.
__global__ void l2_prefetch_kernel(const uint8_t *__restrict__ ptr, unsigned long long bytes) {
  pdl_launch_dependents();
  const unsigned long long o = (static_cast<unsigned long long>(blockIdx.x) * blockDim.x + threadIdx.x) * 16384ull;
  if (o < bytes) {
    const unsigned long long n = bytes - o < 16384ull ? bytes - o : 16384ull;
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(ptr + o), "r"(static_cast<uint32_t>(n)) : "memory");
  }
  pdl_wait();
}

cudaError_t launch_l2_prefetch(const void *ptr, unsigned long long bytes, cudaStream_t st) {
  bytes &= ~15ull;
  if (bytes == 0) return cudaSuccess;
  const unsigned long long pieces = (bytes + 16383ull) / 16384ull;
  return launch_pdl(l2_prefetch_kernel, dim3(static_cast<unsigned>((pieces + 31) / 32)), dim3(32), 0, st,
                    static_cast<const uint8_t *>(ptr), bytes);
}

// K, V [B][L][H*D] -> cache layout K [B][H][L_cap][D], V^T [B][H][D][L_cap] (one block's worth).
__global__ void load_kv_kernel(const bf16 *__restrict__ K, const bf16 *__restrict__ V, int L, int H, int D, int L_cap,
                               bf16 *__restrict__ kc, bf16 *__restrict__ vt) {
  pdl_wait();
  pdl_launch_dependents();
  const int b = blockIdx.z, h = blockIdx.y;
  const int C = H * D;
  for (long long t = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; t < static_cast<long long>(L) * D;
       t += static_cast<long long>(gridDim.x) * blockDim.x) {
    const int l = static_cast<int>(t / D), d = static_cast<int>(t - static_cast<long long>(l) * D);
    const long long src = (static_cast<long long>(b) * L + l) * C + h * D + d;
    kc[((static_cast<long long>(b) * H + h) * L_cap + l) * D + d] = K[src];
    vt[((static_cast<long long>(b) * H + h) * D + d) * L_cap + l] = V[src];
  }
}

cudaError_t launch_load_kv(const bf16 *K, const bf16 *V, int B, int L, int H, int D, int L_cap, bf16 *kc, bf16 *vt,
                           cudaStream_t st) {
  if (L <= 0) return cudaSuccess;
  dim3 grid(static_cast<unsigned>((static_cast<long long>(L) * D + 255) / 256), H, B);
  return launch_pdl(load_kv_kernel, dim3(grid), dim3(256), 0, st, K, V, L, H, D, L_cap, kc, vt);
}

}  // namespace fvar
