// Kernels of the LLS restoration (Sec. 3.3 RP, Eq. "lstsq"; App. A.3): fp32 throughout.  The restoration matrices
// come out of normal equations, whose solve amplifies operand rounding by the condition number of an r x r Gram
// matrix; bf16 (or tf32) tensor-core operands would lose exactly the digits that solve needs, so these products run
// as plain fp32 FMA tiles.  Sizes are small next to the blocks' GEMMs (r <= 192 rows).
#include "internal.h"
#include "ptx.cuh"

namespace fvar {

constexpr int kSgM = 128, kSgN = 64, kSgK = 16;      // output tile 128 x 64, 256 threads, 8 x 4 outputs each

// out[z][m][n] (+)= sum_k A[z][m][k] * B'[z][k][n], B' = B^T for TRANS_B (B stored [n][k], both operands K-major)
// or B (stored [k][n]).  Row pitches lda / ldb / ldo in floats; batch z at a_off + z * a_stride floats, etc.
template <bool TRANS_B>
__global__ void __launch_bounds__(256) sgemm_kernel(const float *__restrict__ A, const float *__restrict__ B, float *__restrict__ out,
                                                    int m, int n, int k, long long lda, long long ldb, long long ldo,
                                                    long long a_off, long long a_stride, long long b_off, long long b_stride,
                                                    long long o_off, long long o_stride, int accumulate, int ksplit, int kchunk) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ __align__(16) float sa[kSgK][kSgM + 4];
  __shared__ __align__(16) float sb[kSgK][kSgN + 4];
  // blockIdx.z = batch * ksplit + s: K range s of the batch's product goes to partial result z (o_stride apart); the
  // partials are added afterwards in order of s (sum_partials_kernel), so the result does not depend on timing
  const int zb = blockIdx.z / ksplit, zs = blockIdx.z - zb * ksplit;
  const long long koff = static_cast<long long>(zs) * kchunk;
  const float *Az = A + a_off + zb * a_stride + koff;
  const float *Bz = B + b_off + zb * b_stride + (TRANS_B ? koff : koff * ldb);
  float *Oz = out + o_off + (ksplit > 1 ? static_cast<long long>(blockIdx.z) : static_cast<long long>(zb)) * o_stride;
  k = min(k - zs * kchunk, kchunk);
  const int m0 = blockIdx.y * kSgM, n0 = blockIdx.x * kSgN;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;      // outputs: rows ty * 8 .. + 7, columns tx * 4 .. + 3
  float acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  const int lk = threadIdx.x & 15, lr = threadIdx.x >> 4;      // loads: K index lk of rows lr, lr + 16, ...
  for (int k0 = 0; k0 < k; k0 += kSgK) {
    const bool kin = k0 + lk < k;
#pragma unroll
    for (int i = 0; i < kSgM / 16; ++i) {
      const int r = lr + 16 * i;
      sa[lk][r] = (kin && m0 + r < m) ? Az[static_cast<long long>(m0 + r) * lda + k0 + lk] : 0.f;
    }
    if (TRANS_B) {
#pragma unroll
      for (int i = 0; i < kSgN / 16; ++i) {
        const int c = lr + 16 * i;
        sb[lk][c] = (kin && n0 + c < n) ? Bz[static_cast<long long>(n0 + c) * ldb + k0 + lk] : 0.f;
      }
    } else {
      const int c = threadIdx.x & 63, kk0 = threadIdx.x >> 6;
#pragma unroll
      for (int i = 0; i < kSgK / 4; ++i) {
        const int kk = kk0 + 4 * i;
        sb[kk][c] = (k0 + kk < k && n0 + c < n) ? Bz[static_cast<long long>(k0 + kk) * ldb + n0 + c] : 0.f;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kSgK; ++kk) {
      const float4 a0 = *reinterpret_cast<const float4 *>(&sa[kk][ty * 8]), a1 = *reinterpret_cast<const float4 *>(&sa[kk][ty * 8 + 4]);
      const float4 b4 = *reinterpret_cast<const float4 *>(&sb[kk][tx * 4]);
      const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = m0 + ty * 8 + i;
    if (row >= m) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int col = n0 + tx * 4 + j;
      if (col < n) {
        float *o = Oz + static_cast<long long>(row) * ldo + col;
        *o = accumulate ? *o + acc[i][j] : acc[i][j];
      }
    }
  }
}

// out[i] = sum over s < ksplit of partial[(i / per) * ksplit + s][i % per], s in order.
__global__ void __launch_bounds__(256) sum_partials_kernel(const float *__restrict__ partial, float *__restrict__ out, long long per,
                                                           long long o_off, long long o_stride, long long ldo, int n, int ksplit,
                                                           long long total) {
  pdl_wait();
  pdl_launch_dependents();
  const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const long long z = i / per, off = i - z * per;
  float acc = 0.f;
  for (int s2 = 0; s2 < ksplit; ++s2) acc += partial[(z * ksplit + s2) * per + off];
  out[o_off + z * o_stride + (off / n) * ldo + off % n] = acc;
}

// ksplit > 1: the K range is cut into ksplit pieces whose partial products go through `scratch` (batch * ksplit * m * n
// floats) and are then added in order; for products with few output tiles and a long reduction.
cudaError_t launch_sgemm(bool trans_b, const float *A, const float *B, float *out, int m, int n, int k, long long lda, long long ldb,
                         long long ldo, long long a_off, long long a_stride, long long b_off, long long b_stride, long long o_off,
                         long long o_stride, int batch, bool accumulate, cudaStream_t st, int ksplit, float *scratch) {
  if (m <= 0 || n <= 0 || k <= 0 || batch <= 0) return cudaSuccess;
  if (ksplit < 1 || scratch == nullptr || accumulate) ksplit = 1;
  int kchunk = ((k + ksplit - 1) / ksplit + kSgK - 1) / kSgK * kSgK;
  ksplit = (k + kchunk - 1) / kchunk;
  if (ksplit == 1) kchunk = k;
  dim3 grid((n + kSgN - 1) / kSgN, (m + kSgM - 1) / kSgM, batch * ksplit);
  float *dst = ksplit > 1 ? scratch : out;
  const long long d_ld = ksplit > 1 ? n : ldo, d_off = ksplit > 1 ? 0 : o_off, d_stride = ksplit > 1 ? static_cast<long long>(m) * n : o_stride;
  cudaError_t e;
  if (trans_b)
    e = launch_pdl(sgemm_kernel<true>, grid, dim3(256), 0, st, A, B, dst, m, n, k, lda, ldb, d_ld, a_off, a_stride, b_off, b_stride,
                   d_off, d_stride, accumulate ? 1 : 0, ksplit, kchunk);
  else
    e = launch_pdl(sgemm_kernel<false>, grid, dim3(256), 0, st, A, B, dst, m, n, k, lda, ldb, d_ld, a_off, a_stride, b_off, b_stride,
                   d_off, d_stride, accumulate ? 1 : 0, ksplit, kchunk);
  if (e != cudaSuccess || ksplit == 1) return e;
  const long long per = static_cast<long long>(m) * n, total = per * batch;
  return launch_pdl(sum_partials_kernel, dim3(static_cast<unsigned>((total + 255) / 256)), dim3(256), 0, st,
                    static_cast<const float *>(scratch), out, per, o_off, o_stride, ldo, n, ksplit, total);
}

__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Inverse of a symmetric positive definite r x r matrix (r <= kLlsMaxRank) through its Cholesky factor.  Every CTA
// (blockIdx.x: the matrix, blockIdx.y: a group of eight columns of the inverse) factorises G = L L^T in shared memory
// (right-looking, column by column; redundant across the CTAs of a matrix, r^3 / 3 operations), then each warp solves
// L y = e_c and L^T x = y for one column c of the identity, the lanes sharing every row's dot product.  A pivot that is not positive (G numerically singular) sets the
// status word's bad-index bit and is replaced by 1, so that nothing divides by zero.
__global__ void __launch_bounds__(256) chol_inverse_kernel(const float *__restrict__ G, float *__restrict__ Ginv, int r, unsigned *status) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ float L[];                       // [r][r + 1], then eight solution vectors of r floats
  const int ld = r + 1;
  const float *g = G + static_cast<long long>(blockIdx.x) * r * r;
  float *inv = Ginv + static_cast<long long>(blockIdx.x) * r * r;
  for (int i = threadIdx.x; i < r * r; i += blockDim.x) L[(i / r) * ld + (i % r)] = g[i];
  __syncthreads();
  for (int j = 0; j < r; ++j) {
    if (threadIdx.x == 0) {
      float d = L[j * ld + j];
      if (!(d > 0.f)) { atomicOr(status, kStatusBadIndex); d = 1.f; }
      L[j * ld + j] = sqrtf(d);
    }
    __syncthreads();
    const float djj = L[j * ld + j];
    for (int i = j + 1 + threadIdx.x; i < r; i += blockDim.x) L[i * ld + j] /= djj;
    __syncthreads();
    // trailing update: L[i][k] -= L[i][j] * L[k][j] for j < k <= i
    for (int i = j + 1 + (threadIdx.x >> 5); i < r; i += blockDim.x >> 5) {      // a warp per row, lanes over the columns
      const float lij = L[i * ld + j];
      for (int k = j + 1 + (threadIdx.x & 31); k <= i; k += 32) L[i * ld + k] -= lij * L[k * ld + j];
    }
    __syncthreads();
  }
  // Columns of the inverse: blockIdx.y picks eight of them, one per warp; the lanes share each row's dot product.
  float *vec = L + r * ld + (threadIdx.x >> 5) * r;    // this warp's solution vector (shared memory)
  const int c = blockIdx.y * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (c < r) {
    for (int i = 0; i < r; ++i) {                      // forward: L y = e_c (y_k = 0 for k < c)
      float s = 0.f;
      for (int k = c + lane; k < i; k += 32) s += L[i * ld + k] * vec[k];
      s = warp_sum_f(s);
      if (lane == 0) vec[i] = (i < c) ? 0.f : (((i == c) ? 1.f : 0.f) - s) / L[i * ld + i];
      __syncwarp();
    }
    for (int i = r - 1; i >= 0; --i) {                 // backward: L^T x = y
      float s = 0.f;
      for (int k = i + 1 + lane; k < r; k += 32) s += L[k * ld + i] * vec[k];
      s = warp_sum_f(s);
      if (lane == 0) vec[i] = (vec[i] - s) / L[i * ld + i];
      __syncwarp();
    }
    for (int i = lane; i < r; i += 32) inv[static_cast<long long>(i) * r + c] = vec[i];
  }
}

cudaError_t lls_prepare() {
  return cudaFuncSetAttribute(chol_inverse_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              kLlsMaxRank * (kLlsMaxRank + 9) * static_cast<int>(sizeof(float)));
}

cudaError_t launch_chol_inverse(const float *G, float *Ginv, int r, int count, unsigned *status, cudaStream_t st) {
  if (r <= 0 || r > kLlsMaxRank || count <= 0) return cudaErrorInvalidValue;
  return launch_pdl(chol_inverse_kernel, dim3(count, (r + 7) / 8), dim3(256), static_cast<size_t>(r) * (r + 9) * sizeof(float), st, G, Ginv,
                    r, status);
}

// fp32 rows -> their two-term bf16 split in the [E][2][mk][C] layout (hi = bf16(x), lo = bf16(x - hi)).
__global__ void __launch_bounds__(256) split_rows_kernel(const float *__restrict__ x, long long x_off, long long x_stride, int M, int C,
                                                         bf16 *__restrict__ xsplit, int mk) {
  pdl_wait();
  pdl_launch_dependents();
  const int e = blockIdx.y;
  const long long per4 = static_cast<long long>(M) * C / 4;
  const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= per4) return;
  const float4 v = reinterpret_cast<const float4 *>(x + x_off + e * x_stride)[i];
  const float f[4] = {v.x, v.y, v.z, v.w};
  bf16 hi[4], lo[4];
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    hi[u] = __float2bfloat16_rn(f[u]);
    lo[u] = __float2bfloat16_rn(f[u] - __bfloat162float(hi[u]));
  }
  bf16 *dst = xsplit + static_cast<long long>(e) * 2 * mk * C + i * 4;
  *reinterpret_cast<uint2 *>(dst) = *reinterpret_cast<const uint2 *>(hi);
  *reinterpret_cast<uint2 *>(dst + static_cast<long long>(mk) * C) = *reinterpret_cast<const uint2 *>(lo);
}

cudaError_t launch_split_rows(const float *x, long long x_off, long long x_stride, int E, int M, int C, bf16 *xsplit, int mk,
                              cudaStream_t st) {
  const long long per4 = static_cast<long long>(M) * C / 4;
  if (per4 <= 0 || E <= 0) return cudaSuccess;
  return launch_pdl(split_rows_kernel, dim3(static_cast<unsigned>((per4 + 255) / 256), E), dim3(256), 0, st, x, x_off, x_stride, M, C,
                    xsplit, mk);
}

}  // namespace fvar
