// Kernels of the LLS restoration (Sec. 3.3 RP, Eq. "lstsq"; App. A.3): fp32 throughout.  The restoration matrices
// come out of normal equations, whose solve amplifies operand rounding by the condition number of an r x r Gram
// matrix; bf16 (or tf32) tensor-core operands would lose exactly the digits that solve needs, so these products run
// as plain fp32 FMA tiles.  Sizes are small next to the blocks' GEMMs (r <= 192 rows).
#include "internal.h"
#include "ptx.cuh"

namespace fvar {

constexpr int kSgTile = 64;      // output tile 64 x 64, 256 threads, 4 x 4 outputs each
constexpr int kSgK = 16;

// out[z][m][n] (+)= sum_k A[z][m][k] * B'[z][k][n], B' = B^T for TRANS_B (B stored [n][k], both operands K-major)
// or B (stored [k][n]).  Row pitches lda / ldb / ldo in floats; batch z at a_off + z * a_stride floats, etc.
template <bool TRANS_B>
__global__ void __launch_bounds__(256) sgemm_kernel(const float *__restrict__ A, const float *__restrict__ B, float *__restrict__ out,
                                                    int m, int n, int k, long long lda, long long ldb, long long ldo,
                                                    long long a_off, long long a_stride, long long b_off, long long b_stride,
                                                    long long o_off, long long o_stride, int accumulate) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ float sa[kSgK][kSgTile + 4];
  __shared__ float sb[kSgK][kSgTile + 4];
  const float *Az = A + a_off + blockIdx.z * a_stride;
  const float *Bz = B + b_off + blockIdx.z * b_stride;
  float *Oz = out + o_off + blockIdx.z * o_stride;
  const int m0 = blockIdx.y * kSgTile, n0 = blockIdx.x * kSgTile;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  for (int k0 = 0; k0 < k; k0 += kSgK) {
    // A tile: 64 rows x 16 k; thread t loads row t / 4, k quad t % 4
    {
      const int r = threadIdx.x >> 2, kq = (threadIdx.x & 3) * 4;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int kk = k0 + kq + u;
        sa[kq + u][r] = (m0 + r < m && kk < k) ? Az[static_cast<long long>(m0 + r) * lda + kk] : 0.f;
      }
    }
    if (TRANS_B) {
      const int r = threadIdx.x >> 2, kq = (threadIdx.x & 3) * 4;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int kk = k0 + kq + u;
        sb[kq + u][r] = (n0 + r < n && kk < k) ? Bz[static_cast<long long>(n0 + r) * ldb + kk] : 0.f;
      }
    } else {
      const int kk = threadIdx.x >> 4, c4 = (threadIdx.x & 15) * 4;
#pragma unroll
      for (int u = 0; u < 4; ++u)
        sb[kk][c4 + u] = (k0 + kk < k && n0 + c4 + u < n) ? Bz[static_cast<long long>(k0 + kk) * ldb + n0 + c4 + u] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kSgK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = sa[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = sb[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = m0 + ty * 4 + i;
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

cudaError_t launch_sgemm(bool trans_b, const float *A, const float *B, float *out, int m, int n, int k, long long lda, long long ldb,
                         long long ldo, long long a_off, long long a_stride, long long b_off, long long b_stride, long long o_off,
                         long long o_stride, int batch, bool accumulate, cudaStream_t st) {
  if (m <= 0 || n <= 0 || k <= 0 || batch <= 0) return cudaSuccess;
  dim3 grid((n + kSgTile - 1) / kSgTile, (m + kSgTile - 1) / kSgTile, batch);
  if (trans_b)
    return launch_pdl(sgemm_kernel<true>, grid, dim3(256), 0, st, A, B, out, m, n, k, lda, ldb, ldo, a_off, a_stride, b_off, b_stride,
                      o_off, o_stride, accumulate ? 1 : 0);
  return launch_pdl(sgemm_kernel<false>, grid, dim3(256), 0, st, A, B, out, m, n, k, lda, ldb, ldo, a_off, a_stride, b_off, b_stride,
                    o_off, o_stride, accumulate ? 1 : 0);
}

// Inverse of a symmetric positive definite r x r matrix (r <= kLlsMaxRank) through its Cholesky factor: one CTA per
// matrix.  G = L L^T is factorised in shared memory (right-looking, column by column); then thread c solves
// L y = e_c and L^T x = y for column c of the identity, keeping its vector in the output matrix (column c, so that the
// threads of a warp touch consecutive addresses).  A pivot that is not positive (G numerically singular) sets the
// status word's bad-index bit and is replaced by 1, so that nothing divides by zero.
__global__ void __launch_bounds__(256) chol_inverse_kernel(const float *__restrict__ G, float *__restrict__ Ginv, int r, unsigned *status) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ float L[];                       // [r][r + 1]
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
    const int rem = r - j - 1;
    for (int t = threadIdx.x; t < rem * rem; t += blockDim.x) {
      const int i = j + 1 + t / rem, k = j + 1 + t % rem;
      if (k <= i) L[i * ld + k] -= L[i * ld + j] * L[k * ld + j];
    }
    __syncthreads();
  }
  for (int c = threadIdx.x; c < r; c += blockDim.x) {
    for (int i = 0; i < r; ++i) {                    // forward: L y = e_c
      float s = (i == c) ? 1.f : 0.f;
      for (int k = c; k < i; ++k) s -= L[i * ld + k] * inv[static_cast<long long>(k) * r + c];     // y_k = 0 for k < c
      inv[static_cast<long long>(i) * r + c] = (i < c) ? 0.f : s / L[i * ld + i];
    }
    for (int i = r - 1; i >= 0; --i) {               // backward: L^T x = y
      float s = inv[static_cast<long long>(i) * r + c];
      for (int k = i + 1; k < r; ++k) s -= L[k * ld + i] * inv[static_cast<long long>(k) * r + c];
      inv[static_cast<long long>(i) * r + c] = s / L[i * ld + i];
    }
  }
}

cudaError_t lls_prepare() {
  return cudaFuncSetAttribute(chol_inverse_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              kLlsMaxRank * (kLlsMaxRank + 1) * static_cast<int>(sizeof(float)));
}

cudaError_t launch_chol_inverse(const float *G, float *Ginv, int r, int count, unsigned *status, cudaStream_t st) {
  if (r <= 0 || r > kLlsMaxRank || count <= 0) return cudaErrorInvalidValue;
  return launch_pdl(chol_inverse_kernel, dim3(count), dim3(256), static_cast<size_t>(r) * (r + 1) * sizeof(float), st, G, Ginv, r, status);
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
