// Kernels of the transition between two scale steps (the paper's Algorithm 1, "Vanilla VAR" lines;
// Eq. "var_upf", Eq. "var_downf"): R_k = Q(F_k^o), F_k = F_{k-1} + Up(R_k, (h_K, w_K)), next input =
// Down(F_k, (h_{k+1}, w_{k+1})).  Q is the nearest codeword: its scores F_k^o Z^T - |Z_v|^2 / 2 come from the
// tensor-core GEMM with the arg-max epilogue; the kernels here supply the half-norms, unpack the winning
// columns, gather + upsample + accumulate the codewords (HBM-bound, 16-byte accesses) and average the
// accumulated map down to the next scale.
#include "internal.h"
#include "ptx.cuh"

namespace fvar {

// hn[v] = |Z_v|^2 / 2 in fp32: one warp per codeword.
__global__ void __launch_bounds__(256) half_norms_kernel(const bf16 *__restrict__ Z, int V, int C, float *__restrict__ hn) {
  const int v = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (v >= V) return;
  const uint4 *row = reinterpret_cast<const uint4 *>(Z + static_cast<long long>(v) * C);
  float acc = 0.f;
  for (int g = lane; g < C / 8; g += 32) {
    const uint4 u = __ldg(row + g);
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&u);
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const float2 f = __bfloat1622float2(h[t]);
      acc = fmaf(f.x, f.x, acc);
      acc = fmaf(f.y, f.y, acc);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) hn[v] = 0.5f * acc;
}

cudaError_t launch_half_norms(const bf16 *Z, int V, int C, float *hn, cudaStream_t st) {
  if (V <= 0) return cudaSuccess;
  half_norms_kernel<<<(V + 7) / 8, 256, 0, st>>>(Z, V, C, hn);
  return cudaGetLastError();
}

// The winning column of every row out of its packed word (low half = ~column).  A row no tile wrote
// (word still zero) or a column out of range flags the status word and yields code 0.
__global__ void __launch_bounds__(256) unpack_codes_kernel(const unsigned long long *__restrict__ best, long long n, int V,
                                                           int *__restrict__ codes, unsigned *status) {
  pdl_wait();
  pdl_launch_dependents();
  const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const unsigned long long w = best[i];
  const unsigned c = 0xFFFFFFFFu - static_cast<unsigned>(w & 0xFFFFFFFFull);
  const bool bad = (w == 0ull) || c >= static_cast<unsigned>(V);
  if (bad) atomicOr(status, kStatusBadIndex);
  codes[i] = bad ? 0 : static_cast<int>(c);
}

cudaError_t launch_unpack_codes(const unsigned long long *best, long long n, int V, int *codes, unsigned *status,
                                cudaStream_t st) {
  if (n <= 0) return cudaSuccess;
  return launch_pdl(unpack_codes_kernel, dim3(static_cast<unsigned>((n + 255) / 256)), dim3(256), 0, st, best, n, V, codes, status);
}

// F[b][p][:] (+)= sum over the four bilinear neighbours of pixel p on the (h0, w0) grid of weight x
// Z[codes[b][neighbour]][:] (half-pixel centres, source coordinate clamped at 0, neighbours clamped at the
// edge: the library's Up).  One warp per target pixel; fp32 accumulator map.  C % 8 == 0.
__global__ void __launch_bounds__(256) up_accumulate_kernel(const bf16 *__restrict__ Z, const int *__restrict__ codes, int B,
                                                            int h0, int w0, int h1, int w1, int C, int overwrite,
                                                            float *__restrict__ F) {
  pdl_wait();
  pdl_launch_dependents();
  const int M1 = h1 * w1;
  const long long gw = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  if (gw >= static_cast<long long>(B) * M1) return;
  const int b = static_cast<int>(gw / M1), i = static_cast<int>(gw - static_cast<long long>(b) * M1);
  const int y = i / w1, xq = i - y * w1;
  const BilinearTap tap = bilinear_tap(y, xq, h0, w0, h1, w1);
  const int y0 = tap.y0, y1 = tap.y1, x0 = tap.x0, x1 = tap.x1;
  const int *cb = codes + static_cast<long long>(b) * h0 * w0;
  const uint4 *p00 = reinterpret_cast<const uint4 *>(Z + static_cast<long long>(__ldg(cb + y0 * w0 + x0)) * C);
  const uint4 *p01 = reinterpret_cast<const uint4 *>(Z + static_cast<long long>(__ldg(cb + y0 * w0 + x1)) * C);
  const uint4 *p10 = reinterpret_cast<const uint4 *>(Z + static_cast<long long>(__ldg(cb + y1 * w0 + x0)) * C);
  const uint4 *p11 = reinterpret_cast<const uint4 *>(Z + static_cast<long long>(__ldg(cb + y1 * w0 + x1)) * C);
  const float w00 = tap.w00, w01 = tap.w01, w10 = tap.w10, w11 = tap.w11;
  float4 *dst = reinterpret_cast<float4 *>(F + (static_cast<long long>(b) * M1 + i) * C);
  for (int g = threadIdx.x & 31; g < C / 8; g += 32) {
    const uint4 a = __ldg(p00 + g), bq = __ldg(p01 + g), cq = __ldg(p10 + g), d = __ldg(p11 + g);
    const __nv_bfloat162 *ha = reinterpret_cast<const __nv_bfloat162 *>(&a), *hb = reinterpret_cast<const __nv_bfloat162 *>(&bq);
    const __nv_bfloat162 *hc = reinterpret_cast<const __nv_bfloat162 *>(&cq), *hd = reinterpret_cast<const __nv_bfloat162 *>(&d);
    float o[8];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const float2 fa = __bfloat1622float2(ha[t]), fb = __bfloat1622float2(hb[t]);
      const float2 fc = __bfloat1622float2(hc[t]), fd = __bfloat1622float2(hd[t]);
      o[2 * t] = w00 * fa.x + w01 * fb.x + w10 * fc.x + w11 * fd.x;
      o[2 * t + 1] = w00 * fa.y + w01 * fb.y + w10 * fc.y + w11 * fd.y;
    }
    float4 lo = make_float4(o[0], o[1], o[2], o[3]), hi = make_float4(o[4], o[5], o[6], o[7]);
    if (!overwrite) {
      const float4 plo = dst[2 * g], phi = dst[2 * g + 1];
      lo.x += plo.x; lo.y += plo.y; lo.z += plo.z; lo.w += plo.w;
      hi.x += phi.x; hi.y += phi.y; hi.z += phi.z; hi.w += phi.w;
    }
    dst[2 * g] = lo;
    dst[2 * g + 1] = hi;
  }
}

cudaError_t launch_up_accumulate(const bf16 *Z, const int *codes, int B, int h0, int w0, int h1, int w1, int C,
                                 bool overwrite, float *F, cudaStream_t st) {
  const long long warps = static_cast<long long>(B) * h1 * w1;
  if (warps <= 0) return cudaSuccess;
  if (C % 8 != 0) return cudaErrorInvalidValue;
  return launch_pdl(up_accumulate_kernel, dim3(static_cast<unsigned>((warps + 7) / 8)), dim3(256), 0, st, Z, codes, B, h0, w0,
                    h1, w1, C, overwrite ? 1 : 0, F);
}

// tokens[b][q][:] = mean of F over the source cells target cell q = (y, x) of the (h1, w1) grid covers:
// rows [floor(y h0 / h1), ceil((y + 1) h0 / h1)), columns likewise ("area" resampling); bf16 out.
// One warp per target cell: the lanes walk the channels four float4 groups at a time (so that several
// loads per lane are in flight), the window cell by cell inside.  C % 4 == 0.
__global__ void __launch_bounds__(256) down_area_kernel(const float *__restrict__ F, int B, int h0, int w0, int h1, int w1,
                                                        int C, bf16 *__restrict__ tokens, int dup) {
  pdl_wait();
  pdl_launch_dependents();
  const int M1 = h1 * w1, lane = threadIdx.x & 31;
  const long long cell = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  if (cell >= static_cast<long long>(B) * M1) return;
  const int b = static_cast<int>(cell / M1), q = static_cast<int>(cell - static_cast<long long>(b) * M1);
  const int y = q / w1, x = q - y * w1;
  const int ya = (y * h0) / h1, yb = ((y + 1) * h0 + h1 - 1) / h1;
  const int xa = (x * w0) / w1, xb = ((x + 1) * w0 + w1 - 1) / w1;
  const float inv = 1.0f / static_cast<float>((yb - ya) * (xb - xa));
  const float4 *src = reinterpret_cast<const float4 *>(F + static_cast<long long>(b) * h0 * w0 * C);
  // dup: element b is written twice, as elements 2b and 2b + 1 (both branches of a CFG pair read the same tokens)
  uint2 *dst = reinterpret_cast<uint2 *>(tokens + (static_cast<long long>(dup ? 2 * b : b) * M1 + q) * C);
  const long long dup_off = static_cast<long long>(M1) * C / 4;      // one element further on, in uint2 units
  const int ngroups = C / 4, row4 = C / 4;
  for (int g0 = lane; g0 < ngroups; g0 += 128) {
    float4 acc[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int yy = ya; yy < yb; ++yy)
      for (int xx = xa; xx < xb; ++xx) {
        const float4 *cellp = src + (static_cast<long long>(yy) * w0 + xx) * row4;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int g = g0 + 32 * u;
          if (g < ngroups) {
            const float4 v = __ldg(cellp + g);
            acc[u].x += v.x; acc[u].y += v.y; acc[u].z += v.z; acc[u].w += v.w;
          }
        }
      }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int g = g0 + 32 * u;
      if (g < ngroups) {
        const __nv_bfloat162 o0 = __floats2bfloat162_rn(acc[u].x * inv, acc[u].y * inv);
        const __nv_bfloat162 o1 = __floats2bfloat162_rn(acc[u].z * inv, acc[u].w * inv);
        uint2 pk;
        pk.x = *reinterpret_cast<const uint32_t *>(&o0);
        pk.y = *reinterpret_cast<const uint32_t *>(&o1);
        dst[g] = pk;
        if (dup) dst[g + dup_off] = pk;
      }
    }
  }
}

cudaError_t launch_down_area(const float *F, int B, int h0, int w0, int h1, int w1, int C, bf16 *tokens, bool dup, cudaStream_t st) {
  if (C % 4 != 0) return cudaErrorInvalidValue;
  const long long warps = static_cast<long long>(B) * h1 * w1;
  if (warps <= 0) return cudaSuccess;
  return launch_pdl(down_area_kernel, dim3(static_cast<unsigned>((warps + 7) / 8)), dim3(256), 0, st, F, B, h0, w0, h1, w1, C,
                    tokens, dup ? 1 : 0);
}

// Classifier-free guidance on CFG pairs: out[p] = null + s (prompt - null) with (prompt, null) = elements
// (2p, 2p + 1); fp32 arithmetic on bf16 inputs, one rounding.  Eight elements per thread.
__global__ void __launch_bounds__(256) cfg_combine_kernel(const bf16 *__restrict__ pair, long long n8_per_elem, long long total8,
                                                          float s, bf16 *__restrict__ out) {
  pdl_wait();
  pdl_launch_dependents();
  const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= total8) return;
  const long long pidx = i / n8_per_elem, off = i - pidx * n8_per_elem;
  const uint4 ua = __ldg(reinterpret_cast<const uint4 *>(pair) + (2 * pidx) * n8_per_elem + off);
  const uint4 ub = __ldg(reinterpret_cast<const uint4 *>(pair) + (2 * pidx + 1) * n8_per_elem + off);
  const __nv_bfloat162 *ha = reinterpret_cast<const __nv_bfloat162 *>(&ua), *hb = reinterpret_cast<const __nv_bfloat162 *>(&ub);
  uint32_t w[4];
#pragma unroll
  for (int t = 0; t < 4; ++t) {
    const float2 a = __bfloat1622float2(ha[t]), b = __bfloat1622float2(hb[t]);
    const __nv_bfloat162 o = __floats2bfloat162_rn(fmaf(s, a.x - b.x, b.x), fmaf(s, a.y - b.y, b.y));
    w[t] = *reinterpret_cast<const uint32_t *>(&o);
  }
  reinterpret_cast<uint4 *>(out)[i] = make_uint4(w[0], w[1], w[2], w[3]);
}

cudaError_t launch_cfg_combine(const bf16 *pair, int pairs, long long per_elem, float s, bf16 *out, cudaStream_t st) {
  if (per_elem % 8 != 0) return cudaErrorInvalidValue;
  const long long total8 = static_cast<long long>(pairs) * (per_elem / 8);
  if (total8 <= 0) return cudaSuccess;
  return launch_pdl(cfg_combine_kernel, dim3(static_cast<unsigned>((total8 + 255) / 256)), dim3(256), 0, st, pair, per_elem / 8,
                    total8, s, out);
}

}  // namespace fvar
