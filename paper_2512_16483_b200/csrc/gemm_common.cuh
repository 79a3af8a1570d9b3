// Epilogue code shared by the tensor-core GEMM kernels: bias, tanh-GELU, gate + residual, the
// QKV / KV-cache split and warp-wide row-segment stores through a shared-memory staging tile.
#pragma once
#include <math.h>
#include "internal.h"
#include "ptx.cuh"

namespace fvar {

constexpr int kBlockM = 128;
constexpr int kBlockK = 64;             // 64 bf16 = one 128-byte swizzle row (one "atom" along K)
// Epilogue warps per CTA: a warp can only read the 32 TMEM lanes of its quadrant (warp index mod 4), so
// the warps come in groups of four; each group takes every kEpiColGroups-th 32-column chunk of a tile.
constexpr int kEpiWarps = 8;
constexpr int kEpiColGroups = kEpiWarps / 4;

__device__ __forceinline__ float gelu_tanh_f(float x) {
  const float k0 = 0.7978845608028654f, k1 = 0.044715f;
  float u = k0 * (x + k1 * x * x * x);
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
  return 0.5f * x * (1.0f + t);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

// Warp-wide row-major stores through a 4 KiB shared-memory staging tile.  After tcgen05.ld each lane
// holds 32 consecutive columns of its own row; storing those directly makes every instruction touch
// 32 different rows 16 bytes at a time.  Instead the lanes park their pieces in shared memory (16-byte
// chunks XOR-swizzled by row, conflict-free both ways) and the warp writes whole 128-byte (fp32) or
// 64-byte (bf16) row segments, 4 or 8 rows per instruction.  `dst` is this lane's row segment (nullptr:
// row past the end); every lane of the warp must call.
__device__ __forceinline__ void warp_store_f32(uint32_t stage, int lane, const float (&v)[32], float *dst) {
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    const uint32_t addr = stage + lane * 128 + ((q ^ (lane & 7)) << 4);
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v[q * 4]), "f"(v[q * 4 + 1]), "f"(v[q * 4 + 2]),
                 "f"(v[q * 4 + 3]) : "memory");
  }
  __syncwarp();
  const int c = lane & 7;
#pragma unroll
  for (int it = 0; it < 8; ++it) {
    const int r = it * 4 + (lane >> 3);
    float4 o;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(o.x), "=f"(o.y), "=f"(o.z), "=f"(o.w)
                 : "r"(stage + r * 128 + ((c ^ (r & 7)) << 4)));
    float *pr = reinterpret_cast<float *>(__shfl_sync(0xffffffffu, reinterpret_cast<unsigned long long>(dst), r));
    if (pr != nullptr) reinterpret_cast<float4 *>(pr)[c] = o;
  }
  __syncwarp();
}

__device__ __forceinline__ void warp_store_bf16(uint32_t stage, int lane, const float (&v)[32], bf16 *dst) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const uint32_t addr = stage + lane * 64 + ((q ^ ((lane >> 1) & 3)) << 4);
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(pack_bf16(v[q * 8], v[q * 8 + 1])),
                 "r"(pack_bf16(v[q * 8 + 2], v[q * 8 + 3])), "r"(pack_bf16(v[q * 8 + 4], v[q * 8 + 5])),
                 "r"(pack_bf16(v[q * 8 + 6], v[q * 8 + 7])) : "memory");
  }
  __syncwarp();
  const int c = lane & 3;
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    const int r = it * 8 + (lane >> 2);
    uint4 o;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(o.x), "=r"(o.y), "=r"(o.z), "=r"(o.w)
                 : "r"(stage + r * 64 + ((c ^ ((r >> 1) & 3)) << 4)));
    bf16 *pr = reinterpret_cast<bf16 *>(__shfl_sync(0xffffffffu, reinterpret_cast<unsigned long long>(dst), r));
    if (pr != nullptr) reinterpret_cast<uint4 *>(pr)[c] = o;
  }
  __syncwarp();
}

// Epilogue of one warp for 32 rows x 32 consecutive columns starting at col0 (col0 % 32 == 0): each
// lane owns one row (`valid` false: row past the end).  Every lane of the warp must call.
template <int EPI>
__device__ __forceinline__ void epilogue_chunk(const GemmArgs &p, const uint32_t (&acc)[32], int batch, int row,
                                               int col0, bool valid, uint32_t stage, int lane,
                                               const float4 *resid_pre = nullptr) {
  float v[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(acc[i]);
  const bool full = (col0 + 32 <= p.N);
  if (p.bias != nullptr) {
    if (full) {
      const uint4 *bp = reinterpret_cast<const uint4 *>(p.bias + col0);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint4 u = __ldg(bp + q);
        const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&u);
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          float2 f = __bfloat1622float2(h[t]);
          v[q * 8 + t * 2] += f.x;
          v[q * 8 + t * 2 + 1] += f.y;
        }
      }
    } else {
      for (int i = 0; i < 32; ++i)
        if (col0 + i < p.N) v[i] += __bfloat162float(p.bias[col0 + i]);
    }
  }
  const long long grow = static_cast<long long>(batch) * p.R + row;   // row in the flattened output

  if constexpr (EPI == EPI_F32) {
    float *dst = p.out_f32 + grow * p.ld_out + col0;
    if (full && (p.ld_out & 3) == 0) {            // uniform across the warp
      warp_store_f32(stage, lane, v, valid ? dst : nullptr);
    } else if (valid) {
      for (int i = 0; i < 32; ++i)
        if (col0 + i < p.N) dst[i] = v[i];
    }
  } else if constexpr (EPI == EPI_BF16 || EPI == EPI_GELU_BF16) {
    if constexpr (EPI == EPI_GELU_BF16) {
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = gelu_tanh_f(v[i]);
    }
    warp_store_bf16(stage, lane, v, valid ? p.out_bf16 + grow * p.ld_out + col0 : nullptr);
  } else if constexpr (EPI == EPI_ARGMAX) {
    if (valid) {
      float best_v = -INFINITY;
      int best_c = -1;
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const int c = col0 + i;
        if (c < p.N) {
          float sc = v[i] - __ldg(p.col_sub + c);
          if (sc != sc) sc = -INFINITY;         // NaN never wins
          if (sc > best_v || best_c < 0) {      // strict: the lowest column wins a tie
            best_v = sc;
            best_c = c;
          }
        }
      }
      if (best_c >= 0) {
        const unsigned u = __float_as_uint(best_v);
        const unsigned key = (u & 0x80000000u) ? ~u : (u | 0x80000000u);  // unsigned order = float order
        atomicMax(p.best + grow, (static_cast<unsigned long long>(key) << 32) | (0xFFFFFFFFu - static_cast<unsigned>(best_c)));
      }
    }
  } else if constexpr (EPI == EPI_QKV) {
    const int e = row / p.rows_per_batch, j = row - e * p.rows_per_batch;
    const int b = e * p.bmul + p.boff;
    const int vc = col0 + p.col_base;             // uniform across the warp
    if (vc < p.C) {
      warp_store_bf16(stage, lane, v, valid ? p.out_bf16 + static_cast<long long>(row) * p.ld_out + vc : nullptr);
    } else if (vc < 2 * p.C) {
      const int c = vc - p.C, h = c / p.D, d0 = c - h * p.D;
      bf16 *base = p.kc + ((static_cast<long long>(b) * p.H + h) * p.L_cap + p.L_prev + j) * p.D + d0;
      warp_store_bf16(stage, lane, v, valid ? base : nullptr);
    } else if (valid) {
      // transposed V cache: consecutive rows of the warp are consecutive addresses already
      const int c = vc - 2 * p.C, h = c / p.D, d0 = c - h * p.D;
      bf16 *base = p.vt + ((static_cast<long long>(b) * p.H + h) * p.D + d0) * p.L_cap + p.L_prev + j;
#pragma unroll
      for (int i = 0; i < 32; ++i) base[static_cast<long long>(i) * p.L_cap] = __float2bfloat16_rn(v[i]);
    }
  } else {  // EPI_RESID
    float *dst = nullptr;
    if (valid) {
      const int e = row / p.rows_per_batch, j = row - e * p.rows_per_batch;
      const int b = e * p.bmul + p.boff;
      const float *res = p.resid + (static_cast<long long>(e * p.rmap.bmul + p.rmap.boff) * p.rmap.rpb + j) * p.ld_out + col0;
      const int jo = p.scatter ? __ldg(p.scatter + static_cast<long long>(e) * p.rows_per_batch + j) : j;
      dst = p.out_f32 + (static_cast<long long>(e * p.omap.bmul + p.omap.boff) * p.omap.rpb + jo) * p.ld_out + col0;
      const float *g = p.gate ? p.gate + static_cast<long long>(b) * p.gate_stride + col0 : nullptr;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        float4 r4 = resid_pre ? resid_pre[q] : reinterpret_cast<const float4 *>(res)[q];
        float4 g4 = g ? __ldg(reinterpret_cast<const float4 *>(g) + q) : make_float4(1.f, 1.f, 1.f, 1.f);
        v[q * 4] = fmaf(g4.x, v[q * 4], r4.x);
        v[q * 4 + 1] = fmaf(g4.y, v[q * 4 + 1], r4.y);
        v[q * 4 + 2] = fmaf(g4.z, v[q * 4 + 2], r4.z);
        v[q * 4 + 3] = fmaf(g4.w, v[q * 4 + 3], r4.w);
      }
    }
    warp_store_f32(stage, lane, v, dst);
    if (p.xsplit != nullptr) {                   // uniform across the grid
      bf16 *hi = nullptr;
      if (valid) {
        const int e = row / p.rows_per_batch, j = row - e * p.rows_per_batch;
        const int jo = p.scatter ? __ldg(p.scatter + static_cast<long long>(e) * p.rows_per_batch + j) : j;
        hi = p.xsplit + (static_cast<long long>(e) * 2 * p.xsplit_mk + jo) * p.ld_out + col0;
      }
      float lo[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) lo[i] = v[i] - __bfloat162float(__float2bfloat16_rn(v[i]));
      warp_store_bf16(stage, lane, v, hi);
      warp_store_bf16(stage, lane, lo, hi ? hi + static_cast<long long>(p.xsplit_mk) * p.ld_out : nullptr);
    }
  }
}

}  // namespace fvar
