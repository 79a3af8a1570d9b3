// Flash-style attention of one scale's query rows over the multi-scale KV cache, sm_100a.
//
// One CTA handles 128 query rows of one (batch element, head).  Warp 0 streams K / V^T tiles of
// 128 keys with TMA; warp 1 issues S = Q K^T and O_j = P V on the tensor cores (accumulators in
// TMEM); warps 2-5 own one query row per thread: they read S from TMEM, keep the running max and
// sum, write P (bf16) into a swizzled shared-memory tile for the second MMA, and fold each O_j
// into a register accumulator with the usual rescaling.  S is double-buffered so that Q K^T of
// block j+1 overlaps the softmax of block j.  Keys at or beyond L are masked.  Every wait is
// bounded (see ptx.cuh).
#include <math.h>

#include "internal.h"
#include "ptx.cuh"

namespace fvar {

constexpr int kAttnThreads = 192;
constexpr int kQRows = 128;
constexpr int kKeys = 128;
constexpr int kAtomBytes = 128 * 128;   // [128 rows][64 bf16] swizzled tile

template <int D>
struct AttnCfg {
  static constexpr int kStages = (D == 64) ? 4 : 2;
  static constexpr int kQBytes = kQRows * D * 2;
  static constexpr int kKBytes = kKeys * D * 2;
  static constexpr int kVBytes = D * kKeys * 2;
  static constexpr int kStageBytes = kKBytes + kVBytes;
  static constexpr int kPBytes = kQRows * kKeys * 2;
  static constexpr int kSmemBytes = kQBytes + kStages * kStageBytes + kPBytes + 1024 + 256;
  static constexpr int kTmemCols = 512;   // S0 [0,128), S1 [128,256), O [256, 256 + D)
  static_assert(kSmemBytes > 116 * 1024, "one CTA per SM (the CTA allocates all of TMEM)");
  static_assert(kSmemBytes <= 227 * 1024, "shared memory");
};

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const __grid_constant__ AttnArgs p) {
  using Cfg = AttnCfg<D>;
  constexpr int S = Cfg::kStages;
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint32_t tmem_base_holder;
  __shared__ volatile int abort_flag;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t q_smem = smem_base;
  const uint32_t kv_smem = q_smem + Cfg::kQBytes;
  const uint32_t p_smem = kv_smem + S * Cfg::kStageBytes;
  const uint32_t bar_base = p_smem + Cfg::kPBytes;
  const uint32_t q_full = bar_base;
  auto kv_full = [&](int s) { return bar_base + 8u * (1 + s); };
  auto kv_empty = [&](int s) { return bar_base + 8u * (1 + S + s); };
  auto s_full = [&](int b) { return bar_base + 8u * (1 + 2 * S + b); };
  const uint32_t p_full = bar_base + 8u * (3 + 2 * S);
  const uint32_t o_full = bar_base + 8u * (4 + 2 * S);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qt = blockIdx.x, h = blockIdx.y, e = blockIdx.z;
  const int b = e * p.bmul + p.boff;
  const int bh = b * p.H + h;
  const int nkv = (p.L + kKeys - 1) / kKeys;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(q_full, 1);
    for (int s = 0; s < S; ++s) {
      mbar_init(kv_full(s), 1);
      mbar_init(kv_empty(s), 1);
    }
    mbar_init(s_full(0), 1);
    mbar_init(s_full(1), 1);
    mbar_init(p_full, 128);
    mbar_init(o_full, 1);
    mbar_fence_init();
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmV);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_holder), Cfg::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_holder;
  const uint32_t tmem_o = tmem_base + 256;
  pdl_wait();
  pdl_launch_dependents();

  if (warp == 0) {
    if (lane == 0) {
      // ---------------------------------------------------------------- TMA producer
      mbar_expect_tx(q_full, Cfg::kQBytes);
      const int qrow0 = e * p.r + qt * kQRows;
#pragma unroll
      for (int a = 0; a < D / 64; ++a) tma_load_2d(q_smem + a * kAtomBytes, &tmQ, q_full, h * D + a * 64, qrow0);
      uint32_t armed = 0, last_parity = 0;
      bool ok = true;
      for (int j = 0; j < nkv; ++j) {
        const int stage = j % S;
        const uint32_t phase = (j / S) & 1u;
        if (!mbar_wait(kv_empty(stage), phase ^ 1u, p.status, &abort_flag)) { ok = false; break; }
        mbar_expect_tx(kv_full(stage), Cfg::kStageBytes);
        const uint32_t ks = kv_smem + stage * Cfg::kStageBytes;
        const uint32_t vs = ks + Cfg::kKBytes;
#pragma unroll
        for (int a = 0; a < D / 64; ++a) tma_load_3d(ks + a * kAtomBytes, &tmK, kv_full(stage), a * 64, j * kKeys, bh);
#pragma unroll
        for (int a = 0; a < 2; ++a) tma_load_3d(vs + a * (D * 128), &tmV, kv_full(stage), j * kKeys + a * 64, 0, bh);
        armed |= 1u << stage;
        last_parity = (last_parity & ~(1u << stage)) | (phase << stage);
      }
      if (!ok) {
        const long long t0 = clock64();
        while (!mbar_try_wait(q_full, 0) && clock64() - t0 < kWaitCycles) {}
        for (int s = 0; s < S; ++s)
          if (armed & (1u << s)) {
            const long long t1 = clock64();
            while (!mbar_try_wait(kv_full(s), (last_parity >> s) & 1u) && clock64() - t1 < kWaitCycles) {}
          }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------------------------------------------------------- MMA issuer
      constexpr uint32_t idesc_s = umma_idesc_bf16(kQRows, kKeys);
      constexpr uint32_t idesc_o = umma_idesc_bf16(kQRows, D);
      auto issue_s = [&](int j) {
        const uint32_t ks = kv_smem + (j % S) * Cfg::kStageBytes;
        const uint32_t d_tmem = tmem_base + (j & 1) * kKeys;
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint64_t da = smem_desc_sw128(q_smem + (k / 4) * kAtomBytes) + 2 * (k % 4);
          const uint64_t db = smem_desc_sw128(ks + (k / 4) * kAtomBytes) + 2 * (k % 4);
          umma_bf16(d_tmem, da, db, idesc_s, k != 0);
        }
        umma_commit(s_full(j & 1));
      };
      bool ok = mbar_wait(q_full, 0, p.status, &abort_flag);
      if (ok) ok = mbar_wait(kv_full(0), 0, p.status, &abort_flag);
      if (ok) {
        tc_fence_after();
        issue_s(0);
      }
      for (int j = 0; ok && j < nkv; ++j) {
        if (j + 1 < nkv) {
          if (!mbar_wait(kv_full((j + 1) % S), ((j + 1) / S) & 1u, p.status, &abort_flag)) { ok = false; break; }
          tc_fence_after();
          issue_s(j + 1);
        }
        if (!mbar_wait(p_full, j & 1u, p.status, &abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t vs = kv_smem + (j % S) * Cfg::kStageBytes + Cfg::kKBytes;
#pragma unroll
        for (int k = 0; k < kKeys / 16; ++k) {
          const uint64_t da = smem_desc_sw128(p_smem + (k / 4) * kAtomBytes) + 2 * (k % 4);
          const uint64_t db = smem_desc_sw128(vs + (k / 4) * (D * 128)) + 2 * (k % 4);
          umma_bf16(tmem_o, da, db, idesc_o, k != 0);
        }
        umma_commit(kv_empty(j % S));
        umma_commit(o_full);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax / accumulate
    const int quad = warp & 3;
    const int row_local = quad * 32 + lane;
    const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
    const float c = p.scale_log2;
    float o_acc[D];
#pragma unroll
    for (int i = 0; i < D; ++i) o_acc[i] = 0.f;
    float m_run = -INFINITY, l_run = 0.f, alpha_prev = 0.f;
    bool ok = true;

    auto fold_o = [&](float alpha) {          // o_acc = o_acc * alpha + O_j (from TMEM)
#pragma unroll
      for (int cc = 0; cc < D / 32; ++cc) {
        uint32_t t[32];
        tmem_ld32(tmem_o + lane_addr + cc * 32, t);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) o_acc[cc * 32 + i] = fmaf(o_acc[cc * 32 + i], alpha, __uint_as_float(t[i]));
      }
    };

    for (int j = 0; j < nkv; ++j) {
      ok = __all_sync(0xffffffffu, mbar_wait(s_full(j & 1), (j >> 1) & 1u, p.status, &abort_flag));
      if (!ok) break;
      tc_fence_after();
      const uint32_t s_addr = tmem_base + (j & 1) * kKeys + lane_addr;
      const int valid = p.L - j * kKeys;        // keys of this block below L (>= 128: all)
      float m_blk = -INFINITY;
#pragma unroll 1
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t t[32];
        tmem_ld32(s_addr + cc * 32, t);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float s = (cc * 32 + i < valid) ? __uint_as_float(t[i]) : -INFINITY;
          m_blk = fmaxf(m_blk, s);
        }
      }
      const float m_new = fmaxf(m_run, m_blk);
      const float alpha = exp2f((m_run - m_new) * c);
      const float neg_mc = -m_new * c;
      if (j > 0) {
        // O_{j-1} must be folded (and P's buffer released by the tensor core) before P_j is written.
        ok = __all_sync(0xffffffffu, mbar_wait(o_full, (j - 1) & 1u, p.status, &abort_flag));
        if (!ok) break;
        tc_fence_after();
        fold_o(alpha_prev);
      }
      float l_blk = 0.f;
#pragma unroll 1
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t t[32];
        tmem_ld32(s_addr + cc * 32, t);
        tmem_ld_wait();
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          float p0 = (cc * 32 + i < valid) ? exp2f(fmaf(__uint_as_float(t[i]), c, neg_mc)) : 0.f;
          float p1 = (cc * 32 + i + 1 < valid) ? exp2f(fmaf(__uint_as_float(t[i + 1]), c, neg_mc)) : 0.f;
          l_blk += p0 + p1;
          __nv_bfloat162 v2 = __floats2bfloat162_rn(p0, p1);
          pk[i >> 1] = *reinterpret_cast<uint32_t *>(&v2);
        }
        // columns cc*32 .. cc*32+31 of row row_local: four 16-byte chunks of the swizzled tile
        const uint32_t atom = p_smem + (cc >> 1) * kAtomBytes + row_local * 128;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint32_t chunk = static_cast<uint32_t>((cc & 1) * 4 + q);
          const uint32_t addr = atom + ((chunk ^ (row_local & 7)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(pk[q * 4]), "r"(pk[q * 4 + 1]),
                       "r"(pk[q * 4 + 2]), "r"(pk[q * 4 + 3])
                       : "memory");
        }
      }
      l_run = l_run * alpha + l_blk;
      m_run = m_new;
      alpha_prev = alpha;
      fence_proxy_async_smem();
      tc_fence_before();
      mbar_arrive(p_full);
    }
    if (ok && nkv > 0) {
      if (__all_sync(0xffffffffu, mbar_wait(o_full, (nkv - 1) & 1u, p.status, &abort_flag))) {
        tc_fence_after();
        fold_o(alpha_prev);
        const int rib = qt * kQRows + row_local;
        if (rib < p.r) {
          const float inv_l = 1.0f / l_run;
          bf16 *dst = p.out + (static_cast<long long>(e) * p.r + rib) * (p.H * D) + h * D;
#pragma unroll
          for (int q = 0; q < D / 8; ++q) {
            uint32_t w[4];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
              __nv_bfloat162 v2 = __floats2bfloat162_rn(o_acc[q * 8 + t * 2] * inv_l, o_acc[q * 8 + t * 2 + 1] * inv_l);
              w[t] = *reinterpret_cast<uint32_t *>(&v2);
            }
            reinterpret_cast<uint4 *>(dst)[q] = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
}

template <int D>
static cudaError_t set_attr() {
  static bool attr_set = false;
  if (attr_set) return cudaSuccess;
  cudaError_t err = cudaFuncSetAttribute(attention_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         AttnCfg<D>::kSmemBytes);
  if (err == cudaSuccess) attr_set = true;
  return err;
}

cudaError_t attention_prepare() {
  cudaError_t e = set_attr<64>();
  if (e == cudaSuccess) e = set_attr<128>();
  return e;
}

template <int D>
static cudaError_t launch_d(const CUtensorMap &tmQ, const CUtensorMap &tmK, const CUtensorMap &tmV, const AttnArgs &a,
                            cudaStream_t st) {
  using Cfg = AttnCfg<D>;
  cudaError_t err = set_attr<D>();
  if (err != cudaSuccess) return err;
  dim3 grid((a.r + kQRows - 1) / kQRows, a.H, a.B_eff);
  return launch_pdl(attention_kernel<D>, grid, dim3(kAttnThreads), Cfg::kSmemBytes, st, tmQ, tmK, tmV, a);
}

cudaError_t launch_attention(const CUtensorMap &tmQ, const CUtensorMap &tmK, const CUtensorMap &tmV,
                             const AttnArgs &a, cudaStream_t st) {
  if (a.r <= 0 || a.L <= 0) return cudaErrorInvalidValue;
  if (a.D == 64) return launch_d<64>(tmQ, tmK, tmV, a, st);
  if (a.D == 128) return launch_d<128>(tmQ, tmK, tmV, a, st);
  return cudaErrorInvalidValue;
}

}  // namespace fvar
