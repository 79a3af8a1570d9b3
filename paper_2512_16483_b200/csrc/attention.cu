// Flash-style attention of one scale's query rows over the multi-scale KV cache, sm_100a.
//
// One CTA handles up to 256 query rows (two tiles of 128) of one (batch element, head).
//   warp 0      streams K and V^T tiles of 128 keys through a ring of shared-memory slots (TMA);
//   warp 1      issues S_t = Q_t K^T and O_t += P_t V on the tensor cores, accumulators in TMEM;
//   warps 2-5   softmax of tile 0, one query row per thread;   warps 6-9: softmax of tile 1.
// The two tiles run out of phase: while one warp-group turns S into P (row max, exp2, bf16 P
// written back into the TMEM columns S came from), the tensor core works for the other tile (P V of
// block j, with P read from TMEM as the A operand, then Q K^T of block j+1).  Keeping P out of shared
// memory matters: the operand reads of the MMAs alone nearly fill the 128 B/clk of shared-memory
// bandwidth, and a P tile costs one write and one read on top.  O stays in TMEM for the whole key loop; its rows are rescaled only when the
// running maximum has grown by more than 2^8 since the last rescale, so the common case costs no
// TMEM round trip.  Keys at or beyond L are masked.  Every wait is bounded (see ptx.cuh).
//
// Few queries over a long cache (few CTAs, many key blocks): the key range is split over a thread-block cluster of
// up to 6 CTAs.  Each parks its unnormalised (O, m, l) in its own shared memory; after a cluster barrier every
// CTA merges a slice of the query rows over all ranges through distributed shared memory, in range order (the
// result does not depend on timing), normalises and stores.  Nothing goes through global scratch.
#include <math.h>

#include "internal.h"
#include "ptx.cuh"

namespace fvar {

constexpr int kAttnThreads = 320;
constexpr int kQRows = 128;
constexpr int kKeys = 128;
constexpr int kAtomBytes = 128 * 128;   // [128 rows][64 bf16] swizzled tile
constexpr float kRescaleThreshold = 8.0f;   // log2 units

template <int D>
struct AttnCfg {
  static constexpr int kTileBytes = 128 * D * 2;          // a Q tile, a K tile [128 keys][D] or a V^T tile [D][128 keys]
  static constexpr int kRing = (D == 64) ? 10 : 5;        // K_j, V_j, K_{j+1}, ...
  static constexpr int kQBytes = 2 * kTileBytes;
  static constexpr int kSmemBytes = kQBytes + kRing * kTileBytes + 1024 + 256;
  // TMEM: S0 [0,128), S1 [128,256), O0 [256,256+D), O1 [256+D,256+2D).  P (bf16, two keys per 32-bit
  // column) overwrites columns [0,64) of the S buffer it was computed from.
  static constexpr int kTmemCols = 512;
  static_assert(kSmemBytes > 116 * 1024, "one CTA per SM (the CTA allocates all of TMEM)");
  static_assert(kSmemBytes + 64 <= 227 * 1024, "shared memory");
  static_assert(256 + 2 * D <= 512, "TMEM columns");
};

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const __grid_constant__ AttnArgs p) {
  using Cfg = AttnCfg<D>;
  constexpr int NR = Cfg::kRing;
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint32_t tmem_base_holder;
  __shared__ volatile int abort_flag;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t q_smem = smem_base;
  const uint32_t ring_smem = q_smem + Cfg::kQBytes;
  const uint32_t bar_base = ring_smem + NR * Cfg::kTileBytes;
  const uint32_t q_full = bar_base;
  auto ring_full = [&](int s) { return bar_base + 8u * (1 + s); };
  auto ring_empty = [&](int s) { return bar_base + 8u * (1 + NR + s); };
  auto s_full = [&](int t) { return bar_base + 8u * (1 + 2 * NR + t); };
  auto p_full = [&](int t) { return bar_base + 8u * (3 + 2 * NR + t); };
  auto o_full = [&](int t) { return bar_base + 8u * (5 + 2 * NR + t); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long wb = wait_budget(p.wait_cycles);
  // kv_splits CTAs (one cluster) share a query tile pair, each covering a contiguous range of key blocks.
  const int splits = p.kv_splits > 1 ? p.kv_splits : 1;
  const int qt = blockIdx.x / splits, sp = blockIdx.x - qt * splits, h = blockIdx.y, e = blockIdx.z;   // sp = rank in the cluster
  const int b = e * p.bmul + p.boff;
  const int bh = b * p.H + h;
  const int nkv_total = (p.L + kKeys - 1) / kKeys;
  const int kv_per = (nkv_total + splits - 1) / splits;
  const int jb0 = sp * kv_per;                                    // first key block of this CTA
  const int nkv = min(kv_per, nkv_total - jb0);                   // >= 1: the host sizes splits so
  const int tpc = p.tiles_per_cta == 1 ? 1 : 2;                   // query tiles a CTA takes: two, or one when CTAs are scarce
  const int q0 = qt * tpc * kQRows;                               // first query row of this CTA within its element
  const int ntiles = (tpc == 2 && p.r - q0 > kQRows) ? 2 : 1;     // query tiles this CTA really has

  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(q_full, 1);
    for (int s = 0; s < NR; ++s) {
      mbar_init(ring_full(s), 1);
      mbar_init(ring_empty(s), 1);
    }
    for (int t = 0; t < 2; ++t) {
      mbar_init(s_full(t), 1);
      mbar_init(p_full(t), 128);
      mbar_init(o_full(t), 1);
    }
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
  pdl_launch_dependents();      // the successor (a GEMM) only requests weights before its own wait
  pdl_wait();
  float m_ref = -INFINITY, l_run = 0.f;      // softmax threads: running maximum and sum of this thread's query row
  bool final_ok = false;                      // softmax threads: the last P V of the row's tile has completed

  if (warp == 0) {
    if (lane == 0) {
      // ---------------------------------------------------------------- TMA producer
      mbar_expect_tx(q_full, ntiles * Cfg::kTileBytes);
      const int qrow0 = e * p.r + q0;
      for (int t = 0; t < ntiles; ++t)
#pragma unroll
        for (int a = 0; a < D / 64; ++a)
          tma_load_2d(q_smem + t * Cfg::kTileBytes + a * kAtomBytes, &tmQ, q_full, h * D + a * 64, qrow0 + t * kQRows);
      uint32_t armed = 0, last_parity = 0;
      bool ok = true;
      for (int i = 0; i < 2 * nkv; ++i) {            // even i: K of block i/2, odd i: V^T of block i/2
        const int slot = i % NR, j = i >> 1;
        const uint32_t phase = (i / NR) & 1u;
        if (!mbar_wait(ring_empty(slot), phase ^ 1u, p.status, &abort_flag, wb)) { ok = false; break; }
        mbar_expect_tx(ring_full(slot), Cfg::kTileBytes);
        const uint32_t dst = ring_smem + slot * Cfg::kTileBytes;
        if ((i & 1) == 0) {
#pragma unroll
          for (int a = 0; a < D / 64; ++a) tma_load_3d(dst + a * kAtomBytes, &tmK, ring_full(slot), a * 64, (jb0 + j) * kKeys, bh);
        } else {
#pragma unroll
          for (int a = 0; a < 2; ++a) tma_load_3d(dst + a * (D * 128), &tmV, ring_full(slot), (jb0 + j) * kKeys + a * 64, 0, bh);
        }
        armed |= 1u << slot;
        last_parity = (last_parity & ~(1u << slot)) | (phase << slot);
      }
      if (!ok) {   // let every copy that was issued land before the shared memory is released
        const long long t0 = clock64();
        while (!mbar_try_wait(q_full, 0) && clock64() - t0 < kWaitCycles) {}
        for (int s = 0; s < NR; ++s)
          if (armed & (1u << s)) {
            const long long t1 = clock64();
            while (!mbar_try_wait(ring_full(s), (last_parity >> s) & 1u) && clock64() - t1 < kWaitCycles) {}
          }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------------------------------------------------------- MMA issuer
      constexpr uint32_t idesc_s = umma_idesc_bf16(kQRows, kKeys);
      constexpr uint32_t idesc_o = umma_idesc_bf16(kQRows, D);
      auto issue_s = [&](int t, int buf, int slot) {   // S buffer `buf` = Q_t K^T
        const uint32_t ks = ring_smem + slot * Cfg::kTileBytes, qs = q_smem + t * Cfg::kTileBytes;
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint64_t da = smem_desc_sw128(qs + (k / 4) * kAtomBytes) + 2 * (k % 4);
          const uint64_t db = smem_desc_sw128(ks + (k / 4) * kAtomBytes) + 2 * (k % 4);
          umma_bf16(tmem_base + buf * kKeys, da, db, idesc_s, k != 0);
        }
        umma_commit(s_full(buf));
      };
      auto issue_pv = [&](int t, int pbuf, int slot, bool accumulate) {   // O_t (+)= P V, P in S buffer `pbuf`
        const uint32_t vs = ring_smem + slot * Cfg::kTileBytes;
#pragma unroll
        for (int k = 0; k < kKeys / 16; ++k) {
          const uint64_t db = smem_desc_sw128(vs + (k / 4) * (D * 128)) + 2 * (k % 4);
          // 16 keys of P = 8 columns of TMEM (two bf16 per column)
          umma_bf16_tmem_a(tmem_base + 256 + t * D, tmem_base + pbuf * kKeys + 8 * k, db, idesc_o, (accumulate || k != 0) ? 1u : 0u);
        }
        umma_commit(o_full(t));
      };
      bool ok = mbar_wait(q_full, 0, p.status, &abort_flag, wb);
      if (ok) ok = mbar_wait(ring_full(0), 0, p.status, &abort_flag, wb);
      if (ok) {
        tc_fence_after();
        for (int t = 0; t < ntiles; ++t) issue_s(t, t, 0);
        umma_commit(ring_empty(0));
      }
      if (ntiles == 1) {
        // A single query tile has no partner to alternate with: the idle tile's S columns serve as
        // a second S buffer, so that Q K^T of block j+1 runs while the softmax works on block j.
        for (int j = 0; ok && j < nkv; ++j) {
          const int vi = 2 * j + 1, ki = 2 * j + 2;
          if (j + 1 < nkv) {
            if (!mbar_wait(ring_full(ki % NR), (ki / NR) & 1u, p.status, &abort_flag, wb)) { ok = false; break; }
            tc_fence_after();
            issue_s(0, (j + 1) & 1, ki % NR);
            umma_commit(ring_empty(ki % NR));
          }
          if (!mbar_wait(p_full(0), j & 1u, p.status, &abort_flag, wb)) { ok = false; break; }
          if (!mbar_wait(ring_full(vi % NR), (vi / NR) & 1u, p.status, &abort_flag, wb)) { ok = false; break; }
          tc_fence_after();
          issue_pv(0, j & 1, vi % NR, j > 0);
          umma_commit(ring_empty(vi % NR));
        }
      } else
      for (int j = 0; ok && j < nkv; ++j) {
        const int vi = 2 * j + 1, ki = 2 * j + 2;
        for (int t = 0; ok && t < ntiles; ++t) {
          if (!mbar_wait(p_full(t), j & 1u, p.status, &abort_flag, wb)) { ok = false; break; }
          if (t == 0 && !mbar_wait(ring_full(vi % NR), (vi / NR) & 1u, p.status, &abort_flag, wb)) { ok = false; break; }
          tc_fence_after();
          issue_pv(t, t, vi % NR, j > 0);
          if (t == ntiles - 1) umma_commit(ring_empty(vi % NR));
          if (j + 1 < nkv) {
            if (t == 0 && !mbar_wait(ring_full(ki % NR), (ki / NR) & 1u, p.status, &abort_flag, wb)) { ok = false; break; }
            tc_fence_after();
            issue_s(t, t, ki % NR);
            if (t == ntiles - 1) umma_commit(ring_empty(ki % NR));
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax warp-groups
    const int t = (warp - 2) >> 2;                       // query tile of this warp-group
    if (t < ntiles) {
      const int quad = warp & 3;                         // TMEM lanes [32 * quad, 32 * quad + 32)
      const int row_local = quad * 32 + lane;
      const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
      const bool single = (ntiles == 1);               // then S alternates between the two S buffers
      const uint32_t s_base = tmem_base + lane_addr;
      const uint32_t o_addr = tmem_base + 256 + t * D + lane_addr;
      const float c = p.scale_log2;
      bool ok = true;

      for (int j = 0; j < nkv; ++j) {
        const int sbuf = single ? (j & 1) : t;
        const uint32_t s_addr = s_base + sbuf * kKeys;
        ok = __all_sync(0xffffffffu, mbar_wait(s_full(sbuf), (single ? (j >> 1) : j) & 1u, p.status, &abort_flag, wb));
        if (!ok) break;
        tc_fence_after();
        const int valid = p.L - (jb0 + j) * kKeys;       // keys of this block below L (>= 128: all)
        // the whole S row (128 fp32) in registers: four TMEM loads in flight, one wait
        uint32_t v[4][32];
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) tmem_ld32(s_addr + cc * 32, v[cc]);
        tmem_ld_wait();
        if (valid < kKeys) {                             // last block: mask keys at or beyond L
#pragma unroll
          for (int cc = 0; cc < 4; ++cc)
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (cc * 32 + i >= valid) v[cc][i] = 0xff800000u;   // -inf
        }
        float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int cc = 0; cc < 4; ++cc)
#pragma unroll
          for (int i = 0; i < 32; ++i) mx[i & 3] = fmaxf(mx[i & 3], __uint_as_float(v[cc][i]));
        const float m_blk = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
        const float m_cand = fmaxf(m_ref, m_blk);
        const bool need = (m_cand - m_ref) * c > kRescaleThreshold;      // true on the first block (m_ref = -inf)
        if (j > 0) {
          // P V of block j-1 must be complete before P's buffer is overwritten or O is touched
          ok = __all_sync(0xffffffffu, mbar_wait(o_full(t), (j - 1) & 1u, p.status, &abort_flag, wb));
          if (!ok) break;
          tc_fence_after();
        }
        if (__any_sync(0xffffffffu, need)) {
          const float alpha = need ? exp2f((m_ref - m_cand) * c) : 1.0f;
          if (need) m_ref = m_cand;
          l_run *= alpha;
          if (j > 0) {
#pragma unroll 1
            for (int cc = 0; cc < D / 32; ++cc) {
              uint32_t o[32];
              tmem_ld32(o_addr + cc * 32, o);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
              tmem_st32(o_addr + cc * 32, o);
            }
            tmem_st_wait();
          }
        }
        const float neg_mc = -m_ref * c;
        float ls[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          // keys 64 * half .. 64 * half + 63 of this row, two per word: 32 TMEM columns.  The whole S
          // row is in registers by now, so overwriting its first columns loses nothing.
          uint32_t pk[32];
#pragma unroll
          for (int cc = 2 * half; cc < 2 * half + 2; ++cc) {
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              const float p0 = exp2f(fmaf(__uint_as_float(v[cc][i]), c, neg_mc));       // exp2(-inf) = 0 for masked keys
              const float p1 = exp2f(fmaf(__uint_as_float(v[cc][i + 1]), c, neg_mc));
              ls[(i >> 1) & 3] += p0 + p1;
              __nv_bfloat162 v2 = __floats2bfloat162_rn(p0, p1);
              pk[(cc & 1) * 16 + (i >> 1)] = *reinterpret_cast<uint32_t *>(&v2);
            }
          }
          tmem_st32(s_addr + half * 32, pk);
        }
        const float l_blk = (ls[0] + ls[1]) + (ls[2] + ls[3]);
        l_run += l_blk;
        tmem_st_wait();
        tc_fence_before();
        mbar_arrive(p_full(t));
      }
      final_ok = ok && __all_sync(0xffffffffu, mbar_wait(o_full(t), (nkv - 1) & 1u, p.status, &abort_flag, wb));
      if (final_ok && splits == 1) {
        tc_fence_after();
        const int rib = q0 + t * kQRows + row_local;
        bf16 *dst = p.out + (static_cast<long long>(e) * p.r + rib) * (p.H * D) + h * D;
        const float inv_l = 1.0f / l_run;
#pragma unroll 1
        for (int cc = 0; cc < D / 32; ++cc) {
          uint32_t v[32];
          tmem_ld32(o_addr + cc * 32, v);
          tmem_ld_wait();
          if (rib < p.r) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              uint32_t w[4];
#pragma unroll
              for (int u = 0; u < 4; ++u) {
                __nv_bfloat162 v2 = __floats2bfloat162_rn(__uint_as_float(v[q * 8 + u * 2]) * inv_l, __uint_as_float(v[q * 8 + u * 2 + 1]) * inv_l);
                w[u] = *reinterpret_cast<uint32_t *>(&v2);
              }
              reinterpret_cast<uint4 *>(dst + cc * 32)[q] = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
      }
    }
  }

  if (splits > 1) {
    // ---------------------------------------------------------------- merge of the key ranges over the cluster
    // Every thread of every CTA of the cluster passes the same barriers, whatever happened to its waits.
    constexpr uint32_t kPitch = (D + 4) * 4;                       // bytes per parked row: conflict-free 16-byte accesses
    const uint32_t part_o = ring_smem;                             // [2 tiles][128 rows][D + 4] fp32; the ring is idle by now
    const uint32_t part_m = part_o + 2 * kQRows * kPitch;          // [2][128] running maxima, then [2][128] sums
    tc_fence_before();
    __syncthreads();                                               // all roles done: no MMA reads the ring any more
    if (warp >= 2 && final_ok) {
      tc_fence_after();
      const int t = (warp - 2) >> 2, row_local = (warp & 3) * 32 + lane;
      const uint32_t o_addr = tmem_base + 256 + t * D + (static_cast<uint32_t>((warp & 3) * 32) << 16);
      const uint32_t dst = part_o + static_cast<uint32_t>(t * kQRows + row_local) * kPitch;
#pragma unroll 1
      for (int cc = 0; cc < D / 32; ++cc) {
        uint32_t v[32];
        tmem_ld32(o_addr + cc * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int q = 0; q < 8; ++q)
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (cc * 32 + q * 4) * 4), "r"(v[q * 4]), "r"(v[q * 4 + 1]),
                       "r"(v[q * 4 + 2]), "r"(v[q * 4 + 3]) : "memory");
      }
      asm volatile("st.shared.f32 [%0], %1;" ::"r"(part_m + (t * kQRows + row_local) * 4), "f"(m_ref) : "memory");
      asm volatile("st.shared.f32 [%0], %1;" ::"r"(part_m + (2 * kQRows + t * kQRows + row_local) * 4), "f"(l_run) : "memory");
    }
    tc_fence_before();
    cluster_sync_all();
    if (warp >= 2 && abort_flag == 0) {
      constexpr int G = D / 4;                                     // threads per row, one float4 each
      const int st = static_cast<int>(threadIdx.x) - 64, d4 = (st % G) * 4;
      uint32_t peer_o[8], peer_m[8];
#pragma unroll
      for (int s2 = 0; s2 < 8; ++s2) {
        peer_o[s2] = mapa_shared(part_o, static_cast<uint32_t>(s2 < splits ? s2 : 0));
        peer_m[s2] = mapa_shared(part_m, static_cast<uint32_t>(s2 < splits ? s2 : 0));
      }
      const float c = p.scale_log2;
      for (int tt = 0; tt < ntiles; ++tt) {
        const int rows_valid = min(kQRows, p.r - q0 - tt * kQRows);
        const int rpr = (rows_valid + splits - 1) / splits;        // this CTA merges rows [lo, hi) of the tile
        const int lo = sp * rpr, hi = min(rows_valid, lo + rpr);
        for (int row = lo + st / G; row < hi; row += 256 / G) {
          const uint32_t moff = static_cast<uint32_t>(tt * kQRows + row) * 4;
          float ms[8], m_all = -INFINITY;
#pragma unroll
          for (int s2 = 0; s2 < 8; ++s2)
            if (s2 < splits) { ms[s2] = ld_dsmem_f32(peer_m[s2] + moff); m_all = fmaxf(m_all, ms[s2]); }
          float l_all = 0.f;
          float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
          const uint32_t ooff = static_cast<uint32_t>(tt * kQRows + row) * kPitch + d4 * 4;
#pragma unroll
          for (int s2 = 0; s2 < 8; ++s2)
            if (s2 < splits) {                                     // range order: the sum does not depend on timing
              const float w = exp2f((ms[s2] - m_all) * c);
              l_all = fmaf(ld_dsmem_f32(peer_m[s2] + 2 * kQRows * 4 + moff), w, l_all);
              const float4 v = ld_dsmem_f4(peer_o[s2] + ooff);
              o.x = fmaf(w, v.x, o.x); o.y = fmaf(w, v.y, o.y); o.z = fmaf(w, v.z, o.z); o.w = fmaf(w, v.w, o.w);
            }
          const float inv_l = 1.0f / l_all;
          const int rib = q0 + tt * kQRows + row;
          __nv_bfloat162 h0 = __floats2bfloat162_rn(o.x * inv_l, o.y * inv_l), h1 = __floats2bfloat162_rn(o.z * inv_l, o.w * inv_l);
          *reinterpret_cast<uint2 *>(p.out + (static_cast<long long>(e) * p.r + rib) * (p.H * D) + h * D + d4) =
              make_uint2(*reinterpret_cast<uint32_t *>(&h0), *reinterpret_cast<uint32_t *>(&h1));
        }
      }
    }
    __syncwarp();
    cluster_sync_all();                                            // nobody leaves while a peer still reads its rows
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
  const int splits = a.kv_splits > 1 ? a.kv_splits : 1;
  if (splits > 8) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  const int rows_cta = (a.tiles_per_cta == 1 ? 1 : 2) * kQRows;
  cfg.gridDim = dim3((a.r + rows_cta - 1) / rows_cta * splits, a.H, a.B_eff);
  cfg.blockDim = dim3(kAttnThreads);
  cfg.dynamicSmemBytes = Cfg::kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;            // the key ranges of one query tile pair form a cluster
  attr[0].val.clusterDim.x = splits;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, attention_kernel<D>, tmQ, tmK, tmV, a);
}

// Launch shape of an attention call: query tiles per CTA (two: each K / V block feeds two tiles, the softmax of one
// overlapping the MMAs of the other; one: twice the CTAs when they would not fill the SMs) and key ranges per query
// tile group (a cluster of at most 6 CTAs, each range at least four key blocks long).
// Largest cluster of key ranges.  Clusters of 7 or 8 CTAs (one CTA per SM here) do not pack the GPCs and part of the
// grid falls into a second wave: measured in the step at the Infinity-2B shape, 8 -> 6 ranges took a block with r = 16
// rows over 6.4 k keys from 110 to 100 us (5 ranges: 102, 4: 103).
constexpr int kMaxRanges = 6;

void attention_plan(int B_eff, int H, int r, int L, int num_sms, int *tiles_per_cta, int *kv_splits) {
  const int nkv = (L + kKeys - 1) / kKeys;
  auto ranges = [&](long long ctas) {                       // key ranges when `ctas` CTAs would run without a split
    if (ctas * 2 > num_sms || nkv < 8) return 1;            // enough CTAs already, or too few key blocks to share
    int s = static_cast<int>(num_sms * 9 / 10 / ctas);       // clusters do not pack the last tenth of the SMs (measured)
    if (s > nkv / 4) s = nkv / 4;                           // at least four key blocks per range (measured: finer is slower)
    if (s > kMaxRanges) s = kMaxRanges;
    if (s < 2) return 1;
    const int per = (nkv + s - 1) / s;
    return (nkv + per - 1) / per;                           // every range gets at least one block
  };
  const long long pairs = static_cast<long long>((r + 2 * kQRows - 1) / (2 * kQRows)) * H * B_eff;
  const long long singles = static_cast<long long>((r + kQRows - 1) / kQRows) * H * B_eff;
  // One tile per CTA when the tile pairs alone would leave more than half of the SMs idle: a lone tile cannot hide its
  // softmax behind the other tile's MMAs, but twice the CTAs share the tensor work.  Measured in the step at the
  // Infinity-2B shape: r = 170 over 6.6 k keys 150 -> 130 us per block, r = 218 over 2.7 k keys 123 -> 115; a model
  // weighing 2 x 1800 cycles per key block of a pair against 2500 of a lone tile picked no better.
  const bool single = r > kQRows && pairs * 2 <= num_sms;
  *tiles_per_cta = single ? 1 : 2;
  *kv_splits = ranges(single ? singles : pairs);
}

cudaError_t launch_attention(const CUtensorMap &tmQ, const CUtensorMap &tmK, const CUtensorMap &tmV,
                             const AttnArgs &a, cudaStream_t st) {
  if (a.r <= 0 || a.L <= 0) return cudaErrorInvalidValue;
  if (a.D == 64) return launch_d<64>(tmQ, tmK, tmV, a, st);
  if (a.D == 128) return launch_d<128>(tmQ, tmK, tmV, a, st);
  return cudaErrorInvalidValue;
}

}  // namespace fvar
