// Tensor-core GEMM for sm_100a: out[R][N] = A[R][K] * W[N][K]^T with fused epilogues.
//
// One persistent CTA per SM walks the tile list.  Warp 0 feeds a ring of shared-memory stages
// with TMA (128-byte swizzle), warp 1 issues tcgen05.mma into one of two TMEM accumulators,
// warps 2-9 drain the other accumulator (tcgen05.ld) and apply the epilogue, so the epilogue of
// tile i overlaps the main loop of tile i+1.  Every wait is bounded; on expiry the CTA flags the
// status word, lets its outstanding copies land, frees its TMEM and returns.
#include "gemm_common.cuh"

namespace fvar {

// Atoms per pipeline stage: one barrier round trip covers 64 * atoms of K.  Narrow tiles are bound by
// the round trip, not by bytes, so they take two atoms per stage (measured: 25 % faster at BN = 64).
__host__ __device__ constexpr int k_atoms(int bn) { return bn <= 128 ? 2 : 1; }
constexpr int kGemmThreads = 64 + 32 * kEpiWarps;
constexpr int kSmemBudget = 196608;     // bytes of operand stages per CTA (192 KiB)


template <int BN>
struct GemmCfg {
  static constexpr int kAtomBytesA = kBlockM * kBlockK * 2;
  static constexpr int kAtomBytesB = BN * kBlockK * 2;
  static constexpr int kKAtoms = k_atoms(BN);
  static constexpr int kStageBytesA = kAtomBytesA * kKAtoms;
  static constexpr int kStageBytesB = kAtomBytesB * kKAtoms;
  static constexpr int kStageBytes = kStageBytesA + kStageBytesB;
  static constexpr int kStages = kSmemBudget / kStageBytes;
  static constexpr int kTmemCols = 2 * BN < 32 ? 32 : 2 * BN;     // two accumulators
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment*/ + 256 /*barriers*/ + kEpiWarps * 4096 /*epilogue staging*/;
  static_assert(kSmemBytes <= 227 * 1024, "shared memory");
  static_assert(kStages >= 2 && kStages <= 12, "stage count");
  static_assert((kTmemCols & (kTmemCols - 1)) == 0 && kTmemCols <= 512, "TMEM columns");
  // More than half of an SM's shared memory per CTA: at most one CTA per SM, so the TMEM
  // allocation (up to all 512 columns) can never wait on a co-resident CTA.
  static_assert(kSmemBytes > 116 * 1024, "one CTA per SM");
};

template <int BN, int EPI>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
            const __grid_constant__ GemmArgs p) {
  using Cfg = GemmCfg<BN>;
  constexpr int S = Cfg::kStages;
  constexpr int kKAtoms = Cfg::kKAtoms;
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint32_t tmem_base_holder;
  __shared__ volatile int abort_flag;
  __shared__ volatile int split_last;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = smem_base + S * Cfg::kStageBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * S + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * S + 2 + a); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long wb = wait_budget(p.wait_cycles);
  const int tiles_m = (p.R + kBlockM - 1) / kBlockM;
  const int tiles_n = (p.N + BN - 1) / BN;
  const int tiles_per_batch = tiles_m * tiles_n;
  const int splits = p.splits > 1 ? p.splits : 1;      // split-K: each work item covers a K range of one tile
  const int total_tiles = tiles_per_batch * p.nbatch * splits;
  const int num_kb = (p.K + kBlockK * kKAtoms - 1) / (kBlockK * kKAtoms);
  const int kb_per_split = (num_kb + splits - 1) / splits;
  // The A box may be shorter than the 128-row tile (few rows: no point in fetching rows nobody stores);
  // the rest of the shared-memory tile then holds stale data whose accumulator rows are never written.
  const uint32_t a_tx_bytes = static_cast<uint32_t>(p.a_box_rows > 0 ? p.a_box_rows : kBlockM) * (kBlockK * 2 * kKAtoms);

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), 32 * kEpiWarps);
    }
    mbar_fence_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmW);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_holder), Cfg::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_holder;
  pdl_wait();
  pdl_launch_dependents();

  if (warp == 0) {
    if (lane == 0) {
      // ---------------------------------------------------------------- TMA producer
      int stage = 0;
      uint32_t phase = 0;
      uint32_t armed = 0;                      // bit s set: stage s has been armed at least once
      uint32_t last_parity = 0;                // bit s: parity of the phase last armed on stage s
      bool ok = true;
      for (int work = blockIdx.x; ok && work < total_tiles; work += gridDim.x) {
        const int tile = work / splits, sp = work - tile * splits;
        const int e = tile / tiles_per_batch, rem = tile - e * tiles_per_batch;
        const int n_idx = rem / tiles_m, m_idx = rem - n_idx * tiles_m;
        const int row_a = e * p.a_batch_rows + m_idx * kBlockM;
        const int row_w = p.w_mn_major ? e * p.b_batch_rows : e * p.b_batch_rows + n_idx * BN;
        const int kb0 = sp * kb_per_split, kb1 = min(num_kb, kb0 + kb_per_split);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, p.status, &abort_flag, wb)) { ok = false; break; }
          mbar_expect_tx(full_bar(stage), a_tx_bytes + Cfg::kStageBytesB);
          const uint32_t sa = smem_base + stage * Cfg::kStageBytes;
#pragma unroll
          for (int ka = 0; ka < kKAtoms; ++ka) {
            const int kx = (kb * kKAtoms + ka) * kBlockK;      // fully out-of-range atoms are zero-filled
            tma_load_2d(sa + ka * Cfg::kAtomBytesA, &tmA, full_bar(stage), kx, row_a);
            if (!p.w_mn_major) {
              tma_load_2d(sa + Cfg::kStageBytesA + ka * Cfg::kAtomBytesB, &tmW, full_bar(stage), kx, row_w);
            } else {
              // 64-column blocks of W^T, each a run of K rows: block j of the stage holds kKAtoms x 64 rows of 128 bytes
#pragma unroll
              for (int j = 0; j < BN / 64; ++j)
                tma_load_2d(sa + Cfg::kStageBytesA + (j * kKAtoms + ka) * 8192, &tmW, full_bar(stage), n_idx * BN + j * 64, row_w + kx);
            }
          }
          armed |= 1u << stage;
          last_parity = (last_parity & ~(1u << stage)) | (phase << stage);
          if (++stage == S) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // Let every copy that was issued land before the CTA's shared memory is released.
        for (int s = 0; s < S; ++s)
          if (armed & (1u << s)) {
            const long long t0 = clock64();
            while (!mbar_try_wait(full_bar(s), (last_parity >> s) & 1u) && clock64() - t0 < kWaitCycles) {}
          }
      }
    }
  } else if (warp == 1) {
    {
      // ---------------------------------------------------------------- MMA issuer
      // The whole warp walks the loop (so that stage counters, addresses and descriptors are
      // warp-uniform values); one elected lane issues the MMAs and the commits.
      const bool leader = elect_one();
      const uint32_t idesc = umma_idesc_bf16(kBlockM, BN) | (p.w_mn_major ? (1u << 16) : 0u);   // bit 16: B is MN-major
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int work = blockIdx.x; ok && work < total_tiles; work += gridDim.x, ++it) {
        const int sp = work % splits;
        const int kb0 = sp * kb_per_split, kb1 = min(num_kb, kb0 + kb_per_split);
        const int a = it & 1;
        const uint32_t aphase = (it >> 1) & 1u;
        ok = __all_sync(0xffffffffu, mbar_wait(tempty_bar(a), aphase ^ 1u, p.status, &abort_flag, wb));
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + a * BN;
        for (int kb = kb0; kb < kb1; ++kb) {
          ok = __all_sync(0xffffffffu, mbar_wait(full_bar(stage), phase, p.status, &abort_flag, wb));
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = smem_base + stage * Cfg::kStageBytes;
          // descriptors are computed by the whole warp (warp-uniform values); only the issue is elected
          uint64_t da[kKAtoms], db[kKAtoms];
#pragma unroll
          for (int ka = 0; ka < kKAtoms; ++ka) {
            da[ka] = smem_desc_sw128(sa + ka * Cfg::kAtomBytesA);
            db[ka] = p.w_mn_major ? smem_desc_sw128_mn(sa + Cfg::kStageBytesA + ka * 8192, kKAtoms * 8192)
                                  : smem_desc_sw128(sa + Cfg::kStageBytesA + ka * Cfg::kAtomBytesB);
          }
          const uint32_t kstep_b = p.w_mn_major ? (2048u >> 4) : 2u;      // descriptor advance per 16 of K
          const uint32_t acc_first = (kb > kb0) ? 1u : 0u;
          if (leader) {
#pragma unroll
          for (int ka = 0; ka < kKAtoms; ++ka) {
#pragma unroll
            for (int k = 0; k < kBlockK / 16; ++k)
              umma_bf16(d_tmem, da[ka] + 2 * k, db[ka] + kstep_b * k, idesc, (ka != 0 || k != 0) ? 1u : acc_first);
          }
          umma_commit(empty_bar(stage));
          }
          __syncwarp();
          if (++stage == S) { stage = 0; phase ^= 1u; }
        }
        if (ok && leader) umma_commit(tfull_bar(a));
        __syncwarp();
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9)
    // A warp reads the TMEM lanes of its quadrant (warp index mod 4); the two warps of a quadrant
    // take alternate 32-column chunks of the tile.
    const int quad = warp & 3;                 // TMEM lanes [32 * quad, 32 * quad + 32)
    const int cg = (warp - 2) >> 2;            // column group of this warp
    constexpr int kChunks = (BN / 32 + kEpiColGroups - 1) / kEpiColGroups;   // chunks per warp
    const uint32_t ep_stage = bar_base + 256 + (warp - 2) * 4096;   // this warp's staging tile
    int it = 0;
    bool ok = true;
    for (int work = blockIdx.x; ok && work < total_tiles; work += gridDim.x, ++it) {
      const int tile = work / splits, sp = work - tile * splits;
      const int e = tile / tiles_per_batch, rem = tile - e * tiles_per_batch;
      const int n_idx = rem / tiles_m, m_idx = rem - n_idx * tiles_m;
      const int a = it & 1;
      const uint32_t aphase = (it >> 1) & 1u;
      const int row_local = quad * 32 + lane;
      const int row = m_idx * kBlockM + row_local;
      // The residual rows of the first two column chunks are fetched while the main loop still runs:
      // with one tile per CTA nothing else hides that latency.
      constexpr int kPre = (kChunks < 2) ? kChunks : 2;
      float4 pre[kPre][8];
      bool have_pre = false;
      if constexpr (EPI == EPI_RESID) {
        if (splits == 1 && row < p.R) {
          const int e2 = row / p.rows_per_batch, j2 = row - e2 * p.rows_per_batch;
          const float *res = p.resid + (static_cast<long long>(e2 * p.rmap.bmul + p.rmap.boff) * p.rmap.rpb + j2) * p.ld_out + n_idx * BN;
#pragma unroll
          for (int ci = 0; ci < kPre; ++ci) {
            const int c = ci * kEpiColGroups + cg;
            if (n_idx * BN + c * 32 < p.N) {
#pragma unroll
              for (int q = 0; q < 8; ++q) pre[ci][q] = reinterpret_cast<const float4 *>(res + c * 32)[q];
            }
          }
          have_pre = true;
        }
      }
      ok = __all_sync(0xffffffffu, mbar_wait(tfull_bar(a), aphase, p.status, &abort_flag, wb));
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + a * BN + (static_cast<uint32_t>(quad * 32) << 16);
      if (splits == 1) {
        auto do_chunk = [&](int ci, const float4 *prep) {
          const int c = ci * kEpiColGroups + cg;
          const int col0 = n_idx * BN + c * 32;
          if (c * 32 < BN && col0 < p.N) {       // uniform across the warp
            uint32_t acc[32];
            tmem_ld32(taddr + c * 32, acc);
            tmem_ld_wait();
            epilogue_chunk<EPI>(p, acc, e, row, col0, row < p.R, ep_stage, lane, prep);
          }
        };
#pragma unroll
        for (int ci = 0; ci < kPre; ++ci) do_chunk(ci, have_pre ? pre[ci] : nullptr);
#pragma unroll 1
        for (int ci = kPre; ci < kChunks; ++ci) do_chunk(ci, nullptr);
        tc_fence_before();
        mbar_arrive(tempty_bar(a));
      } else {
        // Split-K: park this K range's partial tile in the scratch area; the CTA that finishes a
        // tile last adds the partials in split order (so the sum does not depend on timing) and
        // applies the epilogue.
        // Layout of a partial tile: float4 number (c * 8 + q) * 128 + row, so that the 32 lanes of a
        // warp (consecutive rows) touch 512 contiguous bytes per access.
        float4 *mine = reinterpret_cast<float4 *>(p.partial + (static_cast<size_t>(tile) * splits + sp) * (kBlockM * BN)) + row_local;
#pragma unroll 1
        for (int c = cg; c < BN / 32; c += kEpiColGroups) {
          uint32_t acc[32];
          tmem_ld32(taddr + c * 32, acc);
          tmem_ld_wait();
          if (row < p.R)                       // rows past the end carry nothing anybody reads
#pragma unroll
          for (int q = 0; q < 8; ++q)
            __stcg(mine + (c * 8 + q) * kBlockM,
                   make_float4(__uint_as_float(acc[q * 4]), __uint_as_float(acc[q * 4 + 1]),
                               __uint_as_float(acc[q * 4 + 2]), __uint_as_float(acc[q * 4 + 3])));
        }
        tc_fence_before();
        mbar_arrive(tempty_bar(a));
        __threadfence();
        asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpiWarps) : "memory");
        if (threadIdx.x == 64) split_last = (atomicAdd(p.counters + tile, 1) == splits - 1) ? 1 : 0;
        asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpiWarps) : "memory");
        if (split_last) {
          __threadfence();
          const float4 *base = reinterpret_cast<const float4 *>(p.partial + static_cast<size_t>(tile) * splits * (kBlockM * BN)) + row_local;
#pragma unroll 1
          for (int c = cg; c < BN / 32; c += kEpiColGroups) {
            const int col0 = n_idx * BN + c * 32;
            if (col0 >= p.N) break;
            float sum[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) sum[i] = 0.f;
            for (int s2 = 0; s2 < splits && row < p.R; ++s2) {
              const float4 *src = base + static_cast<size_t>(s2) * (kBlockM * BN / 4) + c * 8 * kBlockM;
#pragma unroll
              for (int q = 0; q < 8; ++q) {
                const float4 v = __ldcg(src + q * kBlockM);
                sum[q * 4] += v.x; sum[q * 4 + 1] += v.y; sum[q * 4 + 2] += v.z; sum[q * 4 + 3] += v.w;
              }
            }
            uint32_t acc[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) acc[i] = __float_as_uint(sum[i]);
            epilogue_chunk<EPI>(p, acc, e, row, col0, row < p.R, ep_stage, lane);
          }
          if (threadIdx.x == 64) p.counters[tile] = 0;      // ready for the next launch
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

// Cost model fitted to measurements on B200: an SM takes in about 100 GB/s from L2, so one K step
// of a 128 x BN tile (16 KiB of A + BN * 128 B of W) costs t_k microseconds; a wave of work items
// costs its K steps plus an epilogue that is only hidden behind the next item of the same CTA.
// Splitting K trades a reduction through the scratch area for more CTAs streaming the operands.
// microseconds per K block and per epilogue of a single-CTA tile of 64 / 128 / 256 columns
static const float kTileTk[3] = {0.24f, 0.30f, 0.47f}, kTileTepi[3] = {1.0f, 1.5f, 2.5f};

void gemm_pick_tile(int tiles_m_total, int N, int K, int num_sms, int max_splits, size_t scratch_bytes, int *block_n,
                    int *splits) {
  const int cand[3] = {64, 128, 256};
  const int num_kb = (K + kBlockK - 1) / kBlockK;
  float best_cost = 1e30f;
  *block_n = 64;
  *splits = 1;
  for (int i = 0; i < 3; ++i) {
    const long long tiles = static_cast<long long>(tiles_m_total) * ((N + cand[i] - 1) / cand[i]);
    for (int sp = 1; sp <= max_splits; sp *= 2) {
      // splitting pays only for long reductions that would otherwise leave most SMs idle (measured)
      if (sp > 1 && (num_kb < 64 || tiles * sp > num_sms || tiles > 4096 ||
                     static_cast<size_t>(tiles) * sp * kBlockM * cand[i] * 4 > scratch_bytes))
        break;
      const long long waves = (tiles * sp + num_sms - 1) / num_sms;
      const int kb = (num_kb + sp - 1) / sp;
      float cost = waves * (kb * kTileTk[i] + kTileTepi[i]);
      if (sp > 1) cost += 1.5f + 0.6f * sp * cand[i] / 128.0f;      // park + fixed-order reduction by one CTA
      if (cost < best_cost) {
        best_cost = cost;
        *block_n = cand[i];
        *splits = sp;
      }
    }
  }
}


GemmPlan gemm_plan(int R, int nbatch, int N, int K, int num_sms, int max_clusters, int max_splits, size_t scratch_bytes) {
  GemmPlan plan{false, 64, 1};
  const int tiles_m = (R + kBlockM - 1) / kBlockM * nbatch;
  gemm_pick_tile(tiles_m, N, K, num_sms, max_splits, scratch_bytes, &plan.block_n, &plan.splits);
  if (nbatch != 1 || R <= kBlockM || max_clusters <= 0) return plan;
  // Cost of the single-CTA choice.
  const int num_kb = (K + kBlockK - 1) / kBlockK;
  const int i1 = plan.block_n == 64 ? 0 : (plan.block_n == 128 ? 1 : 2);
  const long long tiles1 = static_cast<long long>(tiles_m) * ((N + plan.block_n - 1) / plan.block_n) * plan.splits;
  float cost1 = ((tiles1 + num_sms - 1) / num_sms) * (((num_kb + plan.splits - 1) / plan.splits) * kTileTk[i1] + kTileTepi[i1]);
  if (plan.splits > 1) cost1 += 1.5f + 0.6f * plan.splits * plan.block_n / 128.0f;
  // A pair CTA moves, per K step, what a single CTA of half the tile width moves, for twice the output.
  const int cand2[2] = {128, 256};
  const int tiles_m2 = (R + 2 * kBlockM - 1) / (2 * kBlockM);
  float best2 = 1e30f;
  int bn2 = 0;
  for (int i = 0; i < 2; ++i) {
    const long long t2 = static_cast<long long>(tiles_m2) * ((N + cand2[i] - 1) / cand2[i]);
    const float c = ((t2 + max_clusters - 1) / max_clusters) * (num_kb * kTileTk[i] + kTileTepi[i + 1]);
    if (c < best2) { best2 = c; bn2 = cand2[i]; }
  }
  if (bn2 && best2 < cost1) plan = GemmPlan{true, bn2, 1};
  return plan;
}

int gemm_pick_block_n(int tiles_m_total, int N, int K, int num_sms) {
  int bn, sp;
  gemm_pick_tile(tiles_m_total, N, K, num_sms, 1, 0, &bn, &sp);
  return bn;
}

template <int BN, int EPI>
static cudaError_t set_attr() {
  static bool attr_set = false;
  if (attr_set) return cudaSuccess;
  cudaError_t err = cudaFuncSetAttribute(gemm_kernel<BN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         GemmCfg<BN>::kSmemBytes);
  if (err == cudaSuccess) attr_set = true;
  return err;
}

template <int BN>
static cudaError_t set_attr_bn() {
  cudaError_t e = set_attr<BN, EPI_F32>();
  if (e == cudaSuccess) e = set_attr<BN, EPI_BF16>();
  if (e == cudaSuccess) e = set_attr<BN, EPI_GELU_BF16>();
  if (e == cudaSuccess) e = set_attr<BN, EPI_QKV>();
  if (e == cudaSuccess) e = set_attr<BN, EPI_RESID>();
  if (e == cudaSuccess) e = set_attr<BN, EPI_ARGMAX>();
  return e;
}

cudaError_t gemm_prepare() {
  cudaError_t e = set_attr_bn<64>();
  if (e == cudaSuccess) e = set_attr_bn<128>();
  if (e == cudaSuccess) e = set_attr_bn<256>();
  return e;
}

template <int BN, int EPI>
static cudaError_t launch_one(const CUtensorMap &tmA, const CUtensorMap &tmW, const GemmArgs &a, int num_sms,
                              cudaStream_t st) {
  using Cfg = GemmCfg<BN>;
  cudaError_t err = set_attr<BN, EPI>();
  if (err != cudaSuccess) return err;
  const long long tiles = static_cast<long long>((a.R + kBlockM - 1) / kBlockM) * ((a.N + BN - 1) / BN) * a.nbatch *
                          (a.splits > 1 ? a.splits : 1);
  if (tiles <= 0) return cudaSuccess;
  const int grid = static_cast<int>(tiles < num_sms ? tiles : num_sms);
  return launch_pdl(gemm_kernel<BN, EPI>, dim3(grid), dim3(kGemmThreads), Cfg::kSmemBytes, st, tmA, tmW, a);
}

template <int BN>
static cudaError_t launch_bn(int epi, const CUtensorMap &tmA, const CUtensorMap &tmW, const GemmArgs &a, int num_sms,
                             cudaStream_t st) {
  switch (epi) {
    case EPI_F32: return launch_one<BN, EPI_F32>(tmA, tmW, a, num_sms, st);
    case EPI_BF16: return launch_one<BN, EPI_BF16>(tmA, tmW, a, num_sms, st);
    case EPI_GELU_BF16: return launch_one<BN, EPI_GELU_BF16>(tmA, tmW, a, num_sms, st);
    case EPI_QKV: return launch_one<BN, EPI_QKV>(tmA, tmW, a, num_sms, st);
    case EPI_RESID: return launch_one<BN, EPI_RESID>(tmA, tmW, a, num_sms, st);
    case EPI_ARGMAX: return launch_one<BN, EPI_ARGMAX>(tmA, tmW, a, num_sms, st);
  }
  return cudaErrorInvalidValue;
}

cudaError_t launch_gemm(int epi, int block_n, const CUtensorMap &tmA, const CUtensorMap &tmW, const GemmArgs &a,
                        int num_sms, cudaStream_t st) {
  switch (block_n) {
    case 64: return launch_bn<64>(epi, tmA, tmW, a, num_sms, st);
    case 128: return launch_bn<128>(epi, tmA, tmW, a, num_sms, st);
    case 256: return launch_bn<256>(epi, tmA, tmW, a, num_sms, st);
  }
  return cudaErrorInvalidValue;
}

}  // namespace fvar
