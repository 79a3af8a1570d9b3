// CTA-pair form of the tensor-core GEMM for sm_100a: out[R][N] = A[R][K] * W[N][K]^T.
//
// Two CTAs on neighbouring SMs (a cluster of two) own one 256 x BN output tile.  Each CTA stages its
// own 128 rows of A and its own BN/2 rows of W per K step; the rank-0 CTA issues one
// tcgen05.mma.cta_group::2 (256 x BN x 16) for both, and each CTA's TMEM receives the 128 x BN
// accumulator of its own rows.  Per CTA and K step that is half of the W bytes the single-CTA kernel
// fetches and reads back for the same amount of math, which is what bounds that kernel (shared-memory
// and L2->SM bandwidth, not the tensor pipe).  Roles per CTA are those of gemm_kernel: warp 0 feeds the
// stage ring with TMA, warp 1 (rank 0 only) issues the MMAs into one of two TMEM accumulators, warps
// 2-9 drain the other one and apply the epilogue.  Every wait is bounded; on expiry the CTA flags the
// status word, gives its copies time to land, joins the pair's final barrier and frees its TMEM.
#include "gemm_common.cuh"

namespace fvar {

constexpr int kPairThreads = 64 + 32 * kEpiWarps;
constexpr int kPairSmemBudget = 196608;     // bytes of operand stages per CTA (192 KiB)

template <int BN>
struct PairCfg {
  static constexpr int kHalfN = BN / 2;
  static constexpr int kAtomBytesA = kBlockM * kBlockK * 2;
  static constexpr int kAtomBytesB = kHalfN * kBlockK * 2;
  static constexpr int kKAtoms = BN <= 128 ? 2 : 1;
  static constexpr int kStageBytesA = kAtomBytesA * kKAtoms;
  static constexpr int kStageBytesB = kAtomBytesB * kKAtoms;
  static constexpr int kStageBytes = kStageBytesA + kStageBytesB;
  static constexpr int kStages = kPairSmemBudget / kStageBytes;
  static constexpr int kTmemCols = 2 * BN;                        // two accumulators of BN columns
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment*/ + 256 /*barriers*/ + kEpiWarps * 4096 /*epilogue staging*/;
  static_assert(BN == 128 || BN == 256, "pair tile width");
  static_assert(kSmemBytes <= 227 * 1024, "shared memory");
  static_assert(kStages >= 2 && kStages <= 12, "stage count");
  static_assert((kTmemCols & (kTmemCols - 1)) == 0 && kTmemCols <= 512, "TMEM columns");
  static_assert(kSmemBytes > 116 * 1024, "one CTA per SM (the TMEM allocation must never wait on a neighbour)");
};

template <int BN, int EPI>
__global__ void __launch_bounds__(kPairThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
                 const __grid_constant__ GemmArgs p) {
  using Cfg = PairCfg<BN>;
  constexpr int S = Cfg::kStages;
  constexpr int kKAtoms = Cfg::kKAtoms;
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint32_t tmem_base_holder;
  __shared__ volatile int abort_flag;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = smem_base + S * Cfg::kStageBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };               // used in rank 0: both CTAs' bytes
  auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };        // one per CTA, signalled by the MMA commit
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * S + a); };    // one per CTA, signalled by the MMA commit
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * S + 2 + a); };   // used in rank 0: both CTAs' epilogue threads

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long wb = wait_budget(p.wait_cycles);
  const uint32_t rank = cluster_ctarank();
  const int pair = static_cast<int>(cluster_id_x()), npairs = static_cast<int>(cluster_nctaid_x());
  const int tiles_m2 = (p.R + 2 * kBlockM - 1) / (2 * kBlockM);
  const int tiles_n = (p.N + BN - 1) / BN;
  const int total_tiles = tiles_m2 * tiles_n;
  const int num_kb = (p.K + kBlockK * kKAtoms - 1) / (kBlockK * kKAtoms);

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), 2 * 32 * kEpiWarps);
    }
    mbar_fence_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmW);
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(&tmem_base_holder), Cfg::kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                 // the peer's barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_holder;
  pdl_wait();
  pdl_launch_dependents();

  if (warp == 0) {
    if (lane == 0) {
      // ---------------------------------------------------------------- TMA producer (both CTAs)
      const uint32_t full0 = mapa_shared(full_bar(0), 0);      // the stage barriers of rank 0
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true, issued = false;
      for (int work = pair; ok && work < total_tiles; work += npairs) {
        const int n_idx = work / tiles_m2, m2 = work - n_idx * tiles_m2;
        const int row_a = (2 * m2 + static_cast<int>(rank)) * kBlockM;
        const int row_w = n_idx * BN + static_cast<int>(rank) * Cfg::kHalfN;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, p.status, &abort_flag, wb)) { ok = false; break; }
          if (rank == 0) mbar_expect_tx(full_bar(stage), 2u * Cfg::kStageBytes);
          const uint32_t sa = smem_base + stage * Cfg::kStageBytes;
          const uint32_t fb = full0 + 8u * stage;
#pragma unroll
          for (int ka = 0; ka < kKAtoms; ++ka) {
            const int kx = (kb * kKAtoms + ka) * kBlockK;      // fully out-of-range atoms are zero-filled
            tma_load_2d_pair(sa + ka * Cfg::kAtomBytesA, &tmA, fb, kx, row_a);
            tma_load_2d_pair(sa + Cfg::kStageBytesA + ka * Cfg::kAtomBytesB, &tmW, fb, kx, row_w);
          }
          issued = true;
          if (++stage == S) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok && issued) {
        // The byte counts of this CTA's copies go to rank 0's barriers, which cannot be polled from
        // here: give the copies in flight a fixed time to land before shared memory is released.
        const long long t0 = clock64();
        while (clock64() - t0 < 4000000ll) {}
      }
    }
  } else if (warp == 1) {
    if (rank == 0) {
      // ---------------------------------------------------------------- MMA issuer (rank 0 only)
      const bool leader = elect_one();
      constexpr uint32_t idesc = umma_idesc_bf16(2 * kBlockM, BN);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int work = pair; ok && work < total_tiles; work += npairs, ++it) {
        const int a = it & 1;
        const uint32_t aphase = (it >> 1) & 1u;
        ok = __all_sync(0xffffffffu, mbar_wait(tempty_bar(a), aphase ^ 1u, p.status, &abort_flag, wb));
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + a * BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = __all_sync(0xffffffffu, mbar_wait(full_bar(stage), phase, p.status, &abort_flag, wb));
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = smem_base + stage * Cfg::kStageBytes;
          uint64_t da[kKAtoms], db[kKAtoms];
#pragma unroll
          for (int ka = 0; ka < kKAtoms; ++ka) {
            da[ka] = smem_desc_sw128(sa + ka * Cfg::kAtomBytesA);
            db[ka] = smem_desc_sw128(sa + Cfg::kStageBytesA + ka * Cfg::kAtomBytesB);
          }
          const uint32_t acc_first = (kb > 0) ? 1u : 0u;
          if (leader) {
#pragma unroll
            for (int ka = 0; ka < kKAtoms; ++ka) {
#pragma unroll
              for (int k = 0; k < kBlockK / 16; ++k)
                umma_bf16_pair(d_tmem, da[ka] + 2 * k, db[ka] + 2 * k, idesc, (ka != 0 || k != 0) ? 1u : acc_first);
            }
            umma_commit_pair(empty_bar(stage));       // frees this stage in both CTAs
          }
          __syncwarp();
          if (++stage == S) { stage = 0; phase ^= 1u; }
        }
        if (ok && leader) umma_commit_pair(tfull_bar(a));   // accumulator ready in both CTAs
        __syncwarp();
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
    const int quad = warp & 3;                 // TMEM lanes [32 * quad, 32 * quad + 32)
    const int cg = (warp - 2) >> 2;            // column group: alternate 32-column chunks of the tile
    constexpr int kChunks = BN / 32 / kEpiColGroups;   // chunks per warp
    const uint32_t ep_stage = bar_base + 256 + (warp - 2) * 4096;   // this warp's staging tile
    const uint32_t tempty0 = mapa_shared(tempty_bar(0), 0);
    int it = 0;
    bool ok = true;
    for (int work = pair; ok && work < total_tiles; work += npairs, ++it) {
      const int n_idx = work / tiles_m2, m2 = work - n_idx * tiles_m2;
      const int a = it & 1;
      const uint32_t aphase = (it >> 1) & 1u;
      const int row_local = quad * 32 + lane;
      const int row = (2 * m2 + static_cast<int>(rank)) * kBlockM + row_local;
      // residual rows of the first two column chunks are fetched while the main loop still runs
      constexpr int kPre = 2;
      float4 pre[kPre][8];
      bool have_pre = false;
      if constexpr (EPI == EPI_RESID) {
        if (row < p.R) {
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
      auto do_chunk = [&](int ci, const float4 *prep) {
        const int c = ci * kEpiColGroups + cg;
        const int col0 = n_idx * BN + c * 32;
        if (col0 < p.N) {                      // uniform across the warp
          uint32_t acc[32];
          tmem_ld32(taddr + c * 32, acc);
          tmem_ld_wait();
          epilogue_chunk<EPI>(p, acc, 0, row, col0, row < p.R, ep_stage, lane, prep);
        }
      };
#pragma unroll
      for (int ci = 0; ci < kPre; ++ci) do_chunk(ci, have_pre ? pre[ci] : nullptr);
#pragma unroll 1
      for (int ci = kPre; ci < kChunks; ++ci) do_chunk(ci, nullptr);
      tc_fence_before();
      mbar_arrive_cluster(tempty0 + 8u * a);   // rank 0's barrier collects both CTAs' epilogue threads
    }
  }

  // Nobody leaves (and no TMEM is freed) while the peer may still signal this CTA's barriers or the
  // pair's MMAs may still write this CTA's TMEM.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, Cfg::kTmemCols);
  }
}

// ------------------------------------------------------------------------------------------------ host
template <int BN, int EPI>
struct PairState {
  static bool attr_set;
  static int max_clusters;
};
template <int BN, int EPI> bool PairState<BN, EPI>::attr_set = false;
template <int BN, int EPI> int PairState<BN, EPI>::max_clusters = 0;

template <int BN, int EPI>
static cudaError_t pair_prepare_one() {
  using St = PairState<BN, EPI>;
  if (St::attr_set) return cudaSuccess;
  cudaError_t err = cudaFuncSetAttribute(gemm_pair_kernel<BN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         PairCfg<BN>::kSmemBytes);
  if (err != cudaSuccess) return err;
  int dev = 0, sms = 0;
  if ((err = cudaGetDevice(&dev)) != cudaSuccess) return err;
  if ((err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return err;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(sms / 2 * 2);
  cfg.blockDim = dim3(kPairThreads);
  cfg.dynamicSmemBytes = PairCfg<BN>::kSmemBytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  err = cudaOccupancyMaxActiveClusters(&n, gemm_pair_kernel<BN, EPI>, &cfg);
  if (err != cudaSuccess) return err;
  St::max_clusters = n;
  St::attr_set = true;
  return cudaSuccess;
}

template <int BN>
static cudaError_t pair_prepare_bn() {
  cudaError_t e = pair_prepare_one<BN, EPI_F32>();
  if (e == cudaSuccess) e = pair_prepare_one<BN, EPI_BF16>();
  if (e == cudaSuccess) e = pair_prepare_one<BN, EPI_GELU_BF16>();
  if (e == cudaSuccess) e = pair_prepare_one<BN, EPI_QKV>();
  if (e == cudaSuccess) e = pair_prepare_one<BN, EPI_RESID>();
  if (e == cudaSuccess) e = pair_prepare_one<BN, EPI_ARGMAX>();
  return e;
}

cudaError_t gemm_pair_prepare() {
  cudaError_t e = pair_prepare_bn<128>();
  if (e == cudaSuccess) e = pair_prepare_bn<256>();
  return e;
}

int gemm_pair_max_clusters() {
  if (gemm_pair_prepare() != cudaSuccess) return 0;
  const int a = PairState<128, EPI_F32>::max_clusters, b = PairState<256, EPI_F32>::max_clusters;
  return a < b ? a : b;
}

template <int BN, int EPI>
static cudaError_t pair_launch_one(const CUtensorMap &tmA, const CUtensorMap &tmW, const GemmArgs &a, cudaStream_t st) {
  using Cfg = PairCfg<BN>;
  using St = PairState<BN, EPI>;
  cudaError_t err = pair_prepare_one<BN, EPI>();
  if (err != cudaSuccess) return err;
  if (St::max_clusters <= 0) return cudaErrorLaunchOutOfResources;
  const long long tiles = static_cast<long long>((a.R + 2 * kBlockM - 1) / (2 * kBlockM)) * ((a.N + BN - 1) / BN);
  if (tiles <= 0) return cudaSuccess;
  const int clusters = static_cast<int>(tiles < St::max_clusters ? tiles : St::max_clusters);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * clusters);
  cfg.blockDim = dim3(kPairThreads);
  cfg.dynamicSmemBytes = Cfg::kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, gemm_pair_kernel<BN, EPI>, tmA, tmW, a);
}

template <int BN>
static cudaError_t pair_launch_bn(int epi, const CUtensorMap &tmA, const CUtensorMap &tmW, const GemmArgs &a, cudaStream_t st) {
  switch (epi) {
    case EPI_F32: return pair_launch_one<BN, EPI_F32>(tmA, tmW, a, st);
    case EPI_BF16: return pair_launch_one<BN, EPI_BF16>(tmA, tmW, a, st);
    case EPI_GELU_BF16: return pair_launch_one<BN, EPI_GELU_BF16>(tmA, tmW, a, st);
    case EPI_QKV: return pair_launch_one<BN, EPI_QKV>(tmA, tmW, a, st);
    case EPI_RESID: return pair_launch_one<BN, EPI_RESID>(tmA, tmW, a, st);
    case EPI_ARGMAX: return pair_launch_one<BN, EPI_ARGMAX>(tmA, tmW, a, st);
  }
  return cudaErrorInvalidValue;
}

// tmA: box of 128 rows; tmW: box of block_n / 2 rows.  One problem per launch (nbatch == 1), no split-K.
cudaError_t launch_gemm_pair(int epi, int block_n, const CUtensorMap &tmA, const CUtensorMap &tmW, const GemmArgs &a,
                             cudaStream_t st) {
  if (a.nbatch != 1 || a.splits > 1) return cudaErrorInvalidValue;
  switch (block_n) {
    case 128: return pair_launch_bn<128>(epi, tmA, tmW, a, st);
    case 256: return pair_launch_bn<256>(epi, tmA, tmW, a, st);
  }
  return cudaErrorInvalidValue;
}

}  // namespace fvar
