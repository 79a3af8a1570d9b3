// Weight-streaming GEMM for few rows, sm_100a: out[R][N] = A[R][K] * W[N][K]^T with R <= 512.
//
// With few rows the product is bound by streaming W once from HBM, so the roles of the two operands are
// swapped: a CTA takes 128 rows of W (128 output features) as the M side of tcgen05.mma and all R rows of
// A as the N side (one or two column chunks of up to 256 rows), so every weight byte enters shared memory
// exactly once and the small A panel is what gets re-read (from L2).  To put every SM on the stream the
// reduction is split over a thread-block cluster of S <= 8 CTAs: CTA s of a cluster covers K range s of
// its 128-feature tile, parks its fp32 partial tile in its own shared memory, and after a cluster barrier
// reduces a 1/S slice of the rows over all S partials through distributed shared memory, in rank order
// (the sum does not depend on timing), and applies the epilogue.  Nothing goes through global scratch.
//
// A pipeline stage covers up to four 64-wide K blocks fetched by ONE TMA instruction per operand: the operands are
// described as 3-D tensors {64 K elements, rows, K / 64} and a box {64, rows, nk} lands as nk consecutive
// 128-byte-swizzled K-major tiles (fewer barrier round trips per byte; in a load-only probe the bytes per instruction
// set the throughput of a single SM's copy unit).
//
// Roles: warp 0 feeds the stage ring with TMA (the weight halves of the first stages are requested before
// griddepcontrol.wait: weights never depend on the preceding kernel), warp 1 issues the MMAs into TMEM,
// warps 2-9 dump, reduce and store.  After its last load the producer asks L2 to prefetch this CTA's share
// of the weights the next GEMM of the chain will stream.  Every mbarrier wait is bounded; a CTA that gives
// up flags the status word and still joins every cluster barrier, so its peers never wait for it.
#include "gemm_common.cuh"

namespace fvar {

constexpr int kSkinnyThreads = 64 + 32 * kEpiWarps;
constexpr int kSkinnyRing = 196608;                       // bytes of operand stages per CTA (192 KiB) ...
constexpr int kSkinnyRingSmall = 98304;                   // ... or 96 KiB when four stages fit: two CTAs per SM, so that
                                                          // the next GEMM of a chain sets up and requests its weights
                                                          // while this one drains
constexpr int kSkinnyBarBytes = 1024;
constexpr int kSkinnySmemBytes = 1024 /*alignment*/ + kSkinnyBarBytes + kSkinnyRing;
constexpr int kSkinnySmemSmall = 1024 + kSkinnyBarBytes + kSkinnyRingSmall;
constexpr int kSkinnyMaxStages = 12;
constexpr int kSkinnyWAtom = kBlockM * kBlockK * 2;       // 128 weight rows x 64 K

// TMEM: the small form allocates at most 64 columns, so co-resident CTAs never wait for each other's columns; the
// large form (up to 512 columns) takes more than half of an SM's shared memory and is alone on its SM.
static_assert(kSkinnySmemBytes > 116 * 1024, "one large CTA per SM");
static_assert(2 * (kSkinnySmemSmall + 1024) <= 227 * 1024, "two small CTAs per SM");

__device__ __forceinline__ void l2_prefetch_bulk(const void *ptr, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(ptr), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint2 pack4_bf16(float a, float b, float c, float d) {
  return make_uint2(pack_bf16(a, b), pack_bf16(c, d));
}

// Epilogue of one thread for output row `row` (row of the flattened [R] rows), features n .. n + 3 (n % 4 == 0,
// n + 3 < N): the four sums arrive in `acc`.
template <int EPI>
__device__ __forceinline__ void skinny_store(const GemmArgs &p, float4 acc, int row, int n) {
  float v[4] = {acc.x, acc.y, acc.z, acc.w};
  if (p.bias != nullptr) {
    const uint2 u = __ldg(reinterpret_cast<const uint2 *>(p.bias + n));
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&u);
    const float2 f0 = __bfloat1622float2(h[0]), f1 = __bfloat1622float2(h[1]);
    v[0] += f0.x; v[1] += f0.y; v[2] += f1.x; v[3] += f1.y;
  }
  if constexpr (EPI == EPI_F32) {
    *reinterpret_cast<float4 *>(p.out_f32 + static_cast<long long>(row) * p.ld_out + n) = make_float4(v[0], v[1], v[2], v[3]);
  } else if constexpr (EPI == EPI_BF16 || EPI == EPI_GELU_BF16) {
    if constexpr (EPI == EPI_GELU_BF16) {
#pragma unroll
      for (int i = 0; i < 4; ++i) v[i] = gelu_tanh_f(v[i]);
    }
    *reinterpret_cast<uint2 *>(p.out_bf16 + static_cast<long long>(row) * p.ld_out + n) = pack4_bf16(v[0], v[1], v[2], v[3]);
  } else if constexpr (EPI == EPI_QKV) {
    const int e = row / p.rows_per_batch, j = row - e * p.rows_per_batch;
    const int b = e * p.bmul + p.boff;
    const int vc = n + p.col_base;
    if (vc < p.C) {
      *reinterpret_cast<uint2 *>(p.out_bf16 + static_cast<long long>(row) * p.ld_out + vc) = pack4_bf16(v[0], v[1], v[2], v[3]);
    } else if (vc < 2 * p.C) {
      const int c = vc - p.C, h = c / p.D, d0 = c - h * p.D;
      bf16 *dst = p.kc + ((static_cast<long long>(b) * p.H + h) * p.L_cap + p.L_prev + j) * p.D + d0;
      *reinterpret_cast<uint2 *>(dst) = pack4_bf16(v[0], v[1], v[2], v[3]);
    } else {
      const int c = vc - 2 * p.C, h = c / p.D, d0 = c - h * p.D;
      bf16 *dst = p.vt + ((static_cast<long long>(b) * p.H + h) * p.D + d0) * p.L_cap + p.L_prev + j;
#pragma unroll
      for (int i = 0; i < 4; ++i) dst[static_cast<long long>(i) * p.L_cap] = __float2bfloat16_rn(v[i]);
    }
  } else if constexpr (EPI == EPI_RESID) {
    const int e = row / p.rows_per_batch, j = row - e * p.rows_per_batch;
    const int b = e * p.bmul + p.boff;
    const float4 r4 = *reinterpret_cast<const float4 *>(
        p.resid + (static_cast<long long>(e * p.rmap.bmul + p.rmap.boff) * p.rmap.rpb + j) * p.ld_out + n);
    const int jo = p.scatter ? __ldg(p.scatter + static_cast<long long>(e) * p.rows_per_batch + j) : j;
    const float4 g4 = p.gate ? __ldg(reinterpret_cast<const float4 *>(p.gate + static_cast<long long>(b) * p.gate_stride + n))
                             : make_float4(1.f, 1.f, 1.f, 1.f);
    v[0] = fmaf(g4.x, v[0], r4.x);
    v[1] = fmaf(g4.y, v[1], r4.y);
    v[2] = fmaf(g4.z, v[2], r4.z);
    v[3] = fmaf(g4.w, v[3], r4.w);
    *reinterpret_cast<float4 *>(p.out_f32 + (static_cast<long long>(e * p.omap.bmul + p.omap.boff) * p.omap.rpb + jo) * p.ld_out + n) =
        make_float4(v[0], v[1], v[2], v[3]);
    if (p.xsplit != nullptr) {
      bf16 *hi = p.xsplit + (static_cast<long long>(e) * 2 * p.xsplit_mk + jo) * p.ld_out + n;
      float lo[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) lo[i] = v[i] - __bfloat162float(__float2bfloat16_rn(v[i]));
      *reinterpret_cast<uint2 *>(hi) = pack4_bf16(v[0], v[1], v[2], v[3]);
      *reinterpret_cast<uint2 *>(hi + static_cast<long long>(p.xsplit_mk) * p.ld_out) = pack4_bf16(lo[0], lo[1], lo[2], lo[3]);
    }
  }
}

// tmA: the activation rows [R][K], box of sk_rp rows; tmW: the weight rows [N][K], box of 128 rows (gemm_skinny_map).
// ROWS = false: the form described at the top (weights on the M side, all rows on the N side).  ROWS = true: the same
// pipeline, K split and cluster reduction for 128 x 128 output tiles with the rows back on the M side -- for a few
// hundred rows and a narrow output, where the row-tiled kernels have too few tiles to fill the SMs and each of their
// CTAs walks all of K; cluster c then owns tile (row tile c % sk_tiles_m, feature tile c / sk_tiles_m).
template <int EPI, bool ROWS>
__global__ void __launch_bounds__(kSkinnyThreads, 1)
gemm_skinny_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
                   const __grid_constant__ GemmArgs p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint32_t tmem_base_holder;
  __shared__ volatile int abort_flag;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = smem_base;
  const uint32_t ring = smem_base + kSkinnyBarBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kSkinnyMaxStages + s); };
  const uint32_t tfull_bar = bar_base + 8u * (2 * kSkinnyMaxStages);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long wb = wait_budget(p.wait_cycles);
  const int S = p.splits > 1 ? p.splits : 1;                 // cluster size = K ranges per tile
  const int sp = static_cast<int>(cluster_ctarank());
  const int cid = static_cast<int>(cluster_id_x());
  const int tile = ROWS ? cid / p.sk_tiles_m : cid;          // 128-feature tile
  const int row0 = ROWS ? (cid % p.sk_tiles_m) * kBlockM : 0;  // first row of the tile (ROWS)
  const int nstages = p.sk_stages, rp = p.sk_rp, rc = p.sk_rows_chunk, nchunks = p.sk_nchunks;
  const int rp32 = (rp + 31) & ~31;                          // TMEM columns between the accumulators of two chunks
  const int nk = p.sk_nk;                                   // K blocks per pipeline stage (one TMA instruction per operand)
  const uint32_t a_bytes = static_cast<uint32_t>(rp) * (kBlockK * 2);       // one K block of one chunk of A
  const uint32_t w_stage = static_cast<uint32_t>(nk) * kSkinnyWAtom;
  const uint32_t stage_bytes = w_stage + nchunks * nk * a_bytes;
  const int num_kb = (p.K + kBlockK - 1) / kBlockK;
  const int kbps = (num_kb + S - 1) / S;
  const int kb0 = sp * kbps;
  const int nkb = max(0, min(num_kb, kb0 + kbps) - kb0);     // the host sizes S so that every range has work
  const int nst = (nkb + nk - 1) / nk;                       // pipeline stages this CTA walks
  uint32_t tmem_cols = 32;
  while (static_cast<int>(tmem_cols) < nchunks * rp32) tmem_cols <<= 1;

  // a stage that reaches past this CTA's K range fetches blocks nobody multiplies (zeros past the end of K)
  auto load_w = [&](int i) {
    const uint32_t dst = ring + (i % nstages) * stage_bytes;
    if (nk > 1) tma_load_3d(dst, &tmW, full_bar(i % nstages), 0, tile * kBlockM, kb0 + i * nk);
    else tma_load_2d(dst, &tmW, full_bar(i % nstages), (kb0 + i) * kBlockK, tile * kBlockM);
  };
  auto load_a = [&](int i) {
    const uint32_t dst = ring + (i % nstages) * stage_bytes + w_stage;
    for (int ch = 0; ch < nchunks; ++ch) {
      if (nk > 1) tma_load_3d(dst + ch * nk * a_bytes, &tmA, full_bar(i % nstages), 0, row0 + ch * rc, kb0 + i * nk);
      else tma_load_2d(dst + ch * a_bytes, &tmA, full_bar(i % nstages), (kb0 + i) * kBlockK, row0 + ch * rc);
    }
  };
  const int pre = min(nstages, nst);
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < nstages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(tfull_bar, 1);
    mbar_fence_init();
    // The weights of the first stages are requested at once, by the thread that will go on producing: they depend
    // on no other kernel, and on nothing of this CTA but the barriers just initialised.
    for (int i = 0; i < pre; ++i) {
      mbar_expect_tx(full_bar(i), stage_bytes);
      load_w(i);
    }
    prefetch_tmap(&tmA);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_holder), tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_holder;
  bool ok = true;

  if (warp == 0) {
    if (lane == 0) {
      // ---------------------------------------------------------------- TMA producer
      pdl_wait();
      pdl_launch_dependents();
      for (int i = 0; i < pre; ++i) load_a(i);
      uint32_t armed = pre > 0 ? ((1u << pre) - 1u) : 0u, last_parity = 0;
      for (int i = pre; ok && i < nst; ++i) {
        const int stage = i % nstages;
        const uint32_t phase = (i / nstages) & 1u;
        if (!mbar_wait(empty_bar(stage), phase ^ 1u, p.status, &abort_flag, wb)) { ok = false; break; }
        mbar_expect_tx(full_bar(stage), stage_bytes);
        load_w(i);
        load_a(i);
        last_parity = (last_parity & ~(1u << stage)) | (phase << stage);
      }
      if (ok && p.pf_ptr != nullptr) {
        // this CTA's share of the next GEMM's weights, in pieces of 16 KiB
        const unsigned long long per = ((p.pf_bytes + gridDim.x - 1) / gridDim.x + 15ull) & ~15ull;
        const unsigned long long lo = per * blockIdx.x, hi = min(p.pf_bytes & ~15ull, lo + per);
        for (unsigned long long o = lo; o < hi; o += 16384ull)
          l2_prefetch_bulk(static_cast<const uint8_t *>(p.pf_ptr) + o, static_cast<uint32_t>(min(16384ull, hi - o)));
      }
      if (!ok) {
        // let every copy that was issued land before the shared memory is reused or released
        for (int s = 0; s < nstages; ++s)
          if (armed & (1u << s)) {
            const long long t0 = clock64();
            while (!mbar_try_wait(full_bar(s), (last_parity >> s) & 1u) && clock64() - t0 < kWaitCycles) {}
          }
      }
    } else {
      pdl_wait();
      pdl_launch_dependents();
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    pdl_wait();
    pdl_launch_dependents();
    const bool leader = elect_one();
    const uint32_t idesc = umma_idesc_bf16(kBlockM, rp);
    for (int i = 0; i < nst; ++i) {
      const int stage = i % nstages;
      ok = __all_sync(0xffffffffu, mbar_wait(full_bar(stage), (i / nstages) & 1u, p.status, &abort_flag, wb));
      if (!ok) break;
      tc_fence_after();
      const uint32_t sa = ring + stage * stage_bytes;
      const int kvalid = min(nk, nkb - i * nk);              // K blocks of this stage inside the CTA's range
      if (leader) {
        // descriptor words: the address field counts 16-byte units, so a K block further on adds its size >> 4
        uint64_t dw = smem_desc_sw128(sa), da0 = smem_desc_sw128(sa + w_stage);
        const uint64_t da1_off = static_cast<uint64_t>((nk * a_bytes) >> 4);
        uint32_t acc = i > 0 ? 1u : 0u;
        for (int kk = 0; kk < kvalid; ++kk) {
#pragma unroll
          for (int k = 0; k < kBlockK / 16; ++k) {
            if (ROWS) {
              umma_bf16(tmem_base, da0 + 2 * k, dw + 2 * k, idesc, acc);       // rows x features
            } else {
              umma_bf16(tmem_base, dw + 2 * k, da0 + 2 * k, idesc, acc);       // features x rows
              if (nchunks > 1) umma_bf16(tmem_base + rp32, dw + 2 * k, da0 + da1_off + 2 * k, idesc, acc);
            }
            acc = 1u;
          }
          dw += kSkinnyWAtom >> 4;
          da0 += a_bytes >> 4;
        }
        umma_commit(empty_bar(stage));
      }
      __syncwarp();
    }
    if (ok && leader) umma_commit(tfull_bar);
    __syncwarp();
  } else {
    pdl_wait();
    pdl_launch_dependents();
    ok = nkb > 0 && __all_sync(0xffffffffu, mbar_wait(tfull_bar, 0, p.status, &abort_flag, wb));
    tc_fence_after();
  }

  // ------------------------------------------------------------------ reduction over the cluster + epilogue
  // Every thread of every CTA of the cluster passes the same cluster barriers; warps 2-9 do the work.
  const int et = static_cast<int>(threadIdx.x) - 64;         // 0 .. 255 in the epilogue warps
  const uint32_t red = ring;                                   // fp32 [rows of the chunk][128 features]; the ring is free by now
  // parked tile: [row][128 features] fp32; ROWS pads a row to 132 floats so that the 16-byte writes of the 32 lanes
  // (one row each) do not collide
  constexpr uint32_t kPitch = ROWS ? 528u : 512u;
  for (int ch = 0; ch < nchunks; ++ch) {
    const int rows_ch = ROWS ? min(kBlockM, p.R - row0) : min(rc, p.R - ch * rc);
    if (warp >= 2 && ok) {
      const int quad = warp & 3, cg = (warp - 2) >> 2;
      const uint32_t taddr = tmem_base + ch * rp32 + (static_cast<uint32_t>(quad * 32) << 16);
      if (ROWS) {
        const int row_local = quad * 32 + lane;              // TMEM lane = row of the tile, columns = features
        for (int c = cg; c < kBlockM / 32; c += kEpiColGroups) {
          uint32_t acc[32];
          tmem_ld32(taddr + c * 32, acc);
          tmem_ld_wait();
          if (row_local < rows_ch) {
            const uint32_t dst = red + static_cast<uint32_t>(row_local) * kPitch + static_cast<uint32_t>(c * 32) * 4u;
#pragma unroll
            for (int q = 0; q < 8; ++q)
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + q * 16u), "r"(acc[q * 4]), "r"(acc[q * 4 + 1]),
                           "r"(acc[q * 4 + 2]), "r"(acc[q * 4 + 3]) : "memory");
          }
        }
      } else {
        for (int c = cg; c * 32 < rows_ch; c += kEpiColGroups) {   // TMEM lane = feature, columns = rows
          uint32_t acc[32];
          tmem_ld32(taddr + c * 32, acc);
          tmem_ld_wait();
          const uint32_t dst = red + static_cast<uint32_t>(c * 32) * 512u + static_cast<uint32_t>(quad * 32 + lane) * 4u;
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (c * 32 + i < rows_ch) asm volatile("st.shared.b32 [%0], %1;" ::"r"(dst + i * 512u), "r"(acc[i]) : "memory");
        }
      }
    }
    tc_fence_before();
    cluster_sync_all();
    if (warp >= 2 && ok) {
      const int rpr = (rows_ch + S - 1) / S;
      const int lo = sp * rpr, hi = min(rows_ch, lo + rpr);
      const int n4 = (et & 31) * 4, n = tile * kBlockM + n4;
      if (n < p.N) {
        uint32_t peer[8];
#pragma unroll
        for (int t = 0; t < 8; ++t) peer[t] = mapa_shared(red, static_cast<uint32_t>(t < S ? t : 0));
        for (int jj = lo + (et >> 5); jj < hi; jj += 8) {
          const uint32_t off = static_cast<uint32_t>(jj) * kPitch + static_cast<uint32_t>(n4) * 4u;
          float4 sum = ld_dsmem_f4(peer[0] + off);
#pragma unroll
          for (int t = 1; t < 8; ++t)
            if (t < S) {                        // rank order: the sum does not depend on timing
              const float4 v = ld_dsmem_f4(peer[t] + off);
              sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
            }
          skinny_store<EPI>(p, sum, row0 + ch * rc + jj, n);
        }
      }
    }
    __syncwarp();
    cluster_sync_all();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, tmem_cols);
  }
}

// ------------------------------------------------------------------------------------------------ host
template <int EPI, bool ROWS>
struct SkinnyState {
  static bool ready;
  static int max_clusters[9];        // resident clusters of size S (0: not launchable)
};
template <int EPI, bool ROWS> bool SkinnyState<EPI, ROWS>::ready = false;
template <int EPI, bool ROWS> int SkinnyState<EPI, ROWS>::max_clusters[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};

template <int EPI, bool ROWS>
static cudaError_t skinny_prepare_one() {
  using St = SkinnyState<EPI, ROWS>;
  if (St::ready) return cudaSuccess;
  cudaError_t err = cudaFuncSetAttribute(gemm_skinny_kernel<EPI, ROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSkinnySmemBytes);
  if (err != cudaSuccess) return err;
  int dev = 0, sms = 0;
  if ((err = cudaGetDevice(&dev)) != cudaSuccess) return err;
  if ((err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return err;
  for (int s = 1; s <= 8; ++s) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(sms / s * s);
    cfg.blockDim = dim3(kSkinnyThreads);
    cfg.dynamicSmemBytes = kSkinnySmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = s;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_skinny_kernel<EPI, ROWS>, &cfg) != cudaSuccess) {
      cudaGetLastError();            // this cluster size is not launchable here: leave it at 0
      n = 0;
    }
    St::max_clusters[s] = n;
  }
  St::ready = true;
  return cudaSuccess;
}

cudaError_t gemm_skinny_prepare() {
  cudaError_t e = skinny_prepare_one<EPI_F32, false>();
  if (e == cudaSuccess) e = skinny_prepare_one<EPI_BF16, false>();
  if (e == cudaSuccess) e = skinny_prepare_one<EPI_GELU_BF16, false>();
  if (e == cudaSuccess) e = skinny_prepare_one<EPI_QKV, false>();
  if (e == cudaSuccess) e = skinny_prepare_one<EPI_RESID, false>();
  if (e == cudaSuccess) e = skinny_prepare_one<EPI_F32, true>();
  if (e == cudaSuccess) e = skinny_prepare_one<EPI_BF16, true>();
  if (e == cudaSuccess) e = skinny_prepare_one<EPI_GELU_BF16, true>();
  if (e == cudaSuccess) e = skinny_prepare_one<EPI_QKV, true>();
  if (e == cudaSuccess) e = skinny_prepare_one<EPI_RESID, true>();
  return e;
}

bool gemm_skinny_supported(int epi, int R, int N, int K) {
  return epi != EPI_ARGMAX && R >= 1 && R <= 512 && N % 8 == 0 && K % 8 == 0 && N >= 8;
}

// Which of the two cluster-split modes, if any, beats the row-tiled kernels -- set from measurements in the step on B200
// (Infinity-2B-shaped GEMMs).  Narrow outputs (at most 2048 features: out-proj, cross-attention projections, fc2) have
// too few tiles to fill the SMs row-tiled and each CTA walks all of K: the 128 x 128-tile mode with the K range over a
// cluster wins for every row count up to 256, up to 512 with a long reduction (fc2: 25 -> 13 - 22 us).  It also beats
// the weight-streaming form there, down to 16 rows (a block at r = 16: 94.5 -> 90.6 us, at r = 59: 107.8 -> 100.3).
// Wide outputs (QKV, fc1) fill the SMs row-tiled from 33 rows on; below, the weight-streaming form wins (15.5 -> 7.8 us
// at R = 16) and the 128 x 128 mode does not (90.6 -> 93.9 us per block).
int gemm_skinny_row_limit(int N, int K) {
  (void)N; (void)K;
  return 32;
}

bool gemm_ksplit_wins(int R, int N, int K) {
  if (N > 2048) return false;
  if (R <= 256) return true;
  return K >= 4096 && R <= 512;
}

// K ranges per tile (128 features x all rows, or x 128 rows when row_tiles > 0 row tiles are given): the split whose
// slowest CTA walks the fewest K blocks while all clusters are resident at once.  Measured on B200: clusters of 7 or 8
// and grids above about 0.9 of the SMs (odd cluster sizes do not pack the GPCs) fall into a second wave and cost 1.5 -
// 2x, whatever the occupancy query says; the small form fits two CTAs per SM.  forced > 0 takes that split when it is
// launchable.
int gemm_skinny_pick_splits(int N, int K, int forced, int row_tiles, int small_form) {
  if (gemm_skinny_prepare() != cudaSuccess) return 0;
  const int *mc = row_tiles > 0 ? SkinnyState<EPI_RESID, true>::max_clusters : SkinnyState<EPI_RESID, false>::max_clusters;
  const int tiles = (N + kBlockM - 1) / kBlockM * (row_tiles > 0 ? row_tiles : 1), num_kb = (K + kBlockK - 1) / kBlockK;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int capacity = (small_form ? 2 : 1) * sms * 9 / 10;
  int best = 0;
  long long best_cost = 0;
  for (int s = 1; s <= 8; ++s) {
    if (mc[s] <= 0 || (forced > 0 && s != forced)) continue;
    const int kbps = (num_kb + s - 1) / s;
    if ((num_kb + kbps - 1) / kbps != s) continue;          // some range would be empty
    if (forced <= 0 && s > 1 && (kbps < 2 || s > 6 || tiles * s > capacity)) continue;
    const long long cost = 10ll * (kbps + 3) + s;            // K blocks of the slowest CTA plus fixed time; smaller clusters on ties
    if (best == 0 || cost < best_cost) { best = s; best_cost = cost; }
  }
  return best;
}

template <int EPI, bool ROWS>
static cudaError_t skinny_launch_one(const CUtensorMap &tmA, const CUtensorMap &tmW, const GemmArgs &a, cudaStream_t st) {
  cudaError_t err = skinny_prepare_one<EPI, ROWS>();
  if (err != cudaSuccess) return err;
  const int S = a.splits > 1 ? a.splits : 1;
  if (S > 8 || SkinnyState<EPI, ROWS>::max_clusters[S] <= 0) return cudaErrorInvalidValue;
  const int tiles = (a.N + kBlockM - 1) / kBlockM * (ROWS ? a.sk_tiles_m : 1);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(tiles * S);
  cfg.blockDim = dim3(kSkinnyThreads);
  cfg.dynamicSmemBytes = a.sk_small ? kSkinnySmemSmall : kSkinnySmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = S;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, gemm_skinny_kernel<EPI, ROWS>, tmA, tmW, a);
}

// Fills the chunking fields of `a` for R rows (R <= 512): rows per chunk, padded MMA width, stage count.
void gemm_skinny_shape(GemmArgs &a) {
  if (a.sk_tiles_m > 0) {                    // 128 x 128 tiles: two K blocks of each operand per stage, three stages
    a.sk_nchunks = 1; a.sk_rows_chunk = kBlockM; a.sk_rp = kBlockM; a.sk_small = 0;
    const int num_kb = (a.K + kBlockK - 1) / kBlockK, S = a.splits > 1 ? a.splits : 1;
    a.sk_nk = (a.K % kBlockK == 0 && (num_kb + S - 1) / S >= 2) ? 2 : 1;
    a.sk_stages = kSkinnyRing / (a.sk_nk * 2 * kSkinnyWAtom);
    if (a.sk_stages > kSkinnyMaxStages) a.sk_stages = kSkinnyMaxStages;
    return;
  }
  a.sk_nchunks = a.R > 256 ? 2 : 1;
  a.sk_rows_chunk = a.sk_nchunks == 1 ? a.R : (((a.R + 1) / 2 + 15) & ~15);
  a.sk_rp = (a.sk_rows_chunk + 15) & ~15;
  // K blocks per stage (one TMA instruction per operand; K must be whole blocks for the 3-D maps).  Up to 64 rows
  // the small ring is preferred: two CTAs share an SM, so the next GEMM of a chain is resident, set up and has
  // its first weights in shared memory while this one still computes.  Otherwise as many blocks per stage as
  // leave two stages in the large ring.
  const int kb_bytes = kSkinnyWAtom + a.sk_nchunks * a.sk_rp * kBlockK * 2;
  const int num_kb = (a.K + kBlockK - 1) / kBlockK, S = a.splits > 1 ? a.splits : 1;
  const int kbps = (num_kb + S - 1) / S;
  const bool whole = a.K % kBlockK == 0;
  a.sk_small = (a.sk_nchunks == 1 && a.sk_rp <= 64) ? 1 : 0;
  const int ring = a.sk_small ? kSkinnyRingSmall : kSkinnyRing;
  int nk = 1;
  if (whole)
    for (int c = 4; c > 1; c >>= 1)
      if (2 * c * kb_bytes <= ring && c <= kbps) { nk = c; break; }
  a.sk_nk = nk;
  const int stages = ring / (nk * kb_bytes);
  a.sk_stages = stages > kSkinnyMaxStages ? kSkinnyMaxStages : stages;
}

// Tensor map of a K-major bf16 matrix [rows][K] (row pitch ld elements) for this kernel: with nk > 1 the 3-D form
// {64, rows, K / 64} with box {64, box_rows, nk} (K a multiple of 64), else the plain 2-D form with box {64, box_rows}.
bool gemm_skinny_map(CUtensorMap *m, const void *base, uint64_t rows, uint64_t K, uint64_t ld, uint32_t box_rows, int nk) {
  if (nk <= 1) return tmap_2d(m, base, K, rows, ld, box_rows);
  return tmap_kblocks(m, base, rows, K / kBlockK, ld, box_rows, static_cast<uint32_t>(nk));
}

// tmA / tmW: gemm_skinny_map over the activation rows (box of a.sk_rp rows) and the weight rows (box of 128 rows).
// a.splits = cluster size, set before gemm_skinny_shape.
cudaError_t launch_gemm_skinny(int epi, const CUtensorMap &tmA, const CUtensorMap &tmW, const GemmArgs &a, cudaStream_t st) {
  if (a.nbatch != 1 || a.w_mn_major || a.sk_stages < 1 || epi == EPI_ARGMAX || a.N % 8 || a.K % 8 ||
      (a.sk_tiles_m <= 0 && !gemm_skinny_supported(epi, a.R, a.N, a.K)))
    return cudaErrorInvalidValue;
  if (a.sk_tiles_m > 0) {
    switch (epi) {
      case EPI_F32: return skinny_launch_one<EPI_F32, true>(tmA, tmW, a, st);
      case EPI_BF16: return skinny_launch_one<EPI_BF16, true>(tmA, tmW, a, st);
      case EPI_GELU_BF16: return skinny_launch_one<EPI_GELU_BF16, true>(tmA, tmW, a, st);
      case EPI_QKV: return skinny_launch_one<EPI_QKV, true>(tmA, tmW, a, st);
      case EPI_RESID: return skinny_launch_one<EPI_RESID, true>(tmA, tmW, a, st);
    }
    return cudaErrorInvalidValue;
  }
  switch (epi) {
    case EPI_F32: return skinny_launch_one<EPI_F32, false>(tmA, tmW, a, st);
    case EPI_BF16: return skinny_launch_one<EPI_BF16, false>(tmA, tmW, a, st);
    case EPI_GELU_BF16: return skinny_launch_one<EPI_GELU_BF16, false>(tmA, tmW, a, st);
    case EPI_QKV: return skinny_launch_one<EPI_QKV, false>(tmA, tmW, a, st);
    case EPI_RESID: return skinny_launch_one<EPI_RESID, false>(tmA, tmW, a, st);
  }
  return cudaErrorInvalidValue;
}

}  // namespace fvar
