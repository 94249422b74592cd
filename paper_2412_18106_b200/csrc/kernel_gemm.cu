// SmoothGEMM (Section 5): C[M,N] = A[M,K] W[N,K]^T on tcgen05, fixed 128 x kTileN tiles with
// virtual padding of M (TMA zero-fills rows past M; the epilogue stores rows below M only).
//
// One persistent CTA per SM, 192 threads:
//   warp 0, one lane   TMA producer: per 64-element K chunk one box of A (128 rows) and one of W
//                      (kTileN rows) into the next free stage of a shared-memory ring
//   warp 1, one lane   MMA issuer: four tcgen05.mma (K = 16 each) per chunk into one of two
//                      accumulators in tensor memory; tcgen05.commit frees the stage and, after
//                      the last chunk, hands the accumulator to the epilogue
//   warps 2-5          epilogue: tensor memory -> bf16 -> global (thread = row), then return the
//                      accumulator; runs while the issuer fills the other accumulator
// Every wait is bounded; on expiry the kernel records XY_ERR_DEVICE_TIMEOUT and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "ptx.cuh"
#include "xy_gemm.h"

namespace xy {
namespace {

using namespace ptx;

constexpr int kTileM = 128;
constexpr int kChunkK = 64;  // elements per K chunk = one 128-byte swizzle row
constexpr int kGemmThreads = 192;
constexpr int kABytes = kTileM * kChunkK * 2;  // 16 KiB
__device__ int32_t g_gemm_status;

template <int kTileN>
struct GemmCfg {
  static constexpr int kWBytes = kTileN * kChunkK * 2;
  static constexpr int kStageBytes = kABytes + kWBytes;
  static constexpr int kStages = kTileN == 256 ? 4 : (kTileN == 128 ? 6 : 8);
  static constexpr int kSmem = 1024 + kStages * kStageBytes + 256;
  static constexpr uint32_t kTmemCols = 2 * kTileN < 32 ? 32 : 2 * kTileN;  // two accumulators (power of two >= 32)
};

struct GemmParams {
  uint16_t* c;
  int64_t ldc;
  int32_t M, N, K;
  int32_t m_tiles, n_tiles;
  // Work split.  Tiles [0, wave_tiles) are computed whole, tile blockIdx.x + i * gridDim.x by CTA
  // blockIdx.x (wave_tiles is a multiple of the grid size).  The K chunks of the remaining sk_tiles
  // tiles form one line of sk_tiles * k_chunks units, of which CTA b takes units [b * upc, (b + 1) * upc):
  // at most two segments, each part of one tile (upc <= k_chunks).
  int32_t wave_tiles, sk_tiles, upc;
  float* ws;     // partial sums: slot 2 b + s of CTA b's segment s, [kTileN / 4][128] float4
  int32_t grid;  // CTAs of the GEMM kernel (the fix-up kernel derives the segments from it)
};

// One piece of work of a CTA: K chunks [kc_lo, kc_hi) of a tile; slot < 0: the whole tile.
struct GemmItem {
  int tile, kc_lo, kc_hi, slot;
};
__device__ __forceinline__ bool gemm_item(const GemmParams& P, int k_chunks, int idx, GemmItem& it) {
  const int G = static_cast<int>(gridDim.x), b = static_cast<int>(blockIdx.x);
  if (b + idx * G < P.wave_tiles) {
    it.tile = b + idx * G;
    it.kc_lo = 0;
    it.kc_hi = k_chunks;
    it.slot = -1;
    return true;
  }
  if (P.sk_tiles == 0) return false;
  const int s = idx - P.wave_tiles / G;  // with split tiles, wave_tiles is a multiple of the grid size
  if (s < 0 || s > 1) return false;
  const int u0 = b * P.upc, u1 = min(u0 + P.upc, P.sk_tiles * k_chunks);
  if (u0 >= u1) return false;
  const int first = u0 / k_chunks;
  const int lo = s == 0 ? u0 : (first + 1) * k_chunks;
  const int hi = s == 0 ? min(u1, (first + 1) * k_chunks) : u1;
  if (lo >= hi) return false;
  it.tile = P.wave_tiles + first + s;
  it.kc_lo = lo - (first + s) * k_chunks;
  it.kc_hi = hi - (first + s) * k_chunks;
  it.slot = (it.kc_lo == 0 && it.kc_hi == k_chunks) ? -1 : 2 * b + s;
  return true;
}

struct __align__(8) GemmBarriers {
  uint64_t full[8], empty[8];
  uint64_t acc_full[2], acc_empty[2];
  uint32_t tmem_base;
};

template <int kTileN>
__global__ void __launch_bounds__(kGemmThreads, 1)
smooth_gemm_kernel(const GemmParams P, const __grid_constant__ CUtensorMap a_map,
                   const __grid_constant__ CUtensorMap w_map) {
  using Cfg = GemmCfg<kTileN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  GemmBarriers* bars =
      reinterpret_cast<GemmBarriers*>(smem_raw + (base - smem_u32(smem_raw)) + Cfg::kStages * Cfg::kStageBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const volatile int32_t* status = &g_gemm_status;
  if (threadIdx.x == 0) {
    for (int s = 0; s < Cfg::kStages; ++s) {
      mbar_init(smem_u32(&bars->full[s]), 1);
      mbar_init(smem_u32(&bars->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars->acc_full[b]), 1);
      mbar_init(smem_u32(&bars->acc_empty[b]), 4);
    }
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&bars->tmem_base), Cfg::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  const int num_tiles = P.m_tiles * P.n_tiles;
  const int k_chunks = (P.K + kChunkK - 1) / kChunkK;

  if (warp == 0 && lane == 0) {
    // ---------------------------------------------------------------- producer
    prefetch_tensormap(&a_map);
    prefetch_tensormap(&w_map);
    uint32_t pos = 0;
    bool dead = false;
    GemmItem it;
    for (int idx = 0; !dead && gemm_item(P, k_chunks, idx, it); ++idx) {
      const int t = it.tile;
      const int m0 = (t % P.m_tiles) * kTileM, n0 = (t / P.m_tiles) * kTileN;
      for (int kc = it.kc_lo; kc < it.kc_hi; ++kc, ++pos) {
        const uint32_t s = pos % Cfg::kStages, use = pos / Cfg::kStages;
        if (use > 0 && !mbar_wait(smem_u32(&bars->empty[s]), (use - 1) & 1u, status)) {
          atomicExch(&g_gemm_status, XY_ERR_DEVICE_TIMEOUT);
          dead = true;
          break;
        }
        const uint32_t full = smem_u32(&bars->full[s]);
        mbar_arrive_expect_tx(full, Cfg::kStageBytes);
        const uint32_t dst = base + s * Cfg::kStageBytes;
        tma_load_2d(dst, &a_map, full, kc * kChunkK, m0);           // rows past M arrive as zeros
        tma_load_2d(dst + kABytes, &w_map, full, kc * kChunkK, n0);  // rows past N likewise
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------------------------------------------------------- MMA issuer
    // Shared-memory descriptors: K-major operands in the 128-byte swizzle, 8-row groups 1024 B
    // apart; a K step of 16 elements advances the start address by 32 B.
    constexpr uint64_t kDescHi = static_cast<uint64_t>((1024u >> 4) | (1u << 14) | (2u << 29)) << 32;
    constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((static_cast<uint32_t>(kTileN) >> 3) << 17) |
                                ((static_cast<uint32_t>(kTileM) >> 4) << 24);
    uint32_t pos = 0, local = 0;
    bool dead = false;
    GemmItem it;
    for (int idx = 0; !dead && gemm_item(P, k_chunks, idx, it); ++idx, ++local) {
      const uint32_t buf = local & 1u, use = local >> 1;
      if (use > 0 && !mbar_wait(smem_u32(&bars->acc_empty[buf]), (use - 1) & 1u, status)) {
        atomicExch(&g_gemm_status, XY_ERR_DEVICE_TIMEOUT);
        break;
      }
      tc_fence_after();
      const uint32_t d_tmem = tmem + buf * kTileN;
      for (int kc = it.kc_lo; kc < it.kc_hi; ++kc, ++pos) {
        const uint32_t s = pos % Cfg::kStages;
        if (!mbar_wait(smem_u32(&bars->full[s]), (pos / Cfg::kStages) & 1u, status)) {
          atomicExch(&g_gemm_status, XY_ERR_DEVICE_TIMEOUT);
          dead = true;
          break;
        }
        tc_fence_after();
        const uint32_t a_lo = (((base + s * Cfg::kStageBytes) >> 4) & 0x3FFFu) | (1u << 16);
        const uint32_t w_lo = (((base + s * Cfg::kStageBytes + kABytes) >> 4) & 0x3FFFu) | (1u << 16);
#pragma unroll
        for (int k16 = 0; k16 < 4; ++k16)
          umma_ss64(d_tmem, kDescHi | (a_lo + k16 * 2), kDescHi | (w_lo + k16 * 2), kIdesc,
                    (kc > it.kc_lo || k16) ? 1u : 0u);
        umma_commit(smem_u32(&bars->empty[s]));  // the stage is free once these MMAs have read it
      }
      if (!dead) umma_commit(smem_u32(&bars->acc_full[buf]));
    }
  } else if (warp >= 2) {
    // ---------------------------------------------------------------- epilogue
    const int q = warp & 3;  // tensor-memory lanes 32 q .. 32 q + 31 belong to this warp
    const int row_in_tile = q * 32 + lane;
    uint32_t local = 0;
    GemmItem it;
    for (int idx = 0; gemm_item(P, k_chunks, idx, it); ++idx, ++local) {
      const uint32_t buf = local & 1u;
      if (!mbar_wait(smem_u32(&bars->acc_full[buf]), (local >> 1) & 1u, status)) {
        atomicExch(&g_gemm_status, XY_ERR_DEVICE_TIMEOUT);
        break;
      }
      tc_fence_after();
      const int t = it.tile;
      const int m0 = (t % P.m_tiles) * kTileM, n0 = (t / P.m_tiles) * kTileN;
      const int row = m0 + row_in_tile;
      const uint32_t t_acc = tmem + (static_cast<uint32_t>(q * 32) << 16) + buf * kTileN;
      uint16_t* crow = P.c + static_cast<int64_t>(row) * P.ldc + n0;
      if (it.slot < 0) {
#pragma unroll 2
        for (int c0 = 0; c0 < kTileN; c0 += 32) {
          uint32_t v[32];
          tmem_ld_32x32b_x32(t_acc + c0, v);
          tmem_wait_ld();
          if (row < P.M) {  // selective write: virtual padding rows are never stored
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              if (n0 + c0 + g * 8 < P.N) {
                uint4 o;
                o.x = pack_bf16(__uint_as_float(v[g * 8 + 0]), __uint_as_float(v[g * 8 + 1]));
                o.y = pack_bf16(__uint_as_float(v[g * 8 + 2]), __uint_as_float(v[g * 8 + 3]));
                o.z = pack_bf16(__uint_as_float(v[g * 8 + 4]), __uint_as_float(v[g * 8 + 5]));
                o.w = pack_bf16(__uint_as_float(v[g * 8 + 6]), __uint_as_float(v[g * 8 + 7]));
                *reinterpret_cast<uint4*>(crow + c0 + g * 8) = o;
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars->acc_empty[buf]));
        continue;
      }
      // A segment of a split tile: leave the fp32 partial sums in this segment's slot (column
      // group by column group, 128 consecutive rows each: coalesced).  gemm_fixup_kernel, launched
      // behind this kernel, adds a tile's segments in the order of the CTAs and stores the tile.
      // (Letting the segment that arrives last add them was measured first: one CTA then reads
      // every partial sum of its tile with 32 - 64 KiB in flight, 20 - 40 us for a 128 x 256 tile.)
      float4* slot = reinterpret_cast<float4*>(P.ws) + static_cast<int64_t>(it.slot) * (kTileN / 4) * kTileM;
#pragma unroll 2
      for (int c0 = 0; c0 < kTileN; c0 += 32) {
        uint32_t v[32];
        tmem_ld_32x32b_x32(t_acc + c0, v);
        tmem_wait_ld();
#pragma unroll
        for (int g = 0; g < 8; ++g)
          slot[(c0 / 4 + g) * kTileM + row_in_tile] =
              make_float4(__uint_as_float(v[4 * g]), __uint_as_float(v[4 * g + 1]), __uint_as_float(v[4 * g + 2]),
                          __uint_as_float(v[4 * g + 3]));
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->acc_empty[buf]));
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, Cfg::kTmemCols);
  }
}


// ------------------------------------------------------------------------------------------
// CTA-pair variant for large problems: a cluster of two CTAs computes a 256 x kTileN tile with
// tcgen05.mma.cta_group::2 (M = 256).  CTA r holds rows [128 r, 128 r + 128) of the tile's A and of
// its accumulator and stages rows [kTileN / 2 * r, + kTileN / 2) of W: per 64-element K chunk a CTA
// loads 16 KiB of A and kTileN * 64 bytes of W for 256 x kTileN x 64 multiply-adds of the pair,
// two thirds of the single-CTA kernel's operand bytes per flop (what the full waves of the
// single-CTA kernel are bound by: 28 us per wave against 22 us of MMAs), and an MMA of the pair
// costs 64 cycles per 128 columns against 81.  Every CTA issues its own copies (no multicast);
// their bytes are counted on the leader's barrier; completions (tcgen05.commit) arrive in both
// CTAs; the peer's epilogue warps return an accumulator with a remote arrive.
template <int kTileN>
struct PairGemmCfg {
  static constexpr int kWBytes = (kTileN / 2) * kChunkK * 2;
  static constexpr int kStageBytes = kABytes + kWBytes;
  static constexpr int kStages = kTileN == 256 ? 6 : 8;
  static constexpr int kSmem = 1024 + kStages * kStageBytes + 256;
  static constexpr uint32_t kTmemCols = 2 * kTileN;
};

template <int kTileN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
smooth_gemm_pair_kernel(const GemmParams P, const __grid_constant__ CUtensorMap a_map,
                        const __grid_constant__ CUtensorMap w_map) {
  using Cfg = PairGemmCfg<kTileN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  GemmBarriers* bars =
      reinterpret_cast<GemmBarriers*>(smem_raw + (base - smem_u32(smem_raw)) + Cfg::kStages * Cfg::kStageBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const volatile int32_t* status = &g_gemm_status;
  if (threadIdx.x == 0) {
    for (int s = 0; s < Cfg::kStages; ++s) {
      mbar_init(smem_u32(&bars->full[s]), 1);   // leader: one arming arrive, bytes of both CTAs
      mbar_init(smem_u32(&bars->empty[s]), 1);  // each CTA: one commit
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars->acc_full[b]), 1);   // each CTA: one commit
      mbar_init(smem_u32(&bars->acc_empty[b]), 8);  // leader: four epilogue warps of each CTA
    }
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(&bars->tmem_base), Cfg::kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  const int num_tiles = P.m_tiles * P.n_tiles;  // m_tiles counts 256-row tiles here
  const int k_chunks = (P.K + kChunkK - 1) / kChunkK;
  const int cluster = static_cast<int>(blockIdx.x >> 1), clusters = static_cast<int>(gridDim.x >> 1);
  auto wait_cluster = [&](uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < (1u << 22); ++i) {
      if (mbar_try_wait_cluster(bar, parity)) return true;
      if ((i & 4095u) == 4095u && status[0] != 0) return false;
    }
    return false;
  };

  if (warp == 0 && lane == 0) {
    // ---------------------------------------------------------------- producer (both CTAs)
    prefetch_tensormap(&a_map);
    prefetch_tensormap(&w_map);
    const uint32_t full_leader = cluster_map(smem_u32(&bars->full[0]), 0);
    uint32_t pos = 0;
    bool dead = false;
    for (int t = cluster; t < num_tiles && !dead; t += clusters) {
      const int m0 = (t % P.m_tiles) * 256 + 128 * static_cast<int>(rank);
      const int n0 = (t / P.m_tiles) * kTileN + (kTileN / 2) * static_cast<int>(rank);
      for (int kc = 0; kc < k_chunks; ++kc, ++pos) {
        const uint32_t s = pos % Cfg::kStages, use = pos / Cfg::kStages;
        if (use > 0 && !wait_cluster(smem_u32(&bars->empty[s]), (use - 1) & 1u)) {
          atomicExch(&g_gemm_status, XY_ERR_DEVICE_TIMEOUT);
          dead = true;
          break;
        }
        if (leader) mbar_arrive_expect_tx(smem_u32(&bars->full[s]), 2 * Cfg::kStageBytes);
        const uint32_t dst = base + s * Cfg::kStageBytes, bar = full_leader + s * 8u;
        tma_load_2d_pair(dst, &a_map, bar, kc * kChunkK, m0);           // rows past M arrive as zeros
        tma_load_2d_pair(dst + kABytes, &w_map, bar, kc * kChunkK, n0);  // rows past N likewise
      }
    }
  } else if (warp == 1 && lane == 0 && leader) {
    // ---------------------------------------------------------------- MMA issuer (leader)
    constexpr uint64_t kDescHi = static_cast<uint64_t>((1024u >> 4) | (1u << 14) | (2u << 29)) << 32;
    constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((static_cast<uint32_t>(kTileN) >> 3) << 17) |
                                ((256u >> 4) << 24);
    uint32_t pos = 0, local = 0;
    bool dead = false;
    for (int t = cluster; t < num_tiles && !dead; t += clusters, ++local) {
      const uint32_t buf = local & 1u, use = local >> 1;
      if (use > 0 && !wait_cluster(smem_u32(&bars->acc_empty[buf]), (use - 1) & 1u)) {
        atomicExch(&g_gemm_status, XY_ERR_DEVICE_TIMEOUT);
        break;
      }
      tc_fence_after();
      const uint32_t d_tmem = tmem + buf * kTileN;
      for (int kc = 0; kc < k_chunks; ++kc, ++pos) {
        const uint32_t s = pos % Cfg::kStages;
        if (!wait_cluster(smem_u32(&bars->full[s]), (pos / Cfg::kStages) & 1u)) {
          atomicExch(&g_gemm_status, XY_ERR_DEVICE_TIMEOUT);
          dead = true;
          break;
        }
        tc_fence_after();
        const uint32_t a_lo = (((base + s * Cfg::kStageBytes) >> 4) & 0x3FFFu) | (1u << 16);
        const uint32_t w_lo = (((base + s * Cfg::kStageBytes + kABytes) >> 4) & 0x3FFFu) | (1u << 16);
#pragma unroll
        for (int k16 = 0; k16 < 4; ++k16)
          umma2_ss64(d_tmem, kDescHi | (a_lo + k16 * 2), kDescHi | (w_lo + k16 * 2), kIdesc, (kc | k16) ? 1u : 0u);
        umma2_commit_both(smem_u32(&bars->empty[s]));  // the stage is free in both CTAs
      }
      if (!dead) umma2_commit_both(smem_u32(&bars->acc_full[buf]));
    }
  } else if (warp >= 2) {
    // ---------------------------------------------------------------- epilogue (both CTAs)
    const int q = warp & 3;
    const int row_in_tile = q * 32 + lane;
    const uint32_t acc_empty_leader = cluster_map(smem_u32(&bars->acc_empty[0]), 0);
    uint32_t local = 0;
    for (int t = cluster; t < num_tiles; t += clusters, ++local) {
      const uint32_t buf = local & 1u;
      if (!wait_cluster(smem_u32(&bars->acc_full[buf]), (local >> 1) & 1u)) {
        atomicExch(&g_gemm_status, XY_ERR_DEVICE_TIMEOUT);
        break;
      }
      tc_fence_after();
      const int m0 = (t % P.m_tiles) * 256 + 128 * static_cast<int>(rank), n0 = (t / P.m_tiles) * kTileN;
      const int row = m0 + row_in_tile;
      const uint32_t t_acc = tmem + (static_cast<uint32_t>(q * 32) << 16) + buf * kTileN;
      uint16_t* crow = P.c + static_cast<int64_t>(row) * P.ldc + n0;
#pragma unroll 2
      for (int c0 = 0; c0 < kTileN; c0 += 32) {
        uint32_t v[32];
        tmem_ld_32x32b_x32(t_acc + c0, v);
        tmem_wait_ld();
        if (row < P.M) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            if (n0 + c0 + g * 8 < P.N) {
              uint4 o;
              o.x = pack_bf16(__uint_as_float(v[g * 8 + 0]), __uint_as_float(v[g * 8 + 1]));
              o.y = pack_bf16(__uint_as_float(v[g * 8 + 2]), __uint_as_float(v[g * 8 + 3]));
              o.z = pack_bf16(__uint_as_float(v[g * 8 + 4]), __uint_as_float(v[g * 8 + 5]));
              o.w = pack_bf16(__uint_as_float(v[g * 8 + 6]), __uint_as_float(v[g * 8 + 7]));
              *reinterpret_cast<uint4*>(crow + c0 + g * 8) = o;
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (leader) mbar_arrive(smem_u32(&bars->acc_empty[buf])); else mbar_arrive_remote(acc_empty_leader + buf * 8u);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // neither CTA leaves while the other may still touch its memory
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem, Cfg::kTmemCols);
  }
}

// Adds the partial sums of the split tiles and stores them.  Grid: (column blocks of 32, split
// tiles); 128 threads = the tile's rows.  The segments of tile sk belong to the consecutive CTAs
// whose unit ranges meet [sk * k_chunks, (sk + 1) * k_chunks); a tile with one segment was stored
// whole by the GEMM kernel.  Every load of a thread is independent of the others (up to 8 per
// segment in flight), and the sum runs in the order of the CTAs: bit-reproducible.
template <int kTileN>
__global__ void __launch_bounds__(128) gemm_fixup_kernel(const GemmParams P) {
  const int sk = blockIdx.y, k_chunks = (P.K + kChunkK - 1) / kChunkK;
  const int b_first = (sk * k_chunks) / P.upc, b_last = ((sk + 1) * k_chunks - 1) / P.upc;
  if (b_first == b_last) return;
  const int t = P.wave_tiles + sk;
  const int m0 = (t % P.m_tiles) * kTileM, n0 = (t / P.m_tiles) * kTileN;
  const int row_in_tile = threadIdx.x, row = m0 + row_in_tile;
  const int c0 = blockIdx.x * 32;
  float4 acc[8];
#pragma unroll
  for (int g = 0; g < 8; ++g) acc[g] = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int bb = b_first; bb <= b_last; ++bb) {
    const int seg = sk - (bb * P.upc) / k_chunks;  // 0 or 1: which of that CTA's segments is this tile
    const float4* src = reinterpret_cast<const float4*>(P.ws) +
                        static_cast<int64_t>(2 * bb + seg) * (kTileN / 4) * kTileM + row_in_tile;
    float4 x[8];
#pragma unroll
    for (int g = 0; g < 8; ++g) x[g] = __ldcg(src + (c0 / 4 + g) * kTileM);
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      acc[g].x += x[g].x;
      acc[g].y += x[g].y;
      acc[g].z += x[g].z;
      acc[g].w += x[g].w;
    }
  }
  if (row >= P.M) return;
  uint16_t* crow = P.c + static_cast<int64_t>(row) * P.ldc + n0;
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    if (n0 + c0 + g * 8 < P.N) {
      uint4 o;
      o.x = pack_bf16(acc[2 * g].x, acc[2 * g].y);
      o.y = pack_bf16(acc[2 * g].z, acc[2 * g].w);
      o.z = pack_bf16(acc[2 * g + 1].x, acc[2 * g + 1].y);
      o.w = pack_bf16(acc[2 * g + 1].z, acc[2 * g + 1].w);
      *reinterpret_cast<uint4*>(crow + c0 + g * 8) = o;
    }
  }
}

// ------------------------------------------------------------------------------------------
// Split-K variant for small token counts (few tiles).  A whole-K tile is one serial
// chain of K/64 chunks on one SM, and with fewer tiles than SMs most of the chip idles while the
// weights stream through a few SMs.  Here a cluster of `splits` CTAs shares one 128 x 128 tile:
// CTA r computes the partial product over its slice of K, writes the valid rows of its fp32
// accumulator into its own shared memory, and after a cluster barrier every CTA adds the slices
// of the rows it owns (row mod splits = rank) through distributed shared memory and stores those
// bf16 rows.  One tile per CTA.
struct SplitKParams {
  uint16_t* c;
  int64_t ldc;
  int32_t M, N, K;
  int32_t splits, chunks_per_split, m_tiles;
};

__global__ void __launch_bounds__(kGemmThreads, 1)
smooth_gemm_splitk_kernel(const SplitKParams P, const __grid_constant__ CUtensorMap a_map,
                          const __grid_constant__ CUtensorMap w_map) {
  constexpr int kTileN = 128;
  using Cfg = GemmCfg<kTileN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
  GemmBarriers* bars = reinterpret_cast<GemmBarriers*>(gen_base + Cfg::kStages * Cfg::kStageBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const volatile int32_t* status = &g_gemm_status;
  const uint32_t rank = cluster_ctarank();
  const int tile = static_cast<int>(blockIdx.x / P.splits);
  const int m0 = (tile % P.m_tiles) * kTileM, n0 = (tile / P.m_tiles) * kTileN;
  const int m_rows = min(kTileM, P.M - m0);  // valid rows of this tile
  const int k_chunks = (P.K + kChunkK - 1) / kChunkK;
  const int kc_lo = static_cast<int>(rank) * P.chunks_per_split;
  const int kc_hi = min(k_chunks, kc_lo + P.chunks_per_split);
  const int my_chunks = max(0, kc_hi - kc_lo);
  if (threadIdx.x == 0) {
    for (int s = 0; s < Cfg::kStages; ++s) {
      mbar_init(smem_u32(&bars->full[s]), 1);
      mbar_init(smem_u32(&bars->empty[s]), 1);
    }
    mbar_init(smem_u32(&bars->acc_full[0]), 1);
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&bars->tmem_base), 128);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  if (warp == 0 && lane == 0) {
    prefetch_tensormap(&a_map);
    prefetch_tensormap(&w_map);
    for (int i = 0; i < my_chunks; ++i) {
      const uint32_t s = i % Cfg::kStages, use = i / Cfg::kStages;
      if (use > 0 && !mbar_wait(smem_u32(&bars->empty[s]), (use - 1) & 1u, status)) {
        atomicExch(&g_gemm_status, XY_ERR_DEVICE_TIMEOUT);
        break;
      }
      const uint32_t full = smem_u32(&bars->full[s]);
      mbar_arrive_expect_tx(full, Cfg::kStageBytes);
      const uint32_t dst = base + s * Cfg::kStageBytes;
      tma_load_2d(dst, &a_map, full, (kc_lo + i) * kChunkK, m0);
      tma_load_2d(dst + kABytes, &w_map, full, (kc_lo + i) * kChunkK, n0);
    }
  } else if (warp == 1 && lane == 0) {
    constexpr uint64_t kDescHi = static_cast<uint64_t>((1024u >> 4) | (1u << 14) | (2u << 29)) << 32;
    constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((static_cast<uint32_t>(kTileN) >> 3) << 17) |
                                ((static_cast<uint32_t>(kTileM) >> 4) << 24);
    bool dead = false;
    for (int i = 0; i < my_chunks; ++i) {
      const uint32_t s = i % Cfg::kStages;
      if (!mbar_wait(smem_u32(&bars->full[s]), (i / Cfg::kStages) & 1u, status)) {
        atomicExch(&g_gemm_status, XY_ERR_DEVICE_TIMEOUT);
        dead = true;
        break;
      }
      tc_fence_after();
      const uint32_t a_lo = (((base + s * Cfg::kStageBytes) >> 4) & 0x3FFFu) | (1u << 16);
      const uint32_t w_lo = (((base + s * Cfg::kStageBytes + kABytes) >> 4) & 0x3FFFu) | (1u << 16);
#pragma unroll
      for (int k16 = 0; k16 < 4; ++k16)
        umma_ss64(tmem, kDescHi | (a_lo + k16 * 2), kDescHi | (w_lo + k16 * 2), kIdesc, (i | k16) ? 1u : 0u);
      umma_commit(smem_u32(&bars->empty[s]));
    }
    if (!dead && my_chunks > 0) umma_commit(smem_u32(&bars->acc_full[0]));
  }
  // ---- every CTA: valid rows of the partial accumulator -> own shared memory (fp32, row r at
  // r * 512 B, 16-byte chunks XOR-swizzled by row so that a warp's 32 rows do not collide).
  // The ring is free by then: acc_full completes only after every MMA has read its stage.
  bool ok = true;
  if (warp >= 2) {
    const int q = warp & 3;
    const int row = q * 32 + lane;
    if (my_chunks > 0) {
      if (!mbar_wait(smem_u32(&bars->acc_full[0]), 0u, status)) {
        atomicExch(&g_gemm_status, XY_ERR_DEVICE_TIMEOUT);
        ok = false;
      }
      tc_fence_after();
    }
    if (ok && q * 32 < m_rows) {  // warps whose 32 rows are all padding skip the copy
      const uint32_t t_acc = tmem + (static_cast<uint32_t>(q * 32) << 16);
#pragma unroll 1
      for (int c0 = 0; c0 < kTileN; c0 += 32) {
        uint32_t v[32];
        if (my_chunks > 0) {
          tmem_ld_32x32b_x32(t_acc + c0, v);
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = 0u;
        }
        if (row < m_rows) {
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            const int chunk = (c0 >> 2) + g;
            *reinterpret_cast<uint4*>(gen_base + row * 512 + ((chunk ^ (row & 31)) << 4)) =
                make_uint4(v[g * 4 + 0], v[g * 4 + 1], v[g * 4 + 2], v[g * 4 + 3]);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncwarp();
  cluster_sync_all();
  if (warp >= 2) {
    // Reduce-scatter: CTA r owns the rows congruent to r modulo `splits`; its 128 epilogue threads
    // add that row's slices of all CTAs (thread t: 16-byte chunk t & 31 of every fourth owned
    // row) through distributed shared memory and store the bf16 row.  Two rows are in flight per
    // thread so that the remote loads overlap.
    const int t = threadIdx.x - 64;
    const int chunk = t & 31;
    const int col = n0 + chunk * 4;
    const int step = 4 * P.splits;
    auto reduce_row = [&](int row, float4& acc) {
      const uint32_t off = static_cast<uint32_t>(row * 512 + ((chunk ^ (row & 31)) << 4));
      acc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int r = 0; r < P.splits; ++r) {
        const float4 v = ld_cluster_f4(cluster_map(base + off, static_cast<uint32_t>(r)));
        acc.x += v.x;
        acc.y += v.y;
        acc.z += v.z;
        acc.w += v.w;
      }
    };
    auto store_row = [&](int row, const float4& acc) {
      if (col < P.N) {  // N is a multiple of 8, chunks of 4 columns are all in or all out
        uint2 o;
        o.x = pack_bf16(acc.x, acc.y);
        o.y = pack_bf16(acc.z, acc.w);
        *reinterpret_cast<uint2*>(P.c + static_cast<int64_t>(m0 + row) * P.ldc + col) = o;
      }
    };
    const int m_end = m_rows;
    int row = static_cast<int>(rank) + P.splits * (t >> 5);
    for (; row + step < m_end; row += 2 * step) {
      float4 a0, a1;
      reduce_row(row, a0);
      reduce_row(row + step, a1);
      store_row(row, a0);
      store_row(row + step, a1);
    }
    if (row < m_end) {
      float4 a0;
      reduce_row(row, a0);
      store_row(row, a0);
    }
  }
  __syncwarp();
  cluster_sync_all();  // every CTA's shared memory stays alive until all of them have read it
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 128);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn gemm_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// 2-D map over a row-major bf16 matrix [rows, K] with row stride ld: box = 64 elements x box_rows.
bool encode_matrix_map(CUtensorMap* m, const void* ptr, int64_t rows, int64_t K, int64_t ld, int box_rows) {
  EncodeTiledFn fn = gemm_encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(rows)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld) * 2};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(kChunkK), static_cast<cuuint32_t>(box_rows)};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Bytes of scratch the split of the last, partial wave of tiles needs: two partial-sum slots of a
// 128 x kTileN fp32 tile per CTA.
constexpr int64_t gemm_workspace_bytes(int tile_n, int num_sms) {
  return static_cast<int64_t>(num_sms) * 2 * kTileM * tile_n * 4;
}

template <int kTileN>
cudaError_t launch_gemm(const void* a, int64_t lda, const void* w, int64_t ldw, void* c, int64_t ldc, int M, int N,
                        int K, int num_sms, void* workspace, int64_t workspace_bytes, cudaStream_t s) {
  using Cfg = GemmCfg<kTileN>;
  auto kernel = smooth_gemm_kernel<kTileN>;
  static bool attr_set[64] = {false};  // per device: the opt-in to large dynamic shared memory
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  CUtensorMap a_map, w_map;
  if (!encode_matrix_map(&a_map, a, M, K, lda, kTileM) || !encode_matrix_map(&w_map, w, N, K, ldw, kTileN))
    return cudaErrorInvalidValue;
  GemmParams P;
  P.c = static_cast<uint16_t*>(c);
  P.ldc = ldc;
  P.M = M;
  P.N = N;
  P.K = K;
  P.m_tiles = (M + kTileM - 1) / kTileM;
  P.n_tiles = (N + kTileN - 1) / kTileN;
  const int tiles = P.m_tiles * P.n_tiles, k_chunks = (K + kChunkK - 1) / kChunkK;
  int grid = tiles < num_sms ? tiles : num_sms;
  P.wave_tiles = tiles;
  P.sk_tiles = 0;
  P.upc = k_chunks;
  P.ws = nullptr;
  // With scratch memory, the tiles of the last, partial wave are split along K over every SM when
  // the chain of K chunks is long: a tile is a serial chain on one SM, so a last wave of few
  // tiles otherwise costs a whole tile time.  Measured on the Linear shapes at M = 4096: Down
  // (K = 14336, 512 tiles = 3.46 waves) 401 -> 358 us; with K = 4096 the split tail and its fix-up
  // cost what the shorter wave saves (QKV 155 -> 158 us: full waves there run at the L2's pace,
  // 28 us per wave against 22 us of MMAs, and a thin last wave is already cheaper than a full
  // one), so chains under 128 chunks are left whole.  With fewer tiles than SMs (M <= 512) the
  // split was level with whole tiles (QKV M = 256: 26.3 against 25.3 us) and is not used.
  const int rest = tiles % num_sms;
  if (kTileN >= 32 && workspace != nullptr && workspace_bytes >= gemm_workspace_bytes(kTileN, num_sms) &&
      tiles > num_sms && rest > 0 && k_chunks >= 128 && rest * 5 <= num_sms * 3) {
    const int units = rest * k_chunks;
    P.wave_tiles = tiles - rest;
    P.sk_tiles = rest;
    P.upc = (units + grid - 1) / grid;
    P.ws = static_cast<float*>(workspace);
  }
  P.grid = grid;
  kernel<<<grid, kGemmThreads, Cfg::kSmem, s>>>(P, a_map, w_map);
  if (P.sk_tiles > 0)
    gemm_fixup_kernel<kTileN><<<dim3(kTileN / 32, P.sk_tiles), 128, 0, s>>>(P);
  return cudaGetLastError();
}


template <int kTileN>
cudaError_t launch_gemm_pair(const void* a, int64_t lda, const void* w, int64_t ldw, void* c, int64_t ldc, int M, int N,
                             int K, int num_sms, cudaStream_t s) {
  using Cfg = PairGemmCfg<kTileN>;
  auto kernel = smooth_gemm_pair_kernel<kTileN>;
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  CUtensorMap a_map, w_map;
  if (!encode_matrix_map(&a_map, a, M, K, lda, kTileM) || !encode_matrix_map(&w_map, w, N, K, ldw, kTileN / 2))
    return cudaErrorInvalidValue;
  GemmParams P = {};
  P.c = static_cast<uint16_t*>(c);
  P.ldc = ldc;
  P.M = M;
  P.N = N;
  P.K = K;
  P.m_tiles = (M + 255) / 256;
  P.n_tiles = (N + kTileN - 1) / kTileN;
  const int tiles = P.m_tiles * P.n_tiles, clusters = num_sms / 2;
  const int grid = 2 * (tiles < clusters ? tiles : clusters);
  kernel<<<grid, kGemmThreads, Cfg::kSmem, s>>>(P, a_map, w_map);
  return cudaGetLastError();
}

cudaError_t launch_gemm_splitk(const void* a, int64_t lda, const void* w, int64_t ldw, void* c, int64_t ldc, int M,
                               int N, int K, int splits, cudaStream_t s) {
  using Cfg = GemmCfg<128>;
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    e = cudaFuncSetAttribute(smooth_gemm_splitk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  CUtensorMap a_map, w_map;
  if (!encode_matrix_map(&a_map, a, M, K, lda, kTileM) || !encode_matrix_map(&w_map, w, N, K, ldw, 128))
    return cudaErrorInvalidValue;
  SplitKParams P;
  P.c = static_cast<uint16_t*>(c);
  P.ldc = ldc;
  P.M = M;
  P.N = N;
  P.K = K;
  P.splits = splits;
  const int k_chunks = (K + kChunkK - 1) / kChunkK;
  P.chunks_per_split = (k_chunks + splits - 1) / splits;
  const int n_tiles = (N + 127) / 128;
  P.m_tiles = (M + kTileM - 1) / kTileM;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(P.m_tiles * n_tiles * splits), 1, 1);
  cfg.blockDim = dim3(kGemmThreads, 1, 1);
  cfg.dynamicSmemBytes = Cfg::kSmem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(splits);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, smooth_gemm_splitk_kernel, P, a_map, w_map);
}

}  // namespace
}  // namespace xy

extern "C" int64_t xy_gemm_workspace_bytes(void) {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
    return -1;
  return xy::gemm_workspace_bytes(256, sms);
}

extern "C" int xy_gemm_run(const void* a, int64_t lda, const void* w, int64_t ldw, void* c, int64_t ldc, int32_t M,
                           int32_t N, int32_t K, int32_t tile_n, void* stream) {
  return xy_gemm_run_ws(a, lda, w, ldw, c, ldc, M, N, K, tile_n, nullptr, 0, stream);
}

extern "C" int xy_gemm_run_ws(const void* a, int64_t lda, const void* w, int64_t ldw, void* c, int64_t ldc, int32_t M,
                              int32_t N, int32_t K, int32_t tile_n, void* workspace, int64_t workspace_bytes,
                              void* stream) {
  if (workspace != nullptr && ((reinterpret_cast<uintptr_t>(workspace) & 15) || workspace_bytes < 0))
    return XY_ERR_INVALID_ARG;
  if (M < 0 || N < 8 || K < 8 || (N % 8) || (K % 8) || (lda % 8) || (ldw % 8) || (ldc % 8) || lda < K || ldw < K ||
      ldc < N)
    return XY_ERR_INVALID_ARG;
  bool pair = (tile_n & XY_GEMM_PAIR) != 0;
  if (pair) {
    tile_n &= ~XY_GEMM_PAIR;
    if (tile_n != 128 && tile_n != 256) return XY_ERR_UNSUPPORTED;
  }
  if (tile_n != 0 && tile_n != 32 && tile_n != 64 && tile_n != 128 && tile_n != 256) return XY_ERR_UNSUPPORTED;
  if (M == 0) return XY_OK;
  if (!a || !w || !c || (reinterpret_cast<uintptr_t>(a) & 15) || (reinterpret_cast<uintptr_t>(w) & 15) ||
      (reinterpret_cast<uintptr_t>(c) & 15))
    return XY_ERR_INVALID_ARG;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return XY_ERR_CUDA;
  static int sm_count[64] = {0};
  int sms = (dev >= 0 && dev < 64) ? sm_count[dev] : 0;
  if (sms == 0) {
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
      return XY_ERR_CUDA;
    if (dev >= 0 && dev < 64) sm_count[dev] = sms;
  }
  if (tile_n == 0 && !pair && sms >= 2 && M > 128) {
    // 256 x 256 tiles on CTA pairs when the padding of M to 256 rows stays under 15 % and the tiles
    // give at least half of the pairs work: measured best or level with the best from 1024 tokens
    // on (at 4096 tokens QKV 155 -> 143 us, OProj 105 -> 96, GateUp 667 -> 609, Down 369 -> 339), and
    // at 256 tokens for GateUp only (112 tiles: 67 -> 61 us; the shapes with 16 - 24 tiles stay with
    // 128-column tiles or the cluster split of K).
    const int mp = (M + 255) / 256, np = (N + 255) / 256;
    if ((mp * 256 - M) * 100 <= 15 * mp * 256 && mp * np * 4 >= sms) {
      pair = true;
      tile_n = 256;
    }
  }
  if (pair) {
    if (sms < 2) return XY_ERR_UNSUPPORTED;
    const cudaError_t e =
        tile_n == 256 ? xy::launch_gemm_pair<256>(a, lda, w, ldw, c, ldc, M, N, K, sms, static_cast<cudaStream_t>(stream))
                      : xy::launch_gemm_pair<128>(a, lda, w, ldw, c, ldc, M, N, K, sms, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? XY_OK : XY_ERR_CUDA;
  }
  if (tile_n == 0 && M <= 512) {
    // Few tiles and one long serial chain over K per tile: split K over a cluster when that puts
    // several times as many SMs to work (Down / OProj projections of a decode batch or a short
    // chunk).  Measured: four or more slices pay off from 16 chunks per slice on; two or three
    // only when the chain is long (32 chunks per slice), else the reduction costs what the
    // shorter chain saves.
    const int tiles = ((M + 127) / 128) * ((N + 127) / 128), k_chunks = (K + 63) / 64;
    int splits = sms / tiles;
    if (splits > 8) splits = 8;
    while (splits >= 2 && k_chunks / splits < (splits >= 4 ? 16 : 32)) --splits;
    if (splits >= 2) {
      const cudaError_t e =
          xy::launch_gemm_splitk(a, lda, w, ldw, c, ldc, M, N, K, splits, static_cast<cudaStream_t>(stream));
      return e == cudaSuccess ? XY_OK : XY_ERR_CUDA;
    }
  }
  if (tile_n == 0) {
    // 128 x 256 tiles read the least of A and W per flop; they are used when they give at least
    // half of the SMs a tile (measured: OProj at 1024 tokens, 128 such tiles, 28 us against 44 us
    // with 128 x 128; GateUp at 16 tokens 44 against 49 us).  Below that 128 x 128 (narrower tiles
    // are not faster for small M, where the time is launch and pipeline-fill latency).
    const int64_t tiles256 = static_cast<int64_t>((M + 127) / 128) * ((N + 255) / 256);
    tile_n = tiles256 * 2 >= sms ? 256 : 128;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e;
  switch (tile_n) {
    case 256: e = xy::launch_gemm<256>(a, lda, w, ldw, c, ldc, M, N, K, sms, workspace, workspace_bytes, s); break;
    case 128: e = xy::launch_gemm<128>(a, lda, w, ldw, c, ldc, M, N, K, sms, workspace, workspace_bytes, s); break;
    case 64: e = xy::launch_gemm<64>(a, lda, w, ldw, c, ldc, M, N, K, sms, workspace, workspace_bytes, s); break;
    default: e = xy::launch_gemm<32>(a, lda, w, ldw, c, ldc, M, N, K, sms, workspace, workspace_bytes, s); break;
  }
  return e == cudaSuccess ? XY_OK : XY_ERR_CUDA;
}

extern "C" int xy_gemm_device_status(int32_t* status) {
  if (status == nullptr) return XY_ERR_INVALID_ARG;
  if (cudaDeviceSynchronize() != cudaSuccess) return XY_ERR_CUDA;
  int32_t v = 0;
  if (cudaMemcpyFromSymbol(&v, xy::g_gemm_status, sizeof v) != cudaSuccess) return XY_ERR_CUDA;
  const int32_t zero = 0;
  if (cudaMemcpyToSymbol(xy::g_gemm_status, &zero, sizeof zero) != cudaSuccess) return XY_ERR_CUDA;
  *status = v;
  return XY_OK;
}
