// Hybrid-batch attention meta-kernel (Meta-Attention, Sections 4.1-4.2), sm_100a.
//
// One persistent CTA per worker (SM) of 384 threads runs meta-tasks until none are left: its own
// Task-Table list (Section 3.3.1) or, for balanced plans, the head of one global queue.  Roles:
//   warps 0..7  consumers: softmax (and, on the warp-level paths, the MMAs), O / LSE output
//   warp  8     producer (one lane): takes the next task, looks page ids up in the block table and
//               stages 128-key K and V tiles (one TMA box per page and 64-element half) into a
//               ring of four shared-memory stages; it runs ahead across task boundaries
//   warps 9-10  tcgen05 issuers (one lane each), one per 128-row sub-tile of a dense task
// Shared-memory tiles use the 128-byte TMA swizzle: element (row, d) of a tile lives at
//   (d / 64) * 16 KiB + row * 128 B + (((d % 64) / 8) ^ (row % 8)) * 16 B + (d % 8) * 2 B,
// which both ldmatrix and the tcgen05 shared-memory descriptors read without bank conflicts.
//
// Two task kinds share the ring:
//   dense     (rows > 16: prefill, verify): two 128-row sub-tiles of packed Q rows; S = Q K^T
//             and O += P V run on tcgen05 with S, P and O in tensor memory, and each consumer
//             warpgroup does the online softmax of one sub-tile (thread = row).  In the variant
//             without tensor memory (kUmma = false) a dense task is one 128-row tile on
//             mma.sync, each consumer warp owning 16 rows.
//   streaming (rows <= 16: decode, tiny verify): each consumer warp owns 16 keys of every tile
//             against all rows on mma.sync; the warps' partial (m, l, O) are merged in shared
//             memory at the end of the task.  HBM-bound.
// Online softmax runs in the log2 domain in fp32; P is rounded to bf16 before P V; masked scores
// are selected to -inf, never added.  Every wait is bounded and reports a timeout in the status
// word instead of spinning forever.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <type_traits>

#include "ptx.cuh"
#include "xy_kernels.h"

namespace xy {

namespace {

using namespace ptx;

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 128;  // + one warpgroup: producer, MMA issuer, 2 idle
constexpr int kRegsConsumer = 216;  // setmaxnreg budgets: 256 x 216 + 128 x 72 = 168 x 384, the launch allocation
constexpr int kRegsOther = 72;
constexpr int kStages = 4;
constexpr int kTileBytes = 32768;  // 2 halves x 128 rows x 128 B
constexpr int kHalfBytes = 16384;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleThresholdWarp = 8.0f;  // log2 units, warp-level MMA paths
constexpr float kLn2 = 0.6931471805599453f;

struct __align__(8) SmemBarriers {
  uint64_t full[kStages];
  uint64_t empty[kStages];      // released by the eight consumer warps (warp-level MMA paths)
  uint64_t empty_umma[kStages];  // released by two tcgen05.commit arrivals (tensor-memory path)
};

constexpr int kSmemQ = 2 * kTileBytes;
constexpr int kSmemRing = kStages * kTileBytes;
constexpr int kSmemMl = kConsumerWarps * 16 * 2 * 4;
constexpr int kSmemFp8 = 1024;  // fp8 KV path: per-row Q factors [128] and a ring of per-tile page scales [8][16]
constexpr int kScaleSlots = 8;
constexpr int kSmemTotal = 1024 /*align slack*/ + kSmemQ + kSmemRing + kSmemMl + sizeof(SmemBarriers) + 128 + 256 + kSmemFp8;

__device__ __forceinline__ uint32_t swz(uint32_t row, uint32_t chunk16 /*0..15*/) {
  return (chunk16 >> 3) * kHalfBytes + row * 128u + (((chunk16 & 7u) ^ (row & 7u)) << 4);
}

struct Pipe {
  int stage;
  uint32_t phase;
  __device__ __forceinline__ void advance() {
    if (++stage == kStages) {
      stage = 0;
      phase ^= 1u;
    }
  }
};

struct MetaParams {
  RunArgs a;
};

// Visibility of key column `col` for new token i (Sections 4.1.2, 4.2.2, 5.2).
__device__ __forceinline__ bool visible(const RunArgs& a, const ReqInfo& rq, int i, int col) {
  if (col > rq.kv_len + i) return false;  // causal frontier; also excludes everything >= L
  if (col < rq.kv_len || rq.mask_kind == XY_MASK_CAUSAL) return true;
  const int jp = col - rq.kv_len;
  const uint64_t w = __ldg(a.tree_mask + rq.tree_off + static_cast<int64_t>(i) * rq.tree_words + (jp >> 6));
  return (w >> (jp & 63)) & 1ull;
}

// One consumer warp: 16 packed rows (x0 .. x0+15) against NT*8 keys (key offset koff inside
// every 128-key tile).  Keeps m (log2 domain), l (thread-partial) and O in registers.
// KEEPQ: Q fragments stay in registers for the whole task (streaming); otherwise they are
// re-read from shared memory at every k-step to leave registers for the 128-key score tile.
// F16: operands are f16 (the fp8 KV-cache path: K / V widened exactly from e4m3, Q converted with a
// power-of-two factor per row) and the scores carry per-row and per-page factors (FpScale).
struct FpScale {
  float q_lo, q_hi;        // 2^e of the two rows this thread holds: undoes the row's Q pre-scaling
  const float* tile;       // shared memory: [0..7] K scale, [8..15] V scale of the tile's pages
  int page_shift;
};

template <bool F16>
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  if constexpr (F16) mma_f16_16816(c, a, b0, b1); else mma_bf16_16816(c, a, b0, b1);
}

template <int NT, bool KEEPQ, bool F16 = false>
struct WarpTile {
  float o[16][4];
  float m_lo, m_hi, l_lo, l_hi;
  uint32_t qf[KEEPQ ? 8 : 1][4];
  uint32_t q_addr;  // this lane's ldmatrix row address for k-step 0 (!KEEPQ)

  __device__ __forceinline__ void init() {
#pragma unroll
    for (int n = 0; n < 16; ++n)
#pragma unroll
      for (int e = 0; e < 4; ++e) o[n][e] = 0.f;
    m_lo = m_hi = -INFINITY;
    l_lo = l_hi = 0.f;
  }

  __device__ __forceinline__ void load_q(uint32_t q_smem, int x0, int lane) {
    const int mi = lane >> 3;
    const uint32_t row = x0 + (lane & 7) + (mi & 1) * 8;
    if (KEEPQ) {
#pragma unroll
      for (int ks = 0; ks < 8; ++ks)
        ldmatrix_x4(q_smem + swz(row, ks * 2 + (mi >> 1)), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
    } else {
      q_addr = q_smem + row * 128u;
      q_row7 = row & 7u;
      q_hi = mi >> 1;
    }
  }
  uint32_t q_row7, q_hi;

  // S = Q K^T for this warp's keys; returns scores (raw dot products) in s.
  __device__ __forceinline__ void qk(uint32_t k_smem, int koff, int lane, float (&s)[NT][4]) {
    if constexpr (NT == 2) {
      // Streaming tile: all eight K fragments are fetched first (one shared-memory latency
      // instead of eight), and even / odd k-steps accumulate separately so that the MMAs form
      // four chains of four instead of two chains of eight.
      const int mi = lane >> 3;
      const uint32_t key = koff + (lane & 7) + (mi >> 1) * 8;
      uint32_t kb[8][4];
#pragma unroll
      for (int ks = 0; ks < 8; ++ks)
        ldmatrix_x4(k_smem + swz(key, ks * 2 + (mi & 1)), kb[ks][0], kb[ks][1], kb[ks][2], kb[ks][3]);
      uint32_t qq[8][4];
      if constexpr (!KEEPQ) {
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint32_t ch = ks * 2 + q_hi;
          ldmatrix_x4(q_addr + (ch >> 3) * kHalfBytes + (((ch & 7u) ^ q_row7) << 4), qq[ks][0], qq[ks][1],
                      qq[ks][2], qq[ks][3]);
        }
      }
      float t[2][4];
#pragma unroll
      for (int n = 0; n < 2; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) s[n][e] = t[n][e] = 0.f;
#pragma unroll
      for (int ks = 0; ks < 8; ks += 2) {
        const uint32_t(&qa)[4] = KEEPQ ? qf[KEEPQ ? ks : 0] : qq[ks];
        const uint32_t(&qb)[4] = KEEPQ ? qf[KEEPQ ? ks + 1 : 0] : qq[ks + 1];
        mma16816<F16>(s[0], qa, kb[ks][0], kb[ks][1]);
        mma16816<F16>(s[1], qa, kb[ks][2], kb[ks][3]);
        mma16816<F16>(t[0], qb, kb[ks + 1][0], kb[ks + 1][1]);
        mma16816<F16>(t[1], qb, kb[ks + 1][2], kb[ks + 1][3]);
      }
#pragma unroll
      for (int n = 0; n < 2; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) s[n][e] += t[n][e];
      return;
    }
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
      for (int e = 0; e < 4; ++e) s[n][e] = 0.f;
    const int mi = lane >> 3;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      if (!KEEPQ) {
        const uint32_t ch = ks * 2 + q_hi;
        ldmatrix_x4(q_addr + (ch >> 3) * kHalfBytes + (((ch & 7u) ^ q_row7) << 4), qf[0][0], qf[0][1],
                    qf[0][2], qf[0][3]);
      }
      const uint32_t(&qa)[4] = qf[KEEPQ ? ks : 0];
#pragma unroll
      for (int np = 0; np < NT / 2; ++np) {
        const uint32_t key = koff + np * 16 + (lane & 7) + (mi >> 1) * 8;
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4(k_smem + swz(key, ks * 2 + (mi & 1)), b0, b1, b2, b3);
        mma16816<F16>(s[2 * np], qa, b0, b1);
        mma16816<F16>(s[2 * np + 1], qa, b2, b3);
      }
    }
  }

  // Mask + online softmax (Update rescale) on s; leaves P (bf16 A fragments) in p.
  // koff: key offset of s[0] inside the 128-key tile (selects the page whose scales apply)
  __device__ __forceinline__ void softmax(const RunArgs& a, const ReqInfo& rq, float (&s)[NT][4],
                                          uint32_t (&p)[NT / 2][4], int col0, int i_lo, int i_hi,
                                          bool need_mask, float scale_log2, int lane, const FpScale* fs = nullptr,
                                          int koff = 0) {
    float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      float f_lo = scale_log2, f_hi = scale_log2;
      if constexpr (F16) {
        const float ks = fs->tile[(koff + n * 8) >> fs->page_shift];
        f_lo = scale_log2 * fs->q_lo * ks;
        f_hi = scale_log2 * fs->q_hi * ks;
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float v = s[n][e] * ((e < 2) ? f_lo : f_hi);
        if (need_mask) {
          const int col = col0 + n * 8 + 2 * (lane & 3) + (e & 1);
          if (!visible(a, rq, (e < 2) ? i_lo : i_hi, col)) v = -INFINITY;
        }
        s[n][e] = v;
        if (e < 2) mx_lo = fmaxf(mx_lo, v); else mx_hi = fmaxf(mx_hi, v);
      }
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
    const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
    // Lazy Update: the reference moves (and O, l are rescaled) only when some row of the warp
    // would otherwise exceed it by more than 2^kRescaleThresholdWarp, or has no reference yet.
    const bool grow = (mn_lo - m_lo > kRescaleThresholdWarp) || (mn_hi - m_hi > kRescaleThresholdWarp) ||
                      (m_lo == -INFINITY && mn_lo != -INFINITY) || (m_hi == -INFINITY && mn_hi != -INFINITY);
    if (__any_sync(0xffffffffu, grow)) {
      const float u_lo = (mn_lo == -INFINITY) ? 0.f : mn_lo, u_hi = (mn_hi == -INFINITY) ? 0.f : mn_hi;
      const float al_lo = ex2(m_lo - u_lo), al_hi = ex2(m_hi - u_hi);
      m_lo = mn_lo;
      m_hi = mn_hi;
      l_lo *= al_lo;
      l_hi *= al_hi;
#pragma unroll
      for (int n = 0; n < 16; ++n) {
        o[n][0] *= al_lo;
        o[n][1] *= al_lo;
        o[n][2] *= al_hi;
        o[n][3] *= al_hi;
      }
    }
    const float use_lo = (m_lo == -INFINITY) ? 0.f : m_lo;
    const float use_hi = (m_hi == -INFINITY) ? 0.f : m_hi;
    float sum_lo = 0.f, sum_hi = 0.f;
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      const float p0 = ex2(s[n][0] - use_lo), p1 = ex2(s[n][1] - use_lo);
      const float p2 = ex2(s[n][2] - use_hi), p3 = ex2(s[n][3] - use_hi);
      sum_lo += p0 + p1;
      sum_hi += p2 + p3;
      // A fragment of k-step n/2: a0,a1 from the even n-tile, a2,a3 from the odd one
      if constexpr (F16) {
        // the V scale of the key's page rides on P (l keeps the unscaled sum)
        const float vs = fs->tile[8 + ((koff + n * 8) >> fs->page_shift)];
        p[n >> 1][(n & 1) * 2 + 0] = pack_f16(p0 * vs, p1 * vs);
        p[n >> 1][(n & 1) * 2 + 1] = pack_f16(p2 * vs, p3 * vs);
      } else {
        p[n >> 1][(n & 1) * 2 + 0] = pack_bf16(p0, p1);
        p[n >> 1][(n & 1) * 2 + 1] = pack_bf16(p2, p3);
      }
    }
    l_lo += sum_lo;
    l_hi += sum_hi;
  }

  // O += P V for this warp's keys.
  __device__ __forceinline__ void pv(uint32_t v_smem, int koff, int lane, const uint32_t (&p)[NT / 2][4]) {
    const int mi = lane >> 3;
    if constexpr (NT == 2) {  // streaming tile: fetch the eight V fragments, then 16 MMAs
      const uint32_t key = koff + (lane & 7) + (mi & 1) * 8;
      uint32_t vb[8][4];
#pragma unroll
      for (int dp = 0; dp < 8; ++dp)
        ldmatrix_x4_trans(v_smem + swz(key, dp * 2 + (mi >> 1)), vb[dp][0], vb[dp][1], vb[dp][2], vb[dp][3]);
#pragma unroll
      for (int dp = 0; dp < 8; ++dp) {
        mma16816<F16>(o[2 * dp], p[0], vb[dp][0], vb[dp][1]);
        mma16816<F16>(o[2 * dp + 1], p[0], vb[dp][2], vb[dp][3]);
      }
      return;
    }
#pragma unroll
    for (int kk = 0; kk < NT / 2; ++kk) {
      const uint32_t key = koff + kk * 16 + (lane & 7) + (mi & 1) * 8;
#pragma unroll
      for (int dp = 0; dp < 8; ++dp) {
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4_trans(v_smem + swz(key, dp * 2 + (mi >> 1)), b0, b1, b2, b3);
        mma16816<F16>(o[2 * dp], p[kk], b0, b1);
        mma16816<F16>(o[2 * dp + 1], p[kk], b2, b3);
      }
    }
  }

  __device__ __forceinline__ void reduce_l() {
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
  }
};

// ------------------------------------------------------------------------------------------
// fp8 KV-cache path (a variant beside the paper's bf16 cache; Section 4.1.1's paged layout with
// e4m3 bytes and one fp32 scale per page and kv head).  A 128-key tile arrives as 16 KiB of
// bytes in the upper half of its 32 KiB stage (row = key, 128 B, 16-byte chunks XOR-swizzled by
// row like every other tile); the warp that is going to read 16 of its rows first widens them in
// place to the f16 tile layout (exact: every e4m3 value is an f16 value).  Two lanes share a row;
// the upper-half destination of a row is the very line its bytes came from, hence the warp-wide
// barrier between the loads and the stores.
__device__ __forceinline__ void widen_rows16(uint32_t stage, int row0, int lane) {
  const uint32_t row = row0 + (lane >> 1), half = lane & 1u, r7 = row & 7u;
  const uint32_t src = stage + kHalfBytes + row * 128u;
  uint4 in[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) in[q] = lds128(src + (((half * 4u + q) ^ r7) << 4));
  // the partner lane's source chunks lie in the line this lane is about to overwrite (and vice versa)
  asm volatile("" ::"r"(in[0].x), "r"(in[1].x), "r"(in[2].x), "r"(in[3].x), "r"(in[0].w), "r"(in[1].w), "r"(in[2].w),
               "r"(in[3].w));
  __syncwarp();
  const uint32_t dst = stage + half * kHalfBytes + row * 128u;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const uint32_t w[4] = {in[q].x, in[q].y, in[q].z, in[q].w};
    uint32_t h[8];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      h[2 * k] = e4m3x2_to_f16x2(static_cast<uint16_t>(w[k] & 0xFFFFu));
      h[2 * k + 1] = e4m3x2_to_f16x2(static_cast<uint16_t>(w[k] >> 16));
    }
    sts128(dst + ((static_cast<uint32_t>(2 * q) ^ r7) << 4), make_uint4(h[0], h[1], h[2], h[3]));
    sts128(dst + ((static_cast<uint32_t>(2 * q + 1) ^ r7) << 4), make_uint4(h[4], h[5], h[6], h[7]));
  }
  __syncwarp();
}

// Q rows of the tile in shared memory, bf16 -> f16 in place, each row multiplied by a power of two
// that brings its largest element below 4 (exact in f16 for every element within 2^-14 of the
// row's largest; bf16's exponent range does not fit f16 otherwise).  qmult[row] receives the
// inverse factor, which the softmax folds into the score scale.  kLanesPerRow lanes share a row.
template <int kLanesPerRow>
__device__ __forceinline__ void q_rows_to_f16(uint32_t q_smem, int row0, float* qmult, int lane) {
  constexpr int kChunks = 16 / kLanesPerRow;  // 16-byte chunks (8 elements) per lane
  const uint32_t row = row0 + lane / kLanesPerRow, c0 = (lane % kLanesPerRow) * kChunks;
  uint4 v[kChunks];
  uint32_t emax = 0;
#pragma unroll
  for (int c = 0; c < kChunks; ++c) {
    v[c] = lds128(q_smem + swz(row, c0 + c));
    const uint32_t w[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
#pragma unroll
    for (int k = 0; k < 4; ++k) emax = max(emax, max(w[k] & 0x7F80u, (w[k] >> 16) & 0x7F80u));
  }
#pragma unroll
  for (int o = 1; o < kLanesPerRow; o <<= 1) emax = max(emax, __shfl_xor_sync(0xffffffffu, emax, o));
  uint32_t e = emax >> 7;                       // biased exponent of the row's largest element
  e = e == 0 ? 127u : min(max(e, 2u), 253u);    // an all-zero row keeps factor 1
  const float down = __uint_as_float((254u - e) << 23), up = __uint_as_float(e << 23);
#pragma unroll
  for (int c = 0; c < kChunks; ++c) {
    uint32_t w[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
#pragma unroll
    for (int k = 0; k < 4; ++k)
      w[k] = pack_f16(__uint_as_float(w[k] << 16) * down, __uint_as_float(w[k] & 0xFFFF0000u) * down);
    sts128(q_smem + swz(row, c0 + c), make_uint4(w[0], w[1], w[2], w[3]));
  }
  if (lane % kLanesPerRow == 0) qmult[row] = up;
}

struct TaskView {
  xy_attn_task t;
  ReqInfo rq;
  int G, rows;
};

// Destination of packed row x: final O / LSE or the fp32 partial.
__device__ __forceinline__ void write_row_pair(const RunArgs& a, const TaskView& tv, int x, int col,
                                               float v0, float v1) {
  if (tv.t.part < 0) {
    const int i = tv.t.tok0 + x / tv.G, head = tv.t.kv_head * tv.G + x % tv.G;
    uint32_t* dst = reinterpret_cast<uint32_t*>(
        a.o + static_cast<int64_t>(tv.rq.q_start + i) * a.o_token_stride + head * kHeadDim + col);
    *dst = pack_bf16(v0, v1);
  } else {
    float2* dst = reinterpret_cast<float2*>(a.o_part + static_cast<int64_t>(tv.t.part + x) * kHeadDim + col);
    *dst = make_float2(v0, v1);
  }
}
__device__ __forceinline__ void write_lse(const RunArgs& a, const TaskView& tv, int x, float lse) {
  if (tv.t.part < 0) {
    const int i = tv.t.tok0 + x / tv.G, head = tv.t.kv_head * tv.G + x % tv.G;
    a.lse[static_cast<int64_t>(tv.rq.q_start + i) * a.num_q_heads + head] = lse;
  } else {
    a.lse_part[tv.t.part + x] = lse;
  }
}

// Debug trace of worker 0: one record per call, (tag << 48) | SM cycle counter.  Compiled in
// only with -DXY_ENABLE_TRACE (the stamps cost issue slots on the critical path).
struct Tracer {
#ifdef XY_ENABLE_TRACE
  unsigned long long* p;
  int n;
  __device__ __forceinline__ void init(const RunArgs& a, int role, bool on) {
    p = (a.trace != nullptr && blockIdx.x == 0 && on) ? a.trace + role * kTraceLen : nullptr;
    n = 0;
  }
  __device__ __forceinline__ void operator()(unsigned tag) {
    if (p != nullptr && n < kTraceLen) p[n++] = (static_cast<unsigned long long>(tag) << 48) | (clock64() & 0xFFFFFFFFFFFFull);
  }
#else
  __device__ __forceinline__ void init(const RunArgs&, int, bool) {}
  __device__ __forceinline__ void operator()(unsigned) {}
#endif
};

// Word 0 of the status block is this run's (cleared at every launch, polled by every wait); the
// sticky word is what xy_attn_device_status reads and clears.
__device__ __forceinline__ void report_timeout(const RunArgs& a) {
  atomicExch(a.status, XY_ERR_DEVICE_TIMEOUT);
  atomicExch(a.status + kStatusSticky, XY_ERR_DEVICE_TIMEOUT);
}

// Merge of a split streaming unit inside the attention kernel (the cross-task Update stage of
// Section 4.2.1, run by the task of the unit that finished last).  rows <= 16; one warp per row;
// LSE_c in lanes, the partial rows read eight at a time straight from L2.
__device__ __forceinline__ float ldcg_f(const float* p) { return __ldcg(p); }
__device__ __forceinline__ void merge_unit_in_kernel(const RunArgs& a, const xy_attn_merge_unit& u, int G, int warp,
                                                     int lane) {
  const int rows = u.ntok * G, ns = u.nsplit;
  const ReqInfo rq = a.reqs[u.req];
  for (int x = warp; x < rows; x += kConsumerWarps) {
    const int64_t row0 = static_cast<int64_t>(u.part0) + x;  // partial row of split c: row0 + c * rows
    float mx = -INFINITY;
    for (int c = lane; c < ns; c += 32) mx = fmaxf(mx, ldcg_f(a.lse_part + row0 + static_cast<int64_t>(c) * rows));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float z = 0.f;
    for (int c = lane; c < ns; c += 32) {
      const float lc = ldcg_f(a.lse_part + row0 + static_cast<int64_t>(c) * rows);
      if (lc != -INFINITY) z += __expf(lc - mx);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    const float lse = mx + logf(z);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int c0 = 0; c0 < ns; c0 += 8) {
      float w[8];
      float4 v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int c = c0 + e;
        const float lc = c < ns ? ldcg_f(a.lse_part + row0 + static_cast<int64_t>(c) * rows) : -INFINITY;
        w[e] = lc != -INFINITY ? __expf(lc - lse) : 0.f;
        // an empty split (weight 0) is not read
        v[e] = w[e] != 0.f ? __ldcg(reinterpret_cast<const float4*>(a.o_part + (row0 + static_cast<int64_t>(c) * rows) * kHeadDim) + lane)
                           : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        acc.x += w[e] * v[e].x;
        acc.y += w[e] * v[e].y;
        acc.z += w[e] * v[e].z;
        acc.w += w[e] * v[e].w;
      }
    }
    const int i = u.tok0 + x / G, head = u.kv_head * G + x % G;
    uint2 packed;
    packed.x = pack_bf16(acc.x, acc.y);
    packed.y = pack_bf16(acc.z, acc.w);
    *reinterpret_cast<uint2*>(a.o + static_cast<int64_t>(rq.q_start + i) * a.o_token_stride + head * kHeadDim + lane * 4) = packed;
    if (lane == 0) a.lse[static_cast<int64_t>(rq.q_start + i) * a.num_q_heads + head] = lse;
  }
}

// ------------------------------------------------------------------------------------------
// One streaming task (at most 16 packed rows: decode steps, short verify windows and the thin
// tails of prefill chunks), run by the eight consumer warps.  Every warp owns 16 keys of each
// 128-key tile, keeps its own online-softmax state over those keys, and the eight partial
// results are merged through shared memory when the task ends (the in-CTA Update stage of
// Section 4.2.1).  pipe_state: ring stage | phase << 8 | dead << 16, returned updated.
// kFp8: the stages hold e4m3 bytes; every warp widens its 16 keys before use, the Q rows in shared
// memory are f16 (converted by the caller), qmult / scale_ring carry the row and page factors and
// tile_seq counts the key tiles this worker has consumed (it selects the scale slot).
template <bool kFp8>
__device__ __forceinline__ uint32_t stream_task(const RunArgs& a, const TaskView& tv, uint32_t q_smem, uint32_t ring,
                                             SmemBarriers* bars, float* xch, float* ml, uint32_t pipe_state,
                                             float scale_log2, const float* qmult, const float* scale_ring,
                                             uint32_t& tile_seq, int unit) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  Pipe pipe{static_cast<int>(pipe_state & 0xFFu), (pipe_state >> 8) & 1u};
  bool dead = (pipe_state >> 16) & 1u;
  const int h = tv.rq.kv_len;
  const bool tree = tv.rq.mask_kind == XY_MASK_TREE;
  const int koff = warp * 16;
  WarpTile<2, false, kFp8> w;
  w.init();
  w.load_q(q_smem, 0, lane);
  FpScale fs{1.f, 1.f, scale_ring, a.page_shift};
  if constexpr (kFp8) {
    fs.q_lo = qmult[lane >> 2];
    fs.q_hi = qmult[(lane >> 2) + 8];
  }
  const int r_lo = min(lane >> 2, tv.rows - 1), r_hi = min((lane >> 2) + 8, tv.rows - 1);
  const int i_lo = tv.t.tok0 + r_lo / tv.G, i_hi = tv.t.tok0 + r_hi / tv.G;
  const int i_max = tv.t.tok0 + tv.t.ntok - 1;
  // Tiles that every row of the task sees in full need neither the mask nor the mask-aware
  // skip test; the loop over them is compiled without either.  The last tiles (the causal
  // frontier or the speculative corner) take the general step.
#ifdef XY_ENABLE_TRACE
  long long ph[6] = {0, 0, 0, 0, 0, 0};
#define XY_PH(i) { const long long c_now = clock64(); ph[i] += c_now - c_prev; c_prev = c_now; }
#else
#define XY_PH(i)
#endif
  auto step = [&](int kt, auto tail_tag) {
    constexpr bool kTail = decltype(tail_tag)::value;
    const int col0 = kt * kKeyTile + koff;
    const bool work = kTail ? (col0 <= h + i_max) : true;
    float s[2][4];
    uint32_t p[1][4];
#ifdef XY_ENABLE_TRACE
    long long c_prev = clock64();
    ph[5] += 1;
#endif
    if (!dead && !mbar_wait_block(smem_u32(&bars->full[pipe.stage]), pipe.phase, a.status)) {
      report_timeout(a);
      dead = true;
    }
    XY_PH(0)
    if constexpr (kFp8) {
      fs.tile = scale_ring + (tile_seq % kScaleSlots) * 16;
      ++tile_seq;
      if (work) widen_rows16(ring + pipe.stage * kTileBytes, koff, lane);
    }
    if (work) w.qk(ring + pipe.stage * kTileBytes, koff, lane, s);
    if constexpr (kFp8) fence_proxy_async_smem();  // the widened rows are overwritten by the next bulk copy
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&bars->empty[pipe.stage]));
    pipe.advance();
    XY_PH(1)
    if (work) {
      const bool need_mask = kTail ? (tree ? (col0 + 16 > h) : (col0 + 16 > h + tv.t.tok0 + 1)) : false;
      w.softmax(a, tv.rq, s, p, col0, i_lo, i_hi, need_mask, scale_log2, lane, &fs, koff);
    }
    XY_PH(2)
    if (!dead && !mbar_wait_block(smem_u32(&bars->full[pipe.stage]), pipe.phase, a.status)) {
      report_timeout(a);
      dead = true;
    }
    XY_PH(3)
    if constexpr (kFp8) {
      if (work) widen_rows16(ring + pipe.stage * kTileBytes, koff, lane);
    }
    if (work) w.pv(ring + pipe.stage * kTileBytes, koff, lane, p);
    if constexpr (kFp8) fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&bars->empty[pipe.stage]));
    pipe.advance();
    XY_PH(4)
  };
  const int full_cols = tree ? h : h + tv.t.tok0 + 1;  // columns below this are visible to every row
  const int kt_mid = max(tv.t.kt_lo, min(tv.t.kt_hi, full_cols / kKeyTile));
  int kt = tv.t.kt_lo;
  for (; kt < kt_mid; ++kt) step(kt, std::false_type{});
  for (; kt < tv.t.kt_hi; ++kt) step(kt, std::true_type{});
#ifdef XY_ENABLE_TRACE
  if (a.trace != nullptr && blockIdx.x == 0 && threadIdx.x == 0)
    for (int i = 0; i < 6; ++i) a.trace[4 * kTraceLen - 8 + i] += ph[i];
#endif
#undef XY_PH
  // ---- merge the eight warps' partials (in-CTA Update stage)
  w.reduce_l();
  named_bar_sync(1, kConsumerThreads);  // every warp holds its Q fragments: Q smem is free
  {
    const int xl = lane >> 2, xh = xl + 8;
    float* mine = xch + warp * (16 * kHeadDim);
    // only the task's rows are merged below: padding rows (most of the 16 in a decode step) are
    // not written
    const bool has_lo = xl < tv.rows, has_hi = xh < tv.rows;
#pragma unroll
    for (int n = 0; n < 16; ++n) {
      const int col = n * 8 + 2 * (lane & 3);
      if (has_lo) *reinterpret_cast<float2*>(mine + xl * kHeadDim + col) = make_float2(w.o[n][0], w.o[n][1]);
      if (has_hi) *reinterpret_cast<float2*>(mine + xh * kHeadDim + col) = make_float2(w.o[n][2], w.o[n][3]);
    }
    if ((lane & 3) == 0) {
      ml[(warp * 16 + xl) * 2 + 0] = w.m_lo;
      ml[(warp * 16 + xl) * 2 + 1] = w.l_lo;
      ml[(warp * 16 + xh) * 2 + 0] = w.m_hi;
      ml[(warp * 16 + xh) * 2 + 1] = w.l_hi;
    }
  }
  named_bar_sync(1, kConsumerThreads);
  {
    const int x = threadIdx.x >> 4, seg = threadIdx.x & 15;  // row, 8-column segment
    if (x < tv.rows) {
      float M = -INFINITY;
#pragma unroll
      for (int ww = 0; ww < kConsumerWarps; ++ww) M = fmaxf(M, ml[(ww * 16 + x) * 2]);
      float L = 0.f, acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int ww = 0; ww < kConsumerWarps; ++ww) {
        const float mw = ml[(ww * 16 + x) * 2], lw = ml[(ww * 16 + x) * 2 + 1];
        if (mw == -INFINITY) continue;
        const float f = ex2(mw - M);
        L += f * lw;
        const float4* src = reinterpret_cast<const float4*>(xch + ww * (16 * kHeadDim) + x * kHeadDim + seg * 8);
        const float4 v0 = src[0], v1 = src[1];
        acc[0] += f * v0.x; acc[1] += f * v0.y; acc[2] += f * v0.z; acc[3] += f * v0.w;
        acc[4] += f * v1.x; acc[5] += f * v1.y; acc[6] += f * v1.z; acc[7] += f * v1.w;
      }
      const float inv = L > 0.f ? 1.f / L : 0.f;
#pragma unroll
      for (int e = 0; e < 8; e += 2)
        write_row_pair(a, tv, x, seg * 8 + e, acc[e] * inv, acc[e + 1] * inv);
      if (seg == 0) write_lse(a, tv, x, L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY);
    }
  }
  if (unit >= 0) {
    // This task is one KV split of a unit that is merged here: publish the partial, count the
    // finished splits, and let the task that completes the unit merge it.  (Writers: stores, fence,
    // barrier, one atomic; the last one: atomic, fence, loads that bypass L1.)
    __shared__ int s_last;
    __threadfence();
    named_bar_sync(1, kConsumerThreads);
    if (threadIdx.x == 0) {
      const int ns = a.units[unit].nsplit;
      s_last = atomicAdd(a.unit_count + unit, 1) == ns - 1 ? 1 : 0;
    }
    named_bar_sync(1, kConsumerThreads);
    if (s_last) {
      __threadfence();
      merge_unit_in_kernel(a, a.units[unit], tv.G, warp, lane);
    }
  }
  return static_cast<uint32_t>(pipe.stage) | (pipe.phase << 8) | (dead ? 1u << 16 : 0u);
}

// ------------------------------------------------------------------------------------------
// tcgen05 dense path.  TMEM columns: S_A [0,128) S_B [128,256) O_A [256,384) O_B [384,512);
// P (bf16, two keys per 32-bit column) overwrites the first 64 columns of its S block.
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemS = 0, kTmemO = 256;
constexpr float kRescaleThreshold = 8.0f;  // log2 units: rescale O only when the row max grows by > 2^8

// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 128.
constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescQK = kIdescBase;              // A, B K-major
constexpr uint32_t kIdescPV = kIdescBase | (1u << 16);  // B (V) MN-major

// Task indices travel from the producer (which takes them from the global queue) to the other
// roles of the CTA through a small ring in shared memory.
constexpr int kTaskRing = 8;
struct __align__(8) TaskRing {
  uint64_t full[kTaskRing];   // producer -> readers: the slot holds a task index (or -1: no more)
  uint64_t empty[kTaskRing];  // readers -> producer: every reader has taken the slot's index
  int32_t ti[kTaskRing];
};

struct DenseShape {
  int n[2];  // KV tiles sub-tile A / B visits in this task
  int n_all;
};
__device__ __forceinline__ DenseShape dense_shape(const xy_attn_task& t, const ReqInfo& rq, int G) {
  DenseShape d;
  const int rows = t.ntok * G;
#pragma unroll
  for (int X = 0; X < 2; ++X) {
    if (X * 128 >= rows) {
      d.n[X] = 0;
      continue;
    }
    const int last_tok = t.tok0 + (min(rows, (X + 1) * 128) - 1) / G;
    const int frontier = (rq.kv_len + last_tok + 1 + kKeyTile - 1) / kKeyTile;
    d.n[X] = max(0, min(t.kt_hi, frontier) - t.kt_lo);
  }
  d.n_all = t.kt_hi - t.kt_lo;
  return d;
}

struct __align__(8) UmmaBarriers {
  uint64_t q_full[2];  // consumers -> MMA: packed Q sub-tile is in shared memory
  uint64_t s_full[2];  // MMA -> consumers: S = Q K^T of the next KV tile is in TMEM
  uint64_t p_full[2][2];  // consumers -> MMA: [sub-tile][half] 64 keys of P are in TMEM (O rescaled if need be)
  uint64_t o_done[2];  // MMA -> consumers: the task's last P V has completed
  uint64_t drained[2];  // every MMA an issuer has issued has completed (waited for once, before exit)
  uint32_t tmem_base;
  volatile uint32_t turn;  // index of the next MMA group allowed onto the tensor pipe
};

static_assert(kStatusWaitLimit == kStatusWaitLimitWord, "one word, two names");
static_assert(sizeof(UmmaBarriers) <= 128, "the shared-memory layout reserves 128 bytes for UmmaBarriers");

template <bool kUmma, bool kFp8>
__global__ void __launch_bounds__(kThreads, 1)
meta_attention_kernel(const __grid_constant__ MetaParams P, const __grid_constant__ CUtensorMap k_map,
                      const __grid_constant__ CUtensorMap v_map) {
  extern __shared__ uint8_t smem_raw[];
  const RunArgs& a = P.a;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t q_smem = base;
  const uint32_t ring = base + kSmemQ;
  uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
  float* ml = reinterpret_cast<float*>(gen_base + kSmemQ + kSmemRing);
  SmemBarriers* bars = reinterpret_cast<SmemBarriers*>(gen_base + kSmemQ + kSmemRing + kSmemMl);
  UmmaBarriers* ub = reinterpret_cast<UmmaBarriers*>(gen_base + kSmemQ + kSmemRing + kSmemMl + sizeof(SmemBarriers));
  TaskRing* tq = reinterpret_cast<TaskRing*>(gen_base + kSmemQ + kSmemRing + kSmemMl + sizeof(SmemBarriers) + 128);
  float* xch = reinterpret_cast<float*>(gen_base);  // streaming merge area, aliases the Q tiles
  static_assert(!(kUmma && kFp8), "the fp8 KV path runs on the warp-level MMA paths");
  float* qmult = reinterpret_cast<float*>(gen_base + kSmemQ + kSmemRing + kSmemMl + sizeof(SmemBarriers) + 128 + 256);
  float* scale_ring = qmult + 128;  // [kScaleSlots][16]: K scales [0..7], V scales [8..15] of a tile's pages

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    unsigned long long now;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
    a.worker_times[4 * blockIdx.x] = now;
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&bars->full[s]), 1);
      mbar_init(smem_u32(&bars->empty[s]), kConsumerWarps);
      mbar_init(smem_u32(&bars->empty_umma[s]), 2);
    }
    ub->turn = 0;
    for (int i = 0; i < kTaskRing; ++i) {
      mbar_init(smem_u32(&tq->full[i]), 1);
      mbar_init(smem_u32(&tq->empty[i]), kConsumerWarps + (kUmma ? 2 : 0));
    }
    for (int X = 0; X < 2; ++X) {
      mbar_init(smem_u32(&ub->q_full[X]), 4);
      mbar_init(smem_u32(&ub->s_full[X]), 1);
      mbar_init(smem_u32(&ub->p_full[X][0]), 4);
      mbar_init(smem_u32(&ub->p_full[X][1]), 4);
      mbar_init(smem_u32(&ub->o_done[X]), 1);
      mbar_init(smem_u32(&ub->drained[X]), 1);
    }
    fence_mbar_init();
  }
  if (kUmma && warp == kConsumerWarps + 1) {
    tmem_alloc(smem_u32(&ub->tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = kUmma ? ub->tmem_base : 0u;

  const int t_begin = a.worker_off[blockIdx.x], t_end = a.worker_off[blockIdx.x + 1];
  const bool dynamic = a.dynamic != 0;
  // Every role but the producer reads its task sequence here: the worker's own Task-Table list
  // (static dealing) or the indices the producer publishes (dynamic dealing).  Warp-uniform.
  int seq_static = t_begin;
  uint32_t n_read = 0;
  bool feed_dead = false;
  auto next_task = [&](bool whole_warp) -> int {  // whole_warp: called by all 32 lanes (else by one)
    if (!dynamic) return seq_static < t_end ? seq_static++ : -1;
    const uint32_t slot = n_read % kTaskRing;
    if (!feed_dead && !mbar_wait_block(smem_u32(&tq->full[slot]), (n_read / kTaskRing) & 1u, a.status)) {
      report_timeout(a);
      feed_dead = true;
    }
    const int ti = feed_dead ? -1 : tq->ti[slot];
    if (whole_warp) {
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&tq->empty[slot]));
    } else {
      mbar_arrive(smem_u32(&tq->empty[slot]));
    }
    ++n_read;
    return ti;
  };
  const int G = a.num_q_heads / a.num_kv_heads;
  const float scale_log2 = a.sm_scale * kLog2e;

  if (warp >= kConsumerWarps) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
    if (warp == kConsumerWarps && lane == 0) {
      // ================================ producer =======================================
      prefetch_tensormap(&k_map);
      prefetch_tensormap(&v_map);
      Pipe pipe{0, 0};
      bool dead = false;
      // Who read each stage last (bit set: the tcgen05 path) and the parity to wait for on each
      // of the two empty barriers of a stage; a stage that was never filled needs no wait.
      uint32_t used = 0, last_umma = 0, ph_cons = 0, ph_umma = 0;
      uint32_t fill_par = 0;  // per stage: parity of the `full` phase its latest fill completes
      Tracer tr;
      tr.init(a, 3, true);
      const int ppt = kKeyTile >> a.page_shift;  // pages per 128-key tile
      const uint32_t page_bytes = static_cast<uint32_t>(a.page_size) * 128u;
      const uint64_t pol_stream = make_l2_policy_evict_first(), pol_keep = make_l2_policy_evict_last();
      // Fill one stage (the K or the V tile) once its previous reader has released it.
      int n_fill = 0;
      uint32_t k_fills = 0;  // K tiles filled so far (fp8: selects the scale slot)
      auto fill = [&](int op, bool by_umma, int kv_head, int kt, const int32_t* bt, int npages, int page0,
                      float ks0, float vs0) {
        // Failure-path test hook (xy_attn_debug_inject): this worker leaves out one fill, so the
        // stage's `full` barrier never completes and the readers' bounded waits run out.
        if (n_fill++ == a.debug_skip_fill) {
          pipe.advance();
          return;
        }
        const uint32_t bit = 1u << pipe.stage;
        if (used & bit) {
          bool ok;
          if (last_umma & bit) {
            ok = mbar_wait_block(smem_u32(&bars->empty_umma[pipe.stage]), (ph_umma >> pipe.stage) & 1u, a.status);
            ph_umma ^= bit;
          } else {
            ok = mbar_wait_block(smem_u32(&bars->empty[pipe.stage]), (ph_cons >> pipe.stage) & 1u, a.status);
            ph_cons ^= bit;
          }
          if (!ok) {
            report_timeout(a);
            dead = true;
            return;
          }
        }
        if (used & bit) fill_par ^= bit;
        used |= bit;
        last_umma = by_umma ? (last_umma | bit) : (last_umma & ~bit);
        tr(1 + op);
        const uint32_t full = smem_u32(&bars->full[pipe.stage]);
        const uint32_t dst = ring + pipe.stage * kTileBytes;
        const CUtensorMap* map = op == 0 ? &k_map : &v_map;
        if constexpr (kFp8) {
          // e4m3 bytes: one box per page (128 B per key) into the upper half of the stage; the K
          // fill also leaves the K and V scales of the tile's pages in the tile's scale slot, before
          // the arrive that the readers' wait synchronises with.
          int pages[8];
          pages[0] = page0;
          if (ppt > 1) {
#pragma unroll
            for (int p = 0; p < 8; ++p)
              if (p < ppt) pages[p] = __ldg(bt + min(kt * ppt + p, npages - 1));  // past the end: reload the last
          }
          if (op == 0) {
            float* slot = scale_ring + (k_fills % kScaleSlots) * 16;
            ++k_fills;
            if (ppt == 1) {
              slot[0] = ks0;
              slot[8] = vs0;
            } else {
#pragma unroll
              for (int p = 0; p < 8; ++p) {
                if (p < ppt) {
                  const int64_t si = static_cast<int64_t>(pages[p]) * a.num_kv_heads + kv_head;
                  slot[p] = __ldg(a.k_scale + si);
                  slot[8 + p] = __ldg(a.v_scale + si);
                }
              }
            }
          }
          mbar_arrive_expect_tx(full, kHalfBytes);
          if (ppt == 1) {
            tma_load_4d_hint(dst + kHalfBytes, map, full, 0, 0, kv_head, page0, pol_stream);
          } else {
#pragma unroll
            for (int p = 0; p < 8; ++p)
              if (p < ppt) tma_load_4d(dst + kHalfBytes + p * page_bytes, map, full, 0, 0, kv_head, pages[p]);
          }
          pipe.advance();
          return;
        }
        mbar_arrive_expect_tx(full, kTileBytes);
        if (ppt == 1) {
          // K/V of streaming tasks is read once: mark it evict-first in L2 so that it does not
          // push out the K/V that the q tiles of a prefill share through L2 (kept evict-last).
          const uint64_t pol = by_umma ? pol_keep : pol_stream;
          tma_load_4d_hint(dst, map, full, 0, 0, kv_head, page0, pol);
          tma_load_4d_hint(dst + kHalfBytes, map, full, 64, 0, kv_head, page0, pol);
        } else {
          for (int p = 0; p < ppt; ++p) {
            const int pi = min(kt * ppt + p, npages - 1);  // pages past the end: reload the last
            const int page = __ldg(bt + pi);
            tma_load_4d(dst + p * page_bytes, map, full, 0, 0, kv_head, page);
            tma_load_4d(dst + kHalfBytes + p * page_bytes, map, full, 64, 0, kv_head, page);
          }
        }
        pipe.advance();
      };
      // A cursor over the worker's (task, key tile) sequence.  The block-table entry of a tile is
      // requested three tiles before the tile is issued, so its global-memory latency (and the
      // task / request loads at a task boundary) never sits between a stage's release and its
      // TMA: that latency would otherwise add to every refill of the ring.
      struct Tile {
        const int32_t* bt;
        int kv_head, kt, npages, page;
        float ks, vs;  // fp8, one page per tile: that page's K and V scale
        bool by_umma, valid;
      };
      int f_ti = t_begin, f_kt = 0, f_hi = 0, f_head = 0, f_npages = 1;
      uint32_t n_pub = 0;
      bool f_done = false;
      // Next task of this worker: its own list, or the head of the global queue (published to the
      // other roles through the ring; -1 is published once, when the queue is exhausted).
      auto grab = [&]() -> int {
        if (!dynamic) return f_ti < t_end ? f_ti++ : -1;
        if (f_done) return -1;
        int ti = -1;
        const int k = atomicAdd(a.queue_head, 1);
        if (k < a.num_tasks) ti = __ldg(a.queue + k);
        const uint32_t slot = n_pub % kTaskRing;
        if (n_pub >= kTaskRing &&
            !mbar_wait_block(smem_u32(&tq->empty[slot]), ((n_pub / kTaskRing) - 1u) & 1u, a.status)) {
          report_timeout(a);
          dead = true;
        }
        tq->ti[slot] = ti;
        mbar_arrive(smem_u32(&tq->full[slot]));
        ++n_pub;
        if (ti < 0) f_done = true;
        return ti;
      };
      const int32_t* f_bt = a.block_table;
      bool f_umma = false, f_open = false;
      auto next_tile = [&]() {
        Tile x;
        x.valid = false;
        x.bt = f_bt;
        x.kv_head = x.kt = x.page = 0;
        x.npages = 1;
        x.ks = x.vs = 1.f;
        x.by_umma = false;
        while (!f_open || f_kt >= f_hi) {
          const int ti = grab();
          if (ti < 0) return x;
          const xy_attn_task t = a.tasks[ti];
          const ReqInfo rq = a.reqs[t.req];
          f_kt = t.kt_lo;
          f_hi = t.kt_hi;
          f_head = t.kv_head;
          f_npages = (rq.kv_len + rq.q_len + a.page_size - 1) >> a.page_shift;
          f_bt = a.block_table + static_cast<int64_t>(rq.bt_row) * a.bt_stride;
          f_umma = kUmma && t.kind == 0;
          f_open = true;
        }
        x.valid = true;
        x.bt = f_bt;
        x.kv_head = f_head;
        x.kt = f_kt;
        x.npages = f_npages;
        x.by_umma = f_umma;
        x.page = __ldg(f_bt + min(f_kt * ppt, f_npages - 1));  // consumed three tiles later
        ++f_kt;
        return x;
      };
      // fp8, one page per tile: the page's scales are requested one step after its block-table
      // entry (which they depend on) and used one step later still.
      auto request_scales = [&](Tile& x) {
        if constexpr (kFp8) {
          if (ppt == 1 && x.valid) {
            const int64_t si = static_cast<int64_t>(x.page) * a.num_kv_heads + x.kv_head;
            x.ks = __ldg(a.k_scale + si);
            x.vs = __ldg(a.v_scale + si);
          }
        }
      };
      Tile q0 = next_tile(), q1 = next_tile(), q2 = next_tile();
      request_scales(q0);
      request_scales(q1);
      while (q0.valid && !dead) {
        const Tile cur = q0;
        q0 = q1;
        q1 = q2;
        q2 = next_tile();
        request_scales(q1);
        fill(0, cur.by_umma, cur.kv_head, cur.kt, cur.bt, cur.npages, cur.page, cur.ks, cur.vs);
        if (!dead) fill(1, cur.by_umma, cur.kv_head, cur.kt, cur.bt, cur.npages, cur.page, cur.ks, cur.vs);
      }
      // No bulk copy of this CTA may still be in flight when it exits: the latest fill of every
      // stage has landed once its `full` phase completes (immediate on the normal path, where the
      // readers have long consumed it; a bounded wait after a failure).
      for (int s = 0; s < kStages; ++s)
        if (used & (1u << s)) mbar_wait_block(smem_u32(&bars->full[s]), (fill_par >> s) & 1u, a.status);
    } else if (kUmma && (warp == kConsumerWarps + 1 || warp == kConsumerWarps + 2) && lane == 0) {
      // ================================ tcgen05 MMA issuers =============================
      // One issuing thread per sub-tile (on different schedulers), each walking its own chain
      //   S_X(0);  for j: [P_X(j) ready] O_X += P_X(j) V(j);  S_X(j+1) = Q_X K(j+1)^T.
      // The MMAs of one thread execute in order, which is what lets P overwrite S in place.
      const int X = warp - (kConsumerWarps + 1);
      uint32_t pos = 0;  // ring position: stage = pos % kStages, parity = (pos / kStages) & 1
      bool dead = false;
      uint32_t ph_q = 0, ph_p = 0;
      Tracer tr;
      tr.init(a, 2, X == 0);
      auto wait_or_die = [&](uint32_t bar, uint32_t parity) {
        if (!dead && !mbar_wait_block(bar, parity, a.status)) {
          report_timeout(a);
          dead = true;
        }
      };
      auto wait_full = [&](uint32_t p) {
        wait_or_die(smem_u32(&bars->full[p % kStages]), (p / kStages) & 1u);
        tc_fence_after();
      };
      // Descriptor halves.  High word (same for every operand here): 8-row groups 1024 B apart,
      // sm_100 descriptor version, 128-byte swizzle.  Low word: start address >> 4 in bits 0-13,
      // leading byte offset >> 4 in bits 16-29 (16 B for the K-major Q / K tiles; 16 KiB, the
      // distance to the second 64-element half, for the MN-major V tile).
      constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
      constexpr uint64_t kDescHi64 = static_cast<uint64_t>(kDescHi) << 32;
      const uint32_t ring_lo = (ring >> 4) & 0x3FFFu;
      const uint32_t t_s = tmem + kTmemS + X * 128, t_o = tmem + kTmemO + X * 128;
      // The issuing thread gets few issue slots next to the softmax warps, so everything an MMA
      // needs is computed ahead of the turn: Q descriptors once, K / V descriptors per tile.
      uint64_t qd[8];
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const uint32_t off = (ks >> 2) * (kHalfBytes >> 4) + (ks & 3) * 2;
        qd[ks] = kDescHi64 | (((((q_smem + X * kTileBytes) >> 4) & 0x3FFFu) + off) | (1u << 16));
      }
      // K tile (K-major): 8 k-steps of 16 elements, 32 B apart, the second half 16 KiB away
      auto k_descs = [&](uint32_t p, uint64_t (&kd)[8]) {
        const uint32_t b0 = (ring_lo + (p % kStages) * (kTileBytes >> 4)) | (1u << 16);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
          kd[ks] = kDescHi64 | (b0 + (ks >> 2) * (kHalfBytes >> 4) + (ks & 3) * 2);
      };
      // V tile (MN-major): 8 k-steps of 16 keys, 2 KiB apart; LBO = 16 KiB to the second half
      auto v_descs = [&](uint32_t p, uint64_t (&vd)[8]) {
        const uint32_t b0 = (ring_lo + (p % kStages) * (kTileBytes >> 4)) | ((kHalfBytes >> 4) << 16);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) vd[ks] = kDescHi64 | (b0 + ks * 128);
      };
      auto issue_qk = [&](const uint64_t (&kd)[8]) {  // S_X = Q_X K^T
        umma_ss64(t_s, qd[0], kd[0], kIdescQK, 0u);
#pragma unroll
        for (int ks = 1; ks < 8; ++ks) umma_ss64(t_s, qd[ks], kd[ks], kIdescQK, 1u);
        umma_commit(smem_u32(&ub->s_full[X]));
      };
      // O_X (+)= P_X V with P in TMEM, in two halves of 64 keys: the first half is issued while
      // the softmax warps are still exponentiating the second.
      auto issue_pv_lo = [&](const uint64_t (&vd)[8], bool accumulate) {
        umma_ts64(t_o, t_s, vd[0], kIdescPV, accumulate ? 1u : 0u);
#pragma unroll
        for (int ks = 1; ks < 4; ++ks) umma_ts64(t_o, t_s + ks * 8, vd[ks], kIdescPV, 1u);
      };
      auto issue_pv_hi = [&](const uint64_t (&vd)[8]) {
#pragma unroll
        for (int ks = 4; ks < 8; ++ks) umma_ts64(t_o, t_s + ks * 8, vd[ks], kIdescPV, 1u);
      };
      // A stage's empty barrier counts two arrivals: one per sub-tile that reads it, or both
      // from the only reader.
      auto release = [&](uint32_t p, bool alone) {
        umma_commit(smem_u32(&bars->empty_umma[p % kStages]));
        if (alone) umma_commit(smem_u32(&bars->empty_umma[p % kStages]));
      };
      // The two issuers take strict turns on the tensor pipe (A, B, A, B, ... skipping a sub-tile
      // that has nothing left), so that one sub-tile's softmax always overlaps the other's MMAs
      // instead of both falling into lockstep.  `turn` counts the groups issued so far.
      uint32_t g_base = 0;
      auto take_turn = [&](uint32_t g) {
        if (dead) return;
        for (uint32_t spin = 0; ub->turn != g; ++spin) {
          if (spin > (1u << 22) || ((spin & 4095u) == 4095u && wait_should_give_up(a.status, spin))) {
            report_timeout(a);
            dead = true;
            return;
          }
        }
      };
      auto pass_turn = [&](uint32_t g) { ub->turn = g + 1; };
      for (int ti = next_task(false); ti >= 0; ti = next_task(false)) {
        const xy_attn_task t = a.tasks[ti];
        const uint32_t n_all = t.kt_hi - t.kt_lo;
        const uint32_t pos0 = pos;
        pos += 2 * n_all;
        if (t.kind == 1) continue;  // streaming tasks never touch the tensor-memory path
        const ReqInfo rq = a.reqs[t.req];
        const DenseShape ds = dense_shape(t, rq, G);
        const int nX = ds.n[X], nY = ds.n[1 - X];
        const int nA = ds.n[0], nB = ds.n[1];
        const uint32_t g0 = g_base;                                  // first group of this task
        const uint32_t g1 = g0 + (nA > 0 ? 1u : 0u) + (nB > 0 ? 1u : 0u);  // first group of the j loop
        g_base = g1 + nA + nB;
        if (nX == 0) continue;
        wait_or_die(smem_u32(&ub->q_full[X]), ph_q);
        ph_q ^= 1u;
        uint64_t kd[8], vd[8];
        k_descs(pos0, kd);
        wait_full(pos0);
        {
          const uint32_t g = g0 + ((X == 1 && nA > 0) ? 1u : 0u);
          take_turn(g);
          if (!dead) {
            issue_qk(kd);
            release(pos0, nY == 0);
          }
          pass_turn(g);
        }
        for (int j = 0; j < nX; ++j) {
          const uint32_t pv = pos0 + 2 * j + 1, pk = pv + 1;
          const bool more = j + 1 < nX;
          const uint32_t g = g1 + min(j, nA) + min(j, nB) + ((X == 1 && j < nA) ? 1u : 0u);
          v_descs(pv, vd);
          k_descs(pk, kd);
          wait_full(pv);
          if (more) wait_full(pk);
          wait_or_die(smem_u32(&ub->p_full[X][0]), ph_p);
          tc_fence_after();
          tr(12);
          take_turn(g);
          tr(19);
          if (!dead) issue_pv_lo(vd, j > 0);
          wait_or_die(smem_u32(&ub->p_full[X][1]), ph_p);  // second half of P
          ph_p ^= 1u;
          tc_fence_after();
          if (!dead) {
            issue_pv_hi(vd);
            if (j == nX - 1) umma_commit(smem_u32(&ub->o_done[X]));
            release(pv, j >= nY);
            if (more) {
              issue_qk(kd);
              release(pk, j + 1 >= nY);
            }
          }
          pass_turn(g);
          tr(16);
        }
      }
      // Tensor memory is freed after the final barrier: no MMA of this thread may still be in
      // flight then.  On the normal path they completed long ago (immediate); after a failure
      // this is a bounded wait.
      umma_commit(smem_u32(&ub->drained[X]));
      mbar_wait_block(smem_u32(&ub->drained[X]), 0u, a.status);
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsConsumer));
    // ================================ consumers ========================================
    Pipe pipe{0, 0};
    bool dead = false;
    uint32_t ph_s = 0, ph_o = 0;  // this warpgroup's s_full / o_done parities
    uint32_t tile_seq = 0;        // key tiles consumed so far (fp8: selects the scale slot)
    Tracer tr;
    tr.init(a, warp >> 2, (threadIdx.x & 127) == 0);
    const int X = warp >> 2;       // sub-tile this warpgroup owns on the tcgen05 path
    // Time this worker spends in dense / streaming tasks, kept by thread 0 in shared memory.
    __shared__ unsigned long long acct_ns[2], acct_prev;
    __shared__ int acct_kind;
    if (threadIdx.x == 0) {
      acct_ns[0] = acct_ns[1] = 0ull;
      acct_kind = -1;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(acct_prev));
    }
    auto account = [&](int kind_now) {  // called by thread 0 at every task boundary
      unsigned long long now;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
      if (acct_kind >= 0) acct_ns[acct_kind] += now - acct_prev;
      acct_prev = now;
      acct_kind = kind_now;
    };
    for (int ti = next_task(true); ti >= 0; ti = next_task(true)) {
      TaskView tv;
      tv.t = a.tasks[ti];
      tv.rq = a.reqs[tv.t.req];
      tv.G = G;
      tv.rows = tv.t.ntok * G;
      const int h = tv.rq.kv_len;
      const bool tree = tv.rq.mask_kind == XY_MASK_TREE;
      const bool stream = tv.t.kind == 1;
      if (threadIdx.x == 0) account(stream ? 1 : 0);
      tr(30);

      if (kUmma && !stream) {
        // ---------------- dense on tcgen05: this thread owns packed row x of sub-tile X ----
        const DenseShape ds = dense_shape(tv.t, tv.rq, G);
        {  // the ring moves on without us: 2 n_all positions
          const uint32_t np = static_cast<uint32_t>(pipe.stage) + 2u * static_cast<uint32_t>(ds.n_all);
          pipe.stage = static_cast<int>(np % kStages);
          pipe.phase ^= (np / kStages) & 1u;
        }
        const int r = (warp & 3) * 32 + lane;
        const int x = X * 128 + r;
        const bool exists = X * 128 < tv.rows;
        const bool valid = x < tv.rows;
        if (!exists) continue;
        // A warp whose 32 rows all lie past the tile's last row has nothing to compute: it only
        // keeps step with the hand-offs (its rows of Q are zero, so are its rows of S, P and O).
        const bool warp_active = X * 128 + (warp & 3) * 32 < tv.rows;
        const int nX = ds.n[X];
        const int i_row = tv.t.tok0 + min(x, tv.rows - 1) / G;
        if (nX == 0) {  // a KV split that lies wholly above this sub-tile's causal frontier
          if (valid) {
            for (int c = 0; c < kHeadDim; c += 2) write_row_pair(a, tv, x, c, 0.f, 0.f);
            write_lse(a, tv, x, -INFINITY);
          }
          continue;
        }
        // packed Q sub-tile -> shared memory, then hand it to the async proxy
        {
          // Thread t copies 16-byte chunk (t & 15) of rows (t >> 4) + 8 it; the (token, head) of
          // a row advances by 8 packed rows per step, so one division per task suffices.
          tr(31);
          const int t128 = threadIdx.x & 127;
          const int ch = t128 & 15;
          const int x0 = X * 128 + (t128 >> 4);
          int i_q = x0 / G, h_q = x0 - i_q * G;
          const int di = 8 / G, dh = 8 - di * G;
          const uint16_t* qbase = a.q + static_cast<int64_t>(tv.rq.q_start + tv.t.tok0) * a.q_token_stride +
                                  static_cast<int64_t>(tv.t.kv_head) * G * kHeadDim + ch * 8;
#pragma unroll 4
          for (int it = 0; it < 16; ++it) {
            const int rr = (t128 >> 4) + 8 * it;
            const bool ok = X * 128 + rr < tv.rows;
            const uint16_t* src = ok ? qbase + static_cast<int64_t>(i_q) * a.q_token_stride + h_q * kHeadDim : qbase;
            cp_async_16(q_smem + X * kTileBytes + swz(rr, ch), src, ok);
            i_q += di;
            h_q += dh;
            if (h_q >= G) {
              h_q -= G;
              ++i_q;
            }
          }
          tr(32);
          cp_async_commit_wait_all();
          fence_proxy_async_smem();
          __syncwarp();
          tr(29);
          if (lane == 0) mbar_arrive(smem_u32(&ub->q_full[X]));
        }
        const uint32_t lane_base = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        const uint32_t t_s = lane_base + kTmemS + X * 128, t_o = lane_base + kTmemO + X * 128;
        const int i_min = tv.t.tok0 + (X * 128) / G;
        float m_ref = -INFINITY, l = 0.f;
        for (int j = 0; j < nX; ++j) {
          const int col0 = (tv.t.kt_lo + j) * kKeyTile;
          tr(20);
          if (!dead && !mbar_wait_block(smem_u32(&ub->s_full[X]), ph_s, a.status)) {
            report_timeout(a);
            dead = true;
          }
          ph_s ^= 1u;
          if (!warp_active) {
            __syncwarp();
            if (lane == 0) {
              mbar_arrive(smem_u32(&ub->p_full[X][0]));
              mbar_arrive(smem_u32(&ub->p_full[X][1]));
            }
            continue;
          }
          tc_fence_after();
          uint32_t sr[128];
          tmem_ld_32x32b_x32(t_s, &sr[0]);
          tmem_ld_32x32b_x32(t_s + 32, &sr[32]);
          tmem_ld_32x32b_x32(t_s + 64, &sr[64]);
          tmem_ld_32x32b_x32(t_s + 96, &sr[96]);
          tr(21);
          tmem_wait_ld();
          tr(22);
          const bool need_mask = tree ? (col0 + kKeyTile > h) : (col0 + kKeyTile > h + i_min + 1);
          if (need_mask) {
            // 128-bit visibility mask of this row for columns col0 .. col0 + 127, built with word
            // operations and applied with one test + select per element (no per-element branches).
            const int nvis = min(max(h + i_row - col0 + 1, 0), kKeyTile);  // causal frontier
            uint64_t v_lo = nvis >= 64 ? ~0ull : ((1ull << nvis) - 1ull);
            uint64_t v_hi = nvis >= 128 ? ~0ull : (nvis <= 64 ? 0ull : ((1ull << (nvis - 64)) - 1ull));
            if (tree) {
              // corner bit of column col is bit (col - h) of the row's ancestor-or-self words;
              // columns below h (the cached prefix) are visible to every row.
              const int jp0 = col0 - h;
              const int wbase = max(jp0, 0) >> 6;
              const uint64_t* mrow = a.tree_mask + tv.rq.tree_off + static_cast<int64_t>(i_row) * tv.rq.tree_words;
              uint64_t w0 = 0ull, w1 = 0ull, w2 = 0ull;
              if (wbase < tv.rq.tree_words) w0 = __ldg(mrow + wbase);
              if (wbase + 1 < tv.rq.tree_words) w1 = __ldg(mrow + wbase + 1);
              if (wbase + 2 < tv.rq.tree_words) w2 = __ldg(mrow + wbase + 2);
              uint64_t t_lo, t_hi;
              if (jp0 >= 0) {
                const int sh = jp0 & 63;
                t_lo = sh ? ((w0 >> sh) | (w1 << (64 - sh))) : w0;
                t_hi = sh ? ((w1 >> sh) | (w2 << (64 - sh))) : w1;
              } else {
                const int pre = -jp0;  // 1 .. 127 prefix columns lead the tile
                if (pre < 64) {
                  t_lo = ((1ull << pre) - 1ull) | (w0 << pre);
                  t_hi = (w0 >> (64 - pre)) | (w1 << pre);
                } else {
                  const int p2 = pre - 64;
                  t_lo = ~0ull;
                  t_hi = p2 ? (((1ull << p2) - 1ull) | (w0 << p2)) : w0;
                }
              }
              v_lo &= t_lo;
              v_hi &= t_hi;
            }
            const uint32_t vm[4] = {static_cast<uint32_t>(v_lo), static_cast<uint32_t>(v_lo >> 32),
                                    static_cast<uint32_t>(v_hi), static_cast<uint32_t>(v_hi >> 32)};
#pragma unroll
            for (int k = 0; k < 128; ++k)
              sr[k] = (vm[k >> 5] & (1u << (k & 31))) ? sr[k] : 0xff800000u;  // -inf, selected (never added)
          }
          float mx;
          {  // eight independent chains of three-input max, then a short tree
            float m8[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) m8[q] = fmaxf(__uint_as_float(sr[q]), __uint_as_float(sr[q + 8]));
#pragma unroll
            for (int k = 16; k < 128; k += 16) {
#pragma unroll
              for (int q = 0; q < 8; ++q)
                m8[q] = max3(m8[q], __uint_as_float(sr[k + q]), __uint_as_float(sr[k + q + 8]));
            }
            mx = max3(max3(m8[0], m8[1], m8[2]), max3(m8[3], m8[4], m8[5]), fmaxf(m8[6], m8[7]));
          }
          tr(23);
          const float m_cand = fmaxf(m_ref, mx * scale_log2);
          bool need = false;
          if (j == 0 || m_ref == -INFINITY) {
            m_ref = m_cand;  // nothing accumulated yet for this row: adopt the max, no rescale
          } else {
            need = m_cand - m_ref > kRescaleThreshold;
          }
          if (__any_sync(0xffffffffu, need)) {
            // Update stage: O *= 2^(m_old - m_new).  The previous P V has completed, because
            // this tile's S was issued behind it on the in-order tensor pipe.
            const float alpha = (m_cand == -INFINITY) ? 1.f : ex2(m_ref - m_cand);
            l *= alpha;
            m_ref = m_cand;
#pragma unroll 1
            for (int c = 0; c < 8; ++c) {  // rare path: small chunks, the 128 scores stay live
              uint32_t orow[16];
              tmem_ld_32x32b_x16(t_o + c * 16, orow);
              tmem_wait_ld();
#pragma unroll
              for (int k = 0; k < 16; ++k) orow[k] = __float_as_uint(__uint_as_float(orow[k]) * alpha);
              tmem_st_32x32b_x16(t_o + c * 16, orow);
            }
          }
          tr(24);
          const float neg_off = (m_ref == -INFINITY) ? 0.f : -m_ref;
          // P = 2^(s * scale - m), two keys packed per 32-bit column, written over sr in place.
          // The scale-and-subtract and the row sum run as packed f32x2 instructions.
          const uint64_t scale2 = pack_f32x2(scale_log2, scale_log2), off2 = pack_f32x2(neg_off, neg_off);
          uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
          for (int half = 0; half < 2; ++half) {
#pragma unroll
            for (int k = half * 32; k < half * 32 + 32; ++k) {
              float x0, x1;
              unpack_f32x2(
                  fma_f32x2(pack_f32x2(__uint_as_float(sr[2 * k]), __uint_as_float(sr[2 * k + 1])), scale2, off2), x0,
                  x1);
              const float p0 = ex2(x0), p1 = ex2(x1);
              sum2[k & 3] = add_f32x2(sum2[k & 3], pack_f32x2(p0, p1));
              sr[k] = pack_bf16(p0, p1);
            }
            // hand this half of P (64 keys, 32 columns) to the MMA issuer
            tmem_st_32x32b_x32(t_s + half * 32, &sr[half * 32]);
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ub->p_full[X][half]));
            if (half == 0) tr(25);
          }
          {
            float a0, a1;
            unpack_f32x2(add_f32x2(add_f32x2(sum2[0], sum2[1]), add_f32x2(sum2[2], sum2[3])), a0, a1);
            l += a0 + a1;
          }
          tr(26);
        }
        // ---- epilogue: O / l -> global
        if (!dead && !mbar_wait_block(smem_u32(&ub->o_done[X]), ph_o, a.status)) {
          report_timeout(a);
          dead = true;
        }
        ph_o ^= 1u;
        tc_fence_after();
        tr(27);
        const float inv = l > 0.f ? 1.f / l : 0.f;
        if (tv.t.part < 0) {
          // Final output.  A thread holds one row, so direct stores would touch 32 rows per warp
          // instruction.  The bf16 rows go through this sub-tile's Q area of shared memory instead
          // (its MMAs have completed; 16-byte chunks XOR-swizzled by row so that neither side has
          // bank conflicts) and leave as row-contiguous 256-byte stores, two rows per instruction.
          uint8_t* stage = gen_base + X * kTileBytes;
          if (warp_active) {
            uint32_t orow[128];  // the whole row with one wait: four loads in flight together
            tmem_ld_32x32b_x32(t_o, &orow[0]);
            tmem_ld_32x32b_x32(t_o + 32, &orow[32]);
            tmem_ld_32x32b_x32(t_o + 64, &orow[64]);
            tmem_ld_32x32b_x32(t_o + 96, &orow[96]);
            tmem_wait_ld();
#pragma unroll
            for (int q = 0; q < 16; ++q) {
              uint4 v;
              v.x = pack_bf16(__uint_as_float(orow[q * 8 + 0]) * inv, __uint_as_float(orow[q * 8 + 1]) * inv);
              v.y = pack_bf16(__uint_as_float(orow[q * 8 + 2]) * inv, __uint_as_float(orow[q * 8 + 3]) * inv);
              v.z = pack_bf16(__uint_as_float(orow[q * 8 + 4]) * inv, __uint_as_float(orow[q * 8 + 5]) * inv);
              v.w = pack_bf16(__uint_as_float(orow[q * 8 + 6]) * inv, __uint_as_float(orow[q * 8 + 7]) * inv);
              *reinterpret_cast<uint4*>(stage + r * 256 + ((q ^ (r & 15)) << 4)) = v;
            }
          }
          __syncwarp();
          if (warp_active) {  // a warp stores only rows it staged itself
            const int ch = lane & 15;
            int rr = (warp & 3) * 32 + (lane >> 4);  // row of the sub-tile this lane stores first
            const int xs = X * 128 + rr;
            int i_o = xs / G, h_o = xs - i_o * G;
            const int di = 2 / G, dh = 2 - di * G;
            uint16_t* obase = a.o + static_cast<int64_t>(tv.rq.q_start + tv.t.tok0) * a.o_token_stride +
                              static_cast<int64_t>(tv.t.kv_head) * G * kHeadDim + ch * 8;
#pragma unroll 4
            for (int it = 0; it < 16; ++it) {
              if (X * 128 + rr < tv.rows) {
                const uint4 v = *reinterpret_cast<const uint4*>(stage + rr * 256 + ((ch ^ (rr & 15)) << 4));
                *reinterpret_cast<uint4*>(obase + static_cast<int64_t>(i_o) * a.o_token_stride + h_o * kHeadDim) = v;
              }
              rr += 2;
              i_o += di;
              h_o += dh;
              if (h_o >= G) {
                h_o -= G;
                ++i_o;
              }
            }
          }
          named_bar_sync(2 + X, 128);  // staging reads done before the next task's Q lands here
        } else if (warp_active) {
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t orow[32];
            tmem_ld_32x32b_x32(t_o + c * 32, orow);
            tmem_wait_ld();
            if (valid) {
              float4* dst = reinterpret_cast<float4*>(a.o_part + static_cast<int64_t>(tv.t.part + x) * kHeadDim + c * 32);
#pragma unroll
              for (int q = 0; q < 8; ++q)
                dst[q] = make_float4(__uint_as_float(orow[q * 4 + 0]) * inv, __uint_as_float(orow[q * 4 + 1]) * inv,
                                     __uint_as_float(orow[q * 4 + 2]) * inv, __uint_as_float(orow[q * 4 + 3]) * inv);
            }
          }
        }
        if (valid) write_lse(a, tv, x, l > 0.f ? (m_ref + log2f(l)) * kLn2 : -INFINITY);
        tc_fence_before();  // order this task's TMEM reads before the next task's MMAs
        tr(28);
        continue;
      }

      // ---- packed Q tile -> shared memory (rows past the tile are zero-filled)
      // A warpgroup that had no sub-tile in the previous dense task arrives here while the other
      // one may still be computing on its Q tile, which this load overwrites: meet first.
      if (kUmma) named_bar_sync(1, kConsumerThreads);
      {
        const int rows_pad = stream ? 16 : 128;
        for (int c = threadIdx.x; c < rows_pad * 16; c += kConsumerThreads) {
          const int x = c >> 4, ch = c & 15;
          const bool ok = x < tv.rows;
          const int xx = ok ? x : 0;
          const int i = tv.t.tok0 + xx / G, head = tv.t.kv_head * G + xx % G;
          const uint16_t* src =
              a.q + static_cast<int64_t>(tv.rq.q_start + i) * a.q_token_stride + head * kHeadDim + ch * 8;
          cp_async_16(q_smem + swz(x, ch), src, ok);
        }
        cp_async_commit_wait_all();
        named_bar_sync(1, kConsumerThreads);
        if constexpr (kFp8) {
          // Q rows become f16 with a power-of-two factor per row (dense: each warp its own 16 rows;
          // streaming: the 16 rows shared by all warps, two per warp)
          if (stream) q_rows_to_f16<16>(q_smem, warp * 2, qmult, lane);
          else q_rows_to_f16<2>(q_smem, warp * 16, qmult, lane);
          named_bar_sync(1, kConsumerThreads);
        }
      }

      if (!kUmma && !stream) {  // (with kUmma every dense task took the tcgen05 path above)
        // ---------------- dense: this warp owns rows x0 .. x0+15 -------------------------
        const int x0 = warp * 16;
        const bool active = x0 < tv.rows;
        WarpTile<16, false, kFp8> w;
        w.init();
        if (active) w.load_q(q_smem, x0, lane);
        FpScale fs{1.f, 1.f, scale_ring, a.page_shift};
        if constexpr (kFp8) {
          fs.q_lo = qmult[x0 + (lane >> 2)];
          fs.q_hi = qmult[x0 + (lane >> 2) + 8];
        }
        const int r_lo = min(x0 + (lane >> 2), tv.rows - 1), r_hi = min(x0 + (lane >> 2) + 8, tv.rows - 1);
        const int i_lo = tv.t.tok0 + r_lo / G, i_hi = tv.t.tok0 + r_hi / G;
        const int i_min = tv.t.tok0 + min(x0, tv.rows - 1) / G;
        const int i_max = tv.t.tok0 + min(x0 + 15, tv.rows - 1) / G;
        for (int kt = tv.t.kt_lo; kt < tv.t.kt_hi; ++kt) {
          const int col0 = kt * kKeyTile;
          const bool work = active && col0 <= h + i_max;  // mask-aware skip (Section 4.2.2)
          float s[16][4];
          uint32_t p[8][4];
          if (!dead && !mbar_wait_block(smem_u32(&bars->full[pipe.stage]), pipe.phase, a.status)) {
            report_timeout(a);
            dead = true;
          }
          if constexpr (kFp8) {
            // every warp widens 16 keys of the tile, all warps read all of it
            fs.tile = scale_ring + (tile_seq % kScaleSlots) * 16;
            ++tile_seq;
            widen_rows16(ring + pipe.stage * kTileBytes, warp * 16, lane);
            named_bar_sync(1, kConsumerThreads);
          }
          if (work) w.qk(ring + pipe.stage * kTileBytes, 0, lane, s);
          if constexpr (kFp8) fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&bars->empty[pipe.stage]));
          pipe.advance();
          if (work) {
            const bool need_mask = tree ? (col0 + kKeyTile > h) : (col0 + kKeyTile > h + i_min + 1);
            w.softmax(a, tv.rq, s, p, col0, i_lo, i_hi, need_mask, scale_log2, lane, &fs, 0);
          }
          if (!dead && !mbar_wait_block(smem_u32(&bars->full[pipe.stage]), pipe.phase, a.status)) {
            report_timeout(a);
            dead = true;
          }
          if constexpr (kFp8) {
            widen_rows16(ring + pipe.stage * kTileBytes, warp * 16, lane);
            named_bar_sync(1, kConsumerThreads);
          }
          if (work) w.pv(ring + pipe.stage * kTileBytes, 0, lane, p);
          if constexpr (kFp8) fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&bars->empty[pipe.stage]));
          pipe.advance();
        }
        if (active) {
          w.reduce_l();
          const float inv_lo = w.l_lo > 0.f ? 1.f / w.l_lo : 0.f;
          const float inv_hi = w.l_hi > 0.f ? 1.f / w.l_hi : 0.f;
          const int xl = x0 + (lane >> 2), xh = xl + 8;
#pragma unroll
          for (int n = 0; n < 16; ++n) {
            const int col = n * 8 + 2 * (lane & 3);
            if (xl < tv.rows) write_row_pair(a, tv, xl, col, w.o[n][0] * inv_lo, w.o[n][1] * inv_lo);
            if (xh < tv.rows) write_row_pair(a, tv, xh, col, w.o[n][2] * inv_hi, w.o[n][3] * inv_hi);
          }
          if ((lane & 3) == 0) {
            if (xl < tv.rows)
              write_lse(a, tv, xl, w.l_lo > 0.f ? (w.m_lo + log2f(w.l_lo)) * kLn2 : -INFINITY);
            if (xh < tv.rows)
              write_lse(a, tv, xh, w.l_hi > 0.f ? (w.m_hi + log2f(w.l_hi)) * kLn2 : -INFINITY);
          }
        }
        named_bar_sync(1, kConsumerThreads);  // Q tile may be overwritten by the next task
      } else {
        // ---------------- streaming (see stream_task) ----
        const uint32_t st = stream_task<kFp8>(a, tv, q_smem, ring, bars, xch, ml, pipe.stage | (pipe.phase << 8) |
                                              (dead ? 1u << 16 : 0u), scale_log2, qmult, scale_ring, tile_seq,
                                              (a.task_unit != nullptr && tv.t.part >= 0) ? a.task_unit[ti] : -1);
        pipe.stage = st & 0xFFu;
        pipe.phase = (st >> 8) & 1u;
        dead = (st >> 16) & 1u;
        named_bar_sync(1, kConsumerThreads);
      }
    }
    if (threadIdx.x == 0) {
      account(-1);
      a.worker_times[4 * blockIdx.x + 2] = acct_ns[0];
      a.worker_times[4 * blockIdx.x + 3] = acct_ns[1];
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long now;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
    a.worker_times[4 * blockIdx.x + 1] = now;
  }
  if (kUmma && warp == kConsumerWarps + 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}

#include "kernel_pair.inc"

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
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

// 4-D map over a paged pool [pages, Hkv, B, D]: box = one page of one head, 64 elements wide.
// box_tokens: tokens per box (0: a whole page)
bool encode_pool_map(CUtensorMap* m, const void* pool, int64_t num_pages, int num_kv_heads, int page_size,
                     int64_t page_stride, int64_t head_stride, int64_t token_stride, bool fp8, int box_tokens = 0) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  // bf16: two boxes of 64 elements per row; e4m3 bytes: one box of 128 - 128 B per row either way
  const cuuint64_t esz = fp8 ? 1 : 2;
  cuuint64_t dims[4] = {static_cast<cuuint64_t>(kHeadDim), static_cast<cuuint64_t>(page_size),
                        static_cast<cuuint64_t>(num_kv_heads), static_cast<cuuint64_t>(num_pages)};
  cuuint64_t strides[3] = {static_cast<cuuint64_t>(token_stride) * esz, static_cast<cuuint64_t>(head_stride) * esz,
                           static_cast<cuuint64_t>(page_stride) * esz};
  cuuint32_t box[4] = {fp8 ? 128u : 64u, static_cast<cuuint32_t>(box_tokens > 0 ? box_tokens : page_size), 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(m, fp8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(pool), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace

cudaError_t launch_meta(const RunArgs& a, int num_workers, int64_t num_pages, bool umma, MetaLaunchCache* cache,
                        cudaStream_t s) {
  static_assert(sizeof(CUtensorMap) == 128, "MetaLaunchCache holds a tensor map in 128 bytes");
  const bool fp8 = a.kv_fp8 != 0;
  if (fp8) umma = false;
  auto kernel = fp8 ? meta_attention_kernel<false, true>
                    : (umma ? meta_attention_kernel<true, false> : meta_attention_kernel<false, false>);
  const int which = fp8 ? 2 : (umma ? 1 : 0);
  if (!cache->attr_set[which]) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTotal);
    if (e != cudaSuccess) return e;
    cache->attr_set[which] = true;
  }
  CUtensorMap* k_map = reinterpret_cast<CUtensorMap*>(cache->maps[0]);
  CUtensorMap* v_map = reinterpret_cast<CUtensorMap*>(cache->maps[1]);
  const bool same = cache->valid && cache->k_pool == a.k_pool && cache->v_pool == a.v_pool &&
                    cache->num_pages == num_pages && cache->page_stride == a.page_stride &&
                    cache->head_stride == a.head_stride && cache->token_stride == a.token_stride &&
                    cache->num_kv_heads == a.num_kv_heads && cache->page_size == a.page_size && cache->fp8 == fp8;
  if (!same) {
    cache->valid = false;
    if (!encode_pool_map(k_map, a.k_pool, num_pages, a.num_kv_heads, a.page_size, a.page_stride, a.head_stride,
                         a.token_stride, fp8) ||
        !encode_pool_map(v_map, a.v_pool, num_pages, a.num_kv_heads, a.page_size, a.page_stride, a.head_stride,
                         a.token_stride, fp8))
      return cudaErrorInvalidValue;
    cache->k_pool = a.k_pool;
    cache->v_pool = a.v_pool;
    cache->num_pages = num_pages;
    cache->page_stride = a.page_stride;
    cache->head_stride = a.head_stride;
    cache->token_stride = a.token_stride;
    cache->num_kv_heads = a.num_kv_heads;
    cache->page_size = a.page_size;
    cache->fp8 = fp8;
    cache->valid = true;
  }
  MetaParams P{a};
  kernel<<<num_workers, kThreads, kSmemTotal, s>>>(P, *k_map, *v_map);
  return cudaGetLastError();
}

// Dense tasks on CTA pairs: `a.queue` / `a.num_tasks` / `a.queue_head` describe the dense part of the
// plan's queue.  num_workers CTAs (even) = num_workers / 2 pairs.
cudaError_t launch_pair_dense(const RunArgs& a, int num_workers, int64_t num_pages, MetaLaunchCache* cache,
                              cudaStream_t s) {
  if (num_workers < 2) return cudaErrorInvalidValue;
  if (!cache->attr_set[3]) {
    cudaError_t e = cudaFuncSetAttribute(pair_dense_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTotal);
    if (e != cudaSuccess) return e;
    cache->attr_set[3] = true;
  }
  CUtensorMap* k_map = reinterpret_cast<CUtensorMap*>(cache->pair_maps[0]);
  CUtensorMap* v_map = reinterpret_cast<CUtensorMap*>(cache->pair_maps[1]);
  const bool same = cache->pair_valid && cache->pk_pool == a.k_pool && cache->pv_pool == a.v_pool &&
                    cache->p_num_pages == num_pages && cache->p_page_stride == a.page_stride &&
                    cache->p_head_stride == a.head_stride && cache->p_token_stride == a.token_stride &&
                    cache->p_num_kv_heads == a.num_kv_heads && cache->p_page_size == a.page_size;
  if (!same) {
    cache->pair_valid = false;
    // K: boxes of at most 64 tokens (a CTA stages 64 keys of a tile); V: whole pages, 64 columns
    if (!encode_pool_map(k_map, a.k_pool, num_pages, a.num_kv_heads, a.page_size, a.page_stride, a.head_stride,
                         a.token_stride, false, a.page_size < 64 ? a.page_size : 64) ||
        !encode_pool_map(v_map, a.v_pool, num_pages, a.num_kv_heads, a.page_size, a.page_stride, a.head_stride,
                         a.token_stride, false))
      return cudaErrorInvalidValue;
    cache->pk_pool = a.k_pool;
    cache->pv_pool = a.v_pool;
    cache->p_num_pages = num_pages;
    cache->p_page_stride = a.page_stride;
    cache->p_head_stride = a.head_stride;
    cache->p_token_stride = a.token_stride;
    cache->p_num_kv_heads = a.num_kv_heads;
    cache->p_page_size = a.page_size;
    cache->pair_valid = true;
  }
  MetaParams P{a};
  pair_dense_kernel<<<num_workers & ~1, kThreads, kSmemTotal, s>>>(P, *k_map, *v_map);
  return cudaGetLastError();
}

}  // namespace xy
