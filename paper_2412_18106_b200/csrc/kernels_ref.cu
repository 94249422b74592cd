// Reference attention kernel (plain SIMT, fp32), the split-KV LSE merge and the
// block-table gather.  The reference kernel walks the same Task-Table as the fast
// kernels and is kept for bisecting: one warp per packed row, one key at a time.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>

#include "xy_kernels.h"

namespace xy {

namespace {

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) {
  return __uint_as_float(static_cast<uint32_t>(b) << 16);
}

__device__ __forceinline__ uint16_t float_to_bf16_bits(float f) {
  return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}

// Four consecutive K or V elements of a cached token as fp32: bf16 pools, or (fp8 KV cache) e4m3
// bytes times the page's scale.  `off` counts elements from the pool's base.
__device__ __forceinline__ void load_kv4(const RunArgs& a, const uint16_t* pool, int64_t off, float scale, float (&out)[4]) {
  if (a.kv_fp8) {
    const uint32_t w = *reinterpret_cast<const uint32_t*>(reinterpret_cast<const uint8_t*>(pool) + off);
    const __half2_raw lo = __nv_cvt_fp8x2_to_halfraw2(static_cast<__nv_fp8x2_storage_t>(w & 0xFFFFu), __NV_E4M3);
    const __half2_raw hi = __nv_cvt_fp8x2_to_halfraw2(static_cast<__nv_fp8x2_storage_t>(w >> 16), __NV_E4M3);
    const float2 f0 = __half22float2(__half2(lo)), f1 = __half22float2(__half2(hi));
    out[0] = f0.x * scale;
    out[1] = f0.y * scale;
    out[2] = f1.x * scale;
    out[3] = f1.y * scale;
  } else {
#pragma unroll
    for (int d = 0; d < 4; ++d) out[d] = bf16_bits_to_float(pool[off + d]);
  }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Section 4.2.1 (QK -> Softmax -> SV per tile unit, with the Update rescale), Section 4.1.1
// (K/V rows found through the block table), Sections 4.1.2 / 4.2.2 (row-wise mask control).
__global__ void __launch_bounds__(128) ref_attention_kernel(RunArgs a) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = a.num_q_heads / a.num_kv_heads;
  const int t_begin = a.worker_off[blockIdx.x], t_end = a.worker_off[blockIdx.x + 1];
  for (int ti = t_begin; ti < t_end; ++ti) {
    const xy_attn_task t = a.tasks[ti];
    const ReqInfo rq = a.reqs[t.req];
    const int rows = t.ntok * G;
    const int32_t* bt = a.block_table + static_cast<int64_t>(rq.bt_row) * a.bt_stride;
    for (int x = warp; x < rows; x += 4) {
      const int i = t.tok0 + x / G;
      const int head = t.kv_head * G + x % G;
      const uint16_t* qp =
          a.q + static_cast<int64_t>(rq.q_start + i) * a.q_token_stride + head * kHeadDim + lane * 4;
      float qv[4];
#pragma unroll
      for (int d = 0; d < 4; ++d) qv[d] = bf16_bits_to_float(qp[d]);
      const uint64_t* mrow = nullptr;
      if (rq.mask_kind == XY_MASK_TREE)
        mrow = a.tree_mask + rq.tree_off + static_cast<int64_t>(i) * rq.tree_words;
      const int j_lo = t.kt_lo * kKeyTile;
      const int j_hi = min(t.kt_hi * kKeyTile, rq.kv_len + i + 1);
      float m = -INFINITY, l = 0.f, o[4] = {0.f, 0.f, 0.f, 0.f};
      for (int j = j_lo; j < j_hi; ++j) {
        if (j >= rq.kv_len && mrow != nullptr) {
          const int jp = j - rq.kv_len;
          if (((mrow[jp >> 6] >> (jp & 63)) & 1ull) == 0ull) continue;
        }
        const int64_t page = bt[j >> a.page_shift];
        const int64_t off = page * a.page_stride + static_cast<int64_t>(t.kv_head) * a.head_stride +
                            static_cast<int64_t>(j & (a.page_size - 1)) * a.token_stride + lane * 4;
        float kf[4], vf[4];
        float ksc = 1.f, vsc = 1.f;
        if (a.kv_fp8) {
          ksc = a.k_scale[page * a.num_kv_heads + t.kv_head];
          vsc = a.v_scale[page * a.num_kv_heads + t.kv_head];
        }
        load_kv4(a, a.k_pool, off, ksc, kf);
        load_kv4(a, a.v_pool, off, vsc, vf);
        float dot = 0.f;
#pragma unroll
        for (int d = 0; d < 4; ++d) dot += qv[d] * kf[d];
        const float s = warp_sum(dot) * a.sm_scale;
        const float m_new = fmaxf(m, s);
        const float alpha = __expf(m - m_new);  // m = -inf on the first key: alpha = 0
        const float p = __expf(s - m_new);
        l = l * alpha + p;
#pragma unroll
        for (int d = 0; d < 4; ++d) o[d] = o[d] * alpha + p * vf[d];
        m = m_new;
      }
      const float inv = l > 0.f ? 1.f / l : 0.f;
      const float lse = l > 0.f ? m + logf(l) : -INFINITY;
      if (t.part < 0) {
        uint16_t* op = a.o + static_cast<int64_t>(rq.q_start + i) * a.o_token_stride +
                       head * kHeadDim + lane * 4;
#pragma unroll
        for (int d = 0; d < 4; ++d) op[d] = float_to_bf16_bits(o[d] * inv);
        if (lane == 0) a.lse[static_cast<int64_t>(rq.q_start + i) * a.num_q_heads + head] = lse;
      } else {
        float* op = a.o_part + static_cast<int64_t>(t.part + x) * kHeadDim + lane * 4;
#pragma unroll
        for (int d = 0; d < 4; ++d) op[d] = o[d] * inv;
        if (lane == 0) a.lse_part[t.part + x] = lse;
      }
    }
  }
}

// Cross-task form of the Update stage (Section 4.2.1): combine the partials of every tile
// unit whose KV range was split.  One warp per packed row (a unit has at most 256): lane l holds
// LSE_c of splits l, l + 32, ..., the maximum and the sum go through warp shuffles, and the
// weights exp(LSE_c - LSE) are broadcast while the lanes accumulate four output columns each,
// eight partial rows per round so that their loads are in flight together.
constexpr int kMergeBlocksPerUnit = 64;  // x 4 warps = 256 rows
constexpr int kMergeLaneParts = 8;     // partials per lane on the shuffle path: up to 256 per row
// kWide: some unit has more than 32 partials per row (a single long context cut for every
// worker); that path holds eight partial rows in registers and is kept out of the common kernel.
template <bool kWide>
__global__ void __launch_bounds__(128) merge_units_kernel(MergeArgs a) {
  const xy_attn_merge_unit u = a.units[blockIdx.x];
  const int G = a.num_q_heads / a.num_kv_heads;
  const int rows = u.ntok * G;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (blockIdx.y * 4 >= rows) return;
  const ReqInfo rq = a.reqs[u.req];
  for (int x = blockIdx.y * 4 + warp; x < rows; x += 4 * gridDim.y) {
    float lse;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    // partial row of part c: the unit's own splits first, then the second family (the rows a
    // member of a shared-prefix group has in the group tile's partials)
    const int nparts = u.nsplit + u.nsplit1;
    auto part_row = [&](int c) -> int64_t {
      return c < u.nsplit ? static_cast<int64_t>(u.part0) + static_cast<int64_t>(c) * rows + x
                          : static_cast<int64_t>(u.part1) + static_cast<int64_t>(c - u.nsplit) * u.stride1 + x;
    };
    if (nparts <= 32) {
      // the common case: lane c holds LSE_c; the partial rows are read four at a time
      const float lc = lane < nparts ? a.lse_part[part_row(lane)] : -INFINITY;
      float mx = lc;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float e = lc != -INFINITY ? __expf(lc - mx) : 0.f;
      float z = e;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
      lse = mx + logf(z);
      const float w_mine = z > 0.f ? e / z : 0.f;
      for (int c0 = 0; c0 < nparts; c0 += 4) {
        float w[4];
        float4 v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int c = c0 + q;
          w[q] = __shfl_sync(0xffffffffu, w_mine, c & 31);
          if (c >= nparts) w[q] = 0.f;
          // an empty split (LSE_c = -inf, weight 0) is not read
          v[q] = w[q] != 0.f ? *reinterpret_cast<const float4*>(a.o_part + part_row(c) * kHeadDim + lane * 4)
                             : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          acc.x += w[q] * v[q].x;
          acc.y += w[q] * v[q].y;
          acc.z += w[q] * v[q].z;
          acc.w += w[q] * v[q].w;
        }
      }
    } else if (kWide && nparts <= 32 * kMergeLaneParts) {
      // lane l holds LSE_c of parts l, l + 32, ...; maximum and sum go through shuffles; the
      // partial rows are then read eight at a time (independent loads in flight together)
      float lc[kMergeLaneParts], mx = -INFINITY;
#pragma unroll
      for (int k = 0; k < kMergeLaneParts; ++k) {
        const int c = k * 32 + lane;
        lc[k] = c < nparts ? a.lse_part[part_row(c)] : -INFINITY;
        mx = fmaxf(mx, lc[k]);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      float z = 0.f;
#pragma unroll
      for (int k = 0; k < kMergeLaneParts; ++k) {
        lc[k] = lc[k] != -INFINITY ? __expf(lc[k] - mx) : 0.f;
        z += lc[k];
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
      lse = mx + logf(z);
      const float rz = z > 0.f ? 1.f / z : 0.f;
#pragma unroll
      for (int k = 0; k < kMergeLaneParts; ++k) {
        if (k * 32 >= nparts) break;
        const float w_mine = lc[k] * rz;
        for (int j = 0; j < 32 && k * 32 + j < nparts; j += 8) {
          float w[8];
          float4 v[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const int c = k * 32 + j + e;
            w[e] = __shfl_sync(0xffffffffu, w_mine, (j + e) & 31);
            // an empty split (LSE_c = -inf, weight 0) is not read
            v[e] = (c < nparts && w[e] != 0.f)
                       ? *reinterpret_cast<const float4*>(a.o_part + part_row(c) * kHeadDim + lane * 4)
                       : make_float4(0.f, 0.f, 0.f, 0.f);
            if (c >= nparts) w[e] = 0.f;
          }
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            acc.x += w[e] * v[e].x;
            acc.y += w[e] * v[e].y;
            acc.z += w[e] * v[e].z;
            acc.w += w[e] * v[e].w;
          }
        }
      }
    } else {
      float mx = -INFINITY;
      for (int c = 0; c < nparts; ++c) mx = fmaxf(mx, a.lse_part[part_row(c)]);
      float z = 0.f;
      for (int c = 0; c < nparts; ++c) {
        const float lc = a.lse_part[part_row(c)];
        if (lc != -INFINITY) z += __expf(lc - mx);
      }
      lse = mx + logf(z);
      for (int c = 0; c < nparts; ++c) {
        const float lc = a.lse_part[part_row(c)];
        if (lc == -INFINITY) continue;
        const float w = __expf(lc - lse);
        const float4 v = *reinterpret_cast<const float4*>(a.o_part + part_row(c) * kHeadDim + lane * 4);
        acc.x += w * v.x;
        acc.y += w * v.y;
        acc.z += w * v.z;
        acc.w += w * v.w;
      }
    }
    const int i = u.tok0 + x / G;
    const int head = u.kv_head * G + x % G;
    uint16_t* op =
        a.o + static_cast<int64_t>(rq.q_start + i) * a.o_token_stride + head * kHeadDim + lane * 4;
    uint2 packed;
    packed.x = float_to_bf16_bits(acc.x) | (static_cast<uint32_t>(float_to_bf16_bits(acc.y)) << 16);
    packed.y = float_to_bf16_bits(acc.z) | (static_cast<uint32_t>(float_to_bf16_bits(acc.w)) << 16);
    *reinterpret_cast<uint2*>(op) = packed;
    if (lane == 0) a.lse[static_cast<int64_t>(rq.q_start + i) * a.num_q_heads + head] = lse;
  }
}

// Context-free merge over plain [num_splits, rows, D] partials.
__global__ void __launch_bounds__(128) merge_plain_kernel(const float* o_part, const float* lse_part,
                                                         int num_splits, int64_t rows, uint16_t* o,
                                                         float* lse_out) {
  const int lane = threadIdx.x & 31;
  const int64_t x = static_cast<int64_t>(blockIdx.x) * 4 + (threadIdx.x >> 5);
  if (x >= rows) return;
  float mx = -INFINITY;
  for (int c = 0; c < num_splits; ++c) mx = fmaxf(mx, lse_part[c * rows + x]);
  float z = 0.f;
  for (int c = 0; c < num_splits; ++c) {
    const float lc = lse_part[c * rows + x];
    if (lc != -INFINITY) z += __expf(lc - mx);
  }
  const float lse = mx + logf(z);
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int c = 0; c < num_splits; ++c) {
    const float lc = lse_part[c * rows + x];
    if (lc == -INFINITY) continue;
    const float w = __expf(lc - lse);
    const float* v = o_part + (c * rows + x) * kHeadDim + lane * 4;
#pragma unroll
    for (int d = 0; d < 4; ++d) acc[d] += w * v[d];
  }
#pragma unroll
  for (int d = 0; d < 4; ++d) o[x * kHeadDim + lane * 4 + d] = float_to_bf16_bits(acc[d]);
  if (lane == 0) lse_out[x] = lse;
}

// Merge of per-device results when the context of a request is sharded over devices: every
// shard ran attention over its own slice of the keys and produced a normalised bf16 O_c and
// LSE_c; the merge is the same Update formula (Section 4.2.1).  One warp per row; lane c holds
// LSE_c when there are at most 32 shards; each lane owns four output columns.
__global__ void __launch_bounds__(128) merge_shards_kernel(const uint16_t* o_shards, const float* lse_shards,
                                                          int num_shards, int64_t rows, uint16_t* o,
                                                          float* lse_out) {
  const int lane = threadIdx.x & 31;
  const int64_t x = static_cast<int64_t>(blockIdx.x) * 4 + (threadIdx.x >> 5);
  if (x >= rows) return;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  float lse;
  auto add = [&](int c, float w) {
    const uint2 v = *reinterpret_cast<const uint2*>(o_shards + (static_cast<int64_t>(c) * rows + x) * kHeadDim + lane * 4);
    acc[0] += w * __uint_as_float(v.x << 16);
    acc[1] += w * __uint_as_float(v.x & 0xffff0000u);
    acc[2] += w * __uint_as_float(v.y << 16);
    acc[3] += w * __uint_as_float(v.y & 0xffff0000u);
  };
  if (num_shards <= 32) {
    const float lc = lane < num_shards ? lse_shards[static_cast<int64_t>(lane) * rows + x] : -INFINITY;
    float mx = lc;
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, s));
    const float e = lc != -INFINITY ? __expf(lc - mx) : 0.f;
    float z = e;
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) z += __shfl_xor_sync(0xffffffffu, z, s);
    lse = mx + logf(z);
    const float w_mine = z > 0.f ? e / z : 0.f;
    for (int c = 0; c < num_shards; ++c) {
      const float w = __shfl_sync(0xffffffffu, w_mine, c);
      if (w != 0.f) add(c, w);  // an empty shard (LSE_c = -inf) is not read
    }
  } else {
    float mx = -INFINITY;
    for (int c = 0; c < num_shards; ++c) mx = fmaxf(mx, lse_shards[static_cast<int64_t>(c) * rows + x]);
    float z = 0.f;
    for (int c = 0; c < num_shards; ++c) {
      const float lc = lse_shards[static_cast<int64_t>(c) * rows + x];
      if (lc != -INFINITY) z += __expf(lc - mx);
    }
    lse = mx + logf(z);
    for (int c = 0; c < num_shards; ++c) {
      const float lc = lse_shards[static_cast<int64_t>(c) * rows + x];
      if (lc != -INFINITY) add(c, __expf(lc - lse));
    }
  }
  uint2 packed;
  packed.x = float_to_bf16_bits(acc[0]) | (static_cast<uint32_t>(float_to_bf16_bits(acc[1])) << 16);
  packed.y = float_to_bf16_bits(acc[2]) | (static_cast<uint32_t>(float_to_bf16_bits(acc[3])) << 16);
  *reinterpret_cast<uint2*>(o + x * kHeadDim + lane * 4) = packed;
  if (lane == 0) lse_out[x] = lse;
}

// Step a5 in isolation: copy the rows a request sees, in logical order (Section 4.1.1).
__global__ void gather_kernel(const uint16_t* k_pool, const uint16_t* v_pool, int64_t page_stride,
                              int64_t head_stride, int64_t token_stride, const int32_t* bt,
                              int page_size, int page_shift, int kv_head, int L, uint16_t* out_k,
                              uint16_t* out_v) {
  const int j = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (j >= L) return;
  const int64_t page = bt[j >> page_shift];
  const int64_t off = page * page_stride + static_cast<int64_t>(kv_head) * head_stride +
                      static_cast<int64_t>(j & (page_size - 1)) * token_stride + lane * 4;
  *reinterpret_cast<uint2*>(out_k + static_cast<int64_t>(j) * kHeadDim + lane * 4) =
      *reinterpret_cast<const uint2*>(k_pool + off);
  *reinterpret_cast<uint2*>(out_v + static_cast<int64_t>(j) * kHeadDim + lane * 4) =
      *reinterpret_cast<const uint2*>(v_pool + off);
}

// KV-cache append with fused QKV split (Sections 4.1.1, 5.4): one block per new token; the
// request is found by bisection over the start positions; every thread moves 16 bytes at a time.
__global__ void __launch_bounds__(128) append_kv_kernel(const uint16_t* qkv, int64_t qkv_token_stride,
                                                        uint16_t* k_pool, uint16_t* v_pool, int64_t page_stride,
                                                        int64_t head_stride, int64_t token_stride,
                                                        const int32_t* block_table, int bt_stride,
                                                        const ReqInfo* reqs, int num_reqs, int Hq, int Hkv,
                                                        int page_size, int page_shift) {
  const int t = blockIdx.x;
  int lo = 0, hi = num_reqs - 1;  // last request whose start position is <= t
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (reqs[mid].q_start <= t) lo = mid; else hi = mid - 1;
  }
  const ReqInfo rq = reqs[lo];
  const int j = rq.kv_len + (t - rq.q_start);
  const int64_t page = block_table[static_cast<int64_t>(lo) * bt_stride + (j >> page_shift)];
  const int64_t slot_off = page * page_stride + static_cast<int64_t>(j & (page_size - 1)) * token_stride;
  const uint16_t* src = qkv + static_cast<int64_t>(t) * qkv_token_stride + static_cast<int64_t>(Hq) * kHeadDim;
  const int chunks = 2 * Hkv * (kHeadDim / 8);  // 16-byte chunks of this token's K then V heads
  for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
    const int hv = c / (kHeadDim / 8), d8 = c % (kHeadDim / 8);  // head index within [K heads | V heads]
    const bool is_v = hv >= Hkv;
    const int g = is_v ? hv - Hkv : hv;
    const uint4 val = *reinterpret_cast<const uint4*>(src + static_cast<int64_t>(hv) * kHeadDim + d8 * 8);
    uint16_t* pool = is_v ? v_pool : k_pool;
    *reinterpret_cast<uint4*>(pool + slot_off + static_cast<int64_t>(g) * head_stride + d8 * 8) = val;
  }
}

}  // namespace

cudaError_t launch_append_kv(const uint16_t* qkv, int64_t qkv_token_stride, uint16_t* k_pool, uint16_t* v_pool,
                             int64_t page_stride, int64_t head_stride, int64_t token_stride,
                             const int32_t* block_table, int bt_stride, const ReqInfo* reqs, int num_reqs,
                             int total_q, int Hq, int Hkv, int page_size, int page_shift, cudaStream_t s) {
  if (total_q == 0) return cudaSuccess;
  append_kv_kernel<<<total_q, 128, 0, s>>>(qkv, qkv_token_stride, k_pool, v_pool, page_stride, head_stride,
                                           token_stride, block_table, bt_stride, reqs, num_reqs, Hq, Hkv,
                                           page_size, page_shift);
  return cudaGetLastError();
}

cudaError_t launch_reference(const RunArgs& a, int num_workers, cudaStream_t s) {
  ref_attention_kernel<<<num_workers, 128, 0, s>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_merge_units(const MergeArgs& a, int num_units, int max_rows, int max_parts, cudaStream_t s) {
  if (num_units == 0) return cudaSuccess;
  // one warp per row of the largest unit (four rows per block), at most kMergeBlocksPerUnit blocks
  int by = (max_rows + 3) / 4;
  by = by < 1 ? 1 : (by > kMergeBlocksPerUnit ? kMergeBlocksPerUnit : by);
  if (max_parts > 32)
    merge_units_kernel<true><<<dim3(num_units, by), 128, 0, s>>>(a);
  else
    merge_units_kernel<false><<<dim3(num_units, by), 128, 0, s>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_merge_plain(const float* o_part, const float* lse_part, int num_splits,
                               int64_t rows, uint16_t* o, float* lse, cudaStream_t s) {
  if (rows == 0) return cudaSuccess;
  const unsigned blocks = static_cast<unsigned>((rows + 3) / 4);
  merge_plain_kernel<<<blocks, 128, 0, s>>>(o_part, lse_part, num_splits, rows, o, lse);
  return cudaGetLastError();
}

cudaError_t launch_merge_shards(const uint16_t* o_shards, const float* lse_shards, int num_shards,
                                int64_t rows, uint16_t* o, float* lse, cudaStream_t s) {
  if (rows == 0) return cudaSuccess;
  const unsigned blocks = static_cast<unsigned>((rows + 3) / 4);
  merge_shards_kernel<<<blocks, 128, 0, s>>>(o_shards, lse_shards, num_shards, rows, o, lse);
  return cudaGetLastError();
}

cudaError_t launch_gather(const uint16_t* k_pool, const uint16_t* v_pool, int64_t page_stride,
                          int64_t head_stride, int64_t token_stride, const int32_t* bt,
                          int page_size, int page_shift, int kv_head, int L, uint16_t* out_k,
                          uint16_t* out_v, cudaStream_t s) {
  if (L == 0) return cudaSuccess;
  gather_kernel<<<(L + 3) / 4, 128, 0, s>>>(k_pool, v_pool, page_stride, head_stride, token_stride,
                                            bt, page_size, page_shift, kv_head, L, out_k, out_v);
  return cudaGetLastError();
}

}  // namespace xy
