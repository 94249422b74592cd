// Allocation-free split-KV decode attention.
//
// Some callers cannot allocate device memory at the point where they need attention: code
// running inside a serving loop whose memory pool has already been handed out in full, a
// plugin that is only given a stream and its input/output buffers, or a host program that
// must not touch the allocator while another library owns it.  For them this file offers one
// entry point that never calls cudaMalloc / cudaFree (nor any allocating library routine): its
// split-KV scratch lives in a fixed, file-scope __device__ array that every GPU loading this
// library holds until the process exits.
//
// It is a variant of the reference SIMT attention kernel restricted to decode requests (one
// new token per request): every (request, kv head) unit is cut into chunks of 2048 keys, one
// thread block per (request, kv head, chunk) writes an fp32 partial (O_c, LSE_c) for each q
// head of the group into the static scratch, and a second kernel merges the chunks
// (LSE = ln sum exp LSE_c, O = sum exp(LSE_c - LSE) O_c) into the caller's O and LSE.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <mutex>

#include "xy_attn.h"

namespace {

constexpr int kD = 128;
constexpr int kChunkKeys = 2048;
constexpr int kMaxDevices = 64;

// The scratch: XY_ATTN_STATIC_MAX_ROWS partial rows of 128 fp32 outputs plus one LSE each
// (4 MiB + 32 KiB per GPU).  In host code this name is only a stand-in for the symbol; the
// device address is fetched with cudaGetSymbolAddress below.
static __device__ __align__(256) float g_static_scratch[XY_ATTN_STATIC_MAX_ROWS * (kD + 1)];

std::mutex g_mu;
float* g_scratch_addr[kMaxDevices] = {nullptr};

__device__ __forceinline__ float bf16_to_f32(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// grid = (chunks, kv heads, requests); block = 32 * G threads: one warp per q head of the group.
// Every block writes all of its partial rows, also when its chunk lies beyond the request's
// keys (LSE_c = -inf, O_c = 0), so nothing in the scratch has to be cleared between calls.
__global__ void decode_static_partial_kernel(const uint16_t* q, int64_t q_token_stride, const uint16_t* k_pool,
                                             const uint16_t* v_pool, int64_t page_stride, int64_t head_stride,
                                             int64_t token_stride, const int32_t* block_table, int bt_stride,
                                             const int32_t* kv_len, int G, int Hq, int page_size, int page_shift,
                                             float sm_scale, int num_chunks, int max_kv_len, float* scratch_o,
                                             float* scratch_lse) {
  const int chunk = blockIdx.x, g = blockIdx.y, r = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int head = g * G + warp;
  // cached tokens plus the new one, whose K/V is already in the cache; never beyond what the
  // caller's max_kv_len sized the chunks (and its block-table rows) for: a request that breaks
  // the bound gets NaN from the merge kernel instead of a silently truncated context
  const int L = min(kv_len[r], max_kv_len) + 1;
  const int j_lo = chunk * kChunkKeys, j_hi = min(L, j_lo + kChunkKeys);
  const uint16_t* qp = q + static_cast<int64_t>(r) * q_token_stride + head * kD + lane * 4;
  float qv[4];
#pragma unroll
  for (int d = 0; d < 4; ++d) qv[d] = bf16_to_f32(qp[d]);
  const int32_t* bt = block_table + static_cast<int64_t>(r) * bt_stride;
  float m = -INFINITY, l = 0.f, o[4] = {0.f, 0.f, 0.f, 0.f};
  for (int j = j_lo; j < j_hi; ++j) {
    const int64_t page = bt[j >> page_shift];
    const int64_t off = page * page_stride + static_cast<int64_t>(g) * head_stride +
                        static_cast<int64_t>(j & (page_size - 1)) * token_stride + lane * 4;
    float dot = 0.f;
#pragma unroll
    for (int d = 0; d < 4; ++d) dot += qv[d] * bf16_to_f32(k_pool[off + d]);
    const float s = warp_sum(dot) * sm_scale;
    const float m_new = fmaxf(m, s);
    const float alpha = __expf(m - m_new), p = __expf(s - m_new);
    l = l * alpha + p;
#pragma unroll
    for (int d = 0; d < 4; ++d) o[d] = o[d] * alpha + p * bf16_to_f32(v_pool[off + d]);
    m = m_new;
  }
  const int64_t row = (static_cast<int64_t>(r) * Hq + head) * num_chunks + chunk;
  const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll
  for (int d = 0; d < 4; ++d) scratch_o[row * kD + lane * 4 + d] = o[d] * inv;
  if (lane == 0) scratch_lse[row] = l > 0.f ? m + logf(l) : -INFINITY;
}

// One warp per (request, q head): merge its chunks.
__global__ void decode_static_merge_kernel(const float* scratch_o, const float* scratch_lse, int num_chunks,
                                           int64_t rows, int Hq, const int32_t* kv_len, int max_kv_len, uint16_t* o,
                                           int64_t o_token_stride, float* lse) {
  const int64_t x = static_cast<int64_t>(blockIdx.x) * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (x >= rows) return;
  if (kv_len[x / Hq] > max_kv_len) {  // the caller's bound does not hold for this request: say so loudly
    uint16_t* bad = o + (x / Hq) * o_token_stride + (x % Hq) * kD + lane * 4;
#pragma unroll
    for (int d = 0; d < 4; ++d) bad[d] = 0x7FC0u;  // bf16 NaN
    if (lane == 0) lse[x] = __int_as_float(0x7FC00000);
    return;
  }
  const float* lc = scratch_lse + x * num_chunks;
  float mx = -INFINITY;
  for (int c = 0; c < num_chunks; ++c) mx = fmaxf(mx, lc[c]);
  float z = 0.f;
  for (int c = 0; c < num_chunks; ++c)
    if (lc[c] != -INFINITY) z += __expf(lc[c] - mx);
  const float total = mx + logf(z);
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int c = 0; c < num_chunks; ++c) {
    if (lc[c] == -INFINITY) continue;
    const float w = __expf(lc[c] - total);
    const float* v = scratch_o + (x * num_chunks + c) * kD + lane * 4;
#pragma unroll
    for (int d = 0; d < 4; ++d) acc[d] += w * v[d];
  }
  const int64_t r = x / Hq, head = x % Hq;
  uint16_t* dst = o + r * o_token_stride + head * kD + lane * 4;
#pragma unroll
  for (int d = 0; d < 4; ++d) dst[d] = __bfloat16_as_ushort(__float2bfloat16_rn(acc[d]));
  if (lane == 0) lse[x] = total;
}

}  // namespace

extern "C" int xy_attn_decode_static(const void* q, int64_t q_token_stride, const void* k_pool, const void* v_pool,
                                     int64_t page_stride, int64_t head_stride, int64_t token_stride,
                                     const int32_t* block_table, int32_t block_table_stride, const int32_t* kv_len,
                                     int32_t num_reqs, int32_t max_kv_len, int32_t num_q_heads, int32_t num_kv_heads,
                                     int32_t page_size, float sm_scale, void* o, int64_t o_token_stride, float* lse,
                                     void* stream) {
  if (num_reqs < 0 || max_kv_len < 0 || num_q_heads < 1 || num_kv_heads < 1 || num_q_heads % num_kv_heads != 0)
    return XY_ERR_INVALID_ARG;
  const int G = num_q_heads / num_kv_heads;
  if (G > 32 || page_size < 1 || (page_size & (page_size - 1)) != 0) return XY_ERR_UNSUPPORTED;
  if (num_reqs == 0) return XY_OK;
  if (!q || !k_pool || !v_pool || !block_table || !kv_len || !o || !lse) return XY_ERR_INVALID_ARG;
  if (q_token_stride < static_cast<int64_t>(num_q_heads) * kD || o_token_stride < static_cast<int64_t>(num_q_heads) * kD ||
      token_stride < kD || block_table_stride < 1 || !(sm_scale > 0.f))
    return XY_ERR_INVALID_ARG;
  const int64_t num_chunks64 = (static_cast<int64_t>(max_kv_len) + 1 + kChunkKeys - 1) / kChunkKeys;
  const int64_t rows = static_cast<int64_t>(num_reqs) * num_q_heads;
  const int num_chunks = static_cast<int>(num_chunks64 > XY_ATTN_STATIC_MAX_ROWS ? XY_ATTN_STATIC_MAX_ROWS + 1 : num_chunks64);
  if (rows * num_chunks > XY_ATTN_STATIC_MAX_ROWS) {
    fprintf(stderr,
            "xy_attn_decode_static: num_reqs * num_q_heads * ceil((max_kv_len + 1) / %d) = %lld exceeds the static "
            "scratch of %d partial rows\n",
            kChunkKeys, static_cast<long long>(rows * num_chunks64), XY_ATTN_STATIC_MAX_ROWS);
    return XY_ERR_CAPACITY;
  }
  // Set-up, once per device, with that device current: the device address of the scratch.
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return XY_ERR_CUDA;
  float* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_scratch_addr[dev] == nullptr) {
      float* p = nullptr;
      if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch) != cudaSuccess || p == nullptr)
        return XY_ERR_CUDA;
      g_scratch_addr[dev] = p;
    }
    scratch = g_scratch_addr[dev];
  }
  float* scratch_o = scratch;
  float* scratch_lse = scratch + static_cast<int64_t>(XY_ATTN_STATIC_MAX_ROWS) * kD;
  int page_shift = 0;
  while ((1 << page_shift) < page_size) ++page_shift;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  dim3 grid(num_chunks, num_kv_heads, num_reqs);
  decode_static_partial_kernel<<<grid, 32 * G, 0, s>>>(
      static_cast<const uint16_t*>(q), q_token_stride, static_cast<const uint16_t*>(k_pool),
      static_cast<const uint16_t*>(v_pool), page_stride, head_stride, token_stride, block_table, block_table_stride,
      kv_len, G, num_q_heads, page_size, page_shift, sm_scale, num_chunks, max_kv_len, scratch_o, scratch_lse);
  if (cudaGetLastError() != cudaSuccess) return XY_ERR_CUDA;
  decode_static_merge_kernel<<<static_cast<unsigned>((rows + 3) / 4), 128, 0, s>>>(
      scratch_o, scratch_lse, num_chunks, rows, num_q_heads, kv_len, max_kv_len, static_cast<uint16_t*>(o),
      o_token_stride, lse);
  if (cudaGetLastError() != cudaSuccess) return XY_ERR_CUDA;
  return XY_OK;
}
