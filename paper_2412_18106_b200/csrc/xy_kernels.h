// Kernel launch entry points (host side) and their argument blocks.
#pragma once

#include <cuda_runtime.h>

#include "xy_internal.h"

namespace xy {

struct MergeArgs {
  const xy_attn_merge_unit* units;
  const ReqInfo* reqs;
  const float* o_part;
  const float* lse_part;
  uint16_t* o;
  int64_t o_token_stride;
  float* lse;
  int32_t num_q_heads, num_kv_heads;
};

// What launch_meta keeps between calls: the two TMA tensor maps (128 opaque bytes each) of the
// pools it saw last, keyed by everything they were encoded from, and whether the kernels'
// shared-memory attribute has been set.
struct MetaLaunchCache {
  alignas(64) unsigned char maps[2][128];
  const void* k_pool = nullptr;
  const void* v_pool = nullptr;
  int64_t num_pages = 0, page_stride = 0, head_stride = 0, token_stride = 0;
  int32_t num_kv_heads = 0, page_size = 0;
  bool valid = false, fp8 = false;
  bool attr_set[4] = {false, false, false, false};
  // the CTA-pair kernel's maps (K in boxes of at most 64 tokens)
  alignas(64) unsigned char pair_maps[2][128];
  const void* pk_pool = nullptr;
  const void* pv_pool = nullptr;
  int64_t p_num_pages = 0, p_page_stride = 0, p_head_stride = 0, p_token_stride = 0;
  int32_t p_num_kv_heads = 0, p_page_size = 0;
  bool pair_valid = false;
};

cudaError_t launch_reference(const RunArgs& a, int num_workers, cudaStream_t s);
cudaError_t launch_meta(const RunArgs& a, int num_workers, int64_t num_pages, bool umma, MetaLaunchCache* cache,
                        cudaStream_t s);
cudaError_t launch_pair_dense(const RunArgs& a, int num_workers, int64_t num_pages, MetaLaunchCache* cache, cudaStream_t s);
cudaError_t launch_merge_units(const MergeArgs& a, int num_units, int max_rows, int max_parts, cudaStream_t s);
cudaError_t launch_merge_plain(const float* o_part, const float* lse_part, int num_splits,
                               int64_t rows, uint16_t* o, float* lse, cudaStream_t s);
cudaError_t launch_merge_shards(const uint16_t* o_shards, const float* lse_shards, int num_shards,
                                int64_t rows, uint16_t* o, float* lse, cudaStream_t s);
cudaError_t launch_append_kv(const uint16_t* qkv, int64_t qkv_token_stride, uint16_t* k_pool, uint16_t* v_pool,
                             int64_t page_stride, int64_t head_stride, int64_t token_stride,
                             const int32_t* block_table, int bt_stride, const ReqInfo* reqs, int num_reqs,
                             int total_q, int Hq, int Hkv, int page_size, int page_shift, cudaStream_t s);
cudaError_t launch_gather(const uint16_t* k_pool, const uint16_t* v_pool, int64_t page_stride,
                          int64_t head_stride, int64_t token_stride, const int32_t* bt,
                          int page_size, int page_shift, int kv_head, int L, uint16_t* out_k,
                          uint16_t* out_v, cudaStream_t s);

}  // namespace xy
