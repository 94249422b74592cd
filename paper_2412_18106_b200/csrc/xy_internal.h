// Internal declarations shared by the planner, the API layer and the kernels.
#pragma once

#include <cstdint>
#include <string>
#include <vector>

#include "xy_attn.h"

namespace xy {

constexpr int kHeadDim = 128;
constexpr int kKeyTile = 128;      // keys per KV tile (one MMA N extent)
constexpr int kStreamRowsMax = 16;
// The status block, indexed from the word the kernels receive as `status`:
//   [0]   the current run's status, polled by every bounded wait
//   [16]  the queue head of dynamic dealing (its own cache line)
//   [32 ..] one completion counter per merge unit
// all of which one memset clears when a run starts; and in front of them, untouched by that,
//   [-8]  the sticky record of failures that xy_attn_device_status reports and clears
//   [-7]  the number of polls after which a bounded wait gives up (ptx.cuh reads the same word).
constexpr int kStatusQueueHead = 16;
constexpr int kStatusUnitCounts = 32;
constexpr int kStatusSticky = -8;
constexpr int kStatusWaitLimit = -7;
constexpr int kStatusLead = 8;  // words in front of `status`
constexpr int kTraceRoles = 4;      // sub-tile A, sub-tile B, MMA issuer, producer (worker 0 only)
constexpr int kTraceLen = 2048;    // records per role and run

// Per-request facts the kernels need (device-visible, 32 bytes).
struct ReqInfo {
  int32_t q_start;    // start position: first row of the request in Q / O / LSE
  int32_t q_len;      // tokenNum
  int32_t kv_len;     // historical kvLen
  int32_t mask_kind;  // XY_MASK_*
  int32_t tree_off;   // first 64-bit word of the request's corner mask
  int32_t tree_words; // words per corner-mask row
  int32_t bt_row;     // block-table row the request's pages are looked up in
  int32_t pad1;
};

struct PlanResult {
  std::vector<ReqInfo> reqs;
  std::vector<int32_t> q_start;            // num_reqs + 1
  std::vector<uint64_t> tree_mask;         // all verify requests back to back
  std::vector<xy_attn_task> tasks;         // grouped by worker
  std::vector<float> task_cost;            // parallel to tasks
  std::vector<int32_t> worker_off;         // num_workers + 1
  std::vector<int32_t> queue;              // task indices by descending cost (dynamic dealing)
  int32_t queue_dense = -1;                // pair plans: the first queue_dense entries are the dense tasks (for the
                                           // CTA-pair launch), the rest the streaming tasks; -1: one mixed queue
  std::vector<xy_attn_merge_unit> merges;  // units merged by the merge kernel first, then those merged in the attention kernel
  std::vector<int32_t> task_unit;          // parallel to tasks: index in `merges` of the unit the last finisher merges
                                           // inside the attention kernel, or -1
  int32_t num_launch_merges = 0;           // leading entries of `merges` that the merge kernel handles
  int64_t partial_rows = 0;
  int64_t total_q = 0;
  xy_attn_plan_info info{};
  // Identity of the Task-Table part (tasks, worker_off, queue, merges): the decomposition it was
  // built from.  Two plans with equal `shape` have identical Task-Tables even when the requests'
  // kvLen differ (a decode step moves kvLen by one token but rarely crosses a 128-key tile).
  std::vector<int32_t> shape;
  uint64_t shape_hash = 0;
  bool from_cache = false;
};

// Task-Tables of recent plans, keyed by their decomposition (least recently used goes first).
struct PlanCache {
  struct Entry {
    std::vector<int32_t> shape;
    uint64_t hash = 0;
    std::vector<xy_attn_task> tasks;
    std::vector<float> task_cost;
    std::vector<int32_t> worker_off, queue;
    int32_t queue_dense = -1;
    std::vector<xy_attn_merge_unit> merges;
    std::vector<int32_t> task_unit;
    int32_t num_launch_merges = 0;
    int64_t partial_rows = 0;
    xy_attn_plan_info info{};
    uint64_t last_use = 0;
  };
  std::vector<Entry> entries;
  size_t capacity = 8;
  uint64_t clock = 0, hits = 0, misses = 0;
};

// 128-row sub-tiles one dense task may hold (the tcgen05 path ping-pongs two; the others one).
inline int dense_subtiles(const xy_attn_config& cfg) {
  return (cfg.kernel == XY_KERNEL_AUTO || cfg.kernel == XY_KERNEL_PAIR) && cfg.kv_dtype == XY_KV_BF16 ? 2 : 1;
}

// Host-only planning.  Returns XY_OK or an error code and fills `err`.
// `pair`: plan for the CTA-pair dense kernel: dense units of up to 512 packed rows, the dense and
// the streaming tasks in separate parts of the queue (they run in two launches).
// `cache` (nullable): Task-Tables of earlier plans; a plan whose decomposition equals a cached one
// takes its Task-Table from there and only rebuilds the Token-Table and the tree masks.
// `groups` (nullable): shared-prefix decode groups, see xy_attn_plan_shared.
int build_plan(const xy_attn_config& cfg, int num_workers, int64_t partial_row_capacity,
               const xy_attn_request* reqs, int32_t num_reqs, const int32_t* tree_parents,
               int32_t num_parents, PlanResult* out, std::string* err, PlanCache* cache = nullptr,
               const xy_attn_prefix_group* groups = nullptr, int32_t num_groups = 0, bool pair = false);

// Arguments every attention kernel takes.
struct RunArgs {
  const uint16_t* q;
  int64_t q_token_stride;
  const uint16_t* k_pool;
  const uint16_t* v_pool;
  int64_t page_stride, head_stride, token_stride;
  const int32_t* block_table;
  int32_t bt_stride;
  const uint64_t* tree_mask;
  float sm_scale;
  uint16_t* o;
  int64_t o_token_stride;
  float* lse;
  // context-owned
  const ReqInfo* reqs;
  const xy_attn_task* tasks;
  const int32_t* worker_off;
  float* o_part;
  float* lse_part;
  int32_t* status;                   // the context's status block, see kStatus*
  unsigned long long* worker_times;  // [2 * workers]: globaltimer at entry and exit of each worker
  unsigned long long* trace;  // null unless tracing: kTraceRoles x kTraceLen (tag << 48 | cycle) records
  int32_t num_q_heads, num_kv_heads, page_size, page_shift;
  // dynamic dealing: workers take the next task of `queue` with an atomic counter
  const int32_t* queue;
  int32_t* queue_head;
  int32_t num_tasks, dynamic;
  // split units whose last finishing task merges them inside the kernel (streaming units)
  const int32_t* task_unit;              // per task: unit index or -1 (null: no such unit)
  const xy_attn_merge_unit* units;
  int32_t* unit_count;                   // per unit: tasks finished so far (returns to 0 by itself)
  // fp8 KV cache: k_pool / v_pool hold e4m3 bytes (strides in bytes) and these are the fp32 scales
  // [pages, Hkv] of K and V
  const float* k_scale;
  const float* v_scale;
  int32_t kv_fp8;
  // test hook: the producer of every worker leaves out its debug_skip_fill-th stage fill (-1: none)
  int32_t debug_skip_fill;
};

}  // namespace xy
