// C-ABI layer: context, plan, run, merge, introspection.  Argument checking and
// marshalling only; every step of the path runs in the kernels.
#include <cuda_runtime.h>

#include <algorithm>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "xy_internal.h"
#include "xy_kernels.h"

using namespace xy;

struct xy_attn_ctx {
  xy_attn_config cfg{};
  int num_workers = 0;
  bool host_only = false;
  int page_shift = 0;
  bool planned = false;
  PlanResult plan;
  PlanCache cache;                  // Task-Tables of recent plans
  std::vector<int32_t> dev_shape;   // decomposition whose Task-Table is in the device tables
  bool dev_shape_valid = false;
  // capacities of the device tables
  int64_t cap_tasks = 0, cap_merges = 0, cap_tree_words = 0, cap_partial_rows = 0;
  ReqInfo* d_reqs = nullptr;
  xy_attn_task* d_tasks = nullptr;
  int32_t* d_worker_off = nullptr;
  int32_t* d_queue = nullptr;
  int32_t* d_task_unit = nullptr;
  uint64_t* d_tree = nullptr;
  xy_attn_merge_unit* d_merges = nullptr;
  float* d_o_part = nullptr;
  float* d_lse_part = nullptr;
  int32_t* d_status_base = nullptr;  // allocation; d_status = d_status_base + kStatusLead
  int32_t* d_status = nullptr;
  unsigned long long* d_trace = nullptr;
  unsigned long long* d_worker_times = nullptr;
  int last_launches = 0;
  MetaLaunchCache launch_cache;     // tensor maps of the last pools seen, kernel attributes set once
  int32_t dbg_skip_fill = -1;       // -1: none
  bool pair = false;                // dense tasks run on CTA pairs (two launches per run: dense pairs, then streaming)
  bool debug_validate = false;      // XY_ATTN_DEBUG=1 at create: block tables are range-checked before launch
  std::vector<int32_t> dbg_bt;      // host copy of the block table for that check
  bool timing = false;
  std::vector<cudaEvent_t> events;  // three per timed run: before attention, after it, after merge
  int timed_runs = 0;
  std::string err = "";
};

namespace {

int set_err(xy_attn_ctx* c, int code, const std::string& msg) {
  if (c) c->err = msg;
  return code;
}

int cuda_fail(xy_attn_ctx* c, cudaError_t e, const char* what) {
  return set_err(c, XY_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

#define XY_CUDA(ctx, call)                                   \
  do {                                                       \
    cudaError_t e__ = (call);                                \
    if (e__ != cudaSuccess) return cuda_fail(ctx, e__, #call); \
  } while (0)

constexpr int kMaxTimedRuns = 4096;

bool pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }

void free_device(xy_attn_ctx* c) {
  if (c->host_only) return;
  for (cudaEvent_t ev : c->events) cudaEventDestroy(ev);
  c->events.clear();
  cudaFree(c->d_reqs);
  cudaFree(c->d_tasks);
  cudaFree(c->d_worker_off);
  cudaFree(c->d_queue);
  cudaFree(c->d_task_unit);
  cudaFree(c->d_tree);
  cudaFree(c->d_merges);
  cudaFree(c->d_o_part);
  cudaFree(c->d_lse_part);
  cudaFree(c->d_status_base);
  cudaFree(c->d_trace);
  cudaFree(c->d_worker_times);
}

}  // namespace

extern "C" {

int xy_attn_create(const xy_attn_config* cfg, xy_attn_ctx** out) {
  if (cfg == nullptr || out == nullptr) return XY_ERR_INVALID_ARG;
  *out = nullptr;
  if (cfg->head_dim != kHeadDim) return XY_ERR_UNSUPPORTED;
  if (!pow2(cfg->page_size) || cfg->page_size < 8 || cfg->page_size > 128) return XY_ERR_UNSUPPORTED;
  if (cfg->num_q_heads < 1 || cfg->num_kv_heads < 1 || cfg->num_q_heads % cfg->num_kv_heads != 0)
    return XY_ERR_INVALID_ARG;
  if (cfg->num_q_heads / cfg->num_kv_heads > 128) return XY_ERR_UNSUPPORTED;
  if (cfg->max_requests < 1 || cfg->max_q_tokens < 1 || cfg->max_pages_per_req < 1 ||
      cfg->max_tree_nodes < 0 || cfg->num_workers < 0 || cfg->max_splits < 0 ||
      cfg->workspace_bytes < 0 || cfg->tile_tokens < 0)
    return XY_ERR_INVALID_ARG;
  if (cfg->kernel < XY_KERNEL_AUTO || cfg->kernel > XY_KERNEL_PAIR) return XY_ERR_INVALID_ARG;
  if (cfg->kernel == XY_KERNEL_PAIR && (cfg->kv_dtype != XY_KV_BF16 || cfg->plan_mode != XY_PLAN_BALANCED))
    return XY_ERR_INVALID_ARG;
  if (cfg->plan_mode != XY_PLAN_BALANCED && cfg->plan_mode != XY_PLAN_PAPER) return XY_ERR_INVALID_ARG;
  if (cfg->kv_dtype != XY_KV_BF16 && cfg->kv_dtype != XY_KV_FP8_E4M3) return XY_ERR_INVALID_ARG;
  if (cfg->kv_dtype == XY_KV_FP8_E4M3 && cfg->page_size < 16) return XY_ERR_UNSUPPORTED;

  xy_attn_ctx* c = new (std::nothrow) xy_attn_ctx();
  if (c == nullptr) return XY_ERR_INVALID_ARG;
  c->cfg = *cfg;
  c->host_only = cfg->device < 0;
  while ((1 << c->page_shift) < cfg->page_size) ++c->page_shift;
  c->num_workers = cfg->num_workers;
  if (!c->host_only) {
    cudaError_t e = cudaSetDevice(cfg->device);
    if (e != cudaSuccess) {
      delete c;
      return XY_ERR_CUDA;
    }
    if (c->num_workers == 0) {
      int sms = 0;
      e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cfg->device);
      if (e != cudaSuccess || sms <= 0) {
        delete c;
        return XY_ERR_CUDA;
      }
      c->num_workers = sms;
    }
  } else if (c->num_workers == 0) {
    c->num_workers = 148;
  }

  c->pair = cfg->kernel == XY_KERNEL_PAIR;
  if (c->pair && (c->num_workers < 2 || c->num_workers % 2 != 0)) {
    delete c;
    return XY_ERR_INVALID_ARG;
  }
  const int G = cfg->num_q_heads / cfg->num_kv_heads;
  const int sub_tok = 128 / G > 0 ? 128 / G : 1;
  const int tile_tok = cfg->plan_mode == XY_PLAN_PAPER
                           ? (cfg->tile_tokens > 0 ? cfg->tile_tokens : sub_tok)
                           : dense_subtiles(*cfg) * sub_tok;
  const int64_t units_max = static_cast<int64_t>(cfg->num_kv_heads) *
                            (cfg->max_requests + cfg->max_q_tokens / tile_tok + 1);
  c->cap_tasks = 2 * units_max + 4ll * c->num_workers + 16;
  c->cap_merges = units_max;
  c->cap_tree_words =
      static_cast<int64_t>(cfg->max_q_tokens) * ((cfg->max_tree_nodes + 63) / 64) + 1;
  const int64_t ws = cfg->workspace_bytes > 0 ? cfg->workspace_bytes : (256ll << 20);
  c->cap_partial_rows = ws / ((kHeadDim + 1) * 4);

  if (!c->host_only) {
    cudaError_t e = cudaSuccess;
    auto alloc = [&](void** p, size_t bytes) {
      if (e == cudaSuccess) e = cudaMalloc(p, bytes < 256 ? 256 : bytes);
    };
    alloc(reinterpret_cast<void**>(&c->d_reqs), sizeof(ReqInfo) * cfg->max_requests);
    alloc(reinterpret_cast<void**>(&c->d_tasks), sizeof(xy_attn_task) * c->cap_tasks);
    alloc(reinterpret_cast<void**>(&c->d_worker_off), sizeof(int32_t) * (c->num_workers + 1));
    alloc(reinterpret_cast<void**>(&c->d_queue), sizeof(int32_t) * c->cap_tasks);
    alloc(reinterpret_cast<void**>(&c->d_task_unit), sizeof(int32_t) * c->cap_tasks);
    alloc(reinterpret_cast<void**>(&c->d_tree), sizeof(uint64_t) * c->cap_tree_words);
    alloc(reinterpret_cast<void**>(&c->d_merges), sizeof(xy_attn_merge_unit) * c->cap_merges);
    alloc(reinterpret_cast<void**>(&c->d_o_part), sizeof(float) * kHeadDim * c->cap_partial_rows);
    alloc(reinterpret_cast<void**>(&c->d_lse_part), sizeof(float) * c->cap_partial_rows);
    // status words, then one completion counter per merge unit
    const size_t status_bytes = sizeof(int32_t) * (kStatusLead + kStatusUnitCounts + c->cap_merges);
    alloc(reinterpret_cast<void**>(&c->d_status_base), status_bytes);
    c->d_status = c->d_status_base + kStatusLead;
    alloc(reinterpret_cast<void**>(&c->d_worker_times), sizeof(unsigned long long) * 4 * c->num_workers);
    if (e == cudaSuccess) e = cudaMemset(c->d_status_base, 0, status_bytes);
    const int32_t default_limit = 1 << 22;
    if (e == cudaSuccess)
      e = cudaMemcpy(c->d_status + kStatusWaitLimit, &default_limit, sizeof default_limit, cudaMemcpyHostToDevice);
    const char* dbg = getenv("XY_ATTN_DEBUG");
    c->debug_validate = dbg != nullptr && dbg[0] == '1';
    const char* tr = getenv("XY_ATTN_TRACE");
    if (tr != nullptr && tr[0] == '1') {
      alloc(reinterpret_cast<void**>(&c->d_trace), sizeof(unsigned long long) * kTraceRoles * kTraceLen);
      if (e == cudaSuccess) e = cudaMemset(c->d_trace, 0, sizeof(unsigned long long) * kTraceRoles * kTraceLen);
    }
    if (e != cudaSuccess) {
      free_device(c);
      delete c;
      return XY_ERR_CUDA;
    }
  }
  *out = c;
  return XY_OK;
}

int xy_attn_destroy(xy_attn_ctx* ctx) {
  if (ctx == nullptr) return XY_ERR_INVALID_ARG;
  if (!ctx->host_only) {
    cudaSetDevice(ctx->cfg.device);
    cudaDeviceSynchronize();
    free_device(ctx);
  }
  delete ctx;
  return XY_OK;
}

int xy_attn_plan(xy_attn_ctx* ctx, const xy_attn_request* reqs, int32_t num_reqs,
                 const int32_t* tree_parents, int32_t num_parents, void* stream,
                 xy_attn_plan_info* info) {
  return xy_attn_plan_shared(ctx, reqs, num_reqs, tree_parents, num_parents, nullptr, 0, stream, info);
}

int xy_attn_plan_shared(xy_attn_ctx* ctx, const xy_attn_request* reqs, int32_t num_reqs,
                        const int32_t* tree_parents, int32_t num_parents,
                        const xy_attn_prefix_group* groups, int32_t num_groups, void* stream,
                        xy_attn_plan_info* info) {
  if (ctx == nullptr) return XY_ERR_INVALID_ARG;
  ctx->planned = false;
  std::string err;
  int rc = build_plan(ctx->cfg, ctx->num_workers, ctx->cap_partial_rows, reqs, num_reqs,
                      tree_parents, num_parents, &ctx->plan, &err, ctx->cache.capacity > 0 ? &ctx->cache : nullptr,
                      groups, num_groups, ctx->pair && num_groups == 0);
  if (rc != XY_OK) {
    ctx->plan = PlanResult();
    return set_err(ctx, rc, err);
  }
  PlanResult& p = ctx->plan;
  if (static_cast<int64_t>(p.tasks.size()) > ctx->cap_tasks ||
      static_cast<int64_t>(p.merges.size()) > ctx->cap_merges ||
      static_cast<int64_t>(p.tree_mask.size()) > ctx->cap_tree_words) {
    ctx->plan = PlanResult();
    return set_err(ctx, XY_ERR_CAPACITY, "plan exceeds the table capacities fixed at create");
  }
  if (!ctx->host_only) {
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    XY_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    // Pageable sources: the runtime stages them before returning, so the vectors may change.
    if (!p.reqs.empty())
      XY_CUDA(ctx, cudaMemcpyAsync(ctx->d_reqs, p.reqs.data(), sizeof(ReqInfo) * p.reqs.size(),
                                   cudaMemcpyHostToDevice, s));
    if (!p.tree_mask.empty())
      XY_CUDA(ctx, cudaMemcpyAsync(ctx->d_tree, p.tree_mask.data(),
                                   sizeof(uint64_t) * p.tree_mask.size(), cudaMemcpyHostToDevice, s));
    // The Task-Table part stays on the device while the decomposition does not change (all of
    // these copies are ordered on `stream`; a caller that plans on several streams must order them).
    const bool same_tables = ctx->dev_shape_valid && ctx->dev_shape == p.shape;
    ctx->dev_shape_valid = false;
    if (!same_tables) {
      if (!p.tasks.empty())
        XY_CUDA(ctx, cudaMemcpyAsync(ctx->d_tasks, p.tasks.data(),
                                     sizeof(xy_attn_task) * p.tasks.size(), cudaMemcpyHostToDevice, s));
      if (!p.queue.empty())
        XY_CUDA(ctx, cudaMemcpyAsync(ctx->d_queue, p.queue.data(), sizeof(int32_t) * p.queue.size(),
                                     cudaMemcpyHostToDevice, s));
      if (!p.task_unit.empty())
        XY_CUDA(ctx, cudaMemcpyAsync(ctx->d_task_unit, p.task_unit.data(), sizeof(int32_t) * p.task_unit.size(),
                                     cudaMemcpyHostToDevice, s));
      XY_CUDA(ctx, cudaMemcpyAsync(ctx->d_worker_off, p.worker_off.data(),
                                   sizeof(int32_t) * p.worker_off.size(), cudaMemcpyHostToDevice, s));
      if (!p.merges.empty())
        XY_CUDA(ctx, cudaMemcpyAsync(ctx->d_merges, p.merges.data(),
                                     sizeof(xy_attn_merge_unit) * p.merges.size(),
                                     cudaMemcpyHostToDevice, s));
      ctx->dev_shape = p.shape;
    }
    ctx->dev_shape_valid = true;
  }
  if (info) *info = p.info;
  ctx->planned = true;
  ctx->err = "";
  return XY_OK;
}

int xy_attn_debug_check_block_table(xy_attn_ctx* ctx, const int32_t* block_table, int32_t block_table_stride,
                                    int64_t num_pages) {
  if (ctx == nullptr) return XY_ERR_INVALID_ARG;
  if (!ctx->planned) return set_err(ctx, XY_ERR_NOT_PLANNED, "block-table check before xy_attn_plan");
  if (block_table == nullptr || block_table_stride < 1 || num_pages < 1)
    return set_err(ctx, XY_ERR_INVALID_ARG, "null block table, bad stride or num_pages");
  char buf[200];
  const int B = ctx->cfg.page_size;
  for (size_t r = 0; r < ctx->plan.reqs.size(); ++r) {
    const ReqInfo& rq = ctx->plan.reqs[r];
    const int64_t need = (static_cast<int64_t>(rq.kv_len) + rq.q_len + B - 1) / B;
    if (need > block_table_stride) {
      snprintf(buf, sizeof buf, "request %zu needs %lld block-table entries, the row has %d", r,
               static_cast<long long>(need), block_table_stride);
      return set_err(ctx, XY_ERR_INVALID_ARG, buf);
    }
    const int32_t* row = block_table + static_cast<int64_t>(rq.bt_row) * block_table_stride;
    for (int64_t p = 0; p < need; ++p) {
      if (row[p] < 0 || row[p] >= num_pages) {
        snprintf(buf, sizeof buf, "block table of request %zu, entry %lld: page %d outside [0, %lld)", r,
                 static_cast<long long>(p), row[p], static_cast<long long>(num_pages));
        return set_err(ctx, XY_ERR_INVALID_ARG, buf);
      }
    }
  }
  return XY_OK;
}

}  // extern "C"

namespace {

// The body of xy_attn_run and xy_attn_run_fp8kv (k_scale / v_scale null: bf16 pools).
int run_impl(xy_attn_ctx* ctx, const void* q, int64_t q_token_stride, const void* k_pool,
             const void* v_pool, const float* k_scale, const float* v_scale, int64_t num_pages, int64_t page_stride,
             int64_t head_stride, int64_t token_stride, const int32_t* block_table, int32_t block_table_stride,
             const uint64_t* tree_mask, float sm_scale, void* o, int64_t o_token_stride,
             float* lse, void* stream) {
  if (ctx == nullptr) return XY_ERR_INVALID_ARG;
  ctx->last_launches = 0;
  if (ctx->host_only) return set_err(ctx, XY_ERR_UNSUPPORTED, "host-only context cannot run");
  if (!ctx->planned) return set_err(ctx, XY_ERR_NOT_PLANNED, "xy_attn_run before xy_attn_plan");
  const bool fp8 = k_scale != nullptr;
  if (fp8 != (ctx->cfg.kv_dtype == XY_KV_FP8_E4M3))
    return set_err(ctx, XY_ERR_UNSUPPORTED, "the context's kv_dtype does not match this run call");
  const PlanResult& p = ctx->plan;
  if (p.tasks.empty()) return XY_OK;
  const xy_attn_config& cfg = ctx->cfg;
  if (!q || !k_pool || !v_pool || !block_table || !o || !lse)
    return set_err(ctx, XY_ERR_INVALID_ARG, "null device pointer");
  auto misaligned = [](const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) != 0; };
  if (misaligned(q) || misaligned(k_pool) || misaligned(v_pool) || misaligned(o))
    return set_err(ctx, XY_ERR_INVALID_ARG, "q, k_pool, v_pool and o must be 16-byte aligned");
  if (q_token_stride < static_cast<int64_t>(cfg.num_q_heads) * kHeadDim || q_token_stride % 8 != 0 ||
      o_token_stride < static_cast<int64_t>(cfg.num_q_heads) * kHeadDim || o_token_stride % 8 != 0)
    return set_err(ctx, XY_ERR_INVALID_ARG, "token stride of q / o too small or not a multiple of 8");
  const int64_t sa = fp8 ? 16 : 8;  // strides must keep every row 16-byte aligned
  if (token_stride < kHeadDim || token_stride % sa != 0 || head_stride % sa != 0 || head_stride < 1 ||
      page_stride % sa != 0 || page_stride < 1 || num_pages < 1)
    return set_err(ctx, XY_ERR_INVALID_ARG, "bad K/V pool strides or num_pages");
  if (fp8 && v_scale == nullptr) return set_err(ctx, XY_ERR_INVALID_ARG, "null scale pointer");
  if (block_table_stride < 1) return set_err(ctx, XY_ERR_INVALID_ARG, "bad block_table_stride");
  if (!(sm_scale > 0.f) || !(sm_scale < 1e30f))
    return set_err(ctx, XY_ERR_INVALID_ARG, "sm_scale must be positive and finite");

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  XY_CUDA(ctx, cudaSetDevice(cfg.device));
  if (ctx->debug_validate) {
    // Validation build of the call (XY_ATTN_DEBUG=1 at create): the block table is brought to the
    // host (this synchronises the stream and allocates host memory - a debugging aid, not the
    // serving path) and every entry a planned request uses is range-checked before anything runs.
    int32_t max_row = 0;
    for (const ReqInfo& rq : p.reqs) max_row = std::max(max_row, rq.bt_row);
    ctx->dbg_bt.resize(static_cast<size_t>(max_row + 1) * block_table_stride);
    XY_CUDA(ctx, cudaStreamSynchronize(s));
    XY_CUDA(ctx, cudaMemcpy(ctx->dbg_bt.data(), block_table, ctx->dbg_bt.size() * sizeof(int32_t),
                            cudaMemcpyDeviceToHost));
    const int rc = xy_attn_debug_check_block_table(ctx, ctx->dbg_bt.data(), block_table_stride, num_pages);
    if (rc != XY_OK) return rc;
  }
  RunArgs a{};
  a.q = static_cast<const uint16_t*>(q);
  a.q_token_stride = q_token_stride;
  a.k_pool = static_cast<const uint16_t*>(k_pool);
  a.v_pool = static_cast<const uint16_t*>(v_pool);
  a.page_stride = page_stride;
  a.head_stride = head_stride;
  a.token_stride = token_stride;
  a.block_table = block_table;
  a.bt_stride = block_table_stride;
  a.tree_mask = tree_mask ? tree_mask : ctx->d_tree;
  a.sm_scale = sm_scale;
  a.o = static_cast<uint16_t*>(o);
  a.o_token_stride = o_token_stride;
  a.lse = lse;
  a.reqs = ctx->d_reqs;
  a.tasks = ctx->d_tasks;
  a.worker_off = ctx->d_worker_off;
  a.o_part = ctx->d_o_part;
  a.lse_part = ctx->d_lse_part;
  a.status = ctx->d_status;
  const bool in_kernel_merges = p.num_launch_merges < static_cast<int32_t>(p.merges.size());
  a.trace = ctx->d_trace;
  a.worker_times = ctx->d_worker_times;
  a.num_q_heads = cfg.num_q_heads;
  a.num_kv_heads = cfg.num_kv_heads;
  a.page_size = cfg.page_size;
  a.page_shift = ctx->page_shift;
  a.queue = ctx->d_queue;
  a.queue_head = ctx->d_status + kStatusQueueHead;  // second cache line of the status block
  a.num_tasks = static_cast<int32_t>(p.tasks.size());
  // Balanced plans are dealt dynamically by the meta-kernel; paper-mode plans keep the static
  // Task-Table (each worker walks its own list), as does the reference kernel.
  a.dynamic = (cfg.plan_mode == XY_PLAN_BALANCED && cfg.kernel != XY_KERNEL_REFERENCE) ? 1 : 0;
  a.debug_skip_fill = ctx->dbg_skip_fill;
  a.task_unit = in_kernel_merges ? ctx->d_task_unit : nullptr;
  a.units = ctx->d_merges;
  a.unit_count = ctx->d_status + kStatusUnitCounts;
  a.k_scale = k_scale;
  a.v_scale = v_scale;
  a.kv_fp8 = fp8 ? 1 : 0;
  // Every run starts with a clean status word, queue head and unit counters (one memset): a run
  // after a device-side timeout is an ordinary run.  The sticky record in front of them is kept.
  XY_CUDA(ctx, cudaMemsetAsync(a.status, 0, (kStatusUnitCounts + (in_kernel_merges ? p.merges.size() : 0)) * sizeof(int32_t), s));

  const bool timed = ctx->timing && ctx->timed_runs < kMaxTimedRuns;
  if (timed) {
    while (static_cast<int>(ctx->events.size()) < 3 * (ctx->timed_runs + 1)) {
      cudaEvent_t ev;
      XY_CUDA(ctx, cudaEventCreate(&ev));
      ctx->events.push_back(ev);
    }
    XY_CUDA(ctx, cudaEventRecord(ctx->events[3 * ctx->timed_runs], s));
  }

  if (cfg.kernel == XY_KERNEL_REFERENCE) {
    XY_CUDA(ctx, launch_reference(a, ctx->num_workers, s));
  } else if (p.queue_dense >= 0 && !fp8) {
    // pair plan: the dense tasks on CTA pairs, then the streaming tasks on single CTAs
    RunArgs d = a;
    d.num_tasks = p.queue_dense;
    if (d.num_tasks > 0) {
      XY_CUDA(ctx, launch_pair_dense(d, ctx->num_workers, num_pages, &ctx->launch_cache, s));
      ctx->last_launches += 1;
    }
    RunArgs st = a;
    st.queue = a.queue + p.queue_dense;
    st.num_tasks = a.num_tasks - p.queue_dense;
    st.queue_head = a.queue_head + 1;  // its own head word, cleared by the same memset
    if (st.num_tasks > 0) {
      XY_CUDA(ctx, launch_meta(st, ctx->num_workers, num_pages, false, &ctx->launch_cache, s));
      ctx->last_launches += 1;
    }
    ctx->last_launches -= 1;  // counted once more below
  } else {
    XY_CUDA(ctx, launch_meta(a, ctx->num_workers, num_pages,
                             (cfg.kernel == XY_KERNEL_AUTO || cfg.kernel == XY_KERNEL_PAIR) && p.info.num_dense_tasks > 0,
                             &ctx->launch_cache, s));
  }
  ctx->last_launches += 1;
  if (timed) XY_CUDA(ctx, cudaEventRecord(ctx->events[3 * ctx->timed_runs + 1], s));

  if (p.num_launch_merges > 0) {
    MergeArgs m{};
    m.units = ctx->d_merges;
    m.reqs = ctx->d_reqs;
    m.o_part = ctx->d_o_part;
    m.lse_part = ctx->d_lse_part;
    m.o = a.o;
    m.o_token_stride = o_token_stride;
    m.lse = lse;
    m.num_q_heads = cfg.num_q_heads;
    m.num_kv_heads = cfg.num_kv_heads;
    int max_rows = 1, max_parts = 1;
    for (int32_t k = 0; k < p.num_launch_merges; ++k) {
      const xy_attn_merge_unit& mu = p.merges[k];
      max_rows = std::max(max_rows, mu.ntok * (cfg.num_q_heads / cfg.num_kv_heads));
      max_parts = std::max(max_parts, mu.nsplit + mu.nsplit1);
    }
    XY_CUDA(ctx, launch_merge_units(m, p.num_launch_merges, max_rows, max_parts, s));
    ctx->last_launches += 1;
  }
  if (timed) {
    XY_CUDA(ctx, cudaEventRecord(ctx->events[3 * ctx->timed_runs + 2], s));
    ctx->timed_runs += 1;
  }
  return XY_OK;
}

}  // namespace

extern "C" {

int xy_attn_run(xy_attn_ctx* ctx, const void* q, int64_t q_token_stride, const void* k_pool,
                const void* v_pool, int64_t num_pages, int64_t page_stride, int64_t head_stride,
                int64_t token_stride, const int32_t* block_table, int32_t block_table_stride,
                const uint64_t* tree_mask, float sm_scale, void* o, int64_t o_token_stride,
                float* lse, void* stream) {
  return run_impl(ctx, q, q_token_stride, k_pool, v_pool, nullptr, nullptr, num_pages, page_stride, head_stride,
                  token_stride, block_table, block_table_stride, tree_mask, sm_scale, o, o_token_stride, lse, stream);
}

int xy_attn_run_fp8kv(xy_attn_ctx* ctx, const void* q, int64_t q_token_stride, const void* k_pool,
                      const void* v_pool, const float* k_scale, const float* v_scale, int64_t num_pages,
                      int64_t page_stride, int64_t head_stride, int64_t token_stride,
                      const int32_t* block_table, int32_t block_table_stride, const uint64_t* tree_mask,
                      float sm_scale, void* o, int64_t o_token_stride, float* lse, void* stream) {
  if (ctx == nullptr) return XY_ERR_INVALID_ARG;
  if (k_scale == nullptr || v_scale == nullptr) return set_err(ctx, XY_ERR_INVALID_ARG, "null scale pointer");
  return run_impl(ctx, q, q_token_stride, k_pool, v_pool, k_scale, v_scale, num_pages, page_stride, head_stride,
                  token_stride, block_table, block_table_stride, tree_mask, sm_scale, o, o_token_stride, lse, stream);
}

int xy_attn_set_timing(xy_attn_ctx* ctx, int32_t enable) {
  if (ctx == nullptr) return XY_ERR_INVALID_ARG;
  if (ctx->host_only) return set_err(ctx, XY_ERR_UNSUPPORTED, "host-only context");
  ctx->timing = enable != 0;
  ctx->timed_runs = 0;
  return XY_OK;
}

int xy_attn_get_timing(xy_attn_ctx* ctx, float* attention_ms, float* merge_ms, int32_t* runs) {
  if (ctx == nullptr || !attention_ms || !merge_ms || !runs) return XY_ERR_INVALID_ARG;
  if (ctx->host_only) return set_err(ctx, XY_ERR_UNSUPPORTED, "host-only context");
  float ta = 0.f, tm = 0.f;
  if (ctx->timed_runs > 0) {
    XY_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    XY_CUDA(ctx, cudaEventSynchronize(ctx->events[3 * ctx->timed_runs - 1]));
    for (int i = 0; i < ctx->timed_runs; ++i) {
      float x = 0.f, y = 0.f;
      XY_CUDA(ctx, cudaEventElapsedTime(&x, ctx->events[3 * i], ctx->events[3 * i + 1]));
      XY_CUDA(ctx, cudaEventElapsedTime(&y, ctx->events[3 * i + 1], ctx->events[3 * i + 2]));
      ta += x;
      tm += y;
    }
  }
  *attention_ms = ta;
  *merge_ms = tm;
  *runs = ctx->timed_runs;
  ctx->timed_runs = 0;
  return XY_OK;
}

int xy_attn_append_kv(xy_attn_ctx* ctx, const void* qkv, int64_t qkv_token_stride, void* k_pool, void* v_pool,
                      int64_t num_pages, int64_t page_stride, int64_t head_stride, int64_t token_stride,
                      const int32_t* block_table, int32_t block_table_stride, void* stream) {
  if (ctx == nullptr) return XY_ERR_INVALID_ARG;
  if (ctx->host_only) return set_err(ctx, XY_ERR_UNSUPPORTED, "host-only context cannot run");
  if (ctx->cfg.kv_dtype != XY_KV_BF16) return set_err(ctx, XY_ERR_UNSUPPORTED, "append serves bf16 caches only");
  if (!ctx->planned) return set_err(ctx, XY_ERR_NOT_PLANNED, "xy_attn_append_kv before xy_attn_plan");
  const PlanResult& p = ctx->plan;
  if (p.total_q == 0) return XY_OK;
  const xy_attn_config& cfg = ctx->cfg;
  if (!qkv || !k_pool || !v_pool || !block_table) return set_err(ctx, XY_ERR_INVALID_ARG, "null device pointer");
  auto misaligned = [](const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) != 0; };
  if (misaligned(qkv) || misaligned(k_pool) || misaligned(v_pool))
    return set_err(ctx, XY_ERR_INVALID_ARG, "qkv, k_pool and v_pool must be 16-byte aligned");
  if (qkv_token_stride < static_cast<int64_t>(cfg.num_q_heads + 2 * cfg.num_kv_heads) * kHeadDim ||
      qkv_token_stride % 8 != 0)
    return set_err(ctx, XY_ERR_INVALID_ARG, "qkv token stride too small or not a multiple of 8");
  if (token_stride < kHeadDim || token_stride % 8 != 0 || head_stride % 8 != 0 || head_stride < 1 ||
      page_stride % 8 != 0 || page_stride < 1 || num_pages < 1 || block_table_stride < 1)
    return set_err(ctx, XY_ERR_INVALID_ARG, "bad K/V pool strides, num_pages or block_table_stride");
  XY_CUDA(ctx, cudaSetDevice(cfg.device));
  XY_CUDA(ctx, launch_append_kv(static_cast<const uint16_t*>(qkv), qkv_token_stride, static_cast<uint16_t*>(k_pool),
                                static_cast<uint16_t*>(v_pool), page_stride, head_stride, token_stride, block_table,
                                block_table_stride, ctx->d_reqs, static_cast<int>(p.reqs.size()),
                                static_cast<int>(p.total_q), cfg.num_q_heads, cfg.num_kv_heads, cfg.page_size,
                                ctx->page_shift, static_cast<cudaStream_t>(stream)));
  return XY_OK;
}

int xy_attn_merge(const float* o_part, const float* lse_part, int32_t num_splits, int64_t rows,
                  int32_t head_dim, void* o, float* lse, void* stream) {
  if (head_dim != kHeadDim) return XY_ERR_UNSUPPORTED;
  if (num_splits < 1 || rows < 0) return XY_ERR_INVALID_ARG;
  if (rows == 0) return XY_OK;
  if (!o_part || !lse_part || !o || !lse) return XY_ERR_INVALID_ARG;
  cudaError_t e = launch_merge_plain(o_part, lse_part, num_splits, rows, static_cast<uint16_t*>(o),
                                     lse, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? XY_OK : XY_ERR_CUDA;
}

int xy_attn_find_prefix_groups(const xy_attn_request* reqs, int32_t num_reqs, const int32_t* block_table,
                               int32_t block_table_stride, int32_t page_size, int32_t min_members,
                               int32_t min_prefix_tokens, xy_attn_prefix_group* groups, int32_t capacity,
                               int32_t* num_groups) {
  if (num_groups == nullptr) return XY_ERR_INVALID_ARG;
  *num_groups = 0;
  if (num_reqs < 0 || capacity < 0 || (num_reqs > 0 && (reqs == nullptr || block_table == nullptr)) ||
      (capacity > 0 && groups == nullptr) || page_size < 1 || page_size > kKeyTile ||
      (page_size & (page_size - 1)) != 0 || block_table_stride < 0 || min_members < 2)
    return XY_ERR_INVALID_ARG;
  const int32_t floor_tokens = std::max(min_prefix_tokens, kKeyTile);
  auto is_decode = [&](int32_t r) { return reqs[r].q_len == 1 && reqs[r].mask_kind == XY_MASK_CAUSAL; };
  // tokens of the longest common run of leading page ids of requests a and b, counted in whole
  // 128-token tiles that lie inside both histories
  auto common_tokens = [&](int32_t a, int32_t b, int32_t limit) -> int32_t {
    const int32_t tokens = std::min(std::min(reqs[a].kv_len, reqs[b].kv_len), limit) / kKeyTile * kKeyTile;
    const int32_t pages = std::min(tokens / page_size, block_table_stride);
    const int32_t* ra = block_table + static_cast<int64_t>(a) * block_table_stride;
    const int32_t* rb = block_table + static_cast<int64_t>(b) * block_table_stride;
    int32_t p = 0;
    while (p < pages && ra[p] == rb[p] && ra[p] >= 0) ++p;
    return static_cast<int32_t>(static_cast<int64_t>(p) * page_size / kKeyTile * kKeyTile);
  };
  int32_t r = 0;
  while (r < num_reqs) {
    if (!is_decode(r) || reqs[r].kv_len < floor_tokens) {
      ++r;
      continue;
    }
    int32_t prefix = reqs[r].kv_len / kKeyTile * kKeyTile;
    int32_t end = r + 1;
    while (end < num_reqs && is_decode(end)) {
      const int32_t c = common_tokens(r, end, prefix);
      if (c < floor_tokens) break;
      prefix = c;
      ++end;
    }
    if (end - r >= min_members) {
      if (*num_groups >= capacity) return XY_ERR_CAPACITY;
      groups[*num_groups] = xy_attn_prefix_group{r, end - r, prefix};
      ++*num_groups;
      r = end;
    } else {
      ++r;
    }
  }
  return XY_OK;
}

int xy_attn_merge_shards(const void* o_shards, const float* lse_shards, int32_t num_shards, int64_t rows,
                         int32_t head_dim, void* o, float* lse, void* stream) {
  if (head_dim != kHeadDim) return XY_ERR_UNSUPPORTED;
  if (num_shards < 1 || rows < 0) return XY_ERR_INVALID_ARG;
  if (rows == 0) return XY_OK;
  if (!o_shards || !lse_shards || !o || !lse) return XY_ERR_INVALID_ARG;
  cudaError_t e = launch_merge_shards(static_cast<const uint16_t*>(o_shards), lse_shards, num_shards, rows,
                                      static_cast<uint16_t*>(o), lse, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? XY_OK : XY_ERR_CUDA;
}

int xy_attn_shard_context(int64_t total_tokens, int32_t page_size, int32_t num_shards, int64_t* bounds) {
  if (bounds == nullptr || num_shards < 1 || total_tokens < 1 || page_size < 1) return XY_ERR_INVALID_ARG;
  const int64_t pages = (total_tokens + page_size - 1) / page_size;
  if (pages < num_shards) return XY_ERR_INVALID_ARG;  // every shard must hold at least one token
  // pages dealt as evenly as whole pages allow; the earlier shards take the extra ones so that
  // the last shard, which holds the ragged tail and receives the appends, is never the largest
  const int64_t base = pages / num_shards, extra = pages % num_shards;
  int64_t page = 0;
  for (int32_t k = 0; k < num_shards; ++k) {
    bounds[k] = page * page_size;
    page += base + (k < extra ? 1 : 0);
  }
  bounds[num_shards] = total_tokens;
  return XY_OK;
}

int xy_attn_debug_gather(xy_attn_ctx* ctx, int32_t req, int32_t kv_head, const void* k_pool,
                         const void* v_pool, int64_t page_stride, int64_t head_stride,
                         int64_t token_stride, const int32_t* block_table,
                         int32_t block_table_stride, void* out_k, void* out_v, void* stream) {
  if (ctx == nullptr) return XY_ERR_INVALID_ARG;
  if (ctx->host_only) return set_err(ctx, XY_ERR_UNSUPPORTED, "host-only context cannot run");
  if (ctx->cfg.kv_dtype != XY_KV_BF16) return set_err(ctx, XY_ERR_UNSUPPORTED, "gather serves bf16 caches only");
  if (!ctx->planned) return set_err(ctx, XY_ERR_NOT_PLANNED, "gather before plan");
  if (req < 0 || req >= static_cast<int32_t>(ctx->plan.reqs.size()) || kv_head < 0 ||
      kv_head >= ctx->cfg.num_kv_heads || !k_pool || !v_pool || !block_table || !out_k || !out_v)
    return set_err(ctx, XY_ERR_INVALID_ARG, "bad gather argument");
  const ReqInfo& r = ctx->plan.reqs[req];
  XY_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
  XY_CUDA(ctx, launch_gather(static_cast<const uint16_t*>(k_pool),
                             static_cast<const uint16_t*>(v_pool), page_stride, head_stride,
                             token_stride,
                             block_table + static_cast<int64_t>(req) * block_table_stride,
                             ctx->cfg.page_size, ctx->page_shift, kv_head, r.q_len + r.kv_len,
                             static_cast<uint16_t*>(out_k), static_cast<uint16_t*>(out_v),
                             static_cast<cudaStream_t>(stream)));
  return XY_OK;
}

#define XY_GETTER(name, type, vec)                                              \
  int name(const xy_attn_ctx* ctx, type* out, int32_t cap) {                    \
    if (ctx == nullptr || (out == nullptr && cap > 0)) return XY_ERR_INVALID_ARG; \
    if (!ctx->planned) return XY_ERR_NOT_PLANNED;                               \
    const auto& v = ctx->plan.vec;                                              \
    const size_t n = v.size() < static_cast<size_t>(cap < 0 ? 0 : cap) ? v.size() : (cap < 0 ? 0 : cap); \
    if (n) std::memcpy(out, v.data(), n * sizeof(type));                        \
    return static_cast<int>(v.size());                                          \
  }

XY_GETTER(xy_attn_get_tasks, xy_attn_task, tasks)
XY_GETTER(xy_attn_get_worker_offsets, int32_t, worker_off)
XY_GETTER(xy_attn_get_merge_units, xy_attn_merge_unit, merges)
XY_GETTER(xy_attn_get_tree_mask, uint64_t, tree_mask)
XY_GETTER(xy_attn_get_q_start, int32_t, q_start)
XY_GETTER(xy_attn_get_queue, int32_t, queue)

int xy_attn_plan_cache(xy_attn_ctx* ctx, int32_t capacity, int64_t* hits, int64_t* misses) {
  if (ctx == nullptr || capacity < -1) return XY_ERR_INVALID_ARG;
  if (capacity >= 0) {
    ctx->cache.capacity = static_cast<size_t>(capacity);
    if (ctx->cache.entries.size() > ctx->cache.capacity) ctx->cache.entries.clear();
  }
  if (hits) *hits = static_cast<int64_t>(ctx->cache.hits);
  if (misses) *misses = static_cast<int64_t>(ctx->cache.misses);
  return XY_OK;
}

int xy_attn_worker_times(xy_attn_ctx* ctx, uint64_t* out, int32_t cap) {
  if (ctx == nullptr || (out == nullptr && cap > 0)) return XY_ERR_INVALID_ARG;
  if (ctx->host_only) return set_err(ctx, XY_ERR_UNSUPPORTED, "host-only context");
  const int n = 4 * ctx->num_workers;
  if (cap >= n) {
    XY_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    XY_CUDA(ctx, cudaDeviceSynchronize());
    XY_CUDA(ctx, cudaMemcpy(out, ctx->d_worker_times, sizeof(uint64_t) * n, cudaMemcpyDeviceToHost));
  }
  return n;
}

int xy_attn_debug_trace(xy_attn_ctx* ctx, uint64_t* out, int32_t cap) {
  if (ctx == nullptr || (out == nullptr && cap > 0)) return XY_ERR_INVALID_ARG;
  if (ctx->host_only || ctx->d_trace == nullptr) return 0;
  const int n = kTraceRoles * kTraceLen;
  XY_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
  XY_CUDA(ctx, cudaDeviceSynchronize());
  if (cap >= n) XY_CUDA(ctx, cudaMemcpy(out, ctx->d_trace, sizeof(uint64_t) * n, cudaMemcpyDeviceToHost));
  return n;
}

int xy_attn_debug_inject(xy_attn_ctx* ctx, int32_t wait_limit_polls, int32_t skip_fill) {
  if (ctx == nullptr || wait_limit_polls < 0 || skip_fill < -1) return XY_ERR_INVALID_ARG;
  ctx->dbg_skip_fill = skip_fill;
  if (!ctx->host_only) {
    // the limit lives in the status block, where the kernels' waits look it up on their slow path
    const int32_t limit = wait_limit_polls > 0 ? wait_limit_polls : (1 << 22);
    XY_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    XY_CUDA(ctx, cudaDeviceSynchronize());
    XY_CUDA(ctx, cudaMemcpy(ctx->d_status + kStatusWaitLimit, &limit, sizeof limit, cudaMemcpyHostToDevice));
  }
  return XY_OK;
}

int xy_attn_last_launches(const xy_attn_ctx* ctx) { return ctx ? ctx->last_launches : XY_ERR_INVALID_ARG; }

const char* xy_attn_last_error(const xy_attn_ctx* ctx) { return ctx ? ctx->err.c_str() : "null context"; }

int xy_attn_device_status(xy_attn_ctx* ctx, int32_t* status_out) {
  if (ctx == nullptr || status_out == nullptr) return XY_ERR_INVALID_ARG;
  if (ctx->host_only) return set_err(ctx, XY_ERR_UNSUPPORTED, "host-only context");
  XY_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
  XY_CUDA(ctx, cudaDeviceSynchronize());
  // word 0 is the last run's status (cleared by every run), word kStatusSticky the record of
  // every failure since the last call of this function: report it and clear both.
  int32_t st[kStatusLead + 1];
  XY_CUDA(ctx, cudaMemcpy(st, ctx->d_status_base, sizeof st, cudaMemcpyDeviceToHost));
  const int32_t sticky = st[kStatusLead + kStatusSticky], last = st[kStatusLead];
  const int32_t seen = sticky != 0 ? sticky : last;
  if (seen != 0) {
    XY_CUDA(ctx, cudaMemset(ctx->d_status, 0, sizeof(int32_t)));
    XY_CUDA(ctx, cudaMemset(ctx->d_status + kStatusSticky, 0, sizeof(int32_t)));
  }
  *status_out = seen;
  return XY_OK;
}

}  // extern "C"
