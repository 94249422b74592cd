// Host planner: Token-Table -> decomposition -> Task-Table (Sections 3.2.1 and 3.3.1).
//
// a1  Token-Table: per request {kind, start position = prefix sum of q_len, tokenNum,
//     historical kvLen}; verify requests get their ancestor-or-self bit matrix.
// a2  Decomposition: request -> q tiles -> one tile unit per kv head.  Rows of a unit are
//     GQA-packed (token-major, the G q heads of the kv head innermost).  The unit's visible
//     keys are cut into runs of 128-key tiles (KV splits) when a unit is too heavy for one
//     worker.  Purely logical: no data moves.
// a3  Reordering: cost per task, sort from largest to smallest, deal to the workers in the
//     symmetric round-robin 0..C-1, C-1..0, ...; each worker's list is stored contiguously.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <numeric>

#include <climits>

#include "xy_internal.h"

namespace xy {
namespace {

// Per-SM time model in microseconds (free design constants; parity does not depend on them).
// Measured on B200 from the per-worker time each kind of task takes: a dense task advances one
// key tile per 2.2 - 2.6 us whether one or both of its 128-row sub-tiles are in use (the softmax
// -> MMA chain of a sub-tile sets the pace and the two sub-tiles overlap each other); a streaming
// task one key tile per ~1.0 us while HBM is not saturated (1.4 us when every SM streams); a
// task boundary costs ~3 us (Q load, pipeline refill, epilogue).
constexpr float kDenseVisitUs = 2.30f;
constexpr float kStreamVisitUs = 1.00f;
constexpr float kPairVisitUs = 1.35f;
constexpr float kTaskFixedUs = 3.0f;
constexpr int kMinChunkTiles = 4;
// A task may cost at most this fraction of the mean per-worker load before its KV range is
// split (measured on the five benchmark batches: finer splits lose more to per-task overhead
// and partial traffic than they gain in balance).
constexpr float kTaskCapFraction = 0.77f;
// Dense tasks are split a little finer (cap x 0.65): their per-task overhead is small next to a
// key-tile visit, and finer dense tasks even out the tail of the dynamically dealt queue.
constexpr float kDenseCapFactor = 0.65f;


struct Unit {
  int32_t req, kv_head, tok0, ntok, kind;
  int32_t nkt;       // visible 128-key tiles: the unit's tasks cover tiles kt0 .. nkt-1
  int32_t kt0;       // first tile (> 0: the suffix of a member of a shared-prefix group)
  int32_t group;     // -1, or the shared-prefix group this unit belongs to (then always partial)
  float visit_cost;  // per kv tile
  float paper_load;  // rows x visible keys
};

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

}  // namespace

int build_plan(const xy_attn_config& cfg, int num_workers, int64_t partial_row_capacity,
               const xy_attn_request* reqs, int32_t num_reqs, const int32_t* tree_parents,
               int32_t num_parents, PlanResult* out, std::string* err, PlanCache* cache,
               const xy_attn_prefix_group* groups, int32_t num_groups, bool pair) {
  *out = PlanResult();
  char buf[256];
  auto fail = [&](int code, const char* msg) {
    *err = msg;
    return code;
  };
  if (num_reqs < 0 || (num_reqs > 0 && reqs == nullptr)) return fail(XY_ERR_INVALID_ARG, "reqs is null");
  if (static_cast<int64_t>(num_reqs) + std::max(num_groups, 0) > cfg.max_requests)
    return fail(XY_ERR_CAPACITY, "num_reqs (+ groups) exceeds max_requests");
  if (num_parents < 0) return fail(XY_ERR_INVALID_ARG, "num_parents < 0");
  const int G = cfg.num_q_heads / cfg.num_kv_heads;
  const int B = cfg.page_size;

  // ---- a1: Token-Table ------------------------------------------------------------------
  out->reqs.resize(num_reqs);
  out->q_start.assign(num_reqs + 1, 0);
  int64_t total_q = 0;
  int64_t pairs = 0, kv_tokens = 0;
  for (int r = 0; r < num_reqs; ++r) {
    const xy_attn_request& q = reqs[r];
    if (q.q_len < 1) {
      snprintf(buf, sizeof buf, "request %d: q_len must be >= 1", r);
      return fail(XY_ERR_INVALID_ARG, buf);
    }
    if (q.kv_len < 0) {
      snprintf(buf, sizeof buf, "request %d: kv_len must be >= 0", r);
      return fail(XY_ERR_INVALID_ARG, buf);
    }
    if (q.mask_kind != XY_MASK_CAUSAL && q.mask_kind != XY_MASK_TREE) {
      snprintf(buf, sizeof buf, "request %d: unknown mask_kind", r);
      return fail(XY_ERR_INVALID_ARG, buf);
    }
    const int64_t L = static_cast<int64_t>(q.q_len) + q.kv_len;
    if (L > static_cast<int64_t>(cfg.max_pages_per_req) * B) {
      snprintf(buf, sizeof buf, "request %d: kv_len+q_len exceeds max_pages_per_req pages", r);
      return fail(XY_ERR_CAPACITY, buf);
    }
    total_q += q.q_len;
    if (total_q > cfg.max_q_tokens) return fail(XY_ERR_CAPACITY, "total q tokens exceed max_q_tokens");
    ReqInfo& ri = out->reqs[r];
    ri.q_start = static_cast<int32_t>(total_q - q.q_len);
    ri.q_len = q.q_len;
    ri.kv_len = q.kv_len;
    ri.mask_kind = q.mask_kind;
    ri.tree_off = 0;
    ri.tree_words = 0;
    ri.bt_row = r;
    ri.pad1 = 0;
    out->q_start[r + 1] = static_cast<int32_t>(total_q);
    kv_tokens += L;
    const int64_t n = q.q_len, h = q.kv_len;
    if (q.mask_kind == XY_MASK_TREE) {
      if (q.q_len > cfg.max_tree_nodes) {
        snprintf(buf, sizeof buf, "request %d: tree has more than max_tree_nodes nodes", r);
        return fail(XY_ERR_CAPACITY, buf);
      }
      if (tree_parents == nullptr || q.parent_off < 0 ||
          static_cast<int64_t>(q.parent_off) + q.q_len > num_parents) {
        snprintf(buf, sizeof buf, "request %d: parent_off/q_len outside tree_parents", r);
        return fail(XY_ERR_BAD_TREE, buf);
      }
      const int32_t* par = tree_parents + q.parent_off;
      const int words = ceil_div(q.q_len, 64);
      ri.tree_off = static_cast<int32_t>(out->tree_mask.size());
      ri.tree_words = words;
      out->tree_mask.resize(out->tree_mask.size() + static_cast<size_t>(words) * q.q_len, 0ull);
      uint64_t* base = out->tree_mask.data() + ri.tree_off;
      pairs += n * h;
      for (int i = 0; i < q.q_len; ++i) {
        if (par[i] < -1 || par[i] >= i) {
          snprintf(buf, sizeof buf, "request %d: parent[%d] = %d not in {-1} U [0, %d]", r, i,
                   par[i], i - 1);
          out->tree_mask.clear();
          return fail(XY_ERR_BAD_TREE, buf);
        }
        uint64_t* row = base + static_cast<size_t>(i) * words;
        if (par[i] >= 0) {  // ancestors of the parent are already complete (topological order)
          const uint64_t* prow = base + static_cast<size_t>(par[i]) * words;
          for (int w = 0; w < words; ++w) row[w] = prow[w];
        }
        row[i / 64] |= 1ull << (i % 64);
        int depth = 0;
        for (int w = 0; w < words; ++w) depth += __builtin_popcountll(row[w]);
        pairs += depth;
      }
    } else {
      pairs += n * h + n * (n + 1) / 2;
    }
  }
  out->total_q = total_q;

  // ---- shared-prefix groups: validation, and one virtual request per group ----------------
  // A group's members are consecutive decode requests whose first prefix_tokens keys are the same
  // pages.  Their queries form a virtual request (q rows of the members, kvLen = prefix_tokens,
  // block-table row of the first member) whose tiles cover the shared keys once; every member
  // keeps a task for its own keys behind the prefix; the merge kernel combines the two.
  if (num_groups < 0 || (num_groups > 0 && groups == nullptr)) return fail(XY_ERR_INVALID_ARG, "groups is null");
  if (num_groups > 0 && cfg.plan_mode == XY_PLAN_PAPER)
    return fail(XY_ERR_UNSUPPORTED, "shared-prefix groups need the balanced plan mode");
  std::vector<int32_t> group_of(num_reqs, -1);
  for (int gi = 0; gi < num_groups; ++gi) {
    const xy_attn_prefix_group& gr = groups[gi];
    if (gr.num_reqs < 1 || gr.first_req < 0 || static_cast<int64_t>(gr.first_req) + gr.num_reqs > num_reqs ||
        gr.prefix_tokens < kKeyTile || gr.prefix_tokens % kKeyTile != 0) {
      snprintf(buf, sizeof buf, "group %d: bad request range or prefix_tokens not a positive multiple of 128", gi);
      return fail(XY_ERR_INVALID_ARG, buf);
    }
    for (int r = gr.first_req; r < gr.first_req + gr.num_reqs; ++r) {
      if (group_of[r] >= 0 || reqs[r].q_len != 1 || reqs[r].mask_kind != XY_MASK_CAUSAL ||
          reqs[r].kv_len < gr.prefix_tokens) {
        snprintf(buf, sizeof buf, "group %d: request %d is not a decode request with kv_len >= prefix_tokens, or is in two groups", gi, r);
        return fail(XY_ERR_INVALID_ARG, buf);
      }
      group_of[r] = gi;
    }
    ReqInfo v;
    v.q_start = out->reqs[gr.first_req].q_start;
    v.q_len = gr.num_reqs;
    v.kv_len = gr.prefix_tokens;
    v.mask_kind = XY_MASK_CAUSAL;
    v.tree_off = v.tree_words = 0;
    v.bt_row = gr.first_req;
    v.pad1 = 0;
    out->reqs.push_back(v);
  }

  // ---- a2: decomposition ----------------------------------------------------------------
  const bool paper = cfg.plan_mode == XY_PLAN_PAPER;
  const int sub_tok = std::max(1, 128 / G);  // tokens of one 128-row sub-tile
  const int subtiles = pair ? 4 : dense_subtiles(cfg);  // a CTA pair holds two sub-tiles of 256 rows
  const int dense_tok = paper ? (cfg.tile_tokens > 0 ? cfg.tile_tokens : sub_tok) : subtiles * sub_tok;
  if (paper && cfg.kernel != XY_KERNEL_REFERENCE && dense_tok * G > 128 * subtiles)
    return fail(XY_ERR_UNSUPPORTED, "paper-mode tile_tokens x (Hq/Hkv) exceeds the rows one task may hold");
  std::vector<Unit> units;
  for (int r = 0; r < num_reqs + num_groups; ++r) {
    const bool is_virtual = r >= num_reqs;
    const int n = is_virtual ? groups[r - num_reqs].num_reqs : reqs[r].q_len;
    const int h = is_virtual ? groups[r - num_reqs].prefix_tokens : reqs[r].kv_len;
    const int gidx = is_virtual ? r - num_reqs : group_of[r];
    // q tiles of this request (same for every kv head)
    std::vector<std::pair<int, int>> tiles;  // tok0, ntok
    if (paper) {
      for (int t0 = 0; t0 < n; t0 += dense_tok) tiles.push_back({t0, std::min(dense_tok, n - t0)});
    } else if (n * G <= kStreamRowsMax) {
      tiles.push_back({0, n});
    } else {
      for (int t0 = 0; t0 < n; t0 += dense_tok) tiles.push_back({t0, std::min(dense_tok, n - t0)});
    }
    for (int g = 0; g < cfg.num_kv_heads; ++g) {
      for (auto& t : tiles) {
        Unit u;
        u.req = r;
        u.kv_head = g;
        u.tok0 = t.first;
        u.ntok = t.second;
        const int rows = u.ntok * G;
        u.kind = rows <= kStreamRowsMax ? 1 : 0;
        // a virtual request's tiles stop at the end of the shared prefix (its rows see all of it)
        const int visible = is_virtual ? h : h + u.tok0 + u.ntok;
        u.nkt = ceil_div(visible, kKeyTile);
        u.group = gidx;
        u.kt0 = (!is_virtual && gidx >= 0) ? groups[gidx].prefix_tokens / kKeyTile : 0;
        if (u.kind == 1) {
          u.visit_cost = kStreamVisitUs;
        } else {
          // a pair advances one key tile of a 512-row unit per kPairVisitUs, which keeps two workers busy
          u.visit_cost = pair ? 2.f * kPairVisitUs : kDenseVisitUs * static_cast<float>(std::max(1, ceil_div(rows, 256)));
        }
        u.paper_load = static_cast<float>(rows) * static_cast<float>(visible);
        units.push_back(u);
      }
    }
  }

  // ---- Task-Table cache: everything below depends on the requests only through the units
  // (request, kv head, q tile, kind, visible key tiles), so an equal decomposition has an equal
  // Task-Table.  The useful-flop and byte counts depend on the exact kvLen and are always fresh.
  out->shape.reserve(units.size() * 8 + 4);
  out->shape.push_back(num_workers);
  out->shape.push_back(static_cast<int32_t>(std::min<int64_t>(partial_row_capacity, INT32_MAX)));
  out->shape.push_back(cfg.plan_mode * 4 + cfg.kernel);
  out->shape.push_back(cfg.max_splits);
  out->shape.push_back(cfg.kv_dtype);
  out->shape.push_back(pair ? 1 : 0);
  for (const Unit& u : units) {
    out->shape.push_back(u.req);
    out->shape.push_back(u.kv_head);
    out->shape.push_back(u.tok0);
    out->shape.push_back(u.ntok);
    out->shape.push_back(u.kind);
    out->shape.push_back(paper ? static_cast<int32_t>(reqs[u.req].kv_len) : u.nkt);
    out->shape.push_back(u.kt0);
    out->shape.push_back(u.group);
  }
  {
    uint64_t hsh = 1469598103934665603ull;  // FNV-1a over the 32-bit words
    for (int32_t v : out->shape) hsh = (hsh ^ static_cast<uint32_t>(v)) * 1099511628211ull;
    out->shape_hash = hsh;
  }
  const int64_t flops_now = 4ll * kHeadDim * cfg.num_q_heads * pairs;
  const int64_t kv_bytes_now = 2ll * kv_tokens * cfg.num_kv_heads * kHeadDim * (cfg.kv_dtype == XY_KV_FP8_E4M3 ? 1 : 2);
  if (cache != nullptr) {
    ++cache->clock;
    for (PlanCache::Entry& e : cache->entries) {
      if (e.hash != out->shape_hash || e.shape != out->shape) continue;
      e.last_use = cache->clock;
      ++cache->hits;
      out->tasks = e.tasks;
      out->task_cost = e.task_cost;
      out->worker_off = e.worker_off;
      out->queue = e.queue;
      out->queue_dense = e.queue_dense;
      out->merges = e.merges;
      out->task_unit = e.task_unit;
      out->num_launch_merges = e.num_launch_merges;
      out->partial_rows = e.partial_rows;
      out->info = e.info;
      out->info.useful_flops = flops_now;
      out->info.kv_bytes = kv_bytes_now;
      out->from_cache = true;
      return XY_OK;
    }
    ++cache->misses;
  }

  // KV splits: cap the cost of one task at a fraction of the mean per-worker load.
  // Default bound on the splits of one unit: 32, or, when the batch has only a few streaming
  // units (a single long-context decode), enough for one task per worker.
  int max_splits = cfg.max_splits;
  if (max_splits <= 0) {
    int n_stream = 0;
    for (const Unit& u : units) n_stream += u.kind == 1 ? 1 : 0;
    max_splits = 32;
    if (n_stream > 0) max_splits = std::max(32, std::min(128, ceil_div(num_workers, n_stream)));
  }
  double total_cost = 0.0, total_kind[2] = {0.0, 0.0};
  for (const Unit& u : units) {
    const double c = kTaskFixedUs + u.visit_cost * (u.nkt - u.kt0);
    total_cost += c;
    total_kind[u.kind == 1 ? 1 : 0] += c;
  }
  float cap = static_cast<float>(total_cost / std::max(1, num_workers) * kTaskCapFraction);
  // pair plans run the two kinds one after the other: each kind is capped against its own mean load
  float cap_kind[2] = {static_cast<float>(total_kind[0] / std::max(1, num_workers) * kTaskCapFraction),
                       static_cast<float>(total_kind[1] / std::max(1, num_workers) * kTaskCapFraction)};
  const float dense_factor = kDenseCapFactor;
  std::vector<int> chunk_tiles(units.size(), 0);
  for (int attempt = 0; attempt < 64; ++attempt) {
    int64_t prow = 0;
    for (size_t k = 0; k < units.size(); ++k) {
      const Unit& u = units[k];
      int nsplit = 1;
      if (!paper) {
        const int nt = u.nkt - u.kt0;
        // (a pair task occupies two workers: its duration is half its cost)
        const float cost = pair && u.kind == 0 ? 0.5f * u.visit_cost * nt : u.visit_cost * nt;
        const float cap_u = pair ? (u.kind == 1 ? cap_kind[1] : cap_kind[0] * dense_factor)
                                 : (u.kind == 1 ? cap : cap * dense_factor);
        nsplit = static_cast<int>(std::ceil(cost / std::max(cap_u, 1e-3f)));
        nsplit = std::min(nsplit, max_splits);
        nsplit = std::min(nsplit, std::max(1, nt / kMinChunkTiles));
        nsplit = std::max(nsplit, 1);
      }
      const int nt = std::max(u.nkt - u.kt0, 1);
      int chunk = ceil_div(nt, nsplit);
      nsplit = ceil_div(nt, chunk);
      chunk_tiles[k] = chunk;
      if (nsplit > 1 || u.group >= 0) prow += static_cast<int64_t>(nsplit) * u.ntok * G;
    }
    if (prow <= partial_row_capacity) break;
    cap *= 1.5f;  // fewer splits until the partials fit the workspace
    cap_kind[0] *= 1.5f;
    cap_kind[1] *= 1.5f;
    if (attempt == 63) return fail(XY_ERR_CAPACITY, "split-KV workspace too small");
  }

  struct Pending {
    xy_attn_task t;
    float cost;
  };
  std::vector<Pending> pend;
  int64_t prow = 0;
  std::vector<int32_t> unit_part(units.size(), -1), unit_nsplit(units.size(), 1);
  std::vector<int32_t> pend_merge;  // per pending task: index in out->merges of its (plain) unit, or -1
  for (size_t k = 0; k < units.size(); ++k) {
    const Unit& u = units[k];
    const int chunk = chunk_tiles[k];
    const int nsplit = ceil_div(std::max(u.nkt - u.kt0, 1), chunk);
    const int rows = u.ntok * G;
    const bool partial = nsplit > 1 || u.group >= 0;  // group units always leave partials
    unit_nsplit[k] = nsplit;
    if (partial) unit_part[k] = static_cast<int32_t>(prow);
    int32_t merge_idx = -1;
    if (nsplit > 1 && u.group < 0) {
      xy_attn_merge_unit mu{u.req, u.kv_head, u.tok0, u.ntok, static_cast<int32_t>(prow), nsplit, 0, 0, 0, 0};
      merge_idx = static_cast<int32_t>(out->merges.size());
      out->merges.push_back(mu);
    }
    for (int c = 0; c < nsplit; ++c) {
      pend_merge.push_back(merge_idx);
      Pending p;
      p.t.req = u.req;
      p.t.kv_head = u.kv_head;
      p.t.tok0 = u.tok0;
      p.t.ntok = u.ntok;
      p.t.kt_lo = u.kt0 + c * chunk;
      p.t.kt_hi = std::min(u.nkt, u.kt0 + (c + 1) * chunk);
      p.t.part = partial ? static_cast<int32_t>(prow + static_cast<int64_t>(c) * rows) : -1;
      p.t.kind = u.kind;
      p.cost = paper ? u.paper_load : kTaskFixedUs + u.visit_cost * (p.t.kt_hi - p.t.kt_lo);
      pend.push_back(p);
    }
    if (partial) prow += static_cast<int64_t>(nsplit) * rows;
  }
  // Merge units of the members of shared-prefix groups: the member's own partials (its keys
  // behind the prefix) plus its rows of the group tile's partials (the shared keys).
  for (size_t k = 0; k < units.size(); ++k) {
    const Unit& u = units[k];
    if (u.group < 0 || u.req >= num_reqs) continue;  // members only
    const int m = u.req - groups[u.group].first_req;   // index of the member = its token in the group
    for (size_t v = 0; v < units.size(); ++v) {
      const Unit& w = units[v];
      if (w.req != num_reqs + u.group || w.kv_head != u.kv_head || m < w.tok0 || m >= w.tok0 + w.ntok) continue;
      xy_attn_merge_unit mu{u.req, u.kv_head, 0, 1, unit_part[k], unit_nsplit[k],
                            unit_part[v] + (m - w.tok0) * G, unit_nsplit[v], w.ntok * G, 0};
      out->merges.push_back(mu);
      break;
    }
  }
  out->partial_rows = prow;
  // Streaming units (at most 16 rows: decode, tiny verify) are merged inside the attention kernel
  // by whichever of their tasks finishes last; dense units (up to 256 rows x splits: a merge that
  // is better spread over all workers) and the two-family units of shared-prefix groups go to the
  // merge kernel.  `merges` is reordered: the merge kernel's units first.
  std::vector<int32_t> merge_new(out->merges.size(), -1);
  {
    const bool in_kernel_ok = cfg.kernel != XY_KERNEL_REFERENCE && !paper;
    std::vector<xy_attn_merge_unit> launch, inside;
    std::vector<int32_t> launch_old, inside_old;
    for (size_t m = 0; m < out->merges.size(); ++m) {
      const xy_attn_merge_unit& mu = out->merges[m];
      const bool in_kernel = in_kernel_ok && mu.nsplit1 == 0 && mu.ntok * G <= kStreamRowsMax;
      (in_kernel ? inside : launch).push_back(mu);
      (in_kernel ? inside_old : launch_old).push_back(static_cast<int32_t>(m));
    }
    out->num_launch_merges = static_cast<int32_t>(launch.size());
    for (size_t k = 0; k < launch_old.size(); ++k) merge_new[launch_old[k]] = -1;  // their tasks carry no unit
    for (size_t k = 0; k < inside_old.size(); ++k) merge_new[inside_old[k]] = static_cast<int32_t>(launch.size() + k);
    out->merges = launch;
    out->merges.insert(out->merges.end(), inside.begin(), inside.end());
  }

  // ---- a3: reordering -> Task-Table ------------------------------------------------------
  std::vector<int> order(pend.size());
  std::iota(order.begin(), order.end(), 0);
  std::stable_sort(order.begin(), order.end(),
                   [&](int a, int b) { return pend[a].cost > pend[b].cost; });
  const int C = std::max(1, num_workers);
  std::vector<std::vector<int>> lists(C);
  for (size_t pos = 0; pos < order.size(); ++pos) {
    const size_t lap = pos / C, idx = pos % C;
    const size_t w = (lap % 2 == 0) ? idx : C - 1 - idx;
    lists[w].push_back(order[pos]);
  }
  out->worker_off.assign(C + 1, 0);
  std::vector<int32_t> where(pend.size(), 0);  // position of each pending task in the table
  out->tasks.reserve(pend.size());
  out->task_cost.reserve(pend.size());
  float lmin = 0.f, lmax = 0.f, lsum = 0.f, tmax = 0.f;
  int ndense = 0;
  for (int w = 0; w < C; ++w) {
    float load = 0.f;
    for (int id : lists[w]) {
      where[id] = static_cast<int32_t>(out->tasks.size());
      out->task_unit.push_back(pend_merge[id] >= 0 ? merge_new[pend_merge[id]] : -1);
      out->tasks.push_back(pend[id].t);
      out->task_cost.push_back(pend[id].cost);
      load += pend[id].cost;
      tmax = std::max(tmax, pend[id].cost);
      ndense += pend[id].t.kind == 0;
    }
    out->worker_off[w + 1] = static_cast<int32_t>(out->tasks.size());
    lmin = (w == 0) ? load : std::min(lmin, load);
    lmax = std::max(lmax, load);
    lsum += load;
  }

  // The queue for workers that take tasks as they become free.  Paper mode: the sorted list.
  // Balanced mode: the dense and the streaming tasks, each in descending order of cost, merged
  // so that at every point of the queue the two kinds have handed out the same fraction of
  // their total cost.  Dense tasks are bound by the SM (tensor pipe + softmax), streaming tasks
  // by HBM; a queue that hands out all of one kind first makes every SM stream at once (HBM
  // saturates) and then leaves HBM idle, while the mixed order keeps both busy throughout.
  // Within the dense kind, sibling q tiles of one (request, kv head) are kept together (below).
  out->queue.resize(order.size());
  if (paper) {
    for (size_t pos = 0; pos < order.size(); ++pos) out->queue[pos] = where[order[pos]];
  } else {
    std::vector<int> by_kind[2];
    double total[2] = {0.0, 0.0}, given[2] = {0.0, 0.0};
    for (int id : order) {
      const int kd = pend[id].t.kind == 1 ? 1 : 0;
      by_kind[kd].push_back(id);
      total[kd] += pend[id].cost;
    }
    {
      // Dense tasks of one (request, kv head) read the same K/V: all but the last tenth of the
      // dense list is regrouped so that such siblings are handed out together (groups in the
      // order of their most expensive task, tasks by descending cost inside a group) and share
      // the K/V through L2 instead of re-reading it from HBM at different times.  The last tenth
      // stays in plain descending order, which is what balances the end of the run.
      std::vector<int>& d = by_kind[0];
      const size_t head = d.size() - d.size() / 10;
      std::vector<int64_t> group_of(head);
      std::vector<int64_t> first_seen;  // group keys in order of first appearance
      for (size_t i = 0; i < head; ++i) {
        group_of[i] = static_cast<int64_t>(pend[d[i]].t.req) * cfg.num_kv_heads + pend[d[i]].t.kv_head;
      }
      std::vector<size_t> idx(head);
      std::iota(idx.begin(), idx.end(), size_t{0});
      // keyed by every Token-Table entry, the virtual requests of shared-prefix groups included
      std::vector<size_t> first_pos(out->reqs.size() * static_cast<size_t>(cfg.num_kv_heads), SIZE_MAX);
      for (size_t i = 0; i < head; ++i)
        if (first_pos[group_of[i]] == SIZE_MAX) first_pos[group_of[i]] = i;
      std::stable_sort(idx.begin(), idx.end(),
                       [&](size_t x, size_t y) { return first_pos[group_of[x]] < first_pos[group_of[y]]; });
      std::vector<int> regrouped;
      regrouped.reserve(d.size());
      for (size_t i : idx) regrouped.push_back(d[i]);
      for (size_t i = head; i < d.size(); ++i) regrouped.push_back(d[i]);
      d.swap(regrouped);
    }
    size_t next[2] = {0, 0};
    if (pair) out->queue_dense = static_cast<int32_t>(by_kind[0].size());
    for (size_t pos = 0; pos < order.size(); ++pos) {
      int kd;
      if (pair) kd = next[0] < by_kind[0].size() ? 0 : 1;  // two launches: all dense tasks, then all streaming tasks
      else if (next[0] >= by_kind[0].size()) kd = 1;
      else if (next[1] >= by_kind[1].size()) kd = 0;
      else {
        // A task must start while at least its own length of work per worker remains, or it
        // runs past the end of everything else: from that point on the longer head goes first.
        const double remaining = (total[0] + total[1] - given[0] - given[1]) / C;
        const float c0 = pend[by_kind[0][next[0]]].cost, c1 = pend[by_kind[1][next[1]]].cost;
        if (std::max(c0, c1) > remaining) kd = c0 >= c1 ? 0 : 1;
        else kd = (given[0] * total[1] <= given[1] * total[0]) ? 0 : 1;
      }
      const int id = by_kind[kd][next[kd]++];
      given[kd] += pend[id].cost;
      out->queue[pos] = where[id];
    }
  }

  xy_attn_plan_info& info = out->info;
  info.num_tasks = static_cast<int32_t>(out->tasks.size());
  info.num_dense_tasks = ndense;
  info.num_merge_units = static_cast<int32_t>(out->merges.size());
  info.num_inline_merge_units = info.num_merge_units - out->num_launch_merges;
  info.reserved = 0;
  info.num_workers = C;
  info.useful_flops = flops_now;
  info.kv_bytes = kv_bytes_now;
  info.partial_rows = prow;
  info.load_min = lmin;
  info.load_mean = lsum / C;
  info.load_max = lmax;
  info.max_task_cost = tmax;
  if (cache != nullptr && cache->capacity > 0) {
    PlanCache::Entry* slot = nullptr;
    if (cache->entries.size() < cache->capacity) {
      cache->entries.emplace_back();
      slot = &cache->entries.back();
    } else {
      slot = &cache->entries[0];
      for (PlanCache::Entry& e : cache->entries)
        if (e.last_use < slot->last_use) slot = &e;
    }
    slot->shape = out->shape;
    slot->hash = out->shape_hash;
    slot->tasks = out->tasks;
    slot->task_cost = out->task_cost;
    slot->worker_off = out->worker_off;
    slot->queue = out->queue;
    slot->queue_dense = out->queue_dense;
    slot->merges = out->merges;
    slot->task_unit = out->task_unit;
    slot->num_launch_merges = out->num_launch_merges;
    slot->partial_rows = out->partial_rows;
    slot->info = out->info;
    slot->last_use = cache->clock;
  }
  return XY_OK;
}

}  // namespace xy
