// Host-only driver for the planner, built with -fsanitize=address by tests/test_plan_asan.py.
// Plans batches that reach every index path of the planner (shared-prefix groups whose virtual
// requests own dense tiles, verify trees, long decode rows that are split, paper mode), so that
// an out-of-range access in the host code aborts the process instead of passing silently.
#include <cstdio>
#include <string>
#include <vector>

#include "xy_internal.h"

using namespace xy;

static int plan(const xy_attn_config& cfg, const std::vector<xy_attn_request>& reqs,
                const std::vector<int32_t>& parents, const std::vector<xy_attn_prefix_group>& groups,
                PlanCache* cache) {
  PlanResult out;
  std::string err;
  const int rc = build_plan(cfg, 148, 1 << 20, reqs.data(), static_cast<int32_t>(reqs.size()),
                            parents.empty() ? nullptr : parents.data(), static_cast<int32_t>(parents.size()), &out,
                            &err, cache, groups.empty() ? nullptr : groups.data(),
                            static_cast<int32_t>(groups.size()));
  if (rc != XY_OK) {
    fprintf(stderr, "plan failed: %d %s\n", rc, err.c_str());
    return 1;
  }
  // the queue must be a permutation of the task table
  std::vector<int> seen(out.tasks.size(), 0);
  for (int32_t q : out.queue) {
    if (q < 0 || q >= static_cast<int32_t>(out.tasks.size()) || seen[q]++) return 2;
  }
  return 0;
}

int main() {
  xy_attn_config cfg{};
  cfg.num_q_heads = 32;
  cfg.num_kv_heads = 8;
  cfg.head_dim = 128;
  cfg.page_size = 128;
  cfg.max_requests = 512;
  cfg.max_q_tokens = 1 << 16;
  cfg.max_pages_per_req = 1 << 14;
  cfg.max_tree_nodes = 64;
  cfg.device = -1;
  PlanCache cache;
  int bad = 0;
  {  // 2 groups of 32 decode requests on an 8192-token prefix: the virtual requests hold dense tiles
    std::vector<xy_attn_request> reqs;
    for (int r = 0; r < 64; ++r) reqs.push_back({1, 8192 + 17 * r, XY_MASK_CAUSAL, -1});
    std::vector<xy_attn_prefix_group> groups = {{0, 32, 8192}, {32, 32, 8192}};
    bad |= plan(cfg, reqs, {}, groups, &cache);
    bad |= plan(cfg, reqs, {}, groups, &cache);  // cache hit
  }
  {  // hybrid: prefill on a prefix, long decode rows (split), a verify tree, a group at the end
    std::vector<xy_attn_request> reqs = {{3000, 5000, XY_MASK_CAUSAL, -1}, {1, 400000, XY_MASK_CAUSAL, -1},
                                         {5, 9000, XY_MASK_TREE, 0}, {1, 0, XY_MASK_CAUSAL, -1}};
    for (int r = 0; r < 40; ++r) reqs.push_back({1, 1024 + r, XY_MASK_CAUSAL, -1});
    std::vector<int32_t> parents = {-1, 0, 0, 1, -1};
    std::vector<xy_attn_prefix_group> groups = {{4, 40, 1024}};
    bad |= plan(cfg, reqs, parents, groups, &cache);
    bad |= plan(cfg, reqs, parents, {}, nullptr);
    xy_attn_config paper = cfg;
    paper.plan_mode = XY_PLAN_PAPER;
    bad |= plan(paper, reqs, parents, {}, nullptr);
  }
  printf(bad ? "FAILED\n" : "OK\n");
  return bad;
}
