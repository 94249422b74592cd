// Token-wise chunk former (Section 3.1): host-side scheduling front that turns the prefill and
// decode / verify queues into the per-step request list xy_attn_plan consumes.
#include <cstdint>
#include <deque>
#include <vector>

#include "xy_sched.h"

namespace {

struct Prompt {
  int64_t id;
  int32_t remaining;  // prompt tokens not scheduled yet
  int32_t kv_len;     // cached prefix + tokens scheduled so far
};

struct DvEntry {
  int64_t id;
  int32_t kind;    // XY_SCHED_DECODE or XY_SCHED_VERIFY
  int32_t kv_len;
  int32_t tokens;  // 1, or the nodes of the tree
  std::vector<int32_t> parents;
};

}  // namespace

struct xy_sched {
  xy_sched_config cfg;
  std::deque<Prompt> prefill;
  std::deque<DvEntry> dv;
  int64_t prefill_tokens = 0, dv_tokens = 0;
};

extern "C" {

int xy_sched_create(const xy_sched_config* cfg, xy_sched** out) {
  if (cfg == nullptr || out == nullptr) return XY_ERR_INVALID_ARG;
  *out = nullptr;
  if (cfg->budget_tokens < 1 || cfg->reserved_dv_tokens < 0 || cfg->reserved_dv_tokens > cfg->budget_tokens ||
      cfg->max_requests < 1)
    return XY_ERR_INVALID_ARG;
  xy_sched* s = new xy_sched();
  s->cfg = *cfg;
  *out = s;
  return XY_OK;
}

int xy_sched_destroy(xy_sched* s) {
  delete s;
  return XY_OK;
}

int xy_sched_add_prefill(xy_sched* s, int64_t id, int32_t prompt_tokens, int32_t cached_tokens) {
  if (s == nullptr || cached_tokens < 0 || cached_tokens >= prompt_tokens) return XY_ERR_INVALID_ARG;
  s->prefill.push_back(Prompt{id, prompt_tokens - cached_tokens, cached_tokens});
  s->prefill_tokens += prompt_tokens - cached_tokens;
  return XY_OK;
}

int xy_sched_add_decode(xy_sched* s, int64_t id, int32_t kv_len) {
  if (s == nullptr || kv_len < 0) return XY_ERR_INVALID_ARG;
  s->dv.push_back(DvEntry{id, XY_SCHED_DECODE, kv_len, 1, {}});
  s->dv_tokens += 1;
  return XY_OK;
}

int xy_sched_add_verify(xy_sched* s, int64_t id, int32_t kv_len, const int32_t* parents, int32_t n) {
  if (s == nullptr || parents == nullptr || kv_len < 0 || n < 1 || n > s->cfg.budget_tokens)
    return XY_ERR_INVALID_ARG;
  s->dv.push_back(DvEntry{id, XY_SCHED_VERIFY, kv_len, n, std::vector<int32_t>(parents, parents + n)});
  s->dv_tokens += n;
  return XY_OK;
}

int xy_sched_pending(const xy_sched* s, int64_t* prefill_tokens, int64_t* dv_tokens) {
  if (s == nullptr) return XY_ERR_INVALID_ARG;
  if (prefill_tokens) *prefill_tokens = s->prefill_tokens;
  if (dv_tokens) *dv_tokens = s->dv_tokens;
  return XY_OK;
}

int xy_sched_next_chunk(xy_sched* s, xy_attn_request* reqs, xy_sched_entry* entries, int32_t cap_reqs,
                        int32_t* tree_parents, int32_t cap_parents, int32_t* num_parents) {
  if (s == nullptr || reqs == nullptr || entries == nullptr || num_parents == nullptr ||
      (tree_parents == nullptr && cap_parents > 0))
    return XY_ERR_INVALID_ARG;
  const int budget = s->cfg.budget_tokens, reserved = s->cfg.reserved_dv_tokens, cap = s->cfg.max_requests;
  if (cap_reqs < cap || cap_parents < budget) return XY_ERR_CAPACITY;
  *num_parents = 0;
  int used = 0;
  // (1) decode / verify entries into the reserved slots: they stay in the FIFO for now and are
  // emitted after the prefill parts.
  size_t n_dv = 0;
  while (n_dv < s->dv.size() && static_cast<int>(n_dv) < cap) {
    const int tokens = s->dv[n_dv].tokens;
    if (used + tokens <= reserved || (used == 0 && tokens <= budget)) {
      ++n_dv;
      used += tokens;
      if (used >= reserved) break;
    } else {
      break;
    }
  }
  // (2) prompts into the space left
  int n_out = 0;
  while (!s->prefill.empty() && used < budget && n_out + static_cast<int>(n_dv) < cap) {
    Prompt& head = s->prefill.front();
    const int take = head.remaining < budget - used ? head.remaining : budget - used;
    reqs[n_out] = xy_attn_request{take, head.kv_len, XY_MASK_CAUSAL, -1};
    entries[n_out] = xy_sched_entry{head.id, XY_SCHED_PREFILL, take == head.remaining ? 1 : 0};
    ++n_out;
    head.remaining -= take;
    head.kv_len += take;
    used += take;
    s->prefill_tokens -= take;
    if (head.remaining == 0) s->prefill.pop_front();
  }
  // (3) leftover space to further decode / verify entries
  if (s->prefill.empty()) {
    while (n_dv < s->dv.size() && n_out + static_cast<int>(n_dv) < cap) {
      const int tokens = s->dv[n_dv].tokens;
      if (used + tokens > budget) break;
      ++n_dv;
      used += tokens;
    }
  }
  for (size_t k = 0; k < n_dv; ++k) {
    const DvEntry& e = s->dv.front();
    const bool tree = e.kind == XY_SCHED_VERIFY;
    reqs[n_out] = xy_attn_request{e.tokens, e.kv_len, tree ? XY_MASK_TREE : XY_MASK_CAUSAL, tree ? *num_parents : -1};
    entries[n_out] = xy_sched_entry{e.id, e.kind, 1};
    if (tree) {
      for (int i = 0; i < e.tokens; ++i) tree_parents[*num_parents + i] = e.parents[i];
      *num_parents += e.tokens;
    }
    s->dv_tokens -= e.tokens;
    ++n_out;
    s->dv.pop_front();
  }
  return n_out;
}

}  // extern "C"
