/* Token-wise chunk former: the scheduling step in front of xy_attn_plan (Section 3.1).
 *
 * Section 3.1 forms, every step, one chunk of at most a fixed budget of tokens out of the
 * scheduling queues; the chunk may mix prefill, decode and verify tokens; prefill is
 * prioritised; a prompt longer than the space left is split; some slots are reserved for decode
 * and speculative tokens; a prefill-only chunk is formed only when none of those are waiting;
 * under low load a chunk is smaller than the budget.  The details the paper leaves open are
 * fixed as follows:
 *   - one FIFO of prefill requests and one FIFO shared by decode (1 token) and verify (a whole
 *     tree) entries; entries are never reordered within a queue, and only prompts are split;
 *   - (1) decode / verify entries are taken from the head of their FIFO while they fit into the
 *     reserved slots; the head entry is taken even if it is larger than the reserved slots as
 *     long as those are still empty;
 *   - (2) prompts are taken in order into the rest of the budget, the head prompt contributing
 *     min(remaining, space) tokens; an unfinished prompt stays at the head with its kvLen
 *     advanced;
 *   - (3) if the prefill FIFO ran dry, further decode / verify entries fill the space left;
 *   - a chunk holds at most max_requests entries; prefill parts are listed first.
 * All of it is host code: plain pointers are HOST memory, nothing touches a GPU.  Every call
 * returns XY_OK (0) or a negative XY_ERR_* code of xy_attn.h unless stated otherwise.  A
 * scheduler object is not thread-safe.
 */
#ifndef XY_SCHED_H_
#define XY_SCHED_H_

#include <stdint.h>

#include "xy_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct xy_sched xy_sched;

typedef struct {
  int32_t budget_tokens;      /* tokens per chunk, >= 1 */
  int32_t reserved_dv_tokens; /* slots kept for decode / verify tokens, 0..budget_tokens */
  int32_t max_requests;       /* entries per chunk, >= 1 (xy_attn_config.max_requests of the consumer) */
} xy_sched_config;

enum xy_sched_kind { XY_SCHED_PREFILL = 0, XY_SCHED_DECODE = 1, XY_SCHED_VERIFY = 2 };

/* Who an entry of the chunk is.  `last` = 1 unless the entry is a part of a prompt that is not
 * complete yet (then the rest follows in later chunks). */
typedef struct {
  int64_t id;
  int32_t kind; /* xy_sched_kind */
  int32_t last;
} xy_sched_entry;

int xy_sched_create(const xy_sched_config* cfg, xy_sched** out);
int xy_sched_destroy(xy_sched* s);

/* Queue a prompt of prompt_tokens tokens of which the first cached_tokens are already in the KV
 * cache (0 <= cached_tokens < prompt_tokens): the rest is scheduled, kvLen starting at
 * cached_tokens. */
int xy_sched_add_prefill(xy_sched* s, int64_t id, int32_t prompt_tokens, int32_t cached_tokens);
/* Queue one decode token of a request with kv_len cached tokens. */
int xy_sched_add_decode(xy_sched* s, int64_t id, int32_t kv_len);
/* Queue a token tree of n nodes (1 <= n <= budget_tokens) to verify; parents[i] in {-1} U [0, i-1]
 * is copied (it is validated by xy_attn_plan, not here). */
int xy_sched_add_verify(xy_sched* s, int64_t id, int32_t kv_len, const int32_t* parents, int32_t n);

/* Tokens waiting in the prefill FIFO and in the decode / verify FIFO (either may be null). */
int xy_sched_pending(const xy_sched* s, int64_t* prefill_tokens, int64_t* dv_tokens);

/* Forms the next chunk and removes it from the queues.  Writes one xy_attn_request per entry
 * (ready for xy_attn_plan: q_len, kv_len, mask_kind, parent_off), the matching xy_sched_entry,
 * and the verify entries' parent arrays back to back into tree_parents (*num_parents of them).
 * Returns the number of entries (0: nothing queued) or a negative error.  cap_reqs must be at
 * least max_requests and cap_parents at least budget_tokens, else XY_ERR_CAPACITY is returned and
 * the queues are unchanged. */
int xy_sched_next_chunk(xy_sched* s, xy_attn_request* reqs, xy_sched_entry* entries, int32_t cap_reqs,
                        int32_t* tree_parents, int32_t cap_parents, int32_t* num_parents);

#ifdef __cplusplus
}
#endif
#endif /* XY_SCHED_H_ */
