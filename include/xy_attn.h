/*
 * xy_attn — hybrid-batch attention meta-kernel for NVIDIA B200 (sm_100a).
 *
 * One launch computes matmul-softmax-matmul for a mixed batch of chunked-prefill
 * requests (optionally on a reused cached prefix), single-token decode requests
 * and speculative-verify requests (a token tree under a tree mask), all reading
 * a paged bf16 KV cache, and writes O (bf16) and LSE (fp32).
 *
 * The calls follow the problem statement of XY-Serve (arXiv 2412.18106):
 *   - Token-Table: one entry per stage {stageID, start position, tokenNum,
 *     historical kvLen, tileSize}                                (Section 3.2.1)
 *   - decomposition into tile units and reordering into a Task-Table that maps
 *     each core to its list of tiles                       (Sections 3.2.1, 3.3.1)
 *   - Meta-Attention: QK -> Softmax -> SV per tile unit over K/V blocks read by
 *     block table, with mask-aware skipping            (Sections 4.1.1, 4.2.1, 4.2.2)
 *   - only the specLen x specLen corner of a verify mask is non-trivial and is
 *     supplied from outside                                        (Section 4.1.2)
 *   - Q is read with a stride from a fused QKV tensor and O is written as
 *     [tokens, heads, headSize]                                     (Section 5.4)
 *
 * Conventions.  Every call returns an int status (XY_OK or a negative XY_ERR_*),
 * never throws and never aborts.  "HOST" / "DEVICE" beside a pointer says where
 * the memory lives.  The caller owns every buffer it passes in; the context owns
 * its task tables, tree masks, split-KV workspace and status word.  No call
 * falls back to the CPU: without a usable CUDA device `xy_attn_run` fails.
 */
#ifndef XY_ATTN_H_
#define XY_ATTN_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct xy_attn_ctx xy_attn_ctx; /* opaque */

enum {
  XY_OK = 0,
  XY_ERR_INVALID_ARG = -1,    /* null pointer, bad size, bad stride, bad head ratio */
  XY_ERR_CAPACITY = -2,       /* batch exceeds a capacity given at create */
  XY_ERR_BAD_TREE = -3,       /* parent[i] not in {-1} U [0, i-1] */
  XY_ERR_NOT_PLANNED = -4,    /* run before a successful plan */
  XY_ERR_CUDA = -5,           /* a CUDA runtime/driver call failed; see xy_attn_last_error */
  XY_ERR_DEVICE_TIMEOUT = -6, /* a bounded wait inside a kernel gave up */
  XY_ERR_UNSUPPORTED = -7     /* head_dim != 128, page size not a power of two in 8..128, ... */
};

enum { XY_MASK_CAUSAL = 0, XY_MASK_TREE = 1 };

/* Which kernels xy_attn_run uses. */
enum {
  XY_KERNEL_AUTO = 0,      /* the product path: tcgen05 dense tiles (prefill, verify; 256 packed rows per
                              task) side by side with streaming tiles (decode) in one launch, tasks
                              dealt from one mixed queue */
  XY_KERNEL_REFERENCE = 1, /* plain SIMT kernel for every tile: slow, kept for bisecting */
  XY_KERNEL_MMA = 2,       /* warp-level mma.sync tiles for every task (dense tasks too) */
  XY_KERNEL_PAIR = 3       /* experimental: dense tiles on CTA pairs (tcgen05 cta_group::2, 512 packed
                              rows per task), then the streaming tiles in a second launch.  Needs a
                              bf16 cache, XY_PLAN_BALANCED and an even worker count (create fails
                              otherwise); batches with shared-prefix groups run as XY_KERNEL_AUTO.
                              Measured 8 - 20 % slower than XY_KERNEL_AUTO on the dense workloads. */
};

/* Task-Table construction (Section 3.3.1). */
enum {
  XY_PLAN_BALANCED = 0, /* cost = a measured time per visited 128-key tile (by task kind) plus a
                           per-task term; long runs are cut into KV splits; the Task-Table is
                           sorted + dealt by symmetric round-robin as in the paper, and the
                           MMA kernels take the same tasks from one queue as workers become
                           free (dense and streaming tasks side by side, sibling q tiles of a
                           request together, long tasks first) */
  XY_PLAN_PAPER = 1     /* the paper's table literally: one task per tile unit, no KV split,
                           load = rows x visible keys, sorted + symmetric round-robin, every
                           worker runs its own list */
};

/* Element type of the paged K/V cache. */
enum {
  XY_KV_BF16 = 0,     /* bf16 pools, xy_attn_run (the paper's cache) */
  XY_KV_FP8_E4M3 = 1  /* e4m3 byte pools with fp32 scales per (page, kv head), xy_attn_run_fp8kv */
};

typedef struct {
  int32_t num_q_heads;       /* Hq */
  int32_t num_kv_heads;      /* Hkv, divides Hq; q head a reads kv head a / (Hq/Hkv) */
  int32_t head_dim;          /* 128 */
  int32_t page_size;         /* B: tokens per KV page, power of two in 8..128 */
  int32_t max_requests;      /* capacity: requests per plan */
  int32_t max_q_tokens;      /* capacity: total new tokens per plan */
  int32_t max_pages_per_req; /* capacity: pages a single request may reference */
  int32_t max_tree_nodes;    /* capacity: nodes of one verify tree */
  int32_t device;            /* CUDA device ordinal; -1 = host-only context (plan works, run fails) */
  int32_t num_workers;       /* 0 = one worker per SM of the device (148 on B200) */
  int32_t kernel;            /* XY_KERNEL_* */
  int32_t plan_mode;         /* XY_PLAN_* */
  int32_t tile_tokens;       /* XY_PLAN_PAPER only: tileSize in tokens (0 = 128 / (Hq/Hkv)) */
  int32_t max_splits;        /* upper bound on KV splits of one tile unit (0 = 32, or up to 128 when so few
                              * streaming units exist that 32 splits each would leave workers idle) */
  int32_t kv_dtype;          /* XY_KV_*: decides which run call the context serves (and the tile plan) */
  int64_t workspace_bytes;   /* split-KV workspace (fp32 partial O and LSE); 0 = 256 MiB */
} xy_attn_config;

/* One Token-Table entry as the caller states it (Section 3.2.1).  The start
 * position is the prefix sum of q_len in request order, computed by plan. */
typedef struct {
  int32_t q_len;      /* tokenNum: new tokens this step, >= 1 */
  int32_t kv_len;     /* historical kvLen: cached tokens BEFORE the new ones, >= 0 */
  int32_t mask_kind;  /* XY_MASK_CAUSAL (prefill, decode) or XY_MASK_TREE (verify) */
  int32_t parent_off; /* XY_MASK_TREE: index of this request's first node in tree_parents; else -1 */
} xy_attn_request;

/* One meta-task of the Task-Table: a packed Q tile against a run of 128-key KV
 * tiles.  Row x of the packed tile is (token tok0 + x / G, q head kv_head*G + x % G),
 * G = Hq/Hkv. */
typedef struct {
  int32_t req;     /* request index */
  int32_t kv_head; /* kv head */
  int32_t tok0;    /* first new token of the tile, relative to the request */
  int32_t ntok;    /* tokens in the tile; rows = ntok * G */
  int32_t kt_lo;   /* first 128-key tile of the run */
  int32_t kt_hi;   /* one past the last 128-key tile of the run */
  int32_t part;    /* -1: the task writes final O and LSE; >= 0: first row of its fp32 partial */
  int32_t kind;    /* 0 dense (rows > 16), 1 streaming (rows <= 16: decode, tiny verify) */
} xy_attn_task;

/* A tile unit whose KV range was split: its `nsplit` partials of `rows` rows each
 * start at partial row `part0` and are `rows` apart. */
typedef struct {
  int32_t req, kv_head, tok0, ntok;
  int32_t part0, nsplit;            /* partials of the unit's own KV splits: part0 + c * rows */
  int32_t part1, nsplit1, stride1;  /* a second family (shared-prefix groups): part1 + c * stride1 */
  int32_t reserved;
} xy_attn_merge_unit;

typedef struct {
  int32_t num_tasks;
  int32_t num_dense_tasks;
  int32_t num_merge_units;
  int32_t num_workers;
  int64_t useful_flops;   /* 4 D Hq sum of allowed (row, key) pairs */
  int64_t kv_bytes;       /* K+V bytes with each cached token of each kv head read once per request */
  int64_t partial_rows;   /* fp32 partial rows used in the workspace */
  float load_min, load_mean, load_max; /* per-worker summed task cost */
  float max_task_cost;
  int32_t num_inline_merge_units; /* of num_merge_units: split units of at most 16 rows (decode, tiny verify) that the
                                   * attention kernel merges itself - the task of the unit that finishes last does it;
                                   * the others are merged by the merge kernel (they come first in the unit list) */
  int32_t reserved;
} xy_attn_plan_info;

/* Create a context.  Allocates the device-side tables and the split workspace
 * once (cudaMalloc); plan and run allocate nothing.  cfg->device = -1 makes a
 * host-only context for planning without a GPU. */
int xy_attn_create(const xy_attn_config* cfg /*HOST*/, xy_attn_ctx** out /*HOST*/);
int xy_attn_destroy(xy_attn_ctx* ctx);

/* Token-Table -> decomposition -> Task-Table (Sections 3.2.1, 3.3.1).  Host work
 * plus asynchronous host-to-device copies of the tables on `stream` (a
 * cudaStream_t, may be 0).  `reqs` and `tree_parents` are HOST arrays, read
 * before return.  tree_parents holds the parent arrays of the XY_MASK_TREE
 * requests back to back: parent[i] in {-1} U [0, i-1] (several roots allowed);
 * anything else gives XY_ERR_BAD_TREE.  The ancestor-or-self bit matrix
 * (ceil(n/64) 64-bit words per node, bit j' of row i set iff j' is i or one of
 * its ancestors) is built here.  Zero requests is valid and makes run a no-op.
 * On error the previous plan is discarded. */
int xy_attn_plan(xy_attn_ctx* ctx, const xy_attn_request* reqs /*HOST*/, int32_t num_reqs,
                 const int32_t* tree_parents /*HOST, nullable if no tree*/, int32_t num_parents,
                 void* stream, xy_attn_plan_info* info /*HOST, nullable*/);

/* Shared-prefix ("cascade") decode, a variant the paper's related work names (requests that share
 * a radix-tree prefix batch their queries against it).  Requests first_req .. first_req+num_reqs-1
 * must be decode requests (q_len 1, XY_MASK_CAUSAL) with kv_len >= prefix_tokens whose
 * block-table rows hold THE SAME page ids for the first prefix_tokens tokens (prefix_tokens a
 * positive multiple of 128).  Their query rows are packed into tiles that read the shared K/V
 * once (dense tcgen05 tiles from 17 packed rows on), every member keeps a task for its own keys
 * behind the prefix, and the split-KV merge kernel combines the two partials.  The result is
 * the same attention as without groups; only the K/V traffic differs.  Groups must not overlap. */
typedef struct {
  int32_t first_req, num_reqs, prefix_tokens;
} xy_attn_prefix_group;

/* xy_attn_plan with shared-prefix groups (HOST array, read before return; num_groups = 0 is
 * xy_attn_plan).  XY_PLAN_BALANCED only.  Errors as xy_attn_plan, plus XY_ERR_INVALID_ARG for a
 * group that breaks the rules above and XY_ERR_CAPACITY when requests + groups exceed
 * max_requests. */
int xy_attn_plan_shared(xy_attn_ctx* ctx, const xy_attn_request* reqs /*HOST*/, int32_t num_reqs,
                        const int32_t* tree_parents /*HOST, nullable*/, int32_t num_parents,
                        const xy_attn_prefix_group* groups /*HOST*/, int32_t num_groups, void* stream,
                        xy_attn_plan_info* info /*HOST, nullable*/);

/* Finds shared-prefix groups from the block tables (what a radix-tree prefix cache leaves behind:
 * requests that matched the same cached prefix point at the same pages, Section 4.1.1).  HOST
 * arithmetic only; needs no context.  Scans the requests in order; a group is a maximal run of
 * consecutive decode requests (q_len 1, XY_MASK_CAUSAL) that each share at least
 * max(min_prefix_tokens, 128) leading tokens with the run's first request — same page ids in
 * block_table (HOST int32 [num_reqs, block_table_stride], entries < 0 never match), counted in
 * whole 128-token tiles inside both histories; the group's prefix_tokens is the smallest such
 * overlap.  Runs shorter than min_members (>= 2) are left ungrouped.  Every group written
 * satisfies the rules of xy_attn_prefix_group.  groups HOST [capacity], *num_groups written.
 * Returns XY_OK, XY_ERR_INVALID_ARG (null pointer, bad page_size or min_members) or
 * XY_ERR_CAPACITY (more groups than capacity; the first `capacity` are written). */
int xy_attn_find_prefix_groups(const xy_attn_request* reqs /*HOST*/, int32_t num_reqs,
                               const int32_t* block_table /*HOST*/, int32_t block_table_stride,
                               int32_t page_size, int32_t min_members, int32_t min_prefix_tokens,
                               xy_attn_prefix_group* groups /*HOST*/, int32_t capacity, int32_t* num_groups);

/* Task-Table cache (Section 3.3: the Task-Table is what the kernels consume; Section 3.3.2 keeps
 * pre-built Task-Tables for recurring shapes).  xy_attn_plan keeps the Task-Tables of the last
 * `capacity` distinct decompositions (default 8).  A plan whose decomposition — per request, kv
 * head and q tile: token range, task kind and number of visible 128-key tiles — equals a cached
 * one reuses that Task-Table (bit-identical to a fresh build) and, if it is the one already in
 * the device tables, skips their upload; the Token-Table, the request facts and the tree masks
 * are rebuilt and uploaded every time.  Consecutive decode steps change kvLen by one token and
 * hit until a request crosses a 128-key tile.  capacity = -1 leaves the setting, 0 disables the
 * cache; hits / misses (HOST, nullable) receive the counts since create. */
int xy_attn_plan_cache(xy_attn_ctx* ctx, int32_t capacity, int64_t* hits /*HOST*/, int64_t* misses /*HOST*/);

/* Meta-Attention over the planned batch (Sections 4.1-4.2, 5.2, 5.4).
 * Asynchronous on `stream`; no allocation, no host synchronisation.
 *   q            DEVICE bf16; row of token t, head a at q + t*q_token_stride + a*D
 *                (elements; q_token_stride >= Hq*D and a multiple of 8, so a fused
 *                [tokens, Hq + 2 Hkv, D] tensor can be passed directly)
 *   k_pool/v_pool DEVICE bf16 [num_pages, Hkv, B, D]; element strides page_stride,
 *                head_stride, token_stride (multiples of 8; D contiguous); every
 *                element of every page a request references must be finite
 *   block_table  DEVICE int32 [num_reqs, block_table_stride]; row r holds at least
 *                ceil((kv_len+q_len)/B) page ids in [0, num_pages)
 *   sm_scale     softmax scale, positive and finite (1/sqrt(D) in the usual case)
 *   tree_mask    DEVICE, nullable: a caller-built corner mask in plan's format
 *                replacing the one plan built from the parent arrays
 *   o            DEVICE bf16 [T, Hq, D] with token stride o_token_stride (elements)
 *   lse          DEVICE fp32 [T, Hq]: natural log of sum exp(sm_scale * q.k) over allowed keys
 * The new tokens' K/V must already be in the cache at positions kv_len .. kv_len+q_len-1. */
int xy_attn_run(xy_attn_ctx* ctx, const void* q, int64_t q_token_stride, const void* k_pool,
                const void* v_pool, int64_t num_pages, int64_t page_stride, int64_t head_stride,
                int64_t token_stride, const int32_t* block_table, int32_t block_table_stride,
                const uint64_t* tree_mask, float sm_scale, void* o, int64_t o_token_stride,
                float* lse, void* stream);

/* Meta-Attention over an fp8 KV cache.  The paper's cache is bf16; an fp8 cache is a variant the
 * related-work directions name, and nothing in the paper fixes its format, so this is the
 * library's own definition: K and V are stored as e4m3 bytes (1 sign, 4 exponent bits of bias 7,
 * 3 mantissa bits, no infinities, 0x7F / 0xFF = NaN: never store those) and the attended value
 * is  decode(byte) * scale[page][kv_head]  with one fp32 scale per page and kv head, K and V
 * separately.  Everything else - requests, masks, block tables, Q, O, LSE - is as in xy_attn_run,
 * and the context must have been created with kv_dtype = XY_KV_FP8_E4M3 (xy_attn_run then
 * returns XY_ERR_UNSUPPORTED, and so does this call on a bf16 context).
 *   k_pool/v_pool  DEVICE uint8 [num_pages, Hkv, B, D]; strides in elements (= bytes), multiples
 *                  of 16; D contiguous
 *   k_scale/v_scale DEVICE fp32 [num_pages, Hkv], contiguous, finite and positive
 * Requires page_size >= 16.  Widening e4m3 to f16 is exact; Q is used as f16 after a per-row
 * power-of-two factor (exact for every element within 2^-14 of its row's largest); scores, the
 * softmax and O accumulate in fp32; P is rounded to f16.  Dense tiles run on the warp-level MMA
 * path in this variant.  xy_attn_append_kv and xy_attn_debug_gather do not serve fp8 contexts
 * (quantising on append needs a scale policy that the caller owns). */
int xy_attn_run_fp8kv(xy_attn_ctx* ctx, const void* q, int64_t q_token_stride, const void* k_pool,
                      const void* v_pool, const float* k_scale, const float* v_scale, int64_t num_pages,
                      int64_t page_stride, int64_t head_stride, int64_t token_stride,
                      const int32_t* block_table, int32_t block_table_stride, const uint64_t* tree_mask,
                      float sm_scale, void* o, int64_t o_token_stride, float* lse, void* stream);

/* KV-cache append with fused QKV split (the step before attention: Sections 4.1.1 and 5.4).
 * For every planned request r and new token i the K and V head rows of the fused tensor
 *   qkv DEVICE bf16 [T, Hq + 2 Hkv, D] (token stride qkv_token_stride elements; K heads follow
 *   the Hq query heads, V heads follow the K heads)
 * are copied into the paged cache at logical position kv_len[r] + i, found through the block
 * table, with no intermediate split / permute tensors.  Uses the current plan's Token-Table;
 * asynchronous on `stream`; run it before xy_attn_run of the same step (stream order suffices).
 * The pools are written, everything else is read-only. */
int xy_attn_append_kv(xy_attn_ctx* ctx, const void* qkv, int64_t qkv_token_stride, void* k_pool, void* v_pool,
                      int64_t num_pages, int64_t page_stride, int64_t head_stride, int64_t token_stride,
                      const int32_t* block_table, int32_t block_table_stride, void* stream);

/* Split-KV LSE merge alone (the cross-core form of the Update stage, Section 4.2.1):
 *   LSE = ln sum_c exp(LSE_c),  O = sum_c exp(LSE_c - LSE) O_c.
 * o_part DEVICE fp32 [num_splits, rows, D], lse_part DEVICE fp32 [num_splits, rows];
 * o DEVICE bf16 [rows, D], lse DEVICE fp32 [rows].  A partial with LSE_c = -inf is ignored.
 * Needs no context; asynchronous on `stream`. */
int xy_attn_merge(const float* o_part, const float* lse_part, int32_t num_splits, int64_t rows,
                  int32_t head_dim, void* o, float* lse, void* stream);

/* Context sharded over devices (one long request's keys split across GPUs; the cross-device
 * form of the Update stage, Section 4.2.1).  Device k holds the keys [bounds[k], bounds[k+1]) of
 * the request in its own paged cache and runs xy_attn_run on them as a decode request whose
 * kv_len is the slice length minus one (the last key of the slice stands where the new token
 * would: every key of the slice is visible to the single query row); that yields the slice's
 * normalised O_k (bf16) and LSE_k.  After one all-gather of (O_k, LSE_k) into local memory every
 * device merges:  LSE = ln sum_k exp(LSE_k),  O = sum_k exp(LSE_k - LSE) O_k.
 *
 * xy_attn_shard_context: HOST arithmetic only.  Splits total_tokens (cached + new, >= 1) into
 *   num_shards contiguous slices whose starts are multiples of page_size; page counts differ by
 *   at most one, the ragged tail (and so the position the new token is appended at) lies in the
 *   last slice.  bounds HOST int64 [num_shards + 1], written.  XY_ERR_INVALID_ARG when the
 *   context has fewer pages than shards.
 * xy_attn_merge_shards: o_shards DEVICE bf16 [num_shards, rows, D] and lse_shards DEVICE fp32
 *   [num_shards, rows] in LOCAL memory (the all-gather's output; rows = tokens x q heads);
 *   o DEVICE bf16 [rows, D], lse DEVICE fp32 [rows], written.  A shard with LSE_k = -inf is
 *   ignored and its O_k not read.  Needs no context; asynchronous on `stream`. */
int xy_attn_shard_context(int64_t total_tokens, int32_t page_size, int32_t num_shards, int64_t* bounds);
int xy_attn_merge_shards(const void* o_shards, const float* lse_shards, int32_t num_shards, int64_t rows,
                         int32_t head_dim, void* o, float* lse, void* stream);

/* Allocation-free decode attention.  The paper has no counterpart for this call: it exists
 * for callers that cannot allocate device memory where they need attention - a serving loop
 * whose memory pool is already handed out in full, a plugin that is given only a stream and
 * its buffers, a program that must keep away from the allocator while another library owns
 * it.  It computes the same result as xy_attn_run for a batch of decode requests (one new
 * token each, causal): request r attends to its kv_len[r] cached tokens plus the new token,
 * whose K/V is already in the cache.  No context is needed and nothing is allocated or freed,
 * on the device or through any library: the split-KV scratch is a fixed array inside the
 * library image, XY_ATTN_STATIC_MAX_ROWS rows of 129 floats (about 4.03 MiB), which every GPU
 * that loads the library holds until the process exits.
 *   q, k_pool, v_pool, block_table, o, lse: as for xy_attn_run (token r of q / o / lse is request r)
 *   kv_len      DEVICE int32 [num_reqs]: cached tokens before the new one
 *   max_kv_len  HOST value, >= every kv_len[r]; sets the number of 2048-key chunks.  A request
 *               whose kv_len[r] exceeds it reads nothing beyond max_kv_len + 1 keys and gets NaN
 *               in its rows of o and lse (never a silently truncated context)
 * Limit: num_reqs * num_q_heads * ceil((max_kv_len + 1) / 2048) <= XY_ATTN_STATIC_MAX_ROWS;
 * beyond it the call returns XY_ERR_CAPACITY (and prints one line to stderr) without launching.
 * The first call on each device looks up the scratch's device address; make that first call
 * outside any stream capture.  All calls share the one scratch array and every call rewrites
 * the part it reads, so nothing needs clearing between calls, but two calls whose kernels can
 * overlap on the GPU (different streams, no ordering between them) race on it: order them. */
#define XY_ATTN_STATIC_MAX_ROWS 8192
int xy_attn_decode_static(const void* q, int64_t q_token_stride, const void* k_pool, const void* v_pool,
                          int64_t page_stride, int64_t head_stride, int64_t token_stride,
                          const int32_t* block_table, int32_t block_table_stride,
                          const int32_t* kv_len /*DEVICE*/, int32_t num_reqs, int32_t max_kv_len,
                          int32_t num_q_heads, int32_t num_kv_heads, int32_t page_size, float sm_scale,
                          void* o, int64_t o_token_stride, float* lse, void* stream);

/* Debug/verification: copy the K and V rows a request sees, in logical order,
 * through the block table: out_k/out_v DEVICE bf16 [kv_len+q_len, D] for kv head
 * `kv_head` of planned request `req`. */
int xy_attn_debug_gather(xy_attn_ctx* ctx, int32_t req, int32_t kv_head, const void* k_pool,
                         const void* v_pool, int64_t page_stride, int64_t head_stride,
                         int64_t token_stride, const int32_t* block_table,
                         int32_t block_table_stride, void* out_k, void* out_v, void* stream);

/* Per-worker wall time of the last xy_attn_run (load-balance metric): synchronises the device
 * and copies 4 x num_workers values to `out` (HOST): for each persistent worker its entry and
 * exit time stamps (nanoseconds of the GPU's global timer) and the nanoseconds it spent in dense
 * and in streaming tasks.  Returns the number of entries; copies only if `cap`
 * is large enough.  Only the attention meta-kernel records them (not XY_KERNEL_REFERENCE). */
int xy_attn_worker_times(xy_attn_ctx* ctx, uint64_t* out, int32_t cap);

/* Debug tracing (only in a library built with -DXY_ENABLE_TRACE, i.e. XY_BUILD_TRACE=1 for
 * paper_2412_18106_b200.build; otherwise no records are written and 0 entries are meaningful).
 * When the environment variable XY_ATTN_TRACE=1 is set at create time, the
 * roles of worker 0 (sub-tile A, sub-tile B, MMA issuer, producer) stamp (tag << 48 | SM cycle
 * counter) records into a context-owned buffer of 4 x 2048 entries per run.  This call
 * synchronises the device and copies them to `out` (HOST); it returns the number of entries
 * (0 when tracing is off) and copies only if `cap` is large enough. */
int xy_attn_debug_trace(xy_attn_ctx* ctx, uint64_t* out, int32_t cap);

/* Introspection of the current plan (HOST outputs).  Each returns the number of
 * items of the plan, or a negative error; at most `cap` items are written. */
int xy_attn_get_tasks(const xy_attn_ctx* ctx, xy_attn_task* out, int32_t cap);
int xy_attn_get_worker_offsets(const xy_attn_ctx* ctx, int32_t* out /* num_workers+1 */, int32_t cap);
int xy_attn_get_merge_units(const xy_attn_ctx* ctx, xy_attn_merge_unit* out, int32_t cap);
int xy_attn_get_tree_mask(const xy_attn_ctx* ctx, uint64_t* out, int32_t cap_words);
int xy_attn_get_q_start(const xy_attn_ctx* ctx, int32_t* out /* num_reqs+1 */, int32_t cap);
/* The order in which free workers take tasks (indices into the task table, a permutation of it)
 * when the plan is dealt dynamically: XY_PLAN_BALANCED with the MMA kernels. */
int xy_attn_get_queue(const xy_attn_ctx* ctx, int32_t* out /* num_tasks */, int32_t cap);

/* Per-kernel device timing.  With timing enabled every xy_attn_run records CUDA events on
 * its stream around the attention launch and around the merge launch (at most 4096 runs
 * are kept).  xy_attn_get_timing waits for the last recorded run, returns the summed
 * durations in milliseconds and the number of runs they cover, and clears the record. */
int xy_attn_set_timing(xy_attn_ctx* ctx, int32_t enable);
int xy_attn_get_timing(xy_attn_ctx* ctx, float* attention_ms /*HOST*/, float* merge_ms /*HOST*/,
                       int32_t* runs /*HOST*/);

/* Validation aid (the stand-in for a memory checker on the paged gather, Section 4.1.1).  Checks a
 * HOST copy of the block table against the current plan: every request must find
 * ceil((kv_len + q_len) / B) entries in its row (<= block_table_stride) and each of them must lie
 * in [0, num_pages).  Host arithmetic only; works on a host-only context.  Returns XY_OK,
 * XY_ERR_NOT_PLANNED, or XY_ERR_INVALID_ARG with the offending request and entry in
 * xy_attn_last_error.  A context created while the environment variable XY_ATTN_DEBUG=1 is set
 * runs this check inside every xy_attn_run (it copies the device block table to the host first,
 * which synchronises the stream) and launches nothing when it fails. */
int xy_attn_debug_check_block_table(xy_attn_ctx* ctx, const int32_t* block_table /*HOST*/,
                                    int32_t block_table_stride, int64_t num_pages);

/* Failure-path test hook for the bounded waits of the attention kernel (every wait on a barrier
 * or a turn counter gives up after a limit and records XY_ERR_DEVICE_TIMEOUT, Section 4.2.1's
 * pipelines being chains of such hand-offs).  wait_limit_polls > 0 replaces the limit (0 restores
 * the default of 2^22 polls); skip_fill >= 0 makes the producer of every worker leave out its
 * skip_fill-th K/V stage fill of the following runs (-1: none), so that the readers of that stage
 * never see it filled and their waits run out.  Nothing faults and nothing spins without bound:
 * the kernel returns, frees its tensor memory, and the status shows the timeout; O and LSE of
 * such a run are unspecified.  The next run on the context starts from a clean status word. */
int xy_attn_debug_inject(xy_attn_ctx* ctx, int32_t wait_limit_polls, int32_t skip_fill);

/* Number of kernel launches the last xy_attn_run enqueued. */
int xy_attn_last_launches(const xy_attn_ctx* ctx);

/* Message of the last error on this context (never null). */
const char* xy_attn_last_error(const xy_attn_ctx* ctx);

/* Synchronises the device, reads the status the kernels recorded and clears it: XY_OK, or
 * XY_ERR_DEVICE_TIMEOUT when a bounded wait inside a kernel gave up in any run since the last
 * call.  A run whose status is not XY_OK has unspecified O and LSE.  The context stays usable:
 * every xy_attn_run starts from a clean status word, so the run after a timeout is an ordinary
 * run (the record of the failure is kept until this function reports it). */
int xy_attn_device_status(xy_attn_ctx* ctx, int32_t* status_out /*HOST*/);

#ifdef __cplusplus
}
#endif
#endif /* XY_ATTN_H_ */
