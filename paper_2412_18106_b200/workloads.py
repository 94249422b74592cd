"""Seeded synthetic hybrid batches (structure and tensors).

This module serves both the CUDA path and the CPU oracle with *inputs only*: it
draws request shapes, token trees, block tables and bf16 tensors from seeded
generators.  It holds none of the method's arithmetic (no attention, no
planning, no masks) and imports neither the binding nor the oracle.

Vocabulary follows the paper's Token-Table (Section 3.2): a request ("stage")
has `q_len` new tokens (tokenNum) on top of `kv_len` cached tokens (historical
kvLen); its kind is prefill (P), decode (D) or verify (V).  The new tokens' K/V
already sit in the paged cache at logical positions kv_len .. kv_len+q_len-1
(Section 4.1.1: historical and newly generated blocks are both read through
the block table).
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional

import numpy as np
import torch

MASK_CAUSAL = 0
MASK_TREE = 1

HEAD_DIM = 128


@dataclasses.dataclass
class Batch:
    """Structure of one hybrid batch (no tensors)."""

    name: str
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    q_len: np.ndarray  # int32 [R]
    kv_len: np.ndarray  # int32 [R]
    mask_kind: np.ndarray  # int32 [R]
    parent_off: np.ndarray  # int32 [R], -1 unless TREE
    parents: np.ndarray  # int32 [sum of q_len over TREE requests]
    block_table: np.ndarray  # int32 [R, max_pages], -1 = unused entry
    num_pages: int  # pages in the pool (used + spare)
    seed: int = 0

    @property
    def num_requests(self) -> int:
        return int(self.q_len.shape[0])

    @property
    def total_q(self) -> int:
        return int(self.q_len.sum())

    @property
    def q_start(self) -> np.ndarray:
        out = np.zeros(self.num_requests + 1, dtype=np.int64)
        np.cumsum(self.q_len, out=out[1:])
        return out

    def tree_parents(self, r: int) -> Optional[np.ndarray]:
        if int(self.mask_kind[r]) != MASK_TREE:
            return None
        off = int(self.parent_off[r])
        return self.parents[off : off + int(self.q_len[r])]


@dataclasses.dataclass
class Tensors:
    """bf16 tensors of a batch, on CPU."""

    q: torch.Tensor  # bf16 [T, Hq, D]  (a view into `qkv` when fused)
    k_pool: torch.Tensor  # bf16 [P, Hkv, B, D]
    v_pool: torch.Tensor  # bf16 [P, Hkv, B, D]
    qkv: Optional[torch.Tensor] = None  # bf16 [T, Hq + 2 Hkv, D] when fused
    k_scale: Optional[torch.Tensor] = None  # fp8 KV cache: fp32 [P, Hkv]; the pools are then uint8 e4m3 bytes
    v_scale: Optional[torch.Tensor] = None


def _pages_needed(q_len, kv_len, page_size):
    tot = np.asarray(q_len, dtype=np.int64) + np.asarray(kv_len, dtype=np.int64)
    return (tot + page_size - 1) // page_size


def assemble(
    name: str,
    hq: int,
    hkv: int,
    page_size: int,
    q_len,
    kv_len,
    mask_kind,
    trees: List[Optional[np.ndarray]],
    rng: np.random.Generator,
    seed: int,
    spare_frac: float = 0.10,
    permute_pages: bool = True,
) -> Batch:
    """Build the block table (random permutation of the pool) and pack trees."""
    q_len = np.asarray(q_len, dtype=np.int32)
    kv_len = np.asarray(kv_len, dtype=np.int32)
    mask_kind = np.asarray(mask_kind, dtype=np.int32)
    R = q_len.shape[0]
    need = _pages_needed(q_len, kv_len, page_size)
    used = int(need.sum())
    num_pages = used + max(1, int(math.ceil(used * spare_frac)))
    order = rng.permutation(num_pages) if permute_pages else np.arange(num_pages)
    max_pages = int(need.max()) if R else 1
    bt = np.full((R, max(max_pages, 1)), -1, dtype=np.int32)
    pos = 0
    for r in range(R):
        n = int(need[r])
        bt[r, :n] = order[pos : pos + n]
        pos += n
    parent_off = np.full(R, -1, dtype=np.int32)
    chunks = []
    off = 0
    for r in range(R):
        if int(mask_kind[r]) == MASK_TREE:
            p = np.asarray(trees[r], dtype=np.int32)
            assert p.shape[0] == int(q_len[r])
            parent_off[r] = off
            chunks.append(p)
            off += p.shape[0]
    parents = np.concatenate(chunks).astype(np.int32) if chunks else np.zeros(0, np.int32)
    return Batch(name, hq, hkv, HEAD_DIM, page_size, q_len, kv_len, mask_kind,
                 parent_off, parents, bt, num_pages, seed)


def random_tree(rng: np.random.Generator, n: int, max_depth: int = 8) -> np.ndarray:
    """Random parent array in topological order: parent[0] = -1 and
    parent[i] uniform in [0, i-1], redrawn until the node's depth (root = 1)
    does not exceed `max_depth` (max_depth <= 1: every node is a root)."""
    parent = np.full(n, -1, dtype=np.int32)
    depth = np.ones(n, dtype=np.int32)
    if max_depth <= 1:
        return parent
    for i in range(1, n):
        while True:
            p = int(rng.integers(0, i))
            if depth[p] + 1 <= max_depth:
                break
        parent[i] = p
        depth[i] = depth[p] + 1
    return parent


def chain_tree(n: int) -> np.ndarray:
    return np.arange(-1, n - 1, dtype=np.int32)


def _log_uniform_int(rng, lo, hi):
    return int(round(math.exp(rng.uniform(math.log(lo), math.log(hi)))))


def config1_tiny(seed: int = 0) -> Batch:
    """Tiny hybrid batch: prefill 64 (kv 0), prefill 64 on a 128-token prefix,
    decode at kv 300, verify with a 4-token chain at kv 200. 8/2 heads, page 16."""
    rng = np.random.default_rng(seed)
    q_len = [64, 64, 1, 4]
    kv_len = [0, 128, 300, 200]
    kind = [MASK_CAUSAL, MASK_CAUSAL, MASK_CAUSAL, MASK_TREE]
    trees = [None, None, None, chain_tree(4)]
    return assemble("tiny_hybrid", 8, 2, 16, q_len, kv_len, kind, trees, rng, seed)


def config2_decode(seed: int = 0, num_requests: int = 64, kv_lo: int = 512,
                   kv_hi: int = 8192) -> Batch:
    """Decode-only: 64 x 1 token, kv_len uniform in [512, 8192], 28/4 heads, page 128."""
    rng = np.random.default_rng(seed)
    kv = rng.integers(kv_lo, kv_hi + 1, size=num_requests)
    q_len = np.ones(num_requests, dtype=np.int32)
    kind = np.zeros(num_requests, dtype=np.int32)
    return assemble("decode_only", 28, 4, 128, q_len, kv, kind, [None] * num_requests, rng, seed)


def config3_splitfuse(seed: int = 0, chunk: int = 2048, prefix: int = 6144,
                      num_decode: int = 48, kv_lo: int = 1024, kv_hi: int = 16384) -> Batch:
    """SplitFuse mix: one prefill chunk on a cached prefix plus decode requests.
    32/8 heads, page 128."""
    rng = np.random.default_rng(seed)
    kv = [prefix] + [int(x) for x in rng.integers(kv_lo, kv_hi + 1, size=num_decode)]
    q_len = [chunk] + [1] * num_decode
    R = 1 + num_decode
    return assemble("splitfuse_mix", 32, 8, 128, q_len, kv, [MASK_CAUSAL] * R, [None] * R, rng, seed)


def config4_verify(seed: int = 0, num_requests: int = 32, n_lo: int = 8, n_hi: int = 64,
                   kv_lo: int = 1024, kv_hi: int = 32768, max_depth: int = 8) -> Batch:
    """Speculative verify: random token trees of 8..64 nodes (depth <= 8),
    kv_len uniform in [1k, 32k], 64/8 heads, page 128."""
    rng = np.random.default_rng(seed)
    n = rng.integers(n_lo, n_hi + 1, size=num_requests)
    trees = [random_tree(rng, int(x), max_depth) for x in n]
    kv = rng.integers(kv_lo, kv_hi + 1, size=num_requests)
    return assemble("verify_trees", 64, 8, 128, n, kv, [MASK_TREE] * num_requests, trees, rng, seed)


def config5_full_mix(seed: int = 0, num_requests: int = 96) -> Batch:
    """Full dynamic serving mix: 20% prefill (q_len log-uniform 128..4096, prefix
    hit fraction f uniform in [0, 0.9], cached length floor(n f / (1 - f)),
    token-granular), 60% decode and 20% verify (trees of 4..32 nodes) with kv_len
    log-uniform 256..64k.  64/8 heads, page 128.  Requests are shuffled."""
    rng = np.random.default_rng(seed)
    n_p = int(round(0.2 * num_requests))
    n_v = int(round(0.2 * num_requests))
    n_d = num_requests - n_p - n_v
    q_len, kv_len, kind, trees = [], [], [], []
    for _ in range(n_p):
        n = _log_uniform_int(rng, 128, 4096)
        f = float(rng.uniform(0.0, 0.9))
        q_len.append(n)
        kv_len.append(int(math.floor(n * f / (1.0 - f))))
        kind.append(MASK_CAUSAL)
        trees.append(None)
    for _ in range(n_d):
        q_len.append(1)
        kv_len.append(_log_uniform_int(rng, 256, 65536))
        kind.append(MASK_CAUSAL)
        trees.append(None)
    for _ in range(n_v):
        n = int(rng.integers(4, 33))
        q_len.append(n)
        kv_len.append(_log_uniform_int(rng, 256, 65536))
        kind.append(MASK_TREE)
        trees.append(random_tree(rng, n, 8))
    order = rng.permutation(num_requests)
    q_len = [q_len[i] for i in order]
    kv_len = [kv_len[i] for i in order]
    kind = [kind[i] for i in order]
    trees = [trees[i] for i in order]
    return assemble("full_mix", 64, 8, 128, q_len, kv_len, kind, trees, rng, seed)


def prefill_prefix(seed: int = 0, num_requests: int = 4, q_tokens: int = 4096) -> Batch:
    """Prefill on a reused prefix (shape of the paper's Section 6.2.1 sweep): prompts of
    `q_tokens` new tokens on cached prefixes drawn token by token from [0, 4096].  32/8 heads,
    page 128.  Not one of the five benchmark configurations; used to tune the dense path."""
    rng = np.random.default_rng(seed)
    kv = [int(x) for x in rng.integers(0, 4097, size=num_requests)]
    R = num_requests
    return assemble("prefill_prefix", 32, 8, 128, [q_tokens] * R, kv, [MASK_CAUSAL] * R, [None] * R, rng, seed)


CONFIGS = {
    "tiny_hybrid": config1_tiny,
    "decode_only": config2_decode,
    "splitfuse_mix": config3_splitfuse,
    "verify_trees": config4_verify,
    "full_mix": config5_full_mix,
    "prefill_prefix": prefill_prefix,
}


def shared_prefix_decode(seed: int = 0, num_groups: int = 4, members: int = 32, prefix: int = 8192,
                         suffix_hi: int = 1024, hq: int = 32, hkv: int = 8, page_size: int = 128):
    """Decode requests that share cached prefixes (a common system prompt, a radix-tree branch):
    `num_groups` groups of `members` requests; the members of a group hold THE SAME pages for their
    first `prefix` tokens (a multiple of 128) and then own `0 .. suffix_hi` further tokens each.
    Returns (batch, groups) with groups = [(first_req, num_reqs, prefix_tokens), ...]."""
    assert prefix % 128 == 0 and prefix % page_size == 0
    rng = np.random.default_rng(seed)
    R = num_groups * members
    kv = [prefix + int(x) for x in rng.integers(0, suffix_hi + 1, size=R)]
    b = assemble("decode_shared_prefix", hq, hkv, page_size, [1] * R, kv, [MASK_CAUSAL] * R, [None] * R, rng, seed)
    npre = prefix // page_size
    groups = []
    for g in range(num_groups):
        first = g * members
        for r in range(first + 1, first + members):
            b.block_table[r, :npre] = b.block_table[first, :npre]
        groups.append((first, members, prefix))
    return b, groups


def long_context_decode(seed: int = 0, num_requests: int = 4, kv_lo: int = 131072, kv_hi: int = 524288,
                        hq: int = 32, hkv: int = 8, page_size: int = 128) -> Batch:
    """Few decode requests on very long contexts (log-uniform lengths): every (request, kv head)
    row is split over many workers and merged (the split-KV path)."""
    rng = np.random.default_rng(seed)
    kv = [_log_uniform_int(rng, kv_lo, kv_hi) for _ in range(num_requests)]
    return assemble("long_context_decode", hq, hkv, page_size, [1] * num_requests, kv,
                    [MASK_CAUSAL] * num_requests, [None] * num_requests, rng, seed, spare_frac=0.01)


CONFIGS["long_context_decode"] = long_context_decode


def custom(name: str, hq: int, hkv: int, page_size: int, requests, seed: int = 0,
           permute_pages: bool = True, spare_frac: float = 0.10) -> Batch:
    """`requests` is a list of (q_len, kv_len, kind, parents-or-None) tuples."""
    rng = np.random.default_rng(seed)
    q_len = [r[0] for r in requests]
    kv_len = [r[1] for r in requests]
    kind = [r[2] for r in requests]
    trees = [None if r[3] is None else np.asarray(r[3], dtype=np.int32) for r in requests]
    return assemble(name, hq, hkv, page_size, q_len, kv_len, kind, trees, rng, seed,
                    spare_frac=spare_frac, permute_pages=permute_pages)


def context_shard(batch: Batch, bounds, k: int) -> Batch:
    """Shard k of a decode batch whose contexts are split over devices.  `bounds[r]` holds the
    slice starts of request r's kv_len + 1 tokens (page-aligned, one more entry than shards).  The
    shard is a decode batch over the same pools: request r keeps the pages of its slice, and its
    kv_len is the slice length minus one, so that the single query row sees the whole slice."""
    assert np.all(batch.q_len == 1)
    B = batch.page_size
    lo = np.array([int(bd[k]) for bd in bounds], dtype=np.int64)
    hi = np.array([int(bd[k + 1]) for bd in bounds], dtype=np.int64)
    assert np.all(lo % B == 0) and np.all(hi > lo)
    need = (hi - lo + B - 1) // B
    bt = np.full((batch.num_requests, int(need.max())), -1, dtype=np.int32)
    for r in range(batch.num_requests):
        p0 = int(lo[r]) // B
        bt[r, : int(need[r])] = batch.block_table[r, p0 : p0 + int(need[r])]
    return Batch("%s_shard%d" % (batch.name, k), batch.num_q_heads, batch.num_kv_heads, batch.head_dim, B,
                 batch.q_len.copy(), (hi - lo - 1).astype(np.int32), batch.mask_kind.copy(),
                 batch.parent_off.copy(), batch.parents.copy(), bt, batch.num_pages, batch.seed)


def _randn_bf16(shape, gen: torch.Generator, chunk_elems: int = 1 << 26) -> torch.Tensor:
    """N(0,1) drawn in fp32 and rounded to bf16, produced in chunks to bound memory."""
    total = int(np.prod(shape)) if len(shape) else 1
    out = torch.empty(total, dtype=torch.bfloat16)
    pos = 0
    while pos < total:
        n = min(chunk_elems, total - pos)
        out[pos : pos + n] = torch.randn(n, generator=gen, dtype=torch.float32).to(torch.bfloat16)
        pos += n
    return out.view(*shape)


def make_tensors(batch: Batch, seed: Optional[int] = None, fused_qkv: bool = False,
                 tail_fill: Optional[float] = None) -> Tensors:
    """Q, K pool and V pool ~ N(0,1) in bf16.  Every page of the pool (spare pages
    and last-page tails included) holds finite N(0,1) data, unless `tail_fill` is
    given: then every cache slot at or beyond a request's kv_len+q_len, and every
    unused page, holds that (large, finite) value instead."""
    seed = batch.seed if seed is None else seed
    gen = torch.Generator().manual_seed(seed)
    T, Hq, Hkv, D, B = batch.total_q, batch.num_q_heads, batch.num_kv_heads, batch.head_dim, batch.page_size
    if fused_qkv:
        qkv = _randn_bf16((T, Hq + 2 * Hkv, D), gen)
        q = qkv[:, :Hq, :]
    else:
        qkv = None
        q = _randn_bf16((T, Hq, D), gen)
    k_pool = _randn_bf16((batch.num_pages, Hkv, B, D), gen)
    v_pool = _randn_bf16((batch.num_pages, Hkv, B, D), gen)
    if tail_fill is not None:
        used = np.zeros(batch.num_pages, dtype=bool)
        for r in range(batch.num_requests):
            L = int(batch.q_len[r]) + int(batch.kv_len[r])
            npg = (L + B - 1) // B
            pages = batch.block_table[r, :npg]
            used[pages] = True
            rem = L - (npg - 1) * B
            if npg > 0 and rem < B:
                last = int(pages[-1])
                k_pool[last, :, rem:, :] = tail_fill
                v_pool[last, :, rem:, :] = -tail_fill
        unused = torch.from_numpy(np.nonzero(~used)[0])
        if unused.numel():
            k_pool[unused] = tail_fill
            v_pool[unused] = -tail_fill
    return Tensors(q=q, k_pool=k_pool, v_pool=v_pool, qkv=qkv)


def to_fp8_kv(tensors: Tensors, unit_scale: bool = False) -> Tensors:
    """Inputs for the fp8 KV-cache variant: the K and V pools as e4m3 bytes with one fp32 scale
    per (page, kv head), chosen so that the page's largest magnitude maps to 448 (or scale = 1
    with `unit_scale`).  The cast is the library's (torch.float8_e4m3fn); what the attention
    kernels and the oracle receive are the bytes and the scales."""
    out = []
    for pool in (tensors.k_pool, tensors.v_pool):
        x = pool.float()
        if unit_scale:
            scale = torch.ones(x.shape[:2], dtype=torch.float32)
        else:
            scale = (x.abs().amax(dim=(2, 3)) / 448.0).clamp_min(2.0 ** -20)
        q = (x / scale[:, :, None, None]).to(torch.float8_e4m3fn)
        out.append((q.view(torch.uint8), scale.contiguous()))
    return Tensors(q=tensors.q, k_pool=out[0][0], v_pool=out[1][0], qkv=tensors.qkv, k_scale=out[0][1], v_scale=out[1][1])


def set_tile_onehot_v(batch: Batch, tensors: Tensors, tile: int = 128) -> None:
    """Probe input (in place): the V row of logical key j of every request becomes the unit
    vector e_d with d = (j // tile) mod D.  Each output element is then the probability mass of
    every D-th key tile, so one key tile that is lost, doubled or attributed to the wrong
    request moves an element by that tile's whole mass.  Pure data placement through the block
    table (requests that share pages keep the same logical positions, so they agree)."""
    B, D = batch.page_size, batch.head_dim
    for r in range(batch.num_requests):
        L = int(batch.q_len[r]) + int(batch.kv_len[r])
        npg = (L + B - 1) // B
        pages = torch.from_numpy(batch.block_table[r, :npg].astype(np.int64))
        j = torch.arange(npg * B, dtype=torch.int64).view(npg, B)
        d = (j // tile) % D
        rows = torch.zeros((npg, B, D), dtype=torch.bfloat16)
        rows.scatter_(2, d.unsqueeze(-1), 1.0)
        tensors.v_pool[pages] = rows.unsqueeze(1).expand(npg, batch.num_kv_heads, B, D)


def set_dominant_keys(batch: Batch, tensors: Tensors, positions, q_value: float = 4.0, k_value: float = 8.0) -> None:
    """Probe input (in place): every query row of request r becomes the constant vector q_value
    and the K row at logical position positions[r] (all kv heads) the constant vector k_value, so
    that this key's score exceeds every other by hundreds and its probability is exactly 1 in any
    fp32 softmax: the output row must then be that key's V row, bit for bit.  positions[r] must be
    visible to every row of the request (inside the history, or the first new token of a causal request)."""
    B = batch.page_size
    qs = batch.q_start
    for r in range(batch.num_requests):
        j = int(positions[r])
        h = int(batch.kv_len[r])
        assert 0 <= j < h or (j == h and (int(batch.mask_kind[r]) == MASK_CAUSAL or int(batch.q_len[r]) == 1))
        tensors.q[int(qs[r]) : int(qs[r + 1])] = q_value
        page = int(batch.block_table[r, j // B])
        tensors.k_pool[page, :, j % B, :] = k_value


def pairs_per_request(batch: Batch) -> np.ndarray:
    """Allowed (query row, key) pairs per request and q head: n h + n (n+1) / 2 for
    a causal request, n h + sum of node depths for a tree request.  Pure counting,
    used to state useful FLOPs = 4 D Hq sum(pairs)."""
    out = np.zeros(batch.num_requests, dtype=np.int64)
    for r in range(batch.num_requests):
        n, h = int(batch.q_len[r]), int(batch.kv_len[r])
        if int(batch.mask_kind[r]) == MASK_TREE:
            p = batch.tree_parents(r)
            depth = np.zeros(n, dtype=np.int64)
            for i in range(n):
                depth[i] = 1 if p[i] < 0 else depth[p[i]] + 1
            out[r] = n * h + int(depth.sum())
        else:
            out[r] = n * h + n * (n + 1) // 2
    return out


def useful_flops(batch: Batch) -> int:
    return int(4 * batch.head_dim * batch.num_q_heads * pairs_per_request(batch).sum())


def kv_bytes(batch: Batch) -> int:
    """K and V bytes when each cached token of each kv head is read once per request."""
    tot = (batch.q_len.astype(np.int64) + batch.kv_len.astype(np.int64)).sum()
    return int(2 * tot * batch.num_kv_heads * batch.head_dim * 2)


def algorithmic_bytes(batch: Batch) -> int:
    """KV bytes + Q read + O write (bf16) + LSE write (fp32) + block-table entries."""
    T = batch.total_q
    qo = 2 * T * batch.num_q_heads * batch.head_dim * 2
    lse = T * batch.num_q_heads * 4
    bt = int(_pages_needed(batch.q_len, batch.kv_len, batch.page_size).sum()) * 4
    return kv_bytes(batch) + qo + lse + bt
