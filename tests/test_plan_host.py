"""Host logic of the C-ABI library (no GPU): symbol export, validation and error codes,
Token-Table / decomposition / Task-Table invariants, and the paper-mode table against the
pure-Python restatement in oracle/task_table.py and the paper's worked example."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import task_table as TT
from paper_2412_18106_b200 import binding as xb
from paper_2412_18106_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def host_ctx(hq, hkv, page, **kw):
    kw.setdefault("device", -1)
    kw.setdefault("max_q_tokens", 1 << 16)
    kw.setdefault("max_pages_per_req", 4096)
    return xb.XYAttn(hq, hkv, page, **kw)


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "xy_attn.h")).read()
    declared = set(re.findall(r"\b(xy_attn_[a-z0-9_]+)\s*\(", header))
    assert declared == set(xb.EXPORTS)
    lib = ctypes.CDLL(xb.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name


def test_struct_sizes_match_header():
    assert ctypes.sizeof(xb.xy_attn_task) == 32
    assert ctypes.sizeof(xb.xy_attn_request) == 16
    assert ctypes.sizeof(xb.xy_attn_merge_unit) == 40
    assert ctypes.sizeof(xb.xy_attn_config) == 16 * 4 + 8   # 15 int32, padding, int64


def test_create_rejects_bad_configs():
    with pytest.raises(xb.XYAttnError) as e:
        host_ctx(8, 2, 16, head_dim=64)
    assert e.value.code == xb.XY_ERR_UNSUPPORTED
    with pytest.raises(xb.XYAttnError) as e:
        host_ctx(8, 2, 24)
    assert e.value.code == xb.XY_ERR_UNSUPPORTED
    with pytest.raises(xb.XYAttnError) as e:
        host_ctx(8, 3, 16)
    assert e.value.code == xb.XY_ERR_INVALID_ARG


def test_plan_error_codes():
    c = host_ctx(8, 2, 16, max_requests=4, max_q_tokens=100, max_pages_per_req=8, max_tree_nodes=4)
    def code(*a):
        with pytest.raises(xb.XYAttnError) as e:
            c.plan(*a)
        return e.value.code
    assert code([0], [5], [0], [-1]) == xb.XY_ERR_INVALID_ARG        # q_len < 1
    assert code([1], [-1], [0], [-1]) == xb.XY_ERR_INVALID_ARG       # kv_len < 0
    assert code([1], [1], [7], [-1]) == xb.XY_ERR_INVALID_ARG        # mask kind
    assert code([1] * 5, [1] * 5, [0] * 5, [-1] * 5) == xb.XY_ERR_CAPACITY  # requests
    assert code([101], [0], [0], [-1]) == xb.XY_ERR_CAPACITY         # q tokens
    assert code([1], [128], [0], [-1]) == xb.XY_ERR_CAPACITY         # pages per request
    assert code([5], [0], [1], [0], [-1, 0, 1, 2, 3]) == xb.XY_ERR_CAPACITY  # tree nodes
    assert code([3], [0], [1], [0], [-1, 1, 0]) == xb.XY_ERR_BAD_TREE   # parent >= index
    assert code([3], [0], [1], [0], [-1, -2, 0]) == xb.XY_ERR_BAD_TREE  # parent < -1
    assert code([3], [0], [1], [1], [-1, 0, 0]) == xb.XY_ERR_BAD_TREE   # parents array too short
    assert code([3], [0], [1], [0], None) == xb.XY_ERR_BAD_TREE
    # a failed plan discards the previous one
    c.plan([2], [3], [0], [-1])
    assert len(c.get_tasks()) > 0
    code([0], [5], [0], [-1])
    with pytest.raises(xb.XYAttnError) as e:
        c.get_tasks()
    assert e.value.code == xb.XY_ERR_NOT_PLANNED
    # zero requests is valid
    info = c.plan([], [], [], [])
    assert info.num_tasks == 0
    # host-only context cannot run
    rc = c.lib.xy_attn_run(c._ctx, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 1.0, 0, 0, 0, 0)
    assert rc == xb.XY_ERR_UNSUPPORTED


def test_tree_mask_is_ancestor_or_self():
    rng = np.random.default_rng(3)
    trees = [W.random_tree(rng, n, 8) for n in (1, 5, 63, 64, 65, 130)]
    trees.append(np.array([-1, -1, 0, 1, -1], dtype=np.int32))  # several roots
    c = host_ctx(8, 2, 16, max_tree_nodes=256)
    parents = np.concatenate(trees)
    off = np.cumsum([0] + [len(t) for t in trees[:-1]])
    c.plan([len(t) for t in trees], [7] * len(trees), [1] * len(trees), off, parents)
    words = c.get_tree_mask()
    pos = 0
    for t in trees:
        n = len(t)
        W64 = (n + 63) // 64
        for i in range(n):
            anc = set()
            node = i
            while node >= 0:
                anc.add(node)
                node = int(t[node])
            row = words[pos + i * W64 : pos + (i + 1) * W64]
            got = {j for j in range(n) if (int(row[j // 64]) >> (j % 64)) & 1}
            assert got == anc
            assert all(int(row[j // 64]) >> (j % 64) == 0 for j in [n - 1 + 1] if j % 64)  # no bits beyond n
        pos += n * W64
    assert pos == len(words)


def coverage_check(batch, ctx, info):
    """Every (request, kv head, new token, visible 128-key tile) is covered exactly once;
    no tile above a token's causal frontier is needed; workers partition the tasks."""
    tasks = ctx.get_tasks()
    off = ctx.get_worker_offsets()
    assert off[0] == 0 and off[-1] == len(tasks) and np.all(np.diff(off) >= 0)
    assert len(off) == info.num_workers + 1
    G = batch.num_q_heads // batch.num_kv_heads
    merges = ctx.get_merge_units()
    for r in range(batch.num_requests):
        n, h = int(batch.q_len[r]), int(batch.kv_len[r])
        for g in range(batch.num_kv_heads):
            sel = tasks[(tasks["req"] == r) & (tasks["kv_head"] == g)]
            need = [-(-(h + i + 1) // 128) for i in range(n)]  # tiles row i needs
            cover = [np.zeros(need[i], dtype=np.int32) for i in range(n)]
            for t in sel:
                assert t["ntok"] >= 1 and t["tok0"] >= 0 and t["tok0"] + t["ntok"] <= n
                assert 0 <= t["kt_lo"] < t["kt_hi"]
                # the run never goes beyond what the tile's last row can see
                assert t["kt_hi"] <= -(-(h + t["tok0"] + t["ntok"]) // 128)
                assert t["kind"] == (1 if t["ntok"] * G <= 16 else 0)
                for i in range(t["tok0"], t["tok0"] + t["ntok"]):
                    hi = min(t["kt_hi"], need[i])
                    if hi > t["kt_lo"]:
                        cover[i][t["kt_lo"] : hi] += 1
            for i in range(n):
                assert np.all(cover[i] == 1), (r, g, i)
    # split bookkeeping: partial rows are disjoint and every split unit has a merge entry
    used = np.zeros(max(int(info.partial_rows), 1), dtype=np.int32)
    for t in tasks[tasks["part"] >= 0]:
        rows = t["ntok"] * G
        used[t["part"] : t["part"] + rows] += 1
    assert np.all(used[: info.partial_rows] == 1)
    for m in merges:
        rows = m["ntok"] * G
        sel = tasks[(tasks["req"] == m["req"]) & (tasks["kv_head"] == m["kv_head"]) & (tasks["tok0"] == m["tok0"])]
        assert len(sel) == m["nsplit"] >= 2
        assert sorted(sel["part"]) == [m["part0"] + c * rows for c in range(m["nsplit"])]
        # chunks tile the visible range without gaps
        order = np.argsort(sel["kt_lo"])
        assert sel["kt_lo"][order][0] == 0
        assert np.all(sel["kt_lo"][order][1:] == sel["kt_hi"][order][:-1])
    unsplit = tasks[tasks["part"] < 0]
    keys = {(t["req"], t["kv_head"], t["tok0"]) for t in unsplit}
    assert len(keys) == len(unsplit)
    assert info.num_tasks == len(tasks) and info.num_merge_units == len(merges)
    # the queue free workers take tasks from is a permutation of the task table
    queue = ctx.get_queue()
    assert sorted(queue.tolist()) == list(range(len(tasks)))


@pytest.mark.parametrize("name", ["tiny_hybrid", "decode_only", "splitfuse_mix", "verify_trees", "full_mix"])
def test_balanced_plan_invariants_on_configs(name):
    b = W.CONFIGS[name]()
    c = host_ctx(b.num_q_heads, b.num_kv_heads, b.page_size)
    info = c.plan_batch(b)
    coverage_check(b, c, info)
    assert info.useful_flops == W.useful_flops(b)
    assert info.kv_bytes == W.kv_bytes(b)
    # balance: snake dealing of a sorted list keeps every worker within one task of the mean
    if info.num_tasks >= 4 * info.num_workers:
        assert info.load_max <= info.load_mean + info.max_task_cost + 1e-3
    # determinism
    t1 = c.get_tasks().copy()
    c.plan_batch(b)
    assert np.array_equal(t1, c.get_tasks())


def test_queue_mixes_kinds_and_puts_long_tasks_early():
    """Balanced plans hand out dense and streaming tasks side by side, dense siblings together,
    and no long task is left for the end of the queue."""
    b = W.CONFIGS["splitfuse_mix"]()
    c = host_ctx(b.num_q_heads, b.num_kv_heads, b.page_size)
    info = c.plan_batch(b)
    tasks, queue = c.get_tasks(), c.get_queue()
    kinds = tasks["kind"][queue]
    ntiles = (tasks["kt_hi"] - tasks["kt_lo"])[queue]
    first = kinds[: info.num_workers]
    assert 0 < int(first.sum()) < info.num_workers  # both kinds among the first tasks handed out
    assert np.all(np.diff(ntiles[kinds == 1]) <= 0)  # streaming tasks: longest first
    # dense tasks: sibling q tiles of one (request, kv head) are handed out together (longest
    # first inside a group) except for the last tenth, which is in plain descending order
    dq = queue[kinds == 0]
    head = len(dq) - len(dq) // 10
    grp = tasks["req"][dq].astype(np.int64) * 64 + tasks["kv_head"][dq]
    dt = (tasks["kt_hi"] - tasks["kt_lo"])[dq]
    seen = set()
    for i in range(head):
        if i and grp[i] == grp[i - 1]:
            assert dt[i] <= dt[i - 1]
        else:
            assert int(grp[i]) not in seen  # a group appears as one run
            seen.add(int(grp[i]))
    assert np.all(np.diff(dt[head:]) <= 0)
    # the last tenth of the queue holds only tasks shorter than the median task
    tail = ntiles[-len(queue) // 10:]
    assert tail.max() <= np.median(ntiles)


def test_plan_edge_shapes():
    reqs = [(n, h, 0, None) for n in (1, 15, 16, 17, 127, 128, 129) for h in (0, 5, 128, 200)]
    b = W.custom("edges", 8, 2, 16, reqs, seed=1)
    for workers in (1, 3, 148):
        c = host_ctx(8, 2, 16, num_workers=workers)
        coverage_check(b, c, c.plan_batch(b))
    c = host_ctx(8, 2, 16, num_workers=8, workspace_bytes=(128 + 1) * 4 * 64)  # tiny workspace
    info = c.plan_batch(b)
    assert info.partial_rows <= 64
    coverage_check(b, c, info)


def test_splits_appear_for_long_decode_and_respect_max_splits():
    b = W.custom("long", 8, 1, 128, [(1, 60000, 0, None)], seed=2)
    c = host_ctx(8, 1, 128, max_splits=5)
    info = c.plan_batch(b)
    assert 2 <= info.num_tasks <= 5 and info.num_merge_units == 1
    coverage_check(b, c, info)


def test_default_split_bound_grows_when_few_streaming_units_exist():
    # two units (one request, two kv heads) on 148 workers: 74 splits each, one task per worker
    b = W.custom("one_long", 8, 2, 128, [(1, 1_000_000, 0, None)], seed=2)
    c = host_ctx(8, 2, 128, num_workers=148, max_pages_per_req=8192)
    info = c.plan_batch(b)
    assert info.num_tasks == 148 and int(c.get_merge_units()["nsplit"].max()) == 74
    coverage_check(b, c, info)
    # many units: the bound stays at 32
    b = W.custom("many", 8, 2, 128, [(1, 300_000, 0, None)] * 8 + [(1, 1_000_000, 0, None)], seed=2)
    c = host_ctx(8, 2, 128, num_workers=148, max_pages_per_req=8192)
    info = c.plan_batch(b)
    assert int(c.get_merge_units()["nsplit"].max()) <= 32
    coverage_check(b, c, info)


def test_paper_mode_equals_python_task_table_and_fig3b():
    q_len, kv_len = [300, 1, 16, 1], [0, 700, 900, 350]
    hq, hkv, C, tile = 6, 6, 4, 128
    c = host_ctx(hq, hkv, 16, plan_mode=xb.XY_PLAN_PAPER, tile_tokens=tile, num_workers=C)
    info = c.plan(q_len, kv_len, [0, 0, 1, 0], [-1, -1, 0, -1], W.chain_tree(16))
    tasks, off = c.get_tasks(), c.get_worker_offsets()
    assert info.num_merge_units == 0 and np.all(tasks["part"] == -1)
    # Fig. 3(b): 3 + 1 + 1 + 1 tile blocks, times headNum units
    assert len(tasks) == 6 * hkv
    blocks = [len(set(tasks[tasks["req"] == r]["tok0"])) for r in range(4)]
    assert blocks == [3, 1, 1, 1]
    want = TT.reorder(TT.decompose(TT.token_table(q_len, kv_len, tile), hkv), C)
    for w in range(C):
        got = [(int(t["req"]), int(t["kv_head"]), int(t["tok0"]), int(t["ntok"])) for t in tasks[off[w] : off[w + 1]]]
        exp = [(u.stage_id, u.head, u.row0, u.rows) for u in want[w]]
        assert got == exp
    # the first eight tiles of the sorted list went to workers 0,1,2,3,3,2,1,0
    units = TT.decompose(TT.token_table(q_len, kv_len, tile), hkv)
    order = sorted(range(len(units)), key=lambda k: -units[k].load)
    first8 = [units[k] for k in order[:8]]
    owners = []
    for u in first8:
        for w in range(C):
            if any((int(t["req"]), int(t["kv_head"]), int(t["tok0"])) == (u.stage_id, u.head, u.row0)
                   for t in tasks[off[w] : off[w + 1]]):
                owners.append(w)
    assert owners == [0, 1, 2, 3, 3, 2, 1, 0]
    coverage_check(W.custom("fig3b", hq, hkv, 16, [(300, 0, 0, None), (1, 700, 0, None),
                                                   (16, 900, 1, W.chain_tree(16)), (1, 350, 0, None)]), c, info)


def test_task_table_cache_reuses_equal_decompositions_bit_exactly():
    """A decode step moves every kvLen by one token; while no request crosses a 128-key tile the
    decomposition, hence the Task-Table, is unchanged: the plan comes from the cache and is
    bit-identical to a fresh context's plan.  Crossing a tile (or any other change) misses."""
    rng = np.random.default_rng(5)
    kv = rng.integers(200, 5000, size=24)
    kv = kv - (kv % 128) + rng.integers(1, 60, size=24)  # at least 60 steps before a tile ends
    reqs = [(1, int(x), 0, None) for x in kv] + [(700, 300, 0, None)]
    c = host_ctx(8, 2, 128)
    b0 = W.custom("s0", 8, 2, 128, reqs, seed=1)
    c.plan_batch(b0)
    assert c.plan_cache() == (0, 1)
    for step in range(1, 4):
        reqs_s = [(1, int(x) + step, 0, None) for x in kv] + [(700, 300, 0, None)]
        b = W.custom("s%d" % step, 8, 2, 128, reqs_s, seed=1)
        info = c.plan_batch(b)
        assert c.plan_cache() == (step, 1)
        fresh = host_ctx(8, 2, 128)
        info_f = fresh.plan_batch(b)
        assert np.array_equal(c.get_tasks(), fresh.get_tasks())
        assert np.array_equal(c.get_queue(), fresh.get_queue())
        assert np.array_equal(c.get_worker_offsets(), fresh.get_worker_offsets())
        assert np.array_equal(c.get_merge_units(), fresh.get_merge_units())
        assert (info.useful_flops, info.kv_bytes) == (info_f.useful_flops, info_f.kv_bytes)
        assert info.useful_flops == W.useful_flops(b)
        coverage_check(b, c, info)
    # one request crosses into its next key tile: different decomposition
    reqs_x = [(1, int(kv[0]) + 128, 0, None)] + [(1, int(x), 0, None) for x in kv[1:]] + [(700, 300, 0, None)]
    c.plan_batch(W.custom("x", 8, 2, 128, reqs_x, seed=1))
    assert c.plan_cache() == (3, 2)
    # back to the first shape: still cached
    c.plan_batch(b0)
    assert c.plan_cache() == (4, 2)
    # disabled: every plan is built
    assert c.plan_cache(0) == (4, 2)
    c.plan_batch(b0)
    assert c.plan_cache() == (4, 2)


def test_shared_prefix_groups_cover_every_key_once_and_reject_bad_groups():
    """A shared-prefix group turns the members' first `prefix` keys into tiles of one virtual
    request (read once) and leaves each member a task for its own keys; together they cover every
    (member, kv head, key tile) exactly once, and each member gets one merge unit with both
    families of partials."""
    b, groups = W.shared_prefix_decode(seed=3, num_groups=3, members=20, prefix=1024, suffix_hi=700,
                                       hq=8, hkv=2, page_size=64)
    c = host_ctx(8, 2, 64, max_requests=256)
    info = c.plan_batch(b, groups=groups)
    tasks, merges = c.get_tasks(), c.get_merge_units()
    R, G = b.num_requests, 4
    assert info.useful_flops == W.useful_flops(b)
    for gi, (first, n, prefix) in enumerate(groups):
        vt = tasks[tasks["req"] == R + gi]
        assert len(vt) and np.all(vt["part"] >= 0) and np.all(vt["kt_hi"] <= prefix // 128)
        for g in range(2):
            for m in range(n):
                r = first + m
                need = -(-(int(b.kv_len[r]) + 1) // 128)
                cover = np.zeros(need, np.int32)
                for t in vt[(vt["kv_head"] == g) & (vt["tok0"] <= m) & (m < vt["tok0"] + vt["ntok"])]:
                    cover[t["kt_lo"]: t["kt_hi"]] += 1
                own = tasks[(tasks["req"] == r) & (tasks["kv_head"] == g)]
                assert len(own) >= 1 and np.all(own["part"] >= 0) and own["kt_lo"].min() == prefix // 128
                for t in own:
                    cover[t["kt_lo"]: t["kt_hi"]] += 1
                assert np.all(cover == 1), (r, g)
                mu = merges[(merges["req"] == r) & (merges["kv_head"] == g)]
                assert len(mu) == 1 and mu["nsplit"][0] == len(own) and mu["nsplit1"][0] >= 1
                assert mu["stride1"][0] % G == 0
    # the queue is still a permutation; partial rows are disjoint
    assert sorted(c.get_queue().tolist()) == list(range(len(tasks)))
    used = np.zeros(int(info.partial_rows), np.int32)
    for t in tasks[tasks["part"] >= 0]:
        used[t["part"]: t["part"] + t["ntok"] * G] += 1
    assert np.all(used == 1)
    # bad groups
    def code(gs):
        with pytest.raises(xb.XYAttnError) as e:
            c.plan_batch(b, groups=gs)
        return e.value.code
    assert code([(0, 20, 1000)]) == xb.XY_ERR_INVALID_ARG         # prefix not a multiple of 128
    assert code([(0, 20, 1024), (10, 5, 1024)]) == xb.XY_ERR_INVALID_ARG  # overlap
    assert code([(50, 20, 1024)]) == xb.XY_ERR_INVALID_ARG        # range beyond the batch
    assert code([(0, 20, 4096)]) == xb.XY_ERR_INVALID_ARG         # prefix longer than a member's kv_len
    pb = W.custom("p", 8, 2, 64, [(5, 2000, 0, None), (1, 2000, 0, None)], seed=1)
    with pytest.raises(xb.XYAttnError) as e:
        c.plan_batch(pb, groups=[(0, 2, 1024)])                   # a prefill request in a group
    assert e.value.code == xb.XY_ERR_INVALID_ARG


def test_queue_keeps_sibling_dense_tiles_of_group_requests_together():
    """The dense tiles of a shared-prefix group's virtual request (request index >= num_reqs) are
    regrouped like every other dense tile: in the queue, all but the last tenth of the dense tasks
    of one (request, kv head) follow each other without another key in between."""
    b, groups = W.shared_prefix_decode(seed=1, num_groups=2, members=32, prefix=8192, suffix_hi=512,
                                       hq=32, hkv=8, page_size=128)
    c = host_ctx(32, 8, 128, max_requests=256)
    c.plan_batch(b, groups=groups)
    tasks, queue = c.get_tasks(), c.get_queue()
    dense = [int(q) for q in queue if tasks[int(q)]["kind"] == 0]
    assert len(dense) > 20 and max(int(tasks[q]["req"]) for q in dense) >= b.num_requests
    head = dense[: len(dense) - len(dense) // 10]
    keys = [(int(tasks[q]["req"]), int(tasks[q]["kv_head"])) for q in head]
    closed = set()
    for k, key in enumerate(keys):
        if k and key != keys[k - 1]:
            closed.add(keys[k - 1])
        assert key not in closed, "tiles of %r are not adjacent in the queue" % (key,)


def test_debug_block_table_check_on_the_host():
    """The validation aid: a host copy of the block table is checked against the plan, every entry
    a request uses must lie in [0, num_pages) and fit the row; unused entries (-1) are ignored."""
    b = W.config1_tiny()
    c = host_ctx(8, 2, 16)
    with pytest.raises(xb.XYAttnError) as e:
        c.debug_check_block_table(b.block_table, b.num_pages)
    assert e.value.code == xb.XY_ERR_NOT_PLANNED
    c.plan_batch(b)
    c.debug_check_block_table(b.block_table, b.num_pages)   # rows carry -1 beyond what a request uses
    need = -(-(int(b.kv_len[2]) + int(b.q_len[2])) // 16)
    for bad in (-1, b.num_pages, 2 ** 31 - 1):
        bt = b.block_table.copy()
        bt[2, need - 1] = bad
        with pytest.raises(xb.XYAttnError) as e:
            c.debug_check_block_table(bt, b.num_pages)
        assert e.value.code == xb.XY_ERR_INVALID_ARG and "request 2" in str(e.value)
        bt[2, need - 1] = b.block_table[2, need - 1]
        bt[2, need:] = bad                                   # beyond the request's last page: not read
        c.debug_check_block_table(bt, b.num_pages)
    with pytest.raises(xb.XYAttnError) as e:                 # a row too short for the longest request
        c.debug_check_block_table(b.block_table[:, : need - 1], b.num_pages)
    assert e.value.code == xb.XY_ERR_INVALID_ARG
    # groups: the virtual request reads the first member's row
    gb, groups = W.shared_prefix_decode(seed=3, num_groups=2, members=8, prefix=256, suffix_hi=100, hq=8, hkv=2,
                                        page_size=64)
    g = host_ctx(8, 2, 64)
    g.plan_batch(gb, groups=groups)
    g.debug_check_block_table(gb.block_table, gb.num_pages)
    with pytest.raises(xb.XYAttnError):
        g.debug_inject(-1, 0)
    g.debug_inject(0, -1)


def test_merge_units_are_partitioned_into_merge_kernel_and_inline_units():
    """Split units of at most 16 packed rows are merged inside the attention kernel and sit behind
    the merge kernel's units in the unit list; the SIMT kernel and paper mode leave every unit to
    the merge kernel.  The covering invariants do not depend on the order."""
    rng = np.random.default_rng(3)
    reqs = [(1, 30000, 0, None), (1, 9000, 0, None), (300, 20000, 0, None), (2, 50000, 1, [-1, 0]),
            (40, 60000, 1, W.random_tree(rng, 40, 6))]
    b = W.custom("partition", 8, 2, 128, reqs, seed=3)
    c = host_ctx(8, 2, 128)
    info = c.plan_batch(b)
    mu = c.get_merge_units()
    rows = mu["ntok"] * 4
    n_launch = info.num_merge_units - info.num_inline_merge_units
    assert info.num_inline_merge_units > 0 and n_launch > 0
    assert np.all(rows[:n_launch] > 16) and np.all(rows[n_launch:] <= 16)
    coverage_check(b, c, info)
    r = host_ctx(8, 2, 128, kernel=xb.XY_KERNEL_REFERENCE)
    assert r.plan_batch(b).num_inline_merge_units == 0


@pytest.mark.parametrize("name", ["splitfuse_mix", "verify_trees", "full_mix"])
def test_pair_plans_put_dense_tasks_of_up_to_512_rows_first(name):
    """XY_KERNEL_PAIR plans for the CTA-pair dense kernel: dense tasks hold up to 512 packed rows
    (two 256-row sub-tiles, each split over two CTAs) and come first in the queue, siblings
    together; the streaming tasks follow in descending order of length.  XY_KERNEL_AUTO keeps
    256-row tasks in one mixed queue.  Coverage holds for both."""
    b = W.CONFIGS[name]()
    G = b.num_q_heads // b.num_kv_heads
    for kernel, max_rows in ((xb.XY_KERNEL_PAIR, 512), (xb.XY_KERNEL_AUTO, 256)):
        c = host_ctx(b.num_q_heads, b.num_kv_heads, b.page_size, kernel=kernel)
        info = c.plan_batch(b)
        coverage_check(b, c, info)
        tasks, queue = c.get_tasks(), c.get_queue()
        dense = tasks[tasks["kind"] == 0]
        assert int((dense["ntok"] * G).max()) <= max_rows
        if kernel == xb.XY_KERNEL_PAIR:
            assert int((dense["ntok"] * G).max()) > 256
            kinds = tasks["kind"][queue]
            nd = int((kinds == 0).sum())
            assert np.all(kinds[:nd] == 0) and np.all(kinds[nd:] == 1)
            ntiles = (tasks["kt_hi"] - tasks["kt_lo"])[queue]
            assert np.all(np.diff(ntiles[nd:]) <= 0)
