"""GPU parity: the CUDA path through the C-ABI against the fp64 CPU oracle, element by
element on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_18106_b200 import binding as xb
from paper_2412_18106_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu

KERNELS = [xb.XY_KERNEL_AUTO, xb.XY_KERNEL_REFERENCE, xb.XY_KERNEL_MMA]
KNAMES = {xb.XY_KERNEL_AUTO: "auto", xb.XY_KERNEL_REFERENCE: "reference", xb.XY_KERNEL_MMA: "mma"}


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    xb.load()  # fails loudly if the extension is missing


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAMES[k])
def test_config1_tiny_hybrid(kernel):
    H.parity(W.config1_tiny(), kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAMES[k])
@pytest.mark.parametrize("page", [16, 32, 64, 128])
def test_page_sizes(kernel, page):
    rng = np.random.default_rng(page)
    reqs = [(70, 0, 0, None), (33, 150, 0, None), (1, 257, 0, None), (1, 5, 0, None),
            (20, 300, 1, W.random_tree(rng, 20, 6)), (2, 129, 1, [-1, 0])]
    H.parity(W.custom("pages%d" % page, 8, 2, page, reqs, seed=page), kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAMES[k])
def test_q_len_straddling_tile_and_page_boundaries(kernel):
    reqs = [(n, h, 0, None) for n in (1, 15, 16, 17, 127, 128, 129) for h in (0, 77)]
    H.parity(W.custom("straddle", 8, 2, 16, reqs, seed=7), kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAMES[k])
def test_tree_sizes(kernel):
    rng = np.random.default_rng(9)
    reqs = [(n, 190, 1, W.random_tree(rng, n, 8)) for n in (1, 63, 64, 65)]
    reqs.append((5, 0, 1, [-1, -1, 0, 1, -1]))  # several roots, no history
    H.parity(W.custom("trees", 8, 2, 32, reqs, seed=9), kernel=kernel, max_tree_nodes=128)


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAMES[k])
@pytest.mark.parametrize("heads", [(28, 4), (32, 8), (64, 8), (4, 4), (16, 1)])
def test_head_ratios(kernel, heads):
    hq, hkv = heads
    rng = np.random.default_rng(hq)
    reqs = [(40, 100, 0, None), (1, 700, 0, None), (9, 260, 1, W.random_tree(rng, 9, 4)), (1, 0, 0, None)]
    H.parity(W.custom("heads%d_%d" % heads, hq, hkv, 64, reqs, seed=hq), kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAMES[k])
def test_split_kv_long_decode_and_verify(kernel):
    rng = np.random.default_rng(12)
    reqs = [(1, 9000, 0, None), (1, 4097, 0, None), (12, 6000, 1, W.random_tree(rng, 12, 5)), (200, 3000, 0, None)]
    b = W.custom("split", 8, 2, 128, reqs, seed=12)
    ctx = H.make_ctx(b, kernel=kernel, num_workers=148)
    info = ctx.plan_batch(b)
    assert info.num_merge_units > 0
    t = W.make_tensors(b)
    O, LSE = H.run_gpu(b, t, ctx=ctx)
    # decode / tiny-verify units are merged inside the attention kernel (not by the SIMT kernel,
    # which leaves every unit to the merge kernel); the merge kernel runs only for the others
    inline = info.num_inline_merge_units
    assert (inline > 0) == (kernel != xb.XY_KERNEL_REFERENCE)
    assert ctx.last_launches() == (2 if info.num_merge_units > inline else 1)
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    H.check_against_oracle(O, LSE, O_ref, LSE_ref, "split")


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAMES[k])
def test_fused_qkv_stride_and_paper_plan(kernel):
    b = W.config1_tiny()
    t = W.make_tensors(b, fused_qkv=True)
    assert t.q.stride(0) == (8 + 4) * 128
    O, LSE = H.run_gpu(b, t, kernel=kernel, plan_mode=xb.XY_PLAN_PAPER, tile_tokens=24)
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    H.check_against_oracle(O, LSE, O_ref, LSE_ref, "fused+paper")


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAMES[k])
def test_tail_and_unused_pages_poisoned(kernel):
    b = W.config1_tiny()
    clean = W.make_tensors(b)
    poisoned = W.make_tensors(b, tail_fill=1e30)
    O1, L1 = H.run_gpu(b, clean, kernel=kernel)
    O2, L2 = H.run_gpu(b, poisoned, kernel=kernel)
    assert np.array_equal(O1, O2) and np.array_equal(L1, L2)


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAMES[k])
def test_run_twice_and_page_permutation_are_bitwise_stable(kernel):
    b = W.config1_tiny()
    t = W.make_tensors(b)
    ctx = H.make_ctx(b, kernel=kernel)
    ctx.plan_batch(b)
    O1, L1 = H.run_gpu(b, t, ctx=ctx)
    O2, L2 = H.run_gpu(b, t, ctx=ctx)
    assert np.array_equal(O1, O2) and np.array_equal(L1, L2)
    rng = np.random.default_rng(5)
    perm = rng.permutation(b.num_pages)
    b2 = W.config1_tiny()
    bt = b.block_table.copy()
    bt[bt >= 0] = perm[bt[bt >= 0]]
    b2.block_table = bt
    k2, v2 = torch.empty_like(t.k_pool), torch.empty_like(t.v_pool)
    k2[torch.from_numpy(perm)] = t.k_pool
    v2[torch.from_numpy(perm)] = t.v_pool
    O3, L3 = H.run_gpu(b2, W.Tensors(q=t.q, k_pool=k2, v_pool=v2), ctx=ctx)
    assert np.array_equal(O1, O3) and np.array_equal(L1, L3)


def test_block_table_gather_is_bit_exact():
    b = W.config1_tiny()
    t = W.make_tensors(b)
    ctx = H.make_ctx(b)
    ctx.plan_batch(b)
    d = H.DeviceBatch(b, t)
    for r in range(b.num_requests):
        L = int(b.q_len[r] + b.kv_len[r])
        for g in range(b.num_kv_heads):
            ok = torch.zeros((L, 128), dtype=torch.bfloat16, device="cuda")
            ov = torch.zeros((L, 128), dtype=torch.bfloat16, device="cuda")
            ctx.debug_gather(r, g, d.k_pool, d.v_pool, d.block_table, ok, ov)
            torch.cuda.synchronize()
            K, V = oracle.gather(b, t, r, g)
            assert torch.equal(ok.cpu().view(torch.int16), K.view(torch.int16))
            assert torch.equal(ov.cpu().view(torch.int16), V.view(torch.int16))


def test_merge_kernel_matches_oracle_merge():
    rng = np.random.default_rng(1)
    S, rows = 5, 37
    Oc = rng.normal(size=(S, rows, 128)).astype(np.float32)
    Lc = rng.normal(scale=3.0, size=(S, rows)).astype(np.float32)
    Lc[2, 5] = -np.inf
    Lc[:, 7] = [-np.inf, 0.25, -np.inf, -np.inf, -np.inf]
    o = torch.zeros((rows, 128), dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(rows, dtype=torch.float32, device="cuda")
    xb.xy_attn_merge(torch.from_numpy(Oc).cuda(), torch.from_numpy(Lc).cuda(), o, lse)
    torch.cuda.synchronize()
    O_ref, L_ref = oracle.merge(Oc.astype(np.float64), Lc.astype(np.float64))
    assert np.abs(o.float().cpu().numpy() - O_ref).max() <= 2e-2
    assert np.all(np.abs(lse.cpu().numpy() - L_ref) <= 1e-3 * np.maximum(1, np.abs(L_ref)))


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAMES[k])
def test_invariants_hold_on_the_gpu(kernel):
    """Decode == last prefill row, chain tree == causal, chunked == unchunked, on the device."""
    total, page = 300, 16
    full = W.custom("full", 8, 2, page, [(total, 0, 0, None)], seed=31)
    tf = W.make_tensors(full)
    Of, Lf = H.run_gpu(full, tf, kernel=kernel)
    cuts = [0, 100, 117, 299, 300]
    specs = [(cuts[k + 1] - cuts[k], cuts[k], 0, None) for k in range(4)]
    specs[1] = (17, 100, 1, W.chain_tree(17))  # a chain tree in place of a causal chunk
    part = W.custom("part", 8, 2, page, specs, seed=31)
    for r in range(4):
        need = -(-(cuts[r + 1]) // page)
        part.block_table[r, :] = -1
        part.block_table[r, :need] = full.block_table[0, :need]
    part.num_pages = full.num_pages
    tp = W.Tensors(q=tf.q.clone(), k_pool=tf.k_pool, v_pool=tf.v_pool)
    Op, Lp = H.run_gpu(part, tp, kernel=kernel)
    assert np.abs(Op - Of).max() <= 2e-2 and np.abs(Op - Of).mean() <= 2e-3
    assert np.all(np.abs(Lp - Lf) <= 1e-3 * np.maximum(1, np.abs(Lf)))


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAMES[k])
def test_scale_and_zero_requests(kernel):
    b = W.custom("scale", 8, 2, 16, [(20, 50, 0, None), (1, 90, 0, None)], seed=3)
    t = W.make_tensors(b)
    O, LSE = H.run_gpu(b, t, scale=0.37, kernel=kernel)
    O_ref, LSE_ref = oracle.attention(b, t, 0.37)
    H.check_against_oracle(O, LSE, O_ref, LSE_ref, "scale")
    ctx = H.make_ctx(b, kernel=kernel)
    ctx.plan([], [], [], [])
    d = H.DeviceBatch(b, t)
    ctx.run(d.q, d.k_pool, d.v_pool, d.block_table, 1.0, d.o, d.lse)  # no-op
    torch.cuda.synchronize()
    assert ctx.last_launches() == 0 and torch.isnan(d.lse).all()


def test_run_error_paths_do_not_launch():
    b = W.config1_tiny()
    t = W.make_tensors(b)
    ctx = H.make_ctx(b)
    d = H.DeviceBatch(b, t)
    with pytest.raises(xb.XYAttnError) as e:
        ctx.run(d.q, d.k_pool, d.v_pool, d.block_table, 1.0, d.o, d.lse)
    assert e.value.code == xb.XY_ERR_NOT_PLANNED
    ctx.plan_batch(b)
    with pytest.raises(xb.XYAttnError) as e:
        ctx.run(t.q, d.k_pool, d.v_pool, d.block_table, 1.0, d.o, d.lse)  # CPU tensor
    assert e.value.code == xb.XY_ERR_INVALID_ARG
    rc = ctx.lib.xy_attn_run(ctx._ctx, 0, 1024, d.k_pool.data_ptr(), d.v_pool.data_ptr(), 1, 1, 1, 128,
                             d.block_table.data_ptr(), 1, 0, 1.0, d.o.data_ptr(), 1024, d.lse.data_ptr(), 0)
    assert rc == xb.XY_ERR_INVALID_ARG
    assert ctx.last_launches() == 0


def test_consecutive_steps_through_the_task_table_cache():
    """Three decode steps on one context: the second and third plan hit the Task-Table cache and
    leave the Task-Table on the device as it is (only the request facts are uploaded); each step
    must still match the oracle, including the step where a request enters a new key tile."""
    rng = np.random.default_rng(11)
    kv = [int(x) for x in rng.integers(130, 900, size=12)]
    kv[0] = 254  # crosses into its third 128-key tile at the third step
    tree = W.random_tree(rng, 12, 4)
    ctx = None
    for step in range(4):
        reqs = [(1, h + step, 0, None) for h in kv] + [(40, 100, 0, None), (12, 300 + step, 1, tree)]
        b = W.custom("steps%d" % step, 8, 2, 32, reqs, seed=3)
        t = W.make_tensors(b)
        if ctx is None:
            ctx = H.make_ctx(b)
        ctx.plan_batch(b)
        O, LSE = H.run_gpu(b, t, ctx=ctx)
        O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
        H.check_against_oracle(O, LSE, O_ref, LSE_ref, "step %d" % step)
    hits, misses = ctx.plan_cache()
    assert hits >= 1 and misses >= 2 and hits + misses == 4
    ctx.close()


@pytest.mark.parametrize("workers", [1, 2, 5])
def test_many_task_kind_transitions_per_worker(workers):
    """Few workers, many short tasks of alternating kinds: one-sub-tile dense tasks (<= 128 packed
    rows), two-sub-tile dense tasks and streaming tasks follow each other on the same worker in
    every order, which exercises the hand-over of the shared Q tiles and of tensor memory between
    tasks.  Whole output against the oracle, and bit-identical when repeated."""
    rng = np.random.default_rng(100 + workers)
    reqs = []
    for k in range(36):
        kind = k % 4
        if kind == 0:
            reqs.append((int(rng.integers(17, 33)), int(rng.integers(0, 400)), 0, None))   # one sub-tile
        elif kind == 1:
            reqs.append((1, int(rng.integers(1, 700)), 0, None))                          # streaming
        elif kind == 2:
            reqs.append((int(rng.integers(40, 64)), int(rng.integers(0, 300)), 0, None))   # two sub-tiles
        else:
            n = int(rng.integers(5, 30))
            reqs.append((n, int(rng.integers(10, 500)), 1, W.random_tree(rng, n, 5)))
    b = W.custom("transitions", 8, 2, 32, reqs, seed=workers)
    t = W.make_tensors(b)
    ctx = H.make_ctx(b, num_workers=workers)
    ctx.plan_batch(b)
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    first = None
    for _ in range(3):
        O, LSE = H.run_gpu(b, t, ctx=ctx)
        H.check_against_oracle(O, LSE, O_ref, LSE_ref, "transitions")
        if first is None:
            first = (O, LSE)
        assert np.array_equal(O, first[0]) and np.array_equal(LSE, first[1])
    ctx.close()


def test_maximum_sizes_one_million_token_context_and_largest_tree():
    """The largest shapes the path is meant for: a decode and a 64-node verify tree (the largest
    tree a context accepts by default) on contexts of about a million and 300 thousand tokens,
    next to a fresh one-token prefill; the long rows are split over every worker and merged."""
    rng = np.random.default_rng(99)
    reqs = [(1, 1_000_003, 0, None), (64, 300_001, 1, W.random_tree(rng, 64, 8)), (1, 0, 0, None)]
    b = W.custom("max_sizes", 8, 2, 128, reqs, seed=99, spare_frac=0.01)
    ctx = H.make_ctx(b)
    info = ctx.plan_batch(b)
    assert info.num_merge_units > 0
    t = W.make_tensors(b)
    O, LSE = H.run_gpu(b, t, ctx=ctx)
    ctx.close()
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    H.check_against_oracle(O, LSE, O_ref, LSE_ref, "max_sizes")
    # the comparison can see 128 lost keys even here: the same batch with kv_len - 128 (a valid
    # run on the same pool) must fail it
    reqs2 = [(1, 1_000_003 - 128, 0, None), (64, 300_001 - 128, 1, b.tree_parents(1)), (1, 0, 0, None)]
    b2 = W.custom("max_sizes_short", 8, 2, 128, reqs2, seed=99, spare_frac=0.01)
    b2.block_table, b2.num_pages = b.block_table, b.num_pages
    O_m, LSE_m = H.run_gpu(b2, t)
    with pytest.raises(AssertionError):
        H.check_against_oracle(O_m[:1], LSE_m[:1], O_ref[:1], LSE_ref[:1], "mutant, million-token row")
    with pytest.raises(AssertionError):
        H.check_against_oracle(O_m[1:65], LSE_m[1:65], O_ref[1:65], LSE_ref[1:65], "mutant, tree rows")


@pytest.mark.parametrize("hq,hkv,kv", [(8, 1, 400_000), (8, 2, 1_000_003)])
def test_single_long_context_is_cut_for_every_worker(hq, hkv, kv):
    """One decode request on a very long context: the default bound on splits grows so that every
    worker gets a key range (more than 32 partials per row: the wide merge kernel)."""
    b = W.custom("one_long", hq, hkv, 128, [(1, kv, 0, None)], seed=5, spare_frac=0.01)
    ctx = H.make_ctx(b)
    info = ctx.plan_batch(b)
    mu = ctx.get_merge_units()
    assert int(mu["nsplit"].max()) > 32 and 100 <= info.num_tasks <= 148
    t = W.make_tensors(b)
    O, LSE = H.run_gpu(b, t, ctx=ctx)
    O2, LSE2 = H.run_gpu(b, t, ctx=ctx)
    ctx.close()
    assert np.array_equal(O, O2) and np.array_equal(LSE, LSE2)
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    H.check_against_oracle(O, LSE, O_ref, LSE_ref, "one long context")


@pytest.mark.parametrize("world", [2, 4])
def test_kv_head_split_runs_on_strided_views_of_the_full_tensors(world):
    """The tensor-parallel style sharding on one device: shard k runs the unchanged xy_attn_run
    on kv heads [k Hkv/N, (k+1) Hkv/N) - strided views of the full pools, of Q and of O, no copies,
    no exchange - and the shards' outputs together are the oracle's result for the whole batch."""
    rng = np.random.default_rng(world)
    reqs = [(90, 200, 0, None), (1, 3000, 0, None), (17, 450, 1, W.random_tree(rng, 17, 5)), (1, 0, 0, None)]
    b = W.custom("headsplit", 16, 4, 64, reqs, seed=world)
    t = W.make_tensors(b)
    d = H.DeviceBatch(b, t)
    hkv, g = 4 // world, 4
    ctx = xb.XYAttn(hkv * g, hkv, 64, max_q_tokens=1 << 15, max_pages_per_req=1024)
    ctx.plan_batch(b)   # the plan depends on the requests only: one plan serves every shard
    for k in range(world):
        hs = slice(k * hkv * g, (k + 1) * hkv * g)
        lse_k = torch.full((b.total_q, hkv * g), float("nan"), dtype=torch.float32, device="cuda")
        ctx.run(d.q[:, hs], d.k_pool[:, k * hkv: (k + 1) * hkv], d.v_pool[:, k * hkv: (k + 1) * hkv], d.block_table,
                H.SCALE, d.o[:, hs], lse_k)
        d.lse[:, hs] = lse_k
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    ctx.close()
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    H.check_against_oracle(d.o.float().cpu().numpy().astype(np.float64), d.lse.cpu().numpy().astype(np.float64),
                           O_ref, LSE_ref, "kv-head split")
