"""Shared-prefix ("cascade") decode on the GPU: groups of decode requests whose first tokens are
the same pages.  The grouped plan must give the same attention as the fp64 oracle (which knows
nothing about groups: it reads every request through its own block-table row)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_18106_b200 import binding as xb
from paper_2412_18106_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu

KERNELS = [xb.XY_KERNEL_AUTO, xb.XY_KERNEL_REFERENCE, xb.XY_KERNEL_MMA]


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("members,hq,hkv", [(3, 8, 2), (20, 8, 2), (40, 16, 2), (70, 4, 4)])
def test_grouped_plan_matches_oracle(kernel, members, hq, hkv):
    # 3 x 4 = 12 packed rows: streaming group tile; 20 x 4 = 80: one sub-tile; 40 x 8 = 320 rows:
    # several dense tiles; 70 x 1 = 70 rows with one head per kv head
    assert torch.cuda.is_available()
    b, groups = W.shared_prefix_decode(seed=members, num_groups=2, members=members, prefix=512, suffix_hi=300,
                                       hq=hq, hkv=hkv, page_size=32)
    # a few ungrouped requests around the groups
    t = W.make_tensors(b)
    ctx = H.make_ctx(b, kernel=kernel, max_requests=512)
    ctx.plan_batch(b, groups=groups)
    O, LSE = H.run_gpu(b, t, ctx=ctx)
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    H.check_against_oracle(O, LSE, O_ref, LSE_ref, "shared prefix %d" % members)
    if kernel == xb.XY_KERNEL_AUTO:
        O2, LSE2 = H.run_gpu(b, t, ctx=ctx)
        assert np.array_equal(O, O2) and np.array_equal(LSE, LSE2)
    ctx.close()


def test_groups_beside_other_requests_and_member_without_suffix():
    rng = np.random.default_rng(5)
    # request order: a prefill, a group of 10 (one member with kv_len == prefix), a tree, decodes
    reqs = [(50, 100, 0, None)] + [(1, 256 + (0 if k == 3 else int(rng.integers(1, 200))), 0, None) for k in range(10)]
    reqs += [(9, 400, 1, W.random_tree(rng, 9, 4)), (1, 777, 0, None), (1, 5, 0, None)]
    b = W.custom("mixed_groups", 8, 2, 16, reqs, seed=2)
    npre = 256 // 16
    for r in range(2, 11):
        b.block_table[r, :npre] = b.block_table[1, :npre]
    t = W.make_tensors(b)
    ctx = H.make_ctx(b)
    ctx.plan_batch(b, groups=[(1, 10, 256)])
    O, LSE = H.run_gpu(b, t, ctx=ctx)
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    H.check_against_oracle(O, LSE, O_ref, LSE_ref, "mixed groups")
    ctx.close()


@pytest.mark.parametrize("seed", range(8))
def test_random_groups(seed):
    """Random mixes: several groups of random size and prefix length between ungrouped prefill,
    decode and verify requests; random head ratio, page size and worker count."""
    rng = np.random.default_rng(1000 + seed)
    hkv = int(rng.choice([1, 2, 4]))
    G = int(rng.choice([1, 2, 4, 8]))
    page = int(rng.choice([16, 32, 64, 128]))
    reqs, groups = [], []
    for _ in range(int(rng.integers(1, 4))):
        for _ in range(int(rng.integers(0, 3))):  # ungrouped requests before the group
            k = rng.random()
            if k < 0.4:
                reqs.append((1, int(rng.integers(1, 900)), 0, None))
            elif k < 0.7:
                reqs.append((int(rng.integers(2, 90)), int(rng.integers(0, 500)), 0, None))
            else:
                n = int(rng.integers(2, 20))
                reqs.append((n, int(rng.integers(0, 500)), 1, W.random_tree(rng, n, 5)))
        n = int(rng.integers(1, 45))
        prefix = 128 * int(rng.integers(1, 9))
        groups.append((len(reqs), n, prefix))
        for _ in range(n):
            reqs.append((1, prefix + int(rng.integers(0, 400)), 0, None))
    b = W.custom("rgroups%d" % seed, hkv * G, hkv, page, reqs, seed=seed)
    for first, n, prefix in groups:
        npre = prefix // page
        for r in range(first + 1, first + n):
            b.block_table[r, :npre] = b.block_table[first, :npre]
    t = W.make_tensors(b)
    ctx = H.make_ctx(b, num_workers=int(rng.choice([1, 5, 148])), max_requests=512)
    ctx.plan_batch(b, groups=groups)
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    O, LSE = H.run_gpu(b, t, ctx=ctx)
    H.check_against_oracle(O, LSE, O_ref, LSE_ref, "random groups %d" % seed)
    O2, LSE2 = H.run_gpu(b, t, ctx=ctx)
    assert np.array_equal(O, O2) and np.array_equal(LSE, LSE2)
    ctx.close()


def test_groups_found_from_the_block_table():
    """groups="auto": the groups are read off the block table, the plan uses them, the result is
    the oracle's."""
    b, groups = W.shared_prefix_decode(seed=21, num_groups=3, members=24, prefix=1024, suffix_hi=400, hq=16, hkv=4,
                                       page_size=64)
    t = W.make_tensors(b)
    ctx = H.make_ctx(b, max_requests=512)
    plain_tasks = ctx.plan_batch(b).num_tasks
    info = ctx.plan_batch(b, groups="auto")
    assert info.num_tasks != plain_tasks and info.num_merge_units >= 3 * 24
    O, LSE = H.run_gpu(b, t, ctx=ctx)
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    H.check_against_oracle(O, LSE, O_ref, LSE_ref, "auto groups")
    ctx.close()
