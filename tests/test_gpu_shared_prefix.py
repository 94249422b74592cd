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
