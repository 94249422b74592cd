"""GPU parity of the experimental CTA-pair dense kernel (XY_KERNEL_PAIR: tcgen05 cta_group::2,
up to 512 packed rows per task, streaming tasks in a second launch) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_18106_b200 import binding as xb
from paper_2412_18106_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    xb.load()


def _tree(seed, n, width):
    return W.random_tree(np.random.default_rng(seed), n, width)


CASES = {
    # G = 4: 64 tokens are 256 packed rows -> four slots of 64 rows
    "one_tile": (128, [(64, 0, 0, None)]),
    "full_512_rows": (128, [(128, 0, 0, None)]),
    "prefix_and_ragged_rows": (128, [(128, 300, 0, None), (70, 0, 0, None), (33, 150, 0, None)]),
    "several_tasks_per_request": (64, [(300, 1000, 0, None), (129, 77, 0, None)]),
    "trees": (32, [(40, 500, 1, _tree(1, 40, 6)), (20, 300, 1, _tree(2, 20, 6)), (64, 0, 1, _tree(3, 64, 8))]),
    "small_pages_mixed_with_decode": (16, [(64, 0, 0, None), (64, 128, 0, None), (1, 300, 0, None),
                                          (4, 200, 1, _tree(4, 4, 2)), (1, 5, 0, None)]),
    "split_kv": (128, [(200, 30000, 0, None), (1, 9000, 0, None)]),
}


@pytest.mark.parametrize("name", list(CASES))
def test_pair_kernel_matches_oracle(name):
    page, reqs = CASES[name]
    b = W.custom(name, 8, 2, page, reqs, seed=3)
    t = W.make_tensors(b)
    ctx = H.make_ctx(b, kernel=xb.XY_KERNEL_PAIR, num_workers=148, max_tree_nodes=128)
    info = ctx.plan_batch(b)
    O, LSE = H.run_gpu(b, t, ctx=ctx)
    # dense tasks in the pair launch, streaming tasks (if any) in the single-CTA launch, the merge
    # kernel for the units the attention kernels do not merge themselves
    stream = info.num_tasks - info.num_dense_tasks
    want = 1 + (1 if stream > 0 else 0) + (1 if info.num_merge_units > info.num_inline_merge_units else 0)
    assert ctx.last_launches() == want
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    H.check_against_oracle(O, LSE, O_ref, LSE_ref, name)


def test_pair_kernel_other_head_ratios():
    for hq, hkv in ((32, 8), (28, 4), (16, 1)):
        reqs = [(90, 700, 0, None), (1, 260, 0, None), (17, 0, 0, None)]
        H.parity(W.custom("pair_heads%d_%d" % (hq, hkv), hq, hkv, 64, reqs, seed=hq), kernel=xb.XY_KERNEL_PAIR,
                 num_workers=148)


def test_pair_kernel_needs_bf16_balanced_even_workers():
    for kw in (dict(kv_dtype=xb.XY_KV_FP8_E4M3), dict(plan_mode=xb.XY_PLAN_PAPER), dict(num_workers=7)):
        with pytest.raises(xb.XYAttnError):
            xb.XYAttn(8, 2, 64, kernel=xb.XY_KERNEL_PAIR, **kw)


def test_pair_kernel_wait_that_runs_out_reports_and_context_stays_usable():
    """A producer that skips one fill makes the issuer's wait run out: the launch ends with
    XY_ERR_DEVICE_TIMEOUT in the status word, and the next run on the same context is correct."""
    b = W.custom("pair_fail", 8, 2, 128, [(128, 1000, 0, None)], seed=5)
    t = W.make_tensors(b)
    ctx = H.make_ctx(b, kernel=xb.XY_KERNEL_PAIR, num_workers=148)
    ctx.plan_batch(b)
    ctx.debug_inject(wait_limit_polls=1 << 14, skip_fill=3)
    d = H.DeviceBatch(b, t)
    ctx.run(d.q, d.k_pool, d.v_pool, d.block_table, H.SCALE, d.o, d.lse)
    torch.cuda.synchronize()
    assert ctx.device_status() == xb.XY_ERR_DEVICE_TIMEOUT
    ctx.debug_inject(wait_limit_polls=0, skip_fill=-1)
    O, LSE = H.run_gpu(b, t, ctx=ctx)
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    H.check_against_oracle(O, LSE, O_ref, LSE_ref, "pair after a timed-out run")


@pytest.mark.parametrize("seed", range(8))
def test_pair_kernel_random_batches_match_oracle_and_repeat_bitwise(seed):
    """Random head ratios, page sizes, even worker counts and request mixes on the pair kernel."""
    rng = np.random.default_rng(100 + seed)
    hkv = int(rng.choice([1, 2, 4]))
    G = int(rng.choice([1, 2, 4, 7, 8, 16]))
    page = int(rng.choice([16, 32, 64, 128]))
    reqs = []
    for _ in range(int(rng.integers(1, 20))):
        kind = rng.random()
        kv = int(rng.integers(0, 1500)) if rng.random() < 0.8 else int(rng.integers(1500, 6000))
        if kind < 0.3:
            reqs.append((1, max(kv, 1), 0, None))
        elif kind < 0.7:
            reqs.append((int(rng.integers(2, 300)), kv, 0, None))
        else:
            n = int(rng.integers(2, 48))
            reqs.append((n, kv, 1, W.random_tree(rng, n, int(rng.integers(1, 9)))))
    workers = int(rng.choice([2, 6, 30, 148]))
    b = W.custom("pair_fuzz%d" % seed, hkv * G, hkv, page, reqs, seed=seed)
    t = W.make_tensors(b)
    ctx = H.make_ctx(b, kernel=xb.XY_KERNEL_PAIR, num_workers=workers, max_tree_nodes=64)
    ctx.plan_batch(b)
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    O1, L1 = H.run_gpu(b, t, ctx=ctx)
    H.check_against_oracle(O1, L1, O_ref, LSE_ref, "pair fuzz %d" % seed)
    O2, L2 = H.run_gpu(b, t, ctx=ctx)
    assert np.array_equal(O1, O2) and np.array_equal(L1, L2)
    ctx.close()
