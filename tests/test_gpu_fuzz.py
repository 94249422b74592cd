"""Randomised batches: head ratios, page sizes, worker counts and request mixes drawn at random;
the meta-kernel against the fp64 oracle on every element, and bit-identical when repeated (a race
between roles, tasks or workers would show as a difference between the two launches)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_18106_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu


def random_batch(seed):
    rng = np.random.default_rng(seed)
    hkv = int(rng.choice([1, 2, 4]))
    G = int(rng.choice([1, 2, 4, 7, 8, 16]))
    page = int(rng.choice([16, 32, 64, 128]))
    reqs = []
    for _ in range(int(rng.integers(1, 28))):
        kind = rng.random()
        kv = int(rng.integers(0, 1500)) if rng.random() < 0.8 else int(rng.integers(1500, 9000))
        if kind < 0.35:
            reqs.append((1, max(kv, 1), 0, None))
        elif kind < 0.7:
            reqs.append((int(rng.integers(2, 200)), kv, 0, None))
        else:
            n = int(rng.integers(2, 48))
            reqs.append((n, kv, 1, W.random_tree(rng, n, int(rng.integers(1, 9)))))
    workers = int(rng.choice([1, 2, 7, 31, 148]))
    return W.custom("fuzz%d" % seed, hkv * G, hkv, page, reqs, seed=seed), workers


@pytest.mark.parametrize("seed", range(16))
def test_random_batch_matches_oracle_and_repeats_bitwise(seed):
    assert torch.cuda.is_available()
    b, workers = random_batch(seed)
    t = W.make_tensors(b)
    ctx = H.make_ctx(b, num_workers=workers, max_tree_nodes=64)
    ctx.plan_batch(b)
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    O1, L1 = H.run_gpu(b, t, ctx=ctx)
    H.check_against_oracle(O1, L1, O_ref, LSE_ref, "fuzz %d" % seed)
    O2, L2 = H.run_gpu(b, t, ctx=ctx)
    assert np.array_equal(O1, O2) and np.array_equal(L1, L2)
    ctx.close()
