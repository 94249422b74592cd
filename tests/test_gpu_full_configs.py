"""Parity at the full benchmark sizes, in the launch configuration bench.py times: sampled
outputs (request, q head, new-token row) of configurations 2-5 against the fp64 oracle, which
computes each sampled row on its own.  Samples are random rows plus, for every request, its
first and last row (diagonal / tail / tree-corner cases) on two heads."""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_18106_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu


def sample_rows(batch, rng, n_random):
    req, head, row = [], [], []
    for r in range(batch.num_requests):
        n = int(batch.q_len[r])
        for i in {0, n - 1}:
            for a in (0, batch.num_q_heads - 1):
                req.append(r), head.append(a), row.append(i)
    tok_req = np.repeat(np.arange(batch.num_requests), batch.q_len)
    q_start = batch.q_start
    for t in rng.integers(0, batch.total_q, size=n_random):
        r = int(tok_req[t])
        req.append(r), head.append(int(rng.integers(0, batch.num_q_heads))), row.append(int(t - q_start[r]))
    return np.array(req, np.int32), np.array(head, np.int32), np.array(row, np.int32)


@pytest.mark.parametrize("name", ["decode_only", "splitfuse_mix", "verify_trees", "full_mix"])
def test_full_size_sampled_parity(name):
    batch = W.CONFIGS[name](seed=0)
    tensors = W.make_tensors(batch)
    O, LSE = H.run_gpu(batch, tensors)  # default context = what bench.py launches
    assert not np.isnan(O).any() and not np.isnan(LSE).any()
    rng = np.random.default_rng(7)
    req, head, row = sample_rows(batch, rng, 96)
    O_ref, LSE_ref = oracle.attention_rows(batch, tensors, H.SCALE, req, head, row)
    x = batch.q_start[req] + row
    H.check_against_oracle(O[x, head], LSE[x, head], O_ref, LSE_ref, name)
    # properties that hold at any size: every row is a convex combination of V rows, so
    # |O| is bounded by the largest |V|; LSE of a row with c allowed keys is >= its max score
    vmax = float(tensors.v_pool.float().abs().max())
    assert np.abs(O).max() <= vmax + 1e-2
