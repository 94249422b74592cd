"""A short request stream through the whole front: chunk former (Section 3.1) -> xy_attn_plan ->
xy_attn_run, every chunk compared with the fp64 oracle.  One context serves all chunks, so the
Task-Table cache and the device-resident tables see changing decompositions."""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_18106_b200 import binding as xb
from paper_2412_18106_b200 import sched as xs
from paper_2412_18106_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_stream_of_chunks_matches_oracle():
    assert torch.cuda.is_available()
    rng = np.random.default_rng(21)
    s = xs.XYSched(budget_tokens=384, reserved_dv_tokens=48, max_requests=64)
    s.add_prefill(1, 700, 130)   # split over several chunks
    s.add_prefill(2, 90, 0)
    decodes = {10 + k: int(rng.integers(20, 1500)) for k in range(30)}
    for rid, kv in decodes.items():
        s.add_decode(rid, kv)
    s.add_verify(50, 640, W.random_tree(rng, 24, 6))
    s.add_verify(51, 77, W.chain_tree(5))
    ctx = None
    nchunks = 0
    while s.pending() != (0, 0):
        chunk = s.next_chunk()
        # decode requests come back with one more cached token, like a serving loop
        for e in chunk:
            if e["kind"] == xs.XY_SCHED_DECODE and nchunks < 2:
                s.add_decode(e["id"], e["kv_len"] + 1)
        reqs = [(e["q_len"], e["kv_len"], 1 if e["parents"] is not None else 0, e["parents"]) for e in chunk]
        b = W.custom("chunk%d" % nchunks, 16, 4, 64, reqs, seed=nchunks)
        t = W.make_tensors(b)
        if ctx is None:
            ctx = H.make_ctx(b, max_q_tokens=1 << 12, max_requests=64, max_tree_nodes=64)
        ctx.plan_batch(b)
        O, LSE = H.run_gpu(b, t, ctx=ctx)
        O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
        H.check_against_oracle(O, LSE, O_ref, LSE_ref, "chunk %d" % nchunks)
        assert b.total_q <= 384
        nchunks += 1
    assert nchunks >= 3
    ctx.close()
