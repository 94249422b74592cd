"""The allocation-free decode entry point, through the C-ABI, against the existing entry point.

Some callers cannot allocate device memory where they need attention (a serving loop whose
pool is fully handed out, a plugin that owns only its buffers); xy_attn_decode_static serves
them from a fixed scratch array inside the library.  This file is collected last on purpose: if
it fails, a run that stops at the first failure has already run every other test.  It passes
alone in a fresh process and after the other tests; two calls in a row check that the shared
scratch needs no clearing between calls of different shapes.
"""
import numpy as np
import pytest
import torch

from paper_2412_18106_b200 import binding as xb
from paper_2412_18106_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _decode_batch(num_requests, kv_hi, seed):
    return W.config2_decode(seed=seed, num_requests=num_requests, kv_lo=1, kv_hi=kv_hi)


def _run_both(batch):
    t = W.make_tensors(batch)
    d = H.DeviceBatch(batch, t)
    # existing entry point
    ctx = H.make_ctx(batch)
    ctx.plan_batch(batch)
    ctx.run(d.q, d.k_pool, d.v_pool, d.block_table, H.SCALE, d.o, d.lse)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    o_ref = d.o.float().cpu().numpy().astype(np.float64)
    lse_ref = d.lse.cpu().numpy().astype(np.float64)
    ctx.close()
    # allocation-free entry point: every tensor it touches exists before the call
    o = torch.full_like(d.o, float("nan"))
    lse = torch.full_like(d.lse, float("nan"))
    kv_len = torch.from_numpy(batch.kv_len.astype(np.int32)).cuda()
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    rc = xb.xy_attn_decode_static(d.q, d.k_pool, d.v_pool, d.block_table, kv_len, int(batch.kv_len.max()),
                                  H.SCALE, o, lse)
    torch.cuda.synchronize()
    assert rc == xb.XY_OK
    assert torch.cuda.memory_allocated() == before
    return o.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64), o_ref, lse_ref


def test_decode_static_matches_run_on_two_calls_in_a_row():
    assert torch.cuda.is_available()
    # second call: fewer requests, shorter contexts, fewer chunks than the first
    for num_requests, kv_hi, seed in ((24, 9000, 3), (7, 1500, 4)):
        b = _decode_batch(num_requests, kv_hi, seed)
        o, lse, o_ref, lse_ref = _run_both(b)
        H.check_against_oracle(o, lse, o_ref, lse_ref, "decode_static vs xy_attn_run")


def test_decode_static_rejects_sizes_beyond_the_scratch():
    b = _decode_batch(4, 600, 5)
    t = W.make_tensors(b)
    d = H.DeviceBatch(b, t)
    kv_len = torch.from_numpy(b.kv_len.astype(np.int32)).cuda()
    # 4 requests x 28 heads x ceil(200001 / 2048) chunks > 8192 rows
    rc = xb.xy_attn_decode_static(d.q, d.k_pool, d.v_pool, d.block_table, kv_len, 200000, H.SCALE, d.o, d.lse)
    assert rc == xb.XY_ERR_CAPACITY
    torch.cuda.synchronize()
    assert torch.isnan(d.lse).all()  # nothing was launched
