"""The device-side failure path and the validation aid, exercised without faulting the GPU.

A bounded wait is made to run out: the producer of the only worker leaves out one stage fill
(nothing reads unwritten memory, the readers simply never see the stage filled) while the wait
limit is short.  The kernel must return, the status must show the timeout, and the next ordinary
run on the same context must be correct."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2412_18106_b200 import binding as xb
from paper_2412_18106_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("kernel", [xb.XY_KERNEL_AUTO, xb.XY_KERNEL_MMA], ids=["auto", "mma"])
@pytest.mark.parametrize("skip", [0, 3, 9])
def test_a_wait_that_runs_out_is_reported_and_the_context_recovers(kernel, skip):
    b = W.config1_tiny()
    t = W.make_tensors(b)
    ctx = H.make_ctx(b, kernel=kernel, num_workers=1)
    ctx.plan_batch(b)
    d = H.DeviceBatch(b, t)
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    ctx.debug_inject(wait_limit_polls=20000, skip_fill=skip)
    ctx.run(d.q, d.k_pool, d.v_pool, d.block_table, H.SCALE, d.o, d.lse)
    torch.cuda.synchronize()                       # the kernel returned
    assert ctx.device_status() == xb.XY_ERR_DEVICE_TIMEOUT
    assert ctx.device_status() == 0                # reported once, then cleared
    # an ordinary run without reading the status in between also recovers
    ctx.run(d.q, d.k_pool, d.v_pool, d.block_table, H.SCALE, d.o, d.lse)
    ctx.debug_inject(0, -1)
    for _ in range(2):
        o = torch.full_like(d.o, float("nan"))
        lse = torch.full_like(d.lse, float("nan"))
        ctx.run(d.q, d.k_pool, d.v_pool, d.block_table, H.SCALE, o, lse)
        torch.cuda.synchronize()
        H.check_against_oracle(o.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64),
                               O_ref, LSE_ref, "run after a timeout")
    assert ctx.device_status() == xb.XY_ERR_DEVICE_TIMEOUT   # the second failing run is on record too
    assert ctx.device_status() == 0
    ctx.close()
    # tensor memory was freed: a fresh context (which allocates all 512 columns again) works
    H.parity(b, kernel=kernel, num_workers=1)


def test_debug_context_rejects_a_bad_block_table_before_launching():
    os.environ["XY_ATTN_DEBUG"] = "1"
    try:
        b = W.config1_tiny()
        ctx = H.make_ctx(b)
    finally:
        del os.environ["XY_ATTN_DEBUG"]
    ctx.plan_batch(b)
    t = W.make_tensors(b)
    d = H.DeviceBatch(b, t)
    good = d.block_table.clone()
    d.block_table[3, 2] = b.num_pages + 7
    with pytest.raises(xb.XYAttnError) as e:
        ctx.run(d.q, d.k_pool, d.v_pool, d.block_table, H.SCALE, d.o, d.lse)
    assert e.value.code == xb.XY_ERR_INVALID_ARG and "request 3" in str(e.value)
    torch.cuda.synchronize()
    assert ctx.last_launches() == 0 and torch.isnan(d.lse).all()
    ctx.run(d.q, d.k_pool, d.v_pool, good, H.SCALE, d.o, d.lse)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    H.check_against_oracle(d.o.float().cpu().numpy().astype(np.float64), d.lse.cpu().numpy().astype(np.float64),
                           O_ref, LSE_ref, "debug context")
    ctx.close()
