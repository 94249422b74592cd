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

import oracle
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
    o64, lse64 = o.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)
    # and against the fp64 oracle (an error shared by both GPU paths would pass the comparison above)
    O_ref, LSE_ref = oracle.attention(batch, t, H.SCALE)
    H.check_against_oracle(o64, lse64, O_ref, LSE_ref, "decode_static vs oracle")
    return o64, lse64, o_ref, lse_ref


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


@pytest.mark.parametrize("hq,hkv,page", [(4, 4, 16), (32, 1, 128), (8, 2, 64)])
def test_decode_static_chunk_boundaries_head_ratios_and_small_pages(hq, hkv, page):
    """Contexts that end exactly at, one before and one after a 2048-key chunk boundary
    (kv_len + 1 keys), one q head per kv head and 32, pages of 16 tokens."""
    reqs = [(1, kv, 0, None) for kv in (0, 1, 2046, 2047, 2048, 4094, 4095, 4096, 777)]
    b = W.custom("static_edges", hq, hkv, page, reqs, seed=hq + page)
    o, lse, o_ref, lse_ref = _run_both(b)
    H.check_against_oracle(o, lse, o_ref, lse_ref, "decode_static edges vs xy_attn_run")


def test_decode_static_flags_a_request_beyond_max_kv_len_and_checks_dtypes():
    b = W.custom("static_bound", 8, 2, 64, [(1, 300, 0, None), (1, 5000, 0, None), (1, 900, 0, None)], seed=2)
    t = W.make_tensors(b)
    d = H.DeviceBatch(b, t)
    kv_len = torch.from_numpy(b.kv_len.astype(np.int32)).cuda()
    o = torch.zeros_like(d.o)
    lse = torch.zeros_like(d.lse)
    rc = xb.xy_attn_decode_static(d.q, d.k_pool, d.v_pool, d.block_table, kv_len, 1000, H.SCALE, o, lse)
    torch.cuda.synchronize()
    assert rc == xb.XY_OK
    assert torch.isnan(lse[1]).all() and torch.isnan(o[1].float()).all()   # the request that breaks the bound
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    keep = [0, 2]
    H.check_against_oracle(o[keep].float().cpu().numpy().astype(np.float64), lse[keep].cpu().numpy().astype(np.float64),
                           O_ref[keep], LSE_ref[keep], "decode_static, rows inside the bound")
    with pytest.raises(xb.XYAttnError):
        xb.xy_attn_decode_static(d.q, d.k_pool, d.v_pool, d.block_table, kv_len.long(), 1000, H.SCALE, o, lse)
    rc = xb.xy_attn_decode_static(d.q, d.k_pool, d.v_pool, d.block_table, kv_len, 2 ** 31 - 1, H.SCALE, o, lse)
    assert rc == xb.XY_ERR_CAPACITY
