"""Shared pieces of the GPU parity tests: upload a batch, run it through the C-ABI binding,
and compare with the fp64 oracle within the stated tolerances."""
import math

import numpy as np
import torch

import oracle
from paper_2412_18106_b200 import binding as xb
from paper_2412_18106_b200 import workloads as W

SCALE = 1.0 / math.sqrt(128.0)

# Tolerances (the benchmark spec): O max abs 2e-2, mean abs 2e-3; LSE |d| <= 1e-3 * max(1, |ref|).
O_MAX_ABS = 2e-2
O_MEAN_ABS = 2e-3
LSE_REL = 1e-3


class DeviceBatch:
    def __init__(self, batch, tensors, device="cuda:0"):
        self.batch = batch
        self.tensors = tensors
        src_q = tensors.qkv if tensors.qkv is not None else tensors.q
        dq = src_q.to(device)
        self.q = dq[:, : batch.num_q_heads, :] if tensors.qkv is not None else dq
        self.k_pool = tensors.k_pool.to(device)
        self.v_pool = tensors.v_pool.to(device)
        bt = np.where(batch.block_table < 0, 0, batch.block_table).astype(np.int32)
        self.block_table = torch.from_numpy(bt).to(device)
        T = batch.total_q
        self.o = torch.full((T, batch.num_q_heads, batch.head_dim), float("nan"), dtype=torch.bfloat16, device=device)
        self.lse = torch.full((T, batch.num_q_heads), float("nan"), dtype=torch.float32, device=device)


def make_ctx(batch, **kw):
    kw.setdefault("max_requests", max(256, batch.num_requests))
    kw.setdefault("max_q_tokens", max(1 << 15, batch.total_q))
    kw.setdefault("max_pages_per_req", max(1024, batch.block_table.shape[1]))
    kw.setdefault("max_tree_nodes", max(64, int(batch.q_len.max()) if batch.num_requests else 64))
    return xb.XYAttn(batch.num_q_heads, batch.num_kv_heads, batch.page_size, **kw)


def run_gpu(batch, tensors, ctx=None, scale=SCALE, **ctx_kw):
    own = ctx is None
    if own:
        ctx = make_ctx(batch, **ctx_kw)
        ctx.plan_batch(batch)
    d = DeviceBatch(batch, tensors)
    ctx.run(d.q, d.k_pool, d.v_pool, d.block_table, scale, d.o, d.lse)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    assert ctx.last_launches() >= 1
    O = d.o.float().cpu().numpy().astype(np.float64)
    LSE = d.lse.cpu().numpy().astype(np.float64)
    if own:
        ctx.close()
    return O, LSE


def check_against_oracle(O, LSE, O_ref, LSE_ref, what=""):
    assert not np.isnan(O).any(), "%s: O has NaN (rows not written?)" % what
    assert not np.isnan(LSE).any(), "%s: LSE has NaN" % what
    dO = np.abs(O - O_ref)
    assert dO.max() <= O_MAX_ABS, "%s: max |dO| = %g" % (what, dO.max())
    assert dO.mean() <= O_MEAN_ABS, "%s: mean |dO| = %g" % (what, dO.mean())
    dL = np.abs(LSE - LSE_ref)
    bound = LSE_REL * np.maximum(1.0, np.abs(LSE_ref))
    assert np.all(dL <= bound), "%s: LSE off by %g (bound %g)" % (what, (dL - bound).max(), bound.min())
    return float(dO.max()), float(dO.mean()), float((dL / np.maximum(1.0, np.abs(LSE_ref))).max())


def parity(batch, tensors=None, scale=SCALE, **ctx_kw):
    tensors = W.make_tensors(batch) if tensors is None else tensors
    O, LSE = run_gpu(batch, tensors, scale=scale, **ctx_kw)
    O_ref, LSE_ref = oracle.attention(batch, tensors, scale)
    return check_against_oracle(O, LSE, O_ref, LSE_ref, batch.name)
