"""fp8 KV-cache variant: the CUDA path (xy_attn_run_fp8kv) against the fp64 oracle on the same
e4m3 bytes and scales.  The oracle attends to decode(byte) * scale exactly; the kernels widen
e4m3 to f16 exactly, so the same tolerances as the bf16 path apply (stated in tests/helpers.py)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_18106_b200 import binding as xb
from paper_2412_18106_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu

KERNELS = [xb.XY_KERNEL_AUTO, xb.XY_KERNEL_REFERENCE]
KNAMES = {xb.XY_KERNEL_AUTO: "auto", xb.XY_KERNEL_REFERENCE: "reference"}


def run_fp8(batch, t8, scale=H.SCALE, ctx=None, **kw):
    own = ctx is None
    if own:
        ctx = H.make_ctx(batch, kv_dtype=xb.XY_KV_FP8_E4M3, **kw)
        ctx.plan_batch(batch)
    dev = "cuda:0"
    q, k8, v8 = t8.q.to(dev), t8.k_pool.to(dev), t8.v_pool.to(dev)
    ks, vs = t8.k_scale.to(dev), t8.v_scale.to(dev)
    bt = torch.from_numpy(np.where(batch.block_table < 0, 0, batch.block_table).astype(np.int32)).to(dev)
    o = torch.full((batch.total_q, batch.num_q_heads, 128), float("nan"), dtype=torch.bfloat16, device=dev)
    lse = torch.full((batch.total_q, batch.num_q_heads), float("nan"), dtype=torch.float32, device=dev)
    ctx.run_fp8kv(q, k8, v8, ks, vs, bt, scale, o, lse)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    if own:
        ctx.close()
    return o.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)


def parity_fp8(batch, **kw):
    t8 = W.to_fp8_kv(W.make_tensors(batch))
    O, LSE = run_fp8(batch, t8, **kw)
    O_ref, LSE_ref = oracle.attention_fp8(batch, t8, H.SCALE)
    return H.check_against_oracle(O, LSE, O_ref, LSE_ref, batch.name + " fp8")


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAMES[k])
def test_config1_tiny_hybrid_fp8(kernel):
    parity_fp8(W.config1_tiny(), kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAMES[k])
@pytest.mark.parametrize("page", [16, 32, 64, 128])
def test_page_sizes_fp8(kernel, page):
    rng = np.random.default_rng(page)
    reqs = [(70, 0, 0, None), (33, 150, 0, None), (1, 257, 0, None), (1, 5, 0, None),
            (20, 300, 1, W.random_tree(rng, 20, 6)), (2, 129, 1, [-1, 0]), (1, 4000, 0, None)]
    parity_fp8(W.custom("fp8pages%d" % page, 8, 2, page, reqs, seed=page), kernel=kernel)


@pytest.mark.parametrize("heads", [(28, 4), (32, 8), (64, 8), (4, 4), (16, 1)])
def test_head_ratios_and_splits_fp8(heads):
    hq, hkv = heads
    rng = np.random.default_rng(hq)
    reqs = [(40, 100, 0, None), (1, 9000, 0, None), (9, 260, 1, W.random_tree(rng, 9, 4)), (1, 0, 0, None),
            (300, 2000, 0, None)]
    b = W.custom("fp8heads%d_%d" % heads, hq, hkv, 64, reqs, seed=hq)
    ctx = H.make_ctx(b, kv_dtype=xb.XY_KV_FP8_E4M3, num_workers=148)
    info = ctx.plan_batch(b)
    assert info.num_merge_units > 0
    t8 = W.to_fp8_kv(W.make_tensors(b))
    O, LSE = run_fp8(b, t8, ctx=ctx)
    O2, LSE2 = run_fp8(b, t8, ctx=ctx)
    ctx.close()
    assert np.array_equal(O, O2) and np.array_equal(LSE, LSE2)
    O_ref, LSE_ref = oracle.attention_fp8(b, t8, H.SCALE)
    H.check_against_oracle(O, LSE, O_ref, LSE_ref, "fp8 heads")


def test_q_rows_of_very_different_magnitudes_fp8():
    """The per-row power-of-two factor of Q: rows scaled by 2^-20 .. 2^20 (far outside what f16
    holds without it) give the same attention as the oracle, at a softmax scale that keeps the
    scores moderate."""
    b = W.custom("fp8qmag", 8, 2, 32, [(24, 100, 0, None), (1, 333, 0, None)], seed=4)
    t = W.make_tensors(b)
    exps = torch.tensor([-20, -7, 0, 9, 20])[torch.arange(b.total_q) % 5]
    t.q = (t.q.float() * (2.0 ** exps.float())[:, None, None] * 2.0 ** -20).to(torch.bfloat16)
    t8 = W.to_fp8_kv(t)
    O, LSE = run_fp8(b, t8, scale=H.SCALE)
    O_ref, LSE_ref = oracle.attention_fp8(b, t8, H.SCALE)
    H.check_against_oracle(O, LSE, O_ref, LSE_ref, "fp8 q magnitudes")


def test_entry_points_check_the_context_dtype():
    b = W.config1_tiny()
    t = W.make_tensors(b)
    d = H.DeviceBatch(b, t)
    c8 = H.make_ctx(b, kv_dtype=xb.XY_KV_FP8_E4M3)
    c8.plan_batch(b)
    with pytest.raises(xb.XYAttnError) as e:
        c8.run(d.q, d.k_pool, d.v_pool, d.block_table, H.SCALE, d.o, d.lse)
    assert e.value.code == xb.XY_ERR_UNSUPPORTED
    c16 = H.make_ctx(b)
    c16.plan_batch(b)
    t8 = W.to_fp8_kv(t)
    with pytest.raises(xb.XYAttnError) as e:
        c16.run_fp8kv(d.q, t8.k_pool.cuda(), t8.v_pool.cuda(), t8.k_scale.cuda(), t8.v_scale.cuda(), d.block_table,
                      H.SCALE, d.o, d.lse)
    assert e.value.code == xb.XY_ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert torch.isnan(d.lse).all()
    with pytest.raises(xb.XYAttnError) as e:
        H.make_ctx(W.custom("p8", 8, 2, 8, [(1, 5, 0, None)]), kv_dtype=xb.XY_KV_FP8_E4M3)
    assert e.value.code == xb.XY_ERR_UNSUPPORTED


@pytest.mark.parametrize("name", ["decode_only", "splitfuse_mix", "verify_trees", "full_mix"])
def test_full_size_sampled_parity_fp8(name):
    """The benchmark configurations with an fp8 cache: sampled rows against the oracle, whole
    output bit-identical when repeated and in agreement with the SIMT kernel."""
    from tests.test_gpu_full_configs import sample_rows
    batch = W.CONFIGS[name](seed=0)
    t8 = W.to_fp8_kv(W.make_tensors(batch))
    ctx = H.make_ctx(batch, kv_dtype=xb.XY_KV_FP8_E4M3)
    ctx.plan_batch(batch)
    O, LSE = run_fp8(batch, t8, ctx=ctx)
    O2, LSE2 = run_fp8(batch, t8, ctx=ctx)
    ctx.close()
    assert not np.isnan(O).any() and np.array_equal(O, O2) and np.array_equal(LSE, LSE2)
    rng = np.random.default_rng(7)
    req, head, row = sample_rows(batch, rng, 64)
    O_ref, LSE_ref = oracle.attention_fp8(batch, t8, H.SCALE, rows=(req, head, row))
    x = batch.q_start[req] + row
    H.check_against_oracle(O[x, head], LSE[x, head], O_ref, LSE_ref, name + " fp8")
    if name in ("decode_only", "verify_trees"):
        Or, Lr = run_fp8(batch, t8, kernel=xb.XY_KERNEL_REFERENCE)
        err = np.sqrt(((O - Or) ** 2).sum(-1))
        ref = np.sqrt((Or ** 2).sum(-1))
        assert np.all(err <= 2.0 ** -6 * ref + 2e-5), float((err / (ref + 1e-9)).max())
        assert np.all(np.abs(LSE - Lr) <= 1e-5 * np.maximum(1.0, np.abs(Lr)))
