"""KV-cache append with fused QKV split on the GPU: bit-exact against the oracle's append, and
attention on the appended cache against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_18106_b200 import binding as xb
from paper_2412_18106_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("page", [16, 128])
def test_append_kv_bit_exact_then_attention(page):
    rng = np.random.default_rng(page)
    reqs = [(70, 0, 0, None), (33, 150, 0, None), (1, 257, 0, None), (1, 5, 0, None),
            (20, 300, 1, W.random_tree(rng, 20, 6)), (130, 77, 0, None)]
    b = W.custom("append%d" % page, 8, 2, page, reqs, seed=page)
    t = W.make_tensors(b, fused_qkv=True)
    d = H.DeviceBatch(b, t)
    qkv_dev = t.qkv.cuda()
    ctx = H.make_ctx(b)
    ctx.plan_batch(b)
    ctx.append_kv(qkv_dev, d.k_pool, d.v_pool, d.block_table)
    q_dev = qkv_dev[:, : b.num_q_heads, :]
    ctx.run(q_dev, d.k_pool, d.v_pool, d.block_table, H.SCALE, d.o, d.lse)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    # oracle: same append on the CPU copies, then attention
    oracle.append_kv(b, t.qkv, t.k_pool, t.v_pool)
    assert torch.equal(d.k_pool.cpu().view(torch.int16), t.k_pool.view(torch.int16))
    assert torch.equal(d.v_pool.cpu().view(torch.int16), t.v_pool.view(torch.int16))
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    H.check_against_oracle(d.o.float().cpu().numpy().astype(np.float64), d.lse.cpu().numpy().astype(np.float64),
                           O_ref, LSE_ref, "append+attention")
    # error paths launch nothing
    ctx2 = H.make_ctx(b)
    with pytest.raises(xb.XYAttnError) as e:
        ctx2.append_kv(qkv_dev, d.k_pool, d.v_pool, d.block_table)
    assert e.value.code == xb.XY_ERR_NOT_PLANNED
