"""Context sharded over devices (cross-device form of the Update stage, Section 4.2.1): every
shard runs decode attention over its slice of the keys, the per-shard (O, LSE) are merged by
xy_attn_merge_shards.  The shards run one after the other on one GPU here (no kernel waits on
another); the expected value is the unchanged attention oracle on the unsharded batch."""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_18106_b200 import binding as xb
from paper_2412_18106_b200 import workloads as W

from . import helpers as H

pytestmark = pytest.mark.gpu


def _sharded_run(b, t, shards, workers=0):
    bounds = [xb.xy_attn_shard_context(int(b.kv_len[r]) + 1, b.page_size, shards) for r in range(b.num_requests)]
    dev = "cuda:0"
    q, kp, vp = t.q.to(dev), t.k_pool.to(dev), t.v_pool.to(dev)
    T, Hq = b.total_q, b.num_q_heads
    o_sh = torch.full((shards, T, Hq, 128), float("nan"), dtype=torch.bfloat16, device=dev)
    l_sh = torch.full((shards, T, Hq), float("nan"), dtype=torch.float32, device=dev)
    ctx = H.make_ctx(b, num_workers=workers)
    for k in range(shards):
        sb = W.context_shard(b, bounds, k)
        ctx.plan_batch(sb)
        bt = torch.from_numpy(np.where(sb.block_table < 0, 0, sb.block_table).astype(np.int32)).to(dev)
        ctx.run(q, kp, vp, bt, H.SCALE, o_sh[k], l_sh[k])
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
    ctx.close()
    o = torch.full((T, Hq, 128), float("nan"), dtype=torch.bfloat16, device=dev)
    lse = torch.full((T, Hq), float("nan"), dtype=torch.float32, device=dev)
    xb.xy_attn_merge_shards(o_sh.view(shards, T * Hq, 128), l_sh.view(shards, T * Hq),
                            o.view(T * Hq, 128), lse.view(T * Hq))
    torch.cuda.synchronize()
    return o, lse, o_sh, l_sh, bounds


@pytest.mark.parametrize("page_size", [16, 128])
@pytest.mark.parametrize("shards", [1, 2, 3, 8])
def test_sharded_decode_matches_unsharded_oracle(shards, page_size):
    rng = np.random.default_rng(100 * shards + page_size)
    lo = shards * page_size  # at least one page per shard
    kvs = [lo - 1, lo, lo + 1] + [int(np.exp(rng.uniform(np.log(lo + 2), np.log(24000)))) for _ in range(5)]
    b = W.custom("ctx_shard", 32, 8, page_size, [(1, kv, 0, None) for kv in kvs], seed=7 + shards)
    t = W.make_tensors(b)
    o, lse, o_sh, l_sh, bounds = _sharded_run(b, t, shards)
    O_ref, L_ref = oracle.attention(b, t, H.SCALE)
    H.check_against_oracle(o.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64),
                           O_ref, L_ref, "sharded %d" % shards)
    # every shard alone equals the oracle restricted to its slice of the keys
    r, a = b.num_requests - 1, 5
    for k in range(shards):
        keep = np.zeros(int(b.kv_len[r]) + 1, dtype=np.uint8)
        keep[int(bounds[r][k]) : int(bounds[r][k + 1])] = 1
        o_k, l_k = oracle.attention_keys(b, t, H.SCALE, r, a, 0, keep)
        assert np.abs(o_sh[k, r, a].float().cpu().numpy() - o_k).max() <= H.O_MAX_ABS
        assert abs(float(l_sh[k, r, a]) - l_k) <= H.LSE_REL * max(1.0, abs(l_k))
    if shards == 1:  # one shard: weight 1, the merge copies the bits
        assert torch.equal(o.view(torch.int16), o_sh[0].view(torch.int16))


def test_merge_shards_kernel_matches_oracle_merge():
    rng = np.random.default_rng(3)
    for S, rows in [(1, 9), (5, 37), (32, 130), (40, 21)]:  # 40 takes the path without shuffles
        Oc = torch.from_numpy(rng.normal(size=(S, rows, 128)).astype(np.float32)).to(torch.bfloat16)
        Lc = rng.normal(scale=3.0, size=(S, rows)).astype(np.float32)
        if S >= 5:
            Lc[2, 5] = -np.inf
            Oc[2, 5] = float("nan")  # an empty shard's O is never read
            Lc[:, 7] = -np.inf
            Lc[1, 7] = 0.25
            Oc[0, 7] = float("inf")
        o = torch.zeros((rows, 128), dtype=torch.bfloat16, device="cuda")
        lse = torch.zeros(rows, dtype=torch.float32, device="cuda")
        xb.xy_attn_merge_shards(Oc.cuda(), torch.from_numpy(Lc).cuda(), o, lse)
        torch.cuda.synchronize()
        Of = Oc.float().numpy().astype(np.float64)
        Of[~np.isfinite(Of)] = 0.0  # weight-zero partials: the definition multiplies them by 0
        O_ref, L_ref = oracle.merge(Of, Lc.astype(np.float64))
        got = o.float().cpu().numpy()
        assert np.isfinite(got).all()
        assert np.abs(got - O_ref).max() <= 2e-2
        assert np.all(np.abs(lse.cpu().numpy() - L_ref) <= 1e-3 * np.maximum(1, np.abs(L_ref)))


_NCCL_ONE_RANK = r"""
import os, sys
import numpy as np
import torch
import torch.distributed as dist
sys.path.insert(0, sys.argv[1])
os.environ["NCCL_NVLS_ENABLE"] = "0"
torch.cuda.set_device(0)
try:
    dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%s" % sys.argv[2], rank=0, world_size=1,
                            device_id=torch.device("cuda", 0))
    probe = torch.ones(4, device="cuda")
    dist.all_reduce(probe)
    torch.cuda.synchronize()
except Exception as e:  # the collective library cannot start on this machine: nothing of ours ran
    print("nccl unavailable: %r" % (e,))
    sys.exit(0)
from paper_2412_18106_b200 import context_shard as cs
g = torch.Generator(device="cuda").manual_seed(5)
o_local = torch.randn((7, 8, 128), device="cuda", generator=g).to(torch.bfloat16)
l_local = torch.randn((7, 8), device="cuda", generator=g)
o, lse = cs.gather_and_merge(o_local, l_local)
torch.cuda.synchronize()
# one rank: weight 1 for its only shard, so the merge returns the bits it was given
assert torch.equal(o.view(torch.int16), o_local.view(torch.int16))
assert torch.allclose(lse, l_local, rtol=0, atol=1e-6)
dist.destroy_process_group()
print("one-rank nccl ok")
"""


def test_gather_and_merge_over_nccl_with_one_rank():
    """The CUDA side of the exchange (NCCL all-gather into local memory, then the merge kernel) with
    a process group of one rank; the two-rank exchange itself runs on CPU ranks (gloo)."""
    import os
    import socket
    import subprocess
    import sys
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-c", _NCCL_ONE_RANK, root, str(port)], capture_output=True, text=True,
                       timeout=300)
    if "nccl unavailable" in r.stdout:
        pytest.skip("NCCL could not start a one-rank group here: " + r.stdout.strip()[-300:])
    assert r.returncode == 0 and "one-rank nccl ok" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]
