"""Host side of the context-sharded decode path: slice arithmetic, argument checks, and the
two-rank exchange on CPU ranks (gloo).  In the gloo test every rank computes its slice with the
attention oracle, the package's gather moves (O_k, LSE_k) between the ranks, and the oracle's
merge of what arrived must equal the oracle on the unsharded batch."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2412_18106_b200 import binding as xb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("page_size", [16, 32, 64, 128])
def test_shard_context_slices(page_size):
    rng = np.random.default_rng(page_size)
    for _ in range(200):
        shards = int(rng.integers(1, 17))
        total = int(rng.integers(shards * page_size - page_size + 1, 200000))
        bd = xb.xy_attn_shard_context(total, page_size, shards)
        assert bd.shape == (shards + 1,) and bd[0] == 0 and bd[-1] == total
        assert np.all(np.diff(bd) > 0)  # contiguous, none empty
        assert np.all(bd[:-1] % page_size == 0)  # every slice starts on a page
        pages = -(-np.diff(bd) // page_size)
        assert pages.max() - pages.min() <= 1
        assert pages[-1] == pages.min()  # the slice that takes the appends is never the largest


def test_shard_context_rejects():
    for total, page, shards in [(0, 16, 1), (100, 16, 0), (100, 0, 2), (32, 16, 3), (128, 128, 2)]:
        with pytest.raises(xb.XYAttnError):
            xb.xy_attn_shard_context(total, page, shards)
    assert list(xb.xy_attn_shard_context(33, 16, 3)) == [0, 16, 32, 33]


def test_merge_shards_argument_checks():
    L = xb.load()
    assert L.xy_attn_merge_shards(None, None, 2, 4, 128, None, None, None) == xb.XY_ERR_INVALID_ARG
    assert L.xy_attn_merge_shards(None, None, 2, 4, 64, None, None, None) == xb.XY_ERR_UNSUPPORTED
    assert L.xy_attn_merge_shards(None, None, 0, 4, 128, None, None, None) == xb.XY_ERR_INVALID_ARG
    assert L.xy_attn_merge_shards(None, None, 2, -1, 128, None, None, None) == xb.XY_ERR_INVALID_ARG
    assert L.xy_attn_merge_shards(None, None, 2, 0, 128, None, None, None) == xb.XY_OK


def test_gather_and_merge_has_no_cpu_path():
    from paper_2412_18106_b200 import context_shard as cs
    with pytest.raises(RuntimeError):
        cs.gather_and_merge(torch.zeros((1, 2, 128), dtype=torch.bfloat16), torch.zeros((1, 2)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _batch():
    from paper_2412_18106_b200 import workloads as W
    kvs = [31, 32, 33, 700, 1999]
    return W.custom("ctx_shard_host", 8, 2, 16, [(1, kv, 0, None) for kv in kvs], seed=11)


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2412_18106_b200 import context_shard as cs
    from paper_2412_18106_b200 import workloads as W
    b = _batch()
    t = W.make_tensors(b)
    bounds = [xb.xy_attn_shard_context(int(kv) + 1, b.page_size, world) for kv in b.kv_len]
    sb = W.context_shard(b, bounds, rank)
    O_k, L_k = oracle.attention(sb, t, 0.125)  # this rank's slice only
    T, Hq = b.total_q, b.num_q_heads
    # the exchange carries what the device path carries: O_k rounded to bf16, LSE_k in fp32
    o_local = torch.from_numpy(O_k).to(torch.bfloat16).reshape(T * Hq, 128)
    l_local = torch.from_numpy(L_k).to(torch.float32).reshape(T * Hq)
    o_sh, l_sh = cs.gather_shards(o_local, l_local)
    assert o_sh.shape == (world, T * Hq, 128) and l_sh.shape == (world, T * Hq)
    assert torch.equal(o_sh[rank], o_local) and torch.equal(l_sh[rank], l_local)
    O, L = oracle.merge(o_sh.float().numpy().astype(np.float64), l_sh.numpy().astype(np.float64))
    np.save(out % rank, np.concatenate([O.reshape(-1), L.reshape(-1)]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_context_sharding(tmp_path):
    out = str(tmp_path / "r%d.npy")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    import oracle
    from paper_2412_18106_b200 import workloads as W
    b = _batch()
    O_ref, L_ref = oracle.attention(b, W.make_tensors(b), 0.125)
    want = np.concatenate([O_ref.reshape(-1), L_ref.reshape(-1)])
    got0, got1 = np.load(out % 0), np.load(out % 1)
    assert np.array_equal(got0, got1)  # both ranks end with the same result
    n = O_ref.size
    assert np.abs(got0[:n] - want[:n]).max() <= 2.0 ** -8 * np.abs(O_ref).max()  # bf16 partials
    assert np.abs(got0[n:] - want[n:]).max() <= 1e-5
