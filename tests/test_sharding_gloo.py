"""Multi-GPU path of bench.py on CPU ranks (gloo, world size 2): requests shard across ranks
with no data-path collective; every rank plans its own batch with the host planner, rank
results are combined only for reporting (max of times, sum of work), as bench.py does."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2412_18106_b200 import binding as xb
    from paper_2412_18106_b200 import workloads as W
    batch = W.config3_splitfuse(seed=rank)  # weak scaling: each rank draws its own batch
    ctx = xb.XYAttn(batch.num_q_heads, batch.num_kv_heads, batch.page_size, device=-1,
                    max_q_tokens=1 << 15, max_pages_per_req=1024)
    info = ctx.plan_batch(batch)
    work = torch.tensor([float(info.useful_flops), float(info.kv_bytes)], dtype=torch.float64)
    t = torch.tensor([1.0 + rank], dtype=torch.float64)  # stand-in for a per-rank time
    dist.barrier()
    dist.all_reduce(work, op=dist.ReduceOp.SUM)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        np.save(out, np.array([work[0].item(), work[1].item(), t.item(), info.num_tasks]))
    dist.destroy_process_group()


def test_two_rank_request_sharding(tmp_path):
    out = str(tmp_path / "r0.npy")
    port = _free_port()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    got = np.load(out)
    sys.path.insert(0, ROOT)
    from paper_2412_18106_b200 import workloads as W
    want_flops = sum(W.useful_flops(W.config3_splitfuse(seed=r)) for r in range(2))
    want_bytes = sum(W.kv_bytes(W.config3_splitfuse(seed=r)) for r in range(2))
    assert got[0] == want_flops and got[1] == want_bytes
    assert got[2] == 2.0  # max over ranks
    assert got[3] > 0


def _head_shard(batch, tensors, k, world):
    """Rank k's slice of a batch under the kv-head split: kv heads [k Hkv/N, (k+1) Hkv/N) of every
    page and the q heads that read them; requests, block table and trees are the same on every rank."""
    import dataclasses
    sys.path.insert(0, ROOT)
    from paper_2412_18106_b200 import workloads as W
    hkv = batch.num_kv_heads // world
    g = batch.num_q_heads // batch.num_kv_heads
    sub = dataclasses.replace(batch, num_q_heads=hkv * g, num_kv_heads=hkv)
    q = tensors.q[:, k * hkv * g: (k + 1) * hkv * g, :].contiguous()
    kp = tensors.k_pool[:, k * hkv: (k + 1) * hkv].contiguous()
    vp = tensors.v_pool[:, k * hkv: (k + 1) * hkv].contiguous()
    return sub, W.Tensors(q=q, k_pool=kp, v_pool=vp)


def _head_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2412_18106_b200 import binding as xb
    from paper_2412_18106_b200 import workloads as W
    batch = W.config1_tiny()          # the same batch on every rank
    tensors = W.make_tensors(batch)
    sub, st = _head_shard(batch, tensors, rank, world)
    # the rank's own plan over its heads: the same decomposition for every rank
    ctx = xb.XYAttn(sub.num_q_heads, sub.num_kv_heads, sub.page_size, device=-1)
    info = ctx.plan_batch(sub)
    shape = torch.tensor([info.num_tasks, info.num_merge_units, info.useful_flops], dtype=torch.int64)
    shapes = [torch.zeros_like(shape) for _ in range(world)]
    dist.all_gather(shapes, shape)
    assert all(torch.equal(s, shapes[0]) for s in shapes)
    # the rank's attention over its heads (the oracle stands in for the GPU on this CPU rank);
    # outputs are only gathered for the check: the path itself has no exchange
    O, LSE = oracle.attention(sub, st, 1.0 / 128 ** 0.5)
    Os = [torch.zeros(O.shape, dtype=torch.float64) for _ in range(world)]
    Ls = [torch.zeros(LSE.shape, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(Os, torch.from_numpy(O))
    dist.all_gather(Ls, torch.from_numpy(LSE))
    if rank == 0:
        np.save(out + ".o.npy", torch.cat(Os, dim=1).numpy())
        np.save(out + ".lse.npy", torch.cat(Ls, dim=1).numpy())
        np.save(out + ".flops.npy", np.array([int(shapes[0][2]) * world]))
    dist.destroy_process_group()


def test_two_rank_kv_head_split_matches_the_unsplit_oracle(tmp_path):
    """Tensor-parallel style sharding: rank k holds kv heads [k Hkv/N, (k+1) Hkv/N) of every page
    and the matching q heads, every rank plans the same requests, and no collective is needed on
    the data path.  The concatenation of the ranks' head slices equals the oracle on the whole
    batch bit for bit (heads are independent), and the ranks' useful flops add up."""
    out = str(tmp_path / "heads")
    port = _free_port()
    mp.spawn(_head_worker, args=(2, port, out), nprocs=2, join=True)
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2412_18106_b200 import workloads as W
    batch = W.config1_tiny()
    tensors = W.make_tensors(batch)
    O_ref, LSE_ref = oracle.attention(batch, tensors, 1.0 / 128 ** 0.5)
    assert np.array_equal(np.load(out + ".o.npy"), O_ref)
    assert np.array_equal(np.load(out + ".lse.npy"), LSE_ref)
    assert int(np.load(out + ".flops.npy")[0]) == W.useful_flops(batch)
