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
