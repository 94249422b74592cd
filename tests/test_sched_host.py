"""Token-wise chunk former (Section 3.1), host only: the C-ABI scheduler front against the plain
Python restatement in oracle/chunk_former.py, the hand-worked example, and the properties the
paper states (budget, prefill priority with splitting, reserved decode / verify slots, no
prefill-only chunk while decode / verify tokens wait)."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import chunk_former as CF
from paper_2412_18106_b200 import binding as xb
from paper_2412_18106_b200 import sched as xs
from paper_2412_18106_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
KIND = {"P": 0, "D": 1, "V": 2}


def test_library_exports_every_scheduler_symbol():
    header = open(os.path.join(ROOT, "include", "xy_sched.h")).read()
    declared = set(re.findall(r"\b(xy_sched_[a-z_]+)\s*\(", header))
    assert declared == set(xs.SCHED_EXPORTS)
    lib = ctypes.CDLL(xb.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert ctypes.sizeof(xs.xy_sched_entry) == 16 and ctypes.sizeof(xs.xy_sched_config) == 12


def read_example():
    chunks = []
    for line in open(os.path.join(ROOT, "tests", "golden", "chunk_former_example.txt")):
        if not line.startswith("chunk "):
            continue
        body = line.split(":", 1)[1].strip()
        entries = []
        for part in filter(None, (p.strip() for p in body.split("|"))):
            k, rid, q, kv, last = part.split()
            entries.append((KIND[k], int(rid), int(q), int(kv), bool(int(last))))
        chunks.append(entries)
    return chunks


def submit_example(s):
    s.add_prefill(1, 30, 10)
    s.add_prefill(2, 6, 0)
    s.add_decode(11, 100)
    s.add_verify(21, 50, [-1, 0, 0])
    s.add_decode(12, 7)
    s.add_verify(22, 20, [-1, 0, 1, 1, 0])


def as_tuples(chunk):
    return [(e["kind"], e["id"], e["q_len"], e["kv_len"], bool(e["last"])) for e in chunk]


@pytest.mark.parametrize("impl", ["oracle", "cabi"])
def test_hand_worked_example(impl):
    s = CF.ChunkFormer(16, 4, 8) if impl == "oracle" else xs.XYSched(16, 4, 8)
    submit_example(s)
    assert s.pending() == (26, 10)
    for want in read_example():
        got = s.next_chunk()
        assert as_tuples(got) == want
        for e in got:
            if e["id"] == 21:
                assert e["parents"] == [-1, 0, 0]
            if e["id"] == 22:
                assert e["parents"] == [-1, 0, 1, 1, 0]
    assert s.pending() == (0, 0)


def random_stream(seed, steps, budget, reserved, cap):
    """Drives both implementations with the same arrivals; yields (state before, chunk) pairs."""
    rng = np.random.default_rng(seed)
    a, b = CF.ChunkFormer(budget, reserved, cap), xs.XYSched(budget, reserved, cap)
    next_id = 0
    log = []
    for _ in range(steps):
        for _ in range(int(rng.integers(0, 4))):
            kind = int(rng.integers(0, 3))
            next_id += 1
            if kind == 0:
                prompt = int(rng.integers(1, 3 * budget))
                cached = int(rng.integers(0, prompt))
                a.add_prefill(next_id, prompt, cached), b.add_prefill(next_id, prompt, cached)
                log.append(("P", next_id, prompt - cached, cached))
            elif kind == 1:
                kv = int(rng.integers(0, 5000))
                a.add_decode(next_id, kv), b.add_decode(next_id, kv)
                log.append(("D", next_id, 1, kv))
            else:
                n = int(rng.integers(1, min(budget, 24) + 1))
                tree = W.random_tree(rng, n, 6)
                kv = int(rng.integers(0, 5000))
                a.add_verify(next_id, kv, tree), b.add_verify(next_id, kv, tree)
                log.append(("V", next_id, n, kv))
        before = a.pending()
        assert b.pending() == before
        ca, cb = a.next_chunk(), b.next_chunk()
        assert ca == cb
        yield before, ca, log
    # drain
    while a.pending() != (0, 0):
        before = a.pending()
        ca, cb = a.next_chunk(), b.next_chunk()
        assert ca == cb and ca
        yield before, ca, log
    assert b.pending() == (0, 0) and b.next_chunk() == []


@pytest.mark.parametrize("budget,reserved,cap", [(16, 4, 8), (64, 0, 64), (32, 32, 5), (1, 1, 3), (256, 48, 128)])
def test_cabi_equals_oracle_and_properties_hold(budget, reserved, cap):
    scheduled = {}   # id -> [tokens scheduled, next expected kv_len]
    order_p, order_dv = [], []
    log = []
    for before, chunk, log in random_stream(budget * 7 + reserved, 60, budget, reserved, cap):
        tokens = sum(e["q_len"] for e in chunk)
        assert tokens <= budget and len(chunk) <= cap
        dv = [e for e in chunk if e["kind"] != CF.KIND_PREFILL]
        pf = [e for e in chunk if e["kind"] == CF.KIND_PREFILL]
        assert chunk[: len(pf)] == pf  # prefill parts first
        if before[1] > 0:
            assert dv, "a prefill-only chunk while decode / verify tokens wait"
        if before != (0, 0):
            assert chunk
        # the prefill queue gets everything the decode / verify side did not take, up to its demand
        dv_tokens = sum(e["q_len"] for e in dv)
        if len(chunk) < cap:
            assert sum(e["q_len"] for e in pf) == min(before[0], budget - dv_tokens) or not pf and before[0] == 0
        for e in pf:
            st = scheduled.setdefault(e["id"], [0, None])
            if st[1] is not None:
                assert e["kv_len"] == st[1]  # a split prompt continues where it stopped
            st[0] += e["q_len"]
            st[1] = e["kv_len"] + e["q_len"]
            if not order_p or order_p[-1] != e["id"]:
                order_p.append(e["id"])
        for e in dv:
            assert e["last"]
            scheduled.setdefault(e["id"], [0, None])[0] += e["q_len"]
            order_dv.append(e["id"])
    # every token of every arrival scheduled exactly once, in arrival order within each queue
    want = {rid: n for _, rid, n, _ in log}
    assert {k: v[0] for k, v in scheduled.items()} == want
    assert order_p == [rid for k, rid, _, _ in log if k == "P"]
    assert order_dv == [rid for k, rid, _, _ in log if k != "P"]


def test_error_codes_and_capacity():
    for bad in [(0, 0, 1), (8, 9, 1), (8, -1, 1), (8, 0, 0)]:
        with pytest.raises(xb.XYAttnError) as e:
            xs.XYSched(*bad)
        assert e.value.code == xb.XY_ERR_INVALID_ARG
    s = xs.XYSched(8, 2, 4)
    for call in [lambda: s.add_prefill(1, 5, 5), lambda: s.add_prefill(1, 5, -1), lambda: s.add_decode(1, -1),
                 lambda: s.add_verify(1, 0, [-1] * 9), lambda: s.add_verify(1, -1, [-1])]:
        with pytest.raises(xb.XYAttnError) as e:
            call()
        assert e.value.code == xb.XY_ERR_INVALID_ARG
    s.add_decode(7, 3)
    reqs = (xb.xy_attn_request * 4)()
    ents = (xs.xy_sched_entry * 4)()
    par = np.zeros(8, np.int32)
    n = ctypes.c_int32(0)
    L = s.lib
    rc = L.xy_sched_next_chunk(s._s, ctypes.cast(reqs, ctypes.c_void_p), ctypes.cast(ents, ctypes.c_void_p), 3,
                               ctypes.c_void_p(par.ctypes.data), 8, ctypes.byref(n))
    assert rc == xb.XY_ERR_CAPACITY and s.pending() == (0, 1)  # too few request slots: nothing dequeued
    rc = L.xy_sched_next_chunk(s._s, ctypes.cast(reqs, ctypes.c_void_p), ctypes.cast(ents, ctypes.c_void_p), 4,
                               ctypes.c_void_p(par.ctypes.data), 7, ctypes.byref(n))
    assert rc == xb.XY_ERR_CAPACITY and s.pending() == (0, 1)
    assert [e["id"] for e in s.next_chunk()] == [7]


def test_chunks_feed_the_planner():
    """The request list of a chunk goes into xy_attn_plan as it is (host-only context)."""
    s = xs.XYSched(512, 64, 64)
    rng = np.random.default_rng(3)
    s.add_prefill(1, 1500, 200)
    for k in range(20):
        s.add_decode(100 + k, int(rng.integers(10, 3000)))
    s.add_verify(200, 900, W.random_tree(rng, 16, 5))
    ctx = xb.XYAttn(8, 2, 16, device=-1, max_q_tokens=1 << 12, max_pages_per_req=4096)
    total = 0
    while s.pending() != (0, 0):
        chunk = s.next_chunk()
        reqs = [(e["q_len"], e["kv_len"], 1 if e["parents"] is not None else 0, e["parents"]) for e in chunk]
        b = W.custom("chunk", 8, 2, 16, reqs, seed=1)
        info = ctx.plan_batch(b)
        assert info.useful_flops == W.useful_flops(b)
        total += b.total_q
    assert total == 1300 + 20 + 16
