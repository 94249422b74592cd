"""TEST INFRASTRUCTURE — ctypes front of the fp64 CPU oracle (`attn_oracle.cpp`).

Only tests, the smoke check and the bench's cpu_baseline / reference arm may
import this package.  It shares no code with the CUDA library and does not
import it.  Inputs are the same bf16 tensors the GPU gets; everything is widened
exactly to fp64 inside the C++ code.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "attn_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (C++17, OpenMP).  Rebuilds when the source is newer."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c++17",
                               "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _u16(t: torch.Tensor) -> torch.Tensor:
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.view(torch.int16)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _ptr(a):
    if isinstance(a, torch.Tensor):
        return ctypes.c_void_p(a.data_ptr())
    if a is None:
        return ctypes.c_void_p(0)
    return ctypes.c_void_p(a.ctypes.data)


class _Problem:
    """Marshals a (batch, tensors) pair into the C argument list."""

    def __init__(self, batch, tensors, sm_scale: float):
        self.batch = batch
        self.keep = []  # keep numpy arrays alive
        q, k, v = tensors.q, tensors.k_pool, tensors.v_pool
        assert q.stride(2) == 1 and q.stride(1) == batch.head_dim
        assert k.stride() == v.stride() and k.stride(3) == 1
        self.q, self.k, self.v = _u16(q), _u16(k), _u16(v)
        ql, kl, mk, po = _i32(batch.q_len), _i32(batch.kv_len), _i32(batch.mask_kind), _i32(batch.parent_off)
        pa = _i32(batch.parents) if batch.parents.size else np.zeros(1, np.int32)
        bt = _i32(batch.block_table)
        self.keep += [ql, kl, mk, po, pa, bt]
        self.args = [
            ctypes.c_int(batch.num_requests), ctypes.c_int(batch.num_q_heads),
            ctypes.c_int(batch.num_kv_heads), ctypes.c_int(batch.head_dim),
            ctypes.c_int(batch.page_size), _ptr(ql), _ptr(kl), _ptr(mk), _ptr(po), _ptr(pa),
            _ptr(self.q), ctypes.c_int64(q.stride(0)), _ptr(self.k), _ptr(self.v),
            ctypes.c_int64(k.stride(0)), ctypes.c_int64(k.stride(1)), ctypes.c_int64(k.stride(2)),
            _ptr(bt), ctypes.c_int32(bt.shape[1]), ctypes.c_double(sm_scale),
        ]


def attention(batch, tensors, sm_scale: float, only: Optional[Sequence[int]] = None,
              want_psum: bool = False):
    """Exact attention of the whole batch (or of the requests listed in `only`).

    Returns (O fp64 [T, Hq, D], LSE fp64 [T, Hq]) and, with want_psum, the sum of each
    row's probabilities.  Rows of requests not in `only` are NaN."""
    p = _Problem(batch, tensors, sm_scale)
    T, Hq, D = batch.total_q, batch.num_q_heads, batch.head_dim
    O = np.full((T, Hq, D), np.nan, dtype=np.float64)
    LSE = np.full((T, Hq), np.nan, dtype=np.float64)
    psum = np.full((T, Hq), np.nan, dtype=np.float64) if want_psum else None
    flags = None
    if only is not None:
        flags = np.zeros(batch.num_requests, dtype=np.uint8)
        flags[list(only)] = 1
    rc = lib().oracle_attention(*p.args, _ptr(flags), _ptr(O), _ptr(LSE), _ptr(psum))
    assert rc == 0
    return (O, LSE, psum) if want_psum else (O, LSE)


def attention_rows(batch, tensors, sm_scale: float, req, head, row) -> Tuple[np.ndarray, np.ndarray]:
    """Sampled outputs: O fp64 [S, D], LSE fp64 [S] for (req[s], head[s], row[s])."""
    p = _Problem(batch, tensors, sm_scale)
    req, head, row = _i32(req), _i32(head), _i32(row)
    S = req.shape[0]
    O = np.zeros((S, batch.head_dim), dtype=np.float64)
    LSE = np.zeros(S, dtype=np.float64)
    rc = lib().oracle_attention_rows(*p.args, ctypes.c_int(S), _ptr(req), _ptr(head), _ptr(row),
                                     _ptr(O), _ptr(LSE))
    assert rc == 0
    return O, LSE


def probs(batch, tensors, sm_scale: float, r: int, a: int) -> Tuple[np.ndarray, np.ndarray]:
    """Probability matrix P fp64 [n, L] and the materialised mask M u8 [n, L] of (request, q head)."""
    p = _Problem(batch, tensors, sm_scale)
    n = int(batch.q_len[r])
    L = n + int(batch.kv_len[r])
    P = np.zeros((n, L), dtype=np.float64)
    M = np.zeros((n, L), dtype=np.uint8)
    rc = lib().oracle_probs(*p.args, ctypes.c_int(r), ctypes.c_int(a), _ptr(P), _ptr(M))
    assert rc == 0
    return P, M


def attention_keys(batch, tensors, sm_scale: float, r: int, a: int, i: int, keep) -> Tuple[np.ndarray, float]:
    """One row restricted to the keys flagged in `keep` (u8 [L]): partial (O_c fp64 [D], LSE_c)."""
    p = _Problem(batch, tensors, sm_scale)
    keep = np.ascontiguousarray(np.asarray(keep, dtype=np.uint8))
    O = np.zeros(batch.head_dim, dtype=np.float64)
    LSE = ctypes.c_double(0.0)
    rc = lib().oracle_attention_keys(*p.args, ctypes.c_int(r), ctypes.c_int(a), ctypes.c_int(i),
                                     _ptr(keep), _ptr(O), ctypes.byref(LSE))
    assert rc == 0
    return O, float(LSE.value)


def gather(batch, tensors, r: int, g: int) -> Tuple[torch.Tensor, torch.Tensor]:
    """Gathered K and V rows (bf16 [L, D] each) of request r, kv head g, read through the block table."""
    p = _Problem(batch, tensors, 1.0)
    L = int(batch.q_len[r]) + int(batch.kv_len[r])
    K = torch.zeros((L, batch.head_dim), dtype=torch.bfloat16)
    V = torch.zeros((L, batch.head_dim), dtype=torch.bfloat16)
    rc = lib().oracle_gather(*p.args, ctypes.c_int(r), ctypes.c_int(g), _ptr(_u16(K)), _ptr(_u16(V)))
    assert rc == 0
    return K, V


def merge(O_c: np.ndarray, LSE_c: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Update-stage merge of C partials: O_c fp64 [C, rows, D], LSE_c fp64 [C, rows]."""
    O_c = np.ascontiguousarray(O_c, dtype=np.float64)
    LSE_c = np.ascontiguousarray(LSE_c, dtype=np.float64)
    C, rows, D = O_c.shape
    O = np.zeros((rows, D), dtype=np.float64)
    LSE = np.zeros(rows, dtype=np.float64)
    rc = lib().oracle_merge(ctypes.c_int(C), ctypes.c_int64(rows), ctypes.c_int(D), _ptr(O_c),
                            _ptr(LSE_c), _ptr(O), _ptr(LSE))
    assert rc == 0
    return O, LSE


def append_kv(batch, qkv: torch.Tensor, k_pool: torch.Tensor, v_pool: torch.Tensor) -> None:
    """Writes the K / V head rows of the fused QKV tensor (bf16 [T, Hq + 2 Hkv, D]) into the paged
    cache at positions kv_len .. kv_len + q_len - 1 of every request (in place, bit copy)."""
    assert qkv.dtype == torch.bfloat16 and qkv.stride(2) == 1 and qkv.stride(1) == batch.head_dim
    ql, kl, bt = _i32(batch.q_len), _i32(batch.kv_len), _i32(batch.block_table)
    rc = lib().oracle_append_kv(
        ctypes.c_int(batch.num_requests), ctypes.c_int(batch.num_q_heads), ctypes.c_int(batch.num_kv_heads),
        ctypes.c_int(batch.head_dim), ctypes.c_int(batch.page_size), _ptr(ql), _ptr(kl), _ptr(_u16(qkv)),
        ctypes.c_int64(qkv.stride(0)), _ptr(_u16(k_pool)), _ptr(_u16(v_pool)), ctypes.c_int64(k_pool.stride(0)),
        ctypes.c_int64(k_pool.stride(1)), ctypes.c_int64(k_pool.stride(2)), _ptr(bt), ctypes.c_int32(bt.shape[1]))
    assert rc == 0


def e4m3_table() -> np.ndarray:
    """The oracle's decode of all 256 e4m3 bytes (fp64; NaN at 0x7F and 0xFF)."""
    out = np.zeros(256, dtype=np.float64)
    assert lib().oracle_e4m3_table(_ptr(out)) == 0
    return out


def attention_fp8(batch, tensors, sm_scale: float, rows=None):
    """fp8 KV-cache variant: tensors.k_pool / v_pool are uint8 e4m3 pools [P, Hkv, B, D] and
    tensors.k_scale / v_scale fp32 [P, Hkv]; the attended values are decode(byte) * scale.
    Whole batch -> (O [T, Hq, D], LSE [T, Hq]); with rows = (req, head, row) -> sampled outputs."""
    k8, v8 = tensors.k_pool, tensors.v_pool
    assert k8.dtype == torch.uint8 and v8.dtype == torch.uint8 and k8.stride() == v8.stride() and k8.stride(3) == 1
    ks = np.ascontiguousarray(tensors.k_scale.numpy() if isinstance(tensors.k_scale, torch.Tensor) else tensors.k_scale,
                              dtype=np.float32)
    vs = np.ascontiguousarray(tensors.v_scale.numpy() if isinstance(tensors.v_scale, torch.Tensor) else tensors.v_scale,
                              dtype=np.float32)
    assert ks.shape == (k8.shape[0], batch.num_kv_heads) and vs.shape == ks.shape
    q = tensors.q
    assert q.stride(2) == 1 and q.stride(1) == batch.head_dim
    ql, kl, mk, po = _i32(batch.q_len), _i32(batch.kv_len), _i32(batch.mask_kind), _i32(batch.parent_off)
    pa = _i32(batch.parents) if batch.parents.size else np.zeros(1, np.int32)
    bt = _i32(batch.block_table)
    args = [ctypes.c_int(batch.num_requests), ctypes.c_int(batch.num_q_heads), ctypes.c_int(batch.num_kv_heads),
            ctypes.c_int(batch.head_dim), ctypes.c_int(batch.page_size), _ptr(ql), _ptr(kl), _ptr(mk), _ptr(po), _ptr(pa),
            _ptr(_u16(q)), ctypes.c_int64(q.stride(0)), ctypes.c_void_p(0), ctypes.c_void_p(0),
            ctypes.c_int64(k8.stride(0)), ctypes.c_int64(k8.stride(1)), ctypes.c_int64(k8.stride(2)),
            _ptr(bt), ctypes.c_int32(bt.shape[1]), ctypes.c_double(sm_scale),
            _ptr(k8), _ptr(v8), _ptr(ks), _ptr(vs)]
    D = batch.head_dim
    if rows is None:
        O = np.full((batch.total_q, batch.num_q_heads, D), np.nan, dtype=np.float64)
        LSE = np.full((batch.total_q, batch.num_q_heads), np.nan, dtype=np.float64)
        rc = lib().oracle_attention_fp8(*args, ctypes.c_int(-1), ctypes.c_void_p(0), ctypes.c_void_p(0),
                                        ctypes.c_void_p(0), _ptr(O), _ptr(LSE))
    else:
        req, head, row = (_i32(x) for x in rows)
        S = req.shape[0]
        O = np.zeros((S, D), dtype=np.float64)
        LSE = np.zeros(S, dtype=np.float64)
        rc = lib().oracle_attention_fp8(*args, ctypes.c_int(S), _ptr(req), _ptr(head), _ptr(row), _ptr(O), _ptr(LSE))
    assert rc == 0
    return O, LSE
