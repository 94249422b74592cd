"""Thin ctypes binding of the token-wise chunk former (include/xy_sched.h): argument
marshalling only, same names as the C entry points.  Host code; no GPU is touched."""
from __future__ import annotations

import ctypes
from typing import List, Sequence, Tuple

import numpy as np

from . import binding as xb

SCHED_EXPORTS = (
    "xy_sched_create", "xy_sched_destroy", "xy_sched_add_prefill", "xy_sched_add_decode",
    "xy_sched_add_verify", "xy_sched_pending", "xy_sched_next_chunk",
)

XY_SCHED_PREFILL, XY_SCHED_DECODE, XY_SCHED_VERIFY = 0, 1, 2


class xy_sched_config(ctypes.Structure):
    _fields_ = [("budget_tokens", ctypes.c_int32), ("reserved_dv_tokens", ctypes.c_int32),
                ("max_requests", ctypes.c_int32)]


class xy_sched_entry(ctypes.Structure):
    _fields_ = [("id", ctypes.c_int64), ("kind", ctypes.c_int32), ("last", ctypes.c_int32)]


_ready = False


def _lib():
    global _ready
    L = xb.load()
    if not _ready:
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        L.xy_sched_create.argtypes = [ctypes.POINTER(xy_sched_config), ctypes.POINTER(vp)]
        L.xy_sched_destroy.argtypes = [vp]
        L.xy_sched_add_prefill.argtypes = [vp, i64, i32, i32]
        L.xy_sched_add_decode.argtypes = [vp, i64, i32]
        L.xy_sched_add_verify.argtypes = [vp, i64, i32, vp, i32]
        L.xy_sched_pending.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i64)]
        L.xy_sched_next_chunk.argtypes = [vp, vp, vp, i32, vp, i32, ctypes.POINTER(i32)]
        for name in SCHED_EXPORTS:
            getattr(L, name).restype = ctypes.c_int
        _ready = True
    return L


class XYSched:
    def __init__(self, budget_tokens: int, reserved_dv_tokens: int, max_requests: int):
        self.lib = _lib()
        self.cfg = xy_sched_config(int(budget_tokens), int(reserved_dv_tokens), int(max_requests))
        self._s = ctypes.c_void_p(0)
        self._check(self.lib.xy_sched_create(ctypes.byref(self.cfg), ctypes.byref(self._s)))
        self._reqs = (xb.xy_attn_request * self.cfg.max_requests)()
        self._entries = (xy_sched_entry * self.cfg.max_requests)()
        self._parents = np.zeros(self.cfg.budget_tokens, dtype=np.int32)

    @staticmethod
    def _check(rc: int) -> int:
        if rc < 0:
            raise xb.XYAttnError(rc, "xy_sched call failed")
        return rc

    def close(self) -> None:
        if self._s and self._s.value:
            self.lib.xy_sched_destroy(self._s)
            self._s = ctypes.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def add_prefill(self, rid: int, prompt_tokens: int, cached_tokens: int) -> None:
        self._check(self.lib.xy_sched_add_prefill(self._s, int(rid), int(prompt_tokens), int(cached_tokens)))

    def add_decode(self, rid: int, kv_len: int) -> None:
        self._check(self.lib.xy_sched_add_decode(self._s, int(rid), int(kv_len)))

    def add_verify(self, rid: int, kv_len: int, parents: Sequence[int]) -> None:
        par = np.ascontiguousarray(np.asarray(parents, dtype=np.int32))
        self._check(self.lib.xy_sched_add_verify(self._s, int(rid), int(kv_len),
                                                 ctypes.c_void_p(par.ctypes.data), int(par.size)))

    def pending(self) -> Tuple[int, int]:
        p, d = ctypes.c_int64(0), ctypes.c_int64(0)
        self._check(self.lib.xy_sched_pending(self._s, ctypes.byref(p), ctypes.byref(d)))
        return int(p.value), int(d.value)

    def next_chunk_raw(self):
        """The next chunk without Python objects per entry: (n, requests, entries, parents,
        num_parents) where requests is the xy_attn_request array xy_attn_plan takes as it is
        (valid until the next call)."""
        npar = ctypes.c_int32(0)
        n = self._check(self.lib.xy_sched_next_chunk(
            self._s, ctypes.cast(self._reqs, ctypes.c_void_p), ctypes.cast(self._entries, ctypes.c_void_p),
            self.cfg.max_requests, ctypes.c_void_p(self._parents.ctypes.data), int(self._parents.size),
            ctypes.byref(npar)))
        return n, self._reqs, self._entries, self._parents, int(npar.value)

    def next_chunk(self) -> List[dict]:
        """The next chunk as a list of dicts (id, kind, q_len, kv_len, last, parents)."""
        npar = ctypes.c_int32(0)
        n = self._check(self.lib.xy_sched_next_chunk(
            self._s, ctypes.cast(self._reqs, ctypes.c_void_p), ctypes.cast(self._entries, ctypes.c_void_p),
            self.cfg.max_requests, ctypes.c_void_p(self._parents.ctypes.data), int(self._parents.size),
            ctypes.byref(npar)))
        out = []
        for k in range(n):
            r, e = self._reqs[k], self._entries[k]
            parents = None
            if r.mask_kind == xb.XY_MASK_TREE:
                parents = [int(x) for x in self._parents[r.parent_off: r.parent_off + r.q_len]]
            out.append(dict(id=int(e.id), kind=int(e.kind), q_len=int(r.q_len), kv_len=int(r.kv_len),
                            last=bool(e.last), parents=parents))
        return out
