"""Thin ctypes binding of the C-ABI library (include/xy_attn.h), same names.

Argument marshalling only: every step of the path runs in the CUDA kernels.
PyTorch is used for device memory and streams.  There is no CPU fallback: if the
shared library is missing the import fails loudly, and `run` needs CUDA tensors.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libxy_attn.so")

XY_OK = 0
XY_ERR_INVALID_ARG = -1
XY_ERR_CAPACITY = -2
XY_ERR_BAD_TREE = -3
XY_ERR_NOT_PLANNED = -4
XY_ERR_CUDA = -5
XY_ERR_DEVICE_TIMEOUT = -6
XY_ERR_UNSUPPORTED = -7

XY_MASK_CAUSAL = 0
XY_MASK_TREE = 1

XY_KERNEL_AUTO = 0
XY_KERNEL_REFERENCE = 1
XY_KERNEL_MMA = 2
XY_KERNEL_PAIR = 3

XY_PLAN_BALANCED = 0
XY_PLAN_PAPER = 1

XY_KV_BF16 = 0
XY_KV_FP8_E4M3 = 1


class xy_attn_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "num_q_heads", "num_kv_heads", "head_dim", "page_size", "max_requests", "max_q_tokens",
        "max_pages_per_req", "max_tree_nodes", "device", "num_workers", "kernel", "plan_mode",
        "tile_tokens", "max_splits", "kv_dtype")] + [("workspace_bytes", ctypes.c_int64)]


class xy_attn_request(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("q_len", "kv_len", "mask_kind", "parent_off")]


class xy_attn_task(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "req", "kv_head", "tok0", "ntok", "kt_lo", "kt_hi", "part", "kind")]


class xy_attn_merge_unit(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("req", "kv_head", "tok0", "ntok", "part0", "nsplit",
                                              "part1", "nsplit1", "stride1", "reserved")]


class xy_attn_prefix_group(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("first_req", "num_reqs", "prefix_tokens")]


class xy_attn_plan_info(ctypes.Structure):
    _fields_ = [("num_tasks", ctypes.c_int32), ("num_dense_tasks", ctypes.c_int32),
                ("num_merge_units", ctypes.c_int32), ("num_workers", ctypes.c_int32),
                ("useful_flops", ctypes.c_int64), ("kv_bytes", ctypes.c_int64),
                ("partial_rows", ctypes.c_int64), ("load_min", ctypes.c_float),
                ("load_mean", ctypes.c_float), ("load_max", ctypes.c_float),
                ("max_task_cost", ctypes.c_float), ("num_inline_merge_units", ctypes.c_int32),
                ("reserved", ctypes.c_int32)]


TASK_DTYPE = np.dtype([(n, np.int32) for n in ("req", "kv_head", "tok0", "ntok", "kt_lo", "kt_hi", "part", "kind")])
MERGE_DTYPE = np.dtype([(n, np.int32) for n in ("req", "kv_head", "tok0", "ntok", "part0", "nsplit",
                                                 "part1", "nsplit1", "stride1", "reserved")])

EXPORTS = (
    "xy_attn_create", "xy_attn_destroy", "xy_attn_plan", "xy_attn_run", "xy_attn_merge",
    "xy_attn_debug_gather", "xy_attn_get_tasks", "xy_attn_get_worker_offsets",
    "xy_attn_get_merge_units", "xy_attn_get_tree_mask", "xy_attn_get_q_start",
    "xy_attn_last_launches", "xy_attn_last_error", "xy_attn_device_status",
    "xy_attn_set_timing", "xy_attn_get_timing", "xy_attn_debug_trace", "xy_attn_decode_static",
    "xy_attn_append_kv", "xy_attn_worker_times", "xy_attn_get_queue", "xy_attn_plan_cache",
    "xy_attn_plan_shared", "xy_attn_shard_context", "xy_attn_merge_shards",
    "xy_attn_find_prefix_groups", "xy_attn_debug_check_block_table", "xy_attn_debug_inject",
    "xy_attn_run_fp8kv",
)

_lib = None


def load() -> ctypes.CDLL:
    """Loads libxy_attn.so (built in-tree by `python -m paper_2412_18106_b200.build`)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            "CUDA extension missing: %s not built (run python -m paper_2412_18106_b200.build). "
            "There is no CPU fallback." % LIB_PATH)
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    L.xy_attn_create.argtypes = [ctypes.POINTER(xy_attn_config), ctypes.POINTER(vp)]
    L.xy_attn_destroy.argtypes = [vp]
    L.xy_attn_plan.argtypes = [vp, vp, i32, vp, i32, vp, ctypes.POINTER(xy_attn_plan_info)]
    L.xy_attn_plan_shared.argtypes = [vp, vp, i32, vp, i32, vp, i32, vp, ctypes.POINTER(xy_attn_plan_info)]
    L.xy_attn_run.argtypes = [vp, vp, i64, vp, vp, i64, i64, i64, i64, vp, i32, vp, ctypes.c_float,
                              vp, i64, vp, vp]
    L.xy_attn_run_fp8kv.argtypes = [vp, vp, i64, vp, vp, vp, vp, i64, i64, i64, i64, vp, i32, vp, ctypes.c_float,
                                    vp, i64, vp, vp]
    L.xy_attn_merge.argtypes = [vp, vp, i32, i64, i32, vp, vp, vp]
    L.xy_attn_merge_shards.argtypes = [vp, vp, i32, i64, i32, vp, vp, vp]
    L.xy_attn_find_prefix_groups.argtypes = [vp, i32, vp, i32, i32, i32, i32, vp, i32, ctypes.POINTER(i32)]
    L.xy_attn_shard_context.argtypes = [i64, i32, i32, ctypes.POINTER(i64)]
    L.xy_attn_append_kv.argtypes = [vp, vp, i64, vp, vp, i64, i64, i64, i64, vp, i32, vp]
    L.xy_attn_debug_gather.argtypes = [vp, i32, i32, vp, vp, i64, i64, i64, vp, i32, vp, vp, vp]
    for name in ("xy_attn_get_tasks", "xy_attn_get_worker_offsets", "xy_attn_get_merge_units",
                 "xy_attn_get_tree_mask", "xy_attn_get_q_start", "xy_attn_get_queue"):
        getattr(L, name).argtypes = [vp, vp, i32]
    L.xy_attn_set_timing.argtypes = [vp, i32]
    L.xy_attn_get_timing.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float),
                                     ctypes.POINTER(i32)]
    L.xy_attn_debug_trace.argtypes = [vp, vp, i32]
    L.xy_attn_worker_times.argtypes = [vp, vp, i32]
    L.xy_attn_plan_cache.argtypes = [vp, i32, ctypes.POINTER(i64), ctypes.POINTER(i64)]
    L.xy_attn_decode_static.argtypes = [vp, i64, vp, vp, i64, i64, i64, vp, i32, vp, i32, i32, i32, i32, i32,
                                        ctypes.c_float, vp, i64, vp, vp]
    L.xy_attn_debug_check_block_table.argtypes = [vp, vp, i32, i64]
    L.xy_attn_debug_inject.argtypes = [vp, i32, i32]
    L.xy_attn_last_launches.argtypes = [vp]
    L.xy_attn_last_error.argtypes = [vp]
    L.xy_attn_last_error.restype = ctypes.c_char_p
    L.xy_attn_device_status.argtypes = [vp, ctypes.POINTER(i32)]
    for name in EXPORTS:
        if name != "xy_attn_last_error":
            getattr(L, name).restype = ctypes.c_int
    _lib = L
    return L


class XYAttnError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__("xy_attn error %d: %s" % (code, msg))
        self.code = code


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> ctypes.c_void_p:
    if stream is None:
        if torch.cuda.is_available():
            return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
        return ctypes.c_void_p(0)
    return ctypes.c_void_p(stream.cuda_stream)


class XYAttn:
    """One xy_attn context.  Methods mirror the C entry points."""

    def __init__(self, num_q_heads: int, num_kv_heads: int, page_size: int, *, head_dim: int = 128,
                 max_requests: int = 256, max_q_tokens: int = 1 << 15, max_pages_per_req: int = 1024,
                 max_tree_nodes: int = 64, device: int = 0, num_workers: int = 0,
                 kernel: int = XY_KERNEL_AUTO, plan_mode: int = XY_PLAN_BALANCED, tile_tokens: int = 0,
                 max_splits: int = 0, workspace_bytes: int = 0, kv_dtype: int = XY_KV_BF16):
        self.lib = load()
        self.cfg = xy_attn_config(num_q_heads, num_kv_heads, head_dim, page_size, max_requests,
                                  max_q_tokens, max_pages_per_req, max_tree_nodes, device, num_workers,
                                  kernel, plan_mode, tile_tokens, max_splits, kv_dtype, workspace_bytes)
        self._ctx = ctypes.c_void_p(0)
        rc = self.lib.xy_attn_create(ctypes.byref(self.cfg), ctypes.byref(self._ctx))
        if rc != XY_OK:
            raise XYAttnError(rc, "xy_attn_create failed")
        self.info = xy_attn_plan_info()

    def close(self):
        if self._ctx and self._ctx.value:
            self.lib.xy_attn_destroy(self._ctx)
            self._ctx = ctypes.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int):
        if rc != XY_OK:
            raise XYAttnError(rc, self.lib.xy_attn_last_error(self._ctx).decode())

    # -- xy_attn_plan
    def plan(self, q_len: Sequence[int], kv_len: Sequence[int], mask_kind: Sequence[int],
             parent_off: Sequence[int], parents=None, stream=None) -> xy_attn_plan_info:
        R = len(q_len)
        reqs = (xy_attn_request * max(R, 1))()
        for r in range(R):
            reqs[r] = xy_attn_request(int(q_len[r]), int(kv_len[r]), int(mask_kind[r]), int(parent_off[r]))
        par = np.ascontiguousarray(np.asarray(parents if parents is not None else [], dtype=np.int32))
        par_ptr = ctypes.c_void_p(par.ctypes.data) if par.size else ctypes.c_void_p(0)
        self._check(self.lib.xy_attn_plan(self._ctx, ctypes.cast(reqs, ctypes.c_void_p), R, par_ptr,
                                          int(par.size), _stream_ptr(stream), ctypes.byref(self.info)))
        return self.info

    def plan_raw(self, reqs, num_reqs: int, parents: Optional[np.ndarray], num_parents: int,
                 stream=None) -> xy_attn_plan_info:
        """xy_attn_plan on an xy_attn_request array as the chunk former returns it."""
        par_ptr = ctypes.c_void_p(parents.ctypes.data) if (parents is not None and num_parents) else ctypes.c_void_p(0)
        self._check(self.lib.xy_attn_plan(self._ctx, ctypes.cast(reqs, ctypes.c_void_p), int(num_reqs), par_ptr,
                                          int(num_parents), _stream_ptr(stream), ctypes.byref(self.info)))
        return self.info

    def plan_shared(self, q_len, kv_len, mask_kind, parent_off, parents, groups, stream=None) -> xy_attn_plan_info:
        """xy_attn_plan_shared: `groups` is a list of (first_req, num_reqs, prefix_tokens)."""
        R = len(q_len)
        reqs = (xy_attn_request * max(R, 1))()
        for r in range(R):
            reqs[r] = xy_attn_request(int(q_len[r]), int(kv_len[r]), int(mask_kind[r]), int(parent_off[r]))
        par = np.ascontiguousarray(np.asarray(parents if parents is not None else [], dtype=np.int32))
        par_ptr = ctypes.c_void_p(par.ctypes.data) if par.size else ctypes.c_void_p(0)
        gs = (xy_attn_prefix_group * max(len(groups), 1))()
        for k, g in enumerate(groups):
            gs[k] = xy_attn_prefix_group(int(g[0]), int(g[1]), int(g[2]))
        self._check(self.lib.xy_attn_plan_shared(self._ctx, ctypes.cast(reqs, ctypes.c_void_p), R, par_ptr,
                                                 int(par.size), ctypes.cast(gs, ctypes.c_void_p), len(groups),
                                                 _stream_ptr(stream), ctypes.byref(self.info)))
        return self.info

    def plan_batch(self, batch, stream=None, groups=None) -> xy_attn_plan_info:
        """`groups`: None, a list of (first_req, num_reqs, prefix_tokens), or "auto" to read the
        shared-prefix groups off the batch's block table."""
        if isinstance(groups, str):
            assert groups == "auto"
            groups = xy_attn_find_prefix_groups(batch.q_len, batch.kv_len, batch.mask_kind, batch.block_table,
                                                batch.page_size)
        if groups:
            return self.plan_shared(batch.q_len, batch.kv_len, batch.mask_kind, batch.parent_off, batch.parents,
                                    groups, stream)
        return self.plan(batch.q_len, batch.kv_len, batch.mask_kind, batch.parent_off, batch.parents, stream)

    # -- xy_attn_run
    def run(self, q: torch.Tensor, k_pool: torch.Tensor, v_pool: torch.Tensor,
            block_table: torch.Tensor, sm_scale: float, o: torch.Tensor, lse: torch.Tensor,
            tree_mask: Optional[torch.Tensor] = None, stream=None) -> None:
        for t in (q, k_pool, v_pool, block_table, o, lse):
            if not t.is_cuda:
                raise XYAttnError(XY_ERR_INVALID_ARG, "run needs CUDA tensors (there is no CPU path)")
        assert q.dtype == torch.bfloat16 and k_pool.dtype == torch.bfloat16 and v_pool.dtype == torch.bfloat16
        assert o.dtype == torch.bfloat16 and lse.dtype == torch.float32 and block_table.dtype == torch.int32
        assert q.stride(2) == 1 and q.stride(1) == self.cfg.head_dim
        assert o.stride(2) == 1 and o.stride(1) == self.cfg.head_dim and lse.is_contiguous()
        assert k_pool.stride() == v_pool.stride() and k_pool.stride(3) == 1
        assert block_table.stride(1) == 1
        tm = ctypes.c_void_p(tree_mask.data_ptr()) if tree_mask is not None else ctypes.c_void_p(0)
        self._check(self.lib.xy_attn_run(
            self._ctx, q.data_ptr(), q.stride(0), k_pool.data_ptr(), v_pool.data_ptr(),
            k_pool.shape[0], k_pool.stride(0), k_pool.stride(1), k_pool.stride(2),
            block_table.data_ptr(), block_table.stride(0), tm, float(sm_scale), o.data_ptr(),
            o.stride(0), lse.data_ptr(), _stream_ptr(stream)))

    # -- xy_attn_run_fp8kv
    def run_fp8kv(self, q: torch.Tensor, k_pool: torch.Tensor, v_pool: torch.Tensor, k_scale: torch.Tensor,
                  v_scale: torch.Tensor, block_table: torch.Tensor, sm_scale: float, o: torch.Tensor,
                  lse: torch.Tensor, tree_mask: Optional[torch.Tensor] = None, stream=None) -> None:
        """k_pool / v_pool uint8 (e4m3 bytes) [P, Hkv, B, D], k_scale / v_scale fp32 [P, Hkv]."""
        for t in (q, k_pool, v_pool, k_scale, v_scale, block_table, o, lse):
            if not t.is_cuda:
                raise XYAttnError(XY_ERR_INVALID_ARG, "run_fp8kv needs CUDA tensors (there is no CPU path)")
        assert q.dtype == torch.bfloat16 and k_pool.dtype == torch.uint8 and v_pool.dtype == torch.uint8
        assert k_scale.dtype == torch.float32 and v_scale.dtype == torch.float32
        assert k_scale.is_contiguous() and v_scale.is_contiguous() and k_scale.shape == (k_pool.shape[0], k_pool.shape[1])
        assert v_scale.shape == k_scale.shape
        assert o.dtype == torch.bfloat16 and lse.dtype == torch.float32 and block_table.dtype == torch.int32
        assert q.stride(2) == 1 and q.stride(1) == self.cfg.head_dim
        assert o.stride(2) == 1 and o.stride(1) == self.cfg.head_dim and lse.is_contiguous()
        assert k_pool.stride() == v_pool.stride() and k_pool.stride(3) == 1
        assert block_table.stride(1) == 1
        tm = ctypes.c_void_p(tree_mask.data_ptr()) if tree_mask is not None else ctypes.c_void_p(0)
        self._check(self.lib.xy_attn_run_fp8kv(
            self._ctx, q.data_ptr(), q.stride(0), k_pool.data_ptr(), v_pool.data_ptr(), k_scale.data_ptr(),
            v_scale.data_ptr(), k_pool.shape[0], k_pool.stride(0), k_pool.stride(1), k_pool.stride(2),
            block_table.data_ptr(), block_table.stride(0), tm, float(sm_scale), o.data_ptr(),
            o.stride(0), lse.data_ptr(), _stream_ptr(stream)))

    # -- xy_attn_append_kv
    def append_kv(self, qkv: torch.Tensor, k_pool: torch.Tensor, v_pool: torch.Tensor, block_table: torch.Tensor,
                  stream=None) -> None:
        """Copies the K / V heads of the fused bf16 [T, Hq + 2 Hkv, D] tensor into the paged cache."""
        for t in (qkv, k_pool, v_pool, block_table):
            if not t.is_cuda:
                raise XYAttnError(XY_ERR_INVALID_ARG, "append_kv needs CUDA tensors (there is no CPU path)")
        assert qkv.dtype == torch.bfloat16 and qkv.stride(2) == 1 and qkv.stride(1) == self.cfg.head_dim
        assert k_pool.stride() == v_pool.stride() and k_pool.stride(3) == 1
        self._check(self.lib.xy_attn_append_kv(
            self._ctx, qkv.data_ptr(), qkv.stride(0), k_pool.data_ptr(), v_pool.data_ptr(), k_pool.shape[0],
            k_pool.stride(0), k_pool.stride(1), k_pool.stride(2), block_table.data_ptr(), block_table.stride(0),
            _stream_ptr(stream)))

    # -- xy_attn_debug_gather
    def debug_gather(self, req: int, kv_head: int, k_pool, v_pool, block_table, out_k, out_v, stream=None):
        self._check(self.lib.xy_attn_debug_gather(
            self._ctx, req, kv_head, k_pool.data_ptr(), v_pool.data_ptr(), k_pool.stride(0),
            k_pool.stride(1), k_pool.stride(2), block_table.data_ptr(), block_table.stride(0),
            out_k.data_ptr(), out_v.data_ptr(), _stream_ptr(stream)))

    # -- introspection
    def _get(self, fn, dtype, count_hint=0):
        n = fn(self._ctx, ctypes.c_void_p(0), 0)
        if n < 0:
            self._check(n)
        out = np.zeros(max(n, 1), dtype=dtype)
        fn(self._ctx, ctypes.c_void_p(out.ctypes.data), n)
        return out[:n]

    def get_tasks(self) -> np.ndarray:
        return self._get(self.lib.xy_attn_get_tasks, TASK_DTYPE)

    def get_worker_offsets(self) -> np.ndarray:
        return self._get(self.lib.xy_attn_get_worker_offsets, np.int32)

    def get_merge_units(self) -> np.ndarray:
        return self._get(self.lib.xy_attn_get_merge_units, MERGE_DTYPE)

    def get_tree_mask(self) -> np.ndarray:
        return self._get(self.lib.xy_attn_get_tree_mask, np.uint64)

    def get_q_start(self) -> np.ndarray:
        return self._get(self.lib.xy_attn_get_q_start, np.int32)

    def get_queue(self) -> np.ndarray:
        return self._get(self.lib.xy_attn_get_queue, np.int32)

    def plan_cache(self, capacity: int = -1):
        """Sets the Task-Table cache capacity (-1: leave) and returns (hits, misses)."""
        hits, misses = ctypes.c_int64(0), ctypes.c_int64(0)
        self._check(self.lib.xy_attn_plan_cache(self._ctx, int(capacity), ctypes.byref(hits), ctypes.byref(misses)))
        return int(hits.value), int(misses.value)

    def set_timing(self, enable: bool) -> None:
        self._check(self.lib.xy_attn_set_timing(self._ctx, 1 if enable else 0))

    def get_timing(self):
        """(attention kernel ms, merge kernel ms, runs) summed since the last call."""
        a, m, n = ctypes.c_float(0), ctypes.c_float(0), ctypes.c_int32(0)
        self._check(self.lib.xy_attn_get_timing(self._ctx, ctypes.byref(a), ctypes.byref(m), ctypes.byref(n)))
        return float(a.value), float(m.value), int(n.value)

    def worker_times(self) -> np.ndarray:
        """uint64 [num_workers, 4]: entry and exit stamps (ns) of each worker in the last run and
        the ns it spent in dense and in streaming tasks."""
        n = self.lib.xy_attn_worker_times(self._ctx, ctypes.c_void_p(0), 0)
        if n <= 0:
            self._check(n)
        out = np.zeros(n, dtype=np.uint64)
        self.lib.xy_attn_worker_times(self._ctx, ctypes.c_void_p(out.ctypes.data), n)
        return out.reshape(-1, 4)

    def debug_trace(self) -> np.ndarray:
        """uint64 [4, 2048] trace records of worker 0 (empty unless XY_ATTN_TRACE=1 at create)."""
        n = self.lib.xy_attn_debug_trace(self._ctx, ctypes.c_void_p(0), 0)
        if n <= 0:
            return np.zeros((0,), dtype=np.uint64)
        out = np.zeros(n, dtype=np.uint64)
        self.lib.xy_attn_debug_trace(self._ctx, ctypes.c_void_p(out.ctypes.data), n)
        return out.reshape(4, -1)

    def debug_check_block_table(self, block_table: np.ndarray, num_pages: int) -> None:
        """xy_attn_debug_check_block_table on a HOST int32 [R, stride] array; raises on a bad entry."""
        bt = np.ascontiguousarray(block_table, dtype=np.int32)
        assert bt.ndim == 2
        self._check(self.lib.xy_attn_debug_check_block_table(self._ctx, ctypes.c_void_p(bt.ctypes.data),
                                                             bt.shape[1], int(num_pages)))

    def debug_inject(self, wait_limit_polls: int = 0, skip_fill: int = -1) -> None:
        self._check(self.lib.xy_attn_debug_inject(self._ctx, int(wait_limit_polls), int(skip_fill)))

    def last_launches(self) -> int:
        return int(self.lib.xy_attn_last_launches(self._ctx))

    def last_error(self) -> str:
        return self.lib.xy_attn_last_error(self._ctx).decode()

    def device_status(self) -> int:
        st = ctypes.c_int32(0)
        self._check(self.lib.xy_attn_device_status(self._ctx, ctypes.byref(st)))
        return int(st.value)


def xy_attn_merge(o_part: torch.Tensor, lse_part: torch.Tensor, o: torch.Tensor, lse: torch.Tensor,
                  stream=None) -> None:
    """Split-KV LSE merge: o_part fp32 [S, rows, D], lse_part fp32 [S, rows] -> o bf16, lse fp32."""
    L = load()
    assert o_part.is_cuda and o_part.is_contiguous() and lse_part.is_contiguous()
    S, rows, D = o_part.shape
    rc = L.xy_attn_merge(o_part.data_ptr(), lse_part.data_ptr(), S, rows, D, o.data_ptr(),
                         lse.data_ptr(), _stream_ptr(stream))
    if rc != XY_OK:
        raise XYAttnError(rc, "xy_attn_merge failed")


def xy_attn_find_prefix_groups(q_len, kv_len, mask_kind, block_table: np.ndarray, page_size: int,
                               min_members: int = 2, min_prefix_tokens: int = 128):
    """Shared-prefix groups read off the block tables: list of (first_req, num_reqs, prefix_tokens)."""
    L = load()
    R = len(q_len)
    reqs = (xy_attn_request * max(R, 1))()
    for r in range(R):
        reqs[r] = xy_attn_request(int(q_len[r]), int(kv_len[r]), int(mask_kind[r]), -1)
    bt = np.ascontiguousarray(block_table, dtype=np.int32)
    assert bt.ndim == 2 and bt.shape[0] == R
    gs = (xy_attn_prefix_group * max(R // 2, 1))()
    n = ctypes.c_int32(0)
    rc = L.xy_attn_find_prefix_groups(ctypes.cast(reqs, ctypes.c_void_p), R, ctypes.c_void_p(bt.ctypes.data),
                                      bt.shape[1], int(page_size), int(min_members), int(min_prefix_tokens),
                                      ctypes.cast(gs, ctypes.c_void_p), max(R // 2, 1), ctypes.byref(n))
    if rc != XY_OK:
        raise XYAttnError(rc, "xy_attn_find_prefix_groups failed")
    return [(gs[k].first_req, gs[k].num_reqs, gs[k].prefix_tokens) for k in range(n.value)]


def xy_attn_shard_context(total_tokens: int, page_size: int, num_shards: int) -> np.ndarray:
    """Page-aligned contiguous slices of a context for num_shards devices: int64 [num_shards + 1]."""
    L = load()
    bounds = (ctypes.c_int64 * (num_shards + 1))()
    rc = L.xy_attn_shard_context(int(total_tokens), int(page_size), int(num_shards), bounds)
    if rc != XY_OK:
        raise XYAttnError(rc, "xy_attn_shard_context: %d tokens of page size %d do not split %d ways"
                          % (total_tokens, page_size, num_shards))
    return np.array(bounds[:], dtype=np.int64)


def xy_attn_merge_shards(o_shards: torch.Tensor, lse_shards: torch.Tensor, o: torch.Tensor,
                         lse: torch.Tensor, stream=None) -> None:
    """Merge of per-device results: o_shards bf16 [S, rows, D], lse_shards fp32 [S, rows], both in
    local device memory -> o bf16 [rows, D], lse fp32 [rows]."""
    L = load()
    assert o_shards.is_cuda and o_shards.dtype == torch.bfloat16 and o_shards.is_contiguous()
    assert lse_shards.is_cuda and lse_shards.dtype == torch.float32 and lse_shards.is_contiguous()
    S, rows, D = o_shards.shape
    assert lse_shards.shape == (S, rows) and o.is_contiguous() and lse.is_contiguous()
    rc = L.xy_attn_merge_shards(o_shards.data_ptr(), lse_shards.data_ptr(), S, rows, D, o.data_ptr(),
                                lse.data_ptr(), _stream_ptr(stream))
    if rc != XY_OK:
        raise XYAttnError(rc, "xy_attn_merge_shards failed")


XY_ATTN_STATIC_MAX_ROWS = 8192


def xy_attn_decode_static(q, k_pool, v_pool, block_table, kv_len, max_kv_len: int, sm_scale: float, o, lse,
                          stream=None) -> int:
    """Decode attention for callers that cannot allocate device memory (a full memory pool, a
    plugin that only owns its buffers): no context, no cudaMalloc; the split-KV scratch is a
    fixed array inside the library.  q / o bf16 [R, Hq, 128], lse fp32 [R, Hq], kv_len int32 [R]
    on the device.  Returns the C status code (XY_ERR_CAPACITY beyond the scratch's limit).
    Calls that may overlap on the GPU share the scratch and must be ordered by the caller."""
    L = load()
    for t in (q, k_pool, v_pool, block_table, kv_len, o, lse):
        if not t.is_cuda:
            raise XYAttnError(XY_ERR_INVALID_ARG, "xy_attn_decode_static needs CUDA tensors")
    if not (q.dtype == o.dtype == k_pool.dtype == v_pool.dtype == torch.bfloat16 and lse.dtype == torch.float32
            and kv_len.dtype == torch.int32 and block_table.dtype == torch.int32):
        raise XYAttnError(XY_ERR_INVALID_ARG, "xy_attn_decode_static: q, o and the pools must be bf16, lse fp32, "
                                              "kv_len and block_table int32")
    assert q.stride(2) == 1 and q.stride(1) == 128 and o.stride(2) == 1 and o.stride(1) == 128
    assert lse.is_contiguous() and kv_len.is_contiguous() and block_table.stride(1) == 1
    assert k_pool.stride() == v_pool.stride() and k_pool.stride(3) == 1
    return int(L.xy_attn_decode_static(
        q.data_ptr(), q.stride(0), k_pool.data_ptr(), v_pool.data_ptr(), k_pool.stride(0), k_pool.stride(1),
        k_pool.stride(2), block_table.data_ptr(), block_table.stride(0), kv_len.data_ptr(), q.shape[0],
        int(max_kv_len), q.shape[1], k_pool.shape[1], k_pool.shape[2], float(sm_scale), o.data_ptr(),
        o.stride(0), lse.data_ptr(), _stream_ptr(stream)))


def attention(ctx: XYAttn, batch, q, k_pool, v_pool, block_table, sm_scale, o=None, lse=None,
              tree_mask=None, stream=None):
    """Convenience: allocate O / LSE if needed and run the planned batch."""
    T = q.shape[0]
    if o is None:
        o = torch.empty((T, ctx.cfg.num_q_heads, ctx.cfg.head_dim), dtype=torch.bfloat16, device=q.device)
    if lse is None:
        lse = torch.empty((T, ctx.cfg.num_q_heads), dtype=torch.float32, device=q.device)
    ctx.run(q, k_pool, v_pool, block_table, sm_scale, o, lse, tree_mask=tree_mask, stream=stream)
    return o, lse
