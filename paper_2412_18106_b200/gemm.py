"""Thin ctypes binding of SmoothGEMM (include/xy_gemm.h): argument marshalling only."""
from __future__ import annotations

import ctypes
from typing import Optional

import torch

from . import binding as xb

GEMM_EXPORTS = ("xy_gemm_run", "xy_gemm_run_ws", "xy_gemm_workspace_bytes", "xy_gemm_device_status")

XY_GEMM_PAIR = 0x1000  # tile_n flag: 256-row tiles on CTA pairs

_ready = False


def _lib():
    global _ready
    L = xb.load()
    if not _ready:
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        L.xy_gemm_run.argtypes = [vp, i64, vp, i64, vp, i64, i32, i32, i32, i32, vp]
        L.xy_gemm_run.restype = ctypes.c_int
        L.xy_gemm_run_ws.argtypes = [vp, i64, vp, i64, vp, i64, i32, i32, i32, i32, vp, i64, vp]
        L.xy_gemm_run_ws.restype = ctypes.c_int
        L.xy_gemm_workspace_bytes.argtypes = []
        L.xy_gemm_workspace_bytes.restype = i64
        L.xy_gemm_device_status.argtypes = [ctypes.POINTER(i32)]
        L.xy_gemm_device_status.restype = ctypes.c_int
        _ready = True
    return L


def xy_gemm_workspace(device) -> torch.Tensor:
    """Zero-filled scratch of xy_gemm_workspace_bytes() bytes for xy_gemm_run(..., workspace=...)."""
    with torch.cuda.device(device):
        n = int(_lib().xy_gemm_workspace_bytes())
    if n < 0:
        raise xb.XYAttnError(xb.XY_ERR_CUDA, "xy_gemm_workspace_bytes failed")
    return torch.zeros(n, dtype=torch.uint8, device=device)


def xy_gemm_run(a: torch.Tensor, w: torch.Tensor, c: torch.Tensor, tile_n: int = 0, stream=None,
                workspace: Optional[torch.Tensor] = None) -> None:
    """c[M, N] = a[M, K] w[N, K]^T (bf16 CUDA tensors, last dimension contiguous; rows may be strided).
    With `workspace` (from xy_gemm_workspace) the call goes through xy_gemm_run_ws."""
    for t in (a, w, c):
        if t.dtype != torch.bfloat16 or not t.is_cuda or t.dim() != 2 or (t.numel() and t.stride(1) != 1):
            raise ValueError("xy_gemm_run takes 2-D bf16 CUDA tensors with a contiguous last dimension")
    M, K = a.shape
    N = w.shape[0]
    if w.shape[1] != K or tuple(c.shape) != (M, N):
        raise ValueError("shape mismatch")
    lda = a.stride(0) if M > 1 else max(K, a.stride(0))
    ldc = c.stride(0) if M > 1 else max(N, c.stride(0))
    if workspace is None:
        rc = _lib().xy_gemm_run(a.data_ptr(), lda, w.data_ptr(), w.stride(0), c.data_ptr(), ldc, M, N, K,
                                int(tile_n), xb._stream_ptr(stream))
    else:
        if workspace.dtype != torch.uint8 or not workspace.is_cuda or not workspace.is_contiguous():
            raise ValueError("workspace must be a contiguous uint8 CUDA tensor")
        rc = _lib().xy_gemm_run_ws(a.data_ptr(), lda, w.data_ptr(), w.stride(0), c.data_ptr(), ldc, M, N, K,
                                   int(tile_n), workspace.data_ptr(), workspace.numel(), xb._stream_ptr(stream))
    if rc != 0:
        raise xb.XYAttnError(rc, "xy_gemm_run failed")


def xy_gemm_device_status() -> int:
    s = ctypes.c_int32(0)
    rc = _lib().xy_gemm_device_status(ctypes.byref(s))
    if rc != 0:
        raise xb.XYAttnError(rc, "xy_gemm_device_status failed")
    return int(s.value)
