"""TEST INFRASTRUCTURE — fp64 reference of the Linear GEMM that SmoothGEMM computes (Section 5):
C[M, N] = A[M, K] W[N, K]^T on the exact values of the bf16 inputs.

Only tests, the smoke check and the bench's cpu_baseline / reference arm may import this module.
It shares no code with the CUDA path.  The definition is the textbook matrix product, written as
one library matmul in fp64 (no blocking, no padding: the virtual padding of Section 5.1 must not
change any result, which is what the comparison checks)."""
from __future__ import annotations

import numpy as np
import torch


def widen(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> fp64 array, exactly."""
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.to(torch.float64).numpy()


def linear(a: torch.Tensor, w: torch.Tensor) -> np.ndarray:
    """a bf16 [M, K], w bf16 [N, K] -> fp64 [M, N] = a w^T."""
    return widen(a) @ widen(w).T


def linear_rows(a: torch.Tensor, w: torch.Tensor, rows, cols) -> np.ndarray:
    """Sampled outputs C[rows[s], cols[s]] as plain dot products (for sizes where the whole
    product is too slow)."""
    A, W = widen(a), widen(w)
    return np.array([float(np.dot(A[r], W[c])) for r, c in zip(rows, cols)], dtype=np.float64)
