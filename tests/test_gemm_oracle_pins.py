"""Pins of the GEMM oracle (fp64 product of the bf16 inputs' exact values) and host-side checks
of the SmoothGEMM entry points: closed forms and structure a wrong product would break (a
transposed operand, a dropped K tail, rows and columns swapped)."""
import ctypes
import os
import re

import numpy as np
import torch

from oracle import gemm_oracle as G
from paper_2412_18106_b200 import binding as xb
from paper_2412_18106_b200 import gemm as xg

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def bf(x):
    return torch.tensor(x, dtype=torch.float32).to(torch.bfloat16)


def test_worked_2x3_example():
    # by hand: rows of a against rows of w
    a = bf([[1, 2, 3], [4, 5, 6]])
    w = bf([[1, 0, -1], [2, 2, 2], [0.5, 0, 0], [0, 1, 0]])
    want = np.array([[1 - 3, 2 + 4 + 6, 0.5, 2], [4 - 6, 8 + 10 + 12, 2, 5]], dtype=np.float64)
    assert np.array_equal(G.linear(a, w), want)


def test_identity_weight_returns_a_and_selector_rows_pick_columns():
    g = torch.Generator().manual_seed(1)
    a = torch.randn((5, 16), generator=g).to(torch.bfloat16)
    assert np.array_equal(G.linear(a, torch.eye(16).to(torch.bfloat16)), G.widen(a))
    sel = torch.zeros((3, 16)); sel[0, 7] = 1; sel[1, 0] = 2; sel[2, 15] = -1
    c = G.linear(a, sel.to(torch.bfloat16))
    A = G.widen(a)
    assert np.array_equal(c, np.stack([A[:, 7], 2 * A[:, 0], -A[:, 15]], axis=1))


def test_product_of_powers_of_two_is_exact_and_not_transposed():
    # C[m, n] = sum_k 2^(m-k) 2^(k+n) = K 2^(m+n): exact, and asymmetric in (m, n) shapes
    M, N, K = 3, 5, 8
    a = bf([[2.0 ** (m - k) for k in range(K)] for m in range(M)])
    w = bf([[2.0 ** (k + n) for k in range(K)] for n in range(N)])
    c = G.linear(a, w)
    assert c.shape == (M, N)
    assert np.array_equal(c, np.array([[K * 2.0 ** (m + n) for n in range(N)] for m in range(M)]))


def test_linearity_and_sampled_rows_agree_with_the_full_product():
    g = torch.Generator().manual_seed(2)
    a1 = torch.randn((7, 40), generator=g).to(torch.bfloat16)
    a2 = torch.randn((7, 40), generator=g).to(torch.bfloat16)
    w = torch.randn((9, 40), generator=g).to(torch.bfloat16)
    s = G.widen(a1) + G.widen(a2)
    assert np.allclose(G.linear(a1, w) + G.linear(a2, w), s @ G.widen(w).T, rtol=1e-13, atol=1e-13)
    rows, cols = [0, 6, 3], [8, 0, 4]
    full = G.linear(a1, w)
    assert np.allclose(G.linear_rows(a1, w, rows, cols), full[rows, cols], rtol=1e-14, atol=1e-14)


def test_library_exports_every_gemm_symbol_and_rejects_bad_arguments():
    header = open(os.path.join(ROOT, "include", "xy_gemm.h")).read()
    declared = set(re.findall(r"\b(xy_gemm_[a-z_]+)\s*\(", header))
    assert declared == set(xg.GEMM_EXPORTS)
    lib = ctypes.CDLL(xb.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    L = xg._lib()
    one = ctypes.c_void_p(16)
    # argument checks come before any CUDA call, so they can be exercised without a GPU
    assert L.xy_gemm_run(one, 64, one, 64, one, 64, 4, 64, 64, 48, None) == xb.XY_ERR_UNSUPPORTED   # tile_n
    assert L.xy_gemm_run(one, 64, one, 64, one, 64, -1, 64, 64, 0, None) == xb.XY_ERR_INVALID_ARG   # M < 0
    assert L.xy_gemm_run(one, 64, one, 64, one, 64, 4, 60, 64, 0, None) == xb.XY_ERR_INVALID_ARG    # N % 8
    assert L.xy_gemm_run(one, 60, one, 64, one, 64, 4, 64, 64, 0, None) == xb.XY_ERR_INVALID_ARG    # lda < K
    assert L.xy_gemm_run(one, 64, one, 64, one, 64, 0, 64, 64, 0, None) == xb.XY_OK                 # M = 0: no-op
    assert L.xy_gemm_run(None, 64, one, 64, one, 64, 4, 64, 64, 0, None) == xb.XY_ERR_INVALID_ARG   # null
    assert L.xy_gemm_run(ctypes.c_void_p(8), 64, one, 64, one, 64, 4, 64, 64, 0, None) == xb.XY_ERR_INVALID_ARG
