"""Can the parity bounds see an error?  (No GPU: the oracle plays both sides.)

A comparison that an all-zero output passes proves nothing, and the absolute bounds alone behave
like that on long contexts, where |O| shrinks like 1/sqrt(keys).  Here a mutant - the exact
attention with one 128-key tile left out, or with the last tile missing - must FAIL
check_against_oracle, and the exact result rounded the way the GPU rounds it (P and O to bf16)
must PASS, at context lengths from 8 k to 300 k tokens."""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_18106_b200 import workloads as W
from tests import helpers as H


def _bf16(x):
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16).float().numpy().astype(np.float64)


@pytest.mark.parametrize("kv", [8192, 65536, 300000])
@pytest.mark.parametrize("onehot_v", [False, True])
def test_a_lost_key_tile_fails_the_bounds_and_bf16_rounding_passes(kv, onehot_v):
    b = W.custom("detector", 8, 2, 128, [(1, kv, 0, None)], seed=kv)
    t = W.make_tensors(b)
    if onehot_v:
        W.set_tile_onehot_v(b, t)
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    L = kv + 1
    for lo in (L // 128 // 2 * 128, L - 128):               # a tile in the middle, and the last 128 keys
        keep = np.ones(L, np.uint8)
        keep[lo: lo + 128] = 0
        O_m, LSE_m = np.zeros_like(O_ref), np.zeros_like(LSE_ref)
        for a in range(8):
            O_m[0, a], LSE_m[0, a] = oracle.attention_keys(b, t, H.SCALE, 0, a, 0, keep)
        with pytest.raises(AssertionError):
            H.check_against_oracle(_bf16(O_m), LSE_m.astype(np.float32).astype(np.float64), O_ref, LSE_ref, "mutant")
        if kv >= 65536 and not onehot_v:
            # 128 lost keys are invisible to the absolute bounds at these lengths: that is the point
            H.check_against_oracle(_bf16(O_m), LSE_m, O_ref, LSE_ref, "mutant, absolute bounds only", tight=False)
    # the exact result with the GPU's roundings passes the tight bounds
    O_gpu_like = _bf16(O_ref * (1.0 + np.random.default_rng(0).uniform(-2.0 ** -9, 2.0 ** -9, size=O_ref.shape)))
    H.check_against_oracle(O_gpu_like, LSE_ref.astype(np.float32).astype(np.float64), O_ref, LSE_ref, "rounded")


def test_an_all_zero_output_fails():
    b = W.custom("zero", 8, 2, 128, [(1, 300000, 0, None)], seed=1)
    t = W.make_tensors(b)
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    with pytest.raises(AssertionError):
        H.check_against_oracle(np.zeros_like(O_ref), LSE_ref, O_ref, LSE_ref, "zeros")
