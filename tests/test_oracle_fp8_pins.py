"""Pins of the fp8 KV-cache oracle (test infrastructure; no GPU).

The paper defines no fp8 cache: format (e4m3), scale granularity (one fp32 per page and kv head,
K and V separately) and rounding are this build's reading - parity unpinned by the paper.  What
can be pinned is pinned: the byte decode against a library conversion for all 256 codes; with
scale = 1 and values representable in e4m3 the fp8 oracle must equal the bf16 oracle exactly; a
power-of-two scale must commute with the decode; and the invariants of the bf16 oracle (rows of p
sum to one is implied by the closed forms below) re-run on the fp8 path."""
import math

import numpy as np
import torch

import oracle
from paper_2412_18106_b200 import workloads as W

SCALE = 1.0 / math.sqrt(128.0)


def test_e4m3_decode_table_matches_the_library_cast():
    t = oracle.e4m3_table()
    ref = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).double().numpy()
    assert np.isnan(t[0x7F]) and np.isnan(t[0xFF]) and np.isnan(ref[0x7F]) and np.isnan(ref[0xFF])
    ok = ~np.isnan(ref)
    assert np.array_equal(t[ok], ref[ok])
    # spot values of the format definition: largest normal, smallest subnormal, signed zero
    assert t[0x7E] == 448.0 and t[0x01] == 2.0 ** -9 and t[0x08] == 2.0 ** -6 and t[0x38] == 1.0
    assert t[0x80] == 0.0 and math.copysign(1.0, t[0x80]) == -1.0 and t[0xFE] == -448.0


def _small_batch(page=16):
    rng = np.random.default_rng(5)
    reqs = [(9, 40, 0, None), (1, 77, 0, None), (6, 33, 1, W.random_tree(rng, 6, 4)), (3, 0, 0, None)]
    return W.custom("fp8pin", 8, 2, page, reqs, seed=5)


def test_unit_scale_on_representable_values_equals_the_bf16_oracle():
    b = _small_batch()
    t = W.make_tensors(b)
    # make K and V exactly representable in e4m3 (round once through the library cast)
    t.k_pool = t.k_pool.float().to(torch.float8_e4m3fn).float().to(torch.bfloat16)
    t.v_pool = t.v_pool.float().to(torch.float8_e4m3fn).float().to(torch.bfloat16)
    t8 = W.to_fp8_kv(t, unit_scale=True)
    assert torch.equal(t8.k_pool.view(torch.float8_e4m3fn).float(), t.k_pool.float())
    O, LSE = oracle.attention(b, t, SCALE)
    O8, LSE8 = oracle.attention_fp8(b, t8, SCALE)
    assert np.array_equal(O, O8) and np.array_equal(LSE, LSE8)
    # sampled rows agree with the whole batch
    req, head, row = np.array([0, 2, 3], np.int32), np.array([1, 7, 0], np.int32), np.array([8, 5, 2], np.int32)
    Or, Lr = oracle.attention_fp8(b, t8, SCALE, rows=(req, head, row))
    x = b.q_start[req] + row
    assert np.array_equal(Or, O8[x, head]) and np.array_equal(Lr, LSE8[x, head])


def test_scales_multiply_the_decoded_values():
    """K scale s_k multiplies every score: with all K scales equal to a power of two c, the result
    equals the unit-scale result at softmax scale c * sm_scale; V scales multiply O linearly, page
    by page (checked with two different scales on a request that spans two pages: O is the
    probability-weighted mix)."""
    b = W.custom("fp8scale", 4, 1, 16, [(1, 31, 0, None)], seed=9)   # 32 keys = 2 pages
    t = W.make_tensors(b)
    t8 = W.to_fp8_kv(t, unit_scale=True)
    O1, L1 = oracle.attention_fp8(b, t8, SCALE * 0.25)
    t8.k_scale = torch.full_like(t8.k_scale, 0.25)
    O2, L2 = oracle.attention_fp8(b, t8, SCALE)
    assert np.array_equal(O1, O2) and np.array_equal(L1, L2)
    # V scales 2 and 8 on the two pages of the request: O = 2 * (mass on page 0 part) + 8 * (page 1 part)
    pages = b.block_table[0, :2]
    keep0 = np.zeros(32, np.uint8)
    keep0[:16] = 1
    t8.v_scale = torch.ones_like(t8.v_scale)
    # per-page partial sums from the probabilities (independent route: P @ decoded V)
    Vd = t8.v_pool.view(torch.float8_e4m3fn).double().numpy()
    Kd = t8.k_pool.view(torch.float8_e4m3fn).double().numpy() * 0.25
    q = t.q.double().numpy()
    vs = np.array([2.0, 8.0])
    t8.v_scale[int(pages[0])] = 2.0
    t8.v_scale[int(pages[1])] = 8.0
    O3, L3 = oracle.attention_fp8(b, t8, SCALE)
    for a in range(4):
        K = np.concatenate([Kd[int(pages[0]), 0], Kd[int(pages[1]), 0]])
        V = np.concatenate([Vd[int(pages[0]), 0] * vs[0], Vd[int(pages[1]), 0] * vs[1]])
        s = SCALE * K @ q[0, a]
        p = np.exp(s - s.max())
        p /= p.sum()
        assert np.allclose(O3[0, a], p @ V, rtol=1e-12, atol=1e-14)
        assert abs(L3[0, a] - (s.max() + math.log(np.exp(s - s.max()).sum()))) < 1e-12


def test_fp8_oracle_against_torch_on_dequantised_tensors():
    """Library special case: dequantise with torch (float8 cast x scale, fp64), gather in python,
    softmax / logsumexp in torch fp64."""
    b = _small_batch(page=32)
    t8 = W.to_fp8_kv(W.make_tensors(b))
    O8, LSE8 = oracle.attention_fp8(b, t8, SCALE)
    Kd = t8.k_pool.view(torch.float8_e4m3fn).double() * t8.k_scale.double()[:, :, None, None]
    Vd = t8.v_pool.view(torch.float8_e4m3fn).double() * t8.v_scale.double()[:, :, None, None]
    qs = b.q_start
    for r in range(b.num_requests):
        n, h = int(b.q_len[r]), int(b.kv_len[r])
        L = n + h
        pages = torch.from_numpy(b.block_table[r, : -(-L // 32)].astype(np.int64))
        par = b.tree_parents(r)
        mask = torch.zeros((n, L), dtype=torch.bool)
        mask[:, :h] = True
        for i in range(n):
            if par is None:
                mask[i, h: h + i + 1] = True
            else:
                node = i
                while node >= 0:
                    mask[i, h + node] = True
                    node = int(par[node])
        for a in range(8):
            g = a // 4
            K = Kd[pages, g].reshape(-1, 128)[:L]
            V = Vd[pages, g].reshape(-1, 128)[:L]
            q = t8.q[int(qs[r]): int(qs[r + 1]), a].double()
            s = SCALE * q @ K.T
            s = torch.where(mask, s, torch.full_like(s, -float("inf")))
            O = torch.softmax(s, dim=-1) @ V
            lse = torch.logsumexp(s, dim=-1)
            assert np.allclose(O8[int(qs[r]): int(qs[r + 1]), a], O.numpy(), rtol=1e-11, atol=1e-13)
            assert np.allclose(LSE8[int(qs[r]): int(qs[r + 1]), a], lse.numpy(), rtol=1e-12, atol=1e-12)


def test_quantised_inputs_stay_close_to_the_bf16_inputs():
    """The generator's bytes and scales reproduce the bf16 pools within e4m3's half-ulp (2^-4
    relative to the element, or half a subnormal step of the page's scale)."""
    b = _small_batch()
    t = W.make_tensors(b)
    t8 = W.to_fp8_kv(t)
    for pool, q8, sc in ((t.k_pool, t8.k_pool, t8.k_scale), (t.v_pool, t8.v_pool, t8.v_scale)):
        deq = q8.view(torch.float8_e4m3fn).double() * sc.double()[:, :, None, None]
        err = (deq - pool.double()).abs()
        bound = pool.double().abs() * 2.0 ** -4 + sc.double()[:, :, None, None] * 2.0 ** -10
        assert bool((err <= bound).all())
        assert not bool(torch.isnan(deq).any())
