"""Pins for the fp64 CPU oracle: what the paper and the mathematics fix.

None of these re-types the oracle's formula against itself: they are invariants
(spec equivalences between request kinds), closed forms, an independently
written brute force (different formulation: dense boolean mask from walking the
parent array, no max subtraction, long double), and a library special case
(torch fp64 softmax / logsumexp on contiguous gathered K/V).
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2412_18106_b200 import workloads as W

SCALE = 1.0 / math.sqrt(128.0)


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.to(torch.float64).numpy()


def contiguous_kv(batch, tensors, r, g):
    """Logical K/V rows of request r / kv head g by direct indexing (python loop)."""
    L = int(batch.q_len[r] + batch.kv_len[r])
    B = batch.page_size
    K = np.zeros((L, batch.head_dim))
    V = np.zeros((L, batch.head_dim))
    for j in range(L):
        page = int(batch.block_table[r, j // B])
        K[j] = bf16_to_f64(tensors.k_pool[page, g, j % B])
        V[j] = bf16_to_f64(tensors.v_pool[page, g, j % B])
    return K, V


def dense_mask(batch, r):
    """Boolean [n, L] mask built independently: history visible; corner by kind."""
    n, h = int(batch.q_len[r]), int(batch.kv_len[r])
    M = np.zeros((n, n + h), dtype=bool)
    M[:, :h] = True
    if int(batch.mask_kind[r]) == W.MASK_CAUSAL:
        for i in range(n):
            M[i, h : h + i + 1] = True
    else:
        par = batch.tree_parents(r)
        for i in range(n):
            for jp in range(n):
                # jp is an ancestor-or-self of i ?
                node, hit = i, False
                while node != -1:
                    if node == jp:
                        hit = True
                        break
                    node = int(par[node])
                M[i, h + jp] = hit
    return M


def brute_force(batch, tensors, r, a):
    """Second formulation: exp without max subtraction, long double accumulators."""
    G = batch.num_q_heads // batch.num_kv_heads
    K, V = contiguous_kv(batch, tensors, r, a // G)
    M = dense_mask(batch, r)
    n = int(batch.q_len[r])
    q0 = int(batch.q_start[r])
    O = np.zeros((n, batch.head_dim))
    LSE = np.zeros(n)
    for i in range(n):
        q = bf16_to_f64(tensors.q[q0 + i, a]).astype(np.longdouble)
        num = np.zeros(batch.head_dim, dtype=np.longdouble)
        den = np.longdouble(0)
        for j in range(K.shape[0]):
            if not M[i, j]:
                continue
            w = np.exp(np.longdouble(SCALE) * np.dot(q, K[j].astype(np.longdouble)))
            num += w * V[j].astype(np.longdouble)
            den += w
        O[i] = (num / den).astype(np.float64)
        LSE[i] = float(np.log(den))
    return O, LSE


def small_batches():
    tree7 = [-1, 0, 0, 1, 1, 2, 5]
    return [
        W.custom("mixA", 4, 2, 4, [(5, 0, 0, None), (3, 6, 0, None), (1, 9, 0, None),
                                   (7, 5, 1, tree7)], seed=3),
        W.custom("mixB", 6, 3, 8, [(1, 0, 0, None), (2, 13, 1, [-1, -1]), (9, 3, 0, None)], seed=4),
        W.custom("mha", 2, 2, 2, [(4, 3, 0, None), (4, 3, 1, [-1, 0, 1, 1])], seed=5),
    ]


# ---------------------------------------------------------------- P9 brute force
@pytest.mark.parametrize("bi", range(3))
def test_brute_force_tiny(bi):
    b = small_batches()[bi]
    t = W.make_tensors(b)
    O, LSE = oracle.attention(b, t, SCALE)
    for r in range(b.num_requests):
        q0 = int(b.q_start[r])
        for a in range(b.num_q_heads):
            Ob, Lb = brute_force(b, t, r, a)
            n = int(b.q_len[r])
            np.testing.assert_allclose(O[q0 : q0 + n, a], Ob, rtol=0, atol=1e-12)
            np.testing.assert_allclose(LSE[q0 : q0 + n, a], Lb, rtol=0, atol=1e-12)


def test_mask_materialised_matches_independent_builder():
    for b in small_batches():
        t = W.make_tensors(b)
        for r in range(b.num_requests):
            _, M = oracle.probs(b, t, SCALE, r, 0)
            assert np.array_equal(M.astype(bool), dense_mask(b, r))


# ---------------------------------------------------------------- P10 library special case
@pytest.mark.parametrize("name", ["tiny_hybrid", "mid"])
def test_torch_fp64_library(name):
    if name == "tiny_hybrid":
        b = W.config1_tiny()
    else:
        rng = np.random.default_rng(11)
        b = W.custom("mid", 8, 2, 16, [(40, 77, 0, None), (1, 150, 0, None),
                                        (19, 60, 1, W.random_tree(rng, 19, 5))], seed=11)
    t = W.make_tensors(b)
    O, LSE = oracle.attention(b, t, SCALE)
    G = b.num_q_heads // b.num_kv_heads
    for r in range(b.num_requests):
        n, q0 = int(b.q_len[r]), int(b.q_start[r])
        M = torch.from_numpy(dense_mask(b, r))
        for a in range(b.num_q_heads):
            K, V = contiguous_kv(b, t, r, a // G)
            K, V = torch.from_numpy(K), torch.from_numpy(V)
            q = t.q[q0 : q0 + n, a].to(torch.float64)
            s = (q @ K.T) * SCALE + torch.where(M, 0.0, -math.inf)
            o = torch.softmax(s, dim=-1) @ V
            l = torch.logsumexp(s, dim=-1)
            np.testing.assert_allclose(O[q0 : q0 + n, a], o.numpy(), rtol=0, atol=1e-11)
            np.testing.assert_allclose(LSE[q0 : q0 + n, a], l.numpy(), rtol=0, atol=1e-11)


# ---------------------------------------------------------------- P1 rows sum to one
def test_probability_rows_sum_to_one():
    for b in small_batches() + [W.config1_tiny()]:
        t = W.make_tensors(b)
        _, _, psum = oracle.attention(b, t, SCALE, want_psum=True)
        assert np.all(np.abs(psum - 1.0) < 1e-12)
        for r in range(b.num_requests):
            P, M = oracle.probs(b, t, SCALE, r, b.num_q_heads - 1)
            assert np.all(P[M == 0] == 0.0)
            assert np.all(np.abs(P.sum(axis=1) - 1.0) < 1e-12)


# ---------------------------------------------------------------- shared-cache helpers
def shared_cache_pair(hq, hkv, page, total, specs, seed):
    """Two batches over the SAME cache: `full` = one causal prefill of `total` tokens
    from kv 0; `part` = the requests in `specs`, each (q_len, kv_len, kind, parents) with
    q_len + kv_len <= total, reading the same pages.  Q rows are taken from the full
    prompt's rows kv_len .. kv_len+q_len-1."""
    full = W.custom("full", hq, hkv, page, [(total, 0, 0, None)], seed=seed)
    tf = W.make_tensors(full)
    part = W.custom("part", hq, hkv, page, specs, seed=seed)
    # same physical pages: every partial request reads the prefix of the full request's table
    npg = part.block_table.shape[1]
    for r in range(part.num_requests):
        need = -(-(int(part.q_len[r]) + int(part.kv_len[r])) // page)
        part.block_table[r, :] = -1
        part.block_table[r, :need] = full.block_table[0, :need]
    part.num_pages = full.num_pages
    rows = []
    for r in range(part.num_requests):
        h, n = int(part.kv_len[r]), int(part.q_len[r])
        rows.append(tf.q[h : h + n])
    tp = W.Tensors(q=torch.cat(rows, dim=0).contiguous(), k_pool=tf.k_pool, v_pool=tf.v_pool)
    return full, tf, part, tp


# ---------------------------------------------------------------- P2 chunked == unchunked
def test_chunked_prefill_equals_unchunked():
    total = 53
    cuts = [0, 7, 8, 24, 41, 53]  # page 8: cuts on and off page boundaries
    specs = [(cuts[k + 1] - cuts[k], cuts[k], 0, None) for k in range(len(cuts) - 1)]
    full, tf, part, tp = shared_cache_pair(4, 2, 8, total, specs, seed=21)
    Of, Lf = oracle.attention(full, tf, SCALE)
    Op, Lp = oracle.attention(part, tp, SCALE)
    np.testing.assert_allclose(Op, Of, rtol=0, atol=1e-13)
    np.testing.assert_allclose(Lp, Lf, rtol=0, atol=1e-13)


# ---------------------------------------------------------------- P3 prefix reuse == full recompute
@pytest.mark.parametrize("prefix", [0, 1, 15, 16, 17, 37])
def test_prefix_reuse_equals_full_recompute(prefix):
    total = 48
    full, tf, part, tp = shared_cache_pair(4, 1, 16, total, [(total - prefix, prefix, 0, None)], seed=22)
    Of, Lf = oracle.attention(full, tf, SCALE)
    Op, Lp = oracle.attention(part, tp, SCALE)
    np.testing.assert_allclose(Op, Of[prefix:], rtol=0, atol=1e-13)
    np.testing.assert_allclose(Lp, Lf[prefix:], rtol=0, atol=1e-13)


# ---------------------------------------------------------------- P4 chain tree == causal
def test_chain_tree_equals_causal():
    n, h = 9, 21
    a = W.custom("causal", 4, 2, 4, [(n, h, W.MASK_CAUSAL, None)], seed=23)
    b = W.custom("chain", 4, 2, 4, [(n, h, W.MASK_TREE, W.chain_tree(n))], seed=23)
    ta, tb = W.make_tensors(a), W.make_tensors(b)
    assert torch.equal(ta.q, tb.q) and torch.equal(ta.k_pool, tb.k_pool)
    Oa, La = oracle.attention(a, ta, SCALE)
    Ob, Lb = oracle.attention(b, tb, SCALE)
    assert np.array_equal(Oa, Ob) and np.array_equal(La, Lb)


# ---------------------------------------------------------------- P5 decode == last prefill row
def test_decode_equals_last_prefill_row():
    total = 30
    full, tf, part, tp = shared_cache_pair(6, 2, 4, total, [(1, total - 1, 0, None)], seed=24)
    Of, Lf = oracle.attention(full, tf, SCALE)
    Op, Lp = oracle.attention(part, tp, SCALE)
    np.testing.assert_allclose(Op[0], Of[-1], rtol=0, atol=1e-13)
    np.testing.assert_allclose(Lp[0], Lf[-1], rtol=0, atol=1e-13)


# ---------------------------------------------------------------- P15 config 1 ties to P3 / P4
def test_config1_requests_are_the_invariants():
    b = W.config1_tiny()
    t = W.make_tensors(b)
    O, LSE = oracle.attention(b, t, SCALE)
    q0 = b.q_start
    # fourth request: 4-token chain at kv 200 == causal prefill of 4 tokens at kv 200
    c = W.config1_tiny()
    c.mask_kind = c.mask_kind.copy()
    c.mask_kind[3] = W.MASK_CAUSAL
    Oc, Lc = oracle.attention(c, t, SCALE, only=[3])
    assert np.array_equal(O[q0[3] : q0[4]], Oc[q0[3] : q0[4]])
    # second request: 64 new on 128 cached == rows 128..191 of a 192-token prefill over the same pages
    full = W.custom("full", 8, 2, 16, [(192, 0, 0, None)], seed=0)
    full.block_table = b.block_table[1:2, :12].copy()
    full.num_pages = b.num_pages
    qf = torch.zeros((192, 8, 128), dtype=torch.bfloat16)
    qf[128:] = t.q[q0[1] : q0[2]]
    Of, Lf = oracle.attention(full, W.Tensors(q=qf, k_pool=t.k_pool, v_pool=t.v_pool), SCALE)
    np.testing.assert_allclose(O[q0[1] : q0[2]], Of[128:], rtol=0, atol=1e-13)
    np.testing.assert_allclose(LSE[q0[1] : q0[2]], Lf[128:], rtol=0, atol=1e-13)
    # third request is a decode over 301 keys: last page holds 301 - 18*16 = 13 valid tokens
    P, M = oracle.probs(b, t, SCALE, 2, 0)
    assert P.shape == (1, 301) and M.sum() == 301


# ---------------------------------------------------------------- P6 closed forms
def _depths(par):
    d = np.zeros(len(par), dtype=int)
    for i, p in enumerate(par):
        d[i] = 1 if p < 0 else d[p] + 1
    return d


def test_closed_form_zero_query():
    rng = np.random.default_rng(31)
    par = W.random_tree(rng, 11, 4)
    b = W.custom("q0", 4, 2, 8, [(6, 10, 0, None), (11, 7, 1, par)], seed=31)
    t = W.make_tensors(b)
    t.q.zero_()
    O, LSE = oracle.attention(b, t, SCALE)
    G = 2
    for r in range(2):
        n, h, q0 = int(b.q_len[r]), int(b.kv_len[r]), int(b.q_start[r])
        M = dense_mask(b, r)
        cnt = (h + np.arange(1, n + 1)) if r == 0 else (h + _depths(par))
        for a in range(4):
            _, V = contiguous_kv(b, t, r, a // G)
            for i in range(n):
                assert M[i].sum() == cnt[i]
                np.testing.assert_allclose(LSE[q0 + i, a], math.log(cnt[i]), atol=1e-13)
                np.testing.assert_allclose(O[q0 + i, a], V[M[i]].mean(axis=0), atol=1e-13)


def test_closed_form_equal_keys_and_constant_values():
    b = W.custom("eq", 2, 1, 4, [(5, 6, 0, None)], seed=32)
    t = W.make_tensors(b)
    t.k_pool[:] = t.k_pool[0, 0, 0]  # every key row identical
    t.v_pool[:] = 0.75
    O, LSE = oracle.attention(b, t, SCALE)
    k = bf16_to_f64(t.k_pool[0, 0, 0])
    for a in range(2):
        for i in range(5):
            s = SCALE * float(np.dot(bf16_to_f64(t.q[i, a]), k))
            np.testing.assert_allclose(LSE[i, a], s + math.log(6 + i + 1), atol=1e-12)
            np.testing.assert_allclose(O[i, a], 0.75, atol=1e-13)


def test_closed_form_single_key():
    b = W.custom("one", 2, 2, 4, [(1, 0, 0, None), (1, 0, 1, [-1])], seed=33)
    t = W.make_tensors(b)
    O, LSE = oracle.attention(b, t, SCALE)
    for r in range(2):
        for a in range(2):
            K, V = contiguous_kv(b, t, r, a)
            s = SCALE * float(np.dot(bf16_to_f64(t.q[r, a]), K[0]))
            assert abs(LSE[r, a] - s) < 1e-14
            np.testing.assert_allclose(O[r, a], V[0], rtol=0, atol=1e-15)


# ---------------------------------------------------------------- P7 one-hot V
def test_one_hot_values_expose_attended_keys():
    b = W.custom("onehot", 2, 1, 4, [(3, 9, 0, None), (4, 5, 1, [-1, 0, 0, 2])], seed=34, permute_pages=True)
    t = W.make_tensors(b)
    D, B = 128, 4
    t.v_pool.zero_()
    for r in range(2):
        L = int(b.q_len[r] + b.kv_len[r])
        for j in range(L):
            t.v_pool[int(b.block_table[r, j // B]), 0, j % B, j % D] = 1.0
    O, _ = oracle.attention(b, t, SCALE)
    for r in range(2):
        q0, n = int(b.q_start[r]), int(b.q_len[r])
        L = n + int(b.kv_len[r])
        P, _ = oracle.probs(b, t, SCALE, r, 1)
        M = dense_mask(b, r)
        for i in range(n):
            o = O[q0 + i, 1]
            assert np.all(o[L:] == 0.0)
            assert np.all((o[:L] > 0) == M[i])  # exactly the allowed keys carry weight
            np.testing.assert_allclose(o[:L], P[i], atol=1e-15)


# ---------------------------------------------------------------- P8 star tree
def test_star_tree_rows_see_root_and_self_only():
    n, h = 6, 10
    par = [-1] + [0] * (n - 1)
    b = W.custom("star", 2, 1, 4, [(n, h, 1, par)], seed=35)
    t = W.make_tensors(b)
    P, M = oracle.probs(b, t, SCALE, 0, 0)
    for i in range(n):
        expect = np.zeros(n + h, dtype=np.uint8)
        expect[:h] = 1
        expect[h] = 1
        expect[h + i] = 1
        assert np.array_equal(M[i], expect)
    # swapping two sibling leaves (their Q rows and cache slots) swaps their output rows
    O1, L1 = oracle.attention(b, t, SCALE)
    t2 = W.make_tensors(b)
    i, j = 2, 4
    t2.q[[i, j]] = t.q[[j, i]]
    B = 4
    def slot(x):
        return int(b.block_table[0, (h + x) // B]), (h + x) % B
    (pi, si), (pj, sj) = slot(i), slot(j)
    for pool_new, pool_old in ((t2.k_pool, t.k_pool), (t2.v_pool, t.v_pool)):
        pool_new[pi, :, si] = pool_old[pj, :, sj]
        pool_new[pj, :, sj] = pool_old[pi, :, si]
    O2, L2 = oracle.attention(b, t2, SCALE)
    np.testing.assert_allclose(O2[i], O1[j], atol=1e-14)
    np.testing.assert_allclose(O2[j], O1[i], atol=1e-14)
    np.testing.assert_allclose(O2[1], O1[1], atol=1e-14)


# ---------------------------------------------------------------- P11 page permutation
def test_page_permutation_invariance_is_bit_exact():
    b = W.config1_tiny()
    t = W.make_tensors(b)
    O1, L1 = oracle.attention(b, t, SCALE)
    rng = np.random.default_rng(5)
    perm = rng.permutation(b.num_pages)  # new_page = perm[old_page]
    b2 = W.config1_tiny()
    bt = b.block_table.copy()
    bt[bt >= 0] = perm[bt[bt >= 0]]
    b2.block_table = bt
    k2, v2 = torch.empty_like(t.k_pool), torch.empty_like(t.v_pool)
    k2[torch.from_numpy(perm)] = t.k_pool
    v2[torch.from_numpy(perm)] = t.v_pool
    O2, L2 = oracle.attention(b2, W.Tensors(q=t.q, k_pool=k2, v_pool=v2), SCALE)
    assert np.array_equal(O1, O2) and np.array_equal(L1, L2)
    K1, V1 = oracle.gather(b, t, 1, 1)
    K2, V2 = oracle.gather(b2, W.Tensors(q=t.q, k_pool=k2, v_pool=v2), 1, 1)
    assert torch.equal(K1, K2) and torch.equal(V1, V2)


def test_gather_matches_direct_indexing():
    b = W.config1_tiny()
    t = W.make_tensors(b)
    for r in range(4):
        for g in range(2):
            K, V = oracle.gather(b, t, r, g)
            Kd, Vd = contiguous_kv(b, t, r, g)
            assert np.array_equal(bf16_to_f64(K), Kd) and np.array_equal(bf16_to_f64(V), Vd)


# ---------------------------------------------------------------- P12 key shift
def test_key_shift_moves_lse_only():
    b = W.custom("shift", 2, 1, 4, [(4, 7, 0, None)], seed=36)
    t = W.make_tensors(b)
    # small-integer data so that k + u is exact in bf16
    gen = torch.Generator().manual_seed(1)
    t.k_pool[:] = torch.randint(-3, 4, t.k_pool.shape, generator=gen).to(torch.bfloat16)
    t.q[:] = torch.randint(-2, 3, t.q.shape, generator=gen).to(torch.bfloat16)
    u = torch.randint(-2, 3, (128,), generator=gen).to(torch.bfloat16)
    O1, L1 = oracle.attention(b, t, SCALE)
    P1, _ = oracle.probs(b, t, SCALE, 0, 1)
    t.k_pool[:] = t.k_pool + u
    O2, L2 = oracle.attention(b, t, SCALE)
    P2, _ = oracle.probs(b, t, SCALE, 0, 1)
    np.testing.assert_allclose(P2, P1, atol=1e-14)
    np.testing.assert_allclose(O2, O1, atol=1e-13)
    for i in range(4):
        for a in range(2):
            shift = SCALE * float(np.dot(bf16_to_f64(t.q[i, a]), bf16_to_f64(u)))
            np.testing.assert_allclose(L2[i, a] - L1[i, a], shift, atol=1e-12)


# ---------------------------------------------------------------- P13 merge identity
def test_merge_of_any_partition_equals_unsplit():
    rng = np.random.default_rng(37)
    par = W.random_tree(rng, 9, 4)
    b = W.custom("merge", 4, 2, 4, [(5, 14, 0, None), (9, 11, 1, par)], seed=37)
    t = W.make_tensors(b)
    O, LSE = oracle.attention(b, t, SCALE)
    for r in range(2):
        n, L, q0 = int(b.q_len[r]), int(b.q_len[r] + b.kv_len[r]), int(b.q_start[r])
        for trial in range(3):
            C = 1 + trial * 2
            label = rng.integers(0, C, size=L)  # arbitrary, non-contiguous partition of the keys
            for a in (0, 3):
                for i in (0, n - 1):
                    Oc = np.zeros((C, 1, 128))
                    Lc = np.zeros((C, 1))
                    for c in range(C):
                        Oc[c, 0], Lc[c, 0] = oracle.attention_keys(b, t, SCALE, r, a, i, label == c)
                    Om, Lm = oracle.merge(Oc, Lc)
                    np.testing.assert_allclose(Om[0], O[q0 + i, a], atol=1e-12)
                    np.testing.assert_allclose(Lm[0], LSE[q0 + i, a], atol=1e-12)


def test_merge_closed_form_two_equal_chunks():
    # two chunks with the same LSE average their outputs; LSE grows by ln 2
    Oc = np.stack([np.full((2, 128), 1.0), np.full((2, 128), 3.0)])
    Lc = np.array([[0.5, -2.0], [0.5, -2.0]])
    O, L = oracle.merge(Oc, Lc)
    np.testing.assert_allclose(O, 2.0, atol=1e-15)
    np.testing.assert_allclose(L, Lc[0] + math.log(2.0), atol=1e-15)
    # an empty chunk (LSE = -inf) is ignored
    Lc2 = np.array([[0.5, -2.0], [-np.inf, -np.inf]])
    O2, L2 = oracle.merge(Oc, Lc2)
    np.testing.assert_allclose(O2, 1.0, atol=1e-15)
    np.testing.assert_allclose(L2, Lc2[0], atol=1e-15)


# ---------------------------------------------------------------- P14 GQA
def test_gqa_group_shares_kv_head_and_reduces_to_mha():
    b = W.custom("gqa", 6, 2, 4, [(3, 8, 0, None)], seed=38)
    t = W.make_tensors(b)
    t.q[:, 1] = t.q[:, 0]
    t.q[:, 2] = t.q[:, 0]  # heads 0..2 share kv head 0
    t.q[:, 3] = t.q[:, 0]  # head 3 uses kv head 1: must differ
    O, LSE = oracle.attention(b, t, SCALE)
    assert np.array_equal(O[:, 0], O[:, 1]) and np.array_equal(O[:, 0], O[:, 2])
    assert not np.allclose(O[:, 0], O[:, 3])
    # Hkv = Hq: q head a reads kv head a
    m = W.custom("mha", 3, 3, 4, [(3, 8, 0, None)], seed=39)
    tm = W.make_tensors(m)
    Om, _ = oracle.attention(m, tm, SCALE)
    for a in range(3):
        K, V = contiguous_kv(m, tm, 0, a)
        q = bf16_to_f64(tm.q[:, a])
        s = (q @ K.T) * SCALE
        s[~dense_mask(m, 0)] = -np.inf
        p = np.exp(s - s.max(axis=1, keepdims=True))
        p /= p.sum(axis=1, keepdims=True)
        np.testing.assert_allclose(Om[:, a], p @ V, atol=1e-12)


def test_sampled_rows_entry_matches_full():
    b = W.config1_tiny()
    t = W.make_tensors(b)
    O, LSE = oracle.attention(b, t, SCALE)
    req = [0, 1, 1, 2, 3, 3]
    head = [0, 7, 3, 5, 1, 6]
    row = [63, 0, 40, 0, 0, 3]
    Os, Ls = oracle.attention_rows(b, t, SCALE, req, head, row)
    for s in range(len(req)):
        x = int(b.q_start[req[s]]) + row[s]
        assert np.array_equal(Os[s], O[x, head[s]]) and Ls[s] == LSE[x, head[s]]


def test_tail_poison_does_not_change_the_result():
    b = W.config1_tiny()
    t = W.make_tensors(b)
    tp = W.make_tensors(b, tail_fill=1e30)
    O1, L1 = oracle.attention(b, t, SCALE)
    O2, L2 = oracle.attention(b, tp, SCALE)
    assert np.array_equal(O1, O2) and np.array_equal(L1, L2)


# ---------------------------------------------------------------- KV-cache append (next-row N1)
def test_append_kv_round_trip_and_untouched_slots():
    """Oracle append pinned by direct indexing: after the append, the cache slot of logical
    position kv_len + i of every request holds exactly the K / V heads of token i of the fused
    tensor, and no other slot changed."""
    rng = np.random.default_rng(41)
    b = W.custom("append", 6, 2, 4, [(5, 3, 0, None), (1, 9, 0, None), (7, 0, 1, W.random_tree(rng, 7, 3))], seed=41)
    t = W.make_tensors(b, fused_qkv=True)
    k0, v0 = t.k_pool.clone(), t.v_pool.clone()
    oracle.append_kv(b, t.qkv, t.k_pool, t.v_pool)
    touched = torch.zeros(t.k_pool.shape[:3], dtype=torch.bool)
    B, Hq, Hkv = b.page_size, b.num_q_heads, b.num_kv_heads
    for r in range(b.num_requests):
        for i in range(int(b.q_len[r])):
            tok = int(b.q_start[r]) + i
            j = int(b.kv_len[r]) + i
            page, slot = int(b.block_table[r, j // B]), j % B
            for g in range(Hkv):
                assert torch.equal(t.k_pool[page, g, slot], t.qkv[tok, Hq + g])
                assert torch.equal(t.v_pool[page, g, slot], t.qkv[tok, Hq + Hkv + g])
                touched[page, g, slot] = True
    assert torch.equal(t.k_pool[~touched], k0[~touched]) and torch.equal(t.v_pool[~touched], v0[~touched])
    # the gather of the oracle sees the appended rows at the end of each request
    K, V = oracle.gather(b, t, 0, 1)
    assert torch.equal(K[3:], t.qkv[0:5, Hq + 1]) and torch.equal(V[3:], t.qkv[0:5, Hq + Hkv + 1])
