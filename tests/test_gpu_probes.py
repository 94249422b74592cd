"""GPU probes that can tell a lost key tile, a lost KV split or a wrong page from rounding noise.

(1) Mutation self-test of the comparison: the GPU output of the same batch with 128 keys fewer -
    an ordinary valid run - must FAIL check_against_oracle against the reference of the full
    batch, at 8 k to 300 k tokens (the million-token case sits in test_gpu_parity.py).
(2) Tile-one-hot V: output element d is the probability mass of every 128-th key tile, checked
    element by element against the oracle with a relative bound.
(3) The product path's paged gather, bit-exact: rows whose softmax puts probability exactly 1 on
    one key must return that key's V row bit for bit - through the TMA producer, for every page
    size, for keys in last-page tails, for streaming and dense tasks, with and without KV splits."""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_18106_b200 import binding as xb
from paper_2412_18106_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu

KERNELS = [xb.XY_KERNEL_AUTO, xb.XY_KERNEL_MMA]
KNAMES = {xb.XY_KERNEL_AUTO: "auto", xb.XY_KERNEL_MMA: "mma"}


def _shorter(batch, by=128):
    """The same batch (same pool, same block table, same Q rows) with every kv_len cut by `by`."""
    reqs = [(int(batch.q_len[r]), int(batch.kv_len[r]) - by, int(batch.mask_kind[r]),
             batch.tree_parents(r)) for r in range(batch.num_requests)]
    b2 = W.custom(batch.name + "_short", batch.num_q_heads, batch.num_kv_heads, batch.page_size, reqs, seed=batch.seed)
    b2.block_table = batch.block_table
    b2.num_pages = batch.num_pages
    return b2


@pytest.mark.parametrize("kv", [8192, 65536, 300000])
def test_mutation_a_run_with_128_keys_fewer_fails_the_comparison(kv):
    rng = np.random.default_rng(kv)
    b = W.custom("mut", 8, 2, 128, [(1, kv, 0, None), (24, kv + 77, 1, W.random_tree(rng, 24, 6))], seed=kv,
                 spare_frac=0.01)
    t = W.make_tensors(b)
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    O, LSE = H.run_gpu(b, t)
    H.check_against_oracle(O, LSE, O_ref, LSE_ref, "full run")
    O_m, LSE_m = H.run_gpu(_shorter(b), t)
    with pytest.raises(AssertionError):
        H.check_against_oracle(O_m, LSE_m, O_ref, LSE_ref, "mutant")
    # the decode row alone (its history lost its last 128 keys; the new key moved too) also fails
    with pytest.raises(AssertionError):
        H.check_against_oracle(O_m[:1], LSE_m[:1], O_ref[:1], LSE_ref[:1], "mutant, decode row")


def check_onehot(O, O_ref, what):
    """Element-wise: |dO| <= 2^-7 |O_ref| + 2e-6 (one bf16 rounding of O is 2^-9 relative; the mass
    of a single 128-key tile is at least 1.2 % of an element at a million keys)."""
    d = np.abs(O - O_ref)
    bound = 2.0 ** -7 * np.abs(O_ref) + 2e-6
    assert np.all(d <= bound), "%s: %d elements off, worst %g against %g" % (
        what, int((d > bound).sum()), float(d.max()), float(O_ref.flat[np.argmax(d)]))


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAMES[k])
def test_tile_onehot_v_on_hybrid_batch_with_splits(kernel):
    rng = np.random.default_rng(3)
    reqs = [(1, 9000, 0, None), (1, 40000, 0, None), (300, 5000, 0, None), (33, 12345, 1, W.random_tree(rng, 33, 7)),
            (1, 127, 0, None), (1, 128, 0, None), (160, 0, 0, None)]
    b = W.custom("onehot", 8, 2, 128, reqs, seed=3)
    t = W.make_tensors(b)
    W.set_tile_onehot_v(b, t)
    ctx = H.make_ctx(b, kernel=kernel)
    info = ctx.plan_batch(b)
    assert info.num_merge_units > 0
    O, LSE = H.run_gpu(b, t, ctx=ctx)
    ctx.close()
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    H.check_against_oracle(O, LSE, O_ref, LSE_ref, "onehot")
    check_onehot(O, O_ref, "onehot")
    # masses of all tiles add up to one
    assert np.all(np.abs(O.sum(axis=-1) - 1.0) <= 2.0 ** -7)


def _dominant_case(page, kernel, reqs, positions, **ctx_kw):
    b = W.custom("dominant%d" % page, 8, 2, page, reqs, seed=page)
    t = W.make_tensors(b)
    W.set_dominant_keys(b, t, positions)
    ctx = H.make_ctx(b, kernel=kernel, **ctx_kw)
    info = ctx.plan_batch(b)
    O, LSE = H.run_gpu(b, t, ctx=ctx)
    ctx.close()
    qs = b.q_start
    G = b.num_q_heads // b.num_kv_heads
    for r in range(b.num_requests):
        j = int(positions[r])
        pg = int(b.block_table[r, j // page])
        for a in range(b.num_q_heads):
            want = t.v_pool[pg, a // G, j % page, :].float().numpy().astype(np.float64)
            got = O[int(qs[r]): int(qs[r + 1]), a, :]
            assert np.array_equal(got, np.broadcast_to(want, got.shape)), (
                "request %d head %d: O is not the V row of key %d" % (r, a, j))
    # LSE = the dominant score: scale * 128 * q_value * k_value, everything else underflows
    assert np.all(np.abs(LSE - H.SCALE * 128 * 4.0 * 8.0) <= 1e-3 * H.SCALE * 128 * 32.0)
    return info


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAMES[k])
@pytest.mark.parametrize("page", [16, 32, 64, 128])
def test_gather_through_the_product_path_is_bit_exact(kernel, page):
    """Decode rows (streaming tasks), prefill and verify rows (dense tasks), keys at position 0,
    at page and tile borders, in the ragged tail of the last page, and the new token itself."""
    rng = np.random.default_rng(page)
    reqs, pos = [], []
    for h, j in ((300, 0), (300, 299), (300, 300), (257, 255), (257, 256), (129, 127), (129, 128),
                 (5, 5), (1, 0), (0, 0), (page * 3 + 1, page * 3), (page * 3 - 1, page * 3 - 2)):
        reqs.append((1, h, 0, None))
        pos.append(j)
    for n, h, j in ((40, 500, 499), (40, 500, 0), (70, 131, 129), (200, 77, 64), (64, 0, 0), (130, 1000, 640)):
        reqs.append((n, h, 0, None))
        pos.append(j)
    for n, h, j in ((20, 300, 298), (5, 129, 0), (40, 1000, 999)):
        reqs.append((n, h, 1, W.random_tree(rng, n, 6)))
        pos.append(j)
    _dominant_case(page, kernel, reqs, pos)


@pytest.mark.parametrize("page", [16, 128])
def test_gather_is_bit_exact_across_kv_splits(page):
    """Long rows cut into KV splits: the dominant key sits in the first, a middle and the last
    split; the partials of the other splits carry weight exp(-hundreds) = 0 in the merge."""
    reqs = [(1, 20000, 0, None), (1, 20000, 0, None), (1, 20000, 0, None), (150, 9000, 0, None), (150, 9000, 0, None)]
    pos = [3, 10000, 20000, 8999, 4000]
    info = _dominant_case(page, xb.XY_KERNEL_AUTO, reqs, pos, num_workers=148)
    assert info.num_merge_units > 0


def test_tile_onehot_v_at_the_largest_sizes():
    """A million-token decode and a 64-node tree on 300 k tokens: every one of the ~7800 (~2300)
    key tiles carries at least 1.2 % (4 %) of one output element."""
    rng = np.random.default_rng(99)
    reqs = [(1, 1_000_003, 0, None), (64, 300_001, 1, W.random_tree(rng, 64, 8))]
    b = W.custom("max_onehot", 8, 2, 128, reqs, seed=98, spare_frac=0.01)
    t = W.make_tensors(b)
    W.set_tile_onehot_v(b, t)
    O, LSE = H.run_gpu(b, t)
    O_ref, LSE_ref = oracle.attention(b, t, H.SCALE)
    H.check_against_oracle(O, LSE, O_ref, LSE_ref, "max_onehot")
    check_onehot(O, O_ref, "max_onehot")
