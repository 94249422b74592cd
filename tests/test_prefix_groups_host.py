"""xy_attn_find_prefix_groups: shared-prefix groups read off the block tables (host only).
Checked against a slow restatement of the rule, against the group contract by brute force, on
the generator's own groups, and by handing the result to the planner."""
import numpy as np
import pytest

from paper_2412_18106_b200 import binding as xb
from paper_2412_18106_b200 import workloads as W

TILE = 128


def common_tokens(b, a, c, limit):
    """Leading tokens requests a and c share page by page, in whole 128-token tiles."""
    tokens = min(int(b.kv_len[a]), int(b.kv_len[c]), limit) // TILE * TILE
    n = 0
    for p in range(min(tokens // b.page_size, b.block_table.shape[1])):
        if b.block_table[a, p] != b.block_table[c, p] or b.block_table[a, p] < 0:
            break
        n += 1
    return n * b.page_size // TILE * TILE


def slow_groups(b, min_members, min_prefix):
    floor = max(min_prefix, TILE)
    dec = [int(b.q_len[r]) == 1 and int(b.mask_kind[r]) == 0 for r in range(b.num_requests)]
    out, r = [], 0
    while r < b.num_requests:
        if not dec[r] or b.kv_len[r] < floor:
            r += 1
            continue
        prefix, end = int(b.kv_len[r]) // TILE * TILE, r + 1
        while end < b.num_requests and dec[end]:
            c = common_tokens(b, r, end, prefix)
            if c < floor:
                break
            prefix, end = c, end + 1
        if end - r >= min_members:
            out.append((r, end - r, prefix))
            r = end
        else:
            r += 1
    return out


def check_contract(b, groups):
    seen = np.zeros(b.num_requests, bool)
    for first, n, prefix in groups:
        assert n >= 2 and prefix > 0 and prefix % TILE == 0
        assert not seen[first: first + n].any()
        seen[first: first + n] = True
        pages = prefix // b.page_size
        for r in range(first, first + n):
            assert b.q_len[r] == 1 and b.mask_kind[r] == 0 and b.kv_len[r] >= prefix
            assert np.array_equal(b.block_table[r, :pages], b.block_table[first, :pages])
            assert (b.block_table[r, :pages] >= 0).all()


def random_batch(seed, page_size):
    rng = np.random.default_rng(seed)
    reqs = []
    for _ in range(int(rng.integers(1, 40))):
        kind = rng.random()
        if kind < 0.7:
            reqs.append((1, int(rng.integers(0, 3000)), 0, None))
        elif kind < 0.85:
            reqs.append((int(rng.integers(2, 60)), int(rng.integers(0, 800)), 0, None))
        else:
            n = int(rng.integers(2, 12))
            reqs.append((n, int(rng.integers(0, 800)), 1, W.random_tree(rng, n, 4)))
    b = W.custom("groups_host", 8, 2, page_size, reqs, seed=seed)
    # overwrite leading pages of random runs of requests with those of the run's first request
    for _ in range(int(rng.integers(0, 6))):
        first = int(rng.integers(0, b.num_requests))
        n = int(rng.integers(2, 10))
        pages = int(rng.integers(1, 3000 // page_size))
        for r in range(first + 1, min(first + n, b.num_requests)):
            k = min(pages, b.block_table.shape[1])
            b.block_table[r, :k] = b.block_table[first, :k]
    return b


def find(b, min_members=2, min_prefix=128):
    return xb.xy_attn_find_prefix_groups(b.q_len, b.kv_len, b.mask_kind, b.block_table, b.page_size,
                                         min_members, min_prefix)


@pytest.mark.parametrize("page_size", [16, 32, 64, 128])
def test_random_block_tables(page_size):
    found_any = 0
    for seed in range(60):
        b = random_batch(1000 * page_size + seed, page_size)
        for min_members, min_prefix in [(2, 128), (3, 512), (2, 1)]:
            got = find(b, min_members, min_prefix)
            assert got == slow_groups(b, min_members, min_prefix)
            check_contract(b, got)
            found_any += len(got)
            if got:  # the planner accepts what the finder returns
                ctx = xb.XYAttn(8, 2, page_size, device=-1, max_requests=256, max_q_tokens=1 << 14,
                                max_pages_per_req=b.block_table.shape[1])
                ctx.plan_batch(b, groups=got)
                ctx.close()
    assert found_any > 20


def test_recovers_the_generators_groups():
    b, groups = W.shared_prefix_decode(seed=1, num_groups=3, members=9, prefix=1024, suffix_hi=500, hq=8, hkv=2,
                                       page_size=32)
    assert find(b) == [tuple(g) for g in groups]
    ctx = xb.XYAttn(8, 2, 32, device=-1, max_requests=256, max_pages_per_req=b.block_table.shape[1])
    n_auto = ctx.plan_batch(b, groups="auto").num_tasks
    assert n_auto == ctx.plan_batch(b, groups=groups).num_tasks != ctx.plan_batch(b).num_tasks
    ctx.close()


def test_no_groups_and_argument_checks():
    b = W.custom("plain", 8, 2, 16, [(1, 500, 0, None), (1, 500, 0, None), (7, 100, 0, None)], seed=3)
    assert find(b) == []
    b.block_table[1, :] = b.block_table[0, :]
    assert find(b) == [(0, 2, 384)]  # 500 cached tokens -> three whole tiles
    assert find(b, min_prefix=385) == []
    assert find(b, min_members=3) == []
    with pytest.raises(xb.XYAttnError):
        find(b, min_members=1)
    with pytest.raises(xb.XYAttnError):
        xb.xy_attn_find_prefix_groups(b.q_len, b.kv_len, b.mask_kind, b.block_table, 24)
    L = xb.load()
    assert L.xy_attn_find_prefix_groups(None, 0, None, 0, 16, 2, 128, None, 0, None) == xb.XY_ERR_INVALID_ARG
