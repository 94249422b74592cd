"""SmoothGEMM on the GPU through the C-ABI against the fp64 oracle, element by element: the
virtual padding of M (Section 5.1) and the partial tiles in N and K must not change any result."""
import numpy as np
import pytest
import torch

from oracle import gemm_oracle as G
from paper_2412_18106_b200 import binding as xb
from paper_2412_18106_b200 import gemm as xg

pytestmark = pytest.mark.gpu


def check(M, N, K, tile_n, seed=0, lda=None, ldc=None):
    """Tolerance: the output is rounded once to bf16 (relative 2^-9 of the result, bounded here by
    2^-8 |ref|); the fp32 accumulation of K products of bf16 values adds at most about
    K 2^-24 sum|a||w|, far below that for K <= 8192; results near zero after cancellation get an
    absolute floor of 2^-8 sqrt(K) 2^-6 (a few fp32 roundings of partial sums of size sqrt(K))."""
    g = torch.Generator().manual_seed(seed)
    lda = K if lda is None else lda
    ldc = N if ldc is None else ldc
    a_buf = torch.randn((max(M, 1), lda), generator=g).to(torch.bfloat16)
    w = torch.randn((N, K), generator=g).to(torch.bfloat16)
    a = a_buf[:M, :K]
    c_buf = torch.full((max(M, 1) + 1, ldc), float("nan"), dtype=torch.bfloat16, device="cuda")
    c = c_buf[:M, :N]
    xg.xy_gemm_run(a_buf.cuda()[:M, :K], w.cuda(), c, tile_n=tile_n)
    assert xg.xy_gemm_device_status() == 0
    got = c.float().cpu().numpy().astype(np.float64)
    ref = G.linear(a.contiguous(), w)
    assert not np.isnan(got).any()
    tol = 2.0 ** -8 * np.abs(ref) + 2.0 ** -14 * np.sqrt(K)
    bad = np.abs(got - ref) > tol
    assert not bad.any(), (M, N, K, tile_n, float(np.abs(got - ref).max()), int(bad.sum()))
    # selective write: nothing outside [0, M) x [0, N) was touched
    rest = c_buf.float().cpu().numpy()
    assert np.isnan(rest[M:, :]).all() and np.isnan(rest[:M, N:]).all()


@pytest.mark.parametrize("tile_n", [32, 64, 128, 256])
@pytest.mark.parametrize("M", [1, 7, 16, 127, 128, 129, 300])
def test_any_token_count_matches_oracle(M, tile_n):
    check(M, 384, 320, tile_n, seed=M)  # N and K both end in partial tiles / chunks


@pytest.mark.parametrize("tile_n", [0, 32, 64, 128, 256])
def test_linear_shapes_several_tiles_per_sm(tile_n):
    check(1000, 1536, 1024, tile_n, seed=3)


def test_strided_rows_and_small_sizes():
    check(33, 64, 64, 128, seed=5, lda=96, ldc=80)
    check(5, 8, 8, 128, seed=6)
    check(200, 520, 72, 256, seed=7, lda=80, ldc=528)


def test_zero_rows_is_a_no_op():
    w = torch.zeros((64, 64), dtype=torch.bfloat16, device="cuda")
    a = torch.zeros((0, 64), dtype=torch.bfloat16, device="cuda")
    c = torch.zeros((0, 64), dtype=torch.bfloat16, device="cuda")
    xg.xy_gemm_run(a, w, c)
    assert xg.xy_gemm_device_status() == 0


def test_full_size_qkv_projection_sampled():
    """The QKV projection of the benchmark model at a full chunk: sampled outputs against dot
    products, and the whole output against the library GEMM within two bf16 roundings."""
    M, N, K = 4096, 6144, 4096
    g = torch.Generator(device="cuda").manual_seed(9)
    a = torch.randn((M, K), device="cuda", generator=g).to(torch.bfloat16)
    w = torch.randn((N, K), device="cuda", generator=g).to(torch.bfloat16)
    c = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    xg.xy_gemm_run(a, w, c)
    assert xg.xy_gemm_device_status() == 0
    rng = np.random.default_rng(1)
    rows = np.concatenate([rng.integers(0, M, size=60), [0, M - 1, 127, 128]])
    cols = np.concatenate([rng.integers(0, N, size=60), [0, N - 1, 255, 256]])
    ref = G.linear_rows(a.cpu(), w.cpu(), rows, cols)
    got = c[torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()].float().cpu().numpy()
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 2.0 ** -14 * np.sqrt(K))
    lib = (a @ w.T).float()
    d = (c.float() - lib).abs()
    assert float((d - 2.0 ** -7 * lib.abs()).max()) <= 2.0 ** -13 * np.sqrt(K)


@pytest.mark.parametrize("M", [1, 16, 33, 100, 128, 129, 300, 512])
@pytest.mark.parametrize("N,K", [(512, 4096), (4096, 1024), (1032, 2304), (4096, 14336)])
def test_small_token_counts_take_the_split_k_path(M, N, K):
    """tile_n = 0 with M <= 512 and few tiles splits K over a cluster; the sum of the slices
    must match the oracle like the single-CTA product does (ragged N, K not a multiple of the
    split, rows past M untouched)."""
    check(M, N, K, 0, seed=M + N)


@pytest.mark.parametrize("shape", [(600, 4000, 8264, 128), (640, 7936, 8200, 256), (1100, 4096, 8192, 0)])
def test_last_wave_split_along_k_with_scratch_matches_oracle_and_repeats_bitwise(shape):
    """More tiles than SMs, a thin last wave and a long K: with scratch memory the last wave's
    tiles are split along K over all SMs and a fix-up kernel adds the partial sums.  Ragged M, N
    and K included; the result must match the oracle, repeat bit for bit, and stay inside
    [0, M) x [0, N)."""
    M, N, K, tile_n = shape
    g = torch.Generator().manual_seed(K)
    a = torch.randn((M, K), generator=g).to(torch.bfloat16)
    w = torch.randn((N, K), generator=g).to(torch.bfloat16)
    ws = xg.xy_gemm_workspace(torch.device("cuda:0"))
    ws.fill_(0xFF)  # contents of the scratch must not matter
    c_buf = torch.full((M + 1, N + 8), float("nan"), dtype=torch.bfloat16, device="cuda")
    c = c_buf[:M, :N]
    xg.xy_gemm_run(a.cuda(), w.cuda(), c, tile_n=tile_n, workspace=ws)
    c2 = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    xg.xy_gemm_run(a.cuda(), w.cuda(), c2, tile_n=tile_n, workspace=ws)
    assert xg.xy_gemm_device_status() == 0
    assert torch.equal(c, c2)
    got = c.float().cpu().numpy().astype(np.float64)
    ref = G.linear(a, w)
    tol = 2.0 ** -8 * np.abs(ref) + 2.0 ** -14 * np.sqrt(K)
    bad = np.abs(got - ref) > tol
    assert not bad.any(), (shape, float(np.abs(got - ref).max()), int(bad.sum()))
    rest = c_buf.float().cpu().numpy()
    assert np.isnan(rest[M:, :]).all() and np.isnan(rest[:M, N:]).all()
    # without scratch the same call computes whole tiles: same result within the tolerance
    c3 = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    xg.xy_gemm_run(a.cuda(), w.cuda(), c3, tile_n=tile_n)
    assert not (np.abs(c3.float().cpu().numpy().astype(np.float64) - ref) > tol).any()


PAIR = xg.XY_GEMM_PAIR


@pytest.mark.parametrize("tile_n", [PAIR | 128, PAIR | 256])
@pytest.mark.parametrize("M", [1, 129, 255, 256, 257, 600])
def test_cta_pair_tiles_any_token_count_matches_oracle(M, tile_n):
    check(M, 392, 328, tile_n, seed=M)  # N and K end in partial tiles / chunks; rows of the peer CTA may all be padding


@pytest.mark.parametrize("tile_n", [PAIR | 128, PAIR | 256])
def test_cta_pair_tiles_several_tiles_per_pair_and_strided_rows(tile_n):
    check(1000, 5000, 1024, tile_n, seed=4)          # 4 x 20 (or 40) tiles over 74 pairs: two accumulators in use
    check(300, 520, 72, tile_n, seed=8, lda=80, ldc=528)


def test_library_choice_covers_pair_tiles():
    check(1024, 4096, 512, 0, seed=11)   # picks 256 x 256 pair tiles
    check(520, 28672, 128, 0, seed=12)   # 520 rows pad to 768: stays on single-CTA tiles


@pytest.mark.parametrize("seed", range(12))
def test_random_shapes_and_tile_choices(seed):
    """Random M, N, K (multiples of 8 for N and K), random row strides and every tile choice,
    pair tiles included."""
    rng = np.random.default_rng(seed)
    M = int(rng.integers(1, 700))
    N = 8 * int(rng.integers(1, 90))
    K = 8 * int(rng.integers(1, 90))
    tile_n = int(rng.choice([0, 32, 64, 128, 256, PAIR | 128, PAIR | 256]))
    lda = K + 8 * int(rng.integers(0, 3))
    ldc = N + 8 * int(rng.integers(0, 3))
    check(M, N, K, tile_n, seed=100 + seed, lda=lda, ldc=ldc)
