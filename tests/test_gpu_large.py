"""Full-size members of the square sweep: the whole result against the oracle up to 8192^3, sampled rows,
columns and tiles above, and whole-matrix checksum identities (exact in int64) on the GPU's complete output."""
import numpy as np
import pytest

from oracle import mip_oracle as orc
from paper_2506_11728_b200 import inputs
from gpu_util import first_mismatch, run_gemm

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mg():
    from paper_2506_11728_b200 import binding
    binding.mipgemm_set_tuning()
    return binding


def checksum_identities(A, B, C, M, N, K, rng):
    """C x = A (B x) and y^T C = (y^T A) B for x, y in {ones, small random}; int64, exact."""
    C2 = C.reshape(M, N)
    A2 = A.reshape(M, K)
    B2 = B.reshape(N, K)                      # row j = column j of B
    step = 1024

    def a_times(v):                           # A @ v, v int64 [K]
        return np.concatenate([A2[i:i + step].astype(np.int64) @ v for i in range(0, M, step)])

    def bt_times(v):                          # B^T ... : (B x)[k] = sum_j B(k,j) x[j]
        acc = np.zeros(K, np.int64)
        for j in range(0, N, step):
            acc += v[j:j + step] @ B2[j:j + step].astype(np.int64)
        return acc

    for x in (np.ones(N, np.int64), rng.integers(-2, 3, size=N).astype(np.int64)):
        lhs = np.concatenate([C2[i:i + step].astype(np.int64) @ x for i in range(0, M, step)])
        assert np.array_equal(lhs, a_times(bt_times(x)))
    for y in (np.ones(M, np.int64), rng.integers(-2, 3, size=M).astype(np.int64)):
        lhs = np.zeros(N, np.int64)
        ya = np.zeros(K, np.int64)
        for i in range(0, M, step):
            lhs += y[i:i + step] @ C2[i:i + step].astype(np.int64)
            ya += y[i:i + step] @ A2[i:i + step].astype(np.int64)
        rhs = np.concatenate([B2[j:j + step].astype(np.int64) @ ya for j in range(0, N, step)])
        assert np.array_equal(lhs, rhs)


def sampled_parity(A, B, C, M, N, K, rng, n_rows=32, n_tiles=16, tile=128):
    C2 = C.reshape(M, N)
    A2 = A.reshape(M, K)
    B2 = B.reshape(N, K)
    rows = sorted(set([0, M - 1] + [int(v) for v in rng.integers(0, M, size=n_rows)]))
    want = orc.gemm(np.ascontiguousarray(A2[rows]).reshape(-1), B, len(rows), N, K).reshape(len(rows), N)
    assert np.array_equal(C2[rows], want), "row sample mismatch"
    cols = sorted(set([0, N - 1] + [int(v) for v in rng.integers(0, N, size=8)]))
    want = orc.gemm(A, np.ascontiguousarray(B2[cols]).reshape(-1), M, len(cols), K).reshape(M, len(cols))
    assert np.array_equal(C2[:, cols], want), "column sample mismatch"
    corners = [(0, 0), (0, N - tile), (M - tile, 0), (M - tile, N - tile)]
    straddle = [(128 - 64, 256 - 64), (M // 2 - 64, N // 2 - 64)]
    rand = [(int(rng.integers(0, M - tile)), int(rng.integers(0, N - tile))) for _ in range(n_tiles - 6)]
    for (i0, j0) in corners + straddle + rand:
        a = np.ascontiguousarray(A2[i0:i0 + tile]).reshape(-1)
        b = np.ascontiguousarray(B2[j0:j0 + tile]).reshape(-1)
        want = orc.gemm(a, b, tile, tile, K).reshape(tile, tile)
        assert np.array_equal(C2[i0:i0 + tile, j0:j0 + tile], want), "tile (%d,%d) mismatch" % (i0, j0)


@pytest.mark.parametrize("n", [4096, 8192, 16384])
def test_square_sweep_large_members(mg, n):
    rng = np.random.default_rng(n)
    A = inputs.uniform_s8(n * n, inputs.seed_for(2, n) + 1)
    B = inputs.uniform_s8(n * n, inputs.seed_for(2, n) + 2)
    C, path = run_gemm(mg, "s8", n, n, n, A, B)
    assert path & mg.PATH_MASK in (mg.PATH_DENSE, mg.PATH_DENSE_PAIR)
    if n <= 8192:       # the whole matrix against the oracle (seconds of CPU time up to this size)
        want = orc.gemm(A, B, n, n, n)
        assert np.array_equal(C, want), first_mismatch(C.reshape(n, n), want.reshape(n, n))
    else:               # above that: sampled rows, columns and tiles, exactly
        sampled_parity(A, B, C, n, n, n, rng)
    checksum_identities(A, B, C, n, n, n, rng)


def test_all_minus_128_at_16384(mg):
    n = 16384
    A = np.full(n * n, -128, np.int8)
    C, _ = run_gemm(mg, "s8", n, n, n, A, A)
    assert C.min() == C.max() == 16384 * n == 1 << 28


@pytest.mark.parametrize("T", [4096, 16384])
def test_bert_shapes_large_t_sampled(mg, T):
    rng = np.random.default_rng(T)
    for (name, N, K) in inputs.BERT_GEMMS:
        A = inputs.normal_s8(T * K, inputs.seed_for(4, N + K) + 1, 40.0)
        B = inputs.normal_s8(N * K, inputs.seed_for(4, N + K) + 2, 20.0)
        C, _ = run_gemm(mg, "s8", T, N, K, A, B)
        sampled_parity(A, B, C, T, N, K, rng, n_rows=16, n_tiles=8)
        checksum_identities(A, B, C, T, N, K, rng)


@pytest.mark.parametrize("M,N,K,accumulate", [(3_000_000, 1024, 32, False), (2_500_000, 1100, 48, True)])
def test_more_than_2_to_31_elements_of_c(mg, M, N, K, accumulate):
    """C with more than 2^31 elements (12 GB): every address computation must be 64-bit.  Rows around the
    2^31- and 2^32-element marks, the first and last rows and 300 random rows are checked against the oracle."""
    import torch
    A = inputs.uniform_s8(M * K, 41)
    B = inputs.uniform_s8(N * K, 42)
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    dC = torch.full((M * N,), 7, dtype=torch.int32, device="cuda")
    mg.mipgemm_s8s8s32(M, N, K, dA, K, dB, K, dC, N, accumulate)
    assert mg.mipgemm_device_status() == mg.OK
    marks = np.array([2 ** 31 // N - 1, 2 ** 31 // N, 2 ** 31 // N + 1, 2 ** 32 // N, 2 ** 32 // N + 1]) % M
    rows = np.unique(np.concatenate([np.arange(0, 4), np.arange(M - 4, M), marks,
                                     np.random.default_rng(0).integers(0, M, 300)]))
    got = dC.view(M, N)[torch.from_numpy(rows).cuda()].cpu().numpy()
    want = orc.gemm(np.ascontiguousarray(A.reshape(M, K)[rows]).reshape(-1), B, len(rows), N, K,
                    C=np.full(len(rows) * N, 7, np.int32), accumulate=accumulate).reshape(len(rows), N)
    assert np.array_equal(got, want)
