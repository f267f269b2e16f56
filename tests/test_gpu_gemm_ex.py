"""GPU parity for the general entry point: signedness pairs x storage orders x C order.

The operands are generated in the requested storage order; the oracle (which knows one
canonical layout) gets the same matrices re-laid out with NumPy transposes (data movement only)."""
import itertools

import numpy as np
import pytest

from oracle import mip_oracle as orc
from paper_2506_11728_b200 import inputs
from gpu_util import to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mg():
    from paper_2506_11728_b200 import binding
    binding.mipgemm_set_tuning()
    return binding


def run_ex(mg, au, bu, ao, bo, ccol, M, N, K, *, pad=(0, 0, 0), accumulate=False, seed=0, misalign=0):
    lda = (M if ao else K) + pad[0]
    ldb = (N if bo else K) + pad[1]
    ldc = (M if ccol else N) + pad[2]
    a_rows, b_rows, c_rows = (K if ao else M), (K if bo else N), (N if ccol else M)
    A = (inputs.uniform_u8 if au else inputs.uniform_s8)(a_rows * lda, seed + 1)
    B = (inputs.uniform_u8 if bu else inputs.uniform_s8)(b_rows * ldb, seed + 2)
    C0 = inputs.uniform_s32(c_rows * ldc, seed + 3) if accumulate else np.full(c_rows * ldc, 0x7F7F7F7F, np.int32)
    # canonical views for the oracle: A as [M][K], B as [N][K], C as [M][N]
    A2 = A.reshape(a_rows, lda)[:, :(M if ao else K)]
    A_can = np.ascontiguousarray(A2.T if ao else A2)
    B2 = B.reshape(b_rows, ldb)[:, :(N if bo else K)]
    B_can = np.ascontiguousarray(B2.T if bo else B2)
    C2 = C0.reshape(c_rows, ldc)[:, :(M if ccol else N)]
    C_can = np.ascontiguousarray(C2.T if ccol else C2)
    want_can = orc.gemm(A_can.reshape(-1), B_can.reshape(-1), M, N, K, C=C_can.reshape(-1).copy(),
                        accumulate=accumulate).reshape(M, N)
    want = C0.reshape(c_rows, ldc).copy()
    want[:, :(M if ccol else N)] = want_can.T if ccol else want_can
    dA, _a = to_dev(A, misalign)
    dB, _b = to_dev(B, misalign)
    dC, _c = to_dev(C0)
    mg.mipgemm_gemm_ex(au, bu, ao, bo, ccol, M, N, K, dA, lda, dB, ldb, dC, ldc, accumulate)
    assert mg.mipgemm_device_status() == mg.OK
    got = dC.cpu().numpy().view(np.int32).reshape(c_rows, ldc)
    assert np.array_equal(got, want), "au=%d bu=%d ao=%d bo=%d ccol=%d %dx%dx%d path=%#x" % (
        au, bu, ao, bo, ccol, M, N, K, mg.mipgemm_last_path())
    return mg.mipgemm_last_path()


@pytest.mark.parametrize("ao,bo", list(itertools.product([0, 1], [0, 1])))
def test_storage_orders_aligned(mg, ao, bo):
    """M/N-contiguous operands read in place by MN-major shared-memory descriptors."""
    for (M, N, K) in [(128, 128, 128), (256, 256, 512), (304, 528, 400), (1024, 768, 1040)]:
        p = run_ex(mg, 0, 0, ao, bo, 0, M, N, K, seed=10 * ao + bo)
        assert not p & mg.PATH_REPACK
    run_ex(mg, 1, 0, ao, bo, 0, 640, 384, 272, accumulate=True, seed=33)


@pytest.mark.parametrize("ao,bo", [(0, 1), (1, 0), (1, 1)])
def test_storage_orders_on_both_kernel_forms(mg, ao, bo):
    """One CTA per tile and CTA pairs, tile widths 128 and 256, split K."""
    try:
        for force, bn in [(mg.PATH_DENSE, 128), (mg.PATH_DENSE, 256), (mg.PATH_DENSE_PAIR, 256), (mg.PATH_DENSE, 0)]:
            mg.mipgemm_set_tuning(block_n=bn, force_path=force)
            p = run_ex(mg, 1, 1, ao, bo, 0, 528, 784, 400, seed=90 + 2 * ao + bo)
            assert p & force and not p & mg.PATH_REPACK
            run_ex(mg, 0, 0, ao, bo, 0, 272, 144, 1024, accumulate=True, pad=(16, 32, 0), seed=95 + 2 * ao + bo)
        mg.mipgemm_set_tuning(split_k=3, force_path=mg.PATH_DENSE)
        p = run_ex(mg, 0, 1, ao, bo, 0, 208, 304, 2048, seed=99)
        assert p & mg.PATH_SPLITK
    finally:
        mg.mipgemm_set_tuning()


@pytest.mark.parametrize("au,bu", list(itertools.product([0, 1], [0, 1])))
def test_signedness_pairs(mg, au, bu):
    run_ex(mg, au, bu, 0, 0, 0, 300, 260, 400, seed=40 + 2 * au + bu)
    run_ex(mg, au, bu, 1, 1, 0, 320, 256, 384, seed=50 + 2 * au + bu)
    # extremes: every product at its largest magnitude
    M, N, K = 128, 128, 1024
    a_val, b_val = (255 if au else -128), (255 if bu else -128)
    A = np.full(M * K, a_val, dtype=np.uint8 if au else np.int8)
    B = np.full(N * K, b_val, dtype=np.uint8 if bu else np.int8)
    dA, _a = to_dev(A)
    dB, _b = to_dev(B)
    dC, _c = to_dev(np.zeros(M * N, np.int32))
    mg.mipgemm_gemm_ex(au, bu, 0, 0, 0, M, N, K, dA, K, dB, K, dC, N, 0)
    assert (dC.cpu().numpy().view(np.int32) == a_val * b_val * K).all()


@pytest.mark.parametrize("ao,bo", list(itertools.product([0, 1], [0, 1])))
def test_column_major_c(mg, ao, bo):
    run_ex(mg, 1, 0, ao, bo, 1, 304, 272, 400, seed=60 + 2 * ao + bo)
    run_ex(mg, 0, 0, ao, bo, 1, 130, 520, 144, accumulate=True, pad=(0, 0, 4), seed=70 + 2 * ao + bo)


def test_unaligned_orders_are_transposed_into_scratch(mg):
    p = run_ex(mg, 0, 0, 1, 1, 0, 130, 70, 100, pad=(1, 3, 1), seed=80)         # odd pitches
    assert p & mg.PATH_REPACK
    p = run_ex(mg, 1, 1, 1, 0, 1, 200, 96, 160, misalign=5, seed=81)            # misaligned bases
    assert p & mg.PATH_REPACK
    run_ex(mg, 0, 1, 0, 1, 0, 77, 300, 48, pad=(0, 5, 0), seed=82)


@pytest.mark.parametrize("ao,bo,ccol", list(itertools.product([0, 1], [0, 1], [0, 1])))
def test_tiny_and_degenerate_shapes(mg, ao, bo, ccol):
    for (M, N, K) in [(1, 1, 1), (5, 3, 2), (17, 1, 40), (1, 33, 16), (16, 16, 16), (2, 300, 1)]:
        run_ex(mg, 1, 1, ao, bo, ccol, M, N, K, seed=100 + M + N + K)
        run_ex(mg, 0, 0, ao, bo, ccol, M, N, K, accumulate=True, seed=120 + M + N + K)
    # K == 0: C is zero-filled or left alone; empty problems are no-ops
    dC, _c = to_dev(np.full(6 * 8, 7, np.int32))
    mg.mipgemm_gemm_ex(0, 1, ao, bo, ccol, 6, 8, 0, 0, 8, 0, 8, dC, 8, 0)
    out = dC.cpu().numpy().view(np.int32).reshape(-1, 8)
    if ccol:        # 8 columns of 6 elements, pitch 8: the two padding elements of each keep their value
        assert (out[:, :6] == 0).all() and (out[:, 6:] == 7).all()
    else:
        assert (out == 0).all()
    mg.mipgemm_gemm_ex(0, 1, ao, bo, ccol, 0, 8, 5, 0, 8, 0, 8, dC, 8, 0)
    assert mg.mipgemm_last_path() == mg.PATH_TRIVIAL


def test_ex_argument_errors(mg):
    a = b = c = 256
    f = mg.mipgemm_gemm_ex
    assert f(0, 0, 2, 0, 0, 4, 4, 16, a, 16, b, 16, c, 4, 0, 0, check=False) == mg.ERR_INVALID_ARG
    assert f(0, 0, 1, 0, 0, 8, 4, 16, a, 7, b, 16, c, 4, 0, 0, check=False) == mg.ERR_INVALID_ARG    # lda < M
    assert f(0, 0, 0, 1, 0, 8, 4, 16, a, 16, b, 3, c, 4, 0, 0, check=False) == mg.ERR_INVALID_ARG    # ldb < N
    assert f(0, 0, 0, 0, 1, 8, 4, 16, a, 16, b, 16, c, 7, 0, 0, check=False) == mg.ERR_INVALID_ARG   # ldc < M
    assert f(1, 1, 0, 0, 0, 4, 4, 33026, a, 33026, b, 33026, c, 4, 0, 0, check=False) == mg.ERR_K_TOO_LARGE
    assert f(0, 1, 0, 0, 0, 4, 4, 65794, a, 65794, b, 65794, c, 4, 0, 0, check=False) == mg.ERR_K_TOO_LARGE
