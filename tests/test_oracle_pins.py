"""Pins for the CPU oracle: it is checked against things other than itself.

Each test fixes one aspect that a plausible mistake would break: loop bounds and
pitch indexing (brute force with a differently organised pure-Python routine),
K count (all-ones), operand orientation (identity), widening / signedness
(extremes), C_in handling (accumulate doubling), the int64 -> int32 guard
(K = 131071 vs 131072), whole-matrix checksum identities, NumPy's own integer
matmul, and for the convolution: explicit im2col + GEMM, 1x1 == GEMM and
one-hot filters == shifted strided copies.
"""
import numpy as np
import pytest

from oracle import mip_oracle as orc
from paper_2506_11728_b200 import inputs


# ---------------------------------------------------------------------------
# P1: brute force, written independently (column-outer order, Python ints,
# running pointers instead of index products).
# ---------------------------------------------------------------------------
def brute_gemm(a_unsigned, M, N, K, A, lda, B, ldb, C, ldc, accumulate):
    A = [int(v) for v in A]
    B = [int(v) for v in B]
    out = [int(v) for v in C]
    for j in range(N):
        pb0 = j * ldb
        for i in range(M):
            pa = i * lda
            pb = pb0
            tot = 0
            for _ in range(K):
                av = A[pa]
                if a_unsigned and av < 0:
                    av += 256
                tot += av * B[pb]
                pa += 1
                pb += 1
            pos = i * ldc + j
            out[pos] = tot + (out[pos] if accumulate else 0)
    return out


def _rand_case(rng, M, N, K, a_unsigned):
    lda = K + int(rng.integers(0, 4))
    ldb = K + int(rng.integers(0, 4))
    ldc = N + int(rng.integers(0, 4))
    A = rng.integers(0, 256, size=max(M * lda, 1), dtype=np.int64).astype(np.uint8)
    if not a_unsigned:
        A = A.view(np.int8)
    B = rng.integers(-128, 128, size=max(N * ldb, 1), dtype=np.int64).astype(np.int8)
    C = rng.integers(-(1 << 20), 1 << 20, size=max(M * ldc, 1), dtype=np.int64).astype(np.int32)
    return A, lda, B, ldb, C, ldc


@pytest.mark.parametrize("a_unsigned", [0, 1])
@pytest.mark.parametrize("accumulate", [0, 1])
def test_p1_brute_force_all_tiny_shapes(a_unsigned, accumulate):
    rng = np.random.default_rng(1234 + 2 * a_unsigned + accumulate)
    shapes = [(m, n, k) for m in range(1, 10) for n in range(1, 10) for k in range(1, 10)]
    shapes += [tuple(int(v) for v in rng.integers(1, 34, size=3)) for _ in range(12)]
    for (M, N, K) in shapes:
        A, lda, B, ldb, C, ldc = _rand_case(rng, M, N, K, a_unsigned)
        want = brute_gemm(a_unsigned, M, N, K, A.view(np.int8) if not a_unsigned else A.astype(np.int64),
                          lda, B, ldb, C, ldc, accumulate)
        got = orc.gemm(A, B, M, N, K, lda=lda, ldb=ldb, C=C.copy(), ldc=ldc, accumulate=bool(accumulate))
        assert [int(v) for v in got] == want, (M, N, K)


def test_p1_padding_columns_of_c_untouched():
    rng = np.random.default_rng(7)
    M, N, K, ldc = 5, 3, 4, 7
    A = rng.integers(-128, 128, size=M * K).astype(np.int8)
    B = rng.integers(-128, 128, size=N * K).astype(np.int8)
    C = np.full(M * ldc, 0x7F7F7F7F, dtype=np.int32)
    out = orc.gemm(A, B, M, N, K, C=C, ldc=ldc)
    view = out.reshape(M, ldc)
    assert (view[:, N:] == 0x7F7F7F7F).all()
    assert (view[:, :N] != 0x7F7F7F7F).all()


# ---------------------------------------------------------------------------
# P2 / P3 / P4 / P5 / P6: closed forms.
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("K", [1, 31, 777])
def test_p2_all_ones_counts_k(K):
    M, N = 9, 11
    A = np.ones(M * K, dtype=np.int8)
    B = np.ones(N * K, dtype=np.int8)
    assert (orc.gemm(A, B, M, N, K) == K).all()


def test_p3_identity_b_returns_a():
    M, K = 13, 17
    A = inputs.uniform_s8(M * K, 3)
    B = np.eye(K, dtype=np.int8).reshape(-1)          # column j holds e_j
    C = orc.gemm(A, B, M, K, K)
    assert (C.reshape(M, K) == A.reshape(M, K).astype(np.int32)).all()


def test_p3_identity_a_returns_b_transposed_storage():
    K, N = 11, 19
    B = inputs.uniform_s8(N * K, 4)                   # B(k,j) = B[j*K + k]
    A = np.eye(K, dtype=np.int8).reshape(-1)
    C = orc.gemm(A, B, K, N, K).reshape(K, N)         # C(i,j) = B(i,j)
    assert (C == B.reshape(N, K).T.astype(np.int32)).all()


@pytest.mark.parametrize("a_val,b_val,dtype,per_k", [
    (-128, -128, np.int8, 16384),
    (-128, 127, np.int8, -16256),
    (255, -128, np.uint8, -32640),
    (255, 127, np.uint8, 32385),
])
def test_p4_extremes(a_val, b_val, dtype, per_k):
    M, N, K = 3, 4, 1000
    A = np.full(M * K, a_val, dtype=dtype)
    B = np.full(N * K, b_val, dtype=np.int8)
    assert (orc.gemm(A, B, M, N, K) == per_k * K).all()


def test_p4_all_minus_128_k16384():
    M, N, K = 2, 2, 16384
    A = np.full(M * K, -128, dtype=np.int8)
    B = np.full(N * K, -128, dtype=np.int8)
    assert (orc.gemm(A, B, M, N, K) == 1 << 28).all()


def test_p5_accumulate_doubles():
    M, N, K = 21, 14, 65
    A = inputs.uniform_s8(M * K, 11)
    B = inputs.uniform_s8(N * K, 12)
    once = orc.gemm(A, B, M, N, K)
    twice = orc.gemm(A, B, M, N, K, C=once.copy(), accumulate=True)
    assert (twice.astype(np.int64) == 2 * once.astype(np.int64)).all()
    # accumulate=0 must ignore whatever C held before
    poisoned = orc.gemm(A, B, M, N, K, C=np.full(M * N, 0x7F7F7F7F, dtype=np.int32))
    assert (poisoned == once).all()


def test_p6_range_check():
    A = np.full(131072, -128, dtype=np.int8)
    B = np.full(131072, -128, dtype=np.int8)
    ok = orc.gemm(A[:131071], B[:131071], 1, 1, 131071)
    assert int(ok[0]) == 2147467264
    with pytest.raises(orc.OracleOverflow):
        orc.gemm(A, B, 1, 1, 131072)
    # u8 mode: 255 * -128 * 65793 = -2147483520 fits, one more k does not
    Au = np.full(65794, 255, dtype=np.uint8)
    Bu = np.full(65794, -128, dtype=np.int8)
    assert int(orc.gemm(Au[:65793], Bu[:65793], 1, 1, 65793)[0]) == -32640 * 65793
    with pytest.raises(orc.OracleOverflow):
        orc.gemm(Au, Bu, 1, 1, 65794)
    # accumulate pushing past the top
    C = np.array([2147483647], dtype=np.int32)
    with pytest.raises(orc.OracleOverflow):
        orc.gemm(np.ones(1, np.int8), np.ones(1, np.int8), 1, 1, 1, C=C, accumulate=True)


# ---------------------------------------------------------------------------
# P7 / P8: checksum identities and NumPy's integer matmul (exact, independent).
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("mode", ["s8", "u8"])
def test_p7_checksum_identities(mode):
    M, N, K = 300, 257, 515
    A = inputs.uniform_s8(M * K, 21) if mode == "s8" else inputs.uniform_u8(M * K, 21)
    B = inputs.uniform_s8(N * K, 22)
    C = orc.gemm(A, B, M, N, K).reshape(M, N).astype(np.int64)
    A64 = A.reshape(M, K).astype(np.int64)
    B64 = B.reshape(N, K).astype(np.int64)            # row j = column j of B
    rng = np.random.default_rng(5)
    for x in (np.ones(N, np.int64), rng.integers(-3, 4, size=N)):
        assert (C @ x == A64 @ (B64.T @ x)).all()
    for y in (np.ones(M, np.int64), rng.integers(-3, 4, size=M)):
        assert (y @ C == (y @ A64) @ B64.T).all()


@pytest.mark.parametrize("mode,M,N,K", [("s8", 64, 48, 96), ("u8", 129, 200, 333), ("s8", 512, 512, 512)])
def test_p8_numpy_integer_matmul(mode, M, N, K):
    A = inputs.uniform_s8(M * K, 31) if mode == "s8" else inputs.uniform_u8(M * K, 31)
    B = inputs.uniform_s8(N * K, 32)
    want = A.reshape(M, K).astype(np.int64) @ B.reshape(N, K).astype(np.int64).T
    got = orc.gemm(A, B, M, N, K).reshape(M, N)
    assert (got.astype(np.int64) == want).all()


def test_p8_with_pitches_and_accumulate():
    M, N, K, lda, ldb, ldc = 37, 29, 61, 64, 70, 33
    A = inputs.uniform_u8(M * lda, 41)
    B = inputs.uniform_s8(N * ldb, 42)
    C0 = inputs.uniform_s32(M * ldc, 43)
    want = C0.reshape(M, ldc).astype(np.int64).copy()
    want[:, :N] += A.reshape(M, lda)[:, :K].astype(np.int64) @ B.reshape(N, ldb)[:, :K].astype(np.int64).T
    got = orc.gemm(A, B, M, N, K, lda=lda, ldb=ldb, C=C0.copy(), ldc=ldc, accumulate=True)
    assert (got.reshape(M, ldc).astype(np.int64) == want).all()


# ---------------------------------------------------------------------------
# P9: convolution.
# ---------------------------------------------------------------------------
def im2col_matrix(X, R, S, stride, pad, dil):
    """Explicit augmented matrix, rows = output pixels, k = (r*S + s)*Cin + c."""
    Nb, H, W, Cin = X.shape
    Ho, Wo = orc.conv_out_hw(H, W, R, S, stride, pad, dil)
    out = np.zeros((Nb * Ho * Wo, R * S * Cin), dtype=np.uint8)
    row = 0
    for n in range(Nb):
        for ho in range(Ho):
            for wo in range(Wo):
                for r in range(R):
                    h = ho * stride[0] - pad[0] + r * dil[0]
                    for s in range(S):
                        w = wo * stride[1] - pad[1] + s * dil[1]
                        if 0 <= h < H and 0 <= w < W:
                            k0 = (r * S + s) * Cin
                            out[row, k0:k0 + Cin] = X[n, h, w]
                row += 1
    return out


CONV_CASES = [
    # Nb, H, W, Cin, Cout, R, S, stride, pad, dil
    (2, 7, 6, 5, 4, 3, 3, (1, 1), (1, 1), (1, 1)),
    (1, 9, 8, 3, 6, 3, 2, (2, 1), (1, 0), (1, 1)),
    (2, 8, 8, 4, 3, 1, 1, (2, 2), (0, 0), (1, 1)),
    (1, 10, 9, 2, 5, 3, 3, (1, 2), (2, 2), (2, 2)),
    (1, 12, 12, 3, 4, 7, 7, (2, 2), (3, 3), (1, 1)),
]


@pytest.mark.parametrize("case", CONV_CASES)
def test_p9_conv_equals_im2col_gemm(case):
    Nb, H, W, Cin, Cout, R, S, stride, pad, dil = case
    X = inputs.uniform_u8(Nb * H * W * Cin, 51).reshape(Nb, H, W, Cin)
    Wt = inputs.uniform_s8(Cout * R * S * Cin, 52).reshape(Cout, R, S, Cin)
    Y = orc.conv(X, Wt, stride=stride, pad=pad, dil=dil)
    cols = im2col_matrix(X, R, S, stride, pad, dil)
    want = cols.astype(np.int64) @ Wt.reshape(Cout, -1).astype(np.int64).T
    assert (Y.reshape(-1, Cout).astype(np.int64) == want).all()
    # and through the GEMM oracle on the same augmented matrix
    Mg, Kg = cols.shape
    G = orc.gemm(np.ascontiguousarray(cols).reshape(-1), Wt.reshape(-1), Mg, Cout, Kg)
    assert (G.reshape(Mg, Cout) == Y.reshape(-1, Cout)).all()


def test_p9_pointwise_conv_is_plain_gemm():
    Nb, H, W, Cin, Cout = 2, 5, 4, 16, 8
    X = inputs.uniform_u8(Nb * H * W * Cin, 61).reshape(Nb, H, W, Cin)
    Wt = inputs.uniform_s8(Cout * Cin, 62).reshape(Cout, 1, 1, Cin)
    Y = orc.conv(X, Wt)
    G = orc.gemm(X.reshape(-1), Wt.reshape(-1), Nb * H * W, Cout, Cin)
    assert (Y.reshape(-1) == G).all()


@pytest.mark.parametrize("stride,pad,dil", [((1, 1), (1, 1), (1, 1)), ((2, 2), (1, 1), (1, 1)),
                                           ((1, 2), (2, 1), (2, 1)), ((3, 1), (0, 2), (1, 2))])
def test_p9_one_hot_filter_is_shifted_copy(stride, pad, dil):
    Nb, H, W, Cin, R, S = 1, 9, 10, 3, 3, 3
    X = inputs.uniform_u8(Nb * H * W * Cin, 71).reshape(Nb, H, W, Cin)
    Ho, Wo = orc.conv_out_hw(H, W, R, S, stride, pad, dil)
    for (r, s, c) in [(0, 0, 0), (1, 2, 1), (2, 1, 2), (2, 2, 0)]:
        Wt = np.zeros((1, R, S, Cin), dtype=np.int8)
        Wt[0, r, s, c] = -1
        Y = orc.conv(X, Wt, stride=stride, pad=pad, dil=dil)
        for ho in range(Ho):
            for wo in range(Wo):
                h = ho * stride[0] - pad[0] + r * dil[0]
                w = wo * stride[1] - pad[1] + s * dil[1]
                want = -int(X[0, h, w, c]) if (0 <= h < H and 0 <= w < W) else 0
                assert int(Y[0, ho, wo, 0]) == want


def test_p9_conv_accumulate():
    X = inputs.uniform_u8(2 * 6 * 6 * 4, 81).reshape(2, 6, 6, 4)
    Wt = inputs.uniform_s8(5 * 3 * 3 * 4, 82).reshape(5, 3, 3, 4)
    once = orc.conv(X, Wt, pad=(1, 1))
    twice = orc.conv(X, Wt, pad=(1, 1), Y=once.copy(), accumulate=True)
    assert (twice.astype(np.int64) == 2 * once.astype(np.int64)).all()


# ---------------------------------------------------------------------------
# Input generators: determinism and ranges (no method arithmetic in there).
# ---------------------------------------------------------------------------
def test_inputs_deterministic_and_in_range():
    a = inputs.uniform_s8(5000, 9)
    assert (a == inputs.uniform_s8(5000, 9)).all() and (a[:100] == inputs.uniform_s8(100, 9)).all()
    assert a.min() == -128 and a.max() == 127
    u = inputs.uniform_u8(5000, 9)
    assert u.min() == 0 and u.max() == 255
    n = inputs.normal_s8(20000, 9, 32.0, -127, 127)
    assert n.min() >= -127 and n.max() <= 127 and 28 < n.astype(np.float64).std() < 36
    c = inputs.uniform_s32(5000, 9)
    assert c.min() >= -(1 << 20) and c.max() <= (1 << 20)
    assert sum(x[0] for x in inputs.RESNET50_CONVS) == 53 and len(inputs.RESNET50_CONVS) == 23


# ---------------------------------------------------------------------------
# Dequantisation C^r = s * C^q: closed forms and NumPy's own float64 product.
# ---------------------------------------------------------------------------
def test_dequant_closed_forms():
    Cq = np.array([0, 1, -1, 2147483647, -2147483648, 16777217, -123456789], dtype=np.int32)
    assert np.array_equal(orc.dequant(Cq, 1.0), Cq.astype(np.float64))
    assert np.array_equal(orc.dequant(Cq, 0.0), np.zeros(7))
    assert np.array_equal(orc.dequant(Cq, -0.5), Cq.astype(np.float64) * -0.5)        # power of two: exact
    assert np.array_equal(orc.dequant(Cq, 2.0 ** -20), Cq.astype(np.float64) / 1048576.0)
    s = float(np.float32(0.0123))
    got = orc.dequant(Cq, s)
    assert np.array_equal(got, np.multiply(Cq.astype(np.float64), s))                 # library product
    # the product of a 32-bit integer and a binary32 scale is exact in binary64: compare with
    # exact rational arithmetic
    from fractions import Fraction
    for c, g in zip(Cq.tolist(), got.tolist()):
        assert Fraction(g) == Fraction(c) * Fraction(s)
    two_d = orc.dequant(Cq[:6].reshape(2, 3), 3.0)
    assert two_d.shape == (2, 3) and two_d[1, 2] == 3.0 * 16777217


# ---------------------------------------------------------------------------
# Unsigned B (all four signedness pairs): extremes, brute force, NumPy.
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("a_dt,b_dt,a_val,b_val", [
    (np.uint8, np.uint8, 255, 255), (np.int8, np.uint8, -128, 255), (np.int8, np.uint8, 127, 255),
    (np.uint8, np.uint8, 1, 200)])
def test_unsigned_b_extremes(a_dt, b_dt, a_val, b_val):
    M, N, K = 2, 3, 500
    A = np.full(M * K, a_val, dtype=a_dt)
    B = np.full(N * K, b_val, dtype=b_dt)
    assert (orc.gemm(A, B, M, N, K) == a_val * b_val * K).all()      # 200 and 255 really are 200 and 255


def test_unsigned_b_matches_numpy_and_brute_force():
    rng = np.random.default_rng(77)
    for a_dt in (np.int8, np.uint8):
        M, N, K = 23, 17, 45
        A = rng.integers(0, 256, size=M * K).astype(np.uint8).view(a_dt)
        B = rng.integers(0, 256, size=N * K).astype(np.uint8)
        want = A.reshape(M, K).astype(np.int64) @ B.reshape(N, K).astype(np.int64).T
        got = orc.gemm(A, B, M, N, K).reshape(M, N)
        assert (got.astype(np.int64) == want).all()
    # u8 x u8 range guard: 255 * 255 * 33025 = 2147450625 fits, 33026 does not
    Au = np.full(33026, 255, dtype=np.uint8)
    assert int(orc.gemm(Au[:33025], Au[:33025], 1, 1, 33025)[0]) == 255 * 255 * 33025
    with pytest.raises(orc.OracleOverflow):
        orc.gemm(Au, Au, 1, 1, 33026)


# ---------------------------------------------------------------- requantisation to 8-bit codes
def _round_half_even(fr):
    """Nearest integer of a Fraction, ties to even (exact)."""
    from fractions import Fraction
    fl = fr.numerator // fr.denominator
    rem = fr - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        return fl + 1
    return fl


def test_requant_scale_one_is_a_clamp():
    Cq = np.array([-2 ** 31, -70000, -129, -128, -127, -1, 0, 1, 126, 127, 128, 255, 256, 2 ** 31 - 1], np.int32)
    assert np.array_equal(orc.requant(Cq, 1.0, -128, 127), np.clip(Cq.astype(np.int64), -128, 127))
    assert np.array_equal(orc.requant(Cq, 1.0, 0, 255), np.clip(Cq.astype(np.int64), 0, 255))
    assert np.array_equal(orc.requant(Cq, 1.0, 0, 127), np.clip(Cq.astype(np.int64), 0, 127))      # ReLU then s8
    assert np.array_equal(orc.requant(Cq, -1.0, -128, 127), np.clip(-Cq.astype(np.int64), -128, 127))


def test_requant_ties_go_to_even():
    Cq = np.array([1, 3, 5, 7, -1, -3, -5, 9, 251, 253], np.int32)          # halves after scale 0.5
    want = [0, 2, 2, 4, 0, -2, -2, 4, 126, 126]
    assert orc.requant(Cq, 0.5, -128, 127).tolist() == want
    assert orc.requant(np.array([10, 30, 50, -10, -30], np.int32), 0.05, -128, 127).tolist() != []  # (smoke)


def test_requant_powers_of_two_match_exact_integer_rounding():
    """For |sum| < 2^24 and a power-of-two scale every binary32 step is exact: the codes are the
    exactly rounded quotients."""
    from fractions import Fraction
    rng = np.random.default_rng(5)
    Cq = rng.integers(-2 ** 24 + 1, 2 ** 24, size=4000).astype(np.int32)
    for k in (1, 3, 7, 12, 16, 20):
        got = orc.requant(Cq, 2.0 ** -k, -128, 127)
        want = [min(max(_round_half_even(Fraction(int(v), 2 ** k)), -128), 127) for v in Cq]
        assert got.tolist() == want, k


def test_requant_general_scale_against_exact_rationals():
    """With an arbitrary scale the binary32 rule may differ from the exactly rounded real product by
    one code, and only when the real product lies within the two roundings' reach of a tie."""
    from fractions import Fraction
    rng = np.random.default_rng(6)
    Cq = rng.integers(-3_000_000, 3_000_000, size=6000).astype(np.int32)
    for scale in (1.25e-3, 7.3e-5, 3.1e-2, -4.4e-4, 1.0 / 3.0):
        s32 = float(np.float32(scale))
        got = orc.requant(Cq, s32, -128, 127)
        off_by_one = 0
        for v, g in zip(Cq.tolist(), got.tolist()):
            real = Fraction(v) * Fraction(s32)
            exact = min(max(_round_half_even(real), -128), 127)
            if g != exact:
                off_by_one += 1
                assert abs(g - exact) == 1
                frac = real - (real.numerator // real.denominator)
                assert abs(frac - Fraction(1, 2)) <= abs(real) * Fraction(1, 2 ** 22), (v, scale)
        assert off_by_one <= 6          # a handful of near-ties at most
    # monotone in the sum for a positive scale
    ordered = np.sort(Cq)
    codes = orc.requant(ordered, 1.25e-3, -128, 127)
    assert (np.diff(codes) >= 0).all()


def test_requant_saturates_and_keeps_shape():
    Cq = np.array([[2 ** 31 - 1, -2 ** 31, 10 ** 9], [-10 ** 9, 12345, -12345]], np.int32)
    got = orc.requant(Cq, 0.75, -128, 127)
    assert got.shape == (2, 3) and got.tolist() == [[127, -128, 127], [-128, 127, -128]]
    assert orc.requant(Cq, 1e-9, 0, 255).tolist() == [[2, 0, 1], [0, 0, 0]]
    with pytest.raises(ValueError):
        orc.requant(Cq, float("inf"), -128, 127)


# ---------------------------------------------------------------- per-channel bias
def test_bias_closed_forms_and_numpy():
    rng = np.random.default_rng(5)
    Cq = rng.integers(-(1 << 30), 1 << 30, size=(7, 5), dtype=np.int64).astype(np.int32)
    assert np.array_equal(orc.add_bias(Cq, np.zeros(5, np.int32)), Cq)                     # zero bias: identity
    bias = rng.integers(-(1 << 20), 1 << 20, size=5, dtype=np.int64).astype(np.int32)
    assert np.array_equal(orc.add_bias(Cq, bias), (Cq.astype(np.int64) + bias.astype(np.int64)).astype(np.int32))
    one_hot = np.array([0, 0, 9, 0, 0], np.int32)                                          # only column 2 moves
    moved = orc.add_bias(Cq, one_hot)
    assert np.array_equal(moved[:, [0, 1, 3, 4]], Cq[:, [0, 1, 3, 4]]) and np.array_equal(moved[:, 2], Cq[:, 2] + 9)
    nhwc = Cq.reshape(1, 7, 1, 5)                                                          # channel-last tensors too
    assert np.array_equal(orc.add_bias(nhwc, bias).reshape(7, 5), orc.add_bias(Cq, bias))
    with pytest.raises(orc.OracleOverflow):
        orc.add_bias(np.array([[2 ** 31 - 1]], np.int32), np.array([1], np.int32))
    assert orc.add_bias(np.array([[2 ** 31 - 1]], np.int32), np.array([1], np.int32), allow_overflow=True)[0, 0] == -2 ** 31


def test_bias_equals_one_more_k_row():
    """A bias in the int8 range is the product with one more k: a column of ones appended to A and the bias
    appended to every column of B -- the GEMM oracle itself says what the sum must be."""
    rng = np.random.default_rng(6)
    M, N, K = 9, 6, 13
    A = rng.integers(-128, 128, size=(M, K)).astype(np.int8)
    B = rng.integers(-128, 128, size=(N, K)).astype(np.int8)                               # row j = column j of B
    bias = rng.integers(-128, 128, size=N).astype(np.int32)
    A1 = np.concatenate([A, np.ones((M, 1), np.int8)], axis=1)
    B1 = np.concatenate([B, bias.astype(np.int8).reshape(N, 1)], axis=1)
    want = orc.gemm(A1.reshape(-1), B1.reshape(-1), M, N, K + 1).reshape(M, N)
    got = orc.add_bias(orc.gemm(A.reshape(-1), B.reshape(-1), M, N, K).reshape(M, N), bias)
    assert np.array_equal(got, want)
