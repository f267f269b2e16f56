"""GPU parity for the requantised (8-bit code) outputs: every code must equal the oracle's, which applies
the stated binary32 rule to the oracle's exact int32 sums."""
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


def run_requant(mg, a_unsigned, M, N, K, scale, *, relu=False, pad=(0, 0, 0), misalign=0, seed=0, sigma=None):
    lda, ldb, ldc = K + pad[0], K + pad[1], N + pad[2]
    gen = inputs.uniform_u8 if a_unsigned else inputs.uniform_s8
    A = gen(M * lda, seed + 1) if sigma is None else inputs.normal_s8(M * lda, seed + 1, sigma)
    if a_unsigned and sigma is not None:
        A = A.view(np.uint8)
    B = inputs.uniform_s8(N * ldb, seed + 2) if sigma is None else inputs.normal_s8(N * ldb, seed + 2, sigma)
    sums = orc.gemm(A, B, M, N, K, lda=lda, ldb=ldb).reshape(M, N)
    lo, hi = (0, 255) if a_unsigned else ((0, 127) if relu else (-128, 127))
    want = orc.requant(sums, scale, lo, hi)
    C0 = np.full(M * ldc, 0x5A, np.uint8)
    dA, _a = to_dev(A)
    dB, _b = to_dev(B)
    dC, _c = to_dev(C0, misalign)
    if a_unsigned:
        mg.mipgemm_u8s8u8_requant(M, N, K, dA, lda, dB, ldb, dC, ldc, scale)
    else:
        mg.mipgemm_s8s8s8_requant(M, N, K, dA, lda, dB, ldb, dC, ldc, scale, relu)
    assert mg.mipgemm_device_status() == mg.OK
    raw = dC.cpu().numpy().reshape(M, ldc)
    got = raw[:, :N].astype(np.int32) if a_unsigned else raw[:, :N].view(np.int8).astype(np.int32)
    assert np.array_equal(got, want), "%dx%dx%d scale %g: %d codes differ" % (M, N, K, scale, (got != want).sum())
    assert (raw[:, N:] == 0x5A).all()                      # padding bytes untouched
    return want


@pytest.mark.parametrize("a_unsigned", [False, True])
def test_requant_codes_match_oracle(mg, a_unsigned):
    for (M, N, K) in [(128, 128, 128), (300, 260, 400), (1000, 96, 777), (2048, 512, 1024), (50, 33, 64)]:
        # scales that put the codes' spread across the 8-bit range for uniform operands
        scale = 127.0 / (3.0 * 74.0 * 74.0 * np.sqrt(K)) * (2.0 if a_unsigned else 1.0)
        codes = run_requant(mg, a_unsigned, M, N, K, float(np.float32(scale)), seed=M + N)
        assert len(np.unique(codes)) > 40                  # not a degenerate all-saturated case


def test_requant_relu_and_saturation(mg):
    run_requant(mg, False, 256, 128, 512, 1.0e-3, relu=True, seed=3)
    codes = run_requant(mg, False, 256, 128, 512, 1.0, seed=4)              # scale 1: pure clamp
    assert set(np.unique(codes)) <= set(range(-128, 128)) and (codes == 127).any() and (codes == -128).any()
    run_requant(mg, True, 130, 70, 200, 0.5, seed=5)                         # exact halves: ties to even
    run_requant(mg, False, 130, 70, 200, -2.0 ** -9, seed=6)                 # negative power of two


def test_requant_layouts(mg):
    run_requant(mg, False, 200, 100, 320, 2e-4, pad=(16, 32, 28), seed=7)            # aligned pitches, N % 16 != 0
    run_requant(mg, True, 200, 100, 320, 2e-4, pad=(3, 5, 7), seed=8)                # operands re-pitched, odd ldc
    run_requant(mg, False, 129, 48, 256, 3e-4, misalign=3, seed=9)                   # misaligned C base
    run_requant(mg, False, 8, 4096, 512, 1e-4, seed=10)                              # M <= 16 stays on the dense kernel
    run_requant(mg, False, 4096, 4096, 256, 1e-4, seed=11)                           # CTA pairs


def test_requant_k_zero_and_errors(mg):
    C0 = np.full(6 * 8, 0x5A, np.uint8)
    dC, _c = to_dev(C0)
    mg.mipgemm_s8s8s8_requant(6, 5, 0, 0, 0, 0, 0, dC, 8, 0.5, 0)
    out = dC.cpu().numpy().reshape(6, 8)
    assert (out[:, :5] == 0).all() and (out[:, 5:] == 0x5A).all()
    assert mg.mipgemm_s8s8s8_requant(4, 4, 16, 256, 16, 256, 16, 256, 4, float("nan"), 0, check=False) == mg.ERR_INVALID_ARG
    assert mg.mipgemm_u8s8u8_requant(4, 4, 16, 256, 16, 256, 16, 256, 3, 1.0, check=False) == mg.ERR_INVALID_ARG


CONVS = [
    (2, 14, 14, 128, 128, 3, 3, (1, 1), (1, 1)),          # TMA im2col
    (2, 32, 32, 3, 64, 7, 7, (2, 2), (3, 3)),             # gathered stem
    (2, 14, 14, 256, 96, 1, 1, (1, 1), (0, 0)),           # pointwise
    (1, 10, 11, 5, 7, 3, 2, (2, 1), (1, 0)),              # gathered, Cout % 4 != 0
]


@pytest.mark.parametrize("case", CONVS)
def test_requant_conv(mg, case):
    Nb, H, W, Cin, Cout, R, S, stride, pad = case
    X = inputs.uniform_u8(Nb * H * W * Cin, 31).reshape(Nb, H, W, Cin)
    Wt = inputs.normal_s8(Cout * R * S * Cin, 32, 32.0, -127, 127).reshape(Cout, R, S, Cin)
    sums = orc.conv(X, Wt, stride=stride, pad=pad)
    scale = float(np.float32(255.0 / (4.0 * 32.0 * 147.0 * np.sqrt(R * S * Cin))))
    want = orc.requant(sums, scale, 0, 255)
    Nb_, Ho, Wo, _ = sums.shape
    dX, _x = to_dev(X)
    dW, _w = to_dev(Wt)
    dY, _y = to_dev(np.full(sums.size, 0x5A, np.uint8))
    mg.mipgemm_conv_u8s8u8_requant(Nb, H, W, Cin, Cout, R, S, stride[0], stride[1], pad[0], pad[1], 1, 1,
                                   dX, dW, dY, scale)
    assert mg.mipgemm_device_status() == mg.OK
    got = dY.cpu().numpy().reshape(sums.shape).astype(np.int32)
    assert np.array_equal(got, want)
    assert len(np.unique(want)) > 20
