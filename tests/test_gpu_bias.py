"""GPU parity for the fused output transforms with a per-output-channel bias: the oracle adds the bias to its
exact int32 sums (range-checked) and then applies the same stated binary32 rules as for the forms without
bias.  Codes must be identical; float outputs must be within 2^-23 relative of the binary64 value and
bit-identical to the binary32 rule.  Covered: one CTA, CTA pairs, cluster split-K, M <= 16 (which stays on
the dense kernel when a bias is given), ragged N with an unaligned bias pointer, every conv lowering,
K == 0, and a NULL bias (the entry point without the suffix)."""
import numpy as np
import pytest

from oracle import mip_oracle as orc
from paper_2506_11728_b200 import inputs
from gpu_util import to_dev

pytestmark = pytest.mark.gpu
REL = 2.0 ** -23


@pytest.fixture(scope="module")
def mg():
    from paper_2506_11728_b200 import binding
    binding.mipgemm_set_tuning()
    return binding


def make_bias(n, seed, spread):
    """Bias values of the size of the sums (so that they move most codes), both signs."""
    rng = np.random.default_rng(seed)
    return rng.integers(-spread, spread + 1, size=n, dtype=np.int64).astype(np.int32)


def check_f32(got_f32, sums, scale):
    want64 = orc.dequant(sums, float(np.float32(scale)))
    err = np.abs(got_f32.astype(np.float64) - want64)
    assert (err <= REL * np.abs(want64)).all()
    rule = (sums.astype(np.float32) * np.float32(scale)).astype(np.float32)
    assert np.array_equal(got_f32.view(np.uint32), rule.view(np.uint32))


def run_dequant_bias(mg, mode, M, N, K, scale, seed, ldc=None, bias_misalign=0):
    ldc = N if ldc is None else ldc
    A = inputs.uniform_s8(M * K, seed + 1) if mode == "s8" else inputs.uniform_u8(M * K, seed + 1)
    B = inputs.uniform_s8(N * K, seed + 2)
    bias = make_bias(N, seed + 3, int(3 * 74 * 74 * np.sqrt(max(K, 1))))
    sums = orc.add_bias(orc.gemm(A, B, M, N, K).reshape(M, N), bias)
    dA, _a = to_dev(A)
    dB, _b = to_dev(B)
    dC, _c = to_dev(np.full(M * ldc, np.float32(-7.25), dtype=np.float32))
    dbias, _k = to_dev(bias, bias_misalign)
    fn = mg.mipgemm_s8s8f32_dequant_bias if mode == "s8" else mg.mipgemm_u8s8f32_dequant_bias
    fn(M, N, K, dA, K, dB, K, dC, ldc, scale, dbias)
    assert mg.mipgemm_device_status() == mg.OK
    path = mg.mipgemm_last_path()
    out = dC.cpu().numpy().view(np.float32).reshape(M, ldc)
    assert (out[:, N:] == np.float32(-7.25)).all()
    check_f32(np.ascontiguousarray(out[:, :N]), sums, scale)
    return path


def run_requant_bias(mg, a_unsigned, M, N, K, scale, seed, relu=False, ldc=None, bias_misalign=0):
    ldc = N if ldc is None else ldc
    A = inputs.uniform_u8(M * K, seed + 1) if a_unsigned else inputs.uniform_s8(M * K, seed + 1)
    B = inputs.uniform_s8(N * K, seed + 2)
    bias = make_bias(N, seed + 3, int(3 * 74 * 74 * np.sqrt(max(K, 1))))
    sums = orc.add_bias(orc.gemm(A, B, M, N, K).reshape(M, N), bias)
    lo, hi = (0, 255) if a_unsigned else ((0, 127) if relu else (-128, 127))
    want = orc.requant(sums, scale, lo, hi)
    plain = orc.requant(orc.gemm(A, B, M, N, K).reshape(M, N), scale, lo, hi)
    dA, _a = to_dev(A)
    dB, _b = to_dev(B)
    dC, _c = to_dev(np.full(M * ldc, 0x5A, np.uint8))
    dbias, _k = to_dev(bias, bias_misalign)
    if a_unsigned:
        mg.mipgemm_u8s8u8_requant_bias(M, N, K, dA, K, dB, K, dC, ldc, scale, dbias)
    else:
        mg.mipgemm_s8s8s8_requant_bias(M, N, K, dA, K, dB, K, dC, ldc, scale, dbias, relu)
    assert mg.mipgemm_device_status() == mg.OK
    raw = dC.cpu().numpy().reshape(M, ldc)
    got = raw[:, :N].astype(np.int32) if a_unsigned else raw[:, :N].view(np.int8).astype(np.int32)
    assert np.array_equal(got, want), "%dx%dx%d: %d codes differ" % (M, N, K, (got != want).sum())
    assert (raw[:, N:] == 0x5A).all()
    if K > 0:
        assert (want != plain).mean() > 0.3                 # the bias really decides the codes
    return mg.mipgemm_last_path()


def test_dequant_bias_dense_paths(mg):
    assert run_dequant_bias(mg, "s8", 300, 520, 400, 0.0123, 1) & mg.PATH_MASK == mg.PATH_DENSE
    run_dequant_bias(mg, "u8", 257, 130, 272, 3.5e-4, 2, ldc=133, bias_misalign=4)     # ragged N, 4-byte aligned bias
    mg.mipgemm_set_tuning(force_path=mg.PATH_DENSE_PAIR)
    try:
        assert run_dequant_bias(mg, "s8", 700, 600, 1424, -0.75, 3) & mg.PATH_MASK == mg.PATH_DENSE_PAIR
    finally:
        mg.mipgemm_set_tuning()
    assert run_dequant_bias(mg, "s8", 128, 256, 8192, 1.0 / 3.0, 4) & mg.PATH_SPLITK   # cluster split-K
    run_dequant_bias(mg, "s8", 2048, 2048, 2048, 2.0 ** -9, 5)


@pytest.mark.parametrize("M", [1, 8, 16])
def test_dequant_bias_few_rows_use_the_dense_kernel(mg, M):
    p = run_dequant_bias(mg, "s8", M, 4096, 4096, 0.004, 10 + M)
    assert p & mg.PATH_MASK in (mg.PATH_DENSE, mg.PATH_DENSE_PAIR)
    run_dequant_bias(mg, "u8", M, 333, 528, 0.5, 20 + M, bias_misalign=8)


@pytest.mark.parametrize("a_unsigned", [False, True])
def test_requant_bias_codes(mg, a_unsigned):
    for (M, N, K) in [(128, 128, 128), (300, 260, 400), (1000, 96, 777), (2048, 512, 1024), (50, 33, 64)]:
        scale = float(np.float32(127.0 / (4.0 * 74.0 * 74.0 * np.sqrt(K)) * (2.0 if a_unsigned else 1.0)))
        run_requant_bias(mg, a_unsigned, M, N, K, scale, M + N)


def test_requant_bias_layouts_and_relu(mg):
    run_requant_bias(mg, False, 256, 128, 512, 1.0e-3, 3, relu=True)
    run_requant_bias(mg, False, 200, 100, 320, 2e-4, 7, ldc=128, bias_misalign=12)
    run_requant_bias(mg, True, 129, 49, 256, 3e-4, 9, ldc=53, bias_misalign=4)
    run_requant_bias(mg, False, 8, 4096, 512, 1e-4, 10)
    run_requant_bias(mg, False, 4096, 4096, 256, 1e-4, 11)                              # CTA pairs


def test_k_zero_writes_the_transformed_bias(mg):
    run_requant_bias(mg, False, 6, 37, 0, 0.01, 40, ldc=40)
    run_requant_bias(mg, True, 6, 37, 0, 0.01, 41, ldc=40)
    run_dequant_bias(mg, "s8", 5, 70, 0, 2.5, 42, ldc=72)


def test_null_bias_is_the_plain_entry_point_and_bad_pointer_is_rejected(mg):
    M, N, K = 130, 200, 144
    A, B = inputs.uniform_s8(M * K, 51), inputs.uniform_s8(N * K, 52)
    want = orc.requant(orc.gemm(A, B, M, N, K).reshape(M, N), 1e-3, -128, 127)
    dA, _a = to_dev(A)
    dB, _b = to_dev(B)
    dC, _c = to_dev(np.zeros(M * N, np.uint8))
    mg.mipgemm_s8s8s8_requant_bias(M, N, K, dA, K, dB, K, dC, N, 1e-3, None)
    assert mg.mipgemm_device_status() == mg.OK
    assert np.array_equal(dC.cpu().numpy().view(np.int8).reshape(M, N).astype(np.int32), want)
    assert mg.mipgemm_s8s8s8_requant_bias(M, N, K, dA, K, dB, K, dC, N, 1e-3, 258, check=False) == mg.ERR_INVALID_ARG
    assert mg.mipgemm_s8s8f32_dequant_bias(M, N, K, dA, K, dB, K, dC, N, 1e-3, 257, check=False) == mg.ERR_INVALID_ARG


CONVS = [
    (2, 14, 14, 128, 128, 3, 3, (1, 1), (1, 1)),          # TMA im2col
    (2, 14, 14, 512, 64, 3, 3, (1, 1), (1, 1)),           # TMA im2col, K-heavy (cluster split-K candidate)
    (2, 32, 32, 3, 64, 7, 7, (2, 2), (3, 3)),             # gathered stem
    (2, 14, 14, 256, 96, 1, 1, (1, 1), (0, 0)),           # pointwise
    (1, 10, 11, 5, 7, 3, 2, (2, 1), (1, 0)),              # gathered, Cout % 4 != 0
]


@pytest.mark.parametrize("case", CONVS)
def test_conv_bias_both_transforms(mg, case):
    Nb, H, W, Cin, Cout, R, S, stride, pad = case
    X = inputs.uniform_u8(Nb * H * W * Cin, 31).reshape(Nb, H, W, Cin)
    Wt = inputs.normal_s8(Cout * R * S * Cin, 32, 32.0, -127, 127).reshape(Cout, R, S, Cin)
    bias = make_bias(Cout, 33, int(2 * 32 * 147 * np.sqrt(R * S * Cin)))
    sums = orc.add_bias(orc.conv(X, Wt, stride=stride, pad=pad), bias)
    scale = float(np.float32(255.0 / (4.0 * 32.0 * 147.0 * np.sqrt(R * S * Cin))))
    dX, _x = to_dev(X)
    dW, _w = to_dev(Wt)
    dbias, _k = to_dev(bias)
    dY, _y = to_dev(np.full(sums.size, 0x5A, np.uint8))
    mg.mipgemm_conv_u8s8u8_requant_bias(Nb, H, W, Cin, Cout, R, S, stride[0], stride[1], pad[0], pad[1], 1, 1,
                                        dX, dW, dY, scale, dbias)
    assert mg.mipgemm_device_status() == mg.OK
    want = orc.requant(sums, scale, 0, 255)
    assert np.array_equal(dY.cpu().numpy().reshape(sums.shape).astype(np.int32), want)
    assert len(np.unique(want)) > 20
    dF, _f = to_dev(np.zeros(sums.size, np.float32))
    mg.mipgemm_conv_u8s8f32_dequant_bias(Nb, H, W, Cin, Cout, R, S, stride[0], stride[1], pad[0], pad[1], 1, 1,
                                         dX, dW, dF, 0.00731, dbias)
    assert mg.mipgemm_device_status() == mg.OK
    check_f32(dF.cpu().numpy().view(np.float32).reshape(sums.shape), sums, 0.00731)
