"""GPU parity for the fused dequantisation entry points (C(float32) = scale * exact int32 sum).

Two checks per case: (a) within 2^-23 relative of the oracle's binary64 value scale*sum (two
binary32 roundings: int -> float conversion and the multiplication); (b) bit-identical to the
stated rounding rule evaluated with NumPy in binary32, which also pins that every kernel path
(one CTA, CTA pairs, cluster split-K, both skinny kernels, both conv lowerings) rounds alike."""
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


def check(got_f32, Cq, scale):
    want64 = orc.dequant(Cq, float(np.float32(scale)))
    err = np.abs(got_f32.astype(np.float64) - want64)
    assert (err <= REL * np.abs(want64)).all(), "max rel err %g" % (err / np.maximum(np.abs(want64), 1e-300)).max()
    rule = (Cq.astype(np.float32) * np.float32(scale)).astype(np.float32)
    assert np.array_equal(got_f32.view(np.uint32), rule.view(np.uint32))


def run_gemm_dequant(mg, mode, M, N, K, scale, seed, ldc=None, expect_path=None):
    ldc = N if ldc is None else ldc
    A = inputs.uniform_s8(M * K, seed + 1) if mode == "s8" else inputs.uniform_u8(M * K, seed + 1)
    B = inputs.uniform_s8(N * K, seed + 2)
    Cq = orc.gemm(A, B, M, N, K).reshape(M, N)
    poison = np.full(M * ldc, np.float32(-7.25), dtype=np.float32)
    dA, _a = to_dev(A)
    dB, _b = to_dev(B)
    dC, _c = to_dev(poison)
    fn = mg.mipgemm_s8s8f32_dequant if mode == "s8" else mg.mipgemm_u8s8f32_dequant
    fn(M, N, K, dA, K, dB, K, dC, ldc, scale)
    assert mg.mipgemm_device_status() == mg.OK
    path = mg.mipgemm_last_path()
    if expect_path is not None:
        assert path & mg.PATH_MASK == expect_path, hex(path)
    out = dC.cpu().numpy().view(np.float32).reshape(M, ldc)
    assert (out[:, N:] == np.float32(-7.25)).all()            # padding columns untouched
    check(np.ascontiguousarray(out[:, :N]), Cq, scale)
    return path


def test_dense_paths(mg):
    run_gemm_dequant(mg, "s8", 300, 520, 400, 0.0123, 1, expect_path=mg.PATH_DENSE)
    run_gemm_dequant(mg, "u8", 257, 130, 272, 3.5e-4, 2, ldc=133)                  # row-per-thread stores
    mg.mipgemm_set_tuning(force_path=mg.PATH_DENSE_PAIR)
    try:
        run_gemm_dequant(mg, "s8", 700, 600, 1424, -0.75, 3, expect_path=mg.PATH_DENSE_PAIR)
    finally:
        mg.mipgemm_set_tuning()
    p = run_gemm_dequant(mg, "s8", 128, 256, 8192, 1.0 / 3.0, 4)                    # cluster split-K
    assert p & mg.PATH_SPLITK
    run_gemm_dequant(mg, "s8", 2048, 2048, 2048, 2.0 ** -9, 5)                      # large sums, exact scale


def test_explicit_split_request_is_ignored_for_float_output(mg):
    mg.mipgemm_set_tuning(split_k=4)
    try:
        p = run_gemm_dequant(mg, "s8", 300, 300, 1296, 0.02, 6)
        assert not p & mg.PATH_SPLITK
    finally:
        mg.mipgemm_set_tuning()


@pytest.mark.parametrize("M", [1, 8, 16])
def test_skinny_paths(mg, M):
    run_gemm_dequant(mg, "s8", M, 4096, 4096, 0.004, 10 + M, expect_path=mg.PATH_SKINNY)      # ring form
    run_gemm_dequant(mg, "u8", M, 333, 528, 0.5, 20 + M, expect_path=mg.PATH_SKINNY)          # register form


@pytest.mark.parametrize("case", [
    (2, 14, 14, 128, 96, 3, 3, (1, 1), (1, 1)),       # TMA im2col
    (2, 32, 32, 3, 64, 7, 7, (2, 2), (3, 3)),         # explicit im2col
    (3, 9, 7, 64, 40, 1, 1, (1, 1), (0, 0)),          # pointwise
])
def test_conv_dequant(mg, case):
    Nb, H, W, Cin, Cout, R, S, stride, pad = case
    X = inputs.uniform_u8(Nb * H * W * Cin, 31).reshape(Nb, H, W, Cin)
    Wt = inputs.normal_s8(Cout * R * S * Cin, 32, 32.0, -127, 127).reshape(Cout, R, S, Cin)
    Yq = orc.conv(X, Wt, stride=stride, pad=pad)
    scale = 0.00731
    dX, _x = to_dev(X)
    dW, _w = to_dev(Wt)
    dY, _y = to_dev(np.zeros(Yq.size, np.float32))
    mg.mipgemm_conv_u8s8f32_dequant(Nb, H, W, Cin, Cout, R, S, stride[0], stride[1], pad[0], pad[1], 1, 1,
                                    dX, dW, dY, scale)
    assert mg.mipgemm_device_status() == mg.OK
    check(dY.cpu().numpy().view(np.float32).reshape(Yq.shape), Yq, scale)


def test_k_zero_gives_float_zeros(mg):
    import torch
    dC = torch.full((5 * 7,), 3.0, dtype=torch.float32, device="cuda")
    dA = torch.zeros(16, dtype=torch.int8, device="cuda")
    mg.mipgemm_s8s8f32_dequant(5, 7, 0, dA, 0, dA, 0, dC, 7, 2.5)
    assert (dC.cpu().numpy() == 0.0).all()
