"""GPU parity for the convolution entry point against the direct-convolution oracle."""
import numpy as np
import pytest

from oracle import mip_oracle as orc
from paper_2506_11728_b200 import inputs
from gpu_util import run_conv, first_mismatch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mg():
    from paper_2506_11728_b200 import binding
    binding.mipgemm_set_tuning()
    return binding


def conv_inputs(Nb, H, W, Cin, Cout, R, S, seed):
    X = inputs.uniform_u8(Nb * H * W * Cin, seed + 1).reshape(Nb, H, W, Cin)
    Wt = inputs.normal_s8(Cout * R * S * Cin, seed + 2, 32.0, -127, 127).reshape(Cout, R, S, Cin)
    return X, Wt


def check_conv(mg, Nb, H, W, Cin, Cout, R, S, stride, pad, dil=(1, 1), seed=0, accumulate=False,
               expect_flag=None):
    X, Wt = conv_inputs(Nb, H, W, Cin, Cout, R, S, seed)
    Y0 = None
    if accumulate:
        Ho, Wo = orc.conv_out_hw(H, W, R, S, stride, pad, dil)
        Y0 = inputs.uniform_s32(Nb * Ho * Wo * Cout, seed + 3).reshape(Nb, Ho, Wo, Cout)
    want = orc.conv(X, Wt, stride=stride, pad=pad, dil=dil, Y=None if Y0 is None else Y0.copy(),
                    accumulate=accumulate)
    got, path = run_conv(mg, X, Wt, stride, pad, dil, Y=None if Y0 is None else Y0.copy(),
                         accumulate=accumulate)
    assert np.array_equal(got, want), "conv %s path=%#x: %s" % (
        (Nb, H, W, Cin, Cout, R, S, stride, pad, dil), path, first_mismatch(got, want))
    if expect_flag is not None:
        assert path & expect_flag, hex(path)
    return path


def test_pointwise_is_plain_gemm(mg):
    p = check_conv(mg, 2, 14, 14, 256, 96, 1, 1, (1, 1), (0, 0), seed=1)
    assert not p & (mg.PATH_IM2COL_TMA | mg.PATH_IM2COL_EXPLICIT)
    check_conv(mg, 3, 7, 9, 24, 40, 1, 1, (1, 1), (0, 0), seed=2)            # Cin % 16 != 0 -> repack


TMA_CASES = [
    # Nb, H, W, Cin, Cout, R, S, stride, pad, dil
    (2, 14, 14, 128, 128, 3, 3, (1, 1), (1, 1), (1, 1)),
    (2, 28, 28, 128, 64, 3, 3, (2, 2), (1, 1), (1, 1)),
    (3, 13, 11, 64, 64, 3, 3, (1, 1), (1, 1), (1, 1)),       # 64-byte k-block, odd extents
    (2, 16, 16, 256, 160, 1, 1, (2, 2), (0, 0), (1, 1)),     # strided 1x1 (projection shortcut)
    (1, 20, 18, 128, 96, 3, 3, (1, 1), (2, 2), (2, 2)),      # dilation
    (2, 15, 17, 128, 72, 5, 3, (2, 1), (2, 1), (1, 1)),      # rectangular filter, mixed stride
    (5, 7, 7, 512, 512, 3, 3, (1, 1), (1, 1), (1, 1)),       # tiles straddle images; K = 4608
    (1, 9, 9, 128, 64, 3, 3, (1, 1), (0, 0), (1, 1)),        # no padding
]


@pytest.mark.parametrize("case", TMA_CASES)
def test_implicit_im2col_tma(mg, case):
    Nb, H, W, Cin, Cout, R, S, stride, pad, dil = case
    check_conv(mg, Nb, H, W, Cin, Cout, R, S, stride, pad, dil, seed=10, expect_flag=mg.PATH_IM2COL_TMA)
    check_conv(mg, Nb, H, W, Cin, Cout, R, S, stride, pad, dil, seed=11, accumulate=True,
               expect_flag=mg.PATH_IM2COL_TMA)


GATHER_CASES = [
    (2, 32, 32, 3, 64, 7, 7, (2, 2), (3, 3), (1, 1)),        # stem-like, Cin = 3, K = 147 (slot 32)
    (2, 12, 12, 16, 32, 3, 3, (1, 1), (1, 1), (1, 1)),       # Cin % 16 == 0 but not % 64 (slot = segment)
    (3, 19, 23, 3, 64, 7, 7, (2, 2), (3, 3), (1, 1)),        # odd extents: tiles straddle rows and images
    (1, 10, 11, 5, 7, 3, 2, (2, 1), (1, 0), (2, 1)),         # dilated rows, Cout % 4 != 0
    (2, 9, 9, 24, 40, 3, 3, (1, 1), (1, 1), (1, 1)),         # segment 72 -> slot 80, K' = 240 (two k-blocks)
    (2, 14, 13, 1, 16, 5, 5, (1, 2), (2, 2), (1, 1)),        # one channel
    (1, 6, 5, 3, 8, 3, 11, (1, 1), (1, 5), (1, 1)),          # filter wider than the image
    (2, 11, 10, 7, 33, 4, 3, (3, 2), (0, 2), (1, 1)),        # padding only in w, stride 3
    (1, 40, 40, 100, 48, 3, 3, (1, 1), (1, 1), (1, 1)),      # long rows of A: K' = 912, 8 k-blocks
    (1, 5, 5, 3, 4, 3, 3, (1, 1), (1, 1), (1, 1)),           # the whole batch is 75 bytes
    # image rows that are multiples of 16 bytes: staged in shared memory by bulk copies
    (3, 20, 16, 3, 64, 7, 7, (2, 2), (3, 3), (1, 1)),        # 48-byte rows; tiles straddle output rows and images
    (2, 16, 32, 4, 32, 5, 5, (1, 2), (2, 2), (1, 1)),        # 128-byte rows, slot 32, stride only in w
    (1, 12, 16, 5, 7, 3, 2, (2, 1), (1, 0), (2, 1)),         # 80-byte rows, dilated filter rows, Cout % 4 != 0
    (2, 8, 8, 2, 16, 8, 8, (1, 1), (4, 4), (1, 1)),          # filter as large as the image, padding on all sides
    (5, 4, 16, 1, 8, 3, 3, (1, 1), (1, 1), (1, 1)),          # tiny images: a tile spans several of them
]


@pytest.mark.parametrize("case", GATHER_CASES)
def test_gathered_im2col(mg, case):
    """Operand A built in shared memory by the gather warps (the augmented matrix never exists)."""
    Nb, H, W, Cin, Cout, R, S, stride, pad, dil = case
    check_conv(mg, Nb, H, W, Cin, Cout, R, S, stride, pad, dil, seed=20, expect_flag=mg.PATH_IM2COL_GATHER)
    check_conv(mg, Nb, H, W, Cin, Cout, R, S, stride, pad, dil, seed=21, accumulate=True,
               expect_flag=mg.PATH_IM2COL_GATHER)


def test_gathered_im2col_extreme_values(mg):
    """All taps at their extremes: every sum is the tap count times 255 * -128 (borders have fewer taps)."""
    Nb, H, W, Cin, Cout, R, S = 2, 17, 15, 3, 16, 7, 7
    X = np.full((Nb, H, W, Cin), 255, np.uint8)
    Wt = np.full((Cout, R, S, Cin), -128, np.int8)
    want = orc.conv(X, Wt, stride=(2, 2), pad=(3, 3))
    got, path = run_conv(mg, X, Wt, (2, 2), (3, 3), (1, 1))
    assert path & mg.PATH_IM2COL_GATHER
    assert np.array_equal(got, want)


@pytest.mark.parametrize("misalign", [1, 2, 3, 7])
def test_gathered_im2col_any_image_alignment(mg, misalign):
    Nb, H, W, Cin, Cout, R, S = 2, 21, 18, 3, 24, 7, 7
    X, Wt = conv_inputs(Nb, H, W, Cin, Cout, R, S, 60 + misalign)
    want = orc.conv(X, Wt, stride=(2, 2), pad=(3, 3))
    got, path = run_conv(mg, X, Wt, (2, 2), (3, 3), (1, 1), x_misalign=misalign)
    assert path & mg.PATH_IM2COL_GATHER
    assert np.array_equal(got, want), first_mismatch(got, want)


EXPLICIT_CASES = [
    (1, 10, 11, 5, 7, 3, 2, (2, 1), (1, 0), (1, 2)),         # dilated columns: not contiguous in the image
    (2, 12, 12, 16, 32, 3, 3, (1, 1), (1, 1), (1, 3)),
    (1, 3, 3, 3, 4, 3, 3, (1, 1), (1, 1), (1, 1)),           # the whole batch is 27 bytes
]
FORCED_EXPLICIT_CASES = GATHER_CASES[:3]


@pytest.mark.parametrize("case", EXPLICIT_CASES)
def test_explicit_im2col(mg, case):
    Nb, H, W, Cin, Cout, R, S, stride, pad, dil = case
    check_conv(mg, Nb, H, W, Cin, Cout, R, S, stride, pad, dil, seed=20, expect_flag=mg.PATH_IM2COL_EXPLICIT)
    check_conv(mg, Nb, H, W, Cin, Cout, R, S, stride, pad, dil, seed=21, accumulate=True,
               expect_flag=mg.PATH_IM2COL_EXPLICIT)


@pytest.mark.parametrize("case", FORCED_EXPLICIT_CASES)
def test_forced_explicit_im2col(mg, case):
    Nb, H, W, Cin, Cout, R, S, stride, pad, dil = case
    mg.mipgemm_set_tuning(force_path=mg.PATH_IM2COL_EXPLICIT)
    try:
        check_conv(mg, Nb, H, W, Cin, Cout, R, S, stride, pad, dil, seed=22, expect_flag=mg.PATH_IM2COL_EXPLICIT)
        check_conv(mg, Nb, H, W, Cin, Cout, R, S, stride, pad, dil, seed=23, accumulate=True,
                   expect_flag=mg.PATH_IM2COL_EXPLICIT)
    finally:
        mg.mipgemm_set_tuning()


def test_forced_explicit_matches_tma(mg):
    case = TMA_CASES[1]
    Nb, H, W, Cin, Cout, R, S, stride, pad, dil = case
    mg.mipgemm_set_tuning(force_path=mg.PATH_IM2COL_EXPLICIT)
    try:
        check_conv(mg, Nb, H, W, Cin, Cout, R, S, stride, pad, dil, seed=30, expect_flag=mg.PATH_IM2COL_EXPLICIT)
    finally:
        mg.mipgemm_set_tuning()


@pytest.mark.parametrize("layer", range(len(inputs.RESNET50_CONVS)))
def test_resnet50_layers_batch2_full(mg, layer):
    _cnt, H, W, Cin, Cout, R, S, st, pd = inputs.RESNET50_CONVS[layer]
    check_conv(mg, 2, H, W, Cin, Cout, R, S, (st, st), (pd, pd), seed=inputs.seed_for(3, layer))


@pytest.mark.parametrize("layer", range(len(inputs.RESNET50_CONVS)))
def test_resnet50_layers_batch32_sampled_images(mg, layer):
    """Full batch on the GPU; the oracle recomputes two whole images (the output of image n
    depends on image n only) -- first and last, so tile runs that cross image borders count."""
    _cnt, H, W, Cin, Cout, R, S, st, pd = inputs.RESNET50_CONVS[layer]
    Nb = 32
    X, Wt = conv_inputs(Nb, H, W, Cin, Cout, R, S, inputs.seed_for(3, layer))
    got, _ = run_conv(mg, X, Wt, (st, st), (pd, pd), (1, 1))
    for n in (0, 17, Nb - 1):
        want = orc.conv(X[n:n + 1], Wt, stride=(st, st), pad=(pd, pd))
        assert np.array_equal(got[n:n + 1], want), "image %d: %s" % (n, first_mismatch(got[n:n + 1], want))


@pytest.mark.parametrize("case", TMA_CASES[:4] + TMA_CASES[6:7])
def test_implicit_im2col_cta_pair(mg, case):
    Nb, H, W, Cin, Cout, R, S, stride, pad, dil = case
    mg.mipgemm_set_tuning(force_path=mg.PATH_DENSE_PAIR)
    try:
        p = check_conv(mg, Nb, H, W, Cin, Cout, R, S, stride, pad, dil, seed=40, expect_flag=mg.PATH_IM2COL_TMA)
        assert p & mg.PATH_MASK == mg.PATH_DENSE_PAIR
        check_conv(mg, Nb, H, W, Cin, Cout, R, S, stride, pad, dil, seed=41, accumulate=True)
    finally:
        mg.mipgemm_set_tuning()


@pytest.mark.parametrize("layer", [12, 16, 18, 22])
def test_resnet50_k_heavy_layers_batch32_cta_pair(mg, layer):
    """The K >= 2304 layers once more with the CTA-pair kernel forced (im2col loads in their cta_group::2
    form at full size): three whole images against the oracle."""
    _cnt, H, W, Cin, Cout, R, S, st, pd = inputs.RESNET50_CONVS[layer]
    Nb = 32
    X, Wt = conv_inputs(Nb, H, W, Cin, Cout, R, S, inputs.seed_for(3, layer) + 3)
    mg.mipgemm_set_tuning(force_path=mg.PATH_DENSE_PAIR)
    try:
        got, path = run_conv(mg, X, Wt, (st, st), (pd, pd), (1, 1))
    finally:
        mg.mipgemm_set_tuning()
    assert path & mg.PATH_MASK == mg.PATH_DENSE_PAIR and path & mg.PATH_IM2COL_TMA
    for n in (0, 13, Nb - 1):
        want = orc.conv(X[n:n + 1], Wt, stride=(st, st), pad=(pd, pd))
        assert np.array_equal(got[n:n + 1], want), "image %d: %s" % (n, first_mismatch(got[n:n + 1], want))


@pytest.mark.parametrize("layer", range(len(inputs.RESNET50_CONVS)))
def test_resnet50_layers_batch128_sampled_images(mg, layer):
    """Batch 128 (the largest configuration: the stem's GEMM has 1.6 M rows): full batch on the GPU,
    three whole images recomputed by the oracle."""
    _cnt, H, W, Cin, Cout, R, S, st, pd = inputs.RESNET50_CONVS[layer]
    Nb = 128
    X, Wt = conv_inputs(Nb, H, W, Cin, Cout, R, S, inputs.seed_for(3, layer) + 7)
    got, _ = run_conv(mg, X, Wt, (st, st), (pd, pd), (1, 1))
    for n in (0, 63, Nb - 1):
        want = orc.conv(X[n:n + 1], Wt, stride=(st, st), pad=(pd, pd))
        assert np.array_equal(got[n:n + 1], want), "image %d: %s" % (n, first_mismatch(got[n:n + 1], want))
