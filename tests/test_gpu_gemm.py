"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, bit for bit."""
import numpy as np
import pytest

from oracle import mip_oracle as orc
from paper_2506_11728_b200 import inputs
from gpu_util import run_gemm, first_mismatch, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mg():
    from paper_2506_11728_b200 import binding
    binding.mipgemm_set_tuning()
    return binding


def make_ab(mode, M, N, K, lda, ldb, seed, dist="uniform"):
    if dist == "uniform":
        A = inputs.uniform_s8(M * lda, seed + 1) if mode == "s8" else inputs.uniform_u8(M * lda, seed + 1)
        B = inputs.uniform_s8(N * ldb, seed + 2)
    else:
        A = inputs.normal_s8(M * lda, seed + 1, 40.0)
        B = inputs.normal_s8(N * ldb, seed + 2, 20.0)
    return A, B


def check_case(mg, mode, M, N, K, *, lda=None, ldb=None, ldc=None, accumulate=False, seed=0,
               misalign_a=0, misalign_b=0, expect_path=None, dist="uniform"):
    lda = K if lda is None else lda
    ldb = K if ldb is None else ldb
    ldc = N if ldc is None else ldc
    A, B = make_ab(mode, M, N, K, lda, ldb, seed, dist)
    if accumulate:
        C0 = inputs.uniform_s32(M * ldc, seed + 3)
    else:
        C0 = np.full(M * ldc, 0x7F7F7F7F, dtype=np.int32)
    want = orc.gemm(A, B, M, N, K, lda=lda, ldb=ldb, C=C0.copy(), ldc=ldc, accumulate=accumulate)
    got, path = run_gemm(mg, mode, M, N, K, A, B, lda=lda, ldb=ldb, C=C0.copy(), ldc=ldc,
                         accumulate=accumulate, misalign_a=misalign_a, misalign_b=misalign_b,
                         expect_path=expect_path)
    # padding columns included: they must still hold what C0 held
    assert np.array_equal(got[:M * ldc], want), "%s M=%d N=%d K=%d acc=%d path=%#x: %s" % (
        mode, M, N, K, accumulate, path, first_mismatch(got[:M * ldc].reshape(M, ldc), want.reshape(M, ldc)))
    return path


def test_config1_512_cubed(mg):
    check_case(mg, "s8", 512, 512, 512, seed=inputs.seed_for(1, 0), expect_path=mg.PATH_DENSE)
    # BASELINE wording: zero-initialised C, accumulate=0 -- and accumulate onto it gives the same
    A, B = make_ab("s8", 512, 512, 512, 512, 512, inputs.seed_for(1, 0))
    want = orc.gemm(A, B, 512, 512, 512)
    got, _ = run_gemm(mg, "s8", 512, 512, 512, A, B, C=np.zeros(512 * 512, np.int32), accumulate=True)
    assert np.array_equal(got, want)


RAGGED = [
    (17, 16, 16), (128, 256, 128), (129, 257, 144), (127, 255, 112), (1, 1, 16), (33, 7, 48),
    (200, 40, 1040), (256, 512, 384), (255, 513, 400), (300, 100, 2048), (77, 300, 16),
    (640, 96, 272), (130, 130, 130 // 16 * 16 + 16),
]


@pytest.mark.parametrize("mode", ["s8", "u8"])
@pytest.mark.parametrize("accumulate", [False, True])
def test_ragged_shapes_dense(mg, mode, accumulate):
    mg.mipgemm_set_tuning(force_path=mg.PATH_DENSE)
    try:
        for i, (M, N, K) in enumerate(RAGGED):
            check_case(mg, mode, M, N, K, accumulate=accumulate, seed=100 + i, expect_path=mg.PATH_DENSE)
    finally:
        mg.mipgemm_set_tuning()


@pytest.mark.parametrize("block_n", [64, 96, 128, 160, 192, 224, 256])
def test_tile_widths_and_pitches(mg, block_n):
    mg.mipgemm_set_tuning(block_n=block_n)
    try:
        check_case(mg, "s8", 300, 700, 400, lda=416, ldb=432, ldc=708, seed=7)       # ldc % 4 == 0
        check_case(mg, "u8", 300, 700, 400, lda=400, ldb=400, ldc=705, seed=8, accumulate=True)  # scalar stores
        check_case(mg, "s8", 260, 520, 272, ldc=520, seed=9)
    finally:
        mg.mipgemm_set_tuning()


@pytest.mark.parametrize("stages", [2, 3])
def test_shallow_pipelines_wrap_phases(mg, stages):
    mg.mipgemm_set_tuning(block_n=128, stages=stages)
    try:
        check_case(mg, "s8", 700, 600, 1424, seed=11)
    finally:
        mg.mipgemm_set_tuning()


def test_many_tiles_per_cta_persistent_loop(mg):
    # 32 x 16 = 512 tiles of 128x128 on 148 CTAs: 3-4 tiles per CTA, both accumulators reused
    mg.mipgemm_set_tuning(block_n=128)
    try:
        check_case(mg, "s8", 4096, 2048, 256, seed=13)
    finally:
        mg.mipgemm_set_tuning()


def test_misaligned_operands_take_the_repack_path(mg):
    # config 2b: every pitch odd, accumulate onto a seeded C
    path = check_case(mg, "s8", 1000, 3001, 777, lda=777, ldb=777, ldc=3001, accumulate=True,
                      seed=inputs.seed_for(2, 0))
    assert path & mg.PATH_REPACK
    path = check_case(mg, "u8", 130, 70, 100, lda=101, ldb=103, ldc=71, seed=21)
    assert path & mg.PATH_REPACK
    # aligned pitches but misaligned base pointers
    path = check_case(mg, "s8", 140, 90, 160, misalign_a=3, misalign_b=5, seed=22)
    assert path & mg.PATH_REPACK
    path = check_case(mg, "s8", 5, 9, 13, seed=23)                                  # tiny, K % 16 != 0
    assert path & mg.PATH_REPACK


def test_split_k_reduction(mg):
    path = check_case(mg, "s8", 128, 256, 8192, seed=31)
    assert path & mg.PATH_SPLITK
    path = check_case(mg, "u8", 200, 100, 4096 + 48, accumulate=True, seed=32)
    assert path & mg.PATH_SPLITK
    mg.mipgemm_set_tuning(split_k=5)
    try:
        check_case(mg, "s8", 300, 300, 1296, ldc=301, seed=33)
    finally:
        mg.mipgemm_set_tuning()


def test_k_zero_and_empty(mg):
    M, N = 37, 21
    A = np.zeros(16, np.int8)
    B = np.zeros(16, np.int8)
    C0 = inputs.uniform_s32(M * (N + 3), 5)
    got, path = run_gemm(mg, "s8", M, N, 0, A, B, lda=0, ldb=0, C=C0.copy(), ldc=N + 3, accumulate=False)
    want = C0.reshape(M, N + 3).copy()
    want[:, :N] = 0
    assert np.array_equal(got.reshape(M, N + 3), want) and path & mg.PATH_MASK == mg.PATH_TRIVIAL
    got, _ = run_gemm(mg, "s8", M, N, 0, A, B, lda=0, ldb=0, C=C0.copy(), ldc=N + 3, accumulate=True)
    assert np.array_equal(got, C0)


@pytest.mark.parametrize("mode,a_val,b_val,per_k", [
    ("s8", -128, -128, 16384), ("s8", -128, 127, -16256), ("u8", 255, -128, -32640), ("u8", 255, 127, 32385)])
def test_extreme_values_closed_form(mg, mode, a_val, b_val, per_k):
    M, N, K = 256, 384, 2048
    A = np.full(M * K, a_val, dtype=np.int8 if mode == "s8" else np.uint8)
    B = np.full(N * K, b_val, dtype=np.int8)
    got, _ = run_gemm(mg, mode, M, N, K, A, B)
    assert (got == per_k * K).all()


def test_largest_exact_k(mg):
    # the K limits of the exactness contract, at the worst-case operand values
    for mode, K, a_val, expect in (("s8", 131071 // 16 * 16, -128, None), ("u8", 65793 // 16 * 16, 255, None)):
        M, N = 128, 64
        A = np.full(M * K, a_val, dtype=np.int8 if mode == "s8" else np.uint8)
        B = np.full(N * K, -128, dtype=np.int8)
        got, _ = run_gemm(mg, mode, M, N, K, A, B)
        assert (got.astype(np.int64) == int(a_val) * -128 * K).all()


def test_square_sweep_small_members_full_oracle(mg):
    for n in (1024, 2048):
        check_case(mg, "s8", n, n, n, seed=inputs.seed_for(2, n))
    n = 1024
    A = np.full(n * n, -128, np.int8)
    got, _ = run_gemm(mg, "s8", n, n, n, A, A)
    assert (got == 16384 * n).all()


BERT_T1024 = [(1024, N, K) for (_name, N, K) in inputs.BERT_GEMMS]


@pytest.mark.parametrize("shape", BERT_T1024)
def test_bert_shapes_t1024(mg, shape):
    M, N, K = shape
    check_case(mg, "s8", M, N, K, seed=inputs.seed_for(4, N + K), dist="normal")


@pytest.mark.parametrize("M", inputs.SKINNY_M)
@pytest.mark.parametrize("mode", ["s8", "u8"])
def test_skinny_small(mg, M, mode):
    for (N, K) in [(16, 16), (100, 272), (1000, 1040), (4096 + 7, 4096)]:
        for acc in (False, True):
            check_case(mg, mode, M, N, K, accumulate=acc, seed=200 + M, ldc=N + 1, expect_path=mg.PATH_SKINNY)
    # other M <= 16
    for Mx in (2, 3, 7, 9, 15):
        check_case(mg, mode, Mx, 333, 528, seed=300 + Mx, expect_path=mg.PATH_SKINNY)


@pytest.mark.parametrize("NK", inputs.SKINNY_WEIGHTS)
def test_skinny_full_size_weights(mg, NK):
    N, K = NK
    for M in (1, 16):
        check_case(mg, "s8", M, N, K, seed=inputs.seed_for(5, M), expect_path=mg.PATH_SKINNY)


def test_skinny_with_constant_weights_promise(mg):
    """The early weight fetch changes no result (several launches back to back on one stream)."""
    mg.mipgemm_set_weights_constant(1)
    try:
        for i, (M, N, K) in enumerate([(1, 4096, 4096), (8, 4096, 1024), (16, 2064, 2048), (4, 11008, 4096)]):
            check_case(mg, "s8", M, N, K, seed=700 + i, expect_path=mg.PATH_SKINNY)
            check_case(mg, "u8", M, N, K, seed=710 + i, accumulate=True, expect_path=mg.PATH_SKINNY)
    finally:
        mg.mipgemm_set_weights_constant(0)


def test_skinny_with_registered_weight_ranges(mg):
    """The per-buffer form of the promise: calls whose B lies inside a registered range fetch it early, other
    calls do not; results are the oracle's either way, also when the tokens are the previous call's output."""
    import torch
    M, N, K = 4, 4096, 4096
    A0 = inputs.uniform_s8(M * K, 5100)
    B1 = inputs.uniform_s8(N * K, 5200)
    B2 = inputs.uniform_s8(N * 4 * N, 5300)
    dA0, _k0 = to_dev(A0)
    dB1, _k1 = to_dev(B1)
    dB2, _k2 = to_dev(B2)
    dC = [torch.full((M * N,), 0x7F7F7F7F, dtype=torch.int32, device="cuda") for _ in range(4)]
    mg.mipgemm_register_constant_weights(dB1)                      # whole tensor
    mg.mipgemm_register_constant_weights(dB2, dB2.numel() // 2)    # only the first half: B2 is NOT covered
    try:
        torch.cuda.synchronize()
        mg.mipgemm_s8s8s32(M, N, K, dA0, K, dB1, K, dC[0], N, False)
        assert mg.mipgemm_last_path() & mg.PATH_MASK == mg.PATH_SKINNY
        mg.mipgemm_s8s8s32(M, N, 4 * N, dC[0].view(torch.uint8), 4 * N, dB2, 4 * N, dC[1], N, False)
        mg.mipgemm_s8s8s32(M, N, K, dC[1].view(torch.uint8)[:M * K], K, dB1, K, dC[2], N, False)
        mg.mipgemm_s8s8s32(M, N, K, dC[2].view(torch.uint8)[:M * K], K, dB1, K, dC[3], N, False)
        torch.cuda.synchronize()
        assert mg.mipgemm_device_status() == mg.OK
    finally:
        mg.mipgemm_unregister_constant_weights(dB1)
        mg.mipgemm_unregister_constant_weights(dB2)
    w0 = orc.gemm(A0, B1, M, N, K)
    w1 = orc.gemm(w0.view(np.int8), B2, M, N, 4 * N)
    w2 = orc.gemm(w1.view(np.int8)[:M * K].copy(), B1, M, N, K)
    w3 = orc.gemm(w2.view(np.int8)[:M * K].copy(), B1, M, N, K)
    for d, want in enumerate([w0, w1, w2, w3]):
        got = dC[d].cpu().numpy()
        assert np.array_equal(got, want), "launch %d: %s" % (d, first_mismatch(got, want))


@pytest.mark.parametrize("promise", [0, 1])
def test_skinny_ring_slots_reused_with_two_ctas_per_sm(mg, promise):
    """Few ring slots, several chunks per CTA and two CTAs streaming on every SM: a slot is refilled (an
    asynchronous write) right after its readers release it, so the release must come after their loads have
    been performed.  Releasing on the barrier arrive alone gave thousands of wrong columns in these cases."""
    mg.mipgemm_set_weights_constant(promise)
    try:
        for rep in range(3):
            for i, (M, N, K, acc) in enumerate([(15, 4096, 4096, True), (16, 4096, 4096, False), (4, 5000, 4096, True),
                                                (16, 14336, 4096, False), (8, 11008, 4096, False), (1, 4096, 11008, False)]):
                check_case(mg, "s8", M, N, K, seed=900 + 10 * rep + i, accumulate=acc, expect_path=mg.PATH_SKINNY)
    finally:
        mg.mipgemm_set_weights_constant(0)


@pytest.mark.parametrize("promise", [0, 1])
@pytest.mark.parametrize("M", [1, 4])
def test_skinny_chain_of_dependent_launches(mg, M, promise):
    """Six ring-form launches enqueued back to back, each reading as its tokens the bytes of the previous one's
    int32 output: a launch that starts under its predecessor's tail (programmatic dependent launch, CTAs of two
    calls on one SM) must still see that output complete."""
    import torch
    N, K0, depth = 4096, 4096, 6
    K = 4 * N
    A0 = inputs.uniform_s8(M * K0, 4100 + M)
    B0 = inputs.uniform_s8(N * K0, 4200 + M)
    B = inputs.uniform_s8(N * K, 4300 + M)
    dA0, _k0 = to_dev(A0)
    dB0, _k1 = to_dev(B0)
    dB, _k2 = to_dev(B)
    dC = [torch.full((M * N,), 0x7F7F7F7F, dtype=torch.int32, device="cuda") for _ in range(depth)]
    torch.cuda.synchronize()
    mg.mipgemm_set_weights_constant(promise)
    try:
        mg.mipgemm_s8s8s32(M, N, K0, dA0, K0, dB0, K0, dC[0], N, False)
        assert mg.mipgemm_last_path() & mg.PATH_MASK == mg.PATH_SKINNY
        for d in range(1, depth):
            mg.mipgemm_s8s8s32(M, N, K, dC[d - 1].view(torch.uint8), K, dB, K, dC[d], N, False)
    finally:
        mg.mipgemm_set_weights_constant(0)
    torch.cuda.synchronize()
    assert mg.mipgemm_device_status() == mg.OK
    want = orc.gemm(A0, B0, M, N, K0)
    for d in range(depth):
        got = dC[d].cpu().numpy()
        assert np.array_equal(got, want), "launch %d of the chain: %s" % (d, first_mismatch(got, want))
        if d + 1 < depth:
            want = orc.gemm(want.view(np.int8), B, M, N, K)


@pytest.mark.parametrize("M,N", [(300, 512), (2500, 256), (64, 1024)])
def test_dense_chain_of_dependent_launches(mg, M, N):
    """The same for the dense kernel, whose launches also start under their predecessor's tail: the bytes of one
    launch's int32 output are the next one's A."""
    import torch
    K0, depth = 192, 6
    K = 4 * N
    A0 = inputs.uniform_s8(M * K0, 4400 + M)
    B0 = inputs.uniform_s8(N * K0, 4500 + M)
    B = inputs.uniform_s8(N * K, 4600 + M)
    dA0, _k0 = to_dev(A0)
    dB0, _k1 = to_dev(B0)
    dB, _k2 = to_dev(B)
    dC = [torch.full((M * N,), 0x7F7F7F7F, dtype=torch.int32, device="cuda") for _ in range(depth)]
    torch.cuda.synchronize()
    mg.mipgemm_s8s8s32(M, N, K0, dA0, K0, dB0, K0, dC[0], N, False)
    for d in range(1, depth):
        mg.mipgemm_s8s8s32(M, N, K, dC[d - 1].view(torch.uint8), K, dB, K, dC[d], N, False)
        assert mg.mipgemm_last_path() & mg.PATH_MASK in (mg.PATH_DENSE, mg.PATH_DENSE_PAIR)
    torch.cuda.synchronize()
    assert mg.mipgemm_device_status() == mg.OK
    want = orc.gemm(A0, B0, M, N, K0)
    for d in range(depth):
        got = dC[d].cpu().numpy()
        assert np.array_equal(got, want), "launch %d of the chain: %s" % (d, first_mismatch(got, want))
        if d + 1 < depth:
            want = orc.gemm(want.view(np.int8), B, M, N, K)


def test_skinny_misaligned_falls_back_to_dense(mg):
    path = check_case(mg, "s8", 4, 300, 100, seed=41)
    assert path & mg.PATH_MASK == mg.PATH_DENSE and path & mg.PATH_REPACK


def test_lent_workspace(mg):
    import torch
    need = mg.mipgemm_workspace_query_gemm(130, 70, 100, 0, 101, 0, 103, 0, 71)
    assert need > 0
    buf = torch.empty(need, dtype=torch.uint8, device="cuda")
    assert mg.mipgemm_set_workspace(buf, need) == mg.OK
    try:
        check_case(mg, "u8", 130, 70, 100, lda=101, ldb=103, ldc=71, seed=21)
        small = torch.empty(256, dtype=torch.uint8, device="cuda")
        mg.mipgemm_set_workspace(small, 256)
        A = np.zeros(130 * 101, np.uint8)
        B = np.zeros(70 * 103, np.int8)
        from gpu_util import to_dev
        dA, _a = to_dev(A)
        dB, _b = to_dev(B)
        dC = torch.zeros(130 * 71, dtype=torch.int32, device="cuda")
        assert mg.mipgemm_u8s8s32(130, 70, 100, dA, 101, dB, 103, dC, 71, 0, check=False) == mg.ERR_WORKSPACE
    finally:
        mg.mipgemm_set_workspace(None, 0)


@pytest.mark.parametrize("mode", ["s8", "u8"])
@pytest.mark.parametrize("accumulate", [False, True])
def test_ragged_shapes_cta_pair_kernel(mg, mode, accumulate):
    """The cta_group::2 form on shapes that leave the second CTA of a pair partly or wholly empty."""
    mg.mipgemm_set_tuning(force_path=mg.PATH_DENSE_PAIR)
    try:
        for i, (M, N, K) in enumerate(RAGGED + [(513, 300, 272), (1000, 3000, 784)]):
            check_case(mg, mode, M, N, K, accumulate=accumulate, seed=400 + i, expect_path=mg.PATH_DENSE_PAIR)
        for bn in (64, 96, 128, 160, 192, 224):      # every tile width the planner may choose
            mg.mipgemm_set_tuning(block_n=bn, force_path=mg.PATH_DENSE_PAIR)
            check_case(mg, mode, 700, 600, 1424, accumulate=accumulate, seed=450 + bn, ldc=604,
                       expect_path=mg.PATH_DENSE_PAIR)
    finally:
        mg.mipgemm_set_tuning()


def test_odd_chunk_counts_keep_staging_buffers_apart(mg):
    """Tiles with an odd number of 32-column chunks, many tiles per CTA and almost no main loop: consecutive
    asynchronous stores (and split-K reduce-adds) must still alternate their staging buffers."""
    try:
        for tune, (M, N, K) in [(dict(block_n=96), (150000, 96, 32)), (dict(block_n=32), (100000, 32, 64)),
                                (dict(block_n=160, force_path=mg.PATH_DENSE_PAIR), (120000, 160, 32)),
                                (dict(block_n=32, split_k=3, stages=5), (962, 908, 586)),
                                (dict(block_n=96, split_k=2), (40000, 96, 256))]:
            mg.mipgemm_set_tuning(**tune)
            check_case(mg, "s8", M, N, K, seed=900 + N, accumulate=("split_k" in tune))
        mg.mipgemm_set_tuning()
        check_case(mg, "u8", 160000, 1000 - 8 * 3, 48, seed=950)          # ragged last tile column: 1 chunk of 8
    finally:
        mg.mipgemm_set_tuning()


def test_cta_pair_with_unaligned_c_and_repack(mg):
    mg.mipgemm_set_tuning(force_path=mg.PATH_DENSE_PAIR)
    try:
        path = check_case(mg, "s8", 1000, 3001, 777, lda=777, ldb=777, ldc=3001, accumulate=True, seed=460)
        assert path & mg.PATH_REPACK and path & mg.PATH_MASK == mg.PATH_DENSE_PAIR
        check_case(mg, "u8", 515, 259, 400, ldc=261, seed=461)
    finally:
        mg.mipgemm_set_tuning()


def test_padding_columns_survive_when_n_is_not_a_multiple_of_four(mg):
    """A 16-byte aligned C with N % 4 != 0: tile stores must not spill into the padding columns."""
    for (M, N, K, ldc) in [(300, 70, 400, 72), (257, 1001, 272, 1004), (129, 34, 144, 40)]:
        check_case(mg, "s8", M, N, K, ldc=ldc, seed=500 + N)
        check_case(mg, "u8", M, N, K, ldc=ldc, seed=510 + N, accumulate=True)
    mg.mipgemm_set_tuning(split_k=3)
    try:
        check_case(mg, "s8", 200, 70, 1296, ldc=72, seed=520)
    finally:
        mg.mipgemm_set_tuning()
    mg.mipgemm_set_tuning(force_path=mg.PATH_DENSE_PAIR)
    try:
        check_case(mg, "s8", 600, 1001, 400, ldc=1004, seed=530)
    finally:
        mg.mipgemm_set_tuning()
