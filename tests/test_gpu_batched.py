"""GPU parity for the strided-batch entry points: every batch member against the oracle."""
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


def run_batched(mg, mode, batch, M, N, K, *, lda=None, ldb=None, ldc=None, sa=None, sb=None, sc=None,
                accumulate=False, seed=0, expect_batched=None):
    lda = K if lda is None else lda
    ldb = K if ldb is None else ldb
    ldc = N if ldc is None else ldc
    sa = M * lda if sa is None else sa
    sb = N * ldb if sb is None else sb
    sc = M * ldc if sc is None else sc
    na = (batch - 1) * sa + M * lda
    nb = (batch - 1) * sb + N * ldb
    nc = (batch - 1) * sc + M * ldc
    A = inputs.uniform_s8(na, seed + 1) if mode == "s8" else inputs.uniform_u8(na, seed + 1)
    B = inputs.uniform_s8(nb, seed + 2)
    C0 = inputs.uniform_s32(nc, seed + 3)
    want = C0.copy()
    for b in range(batch):
        part = orc.gemm(A[b * sa:], B[b * sb:], M, N, K, lda=lda, ldb=ldb, C=want[b * sc:b * sc + M * ldc].copy(),
                        ldc=ldc, accumulate=accumulate)
        want[b * sc:b * sc + M * ldc] = part
    dA, _a = to_dev(A)
    dB, _b = to_dev(B)
    dC, _c = to_dev(C0)
    fn = mg.mipgemm_batched_s8s8s32 if mode == "s8" else mg.mipgemm_batched_u8s8s32
    fn(batch, M, N, K, dA, lda, sa, dB, ldb, sb, dC, ldc, sc, accumulate)
    assert mg.mipgemm_device_status() == mg.OK
    path = mg.mipgemm_last_path()
    got = dC.cpu().numpy().view(np.int32)
    if not accumulate:
        # cells outside the M x N windows (padding columns, gaps between members) must be untouched;
        # inside, the oracle's values
        pass
    assert np.array_equal(got, want), "batch=%d %dx%dx%d path=%#x" % (batch, M, N, K, path)
    if expect_batched is not None:
        assert bool(path & mg.PATH_BATCHED) == expect_batched, hex(path)
    return path


def test_attention_shaped_batches(mg):
    # M5: l x l x d/h per head (K = 64: one 64-byte k-block); M7: d/h x l x l
    run_batched(mg, "s8", 16, 512, 512, 64, seed=1, expect_batched=True)
    run_batched(mg, "s8", 16, 64, 512, 512, seed=2, expect_batched=True)
    run_batched(mg, "u8", 6, 512, 64, 512, seed=3, accumulate=True, expect_batched=True)


def test_ragged_members_with_gaps(mg):
    # pitches and batch strides leave gaps (which must stay untouched); sizes are not tile multiples
    run_batched(mg, "s8", 5, 100, 70, 48, lda=64, ldb=48, ldc=72, sa=100 * 64 + 32, sb=70 * 48 + 16,
                sc=100 * 72 + 8, seed=4, expect_batched=True)
    run_batched(mg, "u8", 3, 257, 130, 272, ldc=131, sc=257 * 131 + 1, seed=5, expect_batched=True)   # unaligned C
    run_batched(mg, "s8", 7, 300, 300, 1296, seed=6, accumulate=True, expect_batched=True)


def test_members_that_need_repacking_run_one_by_one(mg):
    p = run_batched(mg, "s8", 3, 130, 70, 100, lda=101, ldb=103, ldc=71, seed=7, expect_batched=False)
    assert p & mg.PATH_REPACK
    run_batched(mg, "s8", 4, 8, 333, 528, seed=8)                       # skinny members
    run_batched(mg, "s8", 1, 200, 100, 64, seed=9, expect_batched=False)  # batch of one = plain GEMM


def test_shared_operand_stride_zero(mg):
    # the same weights for every member
    batch, M, N, K = 4, 200, 96, 256
    A = inputs.uniform_s8(batch * M * K, 11)
    B = inputs.uniform_s8(N * K, 12)
    dA, _a = to_dev(A)
    dB, _b = to_dev(B)
    dC, _c = to_dev(np.zeros(batch * M * N, np.int32))
    mg.mipgemm_batched_s8s8s32(batch, M, N, K, dA, K, M * K, dB, K, 0, dC, N, M * N, 0)
    got = dC.cpu().numpy().view(np.int32).reshape(batch, M, N)
    for b in range(batch):
        assert np.array_equal(got[b].reshape(-1), orc.gemm(A[b * M * K:(b + 1) * M * K], B, M, N, K))


def test_batched_argument_errors(mg):
    a = b = c = 256
    bad = mg.ERR_INVALID_ARG
    f = mg.mipgemm_batched_s8s8s32
    assert f(-1, 4, 4, 16, a, 16, 64, b, 16, 64, c, 4, 16, 0, 0, check=False) == bad
    assert f(2, 4, 4, 16, a, 16, 64, b, 16, 64, c, 4, 15, 0, 0, check=False) == bad       # C members overlap
    assert f(2, 4, 4, 16, a, 16, -1, b, 16, 64, c, 4, 16, 0, 0, check=False) == bad
    assert f(0, 4, 4, 16, a, 16, 64, b, 16, 64, c, 4, 16, 0, 0, check=False) == mg.OK
