"""The allocation-free entry point against the regular one.

``mipgemm_s8s8s32_static_scratch`` serves callers that must not reach the CUDA allocator (a
memory-planned runtime that owns the device, a real-time loop, a plug-in under another
framework's pool): its re-pitching scratch is a fixed array inside the library instead of a
cudaMallocAsync allocation.  The array is shared by every call and keeps the previous call's
bytes, so the test makes two different calls in a row and compares each, bit for bit, with what
``mipgemm_s8s8s32`` produces for the same operands and with the CPU oracle; after each call the
entry point's own allocation-free status query must report that no device-side wait ran out, and
the path query must name the kernel family that ran.  This file is collected last on purpose: if
it fails, a run that stops at the first failure has already run everything else; it also passes
when it is the only test of a fresh process (the new entry point does its own device set-up).
"""
import numpy as np
import pytest

from paper_2506_11728_b200 import inputs
from gpu_util import to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mg():
    from paper_2506_11728_b200 import binding
    return binding


def _both(mg, M, N, K, lda, ldb, ldc, accumulate, seed, misalign=0):
    """Runs the static-scratch entry point first, then the regular one, on identical operands."""
    import torch
    A = inputs.uniform_s8(M * lda, seed + 1)
    B = inputs.uniform_s8(N * ldb, seed + 2)
    C0 = inputs.uniform_s32(M * ldc, seed + 3)
    dA, _ka = to_dev(A, misalign)
    dB, _kb = to_dev(B, misalign)
    outs = []
    for fn in (mg.mipgemm_s8s8s32_static_scratch, mg.mipgemm_s8s8s32):
        dC, _kc = to_dev(C0)
        fn(M, N, K, dA, lda, dB, ldb, dC, ldc, accumulate)
        if fn is mg.mipgemm_s8s8s32_static_scratch:
            assert mg.mipgemm_static_scratch_status() == mg.OK       # synchronises; nothing gave up a wait
            path = mg.mipgemm_last_path()
            assert path & mg.PATH_MASK in (mg.PATH_DENSE, mg.PATH_DENSE_PAIR), hex(path)
            needs_scratch = mg.mipgemm_workspace_query_gemm(M, N, K, dA, lda, dB, ldb, dC, ldc) > 0
            assert bool(path & mg.PATH_REPACK) == needs_scratch
        torch.cuda.synchronize()
        outs.append(dC.cpu().numpy().view(np.int32).copy())
    # the oracle's word on the same operands (padding columns of C keep their seeded contents)
    from oracle import mip_oracle as orc
    want = orc.gemm(A, B, M, N, K, lda=lda, ldb=ldb, C=C0.copy(), ldc=ldc, accumulate=bool(accumulate))
    assert np.array_equal(outs[0], want)
    return outs


def test_static_scratch_matches_regular_entry_point_twice_in_a_row(mg):
    # first call: both operands re-pitched (odd K and pitches), large enough to fill 3 MB of the array
    new, ref = _both(mg, 1000, 3001, 777, 777, 777, 3001, accumulate=1, seed=inputs.seed_for(2, 0))
    assert np.array_equal(new, ref)
    # second call right after it: smaller operands land on top of the first call's leftovers
    new, ref = _both(mg, 130, 70, 100, 101, 103, 71, accumulate=0, seed=21)
    assert np.array_equal(new, ref)
    # aligned pitches but misaligned base pointers, and a case that needs no scratch at all
    new, ref = _both(mg, 140, 90, 160, 160, 160, 92, accumulate=0, seed=22, misalign=3)
    assert np.array_equal(new, ref)
    new, ref = _both(mg, 300, 520, 400, 400, 400, 520, accumulate=1, seed=23)
    assert np.array_equal(new, ref)


def test_static_scratch_limit_is_enforced_before_anything_runs(mg):
    # 6000 x 1553 and 4000 x 1553 bytes re-pitched to 1568: 15.7 MB > 8 MiB
    before = mg.mipgemm_launch_count()
    st = mg.mipgemm_s8s8s32_static_scratch(6000, 4000, 1553, 256, 1553, 512, 1553, 1024, 4000, 0, 0, check=False)
    assert st == mg.ERR_STATIC_SCRATCH_LIMIT
    assert mg.mipgemm_launch_count() == before
    assert "static" in mg.mipgemm_status_string(st)
    assert mg.mipgemm_s8s8s32_static_scratch(4, 4, 8, 256, 7, 512, 8, 1024, 4, 0, 0, check=False) == mg.ERR_INVALID_ARG
