"""GPU parity for the host-buffer entry points (the end-to-end path): operands and result live in host
memory; large problems are cut into row blocks that three streams pipeline."""
import numpy as np
import pytest

from oracle import mip_oracle as orc
from paper_2506_11728_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mg():
    from paper_2506_11728_b200 import binding
    binding.mipgemm_set_tuning()
    return binding


def run_host(mg, mode, M, N, K, *, pad=(0, 0, 0), accumulate=False, pinned=False, seed=0, sampled_rows=None):
    import torch
    lda, ldb, ldc = K + pad[0], K + pad[1], N + pad[2]
    A = (inputs.uniform_u8 if mode == "u8" else inputs.uniform_s8)(M * lda, seed + 1)
    B = inputs.uniform_s8(N * ldb, seed + 2)
    C0 = inputs.uniform_s32(M * ldc, seed + 3) if accumulate else np.full(M * ldc, 0x7F7F7F7F, np.int32)
    hA, hB, hC = torch.from_numpy(A.copy()), torch.from_numpy(B.copy()), torch.from_numpy(C0.copy())
    if pinned:
        hA, hB, hC = hA.pin_memory(), hB.pin_memory(), hC.pin_memory()
    fn = mg.mipgemm_host_u8s8s32 if mode == "u8" else mg.mipgemm_host_s8s8s32
    fn(M, N, K, hA, lda, hB, ldb, hC, ldc, accumulate)           # synchronises before returning
    assert mg.mipgemm_device_status() == mg.OK
    got = hC.numpy().reshape(M, ldc)
    rows = np.arange(M) if sampled_rows is None else np.unique(np.concatenate(
        [np.arange(0, 3), np.arange(M - 3, M), np.random.default_rng(seed).integers(0, M, sampled_rows)]))
    A2 = A.reshape(M, lda)[rows]
    want = orc.gemm(np.ascontiguousarray(A2).reshape(-1), B, len(rows), N, K, lda=lda, ldb=ldb,
                    C=np.ascontiguousarray(C0.reshape(M, ldc)[rows]).reshape(-1), ldc=ldc, accumulate=accumulate)
    assert np.array_equal(got[rows].reshape(-1), want)            # padding columns included
    if sampled_rows is not None:                                  # every row was written (poison gone)
        assert not (got[:, :N] == 0x7F7F7F7F).all(axis=1).any() or accumulate


@pytest.mark.parametrize("mode", ["s8", "u8"])
def test_host_small_single_block(mg, mode):
    run_host(mg, mode, 300, 200, 400, seed=1)
    run_host(mg, mode, 130, 70, 100, pad=(3, 5, 7), accumulate=True, seed=2)
    run_host(mg, mode, 8, 4096, 512, pinned=True, seed=3)        # skinny path behind the host entry


@pytest.mark.parametrize("pinned", [False, True])
def test_host_large_is_pipelined_in_row_blocks(mg, pinned):
    # >= 2048 rows and >= 32 MB: eight row blocks, ragged last block (4100 rows), padded pitches
    run_host(mg, "s8", 4100, 2304, 1024, pad=(16, 0, 8), pinned=pinned, seed=10, sampled_rows=40)
    run_host(mg, "u8", 4096, 2048, 768, accumulate=True, pinned=pinned, seed=11, sampled_rows=40)
    run_host(mg, "s8", 9000, 1024, 512, pinned=pinned, seed=12, sampled_rows=40)        # the maximum of eight blocks


def test_host_argument_errors(mg):
    import torch
    h = torch.zeros(64, dtype=torch.int8)
    c = torch.zeros(64, dtype=torch.int32)
    assert mg.mipgemm_host_s8s8s32(4, 4, 8, h, 7, h, 8, c, 4, 0, check=False) == mg.ERR_INVALID_ARG
    assert mg.mipgemm_host_s8s8s32(4, 4, 8, 0, 8, h, 8, c, 4, 0, check=False) == mg.ERR_INVALID_ARG
    assert mg.mipgemm_host_s8s8s32(0, 4, 8, h, 8, h, 8, c, 4, 0) == mg.OK
