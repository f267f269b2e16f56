"""Host-side runtime behaviour on a GPU: the unwinding path of the bounded device-side waits, the plan /
tensor-map cache, and concurrent calls from two host threads.  Nothing here faults, traps or hangs the
GPU: the expiry test withholds a signal inside the kernel (a flag that nothing sets), the wait runs out
after a fraction of a millisecond, every role leaves its loop and the kernel returns normally."""
import threading

import numpy as np
import pytest

from oracle import mip_oracle as orc
from paper_2506_11728_b200 import inputs
from gpu_util import first_mismatch, run_gemm, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mg():
    from paper_2506_11728_b200 import binding
    binding.mipgemm_set_tuning()
    return binding


def _exact(mg, mode, M, N, K, seed, **kw):
    gen = inputs.uniform_s8 if mode == "s8" else inputs.uniform_u8
    A, B = gen(M * K, seed), inputs.uniform_s8(N * K, seed + 1)
    got, path = run_gemm(mg, mode, M, N, K, A, B, **kw)
    want = orc.gemm(A, B, M, N, K)
    assert np.array_equal(got, want), first_mismatch(got.reshape(M, N), want.reshape(M, N))
    return path


def test_dense_kernel_wait_runs_out_and_the_kernel_returns(mg):
    """One-CTA dense kernel: the MMA warp never signals "accumulator ready", so the epilogue warps' wait
    runs out after 0.2 ms.  The kernel must come back by itself, the status query must report the
    timeout once, and the very next ordinary call must be exact."""
    import torch
    M, N, K = 128, 128, 1024
    A, B = inputs.uniform_s8(M * K, 61), inputs.uniform_s8(N * K, 62)
    dA, _ka = to_dev(A)
    dB, _kb = to_dev(B)
    dC = torch.zeros(M * N, dtype=torch.int32, device="cuda")
    mg.mipgemm_set_tuning(force_path=mg.PATH_DENSE)
    mg.mipgemm_debug_set(flags=1, wait_budget_ns=200_000)
    try:
        assert mg.mipgemm_s8s8s32(M, N, K, dA, K, dB, K, dC, N, 0) == mg.OK      # enqueued fine
        assert mg.mipgemm_last_path() & mg.PATH_MASK == mg.PATH_DENSE
        assert mg.mipgemm_device_status() == mg.ERR_TIMEOUT                      # synchronises; flag set
    finally:
        mg.mipgemm_debug_set(0, 0)
        mg.mipgemm_set_tuning()
    assert mg.mipgemm_device_status() == mg.OK                                   # ... and cleared by the query
    torch.cuda.synchronize()
    mg.mipgemm_set_tuning(force_path=mg.PATH_DENSE)
    try:
        _exact(mg, "s8", M, N, K, 63, expect_path=mg.PATH_DENSE)
        _exact(mg, "u8", 300, 520, 400, 64, expect_path=mg.PATH_DENSE)
    finally:
        mg.mipgemm_set_tuning()
    assert mg.mipgemm_device_status() == mg.OK


@pytest.mark.parametrize("M", [4, 16])
def test_skinny_ring_wait_runs_out_and_the_kernel_returns(mg, M):
    """Skinny ring kernels (the form for up to 8 tokens and the one for 9 to 16): the first CTA never loads the
    second k-chunk of its first unit, so its consumer warps' wait for that slot runs out; all 256 consumer
    threads decide together to leave."""
    import torch
    N, K = 4096, 4096
    A, B = inputs.uniform_s8(M * K, 71), inputs.uniform_s8(N * K, 72)
    dA, _ka = to_dev(A)
    dB, _kb = to_dev(B)
    dC = torch.zeros(M * N, dtype=torch.int32, device="cuda")
    mg.mipgemm_debug_set(flags=1, wait_budget_ns=200_000)
    try:
        assert mg.mipgemm_s8s8s32(M, N, K, dA, K, dB, K, dC, N, 0) == mg.OK
        assert mg.mipgemm_last_path() & mg.PATH_MASK == mg.PATH_SKINNY
        assert mg.mipgemm_device_status() == mg.ERR_TIMEOUT
    finally:
        mg.mipgemm_debug_set(0, 0)
    assert mg.mipgemm_device_status() == mg.OK
    torch.cuda.synchronize()
    _exact(mg, "s8", M, N, K, 73, expect_path=mg.PATH_SKINNY)
    _exact(mg, "s8", 16, 4096, 4096, 74, expect_path=mg.PATH_SKINNY)
    assert mg.mipgemm_device_status() == mg.OK


def test_plan_cache_serves_repeated_calls_and_follows_the_tuning(mg):
    import torch
    on, _h, _m = mg.mipgemm_plan_cache_stats()
    if not on:
        pytest.skip("plan cache switched off in this process")
    M, N, K = 700, 1536, 640
    A, B = inputs.uniform_s8(M * K, 81), inputs.uniform_s8(N * K, 82)
    want = orc.gemm(A, B, M, N, K)
    dA, _ka = to_dev(A)
    dB, _kb = to_dev(B)
    dC = torch.empty(M * N, dtype=torch.int32, device="cuda")

    def call():
        dC.fill_(0x7F7F7F7F)
        mg.mipgemm_s8s8s32(M, N, K, dA, K, dB, K, dC, N, 0)
        assert mg.mipgemm_device_status() == mg.OK
        assert np.array_equal(dC.cpu().numpy(), want)

    _on, h0, m0 = mg.mipgemm_plan_cache_stats()
    call()
    _on, h1, m1 = mg.mipgemm_plan_cache_stats()
    assert m1 == m0 + 1 and h1 == h0                       # first sight of these arguments
    call()
    call()
    _on, h2, m2 = mg.mipgemm_plan_cache_stats()
    assert h2 == h1 + 2 and m2 == m1                       # served from the cache, same result
    mg.mipgemm_set_tuning(block_n=64)                      # a different plan must not be served from the old entry
    try:
        call()
        _on, h3, m3 = mg.mipgemm_plan_cache_stats()
        assert m3 == m2 + 1
    finally:
        mg.mipgemm_set_tuning()
    # accumulate and the unsigned mode are part of the key
    C0 = inputs.uniform_s32(M * N, 83)
    dC.copy_(torch.from_numpy(C0).cuda())
    mg.mipgemm_s8s8s32(M, N, K, dA, K, dB, K, dC, N, 1)
    assert np.array_equal(dC.cpu().numpy(), orc.gemm(A, B, M, N, K, C=C0.copy(), accumulate=True))
    mg.mipgemm_u8s8s32(M, N, K, dA, K, dB, K, dC, N, 0)
    assert np.array_equal(dC.cpu().numpy(), orc.gemm(A.view(np.uint8), B, M, N, K))


def test_two_host_threads_on_two_streams(mg):
    """Two host threads call the library at the same time, each on a stream of its own and with its own
    shapes (dense, CTA-pair, skinny, re-pitched operands); every result must be the oracle's."""
    import torch
    cases = [
        [("s8", 300, 520, 400), ("u8", 1000, 777, 333), ("s8", 8, 4096, 4096), ("s8", 2048, 2048, 512)],
        [("u8", 257, 129, 1000), ("s8", 16, 11008, 4096), ("s8", 513, 640, 77), ("u8", 1024, 4096, 256)],
    ]
    prepared = []
    for t, lst in enumerate(cases):
        items = []
        for i, (mode, M, N, K) in enumerate(lst):
            gen = inputs.uniform_s8 if mode == "s8" else inputs.uniform_u8
            A, B = gen(M * K, 900 + 10 * t + i), inputs.uniform_s8(N * K, 950 + 10 * t + i)
            dA, ka = to_dev(A)
            dB, kb = to_dev(B)
            dC = torch.empty(M * N, dtype=torch.int32, device="cuda")
            items.append((mode, M, N, K, A, B, dA, dB, dC, ka, kb))
        prepared.append(items)
    torch.cuda.synchronize()
    errors = []

    def worker(t):
        try:
            stream = torch.cuda.Stream()
            for rep in range(6):
                for (mode, M, N, K, A, B, dA, dB, dC, _ka, _kb) in prepared[t]:
                    fn = mg.mipgemm_s8s8s32 if mode == "s8" else mg.mipgemm_u8s8s32
                    fn(M, N, K, dA, K, dB, K, dC, N, 0, stream=stream)
            stream.synchronize()
        except Exception as exc:        # noqa: BLE001 (reported by the main thread)
            errors.append(repr(exc))

    threads = [threading.Thread(target=worker, args=(t,)) for t in range(2)]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    assert not errors, errors
    torch.cuda.synchronize()
    assert mg.mipgemm_device_status() == mg.OK
    for items in prepared:
        for (mode, M, N, K, A, B, _dA, _dB, dC, _ka, _kb) in items:
            want = orc.gemm(A, B, M, N, K)
            got = dC.cpu().numpy()
            assert np.array_equal(got, want), (mode, M, N, K, first_mismatch(got.reshape(M, N), want.reshape(M, N)))


def test_dispatch_log_names_the_path_taken():
    """MIPGEMM_LOG=1 prints one line per call with the dispatch decision (read at library load, hence a child
    process)."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = (
        "import torch\n"
        "from paper_2506_11728_b200 import binding as mg\n"
        "a = torch.zeros(1 << 22, dtype=torch.int8, device='cuda')\n"
        "c = torch.empty(1 << 22, dtype=torch.int32, device='cuda')\n"
        "mg.mipgemm_s8s8s32(512, 512, 512, a, 512, a, 512, c, 512, 0)\n"
        "mg.mipgemm_s8s8s32(512, 512, 512, a, 512, a, 512, c, 512, 0)\n"
        "mg.mipgemm_s8s8s32(4, 4096, 1024, a, 1024, a, 1024, c, 4096, 0)\n"
        "mg.mipgemm_u8s8s32(100, 200, 77, a, 77, a, 77, c, 200, 1)\n"
        "mg.mipgemm_conv_u8s8s32(2, 14, 14, 128, 64, 3, 3, 1, 1, 1, 1, 1, 1, a, a, c, 0)\n"
        "mg.mipgemm_conv_u8s8s32(2, 32, 32, 3, 64, 7, 7, 2, 2, 3, 3, 1, 1, a, a, c, 0)\n"
        "assert mg.mipgemm_device_status() == mg.OK\n")
    env = dict(os.environ, MIPGEMM_LOG="1", PYTHONPATH=root)
    out = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stderr.splitlines() if l.startswith("mipgemm:")]
    assert len(lines) == 6, lines
    assert "gemm s8 M=512 N=512 K=512 -> dense" in lines[0] and "plan=new" in lines[0]
    assert "plan=cached" in lines[1]
    assert "skinny" in lines[2]
    assert "re-pitched" in lines[3] and "accumulate" in lines[3]
    assert "conv (TMA im2col)" in lines[4]
    assert "conv (gathered im2col)" in lines[5]
