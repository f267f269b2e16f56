"""Seeded random shapes, pitches, alignments and geometries through every entry point, against the oracle.
MIPGEMM_FUZZ_CASES raises the number of cases per entry point (default 25)."""
import os

import numpy as np
import pytest

from oracle import mip_oracle as orc
from paper_2506_11728_b200 import inputs
from gpu_util import run_gemm, run_conv, to_dev, first_mismatch

pytestmark = pytest.mark.gpu
CASES = int(os.environ.get("MIPGEMM_FUZZ_CASES", "25"))


@pytest.fixture(scope="module")
def mg():
    from paper_2506_11728_b200 import binding
    binding.mipgemm_set_tuning()
    return binding


def dims(rng, big=False):
    pick = lambda: int(rng.choice([rng.integers(1, 20), rng.integers(20, 200), rng.integers(200, 700 if not big else 1500)]))
    return pick(), pick(), int(rng.choice([rng.integers(1, 40), rng.integers(40, 300), rng.integers(300, 1200)]))


def test_fuzz_gemm(mg):
    rng = np.random.default_rng(2024)
    for i in range(CASES):
        M, N, K = dims(rng, big=True)
        mode = "u8" if rng.integers(2) else "s8"
        lda, ldb, ldc = K + int(rng.choice([0, 0, 1, 16, 37])), K + int(rng.choice([0, 0, 3, 16, 48])), N + int(rng.choice([0, 0, 1, 4, 9]))
        acc = bool(rng.integers(2))
        A = (inputs.uniform_u8 if mode == "u8" else inputs.uniform_s8)(M * lda, 1000 + i)
        B = inputs.uniform_s8(N * ldb, 2000 + i)
        C0 = inputs.uniform_s32(M * ldc, 3000 + i) if acc else None
        got, path = run_gemm(mg, mode, M, N, K, A, B, lda=lda, ldb=ldb, ldc=ldc, C=None if C0 is None else C0.copy(),
                             accumulate=acc, misalign_a=int(rng.choice([0, 0, 1, 16])), misalign_b=int(rng.choice([0, 0, 5])))
        base = C0.copy() if acc else np.full(M * ldc, 0x7F7F7F7F, np.int32)
        want = orc.gemm(A, B, M, N, K, lda=lda, ldb=ldb, C=base, ldc=ldc, accumulate=acc)
        assert np.array_equal(got, want), "gemm case %d %s %dx%dx%d ld %d/%d/%d acc %d path %#x: %s" % (
            i, mode, M, N, K, lda, ldb, ldc, acc, path, first_mismatch(got, want))


def test_fuzz_gemm_forced_configurations(mg):
    """Random tile widths, pipeline depths, split factors and kernel forms (the planner's whole space)."""
    rng = np.random.default_rng(2028)
    try:
        for i in range(CASES):
            M, N, K = dims(rng, big=True)
            K = max(K, 16)
            tune = dict(block_n=int(rng.choice([0, 32, 64, 96, 128, 160, 192, 224, 256])),
                        stages=int(rng.choice([0, 2, 3, 5])), split_k=int(rng.choice([0, 0, 1, 2, 3, 7])),
                        force_path=int(rng.choice([0, mg.PATH_DENSE, mg.PATH_DENSE_PAIR])))
            mg.mipgemm_set_tuning(**tune)
            mode = "u8" if rng.integers(2) else "s8"
            acc = bool(rng.integers(2))
            ldc = N + int(rng.choice([0, 0, 4, 5]))
            A = (inputs.uniform_u8 if mode == "u8" else inputs.uniform_s8)(M * K, 12000 + i)
            B = inputs.uniform_s8(N * K, 13000 + i)
            C0 = inputs.uniform_s32(M * ldc, 14000 + i) if acc else None
            got, path = run_gemm(mg, mode, M, N, K, A, B, ldc=ldc, C=None if C0 is None else C0.copy(), accumulate=acc)
            base = C0.copy() if acc else np.full(M * ldc, 0x7F7F7F7F, np.int32)
            want = orc.gemm(A, B, M, N, K, C=base, ldc=ldc, accumulate=acc)
            assert np.array_equal(got, want), "forced case %d %s %dx%dx%d ldc %d acc %d %s path %#x: %s" % (
                i, mode, M, N, K, ldc, acc, tune, path, first_mismatch(got, want))
    finally:
        mg.mipgemm_set_tuning()


def test_fuzz_tall_and_skinny(mg):
    """Many tiles per CTA with short main loops (tall M, small K), and the M <= 16 streaming kernels."""
    rng = np.random.default_rng(2029)
    try:
        for i in range(CASES):
            if rng.integers(2):
                M, N, K = int(rng.integers(20000, 90000)), int(rng.choice([8, 32, 40, 96, 100, 160, 224, 260])), int(rng.choice([16, 32, 64, 80, 128, 200]))
                mg.mipgemm_set_tuning(block_n=int(rng.choice([0, 0, 32, 96, 160])),
                                      force_path=int(rng.choice([0, 0, mg.PATH_DENSE, mg.PATH_DENSE_PAIR])))
            else:
                M, N, K = int(rng.integers(1, 17)), int(rng.choice([16, 100, 2368, 4096, 5000])), int(rng.choice([128, 256, 1000, 2048, 4096]))
                mg.mipgemm_set_tuning()
                mg.mipgemm_set_weights_constant(int(rng.integers(2)))
            mode = "u8" if rng.integers(2) else "s8"
            acc = bool(rng.integers(2))
            A = (inputs.uniform_u8 if mode == "u8" else inputs.uniform_s8)(M * K, 15000 + i)
            B = inputs.uniform_s8(N * K, 16000 + i)
            C0 = inputs.uniform_s32(M * N, 17000 + i) if acc else None
            got, path = run_gemm(mg, mode, M, N, K, A, B, C=None if C0 is None else C0.copy(), accumulate=acc)
            base = C0.copy() if acc else np.full(M * N, 0x7F7F7F7F, np.int32)
            want = orc.gemm(A, B, M, N, K, C=base, accumulate=acc)
            assert np.array_equal(got, want), "tall/skinny case %d %s %dx%dx%d acc %d path %#x: %s" % (
                i, mode, M, N, K, acc, path, first_mismatch(got, want))
    finally:
        mg.mipgemm_set_tuning()
        mg.mipgemm_set_weights_constant(0)


def test_fuzz_batched(mg):
    rng = np.random.default_rng(2030)
    for i in range(CASES):
        batch = int(rng.integers(1, 9))
        M, N, K = int(rng.integers(1, 300)), int(rng.integers(1, 300)), int(rng.choice([16, 48, 64, 100, 256, 512]))
        lda, ldb, ldc = K + 16 * int(rng.integers(2)), K + 16 * int(rng.integers(2)), N + 4 * int(rng.integers(3))
        sa, sb, sc = M * lda + 16 * int(rng.integers(3)), N * ldb, M * ldc + 4 * int(rng.integers(3))
        acc = bool(rng.integers(2))
        A = inputs.uniform_s8(batch * sa, 18000 + i)
        B = inputs.uniform_s8(batch * sb, 19000 + i)
        C0 = inputs.uniform_s32(batch * sc, 20000 + i)
        want = C0.copy()
        for b in range(batch):
            Cb = np.ascontiguousarray(C0[b * sc:b * sc + M * ldc])
            res = orc.gemm(A[b * sa:b * sa + M * lda], B[b * sb:b * sb + N * ldb], M, N, K, lda=lda, ldb=ldb, C=Cb.copy(),
                           ldc=ldc, accumulate=acc)
            want[b * sc:b * sc + M * ldc] = res
            if not acc:     # padding columns keep their old value
                w2 = want[b * sc:b * sc + M * ldc].reshape(M, ldc)
                w2[:, N:] = C0[b * sc:b * sc + M * ldc].reshape(M, ldc)[:, N:]
        dA, _a = to_dev(A)
        dB, _b = to_dev(B)
        dC, _c = to_dev(C0)
        mg.mipgemm_batched_s8s8s32(batch, M, N, K, dA, lda, sa, dB, ldb, sb, dC, ldc, sc, acc)
        assert mg.mipgemm_device_status() == mg.OK
        got = dC.cpu().numpy().view(np.int32)
        assert np.array_equal(got, want), "batched case %d b%d %dx%dx%d ld %d/%d/%d acc %d path %#x: %s" % (
            i, batch, M, N, K, lda, ldb, ldc, acc, mg.mipgemm_last_path(), first_mismatch(got, want))


def test_fuzz_gemm_ex(mg):
    rng = np.random.default_rng(2025)
    for i in range(CASES):
        M, N, K = dims(rng)
        au, bu, ao, bo, cc = (int(rng.integers(2)) for _ in range(5))
        align = bool(rng.integers(2))
        if align:       # pitches TMA can address: the operand is read in place
            M, N, K = (M + 15) // 16 * 16, (N + 15) // 16 * 16, (K + 15) // 16 * 16
        lda, ldb, ldc = (M if ao else K), (N if bo else K), (M if cc else N) + 4 * int(rng.integers(3))
        a_rows, b_rows, c_rows = (K if ao else M), (K if bo else N), (N if cc else M)
        A = (inputs.uniform_u8 if au else inputs.uniform_s8)(a_rows * lda, 4000 + i)
        B = (inputs.uniform_u8 if bu else inputs.uniform_s8)(b_rows * ldb, 5000 + i)
        acc = bool(rng.integers(2))
        C0 = inputs.uniform_s32(c_rows * ldc, 6000 + i)
        A_can = np.ascontiguousarray(A.reshape(a_rows, lda).T if ao else A.reshape(a_rows, lda))
        B_can = np.ascontiguousarray(B.reshape(b_rows, ldb).T if bo else B.reshape(b_rows, ldb))
        C2 = C0.reshape(c_rows, ldc)[:, :(M if cc else N)]
        C_can = np.ascontiguousarray(C2.T if cc else C2)
        res = orc.gemm(A_can.reshape(-1), B_can.reshape(-1), M, N, K, C=C_can.reshape(-1).copy(), accumulate=acc).reshape(M, N)
        want = C0.reshape(c_rows, ldc).copy()
        want[:, :(M if cc else N)] = res.T if cc else res
        dA, _a = to_dev(A)
        dB, _b = to_dev(B)
        dC, _c = to_dev(C0)
        mg.mipgemm_gemm_ex(au, bu, ao, bo, cc, M, N, K, dA, lda, dB, ldb, dC, ldc, acc)
        assert mg.mipgemm_device_status() == mg.OK
        got = dC.cpu().numpy().view(np.int32).reshape(c_rows, ldc)
        assert np.array_equal(got, want), "gemm_ex case %d signs %d%d orders %d%d ccol %d %dx%dx%d path %#x" % (
            i, au, bu, ao, bo, cc, M, N, K, mg.mipgemm_last_path())


def test_fuzz_conv(mg):
    rng = np.random.default_rng(2026)
    for i in range(CASES):
        Cin = int(rng.choice([1, 3, 5, 16, 24, 64, 128, 192]))
        R, S = int(rng.integers(1, 5)), int(rng.integers(1, 5))
        dil = (int(rng.integers(1, 3)), int(rng.integers(1, 3)))
        pad = (int(rng.integers(0, 3)), int(rng.integers(0, 3)))
        stride = (int(rng.integers(1, 4)), int(rng.integers(1, 4)))
        H = int(rng.integers(dil[0] * (R - 1) + 1, 24)) if dil[0] * (R - 1) + 1 < 24 else dil[0] * (R - 1) + 1
        W = int(rng.integers(dil[1] * (S - 1) + 1, 24)) if dil[1] * (S - 1) + 1 < 24 else dil[1] * (S - 1) + 1
        Nb = int(rng.integers(1, 4)) if rng.integers(5) else int(rng.integers(16, 200))     # sometimes many tiles per CTA
        Cout = int(rng.choice([4, 7, 32, 64, 100]))
        X = inputs.uniform_u8(Nb * H * W * Cin, 7000 + i).reshape(Nb, H, W, Cin)
        Wt = inputs.normal_s8(Cout * R * S * Cin, 8000 + i, 32.0, -127, 127).reshape(Cout, R, S, Cin)
        acc = bool(rng.integers(2))
        Ho, Wo = orc.conv_out_hw(H, W, R, S, stride, pad, dil)
        Y0 = inputs.uniform_s32(Nb * Ho * Wo * Cout, 9000 + i).reshape(Nb, Ho, Wo, Cout) if acc else None
        want = orc.conv(X, Wt, stride=stride, pad=pad, dil=dil, Y=None if Y0 is None else Y0.copy(), accumulate=acc)
        got, path = run_conv(mg, X, Wt, stride, pad, dil, Y=None if Y0 is None else Y0.copy(), accumulate=acc,
                             x_misalign=int(rng.choice([0, 0, 0, 3])))
        assert np.array_equal(got, want), "conv case %d %s f%dx%d s%s p%s d%s cout %d acc %d path %#x: %s" % (
            i, X.shape, R, S, stride, pad, dil, Cout, acc, path, first_mismatch(got, want))


def test_fuzz_conv_scaled_outputs_with_bias(mg):
    """Random convolution geometries through the fused transforms, every other case with a per-channel bias."""
    rng = np.random.default_rng(2031)
    for i in range(CASES):
        Cin = int(rng.choice([1, 3, 16, 64, 128]))
        R, S = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        pad = (int(rng.integers(0, 2)), int(rng.integers(0, 2)))
        stride = (int(rng.integers(1, 3)), int(rng.integers(1, 3)))
        H, W = int(rng.integers(R, 20)), int(rng.integers(S, 20))
        Nb = int(rng.integers(1, 4)) if rng.integers(4) else int(rng.integers(16, 120))
        Cout = int(rng.choice([4, 7, 32, 64, 100]))
        X = inputs.uniform_u8(Nb * H * W * Cin, 17000 + i).reshape(Nb, H, W, Cin)
        Wt = inputs.normal_s8(Cout * R * S * Cin, 18000 + i, 32.0, -127, 127).reshape(Cout, R, S, Cin)
        sums = orc.conv(X, Wt, stride=stride, pad=pad)
        dbias = None
        if rng.integers(2):
            bias = rng.integers(-100000, 100001, size=Cout, dtype=np.int64).astype(np.int32)
            sums = orc.add_bias(sums, bias)
            dbias, _k = to_dev(bias, int(rng.choice([0, 4])))
        scale = float(np.float32(255.0 / (4.0 * 32.0 * 147.0 * np.sqrt(R * S * Cin))))
        dX, _x = to_dev(X)
        dW, _w = to_dev(Wt)
        dY, _y = to_dev(np.full(sums.size, 0x5A, np.uint8))
        geo = (Nb, H, W, Cin, Cout, R, S, stride[0], stride[1], pad[0], pad[1], 1, 1)
        mg.mipgemm_conv_u8s8u8_requant_bias(*geo, dX, dW, dY, scale, dbias)
        assert mg.mipgemm_device_status() == mg.OK
        want = orc.requant(sums, scale, 0, 255)
        got = dY.cpu().numpy().reshape(sums.shape).astype(np.int32)
        assert np.array_equal(got, want), "conv requant case %d %s f%dx%d cout %d bias %s" % (i, X.shape, R, S, Cout, dbias is not None)
        dF, _f = to_dev(np.zeros(sums.size, np.float32))
        mg.mipgemm_conv_u8s8f32_dequant_bias(*geo, dX, dW, dF, scale, dbias)
        assert mg.mipgemm_device_status() == mg.OK
        rule = (sums.astype(np.float32) * np.float32(scale)).astype(np.float32)
        assert np.array_equal(dF.cpu().numpy().view(np.float32).reshape(sums.shape), rule), "conv dequant case %d" % i


def test_fuzz_scaled_outputs(mg):
    rng = np.random.default_rng(2027)
    for i in range(CASES):
        M, N, K = dims(rng)
        unsigned = bool(rng.integers(2))
        A = (inputs.uniform_u8 if unsigned else inputs.uniform_s8)(M * K, 10000 + i)
        B = inputs.uniform_s8(N * K, 11000 + i)
        sums = orc.gemm(A, B, M, N, K).reshape(M, N)
        scale = float(np.float32(rng.choice([1.0, 0.5, 2.0 ** -7, 1.3e-3, 7.7e-5]) * (1 if rng.integers(2) else -1)))
        dA, _a = to_dev(A)
        dB, _b = to_dev(B)
        # every other case with a per-column bias (its pointer 4-, 8- or 16-byte aligned)
        dbias = None
        if rng.integers(2):
            bias = rng.integers(-200000, 200001, size=N, dtype=np.int64).astype(np.int32)
            sums = orc.add_bias(sums, bias)
            dbias, _k = to_dev(bias, int(rng.choice([0, 4, 8])))
        # 8-bit codes
        ldc = N + int(rng.choice([0, 3, 16]))
        dC, _c = to_dev(np.full(M * ldc, 0x5A, np.uint8), int(rng.choice([0, 1])))
        if unsigned:
            mg.mipgemm_u8s8u8_requant_bias(M, N, K, dA, K, dB, K, dC, ldc, scale, dbias)
            want = orc.requant(sums, scale, 0, 255)
            got = dC.cpu().numpy().reshape(M, ldc)[:, :N].astype(np.int32)
        else:
            relu = int(rng.integers(2))
            mg.mipgemm_s8s8s8_requant_bias(M, N, K, dA, K, dB, K, dC, ldc, scale, dbias, relu)
            want = orc.requant(sums, scale, 0 if relu else -128, 127)
            got = dC.cpu().numpy().reshape(M, ldc)[:, :N].view(np.int8).astype(np.int32)
        assert mg.mipgemm_device_status() == mg.OK
        assert np.array_equal(got, want), "requant case %d %dx%dx%d scale %g" % (i, M, N, K, scale)
        assert (dC.cpu().numpy().reshape(M, ldc)[:, N:] == 0x5A).all()
        # float32
        dF, _f = to_dev(np.zeros(M * N, np.float32))
        (mg.mipgemm_u8s8f32_dequant_bias if unsigned else mg.mipgemm_s8s8f32_dequant_bias)(M, N, K, dA, K, dB, K, dF, N,
                                                                                         scale, dbias)
        gotf = dF.cpu().numpy().view(np.float32).reshape(M, N)
        rule = (sums.astype(np.float32) * np.float32(scale)).astype(np.float32)
        assert np.array_equal(gotf, rule), "dequant case %d" % i


def test_concurrent_callers_on_their_own_streams(mg):
    """Four host threads, each with its own stream and a mix of paths (dense, skinny, re-pitched, conv, scaled)."""
    import threading
    import torch
    errors = []

    def worker(tid):
        try:
            rng = np.random.default_rng(3000 + tid)
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                for i in range(12):
                    M, N, K = int(rng.choice([5, 300, 1100])), int(rng.integers(40, 600)), int(rng.choice([64, 100, 512, 1000]))
                    A = inputs.uniform_s8(M * K, 30000 + 100 * tid + i)
                    B = inputs.uniform_s8(N * K, 31000 + 100 * tid + i)
                    dA, _a = to_dev(A)
                    dB, _b = to_dev(B)
                    dC, _c = to_dev(np.zeros(M * N, np.int32))
                    sums = orc.gemm(A, B, M, N, K)
                    if i % 3 == 2:
                        mg.mipgemm_s8s8f32_dequant(M, N, K, dA, K, dB, K, dC, N, 0.25, stream=stream)
                        stream.synchronize()
                        got = dC.cpu().numpy().view(np.float32)
                        ok = np.array_equal(got, sums.astype(np.float32) * np.float32(0.25))
                    else:
                        mg.mipgemm_s8s8s32(M, N, K, dA, K, dB, K, dC, N, 0, stream=stream)
                        stream.synchronize()
                        ok = np.array_equal(dC.cpu().numpy().view(np.int32), sums)
                    if not ok:
                        errors.append("thread %d case %d %dx%dx%d" % (tid, i, M, N, K))
        except Exception as exc:      # noqa: BLE001 - reported below
            errors.append("thread %d: %r" % (tid, exc))

    threads = [threading.Thread(target=worker, args=(t,)) for t in range(4)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    assert mg.mipgemm_device_status() == mg.OK


def test_fuzz_host_entry_and_lent_workspace(mg):
    """Host-buffer calls (single block and pipelined row blocks) and device calls with a lent workspace."""
    import torch
    rng = np.random.default_rng(2031)
    ws = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")
    try:
        for i in range(max(6, CASES // 3)):
            big = bool(rng.integers(2))
            M = int(rng.integers(2048, 6000)) if big else int(rng.integers(1, 900))
            N = int(rng.integers(1500, 2600)) if big else int(rng.integers(1, 500))
            K = int(rng.choice([512, 1000, 2048])) if big else int(rng.integers(1, 700))
            mode = "u8" if rng.integers(2) else "s8"
            acc = bool(rng.integers(2))
            lda, ldb, ldc = K + int(rng.choice([0, 5, 16])), K + int(rng.choice([0, 3])), N + int(rng.choice([0, 1, 8]))
            A = (inputs.uniform_u8 if mode == "u8" else inputs.uniform_s8)(M * lda, 21000 + i)
            B = inputs.uniform_s8(N * ldb, 22000 + i)
            C0 = inputs.uniform_s32(M * ldc, 23000 + i)
            rows = np.arange(M) if not big else np.unique(np.concatenate([np.arange(3), np.arange(M - 3, M), rng.integers(0, M, 24)]))
            want = orc.gemm(np.ascontiguousarray(A.reshape(M, lda)[rows]).reshape(-1), B, len(rows), N, K, lda=lda, ldb=ldb,
                            C=np.ascontiguousarray(C0.reshape(M, ldc)[rows]).reshape(-1), ldc=ldc, accumulate=acc)
            # host entry
            hA, hB, hC = torch.from_numpy(A.copy()), torch.from_numpy(B.copy()), torch.from_numpy(C0.copy())
            if rng.integers(2):
                hA, hB, hC = hA.pin_memory(), hB.pin_memory(), hC.pin_memory()
            (mg.mipgemm_host_u8s8s32 if mode == "u8" else mg.mipgemm_host_s8s8s32)(M, N, K, hA, lda, hB, ldb, hC, ldc, acc)
            assert np.array_equal(hC.numpy().reshape(M, ldc)[rows].reshape(-1), want), "host case %d %dx%dx%d" % (i, M, N, K)
            # device entry with a lent workspace (re-pitching scratch comes out of it)
            mg.mipgemm_set_workspace(ws, ws.numel())
            got, path = run_gemm(mg, mode, M, N, K, A, B, lda=lda, ldb=ldb, ldc=ldc, C=C0.copy(), accumulate=acc)
            mg.mipgemm_set_workspace(None, 0)
            assert np.array_equal(got.reshape(M, ldc)[rows].reshape(-1), want), "lent case %d %dx%dx%d path %#x" % (i, M, N, K, path)
    finally:
        mg.mipgemm_set_workspace(None, 0)
