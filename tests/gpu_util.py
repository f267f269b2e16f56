"""Helpers for the GPU parity tests: upload seeded operands, call the C ABI through the
Python binding, bring the result back.  No arithmetic of the method lives here."""
import numpy as np


def _torch():
    import torch
    return torch


def to_dev(arr: np.ndarray, misalign: int = 0):
    """Uploads a flat array; ``misalign`` bytes of offset from a 256-byte boundary."""
    torch = _torch()
    flat = np.ascontiguousarray(arr).reshape(-1)
    raw = flat.view(np.uint8)
    buf = torch.empty(raw.size + misalign + 256, dtype=torch.uint8, device="cuda")
    view = buf[misalign:misalign + raw.size]
    view.copy_(torch.from_numpy(raw.copy()))
    return view, buf


def run_gemm(mg, mode, M, N, K, A, B, *, lda=None, ldb=None, C=None, ldc=None, accumulate=False,
             misalign_a=0, misalign_b=0, expect_path=None):
    """Returns the full C buffer (with padding columns) as a flat int32 array."""
    torch = _torch()
    lda = K if lda is None else lda
    ldb = K if ldb is None else ldb
    ldc = N if ldc is None else ldc
    if C is None:
        C = np.full(max(M, 1) * ldc, 0x7F7F7F7F, dtype=np.int32)     # poison: accumulate=0 must ignore it
    dA, _ka = to_dev(A, misalign_a)
    dB, _kb = to_dev(B, misalign_b)
    dC, _kc = to_dev(C)
    fn = mg.mipgemm_s8s8s32 if mode == "s8" else mg.mipgemm_u8s8s32
    fn(M, N, K, dA, lda, dB, ldb, dC, ldc, accumulate)
    assert mg.mipgemm_device_status() == mg.OK
    path = mg.mipgemm_last_path()
    if expect_path is not None:
        assert path & mg.PATH_MASK == expect_path, hex(path)
    out = dC.cpu().numpy().view(np.int32).copy()
    torch.cuda.synchronize()
    return out, path


def run_conv(mg, X, Wt, stride, pad, dil, Y=None, accumulate=False, x_misalign=0):
    from oracle.mip_oracle import conv_out_hw
    Nb, H, W, Cin = X.shape
    Cout, R, S, _ = Wt.shape
    Ho, Wo = conv_out_hw(H, W, R, S, stride, pad, dil)
    if Y is None:
        Y = np.full((Nb, Ho, Wo, Cout), 0x7F7F7F7F, dtype=np.int32)
    dX, _kx = to_dev(X, x_misalign)
    dW, _kw = to_dev(Wt, x_misalign)
    dY, _ky = to_dev(Y)
    mg.mipgemm_conv_u8s8s32(Nb, H, W, Cin, Cout, R, S, stride[0], stride[1], pad[0], pad[1],
                            dil[0], dil[1], dX, dW, dY, accumulate)
    assert mg.mipgemm_device_status() == mg.OK
    path = mg.mipgemm_last_path()
    out = dY.cpu().numpy().view(np.int32).reshape(Nb, Ho, Wo, Cout).copy()
    return out, path


def first_mismatch(got: np.ndarray, want: np.ndarray) -> str:
    bad = np.argwhere(got != want)
    if bad.size == 0:
        return "equal"
    idx = tuple(int(v) for v in bad[0])
    return "%d mismatches; first at %s: got %d want %d" % (len(bad), idx, int(got[idx]), int(want[idx]))
