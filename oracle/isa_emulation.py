"""Second, structurally independent CPU oracle: GEMM assembled from the instruction semantics the
paper prints (test infrastructure only; nothing in the product imports it).

Each function below restates, lane by lane, what the paper says one instruction computes
(Section 5.1: vmull_s8, vmlal_s8, vpadalq_s16, vpaddq_s32; Section 5.2: vdotq_laneq_s32;
Section 6.1: the 4x4x8 vmadot of the SpacemiT K1 matrix engine; Section 6.2: the 16x16x64
tile product of Intel AMX; Section 6.3: the sum of four outer products of ARM SME), with the lane
widths it states (int8 inputs, int16 or int32 lanes that wrap like the hardware's).  The small
GEMM drivers walk the operands in their own simple order -- they are not the paper's
micro-kernels and use none of its packing -- so that agreement with ``mip_oracle`` pins the
primary oracle against the paper's own description of the arithmetic rather than against itself.

The ARMv8.0 chain accumulates two int8 products in an int16 lane before widening: exact for
weights in [-127, 127], but (-128)(-128) + (-128)(-128) = 32768 wraps.  ``gemm_neon_v80`` shows
that behaviour; the exact definition (and the GPU library) does not share it.
"""
from __future__ import annotations

import numpy as np


def _wrap16(x):
    return ((np.asarray(x, dtype=np.int64) + 32768) % 65536 - 32768).astype(np.int64)


def _wrap32(x):
    return ((np.asarray(x, dtype=np.int64) + (1 << 31)) % (1 << 32) - (1 << 31)).astype(np.int64)


# --------------------------------------------------------------------------- Section 5.1 (ARMv8.0)
def vmull_s8(v0, v1):
    """Eight int8 x int8 products, each kept in an int16 lane."""
    v0 = np.asarray(v0, dtype=np.int64)
    v1 = np.asarray(v1, dtype=np.int64)
    assert v0.shape == v1.shape == (8,)
    return _wrap16(v0 * v1)


def vmlal_s8(v0, v1, v2):
    """Eight int16 lanes, each incremented by an int8 x int8 product (int16 wrap-around)."""
    v0 = np.asarray(v0, dtype=np.int64)
    assert v0.shape == (8,)
    return _wrap16(v0 + np.asarray(v1, dtype=np.int64) * np.asarray(v2, dtype=np.int64))


def vpadalq_s16(v0, v1):
    """Four int32 lanes, lane i incremented by int16 lanes 2i and 2i+1."""
    v0 = np.asarray(v0, dtype=np.int64)
    v1 = np.asarray(v1, dtype=np.int64)
    assert v0.shape == (4,) and v1.shape == (8,)
    return _wrap32(v0 + v1[0::2] + v1[1::2])


def vpaddq_s32(v0, v1):
    """Pairwise sums: [v0[0]+v0[1], v0[2]+v0[3], v1[0]+v1[1], v1[2]+v1[3]]."""
    v0 = np.asarray(v0, dtype=np.int64)
    v1 = np.asarray(v1, dtype=np.int64)
    return _wrap32(np.array([v0[0] + v0[1], v0[2] + v0[3], v1[0] + v1[1], v1[2] + v1[3]]))


def gemm_neon_v80(A, B):
    """C = A * B (A: M x K int8, B: K x N int8, K a multiple of 16) through the ARMv8.0 chain:
    per 16 values of k one vmull_s8, one vmlal_s8 on top of it, one vpadalq_s16 into four int32
    lanes; the four lanes are folded with two rounds of vpaddq_s32 at the end."""
    A = np.asarray(A, dtype=np.int64)
    B = np.asarray(B, dtype=np.int64)
    M, K = A.shape
    K2, N = B.shape
    assert K == K2 and K % 16 == 0
    C = np.zeros((M, N), dtype=np.int64)
    zero4 = np.zeros(4, dtype=np.int64)
    for i in range(M):
        for j in range(N):
            acc = zero4.copy()
            for k in range(0, K, 16):
                lanes = vmull_s8(A[i, k:k + 8], B[k:k + 8, j])
                lanes = vmlal_s8(lanes, A[i, k + 8:k + 16], B[k + 8:k + 16, j])
                acc = vpadalq_s16(acc, lanes)
            once = vpaddq_s32(acc, zero4)          # [acc0+acc1, acc2+acc3, 0, 0]
            C[i, j] = vpaddq_s32(once, zero4)[0]
    return C


# --------------------------------------------------------------------------- Section 5.2 (ARMv8.2)
def vdotq_laneq_s32(v0, v1, v2, lane):
    """vr[i] = v0[i] + sum_{t<4} v1[4i+t] * v2[4*lane+t], i = 0..3."""
    v0 = np.asarray(v0, dtype=np.int64)
    v1 = np.asarray(v1, dtype=np.int64).reshape(4, 4)
    v2 = np.asarray(v2, dtype=np.int64).reshape(4, 4)
    return _wrap32(v0 + v1 @ v2[lane])


def gemm_neon_dot(A, B):
    """C = A * B from 4-way dot products: a register of A holds 4 rows x 4 consecutive k, a
    register of B holds 4 columns x the same 4 k; lane j of the B register yields column j."""
    A = np.asarray(A, dtype=np.int64)
    B = np.asarray(B, dtype=np.int64)
    M, K = A.shape
    _, N = B.shape
    assert M % 4 == 0 and N % 4 == 0 and K % 4 == 0
    C = np.zeros((M, N), dtype=np.int64)
    for i0 in range(0, M, 4):
        for j0 in range(0, N, 4):
            cols = [np.zeros(4, dtype=np.int64) for _ in range(4)]     # cols[j][i] = C[i0+i, j0+j]
            for k in range(0, K, 4):
                va = A[i0:i0 + 4, k:k + 4].reshape(16)                 # row i -> elements 4i..4i+3
                vb = B[k:k + 4, j0:j0 + 4].T.reshape(16)               # column j -> elements 4j..4j+3
                for j in range(4):
                    cols[j] = vdotq_laneq_s32(cols[j], va, vb, j)
            for j in range(4):
                C[i0:i0 + 4, j0 + j] = cols[j]
    return C


# --------------------------------------------------------------------------- Section 6.1 (SpacemiT K1)
def vmadot(C_tile, A_reg, B_reg):
    """C(4x4, int32) += A(4x8, row-major in a 32-byte register) * B(8x4, column-major register)."""
    A = np.asarray(A_reg, dtype=np.int64).reshape(4, 8)          # row-major 4 x 8
    B = np.asarray(B_reg, dtype=np.int64).reshape(4, 8).T        # column-major 8 x 4
    return _wrap32(np.asarray(C_tile, dtype=np.int64) + A @ B)


def gemm_ime(A, B):
    A = np.asarray(A, dtype=np.int64)
    B = np.asarray(B, dtype=np.int64)
    M, K = A.shape
    _, N = B.shape
    assert M % 4 == 0 and N % 4 == 0 and K % 8 == 0
    C = np.zeros((M, N), dtype=np.int64)
    for i0 in range(0, M, 4):
        for j0 in range(0, N, 4):
            tile = np.zeros((4, 4), dtype=np.int64)
            for k in range(0, K, 8):
                a_reg = A[i0:i0 + 4, k:k + 8].reshape(32)               # rows one after the other
                b_reg = B[k:k + 8, j0:j0 + 4].T.reshape(32)             # columns one after the other
                tile = vmadot(tile, a_reg, b_reg)
            C[i0:i0 + 4, j0:j0 + 4] = tile
    return C


# --------------------------------------------------------------------------- Section 6.2 (Intel AMX)
def tile_dpbssd(C_tile, A_tile, B_tile):
    """C(16x16 int32) += A(16 x 64 int8, row-major) * B, where the B tile is stored as 16 rows of
    64 bytes: row p holds, for each of the 16 columns, the four k-values 4p..4p+3 contiguously."""
    A = np.asarray(A_tile, dtype=np.int64).reshape(16, 64)
    Bt = np.asarray(B_tile, dtype=np.int64).reshape(16, 16, 4)        # [k group][column][k in group]
    Bfull = Bt.transpose(0, 2, 1).reshape(64, 16)                     # k = 4*group + t
    return _wrap32(np.asarray(C_tile, dtype=np.int64) + A @ Bfull)


def gemm_amx(A, B):
    A = np.asarray(A, dtype=np.int64)
    B = np.asarray(B, dtype=np.int64)
    M, K = A.shape
    _, N = B.shape
    assert M % 16 == 0 and N % 16 == 0 and K % 64 == 0
    C = np.zeros((M, N), dtype=np.int64)
    for i0 in range(0, M, 16):
        for j0 in range(0, N, 16):
            tile = np.zeros((16, 16), dtype=np.int64)
            for k in range(0, K, 64):
                a_tile = A[i0:i0 + 16, k:k + 64]
                b_blk = B[k:k + 64, j0:j0 + 16]                        # 64 x 16
                b_tile = b_blk.reshape(16, 4, 16).transpose(0, 2, 1)   # [group][column][t]
                tile = tile_dpbssd(tile, a_tile, b_tile)
            C[i0:i0 + 16, j0:j0 + 16] = tile
    return C


# --------------------------------------------------------------------------- Section 6.3 (ARM SME)
def smopa(ZA, Zn, Zm, dim):
    """ZA(dim x dim int32) += sum of four int8 outer products: Zn and Zm each hold `dim` groups of
    four int8 values; ZA[i][j] += sum_{t<4} Zn[4i+t] * Zm[4j+t]."""
    zn = np.asarray(Zn, dtype=np.int64).reshape(dim, 4)
    zm = np.asarray(Zm, dtype=np.int64).reshape(dim, 4)
    return _wrap32(np.asarray(ZA, dtype=np.int64) + zn @ zm.T)


def gemm_sme(A, B, dim=4):
    A = np.asarray(A, dtype=np.int64)
    B = np.asarray(B, dtype=np.int64)
    M, K = A.shape
    _, N = B.shape
    assert M % dim == 0 and N % dim == 0 and K % 4 == 0
    C = np.zeros((M, N), dtype=np.int64)
    for i0 in range(0, M, dim):
        for j0 in range(0, N, dim):
            za = np.zeros((dim, dim), dtype=np.int64)
            for k in range(0, K, 4):
                za = smopa(za, A[i0:i0 + dim, k:k + 4].reshape(-1), B[k:k + 4, j0:j0 + dim].T.reshape(-1), dim)
            C[i0:i0 + dim, j0:j0 + dim] = za
    return C
