"""Pins the primary oracle against the instruction semantics the paper prints.

``oracle/isa_emulation.py`` restates the paper's per-instruction formulas (ARMv8.0 widening
chain, ARMv8.2 4-way dot, SpacemiT K1 vmadot, Intel AMX tile product, ARM SME outer products);
GEMMs assembled from them must equal the exact definition.  The ARMv8.0 chain sums two products
in an int16 lane, so it is exact for weights in [-127, 127] and wraps for all -128 inputs -- the
case BASELINE's "all -128" run is there to separate (the exact definition is what the library
implements)."""
import numpy as np
import pytest

from oracle import isa_emulation as isa
from oracle import mip_oracle as orc
from paper_2506_11728_b200 import inputs


def oracle_gemm(A2, B2):
    """mip_oracle on A (M x K) and B (K x N) given as 2-D arrays."""
    M, K = A2.shape
    _, N = B2.shape
    Bcol = np.ascontiguousarray(B2.T)                    # [N][K]: column-major K x N
    return orc.gemm(np.ascontiguousarray(A2).reshape(-1), Bcol.reshape(-1), M, N, K).reshape(M, N)


def rand_ab(M, N, K, seed, lo=-128):
    A = inputs.uniform_s8(M * K, seed).reshape(M, K)
    B = inputs.uniform_s8(K * N, seed + 1).reshape(K, N)
    if lo > -128:
        A = np.maximum(A, lo)
        B = np.maximum(B, lo)
    return A, B


def test_instruction_formulas_on_hand_values():
    # vmull / vmlal / vpadalq: the lane formulas as printed, on values chosen to hit the int16 edge
    a = np.array([1, -2, 3, -4, 127, -128, -128, 0])
    b = np.array([5, 6, -7, -8, 127, 127, -128, 9])
    m = isa.vmull_s8(a, b)
    assert m.tolist() == [5, -12, -21, 32, 16129, -16256, 16384, 0]
    m2 = isa.vmlal_s8(m, a, b)
    assert m2.tolist() == [10, -24, -42, 64, 32258, -32512, -32768, 0]          # 32768 wraps to -32768
    p = isa.vpadalq_s16(np.array([100, 0, 0, -1]), m2)
    assert p.tolist() == [100 + 10 - 24, -42 + 64, 32258 - 32512, -1 - 32768]
    assert isa.vpaddq_s32([1, 2, 3, 4], [10, 20, 30, 40]).tolist() == [3, 7, 30, 70]
    # vdotq_laneq_s32: lane selects which group of four of v2 multiplies every group of v1
    v1 = np.arange(16) - 8
    v2 = np.arange(16) * 2 - 5
    for lane in range(4):
        want = [int(10 * i + sum(int(v1[4 * i + t]) * int(v2[4 * lane + t]) for t in range(4))) for i in range(4)]
        assert isa.vdotq_laneq_s32([0, 10, 20, 30], v1, v2, lane).tolist() == want


@pytest.mark.parametrize("M,N,K", [(4, 4, 4), (8, 12, 32), (16, 8, 64)])
def test_dot_product_gemm_equals_the_definition(M, N, K):
    A, B = rand_ab(M, N, K, 11)
    assert np.array_equal(isa.gemm_neon_dot(A, B), oracle_gemm(A, B))


@pytest.mark.parametrize("M,N,K", [(4, 4, 8), (8, 8, 24), (12, 4, 64)])
def test_matrix_engine_gemm_equals_the_definition(M, N, K):
    A, B = rand_ab(M, N, K, 21)
    assert np.array_equal(isa.gemm_ime(A, B), oracle_gemm(A, B))


def test_amx_tile_gemm_equals_the_definition():
    A, B = rand_ab(32, 16, 128, 31)
    assert np.array_equal(isa.gemm_amx(A, B), oracle_gemm(A, B))


@pytest.mark.parametrize("dim", [4, 16])
def test_sme_outer_product_gemm_equals_the_definition(dim):
    A, B = rand_ab(dim * 2, dim, 32, 41)
    assert np.array_equal(isa.gemm_sme(A, B, dim), oracle_gemm(A, B))


def test_armv80_chain_is_exact_without_minus_128():
    A, B = rand_ab(6, 5, 64, 51, lo=-127)
    assert np.array_equal(isa.gemm_neon_v80(A, B), oracle_gemm(A, B))


def test_armv80_chain_wraps_on_all_minus_128_and_the_definition_does_not():
    K = 32
    A = np.full((2, K), -128, dtype=np.int8)
    B = np.full((K, 3), -128, dtype=np.int8)
    exact = oracle_gemm(A, B)
    assert (exact == 16384 * K).all()
    wrapped = isa.gemm_neon_v80(A, B)
    # every pair of products (32768) wraps to -32768 in its int16 lane
    assert (wrapped == -16384 * K).all()
    assert not np.array_equal(wrapped, exact)
