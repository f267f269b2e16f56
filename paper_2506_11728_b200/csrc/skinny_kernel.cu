// Skinny-M MIP GEMM (1 <= M <= 16): C[i][j] = sum_k A[i][k] * B[j][k].
//
// This is the matrix-vector end of the method (the paper's fully connected layer at
// batch 1, "2mn useful operations"): the weight matrix B is streamed from HBM exactly
// once and everything else is noise, so the kernel is built around 16-byte streaming
// loads, not around the tensor-memory pipeline.
//
// A CTA owns 16 consecutive weight rows (columns j of C).  Its warps take 128-byte
// slices of K round-robin; for each slice a warp multiplies the 16x128 weight block by
// the M tokens with four warp-level m16n8k32 integer MMAs per group of 8 tokens (weights
// are the 16-row operand, tokens the 8-column operand, so the accumulator fragment is a
// 16x8 piece of C transposed).  The k positions are permuted identically for both
// operands -- integer sums do not depend on the order -- so that every thread loads 16
// contiguous bytes.  Warp partials are added through shared memory; nothing is ever
// waited on across CTAs and no global scratch memory is used.
#include "internal.h"
#include "ptx.cuh"

namespace mip {

template <bool kUnsignedTokens>
__device__ __forceinline__ void mma_16x8x32(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                            uint32_t a3, uint32_t b0, uint32_t b1) {
    if (kUnsignedTokens)
        asm volatile(
            "mma.sync.aligned.m16n8k32.row.col.s32.s8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
            "{%0,%1,%2,%3};"
            : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    else
        asm volatile(
            "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
            "{%0,%1,%2,%3};"
            : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pick(const uint4& v, int q) {
    return q == 0 ? v.x : (q == 1 ? v.y : (q == 2 ? v.z : v.w));
}

constexpr int kSkinnyWarps = 8;

template <bool kUnsignedTokens, bool kSecondTokenBlock>
__global__ void __launch_bounds__(kSkinnyWarps * 32)
mip_skinny_kernel(const SkinnyParams p) {
    __shared__ int red[kSkinnyWarps][16][17];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const long long n0 = static_cast<long long>(blockIdx.x) * 16;

    const long long row_lo = min(n0 + g, static_cast<long long>(p.N) - 1);
    const long long row_hi = min(n0 + g + 8, static_cast<long long>(p.N) - 1);
    const int8_t* b_lo = p.B + row_lo * p.ldb;
    const int8_t* b_hi = p.B + row_hi * p.ldb;
    const uint8_t* A = static_cast<const uint8_t*>(p.A);
    const bool tok0_ok = g < p.M;
    const bool tok1_ok = kSecondTokenBlock && (g + 8 < p.M);
    const uint8_t* x0 = A + static_cast<long long>(tok0_ok ? g : 0) * p.lda;
    const uint8_t* x1 = A + static_cast<long long>(tok1_ok ? g + 8 : 0) * p.lda;

    int acc0[4] = {0, 0, 0, 0};
    int acc1[4] = {0, 0, 0, 0};
    const int n_slices = (p.K + 127) >> 7;
    const uint4 zero = make_uint4(0, 0, 0, 0);

#pragma unroll 2
    for (int c = warp; c < n_slices; c += kSkinnyWarps) {
        const int k_lo = (c << 7) + (t << 4);
        const int k_hi = k_lo + 64;
        const bool v_lo = k_lo < p.K, v_hi = k_hi < p.K;   // K % 16 == 0: a piece is whole or absent
        const uint4 w_ll = v_lo ? ld_stream_v4(b_lo + k_lo) : zero;
        const uint4 w_hl = v_lo ? ld_stream_v4(b_hi + k_lo) : zero;
        const uint4 w_lh = v_hi ? ld_stream_v4(b_lo + k_hi) : zero;
        const uint4 w_hh = v_hi ? ld_stream_v4(b_hi + k_hi) : zero;
        const uint4 x0l = (v_lo && tok0_ok) ? __ldg(reinterpret_cast<const uint4*>(x0 + k_lo)) : zero;
        const uint4 x0h = (v_hi && tok0_ok) ? __ldg(reinterpret_cast<const uint4*>(x0 + k_hi)) : zero;
        uint4 x1l = zero, x1h = zero;
        if (kSecondTokenBlock) {
            x1l = (v_lo && tok1_ok) ? __ldg(reinterpret_cast<const uint4*>(x1 + k_lo)) : zero;
            x1h = (v_hi && tok1_ok) ? __ldg(reinterpret_cast<const uint4*>(x1 + k_hi)) : zero;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            mma_16x8x32<kUnsignedTokens>(acc0, pick(w_ll, q), pick(w_hl, q), pick(w_lh, q), pick(w_hh, q),
                                         pick(x0l, q), pick(x0h, q));
            if (kSecondTokenBlock)
                mma_16x8x32<kUnsignedTokens>(acc1, pick(w_ll, q), pick(w_hl, q), pick(w_lh, q),
                                             pick(w_hh, q), pick(x1l, q), pick(x1h, q));
        }
    }

    // accumulator fragment: d0 (row g, col 2t), d1 (g, 2t+1), d2 (g+8, 2t), d3 (g+8, 2t+1);
    // row = weight row inside the CTA's 16, col = token.
    red[warp][g][2 * t] = acc0[0];
    red[warp][g][2 * t + 1] = acc0[1];
    red[warp][g + 8][2 * t] = acc0[2];
    red[warp][g + 8][2 * t + 1] = acc0[3];
    if (kSecondTokenBlock) {
        red[warp][g][8 + 2 * t] = acc1[0];
        red[warp][g][8 + 2 * t + 1] = acc1[1];
        red[warp][g + 8][8 + 2 * t] = acc1[2];
        red[warp][g + 8][8 + 2 * t + 1] = acc1[3];
    }
    __syncthreads();
    const int tok = threadIdx.x >> 4, n = threadIdx.x & 15;
    if (tok < p.M && (kSecondTokenBlock || tok < 8) && n0 + n < p.N) {
        int sum = 0;
#pragma unroll
        for (int w = 0; w < kSkinnyWarps; ++w) sum += red[w][n][tok];
        int32_t* dst = p.C + static_cast<long long>(tok) * p.ldc + n0 + n;
        if (p.accumulate) sum = static_cast<int>(static_cast<uint32_t>(sum) + static_cast<uint32_t>(*dst));
        *dst = sum;
    }
}

bool skinny_supported(const SkinnyParams& p) {
    if (p.M < 1 || p.M > 16 || p.N < 1 || p.K < 16) return false;
    if (p.K % 16 != 0 || p.lda % 16 != 0 || p.ldb % 16 != 0) return false;
    if (reinterpret_cast<uintptr_t>(p.A) % 16 != 0 || reinterpret_cast<uintptr_t>(p.B) % 16 != 0) return false;
    return true;
}

cudaError_t launch_skinny(const SkinnyParams& p, cudaStream_t stream) {
    const unsigned grid = static_cast<unsigned>((static_cast<long long>(p.N) + 15) / 16);
    const int threads = kSkinnyWarps * 32;
    const bool two = p.M > 8;
    if (p.a_unsigned) {
        if (two) mip_skinny_kernel<true, true><<<grid, threads, 0, stream>>>(p);
        else     mip_skinny_kernel<true, false><<<grid, threads, 0, stream>>>(p);
    } else {
        if (two) mip_skinny_kernel<false, true><<<grid, threads, 0, stream>>>(p);
        else     mip_skinny_kernel<false, false><<<grid, threads, 0, stream>>>(p);
    }
    return cudaGetLastError();
}

}  // namespace mip
