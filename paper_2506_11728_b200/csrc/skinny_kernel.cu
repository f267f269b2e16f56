// Skinny-M MIP GEMM (1 <= M <= 16): C[i][j] = sum_k A[i][k] * B[j][k].
//
// This is the matrix-vector end of the method (the paper's fully connected layer at
// batch 1, "2mn useful operations"): the weight matrix B is streamed from HBM exactly
// once and everything else is noise, so the kernel is built around keeping as many
// 16-byte streaming loads in flight as the machine allows, not around tensor memory.
//
// Work decomposition: a cluster of S CTAs (S = 1 unless N is so small that the grid would
// leave SMs idle; then 2, 4 or 8) owns 16 consecutive weight rows (columns j of C); CTA r
// of the cluster takes the r-th share of K, and its eight warps take 128-byte slices of
// that share round-robin; with 32 resident warps per SM about 9 MB are in flight chip-wide.
// For each slice a warp multiplies the 16 x 128 weight block by the M tokens with four
// warp-level m16n8k32 integer MMAs per group of 8 tokens (weights are the 16-row operand,
// tokens the 8-column operand, so the accumulator fragment is a 16 x 8 piece of C
// transposed).  The k positions are permuted identically for both operands -- integer
// sums do not depend on the order -- so that every thread loads 16 contiguous bytes.
// Warp partials are added through shared memory, CTA partials through distributed shared
// memory into cluster rank 0, which writes C.  No global scratch, no atomics, and nothing
// is ever waited on except the cluster barrier that every CTA reaches unconditionally.
#include "internal.h"
#include "ptx.cuh"

namespace mip {

template <bool kUnsignedTokens>
__device__ __forceinline__ void mma_16x8x32(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                            uint32_t a3, uint32_t b0, uint32_t b1) {
    if (kUnsignedTokens)
        asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
            "{%0,%1,%2,%3};"
            : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    else
        asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
            "{%0,%1,%2,%3};"
            : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pick(const uint4& v, int q) {
    return q == 0 ? v.x : (q == 1 ? v.y : (q == 2 ? v.z : v.w));
}

// 16-byte read-once load; not `volatile`, so the compiler may hoist it above the MMAs of
// the previous slice.
__device__ __forceinline__ uint4 ld_weights(const void* p, bool valid) {
    uint4 r = make_uint4(0, 0, 0, 0);
    if (valid)
        asm("ld.global.nc.L1::no_allocate.v4.b32 {%0, %1, %2, %3}, [%4];"
            : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ uint4 ld_tokens(const void* p, bool valid) {
    uint4 r = make_uint4(0, 0, 0, 0);
    if (valid)
        asm("ld.global.nc.v4.b32 {%0, %1, %2, %3}, [%4];"
            : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

constexpr int kSkinnyWarps = 8;
constexpr int kSkinnyMaxSplit = 8;

// Operands of one 16-row x 128-byte slice as one thread holds them.
struct SliceRegs {
    uint4 w_ll, w_hl, w_lh, w_hh;   // weights: (row g | g+8) x (k low | k high half)
    uint4 x0l, x0h, x1l, x1h;       // tokens g and g+8
};

template <bool kSecondTokenBlock>
__device__ __forceinline__ void load_slice(SliceRegs& s, int c, int n_slices, int K, int t,
                                           const int8_t* b_lo, const int8_t* b_hi,
                                           const uint8_t* x0, const uint8_t* x1, bool tok0_ok, bool tok1_ok) {
    const int k_lo = (c << 7) + (t << 4);
    const int k_hi = k_lo + 64;
    const bool in = c < n_slices;
    const bool v_lo = in && k_lo < K, v_hi = in && k_hi < K;   // K % 16 == 0: a piece is whole or absent
    s.w_ll = ld_weights(b_lo + k_lo, v_lo);
    s.w_hl = ld_weights(b_hi + k_lo, v_lo);
    s.w_lh = ld_weights(b_lo + k_hi, v_hi);
    s.w_hh = ld_weights(b_hi + k_hi, v_hi);
    s.x0l = ld_tokens(x0 + k_lo, v_lo && tok0_ok);
    s.x0h = ld_tokens(x0 + k_hi, v_hi && tok0_ok);
    if (kSecondTokenBlock) {
        s.x1l = ld_tokens(x1 + k_lo, v_lo && tok1_ok);
        s.x1h = ld_tokens(x1 + k_hi, v_hi && tok1_ok);
    }
}

template <bool kUnsignedTokens, bool kSecondTokenBlock>
__device__ __forceinline__ void mma_slice(const SliceRegs& s, int (&acc0)[4], int (&acc1)[4]) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        mma_16x8x32<kUnsignedTokens>(acc0, pick(s.w_ll, q), pick(s.w_hl, q), pick(s.w_lh, q), pick(s.w_hh, q),
                                     pick(s.x0l, q), pick(s.x0h, q));
        if (kSecondTokenBlock)
            mma_16x8x32<kUnsignedTokens>(acc1, pick(s.w_ll, q), pick(s.w_hl, q), pick(s.w_lh, q),
                                         pick(s.w_hh, q), pick(s.x1l, q), pick(s.x1h, q));
    }
}

#ifndef MIP_SKINNY_DEPTH
#define MIP_SKINNY_DEPTH 1
#endif

// Occupancy matters more than depth here (measured: deeper register rings lose more to
// spills and wave quantisation than they gain): the grid is many small CTAs so that the
// tail is smooth, and registers are capped so that 4 CTAs (M <= 8) share an SM.
template <bool kUnsignedTokens, bool kSecondTokenBlock>
__global__ void __launch_bounds__(kSkinnyWarps * 32, kSecondTokenBlock ? 3 : 4)
mip_skinny_kernel(const SkinnyParams p, int split) {
    constexpr int kDepth = MIP_SKINNY_DEPTH;   // slices in flight per warp
    __shared__ int red[kSkinnyWarps][16][17];        // per-warp partials [weight row][token]
    __shared__ int gather[kSkinnyMaxSplit][256];     // rank 0 only: per-CTA partials of the cluster
    pdl_wait();                // (programmatic dependent launch: see ptx.cuh)
    pdl_launch_dependents();   // released only now: at most two kernels of a chain are in flight
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const uint32_t rank = split > 1 ? cluster_ctarank() : 0u;
    const long long n0 = static_cast<long long>(blockIdx.x / split) * 16;

    const long long row_lo = min(n0 + g, static_cast<long long>(p.N) - 1);
    const long long row_hi = min(n0 + g + 8, static_cast<long long>(p.N) - 1);
    const int8_t* b_lo = p.B + row_lo * p.ldb;
    const int8_t* b_hi = p.B + row_hi * p.ldb;
    const uint8_t* A = static_cast<const uint8_t*>(p.A);
    const bool tok0_ok = g < p.M;
    const bool tok1_ok = kSecondTokenBlock && (g + 8 < p.M);
    const uint8_t* x0 = A + static_cast<long long>(tok0_ok ? g : 0) * p.lda;
    const uint8_t* x1 = A + static_cast<long long>(tok1_ok ? g + 8 : 0) * p.lda;

    // this CTA's share of the 128-byte slices of K
    const int n_slices_total = (p.K + 127) >> 7;
    const int per_cta = (n_slices_total + split - 1) / split;
    const int first = static_cast<int>(rank) * per_cta;
    const int n_slices = min(n_slices_total, first + per_cta);

    int acc0[4] = {0, 0, 0, 0};
    int acc1[4] = {0, 0, 0, 0};
    SliceRegs ring[kDepth];
    int c = first + warp;
#pragma unroll
    for (int d = 0; d < kDepth; ++d)
        load_slice<kSecondTokenBlock>(ring[d], c + d * kSkinnyWarps, n_slices, p.K, t, b_lo, b_hi, x0, x1,
                                      tok0_ok, tok1_ok);
#pragma unroll 1
    while (c < n_slices) {
#pragma unroll
        for (int d = 0; d < kDepth; ++d) {
            // absent slices were loaded as zeros and add nothing
            mma_slice<kUnsignedTokens, kSecondTokenBlock>(ring[d], acc0, acc1);
            load_slice<kSecondTokenBlock>(ring[d], c + (d + kDepth) * kSkinnyWarps, n_slices, p.K, t, b_lo, b_hi,
                                          x0, x1, tok0_ok, tok1_ok);
        }
        c += kDepth * kSkinnyWarps;
    }

    // accumulator fragment: d0 (row g, col 2t), d1 (g, 2t+1), d2 (g+8, 2t), d3 (g+8, 2t+1);
    // row = weight row inside the cluster's 16, col = token.
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

    // thread e owns the cell (token e / 16, weight row e % 16)
    const int tok = threadIdx.x >> 4, n = threadIdx.x & 15;
    int sum = 0;
    if (kSecondTokenBlock || tok < 8) {
#pragma unroll
        for (int w = 0; w < kSkinnyWarps; ++w) sum += red[w][n][tok];
    }
    if (split > 1) {
        // CTA partials meet in rank 0's shared memory (distributed shared memory stores)
        const uint32_t base = mapa_u32(smem_u32(&gather[rank][0]), 0);
        asm volatile("st.shared::cluster.b32 [%0], %1;" ::"r"(base + 4u * threadIdx.x), "r"(sum) : "memory");
        cluster_arrive();
        cluster_wait();
        if (rank != 0) return;
        sum = 0;
        for (int r = 0; r < split; ++r) sum += gather[r][threadIdx.x];
    }
    if (tok < p.M && n0 + n < p.N) {
        int32_t* dst = p.C + static_cast<long long>(tok) * p.ldc + n0 + n;
        if (p.accumulate) sum = static_cast<int>(static_cast<uint32_t>(sum) + static_cast<uint32_t>(*dst));
        if (p.out_f32) sum = __float_as_int(__int2float_rn(sum) * p.out_scale);   // fused dequantisation
        *dst = sum;
    }
}

bool skinny_supported(const SkinnyParams& p) {
    if (p.M < 1 || p.M > 16 || p.N < 1 || p.K < 16) return false;
    if (p.K % 16 != 0 || p.lda % 16 != 0 || p.ldb % 16 != 0) return false;
    if (reinterpret_cast<uintptr_t>(p.A) % 16 != 0 || reinterpret_cast<uintptr_t>(p.B) % 16 != 0) return false;
    if ((static_cast<long long>(p.N) + 15) / 16 * kSkinnyMaxSplit > 0x7FFFFFFFLL) return false;
    return true;
}

// K is split over a cluster only when the 16-row groups alone would leave SMs without a CTA,
// and never so far that a warp gets less than two slices.
static int choose_split(const SkinnyParams& p, int sm_count) {
    const long long groups = (static_cast<long long>(p.N) + 15) / 16;
    const int n_slices = (p.K + 127) >> 7;
    int split = 1;
    while (split < kSkinnyMaxSplit && groups * split < sm_count && n_slices / (split * 2) >= 2 * kSkinnyWarps)
        split *= 2;
    return split;
}

template <bool kU, bool kTwo>
static cudaError_t launch_skinny_t(const SkinnyParams& p, int split, cudaStream_t stream) {
    const unsigned groups = static_cast<unsigned>((static_cast<long long>(p.N) + 15) / 16);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(groups * split, 1, 1);
    cfg.blockDim = dim3(kSkinnyWarps * 32, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(split);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // (measured: these many-CTA streaming kernels gain nothing from an early launch of their successor and
    // lose 3-4 % in CUDA-graph chains, so the attribute stays off; the in-kernel instructions are then no-ops)
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 0;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, mip_skinny_kernel<kU, kTwo>, p, split);
}

cudaError_t launch_skinny(const SkinnyParams& p, cudaStream_t stream) {
    static int sm_count = 0;
    if (sm_count == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            sm_count = 148;
    }
    const int split = choose_split(p, sm_count);
    const bool two = p.M > 8;
    if (p.a_unsigned) return two ? launch_skinny_t<true, true>(p, split, stream) : launch_skinny_t<true, false>(p, split, stream);
    return two ? launch_skinny_t<false, true>(p, split, stream) : launch_skinny_t<false, false>(p, split, stream);
}

}  // namespace mip
