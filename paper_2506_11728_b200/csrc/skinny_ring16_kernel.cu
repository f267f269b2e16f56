// Skinny-M MIP GEMM, ring form for 9 to 16 tokens.
//
// With up to eight tokens the ring kernel (skinny_ring_kernel.cu) keeps all tokens in shared memory beside
// its ring of weight chunks.  Sixteen tokens of K = 4096 bytes are 64 KB: beside them only two 16 KB ring
// slots fit in half an SM, too few bytes in flight to keep the weight stream going (measured: 30 % slower
// per launch than eight tokens), and with K = 11008 they do not fit at all.  This kernel therefore walks its
// share of the weight matrix chunk-major instead of unit-major:
//
//   for every group of up to kMaxU work units (16 weight rows each) of this CTA
//     for every 1 KB k-chunk
//       the tokens' bytes of that k-chunk (16 x 1 KB, one of two buffers)
//       for every unit of the group: its 16 x 1 KB weight chunk from the ring  ->  MMAs
//     reduce the eight warps' partial sums of the group's units and store them
//
// so only 2 x 16 KB of tokens are resident, four ring slots fit beside them with two CTAs per SM, and the
// accumulators of the group's units live in registers.  Warps 0-7 consume (warp w owns the w-th 128-byte
// k-slice of every chunk, as in the other ring kernel), warp 8 streams the weights, warp 9 the token chunks;
// under the constant-weights promise only warp 8 runs ahead of the previous kernel's completion.  A unit is
// never split across CTAs: no scratch, no atomics on global memory, no inter-CTA wait.  Every barrier wait is
// bounded and reports through the device status word.
#include "internal.h"
#include "ptx.cuh"

namespace mip {

namespace {

constexpr int kSlots16Max = 8;
constexpr int kSlotBytes = 16 * 1024;          // 8 slices x 16 rows x 128 B
constexpr int kConsumers = 8;
constexpr int kThreads16 = (kConsumers + 2) * 32;
constexpr int kMaxU = 3;                       // units whose accumulators the consumers hold at once
constexpr int kTokRowBytes = 1024 + 16;        // pitch of a token row inside a token buffer (spreads the banks)
constexpr int kTokBufBytes = 16 * kTokRowBytes;
constexpr int kOutBytes = 4096;                // int32 [kMaxU][16 tokens][16 weight rows], padded
constexpr int kCtrlBytes16 = 256;

template <bool kUnsignedTokens>
__device__ __forceinline__ void mma16(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                      uint32_t b1) {
    if (kUnsignedTokens)
        asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    else
        asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t wd(const uint4& v, int q) {
    return q == 0 ? v.x : (q == 1 ? v.y : (q == 2 ? v.z : v.w));
}

__device__ __forceinline__ uint4 lds16(uint32_t addr) {
    uint4 r;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr) : "memory");
    return r;
}

template <bool kUnsignedTokens>
__global__ void __launch_bounds__(kThreads16, 2)
mip_skinny_ring16_kernel(const __grid_constant__ SkinnyRingParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = ((raw_addr + 1023u) & ~1023u) - raw_addr;
    uint8_t* smem = smem_raw + pad;
    const uint32_t ring = raw_addr + pad;
    // shared memory: [slots x 16 KB ring] [group sums] [barriers, abort word] [two token buffers]
    const int slots = p.slots;
    int* out = reinterpret_cast<int*>(smem + slots * kSlotBytes);
    const uint32_t ctrl = ring + slots * kSlotBytes + kOutBytes;
    const uint32_t bar_full = ctrl, bar_empty = ctrl + 8u * kSlots16Max;
    const uint32_t bar_tfull = ctrl + 16u * kSlots16Max, bar_tempty = bar_tfull + 16u;
    volatile uint32_t* abort_flag =
        reinterpret_cast<volatile uint32_t*>(smem + slots * kSlotBytes + kOutBytes + 16 * kSlots16Max + 32);
    const uint32_t tokbuf = ctrl + kCtrlBytes16;

    const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < slots; ++s) {
            mbar_init(bar_full + 8u * s, 1);
            mbar_init(bar_empty + 8u * s, kConsumers);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_tfull + 8u * b, 1);
            mbar_init(bar_tempty + 8u * b, kConsumers);
        }
        *abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&p.tmap_b);
    }
    if (threadIdx.x < 256)
        for (int i = threadIdx.x; i < kMaxU * 256; i += 256) out[i] = 0;
    // Everything above touched only shared memory and kernel parameters and may overlap the tail of the previous
    // kernel in the stream.  From here on every thread that touches global memory first waits for that kernel to
    // complete -- except the weight producer when the caller has promised constant weights.
    __syncthreads();
    if (p.pdl_mode == 1) pdl_launch_dependents();
    const int units = (p.N + 15) >> 4;
    const int chunks = (p.K + 1023) >> 10;
    const int my_units = (units - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
    const uint64_t budget = p.wait_budget_ns;
    // (B is not read before the previous kernel has completed unless the caller promised constant weights, but
    // the L2 may be asked to fetch the first chunks: a prefetch brings no data to the SM and the L2 stays coherent)
    if (p.pdl_mode == 1 && !p.b_constant && warp == kConsumers && elect_one()) {
        int asked = 0;
        const int n_u = min(kMaxU, my_units);
        for (int ch = 0; ch < chunks && asked < p.prefetch_chunks; ++ch)
            for (int j = 0; j < n_u && asked < p.prefetch_chunks; ++j, ++asked)
                tma_prefetch_l2_3d(&p.tmap_b, 0, (static_cast<int>(blockIdx.x) + j * static_cast<int>(gridDim.x)) * 16, ch * 8);
    }
    if (!(p.b_constant && warp == kConsumers)) pdl_wait();

    if (warp == kConsumers) {
        // ------------------------------------------------------------ weight producer
        uint32_t s = 0, phase = 0;
        bool ok = true;
        for (int g0 = 0; g0 < my_units && ok; g0 += kMaxU) {
            const int n_u = min(kMaxU, my_units - g0);
            for (int ch = 0; ch < chunks && ok; ++ch) {
                for (int j = 0; j < n_u; ++j) {
                    const int u = static_cast<int>(blockIdx.x) + (g0 + j) * static_cast<int>(gridDim.x);
                    if (!mbar_wait(bar_empty + 8u * s, phase ^ 1u, abort_flag, budget)) { ok = false; break; }
                    // (test hook, bit 0: CTA 0 leaves out the second chunk of its first unit)
                    const bool withheld = (p.debug_flags & 1) && blockIdx.x == 0 && g0 == 0 && j == 0 && ch == 1;
                    if (elect_one() && !withheld) {
                        mbar_arrive_expect_tx(bar_full + 8u * s, kSlotBytes);
                        tma_load_3d(ring + s * kSlotBytes, &p.tmap_b, bar_full + 8u * s, 0, u * 16, ch * 8);
                    }
                    if (++s == static_cast<uint32_t>(slots)) { s = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == kConsumers + 1) {
        // ------------------------------------------------------------ token producer: one 1 KB k-chunk of every token
        const uint8_t* A = static_cast<const uint8_t*>(p.A);
        uint32_t t = 0;
        bool ok = true;
        for (int g0 = 0; g0 < my_units && ok; g0 += kMaxU) {
            for (int ch = 0; ch < chunks; ++ch, ++t) {
                const uint32_t b = t & 1u;
                if (!mbar_wait(bar_tempty + 8u * b, ((t >> 1) & 1u) ^ 1u, abort_flag, budget)) { ok = false; break; }
                const uint32_t bytes = static_cast<uint32_t>(min(1024, p.K - ch * 1024));
                if (lane == 0) mbar_arrive_expect_tx(bar_tfull + 8u * b, static_cast<uint32_t>(p.M) * bytes);
                __syncwarp();
                if (lane < p.M)
                    bulk_load_1d(tokbuf + b * kTokBufBytes + lane * kTokRowBytes,
                                 A + static_cast<long long>(lane) * p.lda + ch * 1024, bytes, bar_tfull + 8u * b);
            }
        }
    } else {
        // ------------------------------------------------------------ consumers
        const int g = lane >> 2, t4 = lane & 3;
        // this thread's four 16-byte pieces inside a slice: rows g and g+8, chunks t and t+4, swizzled
        const uint32_t off_ll = static_cast<uint32_t>(warp) * 2048u + g * 128u + ((t4 ^ g) << 4);
        const uint32_t off_lh = static_cast<uint32_t>(warp) * 2048u + g * 128u + (((t4 + 4) ^ g) << 4);
        const uint32_t off_hl = off_ll + 1024u;     // row g + 8: same swizzle phase
        const uint32_t off_hh = off_lh + 1024u;
        // tokens g and g + 8, this warp's 128-byte k-slice of the chunk, bytes t*16.. and 64 + t*16..
        const uint32_t tok_lo = static_cast<uint32_t>(g) * kTokRowBytes + static_cast<uint32_t>(warp) * 128u + (t4 << 4);
        const uint32_t tok_hi = tok_lo + 8u * kTokRowBytes;
        const int tok = (threadIdx.x >> 4), n = threadIdx.x & 15;    // the C cell this thread finalises

        uint32_t s = 0, phase = 0, t = 0;
        const int my_chunks = my_units * chunks;
        const uint32_t total_tok = static_cast<uint32_t>(((my_units + kMaxU - 1) / kMaxU) * chunks);   // token chunks in all
        int chunk_no = 0;
        bool ok = true;
        for (int g0 = 0; g0 < my_units; g0 += kMaxU) {
            const int n_u = min(kMaxU, my_units - g0);
            int acc[kMaxU][2][4];
#pragma unroll
            for (int j = 0; j < kMaxU; ++j)
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[j][h][e] = 0;
            for (int ch = 0; ch < chunks && ok; ++ch, ++t) {
                const uint32_t b = t & 1u;
                if (!mbar_wait(bar_tfull + 8u * b, (t >> 1) & 1u, abort_flag, budget)) { ok = false; break; }
                const uint32_t tb = tokbuf + b * kTokBufBytes;
                const uint4 x0l = lds16(tb + tok_lo), x0h = lds16(tb + tok_lo + 64u);
                const uint4 x1l = lds16(tb + tok_hi), x1h = lds16(tb + tok_hi + 64u);
                // (the refill of a buffer is an asynchronous-proxy write to bytes these generic-proxy loads read:
                // the loads must have been performed before the producer is told, hence the proxy fence)
                if (t + 2 < total_tok) {                  // this buffer will be refilled
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_tempty + 8u * b);
                }
#pragma unroll
                for (int j = 0; j < kMaxU; ++j) {
                    if (j < n_u && ok) {
                        if (!mbar_wait(bar_full + 8u * s, phase, abort_flag, budget)) {
                            ok = false;
                        } else {
                            const uint32_t base = ring + s * kSlotBytes;
                            const uint4 w_ll = lds16(base + off_ll), w_hl = lds16(base + off_hl);
                            const uint4 w_lh = lds16(base + off_lh), w_hh = lds16(base + off_hh);
                            if (chunk_no + slots < my_chunks) {          // this slot will be refilled
                                fence_proxy_async_smem();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(bar_empty + 8u * s);
                            }
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                mma16<kUnsignedTokens>(acc[j][0], wd(w_ll, q), wd(w_hl, q), wd(w_lh, q), wd(w_hh, q),
                                                       wd(x0l, q), wd(x0h, q));
                                mma16<kUnsignedTokens>(acc[j][1], wd(w_ll, q), wd(w_hl, q), wd(w_lh, q), wd(w_hh, q),
                                                       wd(x1l, q), wd(x1h, q));
                            }
                            ++chunk_no;
                            if (++s == static_cast<uint32_t>(slots)) { s = 0; phase ^= 1u; }
                        }
                    }
                }
            }
            // Partial sums of the eight warps meet in shared memory (integer adds: exact in any order).
            // accumulator fragment: d0 (row g, col 2t), d1 (g, 2t+1), d2 (g+8, 2t), d3 (g+8, 2t+1); row = weight row of
            // the unit, col = token (second accumulator: tokens 8..15)
#pragma unroll
            for (int j = 0; j < kMaxU; ++j) {
                if (j < n_u) {
                    int* o = out + j * 256;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        atomicAdd(&o[(8 * h + 2 * t4) * 16 + g], acc[j][h][0]);
                        atomicAdd(&o[(8 * h + 2 * t4 + 1) * 16 + g], acc[j][h][1]);
                        atomicAdd(&o[(8 * h + 2 * t4) * 16 + g + 8], acc[j][h][2]);
                        atomicAdd(&o[(8 * h + 2 * t4 + 1) * 16 + g + 8], acc[j][h][3]);
                    }
                }
            }
            // every consumer thread waits on its own clock, but the warps meet here: leaving is decided together
            if (named_bar_or(1, 256, !ok)) { ok = false; break; }
            for (int j = 0; j < n_u; ++j) {
                const int u = static_cast<int>(blockIdx.x) + (g0 + j) * static_cast<int>(gridDim.x);
                const long long col = static_cast<long long>(u) * 16 + n;
                int sum = out[j * 256 + tok * 16 + n];
                out[j * 256 + tok * 16 + n] = 0;
                if (tok < p.M && col < p.N) {
                    int32_t* dst = p.C + static_cast<long long>(tok) * p.ldc + col;
                    if (p.accumulate) sum = static_cast<int>(static_cast<uint32_t>(sum) + static_cast<uint32_t>(*dst));
                    if (p.out_f32) sum = __float_as_int(__int2float_rn(sum) * p.out_scale);   // fused dequantisation
                    *dst = sum;
                }
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");           // the group sums are zero again
        }
        if (!ok) {
            // Unwinding: whatever the producers may have requested must land before the CTA exits; wait
            // (bounded) on every barrier that can still be pending.
            for (uint32_t i = 0; i < 2; ++i) {
                const uint32_t ti = t + i;
                const uint64_t t0 = globaltimer_ns();
                while (!mbar_try_wait(bar_tfull + 8u * (ti & 1u), (ti >> 1) & 1u)) {
                    if (globaltimer_ns() - t0 > 2000000ull) break;
                }
            }
            for (int i = 0; i < slots; ++i) {
                const uint64_t t0 = globaltimer_ns();
                const uint32_t si = s + i;
                while (!mbar_try_wait(bar_full + 8u * (si % slots), (si >= static_cast<uint32_t>(slots)) ? phase ^ 1u : phase)) {
                    if (globaltimer_ns() - t0 > 2000000ull) break;
                }
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag != 0) atomicOr(p.status, 1u);
}

constexpr int kFixed16 = kOutBytes + kCtrlBytes16 + 2 * kTokBufBytes + 1024;

template <bool kU>
cudaError_t launch16_t(SkinnyRingParams p, int sm_count, cudaStream_t stream) {
    // two CTAs per SM, each with half of its shared memory
    const int budget = 228 * 1024 / 2 - 2048;
    int slots = (budget - kFixed16) / kSlotBytes;
    if (slots > kSlots16Max) slots = kSlots16Max;
    p.slots = slots;
    p.tokens_in_smem = 1;
    p.pdl_mode = 1;
    const int units = (p.N + 15) / 16;
    const int grid = units < 2 * sm_count ? units : 2 * sm_count;
    const size_t smem = static_cast<size_t>(slots) * kSlotBytes + kFixed16;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
    cfg.blockDim = dim3(kThreads16, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl_allowed();
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, mip_skinny_ring16_kernel<kU>, p);
}

}  // namespace

cudaError_t skinny_ring16_init() {
    cudaError_t e = cudaFuncSetAttribute(mip_skinny_ring16_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         228 * 1024 / 2);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(mip_skinny_ring16_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 228 * 1024 / 2);
}

// 9 to 16 tokens, K a multiple of 128, 16-byte aligned operands, enough 16-row units that every SM streams.
bool skinny_ring16_supported(const SkinnyParams& p, int sm_count) {
    if (p.M <= 8 || p.M > 16 || !skinny_supported(p)) return false;
    if (p.K % 128 != 0) return false;
    return (static_cast<long long>(p.N) + 15) / 16 >= sm_count;
}

cudaError_t launch_skinny_ring16(const SkinnyRingParams& p, int sm_count, cudaStream_t stream) {
    return p.a_unsigned ? launch16_t<true>(p, sm_count, stream) : launch16_t<false>(p, sm_count, stream);
}

}  // namespace mip
