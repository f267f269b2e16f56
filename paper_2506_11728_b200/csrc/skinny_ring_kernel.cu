// Skinny-M MIP GEMM, ring form: the weight matrix streams through a deep shared-memory ring
// filled by the TMA, so that far more bytes are in flight per SM than registers could hold.
//
// Persistent CTAs, two per SM with half the shared memory each when at least two ring slots fit
// beside the tokens, else one.  A work unit is 16 consecutive weight rows (columns j of C) over
// the whole of K; it arrives as chunks of 16 rows x 1024 bytes, each one TMA load of a
// rank-3 box {128 B, 16 rows, 8 k-slices} into a 16 KB ring slot (up to 12 slots = 192 KB in
// flight per SM, every slice 128-byte swizzled so the warps' 16-byte reads are conflict-free).  Warp 8
// produces; warps 0-7 consume: warp w multiplies slice w of every chunk by the M tokens with
// warp-level m16n8k32 integer MMAs (weights are the 16-row operand, tokens the 8-column
// operand; k positions permuted identically on both sides so that all accesses are 16 bytes),
// keeping its accumulators in registers across the chunks of a unit; at the end of a unit the
// eight warps add their partials through shared memory and write 16 columns of C.  A unit is
// never split across CTAs, so there is no scratch, no atomics and no inter-CTA wait; every
// barrier wait inside the CTA is bounded and reports through the device status word.
// Requires K % 128 == 0 and 16-byte aligned operands; other shapes use the register form.
#include "internal.h"
#include "ptx.cuh"

namespace mip {

namespace {

#ifdef MIPGEMM_TRACE
// stamps of the first CTA in slots 0.., of the last CTA in slots 16..
#define RING_STAMP(slot) do { if (p.trace && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1) && (threadIdx.x & 31) == 0) \
    p.trace[(blockIdx.x == 0 ? 0 : 16) + (slot)] = globaltimer_ns(); } while (0)
#else
#define RING_STAMP(slot) do { } while (0)
#endif

constexpr int kMaxRingSlots = 12;
constexpr int kSlotBytes = 16 * 1024;          // 8 slices x 16 rows x 128 B
constexpr int kRingConsumers = 8;              // consumer warps = k-slices per chunk
constexpr int kRingThreads = (kRingConsumers + 1) * 32;
constexpr int kRedBytes = 8 * 16 * 17 * 4;
constexpr int kRingCtrlBytes = 256;
constexpr int kRingSmemMax = 227 * 1024;
constexpr int kTokenPad = 64;                  // bytes between token rows beyond K: spreads rows over banks

template <bool kUnsignedTokens>
__device__ __forceinline__ void ring_mma(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
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

__device__ __forceinline__ uint32_t word(const uint4& v, int q) {
    return q == 0 ? v.x : (q == 1 ? v.y : (q == 2 ? v.z : v.w));
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 r;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr) : "memory");
    return r;
}

__device__ __forceinline__ uint4 ldg_tokens(const uint8_t* p, bool valid) {
    uint4 r = make_uint4(0, 0, 0, 0);
    if (valid)
        asm volatile("ld.global.nc.v4.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

struct TokenRegs {
    uint4 x0l, x0h, x1l, x1h;
};

template <bool kSecondTokenBlock>
__device__ __forceinline__ void load_tokens(TokenRegs& r, const uint8_t* x0, const uint8_t* x1, int slice,
                                            int K, int t, bool tok0_ok, bool tok1_ok) {
    const int k_lo = (slice << 7) + (t << 4);
    const bool in = k_lo < K;                       // K % 128 == 0: a slice is whole or absent
    r.x0l = ldg_tokens(x0 + k_lo, in && tok0_ok);
    r.x0h = ldg_tokens(x0 + k_lo + 64, in && tok0_ok);
    if (kSecondTokenBlock) {
        r.x1l = ldg_tokens(x1 + k_lo, in && tok1_ok);
        r.x1h = ldg_tokens(x1 + k_lo + 64, in && tok1_ok);
    }
}

// Same from the shared-memory copy of the tokens (only rows < M exist there).
template <bool kSecondTokenBlock>
__device__ __forceinline__ void load_tokens_smem(TokenRegs& r, uint32_t x0, uint32_t x1, int slice, int K, int t,
                                                 bool tok0_ok, bool tok1_ok) {
    const int k_lo = (slice << 7) + (t << 4);
    const uint4 zero = make_uint4(0, 0, 0, 0);
    const bool in = k_lo < K;
    r.x0l = (in && tok0_ok) ? lds128(x0 + k_lo) : zero;
    r.x0h = (in && tok0_ok) ? lds128(x0 + k_lo + 64) : zero;
    if (kSecondTokenBlock) {
        r.x1l = (in && tok1_ok) ? lds128(x1 + k_lo) : zero;
        r.x1h = (in && tok1_ok) ? lds128(x1 + k_lo + 64) : zero;
    }
}

template <bool kUnsignedTokens, bool kSecondTokenBlock>
__global__ void __launch_bounds__(kRingThreads, 1)
mip_skinny_ring_kernel(const __grid_constant__ SkinnyRingParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = ((raw_addr + 1023u) & ~1023u) - raw_addr;
    uint8_t* smem = smem_raw + pad;
    const uint32_t ring = raw_addr + pad;
    // shared memory: [slots x 16 KB ring] [warp partials] [barriers, abort word] [tokens (optional)]
    const int kRingSlots = p.slots;
    int (*red)[16][17] = reinterpret_cast<int (*)[16][17]>(smem + kRingSlots * kSlotBytes);
    const uint32_t ctrl = ring + kRingSlots * kSlotBytes + kRedBytes;
    const uint32_t bar_full = ctrl, bar_empty = ctrl + 8u * kMaxRingSlots;
    const uint32_t bar_tokens = ctrl + 16u * kMaxRingSlots + 8u;
    volatile uint32_t* abort_flag =
        reinterpret_cast<volatile uint32_t*>(smem + kRingSlots * kSlotBytes + kRedBytes + 16 * kMaxRingSlots);
    const uint32_t tok_base = ctrl + kRingCtrlBytes;
    const int tok_pitch = p.K + kTokenPad;

    const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;
    if (threadIdx.x == 0) RING_STAMP(0);
    if (threadIdx.x == 0) {
        for (int s = 0; s < kRingSlots; ++s) {
            mbar_init(bar_full + 8u * s, 1);
            mbar_init(bar_empty + 8u * s, kRingConsumers);
        }
        mbar_init(bar_tokens, 1);
        *abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&p.tmap_b);
    }
    // Everything above touched only shared memory and kernel parameters, so it may overlap the
    // tail of the previous kernel in the stream.  From here on every thread that touches global
    // memory first waits for that kernel to complete -- except the producer when the caller has
    // promised constant weights: its loads of B then start while the previous kernel drains.
    __syncthreads();
    if (p.pdl_mode == 1) pdl_launch_dependents();
    if (warp == 0) RING_STAMP(1);
    const int units = (p.N + 15) >> 4;
    const int chunks = (p.K + 1023) >> 10;
    const uint64_t budget = p.wait_budget_ns;
    // Without that promise B must not be READ before the previous kernel has completed -- but the L2 may be asked
    // to fetch it: a prefetch brings no data to the SM, and the L2 stays coherent with whatever that kernel still
    // writes.  The producer asks for the first chunks it will stream, so that its loads behind the wait start from
    // the L2 instead of from DRAM.
    // (Under the promise the first chunks go straight to shared memory instead; asking the L2 for the ones behind
    // them as well only gets in the previous kernel's way: +4 to +12 % on the step.)
    if (p.pdl_mode == 1 && !p.b_constant && warp == kRingConsumers && elect_one()) {
        int asked = 0;
        for (int u = blockIdx.x; u < units && asked < p.prefetch_chunks; u += gridDim.x)
            for (int ch = 0; ch < chunks && asked < p.prefetch_chunks; ++ch, ++asked)
                tma_prefetch_l2_3d(&p.tmap_b, 0, u * 16, ch * 8);
    }
    if (!(p.b_constant && warp == kRingConsumers)) pdl_wait();
    if (warp == 0) RING_STAMP(2);

    if (warp == kRingConsumers) {
        // ------------------------------------------------------------ producer
        uint32_t s = 0, phase = 0;
        bool ok = true;
        for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
            for (int ch = 0; ch < chunks; ++ch) {
                if (!mbar_wait(bar_empty + 8u * s, phase ^ 1u, abort_flag, budget)) { ok = false; break; }
                // (test hook, bit 0: CTA 0 leaves out the second chunk of its first unit, so its consumers' wait
                // for that slot runs out)
                const bool withheld = (p.debug_flags & 1) && blockIdx.x == 0 && u == 0 && ch == 1;
                if (u == static_cast<int>(blockIdx.x) && ch == 0) RING_STAMP(3);
                if (elect_one() && !withheld) {
                    mbar_arrive_expect_tx(bar_full + 8u * s, kSlotBytes);
                    tma_load_3d(ring + s * kSlotBytes, &p.tmap_b, bar_full + 8u * s, 0, u * 16, ch * 8);
                }
                if (++s == static_cast<uint32_t>(kRingSlots)) { s = 0; phase ^= 1u; }
            }
        }
    } else {
        // ------------------------------------------------------------ consumers
        const int g = lane >> 2, t = lane & 3;
        const uint8_t* A = static_cast<const uint8_t*>(p.A);
        const bool tok0_ok = g < p.M;
        const bool tok1_ok = kSecondTokenBlock && (g + 8 < p.M);
        const uint8_t* x0 = A + static_cast<long long>(tok0_ok ? g : 0) * p.lda;
        const uint8_t* x1 = A + static_cast<long long>(tok1_ok ? g + 8 : 0) * p.lda;
        // this thread's four 16-byte pieces inside a slice: rows g and g+8, chunks t and t+4, swizzled
        const uint32_t off_ll = static_cast<uint32_t>(warp) * 2048u + g * 128u + ((t ^ g) << 4);
        const uint32_t off_lh = static_cast<uint32_t>(warp) * 2048u + g * 128u + (((t + 4) ^ g) << 4);
        const uint32_t off_hl = off_ll + 1024u;     // row g + 8: same swizzle phase
        const uint32_t off_hh = off_lh + 1024u;
        const int tok = (threadIdx.x >> 4), n = threadIdx.x & 15;    // the C cell this thread finalises

        uint32_t s = 0, phase = 0;
        bool ok = true;
        // chunks this CTA streams in all; if they fit the ring, no slot is ever used twice
        const int my_units = (units - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
        // (only chunks whose slot the producer still needs are released: the proxy fence of a release is
        // ~150 clocks in the consumers' dependency chain, and the last `slots` chunks of a CTA are its tail)
        const int my_chunks = my_units * chunks;
        int chunk_no = 0;
        const uint32_t sx0 = tok_base + g * tok_pitch, sx1 = tok_base + (g + 8) * tok_pitch;
        const bool tsm = p.tokens_in_smem != 0;
        if (tsm) {
            // The tokens are read by every unit: one copy per CTA instead of one L2 read per unit,
            // as one bulk copy per token row, all in flight at once (this sits on the critical
            // path right after the previous kernel's completion, and L2 round trips are long
            // while every SM streams weights).
            // (one lane per token row: issuing a bulk copy costs its thread a few hundred clocks, and this sits
            // right behind the previous kernel's completion)
            if (warp == 0) {
                if (lane == 0) mbar_arrive_expect_tx(bar_tokens, static_cast<uint32_t>(p.M) * static_cast<uint32_t>(p.K));
                __syncwarp();
                if (lane < p.M)
                    bulk_load_1d(tok_base + lane * tok_pitch, A + static_cast<long long>(lane) * p.lda,
                                 static_cast<uint32_t>(p.K), bar_tokens);
            }
            ok = mbar_wait(bar_tokens, 0u, abort_flag, budget);
        }
        // Every consumer thread waits on its own clock, but the warps meet at named barriers once per unit:
        // whether to go on is decided by all 256 together (here and at the end of every unit), so that no warp
        // can leave while another still expects it at a barrier.
        ok = !named_bar_or(1, 256, !ok);
        if (warp == 0) RING_STAMP(4);
        TokenRegs cur = {}, nxt;
        if (ok) {
            if (tsm) load_tokens_smem<kSecondTokenBlock>(cur, sx0, sx1, warp, p.K, t, tok0_ok, tok1_ok);
            else load_tokens<kSecondTokenBlock>(cur, x0, x1, warp, p.K, t, tok0_ok, tok1_ok);
        }
        for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
            // two independent accumulator chains per token block (even / odd k-steps): a chunk's MMAs then
            // depend on each other two deep instead of four deep
            int acc0[4] = {0, 0, 0, 0}, acc0b[4] = {0, 0, 0, 0};
            int acc1[4] = {0, 0, 0, 0}, acc1b[4] = {0, 0, 0, 0};
            for (int ch = 0; ch < chunks; ++ch) {
                // tokens of the next chunk (the first chunk again after the last) travel while we wait
                const int next_ch = ch + 1 < chunks ? ch + 1 : 0;
                if (tsm) load_tokens_smem<kSecondTokenBlock>(nxt, sx0, sx1, next_ch * 8 + warp, p.K, t, tok0_ok, tok1_ok);
                else load_tokens<kSecondTokenBlock>(nxt, x0, x1, next_ch * 8 + warp, p.K, t, tok0_ok, tok1_ok);
                if (!mbar_wait(bar_full + 8u * s, phase, abort_flag, budget)) { ok = false; break; }
                if (warp == 0 && u == static_cast<int>(blockIdx.x) && ch == 0) RING_STAMP(5);
                if (warp == 0 && u + static_cast<int>(gridDim.x) >= units && ch == chunks - 1) RING_STAMP(6);
                const uint32_t base = ring + s * kSlotBytes;
                const uint4 w_ll = lds128(base + off_ll), w_hl = lds128(base + off_hl);
                const uint4 w_lh = lds128(base + off_lh), w_hh = lds128(base + off_hh);
                // The refill is a write through the async proxy to bytes these generic-proxy loads
                // read: the loads must have been performed before the producer may be told.  The
                // barrier arrive alone does not wait for loads still queued in the shared-memory
                // pipe (with two CTAs per SM and weights coming from the L2 the refill did overtake
                // them), the proxy fence does.
                if (chunk_no + kRingSlots < my_chunks || (p.debug_flags & 2)) {   // this slot will be refilled
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_empty + 8u * s);      // the slot may be refilled
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    ring_mma<kUnsignedTokens>((q & 1) ? acc0b : acc0, word(w_ll, q), word(w_hl, q), word(w_lh, q), word(w_hh, q),
                                              word(cur.x0l, q), word(cur.x0h, q));
                    if (kSecondTokenBlock)
                        ring_mma<kUnsignedTokens>((q & 1) ? acc1b : acc1, word(w_ll, q), word(w_hl, q), word(w_lh, q), word(w_hh, q),
                                                  word(cur.x1l, q), word(cur.x1h, q));
                }
                cur = nxt;
                ++chunk_no;
                if (++s == static_cast<uint32_t>(kRingSlots)) { s = 0; phase ^= 1u; }
            }
            // (a warp that gave up still brings its partials -- garbage then -- to the barrier below)
            // accumulator fragment: d0 (row g, col 2t), d1 (g, 2t+1), d2 (g+8, 2t), d3 (g+8, 2t+1);
            // row = weight row of the unit, col = token
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                acc0[e] += acc0b[e];
                acc1[e] += acc1b[e];
            }
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
            if (named_bar_or(1, 256, !ok)) { ok = false; break; }   // partials are in place -- or somebody gave up
            const long long col = static_cast<long long>(u) * 16 + n;
            if (tok < p.M && (kSecondTokenBlock || tok < 8) && col < p.N) {
                int sum = 0;
#pragma unroll
                for (int w = 0; w < kRingConsumers; ++w) sum += red[w][n][tok];
                int32_t* dst = p.C + static_cast<long long>(tok) * p.ldc + col;
                if (p.accumulate) sum = static_cast<int>(static_cast<uint32_t>(sum) + static_cast<uint32_t>(*dst));
                if (p.out_f32) sum = __float_as_int(__int2float_rn(sum) * p.out_scale);   // fused dequantisation
                *dst = sum;
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");           // red[] may be overwritten
        }
        if (!ok) {
            // Unwinding: every slot the producer may have filled must land before the CTA exits;
            // wait (bounded) on the barriers that are still pending, the tokens' first.
            if (tsm) {
                const uint64_t t0 = globaltimer_ns();
                while (!mbar_try_wait(bar_tokens, 0u)) {
                    if (globaltimer_ns() - t0 > 2000000ull) break;
                }
            }
            for (int i = 0; i < kRingSlots; ++i) {
                const uint64_t t0 = globaltimer_ns();
                const uint32_t si = s + i;
                while (!mbar_try_wait(bar_full + 8u * (si % kRingSlots), (si >= static_cast<uint32_t>(kRingSlots)) ? phase ^ 1u : phase)) {
                    if (globaltimer_ns() - t0 > 2000000ull) break;
                }
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) RING_STAMP(7);
    if (threadIdx.x == 0 && *abort_flag != 0) atomicOr(p.status, 1u);
}

template <bool kU, bool kTwo>
cudaError_t launch_ring_t(SkinnyRingParams p, int grid, cudaStream_t stream) {
    // tokens move into shared memory when they leave room for at least 6 ring slots
    const int fixed = kRedBytes + kRingCtrlBytes + 1024;
    const int tok_bytes = p.M * (p.K + kTokenPad);
    p.tokens_in_smem = (kRingSmemMax - fixed - tok_bytes) / kSlotBytes >= 6 ? 1 : 0;
    int slots = (kRingSmemMax - fixed - (p.tokens_in_smem ? tok_bytes : 0)) / kSlotBytes;
    if (slots > kMaxRingSlots) slots = kMaxRingSlots;
    // Programmatic dependent launch: the kernel lets its successor start as soon as all of its own CTAs
    // are resident.  Under the constant-weights promise the successor's producer then fetches B at once;
    // without it the successor's CTAs only set up and wait, which still hides their launch and prologue
    // now that half-memory CTAs leave room for them (2.28 -> 2.21 ms over a chain of 264 decode GEMMs; with
    // one 210 KB CTA per SM it had measured 4-9 % slower).
    p.pdl_mode = 1;
    {
        // Two CTAs per SM, each with half the shared memory, whenever at least two ring slots are left
        // beside the tokens: while one CTA reduces and stores a unit (or, under the constant-weights
        // promise, while the previous call drains) the other keeps streaming, and it no longer matters
        // which call's CTAs the block scheduler puts side by side.  Measured over a chain of 264 decode
        // GEMMs: 2.49 -> 2.28 ms without the promise, 2.06 -> 1.96 ms with it.
        // Measured and not kept (same-process A/B over the 264-launch decode step): one CTA per SM with nine
        // slots whenever fewer than three fit beside the tokens (M = 16: 6-8 % slower per launch -- eight
        // consumer warps per SM are too few); under the promise, at most one half-memory CTA per SM and
        // call, so that two calls are always co-resident (+18 % on the step: the chain of dependent launches,
        // not the weight stream, paces the small matrices); tokens of M <= 1/4/8 read from global memory chunk
        // by chunk instead of copied to shared memory (0 / +2 / +6 %).
        const int fit_min = 2;
        const int budget = 228 * 1024 / 2 - 2048;
        const int fit = (budget - fixed - tok_bytes) / kSlotBytes;
        if (fit >= fit_min) {
            p.tokens_in_smem = 1;
            slots = fit < kMaxRingSlots ? fit : kMaxRingSlots;
            const int units = (p.N + 15) / 16;
            grid = units < 2 * grid ? units : 2 * grid;
        }
    }
    p.slots = slots;
    const size_t smem = static_cast<size_t>(slots) * kSlotBytes + fixed + (p.tokens_in_smem ? tok_bytes : 0);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
    cfg.blockDim = dim3(kRingThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl_allowed();
    cfg.attrs = attr;
    cfg.numAttrs = p.pdl_mode ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, mip_skinny_ring_kernel<kU, kTwo>, p);
}

}  // namespace

// Opt in to large dynamic shared memory for the current device (once per device).
cudaError_t skinny_ring_init() {
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(mip_skinny_ring_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  kRingSmemMax)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(mip_skinny_ring_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  kRingSmemMax)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(mip_skinny_ring_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  kRingSmemMax)) != cudaSuccess) return e;
    return cudaFuncSetAttribute(mip_skinny_ring_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                kRingSmemMax);
}

bool skinny_ring_supported(const SkinnyParams& p, int sm_count) {
    if (!skinny_supported(p)) return false;
    if (p.K % 128 != 0) return false;
    // needs enough 16-row units that (almost) every SM streams; smaller N uses the cluster-split form.
    // With more than 8 tokens the consumers' token traffic doubles: the ring then only wins when the
    // tokens fit in shared memory beside it.
    const long long units = (static_cast<long long>(p.N) + 15) / 16;
    if (units < sm_count) return false;
    if (p.M <= 8) return true;
    const long long tok_bytes = static_cast<long long>(p.M) * (p.K + kTokenPad);
    return (kRingSmemMax - kRedBytes - kRingCtrlBytes - 1024 - tok_bytes) / kSlotBytes >= 6;
}

cudaError_t launch_skinny_ring(const SkinnyRingParams& p, int sm_count, cudaStream_t stream) {
    const int units = (p.N + 15) / 16;
    const int grid = units < sm_count ? units : sm_count;
    const bool two = p.M > 8;
    if (p.a_unsigned) return two ? launch_ring_t<true, true>(p, grid, stream) : launch_ring_t<true, false>(p, grid, stream);
    return two ? launch_ring_t<false, true>(p, grid, stream) : launch_ring_t<false, false>(p, grid, stream);
}

}  // namespace mip
