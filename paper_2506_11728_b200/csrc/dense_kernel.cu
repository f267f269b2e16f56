// Dense MIP GEMM kernel for sm_100a: C(int32) [+]= A(8-bit) * B(int8).
//
// This is the macro-kernel + micro-kernel of the paper's Figure 1 recast for
// Blackwell: the packing of A and B into contiguous buffers becomes TMA tile
// loads into 128-byte-swizzled shared-memory stages, the micro-kernel's
// C_r += A_r * B_r loop becomes tcgen05.mma.kind::i8 accumulating in tensor
// memory, loops L1-L5 become a persistent tile scheduler, and the load/store of
// C_r becomes the epilogue that drains tensor memory to global memory.
//
// One CTA = 6 warps: warp 0 lane 0 issues TMA loads, warp 1 lane 0 issues MMAs
// (warp 1 also owns the tensor-memory allocation), warps 2-5 are the epilogue
// (warp w reads TMEM lanes 32*(w%4) .. +31).  Two accumulators alternate so the
// epilogue of tile t overlaps the main loop of tile t+1.  Every wait is bounded;
// on expiry the CTA raises an abort word, all roles unwind, outstanding copies
// and MMAs are drained with a bounded wait, tensor memory is released and bit 0
// of *status is set.
#include "internal.h"
#include "ptx.cuh"

namespace mip {

struct TileCoord {
    int m0, n0, kb_begin, kb_end;
};

__device__ __forceinline__ TileCoord decode_unit(const DenseParams& p, int unit, int rows_per_tile) {
    const int tiles_mn = p.tiles_m * p.tiles_n;
    const int ks = unit / tiles_mn;
    const int t = unit - ks * tiles_mn;
    // Rasterisation: groups of `group_n` tile columns are swept top to bottom with the
    // column index fastest, so the B panel of a group stays in L2 while A streams by.
    const int per_group = p.group_n * p.tiles_m;
    const int g = t / per_group;
    const int first_n = g * p.group_n;
    const int gsize = min(p.group_n, p.tiles_n - first_n);
    const int r = t - g * per_group;
    const int tm = r / gsize;
    const int tn = first_n + (r - tm * gsize);
    TileCoord c;
    c.m0 = tm * rows_per_tile;
    c.n0 = tn * p.block_n;
    c.kb_begin = ks * p.kb_per_split;
    c.kb_end = min(p.k_blocks, c.kb_begin + p.kb_per_split);
    return c;
}

// Writes one 32-column chunk of one row of the tile.
__device__ __forceinline__ void store_chunk(const DenseParams& p, int32_t* dst, uint32_t (&v)[32], int cols) {
    if (p.use_red) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
            if (j < cols) red_add_s32(dst + j, v[j]);
        return;
    }
    if (cols == 32 && p.store_vec >= 4) {
        if (p.accumulate) {
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                uint32_t c[4];
                ld_global_v4(dst + 4 * g, c);
#pragma unroll
                for (int j = 0; j < 4; ++j) v[4 * g + j] += c[j];
            }
        }
        if (p.store_vec == 8) {
#pragma unroll
            for (int g = 0; g < 4; ++g) st_global_v8(dst + 8 * g, &v[8 * g]);
        } else {
#pragma unroll
            for (int g = 0; g < 8; ++g) st_global_v4(dst + 4 * g, &v[4 * g]);
        }
        return;
    }
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        if (j < cols) {
            uint32_t x = v[j];
            if (p.accumulate) x += static_cast<uint32_t>(dst[j]);
            dst[j] = static_cast<int32_t>(x);
        }
    }
}

__global__ void __launch_bounds__(kDenseThreads, 1)
mip_dense_kernel(const __grid_constant__ DenseParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = ((raw_addr + 1023u) & ~1023u) - raw_addr;
    uint8_t* smem = smem_raw + pad;
    const uint32_t smem_base = raw_addr + pad;

    const uint32_t a_bytes = kBlockM * p.block_k;
    const uint32_t b_bytes = p.block_n * p.block_k;
    const uint32_t stage_bytes = a_bytes + b_bytes;
    const uint32_t ctrl = smem_base + p.stages * stage_bytes;
    // control block: full[stages] | empty[stages] | tmem_full[2] | tmem_empty[2] | drain | slot | abort
    const uint32_t bar_full = ctrl;
    const uint32_t bar_empty = bar_full + 8u * p.stages;
    const uint32_t bar_tfull = bar_empty + 8u * p.stages;
    const uint32_t bar_tempty = bar_tfull + 16u;
    const uint32_t bar_drain = bar_tempty + 16u;
    uint8_t* ctrl_ptr = smem + p.stages * stage_bytes;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctrl_ptr + 16 * p.stages + 40);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(bar_full + 8u * s, 1);
            mbar_init(bar_empty + 8u * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull + 8u * a, 1);
            mbar_init(bar_tempty + 8u * a, 4);
        }
        mbar_init(bar_drain, 1);
        *abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&p.tmap_a);
        tma_prefetch_desc(&p.tmap_b);
    }
    if (warp == 1) {
        tmem_alloc<1>(smem_u32(tmem_slot), p.tmem_cols);
        tmem_relinquish<1>();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int total_units = p.tiles_m * p.tiles_n * p.split_k;
    const uint64_t budget = p.wait_budget_ns;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t s = 0, phase = 0, issued = 0;
            bool ok = true;
            for (int unit = blockIdx.x; unit < total_units && ok; unit += gridDim.x) {
                const TileCoord tc = decode_unit(p, unit, kBlockM);
                int cw = 0, chh = 0, cn = 0;
                if (p.a_im2col) {
                    cn = tc.m0 / p.conv_howo;
                    const int rem = tc.m0 - cn * p.conv_howo;
                    const int ho = rem / p.conv_wo;
                    const int wo = rem - ho * p.conv_wo;
                    cw = wo * p.stride_w - p.pad_w;
                    chh = ho * p.stride_h - p.pad_h;
                }
                for (int kb = tc.kb_begin; kb < tc.kb_end; ++kb) {
                    if (!mbar_wait(bar_empty + 8u * s, phase ^ 1u, abort_flag, budget)) { ok = false; break; }
                    const uint32_t full = bar_full + 8u * s;
                    const uint32_t a_dst = smem_base + s * stage_bytes;
                    mbar_arrive_expect_tx(full, stage_bytes);
                    if (p.a_im2col) {
                        const int tap = kb / p.c_chunks;
                        const int cc = kb - tap * p.c_chunks;
                        const int fr = tap / p.conv_s;
                        const int fs = tap - fr * p.conv_s;
                        tma_load_im2col_4d(a_dst, &p.tmap_a, full, cc * p.block_k, cw, chh, cn,
                                           static_cast<uint16_t>(fs * p.dil_w),
                                           static_cast<uint16_t>(fr * p.dil_h));
                    } else {
                        tma_load_2d(a_dst, &p.tmap_a, full, kb * p.block_k, tc.m0);
                    }
                    tma_load_2d(a_dst + a_bytes, &p.tmap_b, full, kb * p.block_k, tc.n0);
                    ++issued;
                    if (++s == static_cast<uint32_t>(p.stages)) { s = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // Unwinding: wait (bounded) until every copy already issued has landed.
                const uint32_t n = min(issued, static_cast<uint32_t>(p.stages));
                for (uint32_t i = 1; i <= n; ++i) {
                    const uint32_t idx = issued - i;
                    const uint32_t st = idx % p.stages;
                    const uint32_t ph = (idx / p.stages) & 1u;
                    const uint64_t t0 = globaltimer_ns();
                    while (!mbar_try_wait(bar_full + 8u * st, ph)) {
                        if (globaltimer_ns() - t0 > budget) break;
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t s = 0, phase = 0;
            const uint32_t k_steps = p.block_k / 32;
            bool ok = true;
            int t = 0;
            for (int unit = blockIdx.x; unit < total_units && ok; unit += gridDim.x, ++t) {
                const TileCoord tc = decode_unit(p, unit, kBlockM);
                const uint32_t acc = t & 1, acc_phase = (t >> 1) & 1;
                if (!mbar_wait(bar_tempty + 8u * acc, acc_phase ^ 1u, abort_flag, budget)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * p.block_n;
                for (int kb = tc.kb_begin; kb < tc.kb_end; ++kb) {
                    if (!mbar_wait(bar_full + 8u * s, phase, abort_flag, budget)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = smem_base + s * stage_bytes;
                    const uint64_t a_desc = make_kmajor_desc(a_addr, p.block_k);
                    const uint64_t b_desc = make_kmajor_desc(a_addr + a_bytes, p.block_k);
                    for (uint32_t k = 0; k < k_steps; ++k) {
                        mma_i8<1>(d_tmem, a_desc + 2ull * k, b_desc + 2ull * k, p.idesc,
                                  (kb > tc.kb_begin || k > 0) ? 1u : 0u);
                    }
                    mma_commit(bar_empty + 8u * s);
                    if (++s == static_cast<uint32_t>(p.stages)) { s = 0; phase ^= 1u; }
                }
                if (ok) mma_commit(bar_tfull + 8u * acc);
            }
            if (!ok) {
                // Unwinding: let every MMA already issued retire before TMEM is released.
                mma_commit(bar_drain);
                const uint64_t t0 = globaltimer_ns();
                while (!mbar_try_wait(bar_drain, 0)) {
                    if (globaltimer_ns() - t0 > budget) break;
                }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int q = warp & 3;
        int t = 0;
        for (int unit = blockIdx.x; unit < total_units; unit += gridDim.x, ++t) {
            const TileCoord tc = decode_unit(p, unit, kBlockM);
            const uint32_t acc = t & 1, acc_phase = (t >> 1) & 1;
            if (!mbar_wait(bar_tfull + 8u * acc, acc_phase, abort_flag, budget)) break;
            tc_fence_after();
            const int row = tc.m0 + q * 32 + lane;
            const int n_rem = p.N - tc.n0;
            const int n_here = min(p.block_n, n_rem);
            if (tc.m0 + q * 32 < p.M) {
                int32_t* crow = p.C + static_cast<long long>(row) * p.ldc + tc.n0;
                const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * p.block_n;
                for (int c0 = 0; c0 < n_here; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld_32x32(t_row + c0, v);
                    tmem_ld_wait();
                    if (row < p.M) store_chunk(p, crow + c0, v, min(32, n_here - c0));
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty + 8u * acc);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc<1>(tmem_base, p.tmem_cols);
    }
    if (threadIdx.x == 0 && *abort_flag != 0) atomicOr(p.status, 1u);
}

cudaError_t dense_init() {
    return cudaFuncSetAttribute(mip_dense_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
}

cudaError_t launch_dense(const DenseParams& p, int grid, size_t smem_bytes, cudaStream_t stream) {
    mip_dense_kernel<<<grid, kDenseThreads, smem_bytes, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace mip
