// Dense MIP GEMM kernel for sm_100a: C(int32) [+]= A(8-bit) * B(int8).
//
// This is the macro-kernel + micro-kernel of the paper's Figure 1 recast for
// Blackwell: the packing of A and B into contiguous buffers becomes TMA tile
// loads into 128-byte-swizzled shared-memory stages, the micro-kernel's
// C_r += A_r * B_r loop becomes tcgen05.mma.kind::i8 accumulating in tensor
// memory, loops L1-L5 become a persistent tile scheduler, and the load/store of
// C_r becomes the epilogue that drains tensor memory to global memory.
//
// One CTA = 6 warps: warp 0 issues TMA loads, warp 1 issues MMAs (one elected lane
// each; warp 1 also owns the tensor-memory allocation), warps 2-5 are the epilogue
// (warp w reads TMEM lanes 32*(w%4) .. +31).  Two accumulators alternate so the
// epilogue of tile t overlaps the main loop of tile t+1.  Every wait is bounded;
// on expiry the CTA raises an abort word, all roles unwind, outstanding copies
// and MMAs are drained with a bounded wait, tensor memory is released and bit 0
// of *status is set.
//
// The kernel exists in two forms.  kPair = false: one CTA per 128 x block_n tile
// (cta_group::1).  kPair = true: clusters of two CTAs share a 256 x block_n tile
// (cta_group::2): each CTA stages its own 128 rows of A and HALF of the B tile, the
// leader CTA (cluster rank 0) issues every MMA, and both CTAs' tensor memories receive
// their 128 rows of the accumulator -- B traffic from L2 and shared memory is halved.
// Both CTAs' TMA loads complete on the leader's "full" barrier; MMA completion is
// committed to each CTA's own "empty" / "tmem_full" barrier with two plain commits (no
// multicast form is used anywhere in this file).
#include "internal.h"
#include "ptx.cuh"

namespace mip {

#ifdef MIPGEMM_TRACE
#define MIP_STAMP(slot) do { if (p.trace && blockIdx.x == 0 && (threadIdx.x & 31) == 0) p.trace[slot] = globaltimer_ns(); } while (0)
#else
#define MIP_STAMP(slot) do { } while (0)
#endif

struct TileCoord {
    int m0, n0, kb_begin, kb_end, batch;
};

__device__ __forceinline__ TileCoord decode_unit(const DenseParams& p, int unit, int rows_per_tile) {
    const int tiles_mn = p.tiles_m * p.tiles_n;
    int batch = 0;
    if (p.batch > 1) {                 // strided batch: the batch index is the slowest (no split-K)
        batch = unit / tiles_mn;
        unit -= batch * tiles_mn;
    }
    // cluster split-K: the CTAs of a cluster (consecutive units) share one tile
    const int ks = p.cluster_split > 1 ? unit % p.cluster_split : unit / tiles_mn;
    const int t = p.cluster_split > 1 ? unit / p.cluster_split : unit - ks * tiles_mn;
    // Rasterisation: groups of `group_n` tile columns are swept top to bottom with the
    // column index fastest, so the B panel of a group stays in L2 while A streams by.
    const int per_group = p.group_n * p.tiles_m;
    const int g = t / per_group;
    const int first_n = g * p.group_n;
    const int gsize = min(p.group_n, p.tiles_n - first_n);
    const int r = t - g * per_group;
    int tm = r / gsize;
    const int tn = first_n + (r - tm * gsize);
    if ((p.raster & 1) && (g & 1)) tm = p.tiles_m - 1 - tm;   // serpentine: the A slabs at the turn are still in L2
    TileCoord c;
    c.m0 = tm * rows_per_tile;
    c.n0 = tn * p.block_n;
    c.kb_begin = ks * p.kb_per_split;
    c.kb_end = min(p.k_blocks, c.kb_begin + p.kb_per_split);
    c.batch = batch;
    return c;
}

// Optional per-output-channel int32 bias, added to the exact sums before they are scaled (an extension
// of the paper's scale-only transform, Section 7.3).  v holds 32 consecutive columns starting at col0;
// every lane of a warp reads the same 32 words (one broadcast request per load, served by L1).
__device__ __forceinline__ void add_bias_chunk(const DenseParams& p, uint32_t (&v)[32], int col0) {
    const int32_t* b = p.bias + col0;
    const int cols = p.N - col0;
#pragma unroll
    for (int j = 0; j < 32; ++j)
        if (j < cols) v[j] += static_cast<uint32_t>(__ldg(b + j));
}

// Fused dequantisation (paper Section 7.3, C^r = s_A s_B C^q): the exact int32 sum is converted to
// binary32 (round to nearest even) and multiplied by the scale in binary32.
__device__ __forceinline__ void dequant_chunk(const DenseParams& p, uint32_t (&v)[32], int col0) {
    if (p.bias) add_bias_chunk(p, v, col0);
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__int2float_rn(static_cast<int>(v[j])) * p.out_scale);
}

// Requantised output: the exact int32 sum is converted to binary32 (round to nearest even), multiplied
// by the scale in binary32, rounded to the nearest integer (ties to even, saturating) and clamped to
// [q_lo, q_hi]; one byte per element.  `dst` addresses the first of the chunk's `cols` bytes.
__device__ __forceinline__ void store_q8_chunk(const DenseParams& p, uint8_t* dst, const uint32_t (&v)[32], int cols) {
    // The float -> integer step avoids the quarter-rate conversion unit (the epilogue's limit): clamping first
    // (the bounds are integers, so clamp and round-to-nearest-even commute) leaves |t| < 2^22, where adding
    // 1.5 * 2^23 rounds t to the nearest integer, ties to even, and leaves its two's complement in the low
    // mantissa bits.  Same codes as cvt.rni + clamp.
    const float lo = static_cast<float>(p.q_lo), hi = static_cast<float>(p.q_hi);
    uint32_t w[8];
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        uint32_t b[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float t = __fmul_rn(__int2float_rn(static_cast<int>(v[4 * g + j])), p.out_scale);
            t = fminf(fmaxf(t, lo), hi);
            b[j] = __float_as_uint(__fadd_rn(t, 12582912.0f));
        }
        // byte 0 of b[0..3] -> one word
        w[g] = __byte_perm(__byte_perm(b[0], b[1], 0x0040), __byte_perm(b[2], b[3], 0x0040), 0x5410);
    }
    if (cols == 32 && p.store_vec == 16) {
        st_global_v4(reinterpret_cast<int32_t*>(dst), &w[0]);
        st_global_v4(reinterpret_cast<int32_t*>(dst + 16), &w[4]);
        return;
    }
#pragma unroll
    for (int j = 0; j < 32; ++j)
        if (j < cols) dst[j] = static_cast<uint8_t>(w[j >> 2] >> (8 * (j & 3)));
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

// Adds one 32 x 32 chunk (thread = row, v = its 32 columns) into C through the TMA: the rows
// go to a 128-byte-swizzled staging buffer, then one elected lane issues a tile reduce-add
// (32-bit integer adds performed at the L2: exact and order-independent), which clips the
// tile at the edges of C.  Used for split-K.  `buf` alternates between two buffers; at most
// one earlier copy may still be reading shared memory.
__device__ __forceinline__ void tma_reduce_chunk(const DenseParams& p, uint32_t buf, const uint32_t (&v)[32],
                                                 int lane, int x, int y) {
    if (elect_one()) tma_store_wait_read<1>();
    __syncwarp();
    const uint32_t row = buf + static_cast<uint32_t>(lane) * 128u;
#pragma unroll
    for (int j = 0; j < 8; ++j) st_shared_v4(row + (static_cast<uint32_t>(j ^ (lane & 7)) << 4), &v[4 * j]);
    fence_proxy_async_smem();
    __syncwarp();
    if (elect_one()) {   // always the same lane: bulk-group bookkeeping is per thread
        tma_reduce_add_2d(&p.tmap_c, buf, x, y);
        tma_store_commit();
    }
}

// Stores one 128 x 32 slab of the tile (all four epilogue warps, thread = row) with a single
// TMA tile store: the rows go to a 128-byte-swizzled 16 KB staging buffer, the four warps
// meet at a named barrier, and one thread issues the store, which clips at the edges of C.
// `buf` alternates between two buffers; `issuer` is true in exactly one warp.
__device__ __forceinline__ void tma_store_slab(const DenseParams& p, uint32_t buf, const uint32_t (&v)[32],
                                               int lane, int q, bool issuer, int x, int y, int z = 0) {
#ifdef MIPGEMM_TRACE
    const long long ts0 = clock64();
#endif
    if (issuer && elect_one()) tma_store_wait_read<1>();
#ifdef MIPGEMM_TRACE
    const long long ts1 = clock64();
#endif
    asm volatile("bar.sync 1, 128;" ::: "memory");      // the buffer is free for all four warps
#ifdef MIPGEMM_TRACE
    const long long ts2 = clock64();
#endif
    const int r = q * 32 + lane;
    const uint32_t row = buf + static_cast<uint32_t>(r) * 128u;
#pragma unroll
    for (int j = 0; j < 8; ++j) st_shared_v4(row + (static_cast<uint32_t>(j ^ (r & 7)) << 4), &v[4 * j]);
#ifdef MIPGEMM_TRACE
    const long long ts3 = clock64();
#endif
    fence_proxy_async_smem();
#ifdef MIPGEMM_TRACE
    const long long ts4 = clock64();
#endif
    asm volatile("bar.sync 1, 128;" ::: "memory");      // all 128 rows are in place
#ifdef MIPGEMM_TRACE
    const long long ts5 = clock64();
#endif
    if (issuer && elect_one()) {
        if (p.accumulate) {   // C += : the slab is added to C at the L2 (32-bit integer adds, exact in any order)
            if (p.batch > 1) tma_reduce_add_3d(&p.tmap_c, buf, x, y, z);
            else tma_reduce_add_2d(&p.tmap_c, buf, x, y);
        } else if (p.batch > 1) {
            tma_store_3d(&p.tmap_c, buf, x, y, z);
        } else {
            tma_store_2d(&p.tmap_c, buf, x, y);
        }
        tma_store_commit();
    }
#ifdef MIPGEMM_TRACE
    if (p.trace && (p.debug_flags & 128) && blockIdx.x == 0 && threadIdx.x == 64) {   // (perturbs: on request only)
        p.trace[50] += ts1 - ts0; p.trace[51] += ts2 - ts1; p.trace[52] += ts3 - ts2; p.trace[53] += ts4 - ts3;
        p.trace[54] += ts5 - ts4; p.trace[55] += clock64() - ts5; p.trace[56] += 1;
    }
#endif
}

// Writes one 32 x 32 chunk (thread = row, v = its 32 columns) with fully coalesced 16-byte
// accesses: the chunk is transposed through a swizzled staging buffer so that every store
// instruction of the warp covers four complete 128-byte rows of C.  With accumulate, the
// incoming C is read with the same access pattern and added.  Needs a 16-byte aligned C
// base and ldc % 4 == 0.  (row0, col0) is the chunk's origin in C.
__device__ __forceinline__ void coalesced_chunk(const DenseParams& p, uint32_t buf, const uint32_t (&v)[32],
                                                int lane, int row0, int col0, long long c_off = 0) {
    __syncwarp();   // the previous chunk's reads of `buf` are done
    const uint32_t mine = buf + static_cast<uint32_t>(lane) * 128u;
#pragma unroll
    for (int j = 0; j < 8; ++j) st_shared_v4(mine + (static_cast<uint32_t>(j ^ (lane & 7)) << 4), &v[4 * j]);
    __syncwarp();
    const int piece = lane & 7;                 // which 16 bytes (4 columns) of a row
    const int col = col0 + 4 * piece;
    const int cols_left = p.N - col;            // <= 0: nothing of this piece is inside C
    // all eight shared-memory reads are issued before the first global access depends on them
    uint32_t x[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = 4 * i + (lane >> 3);
        asm("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
            : "=r"(x[i][0]), "=r"(x[i][1]), "=r"(x[i][2]), "=r"(x[i][3])
            : "r"(buf + static_cast<uint32_t>(r) * 128u + (static_cast<uint32_t>(piece ^ (r & 7)) << 4))
            : "memory");
    }
    int32_t* dst0 = p.C + c_off + static_cast<long long>(row0 + (lane >> 3)) * p.ldc + col;
    const long long step = 4 * p.ldc;
    if (p.accumulate && cols_left >= 4) {
        uint32_t c[8][4];
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (row0 + 4 * i + (lane >> 3) < p.M) ld_global_v4(dst0 + i * step, c[i]);
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) x[i][j] += c[i][j];
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int row = row0 + 4 * i + (lane >> 3);
        if (row < p.M && cols_left > 0) {
            int32_t* dst = dst0 + i * step;
            if (cols_left >= 4) {
                st_global_v4(dst, x[i]);
            } else {
#pragma unroll
                for (int j = 0; j < 3; ++j) {
                    if (j < cols_left) {
                        uint32_t y = x[i][j];
                        if (p.accumulate) y += static_cast<uint32_t>(dst[j]);
                        dst[j] = static_cast<int32_t>(y);
                    }
                }
            }
        }
    }
}

// Gather form: one 16-byte chunk of a row of A is copied from the image with five 4-byte loads
// at the source address rounded down; funnel shifts then bring the sixteen bytes into place.
// The two rare cases are kept off the common path, which stays
// a handful of instructions per chunk -- the gather warps are bound by their instruction latency:
//   * the pixel's window hangs over the left or right edge of the image: the bytes outside
//     [keep_lo, keep_hi) of the chunk (taps outside the image) are cleared with gather_mask;
//   * gather_border_chunk: the chunk begins before the batch or reaches past its end (first and
//     last pixels of the whole batch only).  It is assembled byte by byte from the bytes that
//     exist; all others are either taps outside the image (zero) or meet a zero weight.
// (volatile loads: the loads of a k-block stay ahead of the first shared-memory store, i.e. all
// in flight together, instead of each being sunk to its use)
__device__ __forceinline__ uint32_t ldg_nc_u32(const uint32_t* ptr) {
    uint32_t v;
    asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(v) : "l"(ptr));
    return v;
}

// Byte mask of a 16-byte chunk that keeps bytes [keep_lo, keep_hi) (any integers; clamped here).
__device__ __forceinline__ uint4 gather_mask(int keep_lo, int keep_hi) {
    uint32_t w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t a = static_cast<uint32_t>(min(max(keep_lo - 4 * j, 0), 4)) * 8u;   // bits to clear from below
        const uint32_t b = static_cast<uint32_t>(min(max(keep_hi - 4 * j, 0), 4)) * 8u;   // bits to keep from below
        // (clamped funnel shift: 0xFFFFFFFF << n, and 0 for n = 32)
        w[j] = __funnelshift_lc(0u, 0xFFFFFFFFu, a) & ~__funnelshift_lc(0u, 0xFFFFFFFFu, b);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

__device__ __noinline__ void gather_border_chunk(const uint8_t* gx, int xbytes, int src, int keep_lo, int keep_hi,
                                                 uint32_t smem_dst) {
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    for (int t = 0; t < 16; ++t) {
        const int i = src + t;
        if (t >= keep_lo && t < keep_hi && i >= 0 && i < xbytes) {
            const uint32_t byte = static_cast<uint32_t>(gx[i]) << (8 * (t & 3));
            if (t < 4) w[0] |= byte; else if (t < 8) w[1] |= byte; else if (t < 12) w[2] |= byte; else w[3] |= byte;
        }
    }
    st_shared_v4(smem_dst, w);
}

// Same idea for a C that is only 4-byte aligned (odd pitch or base): the chunk goes through the warp's
// staging buffer and is written one row per instruction, lane = column, so that every access of the
// warp is one contiguous 128-byte run instead of 32 words 4*ldc bytes apart.  With accumulate the
// incoming C is read the same way.  Warp-collective.
__device__ __forceinline__ void rows_chunk(const DenseParams& p, uint32_t buf, const uint32_t (&v)[32], int lane,
                                           int row0, int col0, long long c_off) {
    __syncwarp();   // the previous chunk's reads of `buf` are done
    const uint32_t mine = buf + static_cast<uint32_t>(lane) * 128u;
#pragma unroll
    for (int j = 0; j < 8; ++j) st_shared_v4(mine + (static_cast<uint32_t>(j ^ (lane & 7)) << 4), &v[4 * j]);
    __syncwarp();
    const int col = col0 + lane;
    if (col >= p.N) return;
    int32_t* dst = p.C + c_off + static_cast<long long>(row0) * p.ldc + col;
    const int rows = min(32, p.M - row0);
    if (!p.accumulate) {
        for (int r = 0; r < rows; ++r) {
            uint32_t x;
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(x)
                         : "r"(buf + static_cast<uint32_t>(r) * 128u + (static_cast<uint32_t>((lane >> 2) ^ (r & 7)) << 4) +
                               static_cast<uint32_t>(lane & 3) * 4u) : "memory");
            *dst = static_cast<int32_t>(x);
            dst += p.ldc;
        }
        return;
    }
    // C += : the sums are added at the L2 (32-bit integer reductions, one 128-byte run per instruction): exact in
    // any order, and no thread waits for the old value of C
    for (int r = 0; r < rows; ++r) {
        uint32_t x;
        asm volatile("ld.shared.b32 %0, [%1];" : "=r"(x)
                     : "r"(buf + static_cast<uint32_t>(r) * 128u + (static_cast<uint32_t>((lane >> 2) ^ (r & 7)) << 4) +
                           static_cast<uint32_t>(lane & 3) * 4u) : "memory");
        red_add_s32(dst, x);
        dst += p.ldc;
    }
}

template <bool kPair, bool kMN, bool kGather, bool kQ8>
__global__ void __launch_bounds__(kGather ? kGatherThreads : (kQ8 ? kDenseQ8Threads : kDenseThreads), 1)
mip_dense_kernel(const __grid_constant__ DenseParams p) {
    constexpr int kGroup = kPair ? 2 : 1;
    // epilogue warps: four (one per quarter of the TMEM lanes); the 8-bit-code epilogue, bound by its
    // conversion arithmetic, runs eight (two per quarter, alternating 32-column chunks)
    constexpr int kEpiWarps = (kQ8 && !kGather) ? 8 : 4;
    constexpr int kRowsPerTile = kPair ? 2 * kBlockM : kBlockM;
    const uint32_t cta_rank = kPair ? cluster_ctarank() : 0u;
    const bool leader = cta_rank == 0;
    const int first_unit = kPair ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
    const int unit_stride = kPair ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);
    const int b_rows = kPair ? (p.block_n >> 1) : p.block_n;   // rows of B staged by this CTA
    MIP_STAMP(0);
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = ((raw_addr + 1023u) & ~1023u) - raw_addr;
    uint8_t* smem = smem_raw + pad;
    const uint32_t smem_base = raw_addr + pad;

    const uint32_t a_bytes = kBlockM * p.block_k;
    const uint32_t b_bytes = b_rows * p.block_k;
    const uint32_t stage_bytes = a_bytes + b_bytes;
    // shared memory: [stages x (A tile | B tile)] [epilogue staging] [control block]
    const uint32_t staging = smem_base + p.stages * stage_bytes;
    const uint32_t ctrl = staging + kStagingBytes;
    // control block: full[stages] | empty[stages] | tmem_full[2] | tmem_empty[2] | drain | slot | abort
    const uint32_t bar_full = ctrl;
    const uint32_t bar_empty = bar_full + 8u * p.stages;
    const uint32_t bar_tfull = bar_empty + 8u * p.stages;
    const uint32_t bar_tempty = bar_tfull + 16u;
    const uint32_t bar_drain = bar_tempty + 16u;
    // staged gather: two more barrier pairs at ctrl + 256, the two image-row buffers behind the control block
    const uint32_t bar_rows_full = ctrl + 256u;
    const uint32_t bar_rows_empty = ctrl + 272u;
    const uint32_t rowbuf0 = ctrl + kCtrlBytes + 64u;      // (64 guard bytes in front: windows start left of a row)
    uint8_t* ctrl_ptr = smem + p.stages * stage_bytes + kStagingBytes;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctrl_ptr + 16 * p.stages + 40);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(tmem_slot + 1);

    // Broadcasting the warp index makes it provably warp-uniform for the compiler, so each
    // role's loop runs convergently (addresses, counters and descriptors live in uniform
    // registers) and only the single-thread instructions are issued under elect_one().
    const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(bar_full + 8u * s, kGather ? 1 + 4 * kGatherParities : ((kQ8 && !kGather) ? 1 : 2));   // producer(s) (+ gather warps)
            mbar_init(bar_empty + 8u * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull + 8u * a, 1);
            mbar_init(bar_tempty + 8u * a, kPair ? 2 * kEpiWarps : kEpiWarps);
        }
        mbar_init(bar_drain, 1);
        if (kGather) {
            for (int b = 0; b < 2; ++b) {
                mbar_init(bar_rows_full + 8u * b, 1);
                mbar_init(bar_rows_empty + 8u * b, 4 * kGatherParities);   // one arrival per gather warp
            }
        }
        *abort_flag = 0;
        fence_mbar_init();
        if (!kGather) tma_prefetch_desc(&p.tmap_a);
        tma_prefetch_desc(&p.tmap_b);
        if (p.c_mode == 1 || p.c_mode == 2) tma_prefetch_desc(&p.tmap_c);
    }
    if (warp == 1) {
        tmem_alloc<kGroup>(smem_u32(tmem_slot), p.tmem_cols);
        tmem_relinquish<kGroup>();
    }
    tc_fence_before();
    __syncthreads();
    if (kPair) {   // the peer's barriers must be initialised before anything remote touches them
        cluster_arrive();
        cluster_wait();
    }
    tc_fence_after();
    // Programmatic dependent launch: everything so far touched only shared memory, tensor memory
    // and kernel parameters and may overlap the tail of the previous kernel in the stream; from
    // here on global memory is read and written, which must wait for that kernel to finish.
    pdl_launch_dependents();
    pdl_wait();
    const uint32_t tmem_base = *tmem_slot;
    if (threadIdx.x == 0) MIP_STAMP(1);

    const int total_units = p.tiles_m * p.tiles_n * p.split_k * (p.batch > 1 ? p.batch : 1);
    const uint64_t budget = p.wait_budget_ns;
    uint32_t issued = 0;   // producer warp: k-blocks whose loads have been issued (the unwinding path needs it)
    uint32_t rows_tiles = 0;   // producer warp, staged gather: tiles whose image rows have been requested

    // Two producer warps, one per operand (warp 0: A, warp 2 + kEpiWarps: B): a TMA load costs its issuing
    // thread some 250 clocks, so with both loads of a k-block in one thread the producer itself paced the
    // shapes with short k-blocks (64-channel convolutions: 2 x 250 clocks against 190 clocks of smem fill).
    // Both walk the same tiles and stages; each arms the stage's "full" barrier with its own byte count.
    // (The gather form has one producer: operand A is written by the gather warps.  So has the 8-bit-code form,
    // whose eight epilogue warps need the registers.)
    constexpr bool kTwoProducers = !kGather && !kQ8;
    constexpr int kWarpB = kTwoProducers ? 2 + kEpiWarps : 0;
    if (warp == 0 || warp == kWarpB) {
        // ------------------------------------------------------------ TMA producers (whole warp loops)
        uint32_t s = 0, phase = 0;
        bool ok = true;
        const bool side_a = !kGather && warp == 0;
        const bool side_b = warp == kWarpB;
        const uint32_t tx_bytes = (kPair ? 2u : 1u) * ((side_a ? a_bytes : 0u) + (side_b ? b_bytes : 0u));
        for (int unit = first_unit; unit < total_units && ok; unit += unit_stride) {
            const TileCoord tc = decode_unit(p, unit, kRowsPerTile);
            const int m_cta = tc.m0 + static_cast<int>(cta_rank) * kBlockM;
            const int n_cta = tc.n0 + static_cast<int>(cta_rank) * b_rows;
            int cw = 0, chh = 0, cn = 0;
            if (p.a_im2col) {
                // a peer CTA whose rows all lie beyond M gathers from pixel 0 instead (its
                // accumulator rows are never stored)
                const int m_src = m_cta < p.M ? m_cta : 0;
                cn = m_src / p.conv_howo;
                const int rem = m_src - cn * p.conv_howo;
                const int ho = rem / p.conv_wo;
                const int wo = rem - ho * p.conv_wo;
                cw = wo * p.stride_w - p.pad_w;
                chh = ho * p.stride_h - p.pad_h;
            }
            if (kGather && p.g_staged) {
                // Staged gather: request the image rows this tile's output pixels read.  Output row L (counted
                // through the whole batch) owns g_span row slots of the buffer; slot r * dil_h of them holds input
                // row ho * stride_h - pad_h + r * dil_h if that row exists.
                const uint32_t buf = rows_tiles & 1u, rph = (rows_tiles >> 1) & 1u;
                if (!mbar_wait(bar_rows_empty + 8u * buf, rph ^ 1u, abort_flag, budget)) { ok = false; break; }
                {
                    // one (output row, filter row) pair per lane: a single thread walking all of them paced the
                    // whole tile
                    const uint32_t rows_full = bar_rows_full + 8u * buf;
                    const uint32_t dst0 = rowbuf0 + buf * static_cast<uint32_t>(p.g_rowbuf_stride);
                    const uint32_t m0u = static_cast<uint32_t>(tc.m0);
                    const uint32_t m1u = static_cast<uint32_t>(min(tc.m0 + kBlockM, p.M) - 1);
                    const uint32_t L0 = (__umulhi(p.g_wo_mul, m0u) + m0u) >> p.g_wo_shift;
                    const uint32_t L1 = (__umulhi(p.g_wo_mul, m1u) + m1u) >> p.g_wo_shift;
                    const int pairs = static_cast<int>(L1 - L0 + 1) * p.g_r;
                    for (int idx = lane; idx < pairs; idx += 32) {
                        const int o = idx / p.g_r;
                        const int r = idx - o * p.g_r;
                        const uint32_t L = L0 + static_cast<uint32_t>(o);
                        const uint32_t n_img = (__umulhi(p.g_ho_mul, L) + L) >> p.g_ho_shift;
                        const int h = static_cast<int>(L - n_img * static_cast<uint32_t>(p.g_ho)) * p.stride_h - p.pad_h +
                                      r * p.dil_h;
                        if (h >= 0 && h < p.g_h) {
                            mbar_expect_tx(rows_full, static_cast<uint32_t>(p.g_row_bytes));
                            bulk_load_1d(dst0 + static_cast<uint32_t>((o * p.g_span + r * p.dil_h) * p.g_row_bytes),
                                         p.gx + (static_cast<long long>(n_img) * p.g_h + h) * p.g_row_bytes,
                                         static_cast<uint32_t>(p.g_row_bytes), rows_full);
                        }
                    }
                    __syncwarp();                      // every lane's transaction count is in before the arrival
                    if (lane == 0) mbar_arrive(rows_full);
                }
                ++rows_tiles;
            }
            int tap = 0, cc = 0, fr = 0, fs = 0;
            if (p.a_im2col) {
                tap = tc.kb_begin / p.c_chunks;
                cc = tc.kb_begin - tap * p.c_chunks;
                fr = tap / p.conv_s;
                fs = tap - fr * p.conv_s;
            }
            for (int kb = tc.kb_begin; kb < tc.kb_end; ++kb) {
                if (!mbar_wait(bar_empty + 8u * s, phase ^ 1u, abort_flag, budget)) { ok = false; break; }
                // both CTAs' bytes complete on the leader's barrier, which expects all of them
                const uint32_t full_local = bar_full + 8u * s;
                const uint32_t full = kPair ? mapa_u32(full_local, 0) : full_local;
                const uint32_t a_dst = smem_base + s * stage_bytes;
                if (elect_one()) {
                    if (leader) mbar_arrive_expect_tx(full_local, tx_bytes);
                    if (!side_a) {
                        // operand A is the other producer warp's (or, in the gather form, the gather warps')
                    } else if (p.a_im2col) {
                        if (kPair)
                            tma_load_im2col_4d_pair(a_dst, &p.tmap_a, full, cc * p.block_k, cw, chh, cn,
                                                    static_cast<uint16_t>(fs * p.dil_w),
                                                    static_cast<uint16_t>(fr * p.dil_h));
                        else
                            tma_load_im2col_4d(a_dst, &p.tmap_a, full, cc * p.block_k, cw, chh, cn,
                                               static_cast<uint16_t>(fs * p.dil_w),
                                               static_cast<uint16_t>(fr * p.dil_h));
                    } else if (kMN && p.a_mn) {   // tensor {M, K}: 128 bytes of M per k row
                        if (kPair) tma_load_2d_pair(a_dst, &p.tmap_a, full, m_cta, kb * p.block_k);
                        else tma_load_2d(a_dst, &p.tmap_a, full, m_cta, kb * p.block_k);
                    } else if (kPair) {
                        tma_load_2d_pair(a_dst, &p.tmap_a, full, kb * p.block_k, m_cta);
                    } else if (p.batch > 1) {
                        tma_load_3d(a_dst, &p.tmap_a, full, kb * p.block_k, m_cta, tc.batch);
                    } else {
                        tma_load_2d(a_dst, &p.tmap_a, full, kb * p.block_k, m_cta);
                    }
                    if (!side_b) {
                        // operand B is the other producer warp's
                    } else if (kMN && p.b_mn) {   // tensor {N, K}: one [k][128 B] block per 128 columns
                        for (int blk = 0; blk * 128 < b_rows; ++blk) {
                            const uint32_t dst = a_dst + a_bytes + blk * p.block_k * 128;
                            if (kPair) tma_load_2d_pair(dst, &p.tmap_b, full, n_cta + blk * 128, kb * p.block_k);
                            else tma_load_2d(dst, &p.tmap_b, full, n_cta + blk * 128, kb * p.block_k);
                        }
                    } else if (kPair) {
                        tma_load_2d_pair(a_dst + a_bytes, &p.tmap_b, full, kb * p.block_k, n_cta);
                    } else if (p.batch > 1) {
                        tma_load_3d(a_dst + a_bytes, &p.tmap_b, full, kb * p.block_k, n_cta, tc.batch);
                    } else {
                        tma_load_2d(a_dst + a_bytes, &p.tmap_b, full, kb * p.block_k, n_cta);
                    }
                }
                if (issued == 0) MIP_STAMP(2);
                if (p.a_im2col && ++cc == p.c_chunks) {   // next filter tap (r, s)
                    cc = 0;
                    if (++fs == p.conv_s) { fs = 0; ++fr; }
                }
                ++issued;
                if (++s == static_cast<uint32_t>(p.stages)) { s = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (whole warp loops)
        if (leader) {
            uint32_t s = 0, phase = 0;
            const uint32_t k_steps = p.block_k / 32;
            bool ok = true;
            int t = 0;
#ifdef MIPGEMM_TRACE
            // (trace builds: waits and issue time of CTA 0's MMA warp, summed in registers and written once)
            long long acc_tempty = 0, acc_full = 0, n_tempty = 0, n_full = 0, acc_issue = 0;
            const long long role_t0 = clock64();
#endif
            for (int unit = first_unit; unit < total_units && ok; unit += unit_stride, ++t) {
                const TileCoord tc = decode_unit(p, unit, kRowsPerTile);
                const uint32_t acc = t & 1, acc_phase = (t >> 1) & 1;
#ifdef MIPGEMM_TRACE
                long long tm0 = clock64();
#endif
                if (!mbar_wait<kPair>(bar_tempty + 8u * acc, acc_phase ^ 1u, abort_flag, budget)) { ok = false; break; }
#ifdef MIPGEMM_TRACE
                acc_tempty += clock64() - tm0; ++n_tempty;
#endif
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * p.block_n;
                for (int kb = tc.kb_begin; kb < tc.kb_end; ++kb) {
#ifdef MIPGEMM_TRACE
                    tm0 = clock64();
#endif
                    if (!mbar_wait(bar_full + 8u * s, phase, abort_flag, budget)) { ok = false; break; }
#ifdef MIPGEMM_TRACE
                    acc_full += clock64() - tm0; ++n_full;
                    const long long ti0 = clock64();
#endif
                    if (t == 0 && kb == tc.kb_begin) MIP_STAMP(3);
                    tc_fence_after();
                    const uint32_t a_addr = smem_base + s * stage_bytes;
                    // K-major tiles advance 32 bytes per K = 32 step, MN-major tiles 32 rows of 128 bytes
                    const bool a_mn = kMN && p.a_mn, b_mn = kMN && p.b_mn;
                    const uint64_t a_desc = a_mn ? make_mnmajor_desc(a_addr, p.block_k * 128)
                                                 : make_kmajor_desc(a_addr, p.block_k);
                    const uint64_t b_desc = b_mn ? make_mnmajor_desc(a_addr + a_bytes, p.block_k * 128)
                                                 : make_kmajor_desc(a_addr + a_bytes, p.block_k);
                    const uint64_t a_step = a_mn ? 256ull : 2ull, b_step = b_mn ? 256ull : 2ull;
                    const uint32_t empty_local = bar_empty + 8u * s;
                    const uint32_t empty_peer = kPair ? mapa_u32(empty_local, 1) : 0u;
                    if (elect_one()) {
                        for (uint32_t k = 0; k < k_steps; ++k) {
                            mma_i8<kGroup>(d_tmem, a_desc + a_step * k, b_desc + b_step * k, p.idesc,
                                           (kb > tc.kb_begin || k > 0) ? 1u : 0u);
                        }
                        if (kPair) {
                            mma_commit_pair(empty_local);
                            mma_commit_pair(empty_peer);
                        } else {
                            mma_commit(empty_local);
                        }
                    }
#ifdef MIPGEMM_TRACE
                    __syncwarp();
                    acc_issue += clock64() - ti0;
#endif
                    if (++s == static_cast<uint32_t>(p.stages)) { s = 0; phase ^= 1u; }
                }
                if (t == 0) MIP_STAMP(4);
                if (ok && !(p.debug_flags & 1)) {   // (test hook, bit 0: the "accumulator ready" signal is withheld)
                    const uint32_t tfull_local = bar_tfull + 8u * acc;
                    const uint32_t tfull_peer = kPair ? mapa_u32(tfull_local, 1) : 0u;
                    if (elect_one()) {
                        if (kPair) {
                            mma_commit_pair(tfull_local);
                            mma_commit_pair(tfull_peer);
                        } else {
                            mma_commit(tfull_local);
                        }
                    }
                }
            }
#ifdef MIPGEMM_TRACE
            if (p.trace && blockIdx.x == 0 && lane == 0) {
                p.trace[32] = acc_tempty; p.trace[33] = n_tempty; p.trace[34] = acc_full; p.trace[35] = n_full;
                p.trace[36] = clock64() - role_t0; p.trace[37] = acc_issue;
            }
#endif
        }
    } else if (kGather && warp >= kGatherFirstWarp) {
        // ------------------------------------------------------------ software im2col
        // Thread = every kGatherParities-th 16-byte chunk of one row of the tile (one output
        // pixel).  For every k-block a thread writes its chunks into the stage in the 128-byte-swizzled K-major
        // layout the TMA would have produced, makes them visible to the tensor core's proxy and
        // arrives.  (Issuing the next k-block's loads before the current one is stored was measured
        // and bought nothing: the warps are bound by instruction latency, not by the loads.)  Byte
        // offsets into the batch fit 31 bits (checked by the host).
        const int row = ((warp - kGatherFirstWarp) & 3) * 32 + lane;
        const int parity = (warp - kGatherFirstWarp) >> 2;
        constexpr int kCh = 8 / kGatherParities;        // chunks per thread and k-block
        if (p.g_staged) {
            // Staged form: the rows this tile reads are in shared memory (see the producer warp); a chunk is five
            // aligned 4-byte shared-memory loads, four funnel shifts and one swizzled 16-byte store.  The warps
            // are bound by their instruction count, so everything that does not depend on the pixel is looked
            // up: a table in shared memory holds, for every 16-byte chunk q of a row of A, its byte offset from
            // the window's first byte (filter row * image row pitch + offset in the slot), the filter row's
            // distance in image rows and the offset in the slot; the two divisions per pixel use multipliers
            // prepared by the host.
            constexpr int kStrideB = 16 * kGatherParities;
            const bool fixed = kStrideB % p.g_slot == 0;     // every chunk of this thread at the same offset in its slot
            const uint32_t tab = rowbuf0 + 2u * static_cast<uint32_t>(p.g_rowbuf_stride);
            {
                const int entries = p.k_blocks * 8;
                for (int q = static_cast<int>(threadIdx.x) - 32 * kGatherFirstWarp; q < entries; q += 128 * kGatherParities) {
                    const int r = (q * 16) / p.g_slot;
                    const int off = q * 16 - r * p.g_slot;
                    const bool valid = q < p.g_chunks && off < p.g_seg;
                    // (chunks of the padding behind the last slot read the window's first bytes and are cleared)
                    const uint32_t lo32 = valid ? static_cast<uint32_t>(r * p.dil_h * p.g_row_bytes + off) : 0u;
                    const uint32_t hi32 = valid ? (static_cast<uint32_t>(r * p.dil_h) | (static_cast<uint32_t>(off) << 12))
                                                : 0x80000000u;
                    asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(tab + 8u * q), "r"(lo32), "r"(hi32) : "memory");
                }
                asm volatile("bar.sync 2, %0;" ::"n"(128 * kGatherParities) : "memory");     // the gather warps only
            }
            const int off_c = (parity * 16) % p.g_slot;      // (fixed case) this thread's offset in its slots
            uint32_t s = 0, phase = 0, tile_no = 0;
            bool ok = true;
            for (int unit = first_unit; unit < total_units && ok; unit += unit_stride, ++tile_no) {
                const TileCoord tc = decode_unit(p, unit, kRowsPerTile);
                const int m = tc.m0 + row;
                const uint32_t mm = static_cast<uint32_t>(m < p.M ? m : tc.m0);
                const uint32_t L = (__umulhi(p.g_wo_mul, mm) + mm) >> p.g_wo_shift;     // output row, counted through the batch
                const uint32_t L0 = (__umulhi(p.g_wo_mul, static_cast<uint32_t>(tc.m0)) + static_cast<uint32_t>(tc.m0)) >> p.g_wo_shift;
                const int wo = static_cast<int>(mm - L * static_cast<uint32_t>(p.conv_wo));
                const uint32_t n_img = (__umulhi(p.g_ho_mul, L) + L) >> p.g_ho_shift;
                const int h0 = static_cast<int>(L - n_img * static_cast<uint32_t>(p.g_ho)) * p.stride_h - p.pad_h;
                const int wb = (wo * p.stride_w - p.pad_w) * p.g_cin;     // window start, bytes into the image row
                const int lo = max(0, -wb);
                const int hi = (p.g_row_bytes - wb >= p.g_seg) ? p.g_slot : p.g_row_bytes - wb;
                const uint32_t buf = tile_no & 1u;
                // address of byte 0 of slot 0 of this pixel's window (may lie a few bytes left of its row)
                const int base = static_cast<int>(rowbuf0) + static_cast<int>(buf) * p.g_rowbuf_stride +
                                 static_cast<int>(L - L0) * p.g_span * p.g_row_bytes + wb;
                uint4 tile_mask = make_uint4(~0u, ~0u, ~0u, ~0u);
                bool row_ok = m < p.M;
                if (fixed) {
                    tile_mask = gather_mask(lo - off_c, hi - off_c);
                    row_ok = row_ok & (off_c < hi) & (off_c + 16 > lo);
                }
                if (!mbar_wait(bar_rows_full + 8u * buf, (tile_no >> 1) & 1u, abort_flag, budget)) { ok = false; break; }
                for (int kb = tc.kb_begin; kb < tc.kb_end; ++kb) {
                    if (!mbar_wait(bar_empty + 8u * s, phase ^ 1u, abort_flag, budget)) { ok = false; break; }
                    const uint32_t dst = smem_base + s * stage_bytes + static_cast<uint32_t>(row) * 128u;
#pragma unroll
                    for (int c = 0; c < kCh; ++c) {
                        const int j = parity + kGatherParities * c;            // chunk within the k-block
                        uint32_t e_lo, e_hi;
                        asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(e_lo), "=r"(e_hi)
                                     : "r"(tab + 8u * static_cast<uint32_t>(kb * 8 + j)) : "memory");
                        const int h = h0 + static_cast<int>(e_hi & 0xFFFu);
                        bool use = row_ok & (static_cast<int>(e_hi) >= 0) &
                                   (static_cast<unsigned>(h) < static_cast<unsigned>(p.g_h));
                        uint4 mk = tile_mask;
                        if (!fixed) {
                            const int off = static_cast<int>((e_hi >> 12) & 0x3FFFu);
                            use = use & (off < hi) & (off + 16 > lo);
                            mk = gather_mask(lo - off, hi - off);
                        }
                        const uint32_t a = static_cast<uint32_t>(base + static_cast<int>(e_lo));
                        const uint32_t al = a & ~3u;
                        const uint32_t sh = (a & 3u) * 8u;
                        uint32_t x[5];
#pragma unroll
                        for (int i = 0; i < 5; ++i)
                            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(x[i]) : "r"(al + 4u * i) : "memory");
                        const uint32_t keep = use ? ~0u : 0u;
                        uint32_t vv[4];
                        vv[0] = __funnelshift_r(x[0], x[1], sh) & (mk.x & keep);
                        vv[1] = __funnelshift_r(x[1], x[2], sh) & (mk.y & keep);
                        vv[2] = __funnelshift_r(x[2], x[3], sh) & (mk.z & keep);
                        vv[3] = __funnelshift_r(x[3], x[4], sh) & (mk.w & keep);
                        st_shared_v4(dst + (static_cast<uint32_t>(j ^ (row & 7)) << 4), vv);
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_full + 8u * s);
                    if (++s == static_cast<uint32_t>(p.stages)) { s = 0; phase ^= 1u; }
                }
                if (!ok) break;
                __syncwarp();                                   // every lane has read its last bytes of the row buffer
                if (lane == 0) mbar_arrive(bar_rows_empty + 8u * buf);
            }
        } else {
        const int xbytes = static_cast<int>(p.g_xbytes);
        const uint32_t align = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(p.gx)) & 3u;
        constexpr int kNone = -0x40000000;
        struct Item {                 // one k-block of one tile, as seen by this thread
            int src[kCh], offs[kCh];      // source byte offset of each chunk (kNone: all zero), offset in its slot
            int lo, hi, q0;
            uint4 mask;               // slots of 16 or 32 bytes: every chunk of this thread has the same offset
            uint32_t x[kCh][5];
        };
        constexpr int kStride = 16 * kGatherParities;   // bytes of a row of A between two chunks of a thread
        const bool fixed_off = kStride % p.g_slot == 0;
        const int r_step = kStride / p.g_slot, off_step = kStride - r_step * p.g_slot;
        // per-tile state of the tile that `prepare` is walking through
        int unit = first_unit, kb = 0, kb_end = 0;
        int h0 = 0, lo = 0, hi = 0, src0 = 0;
        uint4 tile_mask = make_uint4(~0u, ~0u, ~0u, ~0u);
        auto next_item = [&](Item& it) -> bool {     // false: no more work
            while (kb >= kb_end) {
                if (unit >= total_units) return false;
                const TileCoord tc = decode_unit(p, unit, kRowsPerTile);
                unit += unit_stride;
                kb = tc.kb_begin;
                kb_end = tc.kb_end;
                const int m = tc.m0 + row;
                const int mm = m < p.M ? m : 0;
                const int n_img = mm / p.conv_howo;
                const int rem = mm - n_img * p.conv_howo;
                const int ho = rem / p.conv_wo;
                const int wo = rem - ho * p.conv_wo;
                // rows beyond M: every filter row falls outside the image, the row of A is zero
                h0 = m < p.M ? ho * p.stride_h - p.pad_h : kNone;
                const int wb = (wo * p.stride_w - p.pad_w) * p.g_cin;   // window start, bytes into the image row
                // taps inside the image row: bytes [lo, hi) of every slot.  When nothing is cut off on
                // the right, the slot's padding bytes are copied as they come (they meet zero weights).
                lo = max(0, -wb);
                hi = (p.g_row_bytes - wb >= p.g_seg) ? p.g_slot : p.g_row_bytes - wb;
                src0 = n_img * p.g_h * p.g_row_bytes + wb;
                // slots of 16 or 32 bytes: every chunk of this thread sits at the same offset in its slot,
                // so one mask serves the whole tile
                if (fixed_off) {
                    const int off_c = (parity * 16) % p.g_slot;
                    tile_mask = gather_mask(lo - off_c, hi - off_c);
                }
            }
            it.lo = lo; it.hi = hi;
            it.q0 = kb * 8 + parity;
            int r = (it.q0 * 16) / p.g_slot;
            int off = it.q0 * 16 - r * p.g_slot;
            it.mask = tile_mask;
            // (no branches from here on: the four chunks' dependency chains interleave, which is
            // what hides the arithmetic latency of a warp that has its scheduler almost to itself)
#pragma unroll
            for (int c = 0; c < kCh; ++c) {
                const int h = h0 + r * p.dil_h;
                const bool use = (it.q0 + kGatherParities * c < p.g_chunks) & (off < p.g_seg) &
                                 (static_cast<unsigned>(h) < static_cast<unsigned>(p.g_h)) & (off < hi) &
                                 (off + 16 > lo);
                it.src[c] = use ? src0 + h * p.g_row_bytes + off : kNone;
                it.offs[c] = off;
                off += off_step;                       // on to the thread's next chunk: r_step slots + off_step bytes
                r += r_step;
                const bool wrap = off >= p.g_slot;
                off -= wrap ? p.g_slot : 0;
                r += wrap ? 1 : 0;
            }
            // all loads back to back and unconditional (chunks that are all zero, and the few at the
            // very ends of the batch, load the batch's first words instead)
#pragma unroll
            for (int c = 0; c < kCh; ++c) {
                const bool plain = (it.src[c] >= 4) & (it.src[c] <= xbytes - 24);
                const uint32_t* w = reinterpret_cast<const uint32_t*>(
                    (reinterpret_cast<uintptr_t>(p.gx) + static_cast<uintptr_t>(plain ? it.src[c] : 4)) &
                    ~static_cast<uintptr_t>(3));
#pragma unroll
                for (int j = 0; j < 5; ++j) it.x[c][j] = ldg_nc_u32(w + j);
            }
            ++kb;
            return true;
        };
        uint32_t s = 0, phase = 0;
        Item cur;
        while (next_item(cur)) {
            if (!mbar_wait(bar_empty + 8u * s, phase ^ 1u, abort_flag, budget)) break;
            const uint32_t dst = smem_base + s * stage_bytes + static_cast<uint32_t>(row) * 128u;
            // Chunks past the end of a row of A (last k-block) are stored as well: they meet the
            // zero fill of B.  Chunks at the very ends of the batch are stored as zero here and
            // patched below.
            bool border = false;
#pragma unroll
            for (int c = 0; c < kCh; ++c) {
                const int sc = cur.src[c];
                const bool plain = (sc >= 4) & (sc <= xbytes - 24);
                border |= (sc != kNone) & !plain;
                const uint32_t sh = ((static_cast<uint32_t>(sc) + align) & 3u) * 8u;
                uint4 mk = cur.mask;
                if (!fixed_off) mk = gather_mask(cur.lo - cur.offs[c], cur.hi - cur.offs[c]);   // (uniform)
                const uint32_t keep = plain ? ~0u : 0u;
                uint32_t vv[4];
                vv[0] = __funnelshift_r(cur.x[c][0], cur.x[c][1], sh) & mk.x & keep;
                vv[1] = __funnelshift_r(cur.x[c][1], cur.x[c][2], sh) & mk.y & keep;
                vv[2] = __funnelshift_r(cur.x[c][2], cur.x[c][3], sh) & mk.z & keep;
                vv[3] = __funnelshift_r(cur.x[c][3], cur.x[c][4], sh) & mk.w & keep;
                st_shared_v4(dst + (static_cast<uint32_t>((parity + kGatherParities * c) ^ (row & 7)) << 4), vv);
            }
            if (border) {
#pragma unroll
                for (int c = 0; c < kCh; ++c) {
                    const int sc = cur.src[c];
                    if (sc != kNone && !(sc >= 4 && sc <= xbytes - 24))
                        gather_border_chunk(p.gx, xbytes, sc, cur.lo - cur.offs[c], cur.hi - cur.offs[c],
                                            dst + (static_cast<uint32_t>((parity + kGatherParities * c) ^ (row & 7)) << 4));
                }
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_full + 8u * s);
            if (++s == static_cast<uint32_t>(p.stages)) { s = 0; phase ^= 1u; }
        }
        }
    } else if (warp < 2 + kEpiWarps) {
        // ------------------------------------------------------------ epilogue
        const int q = warp & 3;
        int t = 0;
        // Chunks stored so far.  The two staging buffers of the asynchronous store paths alternate with this
        // running count, not with the chunk's position in its tile: a tile with an odd number of chunks would
        // otherwise hand the same buffer to two consecutive copies, the second overwriting what the first may
        // still be reading.
        uint32_t chunk_no = 0;
#ifdef MIPGEMM_TRACE
        // (trace builds: CTA 0's first epilogue warp, summed in registers and written once)
        long long acc_e_wait = 0, acc_e_body = 0, n_e_tiles = 0;
        const long long e_role_t0 = clock64();
#endif
        for (int unit = first_unit; unit < total_units; unit += unit_stride, ++t) {
            const TileCoord tc = decode_unit(p, unit, kRowsPerTile);
            const uint32_t acc = t & 1, acc_phase = (t >> 1) & 1;
#ifdef MIPGEMM_TRACE
            const long long tt0 = clock64();
#endif
            bool gave_up = !mbar_wait(bar_tfull + 8u * acc, acc_phase, abort_flag, budget);
            // Each warp waits on its own clock, but slab stores meet at named barriers: the four warps decide
            // together whether to go on, so none can leave while another still expects it there.
            if (p.c_mode == 1 && p.cluster_split <= 1) gave_up = named_bar_or(1, 128, gave_up);
            if (gave_up) break;
#ifdef MIPGEMM_TRACE
            const long long tt1 = clock64();
            acc_e_wait += tt1 - tt0; ++n_e_tiles;
#endif
            if (t == 0 && warp == 2) MIP_STAMP(5);
            tc_fence_after();
            const int m_cta = tc.m0 + static_cast<int>(cta_rank) * kBlockM;
            const int row = m_cta + q * 32 + lane;
            const int n_rem = p.N - tc.n0;
            const int n_here = min(p.block_n, n_rem);
            if (p.cluster_split > 1) {
                // the accumulator stays in tensor memory; the cluster reduces it below
            } else if (p.c_mode == 1 || m_cta + q * 32 < p.M) {   // (slab stores need all four warps)
                const long long c_off = static_cast<long long>(tc.batch) * p.stride_c;
                int32_t* crow = p.C + c_off + static_cast<long long>(row) * p.ldc + tc.n0;
                uint8_t* crow8 = kQ8 ? reinterpret_cast<uint8_t*>(p.C) + static_cast<long long>(row) * p.ldc + tc.n0 : nullptr;
                const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * p.block_n;
                const uint32_t my_staging = staging + static_cast<uint32_t>(q) * 8192u;
                // two register buffers: the TMEM load of the next chunk is in flight while the
                // current one is written out
                uint32_t va[32], vb[32];
                if (kQ8 && p.c_mode == 4) {
                    // 8-bit codes: this warp's chunks are `step` columns apart (the other warp of the
                    // lane quarter takes the ones in between when there are eight epilogue warps)
                    constexpr int step = kEpiWarps == 8 ? 64 : 32;
                    int c0 = kEpiWarps == 8 ? ((warp - 2) >> 2) * 32 : 0;
                    if (c0 < n_here) tmem_ld_32x32(t_row + c0, va);
                    for (; c0 < n_here; c0 += 2 * step) {
                        tmem_ld_wait();
                        if (c0 + step < n_here) tmem_ld_32x32(t_row + c0 + step, vb);
                        if (p.bias) add_bias_chunk(p, va, tc.n0 + c0);
                        if (row < p.M) store_q8_chunk(p, crow8 + c0, va, min(32, n_here - c0));
                        if (c0 + step < n_here) {
                            tmem_ld_wait();
                            if (c0 + 2 * step < n_here) tmem_ld_32x32(t_row + c0 + 2 * step, va);
                            if (p.bias) add_bias_chunk(p, vb, tc.n0 + c0 + step);
                            if (row < p.M) store_q8_chunk(p, crow8 + c0 + step, vb, min(32, n_here - c0 - step));
                        }
                    }
                } else if (kGather) {
                    // (768 threads leave 80 registers per thread: one register buffer, no look-ahead)
                    for (int c0 = 0; c0 < n_here; c0 += 32) {
                        tmem_ld_32x32(t_row + c0, va);
                        tmem_ld_wait();
                        if (p.out_f32) dequant_chunk(p, va, tc.n0 + c0);
                        if (p.c_mode == 1) tma_store_slab(p, staging + (chunk_no & 1u) * 16384u, va, lane, q, warp == 2, tc.n0 + c0, m_cta, tc.batch);
                        else if (p.c_mode == 3) coalesced_chunk(p, my_staging + (chunk_no & 1u) * 4096u, va, lane, m_cta + q * 32, tc.n0 + c0, c_off);
                        else if (p.c_mode == 5) rows_chunk(p, my_staging, va, lane, m_cta + q * 32, tc.n0 + c0, c_off);
                        else if (row < p.M) store_chunk(p, crow + c0, va, min(32, n_here - c0));
                        ++chunk_no;
                    }
                } else {
                tmem_ld_32x32(t_row, va);
                for (int c0 = 0; c0 < n_here; c0 += 64) {
#ifdef MIPGEMM_TRACE
                    const long long tw0 = clock64();
#endif
                    tmem_ld_wait();
#ifdef MIPGEMM_TRACE
                    if (p.trace && (p.debug_flags & 128) && blockIdx.x == 0 && threadIdx.x == 64) { p.trace[57] += clock64() - tw0; p.trace[58] += 1; }
#endif
                    if (c0 + 32 < n_here) tmem_ld_32x32(t_row + c0 + 32, vb);
                    if (p.out_f32) dequant_chunk(p, va, tc.n0 + c0);
                    if (p.c_mode == 1) tma_store_slab(p, staging + (chunk_no & 1u) * 16384u, va, lane, q, warp == 2, tc.n0 + c0, m_cta, tc.batch);
                    else if (p.c_mode == 3) coalesced_chunk(p, my_staging, va, lane, m_cta + q * 32, tc.n0 + c0, c_off);
                    else if (p.c_mode == 2) tma_reduce_chunk(p, my_staging + (chunk_no & 1u) * 4096u, va, lane, tc.n0 + c0, m_cta + q * 32);
                    else if (p.c_mode == 5) rows_chunk(p, my_staging, va, lane, m_cta + q * 32, tc.n0 + c0, c_off);
                    else if (row < p.M) store_chunk(p, crow + c0, va, min(32, n_here - c0));
                    ++chunk_no;
                    if (c0 + 32 < n_here) {
                        tmem_ld_wait();
                        if (c0 + 64 < n_here) tmem_ld_32x32(t_row + c0 + 64, va);
                        if (p.out_f32) dequant_chunk(p, vb, tc.n0 + c0 + 32);
                        if (p.c_mode == 1) tma_store_slab(p, staging + (chunk_no & 1u) * 16384u, vb, lane, q, warp == 2, tc.n0 + c0 + 32, m_cta, tc.batch);
                        else if (p.c_mode == 3) coalesced_chunk(p, my_staging + 4096u, vb, lane, m_cta + q * 32, tc.n0 + c0 + 32, c_off);
                        else if (p.c_mode == 2) tma_reduce_chunk(p, my_staging + (chunk_no & 1u) * 4096u, vb, lane, tc.n0 + c0 + 32, m_cta + q * 32);
                        else if (p.c_mode == 5) rows_chunk(p, my_staging + 4096u, vb, lane, m_cta + q * 32, tc.n0 + c0 + 32, c_off);
                        else if (row < p.M) store_chunk(p, crow + c0 + 32, vb, min(32, n_here - c0 - 32));
                        ++chunk_no;
                    }
                }
                }
            }
            if (warp == 2) { if (t == 0) MIP_STAMP(6); MIP_STAMP(7); }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (kPair && !leader) mbar_arrive_remote(bar_tempty + 8u * acc, 0);
                else mbar_arrive(bar_tempty + 8u * acc);
            }
#ifdef MIPGEMM_TRACE
            acc_e_body += clock64() - tt1;
#endif
        }
#ifdef MIPGEMM_TRACE
        if (p.trace && blockIdx.x == 0 && threadIdx.x == 64) {
            p.trace[59] = acc_e_wait; p.trace[60] = n_e_tiles; p.trace[61] = acc_e_body; p.trace[62] = clock64() - e_role_t0;
        }
#endif
        // every tile copy issued by this warp must be complete before the CTA may exit
        if (p.cluster_split <= 1 && (p.c_mode == 2 || (p.c_mode == 1 && warp == 2)) && elect_one())
            tma_store_wait<0>();
    }

    if (!kPair && p.cluster_split > 1) {
        // ---------------------------------------------------------------- cluster split-K
        // The S CTAs of a cluster hold partial sums of the same tile (one K share each) in
        // their tensor memories.  Reduce-scatter through distributed shared memory: CTA r owns
        // the r-th slice of the tile's columns; every CTA sends its partial of slice d to CTA
        // d, which adds the S partials (exact integer adds, any order) and stores its slice.
        // The receive buffers alias the pipeline stages, hence the first cluster barrier: it
        // completes only when every CTA's epilogue warps have seen their accumulator ready,
        // i.e. when no MMA in the cluster can still read stage memory.
        const uint32_t S = static_cast<uint32_t>(p.cluster_split);
        const uint32_t rank = cluster_ctarank();
        const int slice_cols = p.block_n / static_cast<int>(S);
        const int chunks = slice_cols >> 5;
        const int q = warp & 3;
        const int r_tile = q * 32 + lane;                       // this thread's row of the tile
        const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
        const TileCoord tc = decode_unit(p, first_unit, kRowsPerTile);
        tc_fence_before();
        cluster_arrive();
        cluster_wait();
        tc_fence_after();
        if (warp >= 2 && warp < 2 + kEpiWarps && *abort_flag == 0) {
            for (uint32_t d = 0; d < S; ++d) {
                if (d == rank) continue;
                const uint32_t slot = rank < d ? rank : rank - 1;            // my slot among d's S-1 senders
                for (int c = 0; c < chunks; ++c) {
                    uint32_t v[32];
                    tmem_ld_32x32(t_row + d * slice_cols + c * 32, v);
                    tmem_ld_wait();
                    const uint32_t local = smem_base + ((slot * chunks + c) * 128u + r_tile) * 128u;
                    const uint32_t remote = mapa_u32(local, d);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};"
                                     ::"r"(remote + (static_cast<uint32_t>(j ^ (r_tile & 7)) << 4)), "r"(v[4 * j]),
                                       "r"(v[4 * j + 1]), "r"(v[4 * j + 2]), "r"(v[4 * j + 3]) : "memory");
                }
            }
        }
        cluster_arrive();
        cluster_wait();
        if (warp >= 2 && warp < 2 + kEpiWarps && *abort_flag == 0) {
            const int m_cta = tc.m0;
            const int row = m_cta + r_tile;
            const uint32_t my_staging = staging + static_cast<uint32_t>(q) * 8192u;
            for (int c = 0; c < chunks; ++c) {
                const int col0 = tc.n0 + static_cast<int>(rank) * slice_cols + c * 32;
                if (col0 >= p.N) break;                                     // uniform over the CTA
                uint32_t v[32];
                tmem_ld_32x32(t_row + rank * slice_cols + c * 32, v);
                tmem_ld_wait();
                for (uint32_t slot = 0; slot + 1 < S; ++slot) {
                    const uint32_t src = smem_base + ((slot * chunks + c) * 128u + r_tile) * 128u;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        uint32_t x[4];
                        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                     : "=r"(x[0]), "=r"(x[1]), "=r"(x[2]), "=r"(x[3])
                                     : "r"(src + (static_cast<uint32_t>(j ^ (r_tile & 7)) << 4)) : "memory");
#pragma unroll
                        for (int e = 0; e < 4; ++e) v[4 * j + e] += x[e];
                    }
                }
                if (p.out_f32) dequant_chunk(p, v, col0);
                if (p.c_mode == 1) tma_store_slab(p, staging + (c & 1) * 16384u, v, lane, q, warp == 2, col0, m_cta);
                else if (p.c_mode == 3) coalesced_chunk(p, my_staging + (c & 1) * 4096u, v, lane, m_cta + q * 32, col0);
                else if (p.c_mode == 5) rows_chunk(p, my_staging + (c & 1) * 4096u, v, lane, m_cta + q * 32, col0, 0);
                else if (row < p.M) store_chunk(p, p.C + static_cast<long long>(row) * p.ldc + col0, v, min(32, p.N - col0));
            }
            if (p.c_mode == 1 && warp == 2 && elect_one()) tma_store_wait<0>();
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag != 0) {
        // Unwinding (uniform: every role has left its loop, so nobody writes the flag any more).  Some role gave
        // up a wait; whatever is still on its way to this CTA must arrive before shared and tensor memory are
        // given back, whichever role it was that gave up:
        //  * the producer warp waits (bounded) until the copies of the last `stages` k-blocks it issued have
        //    landed (a peer CTA cannot observe its own copies -- they complete on the leader's barrier; it is
        //    held by the cluster barrier below until the leader has finished here);
        //  * the MMA warp lets every MMA it issued retire (one more commit, bounded wait).
        if (kGather && warp == 0 && p.g_staged) {       // image rows requested for the last two tiles
            for (uint32_t i = 1; i <= min(rows_tiles, 2u); ++i) {
                const uint32_t t = rows_tiles - i;
                const uint64_t t0 = globaltimer_ns();
                while (!mbar_try_wait(bar_rows_full + 8u * (t & 1u), (t >> 1) & 1u)) {
                    if (globaltimer_ns() - t0 > budget) break;
                }
            }
        }
        if (warp == 0 && leader) {
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
        if (warp == 1 && leader) {
            if (elect_one()) {
                if (kPair) mma_commit_pair(bar_drain); else mma_commit(bar_drain);
            }
            const uint64_t t0 = globaltimer_ns();
            while (!mbar_try_wait(bar_drain, 0)) {
                if (globaltimer_ns() - t0 > budget) break;
            }
            tc_fence_before();
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) MIP_STAMP(8);
    if (kPair) {   // neither CTA may leave while the other can still reach its shared memory
        cluster_arrive();
        cluster_wait();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc<kGroup>(tmem_base, p.tmem_cols);
    }
    if (threadIdx.x == 0) MIP_STAMP(9);
    if (threadIdx.x == 0 && *abort_flag != 0) atomicOr(p.status, 1u);
}

cudaError_t dense_init() {
    cudaError_t e = cudaFuncSetAttribute(mip_dense_kernel<false, false, false, false>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(mip_dense_kernel<false, true, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSmemBudget);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(mip_dense_kernel<true, false, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSmemBudget);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(mip_dense_kernel<true, true, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSmemBudget);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(mip_dense_kernel<false, false, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSmemBudget);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(mip_dense_kernel<false, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSmemBudget);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(mip_dense_kernel<true, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSmemBudget);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(mip_dense_kernel<false, false, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSmemBudget);
    return e;
}

// All launches allow programmatic stream serialisation (see pdl_wait() in the kernel).
static void pdl_attribute(cudaLaunchAttribute& a) {
    a.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    a.val.programmaticStreamSerializationAllowed = pdl_allowed();
}

cudaError_t launch_dense(const DenseParams& p, int grid, size_t smem_bytes, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
    cfg.blockDim = dim3(kDenseThreads, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    pdl_attribute(attr[0]);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // (the M-/N-contiguous operand forms live in an instantiation of their own, so the common
    // kernel's issue loops carry none of their address arithmetic)
    if (p.a_mn || p.b_mn) return cudaLaunchKernelEx(&cfg, mip_dense_kernel<false, true, false, false>, p);
    // (so do the 8-bit-code epilogue and the gather form)
    if (p.out_q8) {
        cfg.blockDim = dim3(kDenseQ8Threads, 1, 1);
        return cudaLaunchKernelEx(&cfg, mip_dense_kernel<false, false, false, true>, p);
    }
    return cudaLaunchKernelEx(&cfg, mip_dense_kernel<false, false, false, false>, p);
}

// One CTA per tile with additional warps (4 * kGatherParities) that gather operand A from an image batch.
cudaError_t launch_dense_gather(const DenseParams& p, int grid, size_t smem_bytes, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
    cfg.blockDim = dim3(kGatherThreads, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    pdl_attribute(attr[0]);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (p.out_q8) return cudaLaunchKernelEx(&cfg, mip_dense_kernel<false, false, true, true>, p);
    return cudaLaunchKernelEx(&cfg, mip_dense_kernel<false, false, true, false>, p);
}

// One-CTA-per-tile kernel launched in clusters of `cluster` CTAs (cluster split-K); `grid` is a
// multiple of `cluster`.
cudaError_t launch_dense_cluster(const DenseParams& p, int grid, int cluster, size_t smem_bytes,
                                 cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
    cfg.blockDim = dim3(kDenseThreads, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(cluster);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    pdl_attribute(attr[1]);
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, mip_dense_kernel<false, false, false, false>, p);
}

// `grid` counts CTAs and must be even: consecutive CTAs form a cluster of two.
cudaError_t launch_dense_pair(const DenseParams& p, int grid, size_t smem_bytes, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
    cfg.blockDim = dim3(kDenseThreads, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    pdl_attribute(attr[1]);
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (p.a_mn || p.b_mn) return cudaLaunchKernelEx(&cfg, mip_dense_kernel<true, true, false, false>, p);
    if (p.out_q8) {
        cfg.blockDim = dim3(kDenseQ8Threads, 1, 1);
        return cudaLaunchKernelEx(&cfg, mip_dense_kernel<true, false, false, true>, p);
    }
    return cudaLaunchKernelEx(&cfg, mip_dense_kernel<true, false, false, false>, p);
}

// Largest number of co-resident 2-CTA clusters for the pair kernel (0 on failure).
int dense_pair_max_clusters(size_t smem_bytes) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2, 1, 1);
    cfg.blockDim = dim3(kDenseThreads, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, mip_dense_kernel<true, false, false, false>, &cfg) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    return n;
}

}  // namespace mip
