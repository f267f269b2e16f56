// Host-side declarations shared by the translation units of libmipgemm.
#pragma once
#include <cstddef>
#include <cstdint>
#include <cstdlib>
#include <cuda.h>
#include <cuda_runtime.h>

namespace mip {

// Programmatic dependent launch may be switched off for experiments (MIPGEMM_NO_PDL=1): every launch then
// waits for its predecessor in the stream to complete before any of its blocks starts.
inline int pdl_allowed() {
    static const int v = [] { const char* e = std::getenv("MIPGEMM_NO_PDL"); return (e && std::atoi(e)) ? 0 : 1; }();
    return v;
}

// Integer environment variable read once per name (experiment switches; `fallback` when unset).
inline int env_int(const char* name, int fallback) {
    const char* e = std::getenv(name);
    return e ? std::atoi(e) : fallback;
}

// Experiment switch: read once, or on every call when MIPGEMM_LIVE_ENV=1 (A/B runs inside one process;
// cached plans are bypassed then).
inline bool live_env() {
    static const bool v = env_int("MIPGEMM_LIVE_ENV", 0) != 0;
    return v;
}
#define MIP_ENV_KNOB(name, fallback) \
    ([]() -> int { static const int cached = ::mip::env_int(name, fallback); \
                   return ::mip::live_env() ? ::mip::env_int(name, fallback) : cached; }())

constexpr int kBlockM = 128;          // rows of C per CTA (TMEM lanes)
constexpr int kDenseThreads = 224;    // producer warp (A), MMA warp, 4 epilogue warps, producer warp (B)
constexpr int kDenseQ8Threads = 320;  // 8-bit-code epilogue: one producer warp, MMA warp, 8 epilogue warps
// Gather form of the dense kernel: 4 * kGatherParities more warps build operand A from an image;
// warp w of them takes rows 32*(w%4).. of the tile and every kGatherParities-th 16-byte chunk.
constexpr int kGatherParities = 4;
constexpr int kGatherFirstWarp = 8;
constexpr int kGatherThreads = 32 * (kGatherFirstWarp + 4 * kGatherParities);
constexpr int kMaxStages = 12;
constexpr int kCtrlBytes = 512;       // barriers + TMEM slot + abort word
constexpr int kStagingBytes = 4 * 2 * 4096;   // epilogue: 4 warps x 2 buffers x (32 rows x 128 B)
#ifdef MIPGEMM_TRACE
constexpr int kSmemBudget = 226 * 1024;   // leaves room for the static trace array
#else
constexpr int kSmemBudget = 227 * 1024;
#endif

// Everything the dense kernel needs; passed by value as a __grid_constant__.
struct alignas(64) DenseParams {
    CUtensorMap tmap_a;      // tiled {K, M} byte tensor, or im2col-mode NHWC tensor
    CUtensorMap tmap_b;      // tiled {K, N} byte tensor (weights, K contiguous)
    CUtensorMap tmap_c;      // tiled {N, M} int32 tensor: 32 x 128 boxes (c_mode 1) or 32 x 32 boxes (c_mode 2)
    int32_t* C;
    long long ldc;
    int M, N;
    int k_blocks;            // ceil(K / block_k)
    int block_n;             // multiple of 32, <= 256
    int block_k;             // bytes of K per pipeline stage: 128 (SWIZZLE_128B) or 64 (SWIZZLE_64B)
    int stages;
    int tiles_m, tiles_n;
    int split_k, kb_per_split;
    int a_mn, b_mn;          // 1: that operand is M- / N-contiguous in memory (k-block 128, one CTA per tile)
    int batch;               // > 1: strided batch; the tensor maps are rank 3 (z = batch index)
    long long stride_c;      // elements between consecutive C matrices of a batch
    int cluster_split;       // > 1: the split_k CTAs sharing a tile form a cluster and reduce through DSMEM
    int group_n;             // n-tiles per rasterisation group
    int raster;              // bit 0: serpentine (odd groups are swept bottom to top)
    int accumulate;          // epilogue adds the incoming C
    int use_red;             // epilogue reduces with red.global.add (split-K)
    int store_vec;           // 8, 4 or 1 int32 per store instruction
    int out_f32;             // 1: the epilogue writes float32 scale * sum instead of the int32 sum
    float out_scale;
    int out_q8;              // 1: the epilogue writes 8-bit codes min(max(rne(scale * sum), q_lo), q_hi); C and ldc
    int q_lo, q_hi;          //    then address bytes (c_mode 4)
    const int32_t* bias;     // optional, length N: added to the exact sums before the output transform
    int c_mode;              // 0: row-per-thread stores (any alignment); 1: TMA tile stores of 128 x 32 slabs -- tile
                             // reduce-adds when `accumulate` is set; 2: TMA tile reduce-add of 32 x 32 boxes (explicit
                             // split-K); 3: 16-byte pieces through a transposing shared-memory buffer; 4: 8-bit codes,
                             // row-per-thread; 5: rows through shared memory, 4-byte accesses, one 128-byte run per
                             // instruction (any alignment; `accumulate` adds at the L2 with red.global.add).
                             // 1, 2 and 3 need a 16-byte aligned C base and ldc % 4 == 0, 1 and 2 also N % 4 == 0
    uint32_t idesc;          // tcgen05 instruction descriptor
    uint32_t tmem_cols;      // power of two >= 2*block_n
    // implicit im2col (operand A gathered by TMA im2col loads)
    int a_im2col;
    int conv_wo, conv_howo, conv_s, c_chunks;
    int stride_w, stride_h, pad_w, pad_h, dil_w, dil_h;
    // software-gathered im2col (operand A built in shared memory by extra warps; for images
    // whose channel count TMA cannot address).  A row of A is R slots of g_slot bytes; slot r is
    // a copy of the g_slot input bytes that start at the window's first pixel in filter row r
    // (the first g_seg = S*Cin of them are real taps, the rest meet zero weights).
    int a_gather;
    const uint8_t* gx;       // NHWC image batch
    long long g_xbytes;      // its size (loads never leave [gx, gx + g_xbytes))
    int g_h, g_row_bytes;    // image rows, bytes per image row (W * Cin)
    int g_cin, g_seg, g_slot;
    int g_chunks;            // 16-byte chunks per row of A (R * g_slot / 16)
    // staged form of the gather (image rows are multiples of 16 bytes and few enough fit shared memory): the
    // producer warp copies the input rows a tile needs into one of two row buffers with bulk copies, and the
    // gather warps realign from shared memory instead of from global memory.  Output row o of the tile
    // (o = 0 .. g_rows_max-1) owns g_span = (R-1)*dil_h + 1 consecutive slots of g_row_bytes.
    int g_staged;
    int g_span, g_rows_max;
    int g_rowbuf_stride;     // bytes between the two row buffers (payload + guard bytes, multiple of 128)
    int g_table_bytes;       // chunk table behind the row buffers: 8 bytes per 16-byte chunk of a (padded) row of A
    int g_r, g_ho;           // filter rows, output rows per image
    // exact division of any n < 2^31 by Wo and by Ho without a divide: q = (umulhi(mul, n) + n) >> shift
    uint32_t g_wo_mul, g_wo_shift, g_ho_mul, g_ho_shift;
    unsigned int* status;    // device word, bit 0 set when a bounded wait expired
    unsigned long long wait_budget_ns;
    int debug_flags;         // test hook (mipgemm_debug_set): bit 0 = never signal "accumulator ready"
    unsigned long long* trace;   // timeline stamps of CTA 0; only read by builds with -DMIPGEMM_TRACE
};

cudaError_t launch_dense_gather(const DenseParams& p, int grid, size_t smem_bytes, cudaStream_t stream);
cudaError_t launch_dense(const DenseParams& p, int grid, size_t smem_bytes, cudaStream_t stream);
cudaError_t launch_dense_cluster(const DenseParams& p, int grid, int cluster, size_t smem_bytes, cudaStream_t stream);
cudaError_t launch_dense_pair(const DenseParams& p, int grid, size_t smem_bytes, cudaStream_t stream);
int dense_pair_max_clusters(size_t smem_bytes);
cudaError_t dense_init();  // opt in to large dynamic shared memory (once per device)

// Skinny-M streaming kernel (M <= 16).
struct SkinnyParams {
    const void* A; long long lda;
    const int8_t* B; long long ldb;
    int32_t* C; long long ldc;
    int M, N, K;
    int a_unsigned, accumulate;
    int out_f32; float out_scale;   // fused dequantisation (see DenseParams)
};
cudaError_t launch_skinny(const SkinnyParams& p, cudaStream_t stream);
bool skinny_supported(const SkinnyParams& p);

// Ring form of the skinny kernel (weights streamed through a TMA-fed shared-memory ring).
struct alignas(64) SkinnyRingParams {
    CUtensorMap tmap_b;      // rank-3 byte tensor {128, N, K/128}, strides {ldb, 128}, box {128, 16, 8}
    const void* A; long long lda;
    int32_t* C; long long ldc;
    int M, N, K;
    int a_unsigned, accumulate;
    int out_f32; float out_scale;   // fused dequantisation (see DenseParams)
    int pdl_mode;                // 1: launched with programmatic stream serialisation (filled in by the launcher)
    int b_constant;              // 1: B may be fetched before the previous kernel on the stream has completed
    int slots, tokens_in_smem;   // filled in by the launcher
    int prefetch_chunks;         // 16 KB chunks of B each CTA asks the L2 for before the dependency wait (no promise)
    unsigned int* status;
    unsigned long long wait_budget_ns;
    int debug_flags;             // test hook (mipgemm_debug_set): bit 0 = the first CTA never loads its second chunk
    unsigned long long* trace;   // timeline stamps of the first and last CTA; only read by builds with -DMIPGEMM_TRACE
};
bool skinny_ring_supported(const SkinnyParams& p, int sm_count);
cudaError_t skinny_ring_init();  // once per device
cudaError_t launch_skinny_ring(const SkinnyRingParams& p, int sm_count, cudaStream_t stream);
// Ring form for 9 to 16 tokens (chunk-major walk, token chunks streamed through two buffers).
bool skinny_ring16_supported(const SkinnyParams& p, int sm_count);
cudaError_t skinny_ring16_init();  // once per device
cudaError_t launch_skinny_ring16(const SkinnyRingParams& p, int sm_count, cudaStream_t stream);

// Auxiliary kernels.
cudaError_t launch_repack(const void* src, long long src_pitch, void* dst, long long dst_pitch,
                          long long rows, long long cols, cudaStream_t stream);
cudaError_t launch_repack2(const void* src0, long long src_pitch0, void* dst0, long long rows0, const void* src1,
                           long long src_pitch1, void* dst1, long long rows1, long long dst_pitch, long long cols,
                           cudaStream_t stream);
cudaError_t launch_transpose_repack(const void* src, long long src_pitch, void* dst, long long dst_pitch,
                                    long long rows_out, long long cols_out, cudaStream_t stream);
// Weights [rows][R][seg] -> [rows][R][slot], zero padded (slot >= seg, slot % 16 == 0).
cudaError_t launch_weight_slots(const int8_t* src, int8_t* dst, long long rows, int R, int seg, int slot,
                                cudaStream_t stream);
cudaError_t launch_fill_zero(int32_t* C, long long ldc, long long M, long long N, cudaStream_t stream);
cudaError_t launch_bias_rows(void* out, long long ld, long long M, long long N, const int32_t* bias, int q8,
                             float scale, int q_lo, int q_hi, cudaStream_t stream);
struct Im2colParams {
    const uint8_t* X; uint8_t* out;
    long long Nb, H, W, Cin, Ho, Wo;
    int R, S, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w;
    long long k_real, k_pitch;   // R*S*Cin and its padded pitch (pad bytes are zero-filled)
};
cudaError_t launch_im2col(const Im2colParams& p, cudaStream_t stream);
cudaError_t launch_probe(int iters, int grid, int32_t* sink, cudaStream_t stream);

}  // namespace mip
