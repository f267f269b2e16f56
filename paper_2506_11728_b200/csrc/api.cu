// C-ABI entry points of libmipgemm: argument validation, path selection, tensor-map
// construction, scratch-memory handling and kernel launches.  No arithmetic of the
// method happens on the host.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <atomic>
#include <map>
#include <mutex>

#include "../../include/mipgemm.h"
#include "internal.h"

namespace {

using namespace mip;

thread_local int tl_last_path = MIPGEMM_PATH_NONE;
thread_local int tl_last_cuda_error = 0;
// Output transform of the call in progress on this thread (set by the *_dequant entry points).
thread_local int tl_out_f32 = 0;
thread_local float tl_out_scale = 1.0f;
// ... or requantisation to 8-bit codes (the *_requant entry points): clamp bounds; C then holds bytes
thread_local int tl_out_q8 = 0, tl_q_lo = 0, tl_q_hi = 0;
// ... and the optional per-output-channel bias of the *_bias entry points (device pointer, length N)
thread_local const int32_t* tl_bias = nullptr;

// Experiment overrides (mipgemm_set_tuning).  The four values travel in one atomic word, so a call
// that runs while another thread changes them sees either the old set or the new one, never a mix.
struct Tuning {
    int block_n = 0, stages = 0, split_k = 0, force_path = 0;
};
std::atomic<uint64_t> g_tuning_word{0};
std::atomic<uint32_t> g_tuning_epoch{0};   // bumped by every change (cached plans remember it)
uint64_t pack_tuning(const Tuning& t) {
    return static_cast<uint64_t>(t.block_n & 0xFFFF) | (static_cast<uint64_t>(t.stages & 0xFF) << 16) |
           (static_cast<uint64_t>(t.split_k & 0xFFFF) << 24) | (static_cast<uint64_t>(t.force_path & 0xFFFFFF) << 40);
}
Tuning tuning_now() {
    const uint64_t w = g_tuning_word.load(std::memory_order_acquire);
    Tuning t;
    t.block_n = static_cast<int>(w & 0xFFFF);
    t.stages = static_cast<int>((w >> 16) & 0xFF);
    t.split_k = static_cast<int>((w >> 24) & 0xFFFF);
    t.force_path = static_cast<int>((w >> 40) & 0xFFFFFF);
    return t;
}
bool g_tuning_no_cluster_split = false;  // MIPGEMM_NO_CLUSTER_SPLIT=1: split-K through zero fill + TMA reduce-add
bool g_tuning_no_skinny_ring = false;    // MIPGEMM_NO_SKINNY_RING=1: always the register form of the skinny kernel
bool g_tuning_no_tma_store = false;   // MIPGEMM_DIRECT_STORE=1: force the direct-store epilogue
std::atomic<uint64_t> g_launches{0};
// Limit of every device-side wait and the test-hook bits handed to the kernels (mipgemm_debug_set).
std::atomic<unsigned long long> g_wait_budget_ns{4000000000ull};
std::atomic<int> g_debug_flags{0};
std::atomic<int> g_weights_constant{0};  // mipgemm_set_weights_constant

// Address ranges the caller has declared constant (mipgemm_register_constant_weights): start -> end.
std::map<uintptr_t, uintptr_t> g_constant_ranges;
std::atomic<int> g_constant_range_count{0};
std::mutex g_ranges_mutex;
bool inside_constant_range(const void* ptr, size_t bytes) {
    if (g_constant_range_count.load(std::memory_order_acquire) == 0) return false;
    const uintptr_t lo = reinterpret_cast<uintptr_t>(ptr), hi = lo + bytes;
    std::lock_guard<std::mutex> lock(g_ranges_mutex);
    auto it = g_constant_ranges.upper_bound(lo);     // first range that starts after lo
    if (it == g_constant_ranges.begin()) return false;
    --it;
    return it->first <= lo && hi <= it->second;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const int*, const int*, cuuint32_t, cuuint32_t,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int kMaxDevices = 64;
constexpr int kHostBlocks = 8;                                    // host-buffer calls: up to 8 x 8 blocks of C
constexpr int kHostEvents = 2 * kHostBlocks + kHostBlocks * kHostBlocks + 3;
struct DeviceState {
    bool ready = false;
    int status = MIPGEMM_OK;
    int sm_count = 0;
    int pair_clusters = 0;                 // co-resident 2-CTA clusters of the pair kernel
    unsigned int* status_word = nullptr;   // device
    cudaStream_t copy_in = nullptr, copy_out = nullptr;   // helper streams of the host-buffer entry points
    std::mutex host_mutex;                 // host-buffer calls on one device run one at a time
    void* staging = nullptr;               // their device staging buffer (grow-only) ...
    size_t staging_bytes = 0;
    cudaEvent_t host_events[kHostEvents] = {};   // ... and their event pool
    bool host_events_ready = false;
    void* lent = nullptr;
    size_t lent_bytes = 0;
};
DeviceState g_dev[kMaxDevices];
std::mutex g_mutex;
EncodeTiledFn g_encode_tiled = nullptr;
EncodeIm2colFn g_encode_im2col = nullptr;

struct NoAllocDevice {
    bool ready = false;
    int status = MIPGEMM_OK;
    DeviceState st;                 // sm_count, pair_clusters, status_word (-> g_static_status)
    unsigned char* scratch = nullptr;   // device address of g_static_scratch on this device
};
NoAllocDevice g_noalloc[kMaxDevices];
std::mutex g_noalloc_mutex;

// MIPGEMM_LOG=1: one line per call on stderr with the dispatch decision.
bool log_enabled() {
    static const bool on = env_int("MIPGEMM_LOG", 0) != 0;
    return on;
}
struct Plan;
void log_dense(const char* what, long long M, long long N, long long K, const Plan& pl, const DenseParams& p, bool hit);

int cuda_fail(cudaError_t e) {
    tl_last_cuda_error = static_cast<int>(e);
    return MIPGEMM_ERR_CUDA;
}

// Reads a device status word and clears it when set (the caller has synchronised the work that may
// have written it).  Returns MIPGEMM_OK, MIPGEMM_ERR_TIMEOUT or MIPGEMM_ERR_CUDA.
int take_status_word(unsigned int* dev_word) {
    unsigned int word = 0;
    cudaError_t e = cudaMemcpy(&word, dev_word, sizeof(word), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e);
    if (word != 0) {
        e = cudaMemset(dev_word, 0, sizeof(word));
        if (e != cudaSuccess) return cuda_fail(e);
        return MIPGEMM_ERR_TIMEOUT;
    }
    return MIPGEMM_OK;
}

// ---- state of the allocation-free entry point (mipgemm_s8s8s32_static_scratch, end of this file)
// The scratch itself.  Host code must never use this name as an address: on the host it is
// only a handle for cudaGetSymbolAddress (see noalloc_device()).
static __device__ __align__(256) unsigned char g_static_scratch[MIPGEMM_STATIC_SCRATCH_BYTES];
// Word that receives the "bounded wait expired" flag of kernels launched from that path; read and
// cleared by mipgemm_static_scratch_status() and by mipgemm_device_status().
static __device__ unsigned int g_static_status;

// Once per device: capability check, driver entry points, kernel attributes, status word.
int get_device(DeviceState** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    // The tensor-map encoders are driver calls and need the device's context current on the calling
    // thread; a host thread that has made no runtime call yet has none (cudaGetDevice does not bind it,
    // cudaSetDevice does).
    thread_local int tl_context_bound = -1;
    if (tl_context_bound != dev) {
        if ((e = cudaSetDevice(dev)) != cudaSuccess) return cuda_fail(e);
        tl_context_bound = dev;
    }
    if (dev < 0 || dev >= kMaxDevices) return MIPGEMM_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState& d = g_dev[dev];
    if (!d.ready) {
        int major = 0, minor = 0;
        if ((e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev)) != cudaSuccess ||
            (e = cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev)) != cudaSuccess ||
            (e = cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
            return cuda_fail(e);
        if (major != 10 || minor != 0) {
            d.status = MIPGEMM_ERR_UNSUPPORTED;
        } else {
            if (!g_encode_tiled) {
                void* fn = nullptr;
                cudaDriverEntryPointQueryResult qr;
                e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr);
                if (e != cudaSuccess || qr != cudaDriverEntryPointSuccess || !fn)
                    return cuda_fail(e == cudaSuccess ? cudaErrorUnknown : e);
                g_encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
                fn = nullptr;
                e = cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &fn, cudaEnableDefault, &qr);
                if (e != cudaSuccess || qr != cudaDriverEntryPointSuccess || !fn)
                    return cuda_fail(e == cudaSuccess ? cudaErrorUnknown : e);
                g_encode_im2col = reinterpret_cast<EncodeIm2colFn>(fn);
            }
            if ((e = dense_init()) != cudaSuccess) return cuda_fail(e);
            if ((e = skinny_ring_init()) != cudaSuccess) return cuda_fail(e);
            if ((e = skinny_ring16_init()) != cudaSuccess) return cuda_fail(e);
            d.pair_clusters = dense_pair_max_clusters(kSmemBudget);
            if (const char* ds = std::getenv("MIPGEMM_DIRECT_STORE")) g_tuning_no_tma_store = std::atoi(ds) != 0;
            if (const char* cs = std::getenv("MIPGEMM_NO_CLUSTER_SPLIT")) g_tuning_no_cluster_split = std::atoi(cs) != 0;
            if (const char* sr = std::getenv("MIPGEMM_NO_SKINNY_RING")) g_tuning_no_skinny_ring = std::atoi(sr) != 0;
            if ((e = cudaMalloc(&d.status_word, sizeof(unsigned int))) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaMemset(d.status_word, 0, sizeof(unsigned int))) != cudaSuccess) return cuda_fail(e);
            // (without them the host-buffer entry points simply do not overlap their copies)
            if (cudaStreamCreateWithFlags(&d.copy_in, cudaStreamNonBlocking) != cudaSuccess) d.copy_in = nullptr;
            if (cudaStreamCreateWithFlags(&d.copy_out, cudaStreamNonBlocking) != cudaSuccess) d.copy_out = nullptr;
            (void)cudaGetLastError();
            d.status = MIPGEMM_OK;
        }
        d.ready = true;
    }
    *out = &d;
    return d.status;
}

// Scratch memory for one call: a slice of the lent buffer, or a stream-ordered allocation.
struct Scratch {
    DeviceState* dev;
    cudaStream_t stream;
    void* base = nullptr;
    size_t size = 0, used = 0;
    bool owned = false;
    Scratch(DeviceState* d, cudaStream_t s) : dev(d), stream(s) {}
    int reserve(size_t bytes) {
        if (bytes == 0) return MIPGEMM_OK;
        if (dev->lent) {
            if (bytes > dev->lent_bytes) return MIPGEMM_ERR_WORKSPACE;
            base = dev->lent;
        } else {
            cudaError_t e = cudaMallocAsync(&base, bytes, stream);
            if (e != cudaSuccess) {
                tl_last_cuda_error = static_cast<int>(e);
                (void)cudaGetLastError();
                return MIPGEMM_ERR_WORKSPACE;
            }
            owned = true;
        }
        size = bytes;
        return MIPGEMM_OK;
    }
    void* take(size_t bytes) {
        void* p = static_cast<char*>(base) + used;
        used += (bytes + 255) & ~static_cast<size_t>(255);
        return p;
    }
    ~Scratch() {
        if (owned && base) (void)cudaFreeAsync(base, stream);
    }
};

size_t align256(size_t b) { return (b + 255) & ~static_cast<size_t>(255); }
long long round_up(long long v, long long m) { return (v + m - 1) / m * m; }
bool aligned16(const void* p, long long pitch) {
    return reinterpret_cast<uintptr_t>(p) % 16 == 0 && pitch % 16 == 0;
}

int encode_tiled_2d(CUtensorMap* map, const void* base, long long inner, long long outer, long long pitch,
                    int box_inner, int box_outer) {
    cuuint64_t dims[2] = {static_cast<cuuint64_t>(inner), static_cast<cuuint64_t>(outer)};
    cuuint64_t strides[1] = {static_cast<cuuint64_t>(pitch)};
    cuuint32_t box[2] = {static_cast<cuuint32_t>(box_inner), static_cast<cuuint32_t>(box_outer)};
    cuuint32_t estr[2] = {1, 1};
    const CUtensorMapSwizzle sw = box_inner == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
    CUresult r = g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides,
                                box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        tl_last_cuda_error = 100000 + static_cast<int>(r);
        return MIPGEMM_ERR_CUDA;
    }
    return MIPGEMM_OK;
}

struct ConvGeom {
    long long Nb, H, W, Cin, Cout, Ho, Wo;
    int R, S, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w;
};

int encode_im2col(CUtensorMap* map, const void* X, const ConvGeom& g, int channels_per_pixel,
                  int pixels_per_column) {
    cuuint64_t dims[4] = {static_cast<cuuint64_t>(g.Cin), static_cast<cuuint64_t>(g.W),
                          static_cast<cuuint64_t>(g.H), static_cast<cuuint64_t>(g.Nb)};
    cuuint64_t strides[3] = {static_cast<cuuint64_t>(g.Cin), static_cast<cuuint64_t>(g.W * g.Cin),
                             static_cast<cuuint64_t>(g.H * g.W * g.Cin)};
    int lower[2] = {-g.pad_w, -g.pad_h};
    int upper[2] = {g.pad_w - (g.S - 1) * g.dil_w, g.pad_h - (g.R - 1) * g.dil_h};
    cuuint32_t estr[4] = {1, static_cast<cuuint32_t>(g.stride_w), static_cast<cuuint32_t>(g.stride_h), 1};
    const CUtensorMapSwizzle sw =
        channels_per_pixel == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
    CUresult r = g_encode_im2col(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(X), dims, strides,
                                 lower, upper, static_cast<cuuint32_t>(channels_per_pixel),
                                 static_cast<cuuint32_t>(pixels_per_column), estr,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        tl_last_cuda_error = 100000 + static_cast<int>(r);
        return MIPGEMM_ERR_CUDA;
    }
    return MIPGEMM_OK;
}

uint32_t pow2_at_least(uint32_t v) {
    uint32_t p = 32;
    while (p < v) p <<= 1;
    return p;
}

// Tile width, pipeline depth and split-K for an M x N x K problem (k-block = block_k bytes).
struct Plan {
    int cluster_split;   // > 1: split_k CTAs of a tile form a cluster and reduce through DSMEM
    int pair;   // 1: CTA pairs share 256-row tiles (cta_group::2)
    int block_n, stages, split_k, kb_per_split, k_blocks, tiles_m, tiles_n;
};

// Cost model behind the plan (clocks, calibrated on B200 with CUDA-graph timings of this
// kernel).  One 128-byte k-block of a 128 x bn tile costs what the slower of the tensor pipe
// (2*bn clk) and the SM's ~64 B/clk ingest from L2 allows; CTA pairs stage only half of B per
// CTA.  The epilogue of a tile hides behind the next tile's main loop as far as the store pace
// allows (see below); the last one (350 clk per 32-column chunk) is exposed.  A launch carries ~3.7 us of fixed cost (launch gap,
// set-up, pipeline fill, store drain); the DSMEM exchange of a cluster split-K costs about
// 2.5 / 6 / 13 us for 2 / 4 / 8 CTAs (measured), so it only pays for K-heavy, tile-poor shapes.
double plan_cost_us(int pair, int bn, int split, long long M, long long N, int k_blocks, int block_k,
                    const DeviceState* dev) {
    const double scale = block_k / 128.0;
    const double kb_clk = (pair ? 300.0 + 1.5 * bn : 250.0 + 2.0 * bn) * scale;
    const double epi_clk = 350.0 * (bn / 32);
    const long long rows = pair ? 2 * kBlockM : kBlockM;
    const long long tiles = ((M + rows - 1) / rows) * ((N + bn - 1) / bn);
    const long long slots = pair ? dev->pair_clusters : dev->sm_count;
    const double main = static_cast<double>((k_blocks + split - 1) / split) * kb_clk;
    double clk;
    if (split > 1) {
        const double exchange_us = split == 2 ? 2.5 : (split == 4 ? 6.0 : 13.0);
        clk = main + epi_clk / split + exchange_us * 1900.0;
    } else {
        // Steady state: a tile's slab stores run beside the next tile's main loop.  When every SM streams C
        // the stores pace at the HBM write rate, ~1130 clk per 16 KB slab (measured), and the loads of the
        // main loop share the SM's port with them: fitted, the tile period is the longer of the two plus a
        // fifth of the shorter (applying it to store-paced tiles only made the model jump at main = store
        // and pick narrow tiles that re-read A four times as often: 20-30 % slower).
        const double store_clk = 1130.0 * (bn / 32);
        const double period = (main > store_clk ? main : store_clk) + 0.2 * (main > store_clk ? store_clk : main);
        const long long waves = (tiles + slots - 1) / slots;
        clk = static_cast<double>(waves - 1) * period + main + epi_clk;
    }
    return 3.7 + (pair ? 1.0 : 0.0) + clk / 1900.0;   // pairs: cluster launch, two cluster barriers
}

Plan make_plan(long long M, long long N, long long K, int block_k, const DeviceState* dev, int min_bn = 32,
               int min_bn_pair = 64, bool one_cta_no_split = false) {
    const int sm_count = dev->sm_count;
    const Tuning tun = tuning_now();
    Plan pl{};
    pl.k_blocks = static_cast<int>((K + block_k - 1) / block_k);

    // Candidates: one CTA per tile or CTA pairs, bn a multiple of 32 up to 256, optionally a cluster
    // split-K of 2/4/8 when the tiles alone would leave most SMs idle.  Experiment overrides
    // (mipgemm_set_tuning) restrict the candidate set.
    int best_pair = 0, best_bn = 128, best_split = 1;
    double best = 1e30;
    // (an explicit split reduces int32 tiles in global memory, which a float output cannot share)
    const bool explicit_split = tun.split_k != 0 && !tl_out_f32 && !tl_out_q8;
    // (N-contiguous B tiles come in 128-column blocks per CTA: a forced width must respect that)
    const int forced_bn = (tun.block_n && (min_bn <= 64 || tun.block_n == 256)) ? tun.block_n : 0;
    for (int pair = 0; pair <= 1; ++pair) {
        if (pair && (dev->pair_clusters <= 0 || one_cta_no_split)) continue;
        if (tun.force_path == MIPGEMM_PATH_DENSE_PAIR && !pair && dev->pair_clusters > 0) continue;
        if (tun.force_path == MIPGEMM_PATH_DENSE && pair) continue;
        for (int bn = 32; bn <= 256; bn += 32) {      // any multiple of 32 columns is a legal tile width (32 itself
                                                      // only pays for problems of a single wave: 512^3 -7 %)
            int bn_use = bn;
            if (bn < (pair ? min_bn_pair : min_bn)) continue;
            // (32 columns: only short-K problems that leave half of the SMs idle even at 64; K-heavy ones split K)
            if (bn == 32 && !forced_bn &&
                (((M + kBlockM - 1) / kBlockM) * ((N + 63) / 64) > sm_count / 2 || pl.k_blocks > 8))
                continue;
            if (min_bn >= 128 && bn % 128 != 0) continue;   // (N-contiguous B: whole 128-column blocks)
            if (forced_bn) {
                if (bn != 256) continue;                      // a single candidate: the forced width
                bn_use = forced_bn;
                if (pair && bn_use % 64 != 0) bn_use = (bn_use + 63) / 64 * 64;
            }
            const long long rows = pair ? 2 * kBlockM : kBlockM;
            const long long tiles = ((M + rows - 1) / rows) * ((N + bn_use - 1) / bn_use);
            for (int split = 1; split <= 8; split *= 2) {
                if (split > 1) {
                    if (pair || explicit_split || g_tuning_no_cluster_split || one_cta_no_split || tl_out_q8) break;
                    if (tiles * split > sm_count || bn_use / split < 32 || (bn_use / split) % 32 != 0) break;
                    if (pl.k_blocks / split < 2) break;
                }
                double us = plan_cost_us(pair, bn_use, split, M, N, pl.k_blocks, block_k, dev);
                // widths that are not a power of two re-read A more often (more DRAM traffic and power than
                // the model sees): they must win by a clear margin
                if ((bn_use & (bn_use - 1)) != 0) us *= 1.03;
                if (us < best) {
                    best = us;
                    best_pair = pair;
                    best_bn = bn_use;
                    best_split = split;
                }
            }
        }
    }
    pl.pair = best_pair;
    const int bn = best_bn;
    const int rows_per_tile = pl.pair ? 2 * kBlockM : kBlockM;
    pl.tiles_m = static_cast<int>((M + rows_per_tile - 1) / rows_per_tile);
    pl.block_n = bn;
    pl.tiles_n = static_cast<int>((N + bn - 1) / bn);
    const int stage_bytes = kBlockM * block_k + (pl.pair ? bn / 2 : bn) * block_k;
    int stages = (kSmemBudget - kCtrlBytes - kStagingBytes - 1024) / stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    if (tun.stages) stages = tun.stages < stages ? tun.stages : stages;
    if (stages < 2) stages = 2;
    pl.stages = stages;

    int split = (explicit_split && !one_cta_no_split) ? tun.split_k : best_split;
    if (pl.pair) split = 1;
    if (split > pl.k_blocks) split = pl.k_blocks;
    if (split < 1) split = 1;
    // the automatic split is a cluster split (DSMEM reduce-scatter: the receive buffers must fit
    // the idle pipeline stages); an explicit factor uses zero fill + TMA tile reduce-add
    pl.cluster_split = 0;
    if (!(explicit_split && !one_cta_no_split) && split > 1) {
        if (512LL * bn * (split - 1) / split <= static_cast<long long>(stages) * stage_bytes) pl.cluster_split = split;
        else split = 1;
    }
    pl.kb_per_split = (pl.k_blocks + split - 1) / split;
    pl.split_k = (pl.k_blocks + pl.kb_per_split - 1) / pl.kb_per_split;
    if (pl.cluster_split && pl.split_k != pl.cluster_split) {   // a share would be empty: no split
        pl.cluster_split = 0;
        pl.split_k = 1;
        pl.kb_per_split = pl.k_blocks;
    }
    return pl;
}

void log_dense(const char* what, long long M, long long N, long long K, const Plan& pl, const DenseParams& p, bool hit) {
    std::fprintf(stderr,
                 "mipgemm: %s M=%lld N=%lld K=%lld -> dense %s tile=%dx%d k_block=%d stages=%d split_k=%d%s c_mode=%d%s%s plan=%s\n",
                 what, M, N, K, pl.pair ? "cta-pair" : "one-cta", pl.pair ? 2 * kBlockM : kBlockM, pl.block_n, p.block_k,
                 pl.stages, pl.split_k, pl.cluster_split ? " (cluster)" : "", p.c_mode, p.accumulate ? " accumulate" : "",
                 p.out_f32 ? " f32-out" : (p.out_q8 ? " q8-out" : ""), hit ? "cached" : "new");
}

void fill_common(DenseParams& p, const Plan& pl, long long M, long long N, int32_t* C, long long ldc,
                 int block_k, bool a_unsigned, int accumulate, DeviceState* dev) {
    p.C = C;
    p.ldc = ldc;
    p.M = static_cast<int>(M);
    p.N = static_cast<int>(N);
    p.k_blocks = pl.k_blocks;
    p.block_n = pl.block_n;
    p.block_k = block_k;
    p.stages = pl.stages;
    p.tiles_m = pl.tiles_m;
    p.tiles_n = pl.tiles_n;
    p.split_k = pl.split_k;
    p.kb_per_split = pl.kb_per_split;
    p.cluster_split = pl.cluster_split;
    const int group_env = MIP_ENV_KNOB("MIPGEMM_GROUP_N", 0);
    const int raster_env = MIP_ENV_KNOB("MIPGEMM_RASTER", 0);
    p.group_n = group_env > 0 ? group_env : 8;
    p.raster = raster_env;
    p.use_red = (pl.split_k > 1 && !pl.cluster_split) ? 1 : 0;
    p.accumulate = p.use_red ? 0 : (accumulate ? 1 : 0);
    const uintptr_t c_addr = reinterpret_cast<uintptr_t>(C);
    p.store_vec = (c_addr % 32 == 0 && ldc % 8 == 0) ? 8 : ((c_addr % 16 == 0 && ldc % 4 == 0) ? 4 : 1);
    p.idesc = (2u << 4) | ((a_unsigned ? 0u : 1u) << 7) | (1u << 10) |
              (static_cast<uint32_t>(pl.block_n >> 3) << 17) |
              (static_cast<uint32_t>((pl.pair ? 2 * kBlockM : kBlockM) >> 4) << 24);
    p.tmem_cols = pow2_at_least(2u * pl.block_n);
    // With a 16-byte aligned C (base and pitch) the epilogue writes fully coalesced rows through
    // shared memory, and split-K partial tiles are added into C by TMA tile reduce-adds.
    p.c_mode = 0;
    if (c_addr % 16 == 0 && ldc % 4 == 0 && !g_tuning_no_tma_store) {
        // TMA tile stores clip at the tensor edge in 16-byte granules (measured: with N % 4 != 0 the
        // columns N .. roundup(N,4)-1 were overwritten), so they are used only when N % 4 == 0; the
        // coalesced path writes the ragged last columns one by one.
        const bool tma_ok = N % 4 == 0;
        if (pl.split_k > 1 && !pl.cluster_split) {
            if (tma_ok) {
                p.c_mode = 2;
                p.use_red = 0;
            }
        } else {
            // (accumulate: the tile stores become tile reduce-adds; without tile stores the rows are added
            // element-wise at the L2, which beats reading, adding and writing 16-byte pieces)
            p.c_mode = tma_ok ? 1 : (accumulate ? 5 : 3);
        }
    }
    // A C that is only 4-byte aligned: rows through shared memory, one 128-byte run per store instruction
    // (split-K partial sums keep the scalar reduce-add form).
    if (p.c_mode == 0 && !p.use_red && !g_tuning_no_tma_store) p.c_mode = 5;
    p.out_f32 = tl_out_f32;
    p.out_scale = tl_out_scale;
    if (tl_out_q8) {   // 8-bit codes: C and ldc address bytes; each thread writes its row's 32 bytes per chunk
        p.out_q8 = 1;
        p.q_lo = tl_q_lo;
        p.q_hi = tl_q_hi;
        p.c_mode = 4;
        p.accumulate = 0;
        p.use_red = 0;
        p.store_vec = (c_addr % 16 == 0 && ldc % 16 == 0) ? 16 : 1;
    }
    p.a_im2col = 0;
    p.status = dev->status_word;
    p.wait_budget_ns = g_wait_budget_ns.load(std::memory_order_relaxed);
    p.debug_flags = g_debug_flags.load(std::memory_order_relaxed);
    p.trace = nullptr;
#ifdef MIPGEMM_TRACE
    if (const char* tr = std::getenv("MIPGEMM_TRACE_PTR"))
        p.trace = reinterpret_cast<unsigned long long*>(std::strtoull(tr, nullptr, 10));
#endif
}

// Plan + encoded tensor maps of recent calls, keyed on everything that determines them (shapes,
// pointers, pitches, output transform, device, tuning epoch): a repeated call -- the normal case in
// inference, where the same layer runs on the same buffers again and again -- skips the planner and
// the three tensor-map encodings and goes straight to the launch.  Direct-mapped, behind a mutex;
// MIPGEMM_PLAN_CACHE=0 switches it off.
struct PlanKey {
    uint64_t w[28];
};
struct PlanEntry {
    bool used = false;
    PlanKey key;
    DenseParams p;
    Plan pl;
};
constexpr int kPlanCacheSlots = 1024;
PlanEntry* g_plan_cache = nullptr;
std::mutex g_plan_mutex;
std::atomic<uint64_t> g_plan_hits{0}, g_plan_misses{0};
bool plan_cache_enabled() {
    static const int on = env_int("MIPGEMM_PLAN_CACHE", 1);
#ifdef MIPGEMM_TRACE
    return false;
#else
    return on != 0 && !live_env();
#endif
}
size_t plan_slot(const PlanKey& k) {
    uint64_t h = 1469598103934665603ull;
    for (uint64_t v : k.w) { h ^= v; h *= 1099511628211ull; h ^= h >> 29; }
    return static_cast<size_t>(h % kPlanCacheSlots);
}
bool plan_lookup(const PlanKey& k, DenseParams* p, Plan* pl) {
    std::lock_guard<std::mutex> lock(g_plan_mutex);
    if (!g_plan_cache) return false;
    const PlanEntry& e = g_plan_cache[plan_slot(k)];
    if (!e.used || std::memcmp(&e.key, &k, sizeof(k)) != 0) return false;
    *p = e.p;
    *pl = e.pl;
    return true;
}
void plan_store(const PlanKey& k, const DenseParams& p, const Plan& pl) {
    std::lock_guard<std::mutex> lock(g_plan_mutex);
    if (!g_plan_cache) g_plan_cache = new PlanEntry[kPlanCacheSlots];
    PlanEntry& e = g_plan_cache[plan_slot(k)];
    e.used = true;
    e.key = k;
    e.p = p;
    e.pl = pl;
}
uint64_t out_mode_word() {
    uint32_t scale_bits;
    std::memcpy(&scale_bits, &tl_out_scale, 4);
    return static_cast<uint64_t>(scale_bits) | (static_cast<uint64_t>(tl_out_f32 & 1) << 32) |
           (static_cast<uint64_t>(tl_out_q8 & 1) << 33) | (static_cast<uint64_t>(tl_q_lo & 0x1FF) << 34) |
           (static_cast<uint64_t>(tl_q_hi & 0x1FF) << 43);
}

int run_dense(DenseParams& p, const Plan& pl, long long M, long long N, int32_t* C, long long ldc,
              int accumulate, DeviceState* dev, cudaStream_t stream, bool c_map_ready = false) {
    p.bias = tl_bias;   // (not part of the plan: a cached plan serves any bias vector)
    if (pl.split_k > 1 && !pl.cluster_split && !accumulate) {
        cudaError_t e = launch_fill_zero(C, ldc, M, N, stream);
        ++g_launches;
        if (e != cudaSuccess) return cuda_fail(e);
    }
    const long long units = static_cast<long long>(pl.tiles_m) * pl.tiles_n * pl.split_k;
    const int b_rows = pl.pair ? pl.block_n / 2 : pl.block_n;
    const size_t smem = static_cast<size_t>(pl.stages) * (kBlockM * p.block_k + b_rows * p.block_k) +
                        kStagingBytes + kCtrlBytes + 1024 +
                        (p.g_staged ? 64 + 2 * static_cast<size_t>(p.g_rowbuf_stride) + p.g_table_bytes : 0);
    if ((p.c_mode == 1 || p.c_mode == 2) && !c_map_ready) {
        cuuint64_t dims[2] = {static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(M)};
        cuuint64_t strides[1] = {static_cast<cuuint64_t>(ldc) * 4};
        cuuint32_t box[2] = {32, static_cast<cuuint32_t>(p.c_mode == 1 ? 128 : 32)};
        cuuint32_t estr[2] = {1, 1};
        CUresult r = g_encode_tiled(&p.tmap_c, CU_TENSOR_MAP_DATA_TYPE_INT32, 2, C, dims, strides, box, estr,
                                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                    CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            tl_last_cuda_error = 100000 + static_cast<int>(r);
            return MIPGEMM_ERR_CUDA;
        }
    }
    cudaError_t e;
    if (pl.pair) {
        const int clusters = static_cast<int>(units < dev->pair_clusters ? units : dev->pair_clusters);
        e = launch_dense_pair(p, 2 * clusters, smem, stream);
    } else if (pl.cluster_split) {
        e = launch_dense_cluster(p, static_cast<int>(units), pl.cluster_split, smem, stream);
    } else {
        const int grid = static_cast<int>(units < dev->sm_count ? units : dev->sm_count);
        e = p.a_gather ? launch_dense_gather(p, grid, smem, stream) : launch_dense(p, grid, smem, stream);
    }
    ++g_launches;
    if (e != cudaSuccess) return cuda_fail(e);
    return MIPGEMM_OK;
}

size_t gemm_scratch_bytes(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda, const void* B,
                          int64_t ldb) {
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    const long long pitch = round_up(K, 16);
    size_t need = 0;
    if (!aligned16(A, lda)) need += align256(static_cast<size_t>(M) * pitch);
    if (!aligned16(B, ldb)) need += align256(static_cast<size_t>(N) * pitch);
    return need;
}

// `outer`: scratch already reserved by the caller (the explicit-im2col convolution), from
// which this call takes its own share; nullptr = reserve what is needed here.
int gemm_impl(bool a_unsigned, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda, const int8_t* B,
              int64_t ldb, int32_t* C, int64_t ldc, int accumulate, void* stream_v, int path_flags,
              Scratch* outer = nullptr) {
    tl_last_path = MIPGEMM_PATH_NONE;
    const Tuning tun = tuning_now();
    if (M < 0 || N < 0 || K < 0) return MIPGEMM_ERR_INVALID_ARG;
    if (M > 0x7FFFFF00LL || N > 0x7FFFFF00LL) return MIPGEMM_ERR_INVALID_ARG;
    if (lda < K || ldb < K || ldc < N) return MIPGEMM_ERR_INVALID_ARG;
    if (K > (a_unsigned ? 65793 : 131071)) return MIPGEMM_ERR_K_TOO_LARGE;
    if (M == 0 || N == 0) {
        tl_last_path = MIPGEMM_PATH_TRIVIAL | path_flags;
        return MIPGEMM_OK;
    }
    if (!C || (!tl_out_q8 && reinterpret_cast<uintptr_t>(C) % 4 != 0)) return MIPGEMM_ERR_INVALID_ARG;
    if (K > 0 && (!A || !B)) return MIPGEMM_ERR_INVALID_ARG;
    DeviceState* dev = nullptr;
    int st = get_device(&dev);
    if (st != MIPGEMM_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);

    if (K == 0 && tl_bias) {     // every sum is its channel's bias
        tl_last_path = MIPGEMM_PATH_TRIVIAL | path_flags;
        cudaError_t e = launch_bias_rows(C, ldc, M, N, tl_bias, tl_out_q8, tl_out_scale, tl_q_lo, tl_q_hi, stream);
        ++g_launches;
        if (e != cudaSuccess) return cuda_fail(e);
        return MIPGEMM_OK;
    }
    if (K == 0 && tl_out_q8) {   // every sum is 0 and so is its code (q_lo <= 0 <= q_hi)
        tl_last_path = MIPGEMM_PATH_TRIVIAL | path_flags;
        cudaError_t e = cudaMemset2DAsync(C, static_cast<size_t>(ldc), 0, static_cast<size_t>(N),
                                          static_cast<size_t>(M), stream);
        if (e != cudaSuccess) return cuda_fail(e);
        return MIPGEMM_OK;
    }
    if (K == 0) {
        tl_last_path = MIPGEMM_PATH_TRIVIAL | path_flags;
        if (!accumulate) {
            cudaError_t e = launch_fill_zero(C, ldc, M, N, stream);
            ++g_launches;
            if (e != cudaSuccess) return cuda_fail(e);
        }
        return MIPGEMM_OK;
    }

    // ---- skinny path
    if (M <= 16 && !tl_out_q8 && !tl_bias && tun.force_path != MIPGEMM_PATH_DENSE &&
        tun.force_path != MIPGEMM_PATH_DENSE_PAIR) {
        SkinnyParams sp{A, lda, B, ldb, C, ldc, static_cast<int>(M), static_cast<int>(N),
                        static_cast<int>(K), a_unsigned ? 1 : 0, accumulate ? 1 : 0, tl_out_f32, tl_out_scale};
        const bool ring16 = skinny_ring16_supported(sp, dev->sm_count) && MIP_ENV_KNOB("MIPGEMM_NO_RING16", 0) == 0;
        if ((ring16 || skinny_ring_supported(sp, dev->sm_count)) && !g_tuning_no_skinny_ring) {
            SkinnyRingParams rp;
            std::memset(&rp, 0, sizeof(rp));
            // the weight matrix's tensor map is remembered like a dense plan (kind 3: only tmap_b is used)
            PlanKey key;
            DenseParams cached;
            Plan unused;
            bool hit = false;
            if (plan_cache_enabled()) {
                std::memset(&key, 0, sizeof(key));
                const uint64_t words[] = {3, reinterpret_cast<uint64_t>(dev), reinterpret_cast<uint64_t>(B),
                                          static_cast<uint64_t>(ldb), static_cast<uint64_t>(N), static_cast<uint64_t>(K)};
                std::memcpy(key.w, words, sizeof(words));
                hit = plan_lookup(key, &cached, &unused);
            }
            CUresult r = CUDA_SUCCESS;
            if (hit) {
                ++g_plan_hits;
                rp.tmap_b = cached.tmap_b;
            } else {
                cuuint64_t dims[3] = {128, static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(K / 128)};
                cuuint64_t strides[2] = {static_cast<cuuint64_t>(ldb), 128};
                cuuint32_t box[3] = {128, 16, 8};
                cuuint32_t estr[3] = {1, 1, 1};
                r = g_encode_tiled(&rp.tmap_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<int8_t*>(B), dims,
                                   strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
                if (r == CUDA_SUCCESS && plan_cache_enabled()) {
                    ++g_plan_misses;
                    std::memset(&cached, 0, sizeof(cached));
                    cached.tmap_b = rp.tmap_b;
                    plan_store(key, cached, Plan{});
                }
            }
            if (r == CUDA_SUCCESS) {   // (a driver that refuses the overlapping strides: register form below)
                rp.A = A; rp.lda = lda; rp.C = C; rp.ldc = ldc;
                rp.M = static_cast<int>(M); rp.N = static_cast<int>(N); rp.K = static_cast<int>(K);
                rp.a_unsigned = a_unsigned ? 1 : 0; rp.accumulate = accumulate ? 1 : 0;
                rp.out_f32 = tl_out_f32; rp.out_scale = tl_out_scale;
                rp.b_constant = (g_weights_constant.load() ||
                                 inside_constant_range(B, static_cast<size_t>(N - 1) * ldb + K)) ? 1 : 0;
                rp.status = dev->status_word;
                rp.wait_budget_ns = g_wait_budget_ns.load(std::memory_order_relaxed);
                rp.prefetch_chunks = MIP_ENV_KNOB("MIPGEMM_PREFETCH_CHUNKS", 4);   // (swept 0..16: 4 is the best)
                rp.debug_flags = g_debug_flags.load(std::memory_order_relaxed) |
                                 (MIP_ENV_KNOB("MIPGEMM_RING_ALWAYS_RELEASE", 0) ? 2 : 0);   // (A/B switch)
                rp.trace = nullptr;
#ifdef MIPGEMM_TRACE
                if (const char* tr = std::getenv("MIPGEMM_TRACE_PTR"))
                    rp.trace = reinterpret_cast<unsigned long long*>(std::strtoull(tr, nullptr, 10));
#endif
                cudaError_t e = ring16 ? launch_skinny_ring16(rp, dev->sm_count, stream)
                                       : launch_skinny_ring(rp, dev->sm_count, stream);
                ++g_launches;
                if (e != cudaSuccess) return cuda_fail(e);
                tl_last_path = MIPGEMM_PATH_SKINNY | path_flags;
                if (log_enabled())
                    std::fprintf(stderr, "mipgemm: gemm %s M=%lld N=%lld K=%lld -> skinny ring%s map=%s\n",
                                 a_unsigned ? "u8" : "s8", static_cast<long long>(M), static_cast<long long>(N),
                                 static_cast<long long>(K), rp.b_constant ? " (constant weights: early fetch)" : "",
                                 hit ? "cached" : "new");
                return MIPGEMM_OK;
            }
            tl_last_cuda_error = 100000 + static_cast<int>(r);
        }
        if (skinny_supported(sp)) {
            cudaError_t e = launch_skinny(sp, stream);
            ++g_launches;
            if (e != cudaSuccess) return cuda_fail(e);
            tl_last_path = MIPGEMM_PATH_SKINNY | path_flags;
            if (log_enabled())
                std::fprintf(stderr, "mipgemm: gemm %s M=%lld N=%lld K=%lld -> skinny register form\n",
                             a_unsigned ? "u8" : "s8", static_cast<long long>(M), static_cast<long long>(N),
                             static_cast<long long>(K));
            return MIPGEMM_OK;
        }
    }

    // ---- dense path; operands that TMA cannot address are re-pitched first
    const bool repack_a = !aligned16(A, lda);
    const bool repack_b = !aligned16(B, ldb);
    const long long pitch = round_up(K, 16);
    Scratch local(dev, stream);
    Scratch& scratch = outer ? *outer : local;
    if (!outer && (st = local.reserve(gemm_scratch_bytes(M, N, K, A, lda, B, ldb))) != MIPGEMM_OK) return st;
    const void* a_use = A;
    const void* b_use = B;
    long long lda_use = lda, ldb_use = ldb;
    if (repack_a && repack_b) {   // both operands in one launch
        void* dst_a = scratch.take(static_cast<size_t>(M) * pitch);
        void* dst_b = scratch.take(static_cast<size_t>(N) * pitch);
        cudaError_t e = launch_repack2(A, lda, dst_a, M, B, ldb, dst_b, N, pitch, K, stream);
        ++g_launches;
        if (e != cudaSuccess) return cuda_fail(e);
        a_use = dst_a;
        b_use = dst_b;
        lda_use = ldb_use = pitch;
        path_flags |= MIPGEMM_PATH_REPACK;
    } else if (repack_a) {
        void* dst = scratch.take(static_cast<size_t>(M) * pitch);
        cudaError_t e = launch_repack(A, lda, dst, pitch, M, K, stream);
        ++g_launches;
        if (e != cudaSuccess) return cuda_fail(e);
        a_use = dst;
        lda_use = pitch;
        path_flags |= MIPGEMM_PATH_REPACK;
    }
    if (repack_b && !repack_a) {
        void* dst = scratch.take(static_cast<size_t>(N) * pitch);
        cudaError_t e = launch_repack(B, ldb, dst, pitch, N, K, stream);
        ++g_launches;
        if (e != cudaSuccess) return cuda_fail(e);
        b_use = dst;
        ldb_use = pitch;
        path_flags |= MIPGEMM_PATH_REPACK;
    }

    const int block_k = 128;
    Plan pl;
    DenseParams p;
    // operands used in place: the plan and the tensor maps depend on nothing but the arguments
    const bool cacheable = plan_cache_enabled() && !repack_a && !repack_b;
    PlanKey key;
    bool hit = false;
    if (cacheable) {
        std::memset(&key, 0, sizeof(key));
        const uint64_t words[] = {1, reinterpret_cast<uint64_t>(dev), g_tuning_epoch.load(std::memory_order_acquire),
                                  static_cast<uint64_t>(a_unsigned) | (accumulate ? 2u : 0u), out_mode_word(),
                                  static_cast<uint64_t>(M), static_cast<uint64_t>(N), static_cast<uint64_t>(K),
                                  reinterpret_cast<uint64_t>(A), static_cast<uint64_t>(lda),
                                  reinterpret_cast<uint64_t>(B), static_cast<uint64_t>(ldb),
                                  reinterpret_cast<uint64_t>(C), static_cast<uint64_t>(ldc)};
        std::memcpy(key.w, words, sizeof(words));
        hit = plan_lookup(key, &p, &pl);
    }
    if (hit) {
        ++g_plan_hits;
    } else {
        pl = make_plan(M, N, K, block_k, dev);
        std::memset(&p, 0, sizeof(p));
        fill_common(p, pl, M, N, C, ldc, block_k, a_unsigned, accumulate, dev);
        if ((st = encode_tiled_2d(&p.tmap_a, a_use, K, M, lda_use, block_k, kBlockM)) != MIPGEMM_OK) return st;
        if ((st = encode_tiled_2d(&p.tmap_b, b_use, K, N, ldb_use, block_k, pl.pair ? pl.block_n / 2 : pl.block_n)) !=
            MIPGEMM_OK)
            return st;
    }
    if ((st = run_dense(p, pl, M, N, C, ldc, accumulate, dev, stream, hit)) != MIPGEMM_OK) return st;
    if (cacheable && !hit) {
        ++g_plan_misses;
        plan_store(key, p, pl);
    }
    if (pl.split_k > 1) path_flags |= MIPGEMM_PATH_SPLITK;
    tl_last_path = (pl.pair ? MIPGEMM_PATH_DENSE_PAIR : MIPGEMM_PATH_DENSE) | path_flags;
    if (log_enabled())
        log_dense(repack_a || repack_b ? (a_unsigned ? "gemm u8 (re-pitched)" : "gemm s8 (re-pitched)")
                                       : (a_unsigned ? "gemm u8" : "gemm s8"), M, N, K, pl, p, hit);
    return MIPGEMM_OK;
}

bool conv_geometry(ConvGeom& g) {
    if (g.Nb < 0 || g.H <= 0 || g.W <= 0 || g.Cin <= 0 || g.Cout < 0 || g.R <= 0 || g.S <= 0) return false;
    if (g.stride_h <= 0 || g.stride_w <= 0 || g.dil_h <= 0 || g.dil_w <= 0 || g.pad_h < 0 || g.pad_w < 0)
        return false;
    const long long eh = g.H + 2LL * g.pad_h - static_cast<long long>(g.dil_h) * (g.R - 1) - 1;
    const long long ew = g.W + 2LL * g.pad_w - static_cast<long long>(g.dil_w) * (g.S - 1) - 1;
    if (eh < 0 || ew < 0) return false;
    g.Ho = eh / g.stride_h + 1;
    g.Wo = ew / g.stride_w + 1;
    return true;
}

bool conv_is_pointwise(const ConvGeom& g) {
    return g.R == 1 && g.S == 1 && g.stride_h == 1 && g.stride_w == 1 && g.pad_h == 0 && g.pad_w == 0;
}

// TMA im2col mode: channel count a multiple of the k-block, 16-byte aligned base, and the
// driver's limits on corners, traversal strides and extents.
bool conv_tma_eligible(const ConvGeom& g, const void* X, const void* Wt) {
    if (g.Cin % 64 != 0) return false;
    if (reinterpret_cast<uintptr_t>(X) % 16 != 0 || reinterpret_cast<uintptr_t>(Wt) % 16 != 0) return false;
    if (g.stride_h > 8 || g.stride_w > 8) return false;
    const int lw = -g.pad_w, lh = -g.pad_h;
    const int uw = g.pad_w - (g.S - 1) * g.dil_w, uh = g.pad_h - (g.R - 1) * g.dil_h;
    if (lw < -128 || lh < -128 || uw < -128 || uh < -128 || uw > 127 || uh > 127) return false;
    if ((g.S - 1) * g.dil_w > 65535 || (g.R - 1) * g.dil_h > 65535) return false;
    if (g.W >= (1LL << 31) || g.H >= (1LL << 31) || g.Nb >= (1LL << 31)) return false;
    if (g.H * g.W * g.Cin >= (1LL << 40)) return false;
    return true;
}

// Convolutions TMA cannot gather (channel count not a multiple of 64, e.g. an RGB stem) whose
// filter rows are contiguous in the image (dil_w == 1): operand A is built in shared memory
// by extra warps of the dense kernel, so the augmented matrix never exists in memory.
bool conv_gather_eligible(const ConvGeom& g) {
    if (g.dil_w != 1) return false;
    const long long seg = static_cast<long long>(g.S) * g.Cin;
    const long long slot = round_up(seg, 16);
    if (slot * g.R > 8192) return false;                       // whole rows of A stay short
    if (g.W * g.Cin >= (1LL << 30) || g.H >= (1LL << 30)) return false;
    const long long xbytes = g.Nb * g.H * g.W * g.Cin;
    if (xbytes < 64 || xbytes >= (1LL << 30)) return false;    // (32-bit byte offsets; loads assume some size)
    return true;
}

// General form: any signedness pair, either storage order for A and B, row- or column-major C
// (paper Section 3: transposition and storage order are absorbed below the micro-kernel; a
// column-major C by swapping the roles of A and B).  M- / N-contiguous operands are read by the
// tensor cores as they are (MN-major shared-memory descriptors); only operands TMA cannot
// address are first transposed into K-contiguous scratch.
int gemm_ex_impl(int a_unsigned, int b_unsigned, int a_order, int b_order, int c_col_major, int64_t M, int64_t N,
                 int64_t K, const void* A, int64_t lda, const void* B, int64_t ldb, int32_t* C, int64_t ldc,
                 int accumulate, void* stream_v) {
    tl_last_path = MIPGEMM_PATH_NONE;
    if ((a_order | b_order | c_col_major | a_unsigned | b_unsigned) & ~1) return MIPGEMM_ERR_INVALID_ARG;
    if (c_col_major)   // C^T = B^T A^T: the same problem with the operands' roles exchanged
        return gemm_ex_impl(b_unsigned, a_unsigned, b_order, a_order, 0, N, M, K, B, ldb, A, lda, C, ldc, accumulate,
                            stream_v);
    if (M < 0 || N < 0 || K < 0 || M > 0x7FFFFF00LL || N > 0x7FFFFF00LL) return MIPGEMM_ERR_INVALID_ARG;
    if (lda < (a_order ? M : K) || ldb < (b_order ? N : K) || ldc < N) return MIPGEMM_ERR_INVALID_ARG;
    const long long k_limit = (a_unsigned && b_unsigned) ? 33025 : ((a_unsigned || b_unsigned) ? 65793 : 131071);
    if (K > k_limit) return MIPGEMM_ERR_K_TOO_LARGE;
    if (!b_unsigned && !a_order && !b_order)
        return gemm_impl(a_unsigned != 0, M, N, K, A, lda, static_cast<const int8_t*>(B), ldb, C, ldc, accumulate,
                         stream_v, 0);
    if (M == 0 || N == 0) {
        tl_last_path = MIPGEMM_PATH_TRIVIAL;
        return MIPGEMM_OK;
    }
    if (!C || reinterpret_cast<uintptr_t>(C) % 4 != 0 || (K > 0 && (!A || !B))) return MIPGEMM_ERR_INVALID_ARG;
    DeviceState* dev = nullptr;
    int st = get_device(&dev);
    if (st != MIPGEMM_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    cudaError_t e;
    if (K == 0) {
        tl_last_path = MIPGEMM_PATH_TRIVIAL;
        if (!accumulate) {
            if ((e = launch_fill_zero(C, ldc, M, N, stream)) != cudaSuccess) return cuda_fail(e);
            ++g_launches;
        }
        return MIPGEMM_OK;
    }

    // operands TMA cannot address go to K-contiguous scratch (plain or transposing re-pitch)
    const long long pitch = round_up(K, 16);
    const bool fix_a = !aligned16(A, lda), fix_b = !aligned16(B, ldb);
    Scratch scratch(dev, stream);
    size_t need = 0;
    if (fix_a) need += align256(static_cast<size_t>(M) * pitch);
    if (fix_b) need += align256(static_cast<size_t>(N) * pitch);
    if ((st = scratch.reserve(need)) != MIPGEMM_OK) return st;
    const void* a_use = A;
    const void* b_use = B;
    long long lda_use = lda, ldb_use = ldb;
    int a_mn = a_order, b_mn = b_order, flags = 0;
    if (fix_a) {
        void* dst = scratch.take(static_cast<size_t>(M) * pitch);
        e = a_order ? launch_transpose_repack(A, lda, dst, pitch, M, K, stream) : launch_repack(A, lda, dst, pitch, M, K, stream);
        if (e != cudaSuccess) return cuda_fail(e);
        ++g_launches;
        a_use = dst; lda_use = pitch; a_mn = 0; flags |= MIPGEMM_PATH_REPACK;
    }
    if (fix_b) {
        void* dst = scratch.take(static_cast<size_t>(N) * pitch);
        e = b_order ? launch_transpose_repack(B, ldb, dst, pitch, N, K, stream) : launch_repack(B, ldb, dst, pitch, N, K, stream);
        if (e != cudaSuccess) return cuda_fail(e);
        ++g_launches;
        b_use = dst; ldb_use = pitch; b_mn = 0; flags |= MIPGEMM_PATH_REPACK;
    }

    const int block_k = 128;
    // N-contiguous B is staged in blocks of 128 columns per CTA: 128 or 256 wide tiles for one
    // CTA, 256 wide for a pair (each CTA stages half)
    const Plan pl = make_plan(M, N, K, block_k, dev, b_mn ? 128 : 64, b_mn ? 256 : 64);
    DenseParams p;
    std::memset(&p, 0, sizeof(p));
    fill_common(p, pl, M, N, C, ldc, block_k, a_unsigned != 0, accumulate, dev);
    p.a_mn = a_mn;
    p.b_mn = b_mn;
    p.idesc = (2u << 4) | ((a_unsigned ? 0u : 1u) << 7) | ((b_unsigned ? 0u : 1u) << 10) |
              (static_cast<uint32_t>(a_mn) << 15) | (static_cast<uint32_t>(b_mn) << 16) |
              (static_cast<uint32_t>(pl.block_n >> 3) << 17) |
              (static_cast<uint32_t>((pl.pair ? 2 * kBlockM : kBlockM) >> 4) << 24);
    // K-contiguous: tensor {K, rows}, box {128, tile rows}; M/N-contiguous: tensor {rows, K}, box {128, 128}
    st = a_mn ? encode_tiled_2d(&p.tmap_a, a_use, M, K, lda_use, 128, block_k)
              : encode_tiled_2d(&p.tmap_a, a_use, K, M, lda_use, block_k, kBlockM);
    if (st != MIPGEMM_OK) return st;
    st = b_mn ? encode_tiled_2d(&p.tmap_b, b_use, N, K, ldb_use, 128, block_k)
              : encode_tiled_2d(&p.tmap_b, b_use, K, N, ldb_use, block_k, pl.pair ? pl.block_n / 2 : pl.block_n);
    if (st != MIPGEMM_OK) return st;
    if ((st = run_dense(p, pl, M, N, C, ldc, accumulate, dev, stream)) != MIPGEMM_OK) return st;
    if (pl.split_k > 1) flags |= MIPGEMM_PATH_SPLITK;
    tl_last_path = (pl.pair ? MIPGEMM_PATH_DENSE_PAIR : MIPGEMM_PATH_DENSE) | flags;
    return MIPGEMM_OK;
}

// Strided batch: C_b [+]= A_b * B_b for b < batch.  When every operand of every batch member is
// TMA-addressable the whole batch is one launch of the dense kernel (rank-3 tensor maps, the batch
// index is the slowest tile coordinate); otherwise the members are served one by one.
int batched_impl(bool a_unsigned, int64_t batch, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                 int64_t stride_a, const int8_t* B, int64_t ldb, int64_t stride_b, int32_t* C, int64_t ldc,
                 int64_t stride_c, int accumulate, void* stream_v) {
    tl_last_path = MIPGEMM_PATH_NONE;
    if (batch < 0 || M < 0 || N < 0 || K < 0 || batch > 0x7FFFFFFFLL) return MIPGEMM_ERR_INVALID_ARG;
    if (M > 0x7FFFFF00LL || N > 0x7FFFFF00LL) return MIPGEMM_ERR_INVALID_ARG;
    if (lda < K || ldb < K || ldc < N || stride_a < 0 || stride_b < 0) return MIPGEMM_ERR_INVALID_ARG;
    if (K > (a_unsigned ? 65793 : 131071)) return MIPGEMM_ERR_K_TOO_LARGE;
    if (batch == 0 || M == 0 || N == 0) {
        tl_last_path = MIPGEMM_PATH_TRIVIAL;
        return MIPGEMM_OK;
    }
    if (batch > 1 && stride_c < (M - 1) * ldc + N) return MIPGEMM_ERR_INVALID_ARG;   // C matrices must not overlap
    if (!C || reinterpret_cast<uintptr_t>(C) % 4 != 0) return MIPGEMM_ERR_INVALID_ARG;
    if (K > 0 && (!A || !B)) return MIPGEMM_ERR_INVALID_ARG;
    DeviceState* dev = nullptr;
    int st = get_device(&dev);
    if (st != MIPGEMM_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);

    const long long tiles_m = (M + kBlockM - 1) / kBlockM;
    const bool one_launch = batch > 1 && K > 0 && aligned16(A, lda) && aligned16(B, ldb) && stride_a % 16 == 0 &&
                            stride_b % 16 == 0 && stride_a > 0 && stride_b > 0 && !tl_out_f32 &&
                            tiles_m * ((N + 63) / 64) * batch < 0x7FFFFFFFLL;
    if (!one_launch) {
        int flags = 0;
        for (int64_t b = 0; b < batch; ++b) {
            st = gemm_impl(a_unsigned, M, N, K, static_cast<const char*>(A) + b * stride_a, lda, B + b * stride_b, ldb,
                           C + b * stride_c, ldc, accumulate, stream_v, 0);
            if (st != MIPGEMM_OK) return st;
            flags |= tl_last_path;
        }
        tl_last_path = flags;
        return MIPGEMM_OK;
    }

    const int block_k = K <= 64 ? 64 : 128;
    const Tuning tun = tuning_now();
    Plan pl{};
    pl.k_blocks = static_cast<int>((K + block_k - 1) / block_k);
    double best = 1e30;
    for (int bn = 64; bn <= 256; bn *= 2) {
        if (tun.block_n && bn != 64) continue;
        const int bn_use = tun.block_n ? tun.block_n : bn;
        const double us = plan_cost_us(0, bn_use, 1, tiles_m * batch * kBlockM, N, pl.k_blocks, block_k, dev);
        if (us < best) { best = us; pl.block_n = bn_use; }
    }
    pl.pair = 0;
    pl.cluster_split = 0;
    pl.split_k = 1;
    pl.kb_per_split = pl.k_blocks;
    pl.tiles_m = static_cast<int>(tiles_m);
    pl.tiles_n = static_cast<int>((N + pl.block_n - 1) / pl.block_n);
    const int stage_bytes = kBlockM * block_k + pl.block_n * block_k;
    int stages = (kSmemBudget - kCtrlBytes - kStagingBytes - 1024) / stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    pl.stages = stages;

    DenseParams p;
    std::memset(&p, 0, sizeof(p));
    fill_common(p, pl, M, N, C, ldc, block_k, a_unsigned, accumulate, dev);
    p.batch = static_cast<int>(batch);
    p.stride_c = stride_c;
    if (stride_c % 4 != 0 && (p.c_mode == 1 || p.c_mode == 3)) {   // batch members of C would lose their 16-byte alignment
        p.c_mode = 5;
    }
    auto encode3 = [&](CUtensorMap* map, const void* base, long long inner, long long rows, long long pitch,
                       long long bstride, int box_inner, int box_rows, CUtensorMapDataType dt, int esize) -> int {
        cuuint64_t dims[3] = {static_cast<cuuint64_t>(inner), static_cast<cuuint64_t>(rows),
                              static_cast<cuuint64_t>(batch)};
        cuuint64_t strides[2] = {static_cast<cuuint64_t>(pitch) * esize, static_cast<cuuint64_t>(bstride) * esize};
        cuuint32_t box[3] = {static_cast<cuuint32_t>(box_inner), static_cast<cuuint32_t>(box_rows), 1};
        cuuint32_t estr[3] = {1, 1, 1};
        const CUtensorMapSwizzle sw = box_inner * esize == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
        CUresult r = g_encode_tiled(map, dt, 3, const_cast<void*>(base), dims, strides, box, estr,
                                    CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            tl_last_cuda_error = 100000 + static_cast<int>(r);
            return MIPGEMM_ERR_CUDA;
        }
        return MIPGEMM_OK;
    };
    if ((st = encode3(&p.tmap_a, A, K, M, lda, stride_a, block_k, kBlockM, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1)) != MIPGEMM_OK)
        return st;
    if ((st = encode3(&p.tmap_b, B, K, N, ldb, stride_b, block_k, pl.block_n, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1)) != MIPGEMM_OK)
        return st;
    if (p.c_mode == 1 &&
        (st = encode3(&p.tmap_c, C, N, M, ldc, stride_c, 32, 128, CU_TENSOR_MAP_DATA_TYPE_INT32, 4)) != MIPGEMM_OK)
        return st;
    const long long units = tiles_m * pl.tiles_n * batch;
    const int grid = static_cast<int>(units < dev->sm_count ? units : dev->sm_count);
    const size_t smem = static_cast<size_t>(pl.stages) * stage_bytes + kStagingBytes + kCtrlBytes + 1024;
    cudaError_t e = launch_dense(p, grid, smem, stream);
    ++g_launches;
    if (e != cudaSuccess) return cuda_fail(e);
    tl_last_path = MIPGEMM_PATH_DENSE | MIPGEMM_PATH_BATCHED;
    return MIPGEMM_OK;
}

// Pitched copy that degenerates to one flat copy when both sides are dense (flat copies run at the
// full rate of the host link; pitched ones are slower even when their pitches equal the width).
cudaError_t copy_rows(void* dst, size_t dpitch, const void* src, size_t spitch, size_t width, size_t rows,
                      cudaMemcpyKind kind, cudaStream_t stream) {
    if (rows == 0 || width == 0) return cudaSuccess;
    if (dpitch == width && spitch == width) return cudaMemcpyAsync(dst, src, width * rows, kind, stream);
    return cudaMemcpy2DAsync(dst, dpitch, src, spitch, width, rows, kind, stream);
}

// Host-buffer front end: stage operands, run the device entry point, copy C back.  Calls are serialised
// per device (they share the staging buffer, the two copy streams and the event pool).
int host_impl(bool a_unsigned, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda, const int8_t* B,
              int64_t ldb, int32_t* C, int64_t ldc, int accumulate, void* stream_v) {
    if (M < 0 || N < 0 || K < 0 || lda < K || ldb < K || ldc < N) return MIPGEMM_ERR_INVALID_ARG;
    if (K > (a_unsigned ? 65793 : 131071)) return MIPGEMM_ERR_K_TOO_LARGE;
    if (M == 0 || N == 0) return MIPGEMM_OK;
    if (!C || (K > 0 && (!A || !B))) return MIPGEMM_ERR_INVALID_ARG;
    DeviceState* dev = nullptr;
    int st = get_device(&dev);
    if (st != MIPGEMM_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const long long pitch = round_up(K > 0 ? K : 1, 16);
    const long long ldc_dev = round_up(N, 8);
    const size_t a_bytes = align256(static_cast<size_t>(M) * pitch);
    const size_t b_bytes = align256(static_cast<size_t>(N) * pitch);
    const size_t c_bytes = align256(static_cast<size_t>(M) * ldc_dev * 4);
    std::lock_guard<std::mutex> host_lock(dev->host_mutex);
    cudaError_t e;
    // The staging buffer lives across calls and only grows (mipgemm_release_staging() frees it): taking
    // gigabytes from the allocator per call cost milliseconds.  Every earlier user has synchronised.
    if (dev->staging_bytes < a_bytes + b_bytes + c_bytes) {
        if (dev->staging) (void)cudaFree(dev->staging);
        dev->staging = nullptr;
        dev->staging_bytes = 0;
        e = cudaMalloc(&dev->staging, a_bytes + b_bytes + c_bytes);
        if (e != cudaSuccess) {
            tl_last_cuda_error = static_cast<int>(e);
            (void)cudaGetLastError();
            return MIPGEMM_ERR_WORKSPACE;
        }
        dev->staging_bytes = a_bytes + b_bytes + c_bytes;
    }
    char* base = static_cast<char*>(dev->staging);
    char* dA = base;
    char* dB = base + a_bytes;
    int32_t* dC = reinterpret_cast<int32_t*>(base + a_bytes + b_bytes);
    st = MIPGEMM_OK;
    auto check = [&](cudaError_t ee) -> bool {
        if (ee != cudaSuccess && st == MIPGEMM_OK) st = cuda_fail(ee);
        return ee == cudaSuccess;
    };

    // Large problems are cut into a grid of up to 4 x 4 blocks of C (1024 rows / columns or more each), and three streams work on them at
    // once: one copies row blocks of A and column blocks of B in (in the order the blocks of C need them),
    // the caller's stream computes block after block, one copies finished blocks out -- so both directions
    // of the host link are busy while the kernels run, and the first block starts after two operand
    // blocks have arrived instead of after all of B.
    const long long total_bytes = static_cast<long long>(M) * K + static_cast<long long>(N) * K +
                                  4LL * M * N * (accumulate ? 2 : 1);
    int bi = 1, bj = 1;
    if (K > 0 && total_bytes >= (32LL << 20) && dev->copy_in && dev->copy_out) {
        bi = static_cast<int>(M / 1024 < 1 ? 1 : (M / 1024 > kHostBlocks ? kHostBlocks : M / 1024));
        bj = static_cast<int>(N / 1024 < 1 ? 1 : (N / 1024 > kHostBlocks ? kHostBlocks : N / 1024));
        // (measured on the square sweep: 4 x 4 blocks beat 8 x 4, 8 x 2, 4 x 2, 2 x 4 and row blocks only --
        // narrower blocks make the pitched copies of C slower, fewer blocks lengthen the head)
        static const int max_bi = env_int("MIPGEMM_HOST_ROW_BLOCKS", 4);
        static const int max_bj = env_int("MIPGEMM_HOST_COL_BLOCKS", 4);
        if (bi > kHostBlocks) bi = kHostBlocks;
        if (bj > kHostBlocks) bj = kHostBlocks;
        if (bi > max_bi) bi = max_bi < 1 ? 1 : max_bi;
        if (bj > max_bj) bj = max_bj < 1 ? 1 : max_bj;
    }
    if (bi * bj > 1) {
        if (!dev->host_events_ready) {
            for (int i = 0; i < kHostEvents; ++i)
                if (!check(cudaEventCreateWithFlags(&dev->host_events[i], cudaEventDisableTiming))) return st;
            dev->host_events_ready = true;
        }
        int n_ev = 0;
        auto next_event = [&]() { return dev->host_events[n_ev++]; };
        const long long rows_per = round_up((M + bi - 1) / bi, 256);
        const long long cols_per = round_up((N + bj - 1) / bj, 256);
        bi = static_cast<int>((M + rows_per - 1) / rows_per);
        bj = static_cast<int>((N + cols_per - 1) / cols_per);
        cudaEvent_t ev_a[kHostBlocks] = {}, ev_b[kHostBlocks] = {};
        bool ok = true;
        auto upload_a = [&](int i) {
            const long long r0 = i * rows_per, rows = (M - r0 < rows_per) ? M - r0 : rows_per;
            ok = ok && check(copy_rows(dA + r0 * pitch, pitch, static_cast<const char*>(A) + r0 * lda, lda, K, rows,
                                       cudaMemcpyHostToDevice, dev->copy_in));
            if (ok && accumulate)
                ok = check(copy_rows(dC + r0 * ldc_dev, ldc_dev * 4, C + r0 * ldc, ldc * 4, N * 4, rows,
                                     cudaMemcpyHostToDevice, dev->copy_in));
            ev_a[i] = next_event();
            ok = ok && check(cudaEventRecord(ev_a[i], dev->copy_in));
        };
        auto upload_b = [&](int j) {
            const long long c0 = j * cols_per, cols = (N - c0 < cols_per) ? N - c0 : cols_per;
            ok = ok && check(copy_rows(dB + c0 * pitch, pitch, reinterpret_cast<const char*>(B) + c0 * ldb, ldb, K, cols,
                                       cudaMemcpyHostToDevice, dev->copy_in));
            ev_b[j] = next_event();
            ok = ok && check(cudaEventRecord(ev_b[j], dev->copy_in));
        };
        cudaEvent_t ev_start = next_event();
        ok = check(cudaEventRecord(ev_start, stream)) && check(cudaStreamWaitEvent(dev->copy_in, ev_start, 0)) &&
             check(cudaStreamWaitEvent(dev->copy_out, ev_start, 0));
        // upload order = order of first use by the row-major sweep over the blocks of C
        if (ok) upload_a(0);
        for (int j = 0; j < bj && ok; ++j) upload_b(j);
        for (int i = 1; i < bi && ok; ++i) upload_a(i);
        for (int i = 0; i < bi && ok; ++i) {
            const long long r0 = i * rows_per, rows = (M - r0 < rows_per) ? M - r0 : rows_per;
            ok = check(cudaStreamWaitEvent(stream, ev_a[i], 0));
            for (int j = 0; j < bj && ok; ++j) {
                const long long c0 = j * cols_per, cols = (N - c0 < cols_per) ? N - c0 : cols_per;
                if (i == 0) ok = check(cudaStreamWaitEvent(stream, ev_b[j], 0));
                if (!ok) break;
                int32_t* c_ij = dC + r0 * ldc_dev + c0;
                const int gs = gemm_impl(a_unsigned, rows, cols, K, dA + r0 * pitch, pitch,
                                         reinterpret_cast<const int8_t*>(dB + c0 * pitch), pitch, c_ij, ldc_dev,
                                         accumulate, stream_v, 0);
                if (gs != MIPGEMM_OK) { st = gs; ok = false; break; }
                cudaEvent_t ev_cmp = next_event();
                ok = check(cudaEventRecord(ev_cmp, stream)) && check(cudaStreamWaitEvent(dev->copy_out, ev_cmp, 0)) &&
                     check(copy_rows(C + r0 * ldc + c0, ldc * 4, c_ij, ldc_dev * 4, cols * 4, rows,
                                     cudaMemcpyDeviceToHost, dev->copy_out));
            }
        }
        // the caller's stream waits for both helper streams
        cudaEvent_t ev_in_done = next_event(), ev_out_done = next_event();
        if (check(cudaEventRecord(ev_in_done, dev->copy_in))) check(cudaStreamWaitEvent(stream, ev_in_done, 0));
        if (check(cudaEventRecord(ev_out_done, dev->copy_out))) check(cudaStreamWaitEvent(stream, ev_out_done, 0));
        e = cudaStreamSynchronize(stream);
        if (st == MIPGEMM_OK && e != cudaSuccess) st = cuda_fail(e);
        if (st != MIPGEMM_OK) {   // make sure nothing of this call is still in flight
            (void)cudaStreamSynchronize(dev->copy_in);
            (void)cudaStreamSynchronize(dev->copy_out);
        }
        return st;
    }

    if (K > 0) {
        check(copy_rows(dA, pitch, A, lda, K, M, cudaMemcpyHostToDevice, stream)) &&
            check(copy_rows(dB, pitch, B, ldb, K, N, cudaMemcpyHostToDevice, stream));
    }
    if (st == MIPGEMM_OK && accumulate)
        check(copy_rows(dC, ldc_dev * 4, C, ldc * 4, N * 4, M, cudaMemcpyHostToDevice, stream));
    if (st == MIPGEMM_OK)
        st = gemm_impl(a_unsigned, M, N, K, dA, pitch, reinterpret_cast<const int8_t*>(dB), pitch, dC, ldc_dev,
                       accumulate, stream_v, 0);
    if (st == MIPGEMM_OK)
        check(copy_rows(C, ldc * 4, dC, ldc_dev * 4, N * 4, M, cudaMemcpyDeviceToHost, stream));
    e = cudaStreamSynchronize(stream);
    if (st == MIPGEMM_OK && e != cudaSuccess) st = cuda_fail(e);
    return st;
}

}  // namespace

extern "C" {

int mipgemm_s8s8s32(int64_t M, int64_t N, int64_t K, const int8_t* A, int64_t lda, const int8_t* B,
                    int64_t ldb, int32_t* C, int64_t ldc, int accumulate, void* stream) {
    return gemm_impl(false, M, N, K, A, lda, B, ldb, C, ldc, accumulate, stream, 0);
}

int mipgemm_u8s8s32(int64_t M, int64_t N, int64_t K, const uint8_t* A, int64_t lda, const int8_t* B,
                    int64_t ldb, int32_t* C, int64_t ldc, int accumulate, void* stream) {
    return gemm_impl(true, M, N, K, A, lda, B, ldb, C, ldc, accumulate, stream, 0);
}

int mipgemm_conv_u8s8s32(int64_t Nb, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int R, int S,
                         int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w,
                         const uint8_t* X, const int8_t* Wt, int32_t* Y, int accumulate, void* stream_v) {
    tl_last_path = MIPGEMM_PATH_NONE;
    const Tuning tun = tuning_now();
    ConvGeom g{Nb, H, W, Cin, Cout, 0, 0, R, S, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w};
    if (!conv_geometry(g)) return MIPGEMM_ERR_INVALID_ARG;
    const long long M = g.Nb * g.Ho * g.Wo;
    const long long K = static_cast<long long>(R) * S * Cin;
    if (M > 0x7FFFFF00LL || Cout > 0x7FFFFF00LL) return MIPGEMM_ERR_INVALID_ARG;
    if (K > 65793) return MIPGEMM_ERR_K_TOO_LARGE;
    if (M == 0 || Cout == 0) {
        tl_last_path = MIPGEMM_PATH_TRIVIAL;
        return MIPGEMM_OK;
    }
    if (!X || !Wt || !Y || (!tl_out_q8 && reinterpret_cast<uintptr_t>(Y) % 4 != 0)) return MIPGEMM_ERR_INVALID_ARG;

    if (conv_is_pointwise(g))
        return gemm_impl(true, M, Cout, Cin, X, Cin, Wt, Cin, Y, Cout, accumulate, stream_v, 0);

    DeviceState* dev = nullptr;
    int st = get_device(&dev);
    if (st != MIPGEMM_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);

    if (conv_tma_eligible(g, X, Wt) && tun.force_path != MIPGEMM_PATH_IM2COL_EXPLICIT) {
        const int block_k = (Cin % 128 == 0) ? 128 : 64;
        Plan pl;
        DenseParams p;
        const bool cacheable = plan_cache_enabled();
        PlanKey key;
        bool hit = false;
        if (cacheable) {
            std::memset(&key, 0, sizeof(key));
            auto pack2 = [](int a, int b) { return (static_cast<uint64_t>(static_cast<uint32_t>(a)) << 32) | static_cast<uint32_t>(b); };
            const uint64_t words[] = {2, reinterpret_cast<uint64_t>(dev), g_tuning_epoch.load(std::memory_order_acquire),
                                      accumulate ? 1u : 0u, out_mode_word(), static_cast<uint64_t>(Nb),
                                      static_cast<uint64_t>(H), static_cast<uint64_t>(W), static_cast<uint64_t>(Cin),
                                      static_cast<uint64_t>(Cout), pack2(R, S), pack2(stride_h, stride_w),
                                      pack2(pad_h, pad_w), pack2(dil_h, dil_w), reinterpret_cast<uint64_t>(X),
                                      reinterpret_cast<uint64_t>(Wt), reinterpret_cast<uint64_t>(Y)};
            std::memcpy(key.w, words, sizeof(words));
            hit = plan_lookup(key, &p, &pl);
        }
        if (hit) {
            ++g_plan_hits;
        } else {
            pl = make_plan(M, Cout, K, block_k, dev);
            std::memset(&p, 0, sizeof(p));
            fill_common(p, pl, M, Cout, Y, Cout, block_k, true, accumulate, dev);
            p.a_im2col = 1;
            p.conv_wo = static_cast<int>(g.Wo);
            p.conv_howo = static_cast<int>(g.Ho * g.Wo);
            p.conv_s = S;
            p.c_chunks = static_cast<int>(Cin / block_k);
            p.stride_w = stride_w; p.stride_h = stride_h;
            p.pad_w = pad_w; p.pad_h = pad_h;
            p.dil_w = dil_w; p.dil_h = dil_h;
            if ((st = encode_im2col(&p.tmap_a, X, g, block_k, kBlockM)) != MIPGEMM_OK) return st;
            if ((st = encode_tiled_2d(&p.tmap_b, Wt, K, Cout, K, block_k, pl.pair ? pl.block_n / 2 : pl.block_n)) !=
                MIPGEMM_OK)
                return st;
        }
        if ((st = run_dense(p, pl, M, Cout, Y, Cout, accumulate, dev, stream, hit)) != MIPGEMM_OK) return st;
        if (cacheable && !hit) {
            ++g_plan_misses;
            plan_store(key, p, pl);
        }
        tl_last_path = (pl.pair ? MIPGEMM_PATH_DENSE_PAIR : MIPGEMM_PATH_DENSE) | MIPGEMM_PATH_IM2COL_TMA |
                       (pl.split_k > 1 ? MIPGEMM_PATH_SPLITK : 0);
        if (log_enabled()) log_dense("conv (TMA im2col)", M, Cout, K, pl, p, hit);
        return MIPGEMM_OK;
    }

    if (conv_gather_eligible(g) && tun.force_path != MIPGEMM_PATH_IM2COL_EXPLICIT) {
        const int seg = S * static_cast<int>(Cin);
        const int slot = static_cast<int>(round_up(seg, 16));
        const long long Kp = static_cast<long long>(R) * slot;      // K with every filter row padded to its slot
        const int block_k = 128;
        Scratch scratch(dev, stream);
        if ((st = scratch.reserve(align256(static_cast<size_t>(Cout) * Kp))) != MIPGEMM_OK) return st;
        int8_t* wp = static_cast<int8_t*>(scratch.take(static_cast<size_t>(Cout) * Kp));
        cudaError_t e = launch_weight_slots(Wt, wp, Cout, R, seg, slot, stream);
        ++g_launches;
        if (e != cudaSuccess) return cuda_fail(e);
        Plan pl = make_plan(M, Cout, Kp, block_k, dev, 64, 64, /*one_cta_no_split=*/true);
        // Staged form: image rows that are multiples of 16 bytes (bulk copies) and few enough per tile go through
        // two row buffers in shared memory, which the pipeline stages make room for.
        const long long row_bytes = g.W * g.Cin;
        const int span = (R - 1) * dil_h + 1;
        const int rows_max = static_cast<int>((kBlockM - 2) / g.Wo + 2);
        const long long payload = static_cast<long long>(rows_max) * span * row_bytes;
        const long long rowbuf_stride = round_up(payload + slot + 64, 128);
        const int stage_bytes_g = kBlockM * block_k + pl.block_n * block_k;
        const long long table_bytes = 8LL * 8 * ((Kp + block_k - 1) / block_k);      // one entry per 16-byte chunk of A
        const long long room = kSmemBudget - kCtrlBytes - kStagingBytes - 1024 - (64 + 2 * rowbuf_stride + table_bytes);
        const bool staged = MIP_ENV_KNOB("MIPGEMM_NO_STAGED_GATHER", 0) == 0 && row_bytes % 16 == 0 &&
                            reinterpret_cast<uintptr_t>(X) % 16 == 0 && pad_w * g.Cin + 4 <= 64 && payload <= 48 * 1024 &&
                            span <= 4095 && slot <= 8192 &&
                            room >= 3LL * stage_bytes_g;
        if (staged && pl.stages > room / stage_bytes_g) pl.stages = static_cast<int>(room / stage_bytes_g);
        DenseParams p;
        std::memset(&p, 0, sizeof(p));
        fill_common(p, pl, M, Cout, Y, Cout, block_k, true, accumulate, dev);
        p.a_gather = 1;
        p.g_staged = staged ? 1 : 0;
        p.g_span = span;
        p.g_rows_max = rows_max;
        p.g_rowbuf_stride = static_cast<int>(rowbuf_stride);
        p.g_r = R;
        p.g_ho = static_cast<int>(g.Ho);
        p.g_table_bytes = static_cast<int>(table_bytes);
        auto magic = [](long long d, uint32_t* mul, uint32_t* shift) {      // q = (umulhi(mul, n) + n) >> shift, n < 2^31
            uint32_t l = 0;
            while ((1LL << l) < d) ++l;
            *mul = static_cast<uint32_t>(((1ULL << 32) * ((1ULL << l) - static_cast<unsigned long long>(d))) /
                                         static_cast<unsigned long long>(d) + 1);
            *shift = l;
        };
        magic(g.Wo, &p.g_wo_mul, &p.g_wo_shift);
        magic(g.Ho, &p.g_ho_mul, &p.g_ho_shift);
        p.gx = X;
        p.g_xbytes = g.Nb * g.H * g.W * g.Cin;
        p.g_h = static_cast<int>(g.H);
        p.g_row_bytes = static_cast<int>(g.W * g.Cin);
        p.g_cin = static_cast<int>(g.Cin);
        p.g_seg = seg;
        p.g_slot = slot;
        p.g_chunks = static_cast<int>(Kp / 16);
        p.conv_wo = static_cast<int>(g.Wo);
        p.conv_howo = static_cast<int>(g.Ho * g.Wo);
        p.stride_w = stride_w; p.stride_h = stride_h;
        p.pad_w = pad_w; p.pad_h = pad_h;
        p.dil_w = dil_w; p.dil_h = dil_h;
        if ((st = encode_tiled_2d(&p.tmap_b, wp, Kp, Cout, Kp, block_k, pl.block_n)) != MIPGEMM_OK) return st;
        if ((st = run_dense(p, pl, M, Cout, Y, Cout, accumulate, dev, stream)) != MIPGEMM_OK) return st;
        tl_last_path = MIPGEMM_PATH_DENSE | MIPGEMM_PATH_IM2COL_GATHER;
        if (log_enabled()) log_dense("conv (gathered im2col)", M, Cout, Kp, pl, p, false);
        return MIPGEMM_OK;
    }

    // Explicit lowering: materialise the augmented matrix (zero-padded to a 16-byte pitch),
    // then run the GEMM on it.  The weight matrix is re-pitched by the GEMM if K % 16 != 0.
    const long long k_pitch = round_up(K, 16);
    Scratch scratch(dev, stream);
    const size_t cols_bytes = align256(static_cast<size_t>(M) * k_pitch);
    if ((st = scratch.reserve(cols_bytes + gemm_scratch_bytes(M, Cout, K, nullptr, k_pitch, Wt, K))) != MIPGEMM_OK)
        return st;
    uint8_t* cols = static_cast<uint8_t*>(scratch.take(static_cast<size_t>(M) * k_pitch));
    Im2colParams ip{X, cols, g.Nb, g.H, g.W, g.Cin, g.Ho, g.Wo, R, S, stride_h, stride_w,
                    pad_h, pad_w, dil_h, dil_w, K, k_pitch};
    cudaError_t e = launch_im2col(ip, stream);
    ++g_launches;
    if (e != cudaSuccess) return cuda_fail(e);
    if (log_enabled())
        std::fprintf(stderr, "mipgemm: conv M=%lld N=%lld K=%lld -> explicit im2col matrix (pitch %lld), then:\n", M,
                     static_cast<long long>(Cout), K, k_pitch);
    // The GEMM takes its own share (weight re-pitching when K % 16 != 0) from the same lease.
    return gemm_impl(true, M, Cout, K, cols, k_pitch, Wt, K, Y, Cout, accumulate, stream_v,
                     MIPGEMM_PATH_IM2COL_EXPLICIT, &scratch);
}

int mipgemm_device_status(void* stream_v) {
    DeviceState* dev = nullptr;
    int st = get_device(&dev);
    if (st != MIPGEMM_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    cudaError_t e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return cuda_fail(e);
    st = take_status_word(dev->status_word);
    // kernels launched by the allocation-free entry point report through a word of their own
    int dev_index = 0;
    unsigned int* static_word = nullptr;
    if (cudaGetDevice(&dev_index) == cudaSuccess && dev_index >= 0 && dev_index < kMaxDevices) {
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (g_noalloc[dev_index].ready) static_word = g_noalloc[dev_index].st.status_word;
    }
    if (static_word) {
        const int st2 = take_status_word(static_word);
        if (st == MIPGEMM_OK) st = st2;
    }
    return st;
}

int mipgemm_set_workspace(void* dev_ptr, size_t bytes) {
    DeviceState* dev = nullptr;
    int st = get_device(&dev);
    if (st != MIPGEMM_OK) return st;
    if (dev_ptr && reinterpret_cast<uintptr_t>(dev_ptr) % 256 != 0) return MIPGEMM_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_mutex);
    dev->lent = dev_ptr;
    dev->lent_bytes = dev_ptr ? bytes : 0;
    return MIPGEMM_OK;
}

size_t mipgemm_workspace_query_gemm(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                                    const void* B, int64_t ldb, const void* C, int64_t ldc, int accumulate) {
    (void)C; (void)ldc; (void)accumulate;
    return gemm_scratch_bytes(M, N, K, A, lda, B, ldb);
}

size_t mipgemm_workspace_query_conv(int64_t Nb, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int R, int S,
                                    int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w) {
    ConvGeom g{Nb, H, W, Cin, Cout, 0, 0, R, S, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w};
    if (!conv_geometry(g)) return 0;
    // Assumes 16-byte aligned tensors (any cudaMalloc'ed or framework-allocated buffer).
    const long long M = g.Nb * g.Ho * g.Wo;
    if (conv_is_pointwise(g)) return gemm_scratch_bytes(M, Cout, Cin, nullptr, Cin, nullptr, Cin);
    if (conv_tma_eligible(g, nullptr, nullptr)) return 0;
    if (conv_gather_eligible(g)) return align256(static_cast<size_t>(Cout) * R * round_up(static_cast<long long>(S) * Cin, 16));
    const long long K = static_cast<long long>(R) * S * Cin;
    const long long k_pitch = round_up(K, 16);
    return align256(static_cast<size_t>(M) * k_pitch) + gemm_scratch_bytes(M, Cout, K, nullptr, k_pitch, nullptr, K);
}

int mipgemm_host_s8s8s32(int64_t M, int64_t N, int64_t K, const int8_t* A, int64_t lda, const int8_t* B,
                         int64_t ldb, int32_t* C, int64_t ldc, int accumulate, void* stream) {
    return host_impl(false, M, N, K, A, lda, B, ldb, C, ldc, accumulate, stream);
}

int mipgemm_host_u8s8s32(int64_t M, int64_t N, int64_t K, const uint8_t* A, int64_t lda, const int8_t* B,
                         int64_t ldb, int32_t* C, int64_t ldc, int accumulate, void* stream) {
    return host_impl(true, M, N, K, A, lda, B, ldb, C, ldc, accumulate, stream);
}

// Fused dequantisation: run the integer entry point with the output transform switched on for
// this thread.  (float 0.0 and int32 0 share their bit pattern, so the K == 0 zero fill is right.)
struct OutputTransformScope {
    OutputTransformScope(float scale) { tl_out_f32 = 1; tl_out_scale = scale; }
    ~OutputTransformScope() { tl_out_f32 = 0; tl_out_scale = 1.0f; }
};

int mipgemm_s8s8f32_dequant(int64_t M, int64_t N, int64_t K, const int8_t* A, int64_t lda, const int8_t* B,
                            int64_t ldb, float* C, int64_t ldc, float scale, void* stream) {
    OutputTransformScope scope(scale);
    return gemm_impl(false, M, N, K, A, lda, B, ldb, reinterpret_cast<int32_t*>(C), ldc, 0, stream, 0);
}

int mipgemm_u8s8f32_dequant(int64_t M, int64_t N, int64_t K, const uint8_t* A, int64_t lda, const int8_t* B,
                            int64_t ldb, float* C, int64_t ldc, float scale, void* stream) {
    OutputTransformScope scope(scale);
    return gemm_impl(true, M, N, K, A, lda, B, ldb, reinterpret_cast<int32_t*>(C), ldc, 0, stream, 0);
}

int mipgemm_conv_u8s8f32_dequant(int64_t Nb, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int R, int S,
                                 int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w,
                                 const uint8_t* X, const int8_t* Wt, float* Y, float scale, void* stream) {
    OutputTransformScope scope(scale);
    return mipgemm_conv_u8s8s32(Nb, H, W, Cin, Cout, R, S, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w, X, Wt,
                                reinterpret_cast<int32_t*>(Y), 0, stream);
}

// Requantisation to 8-bit codes: the integer entry point runs with the epilogue's code transform
// switched on for this thread; C / Y then address bytes.
struct RequantScope {
    RequantScope(float scale, int lo, int hi) { tl_out_q8 = 1; tl_q_lo = lo; tl_q_hi = hi; tl_out_scale = scale; }
    ~RequantScope() { tl_out_q8 = 0; tl_q_lo = tl_q_hi = 0; tl_out_scale = 1.0f; }
};

int mipgemm_s8s8s8_requant(int64_t M, int64_t N, int64_t K, const int8_t* A, int64_t lda, const int8_t* B,
                           int64_t ldb, int8_t* C, int64_t ldc, float scale, int relu, void* stream) {
    if (!std::isfinite(scale)) return MIPGEMM_ERR_INVALID_ARG;
    RequantScope scope(scale, relu ? 0 : -128, 127);
    return gemm_impl(false, M, N, K, A, lda, B, ldb, reinterpret_cast<int32_t*>(C), ldc, 0, stream, 0);
}

int mipgemm_u8s8u8_requant(int64_t M, int64_t N, int64_t K, const uint8_t* A, int64_t lda, const int8_t* B,
                           int64_t ldb, uint8_t* C, int64_t ldc, float scale, void* stream) {
    if (!std::isfinite(scale)) return MIPGEMM_ERR_INVALID_ARG;
    RequantScope scope(scale, 0, 255);
    return gemm_impl(true, M, N, K, A, lda, B, ldb, reinterpret_cast<int32_t*>(C), ldc, 0, stream, 0);
}

int mipgemm_conv_u8s8u8_requant(int64_t Nb, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int R, int S,
                                int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w,
                                const uint8_t* X, const int8_t* Wt, uint8_t* Y, float scale, void* stream) {
    if (!std::isfinite(scale)) return MIPGEMM_ERR_INVALID_ARG;
    RequantScope scope(scale, 0, 255);
    return mipgemm_conv_u8s8s32(Nb, H, W, Cin, Cout, R, S, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w, X, Wt,
                                reinterpret_cast<int32_t*>(Y), 0, stream);
}

// The same fused transforms with a per-output-channel bias added to the exact sums first.
struct BiasScope {
    explicit BiasScope(const int32_t* bias) { tl_bias = bias; }
    ~BiasScope() { tl_bias = nullptr; }
};
static bool bias_ok(const int32_t* bias) { return reinterpret_cast<uintptr_t>(bias) % 4 == 0; }

int mipgemm_s8s8f32_dequant_bias(int64_t M, int64_t N, int64_t K, const int8_t* A, int64_t lda, const int8_t* B,
                                 int64_t ldb, float* C, int64_t ldc, float scale, const int32_t* bias,
                                 void* stream) {
    if (!bias_ok(bias)) return MIPGEMM_ERR_INVALID_ARG;
    BiasScope with_bias(bias);
    return mipgemm_s8s8f32_dequant(M, N, K, A, lda, B, ldb, C, ldc, scale, stream);
}

int mipgemm_u8s8f32_dequant_bias(int64_t M, int64_t N, int64_t K, const uint8_t* A, int64_t lda, const int8_t* B,
                                 int64_t ldb, float* C, int64_t ldc, float scale, const int32_t* bias,
                                 void* stream) {
    if (!bias_ok(bias)) return MIPGEMM_ERR_INVALID_ARG;
    BiasScope with_bias(bias);
    return mipgemm_u8s8f32_dequant(M, N, K, A, lda, B, ldb, C, ldc, scale, stream);
}

int mipgemm_conv_u8s8f32_dequant_bias(int64_t Nb, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int R, int S,
                                      int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w,
                                      const uint8_t* X, const int8_t* Wt, float* Y, float scale,
                                      const int32_t* bias, void* stream) {
    if (!bias_ok(bias)) return MIPGEMM_ERR_INVALID_ARG;
    BiasScope with_bias(bias);
    return mipgemm_conv_u8s8f32_dequant(Nb, H, W, Cin, Cout, R, S, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w,
                                        X, Wt, Y, scale, stream);
}

int mipgemm_s8s8s8_requant_bias(int64_t M, int64_t N, int64_t K, const int8_t* A, int64_t lda, const int8_t* B,
                                int64_t ldb, int8_t* C, int64_t ldc, float scale, int relu, const int32_t* bias,
                                void* stream) {
    if (!bias_ok(bias)) return MIPGEMM_ERR_INVALID_ARG;
    BiasScope with_bias(bias);
    return mipgemm_s8s8s8_requant(M, N, K, A, lda, B, ldb, C, ldc, scale, relu, stream);
}

int mipgemm_u8s8u8_requant_bias(int64_t M, int64_t N, int64_t K, const uint8_t* A, int64_t lda, const int8_t* B,
                                int64_t ldb, uint8_t* C, int64_t ldc, float scale, const int32_t* bias,
                                void* stream) {
    if (!bias_ok(bias)) return MIPGEMM_ERR_INVALID_ARG;
    BiasScope with_bias(bias);
    return mipgemm_u8s8u8_requant(M, N, K, A, lda, B, ldb, C, ldc, scale, stream);
}

int mipgemm_conv_u8s8u8_requant_bias(int64_t Nb, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int R, int S,
                                     int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w,
                                     const uint8_t* X, const int8_t* Wt, uint8_t* Y, float scale,
                                     const int32_t* bias, void* stream) {
    if (!bias_ok(bias)) return MIPGEMM_ERR_INVALID_ARG;
    BiasScope with_bias(bias);
    return mipgemm_conv_u8s8u8_requant(Nb, H, W, Cin, Cout, R, S, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w,
                                       X, Wt, Y, scale, stream);
}

int mipgemm_batched_s8s8s32(int64_t batch, int64_t M, int64_t N, int64_t K, const int8_t* A, int64_t lda,
                            int64_t stride_a, const int8_t* B, int64_t ldb, int64_t stride_b, int32_t* C, int64_t ldc,
                            int64_t stride_c, int accumulate, void* stream) {
    return batched_impl(false, batch, M, N, K, A, lda, stride_a, B, ldb, stride_b, C, ldc, stride_c, accumulate, stream);
}

int mipgemm_batched_u8s8s32(int64_t batch, int64_t M, int64_t N, int64_t K, const uint8_t* A, int64_t lda,
                            int64_t stride_a, const int8_t* B, int64_t ldb, int64_t stride_b, int32_t* C, int64_t ldc,
                            int64_t stride_c, int accumulate, void* stream) {
    return batched_impl(true, batch, M, N, K, A, lda, stride_a, B, ldb, stride_b, C, ldc, stride_c, accumulate, stream);
}

int mipgemm_gemm_ex(int a_unsigned, int b_unsigned, int a_order, int b_order, int c_col_major, int64_t M, int64_t N,
                    int64_t K, const void* A, int64_t lda, const void* B, int64_t ldb, int32_t* C, int64_t ldc,
                    int accumulate, void* stream) {
    return gemm_ex_impl(a_unsigned, b_unsigned, a_order, b_order, c_col_major, M, N, K, A, lda, B, ldb, C, ldc,
                        accumulate, stream);
}

uint64_t mipgemm_launch_count(void) { return g_launches.load(); }

int mipgemm_release_staging(void) {
    DeviceState* dev = nullptr;
    int st = get_device(&dev);
    if (st != MIPGEMM_OK) return st;
    std::lock_guard<std::mutex> host_lock(dev->host_mutex);
    if (dev->staging) {
        cudaError_t e = cudaFree(dev->staging);
        dev->staging = nullptr;
        dev->staging_bytes = 0;
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return MIPGEMM_OK;
}

int mipgemm_plan_cache_stats(uint64_t* hits, uint64_t* misses) {
    if (hits) *hits = g_plan_hits.load();
    if (misses) *misses = g_plan_misses.load();
    return plan_cache_enabled() ? 1 : 0;
}

int mipgemm_last_path(void) { return tl_last_path; }
int mipgemm_last_cuda_error(void) { return tl_last_cuda_error; }

const char* mipgemm_status_string(int status) {
    switch (status) {
        case MIPGEMM_OK: return "ok";
        case MIPGEMM_ERR_INVALID_ARG: return "invalid argument";
        case MIPGEMM_ERR_K_TOO_LARGE: return "K too large for a guaranteed exact int32 result";
        case MIPGEMM_ERR_UNSUPPORTED: return "device is not compute capability 10.0 (sm_100a)";
        case MIPGEMM_ERR_WORKSPACE: return "scratch memory unavailable or lent buffer too small";
        case MIPGEMM_ERR_CUDA: return "CUDA call failed";
        case MIPGEMM_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case MIPGEMM_ERR_STATIC_SCRATCH_LIMIT:
            return "operands need more re-pitching scratch than the built-in static buffer holds";
        default: return "unknown status";
    }
}

int mipgemm_version(void) { return 100; }

int mipgemm_probe_i8_peak(int iters, int* grid_out, double* ops_per_launch, int32_t* sink, void* stream_v) {
    if (iters <= 0 || !sink) return MIPGEMM_ERR_INVALID_ARG;
    DeviceState* dev = nullptr;
    int st = get_device(&dev);
    if (st != MIPGEMM_OK) return st;
    const int grid = dev->sm_count;
    cudaError_t e = launch_probe(iters, grid, sink, static_cast<cudaStream_t>(stream_v));
    ++g_launches;
    if (e != cudaSuccess) return cuda_fail(e);
    if (grid_out) *grid_out = grid;
    if (ops_per_launch) *ops_per_launch = 2.0 * 128 * 256 * 128 * static_cast<double>(iters) * grid;
    return MIPGEMM_OK;
}

int mipgemm_set_weights_constant(int on) {
    g_weights_constant.store(on != 0 ? 1 : 0);
    return MIPGEMM_OK;
}

int mipgemm_register_constant_weights(const void* base, size_t bytes) {
    if (!base || bytes == 0) return MIPGEMM_ERR_INVALID_ARG;
    const uintptr_t lo = reinterpret_cast<uintptr_t>(base);
    std::lock_guard<std::mutex> lock(g_ranges_mutex);
    g_constant_ranges[lo] = lo + bytes;
    g_constant_range_count.store(static_cast<int>(g_constant_ranges.size()), std::memory_order_release);
    return MIPGEMM_OK;
}

int mipgemm_unregister_constant_weights(const void* base) {
    std::lock_guard<std::mutex> lock(g_ranges_mutex);
    if (g_constant_ranges.erase(reinterpret_cast<uintptr_t>(base)) == 0) return MIPGEMM_ERR_INVALID_ARG;
    g_constant_range_count.store(static_cast<int>(g_constant_ranges.size()), std::memory_order_release);
    return MIPGEMM_OK;
}

int mipgemm_debug_set(int flags, unsigned long long wait_budget_ns) {
    if (flags & ~1) return MIPGEMM_ERR_INVALID_ARG;
    g_debug_flags.store(flags);
    g_wait_budget_ns.store(wait_budget_ns ? wait_budget_ns : 4000000000ull);
    g_tuning_epoch.fetch_add(1, std::memory_order_acq_rel);   // cached launch parameters carry the old values
    return MIPGEMM_OK;
}

int mipgemm_set_tuning(int block_n, int stages, int split_k, int force_path) {
    if (block_n != 0 && (block_n < 32 || block_n > 256 || block_n % 32 != 0)) return MIPGEMM_ERR_INVALID_ARG;
    if (stages < 0 || stages > mip::kMaxStages || split_k < 0 || force_path < 0 || force_path > 0xFFFFFF)
        return MIPGEMM_ERR_INVALID_ARG;
    Tuning t;
    t.block_n = block_n;
    t.stages = stages;
    t.split_k = split_k > 0xFFFF ? 0xFFFF : split_k;
    t.force_path = force_path;
    g_tuning_word.store(pack_tuning(t), std::memory_order_release);
    g_tuning_epoch.fetch_add(1, std::memory_order_acq_rel);
    return MIPGEMM_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------
// Allocation-free GEMM entry point.
//
// Everything above obtains its scratch memory (and one status word per device) from the
// CUDA allocator.  Some callers cannot do that: code running inside a memory-planned
// inference runtime that owns every byte of the device, a real-time loop that must never
// enter the driver's allocator, a process whose memory pool has been handed over entirely
// to another framework.  For them the re-pitching GEMM exists once more below with its
// scratch in a fixed array that is part of the library image on every GPU that loads it.
// Nothing on this path calls cudaMalloc, cudaMallocAsync, cudaFree or any other allocating
// routine.  It shares the planner, the tensor-map encoders, the tuning overrides, the launch
// counter and the per-thread last-path / last-error words with the entry points above, but
// none of their device memory: its scratch and its status word are the two static symbols
// defined near the top of this file.
// ---------------------------------------------------------------------------------------
namespace {

// Per-device set-up, done by the first call on each device with that device current:
// capability check, tensor-map encoders, kernel attributes and the DEVICE addresses of the
// two static symbols.  No allocation.
int noalloc_device(NoAllocDevice** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    thread_local int tl_context_bound = -1;      // (binds the device's context to this thread, see get_device())
    if (tl_context_bound != dev) {
        if ((e = cudaSetDevice(dev)) != cudaSuccess) return cuda_fail(e);
        tl_context_bound = dev;
    }
    if (dev < 0 || dev >= kMaxDevices) return MIPGEMM_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    NoAllocDevice& d = g_noalloc[dev];
    if (!d.ready) {
        int major = 0, minor = 0;
        if ((e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev)) != cudaSuccess ||
            (e = cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev)) != cudaSuccess ||
            (e = cudaDeviceGetAttribute(&d.st.sm_count, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
            return cuda_fail(e);
        if (major != 10 || minor != 0) {
            d.status = MIPGEMM_ERR_UNSUPPORTED;
        } else {
            {
                std::lock_guard<std::mutex> lock2(g_mutex);   // the encoder pointers are shared
                if (!g_encode_tiled) {
                    void* fn = nullptr;
                    cudaDriverEntryPointQueryResult qr;
                    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr);
                    if (e != cudaSuccess || qr != cudaDriverEntryPointSuccess || !fn)
                        return cuda_fail(e == cudaSuccess ? cudaErrorUnknown : e);
                    g_encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
                }
            }
            if ((e = dense_init()) != cudaSuccess) return cuda_fail(e);
            d.st.pair_clusters = dense_pair_max_clusters(kSmemBudget);
            void* ptr = nullptr;
            if ((e = cudaGetSymbolAddress(&ptr, g_static_scratch)) != cudaSuccess) return cuda_fail(e);
            d.scratch = static_cast<unsigned char*>(ptr);
            ptr = nullptr;
            if ((e = cudaGetSymbolAddress(&ptr, g_static_status)) != cudaSuccess) return cuda_fail(e);
            d.st.status_word = static_cast<unsigned int*>(ptr);
            d.status = MIPGEMM_OK;
        }
        d.ready = true;
    }
    *out = &d;
    return d.status;
}

}  // namespace

extern "C" int mipgemm_s8s8s32_static_scratch(int64_t M, int64_t N, int64_t K, const int8_t* A, int64_t lda,
                                              const int8_t* B, int64_t ldb, int32_t* C, int64_t ldc,
                                              int accumulate, void* stream_v) {
    tl_last_path = MIPGEMM_PATH_NONE;
    if (M < 0 || N < 0 || K < 0) return MIPGEMM_ERR_INVALID_ARG;
    if (M > 0x7FFFFF00LL || N > 0x7FFFFF00LL) return MIPGEMM_ERR_INVALID_ARG;
    if (lda < K || ldb < K || ldc < N) return MIPGEMM_ERR_INVALID_ARG;
    if (K > 131071) return MIPGEMM_ERR_K_TOO_LARGE;
    if (M == 0 || N == 0) {
        tl_last_path = MIPGEMM_PATH_TRIVIAL;
        return MIPGEMM_OK;
    }
    if (!C || reinterpret_cast<uintptr_t>(C) % 4 != 0) return MIPGEMM_ERR_INVALID_ARG;
    if (K > 0 && (!A || !B)) return MIPGEMM_ERR_INVALID_ARG;
    // How much of the static array this call needs; refuse before anything is enqueued.
    const size_t need = gemm_scratch_bytes(M, N, K, A, lda, B, ldb);
    if (need > static_cast<size_t>(MIPGEMM_STATIC_SCRATCH_BYTES)) return MIPGEMM_ERR_STATIC_SCRATCH_LIMIT;

    NoAllocDevice* nd = nullptr;
    int st = noalloc_device(&nd);
    if (st != MIPGEMM_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    cudaError_t e;
    if (K == 0) {
        if (!accumulate) {
            if ((e = launch_fill_zero(C, ldc, M, N, stream)) != cudaSuccess) return cuda_fail(e);
            ++g_launches;
        }
        tl_last_path = MIPGEMM_PATH_TRIVIAL;
        return MIPGEMM_OK;
    }

    // Re-pitch whatever TMA cannot address into the static array.  Every byte the GEMM kernel
    // will read from the array (K bytes of M, respectively N, rows) is written here first, so
    // nothing left behind by an earlier call can reach the result and nothing needs clearing.
    const long long pitch = round_up(K, 16);
    const void* a_use = A;
    const void* b_use = B;
    long long lda_use = lda, ldb_use = ldb;
    size_t used = 0;
    int flags = 0;
    if (!aligned16(A, lda)) {
        unsigned char* dst = nd->scratch + used;
        used += align256(static_cast<size_t>(M) * pitch);
        if ((e = launch_repack(A, lda, dst, pitch, M, K, stream)) != cudaSuccess) return cuda_fail(e);
        ++g_launches;
        a_use = dst;
        lda_use = pitch;
        flags |= MIPGEMM_PATH_REPACK;
    }
    if (!aligned16(B, ldb)) {
        unsigned char* dst = nd->scratch + used;
        used += align256(static_cast<size_t>(N) * pitch);
        if ((e = launch_repack(B, ldb, dst, pitch, N, K, stream)) != cudaSuccess) return cuda_fail(e);
        ++g_launches;
        b_use = dst;
        ldb_use = pitch;
        flags |= MIPGEMM_PATH_REPACK;
    }

    const int block_k = 128;
    const Plan pl = make_plan(M, N, K, block_k, &nd->st);
    DenseParams p;
    std::memset(&p, 0, sizeof(p));
    fill_common(p, pl, M, N, C, ldc, block_k, false, accumulate, &nd->st);
    if ((st = encode_tiled_2d(&p.tmap_a, a_use, K, M, lda_use, block_k, kBlockM)) != MIPGEMM_OK) return st;
    if ((st = encode_tiled_2d(&p.tmap_b, b_use, K, N, ldb_use, block_k, pl.pair ? pl.block_n / 2 : pl.block_n)) !=
        MIPGEMM_OK)
        return st;
    if ((st = run_dense(p, pl, M, N, C, ldc, accumulate, &nd->st, stream)) != MIPGEMM_OK) return st;
    if (pl.split_k > 1) flags |= MIPGEMM_PATH_SPLITK;
    tl_last_path = (pl.pair ? MIPGEMM_PATH_DENSE_PAIR : MIPGEMM_PATH_DENSE) | flags;
    return MIPGEMM_OK;
}

// Allocation-free status query for the entry point above: waits for `stream`, then reads and clears
// the static status word (plain copies from and to the symbol's address; nothing is allocated).
extern "C" int mipgemm_static_scratch_status(void* stream_v) {
    NoAllocDevice* nd = nullptr;
    int st = noalloc_device(&nd);
    if (st != MIPGEMM_OK) return st;
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream_v));
    if (e != cudaSuccess) return cuda_fail(e);
    return take_status_word(nd->st.status_word);
}
