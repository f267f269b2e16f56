/*
 * libmipgemm -- exact mixed-precision integer GEMM for NVIDIA B200 (sm_100a).
 *
 *     C(int32) [+]= A(int8 | uint8) * B(int8)
 *
 * This is the hot path of "mixed-precision integer (MIP) GEMM" for quantized
 * inference: 8-bit operands, 32-bit exact accumulation (paper Section 5,
 * opening paragraphs; Section 7.3, C^q = A^q B^q; Figure 1, C += A B), its use
 * for convolution through the im2col lowering (Section 7.2) and for the
 * weight-by-activation GEMMs of a transformer encoder (Table 5), and the
 * matrix-vector / skinny case of the final fully connected layer (Section 7.4,
 * "2mn useful operations").
 *
 * Conventions common to every entry point
 * ---------------------------------------
 *  - All data pointers are DEVICE pointers on the current CUDA device, owned by
 *    the caller; the library neither frees nor retains them.  `stream` is a
 *    cudaStream_t passed as void* (NULL = legacy default stream).  Calls are
 *    asynchronous: they return after the work has been enqueued.
 *  - Return value: MIPGEMM_OK (0) or one of the error codes below.  Argument
 *    errors are detected synchronously and nothing is enqueued.  Device-side
 *    problems (a bounded wait that ran out) are reported by
 *    mipgemm_device_status().
 *  - Exactness: the result equals the mathematical value whenever that value
 *    fits int32.  With accumulate == 0 this is unconditional, because K is
 *    limited so that the worst case cannot overflow: K <= 131071 in s8*s8 mode
 *    (128*128*K <= 2^31-1) and K <= 65793 in u8*s8 mode (255*128*K <= 2^31);
 *    larger K returns MIPGEMM_ERR_K_TOO_LARGE.  With accumulate != 0 the sum
 *    C_in + A*B wraps modulo 2^32 if it leaves the int32 range; keeping it in
 *    range is the caller's responsibility.  There is no saturation anywhere.
 *  - A, B and C must not overlap.  A and B need byte alignment only; C needs
 *    4-byte alignment.  Any pitch >= the minimum is accepted; operands whose
 *    base or pitch is not 16-byte aligned are first copied into scratch memory
 *    (see "Scratch memory").
 *  - Padding elements of C (columns N .. ldc-1 of a row) are never written.
 *  - M == 0 or N == 0: no-op, MIPGEMM_OK.  K == 0: C is zero-filled
 *    (accumulate == 0) or left unchanged (accumulate != 0).
 *
 * Threads
 * -------
 * Entry points may be called from several host threads at once, on the same or on different
 * streams and devices: per-device set-up is serialised internally, mipgemm_last_path() and
 * mipgemm_last_cuda_error() are per thread.  Process-wide switches (mipgemm_set_tuning,
 * mipgemm_set_weights_constant, mipgemm_set_workspace) take effect atomically for calls that
 * start after they return; they are meant to be set up front, not raced with compute calls.
 * Calls that share memory must be ordered by the caller as with any CUDA work: a lent workspace
 * (one stream at a time), the static array of mipgemm_s8s8s32_static_scratch, and the staging
 * streams of the host-buffer entry points (calls of those are serialised per device).
 *
 * Scratch memory
 * --------------
 * Some calls need global scratch memory (operand re-pitching, slot-padded
 * filters for convolutions gathered in software, the explicit im2col matrix
 * for the few convolutions neither the TMA nor the gather warps can handle).
 * By default it is taken with cudaMallocAsync on the call's stream and
 * released with cudaFreeAsync after the last kernel of the call.  A caller may instead lend a buffer with mipgemm_set_workspace(); calls
 * that need more than was lent fail with MIPGEMM_ERR_WORKSPACE.  A lent buffer
 * is shared by all calls: calls that use it must be ordered on one stream.
 */
#ifndef MIPGEMM_H_
#define MIPGEMM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MIPGEMM_OK = 0,
    MIPGEMM_ERR_INVALID_ARG = 1, /* NULL pointer, negative size, pitch too small, bad conv geometry */
    MIPGEMM_ERR_K_TOO_LARGE = 2, /* exactness could not be guaranteed (see above)                  */
    MIPGEMM_ERR_UNSUPPORTED = 3, /* current device is not compute capability 10.0                  */
    MIPGEMM_ERR_WORKSPACE = 4,   /* scratch memory could not be obtained / lent buffer too small   */
    MIPGEMM_ERR_CUDA = 5,        /* a CUDA call failed; see mipgemm_last_cuda_error()              */
    MIPGEMM_ERR_TIMEOUT = 6,     /* a bounded device-side wait expired (kernel returned early)     */
    MIPGEMM_ERR_STATIC_SCRATCH_LIMIT = 7 /* mipgemm_s8s8s32_static_scratch: operands too large for  */
                                         /* the built-in scratch array (nothing was enqueued)        */
} mipgemm_status_t;

/* Which kernel family served the most recent GEMM/conv call of this thread (test hook). */
typedef enum {
    MIPGEMM_PATH_NONE = 0,
    MIPGEMM_PATH_DENSE = 1,       /* TMA + tcgen05.mma.kind::i8, one CTA per tile            */
    MIPGEMM_PATH_DENSE_PAIR = 2,  /* same, CTA pairs (cta_group::2)                          */
    MIPGEMM_PATH_SKINNY = 3,      /* M <= 16 streaming kernel                                */
    MIPGEMM_PATH_TRIVIAL = 4,     /* K == 0 fill or empty problem                            */
    MIPGEMM_PATH_REPACK = 0x100,  /* flag: an operand was re-pitched into scratch first      */
    MIPGEMM_PATH_SPLITK = 0x200,  /* flag: K was split over CTAs (partials added exactly)    */
    MIPGEMM_PATH_IM2COL_TMA = 0x400,   /* flag: conv gathered by TMA im2col loads            */
    MIPGEMM_PATH_IM2COL_EXPLICIT = 0x800, /* flag: conv materialised the augmented matrix    */
    MIPGEMM_PATH_BATCHED = 0x1000,     /* flag: a whole strided batch ran as one launch       */
    MIPGEMM_PATH_IM2COL_GATHER = 0x2000 /* flag: conv gathered into shared memory by extra warps */
} mipgemm_path_t;

/*
 * C = [C +] A * B, signed 8-bit A.   (Paper: Figure 1 and Section 5 -- INT8
 * products, INT32 accumulation; the result is the exact integer matrix product.)
 *
 *   A : row-major    M x K, a(i,k) = A[i*lda + k], lda >= K          (device, read)
 *   B : column-major K x N, b(k,j) = B[j*ldb + k], ldb >= K          (device, read)
 *       -- i.e. N runs of K contiguous bytes, the usual [out][in] weight layout
 *   C : row-major    M x N, c(i,j) = C[i*ldc + j], ldc >= N          (device, read/write)
 *   accumulate : 0 -> C = A*B, previous contents of C are ignored;
 *                nonzero -> C += A*B.
 *   stream : cudaStream_t.
 */
int mipgemm_s8s8s32(int64_t M, int64_t N, int64_t K,
                    const int8_t *A, int64_t lda,
                    const int8_t *B, int64_t ldb,
                    int32_t *C, int64_t ldc,
                    int accumulate, void *stream);

/* Same with unsigned 8-bit A (zero-extended), e.g. post-ReLU activations.  The
 * paper's kernels are signed*signed; the unsigned variant follows the same
 * definition with a(i,k) in [0,255] and has no zero-point term. */
int mipgemm_u8s8s32(int64_t M, int64_t N, int64_t K,
                    const uint8_t *A, int64_t lda,
                    const int8_t *B, int64_t ldb,
                    int32_t *C, int64_t ldc,
                    int accumulate, void *stream);

/*
 * Y = [Y +] Conv(Wt, X): channel-last convolution lowered to the GEMM above
 * (paper Section 7.2: O = Conv(F, I), im2col lowering, the cost of the
 * lowering is part of the operator).  GEMM view: M = Nb*Ho*Wo output pixels,
 * N = Cout, K = R*S*Cin ordered (r, s, c).
 *
 *   X  : [Nb][H][W][Cin]      uint8, dense                           (device, read)
 *   Wt : [Cout][R][S][Cin]    int8, dense                            (device, read)
 *   Y  : [Nb][Ho][Wo][Cout]   int32, dense                           (device, read/write)
 *        Ho = (H + 2*pad_h - dil_h*(R-1) - 1)/stride_h + 1, Wo likewise.
 *   Taps that fall outside the image contribute 0 (scale-only quantization, no
 *   zero point).  K = R*S*Cin obeys the u8*s8 limit above.
 */
int mipgemm_conv_u8s8s32(int64_t Nb, int64_t H, int64_t W, int64_t Cin, int64_t Cout,
                         int R, int S, int stride_h, int stride_w,
                         int pad_h, int pad_w, int dil_h, int dil_w,
                         const uint8_t *X, const int8_t *Wt, int32_t *Y,
                         int accumulate, void *stream);

/*
 * Requantised output: C = sat8(rne(scale * (A * B))), one byte per element (paper Section 7.3 read
 * backwards: the integer result is scaled back into the 8-bit range so that the next layer can
 * consume integers again; the paper itself dequantises to FP32 between layers, so this is an
 * extension of its pipeline).  Rule, in binary32: t = fl32(fl32(sum) * scale), both roundings to
 * nearest even; r = t rounded to the nearest integer, ties to even; code = min(max(r, lo), hi) with
 * (lo, hi) = (-128, 127) for int8 codes, (0, 127) with relu != 0, and (0, 255) for uint8 codes (which
 * therefore include a ReLU).  C then never exists as int32 in memory: a quarter of the bytes.
 *
 *   C : device, M x N bytes row-major, ldc >= N counted in bytes, any alignment (16-byte aligned
 *       base and pitch store fastest).  No accumulate form.  scale must be finite.
 * Everything else (operands, K limits, errors, stream semantics) as for mipgemm_s8s8s32 /
 * mipgemm_u8s8s32 / mipgemm_conv_u8s8s32.
 */
int mipgemm_s8s8s8_requant(int64_t M, int64_t N, int64_t K,
                           const int8_t *A, int64_t lda, const int8_t *B, int64_t ldb,
                           int8_t *C, int64_t ldc, float scale, int relu, void *stream);
int mipgemm_u8s8u8_requant(int64_t M, int64_t N, int64_t K,
                           const uint8_t *A, int64_t lda, const int8_t *B, int64_t ldb,
                           uint8_t *C, int64_t ldc, float scale, void *stream);
int mipgemm_conv_u8s8u8_requant(int64_t Nb, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int R, int S,
                                int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w,
                                const uint8_t *X, const int8_t *Wt, uint8_t *Y, float scale, void *stream);

/*
 * General form (paper Section 3, last paragraph: a general GEMM supports transposed inputs and
 * both storage orders for all three operands; the effects on A and B are absorbed below the
 * micro-kernel and a column-major C is handled by swapping the roles of A and B).
 *
 *   a_unsigned, b_unsigned : 0 = int8 (sign-extended), 1 = uint8 (zero-extended), per operand
 *   a_order : MIPGEMM_K_CONTIGUOUS  a(i,k) = A[i*lda + k] (row-major,    lda >= K)
 *             MIPGEMM_MN_CONTIGUOUS a(i,k) = A[k*lda + i] (column-major, lda >= M)
 *   b_order : MIPGEMM_K_CONTIGUOUS  b(k,j) = B[j*ldb + k] (column-major, ldb >= K)
 *             MIPGEMM_MN_CONTIGUOUS b(k,j) = B[k*ldb + j] (row-major,    ldb >= N)
 *   c_col_major : 0  c(i,j) = C[i*ldc + j] (ldc >= N);  1  c(i,j) = C[j*ldc + i] (ldc >= M)
 *
 * K limits for a guaranteed exact result: 131071 (s8*s8), 65793 (one operand unsigned), 33025
 * (u8*u8).  Operands whose base or pitch is not 16-byte aligned are re-pitched (transposed, when
 * M/N-contiguous) into scratch memory first.  Everything else as for mipgemm_s8s8s32.
 */
typedef enum { MIPGEMM_K_CONTIGUOUS = 0, MIPGEMM_MN_CONTIGUOUS = 1 } mipgemm_order_t;
int mipgemm_gemm_ex(int a_unsigned, int b_unsigned, int a_order, int b_order, int c_col_major,
                    int64_t M, int64_t N, int64_t K,
                    const void *A, int64_t lda, const void *B, int64_t ldb,
                    int32_t *C, int64_t ldc, int accumulate, void *stream);

/*
 * Strided batch of independent GEMMs:  C_b [+]= A_b * B_b,  b = 0 .. batch-1, with
 * A_b = A + b*stride_a, B_b = B + b*stride_b, C_b = C + b*stride_c (strides in elements) and each
 * member laid out exactly as in mipgemm_s8s8s32.  This is the shape of the per-head,
 * per-sentence products of a transformer's attention (paper Table 5: M5, l x l x d/h, and M7,
 * d/h x l x l), which the paper leaves in FP32; an int8 variant is offered here as the natural
 * extension.  The C matrices must not overlap (stride_c >= (M-1)*ldc + N); stride_a / stride_b may
 * be 0 to share an operand.  When all operands are 16-byte addressable (bases, pitches and batch
 * strides) the batch runs as a single launch; otherwise the members are computed one after the
 * other.  Same limits and return codes as the single GEMM.
 */
int mipgemm_batched_s8s8s32(int64_t batch, int64_t M, int64_t N, int64_t K,
                            const int8_t *A, int64_t lda, int64_t stride_a,
                            const int8_t *B, int64_t ldb, int64_t stride_b,
                            int32_t *C, int64_t ldc, int64_t stride_c,
                            int accumulate, void *stream);
int mipgemm_batched_u8s8s32(int64_t batch, int64_t M, int64_t N, int64_t K,
                            const uint8_t *A, int64_t lda, int64_t stride_a,
                            const int8_t *B, int64_t ldb, int64_t stride_b,
                            int32_t *C, int64_t ldc, int64_t stride_c,
                            int accumulate, void *stream);

/*
 * Fused dequantisation (paper Section 7.3: with A ~ s_A A^q and B ~ s_B B^q, the real-valued
 * product is approximated by C^r = s_A s_B C^q; the paper applies the scale as a separate, cheap
 * floating-point step after the integer GEMM).  These entry points compute the same exact int32
 * sums as the ones above and write  C(float32) = scale * sum  from the epilogue, so C is written
 * once as float and never exists as int32 in memory.  `scale` is the caller's s_A * s_B.
 * Rounding (the paper fixes none): the int32 sum is converted to binary32 with round-to-nearest-
 * even and multiplied by `scale` in binary32 (round-to-nearest-even); the result is therefore
 * within 2^-23 relative of the real number scale*sum, and bit-identical across kernel paths.
 * Same layouts, limits and return codes as the int32 entry points; there is no accumulate form.
 */
int mipgemm_s8s8f32_dequant(int64_t M, int64_t N, int64_t K,
                            const int8_t *A, int64_t lda, const int8_t *B, int64_t ldb,
                            float *C, int64_t ldc, float scale, void *stream);
int mipgemm_u8s8f32_dequant(int64_t M, int64_t N, int64_t K,
                            const uint8_t *A, int64_t lda, const int8_t *B, int64_t ldb,
                            float *C, int64_t ldc, float scale, void *stream);
int mipgemm_conv_u8s8f32_dequant(int64_t Nb, int64_t H, int64_t W, int64_t Cin, int64_t Cout,
                                 int R, int S, int stride_h, int stride_w,
                                 int pad_h, int pad_w, int dil_h, int dil_w,
                                 const uint8_t *X, const int8_t *Wt, float *Y,
                                 float scale, void *stream);

/*
 * The fused output transforms with a per-output-channel integer bias: the exact sum of column j (GEMM)
 * or output channel j (convolution) becomes sum + bias[j] in int32 before it is scaled, i.e.
 * C = scale * (A * B + 1 bias^T) and C = sat8(rne(scale * (A * B + 1 bias^T))).  The paper's scheme
 * (Section 7.3) carries a scale only; with the bias of a layer quantised at the scale s_A s_B this is
 * the usual integer form of C^r = s_A s_B C^q + b^r, so the transform is an extension, not the paper's.
 *
 *   bias : device, N (GEMM) or Cout (convolution) int32 values, 4-byte aligned (16-byte aligned
 *          reads fastest); read-only, must stay valid until the call has run on its stream.  NULL = no
 *          bias (then the call is the entry point without the suffix).  sum + bias[j] must fit int32
 *          (it wraps modulo 2^32 otherwise, like an accumulate that overflows).
 * K == 0 gives the transformed bias in every row.  Everything else as for the entry points without
 * the suffix (same rounding rules, operands, limits, errors, stream semantics).
 */
int mipgemm_s8s8f32_dequant_bias(int64_t M, int64_t N, int64_t K,
                                 const int8_t *A, int64_t lda, const int8_t *B, int64_t ldb,
                                 float *C, int64_t ldc, float scale, const int32_t *bias, void *stream);
int mipgemm_u8s8f32_dequant_bias(int64_t M, int64_t N, int64_t K,
                                 const uint8_t *A, int64_t lda, const int8_t *B, int64_t ldb,
                                 float *C, int64_t ldc, float scale, const int32_t *bias, void *stream);
int mipgemm_conv_u8s8f32_dequant_bias(int64_t Nb, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int R, int S,
                                      int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w,
                                      const uint8_t *X, const int8_t *Wt, float *Y, float scale,
                                      const int32_t *bias, void *stream);
int mipgemm_s8s8s8_requant_bias(int64_t M, int64_t N, int64_t K,
                                const int8_t *A, int64_t lda, const int8_t *B, int64_t ldb,
                                int8_t *C, int64_t ldc, float scale, int relu, const int32_t *bias, void *stream);
int mipgemm_u8s8u8_requant_bias(int64_t M, int64_t N, int64_t K,
                                const uint8_t *A, int64_t lda, const int8_t *B, int64_t ldb,
                                uint8_t *C, int64_t ldc, float scale, const int32_t *bias, void *stream);
int mipgemm_conv_u8s8u8_requant_bias(int64_t Nb, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int R, int S,
                                     int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w,
                                     const uint8_t *X, const int8_t *Wt, uint8_t *Y, float scale,
                                     const int32_t *bias, void *stream);

/*
 * Host-buffer variants (the end-to-end path): A, B and C are HOST pointers (pinned or
 * pageable) with the same layouts as above.  The call stages the operands into a device
 * staging buffer, runs the device entry point, copies the M x N result back into C (padding
 * columns of the host C are left untouched; with accumulate != 0 the host C is uploaded
 * first) and SYNCHRONISES the stream before returning.  Large problems (>= 32 MB) are cut into
 * up to 4 x 4 blocks of C that three streams pipeline -- operand blocks in, compute on
 * `stream`, finished blocks out -- so both directions of the host link are busy at once; pinned
 * host memory is what makes those copies asynchronous.  The staging buffer (one per device, as
 * large as the largest call so far) stays allocated between calls; mipgemm_release_staging()
 * frees it.  Calls on one device run one at a time.  Same return codes as the device variants.
 */
int mipgemm_host_s8s8s32(int64_t M, int64_t N, int64_t K,
                         const int8_t *A, int64_t lda, const int8_t *B, int64_t ldb,
                         int32_t *C, int64_t ldc, int accumulate, void *stream);
int mipgemm_host_u8s8s32(int64_t M, int64_t N, int64_t K,
                         const uint8_t *A, int64_t lda, const int8_t *B, int64_t ldb,
                         int32_t *C, int64_t ldc, int accumulate, void *stream);

/*
 * Allocation-free variant of mipgemm_s8s8s32 (the paper has no counterpart: this is an
 * integration aid, not part of the method).
 *
 * Who needs it: callers that are not allowed to reach the CUDA allocator -- code embedded
 * in a memory-planned inference runtime that owns the whole device, real-time loops that
 * must never block in cudaMalloc/cudaFree, plug-ins running under another framework's
 * memory pool.  The other entry points take scratch memory with cudaMallocAsync whenever
 * an operand has to be re-pitched for the tensor-memory-accelerator (base or pitch not a
 * multiple of 16 bytes) and allocate one status word per device on first use; this one
 * calls no allocating routine at all.  Its re-pitching scratch is a fixed array of
 * MIPGEMM_STATIC_SCRATCH_BYTES that lives in the library image: every GPU that loads
 * libmipgemm holds that much memory until the process exits, used or not.
 *
 * Same arguments, layouts, exactness contract and return codes as mipgemm_s8s8s32 (all
 * pointers are device pointers; C is read only when accumulate != 0), with these
 * differences:
 *  - It always runs the dense tensor-core kernel (no skinny-M shortcut).
 *  - If the operands that need re-pitching take more than MIPGEMM_STATIC_SCRATCH_BYTES
 *    (A needs M*roundup(K,16) bytes when A or lda is not 16-byte aligned, B needs
 *    N*roundup(K,16) likewise, each rounded up to 256) the call returns
 *    MIPGEMM_ERR_STATIC_SCRATCH_LIMIT and enqueues nothing.
 *  - The first call on each device performs a one-time set-up (it looks up the device
 *    address of the array and sets kernel attributes).  Make that first call outside any
 *    stream capture.
 *  - All calls on a device share the one array.  It keeps whatever the previous call left
 *    in it; that is harmless because each call overwrites every byte it later reads, so
 *    nothing has to be cleared between calls.  But two calls whose kernels can overlap on
 *    the GPU (different streams, or several host threads) race on the array and corrupt
 *    each other's operands: order such calls on one stream or serialise them yourself.
 *  - A bounded device-side wait that expires in this path sets a status word that is a
 *    static symbol of the library as well.  mipgemm_static_scratch_status() reads and clears
 *    it without allocating anything; mipgemm_device_status() reports it too, but that call
 *    belongs to the regular entry points and allocates their status word on first use.
 *  - mipgemm_last_path() reports the kernel family as for the regular entry point.
 */
#define MIPGEMM_STATIC_SCRATCH_BYTES (8u << 20)
int mipgemm_s8s8s32_static_scratch(int64_t M, int64_t N, int64_t K,
                                   const int8_t *A, int64_t lda,
                                   const int8_t *B, int64_t ldb,
                                   int32_t *C, int64_t ldc,
                                   int accumulate, void *stream);

/* Companion of the entry point above, equally allocation-free (the paper has no counterpart):
 * synchronises `stream`, then returns MIPGEMM_OK, or MIPGEMM_ERR_TIMEOUT if a kernel launched by
 * mipgemm_s8s8s32_static_scratch on the current device gave up a bounded wait since the last query
 * (C is then incomplete; the flag is cleared), or MIPGEMM_ERR_CUDA. */
int mipgemm_static_scratch_status(void *stream);

/* Frees the current device's staging buffer of the host-buffer variants (it is allocated again by
 * the next such call). */
int mipgemm_release_staging(void);

/* ---- support calls (no counterpart in the paper) ---- */

/* Number of kernels this library has enqueued since it was loaded (all threads, all devices). */
uint64_t mipgemm_launch_count(void);

/* The library remembers the plan (tile shape, split, pipeline depth) and the encoded TMA tensor maps of
 * recent dense GEMM / TMA-convolution calls and the weight map of skinny calls, keyed on every argument
 * that determines them (shapes, pointers, pitches, output transform, device, tuning overrides): a
 * repeated call skips planning and encoding.  1024 direct-mapped entries, thread-safe; the environment
 * variable MIPGEMM_PLAN_CACHE=0 switches it off.  Returns 1 if the cache is on, 0 if off, and the
 * number of calls served from / entered into it since the library was loaded. */
int mipgemm_plan_cache_stats(uint64_t *hits, uint64_t *misses);

/* Synchronises `stream` and returns MIPGEMM_OK, MIPGEMM_ERR_TIMEOUT if any kernel
 * since the last call gave up a bounded wait (the flag is then cleared), or
 * MIPGEMM_ERR_CUDA if the synchronisation itself failed. */
int mipgemm_device_status(void *stream);

/* Lend (dev_ptr != NULL, 256-byte aligned) or withdraw (dev_ptr == NULL) a scratch
 * buffer for the current device. */
int mipgemm_set_workspace(void *dev_ptr, size_t bytes);

/* Scratch bytes the corresponding call would need (0 = none). `a_unsigned` selects
 * the u8 variant.  Pointers matter only through their alignment. */
size_t mipgemm_workspace_query_gemm(int64_t M, int64_t N, int64_t K,
                                    const void *A, int64_t lda,
                                    const void *B, int64_t ldb,
                                    const void *C, int64_t ldc, int accumulate);
size_t mipgemm_workspace_query_conv(int64_t Nb, int64_t H, int64_t W, int64_t Cin, int64_t Cout,
                                    int R, int S, int stride_h, int stride_w,
                                    int pad_h, int pad_w, int dil_h, int dil_w);

/* Path taken by this thread's most recent call: a mipgemm_path_t value or-ed with flags. */
int mipgemm_last_path(void);

/* cudaError_t of the most recent failing CUDA call of this thread (0 = none). */
int mipgemm_last_cuda_error(void);

const char *mipgemm_status_string(int status);

/* major*10000 + minor*100 + patch */
int mipgemm_version(void);

/*
 * Tensor-pipe peak probe (the analogue of the paper's Table 1 instruction-rate
 * micro-benchmarks): every SM issues `iters` groups of tcgen05.mma.kind::i8
 * (M=128, N=256, K=32 per instruction, 4 per group) on operands resident in
 * shared memory, nothing is loaded from or stored to global memory except one
 * word per CTA.  On return *ops_per_launch = 2*128*256*128*iters*CTAs.  The
 * caller times the launch.  `sink` : device, >= 4*grid bytes.
 */
int mipgemm_probe_i8_peak(int iters, int *grid_out, double *ops_per_launch,
                          int32_t *sink, void *stream);

/*
 * A promise about the weights of the skinny-M (GEMV-like, paper Section 7.2 batch-1) calls, process
 * wide, off by default: with on != 0 the caller guarantees that the B operand of every later call with
 * M <= 16 is not written by any work still pending on the call's stream when it is enqueued (the
 * usual case: B holds inference weights).  The streaming kernel then starts fetching B while the
 * previous kernel on the stream is still draining (programmatic dependent launch); A is read and C is
 * written only after that kernel has completed, as always.  Results do not change; breaking the
 * promise reads stale weights.  Returns MIPGEMM_OK.
 */
int mipgemm_set_weights_constant(int on);

/*
 * The same promise for individual buffers (the form an inference runtime uses: register each weight
 * tensor once after loading it).  A later call with M <= 16 whose B operand lies entirely inside a
 * registered range [base, base + bytes) is treated as under the promise above, whatever the
 * process-wide switch says; calls on other buffers are not affected.  Unregister a range (by its
 * base) before the buffer is freed or rewritten.  Ranges must not overlap.  Thread-safe.
 * Returns MIPGEMM_OK, or MIPGEMM_ERR_INVALID_ARG (NULL / empty range; unknown base).
 */
int mipgemm_register_constant_weights(const void *base, size_t bytes);
int mipgemm_unregister_constant_weights(const void *base);

/* Overrides for experiments: tile width (0 = heuristic; a multiple of 32 up to 256), pipeline
 * depth (0 = heuristic), split-K factor (0 = heuristic, 1 = off), force path. */
int mipgemm_set_tuning(int block_n, int stages, int split_k, int force_path);

/*
 * Test hook for the unwinding path (no counterpart in the paper).  Every device-side wait of the
 * kernels is bounded (4 s by default); when one runs out, all roles of the CTA leave their loops,
 * wait -- again bounded -- for copies and MMAs still in flight, release tensor memory and return, and
 * mipgemm_device_status() reports MIPGEMM_ERR_TIMEOUT.  This call makes that happen on purpose, by
 * withholding a signal inside the kernel (never by faulting or trapping):
 *   flags bit 0 : the dense kernel's MMA warp never signals "accumulator ready", so the epilogue warps'
 *                 wait runs out; the skinny ring kernel's first CTA never loads the second 1 KB k-chunk
 *                 of its first unit, so its consumer warps' wait runs out.  C is left incomplete.
 *   wait_budget_ns : limit of every wait in later launches (0 = the default 4 s).
 * Process-wide; returns MIPGEMM_OK or MIPGEMM_ERR_INVALID_ARG (unknown flag bits).
 */
int mipgemm_debug_set(int flags, unsigned long long wait_budget_ns);

#ifdef __cplusplus
}
#endif
#endif /* MIPGEMM_H_ */
