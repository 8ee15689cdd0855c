/*
 * dropit.h - C ABI of the DropIT layer path for NVIDIA B200 (sm_100a).
 *
 * DropIT (arXiv 2202.13808) shrinks the activation a that a fully-connected or
 * convolutional layer caches for its backward pass: the smallest-|a| gamma
 * fraction of the whole tensor is dropped (Sec. 3.3 "Min-K Elements"), the rest
 * is kept as a sparse cache a-hat = {a_Xr, X_r} (Sec. 3.2), and the weight
 * gradient is computed from R(a-hat), the cache with dropped positions read as
 * zero (Sec. 3.2, Eq. 4-6).
 *
 * Conventions for every entry point
 *  - Pointers marked [device] are CUDA device pointers owned by the caller;
 *    pointers marked [host] are ordinary host pointers.  The library allocates,
 *    frees and synchronises nothing: every device call only enqueues work on
 *    `cuda_stream` (a cudaStream_t passed as void*; NULL = the default stream).
 *  - Device buffers must be 16-byte aligned.
 *  - Errors that the host can see (null or misaligned pointers, bad sizes,
 *    gamma outside [0,1] or NaN, unknown enum, workspace too small) are
 *    returned before anything is launched.  A CUDA launch error is returned as
 *    DROPIT_ERR_CUDA.  Device-side waits are bounded; if one runs out the
 *    kernel stores DROPIT_ERR_TIMEOUT into *dev_status (if given), leaves its
 *    outputs undefined and returns normally.  dev_status is never cleared by
 *    the library.
 *  - Workspaces need no initialisation.  The few words in them that synchronise
 *    CTAs (a grid barrier, tile counters) are stamped with a number the host
 *    draws per call and are left stale when the kernel ends, so a call may be
 *    captured into a CUDA graph and replayed on the same workspace.  After a
 *    launch that reported DROPIT_ERR_TIMEOUT those words may be left
 *    mid-count: clear the workspace before replaying a graph on it.
 *  - gamma is the DROPPED fraction.  n is the number of elements of the layer
 *    input (every token / pixel / channel of the mini-batch counts: one global
 *    selection per layer call).  n must be < 2^31.
 *  - Flat index = row-major offset into the contiguous tensor as passed
 *    ([M, Ca] for Linear, NCHW for Conv2d).
 *
 * Cache layout (what dropit_compress writes, what the gradient calls read)
 *  - values : the k retained elements, raw bits untouched (-0, NaN payloads and
 *             denormals survive), in ascending flat index.
 *  - meta   : DROPIT_FMT_BITMASK - ceil(n/32) little-endian uint32 words, bit
 *             (i mod 32) of word (i div 32) set iff element i is retained,
 *             unused high bits of the last word 0;
 *             DROPIT_FMT_INDEX32 - the k retained flat indices as ascending
 *             int32 (the coordinate format of Sec. 4.1 / App. A.7).
 *  - offsets: ceil(n/DROPIT_CHUNK) uint32; offsets[c] = number of retained
 *             elements with flat index < c*DROPIT_CHUNK (a seek table into
 *             values; not in the paper, needed to start reading mid-tensor).
 */
#ifndef DROPIT_H_
#define DROPIT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DROPIT_OK = 0,
    DROPIT_ERR_INVALID_ARG = 1,
    DROPIT_ERR_UNSUPPORTED = 2,
    DROPIT_ERR_WORKSPACE = 3,
    DROPIT_ERR_CUDA = 4,
    DROPIT_ERR_TIMEOUT = 5
} dropit_status;

typedef enum { DROPIT_BF16 = 0, DROPIT_F32 = 1 } dropit_dtype;
typedef enum { DROPIT_FMT_BITMASK = 0, DROPIT_FMT_INDEX32 = 1 } dropit_format;
/* Element-wise producers of a layer input (see dropit_produce): y = x, y = max(x, 0), or y = table[x]. */
typedef enum { DROPIT_ACT_IDENTITY = 0, DROPIT_ACT_RELU = 1, DROPIT_ACT_TABLE = 2 } dropit_activation;
/* Tables that dropit_activation_table can build. */
typedef enum { DROPIT_TABLE_IDENTITY = 0, DROPIT_TABLE_RELU = 1, DROPIT_TABLE_GELU = 2 } dropit_table_kind;

/* Elements covered by one entry of the offsets table. */
#define DROPIT_CHUNK 128

/* Library version (major*10000 + minor*100 + patch). [host] */
int dropit_version(void);

/* Number of kernels this library has launched in this process since it was loaded (a diagnostic
 * for benchmarks; memsets are not counted). [host] */
uint64_t dropit_launch_count(void);

/* Static, human-readable name of a status code. [host] */
const char* dropit_status_string(dropit_status s);

/*
 * Number of retained elements for a tensor of n elements at drop ratio gamma:
 * k = n - ceil(gamma*n - 1e-6), clamped to [0, n], in IEEE double.
 * (Sec. 3.3: the smallest gamma fraction is dropped; Sec. 4.1: a proportion
 * 1-gamma is retained; Table 4: the cache shrinks precisely by gamma.  The
 * paper does not say how to round; this keeps never more than the 1-gamma
 * budget.)  Returns -1 for n < 0 or gamma outside [0,1] / NaN.  [host]
 */
int64_t dropit_keep_count(int64_t n, double gamma);

/*
 * Byte sizes of the cache buffers and of the scratch workspace that
 * dropit_compress needs for (n, gamma, dtype, format).  Any output pointer may
 * be NULL.  Sizes are exact for values/meta/offsets (0 when k = 0 or n = 0);
 * callers allocate at least that much, 16-byte aligned.  [host]
 */
dropit_status dropit_cache_sizes(int64_t n, double gamma, dropit_dtype dtype, dropit_format format,
                                 size_t* values_bytes, size_t* meta_bytes, size_t* offsets_bytes,
                                 size_t* workspace_bytes);

/*
 * D(a) with the min-k strategy (Sec. 3.3, Sec. 4.1): retain the
 * k = dropit_keep_count(n, gamma) elements of x with the largest |x|, where
 * |x| is ordered by the raw bits with the sign bit cleared (-0 = +0 < finite <
 * Inf < NaN patterns) and ties at the threshold go to the LOWER flat index
 * (the paper leaves ties open).  Writes values / meta / offsets as laid out
 * above.
 *   x [device, n elements of dtype, read only]; values, meta, offsets [device,
 *   written]; workspace [device, scratch of >= workspace_bytes from
 *   dropit_cache_sizes, contents destroyed, need not be initialised];
 *   dev_status [device int32, may be NULL].
 * n = 0 is a no-op.  For k = 0 the mask and offsets are zero-filled.
 */
dropit_status dropit_compress(const void* x, int64_t n, double gamma, dropit_dtype dtype, dropit_format format,
                              void* values, void* meta, uint32_t* offsets, void* workspace, size_t workspace_bytes,
                              int32_t* dev_status, void* cuda_stream);

/*
 * D(a) with the RANDOM strategy (Sec. 3.3 "Random Elements": a gamma fraction of
 * the elements is dropped at random within the mini-batch; the baseline of
 * Table 2).  The paper does not say how the random set is drawn; here exactly
 * k = dropit_keep_count(n, gamma) elements are retained, as under min-k, so the
 * cache has the same size: element i draws a 15-bit rank from Philox4x32-10
 * (Salmon et al., SC'11; the 64-bit block index i div 8 fills the first two
 * counter words, the other two are 0, key = seed; the four output words are
 * eight 16-bit halves, low half first, and element i takes half i mod 8
 * without its top bit), and the k highest ranks stay, ties to the lower flat
 * index.  With 15-bit ranks the elements that share the threshold rank (about
 * n / 32768 of them) are the only ones whose fate depends on their position.
 * The retained set depends on (n, gamma, seed) only, never on the data.
 * Same cache layout and arguments as dropit_compress; workspace of at least
 * dropit_compress_random_workspace bytes (it holds the ranks: about 2 bytes per
 * element), contents destroyed, need not be initialised.
 */
dropit_status dropit_compress_random_workspace(int64_t n, double gamma, size_t* workspace_bytes);
dropit_status dropit_compress_random(const void* x, int64_t n, double gamma, uint64_t seed, dropit_dtype dtype,
                                     dropit_format format, void* values, void* meta, uint32_t* offsets,
                                     void* workspace, size_t workspace_bytes, int32_t* dev_status, void* cuda_stream);

/*
 * The producer in front of the path.  Sec. 3.5: the inputs of conv / fc layers are the outputs of
 * activation and normalisation layers, which keep their own caches; the tensor that such a layer
 * writes is the tensor that DropIT compresses next.  dropit_produce is that element-wise layer for
 * bf16 tensors, fused with the first half of the selection: it reads x once, writes y = act(x),
 * and on the way takes the selection statistics of y (the threshold band from a sample, the band
 * histograms and the counts above the band, per warp and per CTA of the selection kernel's work
 * partition) into `prep`.  dropit_compress_prepared then produces exactly the cache that
 * dropit_compress(y, ...) would, with ONE read of y: no sample step, no first pass, no grid barrier.
 *
 *   dropit_activation_table: table[b] (device, 65536 uint16) = bits of f(value of bf16 pattern b),
 *     f evaluated in double and rounded once to bf16 (ties to even).  kinds: identity, ReLU
 *     (max(x, 0); -0 -> +0; NaN patterns pass), GELU (x Phi(x), Phi(x) = erfc(-x / sqrt 2) / 2; NaN
 *     patterns pass; -Inf gives the NaN pattern 0x7FC0).  Any other element-wise function can be
 *     supplied as a table built by the caller.
 *   dropit_produce: x [device, n bf16, read only]; act: DROPIT_ACT_IDENTITY (y may be NULL: statistics
 *     only), DROPIT_ACT_RELU, or DROPIT_ACT_TABLE with `table` [device]; y [device, n bf16, written]
 *     must not be x (every CTA samples x while others already write y); prep [device, >=
 *     dropit_produce_workspace bytes, written, need not be initialised]; gamma: the drop ratio the
 *     statistics are taken for.  No device-side waits.
 *   dropit_compress_prepared: same arguments, outputs and selection rule as dropit_compress with dtype
 *     DROPIT_BF16, plus `prep` as written by dropit_produce for the same tensor, n and gamma.  If the
 *     statistics do not fit this call (other n / gamma / device, a tensor too small to be sampled, a
 *     threshold outside the sampled band) the call silently does the whole selection itself, so the
 *     result never depends on `prep`; `workspace` as for dropit_compress.
 */
dropit_status dropit_activation_table(dropit_table_kind kind, uint16_t* table, void* cuda_stream);
dropit_status dropit_produce_workspace(int64_t n, size_t* prep_bytes);
dropit_status dropit_produce(const void* x, int64_t n, double gamma, dropit_activation act, const uint16_t* table,
                             void* y, void* prep, size_t prep_bytes, void* cuda_stream);
dropit_status dropit_compress_prepared(const void* y, int64_t n, double gamma, dropit_format format, void* values,
                                       void* meta, uint32_t* offsets, const void* prep, size_t prep_bytes,
                                       void* workspace, size_t workspace_bytes, int32_t* dev_status, void* cuda_stream);

/*
 * Retained values in 8 bits.  Sec. 1 and Table 5 of the paper combine DropIT with 8-bit and 4-bit activation
 * quantisers (on the layers DropIT does not cover); this applies the idea to DropIT's own payload.  Min-k
 * retains the largest magnitudes of a tensor, which span few binades, so one exponent shared by the tensor
 * plus a small float per value holds them to 1 part in 32: the bitmask cache then costs 1 byte per retained
 * element instead of 2 (gamma = 0.9: 12.9 % of the dense bf16 tensor instead of 17.8 %).
 *   code = sign | e (3 bits) | m (4 bits);  u = 2^(E_top - 127 - 10), E_top = the largest exponent field among the
 *   finite values (written to *scale);  e = 0: m * u;  e = 1..7: (16 + m) * 2^(e-1) * u.  Round to nearest
 *   code, ties to even; values above the largest code, Inf and NaN saturate to it; with E_top < 11 all codes
 *   are zero.  |decode(code(v)) - v| <= |v| / 32 for 16 u <= |v|.
 *   dropit_quantize_values: values [device, k bf16, e.g. the `values` that dropit_compress wrote] -> codes
 *     [device, k bytes], scale [device, one uint32].
 *   dropit_dequantize_values: codes + scale -> values [device, k bf16], exactly the values that the codes stand
 *     for; mask / indices and seek table are unchanged, so the weight-gradient calls take the result as is.
 */
dropit_status dropit_quantize_values(const void* values, int64_t k, uint8_t* codes, uint32_t* scale, void* cuda_stream);
dropit_status dropit_dequantize_values(const uint8_t* codes, const uint32_t* scale, int64_t k, void* values,
                                       void* cuda_stream);

/* Largest tensor (elements) that dropit_compress_static accepts. */
#define DROPIT_STATIC_MAX_ELEMS (1 << 28)

/*
 * dropit_compress for bf16 tensors WITHOUT a workspace argument (the paper has no
 * counterpart; this exists for callers that must not allocate device memory).
 * Some callers cannot obtain scratch memory at the moment they need to compress:
 * a runtime whose device-memory plan is frozen before execution starts, a
 * plug-in that lives inside a host application and may not touch that
 * application's allocator (or take its lock from a callback), or an embedded
 * host that has no allocator to call at all.  For them the scratch that
 * dropit_compress takes from its `workspace` argument lives in a fixed array
 * inside the library's device image: dropit_compress_static_scratch_bytes()
 * bytes (about 400 KB) that every GPU which loads the library holds until the
 * process exits.
 *  - Same inputs, outputs, selection rule and cache layout as dropit_compress
 *    with dtype = DROPIT_BF16; the caller still provides x, values, meta, offsets.
 *  - n above DROPIT_STATIC_MAX_ELEMS returns DROPIT_ERR_WORKSPACE and launches
 *    nothing.
 *  - The call allocates and frees nothing.  The first call on each device looks
 *    up the array's device address (with that device current); make that first
 *    call outside any stream capture.
 *  - All calls on a device share the one array, and it keeps whatever the last
 *    call left there; each call resets, when its kernel starts, the few words
 *    that must start fresh (its counters and its barrier word).
 *    Two calls that overlap on the GPU (different streams, no ordering between
 *    them) would trample each other's scratch: order them.
 */
size_t dropit_compress_static_scratch_bytes(void);
dropit_status dropit_compress_static(const void* x, int64_t n, double gamma, dropit_format format, void* values,
                                     void* meta, uint32_t* offsets, int32_t* dev_status, void* cuda_stream);

/*
 * R(a-hat) (Sec. 3.2): inflate the cache back to a dense tensor of n elements
 * with every dropped position +0 and every retained value bit-identical.
 *   values, meta, offsets [device, read only] as written by dropit_compress for
 *   the same (n, dtype, format); k = number of retained elements;
 *   x_dense_out [device, n elements of dtype, written].
 */
dropit_status dropit_decompress(const void* values, const void* meta, const uint32_t* offsets, int64_t n, int64_t k,
                                dropit_dtype dtype, dropit_format format, void* x_dense_out, void* cuda_stream);

/* Scratch bytes that dropit_weight_grad needs for these shapes on the current device (the plan
 * depends on its SM count): the dense scratch, 64 bytes of counters per output tile and, when the
 * token axis is split, one fp32 plane of whole tiles per split.  The environment variable
 * DROPIT_WG_PATH ("single": one CTA per tile instead of CTA pairs; "fused": the kernel of
 * dropit_weight_grad_fused), read at every call, picks another kernel for comparisons and changes
 * the figure; query and call under the same setting. [host] */
dropit_status dropit_weight_grad_workspace(int64_t M, int64_t Ca, int64_t Cz, dropit_dtype dtype, dropit_format format,
                                           size_t* workspace_bytes);

/*
 * Fully-connected weight gradient from the sparsified cache (Eq. 6; App. A.3
 * G' = (A o D) x Z):  dw[j, c] = sum over retained (n, c) of dy[n, j] * a[n, c].
 *   dy [device, M x Cz row-major, dtype]; values/meta/offsets [device] = cache
 *   of the layer input a [M x Ca row-major]; k its retained count;
 *   dw [device, Cz x Ca row-major, float]: overwritten, or added to when
 *   accumulate != 0; workspace [device scratch, contents destroyed].
 * bf16 inputs multiply on the tensor cores with fp32 accumulation; fp32 inputs
 * use fp32 FMA.  The summation order is fixed, so results are reproducible
 * run to run.
 */
dropit_status dropit_weight_grad(const void* dy, const void* values, const void* meta, const uint32_t* offsets,
                                 int64_t M, int64_t Ca, int64_t Cz, int64_t k, dropit_dtype dtype,
                                 dropit_format format, float* dw, int accumulate, void* workspace,
                                 size_t workspace_bytes, int32_t* dev_status, void* cuda_stream);

/*
 * Same result as dropit_weight_grad (Eq. 6), computed WITHOUT inflating the cache to a dense
 * scratch tensor: R(a-hat) (Sec. 3.2: recovery is a temporary) is rebuilt, 128 channels x 16 tokens
 * at a time, straight from mask words, seek-table entries and packed values, and stored into
 * tensor memory, where the tensor cores read it as an MMA operand.  One kernel launch, and the
 * workspace is not touched (it may be NULL / 0 bytes).  Needs dtype = DROPIT_BF16,
 * format = DROPIT_FMT_BITMASK, Ca a multiple of 128 and Cz a multiple of 8; anything else
 * returns DROPIT_ERR_UNSUPPORTED.  On B200 it is the slower of the two variants (the expansion,
 * not the tensor cores, sets its pace), so dropit_weight_grad does not take it on its own; it
 * is for callers that cannot spare the n * 2 bytes of scratch.  Same summation-order guarantee.
 */
dropit_status dropit_weight_grad_fused(const void* dy, const void* values, const void* meta, const uint32_t* offsets,
                                       int64_t M, int64_t Ca, int64_t Cz, int64_t k, dropit_dtype dtype,
                                       dropit_format format, float* dw, int accumulate, void* workspace,
                                       size_t workspace_bytes, int32_t* dev_status, void* cuda_stream);

/* Scratch bytes that dropit_conv_weight_grad needs for these shapes. [host] */
dropit_status dropit_conv_weight_grad_workspace(int B, int Ca, int H, int W, int Cz, int R, int S, int stride, int pad,
                                                dropit_dtype dtype, dropit_format format, size_t* workspace_bytes);

/*
 * Conv2d weight gradient from the sparsified cache (Eq. 4-5, retained term,
 * with an element-wise mask over the input a):
 *   dw[j, c, u, v] = sum_{n, y, x} dy[n, j, y, x] * R(a-hat)[n, c, y*stride + u - pad, x*stride + v - pad],
 * input positions outside the image contribute 0.  Cross-correlation, NCHW,
 * groups = 1, dilation must be 1 (anything else: DROPIT_ERR_UNSUPPORTED).
 *   dy [device, B x Cz x Ho x Wo, dtype] with Ho = (H + 2 pad - R)/stride + 1,
 *   Wo likewise; values/meta/offsets [device] = cache of a [B x Ca x H x W];
 *   dw [device, Cz x Ca x R x S, float], overwritten or accumulated into.
 * bf16 with S <= 7 (and Wo <= W when stride is 1) runs on the tensor cores (one implicit GEMM per
 * filter tap over (n, y, x), fp32 accumulation, fixed summation order); other shapes and
 * fp32 inputs use an fp32 FMA kernel.  A bounded device wait that expires is reported
 * through dev_status as DROPIT_ERR_TIMEOUT.
 */
dropit_status dropit_conv_weight_grad(const void* dy, const void* values, const void* meta, const uint32_t* offsets,
                                      int B, int Ca, int H, int W, int Cz, int R, int S, int stride, int pad,
                                      int dilation, int64_t k, dropit_dtype dtype, dropit_format format, float* dw,
                                      int accumulate, void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                      void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* DROPIT_H_ */
