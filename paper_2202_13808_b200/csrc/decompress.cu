// R(a-hat): inflate the sparse cache to a dense tensor, dropped positions = +0 (Sec. 3.2).
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace dropit {

unsigned long long g_launch_count = 0;

// A warp inflates 1024 consecutive elements (32 mask words, 8 chunks) per step: lane l owns word l.
// The retained values of a step are one contiguous piece of `values` (from the seek-table entry of the
// step's first chunk to that of the next step), which the warp fetches with coalesced 16-byte loads into
// shared memory.  Each lane then drops its values (they start at the chunk's table entry plus the
// population of the chunk's earlier words) into a zeroed shared-memory image of the 1024 elements -
// work proportional to the number of retained values, not to the dense size - and the warp streams the
// image out as 512-byte store instructions.  The grid is persistent; the mask word and the table
// entries of a warp's next step are requested before the current step is processed, so a step waits
// for one round trip to memory (its values), not three.
template <typename Tr> struct DecompWarps { static constexpr int value = Tr::kElemBytes == 2 ? 8 : 4; };   // 36 KB of shared memory per CTA either way
constexpr int kDecompCtasPerSm = 6;

template <typename Tr>
__global__ void __launch_bounds__(32 * DecompWarps<Tr>::value)
decompress_bitmask_kernel(const typename Tr::elem_t* __restrict__ values, const uint32_t* __restrict__ mask,
                          const uint32_t* __restrict__ offsets, int64_t n, int64_t k,
                          typename Tr::elem_t* __restrict__ out) {
    using elem_t = typename Tr::elem_t;
    constexpr int kDecompWarps = DecompWarps<Tr>::value;
    constexpr int G = Tr::kVecElems;                 // elements per 16-byte vector
    constexpr int kPitch = 32 + G;                   // image row = one mask word; one spare vector spreads the banks
    constexpr int kVecPerRow = 32 / G;
    constexpr int kSegElems = 1024 + G;              // a step's values, fetched from a 16-byte boundary
    __shared__ __align__(16) elem_t image[kDecompWarps][32 * kPitch];
    __shared__ __align__(16) elem_t segment[kDecompWarps][kSegElems];
    ptx::grid_dependency_wait();   // launched programmatically: the cache may come from the kernel before this one
    ptx::launch_dependents();      // a weight-gradient kernel behind this one may set itself up meanwhile
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    elem_t* img = image[warp];
    elem_t* seg = segment[warp];
    const int64_t nwords = (n + 31) / 32;
    const int64_t nchunks = (n + DROPIT_CHUNK - 1) / DROPIT_CHUNK;
    const int64_t ntiles = (nwords + 31) / 32;
    const int64_t stride = (int64_t)gridDim.x * kDecompWarps;
    // what a step needs before its values: the lane's mask word, and (lanes 0..8) the table entries of the
    // step's eight chunks and of the chunk behind them (k past the end of the table)
    auto fetch_word = [&](int64_t t) -> uint32_t {
        const int64_t w = t * 32 + lane;
        return (t < ntiles && w < nwords) ? __ldg(mask + w) : 0u;
    };
    auto fetch_entry = [&](int64_t t) -> uint32_t {
        const int64_t c = t * 8 + lane;
        if (t >= ntiles || lane > 8) return 0u;
        return c < nchunks ? __ldg(offsets + c) : (uint32_t)k;
    };
    int64_t t = (int64_t)blockIdx.x * kDecompWarps + warp;
    uint32_t word_next = fetch_word(t), entry_next = fetch_entry(t);
    for (; t < ntiles; t += stride) {
        uint32_t word = word_next;
        const uint32_t entry = entry_next;
        word_next = fetch_word(t + stride);
        entry_next = fetch_entry(t + stride);
        const int64_t e_word = (t * 32 + lane) * 32;
        if (e_word + 32 > n) word = (e_word < n) ? (word & ((1u << (int)(n - e_word)) - 1u)) : 0u;
        const uint32_t seg_begin = __shfl_sync(kFullMask, entry, 0), seg_end = __shfl_sync(kFullMask, entry, 8);
        // the step's values, from the 16-byte boundary at or below its first one
        const uint32_t base = seg_begin & ~(uint32_t)(G - 1);
        uint32_t nvec = (seg_end > base) ? (seg_end - base + G - 1) / G : 0u;
        if (nvec > (uint32_t)(kSegElems / G)) nvec = kSegElems / G;   // a table that does not match the mask must not overrun the buffer
        for (uint32_t c = lane; c < nvec; c += 32) {
            const uint32_t e0 = base + c * G;
            if ((int64_t)e0 + G <= k) {
                reinterpret_cast<uint4*>(seg)[c] = ld_stream(reinterpret_cast<const uint4*>(values + e0));
            } else {   // the last vector of `values` may be partial: element by element
                for (int e = 0; e < G; ++e) seg[c * G + e] = ((int64_t)e0 + e < k) ? values[e0 + e] : (elem_t)0;
            }
        }
        const uint32_t cnt = __popc(word);
        uint32_t incl = cnt;                         // inclusive count over the lanes of this chunk (4 words)
        uint32_t up = __shfl_up_sync(kFullMask, incl, 1);
        if ((lane & 3) >= 1) incl += up;
        up = __shfl_up_sync(kFullMask, incl, 2);
        if ((lane & 3) >= 2) incl += up;
        uint32_t pos = __shfl_sync(kFullMask, entry, lane >> 2) + incl - cnt - base;   // index into the fetched piece
        const uint4 zero = make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int i = 0; i < kPitch / G; ++i) reinterpret_cast<uint4*>(img)[i * 32 + lane] = zero;
        __syncwarp();
        // (a table that does not match the mask must not read outside the buffer)
        if (pos + cnt > (uint32_t)kSegElems) pos = 0;
        while (word) {
            const int b = __ffs(word) - 1;
            word &= word - 1;
            img[lane * kPitch + b] = seg[pos++];
        }
        __syncwarp();
        const int64_t e_tile = t * 1024;
#pragma unroll
        for (int i = 0; i < kVecPerRow; ++i) {
            const int v = i * 32 + lane;             // vector of the tile, in output order
            const int row = v / kVecPerRow, col = v % kVecPerRow;
            const int64_t e0 = e_tile + (int64_t)v * G;
            const uint4 o = *reinterpret_cast<const uint4*>(img + row * kPitch + col * G);
            if (e0 + G <= n) {
                *reinterpret_cast<uint4*>(out + e0) = o;
            } else if (e0 < n) {
                const elem_t* src = img + row * kPitch + col * G;
                for (int e = 0; e0 + e < n; ++e) out[e0 + e] = src[e];
            }
        }
        __syncwarp();
    }
}

template <typename Tr>
__global__ void __launch_bounds__(256)
scatter_index32_kernel(const typename Tr::elem_t* __restrict__ values, const int32_t* __restrict__ idx, int64_t k,
                       int64_t n, typename Tr::elem_t* __restrict__ out) {
    ptx::grid_dependency_wait();
    ptx::launch_dependents();
    for (int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; r < k; r += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = idx[r];
        if (i >= 0 && i < n) out[i] = values[r];
    }
}

template <typename Tr>
static dropit_status run_decompress(const void* values, const void* meta, const uint32_t* offsets, int64_t n, int64_t k,
                                    dropit_format format, void* out, cudaStream_t stream) {
    using elem_t = typename Tr::elem_t;
    constexpr int kDecompWarps = DecompWarps<Tr>::value;
    const int64_t cap = (int64_t)sm_count() * 16;
    if (format == DROPIT_FMT_BITMASK) {
        const int64_t ntiles = (n + 1023) / 1024;       // one warp step each
        int64_t blocks = (ntiles + kDecompWarps - 1) / kDecompWarps;
        const int64_t resident = (int64_t)sm_count() * kDecompCtasPerSm;   // persistent: every CTA is on an SM at once
        if (blocks > resident) blocks = resident;
        // programmatic launch: the kernel may be brought up while the one before it drains; it waits at its top
        cudaLaunchAttribute pdl[1];
        pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        pdl[0].val.programmaticStreamSerializationAllowed = 1;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)blocks);
        cfg.blockDim = dim3(32 * kDecompWarps);
        cfg.stream = stream;
        cfg.attrs = pdl;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, decompress_bitmask_kernel<Tr>, reinterpret_cast<const elem_t*>(values),
                               reinterpret_cast<const uint32_t*>(meta), offsets, n, k, reinterpret_cast<elem_t*>(out)) !=
            cudaSuccess) {
            (void)cudaGetLastError();
            return DROPIT_ERR_CUDA;
        }
        return check_launch();
    }
    if (cudaMemsetAsync(out, 0, (size_t)n * Tr::kElemBytes, stream) != cudaSuccess) return DROPIT_ERR_CUDA;
    if (k == 0) return DROPIT_OK;
    int64_t blocks = (k + 255) / 256;
    if (blocks > cap) blocks = cap;
    scatter_index32_kernel<Tr><<<(unsigned)blocks, 256, 0, stream>>>(reinterpret_cast<const elem_t*>(values),
                                                                   reinterpret_cast<const int32_t*>(meta), k, n,
                                                                   reinterpret_cast<elem_t*>(out));
    return check_launch();
}

dropit_status decompress_dispatch(const void* values, const void* meta, const uint32_t* offsets, int64_t n, int64_t k,
                                  dropit_dtype dtype, dropit_format format, void* out, cudaStream_t stream) {
    if (dtype == DROPIT_BF16) return run_decompress<Bf16Traits>(values, meta, offsets, n, k, format, out, stream);
    return run_decompress<F32Traits>(values, meta, offsets, n, k, format, out, stream);
}

}  // namespace dropit

using namespace dropit;

extern "C" dropit_status dropit_decompress(const void* values, const void* meta, const uint32_t* offsets, int64_t n,
                                           int64_t k, dropit_dtype dtype, dropit_format format, void* x_dense_out,
                                           void* cuda_stream) {
    if (n < 0 || n >= ((int64_t)1 << 31) || k < 0 || k > n) return DROPIT_ERR_INVALID_ARG;
    if ((dtype != DROPIT_BF16 && dtype != DROPIT_F32) || (format != DROPIT_FMT_BITMASK && format != DROPIT_FMT_INDEX32))
        return DROPIT_ERR_INVALID_ARG;
    if (n == 0) return DROPIT_OK;
    if (!x_dense_out || !is_aligned16(x_dense_out)) return DROPIT_ERR_INVALID_ARG;
    if (format == DROPIT_FMT_BITMASK && (!meta || !offsets || !is_aligned16(meta) || !is_aligned16(offsets)))
        return DROPIT_ERR_INVALID_ARG;
    if (k > 0 && (!values || !is_aligned16(values))) return DROPIT_ERR_INVALID_ARG;
    if (k > 0 && format == DROPIT_FMT_INDEX32 && (!meta || !is_aligned16(meta))) return DROPIT_ERR_INVALID_ARG;
    return decompress_dispatch(values, meta, offsets, n, k, dtype, format, x_dense_out, as_stream(cuda_stream));
}

extern "C" int dropit_version(void) { return 100; }

extern "C" uint64_t dropit_launch_count(void) { return g_launch_count; }

extern "C" const char* dropit_status_string(dropit_status s) {
    switch (s) {
        case DROPIT_OK: return "DROPIT_OK";
        case DROPIT_ERR_INVALID_ARG: return "DROPIT_ERR_INVALID_ARG";
        case DROPIT_ERR_UNSUPPORTED: return "DROPIT_ERR_UNSUPPORTED";
        case DROPIT_ERR_WORKSPACE: return "DROPIT_ERR_WORKSPACE";
        case DROPIT_ERR_CUDA: return "DROPIT_ERR_CUDA";
        case DROPIT_ERR_TIMEOUT: return "DROPIT_ERR_TIMEOUT";
    }
    return "DROPIT_ERR_UNKNOWN";
}
