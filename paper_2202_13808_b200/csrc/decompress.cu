// R(a-hat): inflate the sparse cache to a dense tensor, dropped positions = +0 (Sec. 3.2).
#include "common.cuh"

namespace dropit {

unsigned long long g_launch_count = 0;

// One thread per 16-byte output vector.  The number of retained elements before the vector is
// the chunk's table entry plus the mask bits of the chunk that precede it.
template <typename Tr>
__global__ void __launch_bounds__(256)
decompress_bitmask_kernel(const typename Tr::elem_t* __restrict__ values, const uint32_t* __restrict__ mask,
                          const uint32_t* __restrict__ offsets, int64_t n, typename Tr::elem_t* __restrict__ out) {
    using elem_t = typename Tr::elem_t;
    constexpr int G = Tr::kVecElems;
    const int64_t nvec = (n + G - 1) / G;
    const int64_t nwords = (n + 31) / 32;
    for (int64_t vi = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; vi < nvec; vi += (int64_t)gridDim.x * blockDim.x) {
        const int64_t e0 = vi * G;
        const int64_t chunk = e0 / DROPIT_CHUNK;
        const int b = (int)(e0 % DROPIT_CHUNK);
        const int64_t w0 = chunk * (DROPIT_CHUNK / 32);
        uint32_t pos = offsets[chunk];
        const int wi = b >> 5;
        for (int w = 0; w < wi; ++w) pos += __popc(mask[w0 + w]);
        const uint32_t word = (w0 + wi < nwords) ? mask[w0 + wi] : 0u;
        const int sh = b & 31;
        pos += __popc(word & ((1u << sh) - 1u));
        const uint32_t bits = (word >> sh) & ((1u << G) - 1u);
        elem_t r[G];
#pragma unroll
        for (int e = 0; e < G; ++e) {
            r[e] = 0;
            if ((bits >> e) & 1u) r[e] = values[pos++];
        }
        if (e0 + G <= n) {
            uint4 o;
            if constexpr (G == 8) {
                o.x = r[0] | ((uint32_t)r[1] << 16);
                o.y = r[2] | ((uint32_t)r[3] << 16);
                o.z = r[4] | ((uint32_t)r[5] << 16);
                o.w = r[6] | ((uint32_t)r[7] << 16);
            } else {
                o = make_uint4(r[0], r[1], r[2], r[3]);
            }
            reinterpret_cast<uint4*>(out)[vi] = o;
        } else {
            for (int e = 0; e0 + e < n; ++e) out[e0 + e] = r[e];
        }
    }
}

template <typename Tr>
__global__ void __launch_bounds__(256)
scatter_index32_kernel(const typename Tr::elem_t* __restrict__ values, const int32_t* __restrict__ idx, int64_t k,
                       int64_t n, typename Tr::elem_t* __restrict__ out) {
    for (int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; r < k; r += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = idx[r];
        if (i >= 0 && i < n) out[i] = values[r];
    }
}

template <typename Tr>
static dropit_status run_decompress(const void* values, const void* meta, const uint32_t* offsets, int64_t n, int64_t k,
                                    dropit_format format, void* out, cudaStream_t stream) {
    using elem_t = typename Tr::elem_t;
    const int64_t cap = (int64_t)sm_count() * 16;
    if (format == DROPIT_FMT_BITMASK) {
        const int64_t nvec = (n + Tr::kVecElems - 1) / Tr::kVecElems;
        int64_t blocks = (nvec + 255) / 256;   // one vector per thread: short threads, many in flight
        if (blocks > 0x7FFFFFFF) blocks = 0x7FFFFFFF;
        decompress_bitmask_kernel<Tr><<<(unsigned)blocks, 256, 0, stream>>>(
            reinterpret_cast<const elem_t*>(values), reinterpret_cast<const uint32_t*>(meta), offsets, n,
            reinterpret_cast<elem_t*>(out));
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
