// D(.) with the random strategy (Sec. 3.3 "Random Elements": a gamma fraction of the elements is dropped
// at random within the mini-batch).  The same number of elements is retained as under min-k, chosen by a
// pseudo-random rank instead of the magnitude:
//   rank kernel    element i draws a 15-bit rank from Philox4x32-10 (Salmon et al., SC'11): block i div 8
//                  is the counter, the seed the key, the four output words give eight 16-bit halves;
//   selection      the k highest ranks stay, ties to the lower flat index - this is the min-k selection
//                  kernel run on the ranks, which also writes the mask / indices and the seek table;
//   gather         the retained elements of x are packed in ascending flat index.
// The result depends on (n, gamma, seed) only, not on the data, so a layer can reproduce its mask.
#include "common.cuh"

namespace dropit {

size_t fused_compress_workspace_bytes(int64_t n);
dropit_status fused_compress_bf16(const void* x, int64_t n, int64_t k, bool index32, void* values, void* meta,
                                  uint32_t* offsets, void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                  cudaStream_t stream);

// Philox4x32-10: ten rounds of
//   (c0, c1, c2, c3) <- (hi(M1*c2) ^ c1 ^ k0, lo(M1*c2), hi(M0*c0) ^ c3 ^ k1, lo(M0*c0)),
// the key raised by the Weyl constants between rounds.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint32_t k0, uint32_t k1) {
    constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(M0, c.x), lo0 = M0 * c.x;
        const uint32_t hi1 = __umulhi(M1, c.z), lo1 = M1 * c.z;
        c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
        k0 += W0;
        k1 += W1;
    }
    return c;
}

// One thread per block of eight elements: eight 15-bit ranks, laid out like eight bf16 magnitudes.
__global__ void __launch_bounds__(256)
random_ranks_kernel(uint4* __restrict__ ranks, int64_t nblocks, uint32_t seed_lo, uint32_t seed_hi) {
    for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b < nblocks; b += (int64_t)gridDim.x * blockDim.x) {
        uint4 o = philox4x32_10(make_uint4((uint32_t)b, (uint32_t)((uint64_t)b >> 32), 0u, 0u), seed_lo, seed_hi);
        o.x &= 0x7FFF7FFFu; o.y &= 0x7FFF7FFFu; o.z &= 0x7FFF7FFFu; o.w &= 0x7FFF7FFFu;
        ranks[b] = o;
    }
}

// Pack the retained elements of x: a warp per 1024 elements, lane l owns mask word l; its first value
// goes to the chunk's table entry plus the population of the chunk's earlier words.
template <typename Tr>
__global__ void __launch_bounds__(256)
gather_bitmask_kernel(const typename Tr::elem_t* __restrict__ x, const uint32_t* __restrict__ mask,
                      const uint32_t* __restrict__ offsets, int64_t n, int64_t k,
                      typename Tr::elem_t* __restrict__ values) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t nwords = (n + 31) / 32;
    const int64_t ntiles = (nwords + 31) / 32;
    for (int64_t t = (int64_t)blockIdx.x * 8 + warp; t < ntiles; t += (int64_t)gridDim.x * 8) {
        const int64_t w = t * 32 + lane;
        uint32_t word = (w < nwords) ? __ldg(mask + w) : 0u;
        const uint32_t cnt = __popc(word);
        uint32_t incl = cnt;
        uint32_t up = __shfl_up_sync(kFullMask, incl, 1);
        if ((lane & 3) >= 1) incl += up;
        up = __shfl_up_sync(kFullMask, incl, 2);
        if ((lane & 3) >= 2) incl += up;
        uint32_t pos = ((w < nwords) ? __ldg(offsets + (w >> 2)) : 0u) + incl - cnt;
        const int64_t e0 = w * 32;
        while (word) {
            const int b = __ffs(word) - 1;
            word &= word - 1;
            if (e0 + b < n && (int64_t)pos < k) values[pos] = x[e0 + b];
            ++pos;
        }
    }
}

template <typename Tr>
__global__ void __launch_bounds__(256)
gather_index32_kernel(const typename Tr::elem_t* __restrict__ x, const int32_t* __restrict__ idx, int64_t k, int64_t n,
                      typename Tr::elem_t* __restrict__ values) {
    for (int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; r < k; r += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = idx[r];
        if (i >= 0 && i < n) values[r] = x[i];
    }
}

struct RandomPlan {
    size_t select_off, select_bytes;   // the selection kernel's own scratch
    size_t ranks_off, ranks_bytes;     // 15-bit ranks, 2 bytes per element, whole blocks of eight
    size_t rvals_off, rvals_bytes;     // the retained ranks (the selection kernel's `values` output; not used further)
    size_t total_bytes;
};

static RandomPlan make_random_plan(int64_t n, int64_t k) {
    RandomPlan p{};
    p.select_off = 0;
    p.select_bytes = align_up(fused_compress_workspace_bytes(n), 256);
    p.ranks_off = p.select_off + p.select_bytes;
    p.ranks_bytes = align_up((size_t)((n + 7) / 8) * 16, 256);
    p.rvals_off = p.ranks_off + p.ranks_bytes;
    p.rvals_bytes = align_up((size_t)k * 2 + 16, 256);
    p.total_bytes = p.rvals_off + p.rvals_bytes;
    return p;
}

}  // namespace dropit

using namespace dropit;

extern "C" dropit_status dropit_compress_random_workspace(int64_t n, double gamma, size_t* workspace_bytes) {
    if (n < 0 || n >= ((int64_t)1 << 31) || !(gamma >= 0.0 && gamma <= 1.0)) return DROPIT_ERR_INVALID_ARG;
    if (workspace_bytes) *workspace_bytes = make_random_plan(n, dropit_keep_count(n, gamma)).total_bytes;
    return DROPIT_OK;
}

extern "C" dropit_status dropit_compress_random(const void* x, int64_t n, double gamma, uint64_t seed, dropit_dtype dtype,
                                                dropit_format format, void* values, void* meta, uint32_t* offsets,
                                                void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                                void* cuda_stream) {
    if (n < 0 || n >= ((int64_t)1 << 31) || !(gamma >= 0.0 && gamma <= 1.0)) return DROPIT_ERR_INVALID_ARG;
    if ((dtype != DROPIT_BF16 && dtype != DROPIT_F32) || (format != DROPIT_FMT_BITMASK && format != DROPIT_FMT_INDEX32))
        return DROPIT_ERR_INVALID_ARG;
    if (n == 0) return DROPIT_OK;
    const int64_t k = dropit_keep_count(n, gamma);
    if (!x || !offsets || !is_aligned16(x) || !is_aligned16(offsets)) return DROPIT_ERR_INVALID_ARG;
    if (format == DROPIT_FMT_BITMASK && (!meta || !is_aligned16(meta))) return DROPIT_ERR_INVALID_ARG;
    if (k > 0 && (!values || !is_aligned16(values))) return DROPIT_ERR_INVALID_ARG;
    if (k > 0 && format == DROPIT_FMT_INDEX32 && (!meta || !is_aligned16(meta))) return DROPIT_ERR_INVALID_ARG;
    cudaStream_t stream = as_stream(cuda_stream);
    if (k == 0) {   // gamma = 1: nothing retained
        if (format == DROPIT_FMT_BITMASK &&
            cudaMemsetAsync(meta, 0, (size_t)((n + 31) / 32) * 4, stream) != cudaSuccess)
            return DROPIT_ERR_CUDA;
        if (cudaMemsetAsync(offsets, 0, (size_t)((n + DROPIT_CHUNK - 1) / DROPIT_CHUNK) * 4, stream) != cudaSuccess)
            return DROPIT_ERR_CUDA;
        return DROPIT_OK;
    }
    if (!workspace || !is_aligned16(workspace)) return DROPIT_ERR_INVALID_ARG;
    const RandomPlan plan = make_random_plan(n, k);
    if (workspace_bytes < plan.total_bytes) return DROPIT_ERR_WORKSPACE;
    unsigned char* ws = reinterpret_cast<unsigned char*>(workspace);
    uint4* ranks = reinterpret_cast<uint4*>(ws + plan.ranks_off);
    void* rvals = ws + plan.rvals_off;

    const int64_t nblocks = (n + 7) / 8;
    const int64_t cap = (int64_t)sm_count() * 8;
    {
        int64_t grid = (nblocks + 255) / 256;
        if (grid > cap) grid = cap;
        random_ranks_kernel<<<(unsigned)grid, 256, 0, stream>>>(ranks, nblocks, (uint32_t)seed, (uint32_t)(seed >> 32));
        const dropit_status s = check_launch();
        if (s != DROPIT_OK) return s;
    }
    // the k highest ranks, ties to the lower flat index: mask / indices and seek table come out of the selection
    const dropit_status s = fused_compress_bf16(ranks, n, k, format == DROPIT_FMT_INDEX32, rvals, meta, offsets,
                                                ws + plan.select_off, plan.select_bytes, dev_status, stream);
    if (s != DROPIT_OK) return s;
    if (format == DROPIT_FMT_BITMASK) {
        const int64_t ntiles = (n + 1023) / 1024;
        int64_t grid = (ntiles + 7) / 8;
        if (grid > cap) grid = cap;
        if (dtype == DROPIT_BF16)
            gather_bitmask_kernel<Bf16Traits><<<(unsigned)grid, 256, 0, stream>>>(
                reinterpret_cast<const uint16_t*>(x), reinterpret_cast<const uint32_t*>(meta), offsets, n, k,
                reinterpret_cast<uint16_t*>(values));
        else
            gather_bitmask_kernel<F32Traits><<<(unsigned)grid, 256, 0, stream>>>(
                reinterpret_cast<const uint32_t*>(x), reinterpret_cast<const uint32_t*>(meta), offsets, n, k,
                reinterpret_cast<uint32_t*>(values));
    } else {
        int64_t grid = (k + 255) / 256;
        if (grid > cap) grid = cap;
        if (dtype == DROPIT_BF16)
            gather_index32_kernel<Bf16Traits><<<(unsigned)grid, 256, 0, stream>>>(
                reinterpret_cast<const uint16_t*>(x), reinterpret_cast<const int32_t*>(meta), k, n,
                reinterpret_cast<uint16_t*>(values));
        else
            gather_index32_kernel<F32Traits><<<(unsigned)grid, 256, 0, stream>>>(
                reinterpret_cast<const uint32_t*>(x), reinterpret_cast<const int32_t*>(meta), k, n,
                reinterpret_cast<uint32_t*>(values));
    }
    return check_launch();
}
