// R(a-hat): inflate the sparse cache to a dense tensor, dropped positions = +0 (Sec. 3.2).
#include <cstring>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace dropit {

std::atomic<unsigned long long> g_launch_count{0};

// A warp inflates 1024 consecutive elements (32 mask words, 8 chunks) per step: lane l owns word l, and the
// lane's first value sits at the chunk's table entry plus the population of the chunk's earlier words.
// The retained values of a step are one contiguous piece of `values` (from the seek-table entry of the
// step's first chunk to that of the next step), which the warp fetches with coalesced 16-byte loads into
// shared memory.  The grid is persistent and software-pipelined: table entries are requested two steps
// ahead, the mask word and (for steps with at most 64 vectors of values, i.e. gamma >= 0.5) the piece of
// values one step ahead, so that a step does not wait for memory.
// Whole bf16 steps: every lane builds its four output vectors in registers, reading the values of its
// eight elements from the piece with predicated 2-byte loads, and stores them (512 bytes per warp
// instruction).  The last, partial step and fp32: each lane drops its values into a zeroed shared-memory
// image of the 1024 elements and the warp streams the image out.
template <typename Tr> struct DecompWarps { static constexpr int value = Tr::kElemBytes == 2 ? 8 : 4; };   // 36 KB of shared memory per CTA either way
constexpr int kDecompCtasPerSm = 6;

template <int BYTES> __device__ __forceinline__ uint32_t lds_elem(uint32_t addr) {
    uint32_t v;
    if constexpr (BYTES == 2) asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    else asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
template <int BYTES> __device__ __forceinline__ void sts_elem(uint32_t addr, uint32_t v) {
    if constexpr (BYTES == 2) asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
    else asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

template <typename Tr>
__global__ void __launch_bounds__(32 * DecompWarps<Tr>::value, kDecompCtasPerSm)
decompress_bitmask_kernel(const typename Tr::elem_t* __restrict__ values, const uint32_t* __restrict__ mask,
                          const uint32_t* __restrict__ offsets, int64_t n, int64_t k,
                          typename Tr::elem_t* __restrict__ out) {
    using elem_t = typename Tr::elem_t;
    constexpr int kDecompWarps = DecompWarps<Tr>::value;
    constexpr int ES = Tr::kElemBytes;
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
    const uint32_t img_row = ptx::smem_u32(img) + (uint32_t)(lane * kPitch * ES);   // the lane's image row
    const uint32_t seg_addr = ptx::smem_u32(seg);
    // n < 2^31: steps, words and chunks are counted in 32 bits
    const uint32_t nwords = (uint32_t)((n + 31) / 32);
    const uint32_t nchunks = (uint32_t)((n + DROPIT_CHUNK - 1) / DROPIT_CHUNK);
    const uint32_t ntiles = (nwords + 31) / 32;
    const uint32_t full_tiles = (uint32_t)(n / 1024);     // steps that lie wholly inside the tensor
    const uint32_t stride = gridDim.x * kDecompWarps;
    const uint32_t k32 = (uint32_t)k;
    // what a step needs before its values: the lane's mask word, and (lanes 0..8) the table entries of the
    // step's eight chunks and of the chunk behind them (k past the end of the table)
    auto fetch_word = [&](uint32_t t) -> uint32_t {
        const uint32_t w = t * 32 + lane;
        return (t < ntiles && w < nwords) ? __ldg(mask + w) : 0u;
    };
    auto fetch_entry = [&](uint32_t t) -> uint32_t {
        const uint32_t c = t * 8 + lane;
        if (t >= ntiles || lane > 8) return 0u;
        return c < nchunks ? __ldg(offsets + c) : k32;
    };
    // where the lane reads the image for the copy-out: vector v = i * 32 + lane of the step, in output order
    uint32_t img_out[kVecPerRow];
#pragma unroll
    for (int i = 0; i < kVecPerRow; ++i) {
        const int v = i * 32 + lane;
        img_out[i] = ptx::smem_u32(img) + (uint32_t)(((v / kVecPerRow) * kPitch + (v % kVecPerRow) * G) * ES);
    }
    // The piece of `values` that a step needs, as far as it fits two 16-byte vectors per lane (any step at
    // gamma >= 0.5): requested one step ahead into registers, from the table entries that were requested two
    // steps ahead.  A denser step fetches its piece when it is processed.
    constexpr uint32_t kAhead = 64;   // vectors
    auto piece_of = [&](uint32_t entry, uint32_t& base, uint32_t& nvec) {
        const uint32_t seg_begin = __shfl_sync(kFullMask, entry, 0), seg_end = __shfl_sync(kFullMask, entry, 8);
        base = seg_begin & ~(uint32_t)(G - 1);      // the 16-byte boundary at or below the first value
        nvec = (seg_end > base) ? (seg_end - base + G - 1) / G : 0u;
        if (nvec > (uint32_t)(kSegElems / G)) nvec = kSegElems / G;   // a table that does not match the mask must not overrun the buffer
    };
    auto load_vec = [&](uint32_t e0) -> uint4 {
        if (e0 + G <= k32) return ld_stream(reinterpret_cast<const uint4*>(values + e0));
        elem_t tmp[G];   // the last vector of `values` may be partial: element by element
        for (int e = 0; e < G; ++e) tmp[e] = (e0 + e < k32) ? values[e0 + e] : (elem_t)0;
        uint4 v;
        memcpy(&v, tmp, 16);
        return v;
    };
    auto fetch_piece = [&](uint32_t entry, uint4 (&pv)[2]) {
        uint32_t base, nvec;
        piece_of(entry, base, nvec);
        pv[0] = pv[1] = make_uint4(0, 0, 0, 0);
        if (nvec <= kAhead) {
            if ((uint32_t)lane < nvec) pv[0] = load_vec(base + lane * G);
            if ((uint32_t)lane + 32 < nvec) pv[1] = load_vec(base + (lane + 32) * G);
        }
    };
    uint32_t t = blockIdx.x * kDecompWarps + warp;
    uint32_t word_next = fetch_word(t), entry_next = fetch_entry(t), entry_next2 = fetch_entry(t + stride);
    uint4 piece_next[2];
    fetch_piece(entry_next, piece_next);
    for (; t < ntiles; t += stride) {
        uint32_t word = word_next;
        const uint32_t entry = entry_next;
        const uint4 piece0 = piece_next[0], piece1 = piece_next[1];
        word_next = fetch_word(t + stride);
        entry_next = entry_next2;
        entry_next2 = fetch_entry(t + 2 * stride);
        fetch_piece(entry_next, piece_next);
        const bool full = t < full_tiles;              // uniform over the warp
        if (!full) {                                    // last step: bits past the end of the tensor do not count
            const int64_t e_word = ((int64_t)t * 32 + lane) * 32;
            if (e_word + 32 > n) word = (e_word < n) ? (word & ((1u << (int)(n - e_word)) - 1u)) : 0u;
        }
        uint32_t base, nvec;
        piece_of(entry, base, nvec);
        if (nvec <= kAhead) {
            if ((uint32_t)lane < nvec) reinterpret_cast<uint4*>(seg)[lane] = piece0;
            if ((uint32_t)lane + 32 < nvec) reinterpret_cast<uint4*>(seg)[lane + 32] = piece1;
        } else {
            for (uint32_t c = lane; c < nvec; c += 32) reinterpret_cast<uint4*>(seg)[c] = load_vec(base + c * G);
        }
        const uint32_t cnt = __popc(word);
        uint32_t incl = cnt;                         // inclusive count over the lanes of this chunk (4 words)
        uint32_t up = __shfl_up_sync(kFullMask, incl, 1);
        if ((lane & 3) >= 1) incl += up;
        up = __shfl_up_sync(kFullMask, incl, 2);
        if ((lane & 3) >= 2) incl += up;
        uint32_t pos_end = __shfl_sync(kFullMask, entry, lane >> 2) + incl - base;   // behind the lane's last value in the piece
        // (a table that does not match the mask must not read outside the buffer)
        if (pos_end > (uint32_t)kSegElems || pos_end < cnt) pos_end = cnt;
        elem_t* out_t = out + (size_t)t * 1024 + lane * G;
        if constexpr (ES == 2) {
            if (full) {
                // Whole bf16 step: every lane builds its four output vectors (vector i * 32 + lane: byte lane % 4 of
                // mask word i * 8 + lane / 4) in registers, reading the values of its eight elements from the
                // fetched piece with predicated 2-byte loads.  No image: a third fewer trips through shared memory.
                __syncwarp();   // the piece is in shared memory
                const uint32_t pos0 = pos_end - cnt;
                const uint32_t sh = (uint32_t)(lane & 3) * 8;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int owner = i * 8 + (lane >> 2);
                    const uint32_t w = __shfl_sync(kFullMask, word, owner);
                    const uint32_t p0 = __shfl_sync(kFullMask, pos0, owner);
                    uint32_t a = seg_addr + 2u * (p0 + __popc(w & ((1u << sh) - 1u)));
                    const uint32_t mb = w >> sh;
                    uint32_t e[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const uint32_t bit = (mb >> j) & 1u;
                        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\tmov.u32 %0, 0;\n\t@p ld.shared.u16 %0, [%1];\n\t}"
                                     : "=r"(e[j]) : "r"(a), "r"(bit) : "memory");
                        a += 2u * bit;
                    }
                    const uint4 o = make_uint4(e[0] | (e[1] << 16), e[2] | (e[3] << 16), e[4] | (e[5] << 16), e[6] | (e[7] << 16));
                    *reinterpret_cast<uint4*>(out_t + i * 32 * G) = o;
                }
                __syncwarp();
                continue;
            }
        }
        const uint4 zero = make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int i = 0; i < kPitch / G; ++i) reinterpret_cast<uint4*>(img)[i * 32 + lane] = zero;
        __syncwarp();
        uint32_t src = seg_addr + pos_end * ES;
        while (word) {   // the lane's values, last one first
            uint32_t b;
            asm("bfind.u32 %0, %1;" : "=r"(b) : "r"(word));
            word ^= 1u << b;
            src -= ES;
            sts_elem<ES>(img_row + b * ES, lds_elem<ES>(src));
        }
        __syncwarp();
        if (full) {
#pragma unroll
            for (int i = 0; i < kVecPerRow; ++i) {
                uint4 o;
                asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(o.x), "=r"(o.y), "=r"(o.z), "=r"(o.w) : "r"(img_out[i]) : "memory");
                *reinterpret_cast<uint4*>(out_t + i * 32 * G) = o;
            }
        } else {
            const int64_t e_tile = (int64_t)t * 1024;
#pragma unroll
            for (int i = 0; i < kVecPerRow; ++i) {
                const int v = i * 32 + lane;             // vector of the tile, in output order
                const int row = v / kVecPerRow, col = v % kVecPerRow;
                const int64_t e0 = e_tile + (int64_t)v * G;
                const elem_t* srcv = img + row * kPitch + col * G;
                if (e0 + G <= n) {
                    *reinterpret_cast<uint4*>(out + e0) = *reinterpret_cast<const uint4*>(srcv);
                } else if (e0 < n) {
                    for (int e = 0; e0 + e < n; ++e) out[e0 + e] = srcv[e];
                }
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

extern "C" uint64_t dropit_launch_count(void) { return g_launch_count.load(std::memory_order_relaxed); }

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
