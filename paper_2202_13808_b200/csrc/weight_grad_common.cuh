// Pieces shared by the two tcgen05 weight-gradient kernels (dense-B by TMA, and fused cache expansion).
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace dropit {

constexpr int kBM = 128;          // output rows (Cz) per accumulator / MMA
constexpr int kFusedAcc = 2;      // fused kernel: accumulators per CTA (tile = 256 rows of Cz), fills TMEM
constexpr int kBN = 256;          // output columns (Ca) per tile
constexpr int kBK = 64;           // tokens per pipeline stage
constexpr int kAStageBytes = kBM * kBK * 2;
constexpr int kBStageBytes = kBN * kBK * 2;
constexpr uint32_t kWaitLimit = 1u << 22;

// Row-major bf16 matrix [rows, cols]; box = 64 columns (128 bytes) x kBK rows, 128-byte swizzle.
bool make_map_2d_bf16(CUtensorMap* map, const void* base, int64_t rows, int64_t cols);

// Drain one 128 x 256 fp32 accumulator tile from TMEM.  Called by the four warps whose (warp & 3)
// covers the four TMEM lane quarters.  With splits > 1 the tile goes to this split's partial plane.
__device__ __forceinline__ void epilogue_store_tile(uint32_t tmem_base, int warp, int lane, int j0, int c0, int Ca,
                                                    int Cz, int split, int splits, float* __restrict__ dw,
                                                    int accumulate, float* __restrict__ partial) {
    const int g = warp & 3;   // TMEM lane quarter this warp may read
    const int row = j0 + 32 * g + lane;
    float* out = (splits > 1) ? (partial + (size_t)split * Cz * Ca) : dw;
    const bool add = (splits == 1) && accumulate;
#pragma unroll 1
    for (int ch = 0; ch < kBN / 32; ++ch) {
        uint32_t r[32];
        ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(32 * g) << 16) + ch * 32, r);
        ptx::tmem_ld_wait();
        if (row < Cz) {
            float* dst = out + (size_t)row * Ca + c0 + ch * 32;
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
                if (c0 + ch * 32 + e + 4 <= Ca) {
                    float4 v = make_float4(__uint_as_float(r[e]), __uint_as_float(r[e + 1]), __uint_as_float(r[e + 2]),
                                           __uint_as_float(r[e + 3]));
                    if (add) {
                        const float4 o = *reinterpret_cast<const float4*>(dst + e);
                        v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
                    }
                    *reinterpret_cast<float4*>(dst + e) = v;
                }
            }
        }
    }
    if (splits > 1) __threadfence();
}

// Split reduction, called by every thread of the CTA after its partial tile (tile_rows x 256) is
// stored: the last split to arrive adds the partial tiles in split order, so the summation order is fixed.
__device__ __forceinline__ void split_reduce_tile(int tile, int j0, int c0, int Ca, int Cz, int splits,
                                                  float* __restrict__ dw, int accumulate,
                                                  const float* __restrict__ partial, uint32_t* counters, int* s_is_last,
                                                  int tile_rows = kBM) {
    if (threadIdx.x == 0) {
        __threadfence();
        *s_is_last = (atomicAdd(&counters[tile], 1u) == (uint32_t)splits - 1) ? 1 : 0;
    }
    __syncthreads();
    if (!*s_is_last) return;
    __threadfence();
    const size_t plane = (size_t)Cz * Ca;
    // several float4 columns per thread and all splits' loads of them in flight together: the last CTA
    // of a tile runs this alone, so its memory latency is on the kernel's critical path
    constexpr int U = 4;
    const int total = tile_rows * (kBN / 4);
    for (int base = threadIdx.x; base < total; base += blockDim.x * U) {
        float4 acc[U];
        size_t o[U];
        bool ok[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int idx = base + u * blockDim.x;
            const int row = j0 + idx / (kBN / 4);
            const int col = c0 + (idx % (kBN / 4)) * 4;
            ok[u] = idx < total && row < Cz && col + 4 <= Ca;
            o[u] = ok[u] ? ((size_t)row * Ca + col) : 0;
            acc[u] = (accumulate && ok[u]) ? *reinterpret_cast<const float4*>(dw + o[u]) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        for (int s = 0; s < splits; ++s) {   // fixed order over the splits
            float4 v[U];
#pragma unroll
            for (int u = 0; u < U; ++u)
                v[u] = ok[u] ? __ldcg(reinterpret_cast<const float4*>(partial + s * plane + o[u])) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                acc[u].x += v[u].x; acc[u].y += v[u].y; acc[u].z += v[u].z; acc[u].w += v[u].w;
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (ok[u]) *reinterpret_cast<float4*>(dw + o[u]) = acc[u];
    }
}

// Fused variant (defined in weight_grad_fused.cu).
dropit_status launch_wg_fused(const void* dy, const void* values, const void* mask, const uint32_t* offsets, int64_t M,
                              int64_t Ca, int64_t Cz, int64_t k, int tiles_m, int tiles_n, int splits, int kb_per_split,
                              int kb_total, float* dw, int accumulate, float* partial, uint32_t* counters,
                              int32_t* dev_status, cudaStream_t stream);

}  // namespace dropit
