// Pieces shared by the two tcgen05 weight-gradient kernels (dense scratch by TMA; cache expanded into tensor memory).
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace dropit {

constexpr int kBM = 128;          // rows of an accumulator tile = TMEM lanes (outputs j in weight_grad.cu, channels c in weight_grad_tmem.cu)
constexpr int kBN = 256;          // columns of an accumulator tile
constexpr int kBK = 64;           // tokens per pipeline stage
constexpr int kAStageBytes = kBM * kBK * 2;
constexpr int kBStageBytes = kBN * kBK * 2;
constexpr uint32_t kWaitLimit = 1u << 22;

// Row-major bf16 matrix [rows, cols]; box = 64 columns (128 bytes) x box_rows rows, 128-byte swizzle.
bool make_map_2d_bf16(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int box_rows);
// The same matrix as [cols / 64][rows][64] (cols % 64 == 0): one box brings `groups` adjacent 64-column groups.
bool make_map_grouped_bf16(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int groups, int box_rows);

// cluster exchange, receive area: (splits - 1) slots x (256 / splits) columns x 128 rows of fp32; largest for 4 splits
constexpr int kXchgMaxBytes = 3 * kBM * (kBN / 4) * 4;
// Byte offset of the float4 that holds columns 4 * e4 .. 4 * e4 + 3 of chunk `cl` (of the owner's cpo chunks) for
// row 32 * g + lane, in sender slot `slot`.
__device__ __forceinline__ uint32_t xchg_offset(int slot, int cpo, int cl, int g, int e4, int lane) {
    return (uint32_t)slot * (uint32_t)cpo * 16384u + (uint32_t)(((cl * 4 + g) * 8 + e4) * 512 + lane * 16);
}

// Split reduction inside a thread-block cluster (2 or 4 splits of one tile are the CTAs of one cluster).
// The tile's eight 32-column chunks are shared out among the CTAs (chunk ch belongs to CTA ch / (8 / splits)).
// Every epilogue warp sends the chunks of its 32-row quarter that its CTA does not own from TMEM into the
// owner's shared memory, and after a cluster barrier finishes the chunks its CTA owns: it adds the terms in
// split order (its own from TMEM) and writes dW.  All four warps work in both phases.
// Receive area of a CTA: [sender slot][chunk][lane quarter][4-column group (8)][lane (32)] float4, so that one store
// instruction of a warp is 512 contiguous bytes on its way through the cluster, and one load of the receiver too.
// The `subs` warps of a TMEM lane quarter share out the chunks: warp `sub` takes every subs-th one.
__device__ __forceinline__ void cluster_send_chunks(uint32_t tmem_base, uint8_t* xchg, int g, int sub, int subs, int lane,
                                                    int rank, int splits) {
    const int cpo = (kBN / 32) / splits;                     // chunks per owner
#pragma unroll 1
    for (int ch = sub; ch < kBN / 32; ch += subs) {
        const int owner = ch / cpo;
        if (owner == rank) continue;                         // uniform over the warp
        const int slot = rank < owner ? rank : rank - 1;     // the owner keeps no slot for itself
        const uint32_t local = ptx::smem_u32(xchg) + xchg_offset(slot, cpo, ch - owner * cpo, g, 0, lane);
        const uint32_t remote = ptx::map_shared_to_cta(local, (uint32_t)owner);
        uint32_t r[32];
        ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(32 * g) << 16) + ch * 32, r);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int e4 = 0; e4 < 8; ++e4)
            ptx::st_cluster_v4(remote + (uint32_t)e4 * 512u, __uint_as_float(r[4 * e4]), __uint_as_float(r[4 * e4 + 1]),
                               __uint_as_float(r[4 * e4 + 2]), __uint_as_float(r[4 * e4 + 3]));
    }
}

// Cache expanded into tensor memory (weight_grad_tmem.cu): tiles of 128 channels x 256 outputs.
dropit_status launch_wg_tmem(const void* dy, const void* values, const void* mask, const uint32_t* offsets, int64_t M,
                             int64_t Ca, int64_t Cz, int64_t k, int splits, int kb_per_split, int kb_total, float* dw,
                             int accumulate, int32_t* dev_status, cudaStream_t stream);

}  // namespace dropit
