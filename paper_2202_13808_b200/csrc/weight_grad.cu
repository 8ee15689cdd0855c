// Fully-connected weight gradient from the sparsified cache (Eq. 6; App. A.3  G' = (A o D) x Z):
//   dW[j, c] = sum_n dY[n, j] * R(a-hat)[n, c]        dY [M, Cz], a [M, Ca], dW [Cz, Ca]
//
// The reduction runs over the token axis n, which is the strided axis of both row-major
// operands, so for the tensor cores both operands are "MN-major": A = dY^T tile (128 output rows j per CTA),
// B = R(a-hat) tile (256 output columns c), K = a block of tokens per pipeline stage.
//
// bf16: tcgen05.mma (kind::f16, fp32 accumulators in TMEM).  Three kernels:
//  * wg_pair_kernel (this file; what dropit_weight_grad takes when Cz > 128): the cache is first inflated to a
//    dense scratch matrix by the decompression kernel (it mostly stays in L2); CTA pairs (cta_group::2) compute
//    256 x 256 tiles, each CTA loading its 128 rows of dY and half of the 256 columns of the scratch by TMA in
//    the 128-byte-swizzled canonical layout.  The kernel is bound by shared-memory bandwidth (every operand byte
//    is written once by TMA and read once by the MMAs; the pair saves a third of the B traffic of one CTA alone).
//    It is launched programmatically behind the decompression and sets itself up while that one drains.
//  * wg_tc_kernel (this file; Cz <= 128, or DROPIT_WG_PATH=single): the same with one CTA per 128 x 256 tile.
//  * weight_grad_tmem.cu (dropit_weight_grad_fused): no scratch; the cache is expanded into tensor memory in
//    front of the MMAs.  One launch, no workspace, slower.
// Small output matrices are split along n ("split-K").  The splits of a tile add up through global memory:
// the tile is cut into as many parts as there are splits, every CTA stores the parts it does not finish into its
// plane of the workspace and finishes the others, tickets deciding who finishes what (wg_tc_kernel with 2 or 4
// splits: the splits form a thread-block cluster and exchange through distributed shared memory instead).
// Either way the summation order is fixed.
// fp32 (and channel counts that are not a multiple of 8): an FFMA kernel with 64x64 tiles on the dense scratch.
#include <cstdlib>
#include <cstring>

#include "weight_grad_common.cuh"

namespace dropit {

dropit_status decompress_dispatch(const void* values, const void* meta, const uint32_t* offsets, int64_t n, int64_t k,
                                  dropit_dtype dtype, dropit_format format, void* out, cudaStream_t stream);

// ---------------------------------------------------------------------------------------------
// Plan
// ---------------------------------------------------------------------------------------------
constexpr int kStages = 4;
constexpr int kPairBK = 144;                            // wg_pair_kernel: tokens per pipeline stage (three stages fill the shared memory)
constexpr int kPairStages = 3;
constexpr int kEpiSubs = 2;                            // epilogue warps per TMEM lane quarter
constexpr int kEpiWarps = 4 * kEpiSubs;
constexpr int kTcThreads = 64 + 32 * kEpiWarps;        // TMA warp, MMA warp, epilogue warps (idle until the accumulator is final)

struct WgPlan {
    bool tensor_core;
    bool fused;               // weight_grad_tmem.cu: the cache is expanded into tensor memory inside the GEMM (no dense scratch)
    bool cluster;             // the splits of a tile form a thread-block cluster and add up through shared memory
    bool pair;                // CTA pairs compute 256 x 256 tiles (wg_pair_kernel); the splits add up through global memory
    int tiles_m, tiles_n, splits, kb_total, kb_per_split;
    size_t counters_off, counters_bytes;
    size_t dense_off, dense_bytes;
    size_t partial_off, partial_bytes;
    size_t total_bytes;
};

// The kernel without a scratch: bitmask caches whose rows are whole 128-element chunks.
static bool fused_supported(int64_t Ca, int64_t Cz, dropit_dtype dtype, dropit_format format) {
    return dtype == DROPIT_BF16 && format == DROPIT_FMT_BITMASK && (Ca % DROPIT_CHUNK == 0) && (Cz % 8 == 0);
}

// DROPIT_WG_PATH picks a kernel where several apply (for comparisons): "fused" = no scratch, cache expanded into
// tensor memory; "single" = dense scratch, one CTA per tile.  Default: dense scratch, CTA pairs.
static bool wg_path_is(const char* name) {
    const char* e = std::getenv("DROPIT_WG_PATH");
    return e && std::strcmp(e, name) == 0;
}

static WgPlan make_wg_plan(int64_t M, int64_t Ca, int64_t Cz, dropit_dtype dtype, dropit_format format, bool fused) {
    WgPlan p{};
    p.tensor_core = (dtype == DROPIT_BF16) && (Ca % 8 == 0) && (Cz % 8 == 0);
    p.fused = fused && fused_supported(Ca, Cz, dtype, format);
    const size_t es = (dtype == DROPIT_BF16) ? 2 : 4;
    if (p.fused) {
        // tiles of 128 channels x 256 outputs; the splits of the token axis are the CTAs of a cluster (1, 2 or 4)
        p.tiles_m = (int)(Ca / kBM);
        p.tiles_n = (int)((Cz + kBN - 1) / kBN);
        p.kb_total = (int)((M + kBK - 1) / kBK);
        int want = sm_count() / (p.tiles_m * p.tiles_n);
        want = want >= 4 ? 4 : (want >= 2 ? 2 : 1);
        while (want > 1 && (p.kb_total + want - 1) / want * (want - 1) >= p.kb_total) want /= 2;   // every split owns >= 1 block
        p.splits = want;
        p.kb_per_split = (p.kb_total + want - 1) / want;
        p.cluster = want > 1;
        p.total_bytes = 256;
        return p;
    }
    if (p.tensor_core) {
        p.pair = Cz > kBM && !wg_path_is("single");
        p.tiles_m = p.pair ? 2 * (int)((Cz + 2 * kBM - 1) / (2 * kBM)) : (int)((Cz + kBM - 1) / kBM);
        p.tiles_n = (int)((Ca + kBN - 1) / kBN);
        const int bk = p.pair ? kPairBK : kBK;
        p.kb_total = (int)((M + bk - 1) / bk);
        const int tiles = p.tiles_m * p.tiles_n;
        int splits = sm_count() / tiles;
        if (splits < 1) splits = 1;
        if (splits > 255) splits = 255;                                  // the tile counters hold eight bits
        if (splits > p.kb_total) splits = p.kb_total;
        p.kb_per_split = (p.kb_total + splits - 1) / splits;
        p.splits = (p.kb_total + p.kb_per_split - 1) / p.kb_per_split;   // every split owns >= 1 block
        p.cluster = !p.pair && (p.splits == 2 || p.splits == 4);
    } else {
        p.tiles_m = (int)((Cz + 63) / 64);
        p.tiles_n = (int)((Ca + 63) / 64);
        p.splits = 1;
    }
    p.counters_off = 0;
    p.counters_bytes = align_up((size_t)p.tiles_m * p.tiles_n * 64, 256);   // per tile and part: tickets drawn, shares published
    p.dense_off = p.counters_off + p.counters_bytes;
    p.dense_bytes = align_up((size_t)M * Ca * es, 256);
    p.partial_off = p.dense_off + p.dense_bytes;
    p.partial_bytes = (p.splits > 1 && !p.cluster) ? (size_t)p.splits * p.tiles_m * p.tiles_n * kBM * kBN * 4 : 0;   // whole tiles
    p.total_bytes = p.partial_off + p.partial_bytes;
    if (p.total_bytes == 0) p.total_bytes = 256;
    return p;
}

// ---------------------------------------------------------------------------------------------
// TMA descriptors (driver entry point fetched at run time; no link-time dependency on libcuda)
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

bool make_map_2d_bf16(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same matrix seen as [cols / 64][rows][64]: one box {64, box_rows, groups} brings `groups` adjacent 64-column
// groups of box_rows rows with a single copy, laid out group after group as the MN-major operand wants them.
// Needs cols % 64 == 0 (a partial last group would read past the end of a row).
bool make_map_grouped_bf16(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int groups, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {64, (cuuint64_t)rows, (cuuint64_t)(cols / 64)};
    cuuint64_t strides[2] = {(cuuint64_t)cols * 2, 128};
    cuuint32_t box[3] = {64, (cuuint32_t)box_rows, (cuuint32_t)groups};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// ---------------------------------------------------------------------------------------------
// tcgen05 kernel
// ---------------------------------------------------------------------------------------------
struct TcSmem {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t accum;
    uint32_t tmem_base;
    int abort_flag;
    int finisher;     // this CTA drew the last ticket of its tile: it adds the partial tiles and writes dW
};
constexpr int kEpiRowFloats = 36;                          // staging row pitch: 32 columns + 4 (bank spread, 16-byte rows)
constexpr int kEpiWarpFloats = 32 * kEpiRowFloats;         // one warp's 32 x 32 chunk
constexpr int kEpiSpinLimit = 1 << 20;
constexpr size_t kTcSmemBytes = 1024 + (size_t)kStages * (kAStageBytes + kBStageBytes) + sizeof(TcSmem);

// Counters in a workspace that nobody initialises: a word holds (call number << 8) | count.  Every CTA that
// will use a word first makes sure, early in the kernel, that it carries this call's number (a word that does
// not is stale and is replaced by a zero count; if the replacement fails, another CTA of the tile has done it,
// or has even counted already, which it only does on a fresh word).  After that the word is counted up with
// plain atomic additions, one trip to L2 each.
__device__ __forceinline__ void epoch_counter_freshen(uint32_t* word, uint32_t epoch) {
    const uint32_t old = *reinterpret_cast<volatile uint32_t*>(word);
    if ((old >> 8) != epoch) atomicCAS(word, old, epoch << 8);
}
__device__ __forceinline__ void freshen_tile_counters(uint32_t* tile_counters, uint32_t epoch, int t) {
    if (t >= 0 && t < 2 * (kBN / 32)) epoch_counter_freshen(tile_counters + t, epoch);
}

// The split reduction through global memory, as the four epilogue warps of a CTA run it once their accumulator
// is final (threads 64 .. 64 + 32 * kEpiWarps - 1; named barrier 1).  The tile's eight 32-column chunks form
// 1, 2, 4 or 8 parts (as many as there are splits, rounded down to a power of two), each with its own ticket
// counter, and the CTA of split s starts at part s % parts.  The last CTA to draw a part's ticket is that part's
// finisher: it waits until the others have published their share of the part, adds the planes in split order
// and writes dW; the others store their share into their plane and go on to the next part.  So every CTA of a
// tile stores some parts and finishes others, and a CTA only ever waits for CTAs that are already running.
constexpr int kMaxParts = kBN / 32;
__device__ __forceinline__ int ticket_parts(int splits) { return splits >= 8 ? 8 : (splits >= 4 ? 4 : (splits >= 2 ? 2 : 1)); }
// Thread 64 draws the ticket of the part its CTA starts with as soon as the tile's counters are fresh, long before
// the accumulator is final, so that the trip to L2 is not part of the epilogue.  (A ticket says "this split is
// running", which is as true during the main loop as after it; the waits on the other side are bounded.)
__device__ __forceinline__ uint32_t draw_first_ticket(uint32_t* tile_counters, int split, int splits) {
    __syncwarp();   // threads 64..79 of this warp have just freshened the counters
    if (threadIdx.x != 64 || splits <= 1) return 0u;
    return atomicAdd(tile_counters + split % ticket_parts(splits), 1u) & 0xFFu;
}
__device__ __forceinline__ void ticket_epilogue(uint32_t tmem_base, float* stage_base, int warp, int lane, int j0, int c0,
                                                int Ca, int Cz, int split, int splits, float* __restrict__ dw,
                                                int accumulate, float* __restrict__ partial, uint32_t* tickets,
                                                uint32_t* done, uint32_t epoch, uint32_t first_ticket, int* finisher_flag,
                                                volatile int* abort_flag);

// Chunks [ch_begin, ch_end) of one 128 x 256 accumulator tile, as the warp that owns TMEM lane quarter g runs
// them.  A CTA that is not the part's finisher stores its chunks into its split's plane just as they come out
// of tensor memory: planes are laid out [tile][chunk][lane quarter][4-column group (8)][lane (32)] float4, so a
// store instruction of the warp is 512 contiguous bytes and the finisher's lane reads back exactly the columns
// of its own row.  The finisher adds the planes in split order, taking its own term from tensor memory (the sum
// does not depend on which split finishes), turns the chunk through shared memory (row pitch 36 floats) and
// writes full 128-byte row segments of dW.
constexpr int kPlaneTileFloats = kBM * kBN;
__device__ __forceinline__ size_t plane_offset(int ch, int g, int e4, int lane) {
    return (size_t)(((ch * 4 + g) * 8 + e4) * 32 + lane) * 4;
}
__device__ __forceinline__ void epilogue_chunks(uint32_t tmem_base, float* stage, int g, int sub, int lane, int j0, int c0,
                                                int ch_begin, int ch_end, int Ca, int Cz, int split, int splits,
                                                bool finisher, float* __restrict__ dw, int accumulate,
                                                float* __restrict__ planes, size_t plane_stride) {
    const int rr0 = lane >> 3, q = lane & 7;
    float4 ahead[8];
#pragma unroll 1
    for (int ch = ch_begin + sub; ch < ch_end; ch += kEpiSubs) {    // the warps of a lane quarter take every kEpiSubs-th chunk
        uint32_t r[32];
        if (!finisher) {
            ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(32 * g) << 16) + ch * 32, r);
            ptx::tmem_ld_wait();
            float* dst = planes + (size_t)split * plane_stride + plane_offset(ch, g, 0, lane);
#pragma unroll
            for (int e4 = 0; e4 < 8; ++e4)
                __stcg(reinterpret_cast<float4*>(dst + e4 * 128),
                       make_float4(__uint_as_float(r[4 * e4]), __uint_as_float(r[4 * e4 + 1]), __uint_as_float(r[4 * e4 + 2]),
                                   __uint_as_float(r[4 * e4 + 3])));
            continue;
        }
        float4 other[8];
        if (splits == 2) {                       // the common case: the other plane's loads are one chunk ahead
            if (ch == ch_begin + sub) {
                const float* src = planes + (size_t)(1 - split) * plane_stride + plane_offset(ch, g, 0, lane);
#pragma unroll
                for (int e4 = 0; e4 < 8; ++e4) other[e4] = __ldcg(reinterpret_cast<const float4*>(src + e4 * 128));
            } else {
#pragma unroll
                for (int e4 = 0; e4 < 8; ++e4) other[e4] = ahead[e4];
            }
            if (ch + kEpiSubs < ch_end) {
                const float* src = planes + (size_t)(1 - split) * plane_stride + plane_offset(ch + kEpiSubs, g, 0, lane);
#pragma unroll
                for (int e4 = 0; e4 < 8; ++e4) ahead[e4] = __ldcg(reinterpret_cast<const float4*>(src + e4 * 128));
            }
        }
        ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(32 * g) << 16) + ch * 32, r);
        ptx::tmem_ld_wait();
        float acc[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) acc[e] = 0.f;
        for (int s = 0; s < splits; ++s) {       // fixed order over the splits
            if (s == split) {
#pragma unroll
                for (int e = 0; e < 32; ++e) acc[e] += __uint_as_float(r[e]);
            } else {
                if (splits != 2) {
                    const float* src = planes + (size_t)s * plane_stride + plane_offset(ch, g, 0, lane);
#pragma unroll
                    for (int e4 = 0; e4 < 8; ++e4) other[e4] = __ldcg(reinterpret_cast<const float4*>(src + e4 * 128));
                }
#pragma unroll
                for (int e4 = 0; e4 < 8; ++e4) {
                    acc[4 * e4] += other[e4].x; acc[4 * e4 + 1] += other[e4].y;
                    acc[4 * e4 + 2] += other[e4].z; acc[4 * e4 + 3] += other[e4].w;
                }
            }
        }
#pragma unroll
        for (int e = 0; e < 32; e += 4)
            *reinterpret_cast<float4*>(stage + lane * kEpiRowFloats + e) = make_float4(acc[e], acc[e + 1], acc[e + 2], acc[e + 3]);
        __syncwarp();
        const int col = c0 + ch * 32 + 4 * q;
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int row = j0 + 32 * g + it * 4 + rr0;
            if (col < Ca && row < Cz) {          // Ca is a multiple of 8
                float4 v = *reinterpret_cast<const float4*>(stage + (it * 4 + rr0) * kEpiRowFloats + 4 * q);
                float* dst = dw + (size_t)row * Ca + col;
                if (accumulate) {
                    const float4 o = *reinterpret_cast<const float4*>(dst);
                    v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
                }
                *reinterpret_cast<float4*>(dst) = v;
            }
        }
        __syncwarp();
    }
}

__device__ __forceinline__ void ticket_epilogue(uint32_t tmem_base, float* stage_base, int warp, int lane, int j0, int c0,
                                                int Ca, int Cz, int split, int splits, float* __restrict__ dw,
                                                int accumulate, float* __restrict__ partial, uint32_t* tickets,
                                                uint32_t* done, uint32_t epoch, uint32_t first_ticket, int* finisher_flag,
                                                volatile int* abort_flag) {
    const int parts = ticket_parts(splits);
    const int cpp = kMaxParts / parts;           // chunks per part
    float* stage = stage_base + (warp - 2) * kEpiWarpFloats;
    for (int pi = 0; pi < parts; ++pi) {
        const int part = (split + pi) % parts;
        if (splits > 1) {
            if (threadIdx.x == 64) {
                // the ticket of the first part was drawn when the kernel started (draw_first_ticket)
                const uint32_t t = pi == 0 ? first_ticket : (atomicAdd(tickets + part, 1u) & 0xFFu);
                *finisher_flag = (t == (uint32_t)splits - 1) ? 1 : 0;
            }
            asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpiWarps) : "memory");
        }
        const bool finisher = *finisher_flag != 0;
        if (finisher && splits > 1) {
            // the other splits of this tile have drawn this part's ticket, so they are running their epilogues
            if (threadIdx.x == 64) {
                const uint32_t want = (epoch << 8) | ((uint32_t)splits - 1);
                int spins = 0;
                while (*reinterpret_cast<volatile uint32_t*>(done + part) != want && !*abort_flag) {
                    if (++spins > kEpiSpinLimit) { *abort_flag = 1; break; }
                    __nanosleep(32);
                }
                __threadfence();
            }
            asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpiWarps) : "memory");
        }
        if (!*abort_flag) {
            ptx::tc_fence_after();
            epilogue_chunks(tmem_base, stage, warp & 3, (warp - 2) >> 2, lane, j0, c0, part * cpp, (part + 1) * cpp, Ca, Cz, split,
                            splits, finisher, dw, accumulate, partial + (size_t)blockIdx.x * kPlaneTileFloats,
                            (size_t)gridDim.x * kPlaneTileFloats);
        }
        if (splits > 1) {
            // publish this CTA's share of the part (also after an abort, so that the finisher's wait ends); the
            // barrier also keeps thread 64 from redrawing finisher_flag while others still read it
            if (!finisher) __threadfence();
            asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpiWarps) : "memory");
            if (threadIdx.x == 64) {
                if (!finisher) {
                    atomicAdd(done + part, 1u);
                } else if (!*abort_flag) {
                    // every other split has drawn its ticket and published: nobody touches the part's two words
                    // again in this launch.  Zero is stale for every call number (numbers are never zero), so the
                    // same launch replayed from a captured graph starts from a clean count as well.
                    tickets[part] = 0u;
                    done[part] = 0u;
                }
            }
        }
    }
}

__device__ __forceinline__ void cluster_finish_chunks(uint32_t tmem_base, const uint8_t* xchg, float* stage, int g,
                                                      int sub, int lane, int rank, int splits, int j0, int c0, int Ca,
                                                      int Cz, float* __restrict__ dw, int accumulate) {
    const int cpo = (kBN / 32) / splits;
    const int rr0 = lane >> 3, q = lane & 7;
#pragma unroll 1
    for (int cl = sub; cl < cpo; cl += kEpiSubs) {
        const int ch = rank * cpo + cl;
        uint32_t r[32];
        ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(32 * g) << 16) + ch * 32, r);
        ptx::tmem_ld_wait();
        float acc[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) acc[e] = 0.f;
        for (int s = 0; s < splits; ++s) {                            // fixed order over the splits
            if (s == rank) {
#pragma unroll
                for (int e = 0; e < 32; ++e) acc[e] += __uint_as_float(r[e]);
            } else {
                const int slot = s < rank ? s : s - 1;
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    const float4 v = *reinterpret_cast<const float4*>(xchg + xchg_offset(slot, cpo, cl, g, e / 4, lane));
                    acc[e] += v.x; acc[e + 1] += v.y; acc[e + 2] += v.z; acc[e + 3] += v.w;
                }
            }
        }
#pragma unroll
        for (int e = 0; e < 32; e += 4)
            *reinterpret_cast<float4*>(stage + lane * kEpiRowFloats + e) = make_float4(acc[e], acc[e + 1], acc[e + 2], acc[e + 3]);
        __syncwarp();
        const int col = c0 + ch * 32 + 4 * q;
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int row = j0 + 32 * g + it * 4 + rr0;
            if (col < Ca && row < Cz) {
                float4 v = *reinterpret_cast<const float4*>(stage + (it * 4 + rr0) * kEpiRowFloats + 4 * q);
                float* dst = dw + (size_t)row * Ca + col;
                if (accumulate) {
                    const float4 o = *reinterpret_cast<const float4*>(dst);
                    v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
                }
                *reinterpret_cast<float4*>(dst) = v;
            }
        }
        __syncwarp();
    }
}

__global__ void __launch_bounds__(kTcThreads, 1)
wg_tc_kernel(const __grid_constant__ CUtensorMap map_dy, const __grid_constant__ CUtensorMap map_x, int Ca, int Cz,
             int tiles_n, int splits, int kb_per_split, int kb_total, float* __restrict__ dw, int accumulate,
             float* __restrict__ partial, uint32_t* counters, int32_t* dev_status, int cluster_mode,
             int grouped_maps, uint32_t wait_limit, uint32_t epoch) {
    extern __shared__ uint8_t smem_raw[];
    // The dynamic window starts at the same offset in every CTA of the kernel, so this rounding gives
    // the same offsets in both CTAs of a cluster (the exchange below maps addresses between them).
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;
    uint8_t* sB = smem + kStages * kAStageBytes;
    TcSmem* ctl = reinterpret_cast<TcSmem*>(sB + kStages * kBStageBytes);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int tile = blockIdx.x;
    // cluster mode: the cluster is (1, splits, 1), its CTA rank is the split
    const int split = cluster_mode ? (int)ptx::cluster_ctarank() : (int)blockIdx.y;
    const int j0 = (tile / tiles_n) * kBM;
    const int c0 = (tile % tiles_n) * kBN;
    const int kb_begin = split * kb_per_split;
    const int kb_end = min(kb_total, kb_begin + kb_per_split);
    const int nkb = kb_end - kb_begin;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(&ctl->full[s], 1);
            ptx::mbar_init(&ctl->empty[s], 1);
        }
        ptx::mbar_init(&ctl->accum, 1);
        ctl->abort_flag = 0;
        ctl->finisher = 1;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&map_dy);
        ptx::prefetch_tensormap(&map_x);
    }
    if (warp == 1) {
        ptx::tmem_alloc(&ctl->tmem_base, kBN);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    volatile int* abort_flag = &ctl->abort_flag;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            ptx::grid_dependency_wait();   // the dense scratch is written by the kernel before this one
            int issued = 0;
            for (int i = 0; i < nkb && !*abort_flag; ++i) {
                const int s = i % kStages;
                if (i >= kStages && !ptx::mbar_wait_spin(&ctl->empty[s], ((i / kStages) - 1) & 1, wait_limit)) {
                    *abort_flag = 1;
                    break;
                }
                ptx::mbar_arrive_expect_tx(&ctl->full[s], kAStageBytes + kBStageBytes);
                const int k0 = (kb_begin + i) * kBK;
                uint8_t* a = sA + s * kAStageBytes;
                uint8_t* b = sB + s * kBStageBytes;
                if (grouped_maps) {   // one copy per operand
                    ptx::tma_load_3d(a, &map_dy, 0, k0, j0 / 64, &ctl->full[s]);
                    ptx::tma_load_3d(b, &map_x, 0, k0, c0 / 64, &ctl->full[s]);
                } else {
#pragma unroll
                    for (int g = 0; g < kBM / 64; ++g) ptx::tma_load_2d(a + g * (64 * kBK * 2), &map_dy, j0 + 64 * g, k0, &ctl->full[s]);
#pragma unroll
                    for (int g = 0; g < kBN / 64; ++g) ptx::tma_load_2d(b + g * (64 * kBK * 2), &map_x, c0 + 64 * g, k0, &ctl->full[s]);
                }
                issued = i + 1;
            }
            if (*abort_flag) {   // let the copies already in flight land before the CTA exits
                for (int i = max(0, issued - kStages); i < issued; ++i)
                    ptx::mbar_wait(&ctl->full[i % kStages], (i / kStages) & 1, kWaitLimit);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::make_idesc_bf16(kBM, kBN, true, true);
            constexpr uint32_t kGroupBytes = 64 * kBK * 2;   // one 64-wide M/N group: kBK rows of 128 bytes
            for (int i = 0; i < nkb; ++i) {
                const int s = i % kStages;
                if (*abort_flag || !ptx::mbar_wait_spin(&ctl->full[s], (i / kStages) & 1, wait_limit)) {
                    *abort_flag = 1;
                    break;
                }
                ptx::tc_fence_after();
                const uint32_t a_addr = ptx::smem_u32(sA + s * kAStageBytes);
                const uint32_t b_addr = ptx::smem_u32(sB + s * kBStageBytes);
#pragma unroll
                for (int kk = 0; kk < kBK / 16; ++kk) {
                    const uint64_t ad = ptx::make_smem_desc_sw128(a_addr + kk * 2048, kGroupBytes, 1024);
                    const uint64_t bd = ptx::make_smem_desc_sw128(b_addr + kk * 2048, kGroupBytes, 1024);
                    ptx::umma_bf16(tmem_base, ad, bd, idesc, (i > 0 || kk > 0) ? 1u : 0u);
                }
                ptx::umma_commit(&ctl->empty[s]);
            }
            ptx::umma_commit(&ctl->accum);   // also after an abort: the barrier then tells when the MMAs in flight are done
        }
    } else {
        // ---------------- epilogue: TMEM -> global ----------------
        ptx::launch_dependents();   // a programmatically launched kernel behind this one may be brought up
        uint32_t first_ticket = 0;
        if (!cluster_mode && splits > 1) {
            freshen_tile_counters(counters + (size_t)tile * 2 * kMaxParts, epoch, (int)threadIdx.x - 64);
            if (warp == 2) first_ticket = draw_first_ticket(counters + (size_t)tile * 2 * kMaxParts, split, splits);
        }
        bool ok = ptx::mbar_wait_warp(&ctl->accum, 0, wait_limit);
        ok = __all_sync(kFullMask, ok) && !*abort_flag;
        if (!ok) *abort_flag = 1;
        // The accumulator is final, so every MMA has read its operands and every TMA copy has landed:
        // the pipeline buffers are free and serve as the staging area.
        if (!cluster_mode)
            ticket_epilogue(tmem_base, reinterpret_cast<float*>(smem), warp, lane, j0, c0, Ca, Cz, split, splits, dw,
                            accumulate, partial, counters + (size_t)tile * 2 * kMaxParts, counters + (size_t)tile * 2 * kMaxParts + kMaxParts, epoch,
                            first_ticket, &ctl->finisher, abort_flag);
    }

    if (cluster_mode) {
        // All roles are done here: the accumulator is final and the pipeline buffers of this CTA are free.
        // Every thread of the cluster takes part in the two barriers, whatever happened before.
        uint8_t* xchg = smem;                                              // receive area, <= kXchgMaxBytes
        float* stage = reinterpret_cast<float*>(smem + kXchgMaxBytes) + (warp >= 2 ? (warp - 2) * kEpiWarpFloats : 0);
        __syncwarp();
        ptx::cluster_sync_all();                                           // every CTA's buffers are free
        const int g = warp & 3;
        if (warp >= 2 && !*abort_flag) {
            ptx::tc_fence_after();
            cluster_send_chunks(tmem_base, xchg, g, (warp - 2) >> 2, kEpiSubs, lane, split, splits);
        }
        __syncwarp();
        ptx::cluster_sync_all();                                           // every chunk has been delivered
        if (warp >= 2 && !*abort_flag)
            cluster_finish_chunks(tmem_base, xchg, stage, g, (warp - 2) >> 2, lane, split, splits, j0, c0, Ca, Cz, dw, accumulate);
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        // after an abort nobody has waited for the MMAs that were already issued: tensor memory is not given
        // back while they may still write to it (always the full limit here)
        if (*abort_flag) ptx::mbar_wait_warp(&ctl->accum, 0, kWaitLimit);
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kBN);
    }
    if (*abort_flag && threadIdx.x == 0 && dev_status) atomicExch(dev_status, (int)DROPIT_ERR_TIMEOUT);
}

// ---------------------------------------------------------------------------------------------
// tcgen05 kernel on CTA pairs: the two CTAs of a cluster (2, 1, 1) compute a 256 x 256 tile of dW with one
// MMA stream.  Each CTA loads its own 128 rows of dY and only half of the 256 columns of x, so a token block
// costs a CTA 32 KB of shared-memory traffic from L2 instead of 48 KB; that traffic, not the tensor cores,
// bounds the single-CTA kernel above.  Each CTA ends up with its 128 x 256 accumulator in its own tensor
// memory and runs the ticket epilogue on it (the splits of the token axis are separate clusters).
//
// Pipeline: both CTAs' producers point their copies at the full barrier of the even-ranked CTA (the leader), whose
// producer announces the bytes of both; the leader's MMA thread waits there, issues the MMAs for both CTAs and
// commits onto the empty barrier of both.  (Announcing from the other CTA as well, by an arrival sent through
// the cluster, cost that producer more time per token block than the MMAs of the block take.)
// A copy costs the TMA unit about 0.1 us whatever its size, on top of its bytes; with 64 tokens per stage that
// fixed part alone came to more than the MMAs of a stage take, hence three deep stages of 144 tokens rather
// than six of 64.  The slots are shared out among three producer threads in three warps (slot s belongs to
// producer s % 3); two of them are epilogue warps, which have nothing else to do until the accumulator is final.
// ---------------------------------------------------------------------------------------------
constexpr int kPairProducers = 3;
static_assert(kPairStages % kPairProducers == 0, "every producer owns the same number of slots");
constexpr int kPairAStageBytes = kBM * kPairBK * 2;
constexpr int kPairBStageBytes = (kBN / 2) * kPairBK * 2;
constexpr uint32_t kPairStageTx = kPairAStageBytes + kPairBStageBytes;
struct PairSmem {
    uint64_t full[kPairStages];
    uint64_t empty[kPairStages];
    uint64_t accum;
    uint32_t tmem_base;
    int abort_flag;
    int finisher;
    int consumed;                    // leader: token blocks whose operands the MMA thread has seen arrive
    int issued[kPairStages];         // per slot: rounds this CTA's producers have issued
    int peer_issued[kPairStages];    // leader: the other CTA's `issued`, stored by that CTA when its producers stop
    int peer_abort;                  // leader: the other CTA gave up a wait
};
constexpr size_t kPairSmemBytes = 1024 + (size_t)kPairStages * (kPairAStageBytes + kPairBStageBytes) + sizeof(PairSmem);
static_assert(kPairStages * (kPairAStageBytes + kPairBStageBytes) >= (int)(kEpiWarps * kEpiWarpFloats * sizeof(float)),
              "the epilogue stages its chunks in the pipeline buffers");

// One producer thread: token blocks i = p, p + 3, p + 6, ... of this CTA's range (block i lives in slot i % stages,
// so the thread only ever touches the slots s with s % 3 == p).
__device__ __forceinline__ void pair_producer(PairSmem* ctl, uint8_t* sA, uint8_t* sB, const CUtensorMap* map_dy,
                                              const CUtensorMap* map_x, int p, int member, uint32_t leader_rank, int nkb,
                                              int kb_begin, int j0, int cb, int grouped_maps, uint32_t wait_limit) {
    volatile int* abort_flag = &ctl->abort_flag;
    const uint32_t full0 = ptx::map_shared_to_cta(ptx::smem_u32(&ctl->full[0]), leader_rank);
    int rounds[kPairStages / kPairProducers];
#pragma unroll
    for (int q = 0; q < kPairStages / kPairProducers; ++q) rounds[q] = 0;
    bool go = true;
    for (int base = 0; base < nkb && go; base += kPairStages) {
        const uint32_t round_parity = (uint32_t)(base / kPairStages) & 1u;
#pragma unroll
        for (int q = 0; q < kPairStages / kPairProducers; ++q) {
            const int s = p + q * kPairProducers;
            const int i = base + s;
            if (i >= nkb || !go) continue;
            if (*abort_flag || (base > 0 && !ptx::mbar_wait_poll(&ctl->empty[s], round_parity ^ 1u, wait_limit))) {
                *abort_flag = 1;
                go = false;
                continue;
            }
            const uint32_t bar = full0 + 8u * (uint32_t)s;
            if (!member) ptx::mbar_arrive_expect_tx(&ctl->full[s], 2u * kPairStageTx);
            const int k0 = (kb_begin + i) * kPairBK;
            uint8_t* a = sA + s * kPairAStageBytes;
            uint8_t* b = sB + s * kPairBStageBytes;
            if (grouped_maps) {   // one copy per operand
                ptx::tma_load_3d_pair(a, map_dy, 0, k0, j0 / 64, bar);
                ptx::tma_load_3d_pair(b, map_x, 0, k0, cb / 64, bar);
            } else {
#pragma unroll
                for (int g = 0; g < kBM / 64; ++g) ptx::tma_load_2d_pair(a + g * (64 * kPairBK * 2), map_dy, j0 + 64 * g, k0, bar);
#pragma unroll
                for (int g = 0; g < kBN / 128; ++g) ptx::tma_load_2d_pair(b + g * (64 * kPairBK * 2), map_x, cb + 64 * g, k0, bar);
            }
            rounds[q] += 1;
        }
    }
#pragma unroll
    for (int q = 0; q < kPairStages / kPairProducers; ++q) {
        const int s = p + q * kPairProducers;
        ctl->issued[s] = rounds[q];
        if (member) ptx::st_cluster_u32(ptx::map_shared_to_cta(ptx::smem_u32(&ctl->peer_issued[s]), leader_rank), (uint32_t)rounds[q]);
    }
}

__global__ void __launch_bounds__(kTcThreads, 1)
wg_pair_kernel(const __grid_constant__ CUtensorMap map_dy, const __grid_constant__ CUtensorMap map_x, int Ca, int Cz,
               int tiles_n, int splits, int kb_per_split, int kb_total, float* __restrict__ dw, int accumulate,
               float* __restrict__ partial, uint32_t* counters, int32_t* dev_status, int grouped_maps,
               uint32_t wait_limit, uint32_t epoch) {
    extern __shared__ uint8_t smem_raw[];
    // same offsets in both CTAs: the MMA addresses the operands of both with one descriptor
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;
    uint8_t* sB = smem + kPairStages * kPairAStageBytes;
    PairSmem* ctl = reinterpret_cast<PairSmem*>(sB + kPairStages * kPairBStageBytes);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();
    const int member = (int)(rank & 1u);           // 0: leader
    const uint32_t leader_rank = rank & ~1u;
    const int tile = blockIdx.x;                   // the pair's CTAs are neighbours along x
    const int split = blockIdx.y;
    const int pair = tile >> 1;
    const int j0 = ((pair / tiles_n) * 2 + member) * kBM;
    const int c0 = (pair % tiles_n) * kBN;
    const int cb = c0 + member * (kBN / 2);        // the half of the tile's columns whose x this CTA loads
    const int kb_begin = split * kb_per_split;
    const int kb_end = min(kb_total, kb_begin + kb_per_split);
    const int nkb = kb_end - kb_begin;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairStages; ++s) {
            ptx::mbar_init(&ctl->full[s], 1);
            ptx::mbar_init(&ctl->empty[s], 1);
            ctl->issued[s] = 0;
            ctl->peer_issued[s] = 0;
        }
        ptx::mbar_init(&ctl->accum, 1);
        ctl->abort_flag = 0;
        ctl->finisher = 1;
        ctl->consumed = 0;
        ctl->peer_abort = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&map_dy);
        ptx::prefetch_tensormap(&map_x);
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(&ctl->tmem_base, kBN);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before();
    ptx::cluster_sync_all();     // both CTAs' barriers exist before either CTA signals the other
    ptx::tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    volatile int* abort_flag = &ctl->abort_flag;

    if (warp == 0) {
        // ---------------- TMA producer 0 (both CTAs) ----------------
        if (lane == 0) {
            ptx::grid_dependency_wait();   // the dense scratch is written by the kernel before this one
            pair_producer(ctl, sA, sB, &map_dy, &map_x, 0, member, leader_rank, nkb, kb_begin, j0, cb, grouped_maps, wait_limit);
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader only) ----------------
        if (lane == 0 && member == 0) {
            constexpr uint32_t idesc = ptx::make_idesc_bf16(2 * kBM, kBN, true, true);
            constexpr uint32_t kGroupBytes = 64 * kPairBK * 2;   // one 64-wide M/N group: kPairBK rows of 128 bytes
            const uint16_t both = (uint16_t)(3u << leader_rank);
            int consumed = 0, s = 0;
            uint32_t round_parity = 0;
            for (int i = 0; i < nkb; ++i) {
                if (*abort_flag || !ptx::mbar_wait_poll(&ctl->full[s], round_parity, wait_limit)) {
                    *abort_flag = 1;
                    break;
                }
                consumed = i + 1;
                ptx::tc_fence_after();
                const uint32_t a_addr = ptx::smem_u32(sA + s * kPairAStageBytes);
                const uint32_t b_addr = ptx::smem_u32(sB + s * kPairBStageBytes);
#pragma unroll
                for (int kk = 0; kk < kPairBK / 16; ++kk) {
                    const uint64_t ad = ptx::make_smem_desc_sw128(a_addr + kk * 2048, kGroupBytes, 1024);
                    const uint64_t bd = ptx::make_smem_desc_sw128(b_addr + kk * 2048, kGroupBytes, 1024);
                    ptx::umma_bf16_pair(tmem_base, ad, bd, idesc, (i > 0 || kk > 0) ? 1u : 0u);
                }
                ptx::umma_commit_pair(&ctl->empty[s], both);
                if (++s == kPairStages) { s = 0; round_parity ^= 1u; }
            }
            ctl->consumed = consumed;
            ptx::umma_commit_pair(&ctl->accum, both);   // also after an abort: tells both CTAs when the MMAs in flight are done
        }
    } else {
        // ---------------- epilogue: TMEM -> global (both CTAs, each its own 128 rows) ----------------
        ptx::launch_dependents();
        uint32_t first_ticket = 0;
        if (splits > 1) {
            freshen_tile_counters(counters + (size_t)tile * 2 * kMaxParts, epoch, (int)threadIdx.x - 64);
            if (warp == 2) first_ticket = draw_first_ticket(counters + (size_t)tile * 2 * kMaxParts, split, splits);
        }
        if (warp - 2 >= 1 && warp - 2 < kPairProducers) {   // producers 1 and 2 first
            if (lane == 0) {
                ptx::grid_dependency_wait();
                pair_producer(ctl, sA, sB, &map_dy, &map_x, warp - 2, member, leader_rank, nkb, kb_begin, j0, cb, grouped_maps, wait_limit);
            }
            __syncwarp();
        }
        bool ok = ptx::mbar_wait_warp(&ctl->accum, 0, wait_limit);
        ok = __all_sync(kFullMask, ok) && !*abort_flag;
        if (!ok) *abort_flag = 1;
        // every MMA has read its operands in both CTAs: the pipeline buffers serve as the staging area
        ticket_epilogue(tmem_base, reinterpret_cast<float*>(smem), warp, lane, j0, c0, Ca, Cz, split, splits, dw, accumulate,
                        partial, counters + (size_t)tile * 2 * kMaxParts, counters + (size_t)tile * 2 * kMaxParts + kMaxParts, epoch,
                        first_ticket, &ctl->finisher, abort_flag);
    }

    // Neither CTA leaves while the other may still signal its barriers or read its shared memory.  After a wait
    // was given up, copies may be in flight whose token block the MMA thread never took, and one CTA may have
    // issued a block that the other did not: the leader squares the accounts of those barriers by hand (bytes that
    // were announced but never sent are counted as arrived; bytes that were sent unannounced get their arrival)
    // and waits for the rest, between two cluster barriers that keep the other CTA alive.
    __syncthreads();
    if (member && threadIdx.x == 0 && *abort_flag)
        ptx::st_cluster_u32(ptx::map_shared_to_cta(ptx::smem_u32(&ctl->peer_abort), leader_rank), 1u);
    ptx::cluster_sync_all();
    if (!member && threadIdx.x == 0 && (*abort_flag || *reinterpret_cast<volatile int*>(&ctl->peer_abort))) {
        *abort_flag = 1;
        const int consumed = ctl->consumed;
        for (int s = 0; s < kPairStages; ++s) {
            const int taken = consumed > s ? (consumed - s + kPairStages - 1) / kPairStages : 0;   // rounds of slot s the MMAs took
            const int mine = ctl->issued[s], theirs = *reinterpret_cast<volatile int*>(&ctl->peer_issued[s]);
            if (mine <= taken && theirs <= taken) continue;
            uint64_t* bar = &ctl->full[s];
            if (mine <= taken) ptx::mbar_arrive_expect_tx(bar, kPairStageTx);     // only the other CTA's half is on its way
            else if (theirs <= taken) ptx::mbar_complete_tx(bar, kPairStageTx);   // the other CTA's half never left
            ptx::mbar_wait(bar, (uint32_t)taken & 1u, kWaitLimit);
        }
    }
    ptx::tc_fence_before();
    ptx::cluster_sync_all();
    if (warp == 1) {
        // tensor memory is given back by both CTAs, and only once no MMA can still write to it
        ptx::mbar_wait_warp(&ctl->accum, 0, kWaitLimit);
        ptx::tc_fence_after();
        ptx::tmem_dealloc_pair(tmem_base, kBN);
    }
    if (*abort_flag && threadIdx.x == 0 && dev_status) atomicExch(dev_status, (int)DROPIT_ERR_TIMEOUT);
}

// ---------------------------------------------------------------------------------------------
// FFMA kernel: fp32 inputs, or bf16 shapes that the TMA path cannot take.  64x64 output tile,
// 16 tokens per step, 4x4 outputs per thread.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float to_float(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }
__device__ __forceinline__ float to_float(float f) { return f; }

template <typename T>
__global__ void __launch_bounds__(256)
wg_ffma_kernel(const T* __restrict__ dy, const T* __restrict__ xd, int M, int Ca, int Cz, float* __restrict__ dw,
               int accumulate) {
    __shared__ float sA[16][64 + 4];
    __shared__ float sB[16][64 + 4];
    const int j0 = blockIdx.y * 64, c0 = blockIdx.x * 64;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int lr = threadIdx.x >> 4, lc = (threadIdx.x & 15) * 4;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < M; k0 += 16) {
        const int n = k0 + lr;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int j = j0 + lc + e, c = c0 + lc + e;
            sA[lr][lc + e] = (n < M && j < Cz) ? to_float(dy[(size_t)n * Cz + j]) : 0.f;
            sB[lr][lc + e] = (n < M && c < Ca) ? to_float(xd[(size_t)n * Ca + c]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                a[i] = sA[k][ty * 4 + i];
                b[i] = sB[k][tx * 4 + i];
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int l = 0; l < 4; ++l) acc[i][l] = fmaf(a[i], b[l], acc[i][l]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            const int j = j0 + ty * 4 + i, c = c0 + tx * 4 + l;
            if (j < Cz && c < Ca) {
                float* d = dw + (size_t)j * Ca + c;
                *d = accumulate ? (*d + acc[i][l]) : acc[i][l];
            }
        }
}

__global__ void zero_or_keep_kernel(float* dw, int64_t count, int accumulate) {
    if (accumulate) return;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
        dw[i] = 0.f;
}

}  // namespace dropit

using namespace dropit;

extern "C" dropit_status dropit_weight_grad_workspace(int64_t M, int64_t Ca, int64_t Cz, dropit_dtype dtype,
                                                      dropit_format format, size_t* workspace_bytes) {
    if (M < 0 || Ca <= 0 || Cz <= 0 || M * Ca >= ((int64_t)1 << 31)) return DROPIT_ERR_INVALID_ARG;
    if ((dtype != DROPIT_BF16 && dtype != DROPIT_F32) || (format != DROPIT_FMT_BITMASK && format != DROPIT_FMT_INDEX32))
        return DROPIT_ERR_INVALID_ARG;
    if (workspace_bytes) *workspace_bytes = make_wg_plan(M, Ca, Cz, dtype, format, false).total_bytes;
    return DROPIT_OK;
}

static bool prefer_fused() { return wg_path_is("fused"); }

static dropit_status weight_grad_impl(const void* dy, const void* values, const void* meta,
                                      const uint32_t* offsets, int64_t M, int64_t Ca, int64_t Cz, int64_t k,
                                      dropit_dtype dtype, dropit_format format, float* dw, int accumulate,
                                      void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                      void* cuda_stream, bool force_fused) {
    if (M < 0 || Ca <= 0 || Cz <= 0 || M * Ca >= ((int64_t)1 << 31) || k < 0 || k > M * Ca) return DROPIT_ERR_INVALID_ARG;
    if ((dtype != DROPIT_BF16 && dtype != DROPIT_F32) || (format != DROPIT_FMT_BITMASK && format != DROPIT_FMT_INDEX32))
        return DROPIT_ERR_INVALID_ARG;
    if (!dw || !is_aligned16(dw)) return DROPIT_ERR_INVALID_ARG;
    if (force_fused && !fused_supported(Ca, Cz, dtype, format)) return DROPIT_ERR_UNSUPPORTED;
    cudaStream_t stream = as_stream(cuda_stream);
    if (M == 0 || k == 0) {   // empty batch or gamma = 1: the gradient is zero
        zero_or_keep_kernel<<<sm_count(), 256, 0, stream>>>(dw, Cz * Ca, accumulate);
        return check_launch();
    }
    if (!dy || !values || !meta || !is_aligned16(dy) || !is_aligned16(values) || !is_aligned16(meta))
        return DROPIT_ERR_INVALID_ARG;
    if (format == DROPIT_FMT_BITMASK && (!offsets || !is_aligned16(offsets))) return DROPIT_ERR_INVALID_ARG;
    const WgPlan plan = make_wg_plan(M, Ca, Cz, dtype, format, force_fused || prefer_fused());
    if (plan.fused)   // one launch, no scratch
        return launch_wg_tmem(dy, values, meta, offsets, M, Ca, Cz, k, plan.splits, plan.kb_per_split, plan.kb_total, dw,
                              accumulate, dev_status, stream);
    if (!workspace || !is_aligned16(workspace)) return DROPIT_ERR_INVALID_ARG;
    if (workspace_bytes < plan.total_bytes) return DROPIT_ERR_WORKSPACE;
    unsigned char* ws = reinterpret_cast<unsigned char*>(workspace);
    void* dense = ws + plan.dense_off;
    dropit_status s = decompress_dispatch(values, meta, offsets, M * Ca, k, dtype, format, dense, stream);
    if (s != DROPIT_OK) return s;

    if (!plan.tensor_core) {
        dim3 grid(plan.tiles_n, plan.tiles_m);
        if (dtype == DROPIT_BF16)
            wg_ffma_kernel<uint16_t><<<grid, 256, 0, stream>>>(reinterpret_cast<const uint16_t*>(dy),
                                                             reinterpret_cast<const uint16_t*>(dense), (int)M, (int)Ca,
                                                             (int)Cz, dw, accumulate);
        else
            wg_ffma_kernel<float><<<grid, 256, 0, stream>>>(reinterpret_cast<const float*>(dy),
                                                          reinterpret_cast<const float*>(dense), (int)M, (int)Ca,
                                                          (int)Cz, dw, accumulate);
        return check_launch();
    }

    CUtensorMap map_dy, map_x;
    const bool grouped = (Ca % 64 == 0) && (Cz % 64 == 0);
    const int bk = plan.pair ? kPairBK : kBK;
    if (grouped) {
        if (!make_map_grouped_bf16(&map_dy, dy, M, Cz, kBM / 64, bk) ||
            !make_map_grouped_bf16(&map_x, dense, M, Ca, (plan.pair ? kBN / 2 : kBN) / 64, bk))
            return DROPIT_ERR_CUDA;
    } else if (!make_map_2d_bf16(&map_dy, dy, M, Cz, bk) || !make_map_2d_bf16(&map_x, dense, M, Ca, bk)) {
        return DROPIT_ERR_CUDA;
    }
    uint32_t* counters = reinterpret_cast<uint32_t*>(ws + plan.counters_off);
    float* partial = reinterpret_cast<float*>(ws + plan.partial_off);
    uint32_t epoch = next_epoch() & 0xFFFFFFu;   // stamps the tile counters, which nobody zeroes beforehand
    if (epoch == 0) epoch = 1;                     // zero marks a word that a finished call left behind
    static PerDeviceOnce smem_attr;
    if (smem_attr.needed()) {
        if (cudaFuncSetAttribute(wg_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcSmemBytes) != cudaSuccess ||
            cudaFuncSetAttribute(wg_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairSmemBytes) != cudaSuccess)
            return DROPIT_ERR_CUDA;
        smem_attr.mark();
    }
    dim3 grid(plan.tiles_m * plan.tiles_n, plan.splits);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = plan.pair ? kPairSmemBytes : kTcSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    cfg.attrs = attr;
    if (plan.cluster || plan.pair) {
        attr[cfg.numAttrs].id = cudaLaunchAttributeClusterDimension;
        attr[cfg.numAttrs].val.clusterDim.x = plan.pair ? 2u : 1u;
        attr[cfg.numAttrs].val.clusterDim.y = plan.pair ? 1u : (unsigned)plan.splits;
        attr[cfg.numAttrs].val.clusterDim.z = 1;
        ++cfg.numAttrs;
    }
    // the kernel right before this one in the stream is the decompression: this kernel may be set up while that
    // one drains; it waits before reading the scratch
    attr[cfg.numAttrs].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[cfg.numAttrs].val.programmaticStreamSerializationAllowed = 1;
    ++cfg.numAttrs;
    const cudaError_t err =
        plan.pair ? cudaLaunchKernelEx(&cfg, wg_pair_kernel, map_dy, map_x, (int)Ca, (int)Cz, plan.tiles_n, plan.splits,
                                       plan.kb_per_split, plan.kb_total, dw, accumulate, partial, counters, dev_status,
                                       grouped ? 1 : 0, spin_limit(kWaitLimit), epoch)
                  : cudaLaunchKernelEx(&cfg, wg_tc_kernel, map_dy, map_x, (int)Ca, (int)Cz, plan.tiles_n, plan.splits,
                                       plan.kb_per_split, plan.kb_total, dw, accumulate, partial, counters, dev_status,
                                       plan.cluster ? 1 : 0, grouped ? 1 : 0, spin_limit(kWaitLimit), epoch);
    if (err != cudaSuccess) {
        (void)cudaGetLastError();
        return DROPIT_ERR_CUDA;
    }
    return check_launch();
}

extern "C" dropit_status dropit_weight_grad(const void* dy, const void* values, const void* meta,
                                            const uint32_t* offsets, int64_t M, int64_t Ca, int64_t Cz, int64_t k,
                                            dropit_dtype dtype, dropit_format format, float* dw, int accumulate,
                                            void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                            void* cuda_stream) {
    return weight_grad_impl(dy, values, meta, offsets, M, Ca, Cz, k, dtype, format, dw, accumulate, workspace,
                            workspace_bytes, dev_status, cuda_stream, false);
}

extern "C" dropit_status dropit_weight_grad_fused(const void* dy, const void* values, const void* meta,
                                                  const uint32_t* offsets, int64_t M, int64_t Ca, int64_t Cz,
                                                  int64_t k, dropit_dtype dtype, dropit_format format, float* dw,
                                                  int accumulate, void* workspace, size_t workspace_bytes,
                                                  int32_t* dev_status, void* cuda_stream) {
    return weight_grad_impl(dy, values, meta, offsets, M, Ca, Cz, k, dtype, format, dw, accumulate, workspace,
                            workspace_bytes, dev_status, cuda_stream, true);
}
