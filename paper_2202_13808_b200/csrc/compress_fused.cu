// bf16 min-k selection + packing as ONE persistent cooperative kernel (Sec. 3.3 "Min-K Elements",
// Sec. 3.2 a-hat = {a_Xr, X_r}).
//
// Every WARP owns one contiguous run of 1024-element blocks and keeps it for the whole kernel, so
// the ordered compaction needs no block-wide synchronisation and warps drift freely.
//   sample  (separate 1-CTA kernel) a 16 Ki-element jittered sample brackets the threshold key T
//           between two keys [lo, hi] (6-sigma margin on the sample rank); it also clears the selection state.
//   phase 1 one read of the tensor: keys above hi are counted in a register, keys inside the band
//           go to a small per-warp histogram, the rest is ignored (two packed bf16 per 32-bit word
//           are classified with one add each, so the pass is bound by HBM, not by atomics).
//   sync    one grid barrier (bounded wait; the launch is cooperative so all CTAs are resident).
//   phase 2 every CTA sums the per-CTA band histograms: T and the tie quota q follow from the total,
//           the CTA's exclusive prefix from the rows before it, each warp's prefix from the per-warp
//           histograms.  No second counting pass.
//   phase 3 second read (L2 hits for tensors that fit L2): element i is retained iff key_i > T, or
//           key_i == T and fewer than q equal keys precede it; #retained before i =
//           gt_before + min(eq_before, q).  Values are staged per warp and written in 16-byte pieces.
// When the band is wider than the per-warp histogram (small tensors, which are not sampled; key
// distributions that are flat around T; a sample that missed) a general path is taken instead:
// full CTA histogram in shared memory, global histogram by atomics, then one extra counting read.
#include <type_traits>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace dropit {

constexpr int kFusedThreads = 1024;                             // main kernel; 1 CTA per SM
constexpr int kSampleThreads = 1024;
constexpr int kFusedWarps = kFusedThreads / 32;
constexpr int kVpl = 2;                                        // 16-byte vectors per lane per warp block
constexpr int kBlkVecs = 32 * kVpl;                            // vectors per warp block
constexpr int kBlkElems = kBlkVecs * 8;                        // 512 bf16
constexpr int kP1Blocks = 4 / kVpl;                            // blocks loaded per phase-1 iteration (4 loads per lane)
constexpr int kKeySpace = 1 << 15;
constexpr int kWarpBins = 64;                                  // per-warp band histogram
constexpr int kRowWords = kWarpBins + 2;                       // per-CTA row: bins, #key>hi, pad
constexpr int kMaxGrid = 512;
constexpr int kSampleVecs = 2048;                              // 16384 sampled elements
constexpr int64_t kSampleMinElems = 1 << 19;                   // below this the band is the full key range
constexpr int kBarrierSpinLimit = 1 << 22;
constexpr uint32_t kHiBits = 0x80008000u;
constexpr int kRingDepth = 4;                                  // blocks of a warp's run in flight (cp.async ring)
constexpr int kRingSlotBytes = kBlkVecs * 16;                  // one block
constexpr size_t kRingBytes = (size_t)kFusedWarps * kRingDepth * kRingSlotBytes;   // 128 KB
constexpr int kStageVals = kBlkElems + 16;                     // per-warp staging, values
constexpr int kStageIdx = kBlkElems + 8;                       // per-warp staging, indices

struct FusedState {
    uint32_t barrier;            // grid-barrier arrivals
    uint32_t band_lo, band_hi;   // written by the sample kernel
    uint32_t pad0;
    unsigned long long n_hi[2];  // general path: #{key > hi} per attempt
    uint32_t reserved[24];
};
static_assert(sizeof(FusedState) == 128, "FusedState layout");

struct FusedPlan {
    int64_t blocks_total;
    int grid;
    int blocks_per_warp;
    size_t hist_off[2], agg_off, rows_off, total_bytes, zero_bytes;
};

static FusedPlan make_fused_plan(int64_t n) {
    FusedPlan p{};
    p.blocks_total = (n + kBlkElems - 1) / kBlkElems;
    int g = sm_count();
    if (g > kMaxGrid) g = kMaxGrid;
    const int64_t ctas_needed = (p.blocks_total + kFusedWarps - 1) / kFusedWarps;
    if (ctas_needed < g) g = (int)ctas_needed;
    if (g < 1) g = 1;
    p.grid = g;
    p.blocks_per_warp = (int)((p.blocks_total + (int64_t)g * kFusedWarps - 1) / ((int64_t)g * kFusedWarps));
    if (p.blocks_per_warp < 1) p.blocks_per_warp = 1;
    p.hist_off[0] = kStateBytes;
    p.hist_off[1] = p.hist_off[0] + (size_t)kKeySpace * 4;
    p.agg_off = p.hist_off[1] + (size_t)kKeySpace * 4;
    p.zero_bytes = kStateBytes;                                 // the rest is written before it is read
    p.rows_off = p.agg_off + (size_t)kMaxGrid * 8;
    p.total_bytes = p.rows_off + (size_t)kMaxGrid * kRowWords * 4;
    return p;
}

size_t fused_compress_workspace_bytes(int64_t n) { return make_fused_plan(n).total_bytes; }

__device__ __forceinline__ uint32_t ptx_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void keys_of(const uint4& v, uint32_t (&key)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        key[2 * i] = w[i] & 0x7FFFu;
        key[2 * i + 1] = (w[i] >> 16) & 0x7FFFu;
    }
}

// Packed compare constant: adding it to two 15-bit keys held in the halves of a 32-bit word sets
// bit 15 of a half exactly when that key >= bound (no carry crosses the halves).  bound in [0, 32768].
__device__ __forceinline__ uint32_t ge_const(uint32_t bound) { return ((0x8000u - bound) & 0xFFFFu) * 0x00010001u; }

// Four flags held in bit 15 and bit 31 of two words -> 4 bits in element order (x low, x high, y low, y high):
// prmt gathers the two high bytes of each word, a multiply lines the four bit-7s up at bits 21..24.
__device__ __forceinline__ uint32_t flags4(uint32_t x, uint32_t y) {
    const uint32_t t = (__byte_perm(x, y, 0x7531) >> 7) & 0x01010101u;
    return ((t * 0x00204081u) >> 21) & 0xFu;
}

// Exclusive prefix over the block's threads of `v`; also returns the block total.
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* s_warp, uint32_t* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t y = __shfl_up_sync(kFullMask, inc, o);
        if (lane >= o) inc += y;
    }
    __syncthreads();   // protect s_warp from a previous use
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    uint32_t wt = (lane < (int)(blockDim.x >> 5)) ? s_warp[lane] : 0u;
    uint32_t winc = wt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t y = __shfl_up_sync(kFullMask, winc, o);
        if (lane >= o) winc += y;
    }
    const uint32_t wprefix = __shfl_sync(kFullMask, winc - wt, warp);
    *total = __shfl_sync(kFullMask, winc, 31);
    return wprefix + inc - v;
}

// ---------------------------------------------------------------------------------------------
// Sample kernel: zero the scratch, bracket the threshold key.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSampleThreads, 1)
sample_band_kernel(const uint4* __restrict__ x, int64_t n, unsigned long long k, unsigned char* ws, size_t zero_bytes) {
    extern __shared__ uint32_t bins[];
    __shared__ uint32_t s_warp[32];
    __shared__ uint32_t s_band[2];
#ifdef DROPIT_PHASE_TIMING
    unsigned long long t_begin;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_begin));
#endif
    ptx::grid_dependency_wait();   // launched programmatically: x may come from the kernel before this one
    const int64_t nvec = n / 8;
    const bool sampled = n >= kSampleMinElems;
    uint4 sv[kSampleVecs / kSampleThreads];
    if (sampled) {   // issue the sample loads first; they fly while the scratch is zeroed
        const int64_t stride = nvec / kSampleVecs;   // >= 32
#pragma unroll
        for (int r = 0; r < kSampleVecs / kSampleThreads; ++r) {
            const uint32_t s = r * kSampleThreads + threadIdx.x;
            const uint32_t h = (s * 2654435761u) >> 7;   // jitter inside the stride window
            sv[r] = ld_stream(x + (int64_t)s * stride + (int64_t)(h % (uint32_t)stride));
        }
    }
    uint4* z = reinterpret_cast<uint4*>(ws);
    for (size_t i = threadIdx.x; i < zero_bytes / 16; i += blockDim.x) z[i] = make_uint4(0, 0, 0, 0);
    FusedState* st = reinterpret_cast<FusedState*>(ws);
    if (threadIdx.x == 0) {
        s_band[0] = 0;
        s_band[1] = kKeySpace - 1;
    }
    if (sampled) {
        for (int i = threadIdx.x; i < kKeySpace; i += blockDim.x) bins[i] = 0;
        __syncthreads();
#pragma unroll
        for (int r = 0; r < kSampleVecs / kSampleThreads; ++r) {
            uint32_t key[8];
            keys_of(sv[r], key);
#pragma unroll
            for (int e = 0; e < 8; ++e) atomicAdd(&bins[key[e]], 1u);
        }
        __syncthreads();
        // ranks (counted from the largest key) that bracket the threshold with a 6-sigma margin
        const float S = (float)(kSampleVecs * 8);
        const float p = (float)((double)k / (double)n);
        const float ks = p * S;
        const float margin = 6.0f * sqrtf(S * p * (1.0f - p)) + 16.0f;
        const float r_hi = ks - margin, r_lo = ks + margin;
        constexpr int PER = kKeySpace / kSampleThreads;
        const int t = threadIdx.x;
        uint32_t sum = 0;
#pragma unroll
        for (int r = 0; r < PER; ++r) {
            // rotate the start so that the 32 lanes of a warp hit 32 different banks
            const int rr = (r + t) & (PER - 1);
            sum += bins[kKeySpace - 1 - (t * PER + rr)];
        }
        uint32_t total;
        const uint32_t excl = block_exclusive_scan(sum, s_warp, &total);
        // key at descending rank r: cum_before < r <= cum_before + h
        if ((r_hi >= 1.0f && (float)excl < r_hi && r_hi <= (float)(excl + sum)) ||
            (r_lo <= S && (float)excl < r_lo && r_lo <= (float)(excl + sum))) {
            uint32_t cum = excl;
            for (int r = 0; r < PER; ++r) {
                const uint32_t key = kKeySpace - 1 - (t * PER + r);
                const uint32_t hh = bins[key];
                if (hh) {
                    if (r_hi >= 1.0f && (float)cum < r_hi && r_hi <= (float)(cum + hh)) s_band[1] = key;
                    if (r_lo <= S && (float)cum < r_lo && r_lo <= (float)(cum + hh)) s_band[0] = key;
                }
                cum += hh;
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        st->band_lo = s_band[0];
        st->band_hi = s_band[1];
#ifdef DROPIT_PHASE_TIMING
        unsigned long long t;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
        reinterpret_cast<unsigned long long*>(st->reserved)[6] = t;
        reinterpret_cast<unsigned long long*>(st->reserved)[7] = t_begin;
#endif
    }
}

// ---------------------------------------------------------------------------------------------
// Main kernel.
// ---------------------------------------------------------------------------------------------
// Optional phase timestamps of CTA 0 (build with -DDROPIT_PHASE_TIMING): FusedState::reserved holds
// %globaltimer at each stamp.  Off in normal builds.
#ifdef DROPIT_PHASE_TIMING
__device__ __forceinline__ void phase_stamp(FusedState* st, int i) {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
        reinterpret_cast<unsigned long long*>(st->reserved)[i] = t;
    }
}
#else
__device__ __forceinline__ void phase_stamp(FusedState*, int) {}
#endif

struct FusedShared {
    uint32_t warp[32];
    unsigned long long red64[32];
    uint32_t whist[kFusedWarps][kWarpBins];   // per-warp band histograms (fast path)
    uint32_t w_hi[kFusedWarps];               // per-warp #{key > hi}
    uint32_t tot[kRowWords];                  // band histogram over all CTAs (+ #key>hi)
    uint32_t pre[kRowWords];                  // ... over the CTAs before this one
    uint32_t wpre_gt[kFusedWarps], wpre_eq[kFusedWarps];   // exclusive prefix of each warp (absolute)
    uint32_t T, found;
    unsigned long long n_gt, quota;
    int ok;
};

__device__ __forceinline__ bool grid_barrier(uint32_t* counter, uint32_t target, int* s_ok) {
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(counter, 1u);
        int spins = 0;
        bool ok = true;
        while (ld_acquire_u32(counter) < target) {
            if (++spins > kBarrierSpinLimit) { ok = false; break; }
            __nanosleep(32);
        }
        __threadfence();
        *s_ok = ok ? 1 : 0;
    }
    __syncthreads();
    return *s_ok != 0;
}

__device__ __forceinline__ unsigned long long block_sum_u64(unsigned long long v, unsigned long long* s_red) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFullMask, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
    __syncthreads();
    unsigned long long r = ((threadIdx.x & 31) < (blockDim.x >> 5)) ? s_red[threadIdx.x & 31] : 0ull;
    for (int o = 16; o > 0; o >>= 1) r += __shfl_xor_sync(kFullMask, r, o);
    return r;
}

// Load vector vi of the tensor; vectors past the end read as zeros with nvalid = 0, the ragged
// last vector is assembled from scalar loads.
__device__ __forceinline__ uint4 load_vec(const uint4* x, int64_t vi, int64_t nvec_full, int64_t n, int* nvalid) {
    if (vi < nvec_full) {
        *nvalid = 8;
        return ld_stream(x + vi);
    }
    *nvalid = 0;
    uint32_t w[4] = {0, 0, 0, 0};
    if (vi == nvec_full && (n & 7) != 0) {
        const int nv = (int)(n - nvec_full * 8);
        const uint16_t* xe = reinterpret_cast<const uint16_t*>(x) + vi * 8;
        for (int e = 0; e < nv; ++e) w[e >> 1] |= (uint32_t)xe[e] << ((e & 1) * 16);
        *nvalid = nv;
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// Load the 4 vectors of warp block `blk` for this lane (vector j*32 + lane of the block).
__device__ __forceinline__ void load_block(const uint4* x, int64_t blk, int lane, int64_t nvec_full, int64_t n,
                                           uint4 (&v)[kVpl], int (&nvalid)[kVpl]) {
    const int64_t base = blk * kBlkVecs + lane;
    if (base + 32 * (kVpl - 1) < nvec_full) {
#pragma unroll
        for (int j = 0; j < kVpl; ++j) {
            v[j] = ld_stream(x + base + j * 32);
            nvalid[j] = 8;
        }
    } else {
#pragma unroll
        for (int j = 0; j < kVpl; ++j) v[j] = load_vec(x, base + j * 32, nvec_full, n, &nvalid[j]);
    }
}

// The warp's blocks are streamed through a per-warp ring in shared memory fed by cp.async, several
// blocks ahead, so that enough bytes are in flight per SM without holding them in registers.  Each
// lane copies and later reads only its own 16-byte vectors, so a cp.async.wait_group is all the
// synchronisation the ring needs.  `lane_slot` = shared address of the lane's first vector in the slot.
__device__ __forceinline__ void ring_issue(uint32_t lane_slot, const uint4* x, int64_t blk, int lane, int64_t nvec_full,
                                           int64_t n) {
#pragma unroll
    for (int j = 0; j < kVpl; ++j) {
        const int64_t vi = blk * kBlkVecs + j * 32 + lane;
        const uint32_t dst = lane_slot + j * 512;
        if (vi == nvec_full && (n & 7) != 0) {   // ragged last vector of the tensor: assembled by hand
            int nv;
            const uint4 v = load_vec(x, vi, nvec_full, n, &nv);
            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                         : "memory");
        } else {
            const bool in = vi < nvec_full;   // vectors past the end are zero-filled by the copy itself
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(x + (in ? vi : 0)),
                         "r"(in ? 16u : 0u)
                         : "memory");
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}
// The same for a block whose vectors are all whole: `src` = the lane's first vector of the block.
__device__ __forceinline__ void ring_issue_full(uint32_t lane_slot, const uint4* src) {
#pragma unroll
    for (int j = 0; j < kVpl; ++j)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(lane_slot + j * 512), "l"(src + j * 32) : "memory");
    asm volatile("cp.async.commit_group;" ::: "memory");
}
__device__ __forceinline__ void ring_read(uint32_t lane_slot, uint4 (&v)[kVpl]) {
#pragma unroll
    for (int j = 0; j < kVpl; ++j)
        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(v[j].x), "=r"(v[j].y), "=r"(v[j].z), "=r"(v[j].w)
                     : "r"(lane_slot + j * 512)
                     : "memory");
}
// The block issued kRingDepth-1 commits ago has landed.
__device__ __forceinline__ void ring_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(kRingDepth - 1) : "memory"); }
__device__ __forceinline__ int valid_elems(int64_t vi, int64_t nvec_full, int64_t n) {
    return vi < nvec_full ? 8 : (vi == nvec_full ? (int)(n & 7) : 0);
}

// Write the whole 16-byte pieces of a warp's staging buffer and carry the remainder to its front.
// Slot s of the buffer maps to out[base + s] with base a multiple of PIECE elements; the first
// `foreign` slots of the very first piece belong to the previous warp and are never written.
template <typename E, int PIECE>
__device__ __forceinline__ void flush_pieces(E* stage, E* out_base, uint32_t kept, uint32_t& pend, uint32_t& foreign,
                                             int lane) {
    const uint32_t total = pend + kept;
    const uint32_t nfull = total / PIECE;
    uint32_t c0 = 0;
    if (foreign && nfull > 0) {
        if (lane >= (int)foreign && lane < PIECE) out_base[lane] = stage[lane];
        c0 = 1;
        foreign = 0;
    }
    for (uint32_t c = c0 + lane; c < nfull; c += 32)
        reinterpret_cast<uint4*>(out_base)[c] = reinterpret_cast<const uint4*>(stage)[c];
    const uint32_t rem = total - nfull * PIECE;
    E carry = 0;
    if (nfull > 0 && lane < (int)rem) carry = stage[nfull * PIECE + lane];
    __syncwarp();
    if (nfull > 0 && lane < (int)rem) stage[lane] = carry;
    pend = rem;   // == total when nfull == 0
    __syncwarp();
}

template <bool INDEX32>
__global__ void __launch_bounds__(kFusedThreads, 1)
fused_compress_kernel(const uint4* __restrict__ x, int64_t n, unsigned long long k, int blocks_per_warp,
                      unsigned char* ws, size_t hist_off0, size_t hist_off1, size_t agg_off, size_t rows_off,
                      uint16_t* __restrict__ values, uint32_t* __restrict__ mask, int32_t* __restrict__ indices,
                      uint32_t* __restrict__ offsets, int32_t* dev_status) {
    extern __shared__ __align__(16) unsigned char fsm[];
    uint32_t* bins = reinterpret_cast<uint32_t*>(fsm);   // general path, phases 1-2: kKeySpace counters
    // phases 1-2 keep their control block where phase 3 later stages values (phase 3 needs no control block)
    FusedShared& sh = *reinterpret_cast<FusedShared*>(fsm + kRingBytes);
    static_assert(sizeof(FusedShared) <= (size_t)kFusedWarps * kStageVals * 2, "control block must fit the staging area");
    // the input ring shares its memory with the general path's histogram (never live together)
    uint16_t* s_vals_all = reinterpret_cast<uint16_t*>(fsm + kRingBytes);   // phase 3: per-warp staging
    int32_t* s_idx_all = reinterpret_cast<int32_t*>(fsm + kRingBytes + (size_t)kFusedWarps * kStageVals * 2);

    FusedState* st = reinterpret_cast<FusedState*>(ws);
    unsigned long long* agg = reinterpret_cast<unsigned long long*>(ws + agg_off);
    uint32_t* rows = reinterpret_cast<uint32_t*>(ws + rows_off);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ring_lane = ptx_smem(fsm) + (warp * kRingDepth) * kRingSlotBytes + lane * 16;
    const int64_t nvec_full = n / 8;
    const int64_t blocks_total = (n + kBlkElems - 1) / kBlkElems;
    const int64_t blk0 = ((int64_t)blockIdx.x * kFusedWarps + warp) * blocks_per_warp;
    int64_t blk1 = blk0 + blocks_per_warp;
    if (blk1 > blocks_total) blk1 = blocks_total;
    // blocks below this index consist of whole vectors only: they take the paths without bounds arithmetic
    const int64_t blk_full_end = (nvec_full / kBlkVecs < blk1) ? nvec_full / kBlkVecs : blk1;
    auto issue_block = [&](int64_t b, uint32_t dst) {
        if (b < blk_full_end) ring_issue_full(dst, x + b * kBlkVecs + lane);
        else if (b < blk1) ring_issue(dst, x, b, lane, nvec_full, n);
        else asm volatile("cp.async.commit_group;" ::: "memory");
    };
    uint32_t barrier_target = 0;

    uint32_t lo = st->band_lo, hi = st->band_hi;
    uint32_t T = 0, q = 0;
    uint32_t run_gt = 0, run_eq = 0;   // this warp's exclusive prefix (absolute)
    phase_stamp(st, 0);

    for (int attempt = 0; attempt < 2; ++attempt) {
        if (attempt == 1) {
            lo = 0;
            hi = kKeySpace - 1;
        }
        const uint32_t width = hi - lo;
        const bool narrow = width < (uint32_t)kWarpBins;   // uniform over the grid
        uint32_t* ghist = reinterpret_cast<uint32_t*>(ws + (attempt == 0 ? hist_off0 : hist_off1));
        // ---------------- phase 1: band histogram ----------------
        if (narrow) {
            for (int i = threadIdx.x; i < kFusedWarps * kWarpBins; i += blockDim.x) (&sh.whist[0][0])[i] = 0;
        } else {
            for (uint32_t i = threadIdx.x; i <= width; i += blockDim.x) bins[i] = 0;
        }
        __syncthreads();
        uint32_t* hist = narrow ? sh.whist[warp] : bins;
        const uint32_t c_hi = ge_const(hi + 1), c_lo = ge_const(lo);
        uint32_t cnt_hi = 0, cnt_lo = 0;   // keys above the band / keys equal to lo
        auto count_vec = [&](const uint4& v, int nvalid) {
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
            uint32_t a[4], inb[4], any = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t m = w[i] & 0x7FFF7FFFu;
                a[i] = m + c_hi;                       // bit 15 of a half: key > hi
                inb[i] = (m + c_lo) & ~a[i];           // bit 15 of a half: lo <= key <= hi
                any |= inb[i];
            }
            // keys above the band: one popc per pair of words (the flag bytes gathered by prmt)
            cnt_hi += __popc(__byte_perm(a[0], a[1], 0x7531) & 0x80808080u) +
                      __popc(__byte_perm(a[2], a[3], 0x7531) & 0x80808080u);
            if (any & kHiBits) {   // a few percent of the elements: the band histogram
                // one pass per in-band element of the lane's vector (a warp needs about two passes), instead
                // of a divergent test per word and half
                uint32_t pending = (flags4(inb[0], inb[1]) | (flags4(inb[2], inb[3]) << 4)) & ((1u << nvalid) - 1u);
                while (pending) {
                    const uint32_t e = (uint32_t)__ffs(pending) - 1u;
                    pending &= pending - 1u;
                    const uint32_t wlo = (e & 2u) ? w[1] : w[0], whi = (e & 2u) ? w[3] : w[2];
                    const uint32_t ws = (e & 4u) ? whi : wlo;
                    const uint32_t key = ((e & 1u) ? (ws >> 16) : ws) & 0x7FFFu;
                    const uint32_t d = key - lo;
                    if (d == 0) ++cnt_lo; else atomicAdd(&hist[d], 1u);
                }
            }
        };
        if (narrow) {
            // stream the run through the ring, kRingDepth-1 blocks ahead
#pragma unroll
            for (int d = 0; d < kRingDepth - 1; ++d) issue_block(blk0 + d, ring_lane + d * kRingSlotBytes);
            int slot = 0, slot_ahead = kRingDepth - 1;
            for (int64_t blk = blk0; blk < blk1; ++blk) {
                issue_block(blk + kRingDepth - 1, ring_lane + slot_ahead * kRingSlotBytes);
                ring_wait();
                uint4 va[kVpl];
                ring_read(ring_lane + slot * kRingSlotBytes, va);
                if (blk < blk_full_end) {
#pragma unroll
                    for (int j = 0; j < kVpl; ++j) count_vec(va[j], 8);
                } else {
#pragma unroll
                    for (int j = 0; j < kVpl; ++j)
                        count_vec(va[j], valid_elems(blk * kBlkVecs + j * 32 + lane, nvec_full, n));
                }
                slot = (slot + 1 == kRingDepth) ? 0 : slot + 1;
                slot_ahead = (slot_ahead + 1 == kRingDepth) ? 0 : slot_ahead + 1;
            }
            asm volatile("cp.async.wait_all;" ::: "memory");
        } else {
            int64_t blk = blk0;
            for (; blk + kP1Blocks <= blk1; blk += kP1Blocks) {   // 4 loads per lane in flight
                uint4 va[kP1Blocks][kVpl];
                int na[kP1Blocks][kVpl];
#pragma unroll
                for (int u = 0; u < kP1Blocks; ++u) load_block(x, blk + u, lane, nvec_full, n, va[u], na[u]);
#pragma unroll
                for (int u = 0; u < kP1Blocks; ++u)
#pragma unroll
                    for (int j = 0; j < kVpl; ++j) count_vec(va[u][j], na[u][j]);
            }
            for (; blk < blk1; ++blk) {
                uint4 va[kVpl];
                int na[kVpl];
                load_block(x, blk, lane, nvec_full, n, va, na);
#pragma unroll
                for (int j = 0; j < kVpl; ++j) count_vec(va[j], na[j]);
            }
        }
        phase_stamp(st, 1);
        for (int o = 16; o > 0; o >>= 1) {
            cnt_lo += __shfl_xor_sync(kFullMask, cnt_lo, o);
            cnt_hi += __shfl_xor_sync(kFullMask, cnt_hi, o);
        }
        if (lane == 0) {
            if (cnt_lo) atomicAdd(&hist[0], cnt_lo);
            sh.w_hi[warp] = cnt_hi;
        }
        __syncthreads();
        uint32_t cta_hi = 0;
        for (int w = 0; w < kFusedWarps; ++w) cta_hi += sh.w_hi[w];
        if (narrow) {
            // publish this CTA's row: band bins and #key>hi
            if (threadIdx.x < kRowWords) {
                uint32_t v = 0;
                if (threadIdx.x < kWarpBins) {
                    for (int w = 0; w < kFusedWarps; ++w) v += sh.whist[w][threadIdx.x];
                } else if (threadIdx.x == kWarpBins) {
                    v = cta_hi;
                }
                rows[(size_t)blockIdx.x * kRowWords + threadIdx.x] = v;
            }
        } else {
            // the global histogram is scratch that nobody cleared: every CTA clears a slice, and one more
            // grid barrier separates the clearing from the accumulation
            for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i <= width; i += gridDim.x * blockDim.x) ghist[i] = 0;
            barrier_target += gridDim.x;
            if (!grid_barrier(&st->barrier, barrier_target, &sh.ok)) {
                if (threadIdx.x == 0 && dev_status) atomicExch(dev_status, (int)DROPIT_ERR_TIMEOUT);
                return;
            }
            for (uint32_t i = threadIdx.x; i <= width; i += blockDim.x) {
                const uint32_t c = bins[i];
                if (c) atomicAdd(&ghist[i], c);
            }
            if (threadIdx.x == 0 && cta_hi) atomicAdd(&st->n_hi[attempt], (unsigned long long)cta_hi);
        }
        barrier_target += gridDim.x;
        if (!grid_barrier(&st->barrier, barrier_target, &sh.ok)) {
            if (threadIdx.x == 0 && dev_status) atomicExch(dev_status, (int)DROPIT_ERR_TIMEOUT);
            return;
        }
        phase_stamp(st, 2);
        if (threadIdx.x == 0) sh.found = 0;
        // ---------------- phase 2: threshold key, tie quota, prefixes ----------------
        if (narrow) {
            // column sums over all CTAs and over the CTAs before this one (only the band's columns and
            // the #key>hi column carry data); every thread keeps several independent loads in flight
            if (threadIdx.x < kRowWords) {
                sh.tot[threadIdx.x] = 0;
                sh.pre[threadIdx.x] = 0;
            }
            __syncthreads();
            {
                const uint32_t ncol = width + 2;   // bins 0..width, then #key>hi (stored at kWarpBins)
                const uint32_t cells = gridDim.x * ncol;
                for (uint32_t i0 = threadIdx.x; i0 < cells; i0 += 4 * blockDim.x) {
                    uint32_t val[4], col[4], row[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const uint32_t i = i0 + u * blockDim.x;
                        row[u] = i / ncol;
                        const uint32_t c = i - row[u] * ncol;
                        col[u] = (c == width + 1) ? (uint32_t)kWarpBins : c;
                        val[u] = (i < cells) ? __ldcg(&rows[(size_t)row[u] * kRowWords + col[u]]) : 0u;
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        if (val[u]) {
                            atomicAdd(&sh.tot[col[u]], val[u]);
                            if (row[u] < blockIdx.x) atomicAdd(&sh.pre[col[u]], val[u]);
                        }
                    }
                }
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                unsigned long long cum = sh.tot[kWarpBins];   // keys above the band
                for (int d = (int)width; d >= 0; --d) {
                    const uint32_t hcount = sh.tot[d];
                    if (cum < k && k <= cum + hcount) {
                        sh.T = lo + d;
                        sh.n_gt = cum;
                        sh.quota = k - cum;
                        sh.found = 1;
                        break;
                    }
                    cum += hcount;
                }
            }
            __syncthreads();
            if (!sh.found) continue;   // T outside the band (uniform across the grid): widen and redo
            T = sh.T;
            q = (uint32_t)sh.quota;
            const uint32_t dT = T - lo;
            if (warp == 0) {
                // lane = warp index: that warp's (gt, eq), then an exclusive scan over the 32 warps
                uint32_t g = 0, e = 0;
                if (lane < kFusedWarps) {
                    g = sh.w_hi[lane];
                    e = sh.whist[lane][dT];
                    for (uint32_t d = dT + 1; d <= width; ++d) g += sh.whist[lane][d];
                }
                uint32_t gi = g, ei = e;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t yg = __shfl_up_sync(kFullMask, gi, o), ye = __shfl_up_sync(kFullMask, ei, o);
                    if (lane >= o) { gi += yg; ei += ye; }
                }
                uint32_t cta_pre_gt = sh.pre[kWarpBins], cta_pre_eq = sh.pre[dT];
                for (uint32_t d = dT + 1; d <= width; ++d) cta_pre_gt += sh.pre[d];
                if (lane < kFusedWarps) {
                    sh.wpre_gt[lane] = cta_pre_gt + gi - g;
                    sh.wpre_eq[lane] = cta_pre_eq + ei - e;
                }
            }
            __syncthreads();
            run_gt = sh.wpre_gt[warp];
            run_eq = sh.wpre_eq[warp];
            break;
        }
        // ---- general path: T from the global histogram ----
        const unsigned long long n_hi = __ldcg(&st->n_hi[attempt]);
        const uint32_t nb = width + 1;
        const uint32_t per = (nb + kFusedThreads - 1) / kFusedThreads;
        uint32_t sum = 0;
        for (uint32_t r = 0; r < per; ++r) {   // band offsets in descending key order
            const uint32_t pos = threadIdx.x * per + r;
            if (pos < nb) sum += __ldcg(&ghist[width - pos]);
        }
        uint32_t total;
        const uint32_t excl = block_exclusive_scan(sum, sh.warp, &total);
        {
            unsigned long long cum = n_hi + excl;
            if (cum < k && k <= cum + sum) {
                for (uint32_t r = 0; r < per; ++r) {
                    const uint32_t pos = threadIdx.x * per + r;
                    if (pos >= nb) break;
                    const uint32_t hcount = __ldcg(&ghist[width - pos]);
                    if (cum < k && k <= cum + hcount) {
                        sh.T = lo + (width - pos);
                        sh.n_gt = cum;
                        sh.quota = k - cum;
                        sh.found = 1;
                    }
                    cum += hcount;
                }
            }
        }
        __syncthreads();
        if (!sh.found) continue;
        T = sh.T;
        q = (uint32_t)sh.quota;
        // one extra counting read: (#key > T, #key == T) of every warp's run
        {
            const uint32_t c_gt = ge_const(T + 1), c_ge = ge_const(T);
            uint32_t g = 0, e = 0;
            for (int64_t blk = blk0; blk < blk1; ++blk) {
                uint4 va[kVpl];
                int na[kVpl];
                load_block(x, blk, lane, nvec_full, n, va, na);
#pragma unroll
                for (int j = 0; j < kVpl; ++j) {
                    const uint32_t w[4] = {va[j].x, va[j].y, va[j].z, va[j].w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t m = w[i] & 0x7FFF7FFFu;
                        const uint32_t a = m + c_gt;
                        uint32_t eqb = (m + c_ge) & ~a & kHiBits;
                        if (2 * i >= na[j]) eqb &= ~0x8000u;          // elements past the end are not ties
                        if (2 * i + 1 >= na[j]) eqb &= ~0x80000000u;
                        g += __popc(a & kHiBits);
                        e += __popc(eqb);
                    }
                }
            }
            for (int o = 16; o > 0; o >>= 1) {
                g += __shfl_xor_sync(kFullMask, g, o);
                e += __shfl_xor_sync(kFullMask, e, o);
            }
            __syncthreads();
            if (lane == 0) {
                sh.wpre_gt[warp] = g;
                sh.wpre_eq[warp] = e;
            }
            __syncthreads();
            uint32_t cg = 0, ce = 0, wg = 0, we = 0;
            for (int w = 0; w < kFusedWarps; ++w) {
                const uint32_t a = sh.wpre_gt[w], b = sh.wpre_eq[w];
                if (w < warp) { wg += a; we += b; }
                cg += a;
                ce += b;
            }
            if (threadIdx.x == 0) st_relaxed_u64(&agg[blockIdx.x], ((unsigned long long)ce << 32) | cg);
            barrier_target += gridDim.x;
            if (!grid_barrier(&st->barrier, barrier_target, &sh.ok)) {
                if (threadIdx.x == 0 && dev_status) atomicExch(dev_status, (int)DROPIT_ERR_TIMEOUT);
                return;
            }
            unsigned long long pg = 0, pe = 0;
            for (uint32_t b = threadIdx.x; b < blockIdx.x; b += blockDim.x) {
                const unsigned long long a = ld_relaxed_u64(&agg[b]);
                pg += a & 0xFFFFFFFFull;
                pe += a >> 32;
            }
            run_gt = (uint32_t)block_sum_u64(pg, sh.red64) + wg;
            run_eq = (uint32_t)block_sum_u64(pe, sh.red64) + we;
        }
        break;
    }
    __syncthreads();   // shared histograms are dead from here on; phase 3 reuses the memory
    phase_stamp(st, 3);

    // ---------------- phase 3: ordered compaction, one warp per run of blocks ----------------
    ptx::launch_dependents();   // a programmatically launched kernel behind this one may be brought up
    const int64_t nwords = (n + 31) / 32;
    uint16_t* s_vals = s_vals_all + (size_t)warp * kStageVals;
    int32_t* s_idx = s_idx_all + (size_t)warp * kStageIdx;
    const uint32_t c_gt = ge_const(T + 1), c_ge = ge_const(T);
    uint32_t gpos = run_gt + min(run_eq, q);   // retained elements before this warp's next block
    uint32_t pend = gpos & 7u, foreign = pend;       // staged-but-unwritten values; leading slots not ours
    uint32_t pend_i = gpos & 3u, foreign_i = pend_i;
#pragma unroll
    for (int d = 0; d < kRingDepth - 1; ++d) issue_block(blk0 + d, ring_lane + d * kRingSlotBytes);
    int slot = 0, slot_ahead = kRingDepth - 1;
    // One block of the run.  FULL: every vector of the block is whole, so the bounds arithmetic folds away.
    auto compact_block = [&](int64_t blk, auto full_tag) {
        constexpr bool FULL = decltype(full_tag)::value;
        issue_block(blk + kRingDepth - 1, ring_lane + slot_ahead * kRingSlotBytes);
        ring_wait();
        uint4 cur[kVpl];
        ring_read(ring_lane + slot * kRingSlotBytes, cur);
        slot = (slot + 1 == kRingDepth) ? 0 : slot + 1;
        slot_ahead = (slot_ahead + 1 == kRingDepth) ? 0 : slot_ahead + 1;
        uint32_t gt8[kVpl], eq8[kVpl], cnt[kVpl];
#pragma unroll
        for (int j = 0; j < kVpl; ++j) {
            const uint32_t w[4] = {cur[j].x, cur[j].y, cur[j].z, cur[j].w};
            uint32_t a[4], eb[4], eany = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t m = w[i] & 0x7FFF7FFFu;
                a[i] = m + c_gt;                        // bit 15 of a half: key > T
                eb[i] = (m + c_ge) & ~a[i];             // bit 15 of a half: key == T
                eany |= eb[i];
            }
            const uint32_t g8 = flags4(a[0], a[1]) | (flags4(a[2], a[3]) << 4);
            uint32_t e8 = 0;
            if (eany & kHiBits) {
                e8 = flags4(eb[0], eb[1]) | (flags4(eb[2], eb[3]) << 4);
                if constexpr (!FULL) {   // zero padding past the end must not tie with T = 0
                    const int nvalid = valid_elems(blk * kBlkVecs + j * 32 + lane, nvec_full, n);
                    e8 &= (1u << nvalid) - 1u;
                }
            }
            gt8[j] = g8;
            eq8[j] = e8;
            cnt[j] = __popc(g8) | (__popc(e8) << 16);
        }

        // packed (gt | eq << 16) prefix inside the warp in (j, lane) order
        uint32_t excl[kVpl];
        uint32_t row_base = 0;
#pragma unroll
        for (int j = 0; j < kVpl; ++j) {
            uint32_t inc = cnt[j];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t y = __shfl_up_sync(kFullMask, inc, o);
                if (lane >= o) inc += y;
            }
            excl[j] = row_base + inc - cnt[j];
            row_base += __shfl_sync(kFullMask, inc, 31);
        }
        const uint32_t blk_gt = row_base & 0xFFFFu, blk_eq = row_base >> 16;
        const uint32_t blk_kept_base = run_gt + min(run_eq, q);   // == gpos

        uint32_t keep8[kVpl];
#pragma unroll
        for (int j = 0; j < kVpl; ++j) {
            const uint32_t gt_before = run_gt + (excl[j] & 0xFFFFu);
            const uint32_t eq_before = run_eq + (excl[j] >> 16);
            uint32_t keep_eq = eq8[j];
            if (keep_eq) {
                const uint32_t room = (eq_before < q) ? (q - eq_before) : 0u;
                if (room < (cnt[j] >> 16)) {
                    uint32_t m = keep_eq;
                    keep_eq = 0;
                    for (uint32_t r = 0; r < room; ++r) {
                        keep_eq |= m & (0u - m);
                        m &= m - 1;
                    }
                }
            }
            keep8[j] = gt8[j] | keep_eq;
            const uint32_t kept_before = gt_before + min(eq_before, q);
            if constexpr (FULL) {   // vector blk*64 + j*32 + lane opens chunk blk*4 + j*2 + lane/16 when lane % 16 == 0
                if ((lane & 15) == 0) offsets[blk * (kBlkElems / DROPIT_CHUNK) + j * 2 + (lane >> 4)] = kept_before;
            } else {
                const int64_t vi = blk * kBlkVecs + j * 32 + lane;
                if ((lane & 15) == 0 && vi * 8 < n) offsets[(vi * 8) / DROPIT_CHUNK] = kept_before;
            }
            uint32_t pos = kept_before - blk_kept_base;
            const uint32_t w[4] = {cur[j].x, cur[j].y, cur[j].z, cur[j].w};
            [[maybe_unused]] const int32_t first_idx = (int32_t)(blk * kBlkElems) + (j * 32 + lane) * 8;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                if ((keep8[j] >> e) & 1u) {
                    s_vals[pend + pos] = (uint16_t)((w[e >> 1] >> ((e & 1) * 16)) & 0xFFFFu);
                    if constexpr (INDEX32) s_idx[pend_i + pos] = first_idx + e;
                    ++pos;
                }
            }
        }
        if constexpr (!INDEX32) {
            // lanes sharing a 32-bit mask word OR their bytes, then lane i takes word i of the block
            uint32_t word[kVpl];
#pragma unroll
            for (int j = 0; j < kVpl; ++j) {
                uint32_t wv = keep8[j] << (8 * (lane & 3));
                wv |= __shfl_xor_sync(kFullMask, wv, 1);
                wv |= __shfl_xor_sync(kFullMask, wv, 2);
                word[j] = wv;
            }
            uint32_t mine = 0;
            const int src = (lane & 7) * 4;
#pragma unroll
            for (int j = 0; j < kVpl; ++j) {
                const uint32_t got = __shfl_sync(kFullMask, word[j], src);
                if ((lane >> 3) == j) mine = got;
            }
            const int64_t w0 = blk * (kBlkElems / 32);
            if constexpr (FULL) {
                if (lane < 8 * kVpl) mask[w0 + lane] = mine;
            } else {
                if (lane < 8 * kVpl && w0 + lane < nwords) mask[w0 + lane] = mine;
            }
        }
        const uint32_t kept = (run_gt + blk_gt + min(run_eq + blk_eq, q)) - blk_kept_base;
        run_gt += blk_gt;
        run_eq += blk_eq;
        __syncwarp();
        flush_pieces<uint16_t, 8>(s_vals, values + (gpos - pend), kept, pend, foreign, lane);
        if constexpr (INDEX32) flush_pieces<int32_t, 4>(s_idx, indices + (gpos - pend_i), kept, pend_i, foreign_i, lane);
        gpos += kept;
    };
    {
        int64_t blk = blk0;
        for (; blk < blk_full_end; ++blk) compact_block(blk, std::true_type{});
        for (; blk < blk1; ++blk) compact_block(blk, std::false_type{});
    }
    // tails: own values still staged (less than one 16-byte piece); leading foreign slots are skipped
    if (lane >= (int)foreign && lane < (int)pend) values[(gpos - pend) + lane] = s_vals[lane];
    if constexpr (INDEX32) {
        if (lane >= (int)foreign_i && lane < (int)pend_i) indices[(gpos - pend_i) + lane] = s_idx[lane];
    }
    phase_stamp(st, 5);
}

// ---------------------------------------------------------------------------------------------
// Host side.
// ---------------------------------------------------------------------------------------------
dropit_status fused_compress_bf16(const void* x, int64_t n, int64_t k, bool index32, void* values, void* meta,
                                  uint32_t* offsets, void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                  cudaStream_t stream) {
    const FusedPlan plan = make_fused_plan(n);
    if (workspace_bytes < plan.total_bytes) return DROPIT_ERR_WORKSPACE;
    unsigned char* ws = reinterpret_cast<unsigned char*>(workspace);
    const size_t smem_hist = (size_t)kKeySpace * 4;   // sample kernel: one full key histogram
    static_assert(kRingBytes >= (size_t)kKeySpace * 4, "the general path's histogram lives in the ring's memory");
    const size_t smem_mask = kRingBytes + (size_t)kFusedWarps * kStageVals * 2;
    const size_t smem_idx = smem_mask + (size_t)kFusedWarps * kStageIdx * 4;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(sample_band_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_hist) != cudaSuccess ||
            cudaFuncSetAttribute(fused_compress_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_mask) != cudaSuccess ||
            cudaFuncSetAttribute(fused_compress_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_idx) != cudaSuccess)
            return DROPIT_ERR_CUDA;
        attr_set = true;
    }
    {
        cudaLaunchAttribute pdl[1];
        pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        pdl[0].val.programmaticStreamSerializationAllowed = 1;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(1);
        cfg.blockDim = dim3(kSampleThreads);
        cfg.dynamicSmemBytes = smem_hist;
        cfg.stream = stream;
        cfg.attrs = pdl;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, sample_band_kernel, reinterpret_cast<const uint4*>(x), n, (unsigned long long)k, ws,
                               plan.zero_bytes) != cudaSuccess) {
            (void)cudaGetLastError();
            return DROPIT_ERR_CUDA;
        }
    }
    dropit_status s = check_launch();
    if (s != DROPIT_OK) return s;

    const uint4* xp = reinterpret_cast<const uint4*>(x);
    unsigned long long kk = (unsigned long long)k;
    int bpw = plan.blocks_per_warp;
    size_t h0 = plan.hist_off[0], h1 = plan.hist_off[1], ao = plan.agg_off, ro = plan.rows_off;
    uint16_t* vals = reinterpret_cast<uint16_t*>(values);
    uint32_t* maskp = index32 ? nullptr : reinterpret_cast<uint32_t*>(meta);
    int32_t* idxp = index32 ? reinterpret_cast<int32_t*>(meta) : nullptr;
    void* args[] = {&xp, &n, &kk, &bpw, &ws, &h0, &h1, &ao, &ro, &vals, &maskp, &idxp, &offsets, &dev_status};
    const void* fn = index32 ? (const void*)fused_compress_kernel<true> : (const void*)fused_compress_kernel<false>;
    if (cudaLaunchCooperativeKernel(fn, dim3(plan.grid), dim3(kFusedThreads), args, index32 ? smem_idx : smem_mask,
                                    stream) != cudaSuccess) {
        cudaGetLastError();
        return DROPIT_ERR_CUDA;
    }
    return check_launch();
}

}  // namespace dropit

// ---------------------------------------------------------------------------------------------
// Compression without a caller-provided workspace.
// ---------------------------------------------------------------------------------------------
namespace dropit {

// The kernels' scratch (selection state, two key histograms, per-CTA rows) does not grow with the
// tensor, so one fixed array in device memory can serve.  Every GPU that loads the library holds
// these bytes until the process exits.
constexpr size_t kStaticScratchBytes =
    kStateBytes + 2 * (size_t)kKeySpace * 4 + (size_t)kMaxGrid * 8 + (size_t)kMaxGrid * kRowWords * 4;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code `g_static_scratch` is only a handle for the symbol, not an address a kernel may use:
// the device address is looked up once per device, with that device current.
static unsigned char* static_scratch_address() {
    static unsigned char* cached[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!cached[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        cached[dev] = reinterpret_cast<unsigned char*>(p);
    }
    return cached[dev];
}

}  // namespace dropit

extern "C" size_t dropit_compress_static_scratch_bytes(void) { return dropit::kStaticScratchBytes; }

extern "C" dropit_status dropit_compress_static(const void* x, int64_t n, double gamma, dropit_format format,
                                                void* values, void* meta, uint32_t* offsets, int32_t* dev_status,
                                                void* cuda_stream) {
    using namespace dropit;
    if (n < 0 || !(gamma >= 0.0 && gamma <= 1.0)) return DROPIT_ERR_INVALID_ARG;
    if (format != DROPIT_FMT_BITMASK && format != DROPIT_FMT_INDEX32) return DROPIT_ERR_INVALID_ARG;
    if (n > DROPIT_STATIC_MAX_ELEMS) return DROPIT_ERR_WORKSPACE;   // beyond what the built-in scratch is stated for
    if (n == 0) return DROPIT_OK;
    const int64_t k = dropit_keep_count(n, gamma);
    if (!x || !offsets || !is_aligned16(x) || !is_aligned16(offsets)) return DROPIT_ERR_INVALID_ARG;
    if (format == DROPIT_FMT_BITMASK && (!meta || !is_aligned16(meta))) return DROPIT_ERR_INVALID_ARG;
    if (k > 0 && (!values || !is_aligned16(values))) return DROPIT_ERR_INVALID_ARG;
    if (k > 0 && format == DROPIT_FMT_INDEX32 && (!meta || !is_aligned16(meta))) return DROPIT_ERR_INVALID_ARG;
    cudaStream_t stream = as_stream(cuda_stream);
    if (k == 0) {   // gamma = 1: nothing retained, no scratch involved
        if (format == DROPIT_FMT_BITMASK &&
            cudaMemsetAsync(meta, 0, (size_t)((n + 31) / 32) * 4, stream) != cudaSuccess)
            return DROPIT_ERR_CUDA;
        if (cudaMemsetAsync(offsets, 0, (size_t)((n + DROPIT_CHUNK - 1) / DROPIT_CHUNK) * 4, stream) != cudaSuccess)
            return DROPIT_ERR_CUDA;
        return DROPIT_OK;
    }
    if (fused_compress_workspace_bytes(n) > kStaticScratchBytes) return DROPIT_ERR_WORKSPACE;
    unsigned char* scratch = static_scratch_address();
    if (!scratch) return DROPIT_ERR_CUDA;
    // the sample kernel zeroes the part of the scratch that must start at zero on every call
    return fused_compress_bf16(x, n, k, format == DROPIT_FMT_INDEX32, values, meta, offsets, scratch,
                               kStaticScratchBytes, dev_status, stream);
}

