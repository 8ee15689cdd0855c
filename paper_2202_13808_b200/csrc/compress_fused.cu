// bf16 min-k selection + packing as ONE persistent cooperative kernel (Sec. 3.3 "Min-K Elements",
// Sec. 3.2 a-hat = {a_Xr, X_r}).
//
// Every WARP owns one contiguous run of 1024-element super-blocks (two 512-element blocks) and keeps it for the
// whole kernel, so
// the ordered compaction needs no block-wide synchronisation and warps drift freely.
//   sample  every CTA histograms the same 16 Ki-element jittered sample in shared memory and brackets
//           the threshold key T between two keys [lo, hi] (6-sigma margin on the sample rank).
//   phase 1 one read of the tensor: keys above hi are counted in a register, keys inside the band
//           go to a small per-warp histogram, the rest is ignored (two packed bf16 per 32-bit word
//           are classified with one add each, so the pass is bound by HBM, not by atomics).
//   sync    one grid barrier (bounded wait; the launch is cooperative so all CTAs are resident).
//   phase 2 every CTA sums the per-CTA band histograms: T and the tie quota q follow from the total,
//           the CTA's exclusive prefix from the rows before it, each warp's prefix from the per-warp
//           histograms.  No second counting pass.
//   phase 3 second read (L2 hits for tensors that fit L2): element i is retained iff key_i > T, or
//           key_i == T and fewer than q equal keys precede it; #retained before i =
//           gt_before + min(eq_before, q).  A lane owns 32 consecutive elements of a super-block; retained values are
//           staged per warp and leave in aligned 16-byte pieces.
// When the band is wider than the per-warp histogram (small tensors, which are not sampled; key
// distributions that are flat around T; a sample that missed) a general path is taken instead:
// full CTA histogram in shared memory, global histogram by atomics, then one extra counting read.
// Nothing in the scratch has to be cleared before a call: the grid barrier counts arrivals under a
// number unique to the call, everything else is written before it is read.
#include <type_traits>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace dropit {

constexpr int kFusedThreads = 1024;                             // main kernel; 1 CTA per SM
constexpr int kFusedWarps = kFusedThreads / 32;
constexpr int kVpl = 2;                                        // 16-byte vectors per lane per warp block
constexpr int kBlkVecs = 32 * kVpl;                            // vectors per warp block
constexpr int kBlkElems = kBlkVecs * 8;                        // 512 bf16
constexpr int kP1Blocks = 4 / kVpl;                            // blocks loaded per phase-1 iteration (4 loads per lane)
constexpr int kKeySpace = 1 << 15;
constexpr int kWarpBins = 64;                                  // per-warp band histogram
constexpr int kRowWords = kWarpBins + 2;                       // per-CTA row: bins, #key>hi, pad
constexpr int kMaxGrid = 512;                                  // < 4096: departures are counted in 12 bits of the barrier word
constexpr int kSampleVecs = 2048;                              // 16384 sampled elements
constexpr int64_t kSampleMinElems = 1 << 19;                   // below this the band is the full key range
constexpr int kBarrierSpinLimit = 1 << 22;
constexpr uint32_t kHiBits = 0x80008000u;
// The streaming passes work on super-blocks of two blocks (1024 elements): a lane owns 32 CONSECUTIVE
// elements, i.e. one mask word.  Each warp has a ring of two super-block slots fed by cp.async.
constexpr int kSbVecs = 2 * kBlkVecs;                          // 128 vectors
constexpr int kSbElems = 2 * kBlkElems;                        // 1024 bf16
constexpr int kSbBytes = kSbVecs * 16;                         // 2 KB
constexpr int kSbChunks = kSbElems / DROPIT_CHUNK;             // 8 seek-table entries
constexpr int kRingSlots = 2;
constexpr size_t kRingBytes = (size_t)kFusedWarps * kRingSlots * kSbBytes;   // 128 KB
constexpr int kStageVals = kSbElems + 8;                       // per-warp staging: a super-block's retained values behind < 8 carried ones
constexpr size_t kStageBytes = (size_t)kFusedWarps * kStageVals * 2;   // 64.5 KB
static_assert(kStageBytes >= (size_t)kKeySpace * 2, "the sample's 16-bit histogram lives in the staging area");

struct FusedState {
    unsigned long long barrier;  // grid barrier: call epoch << 32 | arrivals (needs no clearing between calls)
    uint32_t pad0[2];
    unsigned long long n_hi[2];  // general path: #{key > hi} per attempt
    uint32_t reserved[24];
};
static_assert(sizeof(FusedState) == 128, "FusedState layout");

struct FusedPlan {
    int64_t blocks_total;
    int grid;
    int blocks_per_warp;
    size_t hist_off[2], agg_off, rows_off, total_bytes;
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
    p.blocks_per_warp = (p.blocks_per_warp + 1) & ~1;          // a run is a whole number of super-blocks
    p.hist_off[0] = kStateBytes;
    p.hist_off[1] = p.hist_off[0] + (size_t)kKeySpace * 4;
    p.agg_off = p.hist_off[1] + (size_t)kKeySpace * 4;
    p.rows_off = p.agg_off + (size_t)kMaxGrid * 8;
    p.total_bytes = p.rows_off + (size_t)kMaxGrid * kRowWords * 4;
    return p;
}

size_t fused_compress_workspace_bytes(int64_t n) { return make_fused_plan(n).total_bytes; }

// ---------------------------------------------------------------------------------------------
// Statistics handed from the producer of a tensor to its compression (produce_kernel below writes them while
// it writes the tensor, fused_compress_kernel then skips its sample step, its first read and its grid barrier):
//   header | per-CTA rows [grid][kRowWords] | per-warp band histograms [grid][32 warps][kPrepWarpWords]
// A row and a per-warp record hold what phase 1 of the selection kernel would have left in shared memory.
// ---------------------------------------------------------------------------------------------
constexpr uint32_t kPrepMagic = 0xD20917F1u;
constexpr int kPrepWarpWords = kWarpBins + 2;                  // band bins, #{key > hi}, pad
struct PrepHeader {
    uint32_t magic, valid;               // valid: the tensor was sampled and the band fits the per-warp histograms
    uint32_t lo, hi;                     // the band of keys around the threshold
    uint32_t grid, blocks_per_warp;      // the work partition the statistics were taken under
    unsigned long long n, k;
    uint32_t reserved[6];
};
static_assert(sizeof(PrepHeader) == 64, "PrepHeader layout");
__host__ __device__ inline const uint32_t* prep_rows(const unsigned char* prep) {
    return reinterpret_cast<const uint32_t*>(prep + sizeof(PrepHeader));
}
__host__ __device__ inline const uint32_t* prep_warp_hist(const unsigned char* prep, uint32_t grid) {
    return prep_rows(prep) + (size_t)grid * kRowWords;
}
static size_t prep_bytes_for(int64_t n) {
    const FusedPlan p = make_fused_plan(n);
    return sizeof(PrepHeader) + (size_t)p.grid * kRowWords * 4 + (size_t)p.grid * kFusedWarps * kPrepWarpWords * 4;
}

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

// Eight flags held in bit 15 and bit 31 of four words -> 8 bits in element order.  prmt gathers the flag
// bytes of each pair of words; flags of the first pair go to bit 0 of each byte, of the second pair to
// bit 4; one multiply lines all eight up at bits 24..31 (no two partial products share a bit, so no carries).
__device__ __forceinline__ uint32_t flags8(uint32_t x0, uint32_t x1, uint32_t x2, uint32_t x3) {
    const uint32_t r0 = __byte_perm(x0, x1, 0x7531), r1 = __byte_perm(x2, x3, 0x7531);
    const uint32_t u = ((r0 >> 7) & 0x01010101u) | ((r1 >> 3) & 0x10101010u);
    return (u * 0x01020408u) >> 24;
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
// Sample step: bracket the threshold key.  Every CTA runs it on the same 16 Ki elements (the first
// CTA to ask brings them in from HBM, the others read them from L2) and therefore arrives at the
// same band without any exchange.  `bins`: kKeySpace counters in shared memory; band[0..1] = lo, hi.
// Ends with a block-wide barrier.
// ---------------------------------------------------------------------------------------------
// `map`: applied to every sampled vector before its keys are taken (the identity for the selection kernel;
// the producer kernel brackets the threshold of act(x), so it maps the sample through act).
template <typename AfterLoads, typename Map>
__device__ __forceinline__ void sample_band(const uint4* __restrict__ x, int64_t n, unsigned long long k, uint32_t* bins,
                                            uint32_t* s_warp, uint32_t* band, FusedState* st, AfterLoads after_loads,
                                            Map map) {
    // after_loads: called once by every thread, after the sample has been counted (or at once when there is no sample)
    const int64_t nvec = n / 8;
    const bool sampled = n >= kSampleMinElems;
    uint4 sv[kSampleVecs / kFusedThreads];
    if (sampled) {   // issue the sample loads first; they fly while the counters are cleared
        const int64_t stride = nvec / kSampleVecs;   // >= 32
#pragma unroll
        for (int r = 0; r < kSampleVecs / kFusedThreads; ++r) {
            const uint32_t s = r * kFusedThreads + threadIdx.x;
            const uint32_t h = (s * 2654435761u) >> 7;   // jitter inside the stride window
            sv[r] = ld_stream(x + (int64_t)s * stride + (int64_t)(h % (uint32_t)stride));
        }
    }
    if (!sampled) after_loads();
    if (threadIdx.x == 0) {
        band[0] = 0;
        band[1] = kKeySpace - 1;
    }
    if (sampled) {
        // two 16-bit counters per word (a counter holds at most the sample size, 16384)
        uint4* z = reinterpret_cast<uint4*>(bins);
        for (int i = threadIdx.x; i < kKeySpace / 8; i += kFusedThreads) z[i] = make_uint4(0, 0, 0, 0);
        __syncthreads();
#pragma unroll
        for (int r = 0; r < kSampleVecs / kFusedThreads; ++r) {
            uint32_t key[8];
            keys_of(map(sv[r]), key);
#pragma unroll
            for (int e = 0; e < 8; ++e) atomicAdd(&bins[key[e] >> 1], 1u << ((key[e] & 1u) * 16));
        }
        __syncthreads();
        // ranks (counted from the largest key) that bracket the threshold with a 6-sigma margin
        const float S = (float)(kSampleVecs * 8);
        const float p = (float)((double)k / (double)n);
        const float ks = p * S;
        const float margin = 6.0f * sqrtf(S * p * (1.0f - p)) + 16.0f;
        const float r_hi = ks - margin, r_lo = ks + margin;
        // as integers: for an integer count c, c < r <=> c < ceil(r) and r <= c <=> ceil(r) <= c.  0 = no such rank.
        const uint32_t R_hi = (r_hi >= 1.0f) ? (uint32_t)ceilf(r_hi) : 0u;
        const uint32_t R_lo = (r_lo <= S) ? (uint32_t)ceilf(r_lo) : 0u;
        constexpr int PER = kKeySpace / kFusedThreads;   // keys per thread, descending: kKeySpace-1 - (t*PER + r)
        const int t = threadIdx.x;
        static_assert(PER == 32, "the walk below assumes 16 words per thread");
        // the thread's 16 words hold its 32 counters; the four 16-byte reads go in an order rotated by (t/2) mod 4,
        // so that the threads of a quarter-warp (64 bytes apart) touch different banks
        const uint4* mine = reinterpret_cast<const uint4*>(bins + (kKeySpace / 2 - (t + 1) * (PER / 2)));
        uint32_t sum = 0;
#pragma unroll
        for (int j = 0; j < PER / 8; ++j) {
            const uint4 v = mine[j ^ ((t >> 1) & 3)];
            sum += (v.x & 0xFFFFu) + (v.x >> 16) + (v.y & 0xFFFFu) + (v.y >> 16) + (v.z & 0xFFFFu) + (v.z >> 16) +
                   (v.w & 0xFFFFu) + (v.w >> 16);
        }
        after_loads();   // what the caller wants in flight while the thresholds are worked out (issued earlier, it delays the sample)
        uint32_t total;
        const uint32_t excl = block_exclusive_scan(sum, s_warp, &total);
        // key at descending rank r: cum_before < r <= cum_before + h
        if ((excl < R_hi && R_hi <= excl + sum) || (excl < R_lo && R_lo <= excl + sum)) {
            // one or two threads of the CTA get here: they read their counters again, in key order
            uint32_t cw[PER / 2];
#pragma unroll
            for (int j = 0; j < PER / 8; ++j) {
                const uint4 v = mine[j];
                cw[4 * j] = v.x; cw[4 * j + 1] = v.y; cw[4 * j + 2] = v.z; cw[4 * j + 3] = v.w;
            }
            uint32_t cum = excl;
#pragma unroll
            for (int r = 0; r < PER; ++r) {
                // key = kKeySpace-1 - (t*PER + r) lives in word 15 - r/2 of the thread, upper half when r is even
                const uint32_t key = kKeySpace - 1 - (t * PER + r);
                const uint32_t cwr = cw[PER / 2 - 1 - r / 2];
                const uint32_t hh = (r & 1) ? (cwr & 0xFFFFu) : (cwr >> 16);
                if (cum < R_hi && R_hi <= cum + hh) band[1] = key;
                if (cum < R_lo && R_lo <= cum + hh) band[0] = key;
                cum += hh;
            }
        }
    }
    __syncthreads();
}

// ---------------------------------------------------------------------------------------------
// Main kernel.
// ---------------------------------------------------------------------------------------------
struct FusedShared {
    uint32_t warp[32];
    unsigned long long red64[32];
    uint32_t whist[kFusedWarps][kWarpBins];   // per-warp band histograms (fast path)
    uint32_t w_hi[kFusedWarps];               // per-warp #{key > hi}
    uint32_t tot[kRowWords];                  // band histogram over all CTAs (+ #key>hi)
    uint32_t pre[kRowWords];                  // ... over the CTAs before this one
    uint32_t wpre_gt[kFusedWarps], wpre_eq[kFusedWarps];   // exclusive prefix of each warp (absolute)
    uint32_t T, found;
    uint32_t band[2];                         // lo, hi from the sample
    unsigned long long n_gt, quota;
    int ok;
};

// Grid barrier on one 64-bit word = (epoch << 32 | arrivals).  `epoch` is unique to the call; CTA 0
// stores (epoch << 32) into the word when the kernel starts (barrier_open), so nothing has to be cleared
// between calls or before the first one.  An arriving CTA waits until the word carries its epoch (it
// does, long since, in any normal run), adds one, and waits for `target` = the arrivals expected so far
// in this call.  Every wait is bounded: returns false when one runs out.
__device__ __forceinline__ void barrier_open(unsigned long long* word, uint32_t epoch) {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        // relaxed: nothing is published with it, and the other CTAs look for it microseconds later
        asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(word), "l"((unsigned long long)epoch << 32) : "memory");
    }
}
__device__ __forceinline__ bool grid_barrier(unsigned long long* word, uint32_t epoch, uint32_t target, int* s_ok,
                                             int spin_max) {
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        bool ok = true;
        int spins = 0;
        unsigned long long v;
        for (;;) {   // the word belongs to this call
            asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(word) : "memory");
            if ((uint32_t)(v >> 32) == epoch) break;
            if (++spins > spin_max) { ok = false; break; }
            __nanosleep(32);
        }
        if (ok) {
            atomicAdd(word, 1ull);
            const unsigned long long goal = ((unsigned long long)epoch << 32) | target;
            for (;;) {
                asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(word) : "memory");
                if (v >= goal) break;
                if (++spins > spin_max) { ok = false; break; }
                __nanosleep(32);
            }
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

// The warp's super-blocks are streamed through a per-warp ring in shared memory fed by cp.async, one
// super-block ahead, so that enough bytes are in flight per SM without holding them in registers.
// The copies are coalesced (lane copies vectors lane, lane+32, lane+64, lane+96 of the super-block);
// a lane then reads the 64 bytes at 64*lane, which other lanes copied, so a __syncwarp follows the wait.
// `lane_slot` = shared address of vector `lane` in the slot.
__device__ __forceinline__ void sb_issue_edge(uint32_t lane_slot, const uint4* x, int64_t sb, int lane, int64_t nvec_full,
                                              int64_t n) {
#pragma unroll
    for (int j = 0; j < kSbVecs / 32; ++j) {
        const int64_t vi = sb * kSbVecs + j * 32 + lane;
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
// The same for a super-block whose vectors are all whole: `src` = vector `lane` of the super-block.
__device__ __forceinline__ void sb_issue_full(uint32_t lane_slot, const uint4* src) {
#pragma unroll
    for (int j = 0; j < kSbVecs / 32; ++j)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(lane_slot + j * 512), "l"(src + j * 32) : "memory");
    asm volatile("cp.async.commit_group;" ::: "memory");
}
// The lane's 32 elements (16 words) of a slot; `own` = shared address of the slot + 64 * lane.  The lanes of a
// warp read 64-byte pieces 64 bytes apart, which would put every other lane of a quarter-warp on the same banks;
// so the lane's j-th load takes its vector j ^ rot (rot = (lane / 2) % 4) and the eight lanes of a quarter-warp
// touch eight different 16-byte columns.  w[4 * j ..] then holds the lane's elements 8 * (j ^ rot) ..
__device__ __forceinline__ void sb_read(uint32_t own, uint32_t rot, uint32_t (&w)[16]) {
#pragma unroll
    for (int j = 0; j < 4; ++j)
        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(w[4 * j]), "=r"(w[4 * j + 1]), "=r"(w[4 * j + 2]), "=r"(w[4 * j + 3])
                     : "r"(own + ((j ^ rot) << 4))
                     : "memory");
}
// All but the most recently committed super-block have landed.
__device__ __forceinline__ void sb_wait() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }
__device__ __forceinline__ int valid_elems(int64_t vi, int64_t nvec_full, int64_t n) {
    return vi < nvec_full ? 8 : (vi == nvec_full ? (int)(n & 7) : 0);
}
__device__ __forceinline__ uint32_t top_bit(uint32_t m) {   // index of the highest set bit (m != 0)
    uint32_t e;
    asm("bfind.u32 %0, %1;" : "=r"(e) : "r"(m));
    return e;
}
__device__ __forceinline__ uint32_t lds_u16(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
// Mask of the lane's elements that exist: the lane owns [first, first + 32) of a tensor of n elements.
__device__ __forceinline__ uint32_t valid_mask32(int64_t first, int64_t n) {
    const int64_t left = n - first;
    return left >= 32 ? 0xFFFFFFFFu : (left > 0 ? (1u << (int)left) - 1u : 0u);
}

template <bool INDEX32>
__global__ void __launch_bounds__(kFusedThreads, 1)
fused_compress_kernel(const uint4* __restrict__ x, int64_t n, unsigned long long k, int blocks_per_warp, uint32_t epoch,
                      unsigned char* ws, size_t hist_off0, size_t hist_off1, size_t agg_off, size_t rows_off,
                      uint16_t* __restrict__ values, uint32_t* __restrict__ mask, int32_t* __restrict__ indices,
                      uint32_t* __restrict__ offsets, int32_t* dev_status, int spin_max, const unsigned char* prep) {
    // shared memory: [input ring, 128 KB | general path: full key histogram]
    //                [phase 3: per-warp value staging, 64 KB | sample step: 16-bit key histogram]
    //                [control block of phases 1-2]
    extern __shared__ __align__(16) unsigned char fsm[];
    uint32_t* bins = reinterpret_cast<uint32_t*>(fsm);
    uint32_t* sample_bins = reinterpret_cast<uint32_t*>(fsm + kRingBytes);
    uint16_t* s_vals_all = reinterpret_cast<uint16_t*>(fsm + kRingBytes);   // phase 3: per-warp staging
    FusedShared& sh = *reinterpret_cast<FusedShared*>(fsm + kRingBytes + kStageBytes);

    FusedState* st = reinterpret_cast<FusedState*>(ws);
    unsigned long long* agg = reinterpret_cast<unsigned long long*>(ws + agg_off);
    uint32_t* rows = reinterpret_cast<uint32_t*>(ws + rows_off);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ring_warp = ptx_smem(fsm) + warp * (kRingSlots * kSbBytes);
    const uint32_t ring_copy = ring_warp + lane * 16;   // where the lane's copies of a slot start
    const uint32_t ring_own = ring_warp + lane * 64;    // the lane's 32 elements of a slot
    const uint32_t rot = (uint32_t)(lane >> 1) & 3u;     // see sb_read
    const int64_t nvec_full = n / 8;
    const int64_t blocks_total = (n + kBlkElems - 1) / kBlkElems;
    const int64_t blk0 = ((int64_t)blockIdx.x * kFusedWarps + warp) * blocks_per_warp;   // even
    int64_t blk1 = blk0 + blocks_per_warp;
    if (blk1 > blocks_total) blk1 = blocks_total;
    // the same run in super-blocks; those below sb_full_end consist of whole vectors only and take the
    // paths without bounds arithmetic
    const int64_t sb0 = blk0 / 2, sb1 = (blk1 + 1) / 2;
    const int64_t sb_full_end = (nvec_full / kSbVecs < sb1) ? nvec_full / kSbVecs : sb1;
    auto issue_sb = [&](int64_t sb, int slot) {
        const uint32_t dst = ring_copy + slot * kSbBytes;
        if (sb < sb_full_end) sb_issue_full(dst, x + sb * kSbVecs + lane);
        else if (sb < sb1) sb_issue_edge(dst, x, sb, lane, nvec_full, n);
        else asm volatile("cp.async.commit_group;" ::: "memory");
    };
    uint32_t barrier_target = 0;

    // the general path's totals start at zero; the grid barriers order this store before their first use
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        st->n_hi[0] = 0;
        st->n_hi[1] = 0;
    }
    barrier_open(&st->barrier, epoch);
    // the first super-block of the run is requested while the sample is evaluated, which hides its latency
    const PrepHeader* ph = reinterpret_cast<const PrepHeader*>(prep);
    // statistics handed over by the producer kernel are used when they describe exactly this call
    const bool prepared = prep != nullptr && ph->magic == kPrepMagic && ph->valid != 0 && ph->n == (unsigned long long)n &&
                          ph->k == k && ph->grid == gridDim.x && ph->blocks_per_warp == (uint32_t)blocks_per_warp;
    if (prepared) {
        if (threadIdx.x == 0) {
            sh.band[0] = ph->lo;
            sh.band[1] = ph->hi;
        }
        const uint32_t* wh = prep_warp_hist(prep, ph->grid) + (size_t)blockIdx.x * kFusedWarps * kPrepWarpWords;
        for (int i = threadIdx.x; i < kFusedWarps * kWarpBins; i += blockDim.x)
            (&sh.whist[0][0])[i] = wh[(i / kWarpBins) * kPrepWarpWords + (i % kWarpBins)];
        if (threadIdx.x < kFusedWarps) sh.w_hi[threadIdx.x] = wh[threadIdx.x * kPrepWarpWords + kWarpBins];
        rows = const_cast<uint32_t*>(prep_rows(prep));
        __syncthreads();
    } else {
        sample_band(x, n, k, sample_bins, sh.warp, sh.band, st, [&] { issue_sb(sb0, 0); }, [](const uint4& v) { return v; });
    }
    bool prefetched = !prepared;
    uint32_t lo = sh.band[0], hi = sh.band[1];
    uint32_t T = 0, q = 0;
    uint32_t run_gt = 0, run_eq = 0;   // this warp's exclusive prefix (absolute)

    for (int attempt = 0; attempt < 2; ++attempt) {
        if (attempt == 1) {
            lo = 0;
            hi = kKeySpace - 1;
        }
        const uint32_t width = hi - lo;
        const bool narrow = width < (uint32_t)kWarpBins;   // uniform over the grid
        uint32_t* ghist = reinterpret_cast<uint32_t*>(ws + (attempt == 0 ? hist_off0 : hist_off1));
        // With the producer's statistics the band histograms, the per-warp counts and the per-CTA rows of the
        // first attempt are already there: no first read of the tensor, no grid barrier.
        if (!(prepared && attempt == 0)) {
            // ---------------- phase 1: band histogram ----------------
            if (narrow) {
                for (int i = threadIdx.x; i < kFusedWarps * kWarpBins; i += blockDim.x) (&sh.whist[0][0])[i] = 0;
            } else {
                if (prefetched) {   // the histogram takes the ring's memory: let the requested blocks land first
                    asm volatile("cp.async.wait_all;" ::: "memory");
                    __syncthreads();
                }
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
                // stream the run through the ring, one super-block ahead
                if (!prefetched) issue_sb(sb0, 0);
                int slot = 0;
                auto count_sb = [&](int64_t sb, auto full_tag) {
                    constexpr bool FULL = decltype(full_tag)::value;
                    issue_sb(sb + 1, slot ^ 1);
                    sb_wait();
                    __syncwarp();   // the lane reads vectors that other lanes copied
                    const uint32_t own = ring_own + slot * kSbBytes;
                    uint32_t w[16];
                    sb_read(own, rot, w);
                    uint32_t hi_flags = 0, pending = 0;
    #pragma unroll
                    for (int g = 0; g < 4; ++g) {   // four words = eight elements at a time
                        uint32_t a[4], b[4];
    #pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const uint32_t m = w[4 * g + i] & 0x7FFF7FFFu;
                            a[i] = m + c_hi;                   // bit 15 of a half: key > hi
                            b[i] = (m + c_lo) & ~a[i];         // bit 15 of a half: lo <= key <= hi
                        }
                        // above the band only the count matters: the flag bytes of all 16 words share one word
                        hi_flags |= ((__byte_perm(a[0], a[1], 0x7531) & 0x80808080u) >> (2 * g)) |
                                    ((__byte_perm(a[2], a[3], 0x7531) & 0x80808080u) >> (2 * g + 1));
                        pending |= flags8(b[0], b[1], b[2], b[3]) << ((g ^ rot) << 3);
                    }
                    cnt_hi += __popc(hi_flags);
                    if constexpr (!FULL) pending &= valid_mask32(sb * kSbElems + lane * 32, n);   // zero padding is no data
                    while (pending) {   // a few percent of the elements: the band histogram (their order is irrelevant)
                        const uint32_t e = top_bit(pending);
                        pending ^= 1u << e;
                        const uint32_t d = (lds_u16(own + 2u * e) & 0x7FFFu) - lo;
                        if (d == 0) ++cnt_lo; else atomicAdd(&hist[d], 1u);
                    }
                    __syncwarp();   // every lane is done with the slot before it is refilled
                    slot ^= 1;
                };
                int64_t sb = sb0;
                for (; sb < sb_full_end; ++sb) count_sb(sb, std::true_type{});
                for (; sb < sb1; ++sb) count_sb(sb, std::false_type{});
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
            prefetched = false;
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
                if (!grid_barrier(&st->barrier, epoch, barrier_target, &sh.ok, spin_max)) {
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
            if (!grid_barrier(&st->barrier, epoch, barrier_target, &sh.ok, spin_max)) {
                if (threadIdx.x == 0 && dev_status) atomicExch(dev_status, (int)DROPIT_ERR_TIMEOUT);
                return;
            }
        }
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
                // thread (g, c) adds column c of rows g, g + kGroups, ...: consecutive threads read consecutive
                // words of a row, and a thread's loads are independent of one another
                constexpr int kGroups = kFusedThreads / kRowWords;
                constexpr int kInFlight = 8;
                const uint32_t g = threadIdx.x / kRowWords, c = threadIdx.x - g * kRowWords;
                if (g < (uint32_t)kGroups && (c <= width || c == (uint32_t)kWarpBins)) {
                    uint32_t t_sum = 0, p_sum = 0;
                    for (uint32_t r0 = g; r0 < gridDim.x; r0 += kInFlight * kGroups) {
                        uint32_t val[kInFlight];
#pragma unroll
                        for (int u = 0; u < kInFlight; ++u) {
                            const uint32_t r = r0 + u * kGroups;
                            val[u] = (r < gridDim.x) ? __ldcg(&rows[(size_t)r * kRowWords + c]) : 0u;
                        }
#pragma unroll
                        for (int u = 0; u < kInFlight; ++u) {
                            t_sum += val[u];
                            if (r0 + u * kGroups < blockIdx.x) p_sum += val[u];
                        }
                    }
                    if (t_sum) atomicAdd(&sh.tot[c], t_sum);
                    if (p_sum) atomicAdd(&sh.pre[c], p_sum);
                }
            }
            __syncthreads();
            if (warp == 0) {
                // bins in descending key order, two per lane: the bin that takes the running count past k is T
                const unsigned long long above = sh.tot[kWarpBins];   // keys above the band
                uint32_t h[2], inc[2];
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const uint32_t pos = j * 32 + lane;
                    h[j] = (pos <= width) ? sh.tot[width - pos] : 0u;
                    inc[j] = h[j];
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const uint32_t y = __shfl_up_sync(kFullMask, inc[j], o);
                        if (lane >= o) inc[j] += y;
                    }
                }
                inc[1] += __shfl_sync(kFullMask, inc[0], 31);
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const uint32_t pos = j * 32 + lane;
                    const unsigned long long cum = above + (inc[j] - h[j]);
                    if (pos <= width && cum < k && k <= cum + h[j]) {
                        sh.T = lo + (width - pos);
                        sh.n_gt = cum;
                        sh.quota = k - cum;
                        sh.found = 1;
                    }
                }
            }
            __syncthreads();
            if (!sh.found) continue;   // T outside the band (uniform across the grid): widen and redo
            T = sh.T;
            q = (uint32_t)sh.quota;
            const uint32_t dT = T - lo;
            {
                // this warp's (#key > T, #key == T) and the same over the CTAs before this one
                uint32_t g = 0, pg = 0;
                for (uint32_t d = dT + 1 + lane; d <= width; d += 32) {
                    g += sh.whist[warp][d];
                    pg += sh.pre[d];
                }
                for (int o = 16; o > 0; o >>= 1) {
                    g += __shfl_xor_sync(kFullMask, g, o);
                    pg += __shfl_xor_sync(kFullMask, pg, o);
                }
                if (lane == 0) {
                    sh.wpre_gt[warp] = g + sh.w_hi[warp];
                    sh.wpre_eq[warp] = sh.whist[warp][dT];
                }
                __syncthreads();
                // exclusive scan over the CTA's warps (lane = warp index), done by every warp for itself
                const uint32_t og = (lane < kFusedWarps) ? sh.wpre_gt[lane] : 0u;
                const uint32_t oe = (lane < kFusedWarps) ? sh.wpre_eq[lane] : 0u;
                uint32_t gi = og, ei = oe;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t yg = __shfl_up_sync(kFullMask, gi, o), ye = __shfl_up_sync(kFullMask, ei, o);
                    if (lane >= o) { gi += yg; ei += ye; }
                }
                run_gt = pg + sh.pre[kWarpBins] + __shfl_sync(kFullMask, gi - og, warp);
                run_eq = sh.pre[dT] + __shfl_sync(kFullMask, ei - oe, warp);
            }
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
            if (!grid_barrier(&st->barrier, epoch, barrier_target, &sh.ok, spin_max)) {
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

    // ---------------- phase 3: ordered compaction, one warp per run of super-blocks ----------------
    // A lane owns 32 consecutive elements = one mask word, so a super-block costs one warp scan and the
    // mask needs no exchange.  Retained values are staged per warp at (final position - head) and leave
    // for global memory in aligned 16-byte pieces after every super-block; the < 8 that remain are
    // carried to the front of the buffer.
    ptx::launch_dependents();   // a programmatically launched kernel behind this one may be brought up
    unsigned long long departed_before = 0;   // see the end of the kernel
    if (barrier_target != 0 && threadIdx.x == 0) departed_before = atomicAdd(&st->barrier, 1ull << 20);
    const int64_t nwords = (n + 31) / 32;
    uint16_t* s_vals = s_vals_all + (size_t)warp * kStageVals;
    const uint32_t s_vals_addr = ptx_smem(s_vals);
    const uint32_t c_gt = ge_const(T + 1), c_ge = ge_const(T);
    uint32_t gpos = run_gt + min(run_eq, q);   // retained elements before this warp's next super-block
    uint32_t head = gpos & ~7u;                // first position not yet written to `values` (16-byte aligned)
    uint32_t foreign = gpos & 7u;              // leading slots of the first piece that belong to the previous warp
    issue_sb(sb0, 0);
    int slot = 0;
    auto compact_sb = [&](int64_t sb, auto full_tag) {
        constexpr bool FULL = decltype(full_tag)::value;
        issue_sb(sb + 1, slot ^ 1);
        sb_wait();
        __syncwarp();   // the lane reads vectors that other lanes copied
        const uint32_t own = ring_own + slot * kSbBytes;
        uint32_t g32 = 0, ge32 = 0;
        {
            uint32_t w[16];
            sb_read(own, rot, w);
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                uint32_t a[4], b[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t m = w[4 * g + i] & 0x7FFF7FFFu;
                    a[i] = m + c_gt;                       // bit 15 of a half: key > T
                    b[i] = m + c_ge;                       // bit 15 of a half: key >= T
                }
                g32 |= flags8(a[0], a[1], a[2], a[3]) << ((g ^ rot) << 3);
                ge32 |= flags8(b[0], b[1], b[2], b[3]) << ((g ^ rot) << 3);
            }
        }
        uint32_t e32 = ge32 & ~g32;   // key == T
        if constexpr (!FULL) e32 &= valid_mask32(sb * kSbElems + lane * 32, n);   // zero padding must not tie with T = 0
        const uint32_t cnt = __popc(g32) | (__popc(e32) << 16);
        // packed (gt | eq << 16) prefix over the lanes = over the super-block's elements
        uint32_t inc = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(kFullMask, inc, o);
            if (lane >= o) inc += y;
        }
        const uint32_t tot = __shfl_sync(kFullMask, inc, 31);
        const uint32_t excl = inc - cnt;
        const uint32_t eq_before = run_eq + (excl >> 16);
        uint32_t keep = g32;
        if (e32) {
            const uint32_t room = (eq_before < q) ? (q - eq_before) : 0u;
            uint32_t ke = e32;
            if (room < (cnt >> 16)) {   // the quota ends inside this lane's ties: the first `room` of them stay
                uint32_t m = e32;
                ke = 0;
                for (uint32_t r = 0; r < room; ++r) {
                    ke |= m & (0u - m);
                    m &= m - 1;
                }
            }
            keep |= ke;
        }
        const uint32_t pos = run_gt + (excl & 0xFFFFu) + min(eq_before, q);   // retained elements before this lane's first
        if ((lane & 3) == 0) {   // the lane opens a 128-element chunk
            if constexpr (FULL) {
                offsets[sb * kSbChunks + (lane >> 2)] = pos;
            } else {
                if (sb * kSbElems + lane * 32 < n) offsets[sb * kSbChunks + (lane >> 2)] = pos;
            }
        }
        if constexpr (!INDEX32) {
            const int64_t wi = sb * (kSbElems / 32) + lane;
            if constexpr (FULL) {
                mask[wi] = keep;
            } else {
                if (wi < nwords) mask[wi] = keep;
            }
        }
        {
            // the lane's retained elements, highest first: read from the ring, staged at their final position
            [[maybe_unused]] const int32_t first_idx = (int32_t)(sb * kSbElems) + lane * 32;
            uint32_t m = keep;
            uint32_t p_abs = pos + __popc(keep);
            while (m) {
                const uint32_t e = top_bit(m);
                m ^= 1u << e;
                --p_abs;
                const uint32_t v = lds_u16(own + 2u * e);
                asm volatile("st.shared.u16 [%0], %1;" ::"r"(s_vals_addr + 2u * (p_abs - head)), "r"(v) : "memory");
                if constexpr (INDEX32) indices[p_abs] = first_idx + (int32_t)e;
            }
        }
        run_gt += tot & 0xFFFFu;
        run_eq += tot >> 16;
        gpos = run_gt + min(run_eq, q);
        __syncwarp();   // staged values visible to the warp; every lane is done with the ring slot
        slot ^= 1;
        // write the whole 16-byte pieces, carry the rest to the front
        const uint32_t staged = gpos - head;
        const uint32_t pieces = staged / 8;
        if (pieces) {
            for (uint32_t c = lane; c < pieces; c += 32) {
                if (c == 0 && foreign) {
                    for (uint32_t e = foreign; e < 8; ++e) values[head + e] = s_vals[e];
                } else {
                    *reinterpret_cast<uint4*>(values + head + c * 8) = *reinterpret_cast<const uint4*>(s_vals + c * 8);
                }
            }
            foreign = 0;
            const uint32_t rem = staged - pieces * 8;
            uint16_t carry = 0;
            if (lane < (int)rem) carry = s_vals[pieces * 8 + lane];
            __syncwarp();
            if (lane < (int)rem) s_vals[lane] = carry;
            head += pieces * 8;
            __syncwarp();
        }
    };
    {
        int64_t sb = sb0;
        for (; sb < sb_full_end; ++sb) compact_sb(sb, std::true_type{});
        for (; sb < sb1; ++sb) compact_sb(sb, std::false_type{});
    }
    // the elements of the last, partial piece (the warp behind this one writes the rest of that piece)
    if (lane >= (int)foreign && head + lane < gpos) values[head + lane] = s_vals[lane];
    // Leave the barrier word stale.  A launch replayed from a captured graph carries the same epoch again; if the
    // word still held this epoch with all arrivals, a CTA that reached the first barrier before CTA 0 has
    // re-stamped the word would pass at once.  Every CTA that went through a barrier (the same ones in every CTA)
    // counts its departure in bits 20..31 of the word, which no wait looks at and which only grow the value; the
    // last one to leave stores zero, an epoch that no call carries.
    // (The count was taken at the start of this phase, behind the last barrier, so that its trip to L2 is not on
    // the kernel's tail.)
    if (barrier_target != 0 && threadIdx.x == 0 &&
        ((departed_before >> 20) & 0xFFFull) == (unsigned long long)gridDim.x - 1ull)
        asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(&st->barrier), "l"(0ull) : "memory");
}

// ---------------------------------------------------------------------------------------------
// Host side.
// ---------------------------------------------------------------------------------------------
dropit_status fused_compress_bf16_prepared(const void* x, int64_t n, int64_t k, bool index32, void* values, void* meta,
                                           uint32_t* offsets, void* workspace, size_t workspace_bytes,
                                           int32_t* dev_status, cudaStream_t stream, const unsigned char* prep) {
    const FusedPlan plan = make_fused_plan(n);
    if (workspace_bytes < plan.total_bytes) return DROPIT_ERR_WORKSPACE;
    unsigned char* ws = reinterpret_cast<unsigned char*>(workspace);
    static_assert(kRingBytes >= (size_t)kKeySpace * 4, "the sample's and the general path's histogram live in the ring's memory");
    const size_t smem_mask = kRingBytes + kStageBytes + sizeof(FusedShared);
    const size_t smem_idx = smem_mask;   // indices are written from registers, not staged
    static PerDeviceOnce attr;
    if (attr.needed()) {
        if (cudaFuncSetAttribute(fused_compress_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_mask) != cudaSuccess ||
            cudaFuncSetAttribute(fused_compress_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_idx) != cudaSuccess)
            return DROPIT_ERR_CUDA;
        attr.mark();
    }
    const uint4* xp = reinterpret_cast<const uint4*>(x);
    unsigned long long kk = (unsigned long long)k;
    int bpw = plan.blocks_per_warp;
    uint32_t epoch = next_epoch();
    if (epoch == 0) epoch = 1;   // zero marks a barrier word that a finished call left behind
    size_t h0 = plan.hist_off[0], h1 = plan.hist_off[1], ao = plan.agg_off, ro = plan.rows_off;
    uint16_t* vals = reinterpret_cast<uint16_t*>(values);
    uint32_t* maskp = index32 ? nullptr : reinterpret_cast<uint32_t*>(meta);
    int32_t* idxp = index32 ? reinterpret_cast<int32_t*>(meta) : nullptr;
    int spin_max = (int)spin_limit((uint32_t)kBarrierSpinLimit);
    void* args[] = {&xp, &n, &kk, &bpw, &epoch, &ws, &h0, &h1, &ao, &ro, &vals, &maskp, &idxp, &offsets, &dev_status, &spin_max,
                    &prep};
    const void* fn = index32 ? (const void*)fused_compress_kernel<true> : (const void*)fused_compress_kernel<false>;
    if (cudaLaunchCooperativeKernel(fn, dim3(plan.grid), dim3(kFusedThreads), args, index32 ? smem_idx : smem_mask,
                                    stream) != cudaSuccess) {
        cudaGetLastError();
        return DROPIT_ERR_CUDA;
    }
    return check_launch();
}

dropit_status fused_compress_bf16(const void* x, int64_t n, int64_t k, bool index32, void* values, void* meta,
                                  uint32_t* offsets, void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                  cudaStream_t stream) {
    return fused_compress_bf16_prepared(x, n, k, index32, values, meta, offsets, workspace, workspace_bytes, dev_status,
                                        stream, nullptr);
}

// ---------------------------------------------------------------------------------------------
// The producer in front of the path: y = act(x) for a bf16 tensor that is about to become a conv / fc input
// (Sec. 3.5: activations and normalisations keep their own caches; what they write is what DropIT compresses),
// with the selection statistics of y taken on the way.  One read of x, one write of y; the selection kernel
// then needs a single read of y.  Same work partition as fused_compress_kernel (a warp owns a run of
// 1024-element super-blocks), same sample, same band, same per-warp histograms.
// act: identity (y may be left out: statistics only), ReLU, or a table over all 65536 bf16 patterns
// (any element-wise function; GELU is built by dropit_activation_table).  The table's entries for
// 2^-9 <= |x| < 16 are kept in shared memory; the few elements outside that window read the table in
// global memory.
// ---------------------------------------------------------------------------------------------
constexpr int kActIdentity = 0, kActRelu = 1, kActTable = 2;
constexpr uint32_t kLutKeyLo = 118u << 7, kLutKeyHi = 131u << 7;   // keys of 2^-9 <= |x| < 2^4
constexpr uint32_t kLutSpan = kLutKeyHi - kLutKeyLo;                // 1664 keys per sign
constexpr size_t kLutBytes = 2 * kLutSpan * 2;

template <int ACT>
__device__ __forceinline__ uint32_t map_word(uint32_t w, uint32_t lut_addr, const uint16_t* __restrict__ table) {
    if constexpr (ACT == kActIdentity) {
        return w;
    } else if constexpr (ACT == kActRelu) {
        // max(x, 0): negative values and -0 become +0; NaN patterns (key > 0x7F80) pass
        const uint32_t neg = w & kHiBits;
        const uint32_t nan = ((w & 0x7FFF7FFFu) + 0x007F007Fu) & kHiBits;
        const uint32_t kill = ((neg & ~nan) >> 15) * 0xFFFFu;
        return w & ~kill;
    } else {
        const uint32_t i0 = (w & 0x7FFFu) - kLutKeyLo, i1 = ((w >> 16) & 0x7FFFu) - kLutKeyLo;
        uint32_t y0, y1;
        if (i0 < kLutSpan && i1 < kLutSpan) {
            asm volatile("ld.shared.u16 %0, [%1];" : "=r"(y0) : "r"(lut_addr + 2u * (((w >> 15) & 1u) * kLutSpan + i0)) : "memory");
            asm volatile("ld.shared.u16 %0, [%1];" : "=r"(y1) : "r"(lut_addr + 2u * ((w >> 31) * kLutSpan + i1)) : "memory");
        } else {
            y0 = __ldg(table + (w & 0xFFFFu));
            y1 = __ldg(table + (w >> 16));
        }
        return y0 | (y1 << 16);
    }
}

template <int ACT>
__global__ void __launch_bounds__(kFusedThreads, 1)
produce_kernel(const uint4* __restrict__ x, uint4* __restrict__ y, int64_t n, unsigned long long k, int blocks_per_warp,
               const uint16_t* __restrict__ table, unsigned char* prep) {
    extern __shared__ __align__(16) unsigned char fsm[];
    uint32_t* sample_bins = reinterpret_cast<uint32_t*>(fsm + kRingBytes);
    FusedShared& sh = *reinterpret_cast<FusedShared*>(fsm + kRingBytes + kStageBytes);
    const uint32_t lut_addr = ptx_smem(fsm + kRingBytes + kStageBytes + ((sizeof(FusedShared) + 15) / 16) * 16);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ring_warp = ptx_smem(fsm) + warp * (kRingSlots * kSbBytes);
    const uint32_t ring_copy = ring_warp + lane * 16;
    const uint32_t ring_own = ring_warp + lane * 64;
    const uint32_t rot = (uint32_t)(lane >> 1) & 3u;
    const int64_t nvec_full = n / 8;
    const int64_t blocks_total = (n + kBlkElems - 1) / kBlkElems;
    const int64_t blk0 = ((int64_t)blockIdx.x * kFusedWarps + warp) * blocks_per_warp;
    int64_t blk1 = blk0 + blocks_per_warp;
    if (blk1 > blocks_total) blk1 = blocks_total;
    const int64_t sb0 = blk0 / 2, sb1 = (blk1 + 1) / 2;
    const int64_t sb_full_end = (nvec_full / kSbVecs < sb1) ? nvec_full / kSbVecs : sb1;
    if constexpr (ACT == kActTable) {
        uint16_t* lut = reinterpret_cast<uint16_t*>(fsm + kRingBytes + kStageBytes + ((sizeof(FusedShared) + 15) / 16) * 16);
        for (uint32_t i = threadIdx.x; i < 2 * kLutSpan; i += blockDim.x)
            lut[i] = table[(i >= kLutSpan ? 0x8000u : 0u) | (kLutKeyLo + (i >= kLutSpan ? i - kLutSpan : i))];
        __syncthreads();
    }
    auto map_vec = [&](const uint4& v) {
        return make_uint4(map_word<ACT>(v.x, lut_addr, table), map_word<ACT>(v.y, lut_addr, table),
                          map_word<ACT>(v.z, lut_addr, table), map_word<ACT>(v.w, lut_addr, table));
    };
    // the same sample as the selection kernel takes, seen through act: every CTA arrives at the same band
    sample_band(x, n, k, sample_bins, sh.warp, sh.band, nullptr,
                [&] { if (sb0 < sb_full_end) sb_issue_full(ring_copy, x + sb0 * kSbVecs + lane); }, map_vec);
    const uint32_t lo = sh.band[0], hi = sh.band[1];
    const uint32_t width = hi - lo;
    const bool stats = n >= kSampleMinElems && width < (uint32_t)kWarpBins;   // uniform over the grid
    for (int i = threadIdx.x; i < kFusedWarps * kWarpBins; i += blockDim.x) (&sh.whist[0][0])[i] = 0;
    __syncthreads();
    uint32_t* hist = sh.whist[warp];
    const uint32_t c_hi = ge_const(hi + 1), c_lo = ge_const(lo);
    uint32_t cnt_hi = 0, cnt_lo = 0;
    // ---- whole super-blocks through the ring ----
    {
        int slot = 0;
        for (int64_t sb = sb0; sb < sb_full_end; ++sb) {
            if (sb + 1 < sb_full_end) sb_issue_full(ring_copy + (slot ^ 1) * kSbBytes, x + (sb + 1) * kSbVecs + lane);
            else asm volatile("cp.async.commit_group;" ::: "memory");
            sb_wait();
            __syncwarp();
            const uint32_t own = ring_own + slot * kSbBytes;
            uint32_t w[16];
            sb_read(own, rot, w);
#pragma unroll
            for (int i = 0; i < 16; ++i) w[i] = map_word<ACT>(w[i], lut_addr, table);
            if (y != nullptr) {
#pragma unroll
                for (int j = 0; j < 4; ++j)   // registers 4j.. hold the lane's vector j ^ rot
                    y[sb * kSbVecs + lane * 4 + (j ^ rot)] = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
            }
            if (stats) {
                if constexpr (ACT != kActIdentity) {   // the band walk below reads keys from the slot: they are y's now
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(own + ((j ^ rot) << 4)), "r"(w[4 * j]),
                                     "r"(w[4 * j + 1]), "r"(w[4 * j + 2]), "r"(w[4 * j + 3]) : "memory");
                }
                uint32_t hi_flags = 0, pending = 0;
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    uint32_t a[4], b[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t m = w[4 * g + i] & 0x7FFF7FFFu;
                        a[i] = m + c_hi;                   // bit 15 of a half: key > hi
                        b[i] = (m + c_lo) & ~a[i];         // bit 15 of a half: lo <= key <= hi
                    }
                    hi_flags |= ((__byte_perm(a[0], a[1], 0x7531) & 0x80808080u) >> (2 * g)) |
                                ((__byte_perm(a[2], a[3], 0x7531) & 0x80808080u) >> (2 * g + 1));
                    pending |= flags8(b[0], b[1], b[2], b[3]) << ((g ^ rot) << 3);
                }
                cnt_hi += __popc(hi_flags);
                while (pending) {
                    const uint32_t e = top_bit(pending);
                    pending ^= 1u << e;
                    const uint32_t d = (lds_u16(own + 2u * e) & 0x7FFFu) - lo;
                    if (d == 0) ++cnt_lo; else atomicAdd(&hist[d], 1u);
                }
            }
            __syncwarp();
            slot ^= 1;
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
    }
    // ---- the ragged last super-block of the tensor (at most one, in one warp): element by element ----
    for (int64_t sb = (sb_full_end > sb0 ? sb_full_end : sb0); sb < sb1; ++sb) {
        const uint16_t* xe = reinterpret_cast<const uint16_t*>(x);
        uint16_t* ye = reinterpret_cast<uint16_t*>(y);
        for (int i = 0; i < 32; ++i) {
            const int64_t e = sb * kSbElems + lane * 32 + i;
            if (e >= n) break;
            const uint32_t xv = xe[e];
            uint32_t yv;
            if constexpr (ACT == kActTable) yv = __ldg(table + xv);
            else yv = map_word<ACT>(xv, lut_addr, table) & 0xFFFFu;
            if (ye != nullptr) ye[e] = (uint16_t)yv;
            if (stats) {
                const uint32_t key = yv & 0x7FFFu;
                if (key > hi) ++cnt_hi;
                else if (key >= lo) {
                    if (key == lo) ++cnt_lo; else atomicAdd(&hist[key - lo], 1u);
                }
            }
        }
    }
    for (int o = 16; o > 0; o >>= 1) {
        cnt_lo += __shfl_xor_sync(kFullMask, cnt_lo, o);
        cnt_hi += __shfl_xor_sync(kFullMask, cnt_hi, o);
    }
    if (lane == 0) {
        if (cnt_lo) atomicAdd(&hist[0], cnt_lo);
        sh.w_hi[warp] = cnt_hi;
    }
    __syncthreads();
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        PrepHeader* ph = reinterpret_cast<PrepHeader*>(prep);
        ph->magic = kPrepMagic;
        ph->valid = stats ? 1u : 0u;
        ph->lo = lo;
        ph->hi = hi;
        ph->grid = gridDim.x;
        ph->blocks_per_warp = (uint32_t)blocks_per_warp;
        ph->n = (unsigned long long)n;
        ph->k = k;
    }
    if (!stats) return;
    uint32_t* rows = const_cast<uint32_t*>(prep_rows(prep));
    uint32_t* wh = const_cast<uint32_t*>(prep_warp_hist(prep, gridDim.x)) + (size_t)blockIdx.x * kFusedWarps * kPrepWarpWords;
    for (int i = threadIdx.x; i < kFusedWarps * kPrepWarpWords; i += blockDim.x) {
        const int w = i / kPrepWarpWords, c = i % kPrepWarpWords;
        wh[i] = c < kWarpBins ? sh.whist[w][c] : (c == kWarpBins ? sh.w_hi[w] : 0u);
    }
    if (threadIdx.x < kRowWords) {
        uint32_t v = 0;
        if (threadIdx.x < kWarpBins) {
            for (int w = 0; w < kFusedWarps; ++w) v += sh.whist[w][threadIdx.x];
        } else if (threadIdx.x == kWarpBins) {
            for (int w = 0; w < kFusedWarps; ++w) v += sh.w_hi[w];
        }
        rows[(size_t)blockIdx.x * kRowWords + threadIdx.x] = v;
    }
}

template <int ACT>
static dropit_status launch_produce(const void* x, void* y, int64_t n, int64_t k, const uint16_t* table, unsigned char* prep,
                                    cudaStream_t stream) {
    const FusedPlan plan = make_fused_plan(n);
    const size_t smem = kRingBytes + kStageBytes + ((sizeof(FusedShared) + 15) / 16) * 16 + kLutBytes;
    static PerDeviceOnce attr;
    if (attr.needed()) {
        if (cudaFuncSetAttribute(produce_kernel<ACT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return DROPIT_ERR_CUDA;
        attr.mark();
    }
    produce_kernel<ACT><<<plan.grid, kFusedThreads, smem, stream>>>(reinterpret_cast<const uint4*>(x),
                                                                    reinterpret_cast<uint4*>(y), n, (unsigned long long)k,
                                                                    plan.blocks_per_warp, table, prep);
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
    // nothing in the scratch has to be cleared first (see the grid barrier); the kernel zeroes its own totals
    return fused_compress_bf16(x, n, k, format == DROPIT_FMT_INDEX32, values, meta, offsets, scratch,
                               kStaticScratchBytes, dev_status, stream);
}


extern "C" dropit_status dropit_produce_workspace(int64_t n, size_t* prep_bytes) {
    if (n < 0 || n >= ((int64_t)1 << 31)) return DROPIT_ERR_INVALID_ARG;
    if (prep_bytes) *prep_bytes = dropit::prep_bytes_for(n);
    return DROPIT_OK;
}

extern "C" dropit_status dropit_produce(const void* x, int64_t n, double gamma, dropit_activation act, const uint16_t* table,
                                        void* y, void* prep, size_t prep_bytes, void* cuda_stream) {
    using namespace dropit;
    if (n < 0 || n >= ((int64_t)1 << 31) || !(gamma >= 0.0 && gamma <= 1.0)) return DROPIT_ERR_INVALID_ARG;
    if (act != DROPIT_ACT_IDENTITY && act != DROPIT_ACT_RELU && act != DROPIT_ACT_TABLE) return DROPIT_ERR_INVALID_ARG;
    if (n == 0) return DROPIT_OK;
    if (!x || !is_aligned16(x) || !prep || !is_aligned16(prep)) return DROPIT_ERR_INVALID_ARG;
    if (y && (!is_aligned16(y) || y == x)) return DROPIT_ERR_INVALID_ARG;       // not in place: every CTA samples x
    if (!y && act != DROPIT_ACT_IDENTITY) return DROPIT_ERR_INVALID_ARG;         // only the identity may leave y out
    if (act == DROPIT_ACT_TABLE && (!table || !is_aligned16(table))) return DROPIT_ERR_INVALID_ARG;
    if (prep_bytes < prep_bytes_for(n)) return DROPIT_ERR_WORKSPACE;
    const int64_t k = dropit_keep_count(n, gamma);
    cudaStream_t stream = as_stream(cuda_stream);
    unsigned char* pp = reinterpret_cast<unsigned char*>(prep);
    if (act == DROPIT_ACT_IDENTITY) return launch_produce<kActIdentity>(x, y, n, k, table, pp, stream);
    if (act == DROPIT_ACT_RELU) return launch_produce<kActRelu>(x, y, n, k, table, pp, stream);
    return launch_produce<kActTable>(x, y, n, k, table, pp, stream);
}

extern "C" dropit_status dropit_compress_prepared(const void* y, int64_t n, double gamma, dropit_format format,
                                                  void* values, void* meta, uint32_t* offsets, const void* prep,
                                                  size_t prep_bytes, void* workspace, size_t workspace_bytes,
                                                  int32_t* dev_status, void* cuda_stream) {
    using namespace dropit;
    if (n < 0 || n >= ((int64_t)1 << 31) || !(gamma >= 0.0 && gamma <= 1.0)) return DROPIT_ERR_INVALID_ARG;
    if (format != DROPIT_FMT_BITMASK && format != DROPIT_FMT_INDEX32) return DROPIT_ERR_INVALID_ARG;
    if (n == 0) return DROPIT_OK;
    if (!prep || !is_aligned16(prep)) return DROPIT_ERR_INVALID_ARG;
    if (prep_bytes < prep_bytes_for(n)) return DROPIT_ERR_WORKSPACE;
    const int64_t k = dropit_keep_count(n, gamma);
    if (k == 0)   // nothing retained: the ordinary entry point zero-fills mask and table
        return dropit_compress(y, n, gamma, DROPIT_BF16, format, values, meta, offsets, workspace, workspace_bytes,
                               dev_status, cuda_stream);
    if (!y || !offsets || !is_aligned16(y) || !is_aligned16(offsets)) return DROPIT_ERR_INVALID_ARG;
    if (!meta || !is_aligned16(meta) || !values || !is_aligned16(values)) return DROPIT_ERR_INVALID_ARG;
    if (!workspace || !is_aligned16(workspace)) return DROPIT_ERR_INVALID_ARG;
    return fused_compress_bf16_prepared(y, n, k, format == DROPIT_FMT_INDEX32, values, meta, offsets, workspace,
                                        workspace_bytes, dev_status, as_stream(cuda_stream),
                                        reinterpret_cast<const unsigned char*>(prep));
}
