// Min-k selection and cache packing (Sec. 3.3 "Min-K Elements", Sec. 3.2 a-hat = {a_Xr, X_r},
// Sec. 4.1 top-k of |a| with proportion 1-gamma).
//
// A radix select over the unsigned key of |x| replaces the sort behind a top-k:
//   1. histogram of one key digit over the whole tensor (shared-memory bins, flushed to a
//      global histogram); the last block to arrive scans the bins from the top and fixes the
//      digit of the threshold key T.  bf16 keys are one 15-bit digit; fp32 keys take three
//      digits (11/10/10 bits), each pass counting only the keys that match the digits so far.
//   2. one ordered compaction pass: element i is retained iff key_i > T, or key_i == T and
//      fewer than q = k - #{key > T} equal keys precede it in flat-index order.  The number of
//      retained elements before i is then  gt_before(i) + min(eq_before(i), q), so a single
//      prefix sum over (gt, eq) counts places every value.  The prefix across tiles is a
//      decoupled look-back over 64-bit tile descriptors with a bounded wait.
#include <unistd.h>

#include <chrono>
#include <cstdlib>

#include "common.cuh"

namespace dropit {

uint32_t next_epoch() {
    static std::atomic<uint32_t> counter{[] {
        const uint64_t t = (uint64_t)std::chrono::steady_clock::now().time_since_epoch().count();
        uint64_t h = (t ^ ((uint64_t)getpid() << 32)) * 0x9E3779B97F4A7C15ull;
        return (uint32_t)(h >> 32);
    }()};
    return counter.fetch_add(1u, std::memory_order_relaxed);
}

uint32_t spin_limit(uint32_t default_limit) {
    const char* e = std::getenv("DROPIT_TEST_SPIN_LIMIT");
    if (!e || !*e) return default_limit;
    const long v = std::strtol(e, nullptr, 10);
    return v > 0 ? (uint32_t)v : default_limit;
}

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
        cached[dev] = v;
    }
    return cached[dev];
}

CompressPlan make_compress_plan(int64_t n, int64_t k, dropit_dtype dtype) {
    CompressPlan p{};
    p.n = n;
    p.k = k;
    const int vec = (dtype == DROPIT_BF16) ? 8 : 4;
    const int64_t tile_elems = (int64_t)kTileVecs * vec;
    p.n_tiles = (n + tile_elems - 1) / tile_elems;
    p.hist_offset = kStateBytes;
    p.hist_bytes = (dtype == DROPIT_BF16) ? (size_t)(1 << 15) * 4 : (size_t)(2048 + 1024 + 1024) * 4;
    p.desc_offset = align_up(p.hist_offset + p.hist_bytes, 256);
    p.desc_bytes = (size_t)p.n_tiles * 8;
    p.total_bytes = align_up(p.desc_offset + p.desc_bytes, 256);
    return p;
}

// ---------------------------------------------------------------------------------------------
// Pass 1: digit histogram + threshold digit (last block).
// ---------------------------------------------------------------------------------------------

template <typename Tr>
__device__ __forceinline__ void unpack_keys(const uint4& v, uint32_t (&key)[Tr::kVecElems]) {
    if constexpr (Tr::kVecElems == 8) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            key[2 * i] = w[i] & 0x7FFFu;
            key[2 * i + 1] = (w[i] >> 16) & 0x7FFFu;
        }
    } else {
        key[0] = v.x & 0x7FFFFFFFu;
        key[1] = v.y & 0x7FFFFFFFu;
        key[2] = v.z & 0x7FFFFFFFu;
        key[3] = v.w & 0x7FFFFFFFu;
    }
}

// BITS: digit width; SHIFT: position of the digit's lowest bit; FIRST: no higher digits to
// match; LAST: this digit completes the key.
template <typename Tr, int BITS, int SHIFT, int PASS, bool FIRST, bool LAST>
__global__ void __launch_bounds__(kHistThreads, 1)
hist_select_kernel(const uint4* __restrict__ x, int64_t n, unsigned long long k_total, SelectState* st,
                   uint32_t* __restrict__ ghist) {
    constexpr int NB = 1 << BITS;
    constexpr int G = Tr::kVecElems;
    extern __shared__ uint32_t bins[];
    __shared__ uint32_t s_warp[32];
    __shared__ uint32_t s_flag;

    for (int i = threadIdx.x; i < NB; i += blockDim.x) bins[i] = 0;
    const uint32_t prefix = FIRST ? 0u : st->prefix;
    __syncthreads();

    uint32_t zero_bin = 0;   // bin 0 is counted in a register: post-ReLU tensors are half zeros
    auto count_key = [&](uint32_t key) {
        if (!FIRST && (key >> (SHIFT + BITS)) != prefix) return;
        const uint32_t b = (key >> SHIFT) & (NB - 1);
        if (b == 0) ++zero_bin;
        else atomicAdd(&bins[b], 1u);
    };

    const int64_t nvec = n / G;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + 3 * stride < nvec; i += 4 * stride) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = ld_stream(x + i + u * stride);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            uint32_t key[G];
            unpack_keys<Tr>(v[u], key);
#pragma unroll
            for (int e = 0; e < G; ++e) count_key(key[e]);
        }
    }
    for (; i < nvec; i += stride) {
        uint32_t key[G];
        unpack_keys<Tr>(ld_stream(x + i), key);
#pragma unroll
        for (int e = 0; e < G; ++e) count_key(key[e]);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {   // ragged tail, fewer than G elements
        const typename Tr::elem_t* xe = reinterpret_cast<const typename Tr::elem_t*>(x);
        for (int64_t e = nvec * G; e < n; ++e) {
            uint32_t key = (uint32_t)xe[e] & ((Tr::kKeyBits == 15) ? 0x7FFFu : 0x7FFFFFFFu);
            count_key(key);
        }
    }

    // bin 0: warp reduce, one shared atomic per warp
    for (int o = 16; o > 0; o >>= 1) zero_bin += __shfl_xor_sync(kFullMask, zero_bin, o);
    if (lane_id() == 0 && zero_bin) atomicAdd(&bins[0], zero_bin);
    __syncthreads();

    for (int b = threadIdx.x; b < NB; b += blockDim.x) {
        const uint32_t c = bins[b];
        if (c) atomicAdd(&ghist[b], c);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_flag = (atomicAdd(&st->blocks_done[PASS], 1u) == gridDim.x - 1) ? 1u : 0u;
    __syncthreads();
    if (!s_flag) return;
    __threadfence();

    // ---- last block: scan the bins from the highest key down ----
    constexpr int PER = NB / kHistThreads;   // bins per thread (32 for bf16, 2 or 1 for fp32 digits)
    static_assert(PER >= 1, "digit too narrow for the block");
    const unsigned long long k_in = FIRST ? k_total : st->k_rem;
    const int t = threadIdx.x;
    uint32_t h[PER];
    uint32_t sum = 0;
#pragma unroll
    for (int r = 0; r < PER; ++r) {   // r-th bin of this thread in DESCENDING key order
        const int b = NB - 1 - (t * PER + r);
        h[r] = __ldcg(&ghist[b]);
        sum += h[r];
    }
    // exclusive scan of `sum` over threads
    uint32_t inc = sum;
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t y = __shfl_up_sync(kFullMask, inc, o);
        if (lane_id() >= (uint32_t)o) inc += y;
    }
    if (lane_id() == 31) s_warp[t >> 5] = inc;
    __syncthreads();
    if (t < 32) {
        uint32_t w = s_warp[t];
        uint32_t wi = w;
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t y = __shfl_up_sync(kFullMask, wi, o);
            if (t >= o) wi += y;
        }
        s_warp[t] = wi - w;   // exclusive
    }
    __syncthreads();
    const unsigned long long excl = (unsigned long long)s_warp[t >> 5] + (inc - sum);
    if (excl < k_in && k_in <= excl + sum) {
        unsigned long long cum = excl;
#pragma unroll
        for (int r = 0; r < PER; ++r) {
            if (cum < k_in && k_in <= cum + h[r]) {
                const uint32_t b = NB - 1 - (t * PER + r);
                const uint32_t np = FIRST ? b : ((prefix << BITS) | b);
                st->prefix = np;
                st->k_rem = k_in - cum;
                if (LAST) {
                    st->threshold = np;
                    st->quota = k_in - cum;
                    st->n_gt = k_total - (k_in - cum);
                }
            }
            cum += h[r];
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Pass 2: ordered compaction.
// ---------------------------------------------------------------------------------------------

__device__ __forceinline__ unsigned long long desc_pack(uint32_t status, uint32_t gt, uint32_t eq) {
    return ((unsigned long long)status << 62) | ((unsigned long long)eq << 31) | (unsigned long long)gt;
}
__device__ __forceinline__ uint32_t desc_status(unsigned long long d) { return (uint32_t)(d >> 62); }
__device__ __forceinline__ uint32_t desc_gt(unsigned long long d) { return (uint32_t)(d & 0x7FFFFFFFull); }
__device__ __forceinline__ uint32_t desc_eq(unsigned long long d) { return (uint32_t)((d >> 31) & 0x7FFFFFFFull); }

template <typename Tr, bool INDEX32>
__global__ void __launch_bounds__(kCompactThreads)
compact_kernel(const uint4* __restrict__ x, int64_t n, SelectState* st, unsigned long long* desc,
               typename Tr::elem_t* __restrict__ values, uint32_t* __restrict__ mask, int32_t* __restrict__ indices,
               uint32_t* __restrict__ offsets, int32_t* dev_status) {
    using elem_t = typename Tr::elem_t;
    constexpr int G = Tr::kVecElems;
    constexpr int VPT = kCompactVecsPerThread;
    constexpr int TILE_ELEMS = kTileVecs * G;
    constexpr int A = 16 / Tr::kElemBytes;            // elements per 16-byte store
    constexpr int LANES_PER_WORD = 32 / G;            // lanes that share one mask word
    constexpr int WORDS_PER_WARP = VPT * G;           // mask words produced by one warp
    constexpr int NWARPS = kCompactThreads / 32;

    extern __shared__ __align__(16) unsigned char smem_raw[];
    elem_t* s_vals = reinterpret_cast<elem_t*>(smem_raw);                       // TILE_ELEMS + A
    int32_t* s_idx = reinterpret_cast<int32_t*>(smem_raw + (size_t)(TILE_ELEMS + A) * Tr::kElemBytes);  // TILE_ELEMS + 4
    __shared__ uint32_t s_warp_tot[NWARPS];
    __shared__ uint32_t s_tile;
    __shared__ uint32_t s_ex[2];
    __shared__ int s_timeout;

    if (threadIdx.x == 0) {
        s_tile = atomicAdd(&st->ticket, 1u);
        s_timeout = 0;
    }
    __syncthreads();
    const uint32_t tile = s_tile;
    const uint32_t T = st->threshold;
    const unsigned long long q64 = st->quota;
    const uint32_t q = (uint32_t)q64;
    const int warp = threadIdx.x >> 5;
    const int lane = lane_id();

    const int64_t nvec_full = n / G;
    const int64_t vec0 = (int64_t)tile * kTileVecs + warp * (32 * VPT);

    // ---- load, key, flag ----
    uint4 v[VPT];
    uint32_t gtm[VPT], eqm[VPT], cnt[VPT];
#pragma unroll
    for (int j = 0; j < VPT; ++j) {
        const int64_t vi = vec0 + j * 32 + lane;
        int nvalid = G;
        if (vi < nvec_full) {
            v[j] = ld_stream(x + vi);
        } else {
            v[j] = make_uint4(0, 0, 0, 0);
            nvalid = 0;
            if (vi == nvec_full && (n % G) != 0) {   // ragged last vector: scalar loads
                nvalid = (int)(n - nvec_full * G);
                const elem_t* xe = reinterpret_cast<const elem_t*>(x) + vi * G;
                uint32_t w[4] = {0, 0, 0, 0};
                for (int e = 0; e < nvalid; ++e) {
                    if constexpr (G == 8) w[e >> 1] |= (uint32_t)xe[e] << ((e & 1) * 16);
                    else w[e] = xe[e];
                }
                v[j] = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
        uint32_t key[G];
        unpack_keys<Tr>(v[j], key);
        uint32_t g = 0, e_ = 0;
#pragma unroll
        for (int e = 0; e < G; ++e) {
            g |= (uint32_t)(key[e] > T) << e;
            e_ |= (uint32_t)(key[e] == T) << e;
        }
        const uint32_t valid = (nvalid >= G) ? ((1u << G) - 1) : ((1u << nvalid) - 1);
        gtm[j] = g & valid;
        eqm[j] = e_ & valid;
        cnt[j] = __popc(gtm[j]) | (__popc(eqm[j]) << 16);
    }

    // ---- packed (gt | eq<<16) prefix inside the warp, in (j, lane) order ----
    uint32_t excl[VPT];
    uint32_t row_base = 0;
#pragma unroll
    for (int j = 0; j < VPT; ++j) {
        uint32_t inc = cnt[j];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t y = __shfl_up_sync(kFullMask, inc, o);
            if (lane >= o) inc += y;
        }
        excl[j] = row_base + inc - cnt[j];
        row_base += __shfl_sync(kFullMask, inc, 31);
    }
    if (lane == 0) s_warp_tot[warp] = row_base;
    __syncthreads();
    uint32_t warp_prefix = 0, tile_tot = 0;
#pragma unroll
    for (int w = 0; w < NWARPS; ++w) {
        const uint32_t t_ = s_warp_tot[w];
        if (w < warp) warp_prefix += t_;
        tile_tot += t_;
    }
    const uint32_t agg_gt = tile_tot & 0xFFFFu, agg_eq = tile_tot >> 16;

    // ---- decoupled look-back across tiles (warp 0) ----
    if (warp == 0) {
        if (lane == 0) st_relaxed_u64(&desc[tile], desc_pack(tile == 0 ? 2u : 1u, agg_gt, agg_eq));
        uint32_t ex_gt = 0, ex_eq = 0;
        if (tile > 0) {
            int64_t look = (int64_t)tile - 1;
            int spins = 0;
            bool timed_out = false;
            while (true) {
                const int64_t idx = look - lane;
                const unsigned long long d = (idx >= 0) ? ld_relaxed_u64(&desc[idx]) : desc_pack(2u, 0, 0);
                const uint32_t status = desc_status(d);
                const uint32_t invalid = __ballot_sync(kFullMask, status == 0);
                const uint32_t has_pref = __ballot_sync(kFullMask, status == 2);
                const int first_pref = has_pref ? (__ffs(has_pref) - 1) : 32;
                const uint32_t need = (first_pref >= 31) ? kFullMask : ((1u << (first_pref + 1)) - 1);
                if (invalid & need) {
                    if (++spins > kSpinLimit) { timed_out = true; break; }
                    __nanosleep(40);
                    continue;
                }
                const bool take = lane <= first_pref;
                uint32_t g = take ? desc_gt(d) : 0u, e = take ? desc_eq(d) : 0u;
                for (int o = 16; o > 0; o >>= 1) {
                    g += __shfl_xor_sync(kFullMask, g, o);
                    e += __shfl_xor_sync(kFullMask, e, o);
                }
                ex_gt += g;
                ex_eq += e;
                if (first_pref < 32) break;
                look -= 32;
            }
            if (lane == 0) {
                // publish even after a timeout so that later tiles do not wait on this one
                st_relaxed_u64(&desc[tile], desc_pack(2u, (ex_gt + agg_gt) & 0x7FFFFFFFu, (ex_eq + agg_eq) & 0x7FFFFFFFu));
                if (timed_out) {
                    s_timeout = 1;
                    if (dev_status) atomicExch(dev_status, (int)DROPIT_ERR_TIMEOUT);
                }
            }
        }
        if (lane == 0) {
            s_ex[0] = ex_gt;
            s_ex[1] = ex_eq;
        }
    }
    __syncthreads();
    if (s_timeout) return;   // outputs undefined, status word set
    const uint32_t tile_gt = s_ex[0], tile_eq = s_ex[1];
    const uint32_t tile_kept_base = tile_gt + min(tile_eq, q);
    const int mis = (int)(tile_kept_base % A);

    // ---- place values; build mask bits ----
    uint32_t keepm[VPT];
#pragma unroll
    for (int j = 0; j < VPT; ++j) {
        const uint32_t p = warp_prefix + excl[j];
        const uint32_t gt_before = tile_gt + (p & 0xFFFFu);
        const uint32_t eq_before = tile_eq + (p >> 16);
        const uint32_t room = (eq_before < q) ? (q - eq_before) : 0u;
        uint32_t keep_eq;
        const uint32_t ne = cnt[j] >> 16;
        if (room >= ne) keep_eq = eqm[j];
        else {
            keep_eq = 0;
            uint32_t m = eqm[j];
            for (uint32_t r = 0; r < room; ++r) {
                keep_eq |= m & (0u - m);
                m &= m - 1;
            }
        }
        keepm[j] = gtm[j] | keep_eq;
        const uint32_t kept_before = gt_before + min(eq_before, q);
        const int64_t vi = vec0 + j * 32 + lane;
        if constexpr (G == 8) {
            if ((lane & 15) == 0 && vi * G < n) offsets[(vi * G) / DROPIT_CHUNK] = kept_before;
        } else {
            if (lane == 0 && vi * G < n) offsets[(vi * G) / DROPIT_CHUNK] = kept_before;
        }
        uint32_t pos = kept_before - tile_kept_base + mis;
        const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
        for (int e = 0; e < G; ++e) {
            if ((keepm[j] >> e) & 1u) {
                elem_t val;
                if constexpr (G == 8) val = (elem_t)((w[e >> 1] >> ((e & 1) * 16)) & 0xFFFFu);
                else val = w[e];
                s_vals[pos] = val;
                if constexpr (INDEX32) s_idx[pos - mis + (tile_kept_base & 3u)] = (int32_t)(vi * G + e);
                ++pos;
            }
        }
    }

    if constexpr (!INDEX32) {
        // lanes that share a word OR their bit groups together, then lane i takes word i of the warp
        uint32_t word[VPT];
#pragma unroll
        for (int j = 0; j < VPT; ++j) {
            uint32_t wv = keepm[j] << (G * (lane % LANES_PER_WORD));
#pragma unroll
            for (int o = 1; o < LANES_PER_WORD; o <<= 1) wv |= __shfl_xor_sync(kFullMask, wv, o);
            word[j] = wv;
        }
        uint32_t mine = 0;
        const int src = (lane % G) * LANES_PER_WORD;
#pragma unroll
        for (int j = 0; j < VPT; ++j) {
            const uint32_t got = __shfl_sync(kFullMask, word[j], src);
            if (lane / G == j) mine = got;
        }
        const int64_t nwords = (n + 31) / 32;
        const int64_t w0 = (int64_t)tile * (TILE_ELEMS / 32) + warp * WORDS_PER_WARP;
        if (lane < WORDS_PER_WARP && w0 + lane < nwords) mask[w0 + lane] = mine;
    }
    __syncthreads();

    // ---- coalesced write of the tile's retained values (and indices) ----
    const uint32_t total = (tile_gt + agg_gt + min(tile_eq + agg_eq, q)) - tile_kept_base;
    {
        const uint32_t end = mis + total;
        const uint32_t fv = mis ? 1u : 0u, lv = end / A;
        elem_t* gbase = values + (tile_kept_base - mis);   // 16-byte aligned
        const uint32_t head_end = min(fv * A, end);
        for (uint32_t s = mis + threadIdx.x; s < head_end; s += blockDim.x) gbase[s] = s_vals[s];
        for (uint32_t sv = fv + threadIdx.x; sv < lv; sv += blockDim.x)
            reinterpret_cast<uint4*>(gbase)[sv] = reinterpret_cast<const uint4*>(s_vals)[sv];
        const uint32_t tail0 = max(lv, fv) * A;
        for (uint32_t s = tail0 + threadIdx.x; s < end; s += blockDim.x) gbase[s] = s_vals[s];
    }
    if constexpr (INDEX32) {
        const uint32_t mi = tile_kept_base & 3u;
        const uint32_t end = mi + total;
        const uint32_t fv = mi ? 1u : 0u, lv = end / 4;
        int32_t* gbase = indices + (tile_kept_base - mi);
        const uint32_t head_end = min(fv * 4, end);
        for (uint32_t s = mi + threadIdx.x; s < head_end; s += blockDim.x) gbase[s] = s_idx[s];
        for (uint32_t sv = fv + threadIdx.x; sv < lv; sv += blockDim.x)
            reinterpret_cast<uint4*>(gbase)[sv] = reinterpret_cast<const uint4*>(s_idx)[sv];
        const uint32_t tail0 = max(lv, fv) * 4;
        for (uint32_t s = tail0 + threadIdx.x; s < end; s += blockDim.x) gbase[s] = s_idx[s];
    }
}

// ---------------------------------------------------------------------------------------------
// Host side.
// ---------------------------------------------------------------------------------------------

template <typename Tr, int BITS, int SHIFT, int PASS, bool FIRST, bool LAST>
static dropit_status launch_hist(const void* x, int64_t n, int64_t k, SelectState* st, uint32_t* ghist,
                                 cudaStream_t stream) {
    auto kern = hist_select_kernel<Tr, BITS, SHIFT, PASS, FIRST, LAST>;
    const size_t smem = (size_t)(1 << BITS) * 4;
    static PerDeviceOnce attr;   // per instantiation
    if (smem > 48 * 1024 && attr.needed()) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return DROPIT_ERR_CUDA;
        attr.mark();
    }
    const int64_t nvec = n / Tr::kVecElems;
    int64_t blocks = (nvec + (int64_t)kHistThreads * 4 - 1) / ((int64_t)kHistThreads * 4);
    const int64_t cap = (int64_t)sm_count() * ((smem > 100 * 1024) ? 1 : 2);
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    kern<<<(unsigned)blocks, kHistThreads, smem, stream>>>(reinterpret_cast<const uint4*>(x), n,
                                                          (unsigned long long)k, st, ghist);
    return check_launch();
}

template <typename Tr, bool INDEX32>
static dropit_status launch_compact(const void* x, const CompressPlan& plan, SelectState* st, unsigned long long* desc,
                                    void* values, void* meta, uint32_t* offsets, int32_t* dev_status,
                                    cudaStream_t stream) {
    auto kern = compact_kernel<Tr, INDEX32>;
    constexpr int TILE_ELEMS = kTileVecs * Tr::kVecElems;
    constexpr int A = 16 / Tr::kElemBytes;
    size_t smem = (size_t)(TILE_ELEMS + A) * Tr::kElemBytes;
    if (INDEX32) smem += (size_t)(TILE_ELEMS + 4) * 4;
    static PerDeviceOnce attr;
    if (smem > 48 * 1024 && attr.needed()) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return DROPIT_ERR_CUDA;
        attr.mark();
    }
    kern<<<(unsigned)plan.n_tiles, kCompactThreads, smem, stream>>>(
        reinterpret_cast<const uint4*>(x), plan.n, st, desc, reinterpret_cast<typename Tr::elem_t*>(values),
        INDEX32 ? nullptr : reinterpret_cast<uint32_t*>(meta), INDEX32 ? reinterpret_cast<int32_t*>(meta) : nullptr,
        offsets, dev_status);
    return check_launch();
}

}  // namespace dropit

namespace dropit {
size_t fused_compress_workspace_bytes(int64_t n);
dropit_status fused_compress_bf16(const void* x, int64_t n, int64_t k, bool index32, void* values, void* meta,
                                  uint32_t* offsets, void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                  cudaStream_t stream);
}  // namespace dropit

using namespace dropit;

extern "C" int64_t dropit_keep_count(int64_t n, double gamma) {
    if (n < 0 || !(gamma >= 0.0 && gamma <= 1.0)) return -1;
    double d = ceil(gamma * (double)n - 1e-6);
    if (d < 0.0) d = 0.0;
    if (d > (double)n) d = (double)n;
    return n - (int64_t)d;
}

extern "C" dropit_status dropit_cache_sizes(int64_t n, double gamma, dropit_dtype dtype, dropit_format format,
                                            size_t* values_bytes, size_t* meta_bytes, size_t* offsets_bytes,
                                            size_t* workspace_bytes) {
    if (n < 0 || n >= ((int64_t)1 << 31) || !(gamma >= 0.0 && gamma <= 1.0)) return DROPIT_ERR_INVALID_ARG;
    if ((dtype != DROPIT_BF16 && dtype != DROPIT_F32) || (format != DROPIT_FMT_BITMASK && format != DROPIT_FMT_INDEX32))
        return DROPIT_ERR_INVALID_ARG;
    const int64_t k = dropit_keep_count(n, gamma);
    const size_t es = (dtype == DROPIT_BF16) ? 2 : 4;
    if (values_bytes) *values_bytes = (size_t)k * es;
    if (meta_bytes) *meta_bytes = (format == DROPIT_FMT_BITMASK) ? (size_t)((n + 31) / 32) * 4 : (size_t)k * 4;
    if (offsets_bytes) *offsets_bytes = (size_t)((n + DROPIT_CHUNK - 1) / DROPIT_CHUNK) * 4;
    if (workspace_bytes)
        *workspace_bytes = (dtype == DROPIT_BF16) ? fused_compress_workspace_bytes(n) : make_compress_plan(n, k, dtype).total_bytes;
    return DROPIT_OK;
}

extern "C" dropit_status dropit_compress(const void* x, int64_t n, double gamma, dropit_dtype dtype,
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
    const size_t off_bytes = (size_t)((n + DROPIT_CHUNK - 1) / DROPIT_CHUNK) * 4;
    if (k == 0) {   // gamma = 1: nothing retained
        if (format == DROPIT_FMT_BITMASK &&
            cudaMemsetAsync(meta, 0, (size_t)((n + 31) / 32) * 4, stream) != cudaSuccess)
            return DROPIT_ERR_CUDA;
        if (cudaMemsetAsync(offsets, 0, off_bytes, stream) != cudaSuccess) return DROPIT_ERR_CUDA;
        return DROPIT_OK;
    }
    if (!workspace || !is_aligned16(workspace)) return DROPIT_ERR_INVALID_ARG;
    if (dtype == DROPIT_BF16)
        return fused_compress_bf16(x, n, k, format == DROPIT_FMT_INDEX32, values, meta, offsets, workspace,
                                   workspace_bytes, dev_status, stream);
    const CompressPlan plan = make_compress_plan(n, k, dtype);
    if (workspace_bytes < plan.total_bytes) return DROPIT_ERR_WORKSPACE;

    unsigned char* ws = reinterpret_cast<unsigned char*>(workspace);
    SelectState* st = reinterpret_cast<SelectState*>(ws);
    uint32_t* hist = reinterpret_cast<uint32_t*>(ws + plan.hist_offset);
    unsigned long long* desc = reinterpret_cast<unsigned long long*>(ws + plan.desc_offset);
    if (cudaMemsetAsync(ws, 0, plan.total_bytes, stream) != cudaSuccess) return DROPIT_ERR_CUDA;

    dropit_status s = launch_hist<F32Traits, 11, 20, 0, true, false>(x, n, k, st, hist, stream);
    if (s != DROPIT_OK) return s;
    s = launch_hist<F32Traits, 10, 10, 1, false, false>(x, n, k, st, hist + 2048, stream);
    if (s != DROPIT_OK) return s;
    s = launch_hist<F32Traits, 10, 0, 2, false, true>(x, n, k, st, hist + 2048 + 1024, stream);
    if (s != DROPIT_OK) return s;
    if (format == DROPIT_FMT_BITMASK)
        return launch_compact<F32Traits, false>(x, plan, st, desc, values, meta, offsets, dev_status, stream);
    return launch_compact<F32Traits, true>(x, plan, st, desc, values, meta, offsets, dev_status, stream);
}
