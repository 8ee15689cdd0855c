// Fully-connected weight gradient straight from the bitmask cache (Eq. 6; Sec. 3.2 R(a-hat)):
// R(a-hat) is never written to global memory.  Per 64-token k-block the CTA needs, for its 256
// channels, 64 mask pieces of 32 bytes, 64 entries of the seek table and 64 short runs of packed
// values.  Those small, mutually dependent reads have a latency far above the time of one k-block,
// so they are prefetched k-blocks ahead into shared-memory rings with per-thread asynchronous copies
// (cp.async, completion counted on mbarriers):
//   warp 0  TMA producer: dY tile (A operand) of every stage
//   warp 1  MMA issuer (one thread), owns the TMEM allocation; every expanded B tile is multiplied
//           with two dY tiles (256 rows of Cz per CTA, two accumulators = all 512 TMEM columns)
//   warp 2  meta loader: mask pieces + table entries, up to 6 k-blocks ahead -> meta ring
//   warps 3, 20  value loaders (half the rows each): once the table entries of a k-block have
//           landed, the first 64 packed values of every row (from the 16-byte-aligned start) ->
//           value ring, eight 16-byte copies per row
//   warps 4..19  expanders: a lane owns one 16-byte piece (8 channels) of a row; it gathers its
//           retained values from the value ring, packs them with zeros and writes the piece of the
//           swizzled B stage with one 16-byte store, then the warp fences to the async proxy and
//           arrives on the stage's mbarrier.  (A row with more retained values in the tile than the
//           prefetched window reads the rest from global memory.)  Warps 4..7 drain TMEM.
// Waiting warps poll with one lane and back off, so that they do not crowd the shared-memory pipe.
#include "weight_grad_common.cuh"

namespace dropit {

namespace {

constexpr int kFStages = 3;                  // A/B pipeline stages
constexpr int kMetaSlots = 4;                // meta ring depth (k-blocks)
constexpr int kValSlots = 3;                 // value ring depth (k-blocks)
constexpr int kExpanders = 16;               // expander warps
constexpr int kTileRows = kBM * kFusedAcc;   // 256 rows of Cz per CTA: two 128 x 256 accumulators = all 512 TMEM columns
constexpr int kAFStageBytes = kTileRows * kBK * 2;   // A stage of the fused kernel
constexpr int kRowsPerExp = kBK / kExpanders;   // 4 rows of a k-block per expander warp
constexpr int kWinVals = 64;                 // packed values per row held in the value ring
constexpr int kValLoaders = 2;                // value loader warps: warp 3 and the last warp, half the rows each
constexpr int kFusedWgThreads = 32 * (4 + kExpanders + (kValLoaders - 1));
constexpr int kLastWarp = kFusedWgThreads / 32 - 1;

struct FusedCtl {
    uint64_t full[kFStages];
    uint64_t empty[kFStages];
    uint64_t meta_full[kMetaSlots];
    uint64_t meta_empty[kMetaSlots];
    uint64_t val_full[kValSlots];
    uint64_t val_empty[kValSlots];
    uint64_t accum;
    uint32_t tmem_base;
    int abort_flag;
    int is_last;
};

constexpr size_t kMaskRingBytes = (size_t)kMetaSlots * kBK * 32;
constexpr size_t kBaseRingBytes = (size_t)kMetaSlots * kBK * 4;
constexpr size_t kValRingBytes = (size_t)kValSlots * kBK * kWinVals * 2;
constexpr size_t kFusedSmemBytes = 1024 + (size_t)kFStages * (kAFStageBytes + kBStageBytes) + kMaskRingBytes +
                                   kBaseRingBytes + kValRingBytes + sizeof(FusedCtl);

static_assert(kFusedSmemBytes <= 232448, "dynamic shared memory of the fused kernel exceeds 227 KB");

// 16-byte copy; with src_bytes = 0 nothing is read and the destination is zero-filled.
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, uint32_t src_bytes = 16) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
// 4-byte copy; with src_bytes = 0 nothing is read and the destination is zero-filled.
__device__ __forceinline__ void cp_async_4(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
// Arrive on the mbarrier once every cp.async issued so far by this thread has landed.
__device__ __forceinline__ void cp_async_arrive(uint64_t* bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(ptx::smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Optional per-role cycle counters of CTA (0,0) (build with -DDROPIT_WG_TIMING): written as int64 behind
// the device status word (dev_status + 4 ...), so the status buffer must then hold at least 64 words.
#ifdef DROPIT_WG_TIMING
#define WG_CLK() clock64()
#define WG_ACC(var, t0) var += clock64() - (t0)
#define WG_DUMP(cond, slot, ...)                                                          \
    if (blockIdx.x == 0 && blockIdx.y == 0 && (cond) && dev_status) {                      \
        const long long v_[] = {__VA_ARGS__};                                             \
        long long* d_ = reinterpret_cast<long long*>(dev_status + 4) + (slot);            \
        for (int z_ = 0; z_ < (int)(sizeof(v_) / sizeof(v_[0])); ++z_) d_[z_] = v_[z_];   \
    }
#else
#define WG_CLK() 0ll
#define WG_ACC(var, t0) (void)(t0)
#define WG_DUMP(cond, slot, ...)
#endif

__global__ void __launch_bounds__(kFusedWgThreads, 1)
wg_fused_kernel(const __grid_constant__ CUtensorMap map_dy, const uint16_t* __restrict__ values,
                const uint32_t* __restrict__ mask, const uint32_t* __restrict__ offsets, unsigned long long k_total,
                int M, int Ca, int Cz, int tiles_n, int splits, int kb_per_split, int kb_total,
                float* __restrict__ dw, int accumulate, float* __restrict__ partial, uint32_t* counters,
                int32_t* dev_status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;
    uint8_t* sB = sA + kFStages * kAFStageBytes;
    uint32_t* s_mask = reinterpret_cast<uint32_t*>(sB + kFStages * kBStageBytes);     // [slot][row][8 words]
    uint32_t* s_base = reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(s_mask) + kMaskRingBytes);   // [slot][row]
    uint16_t* s_vals = reinterpret_cast<uint16_t*>(reinterpret_cast<uint8_t*>(s_base) + kBaseRingBytes);   // [slot][row][64]
    FusedCtl* ctl = reinterpret_cast<FusedCtl*>(reinterpret_cast<uint8_t*>(s_vals) + kValRingBytes);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int tile = blockIdx.x;
    const int split = blockIdx.y;
    const int j0 = (tile / tiles_n) * kTileRows;
    const int c0 = (tile % tiles_n) * kBN;
    const int kb_begin = split * kb_per_split;
    const int kb_end = min(kb_total, kb_begin + kb_per_split);
    const int nkb = kb_end - kb_begin;
    const bool second_half = (c0 + 128) < Ca;   // channels c0+128 .. c0+255 exist (Ca is a multiple of 128)

    if (threadIdx.x == 0) {
        for (int s = 0; s < kFStages; ++s) {
            ptx::mbar_init(&ctl->full[s], 1 + kExpanders);
            ptx::mbar_init(&ctl->empty[s], 1);
        }
        for (int s = 0; s < kMetaSlots; ++s) {
            ptx::mbar_init(&ctl->meta_full[s], 32);
            ptx::mbar_init(&ctl->meta_empty[s], kExpanders);
        }
        for (int s = 0; s < kValSlots; ++s) {
            ptx::mbar_init(&ctl->val_full[s], 32 * kValLoaders);
            ptx::mbar_init(&ctl->val_empty[s], kExpanders);
        }
        ptx::mbar_init(&ctl->accum, 1);
        ctl->abort_flag = 0;
        ctl->is_last = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&map_dy);
    }
    if (warp == 1) {
        ptx::tmem_alloc(&ctl->tmem_base, kBN * kFusedAcc);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    volatile int* abort_flag = &ctl->abort_flag;

    if (warp == 0) {
        // ---------------- TMA producer: dY tiles ----------------
        if (lane == 0) {
            int issued = 0;
            for (int i = 0; i < nkb && !*abort_flag; ++i) {
                const int s = i % kFStages;
                if (i >= kFStages && !ptx::mbar_wait(&ctl->empty[s], ((i / kFStages) - 1) & 1, kWaitLimit)) {
                    *abort_flag = 1;
                    break;
                }
                ptx::mbar_arrive_expect_tx(&ctl->full[s], kAFStageBytes);
                const int k0 = (kb_begin + i) * kBK;
                uint8_t* a = sA + s * kAFStageBytes;
#pragma unroll
                for (int g = 0; g < kTileRows / 64; ++g)
                    ptx::tma_load_2d(a + g * (64 * kBK * 2), &map_dy, j0 + 64 * g, k0, &ctl->full[s]);
                issued = i + 1;
            }
            if (*abort_flag) {   // let the copies already in flight land before the CTA exits
                for (int i = max(0, issued - kFStages); i < issued; ++i)
                    ptx::mbar_wait(&ctl->full[i % kFStages], (i / kFStages) & 1, kWaitLimit);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::make_idesc_bf16(kBM, kBN, true, true);
            constexpr uint32_t kGroupBytes = 64 * kBK * 2;
            bool ok = true;
            [[maybe_unused]] long long t_wait_full = 0;
            for (int i = 0; i < nkb; ++i) {
                const int s = i % kFStages;
                const long long c0_ = WG_CLK();
                if (*abort_flag || !ptx::mbar_wait(&ctl->full[s], (i / kFStages) & 1, kWaitLimit)) {
                    *abort_flag = 1;
                    ok = false;
                    break;
                }
                WG_ACC(t_wait_full, c0_);
                ptx::tc_fence_after();
                const uint32_t a_addr = ptx::smem_u32(sA + s * kAFStageBytes);
                const uint32_t b_addr = ptx::smem_u32(sB + s * kBStageBytes);
#pragma unroll
                for (int kk = 0; kk < kBK / 16; ++kk) {
                    const uint64_t bd = ptx::make_smem_desc_sw128(b_addr + kk * 2048, kGroupBytes, 1024);
#pragma unroll
                    for (int acc = 0; acc < kFusedAcc; ++acc) {   // the expanded B tile feeds both accumulators
                        const uint64_t ad =
                            ptx::make_smem_desc_sw128(a_addr + acc * kAStageBytes + kk * 2048, kGroupBytes, 1024);
                        ptx::umma_bf16(tmem_base + acc * kBN, ad, bd, idesc, (i > 0 || kk > 0) ? 1u : 0u);
                    }
                }
                ptx::umma_commit(&ctl->empty[s]);
            }
            if (ok) ptx::umma_commit(&ctl->accum);
            WG_DUMP(true, 9, t_wait_full);
        }
    }
    else if (warp == 2) {
        // ---------------- meta loader: mask pieces and table entries, two rows per lane ----------------
        for (int i = 0; i < nkb; ++i) {
            const int slot = i % kMetaSlots;
            if (i >= kMetaSlots) {
                const bool ok = ptx::mbar_wait_warp(&ctl->meta_empty[slot], ((i / kMetaSlots) - 1) & 1, kWaitLimit);
                if (!__all_sync(kFullMask, ok)) *abort_flag = 1;
            }
            if (*abort_flag) break;
            const int k0 = (kb_begin + i) * kBK;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int r = lane + 32 * h;
                const int n = k0 + r;
                uint32_t* m_dst = s_mask + ((size_t)slot * kBK + r) * 8;
                uint32_t* b_dst = s_base + (size_t)slot * kBK + r;
                // rows past the last token and channels past the last one are zero-filled by the copy itself
                const bool live = n < M;
                const long long f = live ? ((long long)n * Ca + c0) : 0;
                cp_async_16(ptx::smem_u32(m_dst), mask + (f >> 5), live ? 16u : 0u);
                cp_async_16(ptx::smem_u32(m_dst + 4), mask + (f >> 5) + (second_half ? 4 : 0),
                            (live && second_half) ? 16u : 0u);
                cp_async_4(ptx::smem_u32(b_dst), offsets + (f >> 7), live ? 4u : 0u);
            }
            cp_async_arrive(&ctl->meta_full[slot]);
        }
        cp_async_wait_all();
    } else if (warp == 3 || warp == kLastWarp) {
        // ---------------- value loaders: first 64 packed values of every row, half the rows each ----------------
        const int row_lo = (warp == 3) ? 0 : kBK / 2;
        [[maybe_unused]] long long t_wait_meta = 0, t_wait_slot = 0, t_issue = 0;
        for (int i = 0; i < nkb; ++i) {
            const int mslot = i % kMetaSlots, vslot = i % kValSlots;
            const long long c0_ = WG_CLK();
            bool ok = ptx::mbar_wait_warp(&ctl->meta_full[mslot], (i / kMetaSlots) & 1, kWaitLimit);
            WG_ACC(t_wait_meta, c0_);
            const long long c1_ = WG_CLK();
            if (ok && i >= kValSlots) ok = ptx::mbar_wait_warp(&ctl->val_empty[vslot], ((i / kValSlots) - 1) & 1, kWaitLimit);
            WG_ACC(t_wait_slot, c1_);
            if (!__all_sync(kFullMask, ok)) *abort_flag = 1;
            if (*abort_flag) break;
            const long long c2_ = WG_CLK();
            const uint32_t* bases = s_base + (size_t)mslot * kBK;
            const uint32_t dst0 = ptx::smem_u32(s_vals + (size_t)vslot * kBK * kWinVals) + 16 * (lane & 7);
#pragma unroll 4
            for (int r4 = 0; r4 < kBK / 2; r4 += 4) {   // 8 lanes x 16 bytes per row, 4 rows per instruction
                const int r = row_lo + r4 + (lane >> 3);
                const unsigned long long first = (unsigned long long)(bases[r] & ~7u) + 8u * (lane & 7);   // element index
                uint32_t nbytes = 0;
                if (first < k_total) nbytes = (k_total - first >= 8) ? 16u : (uint32_t)(k_total - first) * 2u;
                const uint16_t* src = nbytes ? (values + first) : values;
                cp_async_16(dst0 + r * (kWinVals * 2), src, nbytes);
            }
            cp_async_arrive(&ctl->val_full[vslot]);
            WG_ACC(t_issue, c2_);
        }
        WG_DUMP(lane == 0 && warp == 3, 6, t_wait_meta, t_wait_slot, t_issue);
        cp_async_wait_all();
    }
    else {
        // ---------------- expanders: mask + packed values -> swizzled B tile ----------------
        // A warp takes two token rows at a time; lane l owns, in each, the 16-byte piece that holds
        // channels c0 + 8l .. c0 + 8l + 7 (mask byte l of the row).  The row's 256 channels are two
        // aligned 128-element chunks of the flat tensor, so the retained count before lane l is the
        // first chunk's table entry plus the mask bits of the lanes before it (one packed warp scan
        // for both rows).  Every lane then gathers its up to 8 values from the row's value window
        // with independent 2-byte shared-memory loads (slot i reads position p + popc(mask below i)),
        // packs them with zeros and writes the whole piece with one 16-byte store: no zero-fill pass,
        // no per-element rounds, all lanes busy.
        const int ew = warp - 4;
        const int grp = lane >> 3, piece = lane & 7;
        [[maybe_unused]] long long t_wait_val = 0, t_wait_empty = 0, t_setup = 0, t_rounds = 0, t_tail = 0;
        for (int i = 0; i < nkb; ++i) {
            const int s = i % kFStages, mslot = i % kMetaSlots, vslot = i % kValSlots;
            const long long c0_ = WG_CLK();
            // the value loaders waited for the meta slot before they filled the value slot
            bool ok = ptx::mbar_wait_warp(&ctl->val_full[vslot], (i / kValSlots) & 1, kWaitLimit);
            WG_ACC(t_wait_val, c0_);
            const long long c1_ = WG_CLK();
            if (ok && i >= kFStages) ok = ptx::mbar_wait_warp(&ctl->empty[s], ((i / kFStages) - 1) & 1, kWaitLimit);
            WG_ACC(t_wait_empty, c1_);
            if (!__all_sync(kFullMask, ok)) *abort_flag = 1;
            if (*abort_flag) break;
            const long long c3_ = WG_CLK();
            // 32-bit shared-memory addresses and explicit ld.shared / st.shared keep the address
            // arithmetic short; all rows of the warp are in flight together
            const uint32_t b_stage = ptx::smem_u32(sB + s * kBStageBytes) + grp * (64 * kBK * 2);
            const uint32_t m_row = ptx::smem_u32(s_mask + ((size_t)mslot * kBK + ew * kRowsPerExp) * 8) + 4 * (lane >> 2);
            const uint32_t b_row = ptx::smem_u32(s_base + (size_t)mslot * kBK + ew * kRowsPerExp);
            const uint32_t v_row = ptx::smem_u32(s_vals + ((size_t)vslot * kBK + ew * kRowsPerExp) * kWinVals);
            uint32_t m[kRowsPerExp], bs[kRowsPerExp], p0[kRowsPerExp];
#pragma unroll
            for (int q = 0; q < kRowsPerExp; ++q) {
                uint32_t word;
                asm("ld.shared.u32 %0, [%1];" : "=r"(word) : "r"(m_row + q * 32));
                asm("ld.shared.u32 %0, [%1];" : "=r"(bs[q]) : "r"(b_row + q * 4));
                m[q] = (word >> (8 * (lane & 3))) & 0xFFu;
            }
#pragma unroll
            for (int q = 0; q < kRowsPerExp; q += 2) {   // two rows per prefix scan (counts in the halves of a word)
                const uint32_t cnt2 = __popc(m[q]) | (__popc(m[q + 1]) << 16);
                uint32_t inc = cnt2;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t y = __shfl_up_sync(kFullMask, inc, o);
                    if (lane >= o) inc += y;
                }
                const uint32_t excl2 = inc - cnt2;
                p0[q] = (bs[q] & 7u) + (excl2 & 0xFFFFu);   // index from the row's 16-byte-aligned start
                p0[q + 1] = (bs[q + 1] & 7u) + (excl2 >> 16);
            }
#pragma unroll
            for (int q = 0; q < kRowsPerExp; ++q) {
                const int r = ew * kRowsPerExp + q;
                const uint32_t win = v_row + q * (kWinVals * 2);
                uint32_t v[8];
                if (p0[q] + __popc(m[q]) <= (uint32_t)kWinVals) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const uint32_t idx = p0[q] + __popc(m[q] & ((1u << e) - 1u));
                        uint16_t t;
                        asm("ld.shared.u16 %0, [%1];" : "=h"(t) : "r"(win + 2 * (idx & (kWinVals - 1))));
                        v[e] = ((m[q] >> e) & 1u) ? (uint32_t)t : 0u;
                    }
                } else {   // a row with more retained values than the prefetched window (rare)
                    const uint16_t* g = values + (bs[q] & ~7u);
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const uint32_t idx = p0[q] + __popc(m[q] & ((1u << e) - 1u));
                        v[e] = 0u;
                        if ((m[q] >> e) & 1u) {
                            if (idx < (uint32_t)kWinVals) {
                                uint16_t t;
                                asm("ld.shared.u16 %0, [%1];" : "=h"(t) : "r"(win + 2 * idx));
                                v[e] = t;
                            } else {
                                v[e] = __ldg(g + idx);
                            }
                        }
                    }
                }
                const uint32_t dst = b_stage + r * 128 + ((piece ^ (r & 7)) << 4);
                asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(v[0] | (v[1] << 16)),
                             "r"(v[2] | (v[3] << 16)), "r"(v[4] | (v[5] << 16)), "r"(v[6] | (v[7] << 16)));
            }
            WG_ACC(t_rounds, c3_);
            const long long c4_ = WG_CLK();
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                ptx::mbar_arrive(&ctl->full[s]);
                ptx::mbar_arrive(&ctl->val_empty[vslot]);
                ptx::mbar_arrive(&ctl->meta_empty[mslot]);
            }
            WG_ACC(t_tail, c4_);
        }
        WG_DUMP(warp == 4 && lane == 0, 0, t_wait_val, t_wait_empty, t_setup, t_rounds, t_tail, (long long)nkb);
        if (warp < 8) {
            // ---------------- epilogue: TMEM -> global ----------------
            bool ok = ptx::mbar_wait_warp(&ctl->accum, 0, kWaitLimit);
            ok = __all_sync(kFullMask, ok) && !*abort_flag;
            if (!ok) {
                *abort_flag = 1;
            } else {
                ptx::tc_fence_after();
#pragma unroll 1
                for (int acc = 0; acc < kFusedAcc; ++acc)
                    epilogue_store_tile(tmem_base + acc * kBN, warp, lane, j0 + acc * kBM, c0, Ca, Cz, split, splits, dw,
                                        accumulate, partial);
            }
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kBN * kFusedAcc);
    }
    if (*abort_flag) {
        if (threadIdx.x == 0 && dev_status) atomicExch(dev_status, (int)DROPIT_ERR_TIMEOUT);
        return;
    }
    if (splits == 1) return;
    split_reduce_tile(tile, j0, c0, Ca, Cz, splits, dw, accumulate, partial, counters, &ctl->is_last, kTileRows);
}

}  // namespace

dropit_status launch_wg_fused(const void* dy, const void* values, const void* mask, const uint32_t* offsets, int64_t M,
                              int64_t Ca, int64_t Cz, int64_t k, int tiles_m, int tiles_n, int splits, int kb_per_split,
                              int kb_total, float* dw, int accumulate, float* partial, uint32_t* counters,
                              int32_t* dev_status, cudaStream_t stream) {
    CUtensorMap map_dy;
    if (!make_map_2d_bf16(&map_dy, dy, M, Cz)) return DROPIT_ERR_CUDA;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(wg_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFusedSmemBytes) !=
            cudaSuccess)
            return DROPIT_ERR_CUDA;
        attr_set = true;
    }
    dim3 grid(tiles_m * tiles_n, splits);
    wg_fused_kernel<<<grid, kFusedWgThreads, kFusedSmemBytes, stream>>>(
        map_dy, reinterpret_cast<const uint16_t*>(values), reinterpret_cast<const uint32_t*>(mask), offsets,
        (unsigned long long)k, (int)M, (int)Ca, (int)Cz, tiles_n, splits, kb_per_split, kb_total, dw, accumulate, partial,
        counters, dev_status);
    return check_launch();
}

}  // namespace dropit
