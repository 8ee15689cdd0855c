// Fully-connected weight gradient straight from the bitmask cache (Eq. 6; Sec. 3.2: R(a-hat) is a temporary):
//   dW[j, c] = sum_n dY[n, j] * R(a-hat)[n, c]
// R(a-hat) is never written to global memory, and not to shared memory as an MMA operand either: it is
// rebuilt, 32 tokens x 32 channels at a time, in registers and stored into TENSOR MEMORY, from where the
// tensor cores read it as their A operand.
//
// Tile of a CTA: 128 channels c (the M rows = the 128 TMEM lanes) x 256 outputs j (N), reduction over tokens.
//   A[c][n] = R(a-hat)[n, c]   K-major in TMEM: lane = channel, a 32-bit column = two consecutive tokens
//   B[n][j] = dY[n, j]          row-major in global memory, i.e. N-major, 128-byte-swizzled stages filled by TMA
//   D[c][j] in TMEM (256 fp32 columns); the epilogue writes it transposed: a warp's 32 lanes are 32 consecutive
//   c, so each of its stores is one 128-byte row segment of dW.
// Per k-block of 64 tokens the CTA needs, for its 128 channels (exactly one 128-element chunk of every token
// row): 64 mask pieces of 16 bytes, 64 seek-table entries and 64 short runs of packed values.  Roles:
//   warp 0   TMA producer: dY stages
//   warp 1   MMA issuer (one thread); owns the TMEM allocation (256 accumulator columns + 4 x 32 operand columns)
//   warp 2   meta loader: mask pieces + table entries, k-blocks ahead, by cp.async -> meta ring
//   (warp 3  idle)
//   warps 4..19  expanders.  A unit is 32 tokens x 32 channels (one mask word per token) and a small image
//            [channel][token] in shared memory.  Lane t owns token t: two of its own k-blocks ahead it reads the
//            token's mask words and table entry, works out where the token's values for these 32 channels
//            lie in `values` (they are consecutive) and requests the one or two 16-byte pieces that hold them,
//            into registers.  When the unit's turn comes the lane parks the pieces in a private slot of shared
//            memory and walks the set bits of its word (work proportional to what is retained), dropping each
//            value into column t of its channel's row.  Then lane c reads row c back as 16 packed registers
//            (two tokens per register) and one tcgen05.st puts them into lane c of tensor memory.  Warps 4..7
//            also drain the accumulator at the end.
// Splits of the token axis (2 or 4) form a thread-block cluster and add up through distributed shared
// memory, always in split order.
#include "weight_grad_common.cuh"

namespace dropit {

namespace {

constexpr int kTmStages = 4;                  // dY (B operand) stages of 32 KB
constexpr int kTmAStages = 4;                 // operand stages in tensor memory (32 columns each)
constexpr int kTmMetaSlots = 8;               // meta ring depth (k-blocks)
constexpr int kTmExpanders = 16;              // expander warps: 8 units per k-block, two k-blocks in flight
constexpr int kTmUnits = 8;                   // units per k-block: 4 lane quarters x 2 halves of 32 tokens
constexpr int kTmGroups = kTmExpanders / kTmUnits;   // k-blocks in flight: group g takes the k-blocks i with i % kTmGroups == g
constexpr int kTmThreads = 32 * (4 + kTmExpanders);
constexpr int kTmWinPieces = 2;               // 16-byte pieces of `values` a lane holds for its token (else: global reads)
constexpr int kTmWinPitch = 48;               // private slot per lane: two pieces, padded to an odd number of pieces (bank spread)
constexpr int kTmRowPitch = 80;               // expander row: 32 tokens x 2 bytes, padded (bank spread, 16-byte aligned)
constexpr int kTmStageBytes = kBN * kBK * 2;  // 32 KB
constexpr int kTmAccCols = kBN;               // accumulator columns
constexpr int kTmACols = kBK / 2;             // operand columns per k-block (two tokens per column)
constexpr int kTmTmemCols = 512;

struct TmCtl {
    uint64_t b_full[kTmStages];
    uint64_t b_empty[kTmStages];
    uint64_t a_full[kTmAStages];
    uint64_t a_empty[kTmAStages];
    uint64_t meta_full[kTmMetaSlots];
    uint64_t meta_empty[kTmMetaSlots];
    uint64_t accum;
    uint32_t tmem_base;
    int abort_flag;
};

constexpr size_t kTmMaskBytes = (size_t)kTmMetaSlots * kBK * 16;        // [slot][row][4 words]
constexpr size_t kTmBaseBytes = (size_t)kTmMetaSlots * kBK * 4;         // [slot][row]
constexpr size_t kTmValBytes = (size_t)kTmExpanders * 32 * kTmWinPitch;   // [expander warp][lane]: the token's pieces
constexpr size_t kTmRowsBytes = (size_t)kTmExpanders * 32 * kTmRowPitch;
constexpr size_t kTmOffMask = (size_t)kTmStages * kTmStageBytes;
constexpr size_t kTmOffBase = kTmOffMask + kTmMaskBytes;
constexpr size_t kTmOffVal = kTmOffBase + kTmBaseBytes;
constexpr size_t kTmOffRows = kTmOffVal + kTmValBytes;
constexpr size_t kTmOffCtl = kTmOffRows + kTmRowsBytes;
constexpr size_t kTmSmemBytes = 1024 + kTmOffCtl + sizeof(TmCtl);
static_assert(kTmAccCols + kTmAStages * kTmACols <= kTmTmemCols, "tensor memory columns");
static_assert(kTmSmemBytes <= 232448, "dynamic shared memory of the tensor-memory kernel exceeds 227 KB");
static_assert(kXchgMaxBytes <= (int)kTmOffCtl, "the cluster exchange area reuses the pipeline buffers (all of them are dead by then)");

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_4(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
// Arrive on the mbarrier once every cp.async issued so far by this thread has landed.
__device__ __forceinline__ void cp_async_arrive(uint64_t* bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(ptx::smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// A load whose result must not meet control flow before it is used: a predicated-off load leaves zeroes in the
// registers and the compiler sees one opaque instruction, so nothing waits for the data where it is issued.
__device__ __forceinline__ uint4 ldg_v4_if(const void* p, bool pred) {
    uint4 v;
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %5, 0;\n\tmov.u32 %0, 0;\n\tmov.u32 %1, 0;\n\tmov.u32 %2, 0;\n\tmov.u32 %3, 0;\n\t"
                 "@q ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];\n\t}"
                 : "=&r"(v.x), "=&r"(v.y), "=&r"(v.z), "=&r"(v.w) : "l"(p), "r"((uint32_t)pred));
    return v;
}

// Transposed finish of the cluster exchange: the lane is channel c, the 16 registers of a piece are 16
// consecutive outputs j.  Terms are added in split order (this CTA's own from TMEM); every store of the warp
// is one 128-byte row segment of dW.  (16 columns at a time keeps the registers few: the expander warps
// set the kernel's register budget.)
__device__ __forceinline__ void cluster_finish_chunks_t(uint32_t tmem_base, const uint8_t* xchg, int g, int lane,
                                                        int rank, int splits, int j0, int c0, int Ca, int Cz,
                                                        float* __restrict__ dw, int accumulate) {
    const int cpo = (kBN / 32) / splits;
    const int c = c0 + 32 * g + lane;
#pragma unroll 1
    for (int piece = 0; piece < 2 * cpo; ++piece) {
        const int col = rank * cpo * 32 + piece * 16;          // column of the tile
        uint32_t r[16];
        ptx::tmem_ld_32x16(tmem_base + ((uint32_t)(32 * g) << 16) + col, r);
        ptx::tmem_ld_wait();
        float acc[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) acc[e] = 0.f;
        for (int s = 0; s < splits; ++s) {                            // fixed order over the splits
            if (s == rank) {
#pragma unroll
                for (int e = 0; e < 16; ++e) acc[e] += __uint_as_float(r[e]);
            } else {
                const int slot = s < rank ? s : s - 1;
#pragma unroll
                for (int e = 0; e < 16; e += 4) {
                    const float4 v = *reinterpret_cast<const float4*>(
                        xchg + xchg_offset(slot, cpo, piece >> 1, g, (piece & 1) * 4 + e / 4, lane));
                    acc[e] += v.x; acc[e + 1] += v.y; acc[e + 2] += v.z; acc[e + 3] += v.w;
                }
            }
        }
        if (c < Ca) {
            const int jb = j0 + col;
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                if (jb + e < Cz) {
                    float* dst = dw + (size_t)(jb + e) * Ca + c;
                    *dst = accumulate ? (*dst + acc[e]) : acc[e];
                }
            }
        }
    }
}

// One split per tile: the accumulator goes straight to dW.
__device__ __forceinline__ void store_tile_t(uint32_t tmem_base, int g, int lane, int j0, int c0, int Ca, int Cz,
                                             float* __restrict__ dw, int accumulate) {
    const int c = c0 + 32 * g + lane;
#pragma unroll 1
    for (int piece = 0; piece < kBN / 16; ++piece) {
        uint32_t r[16];
        ptx::tmem_ld_32x16(tmem_base + ((uint32_t)(32 * g) << 16) + piece * 16, r);
        ptx::tmem_ld_wait();
        if (c < Ca) {
            const int jb = j0 + piece * 16;
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                if (jb + e < Cz) {
                    float* dst = dw + (size_t)(jb + e) * Ca + c;
                    const float v = __uint_as_float(r[e]);
                    *dst = accumulate ? (*dst + v) : v;
                }
            }
        }
    }
}

__global__ void __launch_bounds__(kTmThreads, 1)
wg_tmem_kernel(const __grid_constant__ CUtensorMap map_dy, const uint16_t* __restrict__ values,
               const uint32_t* __restrict__ mask, const uint32_t* __restrict__ offsets, uint32_t k_total, int M, int Ca,
               int Cz, int tiles_n, int splits, int kb_per_split, int kb_total,
               float* __restrict__ dw, int accumulate, int32_t* dev_status, int grouped_map, uint32_t wait_limit) {
    extern __shared__ uint8_t smem_raw[];
    // (the rounding gives the same offsets in every CTA of a cluster: the exchange maps addresses between them)
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sB = smem;
    uint32_t* s_mask = reinterpret_cast<uint32_t*>(smem + kTmOffMask);
    uint32_t* s_base = reinterpret_cast<uint32_t*>(smem + kTmOffBase);
    uint8_t* s_vals = smem + kTmOffVal;
    uint8_t* s_rows = smem + kTmOffRows;
    TmCtl* ctl = reinterpret_cast<TmCtl*>(smem + kTmOffCtl);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int tile = blockIdx.x;
    const int split = (splits > 1) ? (int)ptx::cluster_ctarank() : 0;   // the cluster is (1, splits, 1)
    const int c0 = (tile / tiles_n) * kBM;        // 128 channels
    const int j0 = (tile % tiles_n) * kBN;        // 256 outputs
    const int kb_begin = split * kb_per_split;
    const int kb_end = min(kb_total, kb_begin + kb_per_split);
    const int nkb = kb_end - kb_begin;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kTmStages; ++s) {
            ptx::mbar_init(&ctl->b_full[s], 1);
            ptx::mbar_init(&ctl->b_empty[s], 1);
        }
        for (int s = 0; s < kTmAStages; ++s) {
            ptx::mbar_init(&ctl->a_full[s], kTmUnits);
            ptx::mbar_init(&ctl->a_empty[s], 1);
        }
        for (int s = 0; s < kTmMetaSlots; ++s) {
            ptx::mbar_init(&ctl->meta_full[s], 32);
            ptx::mbar_init(&ctl->meta_empty[s], kTmUnits);
        }
        ptx::mbar_init(&ctl->accum, 1);
        ctl->abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&map_dy);
    }
    if (warp == 1) {
        ptx::tmem_alloc(&ctl->tmem_base, kTmTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const uint32_t tmem_a = tmem_base + kTmAccCols;
    volatile int* abort_flag = &ctl->abort_flag;
    // Everything read below may come from the kernel before this one in the stream.
    ptx::grid_dependency_wait();

    if (warp == 0) {
        // ---------------- TMA producer: dY stages ----------------
        if (lane == 0) {
            int issued = 0;
            for (int i = 0; i < nkb && !*abort_flag; ++i) {
                const int s = i % kTmStages;
                if (i >= kTmStages && !ptx::mbar_wait_spin(&ctl->b_empty[s], ((i / kTmStages) - 1) & 1, wait_limit)) {
                    *abort_flag = 1;
                    break;
                }
                ptx::mbar_arrive_expect_tx(&ctl->b_full[s], kTmStageBytes);
                const int k0 = (kb_begin + i) * kBK;
                uint8_t* b = sB + s * kTmStageBytes;
                if (grouped_map) {
                    ptx::tma_load_3d(b, &map_dy, 0, k0, j0 / 64, &ctl->b_full[s]);
                } else {
#pragma unroll
                    for (int g = 0; g < kBN / 64; ++g)
                        ptx::tma_load_2d(b + g * (64 * kBK * 2), &map_dy, j0 + 64 * g, k0, &ctl->b_full[s]);
                }
                issued = i + 1;
            }
            if (*abort_flag) {   // let the copies already in flight land before the CTA exits
                for (int i = max(0, issued - kTmStages); i < issued; ++i)
                    ptx::mbar_wait(&ctl->b_full[i % kTmStages], (i / kTmStages) & 1, kWaitLimit);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::make_idesc_bf16(kBM, kBN, false, true);
            constexpr uint32_t kGroupBytes = 64 * kBK * 2;   // one 64-wide N group: kBK rows of 128 bytes
            for (int i = 0; i < nkb; ++i) {
                const int s = i % kTmStages, sa = i % kTmAStages;
                if (*abort_flag || !ptx::mbar_wait_spin(&ctl->a_full[sa], (i / kTmAStages) & 1, wait_limit) ||
                    !ptx::mbar_wait_spin(&ctl->b_full[s], (i / kTmStages) & 1, wait_limit)) {
                    *abort_flag = 1;
                    break;
                }
                ptx::tc_fence_after();
                const uint32_t b_addr = ptx::smem_u32(sB + s * kTmStageBytes);
#pragma unroll
                for (int kk = 0; kk < kBK / 16; ++kk) {
                    const uint64_t bd = ptx::make_smem_desc_sw128(b_addr + kk * 2048, kGroupBytes, 1024);
                    ptx::umma_bf16_ts(tmem_base, tmem_a + sa * kTmACols + kk * 8, bd, idesc, (i > 0 || kk > 0) ? 1u : 0u);
                }
                ptx::umma_commit(&ctl->b_empty[s]);
                ptx::umma_commit(&ctl->a_empty[sa]);
            }
            ptx::umma_commit(&ctl->accum);   // also after an abort: the barrier then tells when the MMAs in flight are done
        }
    } else if (warp == 2) {
        // ---------------- meta loader: mask piece (16 bytes) and table entry of every row, two rows per lane ----------------
        for (int i = 0; i < nkb; ++i) {
            const int slot = i % kTmMetaSlots;
            if (i >= kTmMetaSlots) {
                const bool ok = ptx::mbar_wait_warp(&ctl->meta_empty[slot], ((i / kTmMetaSlots) - 1) & 1, wait_limit);
                if (!__all_sync(kFullMask, ok)) *abort_flag = 1;
            }
            if (*abort_flag) break;
            const int k0 = (kb_begin + i) * kBK;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int r = lane + 32 * h;
                const int n = k0 + r;
                const bool live = n < M;   // rows past the last token are zero-filled by the copy itself
                const long long f = live ? ((long long)n * Ca + c0) : 0;
                cp_async_16(ptx::smem_u32(s_mask + ((size_t)slot * kBK + r) * 4), mask + (f >> 5), live ? 16u : 0u);
                cp_async_4(ptx::smem_u32(s_base + (size_t)slot * kBK + r), offsets + (f >> 7), live ? 4u : 0u);
            }
            cp_async_arrive(&ctl->meta_full[slot]);
        }
        cp_async_wait_all();
    } else if (warp == 3) {
        // (no role)
    } else {
        // ---------------- expanders ----------------
        const int ew = warp - 4;
        const int q = warp & 3;                       // TMEM lane quarter of this warp = 32-channel group of the tile
        const int h = (ew >> 2) & 1;                  // which 32 tokens of the k-block
        const int par = ew >> 3;                      // this warp takes the k-blocks i with i % kTmGroups == par
        const uint32_t rows_warp = ptx::smem_u32(s_rows + (size_t)ew * 32 * kTmRowPitch);   // [channel][32 tokens]
        const uint32_t my_row = rows_warp + lane * kTmRowPitch;
        const uint32_t my_win = ptx::smem_u32(s_vals + ((size_t)ew * 32 + lane) * kTmWinPitch);
        const uint32_t dst_t = rows_warp + 2u * lane;         // column `lane` (this token) of the image
        // What a lane knows about its token in one unit: the mask word for the warp's 32 channels, where the
        // token's values for them start in `values` (absolute index), how many, and the pieces that hold them.
        struct Unit {
            uint32_t w, first, cnt;
            uint4 p0, p1;
            bool held;     // the values are all inside p0, p1
        };
        // Read the meta data of k-block j (which has landed, or the wait here ends soon), request the values,
        // give the meta slot back.  Returns false when a wait ran out.
        auto fetch_unit = [&](int j, Unit& u) -> bool {
            const int ms = j % kTmMetaSlots;
            const bool okf = ptx::mbar_wait_warp(&ctl->meta_full[ms], (j / kTmMetaSlots) & 1, wait_limit);
            if (!__all_sync(kFullMask, okf)) return false;
            const int r = 32 * h + lane;                      // lane t: token row r of the k-block
            uint4 mw;
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(mw.x), "=r"(mw.y), "=r"(mw.z), "=r"(mw.w)
                         : "r"(ptx::smem_u32(s_mask + ((size_t)ms * kBK + r) * 4)) : "memory");
            uint32_t bs;
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(bs) : "r"(ptx::smem_u32(s_base + (size_t)ms * kBK + r)) : "memory");
            u.w = q == 0 ? mw.x : q == 1 ? mw.y : q == 2 ? mw.z : mw.w;
            uint32_t pre = 0;
            if (q > 0) pre += __popc(mw.x);
            if (q > 1) pre += __popc(mw.y);
            if (q > 2) pre += __popc(mw.z);
            u.first = bs + pre;
            u.cnt = __popc(u.w);
            const uint32_t a0 = u.first & ~7u, off = u.first & 7u;
            const bool need0 = u.cnt > 0, need1 = off + u.cnt > 8;
            const bool fits = off + u.cnt <= 8u * kTmWinPieces;
            const bool in0 = a0 + 8 <= k_total, in1 = a0 + 16 <= k_total;   // whole pieces only (the end of `values`: global reads)
            u.held = fits && (!need0 || in0) && (!need1 || in1);
            u.p0 = ldg_v4_if(values + a0, u.held && need0);
            u.p1 = ldg_v4_if(values + a0 + 8, u.held && need1);
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&ctl->meta_empty[ms]);
            return true;
        };
        Unit cur, nxt;
        if (par < nkb && !fetch_unit(par, cur)) *abort_flag = 1;
        for (int i = par; i < nkb && !*abort_flag; i += kTmGroups) {
            const int sa = i % kTmAStages;
            if (i + kTmGroups < nkb && !fetch_unit(i + kTmGroups, nxt)) {
                *abort_flag = 1;
                break;
            }
            bool ok = true;
            if (i >= kTmAStages) ok = ptx::mbar_wait_warp(&ctl->a_empty[sa], ((i / kTmAStages) - 1) & 1, wait_limit);
            if (!__all_sync(kFullMask, ok)) *abort_flag = 1;
            if (*abort_flag) break;
            ptx::tc_fence_after();
            // As a channel: lane c owns row c of the warp's [channel][token] image; it starts as zeroes.
#pragma unroll
            for (int z = 0; z < 4; ++z)
                asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(my_row + z * 16), "r"(0u) : "memory");
            // As a token: park the pieces, then walk the retained channels from the highest down; the token's
            // values are taken from the end of its run, so nothing has to be counted.
            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(my_win), "r"(cur.p0.x), "r"(cur.p0.y), "r"(cur.p0.z), "r"(cur.p0.w) : "memory");
            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(my_win + 16), "r"(cur.p1.x), "r"(cur.p1.y), "r"(cur.p1.z), "r"(cur.p1.w) : "memory");
            uint32_t w = cur.w;
            uint32_t vend = (cur.first & 7u) + cur.cnt;       // behind the token's last value, counted from piece 0
            const uint32_t g0 = cur.first & ~7u;
            const bool held = cur.held;
            __syncwarp();   // every row of the image is zeroed
            while (w) {   // four retained channels per trip: their shared-memory reads overlap
                uint32_t c[4], v[4];
                bool has[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    has[u] = w != 0;
                    asm("bfind.u32 %0, %1;" : "=r"(c[u]) : "r"(w));   // 0xFFFFFFFF when w is 0
                    c[u] &= 31u;
                    w &= ~(1u << c[u]);
                }
                if (held) {
#pragma unroll
                    for (int u = 0; u < 4; ++u)   // (slots without a channel read a valid address and are not stored)
                        asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v[u]) : "r"(my_win + 2u * ((vend - 1u - u) & 15u)) : "memory");
                } else {          // a token with more values than the pieces hold, or at the end of `values`
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const uint32_t at = g0 + vend - 1u - u;
                        v[u] = (has[u] && at < k_total) ? (uint32_t)__ldg(values + at) : 0u;
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (has[u]) asm volatile("st.shared.u16 [%0], %1;" ::"r"(dst_t + c[u] * kTmRowPitch), "r"(v[u]) : "memory");
                vend -= 4;
            }
            __syncwarp();   // the image is complete
            cur = nxt;
            uint32_t regs[16];
#pragma unroll
            for (int z = 0; z < 4; ++z)
                asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(regs[4 * z]), "=r"(regs[4 * z + 1]), "=r"(regs[4 * z + 2]), "=r"(regs[4 * z + 3])
                             : "r"(my_row + z * 16) : "memory");
            ptx::tmem_st_32x32_x16(tmem_a + ((uint32_t)(32 * q) << 16) + sa * kTmACols + h * 16, regs);
            ptx::tmem_st_wait();
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&ctl->a_full[sa]);
        }
        if (warp < 8) {
            // ---------------- epilogue (these four warps cover the four TMEM lane quarters) ----------------
            ptx::launch_dependents();
            bool ok = ptx::mbar_wait_warp(&ctl->accum, 0, wait_limit);
            ok = __all_sync(kFullMask, ok) && !*abort_flag;
            if (!ok) *abort_flag = 1;
            if (ok && splits == 1) {
                ptx::tc_fence_after();
                store_tile_t(tmem_base, q, lane, j0, c0, Ca, Cz, dw, accumulate);
            }
        }
    }

    if (splits > 1) {
        // All roles are done: the accumulator is final and the dY stages are free.  Every thread of the cluster
        // takes part in the two barriers, whatever happened before.
        uint8_t* xchg = smem;
        __syncwarp();
        ptx::cluster_sync_all();
        const bool epi_warp = warp >= 4 && warp < 8;
        if (epi_warp && !*abort_flag) {
            ptx::tc_fence_after();
            cluster_send_chunks(tmem_base, xchg, warp & 3, 0, 1, lane, split, splits);
        }
        __syncwarp();
        ptx::cluster_sync_all();
        if (epi_warp && !*abort_flag)
            cluster_finish_chunks_t(tmem_base, xchg, warp & 3, lane, split, splits, j0, c0, Ca, Cz, dw, accumulate);
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        // after an abort nobody has waited for the MMAs that were already issued: tensor memory is not given
        // back while they may still read or write it (always the full limit here)
        if (*abort_flag) ptx::mbar_wait_warp(&ctl->accum, 0, kWaitLimit);
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kTmTmemCols);
    }
    if (*abort_flag && threadIdx.x == 0 && dev_status) atomicExch(dev_status, (int)DROPIT_ERR_TIMEOUT);
}

}  // namespace


// Tiles of 128 channels x 256 outputs; `splits` CTAs per tile along the token axis (1, 2 or 4: a cluster).
dropit_status launch_wg_tmem(const void* dy, const void* values, const void* mask, const uint32_t* offsets, int64_t M,
                             int64_t Ca, int64_t Cz, int64_t k, int splits, int kb_per_split, int kb_total, float* dw,
                             int accumulate, int32_t* dev_status, cudaStream_t stream) {
    CUtensorMap map_dy;
    const bool grouped = (Cz % 64 == 0);
    if (grouped ? !make_map_grouped_bf16(&map_dy, dy, M, Cz, kBN / 64, kBK) : !make_map_2d_bf16(&map_dy, dy, M, Cz, kBK))
        return DROPIT_ERR_CUDA;
    static PerDeviceOnce attr;
    if (attr.needed()) {
        if (cudaFuncSetAttribute(wg_tmem_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTmSmemBytes) !=
            cudaSuccess)
            return DROPIT_ERR_CUDA;
        attr.mark();
    }
    const int tiles_m = (int)(Ca / kBM);
    const int tiles_n = (int)((Cz + kBN - 1) / kBN);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(tiles_m * tiles_n, splits);
    cfg.blockDim = dim3(kTmThreads);
    cfg.dynamicSmemBytes = kTmSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attrs[2];
    cfg.attrs = attrs;
    if (splits > 1) {
        attrs[cfg.numAttrs].id = cudaLaunchAttributeClusterDimension;
        attrs[cfg.numAttrs].val.clusterDim.x = 1;
        attrs[cfg.numAttrs].val.clusterDim.y = (unsigned)splits;
        attrs[cfg.numAttrs].val.clusterDim.z = 1;
        ++cfg.numAttrs;
    }
    attrs[cfg.numAttrs].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[cfg.numAttrs].val.programmaticStreamSerializationAllowed = 1;
    ++cfg.numAttrs;
    if (cudaLaunchKernelEx(&cfg, wg_tmem_kernel, map_dy, reinterpret_cast<const uint16_t*>(values),
                           reinterpret_cast<const uint32_t*>(mask), offsets, (uint32_t)k, (int)M, (int)Ca, (int)Cz,
                           tiles_n, splits, kb_per_split, kb_total, dw, accumulate, dev_status,
                           grouped ? 1 : 0, spin_limit(kWaitLimit)) != cudaSuccess) {
        (void)cudaGetLastError();
        return DROPIT_ERR_CUDA;
    }
    return check_launch();
}

}  // namespace dropit
