// Conv2d weight gradient on the tensor cores (Eq. 4-5, retained term), bf16, stride 1:
//   dW[j,c,u,v] = sum_{n,y,x} dY[n,j,y,x] * R(a-hat)[n,c, y+u-pad, x+v-pad]
// One implicit GEMM per filter tap (u,v): M = output channels j, N = input channels c, and the
// reduction runs over (n, y, x) with x innermost, which is the contiguous axis of both NCHW operands,
// so both are K-major for tcgen05.  A k-block is one image row: 64 x-positions of one (n, y).
// TMA tiles (4-D maps {W, H, C, B}, 128-byte swizzle) bring 128 rows of dY and BN rows of the input;
// the tap's vertical offset u-pad is a TMA coordinate (rows outside the image are zero-filled by the
// hardware), the horizontal offset v-pad cannot be one (a TMA tile must start on a 16-byte boundary),
// so the dense scratch holds one copy of R(a-hat) per horizontal offset, shifted by whole pixels.
// Every split of the reduction stores its partial tile; a second kernel adds them in split order.
#include "weight_grad_common.cuh"

namespace dropit {

dropit_status decompress_dispatch(const void* values, const void* meta, const uint32_t* offsets, int64_t n, int64_t k,
                                  dropit_dtype dtype, dropit_format format, void* out, cudaStream_t stream);

namespace {

constexpr int kCStages = 4;
constexpr int kCThreads = 192;
constexpr int kMaxTapsX = 7;          // widest filter the tensor-core path takes

struct ConvMaps {
    CUtensorMap dy;
    CUtensorMap x;                   // all horizontally shifted copies: {W, H, C, B, tap}
};

struct ConvTcSmem {
    uint64_t full[kCStages];
    uint64_t empty[kCStages];
    uint64_t accum;
    uint32_t tmem_base;
    int abort_flag;
};
constexpr size_t kConvTcSmemBytes = 1024 + (size_t)kCStages * (kAStageBytes + kBStageBytes) + sizeof(ConvTcSmem);

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn conv_encode_fn() {
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

// NCHW bf16 tensor [B, C, H, W]; box = xb x-positions x yb rows x `rows` channels x 1 image.  A box may
// reach outside the tensor in any dimension: those elements arrive as zeros.
bool make_map_nchw(CUtensorMap* map, const void* base, int B, int C, int H, int W, int xb, int yb, int rows) {
    EncodeTiledFn fn = conv_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[4] = {(cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)C, (cuuint64_t)B};
    cuuint64_t strides[3] = {(cuuint64_t)W * 2, (cuuint64_t)H * W * 2, (cuuint64_t)C * H * W * 2};
    cuuint32_t box[4] = {(cuuint32_t)xb, (cuuint32_t)yb, (cuuint32_t)rows, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

__device__ __forceinline__ void tma_load_5d(void* smem_dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            int c4, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(ptx::smem_u32(smem_dst)), "l"(map), "r"(ptx::smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
        : "memory");
}

// The shifted copies lie `copy_stride` bytes apart: a fifth dimension over them lets one box {64, 1, rows, 1, taps}
// bring the tiles of several horizontal taps, stacked tap after tap, with a single copy.
bool make_map_taps(CUtensorMap* map, const void* base, int B, int C, int H, int W, int S, size_t copy_stride, int rows,
                   int taps) {
    EncodeTiledFn fn = conv_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[5] = {(cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)C, (cuuint64_t)B, (cuuint64_t)S};
    cuuint64_t strides[4] = {(cuuint64_t)W * 2, (cuuint64_t)H * W * 2, (cuuint64_t)C * H * W * 2, (cuuint64_t)copy_stride};
    cuuint32_t box[5] = {64, 1, (cuuint32_t)rows, 1, (cuuint32_t)taps};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

__device__ __forceinline__ void tma_load_4d(void* smem_dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(ptx::smem_u32(smem_dst)), "l"(map), "r"(ptx::smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}

// One pass over R(a-hat) writes every horizontally shifted copy the filter needs:
//   out_shift[n,c,y,x] = in[n,c,y,x + shift]  (0 outside the row)  for every shift != 0 with a destination.
// A thread owns 8 pixels (16 bytes, rows are multiples of 8 pixels) and its two neighbour groups.
struct ShiftDst {
    uint4* out[2 * kMaxTapsX - 1];   // indexed by shift + kMaxTapsX - 1; null where the filter has no such tap
};

__global__ void __launch_bounds__(256)
shift_copies_kernel(const uint4* __restrict__ in, ShiftDst dst, int64_t groups, int groups_per_row) {
    ptx::launch_dependents();   // the GEMM behind this kernel may set itself up meanwhile
    for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < groups; g += (int64_t)gridDim.x * blockDim.x) {
        const int gx = (int)(g % groups_per_row);
        const uint4 zero = make_uint4(0, 0, 0, 0);
        const uint4 cur = __ldg(in + g);
        const uint4 prev = gx > 0 ? __ldg(in + g - 1) : zero;
        const uint4 next = gx + 1 < groups_per_row ? __ldg(in + g + 1) : zero;
        const uint32_t w[12] = {prev.x, prev.y, prev.z, prev.w, cur.x, cur.y, cur.z, cur.w, next.x, next.y, next.z, next.w};
#pragma unroll
        for (int sh = -(kMaxTapsX - 1); sh <= kMaxTapsX - 1; ++sh) {
            uint4* out = dst.out[sh + kMaxTapsX - 1];
            if (sh == 0 || out == nullptr) continue;
            const int s = 8 + sh;                 // first window pixel of the shifted group
            uint4 o;
            if ((s & 1) == 0) {
                o = make_uint4(w[s / 2], w[s / 2 + 1], w[s / 2 + 2], w[s / 2 + 3]);
            } else {
                const int a = (s - 1) / 2;
                o = make_uint4(__funnelshift_r(w[a], w[a + 1], 16), __funnelshift_r(w[a + 1], w[a + 2], 16),
                               __funnelshift_r(w[a + 2], w[a + 3], 16), __funnelshift_r(w[a + 3], w[a + 4], 16));
            }
            out[g] = o;
        }
    }
}

// Rows that are not a multiple of 8 pixels cannot be TMA rows (strides are multiples of 16 bytes): this
// kernel rewrites a [rows, W] tensor with row pitch Wp (a multiple of 8, zero padded), once per destination,
// shifted like shift_copies_kernel.  dst.out is indexed by shift + kMaxTapsX - 1 as there, shift 0 included.
__global__ void __launch_bounds__(256)
pad_shift_rows_kernel(const uint16_t* __restrict__ in, ShiftDst dst, int64_t rows, int W, int Wp) {
    ptx::launch_dependents();
    const int64_t total = rows * Wp;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = i / Wp;
        const int x = (int)(i - row * Wp);
        const uint16_t* src = in + row * W;
#pragma unroll
        for (int sh = -(kMaxTapsX - 1); sh <= kMaxTapsX - 1; ++sh) {
            uint16_t* out = reinterpret_cast<uint16_t*>(dst.out[sh + kMaxTapsX - 1]);
            if (out == nullptr) continue;
            const int xs = x + sh;
            out[i] = (x < W && xs >= 0 && xs < W) ? src[xs] : (uint16_t)0;
        }
    }
}

// Strided convolutions: one copy of the input per filter tap, sampled at the output positions,
//   out[t = u*S + v][n,c,y,x] = in[n,c, y*stride + u - pad, x*stride + v - pad]   (0 outside the image),
// with output geometry [Ho, Wp] (row pitch a multiple of 8 pixels, zero padded).  After this every tap is a plain
// GEMM of dY against its own copy.
__global__ void __launch_bounds__(256)
gather_taps_kernel(const uint16_t* __restrict__ in, uint16_t* __restrict__ out, size_t copy_elems, int64_t planes,
                   int H, int W, int Ho, int Wo, int Wp, int R, int S, int stride, int pad) {
    ptx::launch_dependents();
    const int64_t total = planes * Ho * Wp;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int x = (int)(i % Wp);
        const int y = (int)((i / Wp) % Ho);
        const int64_t plane = i / ((int64_t)Wp * Ho);
        const uint16_t* src = in + plane * H * W;
        for (int u = 0; u < R; ++u) {
            const int yi = y * stride + u - pad;
            for (int v = 0; v < S; ++v) {
                const int xi = x * stride + v - pad;
                const bool ok = x < Wo && yi >= 0 && yi < H && xi >= 0 && xi < W;
                out[(size_t)(u * S + v) * copy_elems + i] = ok ? src[(int64_t)yi * W + xi] : (uint16_t)0;
            }
        }
    }
}

// dw[j,c,u,v] (=|+=) sum over splits of partial[split][tap][j][c].  A warp takes 32 consecutive outputs; the eight
// warps of a block share out the splits (warp g adds splits g, g + 8, ... in ascending order, several loads in
// flight), and the eight sums are added in warp order: a fixed order for a given split count.
constexpr int kReduceGroups = 8;
__global__ void __launch_bounds__(32 * kReduceGroups)
conv_tc_reduce_kernel(const float* __restrict__ partial, int splits, int Cz, int Ca, int taps, float* __restrict__ dw,
                      int accumulate) {
    __shared__ float sums[kReduceGroups][32];
    const int64_t plane = (int64_t)taps * Cz * Ca;
    const int lane = threadIdx.x & 31, g = threadIdx.x >> 5;
    ptx::grid_dependency_wait();   // the partial tiles come from the kernel before this one
    for (int64_t base = (int64_t)blockIdx.x * 32; base < plane; base += (int64_t)gridDim.x * 32) {
        const int64_t i = base + lane;
        float acc = 0.f;
        if (i < plane) {
            int s = g;
            for (; s + 3 * kReduceGroups < splits; s += 4 * kReduceGroups) {
                const float v0 = __ldcg(partial + (int64_t)s * plane + i);
                const float v1 = __ldcg(partial + (int64_t)(s + kReduceGroups) * plane + i);
                const float v2 = __ldcg(partial + (int64_t)(s + 2 * kReduceGroups) * plane + i);
                const float v3 = __ldcg(partial + (int64_t)(s + 3 * kReduceGroups) * plane + i);
                acc += v0; acc += v1; acc += v2; acc += v3;
            }
            for (; s < splits; s += kReduceGroups) acc += __ldcg(partial + (int64_t)s * plane + i);
        }
        sums[g][lane] = acc;
        __syncthreads();
        if (g == 0 && i < plane) {
            float t = sums[0][lane];
#pragma unroll
            for (int w = 1; w < kReduceGroups; ++w) t += sums[w][lane];
            const int c = (int)(i % Ca);
            const int j = (int)((i / Ca) % Cz);
            const int tap = (int)(i / ((int64_t)Ca * Cz));
            float* d = dw + ((int64_t)j * Ca + c) * taps + tap;
            *d = accumulate ? (*d + t) : t;
        }
        __syncthreads();
    }
}

struct ConvTcParams {
    int Ca, Cz, R, S, pad;
    int xb, yb, nxb, nyb;        // k-block = xb x yb output positions (xb * yb = 64) of one image
    int bnc, nv, vgroups;        // B tile = nv horizontal taps x bnc input channels (nv * bnc <= 256)
    int a_rows;                  // rows of dY the A copy brings (the rows of a 128-row tile that can exist)
    int gathered;                // strided filter: the scratch holds one pre-sampled copy per tap (u*S + v)
    int flat_w;                  // > 0: planes are flattened into one row of H*W pixels and the vertical tap offset is
                                 // flat_w pixels per filter row along that row (stride 1, output as large as the input)
    int tiles_c;
    int splits, kb_per_split, kb_total;
};

// grid = (tiles_j * tiles_c * R * vgroups, splits).  Warp 0: TMA producer, warp 1: MMA issuer and
// TMEM owner, warps 2..5: epilogue (one TMEM lane quarter each).
__global__ void __launch_bounds__(kCThreads, 1)
conv_wg_tc_kernel(const __grid_constant__ ConvMaps maps, const ConvTcParams p, float* __restrict__ partial,
                  int32_t* dev_status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;
    uint8_t* sB = smem + kCStages * kAStageBytes;
    ConvTcSmem* ctl = reinterpret_cast<ConvTcSmem*>(sB + kCStages * kBStageBytes);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    int t = blockIdx.x;
    const int vg = t % p.vgroups; t /= p.vgroups;
    const int u = t % p.R;        t /= p.R;
    const int c0 = (t % p.tiles_c) * p.bnc;
    const int j0 = (t / p.tiles_c) * kBM;
    const int v0 = vg * p.nv;
    const int nvt = min(p.nv, p.S - v0);          // horizontal taps stacked in this tile
    const int ncols = nvt * p.bnc;                // accumulator columns in use
    const int split = blockIdx.y;
    const int kb_begin = split * p.kb_per_split;
    const int kb_end = min(p.kb_total, kb_begin + p.kb_per_split);
    const int nkb = max(0, kb_end - kb_begin);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kCStages; ++s) {
            ptx::mbar_init(&ctl->full[s], 1);
            ptx::mbar_init(&ctl->empty[s], 1);
        }
        ptx::mbar_init(&ctl->accum, 1);
        ctl->abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&maps.dy);
        ptx::prefetch_tensormap(&maps.x);
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
        if (lane == 0) {
            ptx::grid_dependency_wait();   // the dense copies are written by the kernels before this one
            // both boxes count in full, also where they reach outside the tensors (zero fill)
            const uint32_t stage_bytes = (uint32_t)p.a_rows * 128u + (uint32_t)(p.nv * p.bnc) * 128u;
            int issued = 0;
            int xblk = kb_begin % p.nxb;
            int yblk = (kb_begin / p.nxb) % p.nyb;
            int n = kb_begin / (p.nxb * p.nyb);
            for (int i = 0; i < nkb && !*abort_flag; ++i) {
                const int s = i % kCStages;
                if (i >= kCStages && !ptx::mbar_wait_spin(&ctl->empty[s], ((i / kCStages) - 1) & 1, kWaitLimit)) {
                    *abort_flag = 1;
                    break;
                }
                ptx::mbar_arrive_expect_tx(&ctl->full[s], stage_bytes);
                const int x0 = xblk * p.xb, y0 = yblk * p.yb;
                tma_load_4d(sA + s * kAStageBytes, &maps.dy, x0, y0, j0, n, &ctl->full[s]);
                if (p.gathered) tma_load_5d(sB + s * kBStageBytes, &maps.x, x0, y0, c0, n, u * p.S + v0, &ctl->full[s]);
                else if (p.flat_w) tma_load_5d(sB + s * kBStageBytes, &maps.x, x0 + (u - p.pad) * p.flat_w, y0, c0, n, v0, &ctl->full[s]);
                else tma_load_5d(sB + s * kBStageBytes, &maps.x, x0, y0 + u - p.pad, c0, n, v0, &ctl->full[s]);
                issued = i + 1;
                if (++xblk == p.nxb) {
                    xblk = 0;
                    if (++yblk == p.nyb) { yblk = 0; ++n; }
                }
            }
            if (*abort_flag) {   // let the copies already in flight land before the CTA exits
                for (int i = max(0, issued - kCStages); i < issued; ++i)
                    ptx::mbar_wait(&ctl->full[i % kCStages], (i / kCStages) & 1, kWaitLimit);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = ptx::make_idesc_bf16(kBM, ncols, false, false);   // both operands K-major
            bool ok = true;
            for (int i = 0; i < nkb; ++i) {
                const int s = i % kCStages;
                if (*abort_flag || !ptx::mbar_wait_spin(&ctl->full[s], (i / kCStages) & 1, kWaitLimit)) {
                    *abort_flag = 1;
                    ok = false;
                    break;
                }
                ptx::tc_fence_after();
                const uint32_t a_addr = ptx::smem_u32(sA + s * kAStageBytes);
                const uint32_t b_addr = ptx::smem_u32(sB + s * kBStageBytes);
#pragma unroll
                for (int kk = 0; kk < kBK / 16; ++kk) {   // 16 k-values = 32 bytes inside the swizzled 128-byte row
                    const uint64_t ad = ptx::make_smem_desc_sw128(a_addr + kk * 32, 16, 1024);
                    const uint64_t bd = ptx::make_smem_desc_sw128(b_addr + kk * 32, 16, 1024);
                    ptx::umma_bf16(tmem_base, ad, bd, idesc, (i > 0 || kk > 0) ? 1u : 0u);
                }
                ptx::umma_commit(&ctl->empty[s]);
            }
            if (ok) ptx::umma_commit(&ctl->accum);
        }
    } else if (nkb > 0) {
        ptx::launch_dependents();   // the reduction kernel may be brought up; it waits for this grid to finish
        bool ok = ptx::mbar_wait_warp(&ctl->accum, 0, kWaitLimit);
        ok = __all_sync(kFullMask, ok) && !*abort_flag;
        if (!ok) {
            *abort_flag = 1;
        } else {
            ptx::tc_fence_after();
            // Every MMA has read its operands: the pipeline buffers serve as a staging area.  A 32 x 32 chunk goes
            // TMEM -> registers -> shared memory (row pitch 36 floats) and leaves as full 128-byte row segments
            // (a lane storing its own row straight from registers writes 16 bytes every Ca * 4 bytes: 9 us per tile).
            const int g = warp & 3;
            const int taps = p.R * p.S;
            const bool vec_ok = (p.Ca & 3) == 0;
            constexpr int kRowFloats = 36;
            float* stage = reinterpret_cast<float*>(smem) + (warp - 2) * 32 * kRowFloats;
            const int rr0 = lane >> 3, q = lane & 7;
            if (j0 + 32 * g < p.Cz) {              // uniform over the warp: some of its rows exist
                for (int ch = 0; ch * 32 < ncols; ++ch) {
                    uint32_t r[32];
                    ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(32 * g) << 16) + ch * 32, r);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; e += 4)
                        *reinterpret_cast<float4*>(stage + lane * kRowFloats + e) =
                            make_float4(__uint_as_float(r[e]), __uint_as_float(r[e + 1]), __uint_as_float(r[e + 2]),
                                        __uint_as_float(r[e + 3]));
                    __syncwarp();
                    const int col = ch * 32 + 4 * q;   // bnc is a multiple of 16: 4 columns share one tap
                    if (col < ncols) {
                        const int vi = col / p.bnc;
                        const int c = c0 + (col - vi * p.bnc);
                        const int tap = u * p.S + v0 + vi;
#pragma unroll
                        for (int it = 0; it < 8; ++it) {
                            const int row = j0 + 32 * g + it * 4 + rr0;
                            if (row < p.Cz) {
                                const float4 v = *reinterpret_cast<const float4*>(stage + (it * 4 + rr0) * kRowFloats + 4 * q);
                                float* dst = partial + (((size_t)split * taps + tap) * p.Cz + row) * p.Ca + c;
                                if (vec_ok && c + 4 <= p.Ca) {
                                    *reinterpret_cast<float4*>(dst) = v;
                                } else {
                                    if (c < p.Ca) dst[0] = v.x;
                                    if (c + 1 < p.Ca) dst[1] = v.y;
                                    if (c + 2 < p.Ca) dst[2] = v.z;
                                    if (c + 3 < p.Ca) dst[3] = v.w;
                                }
                            }
                        }
                    }
                    __syncwarp();
                }
            }
        }
    } else {
        // an empty split contributes a zero tile
        const int taps = p.R * p.S;
        for (int idx = threadIdx.x - 64; idx < kBM * ncols; idx += kCThreads - 64) {
            const int row = j0 + idx / ncols, col = idx % ncols;
            const int vi = col / p.bnc;
            const int c = c0 + (col - vi * p.bnc);
            if (row < p.Cz && c < p.Ca)
                partial[(((size_t)split * taps + u * p.S + v0 + vi) * p.Cz + row) * p.Ca + c] = 0.f;
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kBN);
    }
    if (*abort_flag && threadIdx.x == 0 && dev_status) atomicExch(dev_status, (int)DROPIT_ERR_TIMEOUT);
}

struct ConvTcPlan {
    bool ok;
    int H, W, Ho, Wo;          // geometry the kernel sees (a 1x1 filter flattens each plane into one row)
    int tiles;
    ConvTcParams p;
    int row_w;                 // pixels per image row as the shifted copies are written (W of the caller's tensor)
    bool padded;               // the GEMM reads rewritten copies of X (rows not multiples of 8 pixels, or a strided filter)
    bool pad_dy;               // ... and a zero-padded copy of dY
    int copies;                // copies of X in the scratch: S (one per horizontal tap) or R*S (strided filter)
    int Hx;                    // rows per plane of the X copies
    int Wp, Wop;               // row pitch of the X copies / of the dY the GEMM reads
    size_t dense_stride, tmp_off, dy_off, partial_off, total_bytes;
};

ConvTcPlan make_conv_tc_plan(int B, int Ca, int H, int W, int Cz, int R, int S, int stride, int pad, dropit_dtype dtype) {
    ConvTcPlan pl{};
    if (dtype != DROPIT_BF16 || S > kMaxTapsX || pad > kMaxTapsX - 1 || B < 1) return pl;
    int Ho = (H + 2 * pad - R) / stride + 1, Wo = (W + 2 * pad - S) / stride + 1;
    const bool gathered = stride != 1;
    pl.row_w = W;
    int flat_w = 0;
    if (!gathered && R == 1 && S == 1 && pad == 0) {   // plain GEMM over the flattened plane
        W = H * W; H = 1; Wo = W; Ho = 1;
    } else if (!gathered && Ho == H && Wo == W && (W & 7) == 0 && R <= 2 * pad + 1) {
        // Output as large as the input, rows that are whole 16-byte groups: the planes of dY and of the shifted
        // copies are flattened into rows of H*W pixels.  A k-block is 64 consecutive pixels of that row (no padding
        // of short image rows, every tile row a whole aligned 128-byte line); filter row u reads the copy
        // (u - pad) * W pixels further along, and what that puts before the first or after the last pixel of the
        // plane (the image rows above and below) is outside the tensor map and arrives as zeros.  The horizontal
        // taps are the shifted copies as before, whose rows are zero where the tap leaves the image row.
        flat_w = W;
        W = H * W; H = 1; Wo = W; Ho = 1;
    }
    if (!gathered && Wo > W) return pl;
    pl.padded = gathered || (W & 7) || (Wo & 7);   // TMA strides are multiples of 16 bytes
    pl.pad_dy = (Wo & 7) != 0;
    pl.copies = gathered ? R * S : S;
    pl.Hx = gathered ? Ho : H;
    pl.Wp = ((gathered ? Wo : W) + 7) / 8 * 8;
    pl.Wop = (Wo + 7) / 8 * 8;
    ConvTcParams& p = pl.p;
    p.Ca = Ca; p.Cz = Cz; p.R = R; p.S = S; p.pad = pad;
    p.gathered = gathered ? 1 : 0;
    p.flat_w = flat_w;
    // One k-block = 64 consecutive pixels of one image row, so a tile row is exactly one 128-byte
    // swizzle row.  (Boxes with a narrower inner extent and several image rows are not used: their
    // shared-memory footprint under the 128-byte swizzle is not the dense one.)
    p.xb = 64; p.yb = 1;
    p.nxb = (Wo + p.xb - 1) / p.xb;
    p.nyb = (Ho + p.yb - 1) / p.yb;
    const int64_t kb_total = (int64_t)B * p.nxb * p.nyb;
    if (kb_total >= (1ll << 30)) return pl;
    p.kb_total = (int)kb_total;
    p.bnc = Ca >= kBN ? kBN : (Ca + 15) / 16 * 16;
    p.nv = kBN / p.bnc < S ? kBN / p.bnc : S;
    if (p.nv < 1) p.nv = 1;
    p.vgroups = (S + p.nv - 1) / p.nv;
    p.tiles_c = (Ca + p.bnc - 1) / p.bnc;
    p.a_rows = Cz >= kBM ? kBM : (Cz + 7) / 8 * 8;   // tile rows past these hold stale bytes and feed unused D rows
    const int64_t tiles = (int64_t)((Cz + kBM - 1) / kBM) * p.tiles_c * R * p.vgroups;
    if (tiles > (1ll << 30)) return pl;
    pl.tiles = (int)tiles;
    int splits = sm_count() / pl.tiles;
    if (splits < 1) splits = 1;
    if (splits > p.kb_total) splits = p.kb_total;
    p.kb_per_split = (p.kb_total + splits - 1) / splits;
    p.splits = (p.kb_total + p.kb_per_split - 1) / p.kb_per_split;
    if (p.splits > 65535) return pl;
    pl.H = H; pl.W = W; pl.Ho = Ho; pl.Wo = Wo;
    pl.dense_stride = align_up((size_t)B * Ca * pl.Hx * pl.Wp * 2, 256);
    pl.tmp_off = pl.dense_stride * pl.copies;
    pl.dy_off = pl.tmp_off + (pl.padded ? align_up((size_t)B * Ca * H * W * 2, 256) : 0);
    pl.partial_off = pl.dy_off + (pl.pad_dy ? align_up((size_t)B * Cz * Ho * pl.Wop * 2, 256) : 0);
    pl.total_bytes = pl.partial_off + align_up((size_t)p.splits * R * S * Cz * Ca * 4, 256);
    pl.ok = true;
    return pl;
}

}  // namespace

// 0 when the tensor-core path does not take this shape.
size_t conv_tc_workspace_bytes(int B, int Ca, int H, int W, int Cz, int R, int S, int stride, int pad,
                               dropit_dtype dtype) {
    const ConvTcPlan pl = make_conv_tc_plan(B, Ca, H, W, Cz, R, S, stride, pad, dtype);
    return pl.ok ? pl.total_bytes : 0;
}

// Caller has validated pointers, sizes and alignment, and B >= 1, k >= 1.
dropit_status conv_tc_run(const void* dy, const void* values, const void* meta, const uint32_t* offsets, int B, int Ca,
                          int H, int W, int Cz, int R, int S, int stride, int pad, int64_t k, dropit_format format,
                          float* dw, int accumulate, void* workspace, size_t workspace_bytes, int32_t* dev_status,
                          cudaStream_t stream) {
    const ConvTcPlan pl = make_conv_tc_plan(B, Ca, H, W, Cz, R, S, stride, pad, DROPIT_BF16);
    if (!pl.ok) return DROPIT_ERR_UNSUPPORTED;
    if (workspace_bytes < pl.total_bytes) return DROPIT_ERR_WORKSPACE;
    unsigned char* ws = reinterpret_cast<unsigned char*>(workspace);
    const int64_t n = (int64_t)B * Ca * H * W;
    // slot v of the scratch holds the rows shifted by v - pad
    const void* dy_gemm = dy;
    if (!pl.padded) {
        void* dense0 = ws + pl.dense_stride * pad;   // the unshifted copy is the decompressed tensor itself
        dropit_status st0 = decompress_dispatch(values, meta, offsets, n, k, DROPIT_BF16, format, dense0, stream);
        if (st0 != DROPIT_OK) return st0;
        if (S > 1) {
            ShiftDst dst{};
            for (int v = 0; v < S; ++v)
                if (v != pad) dst.out[v - pad + kMaxTapsX - 1] = reinterpret_cast<uint4*>(ws + pl.dense_stride * v);
            const int64_t groups = n / 8;
            int64_t blocks = (groups + 255) / 256;
            if (blocks > (int64_t)sm_count() * 16) blocks = (int64_t)sm_count() * 16;
            shift_copies_kernel<<<(unsigned)blocks, 256, 0, stream>>>(reinterpret_cast<const uint4*>(dense0), dst, groups,
                                                                     (pl.p.flat_w ? pl.row_w : pl.W) / 8);
            st0 = check_launch();
            if (st0 != DROPIT_OK) return st0;
        }
    } else {
        uint16_t* tmp = reinterpret_cast<uint16_t*>(ws + pl.tmp_off);
        dropit_status st0 = decompress_dispatch(values, meta, offsets, n, k, DROPIT_BF16, format, tmp, stream);
        if (st0 != DROPIT_OK) return st0;
        const int cap = sm_count() * 16;
        if (pl.pad_dy) {   // dY with padded rows
            ShiftDst dst{};
            dst.out[kMaxTapsX - 1] = reinterpret_cast<uint4*>(ws + pl.dy_off);
            const int64_t rows = (int64_t)B * Cz * pl.Ho;
            int64_t blocks = (rows * pl.Wop + 255) / 256;
            if (blocks > cap) blocks = cap;
            pad_shift_rows_kernel<<<(unsigned)blocks, 256, 0, stream>>>(reinterpret_cast<const uint16_t*>(dy), dst, rows,
                                                                       pl.Wo, pl.Wop);
            st0 = check_launch();
            if (st0 != DROPIT_OK) return st0;
            dy_gemm = ws + pl.dy_off;
        }
        if (pl.p.gathered) {
            const int64_t planes = (int64_t)B * Ca;
            int64_t blocks = (planes * pl.Ho * pl.Wp + 255) / 256;
            if (blocks > cap) blocks = cap;
            gather_taps_kernel<<<(unsigned)blocks, 256, 0, stream>>>(tmp, reinterpret_cast<uint16_t*>(ws),
                                                                    pl.dense_stride / 2, planes, H, W, pl.Ho, pl.Wo,
                                                                    pl.Wp, R, S, stride, pad);
        } else {
            ShiftDst dst{};
            for (int v = 0; v < S; ++v)
                dst.out[v - pad + kMaxTapsX - 1] = reinterpret_cast<uint4*>(ws + pl.dense_stride * v);
            const int64_t rows = (int64_t)B * Ca * pl.H;
            int64_t blocks = (rows * pl.Wp + 255) / 256;
            if (blocks > cap) blocks = cap;
            pad_shift_rows_kernel<<<(unsigned)blocks, 256, 0, stream>>>(tmp, dst, rows, pl.W, pl.Wp);
        }
        st0 = check_launch();
        if (st0 != DROPIT_OK) return st0;
    }
    dropit_status st = DROPIT_OK;
    ConvMaps maps;
    if (!make_map_nchw(&maps.dy, dy_gemm, B, Cz, pl.Ho, pl.Wop, pl.p.xb, pl.p.yb, pl.p.a_rows)) return DROPIT_ERR_CUDA;
    if (!make_map_taps(&maps.x, ws, B, Ca, pl.Hx, pl.Wp, pl.copies, pl.dense_stride, pl.p.bnc, pl.p.nv))
        return DROPIT_ERR_CUDA;
    static PerDeviceOnce attr;
    if (attr.needed()) {
        if (cudaFuncSetAttribute(conv_wg_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kConvTcSmemBytes) != cudaSuccess)
            return DROPIT_ERR_CUDA;
        attr.mark();
    }
    float* partial = reinterpret_cast<float*>(ws + pl.partial_off);
    dim3 grid(pl.tiles, pl.p.splits);
    cudaLaunchAttribute pdl[1];
    pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kCThreads);
    cfg.dynamicSmemBytes = kConvTcSmemBytes;
    cfg.stream = stream;
    cfg.attrs = pdl;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, conv_wg_tc_kernel, maps, pl.p, partial, dev_status) != cudaSuccess) {
        (void)cudaGetLastError();
        return DROPIT_ERR_CUDA;
    }
    st = check_launch();
    if (st != DROPIT_OK) return st;
    const int64_t count = (int64_t)R * S * Cz * Ca;
    int64_t blocks = (count + 31) / 32;
    if (blocks > (int64_t)sm_count() * 8) blocks = (int64_t)sm_count() * 8;
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(32 * kReduceGroups);
    cfg.dynamicSmemBytes = 0;
    if (cudaLaunchKernelEx(&cfg, conv_tc_reduce_kernel, (const float*)partial, pl.p.splits, Cz, Ca, R * S, dw,
                           accumulate) != cudaSuccess) {
        (void)cudaGetLastError();
        return DROPIT_ERR_CUDA;
    }
    return check_launch();
}

}  // namespace dropit
