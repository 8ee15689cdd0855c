// Conv2d weight gradient from the sparsified cache (Eq. 4-5, retained term):
//   dW[j,c,u,v] = sum_{n,y,x} dY[n,j,y,x] * R(a-hat)[n,c, y*stride+u-pad, x*stride+v-pad]
// NCHW, cross-correlation, groups 1, dilation 1.  The reduction over (n, y, x) is split by image;
// every split writes its partial gradient and a second kernel adds the partials in split order,
// so the summation order is fixed.
#include "common.cuh"

namespace dropit {

dropit_status decompress_dispatch(const void* values, const void* meta, const uint32_t* offsets, int64_t n, int64_t k,
                                  dropit_dtype dtype, dropit_format format, void* out, cudaStream_t stream);

// Tensor-core path (bf16, stride 1, rows a multiple of 8 pixels), defined in conv_weight_grad_tc.cu.
size_t conv_tc_workspace_bytes(int B, int Ca, int H, int W, int Cz, int R, int S, int stride, int pad,
                               dropit_dtype dtype);
dropit_status conv_tc_run(const void* dy, const void* values, const void* meta, const uint32_t* offsets, int B, int Ca,
                          int H, int W, int Cz, int R, int S, int stride, int pad, int64_t k, dropit_format format,
                          float* dw, int accumulate, void* workspace, size_t workspace_bytes, int32_t* dev_status,
                          cudaStream_t stream);

constexpr int kConvTJ = 32;     // output channels per block
constexpr int kConvTC = 8;      // input channels per block
constexpr int kConvMaxUV = 9;   // filter taps accumulated per sweep
constexpr int kConvMaxSplits = 64;

struct ConvPlan {
    int Ho, Wo, splits, tiles_j, tiles_c;
    size_t dense_off, dense_bytes, partial_off, partial_bytes, total_bytes;
    size_t smem_bytes;
};

static ConvPlan make_conv_plan(int B, int Ca, int H, int W, int Cz, int R, int S, int stride, int pad,
                               dropit_dtype dtype) {
    ConvPlan p{};
    p.Ho = (H + 2 * pad - R) / stride + 1;
    p.Wo = (W + 2 * pad - S) / stride + 1;
    p.splits = B < kConvMaxSplits ? B : kConvMaxSplits;
    if (p.splits < 1) p.splits = 1;
    p.tiles_j = (Cz + kConvTJ - 1) / kConvTJ;
    p.tiles_c = (Ca + kConvTC - 1) / kConvTC;
    const size_t es = (dtype == DROPIT_BF16) ? 2 : 4;
    p.dense_off = 0;
    p.dense_bytes = align_up((size_t)B * Ca * H * W * es, 256);
    p.partial_off = p.dense_bytes;
    p.partial_bytes = align_up((size_t)p.splits * Cz * Ca * R * S * 4, 256);
    p.total_bytes = p.partial_off + p.partial_bytes;
    const int wo_pad = p.Wo | 1;
    const int wx = (W + 2 * pad + S) | 1;
    p.smem_bytes = ((size_t)kConvTJ * wo_pad + (size_t)kConvTC * R * wx) * 4;
    return p;
}

__device__ __forceinline__ float conv_to_float(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }
__device__ __forceinline__ float conv_to_float(float f) { return f; }

template <typename T>
__global__ void __launch_bounds__(kConvTJ * kConvTC)
conv_wg_kernel(const T* __restrict__ dy, const T* __restrict__ xd, int B, int Ca, int H, int W, int Cz, int R, int S,
               int stride, int pad, int Ho, int Wo, int tiles_c, int splits, float* __restrict__ partial) {
    extern __shared__ float csm[];
    const int wo_pad = Wo | 1;
    const int wx = (W + 2 * pad + S) | 1;
    float* dys = csm;                              // [kConvTJ][wo_pad]
    float* xs = csm + (size_t)kConvTJ * wo_pad;    // [kConvTC][R][wx], column index = xi + pad

    const int j0 = (blockIdx.x / tiles_c) * kConvTJ;
    const int c0 = (blockIdx.x % tiles_c) * kConvTC;
    const int split = blockIdx.y;
    const int tj = threadIdx.x % kConvTJ, tc = threadIdx.x / kConvTJ;
    const int RS = R * S;
    const size_t plane = (size_t)Cz * Ca * RS;

    for (int uv0 = 0; uv0 < RS; uv0 += kConvMaxUV) {
        float acc[kConvMaxUV];
#pragma unroll
        for (int i = 0; i < kConvMaxUV; ++i) acc[i] = 0.f;
        for (int n = split; n < B; n += splits) {
            for (int y = 0; y < Ho; ++y) {
                __syncthreads();
                for (int i = threadIdx.x; i < kConvTJ * Wo; i += blockDim.x) {
                    const int jj = i / Wo, xx = i % Wo;
                    const int j = j0 + jj;
                    dys[jj * wo_pad + xx] =
                        (j < Cz) ? conv_to_float(dy[(((size_t)n * Cz + j) * Ho + y) * Wo + xx]) : 0.f;
                }
                const int wspan = W + 2 * pad + S;
                for (int i = threadIdx.x; i < kConvTC * R * wspan; i += blockDim.x) {
                    const int col = i % wspan;
                    const int u = (i / wspan) % R;
                    const int cc = i / (wspan * R);
                    const int c = c0 + cc;
                    const int yi = y * stride + u - pad;
                    const int xi = col - pad;
                    float val = 0.f;
                    if (c < Ca && yi >= 0 && yi < H && xi >= 0 && xi < W)
                        val = conv_to_float(xd[(((size_t)n * Ca + c) * H + yi) * W + xi]);
                    xs[(cc * R + u) * wx + col] = val;
                }
                __syncthreads();
                for (int xx = 0; xx < Wo; ++xx) {
                    const float d = dys[tj * wo_pad + xx];
#pragma unroll
                    for (int i = 0; i < kConvMaxUV; ++i) {
                        const int uv = uv0 + i;
                        if (uv < RS) {
                            const int u = uv / S, v = uv % S;
                            acc[i] = fmaf(d, xs[(tc * R + u) * wx + xx * stride + v], acc[i]);
                        }
                    }
                }
            }
        }
        const int j = j0 + tj, c = c0 + tc;
        if (j < Cz && c < Ca) {
#pragma unroll
            for (int i = 0; i < kConvMaxUV; ++i) {
                const int uv = uv0 + i;
                if (uv < RS) partial[split * plane + ((size_t)j * Ca + c) * RS + uv] = acc[i];
            }
        }
    }
}

__global__ void __launch_bounds__(256)
conv_reduce_kernel(const float* __restrict__ partial, int splits, int64_t count, float* __restrict__ dw,
                   int accumulate) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x) {
        float acc = accumulate ? dw[i] : 0.f;
        for (int s = 0; s < splits; ++s) acc += partial[(size_t)s * count + i];
        dw[i] = acc;
    }
}

__global__ void conv_zero_kernel(float* dw, int64_t count) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
        dw[i] = 0.f;
}

static dropit_status conv_check_shape(int B, int Ca, int H, int W, int Cz, int R, int S, int stride, int pad) {
    if (B < 0 || Ca <= 0 || H <= 0 || W <= 0 || Cz <= 0 || R <= 0 || S <= 0 || stride <= 0 || pad < 0)
        return DROPIT_ERR_INVALID_ARG;
    if (H + 2 * pad < R || W + 2 * pad < S) return DROPIT_ERR_INVALID_ARG;
    if ((int64_t)B * Ca * H * W >= ((int64_t)1 << 31)) return DROPIT_ERR_INVALID_ARG;
    return DROPIT_OK;
}

}  // namespace dropit

using namespace dropit;

extern "C" dropit_status dropit_conv_weight_grad_workspace(int B, int Ca, int H, int W, int Cz, int R, int S,
                                                           int stride, int pad, dropit_dtype dtype,
                                                           dropit_format format, size_t* workspace_bytes) {
    dropit_status s = conv_check_shape(B, Ca, H, W, Cz, R, S, stride, pad);
    if (s != DROPIT_OK) return s;
    if ((dtype != DROPIT_BF16 && dtype != DROPIT_F32) || (format != DROPIT_FMT_BITMASK && format != DROPIT_FMT_INDEX32))
        return DROPIT_ERR_INVALID_ARG;
    if (workspace_bytes) {
        const size_t tc = (B > 0) ? conv_tc_workspace_bytes(B, Ca, H, W, Cz, R, S, stride, pad, dtype) : 0;
        const ConvPlan p = make_conv_plan(B, Ca, H, W, Cz, R, S, stride, pad, dtype);
        *workspace_bytes = tc ? tc : (p.total_bytes ? p.total_bytes : 256);
    }
    return DROPIT_OK;
}

extern "C" dropit_status dropit_conv_weight_grad(const void* dy, const void* values, const void* meta,
                                                 const uint32_t* offsets, int B, int Ca, int H, int W, int Cz, int R,
                                                 int S, int stride, int pad, int dilation, int64_t k,
                                                 dropit_dtype dtype, dropit_format format, float* dw, int accumulate,
                                                 void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                                 void* cuda_stream) {
    dropit_status s = conv_check_shape(B, Ca, H, W, Cz, R, S, stride, pad);
    if (s != DROPIT_OK) return s;
    if ((dtype != DROPIT_BF16 && dtype != DROPIT_F32) || (format != DROPIT_FMT_BITMASK && format != DROPIT_FMT_INDEX32))
        return DROPIT_ERR_INVALID_ARG;
    if (dilation != 1) return DROPIT_ERR_UNSUPPORTED;
    const int64_t n = (int64_t)B * Ca * H * W;
    if (k < 0 || k > n || !dw || !is_aligned16(dw)) return DROPIT_ERR_INVALID_ARG;
    cudaStream_t stream = as_stream(cuda_stream);
    const int64_t count = (int64_t)Cz * Ca * R * S;
    if (B == 0 || k == 0) {
        if (!accumulate) conv_zero_kernel<<<sm_count(), 256, 0, stream>>>(dw, count);
        return check_launch();
    }
    if (!dy || !values || !meta || !is_aligned16(dy) || !is_aligned16(values) || !is_aligned16(meta))
        return DROPIT_ERR_INVALID_ARG;
    if (format == DROPIT_FMT_BITMASK && (!offsets || !is_aligned16(offsets))) return DROPIT_ERR_INVALID_ARG;
    if (!workspace || !is_aligned16(workspace)) return DROPIT_ERR_INVALID_ARG;
    if (conv_tc_workspace_bytes(B, Ca, H, W, Cz, R, S, stride, pad, dtype) != 0)
        return conv_tc_run(dy, values, meta, offsets, B, Ca, H, W, Cz, R, S, stride, pad, k, format, dw, accumulate,
                           workspace, workspace_bytes, dev_status, stream);
    const ConvPlan plan = make_conv_plan(B, Ca, H, W, Cz, R, S, stride, pad, dtype);
    if (plan.smem_bytes > 200 * 1024) return DROPIT_ERR_UNSUPPORTED;
    if (workspace_bytes < plan.total_bytes) return DROPIT_ERR_WORKSPACE;
    unsigned char* ws = reinterpret_cast<unsigned char*>(workspace);
    void* dense = ws + plan.dense_off;
    float* partial = reinterpret_cast<float*>(ws + plan.partial_off);

    s = decompress_dispatch(values, meta, offsets, n, k, dtype, format, dense, stream);
    if (s != DROPIT_OK) return s;

    dim3 grid(plan.tiles_j * plan.tiles_c, plan.splits);
    if (dtype == DROPIT_BF16) {
        auto kern = conv_wg_kernel<uint16_t>;
        if (plan.smem_bytes > 48 * 1024 &&
            cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem_bytes) != cudaSuccess)
            return DROPIT_ERR_CUDA;
        kern<<<grid, kConvTJ * kConvTC, plan.smem_bytes, stream>>>(
            reinterpret_cast<const uint16_t*>(dy), reinterpret_cast<const uint16_t*>(dense), B, Ca, H, W, Cz, R, S,
            stride, pad, plan.Ho, plan.Wo, plan.tiles_c, plan.splits, partial);
    } else {
        auto kern = conv_wg_kernel<float>;
        if (plan.smem_bytes > 48 * 1024 &&
            cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem_bytes) != cudaSuccess)
            return DROPIT_ERR_CUDA;
        kern<<<grid, kConvTJ * kConvTC, plan.smem_bytes, stream>>>(
            reinterpret_cast<const float*>(dy), reinterpret_cast<const float*>(dense), B, Ca, H, W, Cz, R, S, stride,
            pad, plan.Ho, plan.Wo, plan.tiles_c, plan.splits, partial);
    }
    s = check_launch();
    if (s != DROPIT_OK) return s;
    int64_t blocks = (count + 255) / 256;
    if (blocks > (int64_t)sm_count() * 8) blocks = (int64_t)sm_count() * 8;
    conv_reduce_kernel<<<(unsigned)blocks, 256, 0, stream>>>(partial, plan.splits, count, dw, accumulate);
    return check_launch();
}
