// Retained values in 8 bits (Sec. 1 and Table 5 combine DropIT with 8-bit / 4-bit activation quantisers on the
// layers DropIT does not cover; this is the same idea applied to DropIT's own payload).  Min-k keeps the largest
// magnitudes of a tensor, which span few binades, so a small float with one exponent shared by the tensor holds
// them to 1 part in 32:
//     code = sign | e (3 bits) | m (4 bits),   u = 2^(E_top - 127 - 10),   E_top = largest exponent field among
//     the finite values;   e = 0: m * u;   e = 1..7: (16 + m) * 2^(e-1) * u  (the top binade is that of E_top).
// Round to nearest code, ties to even; saturate above the largest code (also Inf / NaN); with E_top < 11 every
// code is zero.  Decoding gives bf16 values exactly, so the weight-gradient kernels run unchanged on them.
#include "common.cuh"

namespace dropit {

__global__ void q8_top_exponent_kernel(const uint16_t* __restrict__ values, int64_t k, uint32_t* __restrict__ scale) {
    uint32_t top = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < k; i += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t e = (values[i] >> 7) & 0xFFu;
        if (e != 0xFFu && e > top) top = e;
    }
    for (int o = 16; o > 0; o >>= 1) top = max(top, __shfl_xor_sync(kFullMask, top, o));
    if ((threadIdx.x & 31) == 0 && top) atomicMax(scale, top);
}

// Integer form of the rounding: a value 1.m7 * 2^(E-127) lies d = E_top - E binades below the top one.
__device__ __forceinline__ uint32_t q8_encode_one(uint32_t v, uint32_t e_top) {
    const uint32_t sign = (v >> 8) & 0x80u;
    const uint32_t E = (v >> 7) & 0xFFu, m7 = v & 0x7Fu;
    if (E == 0xFFu) return sign | 0x7Fu;
    if (e_top < 11u || E == 0u) return sign;
    if (E > e_top) return sign | 0x7Fu;                 // above the scale (only with a foreign E_top)
    const uint32_t d = e_top - E;
    if (d <= 6u) {                                       // a full binade: round the 7-bit mantissa to 4 bits
        uint32_t e = 7u - d, m4 = m7 >> 3;
        const uint32_t rest = m7 & 7u;
        if (rest > 4u || (rest == 4u && (m4 & 1u))) ++m4;
        const uint32_t code = (e << 4) + m4;             // m4 = 16 carries into the next binade
        return sign | (code > 127u ? 127u : code);
    }
    // the lowest binade of codes: |v| / u = (128 + m7) / 2^s with s = d - 3 >= 4
    const uint32_t s = d - 3u;
    if (s >= 9u) return sign;
    const uint32_t x = 128u + m7;
    uint32_t q = x >> s;
    const uint32_t rem = x & ((1u << s) - 1u), half = 1u << (s - 1u);
    if (rem > half || (rem == half && (q & 1u))) ++q;
    return sign | q;                                     // 0 .. 16
}

__device__ __forceinline__ uint32_t q8_decode_one(uint32_t q, uint32_t e_top) {
    const uint32_t sign = (q & 0x80u) << 8;
    const uint32_t c = q & 0x7Fu;
    if (c == 0u || e_top < 11u) return sign;
    uint32_t e = c >> 4, m = c & 15u;
    if (e == 0u) {                                       // m * u, m in 1..15: normalise
        const uint32_t lead = 31u - __clz(m);            // 0..3
        return sign | ((e_top - 10u + lead) << 7) | (((m << (7u - lead)) & 0x7Fu));
    }
    return sign | ((e_top - 7u + e) << 7) | (m << 3);
}

__global__ void q8_encode_kernel(const uint16_t* __restrict__ values, int64_t k, const uint32_t* __restrict__ scale,
                                 uint8_t* __restrict__ codes) {
    const uint32_t e_top = *scale;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < k; i += (int64_t)gridDim.x * blockDim.x)
        codes[i] = (uint8_t)q8_encode_one(values[i], e_top);
}

__global__ void q8_decode_kernel(const uint8_t* __restrict__ codes, int64_t k, const uint32_t* __restrict__ scale,
                                 uint16_t* __restrict__ values) {
    const uint32_t e_top = *scale;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < k; i += (int64_t)gridDim.x * blockDim.x)
        values[i] = (uint16_t)q8_decode_one(codes[i], e_top);
}

static unsigned q8_blocks(int64_t k) {
    int64_t b = (k + 1023) / 1024;
    const int64_t cap = (int64_t)sm_count() * 8;
    if (b > cap) b = cap;
    return (unsigned)(b < 1 ? 1 : b);
}

}  // namespace dropit

using namespace dropit;

extern "C" dropit_status dropit_quantize_values(const void* values, int64_t k, uint8_t* codes, uint32_t* scale,
                                                void* cuda_stream) {
    if (k < 0 || !scale) return DROPIT_ERR_INVALID_ARG;
    cudaStream_t stream = as_stream(cuda_stream);
    if (cudaMemsetAsync(scale, 0, sizeof(uint32_t), stream) != cudaSuccess) return DROPIT_ERR_CUDA;
    if (k == 0) return DROPIT_OK;
    if (!values || !codes || !is_aligned16(values)) return DROPIT_ERR_INVALID_ARG;
    q8_top_exponent_kernel<<<q8_blocks(k), 256, 0, stream>>>(reinterpret_cast<const uint16_t*>(values), k, scale);
    dropit_status s = check_launch();
    if (s != DROPIT_OK) return s;
    q8_encode_kernel<<<q8_blocks(k), 256, 0, stream>>>(reinterpret_cast<const uint16_t*>(values), k, scale, codes);
    return check_launch();
}

extern "C" dropit_status dropit_dequantize_values(const uint8_t* codes, const uint32_t* scale, int64_t k, void* values,
                                                  void* cuda_stream) {
    if (k < 0 || !scale) return DROPIT_ERR_INVALID_ARG;
    if (k == 0) return DROPIT_OK;
    if (!values || !codes || !is_aligned16(values)) return DROPIT_ERR_INVALID_ARG;
    q8_decode_kernel<<<q8_blocks(k), 256, 0, as_stream(cuda_stream)>>>(codes, k, scale, reinterpret_cast<uint16_t*>(values));
    return check_launch();
}
