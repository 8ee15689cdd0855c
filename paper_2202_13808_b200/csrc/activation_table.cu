// Tables of element-wise activations over all 65536 bf16 bit patterns (Sec. 3.5: the producers of conv / fc
// inputs).  Every entry is the activation evaluated in double and rounded ONCE to bf16, ties to even, so a
// table lookup is the correctly rounded activation; the producer kernel (compress_fused.cu) applies it.
#include "common.cuh"

namespace dropit {

// A double rounded once to bf16: truncate to fp32 towards zero and remember whether anything was lost;
// then the low 16 bits of the fp32 pattern plus that sticky flag decide the rounding of the high 16.
__device__ __forceinline__ uint32_t round_to_bf16(double v) {
    if (v != v) return 0x7FC0u;
    const float f = __double2float_rz(v);
    const bool sticky = (double)f != v;
    const uint32_t u = __float_as_uint(f);
    const uint32_t sign = (u >> 16) & 0x8000u;
    const uint32_t a = u & 0x7FFFFFFFu;
    if (a >= 0x7F800000u) return sign | 0x7F80u;
    const uint32_t rem = a & 0xFFFFu;
    uint32_t hi = a >> 16;
    if (rem > 0x8000u || (rem == 0x8000u && (sticky || (hi & 1u)))) ++hi;   // a carry may reach the exponent: Inf
    return sign | hi;
}

__global__ void activation_table_kernel(int kind, uint16_t* __restrict__ table) {
    const uint32_t b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= 65536u) return;
    const uint32_t key = b & 0x7FFFu;
    uint32_t y;
    if (kind == (int)DROPIT_TABLE_IDENTITY || key > 0x7F80u) {
        y = b;                                                   // NaN patterns pass through
    } else if (kind == (int)DROPIT_TABLE_RELU) {
        y = ((b & 0x8000u) || key == 0u) ? 0u : b;
    } else {
        const double x = (double)__uint_as_float(b << 16);
        y = round_to_bf16(x * (0.5 * erfc(-x / sqrt(2.0))));     // x Phi(x); the erfc form keeps its digits for x < 0
    }
    table[b] = (uint16_t)y;
}

}  // namespace dropit

extern "C" dropit_status dropit_activation_table(dropit_table_kind kind, uint16_t* table, void* cuda_stream) {
    using namespace dropit;
    if (kind != DROPIT_TABLE_IDENTITY && kind != DROPIT_TABLE_RELU && kind != DROPIT_TABLE_GELU) return DROPIT_ERR_INVALID_ARG;
    if (!table || !is_aligned16(table)) return DROPIT_ERR_INVALID_ARG;
    activation_table_kernel<<<256, 256, 0, as_stream(cuda_stream)>>>((int)kind, table);
    return check_launch();
}
