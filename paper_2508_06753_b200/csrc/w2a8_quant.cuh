// Arithmetic of the per-token activation quantiser (a8_quantize in w2a8.h), shared by the
// stand-alone quantiser kernels and by the streaming kernel that quantises its own input.
// Every step is one IEEE fp32 round-to-nearest-even operation.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace w2a8 {

__device__ __forceinline__ float bf16_bits_to_float(uint32_t h) { return __uint_as_float(h << 16); }

__device__ __forceinline__ uint32_t quant4(uint32_t lo, uint32_t hi, float inv) {
    // lo, hi: two 32-bit words holding four consecutive bf16 values
    const float x0 = __uint_as_float(lo << 16), x1 = __uint_as_float(lo & 0xFFFF0000u);
    const float x2 = __uint_as_float(hi << 16), x3 = __uint_as_float(hi & 0xFFFF0000u);
    int q0 = __float2int_rn(__fmul_rn(x0, inv)), q1 = __float2int_rn(__fmul_rn(x1, inv));
    int q2 = __float2int_rn(__fmul_rn(x2, inv)), q3 = __float2int_rn(__fmul_rn(x3, inv));
    q0 = max(-127, min(127, q0)); q1 = max(-127, min(127, q1));
    q2 = max(-127, min(127, q2)); q3 = max(-127, min(127, q3));
    return (uint32_t)(q0 & 0xFF) | ((uint32_t)(q1 & 0xFF) << 8) | ((uint32_t)(q2 & 0xFF) << 16) |
           ((uint32_t)(q3 & 0xFF) << 24);
}

__device__ __forceinline__ float quant_scale(uint32_t amax_bits, float *inv_out) {
    const float amax = bf16_bits_to_float(amax_bits);
    const float s = __fdiv_rn(amax, 127.0f);
    float inv = __fdiv_rn(1.0f, s);
    const bool dead = !(amax > 0.0f) || !(fabsf(inv) <= 3.402823466e38f);
    *inv_out = dead ? 0.0f : inv;
    return dead ? 0.0f : s;
}

// running maximum of the magnitudes (as bit patterns) of the eight bf16 values of a 16-byte vector
__device__ __forceinline__ uint32_t amax8(uint32_t amax_bits, const uint4 &v) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        amax_bits = max(amax_bits, w[q] & 0x7FFFu);
        amax_bits = max(amax_bits, (w[q] >> 16) & 0x7FFFu);
    }
    return amax_bits;
}

}  // namespace w2a8
