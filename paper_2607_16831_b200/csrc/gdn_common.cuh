// Shared device/host helpers of libgdn (internal; the public boundary is include/gdn.h).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gdn.h"

namespace gdn {

constexpr int kD = 128;      // dk = dv = 128 (the only supported head size)
constexpr int kChunk = 64;   // prefill chunk length

__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits16) {
    return __uint_as_float(bits16 << 16);
}

// Two packed bf16 (low half = element 0) -> two floats.
__device__ __forceinline__ void unpack_bf16x2(uint32_t w, float& lo, float& hi) {
    lo = __uint_as_float(w << 16);
    hi = __uint_as_float(w & 0xffff0000u);
}

// Round-to-nearest-even fp32 -> bf16 bits.
__device__ __forceinline__ uint16_t float_to_bf16_bits(float x) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(x));
}

// Two floats -> packed bf16x2 (element 0 in the low half), one conversion instruction.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// y0,y1 -> packed bf16 hi parts and packed bf16 of the remainders (y - hi): a two-term
// bf16 expansion carrying ~16 significant bits.
__device__ __forceinline__ void split_bf16x2(float y0, float y1, uint32_t& hi, uint32_t& lo) {
    hi = pack_bf16x2(y0, y1);
    const float h0 = __uint_as_float(hi << 16), h1 = __uint_as_float(hi & 0xffff0000u);
    lo = pack_bf16x2(y0 - h0, y1 - h1);
}

// Raw gate parameterisation (Section 3.2 of the paper, first two lines), evaluated in fp32:
//   log-decay g = -exp(A_log) * softplus(a + dt_bias),   beta = sigmoid(b).
__device__ __forceinline__ void raw_gates(float a, float b, float A_log, float dt_bias, float& g, float& beta) {
    const float x = a + dt_bias;
    const float sp = fmaxf(x, 0.f) + log1pf(__expf(-fabsf(x)));
    g = -__expf(A_log) * sp;
    beta = 1.f / (1.f + __expf(-b));
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace gdn
