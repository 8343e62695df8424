// Expansion of quantised cache codes to the bf16 values the attention sees: bf16(code * row scale),
// the product taken in fp32 and rounded once to bf16 (the paper's Discussion: a round trip
// bf16 -> intN -> bf16 of the stored rows).  Shared by the kernels that read code tiles.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace kvf {
namespace {

__device__ __forceinline__ uint32_t pack_bf16_pair(float lo, float hi) {
    __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&b);
}

// Four codes (one 32-bit word, each byte already offset by 128) -> two packed bf16 pairs of
// bf16(code * scale): byte i dropped into the mantissa of 2^23 gives 2^23 + code + 128 exactly.
__device__ __forceinline__ void expand4(uint32_t x, float2 sc, uint32_t &lo, uint32_t &hi) {
    const float2 off = make_float2(-8388736.f, -8388736.f);
    float2 a = make_float2(__uint_as_float(__byte_perm(x, 0x4B000000u, 0x7650)), __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7651)));
    float2 b = make_float2(__uint_as_float(__byte_perm(x, 0x4B000000u, 0x7652)), __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7653)));
    a = __fmul2_rn(__fadd2_rn(a, off), sc);
    b = __fmul2_rn(__fadd2_rn(b, off), sc);
    lo = pack_bf16_pair(a.x, a.y);
    hi = pack_bf16_pair(b.x, b.y);
}

// Eight 4-bit codes (one 32-bit word, each nibble = code + 8, element 2i in the low nibble of byte i)
// -> four packed bf16 pairs of bf16(code * scale), in element order.
__device__ __forceinline__ void expand8(uint32_t w, float2 sc, uint32_t (&o)[4]) {
    const float2 off = make_float2(-8388616.f, -8388616.f);      // 2^23 + 8
    const uint32_t lo = w & 0x0F0F0F0Fu, hi = (w >> 4) & 0x0F0F0F0Fu;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 a = make_float2(__uint_as_float(__byte_perm(lo, 0x4B000000u, 0x7650 + i)),
                               __uint_as_float(__byte_perm(hi, 0x4B000000u, 0x7650 + i)));
        a = __fmul2_rn(__fadd2_rn(a, off), sc);
        o[i] = pack_bf16_pair(a.x, a.y);
    }
}


}  // namespace
}  // namespace kvf
