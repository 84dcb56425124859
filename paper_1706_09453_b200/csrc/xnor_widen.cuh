// Widening of packed sign bits to the 4-bit float e2m1 (+1 = nibble 0x2, -1 = nibble 0xA,
// nothing = nibble 0x0; for activations that stand for (0,1): 1 = nibble 0x2, 0 = nibble 0x0), shared by the XNOR tensor-core kernels, and the constant of the
// float -> integer trick their epilogues use.
#pragma once

#include <stdint.h>

namespace bnn {

constexpr int kMagicBits = 0x4B400000;   // bits of 1.5 * 2^23: x + magic has the integer x in its low bits

// Four output words of one input word: nibble i of word t <- bit 4i + t.
__device__ __forceinline__ uint4 widen(uint32_t w) {
    return make_uint4(((w << 3) & 0x88888888u) ^ 0xAAAAAAAAu, ((w << 2) & 0x88888888u) ^ 0xAAAAAAAAu,
                      ((w << 1) & 0x88888888u) ^ 0xAAAAAAAAu, (w & 0x88888888u) ^ 0xAAAAAAAAu);
}
// The same with the nibbles of invalid positions (bit of `valid` clear) set to +0.
__device__ __forceinline__ uint4 widen_masked(uint32_t w, uint32_t valid) {
    uint4 o = widen(w);
    o.x &= (valid & 0x11111111u) * 15u;
    o.y &= ((valid >> 1) & 0x11111111u) * 15u;
    o.z &= ((valid >> 2) & 0x11111111u) * 15u;
    o.w &= ((valid >> 3) & 0x11111111u) * 15u;
    return o;
}

// Activations in (0,1): bit 1 -> nibble 0x2 (+1), bit 0 -> nibble 0x0 (+0).
__device__ __forceinline__ uint4 widen01(uint32_t w) {
    return make_uint4((w << 1) & 0x22222222u, w & 0x22222222u, (w >> 1) & 0x22222222u, (w >> 2) & 0x22222222u);
}
__device__ __forceinline__ uint4 widen01_masked(uint32_t w, uint32_t valid) { return widen01(w & valid); }

}  // namespace bnn
