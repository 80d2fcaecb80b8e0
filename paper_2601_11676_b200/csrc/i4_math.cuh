// Unpacking of int4 codes (two per byte, nibble = code + 8) without converting a nibble on its own: nibbles k and k + 4
// of a 32-bit word are masked into the two halves of a register and OR-ed with 0x4300, which makes them the bf16
// numbers 128 + nibble; the offset 128 + 8 is taken off once per sum.
#pragma once
#include <stdint.h>

namespace halo {

constexpr float kNibbleBias = 136.0f;      // 128 from the bf16 trick + 8 from the code's zero point

__device__ __forceinline__ uint32_t nibble_pair_bf16(uint32_t word, int k) {
    return ((word >> (4 * k)) & 0x000F000Fu) | 0x43004300u;      // {128 + nibble k, 128 + nibble k+4} as bf16x2
}

// Mask and exponent bits as run-time values held in registers: with two immediates the "and, then or" is two logic
// instructions, with register operands it is one three-input instruction.
struct PairBits { uint32_t mask, magic; };
__device__ __forceinline__ uint32_t nibble_pair_r(uint32_t shifted_word, const PairBits& pb) {
    return (shifted_word & pb.mask) | pb.magic;
}

}  // namespace halo
