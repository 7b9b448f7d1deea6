// Device-side pieces of the block quantiser shared by the quantiser kernel and by the attention
// kernels that quantise probabilities and score gradients in registers.
#pragma once
#include <cstdint>

#include "sm100_ptx.cuh"

namespace attnfp8 {

// Scale of one block of 32 values with maximum magnitude `amax`: the smallest power of two 2^e
// with amax * 2^-e <= 448 (448 = 1.75 * 2^8, so e = E - 8, one more when the mantissa of amax
// exceeds 1.75).  Returns the stored byte e + 127 (0 for an all-zero block) and the exact
// multiplier 2^-e.
__device__ __forceinline__ void block_scale(float amax, uint32_t& byte, float& inv) {
  // adding 0x1FFFFF to the bit pattern carries into the exponent field exactly when the mantissa
  // exceeds 1.75; biased exponents below 8 (zero and subnormal maxima included) clamp to byte 0;
  // a non-finite maximum takes the largest scale
  const uint32_t bits = __float_as_uint(amax);
  int eb = max(static_cast<int>((bits + 0x1FFFFFu) >> 23) - 8, 0);
  eb = bits >= 0x7F800000u ? 254 : eb;
  byte = static_cast<uint32_t>(eb);
  const int ib = 254 - eb;                     // biased exponent of 2^-e
  inv = ib > 0 ? __uint_as_float(static_cast<uint32_t>(ib) << 23) : __uint_as_float(0x00400000u);
}

// The same rule for a maximum known to be finite and non-negative (probabilities, score
// gradients), in five integer operations: adding 0x1FFFFF to the bit pattern carries into the
// exponent field exactly when the mantissa exceeds 1.75.  Maxima below 2^-119 (biased exponent
// under 8, zero included) give byte 0, as block_scale does.
__device__ __forceinline__ void block_scale_finite(float amax, uint32_t& byte, float& inv) {
  const int eb = max(static_cast<int>((__float_as_uint(amax) + 0x1FFFFFu) >> 23) - 8, 0);
  byte = static_cast<uint32_t>(eb);
  inv = __uint_as_float(static_cast<uint32_t>(254 - eb) << 23);
}

// Quantise 32 values held in registers: codes packed four per word (element 0 in the low byte)
// and the block's scale byte.
__device__ __forceinline__ uint32_t quantize_block32(const float* x, uint32_t* words) {
  float amax = 0.f;
#pragma unroll
  for (int i = 0; i < 32; ++i) amax = fmaxf(amax, fabsf(x[i]));
  uint32_t byte;
  float inv;
  block_scale_finite(amax, byte, inv);
  const float2 inv2 = make_float2(inv, inv);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float2 a = __fmul2_rn(make_float2(x[4 * i], x[4 * i + 1]), inv2);
    const float2 b = __fmul2_rn(make_float2(x[4 * i + 2], x[4 * i + 3]), inv2);
    words[i] = sm100::cvt_e4m3x4(a.x, a.y, b.x, b.y);
  }
  return byte;
}

// offset of (row r of a 128-row tile, block k of 4) inside a 512-byte scale tile
__device__ __forceinline__ int sf_tile_offset(int r, int k) { return (r & 31) * 16 + (r >> 5) * 4 + k; }

}  // namespace attnfp8
