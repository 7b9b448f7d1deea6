// Issue loops shared by the attention kernels.  The issuing warps share their schedulers with the
// arithmetic warps, and every extra instruction between two tcgen05.mma delays the tensor pipe, so
// the loops are unrolled at compile time: chunk offsets, scale-factor ids and instruction
// descriptors become immediates and only the trip-count guard stays at run time.
#pragma once
#include "sm100_ptx.cuh"

namespace sm100 {

// D[128 x kN] = A * B^T with both operands in shared memory, K-major, stored as 128-byte-wide
// swizzled chunks (kAChunk16 / kBChunk16: distance between chunks in 16-byte units).  `nk` is the
// number of 32-byte K steps actually present (<= 4 * kChunks).  FP8: step kb takes scale byte
// kb % 4 of the scale columns sfa + 4 * (kb / 4) and sfb + 4 * (kb / 4).
template <bool kFp8, int kChunks, int kN, int kAChunk16, int kBChunk16>
__device__ __forceinline__ void issue_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, int nk, uint32_t sfa,
                                         uint32_t sfb) {
#pragma unroll
  for (int kb = 0; kb < 4 * kChunks; ++kb) {
    if (kb < nk) {
      const int c = kb >> 2, w = kb & 3;
      const uint64_t a = a_desc + (c * kAChunk16 + 2 * w), b = b_desc + (c * kBChunk16 + 2 * w);
      if (kFp8)
        mma_mxf8_ss_elect(d_tmem, a, b, make_idesc_mxf8(128, kN, w, w), sfa + 4 * c, sfb + 4 * c, kb > 0);
      else
        mma_bf16_ss_elect(d_tmem, a, b, make_idesc_bf16(128, kN), kb > 0);
    }
  }
}

// D[128 x n] += A * B^T with A (64 tokens of quantised probabilities or score gradients) in tensor
// memory and B a [n x 128-byte] chunk in shared memory whose rows are taken kRows x 128 at a time
// (`n_total` rows in all; D and the B scale columns advance by 128 and 4 per row tile).  The 64
// tokens are 2 * kEB steps of 32 bytes starting at step 2 * sub of the chunk.  `acc` = accumulate
// into D already on the first step.
template <bool kFp8, int kEB, int kRows>
__device__ __forceinline__ void issue_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, int n_total, int sub,
                                         uint32_t sfa, uint32_t sfb, bool acc) {
  const uint64_t b_sub = b_desc + 4 * sub;
#pragma unroll
  for (int r = 0; r < kRows; ++r) {
    const int n = (r + 1 < kRows) ? 128 : n_total - 128 * r;
    if (r == 0 || n > 0) {
#pragma unroll
      for (int kb = 0; kb < 2 * kEB; ++kb) {
        const uint64_t b = b_sub + (r * (128 * 128 / 16) + 2 * kb);
        if (kFp8)
          mma_mxf8_ts_elect(d_tmem + 128 * r, a_tmem + 8 * kb, b,
                            make_idesc_mxf8(128, n, kb, 0) + (static_cast<uint32_t>(2 * sub + kb) << 4), sfa,
                            sfb + 4 * r, acc || kb > 0);
        else
          mma_bf16_ts_elect(d_tmem + 128 * r, a_tmem + 8 * kb, b, make_idesc_bf16(128, n), acc || kb > 0);
      }
    }
  }
}

// Copies kTiles consecutive 512-byte scale tiles from shared memory into tensor memory (4 columns each).
template <int kTiles>
__device__ __forceinline__ void sf_copy_tiles(uint32_t tmem_dst, const uint8_t* smem_src) {
  const uint64_t d = make_desc_sf(smem_u32(smem_src));
#pragma unroll
  for (int c = 0; c < kTiles; ++c) sf_copy_elect(tmem_dst + 4 * c, d + c * (512 / 16));
}

}  // namespace sm100
