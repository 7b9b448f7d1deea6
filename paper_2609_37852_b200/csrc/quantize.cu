// Block-scaling quantiser: E4M3 codes with one E8M0 scale per 32 consecutive elements, written
// in both orientations (blocks along channels; blocks along tokens, stored transposed).
//
// One CTA owns a tile of 128 tokens x d channels of one (batch, head) slab, so it owns whole
// 512-byte scale tiles of both orientations.  Pass 1 reads the tile from HBM once with 16-byte
// coalesced loads, quantises along channels (4 lanes share a block of 32) and parks the source
// tile in shared memory; pass 2 walks the parked tile along tokens.  Codes of the transposed
// copy are staged in shared memory so that they leave as full 128-byte rows.
#include <cuda_bf16.h>

#include "common.cuh"
#include "mxfp8_device.cuh"
#include "sm100_ptx.cuh"

namespace attnfp8 {
namespace {

constexpr int kTokens = 128;
constexpr int kThreads = 256;

__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ float to_f32(float x) { return x; }

template <typename T>
__global__ void __launch_bounds__(kThreads) quantize_kernel(const T* __restrict__ src, int N, int d,
                                                            uint8_t* __restrict__ row_codes,
                                                            uint8_t* __restrict__ row_scales,
                                                            uint8_t* __restrict__ col_codes,
                                                            uint8_t* __restrict__ col_scales) {
  extern __shared__ __align__(16) uint8_t smem[];
  const int pitch = d + 16 / static_cast<int>(sizeof(T)) * 1;       // elements; +16 bytes per row
  T* tile = reinterpret_cast<T*>(smem);
  const int n_ct = (d / 32 + 3) / 4;                                 // row-copy scale tiles of this CTA
  const int n_rt = (d + 127) / 128;                                  // col-copy scale tiles of this CTA
  uint8_t* s_row_sf = smem + static_cast<size_t>(kTokens) * pitch * sizeof(T);
  uint8_t* s_col_sf = s_row_sf + n_ct * 512;
  uint8_t* s_col_codes = s_col_sf + n_rt * 512;                      // [d][128 + 16]
  constexpr int kColPitch = kTokens + 16;

  const int tid = threadIdx.x;
  const int tok_tile = blockIdx.x;
  const size_t slab = blockIdx.y;
  const size_t tok0 = static_cast<size_t>(tok_tile) * kTokens;
  const T* g_src = src + (slab * N + tok0) * d;
  const bool want_row = row_codes != nullptr;
  const bool want_col = col_codes != nullptr;

  for (int i = tid; i < (n_ct + n_rt) * 512 / 4; i += kThreads) reinterpret_cast<uint32_t*>(s_row_sf)[i] = 0;
  __syncthreads();

  // ---- pass 1: rows.  8 elements per thread per step, 4 lanes per block of 32 channels.
  const int steps = kTokens * d / (8 * kThreads);
  for (int s = 0; s < steps; ++s) {
    const int ci = s * kThreads + tid;
    const int e0 = ci * 8;
    const int tok = e0 / d, ch = e0 - tok * d;
    float x[8];
    if constexpr (sizeof(T) == 2) {
      const uint4 raw = *reinterpret_cast<const uint4*>(g_src + e0);
      const __nv_bfloat16* h = reinterpret_cast<const __nv_bfloat16*>(&raw);
#pragma unroll
      for (int i = 0; i < 8; ++i) x[i] = to_f32(h[i]);
      if (want_col) *reinterpret_cast<uint4*>(tile + tok * pitch + ch) = raw;
    } else {
      const float4 a = *reinterpret_cast<const float4*>(g_src + e0);
      const float4 b = *reinterpret_cast<const float4*>(g_src + e0 + 4);
      x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
      if (want_col) {
        *reinterpret_cast<float4*>(tile + tok * pitch + ch) = a;
        *reinterpret_cast<float4*>(tile + tok * pitch + ch + 4) = b;
      }
    }
    if (want_row) {
      float amax = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(x[i]));
      amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
      amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
      uint32_t byte; float inv;
      block_scale(amax, byte, inv);
      uint2 codes;
      codes.x = sm100::cvt_e4m3x4(x[0] * inv, x[1] * inv, x[2] * inv, x[3] * inv);
      codes.y = sm100::cvt_e4m3x4(x[4] * inv, x[5] * inv, x[6] * inv, x[7] * inv);
      *reinterpret_cast<uint2*>(row_codes + (slab * N + tok0) * d + e0) = codes;
      if ((tid & 3) == 0) {
        const int blk = ch >> 5;
        s_row_sf[(blk >> 2) * 512 + sf_tile_offset(tok, blk & 3)] = static_cast<uint8_t>(byte);
      }
    }
  }
  __syncthreads();
  if (want_row) {
    uint8_t* g = row_scales + (slab * (N / kTokens) + tok_tile) * n_ct * 512;
    for (int i = tid; i < n_ct * 512 / 16; i += kThreads)
      reinterpret_cast<uint4*>(g)[i] = reinterpret_cast<const uint4*>(s_row_sf)[i];
  }
  if (!want_col) return;

  // ---- pass 2: columns.  One (channel, block of 32 tokens) per thread per step.
  for (int item = tid; item < d * 4; item += kThreads) {
    const int c = item % d, tb = item / d;
    float x[32];
    float amax = 0.f;
#pragma unroll
    for (int t = 0; t < 32; ++t) {
      x[t] = to_f32(tile[(tb * 32 + t) * pitch + c]);
      amax = fmaxf(amax, fabsf(x[t]));
    }
    uint32_t byte; float inv;
    block_scale(amax, byte, inv);
    uint32_t w[8];
#pragma unroll
    for (int t = 0; t < 8; ++t)
      w[t] = sm100::cvt_e4m3x4(x[4 * t] * inv, x[4 * t + 1] * inv, x[4 * t + 2] * inv, x[4 * t + 3] * inv);
    uint4* dst = reinterpret_cast<uint4*>(s_col_codes + c * kColPitch + tb * 32);
    dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
    dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
    s_col_sf[(c >> 7) * 512 + sf_tile_offset(c & 127, tb)] = static_cast<uint8_t>(byte);
  }
  __syncthreads();
  for (int i = tid; i < d * 8; i += kThreads) {
    const int c = i >> 3, chunk = i & 7;
    *reinterpret_cast<uint4*>(col_codes + (slab * d + c) * N + tok0 + chunk * 16) =
        *reinterpret_cast<const uint4*>(s_col_codes + c * kColPitch + chunk * 16);
  }
  for (int rt = 0; rt < n_rt; ++rt) {
    uint8_t* g = col_scales + ((slab * n_rt + rt) * (N / kTokens) + tok_tile) * 512;
    for (int i = tid; i < 512 / 16; i += kThreads)
      reinterpret_cast<uint4*>(g)[i] = reinterpret_cast<const uint4*>(s_col_sf + rt * 512)[i];
  }
}

template <typename T>
attn_status_t launch_t(const void* src, int B, int H, int N, int d, attn_qtensor_t out, cudaStream_t stream) {
  const int pitch = d + 16 / static_cast<int>(sizeof(T));
  const int n_ct = (d / 32 + 3) / 4, n_rt = (d + 127) / 128;
  const size_t smem = static_cast<size_t>(kTokens) * pitch * sizeof(T) + (n_ct + n_rt) * 512 +
                      static_cast<size_t>(d) * (kTokens + 16);
  cudaError_t e = cudaFuncSetAttribute(quantize_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(smem));
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "quantize: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  dim3 grid(N / kTokens, B * H);
  quantize_kernel<T><<<grid, kThreads, smem, stream>>>(static_cast<const T*>(src), N, d, out.row_codes,
                                                      out.row_scales, out.col_codes, out.col_scales);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "quantize: launch: %s", cudaGetErrorString(e));
  return ATTN_OK;
}

// BF16 mode: the operands are the tensors themselves, rounded to BF16, in both orientations.
// One CTA transposes a tile of 64 tokens x d channels through shared memory.
constexpr int kCopyTokens = 64;

template <typename T>
__global__ void __launch_bounds__(kThreads) bf16_copies_kernel(const T* __restrict__ src, int N, int d,
                                                               __nv_bfloat16* __restrict__ row_out,
                                                               __nv_bfloat16* __restrict__ col_out) {
  extern __shared__ __align__(16) uint8_t smem[];
  __nv_bfloat16* tile = reinterpret_cast<__nv_bfloat16*>(smem);       // [64][d + 2]
  const int pitch = d + 2;
  const size_t slab = blockIdx.y;
  const size_t tok0 = static_cast<size_t>(blockIdx.x) * kCopyTokens;
  const T* g_src = src + (slab * N + tok0) * d;
  for (int i = threadIdx.x; i < kCopyTokens * d / 2; i += kThreads) {
    const int e0 = 2 * i, tok = e0 / d, ch = e0 - tok * d;
    const __nv_bfloat162 v2 = __floats2bfloat162_rn(to_f32(g_src[e0]), to_f32(g_src[e0 + 1]));
    *reinterpret_cast<__nv_bfloat162*>(tile + tok * pitch + ch) = v2;
    if (row_out) *reinterpret_cast<__nv_bfloat162*>(row_out + (slab * N + tok0) * d + e0) = v2;
  }
  if (!col_out) return;
  __syncthreads();
  for (int i = threadIdx.x; i < d * (kCopyTokens / 2); i += kThreads) {
    const int c = i / (kCopyTokens / 2), tp = i % (kCopyTokens / 2);
    __nv_bfloat162 v2;
    v2.x = tile[(2 * tp) * pitch + c];
    v2.y = tile[(2 * tp + 1) * pitch + c];
    *reinterpret_cast<__nv_bfloat162*>(col_out + (slab * d + c) * N + tok0 + 2 * tp) = v2;
  }
}

template <typename T>
attn_status_t launch_copies_t(const void* src, int B, int H, int N, int d, void* row_out, void* col_out,
                              cudaStream_t stream) {
  const size_t smem = static_cast<size_t>(kCopyTokens) * (d + 2) * sizeof(__nv_bfloat16);
  dim3 grid(N / kCopyTokens, B * H);
  bf16_copies_kernel<T><<<grid, kThreads, smem, stream>>>(static_cast<const T*>(src), N, d,
                                                         static_cast<__nv_bfloat16*>(row_out),
                                                         static_cast<__nv_bfloat16*>(col_out));
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "bf16 copies: launch: %s", cudaGetErrorString(e));
  return ATTN_OK;
}

}  // namespace

attn_status_t launch_bf16_copies(const void* src, int src_dtype, int B, int H, int N, int d, void* row_out, void* col_out,
                                 cudaStream_t stream) {
  if (src_dtype == ATTN_SRC_BF16) return launch_copies_t<__nv_bfloat16>(src, B, H, N, d, row_out, col_out, stream);
  return launch_copies_t<float>(src, B, H, N, d, row_out, col_out, stream);
}

attn_status_t launch_quantize(const void* src, int src_dtype, int B, int H, int N, int d, attn_qtensor_t out,
                              cudaStream_t stream) {
  if (src_dtype == ATTN_SRC_BF16) return launch_t<__nv_bfloat16>(src, B, H, N, d, out, stream);
  return launch_t<float>(src, B, H, N, d, out, stream);
}

}  // namespace attnfp8
