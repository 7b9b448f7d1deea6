// The quantiser with the operand producer fused in front (rotary embedding, key centering, scale
// folding), the token-mean kernel it needs, and the operand copies of BF16 mode.  The plain
// quantiser (no producer steps) lives in quantize_batch.cu.
//
// One CTA owns a tile of 128 tokens x d channels of one (batch, head) slab, so it owns whole
// 512-byte scale tiles of both orientations.  Pass 1 reads the tile from HBM once with 16-byte
// coalesced loads, applies the producer steps in FP32, quantises along channels (4 lanes share a
// block of 32) and parks the FP32 values in shared memory; pass 2 walks the parked tile along
// tokens.  Codes of the transposed copy are staged in shared memory so that they leave as full
// 128-byte rows.
#include <cuda_bf16.h>

#include <type_traits>

#include "common.cuh"
#include "mxfp8_device.cuh"
#include "sm100_ptx.cuh"

namespace attnfp8 {
namespace {

constexpr int kTokens = 128;
constexpr int kThreads = 256;

__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ float to_f32(float x) { return x; }

// Producer steps fused in front of the quantiser (paper Appendix "Operands, Scaling, and
// Accumulation"): rotary embedding in FP32 with the rotated channels rounded to BF16, subtraction
// of the FP32 token mean (key centering), FP32 multiplication by a scale (tau folded into Q).
struct Producer {
  const float* cos;     // [N, d/2] or nullptr
  const float* sin;
  const float* mean;    // [B*H, d] or nullptr
  float scale;
  int use_scale;
};

// One rotated channel: x*cos -+ partner*sin with one rounding for the product and a fused
// multiply-add, then BF16 (the order the header of attn_fp8_quantize_fused states).
__device__ __forceinline__ float rotate_bf16(float x, float partner, float c, float s, bool upper) {
  const float t = __fmul_rn(partner, s);
  const float r = __fmaf_rn(x, c, upper ? t : -t);
  return __bfloat162float(__float2bfloat16_rn(r));
}

template <typename T>
__global__ void __launch_bounds__(kThreads) quantize_fused_kernel(const T* __restrict__ src, int N, int d,
                                                            uint8_t* __restrict__ row_codes,
                                                            uint8_t* __restrict__ row_scales,
                                                            uint8_t* __restrict__ col_codes,
                                                            uint8_t* __restrict__ col_scales, const Producer prod) {
  extern __shared__ __align__(16) uint8_t smem[];
  using TT = float;                                                  // what the parked tile holds
  const int pitch = d + 16 / static_cast<int>(sizeof(TT)) * 1;      // elements; +16 bytes per row
  TT* tile = reinterpret_cast<TT*>(smem);
  const int n_ct = (d / 32 + 3) / 4;                                 // row-copy scale tiles of this CTA
  const int n_rt = (d + 127) / 128;                                  // col-copy scale tiles of this CTA
  uint8_t* s_row_sf = smem + static_cast<size_t>(kTokens) * pitch * sizeof(TT);
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
  // unrolled so that the loads of several steps are in flight together (a CTA is short-lived:
  // the latency of its own loads is most of its life)
#pragma unroll 8
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
    } else {
      const float4 a = *reinterpret_cast<const float4*>(g_src + e0);
      const float4 b = *reinterpret_cast<const float4*>(g_src + e0 + 4);
      x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
    }
    {
      if (prod.cos != nullptr) {
        const int half = d >> 1;
        const bool upper = ch >= half;
        const int pc = upper ? ch - half : ch;                       // pair index; 8 consecutive pairs per thread
        const T* g_partner = g_src + e0 + (upper ? -half : half);
        const size_t tab = (tok0 + tok) * half + pc;
#pragma unroll
        for (int i = 0; i < 8; ++i)
          x[i] = rotate_bf16(x[i], to_f32(g_partner[i]), prod.cos[tab + i], prod.sin[tab + i], upper);
      }
      if (prod.mean != nullptr) {
#pragma unroll
        for (int i = 0; i < 8; ++i) x[i] = __fsub_rn(x[i], prod.mean[slab * d + ch + i]);
      }
      if (prod.use_scale) {
#pragma unroll
        for (int i = 0; i < 8; ++i) x[i] = __fmul_rn(x[i], prod.scale);
      }
      if (want_col) {
        *reinterpret_cast<float4*>(tile + tok * pitch + ch) = make_float4(x[0], x[1], x[2], x[3]);
        *reinterpret_cast<float4*>(tile + tok * pitch + ch + 4) = make_float4(x[4], x[5], x[6], x[7]);
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
attn_status_t launch_t(const void* src, int B, int H, int N, int d, attn_qtensor_t out, const Producer& prod,
                       cudaStream_t stream) {
  const int tile_elem = 4;                                           // the parked tile is FP32
  const int pitch = d + 16 / tile_elem;
  const int n_ct = (d / 32 + 3) / 4, n_rt = (d + 127) / 128;
  const size_t smem = static_cast<size_t>(kTokens) * pitch * tile_elem + (n_ct + n_rt) * 512 +
                      static_cast<size_t>(d) * (kTokens + 16);
  cudaError_t e = cudaFuncSetAttribute(quantize_fused_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(smem));
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "quantize: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  dim3 grid(N / kTokens, B * H);
  quantize_fused_kernel<T><<<grid, kThreads, smem, stream>>>(static_cast<const T*>(src), N, d, out.row_codes,
                                                              out.row_scales, out.col_codes, out.col_scales, prod);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "quantize: launch: %s", cudaGetErrorString(e));
  return ATTN_OK;
}

// FP32 mean over tokens of the (rotated, BF16-rounded) tensor, per (batch, head, channel).  The
// terms are BF16 values, so a double-precision sum is exact whatever its order, and the result is
// the correctly rounded quotient: bitwise reproducible.  One CTA per (batch, head).
constexpr int kMeanThreads = 1024;

template <typename T>
__global__ void __launch_bounds__(kMeanThreads) token_mean_kernel(const T* __restrict__ src, int N, int d,
                                                                  const float* __restrict__ cos,
                                                                  const float* __restrict__ sin,
                                                                  float* __restrict__ mean) {
  extern __shared__ __align__(16) uint8_t smem[];
  double* part = reinterpret_cast<double*>(smem);                   // [phases][d]
  const int half = d >> 1;
  const int phases = kMeanThreads / half;
  const int pc = threadIdx.x % half, ph = threadIdx.x / half;
  const size_t slab = blockIdx.x;
  const T* g = src + slab * N * d;
  double a1 = 0.0, a2 = 0.0;
  if (ph < phases) {
    for (int n = ph; n < N; n += phases) {
      float x1 = to_f32(g[static_cast<size_t>(n) * d + pc]), x2 = to_f32(g[static_cast<size_t>(n) * d + half + pc]);
      if (cos != nullptr) {
        const float c = cos[static_cast<size_t>(n) * half + pc], s = sin[static_cast<size_t>(n) * half + pc];
        const float r1 = rotate_bf16(x1, x2, c, s, false), r2 = rotate_bf16(x2, x1, c, s, true);
        x1 = r1; x2 = r2;
      }
      a1 += static_cast<double>(x1);
      a2 += static_cast<double>(x2);
    }
    part[ph * d + pc] = a1;
    part[ph * d + half + pc] = a2;
  }
  __syncthreads();
  for (int c = threadIdx.x; c < d; c += kMeanThreads) {
    double sum = 0.0;
    for (int i = 0; i < phases; ++i) sum += part[i * d + c];
    mean[slab * d + c] = static_cast<float>(sum / static_cast<double>(N));
  }
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

attn_status_t launch_quantize_fused(const void* src, int src_dtype, int B, int H, int N, int d, const float* cos,
                                    const float* sin, float scale, float* mean, attn_qtensor_t out,
                                    cudaStream_t stream) {
  if (mean != nullptr) {
    const size_t smem = static_cast<size_t>(kMeanThreads / (d / 2)) * d * sizeof(double);
    if (src_dtype == ATTN_SRC_BF16)
      token_mean_kernel<__nv_bfloat16><<<B * H, kMeanThreads, smem, stream>>>(static_cast<const __nv_bfloat16*>(src), N, d, cos, sin, mean);
    else
      token_mean_kernel<float><<<B * H, kMeanThreads, smem, stream>>>(static_cast<const float*>(src), N, d, cos, sin, mean);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "token mean: launch: %s", cudaGetErrorString(e));
  }
  const Producer prod{cos, sin, mean, scale, scale != 1.f ? 1 : 0};
  if (src_dtype == ATTN_SRC_BF16) return launch_t<__nv_bfloat16>(src, B, H, N, d, out, prod, stream);
  return launch_t<float>(src, B, H, N, d, out, prod, stream);
}

}  // namespace attnfp8
