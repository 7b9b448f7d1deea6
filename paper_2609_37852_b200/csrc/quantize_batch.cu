// Block-scaling quantiser: E4M3 codes with one E8M0 scale per 32 consecutive elements, written
// in both orientations (blocks along channels; blocks along tokens, stored transposed), for one
// tensor or for several in one launch (the four operands of a step: Q, K, V, dO).
//
// The tiles (128 tokens x d channels, contiguous in the source) of all tensors form one list.  A
// persistent grid (two CTAs per SM) walks it; each CTA keeps a ring of two source tiles in shared
// memory (one where two would cost the second CTA), filled by bulk asynchronous copies (one
// instruction per tile, completion counted on an mbarrier), so that the next tile is in flight
// while the current one is quantised: the short tails and ramps of four separate launches
// disappear and every SM always has loads outstanding.
// Pass 1 walks the tile along channels (row copy), pass 2 along tokens (column copy, staged in
// shared memory so that it leaves as full 128-byte rows).
#include <cuda_bf16.h>

#include "common.cuh"
#include "mxfp8_device.cuh"
#include "sm100_ptx.cuh"

namespace attnfp8 {
namespace {

using namespace sm100;

constexpr int kTokens = 128;
constexpr int kThreads = 256;
constexpr int kMaxRing = 2;
constexpr int kColPitch = kTokens + 16;

struct BatchJob {
  const void* src;
  uint8_t *row_codes, *row_scales, *col_codes, *col_scales;
  int N, d;
  int first_tile;        // index of this tensor's first tile in the list
};

struct BatchParams {
  BatchJob job[ATTN_QUANTIZE_MAX_JOBS];
  int n_jobs;
  int total_tiles;
  int d_max;
  int ring;              // source tiles a CTA keeps in shared memory (1 or 2)
  int* status;
};

// |a| max |b| per 16-bit lane; a NaN lane yields the other operand, as fmaxf does
__device__ __forceinline__ __nv_bfloat162 absmax2(__nv_bfloat162 acc, uint32_t raw) {
  return __hmax2(acc, __habs2(*reinterpret_cast<const __nv_bfloat162*>(&raw)));
}
// the two BF16 values of a word as FP32 (exact)
__device__ __forceinline__ float2 unpack_bf16x2(uint32_t raw) {
  return make_float2(__uint_as_float(raw << 16), __uint_as_float(raw & 0xFFFF0000u));
}

// Both passes over one source tile in shared memory ([128 tokens][d], unpadded).  kD is the head
// dim when it is one of the built ones (0: use the run-time value).
template <typename T, int kD>
__device__ __forceinline__ void quantize_tile(const T* tile, int d_rt, const BatchJob& job, size_t slab, size_t tok0,
                                              uint8_t* s_row_sf, uint8_t* s_col_sf, uint8_t* s_col_codes, int tid) {
  const int d = kD ? kD : d_rt;
  const int N = job.N;
  // ---- pass 1: rows.  8 elements per thread per step, 4 lanes per block of 32 channels.
  if (job.row_codes != nullptr) {
    uint8_t* g_codes = job.row_codes + (slab * N + tok0) * d;
    const int steps = kTokens * d / (8 * kThreads);
#pragma unroll 4
    for (int s = 0; s < steps; ++s) {
      const int e0 = (s * kThreads + tid) * 8;
      const int tok = e0 / d, ch = e0 - tok * d;
      float amax;
      float2 v[4];
      if constexpr (sizeof(T) == 2) {
        const uint4 raw = *reinterpret_cast<const uint4*>(tile + e0);
        __nv_bfloat162 m = __float2bfloat162_rn(0.f);
        m = absmax2(m, raw.x); m = absmax2(m, raw.y); m = absmax2(m, raw.z); m = absmax2(m, raw.w);
        amax = fmaxf(__low2float(m), __high2float(m));
        v[0] = unpack_bf16x2(raw.x); v[1] = unpack_bf16x2(raw.y); v[2] = unpack_bf16x2(raw.z); v[3] = unpack_bf16x2(raw.w);
      } else {
        const float4 a = *reinterpret_cast<const float4*>(tile + e0);
        const float4 b = *reinterpret_cast<const float4*>(tile + e0 + 4);
        v[0] = make_float2(a.x, a.y); v[1] = make_float2(a.z, a.w); v[2] = make_float2(b.x, b.y); v[3] = make_float2(b.z, b.w);
        amax = 0.f;
#pragma unroll
        for (int k = 0; k < 4; ++k) amax = fmaxf(amax, fmaxf(fabsf(v[k].x), fabsf(v[k].y)));
      }
      amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
      amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
      uint32_t byte; float inv;
      block_scale(amax, byte, inv);
      const float2 inv2 = make_float2(inv, inv);
#pragma unroll
      for (int k = 0; k < 4; ++k) v[k] = __fmul2_rn(v[k], inv2);
      uint2 codes;
      codes.x = cvt_e4m3x4(v[0].x, v[0].y, v[1].x, v[1].y);
      codes.y = cvt_e4m3x4(v[2].x, v[2].y, v[3].x, v[3].y);
      *reinterpret_cast<uint2*>(g_codes + e0) = codes;
      if ((tid & 3) == 0) {
        const int blk = ch >> 5;
        s_row_sf[(blk >> 2) * 512 + sf_tile_offset(tok, blk & 3)] = static_cast<uint8_t>(byte);
      }
    }
  }
  // ---- pass 2: columns.
  if (job.col_codes != nullptr) {
    if constexpr (sizeof(T) == 2) {
      // one pair of neighbouring channels x one block of 32 tokens per thread and step: 32-bit
      // loads, packed maxima
      const int pairs = d >> 1;
      for (int item = tid; item < pairs * 4; item += kThreads) {
        const int c = (item % pairs) * 2, tb = item / pairs;
        const uint32_t* col = reinterpret_cast<const uint32_t*>(tile + tb * 32 * d + c);
        uint32_t raw[32];
        __nv_bfloat162 m = __float2bfloat162_rn(0.f);
#pragma unroll
        for (int t = 0; t < 32; ++t) {
          raw[t] = col[t * pairs];
          m = absmax2(m, raw[t]);
        }
        uint32_t byte_lo, byte_hi;
        float2 inv2;
        block_scale(__low2float(m), byte_lo, inv2.x);
        block_scale(__high2float(m), byte_hi, inv2.y);
        uint32_t w_lo[8], w_hi[8];
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          const float2 a = __fmul2_rn(unpack_bf16x2(raw[4 * t]), inv2), b = __fmul2_rn(unpack_bf16x2(raw[4 * t + 1]), inv2);
          const float2 e = __fmul2_rn(unpack_bf16x2(raw[4 * t + 2]), inv2), f = __fmul2_rn(unpack_bf16x2(raw[4 * t + 3]), inv2);
          w_lo[t] = cvt_e4m3x4(a.x, b.x, e.x, f.x);
          w_hi[t] = cvt_e4m3x4(a.y, b.y, e.y, f.y);
        }
        uint4* dst = reinterpret_cast<uint4*>(s_col_codes + c * kColPitch + tb * 32);
        dst[0] = make_uint4(w_lo[0], w_lo[1], w_lo[2], w_lo[3]);
        dst[1] = make_uint4(w_lo[4], w_lo[5], w_lo[6], w_lo[7]);
        dst = reinterpret_cast<uint4*>(s_col_codes + (c + 1) * kColPitch + tb * 32);
        dst[0] = make_uint4(w_hi[0], w_hi[1], w_hi[2], w_hi[3]);
        dst[1] = make_uint4(w_hi[4], w_hi[5], w_hi[6], w_hi[7]);
        s_col_sf[(c >> 7) * 512 + sf_tile_offset(c & 127, tb)] = static_cast<uint8_t>(byte_lo);
        s_col_sf[(c >> 7) * 512 + sf_tile_offset((c + 1) & 127, tb)] = static_cast<uint8_t>(byte_hi);
      }
    } else {
      // one (channel, block of 32 tokens) per thread and step
      for (int item = tid; item < d * 4; item += kThreads) {
        const int c = item % d, tb = item / d;
        float x[32];
        float amax = 0.f;
#pragma unroll
        for (int t = 0; t < 32; ++t) {
          x[t] = tile[(tb * 32 + t) * d + c];
          amax = fmaxf(amax, fabsf(x[t]));
        }
        uint32_t byte; float inv;
        block_scale(amax, byte, inv);
        uint32_t w[8];
#pragma unroll
        for (int t = 0; t < 8; ++t)
          w[t] = cvt_e4m3x4(x[4 * t] * inv, x[4 * t + 1] * inv, x[4 * t + 2] * inv, x[4 * t + 3] * inv);
        uint4* dst = reinterpret_cast<uint4*>(s_col_codes + c * kColPitch + tb * 32);
        dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
        dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
        s_col_sf[(c >> 7) * 512 + sf_tile_offset(c & 127, tb)] = static_cast<uint8_t>(byte);
      }
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(kThreads, 2) quantize_batch_kernel(const __grid_constant__ BatchParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int tile_bytes_max = kTokens * p.d_max * static_cast<int>(sizeof(T));
  auto ring = [&](int slot) { return reinterpret_cast<T*>(smem + slot * tile_bytes_max); };
  const int n_ring = p.ring;
  const int n_ct_max = (p.d_max / 32 + 3) / 4, n_rt_max = (p.d_max + 127) / 128;
  uint8_t* s_row_sf = smem + n_ring * tile_bytes_max;
  uint8_t* s_col_sf = s_row_sf + n_ct_max * 512;
  uint8_t* s_col_codes = s_col_sf + n_rt_max * 512;                  // [d][128 + 16]
  uint64_t* full = reinterpret_cast<uint64_t*>(s_col_codes + p.d_max * kColPitch);
  int* abort_flag = reinterpret_cast<int*>(full + kMaxRing);

  const int tid = threadIdx.x;
  const int my_tiles = (p.total_tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) /
                       static_cast<int>(gridDim.x);

  // tile index -> (tensor, slab, token tile); the copy of a tile is one contiguous range
  auto locate = [&](int tile, int& j, int& local) {
    j = 0;
#pragma unroll
    for (int i = 1; i < ATTN_QUANTIZE_MAX_JOBS; ++i)
      if (i < p.n_jobs && tile >= p.job[i].first_tile) j = i;
    local = tile - p.job[j].first_tile;
  };
  auto issue = [&](int i) {        // thread 0: request the i-th tile of this CTA into its ring slot
    int j, local;
    locate(static_cast<int>(blockIdx.x) + i * static_cast<int>(gridDim.x), j, local);
    const uint32_t bytes = static_cast<uint32_t>(kTokens * p.job[j].d * sizeof(T));
    const uint8_t* g = static_cast<const uint8_t*>(p.job[j].src) + static_cast<size_t>(local) * bytes;
    mbar_arrive_expect_tx(&full[i % n_ring], bytes);
    bulk_load_1d(ring(i % n_ring), g, bytes, &full[i % n_ring]);
  };

  if (tid == 0) {
    for (int s = 0; s < n_ring; ++s) mbar_init(&full[s], 1);
    *abort_flag = 0;
    fence_mbar_init();
    for (int i = 0; i < n_ring && i < my_tiles; ++i) issue(i);
  }
  __syncthreads();

  for (int i = 0; i < my_tiles; ++i) {
    int j, local;
    locate(static_cast<int>(blockIdx.x) + i * static_cast<int>(gridDim.x), j, local);
    const BatchJob& job = p.job[j];
    const int N = job.N, d = job.d;
    const int tiles_per_slab = N / kTokens;
    const size_t slab = static_cast<size_t>(local / tiles_per_slab);
    const int tok_tile = local % tiles_per_slab;
    const size_t tok0 = static_cast<size_t>(tok_tile) * kTokens;
    const int n_ct = (d / 32 + 3) / 4, n_rt = (d + 127) / 128;
    const bool want_row = job.row_codes != nullptr, want_col = job.col_codes != nullptr;
    const T* tile = ring(i % n_ring);

    for (int w = tid; w < (n_ct_max + n_rt_max) * 512 / 4; w += kThreads) reinterpret_cast<uint32_t*>(s_row_sf)[w] = 0;
    // bounded wait: a copy that never lands ends the CTA with the time-out status, not a hang
    const bool landed = mbar_wait(&full[i % n_ring], (i / n_ring) & 1, abort_flag);
    if (__syncthreads_or(!landed)) break;        // all threads take the same way out

    switch (d) {                      // compile-time head dims: no integer division, constant strides
      case 64:  quantize_tile<T, 64>(tile, d, job, slab, tok0, s_row_sf, s_col_sf, s_col_codes, tid); break;
      case 128: quantize_tile<T, 128>(tile, d, job, slab, tok0, s_row_sf, s_col_sf, s_col_codes, tid); break;
      case 192: quantize_tile<T, 192>(tile, d, job, slab, tok0, s_row_sf, s_col_sf, s_col_codes, tid); break;
      case 256: quantize_tile<T, 256>(tile, d, job, slab, tok0, s_row_sf, s_col_sf, s_col_codes, tid); break;
      default:  quantize_tile<T, 0>(tile, d, job, slab, tok0, s_row_sf, s_col_sf, s_col_codes, tid); break;
    }
    __syncthreads();
    // the source tile is consumed: refill its slot while the staged outputs leave
    if (tid == 0 && i + n_ring < my_tiles) {
      fence_proxy_async_smem();
      issue(i + n_ring);
    }
    if (want_row) {
      uint8_t* g = job.row_scales + (slab * tiles_per_slab + tok_tile) * n_ct * 512;
      for (int w = tid; w < n_ct * 512 / 16; w += kThreads)
        reinterpret_cast<uint4*>(g)[w] = reinterpret_cast<const uint4*>(s_row_sf)[w];
    }
    if (want_col) {
      for (int w = tid; w < d * 8; w += kThreads) {
        const int c = w >> 3, chunk = w & 7;
        *reinterpret_cast<uint4*>(job.col_codes + (slab * d + c) * N + tok0 + chunk * 16) =
            *reinterpret_cast<const uint4*>(s_col_codes + c * kColPitch + chunk * 16);
      }
      for (int rt = 0; rt < n_rt; ++rt) {
        uint8_t* g = job.col_scales + ((slab * n_rt + rt) * tiles_per_slab + tok_tile) * 512;
        for (int w = tid; w < 512 / 16; w += kThreads)
          reinterpret_cast<uint4*>(g)[w] = reinterpret_cast<const uint4*>(s_col_sf + rt * 512)[w];
      }
    }
    __syncthreads();                 // staging buffers free for the next tile
  }
  if (tid == 0 && *abort_flag) atomicExch(p.status, static_cast<int>(ATTN_ERR_TIMEOUT));
}

static size_t batch_smem_bytes(size_t elem, int d_max, int ring) {
  const int n_ct = (d_max / 32 + 3) / 4, n_rt = (d_max + 127) / 128;
  return ring * static_cast<size_t>(kTokens) * d_max * elem + (n_ct + n_rt) * 512 +
         static_cast<size_t>(d_max) * kColPitch + 64;
}

template <typename T>
attn_status_t launch_batch_t(BatchParams& p, cudaStream_t stream) {
  // two CTAs per SM come first (each covers the other's stalls), the deeper ring second: measured
  // at d = 192 one tile x two CTAs 0.078 ms against two tiles x one CTA 0.098 ms
  const size_t half_sm = 113 * 1024, whole_sm = 227 * 1024;
  if (batch_smem_bytes(sizeof(T), p.d_max, kMaxRing) <= half_sm) p.ring = kMaxRing;
  else if (batch_smem_bytes(sizeof(T), p.d_max, 1) <= half_sm) p.ring = 1;
  else p.ring = batch_smem_bytes(sizeof(T), p.d_max, kMaxRing) <= whole_sm ? kMaxRing : 1;
  const size_t smem = batch_smem_bytes(sizeof(T), p.d_max, p.ring);
  cudaError_t e = cudaFuncSetAttribute(quantize_batch_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(smem));
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "quantize: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  int dev = 0, sms = 0, per_sm = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, quantize_batch_kernel<T>, kThreads, smem);
  if (e != cudaSuccess || per_sm < 1 || sms < 1)
    return fail(ATTN_ERR_CUDA, "quantize: occupancy query: %s", cudaGetErrorString(e));
  const int resident = sms * per_sm;
  const int grid = p.total_tiles < resident ? p.total_tiles : resident;
  quantize_batch_kernel<T><<<grid, kThreads, smem, stream>>>(p);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "quantize: launch: %s", cudaGetErrorString(e));
  return ATTN_OK;
}

}  // namespace

attn_status_t launch_quantize_batch(const attn_quantize_job_t* jobs, int n_jobs, int* status, cudaStream_t stream) {
  BatchParams p = {};
  p.n_jobs = n_jobs;
  p.status = status;
  int tiles = 0, d_max = 0;
  for (int j = 0; j < n_jobs; ++j) {
    const attn_quantize_job_t& in = jobs[j];
    BatchJob& b = p.job[j];
    b.src = in.src;
    b.row_codes = in.out.row_codes; b.row_scales = in.out.row_scales;
    b.col_codes = in.out.col_codes; b.col_scales = in.out.col_scales;
    b.N = in.N; b.d = in.d;
    b.first_tile = tiles;
    tiles += in.B * in.H * (in.N / kTokens);
    d_max = in.d > d_max ? in.d : d_max;
  }
  p.total_tiles = tiles;
  p.d_max = d_max;
  if (jobs[0].src_dtype == ATTN_SRC_BF16) return launch_batch_t<__nv_bfloat16>(p, stream);
  return launch_batch_t<float>(p, stream);
}

}  // namespace attnfp8
