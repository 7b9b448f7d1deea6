// Measurement aid: the rate at which the tensor cores of this device execute the block-scaled FP8
// instruction the attention kernels are built on (tcgen05.mma.kind::mxf8f6f4.block_scale, E4M3
// operands with E8M0 scales, M = 128, N = 224, K = 32 per instruction), with nothing else running.
// Two warps per CTA issue back to back from shared-memory operands into their own accumulators (one
// warp cannot issue fast enough to keep the pipe busy; at N = 128 the operand reads from shared
// memory, 8 KB per 64 tensor cycles, would be the limit instead of the tensor pipe), one CTA per SM.  The figure is the
// denominator "measured FP8 peak" of the benchmark's report; the paper has no counterpart.
#include <cuda_runtime.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace attnfp8 {
namespace {

using namespace sm100;

constexpr int kIssuers = 2;
constexpr int kN = 224;

__global__ void __launch_bounds__(128, 1) mma_peak_kernel(int reps, int* status) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* sA = smem_raw;                       // 128 rows x 128 bytes, swizzled layout (the values do not matter)
  uint8_t* sB = smem_raw + 16384;               // kN rows x 128 bytes (32 KB reserved)
  uint8_t* sSF = smem_raw + 49152;              // two 512-byte scale tiles
  __shared__ uint64_t bar[kIssuers];
  __shared__ uint32_t tmem_holder;
  __shared__ int abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5;
  if (smem_u32(smem_raw) & 1023u) {
    if (tid == 0) atomicExch(status, static_cast<int>(ATTN_ERR_ALIGNMENT));
    return;
  }
  for (int i = tid; i < 49152 / 4; i += 128) reinterpret_cast<uint32_t*>(smem_raw)[i] = 0x38383838u;   // E4M3 1.0
  for (int i = tid; i < 1024 / 4; i += 128) reinterpret_cast<uint32_t*>(sSF)[i] = 0x7f7f7f7fu;         // scale 2^0
  if (tid == 0) {
    for (int i = 0; i < kIssuers; ++i) mbar_init(&bar[i], 1);
    abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&tmem_holder, 512);
    tmem_relinquish();
  }
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_holder;
  if (warp < kIssuers) {
    const uint32_t sfa = tmem + 2 * kN + 16 * warp, sfb = sfa + 4;       // B: kN / 32 = 7 columns of two tiles
    sf_copy_elect(sfa, make_desc_sf(smem_u32(sSF)));
    sf_copy_elect(sfb, make_desc_sf(smem_u32(sSF)));
    sf_copy_elect(sfb + 4, make_desc_sf(smem_u32(sSF + 512)));
    const uint64_t da = make_desc_sw128(smem_u32(sA)), db = make_desc_sw128(smem_u32(sB));
    const uint32_t acc = tmem + kN * warp;
    for (int r = 0; r < reps; r += 4) {
#pragma unroll
      for (int kb = 0; kb < 4; ++kb)
        mma_mxf8_ss_elect(acc, da + 2 * kb, db + 2 * kb, make_idesc_mxf8(128, kN, kb, kb), sfa, sfb, (r > 0 || kb > 0));
    }
    mma_commit_elect(&bar[warp]);
    mbar_wait(&bar[warp], 0, &abort_flag);
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
  if (tid == 0 && abort_flag) atomicExch(status, static_cast<int>(ATTN_ERR_TIMEOUT));
}

// What the FP32 reduction of dQ would cost in a merged key-major gradient pass (the shape the paper's
// Limitations name as open engineering: one pass that forms dS once and produces dQ, dK and dV): every
// (key tile of 128, query sub-tile of 64) pair of the workload adds a [64 x dqk] FP32 partial into an FP32
// dQ of the whole problem.  This kernel issues exactly those adds (red.global.add.v4.f32, the partial is
// all ones) and nothing else, one CTA per (KV head, key tile, batch) in the order the key-major kernel
// uses; the result is checkable (element (h, i, c) ends up as the number of key tiles row i sees).
__global__ void __launch_bounds__(256, 1) dq_reduction_kernel(float* dq, int N, int Hq, int Hkv, int dqk, int causal) {
  const int jt = blockIdx.y, g = blockIdx.x, b = blockIdx.z, G = Hq / Hkv, tiles = N / 128;
  for (int h = g * G; h < (g + 1) * G; ++h)
    for (int it = causal ? jt : 0; it < tiles; ++it)
      for (int half = 0; half < 2; ++half) {
        float* dst = dq + (static_cast<size_t>(b * Hq + h) * N + it * 128 + half * 64) * dqk;
        for (int e = threadIdx.x * 4; e < 64 * dqk; e += 256 * 4)
          asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + e), "f"(1.f), "f"(1.f), "f"(1.f), "f"(1.f) : "memory");
      }
}

}  // namespace

attn_status_t measure_mma_peak(double* tflops_out, int* status, cudaStream_t stream) {
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess || sms < 1) return fail(ATTN_ERR_CUDA, "mma peak: SM count: %s", cudaGetErrorString(e));
  const int smem = 49152 + 1024;
  const int reps = 16384;                       // per issuing warp: ~3 ms at the nominal rate
  e = cudaFuncSetAttribute(mma_peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "mma peak: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  e = cudaEventCreate(&e0);
  if (e == cudaSuccess) e = cudaEventCreate(&e1);
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "mma peak: cudaEventCreate: %s", cudaGetErrorString(e));
  float best_ms = 0.f;
  for (int round = 0; round < 3 && e == cudaSuccess; ++round) {      // the first round warms the clocks up
    cudaEventRecord(e0, stream);
    mma_peak_kernel<<<sms, 128, smem, stream>>>(reps, status);
    cudaEventRecord(e1, stream);
    e = cudaEventSynchronize(e1);
    if (e == cudaSuccess) e = cudaGetLastError();
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    if (round > 0 && (best_ms == 0.f || ms < best_ms)) best_ms = ms;
  }
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "mma peak: %s", cudaGetErrorString(e));
  const double flops = 2.0 * 128 * kN * 32 * static_cast<double>(reps) * kIssuers * sms;
  *tflops_out = flops / (best_ms * 1e-3) / 1e12;
  return ATTN_OK;
}

}  // namespace attnfp8

namespace attnfp8 {

attn_status_t measure_dq_reduction(const AttnShape& s, float* dq_f32, double* ms_out, double* bytes_out, cudaStream_t stream) {
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  cudaError_t e = cudaEventCreate(&e0);
  if (e == cudaSuccess) e = cudaEventCreate(&e1);
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "dq reduction: cudaEventCreate: %s", cudaGetErrorString(e));
  const size_t n = static_cast<size_t>(s.B) * s.Hq * s.N * s.dqk;
  const dim3 grid(s.Hkv, s.N / 128, s.B);
  float best_ms = 0.f;
  for (int round = 0; round < 3 && e == cudaSuccess; ++round) {     // the last round leaves the checkable result
    e = cudaMemsetAsync(dq_f32, 0, n * sizeof(float), stream);
    cudaEventRecord(e0, stream);
    dq_reduction_kernel<<<grid, 256, 0, stream>>>(dq_f32, s.N, s.Hq, s.Hkv, s.dqk, s.causal);
    cudaEventRecord(e1, stream);
    if (e == cudaSuccess) e = cudaEventSynchronize(e1);
    if (e == cudaSuccess) e = cudaGetLastError();
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    if (round > 0 && (best_ms == 0.f || ms < best_ms)) best_ms = ms;
  }
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "dq reduction: %s", cudaGetErrorString(e));
  const double tiles = s.N / 128;
  const double pairs = static_cast<double>(s.B) * s.Hq * (s.causal ? tiles * (tiles + 1) / 2 : tiles * tiles) * 2;
  *ms_out = best_ms;
  *bytes_out = pairs * 64 * s.dqk * sizeof(float);
  return ATTN_OK;
}

}  // namespace attnfp8
