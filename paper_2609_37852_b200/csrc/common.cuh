// Declarations shared by the kernels' translation units and the C-ABI layer.
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda.h>
#include <cuda_runtime.h>

#include "../../include/attn_fp8.h"

namespace attnfp8 {

// Records a message for attn_fp8_last_error() and returns `code`.
attn_status_t fail(attn_status_t code, const char* fmt, ...);

// Bytes at the head of every workspace reserved for the device status word.
constexpr size_t kWorkspaceHeaderBytes = ATTN_STATUS_WORKSPACE_BYTES;

// cuTensorMapEncodeTiled fetched through the runtime (no link-time dependency on libcuda).
// Encodes a 2-D uint8 tensor [rows, row_bytes] (row pitch == row_bytes) with a
// (box_rows x 128-byte) box and the 128-byte swizzle.
attn_status_t encode_tmap_u8_sw128(CUtensorMap* out, const void* base, uint64_t row_bytes, uint64_t rows,
                                   uint32_t box_rows);

struct AttnShape {
  int B, N, Hq, Hkv, dqk, dv, causal;   // N: query rows (the length of Q, dO, O, dQ, LSE, delta)
  float scale;
  int eb;   // bytes per operand element: 1 = E4M3 codes with E8M0 block scales, 2 = BF16 without scales
  int ebv;  // the same for the row copies of dO and V, the operands of dP alone (2 with eb == 1: protected dP)
  int Nk;   // keys (the length of K, V, dK, dV); == N unless the caller holds a shard of the queries
  int q0t;  // 128-row tile index of query row 0 in the key sequence: key j is visible to query i iff j <= 128 * q0t + i
  int kv_lim;  // last real key inside the last key tile (127: the tile is full); read without the causal mask only
};

// Kernel launchers (each validates nothing: the C-ABI layer has done so).
attn_status_t launch_quantize_fused(const void* src, int src_dtype, int B, int H, int N, int d, const float* cos,
                                    const float* sin, float scale, float* mean, attn_qtensor_t out,
                                    cudaStream_t stream);
attn_status_t launch_quantize_batch(const attn_quantize_job_t* jobs, int n_jobs, int* status, cudaStream_t stream);
attn_status_t launch_bf16_copies(const void* src, int src_dtype, int B, int H, int N, int d, void* row_out, void* col_out,
                                 cudaStream_t stream);
attn_status_t launch_fwd(const AttnShape& s, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v, void* o,
                         float* lse, int* status, cudaStream_t stream);
attn_status_t launch_fwd_interleaved(const AttnShape& s, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v, void* o,
                                     float* lse, int* status, cudaStream_t stream);
attn_status_t launch_bwd_delta(const AttnShape& s, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                               attn_qtensor_t dO, const float* lse, float* delta, int* status, cudaStream_t stream);
attn_status_t launch_stale_delta(const AttnShape& s, const void* dO_bf16, const void* o_bf16, float* delta,
                                 cudaStream_t stream);
attn_status_t launch_consistent_delta(const AttnShape& s, attn_qtensor_t dO, const void* o_bf16, float* delta,
                                      cudaStream_t stream);
attn_status_t launch_bwd_dq(const AttnShape& s, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                            attn_qtensor_t dO, const float* lse, const float* delta, void* dq, float* rowsum,
                            float* rowabs, float* post_rowsum, float* post_rowabs, int* status, cudaStream_t stream,
                            bool behind_dkdv = false, float* p_abs_dp = nullptr);
attn_status_t launch_bwd_dkdv(const AttnShape& s, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                              attn_qtensor_t dO, const float* lse, const float* delta, void* dk, void* dv,
                              int* status, cudaStream_t stream);

attn_status_t measure_mma_peak(double* tflops_out, int* status, cudaStream_t stream);
attn_status_t measure_dq_reduction(const AttnShape& s, float* dq_f32, double* ms_out, double* bytes_out, cudaStream_t stream);

inline size_t scale_tiles_per_slab(int64_t rows, int64_t cols) {
  return static_cast<size_t>((rows + 127) / 128) * static_cast<size_t>((cols / 32 + 3) / 4);
}

}  // namespace attnfp8
