// C-ABI entry points: argument validation, workspace handling, dispatch to the kernel launchers.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace attnfp8 {

static thread_local char g_last_error[512] = "no error";

attn_status_t fail(attn_status_t code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_last_error, sizeof(g_last_error), fmt, ap);
  va_end(ap);
  return code;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) return nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

attn_status_t encode_tmap_u8_sw128(CUtensorMap* out, const void* base, uint64_t row_bytes, uint64_t rows,
                                   uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return fail(ATTN_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  cuuint64_t dims[2] = {row_bytes, rows};
  cuuint64_t strides[1] = {row_bytes};
  cuuint32_t box[2] = {128, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(ATTN_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
  return ATTN_OK;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

static attn_status_t check_device() {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  int major = 0;
  e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "cudaDeviceGetAttribute: %s", cudaGetErrorString(e));
  if (major != 10) return fail(ATTN_ERR_ARCH, "device compute capability %d.x is not 10.x (sm_100a)", major);
  return ATTN_OK;
}

enum Entry { kEntryFwd = 0, kEntryDelta = 1, kEntryDq = 2, kEntryDkdv = 3 };

// Head-dimension pairs each kernel family is built for, per operand width.
static bool dims_supported(int entry, int eb, int dqk, int dv) {
  (void)entry; (void)eb;
  const bool narrow = (dqk == 64 && dv == 64) || (dqk == 128 && dv == 128);
  const bool wide = (dqk == 192 && dv == 128) || (dqk == 256 && dv == 256);
  return narrow || wide;
}

static attn_status_t check_params(const attn_params_t* p, AttnShape* s, int entry) {
  if (!p) return fail(ATTN_ERR_INVALID_ARG, "params is NULL");
  if (p->batch <= 0 || p->seqlen <= 0 || p->heads_q <= 0 || p->heads_kv <= 0)
    return fail(ATTN_ERR_INVALID_ARG, "batch, seqlen and head counts must be positive");
  if (p->heads_q % p->heads_kv) return fail(ATTN_ERR_INVALID_ARG, "heads_q must be a multiple of heads_kv");
  if (p->causal != 0 && p->causal != 1) return fail(ATTN_ERR_INVALID_ARG, "causal must be 0 or 1");
  if (!(p->softmax_scale > 0.f)) return fail(ATTN_ERR_INVALID_ARG, "softmax_scale must be positive");
  if (p->precision != ATTN_PREC_MXFP8 && p->precision != ATTN_PREC_BF16 && p->precision != ATTN_PREC_MXFP8_PROTECTED_DP)
    return fail(ATTN_ERR_INVALID_ARG, "precision %d unknown", p->precision);
  if (p->seqlen % 128) return fail(ATTN_ERR_UNSUPPORTED, "seqlen must be a multiple of 128");
  if (p->seqlen_k < 0 || p->q_start < 0) return fail(ATTN_ERR_INVALID_ARG, "seqlen_k and q_start must not be negative");
  if (p->seqlen_k == 0 && p->q_start != 0) return fail(ATTN_ERR_INVALID_ARG, "q_start needs seqlen_k");
  const int seqlen_k = p->seqlen_k ? p->seqlen_k : p->seqlen;
  const int q_start = p->causal ? p->q_start : 0;
  if (seqlen_k % 128 || p->q_start % 128) return fail(ATTN_ERR_UNSUPPORTED, "seqlen_k and q_start must be multiples of 128");
  if (p->causal && static_cast<long long>(q_start) + p->seqlen != seqlen_k)
    return fail(ATTN_ERR_UNSUPPORTED, "causal shard: seqlen_k (%d) must equal q_start + seqlen (%d + %d)", seqlen_k, q_start,
                p->seqlen);
  // the kernels form row coordinates of the [B * H * N] and [B * Hkv * d] operand views in 32-bit integers
  {
    const long long q_rows = static_cast<long long>(p->batch) * p->heads_q * p->seqlen;
    const int wide = p->head_dim_qk > p->head_dim_v ? p->head_dim_qk : p->head_dim_v;
    const long long kv_rows = static_cast<long long>(p->batch) * p->heads_kv * (seqlen_k > wide ? seqlen_k : wide);
    if (q_rows > 0x7fffffffLL || kv_rows > 0x7fffffffLL)
      return fail(ATTN_ERR_UNSUPPORTED, "batch * heads * seqlen = %lld exceeds the 2^31 - 1 rows a launch indexes",
                  q_rows > kv_rows ? q_rows : kv_rows);
  }
  const int eb = p->precision == ATTN_PREC_BF16 ? 2 : 1;
  if (!dims_supported(entry, eb, p->head_dim_qk, p->head_dim_v))
    return fail(ATTN_ERR_UNSUPPORTED, "head dims (%d, %d) are not built for this entry point in %s mode",
                p->head_dim_qk, p->head_dim_v, eb == 1 ? "MXFP8" : "BF16");
  // protected dP: the row copies of dO and V (the operands of dP alone) are BF16; the forward never sees them
  const bool protect = p->precision == ATTN_PREC_MXFP8_PROTECTED_DP && entry != kEntryFwd;
  if (protect && !((p->head_dim_qk == 64 && p->head_dim_v == 64) || (p->head_dim_qk == 128 && p->head_dim_v == 128)))
    return fail(ATTN_ERR_UNSUPPORTED, "protected dP is built for head dims (64,64) and (128,128)");
  if (p->keys_valid < 0 || p->keys_valid > seqlen_k || (p->keys_valid && p->keys_valid <= seqlen_k - 128))
    return fail(ATTN_ERR_INVALID_ARG, "keys_valid (%d) must be 0 or lie in the last 128-key tile of seqlen_k (%d)",
                p->keys_valid, seqlen_k);
  const int kv_lim = p->keys_valid ? p->keys_valid - 1 - (seqlen_k - 128) : 127;
  *s = AttnShape{p->batch, p->seqlen, p->heads_q, p->heads_kv, p->head_dim_qk, p->head_dim_v, p->causal,
                 p->softmax_scale, eb, protect ? 2 : eb, seqlen_k, q_start / 128, kv_lim};
  return ATTN_OK;
}

static attn_status_t check_ptr(const void* p, const char* name) {
  if (!p) return fail(ATTN_ERR_INVALID_ARG, "%s is NULL", name);
  if (!aligned16(p)) return fail(ATTN_ERR_ALIGNMENT, "%s is not 16-byte aligned", name);
  return ATTN_OK;
}

// One orientation of an operand: the codes (or BF16 values) always, the scale bytes in FP8 mode.
#define CHECK_OPERAND(t, orient, fp8)                                                   \
  do {                                                                                   \
    CHECK(check_ptr(t.orient##_codes, #t "." #orient "_codes"));                          \
    if (fp8) CHECK(check_ptr(t.orient##_scales, #t "." #orient "_scales"));               \
  } while (0)

#define CHECK(x)                        \
  do {                                  \
    attn_status_t st_ = (x);            \
    if (st_ != ATTN_OK) return st_;     \
  } while (0)

// The status word is sticky: kernels only ever set it, attn_fp8_workspace_init and
// attn_fp8_read_status clear it.  Nothing is enqueued here.
static attn_status_t prepare_workspace(void* ws, size_t ws_bytes, size_t need, cudaStream_t, int** status) {
  if (!ws || ws_bytes < need) return fail(ATTN_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, ws_bytes);
  if (!aligned16(ws)) return fail(ATTN_ERR_ALIGNMENT, "workspace is not 16-byte aligned");
  *status = static_cast<int*>(ws);
  return ATTN_OK;
}

static attn_status_t builtin_scratch_for_current_device(void** out);   // defined with the built-in scratch, below

}  // namespace attnfp8

using namespace attnfp8;

extern "C" {

size_t attn_fp8_scale_offset(int64_t row, int64_t block, int64_t n_blocks) {
  const int64_t tiles_per_row_tile = (n_blocks + 3) / 4;
  const int64_t tile = (row / 128) * tiles_per_row_tile + block / 4;
  return static_cast<size_t>(tile * 512 + (row % 32) * 16 + ((row % 128) / 32) * 4 + (block % 4));
}

size_t attn_fp8_scale_bytes(int64_t B, int64_t H, int64_t rows, int64_t cols) {
  return static_cast<size_t>(B * H) * scale_tiles_per_slab(rows, cols) * 512;
}

static attn_status_t check_quantize_args(const void* src, int32_t src_dtype, int32_t B, int32_t H, int32_t N, int32_t d,
                                         const attn_qtensor_t& out) {
  if (B <= 0 || H <= 0 || N <= 0 || d <= 0) return fail(ATTN_ERR_INVALID_ARG, "sizes must be positive");
  if (src_dtype != ATTN_SRC_BF16 && src_dtype != ATTN_SRC_FP32)
    return fail(ATTN_ERR_INVALID_ARG, "src_dtype %d is neither BF16 nor FP32", src_dtype);
  if (N % 128 || d % 32 || d > 256)
    return fail(ATTN_ERR_UNSUPPORTED, "quantize needs N %% 128 == 0 and d %% 32 == 0, d <= 256 (N=%d d=%d)", N, d);
  CHECK(check_ptr(src, "src"));
  if (!out.row_codes && !out.col_codes) return fail(ATTN_ERR_INVALID_ARG, "no output orientation requested");
  if ((out.row_codes == nullptr) != (out.row_scales == nullptr) ||
      (out.col_codes == nullptr) != (out.col_scales == nullptr))
    return fail(ATTN_ERR_INVALID_ARG, "codes and scales of an orientation must be given together");
  if (out.row_codes) { CHECK(check_ptr(out.row_codes, "row_codes")); CHECK(check_ptr(out.row_scales, "row_scales")); }
  if (out.col_codes) { CHECK(check_ptr(out.col_codes, "col_codes")); CHECK(check_ptr(out.col_scales, "col_scales")); }
  return ATTN_OK;
}

attn_status_t attn_fp8_quantize(const void* src, int32_t src_dtype, int32_t B, int32_t H, int32_t N, int32_t d,
                                attn_qtensor_t out, void* stream) {
  CHECK(check_quantize_args(src, src_dtype, B, H, N, d, out));
  if (static_cast<long long>(B) * H * (N / 128) > 0x7fffffffLL)
    return fail(ATTN_ERR_UNSUPPORTED, "tensor of more than 2^31 - 1 tiles of 128 tokens");
  CHECK(check_device());
  // a batch of one; this entry point has no workspace argument, so the status word of its kernel
  // (a bulk copy that never completed) lands in the library's built-in scratch
  void* scratch = nullptr;
  CHECK(builtin_scratch_for_current_device(&scratch));
  const attn_quantize_job_t job = {src, src_dtype, B, H, N, d, out};
  return launch_quantize_batch(&job, 1, static_cast<int*>(scratch), static_cast<cudaStream_t>(stream));
}

attn_status_t attn_fp8_quantize_batch(const attn_quantize_job_t* jobs, int32_t n_jobs, void* workspace,
                                      size_t workspace_bytes, void* stream) {
  if (!jobs) return fail(ATTN_ERR_INVALID_ARG, "jobs is NULL");
  if (n_jobs < 1 || n_jobs > ATTN_QUANTIZE_MAX_JOBS)
    return fail(ATTN_ERR_INVALID_ARG, "n_jobs must be 1..%d (got %d)", ATTN_QUANTIZE_MAX_JOBS, n_jobs);
  long long tiles = 0;
  for (int j = 0; j < n_jobs; ++j) {
    const attn_quantize_job_t& q = jobs[j];
    CHECK(check_quantize_args(q.src, q.src_dtype, q.B, q.H, q.N, q.d, q.out));
    if (q.src_dtype != jobs[0].src_dtype) return fail(ATTN_ERR_INVALID_ARG, "all jobs of a batch must share one src_dtype");
    tiles += static_cast<long long>(q.B) * q.H * (q.N / 128);
  }
  if (tiles > 0x7fffffffLL) return fail(ATTN_ERR_UNSUPPORTED, "batch of %lld tiles exceeds the 2^31 - 1 a launch indexes", tiles);
  CHECK(check_device());
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int* status = nullptr;
  CHECK(prepare_workspace(workspace, workspace_bytes, kWorkspaceHeaderBytes, st, &status));
  return launch_quantize_batch(jobs, n_jobs, status, st);
}

attn_status_t attn_fp8_quantize_fused(const void* src, int32_t src_dtype, int32_t B, int32_t H, int32_t N, int32_t d,
                                      const float* rope_cos, const float* rope_sin, float scale, float* mean,
                                      attn_qtensor_t out, void* stream) {
  if (B <= 0 || H <= 0 || N <= 0 || d <= 0) return fail(ATTN_ERR_INVALID_ARG, "sizes must be positive");
  if (src_dtype != ATTN_SRC_BF16 && src_dtype != ATTN_SRC_FP32)
    return fail(ATTN_ERR_INVALID_ARG, "src_dtype %d is neither BF16 nor FP32", src_dtype);
  if (N % 128 || d % 32 || d > 256)
    return fail(ATTN_ERR_UNSUPPORTED, "quantize needs N %% 128 == 0 and d %% 32 == 0, d <= 256 (N=%d d=%d)", N, d);
  if ((rope_cos == nullptr) != (rope_sin == nullptr))
    return fail(ATTN_ERR_INVALID_ARG, "rope_cos and rope_sin must be given together");
  if (!(scale > 0.f) || !(scale < 3.0e38f)) return fail(ATTN_ERR_INVALID_ARG, "scale must be positive and finite");
  if (mean != nullptr && src_dtype != ATTN_SRC_BF16)
    return fail(ATTN_ERR_UNSUPPORTED, "key centering needs a BF16 source (the mean is an exact sum of BF16 terms)");
  CHECK(check_ptr(src, "src"));
  if (rope_cos) { CHECK(check_ptr(rope_cos, "rope_cos")); CHECK(check_ptr(rope_sin, "rope_sin")); }
  if (mean) CHECK(check_ptr(mean, "mean"));
  if (!out.row_codes && !out.col_codes) return fail(ATTN_ERR_INVALID_ARG, "no output orientation requested");
  if ((out.row_codes == nullptr) != (out.row_scales == nullptr) ||
      (out.col_codes == nullptr) != (out.col_scales == nullptr))
    return fail(ATTN_ERR_INVALID_ARG, "codes and scales of an orientation must be given together");
  if (out.row_codes) { CHECK(check_ptr(out.row_codes, "row_codes")); CHECK(check_ptr(out.row_scales, "row_scales")); }
  if (out.col_codes) { CHECK(check_ptr(out.col_codes, "col_codes")); CHECK(check_ptr(out.col_scales, "col_scales")); }
  CHECK(check_device());
  return launch_quantize_fused(src, src_dtype, B, H, N, d, rope_cos, rope_sin, scale, mean, out,
                               static_cast<cudaStream_t>(stream));
}

attn_status_t attn_fp8_prepare_bf16(const void* src, int32_t src_dtype, int32_t B, int32_t H, int32_t N, int32_t d,
                                    attn_qtensor_t out, void* stream) {
  if (B <= 0 || H <= 0 || N <= 0 || d <= 0) return fail(ATTN_ERR_INVALID_ARG, "sizes must be positive");
  if (src_dtype != ATTN_SRC_BF16 && src_dtype != ATTN_SRC_FP32)
    return fail(ATTN_ERR_INVALID_ARG, "src_dtype %d is neither BF16 nor FP32", src_dtype);
  if (N % 128 || d % 32 || d > 256)
    return fail(ATTN_ERR_UNSUPPORTED, "prepare_bf16 needs N %% 128 == 0 and d %% 32 == 0, d <= 256 (N=%d d=%d)", N, d);
  CHECK(check_ptr(src, "src"));
  if (!out.row_codes && !out.col_codes) return fail(ATTN_ERR_INVALID_ARG, "no output orientation requested");
  if (out.row_codes) CHECK(check_ptr(out.row_codes, "row_codes"));
  if (out.col_codes) CHECK(check_ptr(out.col_codes, "col_codes"));
  CHECK(check_device());
  return launch_bf16_copies(src, src_dtype, B, H, N, d, out.row_codes, out.col_codes, static_cast<cudaStream_t>(stream));
}

size_t attn_fp8_workspace_bytes(const attn_params_t* p, int32_t which) {
  (void)p;
  (void)which;
  return kWorkspaceHeaderBytes;
}

attn_status_t attn_fp8_fwd(const attn_params_t* p, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                           void* o_bf16, float* lse, void* workspace, size_t workspace_bytes, void* stream) {
  AttnShape s;
  CHECK(check_params(p, &s, kEntryFwd));
  const bool fp8 = s.eb == 1;
  CHECK_OPERAND(q, row, fp8); CHECK_OPERAND(k, row, fp8); CHECK_OPERAND(v, col, fp8);
  CHECK(check_ptr(o_bf16, "o_bf16")); CHECK(check_ptr(lse, "lse"));
  CHECK(check_device());
  int* status = nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CHECK(prepare_workspace(workspace, workspace_bytes, attn_fp8_workspace_bytes(p, ATTN_WS_FWD), st, &status));
  return launch_fwd(s, q, k, v, o_bf16, lse, status, st);
}

attn_status_t attn_fp8_bwd_delta(const attn_params_t* p, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                                 attn_qtensor_t dO, const void* dO_bf16, const void* o_bf16, const float* lse,
                                 float* delta, void* workspace, size_t workspace_bytes, void* stream) {
  AttnShape s;
  CHECK(check_params(p, &s, kEntryDelta));
  const bool fp8 = s.eb == 1;
  CHECK(check_ptr(delta, "delta"));
  CHECK(check_device());
  int* status = nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CHECK(prepare_workspace(workspace, workspace_bytes, attn_fp8_workspace_bytes(p, ATTN_WS_BWD_DELTA), st, &status));
  if (p->delta_mode == ATTN_DELTA_STALE) {
    CHECK(check_ptr(dO_bf16, "dO_bf16")); CHECK(check_ptr(o_bf16, "o_bf16"));
    return launch_stale_delta(s, dO_bf16, o_bf16, delta, st);
  }
  if (p->delta_mode == ATTN_DELTA_CONSISTENT_DO) {
    CHECK(check_ptr(o_bf16, "o_bf16"));
    if (s.ebv == 2) {                                 // BF16 row copy of dO: dO^ is the BF16 dO itself
      CHECK(check_ptr(dO.row_codes, "dO.row_codes"));
      return launch_stale_delta(s, dO.row_codes, o_bf16, delta, st);
    }
    CHECK_OPERAND(dO, row, fp8);
    return launch_consistent_delta(s, dO, o_bf16, delta, st);
  }
  if (p->delta_mode != ATTN_DELTA_MATCHED) return fail(ATTN_ERR_INVALID_ARG, "delta_mode %d unknown", p->delta_mode);
  const bool fp8v = s.ebv == 1;
  CHECK_OPERAND(q, row, fp8); CHECK_OPERAND(k, row, fp8); CHECK_OPERAND(v, row, fp8v); CHECK_OPERAND(dO, row, fp8v);
  CHECK(check_ptr(lse, "lse"));
  return launch_bwd_delta(s, q, k, v, dO, lse, delta, status, st);
}

static attn_status_t bwd_impl(const attn_params_t* p, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                              attn_qtensor_t dO, const float* lse, const float* delta, void* dq_bf16, void* dk_bf16,
                              void* dv_bf16, float* diag_rowsum_ds, float* diag_rowsum_abs_ds, void* workspace,
                              size_t workspace_bytes, void* stream, bool want_dq, bool want_dkdv,
                              float* post_rowsum = nullptr, float* post_rowabs = nullptr, float* p_abs_dp = nullptr) {
  AttnShape s;
  if (want_dq) CHECK(check_params(p, &s, kEntryDq));
  if (want_dkdv) CHECK(check_params(p, &s, kEntryDkdv));
  const bool fp8 = s.eb == 1, fp8v = s.ebv == 1;
  CHECK_OPERAND(q, row, fp8); CHECK_OPERAND(k, row, fp8); CHECK_OPERAND(v, row, fp8v); CHECK_OPERAND(dO, row, fp8v);
  CHECK(check_ptr(lse, "lse")); CHECK(check_ptr(delta, "delta"));
  if (want_dq) {
    CHECK_OPERAND(k, col, fp8);
    CHECK(check_ptr(dq_bf16, "dq_bf16"));
    if ((diag_rowsum_ds == nullptr) != (diag_rowsum_abs_ds == nullptr))
      return fail(ATTN_ERR_INVALID_ARG, "the two diagnostic outputs must be given together");
    if ((post_rowsum == nullptr) != (post_rowabs == nullptr) || (post_rowsum && !diag_rowsum_ds))
      return fail(ATTN_ERR_INVALID_ARG, "the post-cast outputs come as a pair and need the pre-cast pair as well");
    if (p_abs_dp && !diag_rowsum_ds) return fail(ATTN_ERR_INVALID_ARG, "diag_p_abs_dp needs the pre-cast pair as well");
    if (p_abs_dp) CHECK(check_ptr(p_abs_dp, "diag_p_abs_dp"));
  }
  if (want_dkdv) {
    CHECK_OPERAND(q, col, fp8); CHECK_OPERAND(dO, col, fp8);
    CHECK(check_ptr(dk_bf16, "dk_bf16")); CHECK(check_ptr(dv_bf16, "dv_bf16"));
  }
  CHECK(check_device());
  int* status = nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CHECK(prepare_workspace(workspace, workspace_bytes, attn_fp8_workspace_bytes(p, ATTN_WS_BWD), st, &status));
  if (want_dq) {
    // the ticket counter of the persistent dQ kernel (bytes 16..31 of the header) starts at zero; cleared
    // here, ahead of both kernels, so that nothing sits between the key-major launch and the dQ launch
    cudaError_t e = cudaMemsetAsync(static_cast<char*>(workspace) + 16, 0, 16, st);
    if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "bwd: cudaMemsetAsync(ticket counter): %s", cudaGetErrorString(e));
  }
  // Key-major kernel first: its CTAs are few and long, so its last wave leaves SMs idle, which
  // the many short CTAs of the query-major kernel, launched behind it, fill.
  if (want_dkdv) CHECK(launch_bwd_dkdv(s, q, k, v, dO, lse, delta, dk_bf16, dv_bf16, status, st));
  if (want_dq)
    CHECK(launch_bwd_dq(s, q, k, v, dO, lse, delta, dq_bf16, diag_rowsum_ds, diag_rowsum_abs_ds, post_rowsum, post_rowabs,
                        status, st, /*behind_dkdv=*/want_dkdv, p_abs_dp));
  return ATTN_OK;
}

attn_status_t attn_fp8_bwd(const attn_params_t* p, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                           attn_qtensor_t dO, const float* lse, const float* delta, void* dq_bf16, void* dk_bf16,
                           void* dv_bf16, float* diag_rowsum_ds, float* diag_rowsum_abs_ds, void* workspace,
                           size_t workspace_bytes, void* stream) {
  return bwd_impl(p, q, k, v, dO, lse, delta, dq_bf16, dk_bf16, dv_bf16, diag_rowsum_ds, diag_rowsum_abs_ds,
                  workspace, workspace_bytes, stream, true, true);
}

attn_status_t attn_fp8_bwd_dq(const attn_params_t* p, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                              attn_qtensor_t dO, const float* lse, const float* delta, void* dq_bf16,
                              float* diag_rowsum_ds, float* diag_rowsum_abs_ds, void* workspace,
                              size_t workspace_bytes, void* stream) {
  return bwd_impl(p, q, k, v, dO, lse, delta, dq_bf16, nullptr, nullptr, diag_rowsum_ds, diag_rowsum_abs_ds,
                  workspace, workspace_bytes, stream, true, false);
}

attn_status_t attn_fp8_bwd_dq_postcast(const attn_params_t* p, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                                       attn_qtensor_t dO, const float* lse, const float* delta, void* dq_bf16,
                                       float* diag_rowsum_ds, float* diag_rowsum_abs_ds, float* diag_post_rowsum_ds,
                                       float* diag_post_rowsum_abs_ds, void* workspace, size_t workspace_bytes,
                                       void* stream) {
  if (!diag_post_rowsum_ds || !diag_post_rowsum_abs_ds || !diag_rowsum_ds || !diag_rowsum_abs_ds)
    return fail(ATTN_ERR_INVALID_ARG, "attn_fp8_bwd_dq_postcast needs all four diagnostic outputs");
  return bwd_impl(p, q, k, v, dO, lse, delta, dq_bf16, nullptr, nullptr, diag_rowsum_ds, diag_rowsum_abs_ds,
                  workspace, workspace_bytes, stream, true, false, diag_post_rowsum_ds, diag_post_rowsum_abs_ds);
}

attn_status_t attn_fp8_bwd_dq_rowprobe(const attn_params_t* p, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                                       attn_qtensor_t dO, const float* lse, const float* delta, void* dq_bf16,
                                       float* diag_rowsum_ds, float* diag_rowsum_abs_ds, float* diag_p_abs_dp,
                                       void* workspace, size_t workspace_bytes, void* stream) {
  if (!diag_rowsum_ds || !diag_rowsum_abs_ds || !diag_p_abs_dp)
    return fail(ATTN_ERR_INVALID_ARG, "attn_fp8_bwd_dq_rowprobe needs all three diagnostic outputs");
  return bwd_impl(p, q, k, v, dO, lse, delta, dq_bf16, nullptr, nullptr, diag_rowsum_ds, diag_rowsum_abs_ds,
                  workspace, workspace_bytes, stream, true, false, nullptr, nullptr, diag_p_abs_dp);
}

attn_status_t attn_fp8_bwd_dkdv(const attn_params_t* p, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                                attn_qtensor_t dO, const float* lse, const float* delta, void* dk_bf16,
                                void* dv_bf16, void* workspace, size_t workspace_bytes, void* stream) {
  return bwd_impl(p, q, k, v, dO, lse, delta, nullptr, dk_bf16, dv_bf16, nullptr, nullptr, workspace,
                  workspace_bytes, stream, false, true);
}

attn_status_t attn_fp8_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
  if (!workspace || workspace_bytes < kWorkspaceHeaderBytes)
    return fail(ATTN_ERR_WORKSPACE, "workspace of at least %zu bytes needed, %zu given", kWorkspaceHeaderBytes, workspace_bytes);
  if (!aligned16(workspace)) return fail(ATTN_ERR_ALIGNMENT, "workspace is not 16-byte aligned");
  cudaError_t e = cudaMemsetAsync(workspace, 0, kWorkspaceHeaderBytes, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "workspace_init: cudaMemsetAsync: %s", cudaGetErrorString(e));
  return ATTN_OK;
}

attn_status_t attn_fp8_read_status(void* workspace, void* stream) {
  if (!workspace) {                                  // the built-in scratch array of the current device
    CHECK(check_device());
    CHECK(builtin_scratch_for_current_device(&workspace));
  }
  int host = 0;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(&host, workspace, sizeof(int), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e == cudaSuccess && host != 0) {          // reported once: clear the header (status word and the scheduling
                                                // counters a kernel that gave up may have left) for the calls that follow
    e = cudaMemsetAsync(workspace, 0, kWorkspaceHeaderBytes, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  }
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "read_status: %s", cudaGetErrorString(e));
  if (host == ATTN_ERR_ALIGNMENT)
    return fail(ATTN_ERR_ALIGNMENT, "a kernel found its dynamic shared memory not 1024-byte aligned and did not run");
  if (host != 0) return fail(ATTN_ERR_TIMEOUT, "a bounded device-side wait expired (status word %d)", host);
  return ATTN_OK;
}

const char* attn_fp8_last_error(void) { return g_last_error; }

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// Forward for callers that cannot hand over a workspace.
//
// The scratch the forward kernel needs (today: its status header) lives in a fixed array that is
// part of the library image, so every GPU that loads the library carries these bytes until the
// process exits.  In host code the array's name is only a handle: the device address has to be
// asked for, per device, with that device current.
namespace attnfp8 {

constexpr size_t kBuiltinScratchBytes = 4096;
static __device__ __align__(256) unsigned char g_builtin_scratch[kBuiltinScratchBytes];

constexpr int kMaxDevices = 64;
static void* g_builtin_scratch_addr[kMaxDevices];   // device address of the array, per device ordinal
static std::mutex g_builtin_scratch_mutex;

static attn_status_t builtin_scratch_for_current_device(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return fail(ATTN_ERR_UNSUPPORTED, "device ordinal %d is outside 0..%d", dev, kMaxDevices - 1);
  std::lock_guard<std::mutex> lock(g_builtin_scratch_mutex);
  if (!g_builtin_scratch_addr[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_builtin_scratch);
    if (e != cudaSuccess || !ptr)
      return fail(ATTN_ERR_CUDA, "cudaGetSymbolAddress(built-in scratch) on device %d: %s", dev, cudaGetErrorString(e));
    g_builtin_scratch_addr[dev] = ptr;
  }
  *out = g_builtin_scratch_addr[dev];
  return ATTN_OK;
}

}  // namespace attnfp8

extern "C" attn_status_t attn_fp8_fwd_noalloc(const attn_params_t* p, attn_qtensor_t q, attn_qtensor_t k,
                                              attn_qtensor_t v, void* o_bf16, float* lse, void* stream) {
  AttnShape s;
  CHECK(check_params(p, &s, kEntryFwd));
  const bool fp8 = s.eb == 1;
  CHECK_OPERAND(q, row, fp8); CHECK_OPERAND(k, row, fp8); CHECK_OPERAND(v, col, fp8);
  CHECK(check_ptr(o_bf16, "o_bf16")); CHECK(check_ptr(lse, "lse"));
  const size_t need = attn_fp8_workspace_bytes(p, ATTN_WS_FWD);
  if (need > kBuiltinScratchBytes)
    return fail(ATTN_ERR_WORKSPACE,
                "attn_fp8_fwd_noalloc: this problem needs %zu bytes of scratch but the built-in array holds %zu; "
                "use attn_fp8_fwd with a caller workspace", need, kBuiltinScratchBytes);
  CHECK(check_device());
  void* scratch = nullptr;
  CHECK(builtin_scratch_for_current_device(&scratch));
  int* status = nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the array keeps whatever earlier calls left; its status word is only ever set, so nothing needs clearing
  CHECK(prepare_workspace(scratch, kBuiltinScratchBytes, need, st, &status));
  return launch_fwd(s, q, k, v, o_bf16, lse, status, st);
}

// ------------------------------------------------------------------------------------------------
// Self-test of the bounded-wait machinery: one CTA waits on a barrier that nothing completes, with
// a limit of a few milliseconds, gives up, and reports through the workspace status word exactly as
// the attention kernels do.  The context stays usable; nothing traps.
namespace attnfp8 {
__global__ void wait_selftest_kernel(int* status, long long limit_cycles) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    sm100::mbar_init(&bar, 1);
    abort_flag = 0;
    sm100::fence_mbar_init();
  }
  __syncthreads();
  // each thread polls in short bursts so that the limit is looked at every few microseconds
  const bool ok = sm100::mbar_wait_limited(&bar, 0, &abort_flag, limit_cycles, 4);
  __syncthreads();
  if (threadIdx.x == 0 && (abort_flag || !ok)) atomicExch(status, static_cast<int>(ATTN_ERR_TIMEOUT));
}
}  // namespace attnfp8

extern "C" attn_status_t attn_fp8_selftest_timeout(void* workspace, size_t workspace_bytes, void* stream) {
  CHECK(check_device());
  if (!workspace) {                                  // the built-in scratch array of the current device
    CHECK(builtin_scratch_for_current_device(&workspace));
    workspace_bytes = kBuiltinScratchBytes;
  }
  int* status = nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CHECK(prepare_workspace(workspace, workspace_bytes, kWorkspaceHeaderBytes, st, &status));
  wait_selftest_kernel<<<1, 64, 0, st>>>(status, 4000000LL);     // ~2 ms of SM cycles
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "selftest: launch: %s", cudaGetErrorString(e));
  return ATTN_OK;
}

extern "C" attn_status_t attn_fp8_measure_mma_peak(double* tflops, void* workspace, size_t workspace_bytes, void* stream) {
  if (!tflops) return fail(ATTN_ERR_INVALID_ARG, "tflops is NULL");
  CHECK(check_device());
  int* status = nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CHECK(prepare_workspace(workspace, workspace_bytes, kWorkspaceHeaderBytes, st, &status));
  return measure_mma_peak(tflops, status, st);
}

extern "C" attn_status_t attn_fp8_measure_dq_reduction(const attn_params_t* p, float* dq_f32, size_t dq_f32_bytes, double* ms,
                                                        double* bytes, void* stream) {
  AttnShape s;
  CHECK(check_params(p, &s, kEntryDq));
  if (s.Nk != s.N || s.q0t) return fail(ATTN_ERR_UNSUPPORTED, "dq reduction probe: square problems only");
  if (!ms || !bytes) return fail(ATTN_ERR_INVALID_ARG, "ms / bytes is NULL");
  CHECK(check_ptr(dq_f32, "dq_f32"));
  const size_t need = static_cast<size_t>(s.B) * s.Hq * s.N * s.dqk * sizeof(float);
  if (dq_f32_bytes < need) return fail(ATTN_ERR_WORKSPACE, "dq_f32 of %zu bytes needed, %zu given", need, dq_f32_bytes);
  CHECK(check_device());
  return measure_dq_reduction(s, dq_f32, ms, bytes, static_cast<cudaStream_t>(stream));
}
