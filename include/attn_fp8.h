/*
 * attn_fp8.h -- C ABI of the FP8 Delta-Matching attention library for NVIDIA B200 (sm_100a).
 *
 * The library computes causal / grouped-query softmax attention forward and backward with
 * block-scaled FP8 operands in every attention-core matmul (paper Section 2.3:
 * S = Q K^T * scale, P = softmax(S), O = P V, dV = P^T dO, dP = dO V^T, dS = P o (dP - delta),
 * dQ = dS K * scale, dK = dS^T Q * scale).  The backward row correction delta is recomputed
 * as rowsum(P o dP) from the unquantised probabilities and the FP32 product of the same FP8
 * dO and V the gradient pass consumes ("Delta-Matching", paper Section 3.3, Eq. 4-5), so
 * that dS keeps zero row sums; the saved-output shortcut rowsum(dO o O) ("stale delta",
 * Section 3.2) is selectable as an ablation.
 *
 * Number format.  Operands are E4M3 codes (round to nearest even, saturating at +-448; paper
 * Appendix "Operands, Scaling, and Accumulation") with one E8M0 scale byte (value 2^(byte-127))
 * per 32 consecutive elements ALONG THE CONTRACTION DIMENSION of the matmul that consumes the
 * operand.  Every input tensor therefore exists in up to two quantised copies:
 *   "row" copy: blocks along the channel dim d      (used when the matmul contracts over d)
 *   "col" copy: blocks along the token dim N, stored transposed (used when it contracts over N)
 * The scale of a block is the smallest power of two that maps the block maximum to <= 448.
 *
 * Conventions.
 *   - Every pointer is a DEVICE pointer unless stated otherwise; all tensors are contiguous.
 *   - The caller owns every buffer.  The library allocates nothing and frees nothing.
 *   - Every call only enqueues work on `stream` (a cudaStream_t passed as void*) and returns;
 *     it never synchronises and never reads device memory from the host, except
 *     attn_fp8_read_status, which says so.
 *   - Calls that take a `workspace` report device-side failures through its sticky status word
 *     (see attn_fp8_workspace_bytes): initialise a workspace once, read the status when needed.
 *   - Errors are return codes; nothing aborts or traps.  Arguments are validated before any
 *     launch.  attn_fp8_last_error() gives a thread-local message for the last failure.
 *   - Results of quantize, fwd, bwd_delta and bwd are bitwise reproducible run to run.
 *   - Changing delta_mode changes only `delta`, dQ and dK -- never O, LSE or dV.
 *
 * Supported shapes: seqlen a multiple of 128 (causal means key j <= query i; a caller that holds
 * a shard of the queries against a longer key sequence says so with seqlen_k / q_start below);
 * heads_q a multiple of heads_kv; head dims (qk, v): (64,64), (128,128), (192,128), (256,256) for
 * every attention entry point in FP8 and in BF16 mode, (64,64) and (128,128) with protected dP;
 * the quantiser accepts any d that is a multiple of 32 up to 256.  Anything else returns
 * ATTN_ERR_UNSUPPORTED.
 *
 * BF16 mode (attn_params_t.precision = ATTN_PREC_BF16; the paper's BF16 reference point, Section
 * 2.1): the same kernels with BF16 operands and no block scales.  An attn_qtensor_t then carries
 *   row_codes = BF16 [B, H, N, d]   (the tensor itself, rounded to BF16)
 *   col_codes = BF16 [B, H, d, N]   (its transpose)
 * and both scale pointers are ignored (may be NULL); attn_fp8_prepare_bf16 writes the two copies.
 * Probabilities and score gradients are rounded to BF16 where the FP8 mode quantises them; the
 * normaliser, LSE, the row correction and every accumulation stay FP32 exactly as in FP8 mode.
 *
 * Protected dP (precision = ATTN_PREC_MXFP8_PROTECTED_DP; the paper's ablation of that name,
 * Appendix "Protected dP"): FP8 mode in which dP = dO V^T alone is computed from BF16 operands.
 * The backward entry points (bwd_delta, bwd, bwd_dq, bwd_dkdv) then take
 *   dO.row_codes = BF16 [B, Hq, N, dv]  and  v.row_codes = BF16 [B, Hkv, N, dv]
 * (row scales ignored); every other operand, the column copies of dO and V included, stays FP8.
 * The forward treats this precision as ATTN_PREC_MXFP8.  Head dims (64,64) and (128,128).  The
 * paper pairs it with the stale correction; any delta_mode is accepted.
 */
#ifndef ATTN_FP8_H_
#define ATTN_FP8_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  ATTN_OK = 0,
  ATTN_ERR_INVALID_ARG = 1,   /* null pointer, non-positive size, heads_q % heads_kv != 0 ...  */
  ATTN_ERR_UNSUPPORTED = 2,   /* shape / precision / mode outside the supported set             */
  ATTN_ERR_ALIGNMENT = 3,     /* a pointer is not 16-byte aligned                               */
  ATTN_ERR_WORKSPACE = 4,     /* workspace missing or smaller than attn_fp8_workspace_bytes()   */
  ATTN_ERR_ARCH = 5,          /* current device is not compute capability 10.x                  */
  ATTN_ERR_CUDA = 6,          /* a CUDA runtime / driver call failed; see attn_fp8_last_error   */
  ATTN_ERR_TIMEOUT = 7        /* a bounded device-side wait expired (reported by read_status)   */
} attn_status_t;

typedef enum { ATTN_PREC_MXFP8 = 0, ATTN_PREC_BF16 = 1, ATTN_PREC_MXFP8_PROTECTED_DP = 2 } attn_precision_t;
typedef enum { ATTN_DELTA_MATCHED = 0, ATTN_DELTA_STALE = 1, ATTN_DELTA_CONSISTENT_DO = 2 } attn_delta_mode_t;
typedef enum { ATTN_SRC_BF16 = 0, ATTN_SRC_FP32 = 1 } attn_src_dtype_t;
typedef enum { ATTN_WS_FWD = 0, ATTN_WS_BWD_DELTA = 1, ATTN_WS_BWD = 2 } attn_ws_kind_t;

/* Problem description shared by the attention entry points.
 * Tensors: Q, dO, O, dQ are [batch, heads_q, seqlen, dim]; K, V, dK, dV are
 * [batch, heads_kv, seqlen_k, dim]; LSE, delta and the diagnostics are [batch, heads_q, seqlen].
 * Query head h reads KV head h / (heads_q / heads_kv).
 *
 * Sequence shards (the paper's Limitations name a context-parallel exchange of FP8 K / V as the
 * next step; this is the per-shard problem such a scheme runs).  With seqlen_k == 0 the problem is
 * square: seqlen keys, query i at position i.  Otherwise the caller holds `seqlen` consecutive
 * queries that start at position q_start of a sequence and `seqlen_k` keys from position 0 on:
 * under the causal mask key j is visible to local query i iff j <= q_start + i.  seqlen_k and
 * q_start are multiples of 128; with causal == 1, seqlen_k must equal q_start + seqlen (keys past
 * the last query are not part of the shard's problem); with causal == 0, q_start is ignored.
 * dK / dV are the shard's contribution for all seqlen_k keys (a sum over shards gives the
 * gradient).  Rows of O, LSE, delta and dQ are bit-identical to those of the unsharded problem.
 *
 * Ragged lengths.  Tensors are always allocated, and quantised, at a multiple of 128 tokens: a caller
 * with fewer tokens pads Q, K, V and dO with zero rows (zero blocks quantise to zero codes, and a
 * partly filled 32-token block takes the scale of its real tokens).  keys_valid says how many of the
 * seqlen_k keys are real (0: all of them; otherwise seqlen_k - 128 < keys_valid <= seqlen_k): without
 * the causal mask the keys from keys_valid on are masked out of every row; under the causal mask real
 * queries never see them, and keys_valid is not needed.  Rows of the outputs that belong to padded
 * queries hold finite values the caller ignores; because their dO rows are zero they add nothing to
 * dK and dV, and the dK / dV rows of padded keys come out as zeros.                               */
typedef struct {
  int32_t batch, seqlen, heads_q, heads_kv, head_dim_qk, head_dim_v;
  int32_t causal;          /* 0 or 1                                                          */
  float   softmax_scale;   /* multiplies the FP32 score accumulator; NOT folded into Q         */
  int32_t precision;       /* attn_precision_t                                                 */
  int32_t delta_mode;      /* attn_delta_mode_t (read by attn_fp8_bwd_delta only)              */
  int32_t seqlen_k;        /* keys; 0 means seqlen (square problem, q_start must be 0)         */
  int32_t q_start;         /* position of query row 0 in the key sequence                      */
  int32_t keys_valid;      /* real keys among the seqlen_k allocated ones; 0 means all         */
} attn_params_t;

/* One quantised tensor X [B, H, N, d] (caller-allocated device memory).
 *
 *   row_codes  uint8 [B, H, N, d]          E4M3 code of X[b,h,n,c], blocks = 32 channels
 *   col_codes  uint8 [B, H, d, N]          E4M3 code of X[b,h,n,c] at [b,h,c,n], blocks = 32 tokens
 *   row_scales uint8 [B, H, N/128, ceil(d/128), 512]
 *   col_scales uint8 [B, H, ceil(d/128), N/128, 512]
 *
 * Scale bytes are stored in 512-byte tiles, the order in which the tensor cores take them
 * from tensor memory.  A tile covers 128 rows x 4 blocks of the scaled matrix (row copy: rows
 * are tokens, blocks run along d; col copy: rows are channels, blocks run along N).  Inside
 * a tile, the byte of (row r, block k) sits at offset  (r % 32) * 16 + ((r % 128) / 32) * 4 + (k % 4);
 * tiles are ordered [r / 128][k / 4].  Bytes of rows or blocks beyond the tensor are 0.
 * attn_fp8_scale_offset() below returns this offset so that callers need not restate it.
 *
 * Either pair may be NULL when that orientation is not needed by the call.                    */
typedef struct {
  uint8_t *row_codes, *row_scales;
  uint8_t *col_codes, *col_scales;
} attn_qtensor_t;

/* Byte offset, inside one (b, h) slab of a scale tensor, of the scale of (row, block) for a
 * scaled matrix with `n_blocks` blocks per row.  Pure host arithmetic.                        */
size_t attn_fp8_scale_offset(int64_t row, int64_t block, int64_t n_blocks);

/* Bytes of one scale tensor (all B*H slabs) for a scaled matrix of `rows` x (`cols`/32 blocks):
 * row copy: rows = N, cols = d; col copy: rows = d, cols = N.                                 */
size_t attn_fp8_scale_bytes(int64_t B, int64_t H, int64_t rows, int64_t cols);

/* Block-scaling quantiser (paper Appendix "Operands, Scaling, and Accumulation", Eq.
 * app_kernel_quantizer, with the FP32 scale amax/448 replaced by an E8M0 scale per 1x32 block).
 *   src        [B, H, N, d] in `src_dtype` (BF16 or FP32), device memory, 16-byte aligned
 *   out        the orientations whose pointers are non-NULL are written (codes AND scales of an
 *              orientation must both be given); all 16-byte aligned
 *   N % 128 == 0, d % 32 == 0, 32 <= d <= 256.
 * Non-finite inputs do not trap: NaN encodes as 0x7F, +-Inf saturates to +-448.
 * The first call on each device looks up the address of the library's built-in scratch (a
 * one-time runtime query): make that first call outside of any stream capture.                */
attn_status_t attn_fp8_quantize(const void* src, int32_t src_dtype, int32_t B, int32_t H, int32_t N,
                                int32_t d, attn_qtensor_t out, void* stream);

/* One tensor of a batched quantiser call: the arguments of attn_fp8_quantize.                   */
typedef struct {
  const void* src;
  int32_t src_dtype;
  int32_t B, H, N, d;
  attn_qtensor_t out;
} attn_quantize_job_t;

#define ATTN_QUANTIZE_MAX_JOBS 8
#define ATTN_STATUS_WORKSPACE_BYTES 256   /* workspace that carries only the device status word */

/* attn_fp8_quantize of up to ATTN_QUANTIZE_MAX_JOBS tensors (the four operands of a step) in ONE
 * launch: a persistent grid walks the 128-token tiles of all tensors and keeps the next tile in
 * flight (bulk asynchronous copies into a shared-memory ring) while it quantises the current one.
 * Outputs are bit-identical to those of attn_fp8_quantize on each tensor.
 *   jobs       host array; every job as attn_fp8_quantize documents; all jobs share one src_dtype
 *              (ATTN_ERR_INVALID_ARG otherwise); outputs of different jobs must not overlap
 *   workspace  device, >= ATTN_STATUS_WORKSPACE_BYTES, 16-byte aligned: its status word reports a
 *              copy that never completed (attn_fp8_read_status -> ATTN_ERR_TIMEOUT), as for the
 *              attention entry points; a workspace of those calls may be passed
 * attn_fp8_quantize is this call with one job; its status word lands in the library's built-in
 * scratch of the current device, which attn_fp8_read_status(NULL, stream) reads.                 */
attn_status_t attn_fp8_quantize_batch(const attn_quantize_job_t* jobs, int32_t n_jobs, void* workspace,
                                      size_t workspace_bytes, void* stream);

/* The quantiser with the paper's operand producer fused in front (Appendix "Operands, Scaling, and
 * Accumulation"), for callers that hold q / k BEFORE rotary embedding, scale folding or key centering:
 *   1. rotary embedding, if rope_cos / rope_sin (FP32 [N, d/2], device) are given: channel c < d/2 is
 *      paired with c + d/2;  r1 = fma(x1, cos, -fl32(x2 sin)),  r2 = fma(x2, cos, fl32(x1 sin)) in FP32,
 *      rotated channels rounded to BF16;
 *   2. key centering, if `mean` (FP32 [B, H, d], device) is given: the mean over the N tokens of the
 *      values of step 1, per (batch, head, channel), is WRITTEN to `mean` (exact sum, correctly rounded
 *      quotient) and subtracted in FP32; needs a BF16 source;
 *   3. multiplication by `scale` in FP32 when scale != 1 (tau = d^-1/2 folded into Q: the attention
 *      calls then take softmax_scale = 1);
 *   4. attn_fp8_quantize of the result.
 * Bitwise reproducible.  Other arguments and errors as attn_fp8_quantize.                       */
attn_status_t attn_fp8_quantize_fused(const void* src, int32_t src_dtype, int32_t B, int32_t H, int32_t N,
                                      int32_t d, const float* rope_cos, const float* rope_sin, float scale,
                                      float* mean, attn_qtensor_t out, void* stream);

/* Operand preparation for BF16 mode: writes the BF16 rounding of `src` to out.row_codes
 * ([B, H, N, d]) and its transpose to out.col_codes ([B, H, d, N]); an orientation whose pointer
 * is NULL is skipped, the scale pointers are ignored.  A caller whose source already is BF16 may
 * pass the source itself as row_codes of the attention calls and ask only for the transpose.
 *   N % 128 == 0, d % 32 == 0, 32 <= d <= 256; pointers 16-byte aligned.                      */
attn_status_t attn_fp8_prepare_bf16(const void* src, int32_t src_dtype, int32_t B, int32_t H, int32_t N,
                                    int32_t d, attn_qtensor_t out, void* stream);

/* Forward (paper Appendix "Forward Probability Encoding"): per query row, online softmax of
 * S = scale * Q^ K^^T over key tiles with a running INTEGER power-of-two shift, normaliser l
 * taken from the exponentials BEFORE the FP8 cast, probabilities quantised in-register in
 * blocks of 32 keys, O = (P^ V^) / l.
 *   reads   q.row_*, k.row_*, v.col_*
 *   writes  o_bf16 [B, Hq, N, dv] (BF16), lse [B, Hq, N] (FP32, natural log)                  */
attn_status_t attn_fp8_fwd(const attn_params_t* p, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                           void* o_bf16, float* lse, void* workspace, size_t workspace_bytes, void* stream);

/* Row correction (paper Section 3.3 Eq. 4; Appendix "Backward Correction and Gradient
 * Computation", paragraph "Matched correction").
 *   MATCHED: delta_i = sum_j P_ij dP^_ij with P_ij = exp(S_ij - LSE_i) unquantised FP32 and
 *            dP^ = dO^ V^^T accumulated in FP32 from FP8 operands.
 *            reads q.row_*, k.row_*, v.row_*, dO.row_*, lse.  dO_bf16 / o_bf16 are ignored.
 *   STALE:   delta_i = sum_c dO_ic O_ic from BF16 dO and the saved BF16 O (both [B,Hq,N,dv]).
 *            reads dO_bf16, o_bf16 only.
 *   CONSISTENT_DO (paper Section 3.3, Eq. delta_consistent_do_residual; an ablation): the same
 *            shortcut with dO replaced by the operand the backward matmuls consume,
 *            delta_i = sum_c dO^_ic O_ic, dO^ = the dequantised row copy of dO.
 *            reads dO.row_*, o_bf16.
 *   writes  delta [B, Hq, N] (FP32)                                                           */
attn_status_t attn_fp8_bwd_delta(const attn_params_t* p, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                                 attn_qtensor_t dO, const void* dO_bf16, const void* o_bf16,
                                 const float* lse, float* delta,
                                 void* workspace, size_t workspace_bytes, void* stream);

/* Gradient pass (same Appendix, paragraphs "Score-gradient quantization" and "Query
 * gradients"): recomputes S and dP^ from the FP8 operands, P = exp(S - LSE) and
 * dS = P o (dP^ - delta) in FP32, quantises P and dS in-register along each contraction
 * dimension and accumulates dV = P^^T dO^, dK = scale dS^^T Q^, dQ = scale dS^ K^; dK and dV are
 * summed over the query heads of each KV group in FP32 before the BF16 store.
 *   reads   q.row_*, q.col_*, k.row_*, k.col_*, v.row_*, dO.row_*, dO.col_*, lse, delta
 *   writes  dq_bf16 [B,Hq,N,dqk], dk_bf16 [B,Hkv,N,dqk], dv_bf16 [B,Hkv,N,dv] (BF16)
 *   diag_rowsum_ds / diag_rowsum_abs_ds: optional [B,Hq,N] FP32 outputs, sum_j dS_ij and
 *   sum_j |dS_ij| taken before the FP8 cast (the paper's row-sum residual probe); may be NULL. */
attn_status_t attn_fp8_bwd(const attn_params_t* p, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                           attn_qtensor_t dO, const float* lse, const float* delta,
                           void* dq_bf16, void* dk_bf16, void* dv_bf16,
                           float* diag_rowsum_ds, float* diag_rowsum_abs_ds,
                           void* workspace, size_t workspace_bytes, void* stream);

/* The two halves of attn_fp8_bwd, for callers that need only one of them (frozen keys/values,
 * or timing the two kernels separately).  Same arguments and meaning as attn_fp8_bwd:
 *   attn_fp8_bwd_dq    the query-major pass: dQ (and the optional row statistics);
 *                      reads q.row_*, k.row_*, k.col_*, v.row_*, dO.row_*, lse, delta
 *   attn_fp8_bwd_dkdv  the key-major pass: dK and dV;
 *                      reads q.row_*, q.col_*, k.row_*, v.row_*, dO.row_*, dO.col_*, lse, delta
 * attn_fp8_bwd produces exactly their outputs with one call: it launches the key-major kernel first
 * and the query-major kernel behind it (the two are independent; the second starts on the SMs the
 * first one's last wave leaves idle), and both have completed when the stream reaches what follows. */
attn_status_t attn_fp8_bwd_dq(const attn_params_t* p, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                              attn_qtensor_t dO, const float* lse, const float* delta, void* dq_bf16,
                              float* diag_rowsum_ds, float* diag_rowsum_abs_ds,
                              void* workspace, size_t workspace_bytes, void* stream);
attn_status_t attn_fp8_bwd_dkdv(const attn_params_t* p, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                                attn_qtensor_t dO, const float* lse, const float* delta,
                                void* dk_bf16, void* dv_bf16,
                                void* workspace, size_t workspace_bytes, void* stream);

/* attn_fp8_bwd_dq with the post-cast probe of the paper's Appendix "dS Quantization Residuals"
 * (Eq. app_ds_quantization_residuals): besides the pre-cast sums it writes, per query row,
 *   diag_post_rowsum_ds      sum_j dS'_ij     dS' = the cast score gradient the dQ matmul consumes
 *   diag_post_rowsum_abs_ds  sum_j |dS'_ij|   (code * 2^(scale byte - 127); the BF16 value in BF16 mode)
 * both [B, Hq, N] FP32.  From the four outputs a caller forms r_pre, r_post, r_post,own and the
 * signed casting offset kappa.  All four diagnostic pointers are required; dQ is identical to
 * attn_fp8_bwd_dq's.                                                                          */
attn_status_t attn_fp8_bwd_dq_postcast(const attn_params_t* p, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                                       attn_qtensor_t dO, const float* lse, const float* delta, void* dq_bf16,
                                       float* diag_rowsum_ds, float* diag_rowsum_abs_ds,
                                       float* diag_post_rowsum_ds, float* diag_post_rowsum_abs_ds,
                                       void* workspace, size_t workspace_bytes, void* stream);

/* attn_fp8_bwd_dq with the quantities the per-row acceptance of the zero-row-sum invariant needs (paper
 * Section 3.3 Eq. 5; Appendix "Row-Sum Residuals").  With the matched correction the row sum of dS is, in
 * exact arithmetic, delta_i (1 - sum_j P_ij): zero up to the rounding of the FP32-stored LSE, which leaves
 * dust of size ulp(LSE_i) * sum_j P_ij |dP^_ij|.  Besides the pre-cast pair the call writes that last sum,
 *   diag_p_abs_dp   sum_j P_ij |dP^_ij|   [B, Hq, N] FP32,
 * so that a caller can test |sum_j dS| <= 1e-5 sum_j |dS| + (ulp(LSE_i) + c) * diag_p_abs_dp on EVERY row, c = 2^-20
 * for rows of up to 8192 keys (the FP32 summation of the normaliser and of delta), growing in proportion to
 * the key count beyond (rows that see one key, or are one-hot, have sum_j |dS| -> 0 and only the dust).  All three diagnostic
 * pointers are required; dQ is identical to attn_fp8_bwd_dq's.                                        */
attn_status_t attn_fp8_bwd_dq_rowprobe(const attn_params_t* p, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                                       attn_qtensor_t dO, const float* lse, const float* delta, void* dq_bf16,
                                       float* diag_rowsum_ds, float* diag_rowsum_abs_ds, float* diag_p_abs_dp,
                                       void* workspace, size_t workspace_bytes, void* stream);

/* Forward without a workspace argument (the paper has no counterpart; this is a packaging variant
 * of attn_fp8_fwd and computes exactly the same O and LSE).
 *
 * It is meant for callers that have no way to produce device scratch at the call site: code that
 * runs inside a host framework which owns all device memory and forbids allocation from within
 * an operator, services whose device memory is carved up once at start-up and must not grow, and
 * similar set-ups where cudaMalloc (or any allocating library routine) is off limits.  The scratch
 * the forward kernel needs is therefore a fixed 4096-byte array compiled into the library; every
 * GPU that loads the library holds those bytes until the process exits.  The call itself performs
 * no allocation and no free of any kind.
 *
 *   - Problems whose scratch need (attn_fp8_workspace_bytes(p, ATTN_WS_FWD)) exceeds 4096 bytes are
 *     rejected with ATTN_ERR_WORKSPACE and a message naming both sizes.
 *   - The first call on each device looks up the array's device address (a one-time runtime query
 *     made with that device current); make that first call outside of any stream capture.  The
 *     address is cached per device ordinal for the life of the process: it does not survive a
 *     cudaDeviceReset of that device (do not reset a device between calls of this library).
 *   - All calls on a device share the one array, and it keeps what earlier calls left; its
 *     status word is only ever set by a kernel that gave up, so nothing has to be cleared between
 *     calls and overlapping calls (different streams) do not disturb one another.
 *   - The device status word lands in the built-in array: attn_fp8_read_status(NULL, stream) reads
 *     (and, if set, clears) it.
 * Arguments, layouts and error codes are otherwise those of attn_fp8_fwd.                       */
attn_status_t attn_fp8_fwd_noalloc(const attn_params_t* p, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                                   void* o_bf16, float* lse, void* stream);

/* Bytes of workspace the given entry point needs for `p` (attn_ws_kind_t).  The workspace is
 * scratch owned by the caller; one workspace may serve all entry points of a stream.  Its first
 * word is the device-side status word; the rest of its first ATTN_STATUS_WORKSPACE_BYTES bytes holds
 * counters the kernels of one call share (each call clears its own: give concurrent streams
 * separate workspaces).  The status is STICKY: kernels only ever set it (a bounded
 * wait that gave up, a launch that found its shared memory misaligned), no entry point clears it,
 * so one attn_fp8_read_status at the end of a chain of calls reports a failure of any of them.
 * A workspace must be initialised once before its first use (attn_fp8_workspace_init, or any other
 * way of zeroing its first ATTN_STATUS_WORKSPACE_BYTES bytes): an uninitialised status word reads
 * as an error.                                                                                 */
size_t attn_fp8_workspace_bytes(const attn_params_t* p, int32_t which);

/* Enqueues the clearing of the status header of `workspace` (>= ATTN_STATUS_WORKSPACE_BYTES,
 * 16-byte aligned) on `stream`.  Once per workspace, before its first use.                     */
attn_status_t attn_fp8_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/* Waits for `stream`, copies the status word of `workspace` to the host and returns it:
 * ATTN_OK, or ATTN_ERR_TIMEOUT / ATTN_ERR_ALIGNMENT if a kernel of any call since the last read (or
 * the initialisation) gave up (outputs of those calls are then undefined).  A non-OK status is
 * cleared by the read.  workspace == NULL means the library's built-in scratch array on the current
 * device, where the entry points without a workspace argument (attn_fp8_quantize,
 * attn_fp8_fwd_noalloc) report.  This is the one call that synchronises.                        */
attn_status_t attn_fp8_read_status(void* workspace, void* stream);

/* Self-test of the device-side time-out report: enqueues a one-CTA kernel that waits, with a limit
 * of about 2 ms, on a barrier nothing completes, gives up and sets the status word of `workspace`
 * (>= attn_fp8_workspace_bytes) exactly as an attention kernel whose wait expired would.  A later
 * attn_fp8_read_status(workspace) therefore returns ATTN_ERR_TIMEOUT; the context stays usable.
 * workspace == NULL (workspace_bytes ignored) targets the built-in scratch array of the current device.
 * For tests of the error path: nothing faults, traps or hangs.                                 */
attn_status_t attn_fp8_selftest_timeout(void* workspace, size_t workspace_bytes, void* stream);

/* Measurement aid (the paper has no counterpart): the rate, in TFLOP/s, at which this device executes
 * the bare block-scaled FP8 tensor-core instruction the attention kernels are built on (E4M3 operands,
 * E8M0 scales, 128 x 224 x 32 per instruction, two issuing warps per SM, operands resident in shared
 * memory), written to *tflops (host).  Runs a few milliseconds of such instructions on `stream` three
 * times (the first warms the clocks up; the faster of the other two counts) and WAITS for them: unlike
 * the other entry points this one synchronises the stream.  `workspace` as for the attention calls
 * (status word).  Allocates no device memory.                                                       */
attn_status_t attn_fp8_measure_mma_peak(double* tflops, void* workspace, size_t workspace_bytes, void* stream);

/* Measurement aid for one design question (the paper's Limitations name a fused gradient pass as open
 * engineering; it has no such kernel): what the FP32 reduction of dQ alone would cost if the key-major
 * kernel also produced dQ.  Issues, with no other work, the adds such a pass would make for the shape `p`
 * (one [64 x head_dim_qk] FP32 partial per key tile of 128 and query sub-tile of 64 that the mask keeps,
 * red.global.add.v4.f32 of ones, one CTA per (KV head, key tile, batch)) into `dq_f32`
 * ([B, Hq, N, head_dim_qk] FP32, device, >= that many bytes; cleared by the call), three times, and WAITS:
 * *ms = the faster of the last two passes, *bytes = the bytes added per pass.  Afterwards element
 * (b, h, i, c) holds the number of key tiles row i sees.  Allocates nothing.                           */
attn_status_t attn_fp8_measure_dq_reduction(const attn_params_t* p, float* dq_f32, size_t dq_f32_bytes, double* ms,
                                            double* bytes, void* stream);

/* Message for the last non-OK return on this host thread (static storage; never NULL).        */
const char* attn_fp8_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* ATTN_FP8_H_ */
