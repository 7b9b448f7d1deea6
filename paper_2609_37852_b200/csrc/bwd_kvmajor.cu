// Key-major backward kernel: dK and dV (paper Appendix "Backward Correction and Gradient
// Computation", paragraph "Score-gradient quantization", merged with the GQA group reduction).
//
// One CTA owns 128 keys of one (batch, KV head).  It loops over the query heads of the group and,
// for each, over the query tiles from the causal diagonal to the end, 64 query rows at a time.
// Per sub-tile the tensor cores recompute the TRANSPOSED products
//     S^T  = K^ Q^^T    (128 keys x 64 queries; row-blocked FP8 copies)
//     dP^T = V^ dO^^T
// so that a softmax thread owns one key (one TMEM lane) and sees 32 consecutive query rows in
// its registers: exactly one quantisation block of the operands P^T and dS^T, whose matmuls
// contract over the query index.  The thread rebuilds P = 2^(S*scale*log2e - LSE_i*log2e),
// forms dS = P (dP - D_i) in FP32, quantises both in registers, and the tensor cores accumulate
//     dV += P^^T dO^c      dK += dS^^T Q^c      (copies of dO, Q blocked along tokens)
// in tensor memory across all query tiles and all query heads of the group: the group sum is
// an FP32 sum, rounded to BF16 once at the end.
//
// Warp roles: warp 0 TMA producer; warps 1, 2, 3 issue the S^T, dP^T and dV/dK MMAs (one warp
// cannot issue tcgen05.mma fast enough for small tiles); warps 4..19 are two softmax teams that
// take alternate sub-tiles (within a team, warp % 4 selects the 32 TMEM lanes and the column
// group w takes query columns 32w..32w+31).
#include <cuda_bf16.h>

#include <type_traits>

#include "common.cuh"
#include "mxfp8_device.cuh"
#include "sm100_ptx.cuh"

namespace attnfp8 {

#ifdef ATTN_TRACE
// Debug build only: clock stamps of one CTA (roles x steps x events), read back by the host.
__device__ long long g_kv_trace[4][256][4];
#define KV_TRACE(role, step, ev) do { if (blockIdx.x == 0 && blockIdx.y == 0 && (step) < 256) g_kv_trace[role][step][ev] = clock64(); } while (0)
extern "C" int attn_fp8_debug_kv_trace(long long* host_out) {
  return static_cast<int>(cudaMemcpyFromSymbol(host_out, g_kv_trace, sizeof(g_kv_trace)));
}
#else
#define KV_TRACE(role, step, ev) do { } while (0)
#endif

namespace {

using namespace sm100;

constexpr int kTile = 128;
constexpr int kSub = 64;
// Per query tile the CTA streams a 'row' set (Q and dO row copies, their scales, LSE, D: read by
// the S^T / dP^T MMAs and the softmax) and a 'col' set (Q and dO column copies: read by the dV / dK
// MMAs).  The row set is released early and has three stages, so that a reload never sits between
// the end of one tile's gradient MMAs and the start of the next tile's scores.
constexpr int kRowStages = 3;
constexpr int kColStages = 2;
constexpr int kTeams = 2;                       // softmax teams; team t takes sub-tiles u with u % kTeams == t
constexpr int kTeamThreads = 256;               // 8 warps: 4 TMEM lane quadrants x 2 column groups
constexpr int kThreads = 128 + kTeams * kTeamThreads;
constexpr int kPrepThreads = 32;                // warp 2 turns LSE into -LSE*log2(e) once per query tile
constexpr float kLog2e = 1.4426950408889634f;

constexpr uint32_t kColS = 0, kColdP = 64, kColP = 128 /* 2 x 16 */, kColdS = 160 /* 2 x 16 */;
constexpr uint32_t kColdV = 192, kColdK = 320;
constexpr uint32_t kColSFK = 448, kColSFV = 452, kColSFQ = 456 /* 2 x 4 */, kColSFdO = 464 /* 2 x 4 */,
                   kColSFP = 472 /* 2 x 4 */, kColSFdS = 480 /* 2 x 4 */, kColSFdOc = 488 /* 2 x 4 */,
                   kColSFQc = 496 /* 2 x 4 */;
constexpr uint32_t kTmemCols = 512;

struct KvRowStage {
  alignas(1024) uint8_t q[kTile * 128];       // Q row copy  [128 queries][dqk]
  alignas(1024) uint8_t dO[kTile * 128];      // dO row copy [128 queries][dv]
  alignas(16) uint8_t sf_q[512];
  alignas(16) uint8_t sf_dO[512];
  alignas(16) float lse[kTile];
  alignas(16) float delta[kTile];
  alignas(16) float neg_lse2[kTile];          // -LSE * log2(e), written by the prep warp
};
struct KvColStage {
  alignas(1024) uint8_t qc[kTile * 128];      // Q col copy  [dqk][128 queries]
  alignas(1024) uint8_t dOc[kTile * 128];     // dO col copy [dv][128 queries]
  alignas(16) uint8_t sf_qc[512];
  alignas(16) uint8_t sf_dOc[512];
};

struct KvSmem {
  alignas(1024) uint8_t k[kTile * 128];
  alignas(1024) uint8_t v[kTile * 128];
  KvRowStage rst[kRowStages];
  KvColStage cst[kColStages];
  alignas(16) uint8_t sf_k[512];
  alignas(16) uint8_t sf_v[512];
  alignas(16) uint8_t sf_p[2][512];
  alignas(16) uint8_t sf_ds[2][512];
  uint64_t kv_full;
  uint64_t row_full[kRowStages], row_empty[kRowStages];
  uint64_t col_full[kColStages], col_empty[kColStages];
  uint64_t lse_ready[kRowStages];
  uint64_t sdp_full[kTeams], sdp_free[kTeams];
  uint64_t pds_full[2], pds_free[2];
  uint64_t done;
  uint64_t drain[3];
  uint32_t tmem_base;
  int abort_flag;
};

struct KvParams {
  const uint8_t *k_sf, *v_sf, *q_sf, *dO_sf, *qc_sf, *dOc_sf;
  const float* lse;
  const float* delta;
  __nv_bfloat16* dk;
  __nv_bfloat16* dv_out;
  int* status;
  int N, Hq, Hkv, dqk, dv, causal;
  float scale, scale_log2;
};

__global__ void __launch_bounds__(kThreads, 1)
kvmajor_kernel(const KvParams p, const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
               const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_dO,
               const __grid_constant__ CUtensorMap tm_qc, const __grid_constant__ CUtensorMap tm_dOc) {
  extern __shared__ uint8_t smem_raw[];
  KvSmem& sm = *reinterpret_cast<KvSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // blocks are handed out x-fastest: KV heads vary fastest, key tiles in order, so the heaviest
  // tiles (the earliest keys under the causal mask) of all heads go first
  const int jt = blockIdx.y;
  const int g = blockIdx.x, b = blockIdx.z;
  const int G = p.Hq / p.Hkv;
  const int tiles_n = p.N / kTile;
  const int it0 = p.causal ? jt : 0;                // first query tile that sees these keys
  const int tiles_per_head = tiles_n - it0;
  const int n_qtiles = G * tiles_per_head;          // query tiles this CTA walks
  const int n_sub = 2 * n_qtiles;
  const int nk_qk = p.dqk / 32, nk_v = p.dv / 32;
  volatile int* abort_flag = &sm.abort_flag;

  if (tid == 0) {
    mbar_init(&sm.kv_full, 1);
    for (int s = 0; s < kRowStages; ++s) {
      mbar_init(&sm.row_full[s], 1); mbar_init(&sm.row_empty[s], 1);      // released once both softmax teams are done with the tile
      mbar_init(&sm.lse_ready[s], 1);                 // one arrival by the prep warp
    }
    for (int s = 0; s < kColStages; ++s) { mbar_init(&sm.col_full[s], 1); mbar_init(&sm.col_empty[s], 1); }
    for (int t = 0; t < kTeams; ++t) { mbar_init(&sm.sdp_full[t], 2); mbar_init(&sm.sdp_free[t], kTeamThreads); }
    for (int i = 0; i < 2; ++i) { mbar_init(&sm.pds_full[i], kTeamThreads); mbar_init(&sm.pds_free[i], 1); }
    for (int i = 0; i < 3; ++i) mbar_init(&sm.drain[i], 1);
    mbar_init(&sm.done, 1);
    sm.abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&sm.tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sm.tmem_base;


  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      prefetch_tmap(&tm_k); prefetch_tmap(&tm_v); prefetch_tmap(&tm_q); prefetch_tmap(&tm_dO);
      prefetch_tmap(&tm_qc); prefetch_tmap(&tm_dOc);
      const int kv_slab = b * p.Hkv + g;
      mbar_arrive_expect_tx(&sm.kv_full, 2 * (kTile * 128 + 512));
      tma_load_2d(sm.k, &tm_k, &sm.kv_full, 0, kv_slab * p.N + jt * kTile);
      tma_load_2d(sm.v, &tm_v, &sm.kv_full, 0, kv_slab * p.N + jt * kTile);
      bulk_load_1d(sm.sf_k, p.k_sf + (static_cast<size_t>(kv_slab) * tiles_n + jt) * 512, 512, &sm.kv_full);
      bulk_load_1d(sm.sf_v, p.v_sf + (static_cast<size_t>(kv_slab) * tiles_n + jt) * 512, 512, &sm.kv_full);
      int issued_row = 0, issued_col = 0;
      bool ok = true;
      for (int n = 0; n < n_qtiles && ok; ++n) {
        const int rs = n % kRowStages, cs = n % kColStages;
        const int h = g * G + n / tiles_per_head, it = it0 + n % tiles_per_head;
        const int q_slab = b * p.Hq + h;
        const size_t sf_tile = (static_cast<size_t>(q_slab) * tiles_n + it) * 512;
        const size_t row0 = static_cast<size_t>(q_slab) * p.N + it * kTile;
        ok = mbar_wait(&sm.row_empty[rs], ((n / kRowStages) & 1) ^ 1, abort_flag);
        if (!ok) break;
        KvRowStage& r = sm.rst[rs];
        mbar_arrive_expect_tx(&sm.row_full[rs], 2 * kTile * 128 + 2 * 512 + 2 * kTile * 4);
        tma_load_2d(r.q, &tm_q, &sm.row_full[rs], 0, q_slab * p.N + it * kTile);
        tma_load_2d(r.dO, &tm_dO, &sm.row_full[rs], 0, q_slab * p.N + it * kTile);
        bulk_load_1d(r.sf_q, p.q_sf + sf_tile, 512, &sm.row_full[rs]);
        bulk_load_1d(r.sf_dO, p.dO_sf + sf_tile, 512, &sm.row_full[rs]);
        bulk_load_1d(r.lse, p.lse + row0, kTile * 4, &sm.row_full[rs]);
        bulk_load_1d(r.delta, p.delta + row0, kTile * 4, &sm.row_full[rs]);
        ++issued_row;
        ok = mbar_wait(&sm.col_empty[cs], ((n / kColStages) & 1) ^ 1, abort_flag);
        if (!ok) break;
        KvColStage& c = sm.cst[cs];
        mbar_arrive_expect_tx(&sm.col_full[cs], (p.dqk + p.dv) * 128 + 2 * 512);
        tma_load_2d(c.qc, &tm_qc, &sm.col_full[cs], it * kTile, q_slab * p.dqk);
        tma_load_2d(c.dOc, &tm_dOc, &sm.col_full[cs], it * kTile, q_slab * p.dv);
        bulk_load_1d(c.sf_qc, p.qc_sf + sf_tile, 512, &sm.col_full[cs]);
        bulk_load_1d(c.sf_dOc, p.dOc_sf + sf_tile, 512, &sm.col_full[cs]);
        ++issued_col;
      }
      if (!ok) {
        int dummy = 0;
        for (int n = max(0, issued_row - kRowStages); n < issued_row; ++n)
          mbar_wait(&sm.row_full[n % kRowStages], (n / kRowStages) & 1, &dummy);
        for (int n = max(0, issued_col - kColStages); n < issued_col; ++n)
          mbar_wait(&sm.col_full[n % kColStages], (n / kColStages) & 1, &dummy);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ S^T issuer
    // One tcgen05.mma can be issued per ~130 cycles from one warp whatever its size, so the
    // products are spread over three issuing warps; orderings that a single issuer would give
    // for free are carried by mbarriers instead.
    {
      const uint64_t desc_k = make_desc_sw128(smem_u32(sm.k));
      bool ok = mbar_wait(&sm.kv_full, 0, abort_flag);
      if (ok) {
        tc_fence_after_sync();
        sf_copy_elect(tmem + kColSFK, make_desc_sf(smem_u32(sm.sf_k)));
      }
      for (int u = 0; u < n_sub && ok; ++u) {
        const int n = u >> 1, half = u & 1, s = n % kRowStages, slot = n & 1;
        KvRowStage& st = sm.rst[s];
        if (half == 0) {
          ok = mbar_wait(&sm.row_full[s], (n / kRowStages) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          sf_copy_elect(tmem + kColSFQ + 4 * slot, make_desc_sf(smem_u32(st.sf_q)));
        }
        KV_TRACE(0, u, 0);
        if (u > 0) {
          // the team of the previous sub-tile has pulled S and dP into registers
          ok = mbar_wait(&sm.sdp_free[(u - 1) % kTeams], ((u - 1) / kTeams) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
        }
        KV_TRACE(0, u, 1);
        const uint64_t desc_q = make_desc_sw128(smem_u32(st.q)) + half * (kSub * 128 / 16);
        for (int kb = 0; kb < nk_qk; ++kb)
          mma_mxf8_ss_elect(tmem + kColS, desc_k + 2 * kb, desc_q + 2 * kb, make_idesc_mxf8(128, kSub, kb, kb),
                      tmem + kColSFK, tmem + kColSFQ + 4 * slot + 2 * half, kb > 0);
        mma_commit_elect(&sm.sdp_full[u % kTeams]);
        KV_TRACE(0, u, 2);
      }
      if (!ok) {
        int dummy = 0;
        mma_commit_elect(&sm.drain[0]);
        mbar_wait(&sm.drain[0], 0, &dummy);
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ dP^T issuer + LSE preparation
    const uint64_t desc_v = make_desc_sw128(smem_u32(sm.v));
    bool ok = mbar_wait(&sm.kv_full, 0, abort_flag);
    if (ok) {
      tc_fence_after_sync();
      sf_copy_elect(tmem + kColSFV, make_desc_sf(smem_u32(sm.sf_v)));
    }
    for (int u = 0; u < n_sub && ok; ++u) {
      const int n = u >> 1, half = u & 1, s = n % kRowStages, slot = n & 1;
      KvRowStage& st = sm.rst[s];
      if (half == 0) {
        ok = mbar_wait(&sm.row_full[s], (n / kRowStages) & 1, abort_flag);
        if (!ok) break;
        // every lane turns four LSE values into -LSE*log2(e) for the softmax teams
        const float4 l = *reinterpret_cast<const float4*>(&st.lse[4 * lane]);
        *reinterpret_cast<float4*>(&st.neg_lse2[4 * lane]) =
            make_float4(-l.x * kLog2e, -l.y * kLog2e, -l.z * kLog2e, -l.w * kLog2e);
        mbar_arrive_warp(&sm.lse_ready[s]);
        {
          tc_fence_after_sync();
          sf_copy_elect(tmem + kColSFdO + 4 * slot, make_desc_sf(smem_u32(st.sf_dO)));
        }
      }
      if (u > 0) {
        ok = mbar_wait(&sm.sdp_free[(u - 1) % kTeams], ((u - 1) / kTeams) & 1, abort_flag);
        if (!ok) break;
      }
      {
        tc_fence_after_sync();
        const uint64_t desc_dO = make_desc_sw128(smem_u32(st.dO)) + half * (kSub * 128 / 16);
        for (int kb = 0; kb < nk_v; ++kb)
          mma_mxf8_ss_elect(tmem + kColdP, desc_v + 2 * kb, desc_dO + 2 * kb, make_idesc_mxf8(128, kSub, kb, kb),
                      tmem + kColSFV, tmem + kColSFdO + 4 * slot + 2 * half, kb > 0);
        mma_commit_elect(&sm.sdp_full[u % kTeams]);
      }
    }
    if (!ok) {
      int dummy = 0;
      mma_commit_elect(&sm.drain[1]);
      mbar_wait(&sm.drain[1], 0, &dummy);
    }
  } else if (warp == 3) {
    // ------------------------------------------------------------------ dV / dK issuer
    {
      bool ok = true;
      for (int u = 0; u < n_sub && ok; ++u) {
        const int n = u >> 1, half = u & 1, s = n % kColStages, slot = n & 1, buf = u & 1;
        KvColStage& st = sm.cst[s];
        if (half == 0) {
          ok = mbar_wait(&sm.col_full[s], (n / kColStages) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          sf_copy_elect(tmem + kColSFdOc + 4 * slot, make_desc_sf(smem_u32(st.sf_dOc)));
          sf_copy_elect(tmem + kColSFQc + 4 * slot, make_desc_sf(smem_u32(st.sf_qc)));
        }
        KV_TRACE(1, u, 0);
        ok = mbar_wait(&sm.pds_full[buf], (u >> 1) & 1, abort_flag);
        if (!ok) break;
        KV_TRACE(1, u, 1);
        // both halves of the tile have been through the softmax: its row set (scores operands,
        // LSE, D) is no longer read
        if (half == 1 && lane == 0) mbar_arrive(&sm.row_empty[n % kRowStages]);
        tc_fence_after_sync();
        sf_copy_elect(tmem + kColSFP + 4 * buf, make_desc_sf(smem_u32(sm.sf_p[buf])));
        sf_copy_elect(tmem + kColSFdS + 4 * buf, make_desc_sf(smem_u32(sm.sf_ds[buf])));
        const uint64_t desc_dOc = make_desc_sw128(smem_u32(st.dOc));
        const uint64_t desc_qc = make_desc_sw128(smem_u32(st.qc));
        for (int kb = 0; kb < 2; ++kb)
          mma_mxf8_ts_elect(tmem + kColdV, tmem + kColP + 16 * buf + 8 * kb, desc_dOc + 2 * (2 * half + kb),
                      make_idesc_mxf8(128, p.dv, kb, 2 * half + kb), tmem + kColSFP + 4 * buf,
                      tmem + kColSFdOc + 4 * slot, (u > 0 || kb > 0));
        for (int kb = 0; kb < 2; ++kb)
          mma_mxf8_ts_elect(tmem + kColdK, tmem + kColdS + 16 * buf + 8 * kb, desc_qc + 2 * (2 * half + kb),
                      make_idesc_mxf8(128, p.dqk, kb, 2 * half + kb), tmem + kColSFdS + 4 * buf,
                      tmem + kColSFQc + 4 * slot, (u > 0 || kb > 0));
        // codes and scale bytes of this buffer may be overwritten once these MMAs have run; the
        // stage may be refilled after the second half (the S^T / dP^T MMAs that read it finished
        // before the softmax team could even start on this sub-tile)
        mma_commit_elect(&sm.pds_free[buf]);
        KV_TRACE(1, u, 2);
        if (half == 1) mma_commit_elect(&sm.col_empty[s]);
        if (u == n_sub - 1) mma_commit_elect(&sm.done);
      }
      if (!ok) {
        int dummy = 0;
        mma_commit_elect(&sm.drain[2]);
        mbar_wait(&sm.drain[2], 0, &dummy);
      }
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ softmax
    const int team = (warp - 4) >> 3;
    const int grp = ((warp - 4) >> 2) & 1;
    const int quad = warp & 3;
    const int row = quad * 32 + lane;                 // key inside the tile == TMEM lane
    const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
    bool ok = true;
    for (int u = team; u < n_sub; u += kTeams) {
      const int n = u >> 1, half = u & 1, buf = u & 1, s = n % kRowStages;
      const int it = it0 + n % tiles_per_head;
      if (quad == 0 && lane == 0 && grp == 0) KV_TRACE(2, u, 0);
      ok = mbar_wait(&sm.sdp_full[team], (u / kTeams) & 1, abort_flag);
      if (!ok) break;
      if (quad == 0 && lane == 0 && grp == 0) KV_TRACE(2, u, 1);
      tc_fence_after_sync();
      uint32_t sr[32], dpr[32];                       // S then P; dP then dS (in place)
      tmem_ld32(tmem + kColS + lane_addr + 32 * grp, sr);
      tmem_ld32(tmem + kColdP + lane_addr + 32 * grp, dpr);
      tmem_wait_ld();
      tc_fence_before_sync();
      mbar_arrive(&sm.sdp_free[team]);
      if (quad == 0 && lane == 0 && grp == 0) KV_TRACE(2, u, 2);
      ok = mbar_wait(&sm.lse_ready[s], (n / kRowStages) & 1, abort_flag);
      if (!ok) break;
      const int col0 = half * kSub + 32 * grp;        // query row (inside the tile) of this thread's first column
      const KvRowStage& st = sm.rst[s];
      float amax_p = 0.f, max_s = 0.f;
      const float* s_lse = &st.neg_lse2[col0];
      const float* s_delta = &st.delta[col0];
      auto body = [&](auto diag_tag) {
        constexpr bool kDiag = decltype(diag_tag)::value;
#pragma unroll
        for (int c4 = 0; c4 < 32; c4 += 4) {
          const float4 l4 = lds_f4(&s_lse[c4]);
          const float4 d4 = lds_f4(&s_delta[c4]);
          const float lv[4] = {l4.x, l4.y, l4.z, l4.w};
          const float dv4[4] = {d4.x, d4.y, d4.z, d4.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int c = c4 + e;
            float x = fmaf(__uint_as_float(sr[c]), p.scale_log2, lv[e]);
            if (kDiag && (row > col0 + c)) x = -INFINITY;      // key after the query
            const float pv = ex2_approx(x);
            const float dsv = pv * (__uint_as_float(dpr[c]) - dv4[e]);
            sr[c] = __float_as_uint(pv);
            dpr[c] = __float_as_uint(dsv);
            amax_p = fmaxf(amax_p, pv);
            max_s = fmaxf(max_s, fabsf(dsv));
          }
        }
      };
      if (p.causal && it == jt) body(std::true_type{}); else body(std::false_type{});
      uint32_t byte_p, byte_s;
      float inv_p, inv_s;
      block_scale(amax_p, byte_p, inv_p);
      block_scale(max_s, byte_s, inv_s);
      if (u >= 2) {
        // the dV / dK MMAs of sub-tile u-2 have consumed this buffer's codes and scale bytes
        ok = mbar_wait(&sm.pds_free[buf], ((u - 2) >> 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after_sync();
      }
      uint32_t words[8];
#pragma unroll
      for (int i = 0; i < 8; ++i)
        words[i] = cvt_e4m3x4(__uint_as_float(sr[4 * i]) * inv_p, __uint_as_float(sr[4 * i + 1]) * inv_p,
                              __uint_as_float(sr[4 * i + 2]) * inv_p, __uint_as_float(sr[4 * i + 3]) * inv_p);
      tmem_st8(tmem + kColP + 16 * buf + lane_addr + 8 * grp, words);
#pragma unroll
      for (int i = 0; i < 8; ++i)
        words[i] = cvt_e4m3x4(__uint_as_float(dpr[4 * i]) * inv_s, __uint_as_float(dpr[4 * i + 1]) * inv_s,
                              __uint_as_float(dpr[4 * i + 2]) * inv_s, __uint_as_float(dpr[4 * i + 3]) * inv_s);
      tmem_st8(tmem + kColdS + 16 * buf + lane_addr + 8 * grp, words);
      const int sf_at = (row & 31) * 16 + (row >> 5) * 4 + grp;
      sts_u8(&sm.sf_p[buf][sf_at], byte_p);
      sts_u8(&sm.sf_ds[buf][sf_at], byte_s);
      tmem_wait_st();
      fence_proxy_async_smem();
      tc_fence_before_sync();
      mbar_arrive(&sm.pds_full[buf]);
      if (quad == 0 && lane == 0 && grp == 0) KV_TRACE(2, u, 3);
    }
    // the epilogue is done by team 0 (group 0 stores dV, group 1 stores dK)
    if (team != 0) ok = false;
    if (ok) ok = mbar_wait(&sm.done, 0, abort_flag);
    if (ok) {
      tc_fence_after_sync();
      const size_t grow = static_cast<size_t>(b * p.Hkv + g) * p.N + jt * kTile + row;
      // group 0 stores dV, group 1 stores dK (scaled)
      const uint32_t col = grp == 0 ? kColdV : kColdK;
      const int width = grp == 0 ? p.dv : p.dqk;
      const float mul = grp == 0 ? 1.f : p.scale;
      __nv_bfloat16* out_row = (grp == 0 ? p.dv_out : p.dk) + grow * width;
      for (int c0 = 0; c0 < width; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tmem + col + lane_addr + c0, r);
        tmem_wait_ld();
        uint32_t packed[16];
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          __nv_bfloat162 v2 = __floats2bfloat162_rn(__uint_as_float(r[2 * c]) * mul, __uint_as_float(r[2 * c + 1]) * mul);
          packed[c] = *reinterpret_cast<uint32_t*>(&v2);
        }
        uint4* dst = reinterpret_cast<uint4*>(out_row + c0);
#pragma unroll
        for (int c = 0; c < 4; ++c) dst[c] = make_uint4(packed[4 * c], packed[4 * c + 1], packed[4 * c + 2], packed[4 * c + 3]);
      }
    }
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
  if (tid == 0 && sm.abort_flag) atomicExch(p.status, static_cast<int>(ATTN_ERR_TIMEOUT));
}

}  // namespace

attn_status_t launch_bwd_dkdv(const AttnShape& s, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v, attn_qtensor_t dO,
                              const float* lse, const float* delta, void* dk, void* dv, int* status,
                              cudaStream_t stream) {
  CUtensorMap tm_k, tm_v, tm_q, tm_dO, tm_qc, tm_dOc;
  attn_status_t st;
  const uint64_t q_rows = static_cast<uint64_t>(s.B) * s.Hq * s.N, kv_rows = static_cast<uint64_t>(s.B) * s.Hkv * s.N;
  if ((st = encode_tmap_u8_sw128(&tm_k, k.row_codes, s.dqk, kv_rows, kTile)) != ATTN_OK) return st;
  if ((st = encode_tmap_u8_sw128(&tm_v, v.row_codes, s.dv, kv_rows, kTile)) != ATTN_OK) return st;
  if ((st = encode_tmap_u8_sw128(&tm_q, q.row_codes, s.dqk, q_rows, kTile)) != ATTN_OK) return st;
  if ((st = encode_tmap_u8_sw128(&tm_dO, dO.row_codes, s.dv, q_rows, kTile)) != ATTN_OK) return st;
  if ((st = encode_tmap_u8_sw128(&tm_qc, q.col_codes, s.N, static_cast<uint64_t>(s.B) * s.Hq * s.dqk, s.dqk)) != ATTN_OK) return st;
  if ((st = encode_tmap_u8_sw128(&tm_dOc, dO.col_codes, s.N, static_cast<uint64_t>(s.B) * s.Hq * s.dv, s.dv)) != ATTN_OK) return st;
  KvParams p;
  p.k_sf = k.row_scales; p.v_sf = v.row_scales; p.q_sf = q.row_scales; p.dO_sf = dO.row_scales;
  p.qc_sf = q.col_scales; p.dOc_sf = dO.col_scales;
  p.lse = lse; p.delta = delta;
  p.dk = static_cast<__nv_bfloat16*>(dk); p.dv_out = static_cast<__nv_bfloat16*>(dv); p.status = status;
  p.N = s.N; p.Hq = s.Hq; p.Hkv = s.Hkv; p.dqk = s.dqk; p.dv = s.dv; p.causal = s.causal;
  p.scale = s.scale; p.scale_log2 = s.scale * kLog2e;
  const size_t smem = sizeof(KvSmem) + 1024;
  cudaError_t e = cudaFuncSetAttribute(kvmajor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "bwd kv-major: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  dim3 grid(s.Hkv, s.N / kTile, s.B);
  kvmajor_kernel<<<grid, kThreads, smem, stream>>>(p, tm_k, tm_v, tm_q, tm_dO, tm_qc, tm_dOc);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "bwd kv-major: launch: %s", cudaGetErrorString(e));
  return ATTN_OK;
}

}  // namespace attnfp8
