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
//
// The kernel is a template over the operand width (element bytes 1: E4M3 codes with E8M0 block
// scales, 2: BF16 without scales; 128-byte chunks per operand row) and over which gradients it
// accumulates.  The column copies are streamed one 128-byte chunk of the query dimension at a
// time (128 queries of codes, 64 of BF16); the row copies 128 queries at a time in the narrow FP8
// configuration and 64 otherwise.  When dV and dK together do not fit in tensor memory beside the
// score tiles (qk head dim above 128), the launcher runs the kernel twice: a pass that rebuilds P
// and accumulates dV, and a pass that rebuilds P and dS and accumulates dK.
#include <cuda_bf16.h>

#include <type_traits>

#include "common.cuh"
#include "mma_issue.cuh"
#include "mxfp8_device.cuh"
#include "sm100_ptx.cuh"

namespace attnfp8 {

namespace {

using namespace sm100;

constexpr int kTile = 128;
constexpr int kSub = 64;
constexpr int kTeams = 2;                       // softmax teams; team t takes sub-tiles u with u % kTeams == t
constexpr int kTeamThreads = 256;               // 8 warps: 4 TMEM lane quadrants x 2 column groups
constexpr int kThreads = 128 + kTeams * kTeamThreads;
constexpr float kLog2e = 1.4426950408889634f;
constexpr int kSmemLimit = 232448;              // dynamic shared memory a CTA may ask for

enum KvMode { kBoth = 0, kDvOnly = 1, kDkOnly = 2 };

// Operand geometry, ring depths and tensor-memory map of one instantiation.
template <int kEB_, int kCq_, int kCv_, int kMode_, int kEBv_ = kEB_, int kDkTile_ = -1>
struct KvCfg {
  static constexpr int kEB = kEB_, kCq = kCq_, kCv = kCv_, kMode = kMode_;
  static constexpr int kEBv = kEBv_;                   // bytes per element of the V / dO row operands (dP^T only):
                                                       // 2 with kEB == 1 is the protected-dP ablation
  static constexpr bool kFp8 = kEB == 1;
  static constexpr bool kFp8v = kEBv == 1;
  static constexpr bool kHasDv = kMode != kDkOnly;     // accumulates dV (needs P^)
  static constexpr bool kHasDk = kMode != kDvOnly;     // accumulates dK (needs dP^T, D, dS^)
  static constexpr int kRq = kCq / kEB > 0 ? (kCq + kEB - 1) / kEB : 1;   // 128-row tiles of the Q^c operand (dqk / 128, rounded up)
  static constexpr int kRv = (kCv + kEBv - 1) / kEBv;                     // 128-row tiles of the dO^c operand
  // BF16 at head dim 256: K, V and one row stage fill shared memory, so a dK pass takes one 128-column
  // tile of dK (kDkTile = 0, 1) and the launcher runs one pass per tile
  static constexpr int kDkTile = kDkTile_;
  static constexpr int kRqAcc = kDkTile >= 0 ? 1 : kRq;                   // 128-row tiles of Q^c a pass accumulates into dK
  // Per query tile the CTA streams a 'row' set (Q and dO row copies, their scales, LSE, D: read by
  // the S^T / dP^T MMAs and the softmax) and a 'col' set (Q and dO column copies: read by the dV /
  // dK MMAs).  The row set is released early and gets the deeper ring, so that a reload never sits
  // between the end of one tile's gradient MMAs and the start of the next tile's scores.
  static constexpr int kRowTok = (kFp8 && kCq == 1 && kCv == 1) ? 128 : 64;   // queries per row stage
  static constexpr int kColTok = kTile / kEB;                                 // queries per col stage
  static constexpr int kSubPerRow = kRowTok / kSub, kSubPerCol = kColTok / kSub;
  static constexpr int kKvBytes = (kCq + (kHasDk ? kCv : 0)) * kTile * 128;
  static constexpr int kRowBytes = (kCq + (kHasDk ? kCv : 0)) * kRowTok * 128;
  // (192,128) with both gradients in one pass (see kTight below): the Q^c stage holds the 192 rows it is
  // loaded with, not two full row tiles, which leaves room for a third row stage
  static constexpr bool kTightDims = kMode_ == kBoth && ((kEB == 1 && kEBv == 1 && kCq == 2 && kCv == 1) || (kEB == 2 && kEBv == 2 && kCq == 3 && kCv == 2));
  static constexpr int kQcRows = kTightDims ? 192 : kRqAcc * kTile;
  static constexpr int kColBytes = ((kHasDk ? kQcRows : 0) + (kHasDv ? kRv * kTile : 0)) * 128;
  // rings shrink to one stage where two do not fit (wide heads in BF16 mode): loads and MMAs of
  // successive steps then no longer overlap
  static constexpr int kColStages = kKvBytes + 2 * kRowBytes + 2 * kColBytes <= 210 * 1024 ? 2 : 1;
  static constexpr int kRowRaw = (216 * 1024 - kKvBytes - kColStages * kColBytes) / kRowBytes;
  static constexpr bool kTwoRowsFit = kKvBytes + kColStages * kColBytes + 2 * kRowBytes <= 214 * 1024;
  static constexpr int kRowCap = 3;
  static constexpr int kRowStages = kRowRaw < 2 ? (kTwoRowsFit ? 2 : 1) : (kRowRaw > kRowCap ? kRowCap : kRowRaw);
  // 64-query row stages (one sub-tile each): -LSE*log2(e) and -D of a sub-tile live in a small ring
  // of their own, written by the preparation warp, so that the operand part of a row stage is released as soon
  // as the S^T / dP^T MMAs that read it have run, not when the softmax is done with the sub-tile: the reload is
  // in flight a whole softmax step earlier.  Slot reuse is safe kRowStages + 3 sub-tiles later (the row load
  // that precedes the rewrite waits for the MMAs of sub-tile u + 3, which are issued after the team of u has
  // taken S of u + 2, i.e. finished u); an even count keeps each slot with one team.
  // (not at (192,128) in BF16 mode, one pass: a single column stage paces that kernel and the change cost 5 %)
  static constexpr bool kEarly = kRowTok == kSub && !(kEB == 2 && kTightDims);
  // arrivals that release a row stage: the commits behind the S^T and dP^T MMAs; without dP^T, in BF16 mode
  // (LSE arrives in the stage by a bulk copy), the preparation warp once it has read LSE out of the stage
  static constexpr int kRowReleases = !kEarly ? 1 : (kHasDk ? 2 : (kEB == 1 ? 1 : 2));
  static constexpr int kLseSlots = kEarly ? ((kRowStages + 4) & ~1) : kRowStages;
  // tensor memory
  // FP8 at (192, 128) with both gradients in one pass: dV 128 + dK 192 columns beside the score tiles
  // fill tensor memory exactly when the P^ / dS^ operands and every scale-factor slot are single and the
  // scale columns of the two gradient products are shared (they are used one after the other by one
  // issuing thread): 64 + 64 + 16 + 16 + 128 + 192 + SF 32 = 512.
  // (BF16 at the same head dims: no scale factors, 64 + 64 + 32 + 32 + 128 + 192 = 512 with single operand buffers)
  static constexpr bool kTight = kMode == kBoth && ((kFp8 && kFp8v && kCq == 2 && kCv == 1) || (kEB == 2 && kEBv == 2 && kCq == 3 && kCv == 2));
  static constexpr int kOpBufs = kTight ? 1 : 2;       // P^ / dS^ operand buffers
  static constexpr int kSl = kTight ? 1 : 2;           // scale-factor slots per streamed stage
  static constexpr int kOpCols = 16 * kEB;             // columns of one P^ / dS^ buffer (64 queries)
  static constexpr uint32_t kColS = 0;
  static constexpr uint32_t kColdP = 64;
  static constexpr uint32_t kColP = kColdP + (kHasDk ? 64 : 0);
  static constexpr uint32_t kColdS = kColP + (kHasDv ? kOpBufs * kOpCols : 0);
  static constexpr uint32_t kColdV = kColdS + (kHasDk ? kOpBufs * kOpCols : 0);
  static constexpr uint32_t kColdK = kColdV + (kHasDv ? 128 * kRv : 0);
  static constexpr uint32_t kColSFK = kColdK + (kHasDk ? (kTight ? 192 : 128 * kRqAcc) : 0);
  static constexpr uint32_t kColSFV = kColSFK + 4 * kCq;
  static constexpr uint32_t kColSFQ = kColSFV + (kHasDk && kFp8v ? 4 * kCv : 0);   // kSl slots
  static constexpr uint32_t kColSFdO = kColSFQ + 4 * kSl * kCq;                // kSl slots
  static constexpr uint32_t kColSFP = kColSFdO + (kHasDk && kFp8v ? 4 * kSl * kCv : 0);  // kOpBufs x 4
  static constexpr uint32_t kColSFdS = kTight ? kColSFP : kColSFP + (kHasDv ? 8 : 0);   // kOpBufs x 4
  static constexpr uint32_t kColSFdOc = kColSFdS + (kTight ? 4 : (kHasDk ? 8 : 0));     // kSl slots x row tiles
  static constexpr uint32_t kColSFQc = kTight ? kColSFdOc : kColSFdOc + (kHasDv ? 8 * kRv : 0);   // kSl slots x row tiles
  static constexpr uint32_t kColsUsed = kFp8 ? (kTight ? kColSFQc + 4 : kColSFQc + (kHasDk ? 8 * kRqAcc : 0)) : kColSFK;
  static constexpr uint32_t kTmemCols = 512;
  static_assert(kColsUsed <= 512, "tensor memory exceeded");
};

template <class C>
struct KvRowStage {
  alignas(1024) uint8_t q[C::kCq][C::kRowTok * 128];                    // Q row copy  [queries][dqk]
  alignas(1024) uint8_t dO[C::kHasDk ? C::kCv : 1][C::kHasDk ? C::kRowTok * 128 : 16];   // dO row copy [queries][dv]
  alignas(16) uint8_t sf_q[C::kCq * 512];
  alignas(16) uint8_t sf_dO[C::kCv * 512];
  alignas(16) float lse[C::kRowTok];
  alignas(16) float delta[C::kRowTok];
  alignas(16) float neg_lse2[C::kRowTok];       // -LSE * log2(e), written by the prep warp
};
template <class C>
struct KvColStage {
  alignas(1024) uint8_t qc[C::kHasDk ? C::kQcRows * 128 : 16];   // Q col copy  [dqk][queries]
  alignas(1024) uint8_t dOc[C::kHasDv ? C::kRv * kTile * 128 : 16];     // dO col copy [dv][queries]
  alignas(16) uint8_t sf_qc[C::kRqAcc * 512];
  alignas(16) uint8_t sf_dOc[C::kRv * 512];
};

template <class C>
struct KvSmem {
  alignas(1024) uint8_t k[C::kCq][kTile * 128];
  alignas(1024) uint8_t v[C::kHasDk ? C::kCv : 1][C::kHasDk ? kTile * 128 : 16];
  KvRowStage<C> rst[C::kRowStages];
  KvColStage<C> cst[C::kColStages];
  alignas(16) uint8_t sf_k[C::kCq * 512];
  alignas(16) uint8_t sf_v[C::kCv * 512];
  alignas(16) uint8_t sf_p[2][512];
  alignas(16) uint8_t sf_ds[2][512];
  uint64_t kv_full;
  uint64_t row_full[C::kRowStages], row_empty[C::kRowStages];
  uint64_t col_full[C::kColStages], col_empty[C::kColStages];
  uint64_t lse_ready[C::kLseSlots];
  alignas(16) float lse_ring[C::kEarly ? C::kLseSlots : 1][kSub];     // kEarly: -LSE * log2(e) of a sub-tile
  alignas(16) float delta_ring[C::kEarly ? C::kLseSlots : 1][kSub];   // kEarly: -D
  uint64_t sdp_full[kTeams], sdp_free[kTeams];
  // P^ / dS^ hand-off.  "free" barriers are per softmax team (the team that writes the buffer next waits on its
  // own: a team takes every other sub-tile, and a parity wait on a barrier that completes once per sub-tile
  // would pass at once for a waiter a whole phase behind).  With a single operand buffer P^ and dS^ are handed
  // over separately (p_full / p_free for P^), so that the next P^ is written while the dK MMAs still run.
  uint64_t pds_full[2], pds_free[2];
  uint64_t p_full, p_free[2];
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
  int N, Nk, q0t, Hq, Hkv, dqk, dv, causal;   // N query rows, Nk keys, q0t: tile offset of the causal diagonal
  int kv_lim;               // without the causal mask: last real key of the last key tile (127: all real)
  int tail_wait;            // launched behind another key-major pass of the same call (see launch_kvmajor_t)
  float scale, scale_log2;
};

template <class C>
__global__ void __launch_bounds__(kThreads, 1)
kvmajor_kernel(const KvParams p, const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
               const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_dO,
               const __grid_constant__ CUtensorMap tm_qc, const __grid_constant__ CUtensorMap tm_dOc) {
  // declared with the alignment the swizzled operand tiles need, so that the compiler keeps the
  // shared state space of every access derived from it (checked below)
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  constexpr bool kFp8 = C::kFp8, kFp8v = C::kFp8v, kHasDv = C::kHasDv, kHasDk = C::kHasDk;
  constexpr int kEB = C::kEB, kCq = C::kCq, kCv = C::kCv, kRq = C::kRqAcc, kRv = C::kRv;
  constexpr int kRowStages = C::kRowStages, kColStages = C::kColStages, kRowTok = C::kRowTok;
  constexpr int kSubPerRow = C::kSubPerRow, kSubPerCol = C::kSubPerCol, kOpCols = C::kOpCols;
  constexpr bool kTight = C::kTight;
  constexpr int kOpBufs = C::kOpBufs, kSl = C::kSl;
  // 64-query row stages: LSE and D of a stage are fetched by the preparation warp with plain loads, one stage
  // ahead, instead of two more bulk copies per stage by the producer thread (which paces the kernel there)
  // (FP8 only: in BF16 mode the producer is not what paces the kernel, and the change cost 5 % there)
  constexpr bool kPrepLoads = kFp8 && C::kRowTok == kSub;
  constexpr bool kSplit = kOpBufs == 1;          // single operand buffer: P^ and dS^ are handed over separately
  constexpr uint32_t kColS = C::kColS, kColdP = C::kColdP, kColP = C::kColP, kColdS = C::kColdS, kColdV = C::kColdV,
                     kColdK = C::kColdK, kColSFK = C::kColSFK, kColSFV = C::kColSFV, kColSFQ = C::kColSFQ,
                     kColSFdO = C::kColSFdO, kColSFP = C::kColSFP, kColSFdS = C::kColSFdS, kColSFdOc = C::kColSFdOc,
                     kColSFQc = C::kColSFQc, kTmemCols = C::kTmemCols;
  KvSmem<C>& sm = *reinterpret_cast<KvSmem<C>*>(smem_raw);
  if (smem_u32(smem_raw) & 1023u) {               // never expected: report instead of computing garbage
    if (threadIdx.x == 0) atomicExch(p.status, static_cast<int>(ATTN_ERR_ALIGNMENT));
    return;
  }
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // blocks are handed out x-fastest: KV heads vary fastest, key tiles in order, so the heaviest
  // tiles (the earliest keys under the causal mask) of all heads go first
  const int jt = blockIdx.y;
  const int g = blockIdx.x, b = blockIdx.z;
  const int G = p.Hq / p.Hkv;
  const int tiles_n = p.N / kTile, tiles_nk = p.Nk / kTile;
  const int it0 = p.causal ? max(jt - p.q0t, 0) : 0;   // first query tile that sees these keys
  const int tiles_per_head = tiles_n - it0;
  const int n_qtiles = G * tiles_per_head;          // query tiles this CTA walks
  const int n_sub = 2 * n_qtiles;
  const int nk_qk = p.dqk * kEB / 32, nk_v = p.dv * C::kEBv / 32;   // 32-byte K steps of S^T and dP^T
  // columns of dK (rows of Q^c) this pass accumulates: all of them, or one tile of 128
  const int dk_col0 = C::kDkTile >= 0 ? 128 * C::kDkTile : 0;
  const int dk_cols = C::kDkTile >= 0 ? min(128, p.dqk - dk_col0) : p.dqk;
  volatile int* abort_flag = &sm.abort_flag;

  if (tid == 0) {
    mbar_init(&sm.kv_full, 1);
    for (int s = 0; s < kRowStages; ++s) {
      // released once the softmax teams are done with the rows (kEarly: once the S^T and dP^T MMAs have read them)
      mbar_init(&sm.row_full[s], 1); mbar_init(&sm.row_empty[s], C::kRowReleases);
    }
    for (int s = 0; s < C::kLseSlots; ++s) mbar_init(&sm.lse_ready[s], 1);   // one arrival by the prep warp
    for (int s = 0; s < kColStages; ++s) { mbar_init(&sm.col_full[s], 1); mbar_init(&sm.col_empty[s], 1); }
    for (int t = 0; t < kTeams; ++t) { mbar_init(&sm.sdp_full[t], kHasDk ? 2 : 1); mbar_init(&sm.sdp_free[t], kTeamThreads); }
    for (int i = 0; i < 2; ++i) { mbar_init(&sm.pds_full[i], kTeamThreads); mbar_init(&sm.pds_free[i], 1); mbar_init(&sm.p_free[i], 1); }
    mbar_init(&sm.p_full, kTeamThreads);
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
  // the query-major kernel of the same call may be queued behind this grid: let its CTAs take the
  // SMs that this grid's last wave leaves idle (nothing it does depends on this grid's output)
  griddep_launch_dependents();
  const uint32_t tmem = sm.tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      prefetch_tmap(&tm_k); prefetch_tmap(&tm_v); prefetch_tmap(&tm_q); prefetch_tmap(&tm_dO);
      prefetch_tmap(&tm_qc); prefetch_tmap(&tm_dOc);
      const int kv_slab = b * p.Hkv + g;
      mbar_arrive_expect_tx(&sm.kv_full, kCq * (kTile * 128 + (kFp8 ? 512 : 0)) +
                                             (kHasDk ? kCv * (kTile * 128 + (kFp8v ? 512 : 0)) : 0));
      for (int c = 0; c < kCq; ++c) tma_load_2d(sm.k[c], &tm_k, &sm.kv_full, 128 * c, kv_slab * p.Nk + jt * kTile);
      if (kFp8) bulk_load_1d(sm.sf_k, p.k_sf + (static_cast<size_t>(kv_slab) * tiles_nk + jt) * kCq * 512, kCq * 512, &sm.kv_full);
      if (kHasDk) {
        for (int c = 0; c < kCv; ++c) tma_load_2d(sm.v[c], &tm_v, &sm.kv_full, 128 * c, kv_slab * p.Nk + jt * kTile);
        if (kFp8v) bulk_load_1d(sm.sf_v, p.v_sf + (static_cast<size_t>(kv_slab) * tiles_nk + jt) * kCv * 512, kCv * 512, &sm.kv_full);
      }
      int issued_row = 0, issued_col = 0;
      bool ok = true;
      for (int u = 0; u < n_sub && ok; ++u) {
        const int n = u >> 1, half = u & 1;
        const int h = g * G + n / tiles_per_head, it = it0 + n % tiles_per_head;
        const int q_slab = b * p.Hq + h;
        const size_t sf_tile = static_cast<size_t>(q_slab) * tiles_n + it;
        if (u % kSubPerRow == 0) {
          const int ri = u / kSubPerRow, rs = ri % kRowStages;
          const int tok0 = it * kTile + (kSubPerRow == 1 ? half * kSub : 0);     // first query of the stage
          ok = mbar_wait(&sm.row_empty[rs], ((ri / kRowStages) & 1) ^ 1, abort_flag);
          if (!ok) break;
          KvRowStage<C>& r = sm.rst[rs];
          mbar_arrive_expect_tx(&sm.row_full[rs], kCq * (kRowTok * 128 + (kFp8 ? 512 : 0)) +
                                                      (kHasDk ? kCv * (kRowTok * 128 + (kFp8v ? 512 : 0)) : 0) +
                                                      (kPrepLoads ? 0 : (kHasDk ? 2 : 1) * kRowTok * 4));
          for (int c = 0; c < kCq; ++c) tma_load_2d(r.q[c], &tm_q, &sm.row_full[rs], 128 * c, q_slab * p.N + tok0);
          if (kFp8) bulk_load_1d(r.sf_q, p.q_sf + sf_tile * kCq * 512, kCq * 512, &sm.row_full[rs]);
          if (!kPrepLoads) bulk_load_1d(r.lse, p.lse + static_cast<size_t>(q_slab) * p.N + tok0, kRowTok * 4, &sm.row_full[rs]);
          if (kHasDk) {
            for (int c = 0; c < kCv; ++c) tma_load_2d(r.dO[c], &tm_dO, &sm.row_full[rs], 128 * c, q_slab * p.N + tok0);
            if (kFp8v) bulk_load_1d(r.sf_dO, p.dO_sf + sf_tile * kCv * 512, kCv * 512, &sm.row_full[rs]);
            if (!kPrepLoads) bulk_load_1d(r.delta, p.delta + static_cast<size_t>(q_slab) * p.N + tok0, kRowTok * 4, &sm.row_full[rs]);
          }
          ++issued_row;
        }
        if (u % kSubPerCol == 0) {
          const int ci = u / kSubPerCol, cs = ci % kColStages;
          const int x0 = (it * kTile + (kSubPerCol == 1 ? half * kSub : 0)) * kEB;   // byte offset along the query dim
          ok = mbar_wait(&sm.col_empty[cs], ((ci / kColStages) & 1) ^ 1, abort_flag);
          if (!ok) break;
          KvColStage<C>& c = sm.cst[cs];
          mbar_arrive_expect_tx(&sm.col_full[cs], (kHasDk ? dk_cols * 128 + (kFp8 ? kRq * 512 : 0) : 0) +
                                                      (kHasDv ? p.dv * 128 + (kFp8 ? kRv * 512 : 0) : 0));
          if (kHasDk) {
            tma_load_2d(c.qc, &tm_qc, &sm.col_full[cs], x0, q_slab * p.dqk + dk_col0);
            if (kFp8)
              for (int r = 0; r < kRq; ++r)
                bulk_load_1d(c.sf_qc + 512 * r, p.qc_sf + ((static_cast<size_t>(q_slab) * kRq + r) * tiles_n + it) * 512, 512,
                             &sm.col_full[cs]);
          }
          if (kHasDv) {
            tma_load_2d(c.dOc, &tm_dOc, &sm.col_full[cs], x0, q_slab * p.dv);
            if (kFp8)
              for (int r = 0; r < kRv; ++r)
                bulk_load_1d(c.sf_dOc + 512 * r, p.dOc_sf + ((static_cast<size_t>(q_slab) * kRv + r) * tiles_n + it) * 512, 512,
                             &sm.col_full[cs]);
          }
          ++issued_col;
        }
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
      const uint64_t desc_k = make_desc_sw128(smem_u32(sm.k[0]));
      bool ok = mbar_wait(&sm.kv_full, 0, abort_flag);
      if (ok && kFp8) {
        tc_fence_after_sync();
        sf_copy_tiles<kCq>(tmem + kColSFK, sm.sf_k);
      }
      // the row ring is walked with a running (stage, phase) pair: a division by a ring depth of 3 in every
      // iteration is felt in the issue rate
      int s = 0;
      uint32_t s_phase = 0;
      for (int u = 0; u < n_sub && ok; ++u) {
        const int half = u & 1, ri = u / kSubPerRow, slot = kSl == 2 ? (ri & 1) : 0, sub_r = u % kSubPerRow;
        if (u > 0 && sub_r == 0 && ++s == kRowStages) { s = 0; s_phase ^= 1u; }
        KvRowStage<C>& st = sm.rst[s];
        if (sub_r == 0) {
          ok = mbar_wait(&sm.row_full[s], s_phase, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          if (kFp8 && kSl == 2) sf_copy_tiles<kCq>(tmem + kColSFQ + 4 * kCq * slot, st.sf_q);
        }
        if (u > 0) {
          // the team of the previous sub-tile has pulled S and dP into registers
          ok = mbar_wait(&sm.sdp_free[(u - 1) % kTeams], ((u - 1) / kTeams) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
        }
        // a single scale slot is rewritten only now that the product that read it has been consumed
        if (kFp8 && kSl == 1 && sub_r == 0) sf_copy_tiles<kCq>(tmem + kColSFQ, st.sf_q);
        const uint64_t desc_q = make_desc_sw128(smem_u32(st.q[0])) + sub_r * (kSub * 128 / 16);
        issue_ss<kFp8, kCq, kSub, kTile * 128 / 16, kRowTok * 128 / 16>(
            tmem + kColS, desc_k, desc_q, nk_qk, tmem + kColSFK, tmem + kColSFQ + 4 * kCq * slot + 2 * half);
        mma_commit_elect(&sm.sdp_full[u % kTeams]);
        if (C::kEarly) mma_commit_elect(&sm.row_empty[s]);   // the row operands of this sub-tile have been read
      }
      if (!ok) {
        int dummy = 0;
        mma_commit_elect(&sm.drain[0]);
        mbar_wait(&sm.drain[0], 0, &dummy);
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ dP^T issuer + LSE preparation
    const uint64_t desc_v = make_desc_sw128(smem_u32(sm.v[0]));
    bool ok = mbar_wait(&sm.kv_full, 0, abort_flag);
    if (ok && kFp8v && kHasDk) {
      tc_fence_after_sync();
      sf_copy_tiles<kCv>(tmem + kColSFV, sm.sf_v);
    }
    int s = 0;                                        // running (stage, phase) of the row ring
    uint32_t s_phase = 0;
    // kPrepLoads: LSE and D of the next row stage (= sub-tile), in flight while this one is handled
    int pf_h = g * G, pf_it = it0;                    // (head, query tile) of the stage fetched next
    float4 pf_l = make_float4(0.f, 0.f, 0.f, 0.f), pf_d = make_float4(0.f, 0.f, 0.f, 0.f);
    auto prefetch = [&](int uu) {
      if (4 * lane < kRowTok) {
        const size_t at = static_cast<size_t>(b * p.Hq + pf_h) * p.N + pf_it * kTile + (uu & 1) * kSub + 4 * lane;
        pf_l = *reinterpret_cast<const float4*>(p.lse + at);
        if (kHasDk) pf_d = *reinterpret_cast<const float4*>(p.delta + at);
      }
      if ((uu & 1) && ++pf_it == tiles_n) { pf_it = it0; ++pf_h; }
    };
    if (kPrepLoads && n_sub > 0) prefetch(0);
    int ls = 0;                                       // kEarly: slot of the LSE / D ring (sub-tile u modulo its depth)
    for (int u = 0; u < n_sub && ok; ++u) {
      const int half = u & 1, ri = u / kSubPerRow, slot = kSl == 2 ? (ri & 1) : 0, sub_r = u % kSubPerRow;
      if (u > 0 && sub_r == 0 && ++s == kRowStages) { s = 0; s_phase ^= 1u; }
      KvRowStage<C>& st = sm.rst[s];
      if (sub_r == 0) {
        ok = mbar_wait(&sm.row_full[s], s_phase, abort_flag);
        if (!ok) break;
        if (kPrepLoads) {
          if (4 * lane < kRowTok) {
            *reinterpret_cast<float4*>(&sm.lse_ring[ls][4 * lane]) =
                make_float4(-pf_l.x * kLog2e, -pf_l.y * kLog2e, -pf_l.z * kLog2e, -pf_l.w * kLog2e);
            if (kHasDk) *reinterpret_cast<float4*>(&sm.delta_ring[ls][4 * lane]) = make_float4(-pf_d.x, -pf_d.y, -pf_d.z, -pf_d.w);
          }
          if (u + 1 < n_sub) prefetch(u + 1);
        } else
        // every lane turns four LSE values into -LSE*log2(e) for the softmax teams
        if (4 * lane < kRowTok) {
          const float4 l = *reinterpret_cast<const float4*>(&st.lse[4 * lane]);
          *reinterpret_cast<float4*>(C::kEarly ? &sm.lse_ring[ls][4 * lane] : &st.neg_lse2[4 * lane]) =
              make_float4(-l.x * kLog2e, -l.y * kLog2e, -l.z * kLog2e, -l.w * kLog2e);
          if (kHasDk) {                                 // and the row correction into its negative (in place, or into the ring)
            const float4 d = *reinterpret_cast<const float4*>(&st.delta[4 * lane]);
            *reinterpret_cast<float4*>(C::kEarly ? &sm.delta_ring[ls][4 * lane] : &st.delta[4 * lane]) = make_float4(-d.x, -d.y, -d.z, -d.w);
          }
        }
        if (C::kEarly && !kPrepLoads && !kHasDk) mbar_arrive_warp(&sm.row_empty[s]);   // LSE has been read out of the stage
        mbar_arrive_warp(&sm.lse_ready[C::kEarly ? ls : s]);
        if (++ls == C::kLseSlots) ls = 0;
        if (kFp8v && kHasDk && kSl == 2) {
          tc_fence_after_sync();
          sf_copy_tiles<kCv>(tmem + kColSFdO + 4 * kCv * slot, st.sf_dO);
        }
      }
      if (kHasDk) {
        if (u > 0) {
          ok = mbar_wait(&sm.sdp_free[(u - 1) % kTeams], ((u - 1) / kTeams) & 1, abort_flag);
          if (!ok) break;
        }
        tc_fence_after_sync();
        if (kFp8v && kSl == 1 && sub_r == 0) sf_copy_tiles<kCv>(tmem + kColSFdO, st.sf_dO);
        const uint64_t desc_dO = make_desc_sw128(smem_u32(st.dO[0])) + sub_r * (kSub * 128 / 16);
        issue_ss<kFp8v, kCv, kSub, kTile * 128 / 16, kRowTok * 128 / 16>(
            tmem + kColdP, desc_v, desc_dO, nk_v, tmem + kColSFV, tmem + kColSFdO + 4 * kCv * slot + 2 * half);
        mma_commit_elect(&sm.sdp_full[u % kTeams]);
        if (C::kEarly) mma_commit_elect(&sm.row_empty[s]);
      }
    }
    if (!ok && kHasDk) {
      int dummy = 0;
      mma_commit_elect(&sm.drain[1]);
      mbar_wait(&sm.drain[1], 0, &dummy);
    }
  } else if (warp == 3) {
    // ------------------------------------------------------------------ dV / dK issuer
    {
      bool ok = true;
      int rs_done = 0;                                // row stage whose queries go through the softmax next
      for (int u = 0; u < n_sub && ok; ++u) {
        const int buf = kOpBufs == 2 ? (u & 1) : 0, ci = u / kSubPerCol, s = ci % kColStages, slot = kSl == 2 ? (ci & 1) : 0, sub_c = u % kSubPerCol;
        KvColStage<C>& st = sm.cst[s];
        if (sub_c == 0) {
          ok = mbar_wait(&sm.col_full[s], (ci / kColStages) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          if (kFp8 && !kTight) {
            if (kHasDv) sf_copy_tiles<kRv>(tmem + kColSFdOc + 4 * kRv * slot, st.sf_dOc);
            if (kHasDk) sf_copy_tiles<kRq>(tmem + kColSFQc + 4 * kRq * slot, st.sf_qc);
          }
        }
        // (single operand buffer: P^ comes first, dS^ is waited for ahead of the dK product)
        ok = kSplit ? mbar_wait(&sm.p_full, u & 1, abort_flag) : mbar_wait(&sm.pds_full[buf], (kOpBufs == 2 ? u >> 1 : u) & 1, abort_flag);
        if (!ok) break;
        // all queries of a row stage have been through the softmax: the stage (score operands,
        // LSE, D) is no longer read
        if (!C::kEarly && u % kSubPerRow == kSubPerRow - 1) {
          if (lane == 0) mbar_arrive(&sm.row_empty[rs_done]);
          if (++rs_done == kRowStages) rs_done = 0;
        }
        tc_fence_after_sync();
        if (kFp8 && !kTight) {
          if (kHasDv) sf_copy_elect(tmem + kColSFP + 4 * buf, make_desc_sf(smem_u32(sm.sf_p[buf])));
          if (kHasDk) sf_copy_elect(tmem + kColSFdS + 4 * buf, make_desc_sf(smem_u32(sm.sf_ds[buf])));
        }
        if (kTight && kFp8) {
          // One operand buffer, one pair of scale slots: the scales of P^ and dO^c, the dV product, then the
          // scales of dS^ and of each row tile of Q^c in the same columns and the dK product of that tile.
          // Copies and MMAs of one thread run in the order issued.
          const uint64_t desc_qc = make_desc_sw128(smem_u32(st.qc));
          sf_copy_elect(tmem + kColSFP, make_desc_sf(smem_u32(sm.sf_p[0])));
          sf_copy_elect(tmem + kColSFdOc, make_desc_sf(smem_u32(st.sf_dOc)));
          issue_ts<true, 1, 1>(tmem + kColdV, tmem + kColP, make_desc_sw128(smem_u32(st.dOc)), p.dv, sub_c, tmem + kColSFP,
                               tmem + kColSFdOc, u > 0);
          mma_commit_elect(&sm.p_free[(u + 1) & 1]);      // P^ and its scale bytes may be rewritten (by the other team)
          ok = mbar_wait(&sm.pds_full[0], u & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          sf_copy_elect(tmem + kColSFdS, make_desc_sf(smem_u32(sm.sf_ds[0])));
#pragma unroll
          for (int r = 0; r < 2; ++r) {
            sf_copy_elect(tmem + kColSFQc, make_desc_sf(smem_u32(st.sf_qc + 512 * r)));
            issue_ts<true, 1, 1>(tmem + kColdK + 128 * r, tmem + kColdS, desc_qc + r * (128 * 128 / 16), r == 0 ? 128 : dk_cols - 128,
                                 sub_c, tmem + kColSFdS, tmem + kColSFQc, u > 0);
          }
        } else {
        // 64 queries = 2 (codes) or 4 (BF16) steps of 32 bytes; the B operands are taken 128 rows at a time
        if (kHasDv)
          issue_ts<kFp8, kEB, kRv>(tmem + kColdV, tmem + kColP + kOpCols * buf, make_desc_sw128(smem_u32(st.dOc)), p.dv,
                                   sub_c, tmem + kColSFP + 4 * buf, tmem + kColSFdOc + 4 * kRv * slot, u > 0);
        if (kSplit) {
          mma_commit_elect(&sm.p_free[(u + 1) & 1]);
          ok = mbar_wait(&sm.pds_full[0], u & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
        }
        if (kHasDk)
          issue_ts<kFp8, kEB, kRq>(tmem + kColdK, tmem + kColdS + kOpCols * buf, make_desc_sw128(smem_u32(st.qc)), dk_cols,
                                   sub_c, tmem + kColSFdS + 4 * buf, tmem + kColSFQc + 4 * kRq * slot, u > 0);
        }
        // operands and scale bytes of this buffer may be overwritten once these MMAs have run; the
        // col stage may be refilled after its last sub-tile
        mma_commit_elect(&sm.pds_free[kOpBufs == 2 ? buf : ((u + 1) & 1)]);   // indexed by the team that writes next
        if (sub_c == kSubPerCol - 1) mma_commit_elect(&sm.col_empty[s]);
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
    int it = it0;                                     // query tile of the current sub-tile (kTeams == 2: one tile per iteration)
    static_assert(kTeams == 2, "a team advances by one query tile per iteration");
    // running (stage, phase) of the row ring: the team's first sub-tile is in row stage team / kSubPerRow and
    // it advances by kTeams / kSubPerRow stages per iteration
    int s = (team / kSubPerRow) % kRowStages;
    uint32_t s_phase = ((team / kSubPerRow) / kRowStages) & 1;
    int ls = team;                                    // kEarly: running (slot, phase) of the LSE / D ring
    uint32_t ls_phase = 0;
    for (int u = team; u < n_sub; u += kTeams) {
      const int half = u & 1, buf = kOpBufs == 2 ? (u & 1) : 0;
      if (u != team) {
#pragma unroll
        for (int a = 0; a < kTeams / kSubPerRow; ++a)
          if (++s == kRowStages) { s = 0; s_phase ^= 1u; }
        if ((ls += kTeams) >= C::kLseSlots) { ls -= C::kLseSlots; ls_phase ^= 1u; }
      }
      ok = mbar_wait(&sm.sdp_full[team], (u / kTeams) & 1, abort_flag);
      if (!ok) break;
      tc_fence_after_sync();
      uint32_t sr[32], dpr[32];                       // S then P; dP then dS (in place)
      tmem_ld32(tmem + kColS + lane_addr + 32 * grp, sr);
      if (kHasDk) tmem_ld32(tmem + kColdP + lane_addr + 32 * grp, dpr);
      tmem_wait_ld();
      tc_fence_before_sync();
      mbar_arrive(&sm.sdp_free[team]);
      ok = C::kEarly ? mbar_wait(&sm.lse_ready[ls], ls_phase, abort_flag) : mbar_wait(&sm.lse_ready[s], s_phase, abort_flag);
      if (!ok) break;
      const int col0 = half * kSub + 32 * grp;        // query row (inside the tile) of this thread's first column
      const int st0 = (u % kSubPerRow) * kSub + 32 * grp;   // the same inside the row stage
      const KvRowStage<C>& st = sm.rst[s];
      float amax_p = 0.f, max_s = 0.f;
      const float* s_lse = C::kEarly ? &sm.lse_ring[ls][32 * grp] : &st.neg_lse2[st0];
      const float* s_delta = C::kEarly ? &sm.delta_ring[ls][32 * grp] : &st.delta[st0];
      // two elements per instruction (fma / mul .f32x2) wherever the arithmetic allows: the loop is
      // bound by instruction issue, not by a pipe
      const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
      auto body = [&](auto diag_tag) {
        constexpr bool kDiag = decltype(diag_tag)::value;
#pragma unroll
        for (int c4 = 0; c4 < 32; c4 += 4) {
          const float4 l4 = lds_f4(&s_lse[c4]);
          float4 d4 = make_float4(0.f, 0.f, 0.f, 0.f);
          if (kHasDk) d4 = lds_f4(&s_delta[c4]);
#pragma unroll
          for (int e = 0; e < 4; e += 2) {
            const int c = c4 + e;
            const float2 lv2 = e == 0 ? make_float2(l4.x, l4.y) : make_float2(l4.z, l4.w);
            float2 x2 = __ffma2_rn(make_float2(__uint_as_float(sr[c]), __uint_as_float(sr[c + 1])), sc2, lv2);
            if (kDiag) {                                      // key after the query
              if (row > col0 + c) x2.x = -INFINITY;
              if (row > col0 + c + 1) x2.y = -INFINITY;
            }
            const float2 p2 = make_float2(ex2_approx(x2.x), ex2_approx(x2.y));
            sr[c] = __float_as_uint(p2.x);
            sr[c + 1] = __float_as_uint(p2.y);
            amax_p = fmaxf(amax_p, fmaxf(p2.x, p2.y));
            if (kHasDk) {
              const float2 dv2 = e == 0 ? make_float2(d4.x, d4.y) : make_float2(d4.z, d4.w);
              const float2 t2 = __fadd2_rn(make_float2(__uint_as_float(dpr[c]), __uint_as_float(dpr[c + 1])), dv2);   // dP - D (dv2 holds -D)
              const float2 ds2 = __fmul2_rn(p2, t2);          // dS = P (dP - D)
              dpr[c] = __float_as_uint(ds2.x);
              dpr[c + 1] = __float_as_uint(ds2.y);
              max_s = fmaxf(max_s, fmaxf(fabsf(ds2.x), fabsf(ds2.y)));
            }
          }
        }
      };
      if (p.causal && it + p.q0t == jt) body(std::true_type{}); else body(std::false_type{});
      if (__builtin_expect(!p.causal && row > p.kv_lim && jt == p.Nk / kTile - 1, 0)) {
        // a padded key of a ragged sequence (no causal mask): its probabilities and score gradients are zero
#pragma unroll
        for (int c = 0; c < 32; ++c) { sr[c] = 0u; dpr[c] = 0u; }
        amax_p = 0.f;
        max_s = 0.f;
      }
      uint32_t byte_p = 0, byte_s = 0;
      float inv_p = 1.f, inv_s = 1.f;
      if (kFp8) {
        if (kHasDv) block_scale_finite(amax_p, byte_p, inv_p);
        if (kHasDk) block_scale_finite(max_s, byte_s, inv_s);
      }
      if (u >= kOpBufs) {
        // the dV / dK MMAs of the sub-tile that last used this buffer have consumed its operands and scale bytes
        // (single buffer: the dV MMAs have consumed P^; dS^ is waited for below)
        ok = mbar_wait(kSplit ? &sm.p_free[team] : &sm.pds_free[team], ((u - kOpBufs) >> 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after_sync();
      }
      uint32_t words[8 * kEB];
      if (kHasDv) {
        if (kFp8) {
          const float2 inv2 = make_float2(inv_p, inv_p);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float2 a = __fmul2_rn(make_float2(__uint_as_float(sr[4 * i]), __uint_as_float(sr[4 * i + 1])), inv2);
            const float2 bq = __fmul2_rn(make_float2(__uint_as_float(sr[4 * i + 2]), __uint_as_float(sr[4 * i + 3])), inv2);
            words[i] = cvt_e4m3x4(a.x, a.y, bq.x, bq.y);
          }
        } else {
#pragma unroll
          for (int i = 0; i < 8 * kEB; ++i)
            words[i] = cvt_bf16x2(__uint_as_float(sr[(2 * i) & 31]), __uint_as_float(sr[(2 * i + 1) & 31]));
        }
#pragma unroll
        for (int i = 0; i < kEB; ++i) tmem_st8(tmem + kColP + kOpCols * buf + lane_addr + 8 * kEB * grp + 8 * i, words + 8 * i);
      }
      if (kSplit) {
        // hand P^ over, then wait for the dK MMAs of the sub-tile before to have consumed dS^
        if (kFp8) sts_u8(&sm.sf_p[0][(row & 31) * 16 + (row >> 5) * 4 + grp], byte_p);
        tmem_wait_st();
        fence_proxy_async_smem();
        tc_fence_before_sync();
        mbar_arrive(&sm.p_full);
        if (u >= 1) {
          ok = mbar_wait(&sm.pds_free[team], ((u - 1) >> 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
        }
      }
      if (kHasDk) {
        if (kFp8) {
          const float2 inv2 = make_float2(inv_s, inv_s);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float2 a = __fmul2_rn(make_float2(__uint_as_float(dpr[4 * i]), __uint_as_float(dpr[4 * i + 1])), inv2);
            const float2 bq = __fmul2_rn(make_float2(__uint_as_float(dpr[4 * i + 2]), __uint_as_float(dpr[4 * i + 3])), inv2);
            words[i] = cvt_e4m3x4(a.x, a.y, bq.x, bq.y);
          }
        } else {
#pragma unroll
          for (int i = 0; i < 8 * kEB; ++i)
            words[i] = cvt_bf16x2(__uint_as_float(dpr[(2 * i) & 31]), __uint_as_float(dpr[(2 * i + 1) & 31]));
        }
#pragma unroll
        for (int i = 0; i < kEB; ++i) tmem_st8(tmem + kColdS + kOpCols * buf + lane_addr + 8 * kEB * grp + 8 * i, words + 8 * i);
      }
      if (kFp8) {
        const int sf_at = (row & 31) * 16 + (row >> 5) * 4 + grp;
        if (kHasDv && !kSplit) sts_u8(&sm.sf_p[buf][sf_at], byte_p);
        if (kHasDk) sts_u8(&sm.sf_ds[buf][sf_at], byte_s);
      }
      tmem_wait_st();
      fence_proxy_async_smem();
      tc_fence_before_sync();
      mbar_arrive(&sm.pds_full[buf]);
      it = (it + 1 == tiles_n) ? it0 : it + 1;        // next tile of this head, or the first tile of the next head
    }
    // the epilogue is done by team 0 (group 0 stores dV, group 1 stores dK)
    if (team != 0) ok = false;
    if (grp == 0 ? !kHasDv : !kHasDk) ok = false;
    if (ok) ok = mbar_wait(&sm.done, 0, abort_flag);
    if (ok) {
      tc_fence_after_sync();
      const size_t grow = static_cast<size_t>(b * p.Hkv + g) * p.Nk + jt * kTile + row;
      const uint32_t col = grp == 0 ? kColdV : kColdK;
      const int width = grp == 0 ? p.dv : p.dqk;
      const int first = grp == 0 ? 0 : dk_col0, count = grp == 0 ? p.dv : dk_cols;   // columns this pass holds
      const float mul = grp == 0 ? 1.f : p.scale;
      __nv_bfloat16* out_row = (grp == 0 ? p.dv_out : p.dk) + grow * width + first;
      for (int c0 = 0; c0 < count; c0 += 32) {
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
  // This grid may have started while the pass ahead of it was draining.  One CTA, the last in launch
  // order, stays until that grid has completed, so that the completion of this grid implies the
  // completion of both for whatever follows in the stream.
  if (p.tail_wait && tid == 0 && blockIdx.x == gridDim.x - 1 && blockIdx.y == gridDim.y - 1 && blockIdx.z == gridDim.z - 1)
    griddep_wait();
}

// `behind`: the launch follows another key-major pass of the same call, which writes another output
// (dV or dK, or another column tile of dK) from the same inputs.  With few KV heads a pass has fewer
// CTAs than the GPU has SMs, or a long tail behind its heaviest CTAs; programmatic stream serialisation
// lets this pass's CTAs take the SMs the pass ahead leaves idle (every key-major CTA executes
// griddepcontrol.launch_dependents once set up).
template <class C>
attn_status_t launch_kvmajor_t(const AttnShape& s, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v, attn_qtensor_t dO,
                               const float* lse, const float* delta, void* dk, void* dv, int* status,
                               cudaStream_t stream, bool behind = false) {
  static_assert(sizeof(KvSmem<C>) + 1024 <= kSmemLimit, "shared memory exceeded");
  CUtensorMap tm_k, tm_v, tm_q, tm_dO, tm_qc, tm_dOc;
  attn_status_t st;
  const uint64_t eb = C::kEB, ebv = C::kEBv;
  const uint64_t q_rows = static_cast<uint64_t>(s.B) * s.Hq * s.N, kv_rows = static_cast<uint64_t>(s.B) * s.Hkv * s.Nk;
  if ((st = encode_tmap_u8_sw128(&tm_k, k.row_codes, s.dqk * eb, kv_rows, kTile)) != ATTN_OK) return st;
  if ((st = encode_tmap_u8_sw128(&tm_v, v.row_codes, s.dv * ebv, kv_rows, kTile)) != ATTN_OK) return st;
  if ((st = encode_tmap_u8_sw128(&tm_q, q.row_codes, s.dqk * eb, q_rows, C::kRowTok)) != ATTN_OK) return st;
  if ((st = encode_tmap_u8_sw128(&tm_dO, dO.row_codes, s.dv * ebv, q_rows, C::kRowTok)) != ATTN_OK) return st;
  const int qc_rows = C::kDkTile >= 0 ? (s.dqk - 128 * C::kDkTile < 128 ? s.dqk - 128 * C::kDkTile : 128) : s.dqk;
  if ((st = encode_tmap_u8_sw128(&tm_qc, q.col_codes, s.N * eb, static_cast<uint64_t>(s.B) * s.Hq * s.dqk, qc_rows)) != ATTN_OK) return st;
  if ((st = encode_tmap_u8_sw128(&tm_dOc, dO.col_codes, s.N * eb, static_cast<uint64_t>(s.B) * s.Hq * s.dv, s.dv)) != ATTN_OK) return st;
  KvParams p;
  p.k_sf = k.row_scales; p.v_sf = v.row_scales; p.q_sf = q.row_scales; p.dO_sf = dO.row_scales;
  p.qc_sf = q.col_scales; p.dOc_sf = dO.col_scales;
  p.lse = lse; p.delta = delta;
  p.dk = static_cast<__nv_bfloat16*>(dk); p.dv_out = static_cast<__nv_bfloat16*>(dv); p.status = status;
  p.N = s.N; p.Nk = s.Nk; p.q0t = s.q0t; p.kv_lim = s.kv_lim; p.Hq = s.Hq; p.Hkv = s.Hkv; p.dqk = s.dqk; p.dv = s.dv; p.causal = s.causal;
  p.scale = s.scale; p.scale_log2 = s.scale * kLog2e;
  p.tail_wait = behind ? 1 : 0;
  const size_t smem = sizeof(KvSmem<C>) + 1024;
  cudaError_t e = cudaFuncSetAttribute(kvmajor_kernel<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "bwd kv-major: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  dim3 grid(s.Hkv, s.Nk / kTile, s.B);
  if (behind) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kvmajor_kernel<C>, p, tm_k, tm_v, tm_q, tm_dO, tm_qc, tm_dOc);
    if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "bwd kv-major: launch: %s", cudaGetErrorString(e));
  } else {
    kvmajor_kernel<C><<<grid, kThreads, smem, stream>>>(p, tm_k, tm_v, tm_q, tm_dO, tm_qc, tm_dOc);
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "bwd kv-major: launch: %s", cudaGetErrorString(e));
  return ATTN_OK;
}

}  // namespace

attn_status_t launch_bwd_dkdv(const AttnShape& s, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v, attn_qtensor_t dO,
                              const float* lse, const float* delta, void* dk, void* dv, int* status,
                              cudaStream_t stream) {
  const int cq = (s.dqk * s.eb + 127) / 128, cv = (s.dv * s.ebv + 127) / 128;
  if (s.eb == 1 && s.ebv == 2) {                     // protected dP: BF16 row copies of V and dO
    if (cq == 1 && cv == 1)
      return launch_kvmajor_t<KvCfg<1, 1, 1, kBoth, 2>>(s, q, k, v, dO, lse, delta, dk, dv, status, stream);
    if (cq == 1 && cv == 2)
      return launch_kvmajor_t<KvCfg<1, 1, 2, kBoth, 2>>(s, q, k, v, dO, lse, delta, dk, dv, status, stream);
    return fail(ATTN_ERR_UNSUPPORTED, "bwd kv-major: protected dP is built for head dims (64,64) and (128,128)");
  }
  if (s.eb == 1 && cq == 1 && cv == 1)
    return launch_kvmajor_t<KvCfg<1, 1, 1, kBoth>>(s, q, k, v, dO, lse, delta, dk, dv, status, stream);
  if (s.eb == 2 && cq == 1 && cv == 1)
    return launch_kvmajor_t<KvCfg<2, 1, 1, kBoth>>(s, q, k, v, dO, lse, delta, dk, dv, status, stream);
  if (s.eb == 2 && cq == 2 && cv == 2)
    return launch_kvmajor_t<KvCfg<2, 2, 2, kBoth>>(s, q, k, v, dO, lse, delta, dk, dv, status, stream);
  // qk head dim above 128: dV and dK do not fit in tensor memory together; one pass each, the
  // heavier dK pass first and the dV pass launched behind it (see launch_kvmajor_t)
  // (at (192,128) both fit when every operand buffer and scale slot is single: KvCfg::kTight)
  if (s.eb == 1 && cq == 2 && cv == 1)
    return launch_kvmajor_t<KvCfg<1, 2, 1, kBoth>>(s, q, k, v, dO, lse, delta, dk, dv, status, stream);
  if (s.eb == 1 && cq == 2 && cv == 2) {
    attn_status_t st = launch_kvmajor_t<KvCfg<1, 2, 2, kDkOnly>>(s, q, k, v, dO, lse, delta, dk, dv, status, stream);
    if (st != ATTN_OK) return st;
    return launch_kvmajor_t<KvCfg<1, 2, 2, kDvOnly>>(s, q, k, v, dO, lse, delta, dk, dv, status, stream, true);
  }
  if (s.eb == 2 && cq == 3 && cv == 2)
    return launch_kvmajor_t<KvCfg<2, 3, 2, kBoth>>(s, q, k, v, dO, lse, delta, dk, dv, status, stream);
  if (s.eb == 2 && cq == 4 && cv == 4) {
    attn_status_t st = launch_kvmajor_t<KvCfg<2, 4, 4, kDkOnly, 2, 0>>(s, q, k, v, dO, lse, delta, dk, dv, status, stream);
    if (st != ATTN_OK) return st;
    st = launch_kvmajor_t<KvCfg<2, 4, 4, kDkOnly, 2, 1>>(s, q, k, v, dO, lse, delta, dk, dv, status, stream, true);
    if (st != ATTN_OK) return st;
    return launch_kvmajor_t<KvCfg<2, 4, 4, kDvOnly>>(s, q, k, v, dO, lse, delta, dk, dv, status, stream, true);
  }
  return fail(ATTN_ERR_UNSUPPORTED, "bwd kv-major: no kernel for head dims (%d, %d) at %d bytes per element", s.dqk, s.dv,
              s.eb);
}

}  // namespace attnfp8
