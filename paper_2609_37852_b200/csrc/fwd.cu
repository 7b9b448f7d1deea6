// Forward attention (paper Appendix "Forward Probability Encoding", re-designed for tcgen05 / tensor
// memory) for the operand widths the row-owner kernel of fwd_interleaved.cu does not cover: FP8 operands
// at v head dim 256, and BF16 mode.
//
// One CTA owns 128 query rows of one (batch, query head) and walks the keys up to the causal
// diagonal, 64 keys at a time; it uses 256 of the 512 tensor-memory columns and under half of the
// shared memory, so two CTAs share an SM and each fills the other's stalls.  Warp roles:
//   warp 0      TMA producer: Q tile once, then K tiles [128 keys x d] and V tiles [dv x 128 keys]
//   warp 1      issues S = Q K^T (block-scaled, 128 x 64 per sub-tile)
//   warp 2      issues O += P V (A operand = quantised probabilities read from tensor memory)
//   warps 4..11 softmax: two threads per query row (thread <-> TMEM lane x 32-key column group).
//               A thread pulls its 32 scores into registers and releases the score buffer at
//               once, so the next S is computed while it works.  Scores go to log2 units; the running shift M is an
//               INTEGER, so rescaling is by exact powers of two and the E4M3 codes of the
//               probabilities do not depend on the tile order; l accumulates the exponentials
//               BEFORE the FP8 cast; probabilities are quantised in blocks of 32 keys in
//               registers and written to tensor memory as the A operand of the second MMA, their
//               scale bytes going through shared memory into the scale-factor columns.
// M is only raised when the sub-tile maximum exceeds it by more than kLazyShift (the block scales
// absorb the difference), so the accumulator in tensor memory is almost never rescaled.
// Two MMA-issuing warps because one warp issues at most one tcgen05.mma per ~130 cycles.
//
// The kernel is a template over the operand width: element bytes (1: E4M3 codes with E8M0 block
// scales; 2: BF16 without scales, the reference-point mode), 128-byte chunks per row of the
// Q / K tiles (head dims above 128 bytes per row take two) and 128-row tiles of the V operand
// (dv = 256 takes two).  A shared-memory stage always holds one 128-byte chunk of the token
// dimension: 128 keys of codes or 64 keys of BF16.
#include <cuda_bf16.h>

#include <type_traits>

#include "common.cuh"
#include "mma_issue.cuh"
#include "mxfp8_device.cuh"
#include "sm100_ptx.cuh"

namespace attnfp8 {

namespace {

using namespace sm100;

constexpr int kTile = 128;          // query rows per CTA; keys per K / V tile in shared memory
constexpr int kSub = 64;            // keys per softmax step
constexpr int kStages = 2;          // K ring and V ring depth
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2Hi = 0.693359375f;             // ln 2 = kLn2Hi + kLn2Lo, kLn2Hi has 8 significant bits
constexpr float kLn2Lo = -2.12194440054690583e-4f;
constexpr int kLazyShift = 8;

// Operand geometry and tensor-memory map of one instantiation.
template <int kEB_, int kCq_, int kRv_, int kSplit_ = 2>
struct FwdCfg {
  static constexpr int kSplit = kSplit_;                // softmax threads per query row (1 or 2)
  static constexpr int kBpt = 2 / kSplit;               // 32-key quantisation blocks per thread and step
  static constexpr int kSoftmaxThreads = 128 * kSplit;
  static constexpr int kThreads = 128 + kSoftmaxThreads;
  static constexpr int kEB = kEB_;                      // bytes per operand element
  static constexpr int kCq = kCq_;                      // 128-byte chunks per Q / K row
  static constexpr int kRv = kRv_;                      // 128-row tiles of the V^T operand (dv / 128, rounded up)
  static constexpr bool kFp8 = kEB == 1;
  static constexpr int kTileKeys = kTile / kEB;         // keys per K / V stage
  static constexpr int kSubPerTile = kTileKeys / kSub;  // 64-key steps per stage
  static constexpr int kPCols = 16 * kEB;               // columns of one probability buffer (64 keys)
  static constexpr uint32_t kColS = 0;                  // scores of the current sub-tile, 64 columns
  static constexpr uint32_t kColP = 64;                 // probability operand, two buffers
  static constexpr uint32_t kColO = kColP + 2 * kPCols; // output accumulator, dv columns
  // scale factors (FP8 only): Q (4 per chunk), K (2 slots), V (2 slots x row tiles), P (2 x 4)
  static constexpr uint32_t kColSFQ = kColO + 128 * kRv;
  static constexpr uint32_t kColSFK = kColSFQ + 4 * kCq;
  static constexpr uint32_t kColSFV = kColSFK + 8 * kCq;
  static constexpr uint32_t kColSFP = kColSFV + 8 * kRv;
  static constexpr uint32_t kColsUsed = kFp8 ? kColSFP + 8 : kColSFQ;
  static constexpr uint32_t kTmemCols = kColsUsed <= 256 ? 256 : 512;
  static constexpr int kCtasPerSm = kTmemCols == 256 ? 2 : 1;
  static_assert(kColsUsed <= 512, "tensor memory exceeded");
};

template <class C>
struct FwdSmem {
  alignas(1024) uint8_t q[C::kCq][kTile * 128];
  alignas(1024) uint8_t k[kStages][C::kCq][C::kTileKeys * 128];
  alignas(1024) uint8_t v[kStages][C::kRv * kTile * 128];
  alignas(16) uint8_t sf_q[C::kCq * 512];
  alignas(16) uint8_t sf_k[kStages][C::kCq * 512];
  alignas(16) uint8_t sf_v[kStages][C::kRv * 512];
  alignas(16) uint8_t sf_p[2][512];
  alignas(16) float xch[2][2][kTile];       // row maxima (and at the end normaliser shares) of the thread pairs
  uint64_t q_full;
  uint64_t k_full[kStages], k_empty[kStages];
  uint64_t v_full[kStages], v_empty[kStages];
  uint64_t s_full, s_free;
  uint64_t p_full[2], p_free[2];
  uint64_t o_done;
  uint64_t pair[4];                         // one per TMEM lane quadrant: the two warps of a thread pair
  uint64_t drain[2];
  uint32_t tmem_base;
  int abort_flag;
};

struct FwdParams {
  const uint8_t* q_sf;      // row scales of Q
  const uint8_t* k_sf;      // row scales of K
  const uint8_t* v_sf;      // col scales of V
  __nv_bfloat16* o;
  float* lse;
  int* status;
  int N, Nk, q0t, Hq, Hkv, dqk, dv, causal;   // N query rows, Nk keys, q0t: tile offset of the causal diagonal
  int kv_lim;               // without the causal mask: last real key of the last key tile (127: all real)
  float scale_log2;         // softmax_scale * log2(e)
};

template <class C>
__global__ void __launch_bounds__(C::kThreads, C::kCtasPerSm)
fwd_kernel(const FwdParams p, const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
           const __grid_constant__ CUtensorMap tm_v) {
  // declared with the alignment the swizzled operand tiles need, so that the compiler keeps the
  // shared state space of every access derived from it (checked below)
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  FwdSmem<C>& sm = *reinterpret_cast<FwdSmem<C>*>(smem_raw);
  if (smem_u32(smem_raw) & 1023u) {               // never expected: report instead of computing garbage
    if (threadIdx.x == 0) atomicExch(p.status, static_cast<int>(ATTN_ERR_ALIGNMENT));
    return;
  }
  constexpr bool kFp8 = C::kFp8;
  constexpr int kEB = C::kEB, kCq = C::kCq, kRv = C::kRv, kSubPerTile = C::kSubPerTile;
  constexpr int kSplit = C::kSplit, kBpt = C::kBpt, kSoftmaxThreads = C::kSoftmaxThreads;
  constexpr uint32_t kColS = C::kColS, kColP = C::kColP, kColO = C::kColO, kColSFQ = C::kColSFQ, kColSFK = C::kColSFK,
                     kColSFV = C::kColSFV, kColSFP = C::kColSFP, kTmemCols = C::kTmemCols, kPCols = C::kPCols;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // heavy (late) query tiles first
  // blocks are handed out x-fastest: heads vary fastest and the heaviest (latest) query tiles of
  // all heads go first, so the light tiles fill the tail of the launch
  const int qt = p.causal ? (gridDim.y - 1 - blockIdx.y) : blockIdx.y;
  const int h = blockIdx.x, b = blockIdx.z;
  const int g = h / (p.Hq / p.Hkv);
  const int n_tiles = p.causal ? qt + p.q0t + 1 : p.Nk / kTile;
  const int n_sub = 2 * n_tiles;
  const int n_stage_tiles = n_tiles * kEB;      // K / V stages to stream
  const int nk_qk = p.dqk * kEB / 32;           // 32-byte K steps of the score MMA
  volatile int* abort_flag = &sm.abort_flag;

  if (tid == 0) {
    mbar_init(&sm.q_full, 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm.k_full[s], 1); mbar_init(&sm.k_empty[s], 1);
      mbar_init(&sm.v_full[s], 1); mbar_init(&sm.v_empty[s], 1);
    }
    mbar_init(&sm.s_full, 1); mbar_init(&sm.s_free, kSoftmaxThreads);
    for (int i = 0; i < 2; ++i) { mbar_init(&sm.p_full[i], kSoftmaxThreads); mbar_init(&sm.p_free[i], 1); }
    mbar_init(&sm.o_done, 1);
    for (int i = 0; i < 4; ++i) mbar_init(&sm.pair[i], 64);
    mbar_init(&sm.drain[0], 1); mbar_init(&sm.drain[1], 1);
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
      prefetch_tmap(&tm_q); prefetch_tmap(&tm_k); prefetch_tmap(&tm_v);
      const int q_row = (b * p.Hq + h) * p.N + qt * kTile;
      const int tiles_n = p.N / kTile, tiles_nk = p.Nk / kTile;
      mbar_arrive_expect_tx(&sm.q_full, kCq * kTile * 128 + (kFp8 ? kCq * 512 : 0));
      for (int c = 0; c < kCq; ++c) tma_load_2d(sm.q[c], &tm_q, &sm.q_full, 128 * c, q_row);
      if (kFp8)
        bulk_load_1d(sm.sf_q, p.q_sf + (static_cast<size_t>(b * p.Hq + h) * tiles_n + qt) * kCq * 512, kCq * 512, &sm.q_full);
      const int kv_slab = b * p.Hkv + g;
      int issued_k = 0, issued_v = 0;
      bool ok = true;
      for (int t = 0; t < n_stage_tiles && ok; ++t) {
        const int s = t % kStages, u = t / kStages;
        ok = mbar_wait(&sm.k_empty[s], (u & 1) ^ 1, abort_flag);
        if (!ok) break;
        mbar_arrive_expect_tx(&sm.k_full[s], kCq * C::kTileKeys * 128 + (kFp8 ? kCq * 512 : 0));
        for (int c = 0; c < kCq; ++c)
          tma_load_2d(sm.k[s][c], &tm_k, &sm.k_full[s], 128 * c, kv_slab * p.Nk + t * C::kTileKeys);
        if (kFp8)
          bulk_load_1d(sm.sf_k[s], p.k_sf + (static_cast<size_t>(kv_slab) * tiles_nk + t) * kCq * 512, kCq * 512, &sm.k_full[s]);
        ++issued_k;
        ok = mbar_wait(&sm.v_empty[s], (u & 1) ^ 1, abort_flag);
        if (!ok) break;
        mbar_arrive_expect_tx(&sm.v_full[s], p.dv * 128 + (kFp8 ? kRv * 512 : 0));
        tma_load_2d(sm.v[s], &tm_v, &sm.v_full[s], t * 128, kv_slab * p.dv);
        if (kFp8)
          for (int r = 0; r < kRv; ++r)
            bulk_load_1d(sm.sf_v[s] + 512 * r, p.v_sf + ((static_cast<size_t>(kv_slab) * kRv + r) * tiles_nk + t) * 512, 512,
                         &sm.v_full[s]);
        ++issued_v;
      }
      if (!ok) {
        // let the copies already in flight land before the CTA gives its shared memory back
        int dummy = 0;
        for (int t = max(0, issued_k - kStages); t < issued_k; ++t)
          mbar_wait(&sm.k_full[t % kStages], (t / kStages) & 1, &dummy);
        for (int t = max(0, issued_v - kStages); t < issued_v; ++t)
          mbar_wait(&sm.v_full[t % kStages], (t / kStages) & 1, &dummy);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ S = Q K^T issuer
    {
      const uint64_t desc_q = make_desc_sw128(smem_u32(sm.q[0]));
      bool ok = mbar_wait(&sm.q_full, 0, abort_flag);
      if (ok && kFp8) {
        tc_fence_after_sync();
        sf_copy_tiles<kCq>(tmem + kColSFQ, sm.sf_q);
      }
      for (int u = 0; u < n_sub && ok; ++u) {
        const int t = u / kSubPerTile, sub = u % kSubPerTile, s = t % kStages, slot = t & 1;
        if (sub == 0) {
          ok = mbar_wait(&sm.k_full[s], (t / kStages) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          if (kFp8) sf_copy_tiles<kCq>(tmem + kColSFK + 4 * kCq * slot, sm.sf_k[s]);
        }
        if (u > 0) {
          // the softmax threads have pulled the previous scores into registers
          ok = mbar_wait(&sm.s_free, (u - 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
        }
        const uint64_t desc_k = make_desc_sw128(smem_u32(sm.k[s][0])) + sub * (kSub * 128 / 16);
        issue_ss<kFp8, kCq, kSub, kTile * 128 / 16, C::kTileKeys * 128 / 16>(
            tmem + kColS, desc_q, desc_k, nk_qk, tmem + kColSFQ, tmem + kColSFK + 4 * kCq * slot + 2 * sub);
        mma_commit_elect(&sm.s_full);
        if (sub == kSubPerTile - 1) mma_commit_elect(&sm.k_empty[s]);
      }
      if (!ok) {
        int dummy = 0;
        mma_commit_elect(&sm.drain[0]);
        mbar_wait(&sm.drain[0], 0, &dummy);
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ O += P V issuer
    {
      bool ok = true;
      for (int u = 0; u < n_sub && ok; ++u) {
        const int t = u / kSubPerTile, sub = u % kSubPerTile, s = t % kStages, slot = t & 1, buf = u & 1;
        if (sub == 0) {
          ok = mbar_wait(&sm.v_full[s], (t / kStages) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          if (kFp8) sf_copy_tiles<kRv>(tmem + kColSFV + 4 * kRv * slot, sm.sf_v[s]);
        }
        ok = mbar_wait(&sm.p_full[buf], (u >> 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after_sync();
        if (kFp8) sf_copy_elect(tmem + kColSFP + 4 * buf, make_desc_sf(smem_u32(sm.sf_p[buf])));
        // 64 keys = 2 (codes) or 4 (BF16) steps of 32 bytes; the V^T operand is taken 128 rows at a time
        issue_ts<kFp8, kEB, kRv>(tmem + kColO, tmem + kColP + kPCols * buf, make_desc_sw128(smem_u32(sm.v[s])), p.dv, sub,
                                 tmem + kColSFP + 4 * buf, tmem + kColSFV + 4 * kRv * slot, u > 0);
        mma_commit_elect(&sm.p_free[buf]);              // operand (and scale bytes) of this buffer consumed; O updated
        if (sub == kSubPerTile - 1) mma_commit_elect(&sm.v_empty[s]);
        if (u == n_sub - 1) mma_commit_elect(&sm.o_done);
      }
      if (!ok) {
        int dummy = 0;
        mma_commit_elect(&sm.drain[1]);
        mbar_wait(&sm.drain[1], 0, &dummy);
      }
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ softmax
    // kSplit threads per query row.  With two, column group `grp` owns keys 32*grp .. 32*grp+31 of
    // the sub-tile (one quantisation block); the pair lives in two warps with the same TMEM lane
    // quadrant and exchanges its block maxima through shared memory, so that both use the same
    // shift M.  With one, the thread owns both blocks and nothing is exchanged (measured slower on
    // B200: four softmax warps per CTA hide less latency than the exchange costs).
    const int grp = kSplit == 2 ? (warp - 4) >> 2 : 0;
    const int quad = warp & 3;
    const int row = quad * 32 + lane;                 // row inside the tile == TMEM lane
    const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
    const int blk0 = grp * kBpt;                      // first 32-key block of this thread inside a sub-tile
    float M = -INFINITY;                              // integer-valued running shift (log2 units)
    float l = 0.f;                                    // this thread's share of the normaliser
    bool ok = true;
    for (int u = 0; u < n_sub; ++u) {
      const int t = u >> 1, half = u & 1, buf = u & 1;
      ok = mbar_wait(&sm.s_full, u & 1, abort_flag);
      if (!ok) break;
      tc_fence_after_sync();
      float sv[32 * kBpt];
#pragma unroll
      for (int bk = 0; bk < kBpt; ++bk)
        tmem_ld32(tmem + kColS + lane_addr + 32 * (blk0 + bk), reinterpret_cast<uint32_t*>(sv + 32 * bk));
      tmem_wait_ld();
      tc_fence_before_sync();
      mbar_arrive(&sm.s_free);
      // maxima of the raw accumulators per block (the scale is positive), masked on the diagonal tile
      float mxb[kBpt];
      // masked tiles: the diagonal one under the causal mask, else the last one when the sequence ends inside it
      if (p.causal ? t == qt + p.q0t : (p.kv_lim < kTile - 1 && t == n_tiles - 1)) {
        const int lim = p.causal ? row : p.kv_lim;
#pragma unroll
        for (int bk = 0; bk < kBpt; ++bk) {
          const int col0 = half * kSub + 32 * (blk0 + bk);
          float m = -INFINITY;
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            if (col0 + c > lim) sv[32 * bk + c] = -INFINITY;
            m = fmaxf(m, sv[32 * bk + c]);
          }
          mxb[bk] = m;
        }
      } else {
#pragma unroll
        for (int bk = 0; bk < kBpt; ++bk) {
          float m = -INFINITY;
#pragma unroll
          for (int c = 0; c < 32; ++c) m = fmaxf(m, sv[32 * bk + c]);
          mxb[bk] = m;
        }
      }
      float mx = mxb[0];
      if (kBpt == 2) mx = fmaxf(mx, mxb[kBpt - 1]);
      if (kSplit == 2) {
        sts_f32(&sm.xch[u & 1][grp][row], mx);
        mbar_arrive(&sm.pair[quad]);                  // the two warps that share these 32 rows
        ok = mbar_wait(&sm.pair[quad], u & 1, abort_flag);
        if (!ok) break;
        mx = fmaxf(mx, lds_f32(&sm.xch[u & 1][grp ^ 1][row]));
      }
      // a fully masked sub-tile (second half of the diagonal tile for the first 64 rows) gives -inf:
      // it never raises M and contributes zeros
      const float m_new = ceilf(mx * p.scale_log2);
      const bool raise = m_new > M + static_cast<float>(kLazyShift);   // true on the first sub-tile
      if (__any_sync(0xffffffffu, raise)) {             // same rows, same decision in both warps of a pair
        const float factor = raise ? exp2f(M - m_new) : 1.f;            // exact power of two (0 at the start)
        if (raise) { l *= factor; M = m_new; }
        if (u > 0) {
          // the previous P V product must have landed before the accumulator is touched
          ok = mbar_wait(&sm.p_free[(u - 1) & 1], ((u - 1) >> 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          // rare path; each thread of a row rescales its share of the output columns
          const int my_cols = p.dv / kSplit;
          for (int c0 = grp * my_cols; c0 < (grp + 1) * my_cols; c0 += 8) {
            uint32_t r[8];
            tmem_ld8(tmem + kColO + lane_addr + c0, r);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < 8; ++c) r[c] = __float_as_uint(__uint_as_float(r[c]) * factor);
            tmem_st8(tmem + kColO + lane_addr + c0, r);
          }
          tmem_wait_st();
        }
      }
      const float neg_m = -M;
      uint32_t bytes[kBpt];
      uint32_t words[kBpt][8 * kEB];
#pragma unroll
      for (int bk = 0; bk < kBpt; ++bk) {
        const float* x = sv + 32 * bk;
        bytes[bk] = 0;
        if (kFp8) {
          // The block's scale 2^e follows from its largest exponential, which is the exponential of
          // the block's score maximum; folding e into the shift makes ex2 deliver p * 2^-e, the
          // value the E4M3 cast wants, and the block sum is put back on the common scale by one
          // exact multiplication.
          float inv;
          block_scale_finite(ex2_approx(fmaf(mxb[bk], p.scale_log2, neg_m)), bytes[bk], inv);
          const float neg_me = neg_m - static_cast<float>(static_cast<int>(bytes[bk]) - 127);
          const float2 sc2 = make_float2(p.scale_log2, p.scale_log2), nme2 = make_float2(neg_me, neg_me);
          float2 bs01 = make_float2(0.f, 0.f), bs23 = make_float2(0.f, 0.f);   // two chains of pairs for the block sum
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float2 a = __ffma2_rn(make_float2(x[4 * i], x[4 * i + 1]), sc2, nme2);
            const float2 c = __ffma2_rn(make_float2(x[4 * i + 2], x[4 * i + 3]), sc2, nme2);
            const float2 t01 = make_float2(ex2_approx(a.x), ex2_approx(a.y));
            const float2 t23 = make_float2(ex2_approx(c.x), ex2_approx(c.y));
            bs01 = __fadd2_rn(bs01, t01);
            bs23 = __fadd2_rn(bs23, t23);
            words[bk][i] = cvt_e4m3x4(t01.x, t01.y, t23.x, t23.y);
          }
          const float bs0 = bs01.x + bs01.y, bs1 = bs23.x + bs23.y;
          l = fmaf(bs0 + bs1, __uint_as_float(bytes[bk] << 23), l);   // 2^e (0 for an all-masked block, whose sum is 0)
        } else {
          float bs0 = 0.f, bs1 = 0.f;
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const float p0 = ex2_approx(fmaf(x[c], p.scale_log2, neg_m));
            const float p1 = ex2_approx(fmaf(x[c + 1], p.scale_log2, neg_m));
            bs0 += p0;
            bs1 += p1;
            words[bk][c >> 1] = cvt_bf16x2(p0, p1);
          }
          l += bs0 + bs1;
        }
      }
      if (u >= 2) {
        // the P V MMAs of sub-tile u-2 have consumed this buffer's operand and scale bytes
        ok = mbar_wait(&sm.p_free[buf], ((u - 2) >> 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after_sync();
      }
#pragma unroll
      for (int bk = 0; bk < kBpt; ++bk) {
#pragma unroll
        for (int i = 0; i < kEB; ++i)
          tmem_st8(tmem + kColP + kPCols * buf + lane_addr + 8 * kEB * (blk0 + bk) + 8 * i, words[bk] + 8 * i);
        if (kFp8) sts_u8(&sm.sf_p[buf][(row & 31) * 16 + (row >> 5) * 4 + blk0 + bk], bytes[bk]);
      }
      tmem_wait_st();
      fence_proxy_async_smem();
      tc_fence_before_sync();
      mbar_arrive(&sm.p_full[buf]);
    }
    // total normaliser of the row = sum of the shares of its threads
    if (ok && kSplit == 2) {
      sm.xch[0][grp][row] = l;
      mbar_arrive(&sm.pair[quad]);
      ok = mbar_wait(&sm.pair[quad], n_sub & 1, abort_flag);
      if (ok) l += sm.xch[0][grp ^ 1][row];
    }
    if (ok) ok = mbar_wait(&sm.o_done, 0, abort_flag);
    if (ok) {
      tc_fence_after_sync();
      const float inv_l = 1.f / l;
      const size_t grow = static_cast<size_t>(b * p.Hq + h) * p.N + qt * kTile + row;
      __nv_bfloat16* o_row = p.o + grow * p.dv;
      const int my_cols = p.dv / kSplit;              // each thread of a row stores its share of the row
      for (int c0 = grp * my_cols; c0 < (grp + 1) * my_cols; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tmem + kColO + lane_addr + c0, r);
        tmem_wait_ld();
        uint32_t packed[16];
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          __nv_bfloat162 v2 = __floats2bfloat162_rn(__uint_as_float(r[2 * c]) * inv_l, __uint_as_float(r[2 * c + 1]) * inv_l);
          packed[c] = *reinterpret_cast<uint32_t*>(&v2);
        }
        uint4* dst = reinterpret_cast<uint4*>(o_row + c0);
#pragma unroll
        for (int c = 0; c < 4; ++c) dst[c] = make_uint4(packed[4 * c], packed[4 * c + 1], packed[4 * c + 2], packed[4 * c + 3]);
      }
      // LSE = M ln2 + ln l with ln2 split so that M * ln2_hi is exact: one rounding at the end
      if (grp == 0) p.lse[grow] = fmaf(M, kLn2Hi, fmaf(M, kLn2Lo, logf(l)));
    }
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
  if (tid == 0 && sm.abort_flag) atomicExch(p.status, static_cast<int>(ATTN_ERR_TIMEOUT));
}

template <class C>
attn_status_t launch_fwd_t(const AttnShape& s, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v, void* o, float* lse,
                           int* status, cudaStream_t stream) {
  CUtensorMap tm_q, tm_k, tm_v;
  attn_status_t st;
  constexpr int eb = C::kEB;
  st = encode_tmap_u8_sw128(&tm_q, q.row_codes, static_cast<uint64_t>(s.dqk) * eb, static_cast<uint64_t>(s.B) * s.Hq * s.N, kTile);
  if (st != ATTN_OK) return st;
  st = encode_tmap_u8_sw128(&tm_k, k.row_codes, static_cast<uint64_t>(s.dqk) * eb, static_cast<uint64_t>(s.B) * s.Hkv * s.Nk,
                            C::kTileKeys);
  if (st != ATTN_OK) return st;
  st = encode_tmap_u8_sw128(&tm_v, v.col_codes, static_cast<uint64_t>(s.Nk) * eb, static_cast<uint64_t>(s.B) * s.Hkv * s.dv, s.dv);
  if (st != ATTN_OK) return st;
  FwdParams p;
  p.q_sf = q.row_scales; p.k_sf = k.row_scales; p.v_sf = v.col_scales;
  p.o = static_cast<__nv_bfloat16*>(o); p.lse = lse; p.status = status;
  p.N = s.N; p.Nk = s.Nk; p.q0t = s.q0t; p.kv_lim = s.kv_lim; p.Hq = s.Hq; p.Hkv = s.Hkv; p.dqk = s.dqk; p.dv = s.dv; p.causal = s.causal;
  p.scale_log2 = s.scale * kLog2e;
  const size_t smem = sizeof(FwdSmem<C>) + 1024;
  cudaError_t e = cudaFuncSetAttribute(fwd_kernel<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "fwd: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  dim3 grid(s.Hq, s.N / kTile, s.B);
  fwd_kernel<C><<<grid, C::kThreads, smem, stream>>>(p, tm_q, tm_k, tm_v);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "fwd: launch: %s", cudaGetErrorString(e));
  return ATTN_OK;
}

}  // namespace

attn_status_t launch_fwd(const AttnShape& s, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v, void* o, float* lse,
                         int* status, cudaStream_t stream) {
  const int cq = (s.dqk * s.eb + 127) / 128, rv = (s.dv + 127) / 128;
  // FP8 operands at head dims up to 128: the kernel with a row-owning thread per half step (fwd_interleaved.cu)
  // (and at qk head dim 192 with v head dim 128, where two chunks per Q / K row still leave tensor memory for it)
  if (s.eb == 1 && cq <= 2 && rv == 1) return launch_fwd_interleaved(s, q, k, v, o, lse, status, stream);
  if (s.eb == 1) {
    if (cq == 2 && rv == 1) return launch_fwd_t<FwdCfg<1, 2, 1>>(s, q, k, v, o, lse, status, stream);
    if (cq == 2 && rv == 2) return launch_fwd_t<FwdCfg<1, 2, 2>>(s, q, k, v, o, lse, status, stream);
  } else {
    if (cq == 1 && rv == 1) return launch_fwd_t<FwdCfg<2, 1, 1>>(s, q, k, v, o, lse, status, stream);
    if (cq == 2 && rv == 1) return launch_fwd_t<FwdCfg<2, 2, 1>>(s, q, k, v, o, lse, status, stream);
    if (cq == 3 && rv == 1) return launch_fwd_t<FwdCfg<2, 3, 1>>(s, q, k, v, o, lse, status, stream);
    if (cq == 4 && rv == 2) return launch_fwd_t<FwdCfg<2, 4, 2>>(s, q, k, v, o, lse, status, stream);
  }
  return fail(ATTN_ERR_UNSUPPORTED, "fwd: no kernel for head dims (%d, %d) at %d bytes per element", s.dqk, s.dv, s.eb);
}

}  // namespace attnfp8
