// Query-major backward kernels: the matched row correction (Delta-Matching, paper Section 3.3
// Eq. 4) and the query gradient (paper Appendix "Backward Correction and Gradient Computation").
//
// A work item is 128 query rows of one (batch, query head); the CTA that has it sweeps the key
// tiles (128 keys) up to the causal diagonal.  Where shared memory allows, a CTA takes one item
// after another (one CTA per SM; see QmCfg::kPersist for how the items are handed out).  For every
// key tile the tensor cores recompute
//     S  = Q^ K^^T   (row-blocked FP8 copies, contraction over the qk channels)
//     dP = dO^ V^^T  (row-blocked FP8 copies, contraction over the v channels)
// into tensor memory; the softmax warps rebuild P = 2^(S*scale*log2e - LSE*log2e) in FP32 from
// the saved LSE (not renormalised, not quantised) and then either
//   kDelta: accumulate D_i = sum_j P_ij dP_ij, or
//   kDQ:    form dS = P (dP - D), record the pre-cast row statistics, quantise dS in blocks of
//           32 keys in registers, hand the codes back through tensor memory and let the tensor
//           cores accumulate dQ += dS^ K^c (K copy blocked along keys).
// Both modes run the same instruction sequence for P and dP, so the correction the first
// produces is the one that zeroes the row sums of the second up to FP32 rounding.
//
// Warp roles: warp 0 TMA producer; warps 1, 2, 3 issue the S, dP and dQ MMAs (an issuing warp
// spends ~130 cycles per tcgen05 instruction whatever its size, so the MMAs are 128 keys wide and
// spread over three warps); warps 4..19 softmax: warp % 4 selects the 32 TMEM lanes (query rows),
// (warp - 4) / 4 the 32-key column group.  The softmax threads pull S and dP into registers and
// release the buffers at once, so the next tile's MMAs overlap the exponentials of this one.
//
// The kernel is a template over the operand width: element bytes (1: E4M3 codes with E8M0 block
// scales, 2: BF16 without scales) and the number of 128-byte chunks per operand row.  A key step
// always spans one 128-byte chunk of the token dimension (128 keys of codes, 64 keys of BF16).
// When the qk head dim exceeds 128 the dQ accumulator no longer fits beside S and dP in tensor
// memory; the dQ columns are then split in tiles of 128 over CTAs that each repeat the S / dP work.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <type_traits>

#include "common.cuh"
#include "mma_issue.cuh"
#include "mxfp8_device.cuh"
#include "sm100_ptx.cuh"

namespace attnfp8 {

namespace {

using namespace sm100;

constexpr int kTile = 128;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLog2eLo = 1.92596299e-8f;          // log2(e) minus its FP32 rounding
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kSmemLimit = 232448;                  // dynamic shared memory a CTA may ask for

// Operand geometry, ring depths and tensor-memory map of one instantiation.
template <bool kDQ_, int kEB_, int kCq_, int kCv_, int kEBv_ = kEB_>
struct QmCfg {
  static constexpr bool kDQ = kDQ_;
  static constexpr int kEB = kEB_;                      // bytes per operand element
  static constexpr int kCq = kCq_;                      // 128-byte chunks per Q / K row
  static constexpr int kCv = kCv_;                      // 128-byte chunks per dO / V row
  static constexpr int kEBv = kEBv_;                    // bytes per element of the dO / V row operands (dP only):
                                                        // 2 with kEB == 1 is the protected-dP ablation
  static constexpr bool kFp8 = kEB == 1;
  static constexpr bool kFp8v = kEBv == 1;
  // Both kernels are persistent where shared memory allows: a CTA walks a list of query tiles, with
  // the Q / dO tiles double-buffered and the K / V rings, the score buffers and their barriers
  // running on across tile boundaries, so that set-up, pipeline fill and most of the drain are paid
  // once per CTA instead of once per query tile.  The delta kernel takes a static list (all its CTAs
  // start together).  The dQ kernel is launched behind the key-major kernel, so its CTAs start at
  // different times: they draw their tiles from a ticket counter in the workspace instead.
  // FP8 at (256, 256) takes 64 keys per step: the whole dQ row (256 columns) then fits in tensor memory
  // next to S and dP (64 + 64 + 2 x 32 + 256 + 64 columns of scale factors = 512), and one CTA owns it
  static constexpr bool kHalf = kDQ && kEB == 1 && kEBv == 1 && kCq == 2 && kCv == 2;
  static constexpr int kStep = kHalf ? 64 : kTile / kEB; // keys per step
  static constexpr int kStepsPerTile = kTile / kStep;
  // FP8 at (192, 128): the whole dQ row (192 columns) stays in one CTA, which then runs S, dP and the
  // softmax once per item instead of once per 128-column tile of dQ.  Tensor memory holds it exactly when
  // the dS^ operand and every scale-factor slot are single: S 128 + dP 128 + dS^ 32 + dQ 192 + SF 32 = 512.
  // (BF16 at the same head dims has no scale factors and fits with room to spare; it takes the same path)
  static constexpr bool kOneCta = kDQ && ((kEB == 1 && kEBv == 1 && kCq == 2 && kCv == 1) || (kEB == 2 && kEBv == 2 && kCq == 3 && kCv == 2));
  static constexpr int kDsBufs = kOneCta ? 1 : 2;       // dS^ operand buffers (and their scale-byte slots)
  static constexpr int kSfSlots = kOneCta ? 1 : 2;      // scale-factor slots of the K, V and K^c stages
  static constexpr bool kWhole = kOneCta || kHalf;      // one CTA holds every dQ column of its rows
  static constexpr int kKcRows = kOneCta ? 192 : (kHalf ? 256 : 128);   // rows (dQ columns) of a K^c stage
  static constexpr int kDqCols = kKcRows;
  static constexpr int kKb = kStep * kEB / 32;          // 32-byte K steps of the dQ product per key step
  static constexpr bool kPersist =
      2 * (kCq + kCv) * kTile * 128 + 2 * ((kCq + kCv) * kStep * 128 + (kDQ ? kTile * 128 : 0)) <= 216 * 1024;
  static constexpr bool kTicket = kPersist && kDQ;
  static constexpr int kQBufs = kPersist ? 2 : 1;       // Q / dO tile buffers (and scale-factor slots)
  static constexpr int kGroups = kStep / 32;            // 32-key column groups of a step
  static constexpr int kSoftmaxThreads = 128 * kGroups; // 4 TMEM lane quadrants x column groups
  static constexpr int kThreads = 128 + kSoftmaxThreads;
  // K/V ring depth: deep enough to cover the L2 -> shared-memory latency of a tile (what fits);
  // the K^T ring of the dQ product falls back to one stage when two do not fit
  static constexpr int kFixedBytes = kQBufs * (kCq + kCv) * kTile * 128;
  static constexpr int kKvBytes = (kCq + kCv) * kStep * 128;
  static constexpr int kKcBytes = kDQ ? kKcRows * 128 : 0;
  static constexpr int kRaw = ((kPersist ? 216 : 224) * 1024 - kFixedBytes - kKcBytes) / (kKvBytes + kKcBytes);
  // (BF16 at head dim 256: the Q / dO tiles alone take 128 KB and a K / V step 64 KB, so the ring is
  // a single stage there: loads and MMAs of successive steps no longer overlap)
  static constexpr bool kTwoFit = kFixedBytes + 2 * kKvBytes + kKcBytes <= 212 * 1024;
  static constexpr int kStages = kRaw < 2 ? (kTwoFit ? 2 : 1) : (kRaw > 4 ? 4 : kRaw);
  static constexpr int kKcStages = !kDQ ? 1 : (kRaw < 2 ? 1 : kStages);
  // tensor memory
  // BF16 mode has no scale-factor columns and 64-key steps: a second S / dP pair fits, so the products of the
  // next step are issued while the softmax threads still work on this one (with one pair the 8 MMAs of a 64-key
  // step, their completion, the wake-up, the load and the release ran one after the other: 1175 cycles a step in
  // the correction pass at head dim 128, 0.683 -> 0.598 ms on the 8K workload; the wide head dims gain nothing)
  static constexpr int kSBufs = (kEB == 2 && kEBv == 2 && kCq == 2 && kCv == 2) ? 2 : 1;
  static constexpr uint32_t kSdp = 2 * kStep;           // columns of an S / dP pair
  static constexpr uint32_t kColS = 0, kColdP = kStep, kColdS = kSdp * kSBufs /* kDsBufs x 32 */, kColdQ = kColdS + 32 * kDsBufs;
  static constexpr uint32_t kColSFQ = kDQ ? kColdQ + kDqCols : kSdp * kSBufs;   // kQBufs slots (no dS^ / dQ columns without dQ)
  static constexpr uint32_t kColSFdO = kColSFQ + 4 * kCq * kQBufs;   // kQBufs slots
  static constexpr uint32_t kColSFK = kColSFdO + 4 * kCv * kQBufs;   // kSfSlots slots
  static constexpr uint32_t kColSFV = kColSFK + 4 * kSfSlots * kCq;
  static constexpr uint32_t kColSFdS = kColSFV + 4 * kSfSlots * kCv; // kDsBufs x 4
  static constexpr uint32_t kColSFKc = kColSFdS + 4 * kDsBufs;       // kSfSlots x 4 (one row tile of K^c at a time)
  static constexpr uint32_t kColsUsed = kFp8 ? kColSFKc + 4 * kSfSlots : kColSFQ;
  static constexpr uint32_t kTmemCols = 512;
  static_assert(kColsUsed <= 512, "tensor memory exceeded");
};

template <class C>
struct QmSmem {
  static constexpr int kStages = C::kStages;
  alignas(1024) uint8_t q[C::kQBufs][C::kCq][kTile * 128];
  alignas(1024) uint8_t dO[C::kQBufs][C::kCv][kTile * 128];
  alignas(1024) uint8_t k[kStages][C::kCq][C::kStep * 128];
  alignas(1024) uint8_t v[kStages][C::kCv][C::kStep * 128];
  alignas(1024) uint8_t kc[C::kKcStages][C::kDQ ? C::kKcRows * 128 : 1024];   // K^c tiles of the dQ product
  alignas(16) uint8_t sf_q[C::kQBufs][C::kCq * 512];
  alignas(16) uint8_t sf_dO[C::kQBufs][C::kCv * 512];
  alignas(16) uint8_t sf_k[kStages][C::kCq * 512];
  alignas(16) uint8_t sf_v[kStages][C::kCv * 512];
  alignas(16) uint8_t sf_kc[C::kKcStages][C::kWhole ? 1024 : 512];
  alignas(16) uint8_t sf_ds[2][512];
  alignas(16) float red[C::kGroups][5][kTile];   // partial row sums of every column group
  uint64_t q_full[C::kQBufs], q_empty[C::kQBufs];
  uint64_t kv_full[kStages], kv_empty[kStages];
  uint64_t kc_full[C::kKcStages], kc_empty[C::kKcStages];
  uint64_t sdp_full[2], sdp_free[2];   // per S / dP pair
  uint64_t ds_full[2], ds_free[2];
  uint64_t dq_done, dq_free;
  uint64_t item_full[4];        // ticket mode: the producer has published the CTA's i-th work item in item_l[i % 4]
  int item_l[4];
  uint64_t drain[3];
  uint32_t tmem_base;
  int abort_flag;
};

struct QmParams {
  const uint8_t *q_sf, *dO_sf, *k_sf, *v_sf, *kc_sf;
  const float* lse;
  const float* delta_in;
  float* delta_out;
  __nv_bfloat16* dq;
  float* rowsum;
  float* rowabs;
  float* post_rowsum;       // optional: row sums of the CAST score gradient (the dQ operand) and of its magnitude
  float* post_rowabs;
  float* p_abs_dp;          // optional (with rowsum): sum_j P_ij |dP^_ij|, the scale of the rounding dust of a row sum
  int* status;
  int* sched;               // ticket mode: the next item number; the host zeroes it ahead of the launch
  int N, Nk, q0t, Hq, Hkv, dqk, dv, causal;   // N query rows, Nk keys, q0t: tile offset of the causal diagonal
  int kv_lim;               // without the causal mask: last real key of the last key tile (127: all real)
  int gx, gy, gz;           // the (head x column tile, query tile, batch) grid the work items are numbered in
  int tail_wait;            // launched behind the key-major kernel of the same call (see launch_bwd_dq)
  float scale, scale_log2;
};

template <class C>
__global__ void __launch_bounds__(C::kThreads, 1)
qmajor_kernel(const QmParams p, const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_dO,
              const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
              const __grid_constant__ CUtensorMap tm_kc) {
  // declared with the alignment the swizzled operand tiles need, so that the compiler keeps the
  // shared state space of every access derived from it (checked below)
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  constexpr bool kDQ = C::kDQ, kFp8 = C::kFp8, kFp8v = C::kFp8v, kPersist = C::kPersist, kTicket = C::kTicket;
  constexpr int kStages = C::kStages, kKcStages = C::kKcStages, kEB = C::kEB, kCq = C::kCq, kCv = C::kCv;
  constexpr int kStep = C::kStep, kGroups = C::kGroups, kSoftmaxThreads = C::kSoftmaxThreads;
  constexpr uint32_t kColS = C::kColS, kColdP = C::kColdP, kColdS = C::kColdS, kColdQ = C::kColdQ, kColSFQ = C::kColSFQ,
                     kColSFdO = C::kColSFdO, kColSFK = C::kColSFK, kColSFV = C::kColSFV, kColSFdS = C::kColSFdS,
                     kColSFKc = C::kColSFKc, kTmemCols = C::kTmemCols;
  QmSmem<C>& sm = *reinterpret_cast<QmSmem<C>*>(smem_raw);
  if (smem_u32(smem_raw) & 1023u) {               // never expected: report instead of computing garbage
    if (threadIdx.x == 0) atomicExch(p.status, static_cast<int>(ATTN_ERR_ALIGNMENT));
    return;
  }
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // Work items are numbered x-fastest over the grid (gx, gy, gz): heads vary fastest and the heaviest
  // (latest) query tiles of all heads come first, so the light tiles fill the tail.  Without
  // persistence a CTA is its own item.  With a static list a persistent CTA takes the items c,
  // 2n-1-c, 2n+c, ... (n CTAs, c its index): alternate rounds run backwards, so that no CTA collects
  // the heavier item of every round.  In ticket mode the producer thread draws item numbers from a
  // global counter and publishes them to the other warps through shared memory.
  constexpr bool kOneCta = C::kOneCta, kHalf = C::kHalf, kWhole = C::kWhole;
  constexpr int kSBufs = C::kSBufs;
  constexpr uint32_t kSdp = C::kSdp;
  constexpr int kDsBufs = C::kDsBufs, kSfSlots = C::kSfSlots;
  const int rq_sf = (p.dqk + 127) / 128;                   // 128-row tiles of the K^c scale tensor
  const int rq = (kDQ && !kWhole) ? rq_sf : 1;            // dQ column tiles (128 wide) of one head, neighbours in x
  const int total_items = p.gx * p.gy * p.gz;
  const int n_cta = static_cast<int>(gridDim.x);
  const int n_static = !kPersist ? 1
                                 : total_items / n_cta + ((((total_items / n_cta) & 1) ? n_cta - 1 - static_cast<int>(blockIdx.x)
                                                                                         : static_cast<int>(blockIdx.x)) <
                                                              total_items % n_cta
                                                          ? 1 : 0);
  volatile int* abort_flag = &sm.abort_flag;
  struct Item { int qt, h, r_tile, b, g, n_tiles; bool valid; };
  auto decode = [&](int x, int y, int z) {
    Item it;
    it.qt = p.causal ? (p.gy - 1 - y) : y;
    it.h = x / rq; it.r_tile = x % rq; it.b = z;
    it.g = it.h / (p.Hq / p.Hkv);
    it.n_tiles = (p.causal ? it.qt + p.q0t + 1 : p.Nk / kTile) * C::kStepsPerTile;       // key steps
    it.valid = true;
    return it;
  };
  auto decode_linear = [&](int l) { return decode(l % p.gx, (l / p.gx) % p.gy, l / (p.gx * p.gy)); };
  // the i-th item of this CTA (valid = false: no more; in ticket mode also when the wait gave up)
  auto item_at = [&](int i) {
    Item none; none.valid = false; none.qt = none.h = none.r_tile = none.b = none.g = none.n_tiles = 0;
    if (!kPersist) return i == 0 ? decode(blockIdx.x, blockIdx.y, blockIdx.z) : none;
    if (!kTicket) {
      if (i >= n_static) return none;
      const int pos = (i & 1) ? n_cta - 1 - static_cast<int>(blockIdx.x) : static_cast<int>(blockIdx.x);
      return decode_linear(i * n_cta + pos);
    }
    if (!mbar_wait(&sm.item_full[i & 3], (i >> 2) & 1, abort_flag)) return none;
    const int l = *reinterpret_cast<volatile int*>(&sm.item_l[i & 3]);
    return l >= 0 ? decode_linear(l) : none;
  };
  const int nk_qk = p.dqk * kEB / 32, nk_v = p.dv * C::kEBv / 32;       // 32-byte K steps of the two products

  if (tid == 0) {
    for (int i = 0; i < C::kQBufs; ++i) { mbar_init(&sm.q_full[i], 1); mbar_init(&sm.q_empty[i], 2); }
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm.kv_full[s], 1); mbar_init(&sm.kv_empty[s], 2);   // released by the S and the dP issuer
    }
    for (int s = 0; s < kKcStages; ++s) { mbar_init(&sm.kc_full[s], 1); mbar_init(&sm.kc_empty[s], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&sm.sdp_full[i], 2); mbar_init(&sm.sdp_free[i], kSoftmaxThreads); }
    for (int i = 0; i < 2; ++i) { mbar_init(&sm.ds_full[i], kSoftmaxThreads); mbar_init(&sm.ds_free[i], 1); }
    mbar_init(&sm.dq_done, 1); mbar_init(&sm.dq_free, kSoftmaxThreads);
    for (int i = 0; i < 4; ++i) mbar_init(&sm.item_full[i], 1);
    for (int i = 0; i < 3; ++i) mbar_init(&sm.drain[i], 1);
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
      prefetch_tmap(&tm_q); prefetch_tmap(&tm_dO); prefetch_tmap(&tm_k); prefetch_tmap(&tm_v);
      if (kDQ) prefetch_tmap(&tm_kc);
      const int tiles_n = p.N / kTile, tiles_nk = p.Nk / kTile;
      int issued_kv = 0, issued_kc = 0;
      bool ok = true;
      int T = 0;                                      // key steps of the items before this one
      int ticket = kTicket ? atomicAdd(p.sched, 1) : 0;
      for (int i = 0; ok; ++i) {
        const int qb = i % C::kQBufs;
        if (kPersist && i >= C::kQBufs) {
          // both issuers have finished with the item that used this Q / dO buffer (and every warp has
          // long read the slot of the item list that is about to be rewritten)
          ok = mbar_wait(&sm.q_empty[qb], ((i / C::kQBufs) - 1) & 1, abort_flag);
          if (!ok) break;
        }
        Item it;
        if (kTicket) {
          // publish this CTA's i-th item (or the end of the list) to the other warps, and draw the
          // next ticket now: its latency passes while this item's copies are issued
          const int l = ticket < total_items ? ticket : -1;
          sm.item_l[i & 3] = l;
          mbar_arrive(&sm.item_full[i & 3]);
          if (l < 0) break;
          it = decode_linear(l);
          ticket = atomicAdd(p.sched, 1);
        } else {
          it = item_at(i);
          if (!it.valid) break;
        }
        const int q_slab = it.b * p.Hq + it.h, kv_slab = it.b * p.Hkv + it.g;
        mbar_arrive_expect_tx(&sm.q_full[qb], kCq * (kTile * 128 + (kFp8 ? 512 : 0)) + kCv * (kTile * 128 + (kFp8v ? 512 : 0)));
        for (int c = 0; c < kCq; ++c) tma_load_2d(sm.q[qb][c], &tm_q, &sm.q_full[qb], 128 * c, q_slab * p.N + it.qt * kTile);
        for (int c = 0; c < kCv; ++c) tma_load_2d(sm.dO[qb][c], &tm_dO, &sm.q_full[qb], 128 * c, q_slab * p.N + it.qt * kTile);
        if (kFp8)
          bulk_load_1d(sm.sf_q[qb], p.q_sf + (static_cast<size_t>(q_slab) * tiles_n + it.qt) * kCq * 512, kCq * 512, &sm.q_full[qb]);
        if (kFp8v)
          bulk_load_1d(sm.sf_dO[qb], p.dO_sf + (static_cast<size_t>(q_slab) * tiles_n + it.qt) * kCv * 512, kCv * 512, &sm.q_full[qb]);
        for (int t = 0; t < it.n_tiles && ok; ++t) {
          const int gt = T + t;                       // step index over all items of this CTA: the rings run on
          const int s = gt % kStages, u = gt / kStages;
          ok = mbar_wait(&sm.kv_empty[s], (u & 1) ^ 1, abort_flag);
          if (!ok) break;
          mbar_arrive_expect_tx(&sm.kv_full[s], kCq * (kStep * 128 + (kFp8 ? 512 : 0)) + kCv * (kStep * 128 + (kFp8v ? 512 : 0)));
          for (int c = 0; c < kCq; ++c) tma_load_2d(sm.k[s][c], &tm_k, &sm.kv_full[s], 128 * c, kv_slab * p.Nk + t * kStep);
          for (int c = 0; c < kCv; ++c) tma_load_2d(sm.v[s][c], &tm_v, &sm.kv_full[s], 128 * c, kv_slab * p.Nk + t * kStep);
          // (64-key steps: both halves of a key tile load the tile's scale bytes and its K^c chunk)
          const int tt = kHalf ? t >> 1 : t;          // 128-key tile of the scale tensors / 128-byte chunk of K^c
          if (kFp8)
            bulk_load_1d(sm.sf_k[s], p.k_sf + (static_cast<size_t>(kv_slab) * tiles_nk + tt) * kCq * 512, kCq * 512, &sm.kv_full[s]);
          if (kFp8v)
            bulk_load_1d(sm.sf_v[s], p.v_sf + (static_cast<size_t>(kv_slab) * tiles_nk + tt) * kCv * 512, kCv * 512, &sm.kv_full[s]);
          ++issued_kv;
          if (kDQ) {
            const int sc = gt % kKcStages;
            ok = mbar_wait(&sm.kc_empty[sc], ((gt / kKcStages) & 1) ^ 1, abort_flag);
            if (!ok) break;
            if (kWhole) {
              mbar_arrive_expect_tx(&sm.kc_full[sc], C::kKcRows * 128 + (kFp8 ? 2 * 512 : 0));
              tma_load_2d(sm.kc[sc], &tm_kc, &sm.kc_full[sc], tt * 128, kv_slab * p.dqk);
              for (int r = 0; kFp8 && r < 2; ++r)
                bulk_load_1d(sm.sf_kc[sc] + 512 * r, p.kc_sf + ((static_cast<size_t>(kv_slab) * rq_sf + r) * tiles_nk + tt) * 512, 512,
                             &sm.kc_full[sc]);
            } else {
              mbar_arrive_expect_tx(&sm.kc_full[sc], min(128, p.dqk) * 128 + (kFp8 ? 512 : 0));
              tma_load_2d(sm.kc[sc], &tm_kc, &sm.kc_full[sc], t * 128, kv_slab * p.dqk + 128 * it.r_tile);
              if (kFp8)
                bulk_load_1d(sm.sf_kc[sc], p.kc_sf + ((static_cast<size_t>(kv_slab) * rq_sf + it.r_tile) * tiles_nk + t) * 512, 512,
                             &sm.kc_full[sc]);
            }
            ++issued_kc;
          }
        }
        T += it.n_tiles;
      }
      if (!ok) {
        int dummy = 0;
        for (int t = max(0, issued_kv - kStages); t < issued_kv; ++t)
          mbar_wait(&sm.kv_full[t % kStages], (t / kStages) & 1, &dummy);
        for (int t = max(0, issued_kc - kKcStages); t < issued_kc; ++t)
          mbar_wait(&sm.kc_full[t % kKcStages], (t / kKcStages) & 1, &dummy);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ S issuer
    {
      bool ok = true;
      int T = 0;
      for (int i = 0; ok; ++i) {
        const Item it = item_at(i);
        if (!it.valid) break;
        const int qb = i % C::kQBufs;
        const uint64_t desc_q = make_desc_sw128(smem_u32(sm.q[qb][0]));
        const uint32_t t_sfq = tmem + kColSFQ + 4 * kCq * qb;
        ok = mbar_wait(&sm.q_full[qb], (i / C::kQBufs) & 1, abort_flag);
        if (!ok) break;
        if (kFp8) {
          tc_fence_after_sync();
          sf_copy_tiles<kCq>(t_sfq, sm.sf_q[qb]);
        }
        for (int t = 0; t < it.n_tiles && ok; ++t) {
          const int gt = T + t;
          const int s = gt % kStages, slot = kSfSlots == 2 ? (gt & 1) : 0;
          ok = mbar_wait(&sm.kv_full[s], (gt / kStages) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          if (kFp8 && kSfSlots == 2) sf_copy_tiles<kCq>(tmem + kColSFK + 4 * kCq * slot, sm.sf_k[s]);
          const int sb = kSBufs == 2 ? (gt & 1) : 0;   // S / dP pair of this step
          if (gt >= kSBufs) {
            // the softmax threads have pulled the S and dP that last used this pair into registers
            ok = mbar_wait(&sm.sdp_free[sb], (kSBufs == 2 ? (gt >> 1) - 1 : gt - 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after_sync();
          }
          // a single scale slot is rewritten only now that the product that read it has been consumed
          if (kFp8 && kSfSlots == 1) sf_copy_tiles<kCq>(tmem + kColSFK, sm.sf_k[s]);
          const uint64_t desc_k = make_desc_sw128(smem_u32(sm.k[s][0]));
          issue_ss<kFp8, kCq, kStep, kTile * 128 / 16, kStep * 128 / 16>(tmem + kColS + kSdp * sb, desc_q, desc_k, nk_qk, t_sfq,
                                                                          tmem + kColSFK + 4 * kCq * slot + (kHalf ? 2 * (t & 1) : 0));
          mma_commit_elect(&sm.sdp_full[sb]);
          mma_commit_elect(&sm.kv_empty[s]);
        }
        if (kPersist && ok) mma_commit_elect(&sm.q_empty[qb]);     // this item's Q tile has been read
        T += it.n_tiles;
      }
      if (*abort_flag) ok = false;
      if (!ok) {
        int dummy = 0;
        mma_commit_elect(&sm.drain[0]);
        mbar_wait(&sm.drain[0], 0, &dummy);
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ dP issuer
    {
      bool ok = true;
      int T = 0;
      for (int i = 0; ok; ++i) {
        const Item it = item_at(i);
        if (!it.valid) break;
        const int qb = i % C::kQBufs;
        const uint64_t desc_dO = make_desc_sw128(smem_u32(sm.dO[qb][0]));
        const uint32_t t_sfdO = tmem + kColSFdO + 4 * kCv * qb;
        ok = mbar_wait(&sm.q_full[qb], (i / C::kQBufs) & 1, abort_flag);
        if (!ok) break;
        if (kFp8v) {
          tc_fence_after_sync();
          sf_copy_tiles<kCv>(t_sfdO, sm.sf_dO[qb]);
        }
        for (int t = 0; t < it.n_tiles && ok; ++t) {
          const int gt = T + t;
          const int s = gt % kStages, slot = kSfSlots == 2 ? (gt & 1) : 0;
          ok = mbar_wait(&sm.kv_full[s], (gt / kStages) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          if (kFp8v && kSfSlots == 2) sf_copy_tiles<kCv>(tmem + kColSFV + 4 * kCv * slot, sm.sf_v[s]);
          const int sb = kSBufs == 2 ? (gt & 1) : 0;
          if (gt >= kSBufs) {
            ok = mbar_wait(&sm.sdp_free[sb], (kSBufs == 2 ? (gt >> 1) - 1 : gt - 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after_sync();
          }
          if (kFp8v && kSfSlots == 1) sf_copy_tiles<kCv>(tmem + kColSFV, sm.sf_v[s]);
          const uint64_t desc_v = make_desc_sw128(smem_u32(sm.v[s][0]));
          issue_ss<kFp8v, kCv, kStep, kTile * 128 / 16, kStep * 128 / 16>(tmem + kColdP + kSdp * sb, desc_dO, desc_v, nk_v, t_sfdO,
                                                                          tmem + kColSFV + 4 * kCv * slot + (kHalf ? 2 * (t & 1) : 0));
          mma_commit_elect(&sm.sdp_full[sb]);
          mma_commit_elect(&sm.kv_empty[s]);
        }
        if (kPersist && ok) mma_commit_elect(&sm.q_empty[qb]);     // this item's dO tile has been read
        T += it.n_tiles;
      }
      if (*abort_flag) ok = false;
      if (!ok) {
        int dummy = 0;
        mma_commit_elect(&sm.drain[1]);
        mbar_wait(&sm.drain[1], 0, &dummy);
      }
    }
  } else if (warp == 3) {
    // ------------------------------------------------------------------ dQ issuer
    if (kDQ) {
      bool ok = true;
      int T = 0;
      for (int i = 0; ok; ++i) {
        const Item it = item_at(i);
        if (!it.valid) break;
        const int n_tiles = it.n_tiles;
        const int n_dq = kWhole ? p.dqk : min(128, p.dqk - 128 * it.r_tile);   // dQ columns of this CTA
        if (i > 0) {
          // the softmax threads have read the previous item's dQ out of tensor memory
          ok = mbar_wait(&sm.dq_free, (i - 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
        }
        for (int t = 0; t < n_tiles && ok; ++t) {
          const int gt = T + t;                       // the K^T ring and the dS^ buffers run on across items
          const int s = gt % kKcStages, slot = kSfSlots == 2 ? (gt & 1) : 0, buf = kDsBufs == 2 ? (gt & 1) : 0;
          ok = mbar_wait(&sm.kc_full[s], (gt / kKcStages) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          if (kFp8 && !kWhole) sf_copy_elect(tmem + kColSFKc + 4 * slot, make_desc_sf(smem_u32(sm.sf_kc[s])));
          ok = mbar_wait(&sm.ds_full[buf], (kDsBufs == 2 ? gt >> 1 : gt) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          if (kFp8) sf_copy_elect(tmem + kColSFdS + 4 * buf, make_desc_sf(smem_u32(sm.sf_ds[buf])));
          const uint64_t desc_kc = make_desc_sw128(smem_u32(sm.kc[s]));
          if (kWhole) {
            // The dQ columns are two row tiles of K^c (128 + 64, or 128 + 128), one after the other.  With a
            // single scale slot both go through it: copies and MMAs of one thread run in the order issued,
            // and the step before has completed (its commit released the single dS^ buffer this step's
            // operand came through).  With 64-key steps the operand is half of the 128-byte chunk (K steps
            // koff, koff + 1), each row tile has a scale slot of its own and the dS^ buffers alternate.
            const int koff = kHalf ? 2 * (t & 1) : 0;
#pragma unroll
            for (int r = 0; r < 2; ++r) {
              const uint32_t t_sfkc = tmem + kColSFKc + (kHalf ? 4 * r : 0);
              if (kFp8) sf_copy_elect(t_sfkc, make_desc_sf(smem_u32(sm.sf_kc[s] + 512 * r)));
#pragma unroll
              for (int kb = 0; kb < C::kKb; ++kb) {
                if (kFp8)
                  mma_mxf8_ts_elect(tmem + kColdQ + 128 * r, tmem + kColdS + 32 * buf + 8 * kb,
                                    desc_kc + (r * (128 * 128 / 16) + 2 * (koff + kb)),
                                    make_idesc_mxf8(128, r == 0 ? 128 : n_dq - 128, kb, koff + kb), tmem + kColSFdS + 4 * buf,
                                    t_sfkc, (t > 0 || kb > 0));
                else
                  mma_bf16_ts_elect(tmem + kColdQ + 128 * r, tmem + kColdS + 32 * buf + 8 * kb,
                                    desc_kc + (r * (128 * 128 / 16) + 2 * kb), make_idesc_bf16(128, r == 0 ? 128 : n_dq - 128),
                                    (t > 0 || kb > 0));
              }
            }
          } else
#pragma unroll
          for (int kb = 0; kb < 4; ++kb) {
            if (kFp8)
              mma_mxf8_ts_elect(tmem + kColdQ, tmem + kColdS + 32 * buf + 8 * kb, desc_kc + 2 * kb,
                                make_idesc_mxf8(128, n_dq, kb, kb), tmem + kColSFdS + 4 * buf, tmem + kColSFKc + 4 * slot,
                                (t > 0 || kb > 0));
            else
              mma_bf16_ts_elect(tmem + kColdQ, tmem + kColdS + 32 * buf + 8 * kb, desc_kc + 2 * kb,
                                make_idesc_bf16(128, n_dq), (t > 0 || kb > 0));
          }
          mma_commit_elect(&sm.ds_free[buf]);            // operand and scale bytes of this buffer may be overwritten
          mma_commit_elect(&sm.kc_empty[s]);
          if (t == n_tiles - 1) mma_commit_elect(&sm.dq_done);
        }
        T += n_tiles;
      }
      if (*abort_flag) ok = false;
      if (!ok) {
        int dummy = 0;
        mma_commit_elect(&sm.drain[2]);
        mbar_wait(&sm.drain[2], 0, &dummy);
      }
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ softmax
    const int grp = (warp - 4) >> 2;                  // 32-key column group of the tile
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
    auto row_of = [&](const Item& it) {
      return static_cast<size_t>(it.b * p.Hq + it.h) * p.N + it.qt * kTile + row;
    };
    bool ok = true;
    int T = 0;                                        // key steps of the items before this one
    Item it = item_at(0);
    float lse_next = 0.f, d_next = 0.f;
    if (it.valid) {
      lse_next = p.lse[row_of(it)];
      if (kDQ) d_next = p.delta_in[row_of(it)];
    }
    for (int i = 0; ok && it.valid; ++i) {
    const int qt = it.qt, r_tile = it.r_tile, n_tiles = it.n_tiles;
    const int n_dq = kWhole ? p.dqk : min(128, p.dqk - 128 * r_tile);   // dQ columns of this CTA
    // first key of the masked tile (the diagonal one; without the causal mask the last one, when the sequence
    // ends inside it)
    const int mask_from = p.causal ? (qt + p.q0t) * kTile : (p.kv_lim < kTile - 1 ? p.Nk - kTile : 0x7fffffff);
    // LSE * log2(e) as an unevaluated sum hi + lo, so that rebuilding P adds no rounding of its own
    // to the half ulp the FP32 storage of LSE already carries
    const float lse_nat = lse_next;
    const float lse2 = lse_nat * kLog2e;
    const float lse2_lo = fmaf(lse_nat, kLog2e, -lse2) + lse_nat * kLog2eLo;
    const float D = d_next;
    const float f_lo = fmaf(-lse2_lo, kLn2, 1.0f);   // 2^-lo to first order (|lo| < 1e-5)
    const float fD = f_lo * D;
    float acc0 = 0.f, acc1 = 0.f;                     // kDelta: sum P dP (kDQ: used by the final sum only)
    // kDQ with statistics: sum dS and sum |dS| live in shared memory (slots 0 and 1), a step's share added
    // after the step, so that the common path carries no register for them
    if (kDQ && p.rowsum) { sm.red[grp][0][row] = 0.f; sm.red[grp][1][row] = 0.f; }
    // kDQ with statistics, on request: sum P |dP| (without the factor f_lo), kept in shared memory like the
    // post-cast sums so that the common path carries no extra register
    if (kDQ && p.p_abs_dp) sm.red[grp][4][row] = 0.f;
    // kDQ, on request: sum dS', sum |dS'| of the cast values, kept in shared memory so that the
    // common path carries no extra registers
    const bool want_post = kDQ && p.post_rowsum != nullptr;
    if (want_post) {
      sm.red[grp][2][row] = 0.f;
      sm.red[grp][3][row] = 0.f;
    }
    for (int t = 0; t < n_tiles; ++t) {
      const int gt = T + t;                           // step index over all items: the dS^ buffers run on
      const int buf = kDsBufs == 2 ? (gt & 1) : 0;
      const int sb = kSBufs == 2 ? (gt & 1) : 0;
      ok = mbar_wait(&sm.sdp_full[sb], (kSBufs == 2 ? gt >> 1 : gt) & 1, abort_flag);
      if (!ok) break;
      tc_fence_after_sync();
      uint32_t sr[32], dpr[32];
      tmem_ld32(tmem + kColS + kSdp * sb + lane_addr + 32 * grp, sr);
      tmem_ld32(tmem + kColdP + kSdp * sb + lane_addr + 32 * grp, dpr);
      tmem_wait_ld();
      tc_fence_before_sync();
      mbar_arrive(&sm.sdp_free[sb]);
      // column, inside the query tile's own key range, of this thread's first element (negative
      // before the diagonal tile)
      // (without the causal mask: inside the last key tile, where a ragged sequence ends)
      const int col0 = t * kStep - mask_from + 32 * grp;
      float ds[32];
      // P = 2^(x - lo) = 2^x * f with x = S*scale*log2e - hi and f = 2^-lo folded into the factors
      // that multiply P; the causal mask only exists on the diagonal tile, so the other tiles run
      // a loop without it
      // two elements per instruction (fma / mul .f32x2) wherever the arithmetic allows
      const float2 sc2 = make_float2(p.scale_log2, p.scale_log2), nl2 = make_float2(-lse2, -lse2);
      const float2 fl2 = make_float2(f_lo, f_lo), nfd2 = make_float2(-fD, -fD);
      float2 part2 = make_float2(0.f, 0.f);
      float a2 = 0.f;                                  // this step's share of sum P |dP| (statistics only)
      float s0 = 0.f, s1 = 0.f;                        // ... of sum dS and sum |dS|
      auto body = [&](auto diag_tag, auto stats_tag) {
        constexpr bool kDiag = decltype(diag_tag)::value;
        constexpr bool kStats = decltype(stats_tag)::value;      // pre-cast row statistics requested
        const int lim = p.causal ? row : p.kv_lim;               // last visible column of the masked tile
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          float2 x2 = __ffma2_rn(make_float2(__uint_as_float(sr[c]), __uint_as_float(sr[c + 1])), sc2, nl2);
          if (kDiag) {
            if (col0 + c > lim) x2.x = -INFINITY;
            if (col0 + c + 1 > lim) x2.y = -INFINITY;
          }
          const float2 pr2 = make_float2(ex2_approx(x2.x), ex2_approx(x2.y));
          const float2 dp2 = make_float2(__uint_as_float(dpr[c]), __uint_as_float(dpr[c + 1]));
          if (kDQ) {
            const float2 d2 = __fmul2_rn(pr2, __ffma2_rn(dp2, fl2, nfd2));
            ds[c] = d2.x;
            ds[c + 1] = d2.y;
            if (kStats) {
              s0 += d2.x + d2.y;
              s1 += fabsf(d2.x) + fabsf(d2.y);
              a2 = fmaf(pr2.x, fabsf(dp2.x), fmaf(pr2.y, fabsf(dp2.y), a2));
            }
          } else {
            part2 = __ffma2_rn(pr2, dp2, part2);
          }
        }
      };
      const bool diag = t * kStep >= mask_from;
      if (kDQ && p.rowsum != nullptr) {
        if (diag) body(std::true_type{}, std::true_type{}); else body(std::false_type{}, std::true_type{});
        sm.red[grp][0][row] += s0;
        sm.red[grp][1][row] += s1;
        if (p.p_abs_dp) sm.red[grp][4][row] += a2;
      } else {
        if (diag) body(std::true_type{}, std::false_type{}); else body(std::false_type{}, std::false_type{});
      }
      if (!kDQ) {
        acc0 = fmaf(part2.x + part2.y, f_lo, acc0);
      } else {
        uint32_t words[8 * kEB];
        uint32_t byte = 0;
        if (kFp8) {
          byte = quantize_block32(ds, words);
        } else {
#pragma unroll
          for (int i = 0; i < 8 * kEB; ++i) words[i] = cvt_bf16x2(ds[(2 * i) & 31], ds[(2 * i + 1) & 31]);
        }
        if (__builtin_expect(want_post, 0)) {
          // decode what the tensor cores will read: code * 2^(byte - 127), or the BF16 value
          float ps = 0.f, pa = 0.f;
          if (kFp8) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              uint32_t h01, h23;                       // E4M3 -> FP16 is exact
              asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h01) : "h"(static_cast<uint16_t>(words[i] & 0xFFFF)));
              asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h23) : "h"(static_cast<uint16_t>(words[i] >> 16)));
              const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&h01));
              const float2 bq = __half22float2(*reinterpret_cast<const __half2*>(&h23));
              ps += (a.x + a.y) + (bq.x + bq.y);
              pa += (fabsf(a.x) + fabsf(a.y)) + (fabsf(bq.x) + fabsf(bq.y));
            }
            const float sc = __uint_as_float(byte << 23);     // 2^(byte - 127); an all-zero block has byte 0 and sums 0
            ps *= sc;
            pa *= sc;
          } else {
#pragma unroll
            for (int i = 0; i < 8 * kEB; ++i) {
              const float lo = __uint_as_float(words[i] << 16), hi = __uint_as_float(words[i] & 0xFFFF0000u);
              ps += lo + hi;
              pa += fabsf(lo) + fabsf(hi);
            }
          }
          sm.red[grp][2][row] += ps;
          sm.red[grp][3][row] += pa;
        }
        if (gt >= kDsBufs) {
          // the dQ MMAs of the step that last used this buffer have consumed its operand and scale bytes
          ok = mbar_wait(&sm.ds_free[buf], (kDsBufs == 2 ? (gt - 2) >> 1 : gt - 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
        }
#pragma unroll
        for (int i = 0; i < kEB; ++i) tmem_st8(tmem + kColdS + 32 * buf + lane_addr + 8 * kEB * grp + 8 * i, words + 8 * i);
        if (kFp8) sts_u8(&sm.sf_ds[buf][(row & 31) * 16 + (row >> 5) * 4 + grp], byte);
        tmem_wait_st();
        fence_proxy_async_smem();
        tc_fence_before_sync();
        mbar_arrive(&sm.ds_full[buf]);
      }
    }
    // the next item (published by now, as a rule): its LSE and D are in flight during this item's epilogue
    Item nx; nx.valid = false;
    if (kPersist && ok) {
      nx = item_at(i + 1);
      if (nx.valid) {
        lse_next = p.lse[row_of(nx)];
        if (kDQ) d_next = p.delta_in[row_of(nx)];
      }
    }
    const size_t grow = row_of(it);                   // (formed here: not a register of the step loop)
    // combine the row sums of the column groups (fixed order: reproducible).  The persistent
    // delta kernel alternates between two slots, so that the next item's partial sums do not
    // overwrite what group 0 may still be reading.
    const int si = (kPersist && !kDQ) ? (i & 1) : 0;   // the dQ kernel uses slots 0 and 1 and a barrier per item
    if (!kDQ) sm.red[grp][si][row] = acc0;
    if (kDQ && p.p_abs_dp) sm.red[grp][4][row] *= f_lo;
    named_barrier_sync(1, kSoftmaxThreads);
    if (ok && grp == 0) {
      acc0 = 0.f; acc1 = 0.f;
      for (int j = 0; j < kGroups; ++j) {
        acc0 += sm.red[j][si][row];
        if (kDQ) acc1 += sm.red[j][1][row];
      }
      if (!kDQ) {
        p.delta_out[grow] = acc0;
      } else if (p.rowsum && r_tile == 0) {
        p.rowsum[grow] = acc0;
        p.rowabs[grow] = acc1;
        if (p.p_abs_dp) {
          float dust = 0.f;
          for (int j = 0; j < kGroups; ++j) dust += sm.red[j][4][row];
          p.p_abs_dp[grow] = dust;
        }
        if (p.post_rowsum) {
          float post0 = 0.f, post1 = 0.f;
          for (int j = 0; j < kGroups; ++j) { post0 += sm.red[j][2][row]; post1 += sm.red[j][3][row]; }
          p.post_rowsum[grow] = post0;
          p.post_rowabs[grow] = post1;
        }
      }
    }
    if (kDQ && ok) {
      ok = mbar_wait(&sm.dq_done, i & 1, abort_flag);
      if (ok) {
        tc_fence_after_sync();
        __nv_bfloat16* out_row = p.dq + grow * p.dqk + 128 * r_tile;
        for (int c0 = grp * 32; c0 < n_dq; c0 += 32 * kGroups) {
          uint32_t r[32];
          tmem_ld32(tmem + kColdQ + lane_addr + c0, r);
          tmem_wait_ld();
          uint32_t packed[16];
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            __nv_bfloat162 v2 = __floats2bfloat162_rn(__uint_as_float(r[2 * c]) * p.scale, __uint_as_float(r[2 * c + 1]) * p.scale);
            packed[c] = *reinterpret_cast<uint32_t*>(&v2);
          }
          uint4* dst = reinterpret_cast<uint4*>(out_row + c0);
#pragma unroll
          for (int c = 0; c < 4; ++c) dst[c] = make_uint4(packed[4 * c], packed[4 * c + 1], packed[4 * c + 2], packed[4 * c + 3]);
        }
        if (kPersist) {
          // the accumulator may be overwritten by the next item's first dQ MMA
          tc_fence_before_sync();
          mbar_arrive(&sm.dq_free);
        }
      }
    }
    // the row-sum slots may be overwritten by the next item's partial sums
    if (kDQ && kPersist) named_barrier_sync(1, kSoftmaxThreads);
    T += n_tiles;
    it = nx;
    }  // items
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
  if (tid == 0 && sm.abort_flag) atomicExch(p.status, static_cast<int>(ATTN_ERR_TIMEOUT));
  // This grid may have started while the grid ahead of it was draining.  One CTA, the last in
  // launch order, stays until that grid has completed, so that the completion of this grid
  // implies the completion of both for whatever follows in the stream.
  if (p.tail_wait && tid == 0 && blockIdx.x == gridDim.x - 1 && blockIdx.y == gridDim.y - 1 && blockIdx.z == gridDim.z - 1)
    griddep_wait();
}

template <class C>
attn_status_t launch_qmajor_t(const AttnShape& s, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v, attn_qtensor_t dO,
                              const float* lse, const float* delta_in, float* delta_out, void* dq, float* rowsum,
                              float* rowabs, float* post_rowsum, float* post_rowabs, int* status, cudaStream_t stream,
                              bool behind_dkdv, float* p_abs_dp) {
  constexpr bool kDQ = C::kDQ;
  static_assert(sizeof(QmSmem<C>) + 1024 <= kSmemLimit, "shared memory exceeded");
  CUtensorMap tm_q, tm_dO, tm_k, tm_v, tm_kc;
  attn_status_t st;
  const uint64_t eb = C::kEB, ebv = C::kEBv;
  const uint64_t q_rows = static_cast<uint64_t>(s.B) * s.Hq * s.N, kv_rows = static_cast<uint64_t>(s.B) * s.Hkv * s.Nk;
  if ((st = encode_tmap_u8_sw128(&tm_q, q.row_codes, s.dqk * eb, q_rows, kTile)) != ATTN_OK) return st;
  if ((st = encode_tmap_u8_sw128(&tm_dO, dO.row_codes, s.dv * ebv, q_rows, kTile)) != ATTN_OK) return st;
  if ((st = encode_tmap_u8_sw128(&tm_k, k.row_codes, s.dqk * eb, kv_rows, C::kStep)) != ATTN_OK) return st;
  if ((st = encode_tmap_u8_sw128(&tm_v, v.row_codes, s.dv * ebv, kv_rows, C::kStep)) != ATTN_OK) return st;
  if (kDQ) {
    if ((st = encode_tmap_u8_sw128(&tm_kc, k.col_codes, s.Nk * eb, static_cast<uint64_t>(s.B) * s.Hkv * s.dqk,
                                   C::kWhole ? C::kKcRows : (s.dqk < 128 ? s.dqk : 128))) != ATTN_OK)
      return st;
  } else {
    tm_kc = tm_k;
  }
  QmParams p;
  p.q_sf = q.row_scales; p.dO_sf = dO.row_scales; p.k_sf = k.row_scales; p.v_sf = v.row_scales;
  p.kc_sf = kDQ ? k.col_scales : nullptr;
  p.lse = lse; p.delta_in = delta_in; p.delta_out = delta_out;
  p.dq = static_cast<__nv_bfloat16*>(dq); p.rowsum = rowsum; p.rowabs = rowabs; p.post_rowsum = post_rowsum; p.post_rowabs = post_rowabs; p.p_abs_dp = p_abs_dp; p.status = status;
  p.N = s.N; p.Nk = s.Nk; p.q0t = s.q0t; p.kv_lim = s.kv_lim; p.Hq = s.Hq; p.Hkv = s.Hkv; p.dqk = s.dqk; p.dv = s.dv; p.causal = s.causal;
  p.scale = s.scale; p.scale_log2 = s.scale * kLog2e;
  p.tail_wait = behind_dkdv ? 1 : 0;
  p.sched = status + 4;                             // bytes 16..23 of the workspace header
  const size_t smem = sizeof(QmSmem<C>) + 1024;
  cudaError_t e = cudaFuncSetAttribute(qmajor_kernel<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "bwd q-major: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  const int rq = (kDQ && !C::kWhole) ? (s.dqk + 127) / 128 : 1;
  dim3 grid(s.Hq * rq, s.N / kTile, s.B);
  p.gx = static_cast<int>(grid.x); p.gy = static_cast<int>(grid.y); p.gz = static_cast<int>(grid.z);
  if (C::kPersist) {
    // one CTA per SM (the kernel takes a whole SM's shared memory) walks the item list
    int dev = 0, sms = 0;
    e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess || sms < 1) return fail(ATTN_ERR_CUDA, "bwd q-major: SM count: %s", cudaGetErrorString(e));
    const long long items = static_cast<long long>(p.gx) * p.gy * p.gz;
    if (items > 0x7fffffffLL) return fail(ATTN_ERR_UNSUPPORTED, "bwd q-major: %lld work items exceed 2^31 - 1", items);
    grid = dim3(static_cast<unsigned>(items < sms ? items : sms), 1, 1);
  }
  if (behind_dkdv) {
    // the key-major kernel ahead in the stream reads what this one reads and writes other buffers:
    // this grid may take the SMs that kernel's last wave leaves idle
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = dim3(C::kThreads); cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, qmajor_kernel<C>, p, tm_q, tm_dO, tm_k, tm_v, tm_kc);
    if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "bwd q-major: launch: %s", cudaGetErrorString(e));
  } else {
    qmajor_kernel<C><<<grid, C::kThreads, smem, stream>>>(p, tm_q, tm_dO, tm_k, tm_v, tm_kc);
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "bwd q-major: launch: %s", cudaGetErrorString(e));
  return ATTN_OK;
}

template <bool kDQ>
attn_status_t launch_qmajor(const AttnShape& s, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v, attn_qtensor_t dO,
                            const float* lse, const float* delta_in, float* delta_out, void* dq, float* rowsum,
                            float* rowabs, float* post_rowsum, float* post_rowabs, int* status, cudaStream_t stream,
                            bool behind_dkdv = false, float* p_abs_dp = nullptr) {
  const int cq = (s.dqk * s.eb + 127) / 128, cv = (s.dv * s.ebv + 127) / 128;
#define ATTN_QM_CASE(EB, CQ, CV, EBV)                                                                         \
  if (s.eb == EB && s.ebv == EBV && cq == CQ && cv == CV)                                                     \
    return launch_qmajor_t<QmCfg<kDQ, EB, CQ, CV, EBV>>(s, q, k, v, dO, lse, delta_in, delta_out, dq, rowsum, rowabs, \
                                                       post_rowsum, post_rowabs, status, stream, behind_dkdv, p_abs_dp);
  ATTN_QM_CASE(1, 1, 1, 1)
  ATTN_QM_CASE(1, 2, 1, 1)
  ATTN_QM_CASE(1, 2, 2, 1)
  ATTN_QM_CASE(2, 1, 1, 2)
  ATTN_QM_CASE(2, 2, 2, 2)
  ATTN_QM_CASE(2, 3, 2, 2)
  ATTN_QM_CASE(2, 4, 4, 2)
  ATTN_QM_CASE(1, 1, 1, 2)   // protected dP, d = 64
  ATTN_QM_CASE(1, 1, 2, 2)   // protected dP, d = 128
#undef ATTN_QM_CASE
  return fail(ATTN_ERR_UNSUPPORTED, "bwd q-major: no kernel for head dims (%d, %d) at %d bytes per element", s.dqk, s.dv,
              s.eb);
}

// Stale delta: D_i = sum_c dO_ic O_ic from the BF16 tensors (paper Section 3.2).  One warp per row.
__global__ void stale_delta_kernel(const __nv_bfloat16* __restrict__ dO, const __nv_bfloat16* __restrict__ o,
                                   float* __restrict__ delta, size_t rows, int dv) {
  const size_t row = (static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  float acc = 0.f;
  for (int c = lane * 2; c < dv; c += 64) {
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(dO + row * dv + c);
    const __nv_bfloat162 bb = *reinterpret_cast<const __nv_bfloat162*>(o + row * dv + c);
    acc = fmaf(__bfloat162float(a.x), __bfloat162float(bb.x), acc);
    acc = fmaf(__bfloat162float(a.y), __bfloat162float(bb.y), acc);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
  if (lane == 0) delta[row] = acc;
}

// Consistent dO (paper Section 3.3): the saved-output shortcut with dO replaced by the FP8 operand
// the backward matmuls consume, D_i = sum_c dO^_ic O_ic with dO^ = code * 2^(byte - 127) from the
// row-blocked copy.  One warp per row, four codes per lane and step.
__global__ void consistent_delta_kernel(const uint8_t* __restrict__ dO_codes, const uint8_t* __restrict__ dO_scales,
                                        const __nv_bfloat16* __restrict__ o, float* __restrict__ delta, size_t rows,
                                        int N, int dv) {
  const size_t row = (static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const size_t slab = row / N;
  const int r = static_cast<int>(row % N);
  const int n_ct = (dv / 32 + 3) / 4;                 // 512-byte scale tiles per 128-row tile
  const uint8_t* sf = dO_scales + (slab * (N / 128) + r / 128) * n_ct * 512 + sf_tile_offset(r & 127, 0);
  float acc = 0.f;
  for (int c = lane * 4; c < dv; c += 128) {
    const uint32_t codes = *reinterpret_cast<const uint32_t*>(dO_codes + row * dv + c);
    const int blk = c >> 5;
    const float sc = __uint_as_float(static_cast<uint32_t>(sf[(blk >> 2) * 512 + (blk & 3)]) << 23);   // 2^(byte-127); 0 for byte 0
    const uint2 ov = *reinterpret_cast<const uint2*>(o + row * dv + c);
    const __nv_bfloat162 o01 = *reinterpret_cast<const __nv_bfloat162*>(&ov.x);
    const __nv_bfloat162 o23 = *reinterpret_cast<const __nv_bfloat162*>(&ov.y);
    uint32_t h01, h23;                                 // E4M3 -> FP16 is exact
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h01) : "h"(static_cast<uint16_t>(codes & 0xFFFF)));
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h23) : "h"(static_cast<uint16_t>(codes >> 16)));
    const float2 d01 = __half22float2(*reinterpret_cast<const __half2*>(&h01));
    const float2 d23 = __half22float2(*reinterpret_cast<const __half2*>(&h23));
    float part = d01.x * __bfloat162float(o01.x);
    part = fmaf(d01.y, __bfloat162float(o01.y), part);
    part = fmaf(d23.x, __bfloat162float(o23.x), part);
    part = fmaf(d23.y, __bfloat162float(o23.y), part);
    acc = fmaf(part, sc, acc);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
  if (lane == 0) delta[row] = acc;
}

}  // namespace

attn_status_t launch_consistent_delta(const AttnShape& s, attn_qtensor_t dO, const void* o_bf16, float* delta,
                                      cudaStream_t stream) {
  const size_t rows = static_cast<size_t>(s.B) * s.Hq * s.N;
  const int threads = 256;
  const size_t blocks = (rows * 32 + threads - 1) / threads;
  consistent_delta_kernel<<<static_cast<unsigned>(blocks), threads, 0, stream>>>(
      dO.row_codes, dO.row_scales, static_cast<const __nv_bfloat16*>(o_bf16), delta, rows, s.N, s.dv);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "consistent delta: launch: %s", cudaGetErrorString(e));
  return ATTN_OK;
}

attn_status_t launch_bwd_delta(const AttnShape& s, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v,
                               attn_qtensor_t dO, const float* lse, float* delta, int* status, cudaStream_t stream) {
  return launch_qmajor<false>(s, q, k, v, dO, lse, nullptr, delta, nullptr, nullptr, nullptr, nullptr, nullptr, status, stream);
}

attn_status_t launch_bwd_dq(const AttnShape& s, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v, attn_qtensor_t dO,
                            const float* lse, const float* delta, void* dq, float* rowsum, float* rowabs,
                            float* post_rowsum, float* post_rowabs, int* status, cudaStream_t stream, bool behind_dkdv,
                            float* p_abs_dp) {
  return launch_qmajor<true>(s, q, k, v, dO, lse, delta, nullptr, dq, rowsum, rowabs, post_rowsum, post_rowabs, status, stream,
                             behind_dkdv, p_abs_dp);
}

attn_status_t launch_stale_delta(const AttnShape& s, const void* dO_bf16, const void* o_bf16, float* delta,
                                 cudaStream_t stream) {
  const size_t rows = static_cast<size_t>(s.B) * s.Hq * s.N;
  const int threads = 256;
  const size_t blocks = (rows * 32 + threads - 1) / threads;
  stale_delta_kernel<<<static_cast<unsigned>(blocks), threads, 0, stream>>>(
      static_cast<const __nv_bfloat16*>(dO_bf16), static_cast<const __nv_bfloat16*>(o_bf16), delta, rows, s.dv);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "stale delta: launch: %s", cudaGetErrorString(e));
  return ATTN_OK;
}

}  // namespace attnfp8
