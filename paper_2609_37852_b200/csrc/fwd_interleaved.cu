// Forward attention with block-scaled FP8 operands for v head dims up to 128 and qk head dims up to 192 (paper Appendix
// "Forward Probability Encoding", re-designed for tcgen05 / tensor memory): the variant in which a
// softmax thread owns a whole query row of a key step, the key steps of a query tile are dealt
// round-robin to the softmax warpgroups, and a separate warpgroup keeps the output accumulator's
// power-of-two unit.
//
// One CTA per SM owns 128 query rows of one (batch, query head) and walks the key tiles up to the
// causal diagonal.  Score tiles of kWG consecutive key steps live in tensor memory at once, one per
// softmax warpgroup, so the tensor cores compute S of step u+1 while the exponentials of step u run:
//   warp 0        TMA producer: Q tile once, then K tiles [128 keys x d] and V^T tiles [dv x 128 keys]
//   warp 1        issues S_u = Q K_u^T into score buffer u % kWG
//   warp 2        issues O += P^_u V_u (A operand = quantised probabilities read from tensor memory)
//   warps 4..7    unit keepers: thread <-> query row (see below); they also write O and LSE at the end
//   warpgroup w   (warps 8+4w .. 11+4w) softmax of the steps u = w, w + kWG, ...: thread <-> query row.
// A softmax thread keeps a PRIVATE integer shift M and normaliser share l for the steps it sees: the
// E4M3 codes of a block do not depend on the shift (the block scale absorbs any power of two), and l
// sums the exponentials before the cast.  It never waits for another softmax thread: it writes the
// codes to tensor memory, the scale bytes (relative to its M) and M itself to shared memory, and goes
// on.  What the steps of a row must agree on is only the power of two the output accumulator is
// expressed in, M_O.  The row's unit keeper holds it in a register and takes the steps in order: it
// adds M - M_O to the step's scale bytes (exact), hands the step to the P V issuer, and on the rare
// occasion that M exceeds M_O by more than kLazyUnit it first rescales the accumulator row in tensor
// memory between two P V products.
#include <cuda_bf16.h>

#include "common.cuh"
#include "mma_issue.cuh"
#include "mxfp8_device.cuh"
#include "sm100_ptx.cuh"

namespace attnfp8 {

namespace {

using namespace sm100;

constexpr int kTile = 128;          // query rows per CTA; keys per K / V tile in shared memory
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2Hi = 0.693359375f;             // ln 2 = kLn2Hi + kLn2Lo, kLn2Hi has 8 significant bits
constexpr float kLn2Lo = -2.12194440054690583e-4f;
constexpr int kLazyShift = 8;       // a thread raises its private shift when a step's maximum exceeds it by more
constexpr int kLazyUnit = 24;       // the accumulator's unit is raised when a step's shift exceeds it by more

__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

template <int kWG_, int kSW_, int kSplit_, int kCq_ = 1>
struct IlCfg {
  static constexpr int kCq = kCq_;                      // 128-byte chunks per Q / K row (2: qk head dim 192)
  // Ring depths (what shared memory holds).  A V stage is held from its copy until the P V product of its tile,
  // about two steps after the score product that frees the K stage of the same tile, so the V ring is the one
  // that needs the depth: at qk head dim 192, two K stages and four V stages (0.278 -> 0.224 ms on mla8k against
  // two and two, where every third step waited a step's time for V).
  static constexpr int kStages = kCq == 1 ? 4 : 2;      // K ring depth
  static constexpr int kVStages = 4;                    // V ring depth
  static constexpr int kWG = kWG_;                      // softmax teams == score buffers in flight
  static constexpr int kSW = kSW_;                      // keys per step (64 or 128)
  static constexpr int kSplit = kSplit_;                // threads per query row and step (each takes kSW / kSplit keys)
  static constexpr int kBlk = kSW / 32;                 // quantisation blocks per step
  static constexpr int kBlkT = kBlk / kSplit;           // ... per thread
  static constexpr int kColsT = kSW / kSplit;           // score columns per thread and step
  static constexpr int kSubPerTile = kTile / kSW;       // steps per K / V tile
  static constexpr int kSoftmaxThreads = 128 * kWG * kSplit;
  static constexpr int kThreads = 256 + kSoftmaxThreads;
  static constexpr int kPCols = kSW / 4;                // columns of one probability buffer
  static constexpr uint32_t kColS = 0;                  // kWG score buffers
  static constexpr uint32_t kColO = kWG * kSW;          // output accumulator, up to 128 columns
  static constexpr uint32_t kColP = kColO + 128;        // kWG probability buffers
  static constexpr uint32_t kColSFQ = kColP + kWG * kPCols;
  static constexpr uint32_t kColSFK = kColSFQ + 8 * kCq;   // 2 slots (Q: 2 slots), 4 columns per chunk
  static constexpr uint32_t kColSFV = kColSFK + 8 * kCq;   // 2 slots
  static constexpr uint32_t kColSFP = kColSFV + 8;      // kWG x 4
  static constexpr uint32_t kColsUsed = kColSFP + 4 * kWG;
  static_assert(kColsUsed <= 512, "tensor memory exceeded");
  // registers (the CTA's pool is what it was launched with: 65536 / kThreads per thread, rounded
  // down to a multiple of 8): the issuing warpgroup and the unit keepers give registers to the
  // softmax warpgroups
  static constexpr int kRegsIssue = 40;
  static constexpr int kRegsKeeper = kSplit == 1 ? 64 : 56;
  static constexpr int kRegsLaunch = (65536 / kThreads) / 8 * 8;
  static constexpr int kRegsSoftmax = ((kRegsLaunch * kThreads - 128 * (kRegsIssue + kRegsKeeper)) / kSoftmaxThreads) / 8 * 8;
};

template <class C>
struct IlSmem {
  static constexpr int kStages = C::kStages;
  alignas(1024) uint8_t q[2][C::kCq][kTile * 128];
  alignas(1024) uint8_t k[kStages][C::kCq][kTile * 128];
  alignas(1024) uint8_t v[C::kVStages][kTile * 128];
  alignas(16) uint8_t sf_q[2][C::kCq * 512];
  alignas(16) uint8_t sf_k[kStages][C::kCq * 512];
  alignas(16) uint8_t sf_v[C::kVStages][512];
  alignas(16) uint8_t sf_p[C::kWG][512];
  alignas(16) uint32_t raw_sf[C::kWG][C::kSplit][kTile];    // scale bytes of a step relative to the softmax thread's shift
  alignas(16) float step_m[C::kWG][C::kSplit][kTile];       // that shift
  alignas(16) float fin_l[4][C::kWG * C::kSplit][kTile];    // normaliser shares at the end of an item (four slots, by item
  alignas(16) float fin_m[4][C::kWG * C::kSplit][kTile];    // number), and the shifts they are expressed in
  uint64_t q_full[2], q_empty[2];
  uint64_t k_full[kStages], k_empty[kStages];
  uint64_t v_full[C::kVStages], v_empty[C::kVStages];
  uint64_t s_full[C::kWG], s_free[C::kWG];
  uint64_t p_ready[C::kWG], p_full[C::kWG], p_free[C::kWG];
  uint64_t o_done, o_free;
  uint64_t drain[2];
  uint32_t tmem_base;
  int abort_flag;
};

struct IlParams {
  const uint8_t* q_sf;      // row scales of Q
  const uint8_t* k_sf;      // row scales of K
  const uint8_t* v_sf;      // col scales of V
  __nv_bfloat16* o;
  float* lse;
  int* status;
  int N, Nk, q0t, Hq, Hkv, dqk, dv, causal;   // N query rows, Nk keys, q0t: tile offset of the causal diagonal
  int kv_lim;               // without the causal mask: last real key of the last key tile (127: all real)
  int gx, gy, gz;           // the (head, query tile, batch) grid the work items are numbered in
  float scale_log2;         // softmax_scale * log2(e)
};

// 2^d for an integer-valued d <= 127 (0 below the normal range, -inf included)
__device__ __forceinline__ float pow2_int(float d) {
  const int e = d < -126.f ? 0 : 127 + static_cast<int>(d);
  return __uint_as_float(static_cast<uint32_t>(e) << 23);
}

template <class C>
__global__ void __launch_bounds__(C::kThreads, 1)
fwd_il_kernel(const IlParams p, const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
              const __grid_constant__ CUtensorMap tm_v) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  IlSmem<C>& sm = *reinterpret_cast<IlSmem<C>*>(smem_raw);
  if (smem_u32(smem_raw) & 1023u) {               // never expected: report instead of computing garbage
    if (threadIdx.x == 0) atomicExch(p.status, static_cast<int>(ATTN_ERR_ALIGNMENT));
    return;
  }
  constexpr int kWG = C::kWG, kSW = C::kSW, kBlk = C::kBlk, kSubPerTile = C::kSubPerTile, kPCols = C::kPCols;
  constexpr int kSplit = C::kSplit, kBlkT = C::kBlkT, kColsT = C::kColsT;
  constexpr uint32_t kColS = C::kColS, kColO = C::kColO, kColP = C::kColP, kColSFQ = C::kColSFQ, kColSFK = C::kColSFK,
                     kColSFV = C::kColSFV, kColSFP = C::kColSFP;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // Work items (128 query rows of one head) are numbered x-fastest over (head, query tile, batch):
  // heads vary fastest and the heaviest (latest) query tiles of all heads come first.  CTA c of n
  // takes the items c, 2n-1-c, 2n+c, ...: alternate rounds run backwards, so that no CTA collects the
  // heavier item of every round.  The K / V rings, the score and probability buffers and their
  // barriers run on across items; Q is double-buffered; the output accumulator is handed from the
  // unit keepers (who store the finished item) back to the P V issuer once per item.
  const int n_cta = static_cast<int>(gridDim.x), cta = static_cast<int>(blockIdx.x);
  const int total_items = p.gx * p.gy * p.gz;
  struct Item { int qt, h, b, g, n_tiles, n_steps; bool valid; };
  auto item_at = [&](int i) {
    Item it;
    const int l = i * n_cta + ((i & 1) ? n_cta - 1 - cta : cta);
    it.valid = l < total_items;
    const int x = l % p.gx, y = (l / p.gx) % p.gy, z = l / (p.gx * p.gy);
    it.qt = p.causal ? (p.gy - 1 - y) : y;
    it.h = x; it.b = z;
    it.g = it.h / (p.Hq / p.Hkv);
    it.n_tiles = p.causal ? it.qt + p.q0t + 1 : p.Nk / kTile;
    it.n_steps = it.n_tiles * kSubPerTile;
    return it;
  };
  constexpr int kStages = C::kStages, kVStages = C::kVStages, kCq = C::kCq;
  const int nk_qk = p.dqk / 32;                 // 32-byte K steps of the score MMA
  volatile int* abort_flag = &sm.abort_flag;

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) { mbar_init(&sm.q_full[i], 1); mbar_init(&sm.q_empty[i], 1); }
    for (int s = 0; s < kStages; ++s) { mbar_init(&sm.k_full[s], 1); mbar_init(&sm.k_empty[s], 1); }
    for (int s = 0; s < kVStages; ++s) { mbar_init(&sm.v_full[s], 1); mbar_init(&sm.v_empty[s], 1); }
    for (int w = 0; w < kWG; ++w) {
      // every thread arrives for itself (one elected arrival per warp behind a warp barrier measured slower)
      mbar_init(&sm.s_full[w], 1); mbar_init(&sm.s_free[w], 128 * kSplit);
      mbar_init(&sm.p_ready[w], 128 * kSplit); mbar_init(&sm.p_full[w], 128); mbar_init(&sm.p_free[w], 1);
    }
    mbar_init(&sm.o_done, 1);
    mbar_init(&sm.o_free, 4);
    mbar_init(&sm.drain[0], 1); mbar_init(&sm.drain[1], 1);
    sm.abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&sm.tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sm.tmem_base;

  if (warp < 4) {
    reg_dealloc<C::kRegsIssue>();
    if (warp == 0) {
      // ------------------------------------------------------------------ producer
      if (lane == 0) {
        prefetch_tmap(&tm_q); prefetch_tmap(&tm_k); prefetch_tmap(&tm_v);
        const int tiles_n = p.N / kTile, tiles_nk = p.Nk / kTile;
        int issued_k = 0, issued_v = 0;
        int T = 0;                                    // key tiles of the items before this one
        bool ok = true;
        for (int i = 0; ok; ++i) {
          const Item it = item_at(i);
          if (!it.valid) break;
          const int qb = i & 1;
          if (i >= 2) {
            // the S issuer has finished with the item that used this Q buffer
            ok = mbar_wait(&sm.q_empty[qb], ((i >> 1) - 1) & 1, abort_flag);
            if (!ok) break;
          }
          const int q_slab = it.b * p.Hq + it.h, kv_slab = it.b * p.Hkv + it.g;
          mbar_arrive_expect_tx(&sm.q_full[qb], kCq * (kTile * 128 + 512));
          for (int c = 0; c < kCq; ++c) tma_load_2d(sm.q[qb][c], &tm_q, &sm.q_full[qb], 128 * c, q_slab * p.N + it.qt * kTile);
          bulk_load_1d(sm.sf_q[qb], p.q_sf + (static_cast<size_t>(q_slab) * tiles_n + it.qt) * kCq * 512, kCq * 512,
                       &sm.q_full[qb]);
          for (int t = 0; t < it.n_tiles && ok; ++t) {
            const int gt = T + t, s = gt % kStages, r = gt / kStages;
            ok = mbar_wait(&sm.k_empty[s], (r & 1) ^ 1, abort_flag);
            if (!ok) break;
            mbar_arrive_expect_tx(&sm.k_full[s], kCq * (kTile * 128 + 512));
            for (int c = 0; c < kCq; ++c) tma_load_2d(sm.k[s][c], &tm_k, &sm.k_full[s], 128 * c, kv_slab * p.Nk + t * kTile);
            bulk_load_1d(sm.sf_k[s], p.k_sf + (static_cast<size_t>(kv_slab) * tiles_nk + t) * kCq * 512, kCq * 512,
                         &sm.k_full[s]);
            ++issued_k;
            const int sv = gt % kVStages, rv = gt / kVStages;
            ok = mbar_wait(&sm.v_empty[sv], (rv & 1) ^ 1, abort_flag);
            if (!ok) break;
            mbar_arrive_expect_tx(&sm.v_full[sv], p.dv * 128 + 512);
            tma_load_2d(sm.v[sv], &tm_v, &sm.v_full[sv], t * 128, kv_slab * p.dv);
            bulk_load_1d(sm.sf_v[sv], p.v_sf + (static_cast<size_t>(kv_slab) * tiles_nk + t) * 512, 512, &sm.v_full[sv]);
            ++issued_v;
          }
          T += it.n_tiles;
        }
        if (!ok) {
          // let the copies already in flight land before the CTA gives its shared memory back
          int dummy = 0;
          for (int t = max(0, issued_k - kStages); t < issued_k; ++t)
            mbar_wait(&sm.k_full[t % kStages], (t / kStages) & 1, &dummy);
          for (int t = max(0, issued_v - kVStages); t < issued_v; ++t)
            mbar_wait(&sm.v_full[t % kVStages], (t / kVStages) & 1, &dummy);
        }
      }
    } else if (warp == 1) {
      // ------------------------------------------------------------------ S = Q K^T issuer
      bool ok = true;
      int T = 0, G = 0;                               // key tiles and key steps of the items before this one
      for (int i = 0; ok; ++i) {
        const Item it = item_at(i);
        if (!it.valid) break;
        const int qb = i & 1;
        const uint64_t desc_q = make_desc_sw128(smem_u32(sm.q[qb][0]));
        ok = mbar_wait(&sm.q_full[qb], (i >> 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after_sync();
        sf_copy_tiles<kCq>(tmem + kColSFQ + 4 * kCq * qb, sm.sf_q[qb]);
        for (int u = 0; u < it.n_steps && ok; ++u) {
          const int gu = G + u, gt = T + u / kSubPerTile;
          const int sub = u % kSubPerTile, s = gt % kStages, slot = gt & 1, w = gu % kWG;
          if (sub == 0) {
            ok = mbar_wait(&sm.k_full[s], (gt / kStages) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after_sync();
            sf_copy_tiles<kCq>(tmem + kColSFK + 4 * kCq * slot, sm.sf_k[s]);
          }
          if (gu >= kWG) {
            // team w has pulled the scores of its previous step into registers
            ok = mbar_wait(&sm.s_free[w], ((gu / kWG) - 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after_sync();
          }
          const uint64_t desc_k = make_desc_sw128(smem_u32(sm.k[s][0])) + sub * (kSW * 128 / 16);
          issue_ss<true, kCq, kSW, kTile * 128 / 16, kTile * 128 / 16>(tmem + kColS + kSW * w, desc_q, desc_k, nk_qk,
                                                                        tmem + kColSFQ + 4 * kCq * qb,
                                                                        tmem + kColSFK + 4 * kCq * slot + kBlk * sub);
          mma_commit_elect(&sm.s_full[w]);
          if (sub == kSubPerTile - 1) mma_commit_elect(&sm.k_empty[s]);
        }
        if (ok) mma_commit_elect(&sm.q_empty[qb]);       // this item's Q tile has been read
        T += it.n_tiles; G += it.n_steps;
      }
      if (*abort_flag) ok = false;
      if (!ok) {
        int dummy = 0;
        mma_commit_elect(&sm.drain[0]);
        mbar_wait(&sm.drain[0], 0, &dummy);
      }
    } else if (warp == 2) {
      // ------------------------------------------------------------------ O += P V issuer
      bool ok = true;
      const uint32_t n_dv = static_cast<uint32_t>(p.dv);
      int T = 0, G = 0;
      for (int i = 0; ok; ++i) {
        const Item it = item_at(i);
        if (!it.valid) break;
        for (int u = 0; u < it.n_steps && ok; ++u) {
          const int gu = G + u, gt = T + u / kSubPerTile;
          const int sub = u % kSubPerTile, s = gt % kVStages, slot = gt & 1, w = gu % kWG;
          if (sub == 0) {
            ok = mbar_wait(&sm.v_full[s], (gt / kVStages) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after_sync();
            sf_copy_tiles<1>(tmem + kColSFV + 4 * slot, sm.sf_v[s]);
          }
          ok = mbar_wait(&sm.p_full[w], (gu / kWG) & 1, abort_flag);
          if (!ok) break;
          if (u == 0 && i > 0) {
            // the unit keepers have read the previous item out of the accumulator
            ok = mbar_wait(&sm.o_free, (i - 1) & 1, abort_flag);
            if (!ok) break;
          }
          tc_fence_after_sync();
          sf_copy_elect(tmem + kColSFP + 4 * w, make_desc_sf(smem_u32(sm.sf_p[w])));
          const uint64_t desc_v = make_desc_sw128(smem_u32(sm.v[s]));
#pragma unroll
          for (int kb = 0; kb < kBlk; ++kb) {
            const int kstep = sub * kBlk + kb;              // 32-key block inside the 128-key tile
            mma_mxf8_ts_elect(tmem + kColO, tmem + kColP + kPCols * w + 8 * kb, desc_v + 2 * kstep,
                              make_idesc_mxf8(128, n_dv, kb, kstep), tmem + kColSFP + 4 * w, tmem + kColSFV + 4 * slot,
                              (u > 0 || kb > 0));
          }
          mma_commit_elect(&sm.p_free[w]);                  // operand and scale bytes of this buffer consumed; O updated
          if (sub == kSubPerTile - 1) mma_commit_elect(&sm.v_empty[s]);
          if (u == it.n_steps - 1) mma_commit_elect(&sm.o_done);
        }
        T += it.n_tiles; G += it.n_steps;
      }
      if (*abort_flag) ok = false;
      if (!ok) {
        int dummy = 0;
        mma_commit_elect(&sm.drain[1]);
        mbar_wait(&sm.drain[1], 0, &dummy);
      }
    }
  } else if (warp < 8) {
    // -------------------------------------------------------------------- unit keepers
    reg_dealloc<C::kRegsKeeper>();
    const int quad = warp & 3;
    const int row = quad * 32 + lane;                   // row inside the tile == TMEM lane
    const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
    bool ok = true;
    int G = 0;
    for (int i = 0; ok; ++i) {
      const Item it = item_at(i);
      if (!it.valid) break;
      float MO = -INFINITY;                             // the accumulator row is expressed in units of 2^MO
      for (int u = 0; u < it.n_steps; ++u) {
        const int gu = G + u, w = gu % kWG, use = gu / kWG;
        ok = mbar_wait(&sm.p_ready[w], use & 1, abort_flag);
        if (!ok) break;
        float Mh[kSplit];                               // -inf: the thread has seen nothing but masked keys
        uint32_t raw[kSplit];
#pragma unroll
        for (int hf = 0; hf < kSplit; ++hf) {
          Mh[hf] = lds_f32(&sm.step_m[w][hf][row]);
          asm volatile("ld.shared.b32 %0, [%1];" : "=r"(raw[hf]) : "r"(smem_u32(&sm.raw_sf[w][hf][row])));
        }
        float M = Mh[0];
#pragma unroll
        for (int hf = 1; hf < kSplit; ++hf) M = fmaxf(M, Mh[hf]);
        const bool raise = M > MO + static_cast<float>(kLazyUnit);       // always on the item's first step
        if (__any_sync(0xffffffffu, raise)) {
          if (u > 0) {
            // rare: the previous P V product must have landed before the accumulator row is rescaled
            ok = mbar_wait(&sm.p_free[(gu - 1) % kWG], ((gu - 1) / kWG) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after_sync();
            const float factor = raise ? pow2_int(MO - M) : 1.f;
            for (int c0 = 0; c0 < p.dv; c0 += 16) {
              uint32_t r[16];
              tmem_ld16(tmem + kColO + lane_addr + c0, r);
              tmem_wait_ld();
#pragma unroll
              for (int c = 0; c < 16; ++c) r[c] = __float_as_uint(__uint_as_float(r[c]) * factor);
              tmem_st16(tmem + kColO + lane_addr + c0, r);
            }
            tmem_wait_st();
            tc_fence_before_sync();
          }
          if (raise) MO = M;
        }
        // scale bytes relative to the accumulator's unit; a block more than 2^-127 below it keeps byte 0
        uint32_t packed = 0;
#pragma unroll
        for (int hf = 0; hf < kSplit; ++hf) {
          const int shift = Mh[hf] == -INFINITY ? 0 : static_cast<int>(fmaxf(Mh[hf] - MO, -1024.f));
#pragma unroll
          for (int bk = 0; bk < kBlkT; ++bk) {
            const int byte = static_cast<int>((raw[hf] >> (8 * bk)) & 0xFFu);
            const int bnew = byte == 0 ? 0 : max(byte + shift, 0);
            packed |= static_cast<uint32_t>(bnew) << (8 * (hf * kBlkT + bk));
          }
        }
        uint8_t* sf_dst = &sm.sf_p[w][(row & 31) * 16 + (row >> 5) * 4];
        if (kBlk == 4)
          asm volatile("st.shared.b32 [%0], %1;" ::"r"(smem_u32(sf_dst)), "r"(packed) : "memory");
        else
          asm volatile("st.shared.b16 [%0], %1;" ::"r"(smem_u32(sf_dst)), "h"(static_cast<uint16_t>(packed)) : "memory");
        fence_proxy_async_smem();
        mbar_arrive(&sm.p_full[w]);
      }
      // The row's normaliser = sum of the shares of its softmax threads, in the accumulator's unit.  A
      // team wrote its shares ahead of the arrival that announced its last step of the item (a team
      // without a step in a one-step item wrote nothing).
      if (ok) ok = mbar_wait(&sm.o_done, i & 1, abort_flag);
      if (!ok) break;
      tc_fence_after_sync();
      float lt = 0.f;
#pragma unroll
      for (int j = 0; j < kWG * kSplit; ++j) {
        const int first_u = (j / kSplit + kWG - G % kWG) % kWG;     // the team's first step of this item
        if (first_u < it.n_steps)
          lt += lds_f32(&sm.fin_l[i & 3][j][row]) * pow2_int(lds_f32(&sm.fin_m[i & 3][j][row]) - MO);   // M = -inf goes with l = 0
      }
      const float inv_l = 1.f / lt;
      const size_t grow = static_cast<size_t>(it.b * p.Hq + it.h) * p.N + it.qt * kTile + row;
      __nv_bfloat16* o_row = p.o + grow * p.dv;
      for (int c0 = 0; c0 < p.dv; c0 += 16) {
        uint32_t r[16];
        tmem_ld16(tmem + kColO + lane_addr + c0, r);
        tmem_wait_ld();
        uint32_t packed[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          __nv_bfloat162 v2 = __floats2bfloat162_rn(__uint_as_float(r[2 * c]) * inv_l, __uint_as_float(r[2 * c + 1]) * inv_l);
          packed[c] = *reinterpret_cast<uint32_t*>(&v2);
        }
        uint4* dst = reinterpret_cast<uint4*>(o_row + c0);
        dst[0] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
        dst[1] = make_uint4(packed[4], packed[5], packed[6], packed[7]);
      }
      // the accumulator may be overwritten by the next item's first P V product
      tc_fence_before_sync();
      mbar_arrive_warp(&sm.o_free);
      // LSE = M_O ln2 + ln l with ln2 split so that M_O * ln2_hi is exact: one rounding at the end
      p.lse[grow] = fmaf(MO, kLn2Hi, fmaf(MO, kLn2Lo, logf(lt)));
      G += it.n_steps;
    }
  } else {
    // -------------------------------------------------------------------- softmax
    reg_alloc<C::kRegsSoftmax>();
    const int w = (warp - 8) / (4 * kSplit);            // team: takes the steps whose running number is w modulo kWG
    const int hf = ((warp - 8) >> 2) % kSplit;          // which kColsT keys of a step
    const int quad = warp & 3;
    const int row = quad * 32 + lane;                   // row inside the tile == TMEM lane
    const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
    bool ok = true;
    int G = 0;
    for (int i = 0; ok; ++i) {
      const Item it = item_at(i);
      if (!it.valid) break;
      const int qt = it.qt;
      float M = -INFINITY;                              // private integer-valued shift (log2 units)
      float l = 0.f;                                    // this thread's share of the normaliser, in units of 2^M
      for (int u = (w + kWG - G % kWG) % kWG; u < it.n_steps; u += kWG) {
        const int gu = G + u, t = u / kSubPerTile, sub = u % kSubPerTile, use = gu / kWG;
        ok = mbar_wait(&sm.s_full[w], use & 1, abort_flag);
        if (!ok) break;
        tc_fence_after_sync();
        float sv[kColsT];
#pragma unroll
        for (int bk = 0; bk < kBlkT; ++bk)
          tmem_ld32(tmem + kColS + kSW * w + kColsT * hf + lane_addr + 32 * bk, reinterpret_cast<uint32_t*>(sv + 32 * bk));
        tmem_wait_ld();
        tc_fence_before_sync();
        mbar_arrive(&sm.s_free[w]);                // the scores are in registers: the next S of this buffer may be issued
        // maxima of the raw accumulators per block (the scale is positive), masked on the diagonal tile
        float mxb[kBlkT];
        // masked tiles: the diagonal one under the causal mask (keys after the query), else the last one
        // when the sequence ends inside it (keys after the last real key)
        if (p.causal ? t == qt + p.q0t : (p.kv_lim < kTile - 1 && t == it.n_tiles - 1)) {
          const int lim = p.causal ? row : p.kv_lim;
#pragma unroll
          for (int bk = 0; bk < kBlkT; ++bk) {
            const int col0 = sub * kSW + kColsT * hf + 32 * bk;
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
          for (int bk = 0; bk < kBlkT; ++bk) {
            // 16 three-input maxima as a tree of depth 4
            const float* x = sv + 32 * bk;
            float a[10];
#pragma unroll
            for (int j = 0; j < 10; ++j) a[j] = max3(x[3 * j], x[3 * j + 1], x[3 * j + 2]);
            const float b0 = max3(a[0], a[1], a[2]), b1 = max3(a[3], a[4], a[5]), b2 = max3(a[6], a[7], a[8]);
            const float b3 = max3(a[9], x[30], x[31]);
            mxb[bk] = fmaxf(max3(b0, b1, b2), b3);
          }
        }
        float mx = mxb[0];
#pragma unroll
        for (int bk = 1; bk < kBlkT; ++bk) mx = fmaxf(mx, mxb[bk]);
        // a fully masked step (second half of the diagonal tile for the first 64 rows) gives -inf: it
        // never raises M and contributes zeros
        const float mx2 = mx * p.scale_log2;
        if (mx2 > M + static_cast<float>(kLazyShift)) {   // true on the thread's first unmasked step of the item
          const float m_new = ceilf(mx2);
          l *= pow2_int(M - m_new);                       // exact power of two (0 at the start)
          M = m_new;
        }
        const float neg_m = M == -INFINITY ? 0.f : -M;    // nothing seen yet: every score is -inf, any finite shift gives zeros
        uint32_t bytes[kBlkT];
        // The scale 2^e of a block follows from its largest exponential, which is the exponential of
        // the block's score maximum; folding e into the shift makes ex2 deliver p * 2^-e, the value
        // the E4M3 cast wants, and the block sum is put back on the thread's scale by one exact
        // multiplication.
        float2 nme2[kBlkT];
#pragma unroll
        for (int bk = 0; bk < kBlkT; ++bk) {
          float inv;
          block_scale_finite(ex2_approx(fmaf(mxb[bk], p.scale_log2, neg_m)), bytes[bk], inv);
          const float neg_me = neg_m - static_cast<float>(static_cast<int>(bytes[bk]) - 127);
          nme2[bk] = make_float2(neg_me, neg_me);
        }
        uint32_t packed_sf = 0;
#pragma unroll
        for (int bk = 0; bk < kBlkT; ++bk) packed_sf |= bytes[bk] << (8 * bk);
        // Groups of four keys, the exponentials of group i written kLag groups ahead of the sums and
        // casts that consume them.  The codes of a block go to tensor memory as soon as it is complete.
        {
          constexpr int kGroups = kColsT / 4, kLag = 3;
          const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
          float2 e01[kGroups], e23[kGroups];
          float2 bs01[kBlkT], bs23[kBlkT];
          uint32_t words[kBlkT][8];
#pragma unroll
          for (int bk = 0; bk < kBlkT; ++bk) bs01[bk] = bs23[bk] = make_float2(0.f, 0.f);
#pragma unroll
          for (int j0 = 0; j0 < kGroups + kLag; ++j0) {
            if (j0 < kGroups) {
              const float2 a = __ffma2_rn(make_float2(sv[4 * j0], sv[4 * j0 + 1]), sc2, nme2[j0 / 8]);
              const float2 c = __ffma2_rn(make_float2(sv[4 * j0 + 2], sv[4 * j0 + 3]), sc2, nme2[j0 / 8]);
              e01[j0] = make_float2(ex2_approx(a.x), ex2_approx(a.y));
              e23[j0] = make_float2(ex2_approx(c.x), ex2_approx(c.y));
            }
            if (j0 >= kLag) {
              const int j = j0 - kLag;
              bs01[j / 8] = __fadd2_rn(bs01[j / 8], e01[j]);
              bs23[j / 8] = __fadd2_rn(bs23[j / 8], e23[j]);
              words[j / 8][j % 8] = cvt_e4m3x4(e01[j].x, e01[j].y, e23[j].x, e23[j].y);
              if (j == 7) {
                // The first block is done.  Before anything of this step is stored: the P V MMAs of
                // the team's previous step have consumed its operand buffer (and the unit keepers its
                // scale bytes and shift before that); that product was issued when the previous step
                // ended, so the wait is over by now as a rule.
                if (gu >= kWG) {
                  ok = mbar_wait(&sm.p_free[w], (use - 1) & 1, abort_flag);
                  if (!ok) break;
                  tc_fence_after_sync();
                }
                asm volatile("st.shared.b32 [%0], %1;" ::"r"(smem_u32(&sm.raw_sf[w][hf][row])), "r"(packed_sf) : "memory");
                sts_f32(&sm.step_m[w][hf][row], M);
              }
              if (j % 8 == 7) tmem_st8(tmem + kColP + kPCols * w + lane_addr + 8 * (hf * kBlkT + j / 8), words[j / 8]);
            }
          }
          if (!ok) break;
#pragma unroll
          for (int bk = 0; bk < kBlkT; ++bk) {
            const float bs0 = bs01[bk].x + bs01[bk].y, bs1 = bs23[bk].x + bs23[bk].y;
            l = fmaf(bs0 + bs1, __uint_as_float(bytes[bk] << 23), l);   // 2^e (0 for an all-masked block, whose sum is 0)
          }
        }
        if (u + kWG >= it.n_steps) {
          // the team's last step of the item: its normaliser shares go with this arrival (the slot was
          // last read four items ago)
          sts_f32(&sm.fin_l[i & 3][w * kSplit + hf][row], l);
          sts_f32(&sm.fin_m[i & 3][w * kSplit + hf][row], M);
        }
        tmem_wait_st();
        tc_fence_before_sync();
        mbar_arrive(&sm.p_ready[w]);               // codes in tensor memory, scale bytes and shift in shared memory
      }
      if (!ok) break;
      G += it.n_steps;
    }
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
  if (tid == 0 && sm.abort_flag) atomicExch(p.status, static_cast<int>(ATTN_ERR_TIMEOUT));
}

template <class C>
attn_status_t launch_fwd_il_t(const AttnShape& s, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v, void* o, float* lse,
                              int* status, cudaStream_t stream) {
  CUtensorMap tm_q, tm_k, tm_v;
  attn_status_t st;
  st = encode_tmap_u8_sw128(&tm_q, q.row_codes, static_cast<uint64_t>(s.dqk), static_cast<uint64_t>(s.B) * s.Hq * s.N, kTile);
  if (st != ATTN_OK) return st;
  st = encode_tmap_u8_sw128(&tm_k, k.row_codes, static_cast<uint64_t>(s.dqk), static_cast<uint64_t>(s.B) * s.Hkv * s.Nk, kTile);
  if (st != ATTN_OK) return st;
  st = encode_tmap_u8_sw128(&tm_v, v.col_codes, static_cast<uint64_t>(s.Nk), static_cast<uint64_t>(s.B) * s.Hkv * s.dv, s.dv);
  if (st != ATTN_OK) return st;
  IlParams p;
  p.q_sf = q.row_scales; p.k_sf = k.row_scales; p.v_sf = v.col_scales;
  p.o = static_cast<__nv_bfloat16*>(o); p.lse = lse; p.status = status;
  p.N = s.N; p.Nk = s.Nk; p.q0t = s.q0t; p.kv_lim = s.kv_lim; p.Hq = s.Hq; p.Hkv = s.Hkv; p.dqk = s.dqk; p.dv = s.dv; p.causal = s.causal;
  p.scale_log2 = s.scale * kLog2e;
  const size_t smem = sizeof(IlSmem<C>) + 1024;
  cudaError_t e = cudaFuncSetAttribute(fwd_il_kernel<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "fwd: cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  p.gx = s.Hq; p.gy = s.N / kTile; p.gz = s.B;
  const long long items = static_cast<long long>(p.gx) * p.gy * p.gz;
  if (items > 0x7fffffffLL) return fail(ATTN_ERR_UNSUPPORTED, "fwd: %lld work items exceed 2^31 - 1", items);
  // one CTA per SM (the kernel takes all of an SM's tensor memory) walks the item list
  int dev = 0, sms = 0;
  e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess || sms < 1) return fail(ATTN_ERR_CUDA, "fwd: SM count: %s", cudaGetErrorString(e));
  dim3 grid(static_cast<unsigned>(items < sms ? items : sms), 1, 1);
  fwd_il_kernel<C><<<grid, C::kThreads, smem, stream>>>(p, tm_q, tm_k, tm_v);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(ATTN_ERR_CUDA, "fwd: launch: %s", cudaGetErrorString(e));
  return ATTN_OK;
}

}  // namespace

// FP8 operands, head dims (64,64) and (128,128): two teams, 128-key steps, two threads per row and step.
attn_status_t launch_fwd_interleaved(const AttnShape& s, attn_qtensor_t q, attn_qtensor_t k, attn_qtensor_t v, void* o,
                                     float* lse, int* status, cudaStream_t stream) {
  if (s.dqk > 128) return launch_fwd_il_t<IlCfg<2, 128, 2, 2>>(s, q, k, v, o, lse, status, stream);
  return launch_fwd_il_t<IlCfg<2, 128, 2>>(s, q, k, v, o, lse, status, stream);
}

}  // namespace attnfp8
