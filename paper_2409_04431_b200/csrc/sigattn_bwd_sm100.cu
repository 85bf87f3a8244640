// bf16 backward of sigmoid attention for sm_100a (Algorithm 2 of Appendix F.1, redesigned
// for Blackwell).  Per (batch*head, 128-key tile j) work item, looping over query tiles i:
//
//     S^T  = K_j Q_i^T                      (tensor memory region A, fp32)
//     P^T  = sigmoid(scale S^T + b ...)     (registers -> bf16 over region A)
//     dV_j += P^T dO_i                      (A operand from tensor memory)
//     dP^T = V_j dO_i^T                     (region B)
//     dS^T = P^T (1 - P^T) dP^T             (registers -> bf16, over region B and in shared memory)
//     dK_j += dS^T Q_i                      (A operand from tensor memory)
//     dQ_i  = dS K_j                        (region B again, then fp32 reduce-add to HBM)
//
// Everything is kept transposed (keys on the 128 TMEM lanes, queries along columns) so
// that P^T and dS^T can feed the dV and dK products straight from tensor memory; only dQ
// needs dS with queries as rows, and reads the shared-memory copy as an MN-major A operand.
// No row statistic of any kind is read or written: dS is a point-wise function of S and
// dP (Section 4 / Appendix F.1), and P is recomputed from Q and K alone.
//
// dK_j and dV_j stay in tensor memory across the whole query loop.  dQ_i is complete only
// after all key tiles have contributed, so each CTA adds its fp32 partial tile into a
// [B, H, N, D] fp32 workspace with TMA reduce-add; the workspace is zeroed before and
// converted to bf16 (times scale) after the main kernel: the two helper steps that
// survive from the paper's backward.  scale is also folded into dK's epilogue.
//
// Warp roles (448 threads): warps 0-7 two activation groups (query columns 0-63 and
// 64-127 of the tile; every thread owns one key row), warps 8-11 dQ drain group,
// warp 12 TMA producer, warp 13 MMA issuer.
#include <atomic>

#include "sigattn_internal.h"
#include "sigattn_activation.cuh"
#include "sm100_primitives.cuh"
#include "tensor_map.h"
#include "../../include/sigattn.h"

namespace sigattn {
namespace {

using namespace sm100;

constexpr int kT = 128;  // tile edge: keys per item (TMEM lanes) and queries per step
constexpr int kBwdThreads = 448;
constexpr int kBwdLoadWarp = 12;
constexpr int kBwdMmaWarp = 13;
constexpr float kLog2eB = 1.4426950408889634f;

template <int D>
struct BwdSmem {
  static constexpr int kPanels = D / 64;
  static constexpr int kPanelBytes = kT * 128;
  static constexpr int kTileBytes = kPanels * kPanelBytes;  // a K, V, Q or dO tile
  static constexpr int kKOff = 0;
  static constexpr int kVOff = kTileBytes;
  // Q stages: two at D = 128 (shared memory is full); three at D = 64, where S^T runs two steps ahead
  // (four, which would make stage and phase a mask and a shift, measured no faster)
  static constexpr int kQStages = (D == 64) ? 3 : 2;
  static constexpr int kQOff = 2 * kTileBytes;
  static constexpr int kDoOff = (2 + kQStages) * kTileBytes;   // one stage
  static constexpr int kDsOff = (3 + kQStages) * kTileBytes;   // dS^T, 128 x 128 bf16 = two panels
  static constexpr int kDqOff = kDsOff + 2 * kPanelBytes;   // two fp32 staging boxes of 128 x 32
  static constexpr int kTotal = kDqOff + 2 * kPanelBytes;
  static constexpr int kDynBytes = kTotal + 1024;
};

struct BwdBarriers {
  uint64_t kv_full, kv_empty;
  uint64_t q_full[3], q_empty[3];
  uint64_t do_full, do_empty;
  // s_full, p_ready, dq_full, dq_empty: one per region of tensor memory that holds S^T / P^T (see BwdTmem);
  // a region's barriers flip once per use of that region
  uint64_t s_full[2], dp_full;
  uint64_t p_ready[2], ds_ready;
  uint64_t dq_full[2], dq_empty[2];
  uint64_t dkv_full, dkv_empty;
  // dynamic schedule (batches without padding): the TMA thread draws the next work item from a
  // global counter and hands it to the other roles through this two-slot ring
  uint64_t sched_full[2], sched_empty[2];
  int sched_item[2];
};

struct BwdParams {
  int BH, H, N;    // BH counts (batch, key/value head) pairs: the work items are per key/value head
  int H_kv, group; // heads of K, V and query heads per key/value head (H = H_kv * group)
  int n_tiles;    // query tiles: ceil(N / 128), N = rows of Q
  int n_tiles_k;  // key tiles: ceil(rows of K / 128)
  int pos0;       // position of query row 0 relative to key row 0 (see FwdParams of the forward)
  const int* seqlens;   // padded batch: valid length per batch entry (keys and queries), or nullptr
  // batch stored without padding (B = 1): sequence s owns rows [cu_seqlens[s], cu_seqlens[s + 1]);
  // bias_vec and dbias then hold one entry per (sequence, head)
  const int* cu_seqlens;
  int n_seqs;
  int* sched_counter;   // dynamic schedule: next work item to hand out (zero at launch), or nullptr
  // Few (batch, key/value head) pairs (multi-query attention at a small batch): the query heads of a
  // group are split over n_sub work items of heads_per_sub heads each, which add their dK_j, dV_j
  // (bf16 TMA reduce-adds into the cleared outputs) instead of storing them.  n_sub = 1: off.
  int n_sub, heads_per_sub;
  // Few work items with one query head per key/value head (one long sequence, few heads): the query
  // tiles of a key tile are divided over two items (i_split = 2) that add their dK_j, dV_j likewise.
  int i_split;
  int dkv_add;   // 1: dK_j, dV_j are added (bf16 TMA reduce-adds) into outputs the caller cleared: several calls sum up
  int n_items;
  float scale, scale_log2e, bias_log2e;
  const float* bias_vec;   // one bias per (batch, head) instead of the scalar, or nullptr
  float* dbias;            // receives sum dS per (batch, head), or nullptr
  const float* slopes;
  int* status;
};

struct BwdItem {
  int bh;       // (batch, key/value head) index: K_j, V_j, dK_j, dV_j
  int bh_q0;    // first of the `group` query heads that read this key/value head
  int j, i_begin;
  int n;        // query tiles per query head
  int steps;    // group * n, visited head by head
  int n_valid;  // rows of this sequence that count (N unless the batch is padded)
};

// Ranks are ordered by decreasing cost; rounds alternate direction over the CTAs so that
// expensive and cheap items pair up (static stand-in for longest-first scheduling).
__device__ __forceinline__ int bwd_snake_rank(int round, int n_items) {
  const int g = gridDim.x;
  const int c = (round & 1) ? (g - 1 - static_cast<int>(blockIdx.x)) : static_cast<int>(blockIdx.x);
  const int rank = round * g + c;
  return rank < n_items ? rank : -1;
}

__device__ __forceinline__ int bwd_num_rounds(int n_items) { return (n_items + gridDim.x - 1) / gridDim.x; }

// Dynamic schedule for batches without padding, where an item's cost follows the position of its
// key tile inside its own sequence and the static order above no longer sorts by cost: the CTAs
// draw items from a global counter in key-tile order (every sequence hands out its expensive key
// tiles first).  One thread per CTA draws; the MMA thread, the activation groups and the drain
// group read the item from a two-slot ring.  false: a bounded wait expired; *item < 0: none left.
constexpr int kBwdSchedConsumers = 1 + 256 + 128;
__device__ __forceinline__ bool bwd_sched_draw(const BwdParams& p, BwdBarriers* bars, int round, int* item,
                                               volatile int* cta_err) {
  const uint32_t slot = round & 1, phase = (round >> 1) & 1;
  if (!mbar_wait(smem_u32(&bars->sched_empty[slot]), phase ^ 1, cta_err, 70)) return false;
  int it = atomicAdd(p.sched_counter, 1);
  // every thread block draws until its first value >= n_items, so one launch draws n_items + gridDim.x
  // values in all; a larger value means another launch in flight shares the counter (more launches
  // overlapping than the library has counters): report it instead of silently skipping or repeating items
  if (it >= p.n_items + static_cast<int>(gridDim.x)) *cta_err = 76;
  if (it >= p.n_items) it = -1;
  *reinterpret_cast<volatile int*>(&bars->sched_item[slot]) = it;
  mbar_arrive(smem_u32(&bars->sched_full[slot]));
  *item = it;
  return true;
}
__device__ __forceinline__ bool bwd_sched_take(BwdBarriers* bars, int round, int* item, volatile int* cta_err) {
  const uint32_t slot = round & 1, phase = (round >> 1) & 1;
  if (!mbar_wait(smem_u32(&bars->sched_full[slot]), phase, cta_err, 71)) return false;
  *item = *reinterpret_cast<volatile int*>(&bars->sched_item[slot]);
  mbar_arrive(smem_u32(&bars->sched_empty[slot]));
  return true;
}

// GROUPED = false compiles the plain case (one query head per key/value head, no padded batch)
// without the head loop and without the per-sequence lengths; it is the benchmarked path.
// GROUPED = true serves grouped heads, padded batches and batches stored without padding.
// Sequence that owns `row` in a batch stored without padding: the largest s with cu[s] <= row.
__device__ __forceinline__ int bwd_seq_of_row(const int* __restrict__ cu, int n_seqs, int row) {
  int lo = 0, hi = n_seqs;   // cu[lo] <= row < cu[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (__ldg(cu + mid) <= row) lo = mid; else hi = mid;
  }
  return lo;
}

template <bool CAUSAL, bool GROUPED>
__device__ __forceinline__ BwdItem decode_bwd_item(const BwdParams& p, int item) {
  BwdItem w;
  w.j = item / p.BH;  // ascending key tile = descending work when causal
  w.bh = item - w.j * p.BH;
  int sub = 0;
  if (GROUPED && p.n_sub > 1) {   // item = (key tile, key/value head, part of its query heads)
    const int per_j = p.BH * p.n_sub;
    w.j = item / per_j;
    const int r = item - w.j * per_j;
    w.bh = r / p.n_sub;
    sub = r - w.bh * p.n_sub;
  }
  int part = 0;
  if (GROUPED && p.i_split > 1) {   // item = (key tile, head, half of its query tiles)
    const int per_j = p.BH * 2;
    w.j = item / per_j;
    const int r = item - w.j * per_j;
    w.bh = r >> 1;
    part = r & 1;
  }
  w.bh_q0 = GROUPED ? (w.bh / p.H_kv) * p.H + (w.bh % p.H_kv) * p.group + sub * p.heads_per_sub : w.bh;
  // causal: the first query tile whose last row, at position 128 i + 127 + pos0, reaches key 128 j
  // padded batch: query tiles past the sequence's end are not visited at all
  const bool padded = GROUPED && p.seqlens != nullptr;
  w.n_valid = padded ? max(0, min(p.N, __ldg(p.seqlens + w.bh / p.H_kv))) : p.N;
  const int n_tiles_q = padded ? max(1, (w.n_valid + kT - 1) / kT) : p.n_tiles;
  // (a key tile that lies after every query still visits the last query tile, fully masked: zeros)
  w.i_begin = CAUSAL ? min(n_tiles_q - 1, max(0, (w.j * kT - p.pos0) / kT)) : 0;
  // a key tile wholly past the sequence's end needs one (fully masked) query tile to write its zeros
  if (padded && w.j * kT >= w.n_valid) w.i_begin = n_tiles_q - 1;
  w.n = n_tiles_q - w.i_begin;
  if (GROUPED && p.cu_seqlens != nullptr) {
    // batch without padding: the queries that see this key tile run from the start of its first
    // key's sequence (causal: from the first key itself) to the end of its last key's sequence
    const int k_first = w.j * kT, k_last = min(p.N, k_first + kT) - 1;
    const int q_lo = CAUSAL ? k_first : __ldg(p.cu_seqlens + bwd_seq_of_row(p.cu_seqlens, p.n_seqs, k_first));
    const int q_hi = __ldg(p.cu_seqlens + bwd_seq_of_row(p.cu_seqlens, p.n_seqs, k_last) + 1);
    // (offsets that do not rise from 0 to N give wrong results, but the clamps keep every loop bounded)
    w.i_begin = max(0, min(p.n_tiles - 1, q_lo / kT));
    w.n = max(1, min(p.n_tiles, (q_hi + kT - 1) / kT) - w.i_begin);
  }
  if (GROUPED && p.i_split > 1) {
    const int first_half = (w.n + 1) / 2;
    if (part == 0) {
      w.n = first_half;
    } else if (w.n > first_half) {
      w.i_begin += first_half;
      w.n -= first_half;
    } else {
      // a single query tile cannot be divided (the last key tile of a causal call): the second item
      // visits the query tile before it, which the mask blanks completely, and adds zeros
      w.i_begin = max(0, w.i_begin - 1);
      w.n = 1;
    }
  }
  w.steps = GROUPED ? p.heads_per_sub * w.n : w.n;
  return w;
}

// TMEM column map (fp32 columns).
// D = 128: region A = S^T / P^T, region B = dP^T / dS^T / dQ, then dV and dK: 4 x 128 columns, tensor memory
// is full.  S^T(i+1) has to wait for dV(i), which reads P^T(i) from A, and dP^T(i+1) for the drain of dQ(i).
// D = 64: dV and dK take 64 columns each and 128 are left over.  They make a second region A: steps
// alternate between A0 and A1, S^T runs two steps ahead of the activation, and dQ(i) is written over the
// first 64 columns of the step's own region A (its P^T has been consumed by dV(i), which the same thread
// issued earlier) so that region B is free for dP^T(i+1) at once.  S^T(i+2) waits for the drain of dQ(i).
template <int D>
struct BwdTmem {
  static constexpr bool kTwoA = (D == 64);
  static constexpr uint32_t kB = 128;
  static constexpr uint32_t kDv = 256;
  static constexpr uint32_t kDk = 256 + D;
  // region A of (global) step `step`, its index, and how often that region has been used before
  __device__ static __forceinline__ uint32_t a_col(uint32_t step) { return (kTwoA && (step & 1)) ? 384u : 0u; }
  __device__ static __forceinline__ uint32_t r_index(uint32_t step) { return kTwoA ? (step & 1) : 0u; }
  __device__ static __forceinline__ uint32_t r_use(uint32_t step) { return kTwoA ? (step >> 1) : step; }
  // where dQ of that step is accumulated
  __device__ static __forceinline__ uint32_t dq_col(uint32_t step) { return kTwoA ? a_col(step) : kB; }
};

// ------------------------------------------------------------------ producer

template <int D, bool CAUSAL, bool GROUPED, bool DYNAMIC>
__device__ void bwd_load_role(const BwdParams& p, const CUtensorMap* tmQ, const CUtensorMap* tmK,
                              const CUtensorMap* tmV, const CUtensorMap* tmDo, uint32_t smem_base,
                              BwdBarriers* bars, volatile int* cta_err) {
  using L = BwdSmem<D>;
  uint32_t q_cnt = 0, do_cnt = 0, item_cnt = 0;
  auto load_tile = [&](const CUtensorMap* tm, uint32_t dst, uint32_t bar, int row, int bh) {
#pragma unroll
    for (int pn = 0; pn < L::kPanels; ++pn) tma_load_3d(dst + pn * L::kPanelBytes, tm, bar, pn * 64, row, bh);
  };
  auto load_q = [&](int i, int bh) -> bool {
    const uint32_t st = q_cnt % L::kQStages, ph = (q_cnt / L::kQStages) & 1;
    if (!mbar_wait(smem_u32(&bars->q_empty[st]), ph ^ 1, cta_err, 40)) return false;
    const uint32_t bar = smem_u32(&bars->q_full[st]);
    mbar_arrive_expect_tx(bar, L::kTileBytes);
    load_tile(tmQ, smem_base + L::kQOff + st * L::kTileBytes, bar, i * kT, bh);
    ++q_cnt;
    return true;
  };
  auto load_do = [&](int i, int bh) -> bool {
    if (!mbar_wait(smem_u32(&bars->do_empty), (do_cnt & 1) ^ 1, cta_err, 41)) return false;
    const uint32_t bar = smem_u32(&bars->do_full);
    mbar_arrive_expect_tx(bar, L::kTileBytes);
    load_tile(tmDo, smem_base + L::kDoOff, bar, i * kT, bh);
    ++do_cnt;
    return true;
  };
  for (int round = 0, rounds = bwd_num_rounds(p.n_items); DYNAMIC || round < rounds; ++round) {
    int item;
    if (DYNAMIC) {
      if (!bwd_sched_draw(p, bars, round, &item, cta_err)) return;
      if (item < 0) break;
    } else {
      item = bwd_snake_rank(round, p.n_items);
      if (item < 0) continue;
    }
    const BwdItem w = decode_bwd_item<CAUSAL, GROUPED>(p, item);
    if (!load_q(w.i_begin, w.bh_q0)) return;
    if (!load_do(w.i_begin, w.bh_q0)) return;
    if (!mbar_wait(smem_u32(&bars->kv_empty), (item_cnt & 1) ^ 1, cta_err, 42)) return;
    {
      const uint32_t bar = smem_u32(&bars->kv_full);
      mbar_arrive_expect_tx(bar, 2 * L::kTileBytes);
      load_tile(tmK, smem_base + L::kKOff, bar, w.j * kT, w.bh);
      load_tile(tmV, smem_base + L::kVOff, bar, w.j * kT, w.bh);
    }
    ++item_cnt;
    // The remaining steps, head by head.  With two regions A (D = 64) S^T runs a step further ahead than
    // dP^T, so Q stays one tile ahead of dO: dO(s) can only be loaded after dV(s-1), and S^T(s+1) is issued
    // before that product's inputs exist.
    constexpr int lead = BwdTmem<D>::kTwoA ? 1 : 0;
    auto load_step = [&](int s, bool is_q) -> bool {
      const int g = GROUPED ? s / w.n : 0;
      const int i = w.i_begin + (s - g * w.n), bh = w.bh_q0 + g;
      return is_q ? load_q(i, bh) : load_do(i, bh);
    };
    for (int q_next = 1, do_next = 1; do_next < w.steps; ++do_next) {
      for (; q_next < w.steps && q_next <= do_next + lead; ++q_next)
        if (!load_step(q_next, true)) return;
      if (!load_step(do_next, false)) return;
    }
  }
}

// ------------------------------------------------------------------ MMA issuer

template <int D, bool CAUSAL, bool GROUPED, bool DYNAMIC>
__device__ void bwd_mma_role(const BwdParams& p, uint32_t smem_base, uint32_t tmem, BwdBarriers* bars,
                             volatile int* cta_err) {
  using L = BwdSmem<D>;
  using TM = BwdTmem<D>;
  constexpr uint32_t kIdescSt = make_idesc_bf16(kT, kT, 0, 0);   // S^T, dP^T : K-major x K-major
  constexpr uint32_t kIdescAcc = make_idesc_bf16(kT, D, 0, 1);   // dV, dK   : (TMEM | K-major) x MN-major
  constexpr uint32_t kIdescDq = make_idesc_bf16(kT, D, 1, 1);    // dQ       : MN-major x MN-major
  const uint32_t sK = smem_base + L::kKOff, sV = smem_base + L::kVOff, sDo = smem_base + L::kDoOff,
                 sDs = smem_base + L::kDsOff;
  uint32_t q_cnt = 0, do_cnt = 0, item_cnt = 0, step_cnt = 0;

  // [128 x 128] = X[128 x D] * Y[128 x D]^T, both K-major
  auto issue_kk = [&](uint32_t d_col, uint64_t x_desc, uint64_t y_desc) {
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
      const uint32_t off = (ks >> 2) * L::kPanelBytes + (ks & 3) * 32;
      umma_ss(tmem + d_col, desc_advance(x_desc, off), desc_advance(y_desc, off), kIdescSt, ks > 0);
    }
  };
  // Descriptors are built once; each k-step only advances the start address.
  const uint64_t dK_k = make_smem_desc_sw128(sK, 16, 1024);                 // K_j, K-major (S^T)
  const uint64_t dV_k = make_smem_desc_sw128(sV, 16, 1024);                 // V_j, K-major (dP^T)
  const uint64_t dDo_k = make_smem_desc_sw128(sDo, 16, 1024);               // dO_i, K-major (dP^T)
  const uint64_t dDo_mn = make_smem_desc_sw128(sDo, L::kPanelBytes, 1024);  // dO_i, MN-major (dV)
  const uint64_t dK_mn = make_smem_desc_sw128(sK, L::kPanelBytes, 1024);    // K_j, MN-major (dQ)
  const uint64_t dDs_mn = make_smem_desc_sw128(sDs, L::kPanelBytes, 1024);  // dS^T, MN-major (dQ)
  // Stage 0 of Q; the other stages are reached by advancing the start address (an array indexed by the
  // stage at run time would live in local memory, and this thread pays for every load in full)
  const uint64_t dQ_k0 = make_smem_desc_sw128(smem_base + L::kQOff, 16, 1024);                 // Q_i, K-major (S^T)
  const uint64_t dQ_mn0 = make_smem_desc_sw128(smem_base + L::kQOff, L::kPanelBytes, 1024);    // Q_i, MN-major (dK)
  auto q_stage = [](uint32_t cnt) -> uint32_t { return cnt % L::kQStages; };
  auto q_phase = [](uint32_t cnt) -> uint32_t { return (cnt / L::kQStages) & 1; };
  // S^T of global step `step` from the Q tile with running number `qn`.  D = 64: the step's region A last
  // held dQ of two steps earlier, which the drain group must have read.
  auto issue_s = [&](uint32_t step, uint32_t qn, int where) -> bool {
    if (!mbar_wait(smem_u32(&bars->q_full[q_stage(qn)]), q_phase(qn), cta_err, where)) return false;
    if (TM::kTwoA &&
        !mbar_wait(smem_u32(&bars->dq_empty[TM::r_index(step)]), (TM::r_use(step) & 1) ^ 1, cta_err, where + 20))
      return false;
    tc_fence_after_sync();
    issue_kk(TM::a_col(step), dK_k, desc_advance(dQ_k0, q_stage(qn) * L::kTileBytes));
    umma_commit(smem_u32(&bars->s_full[TM::r_index(step)]));
    return true;
  };
  // dP^T of global step `step`.  D = 128: region B last held dQ of the step before.
  auto issue_dp = [&](uint32_t step, int where) -> bool {
    if (!mbar_wait(smem_u32(&bars->do_full), do_cnt & 1, cta_err, where)) return false;
    if (!TM::kTwoA &&
        !mbar_wait(smem_u32(&bars->dq_empty[0]), (step & 1) ^ 1, cta_err, where + 20))
      return false;
    tc_fence_after_sync();
    issue_kk(TM::kB, dV_k, dDo_k);
    umma_commit(smem_u32(&bars->dp_full));
    return true;
  };

  for (int round = 0, rounds = bwd_num_rounds(p.n_items); DYNAMIC || round < rounds; ++round) {
    int item;
    if (DYNAMIC) {
      if (!bwd_sched_take(bars, round, &item, cta_err)) return;
      if (item < 0) break;
    } else {
      item = bwd_snake_rank(round, p.n_items);
      if (item < 0) continue;
    }
    const BwdItem w = decode_bwd_item<CAUSAL, GROUPED>(p, item);
    if (!mbar_wait(smem_u32(&bars->kv_full), item_cnt & 1, cta_err, 50)) return;

    // prologue: S^T(0), dP^T(0) and, with two regions A, S^T(1)
    if (!issue_s(step_cnt, q_cnt, 51)) return;
    if (!issue_dp(step_cnt, 52)) return;
    if (TM::kTwoA && w.steps > 1 && !issue_s(step_cnt + 1, q_cnt + 1, 53)) return;

    for (int it = 0; it < w.steps; ++it) {
      const uint32_t st = q_stage(q_cnt), reg = TM::r_index(step_cnt);
      // dV += P^T dO_i
      if (!mbar_wait(smem_u32(&bars->p_ready[reg]), TM::r_use(step_cnt) & 1, cta_err, 54)) return;
      if (it == 0 && !mbar_wait(smem_u32(&bars->dkv_empty), (item_cnt & 1) ^ 1, cta_err, 55)) return;
      tc_fence_after_sync();
#pragma unroll
      for (int ks = 0; ks < kT / 16; ++ks) {
        umma_ts(tmem + TM::kDv, tmem + TM::a_col(step_cnt) + (ks >> 2) * 64 + (ks & 3) * 8,
                desc_advance(dDo_mn, ks * 2048), kIdescAcc, (it > 0 || ks > 0));
      }
      umma_commit(smem_u32(&bars->do_empty));
      ++do_cnt;
      // one region A: S^T of the next query tile goes where P^T was
      if (!TM::kTwoA && it + 1 < w.steps && !issue_s(step_cnt + 1, q_cnt + 1, 56)) return;
      // dK += dS^T Q_i with dS^T read from region B of tensor memory (the activation groups
      // leave a bf16 copy there, over the dP^T columns they have consumed), then dQ_i = dS K_j,
      // which overwrites region B (D = 128) or the head of the step's region A (D = 64): MMAs of
      // one thread execute in issue order.
      if (!mbar_wait(smem_u32(&bars->ds_ready), step_cnt & 1, cta_err, 57)) return;
      tc_fence_after_sync();
      const uint64_t q_mn = desc_advance(dQ_mn0, st * L::kTileBytes);
#pragma unroll
      for (int ks = 0; ks < kT / 16; ++ks) {
        umma_ts(tmem + TM::kDk, tmem + TM::kB + (ks >> 2) * 64 + (ks & 3) * 8, desc_advance(q_mn, ks * 2048),
                kIdescAcc, (it > 0 || ks > 0));
      }
#pragma unroll
      for (int ks = 0; ks < kT / 16; ++ks) {
        umma_ss(tmem + TM::dq_col(step_cnt), desc_advance(dDs_mn, ks * 2048), desc_advance(dK_mn, ks * 2048),
                kIdescDq, ks > 0);
      }
      umma_commit(smem_u32(&bars->dq_full[reg]));
      umma_commit(smem_u32(&bars->q_empty[st]));
      // dP^T of the next query tile, then (two regions A) S^T of the one after it
      if (it + 1 < w.steps && !issue_dp(step_cnt + 1, 58)) return;
      if (TM::kTwoA && it + 2 < w.steps && !issue_s(step_cnt + 2, q_cnt + 2, 59)) return;
      ++q_cnt;
      ++step_cnt;
    }
    umma_commit(smem_u32(&bars->dkv_full));
    ++item_cnt;
  }
}

// ------------------------------------------------------------------ activation groups

// 32 logits (transposed tile: this thread's key against 32 queries) -> P as bf16x2 for
// the dV product and P (1 - P) in fp32 for dS.
//   a = log2(e) * (scale * s + b - slope * |i - j|);  u = 2^a;  P = u / (1 + u);  1 - P = 1 / (1 + u)
// MASK: 0 no element masked, 1 causal only (queries before mask_lo), 2 both ends (padded batch)
// CAUSAL: a query that keeps its weight sits at or after the key, so the position term is linear in the
// query index: one FMA per logit from a per-call constant (a masked query is blanked afterwards).
template <int MASK, bool ALIBI, bool CAUSAL>
__device__ __forceinline__ void bwd_sigmoid_chunk(const uint32_t (&s)[32], uint32_t (&p_out)[16], float (&pp)[32],
                                                  float scale_log2e, float bias_log2e, float slope_log2e,
                                                  float col_rel, int q_base, float mask_lo, float mask_hi) {
  float a[32];
  const float c_first = fmaf(-slope_log2e, static_cast<float>(q_base) - col_rel, bias_log2e);   // query q_base
#pragma unroll
  for (int e = 0; e < 32; ++e) {
    float c0 = bias_log2e;
    if (ALIBI && CAUSAL) c0 = fmaf(-slope_log2e, static_cast<float>(e), c_first);
    else if (ALIBI) c0 = fmaf(-slope_log2e, fabsf(static_cast<float>(q_base + e) - col_rel), bias_log2e);
    a[e] = fmaf(__uint_as_float(s[e]), scale_log2e, c0);
  }
  float pr[32];
  sigmoid_block<32, true, 0>(a, pr, pp);
  if (MASK == 1) {
#pragma unroll
    for (int e = 0; e < 32; ++e)
      if (static_cast<float>(q_base + e) < mask_lo) { pr[e] = 0.0f; pp[e] = 0.0f; }  // query before key
  }
  if (MASK == 2) {
#pragma unroll
    for (int e = 0; e < 32; ++e)
      // query before key (causal), or, in a padded batch, past the end of the sequence
      if (static_cast<float>(q_base + e) < mask_lo || static_cast<float>(q_base + e) >= mask_hi) {
        pr[e] = 0.0f;
        pp[e] = 0.0f;
      }
  }
#pragma unroll
  for (int e = 0; e < 16; ++e) p_out[e] = pack_bf16x2(pr[2 * e], pr[2 * e + 1]);
}

// One row of a [128 x D] fp32 accumulator -> bf16 (times `mul`) -> swizzled staging tile.
template <int D>
__device__ __forceinline__ void bwd_store_acc_rows(uint32_t t_acc, uint8_t* stage, int tid, float mul) {
  using L = BwdSmem<D>;
#pragma unroll 1
  for (int c = 0; c < D / 32; ++c) {
    uint32_t o[32];
    tmem_ld32(t_acc + c * 32, o);
    tmem_wait_ld();
    uint8_t* panel = stage + (c >> 1) * L::kPanelBytes + tid * 128;
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      uint4 val;
      val.x = pack_bf16x2(mul * __uint_as_float(o[8 * g + 0]), mul * __uint_as_float(o[8 * g + 1]));
      val.y = pack_bf16x2(mul * __uint_as_float(o[8 * g + 2]), mul * __uint_as_float(o[8 * g + 3]));
      val.z = pack_bf16x2(mul * __uint_as_float(o[8 * g + 4]), mul * __uint_as_float(o[8 * g + 5]));
      val.w = pack_bf16x2(mul * __uint_as_float(o[8 * g + 6]), mul * __uint_as_float(o[8 * g + 7]));
      const int chunk = (c & 1) * 4 + g;
      *reinterpret_cast<uint4*>(panel + ((chunk ^ (tid & 7)) * 16)) = val;
    }
  }
}

// KIND: 0 plain, 1 general (grouped heads, padded batch), 2 general plus a batch stored without padding
template <int D, bool CAUSAL, bool ALIBI, bool DBIAS, int KIND>
__device__ void bwd_act_role(const BwdParams& p, const CUtensorMap* tmDk, const CUtensorMap* tmDv, int wg,
                             uint8_t* smem, uint32_t tmem, BwdBarriers* bars, volatile int* cta_err) {
  using L = BwdSmem<D>;
  using TM = BwdTmem<D>;
  constexpr bool GROUPED = KIND >= 1, DYNAMIC = KIND == 2;
  const int tid = threadIdx.x & 127;  // key row within the tile
  const uint32_t lane_off = static_cast<uint32_t>(((threadIdx.x >> 5) & 3) * 32) << 16;
  uint32_t step_cnt = 0, item_cnt = 0;

  for (int round = 0, rounds = bwd_num_rounds(p.n_items); DYNAMIC || round < rounds; ++round) {
    int item;
    if (DYNAMIC) {
      if (!bwd_sched_take(bars, round, &item, cta_err)) return;
      if (item < 0) break;
    } else {
      item = bwd_snake_rank(round, p.n_items);
      if (item < 0) continue;
    }
    const BwdItem w = decode_bwd_item<CAUSAL, GROUPED>(p, item);
    for (int g = 0; g < (GROUPED ? p.heads_per_sub : 1); ++g) {   // the query heads that read this key/value head
    const int bh_q = w.bh_q0 + g;
    float slope_log2e = 0.0f;
    if (ALIBI) slope_log2e = p.slopes[bh_q % p.H] * kLog2eB;
    float bias_log2e = p.bias_vec ? __ldg(p.bias_vec + bh_q) * kLog2eB : p.bias_log2e;
    float ds_sum = 0.0f;   // this thread's share of sum dS over the head's tiles (the bias gradient)
    // batch without padding: the queries [q_lo, q_hi) that see this thread's key (its own sequence,
    // from the key itself on when causal), and the sequence's bias
    constexpr bool ragged = (KIND == 2);
    int q_lo = 0, q_hi = 0, seq = 0;
    if (ragged) {
      const int kr = w.j * kT + tid;
      bias_log2e = p.bias_log2e;
      if (kr < p.N) {
        seq = bwd_seq_of_row(p.cu_seqlens, p.n_seqs, kr);
        q_lo = CAUSAL ? kr : __ldg(p.cu_seqlens + seq);
        q_hi = __ldg(p.cu_seqlens + seq + 1);
        if (p.bias_vec) bias_log2e = __ldg(p.bias_vec + seq * p.H + bh_q) * kLog2eB;
      }
    }

    for (int it = 0; it < w.n; ++it) {
      const int i = w.i_begin + it;
      // this thread's key index minus the position of the tile's first query
      const float col_rel = static_cast<float>((w.j - i) * kT + tid - p.pos0);
      // the mask cuts through the tile unless even its first query sits at or after the last key:
      // the first tile of the loop, and with pos0 not a multiple of 128 also the second
      bool diag = CAUSAL && (i * kT + p.pos0 < w.j * kT + kT - 1);
      // queries [mask_lo, mask_hi) of the tile keep their weight for this thread's key
      float mask_lo = CAUSAL ? col_rel : -1.0f, mask_hi = 1.0e9f;
      if (GROUPED && p.seqlens != nullptr) {
        mask_hi = static_cast<float>(w.n_valid - i * kT);
        if (w.j * kT + tid >= w.n_valid) mask_hi = -1.0f;   // a key past the end: the whole row
        diag = diag || (w.j + 1) * kT > w.n_valid || (i + 1) * kT > w.n_valid;
      }
      if (ragged) {
        mask_lo = static_cast<float>(q_lo - i * kT);
        mask_hi = static_cast<float>(q_hi - i * kT);
        diag = i * kT < q_lo || (i + 1) * kT > q_hi;   // the tile is not wholly inside this key's queries
      }
      float pp0[32], pp1[32];
      if (!mbar_wait(smem_u32(&bars->s_full[TM::r_index(step_cnt)]), TM::r_use(step_cnt) & 1, cta_err, 60 + wg))
        return;
      tc_fence_after_sync();
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const int gc = wg * 2 + c;  // 32-query chunk of the tile
        uint32_t s[32], pk[16];
        tmem_ld32(tmem + TM::a_col(step_cnt) + lane_off + gc * 32, s);
        tmem_wait_ld();
        float(&ppc)[32] = (c == 0) ? pp0 : pp1;
        if (GROUPED && diag)
          bwd_sigmoid_chunk<2, ALIBI, CAUSAL>(s, pk, ppc, p.scale_log2e, bias_log2e, slope_log2e, col_rel, gc * 32, mask_lo,
                                      mask_hi);
        else if (CAUSAL && diag)
          bwd_sigmoid_chunk<1, ALIBI, CAUSAL>(s, pk, ppc, p.scale_log2e, bias_log2e, slope_log2e, col_rel, gc * 32, col_rel,
                                      0.0f);
        else
          bwd_sigmoid_chunk<0, ALIBI, CAUSAL>(s, pk, ppc, p.scale_log2e, bias_log2e, slope_log2e, col_rel, gc * 32, 0.0f,
                                      0.0f);
        tmem_st16(tmem + TM::a_col(step_cnt) + lane_off + wg * 64 + c * 16, pk);
      }
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(smem_u32(&bars->p_ready[TM::r_index(step_cnt)]));

      // dS^T = P (1 - P) dP^T -> bf16 -> shared memory [key][query], 128-byte swizzle
      if (!mbar_wait(smem_u32(&bars->dp_full), step_cnt & 1, cta_err, 62 + wg)) return;
      tc_fence_after_sync();
      uint8_t* ds_row = smem + L::kDsOff + wg * L::kPanelBytes + tid * 128;
#pragma unroll
      for (int c = 0; c < 4; ++c) {  // 16 queries at a time
        uint32_t dp[16];
        tmem_ld16(tmem + TM::kB + lane_off + wg * 64 + c * 16, dp);
        tmem_wait_ld();
        uint32_t ds[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float* f = ((c < 2) ? pp0 : pp1) + (c & 1) * 16 + 2 * e;
          const float ds0 = f[0] * __uint_as_float(dp[2 * e]), ds1 = f[1] * __uint_as_float(dp[2 * e + 1]);
          if (DBIAS) ds_sum += ds0 + ds1;
          ds[e] = pack_bf16x2(ds0, ds1);
        }
        // one copy to shared memory (A operand of dQ, MN-major) ...
#pragma unroll
        for (int g = 0; g < 2; ++g) {
          const int chunk = c * 2 + g;
          *reinterpret_cast<uint4*>(ds_row + ((chunk ^ (tid & 7)) * 16)) =
              make_uint4(ds[4 * g + 0], ds[4 * g + 1], ds[4 * g + 2], ds[4 * g + 3]);
        }
        // ... and one to tensor memory (A operand of dK), over dP^T columns already consumed
        tmem_st8(tmem + TM::kB + lane_off + wg * 64 + c * 8, ds);
      }
      tmem_wait_st();
      tc_fence_before_sync();   // the dP^T reads above precede the dQ MMA that overwrites region B
      fence_proxy_async_smem();
      mbar_arrive(smem_u32(&bars->ds_ready));
      ++step_cnt;
    }

    if (DBIAS && ragged) {   // keys of one warp may belong to different sequences: one atomic per key
      if (q_hi > q_lo) atomicAdd(p.dbias + seq * p.H + bh_q, ds_sum);
    } else if (DBIAS) {   // sum over the warp, one atomic per warp, item and query head
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) ds_sum += __shfl_xor_sync(0xffffffffu, ds_sum, off);
      if ((threadIdx.x & 31) == 0) atomicAdd(p.dbias + bh_q, ds_sum);
    }
    }   // query heads

    // epilogue: group 0 stores dV_j (staged in the V tile), group 1 stores scale * dK_j (K tile)
    if (!mbar_wait(smem_u32(&bars->dkv_full), item_cnt & 1, cta_err, 64 + wg)) return;
    ++item_cnt;
    tc_fence_after_sync();
    uint8_t* stage = smem + (wg == 0 ? L::kVOff : L::kKOff);
    bwd_store_acc_rows<D>(tmem + (wg == 0 ? TM::kDv : TM::kDk) + lane_off, stage, tid, wg == 0 ? 1.0f : p.scale);
    tc_fence_before_sync();
    mbar_arrive(smem_u32(&bars->dkv_empty));
    fence_proxy_async_smem();
    if (wg == 0) named_barrier_sync<1, 128>(); else named_barrier_sync<2, 128>();
    if (tid == 0) {
      const CUtensorMap* tm = (wg == 0) ? tmDv : tmDk;
#pragma unroll
      for (int pn = 0; pn < L::kPanels; ++pn)
        if (GROUPED && (p.n_sub > 1 || p.i_split > 1 || p.dkv_add))   // the parts (or successive calls) add their shares
          tma_reduce_add_3d(tm, smem_u32(stage + pn * L::kPanelBytes), pn * 64, w.j * kT, w.bh);
        else
          tma_store_3d(tm, smem_u32(stage + pn * L::kPanelBytes), pn * 64, w.j * kT, w.bh);
      tma_commit_group();
      tma_wait_group_read<0>();
      mbar_arrive(smem_u32(&bars->kv_empty));
    }
  }
  if (tid == 0) tma_wait_group<0>();
}

// ------------------------------------------------------------------ dQ drain group

template <int D, bool CAUSAL, bool GROUPED, bool DYNAMIC>
__device__ void bwd_drain_role(const BwdParams& p, const CUtensorMap* tmW, uint8_t* smem, uint32_t tmem,
                               BwdBarriers* bars, volatile int* cta_err) {
  using L = BwdSmem<D>;
  using TM = BwdTmem<D>;
  const int tid = threadIdx.x & 127;  // query row within the tile
  const uint32_t lane_off = static_cast<uint32_t>(((threadIdx.x >> 5) & 3) * 32) << 16;
  uint32_t step_cnt = 0;
  for (int round = 0, rounds = bwd_num_rounds(p.n_items); DYNAMIC || round < rounds; ++round) {
    int item;
    if (DYNAMIC) {
      if (!bwd_sched_take(bars, round, &item, cta_err)) return;
      if (item < 0) break;
    } else {
      item = bwd_snake_rank(round, p.n_items);
      if (item < 0) continue;
    }
    const BwdItem w = decode_bwd_item<CAUSAL, GROUPED>(p, item);
    for (int s = 0; s < w.steps; ++s) {
      const int g = GROUPED ? s / w.n : 0, it = s - g * w.n;   // query head within the group, query tile
      const int row0 = (w.i_begin + it) * kT, bh_q = w.bh_q0 + g;
      const uint32_t reg = TM::r_index(step_cnt), dq_col = TM::dq_col(step_cnt);
      if (!mbar_wait(smem_u32(&bars->dq_full[reg]), TM::r_use(step_cnt) & 1, cta_err, 70)) return;
      ++step_cnt;
      tc_fence_after_sync();
      // 64 columns per round: both staging boxes are filled from registers, so region B is
      // released right after the last TMEM read instead of after the last reduce-add.
#pragma unroll 1
      for (int r = 0; r < D / 64; ++r) {
        uint32_t o0[32], o1[32];
        tmem_ld32(tmem + dq_col + lane_off + r * 64, o0);
        tmem_ld32(tmem + dq_col + lane_off + r * 64 + 32, o1);
        tmem_wait_ld();
        if (r == D / 64 - 1) {
          tc_fence_before_sync();
          mbar_arrive(smem_u32(&bars->dq_empty[reg]));
        }
        // both staging boxes must have been read by the reduce-adds issued earlier
        if (tid == 0) tma_wait_group_read<0>();
        named_barrier_sync<3, 128>();
        uint8_t* row0p = smem + L::kDqOff + tid * 128;
        uint8_t* row1p = row0p + L::kPanelBytes;
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          *reinterpret_cast<uint4*>(row0p + ((g ^ (tid & 7)) * 16)) =
              make_uint4(o0[4 * g + 0], o0[4 * g + 1], o0[4 * g + 2], o0[4 * g + 3]);
          *reinterpret_cast<uint4*>(row1p + ((g ^ (tid & 7)) * 16)) =
              make_uint4(o1[4 * g + 0], o1[4 * g + 1], o1[4 * g + 2], o1[4 * g + 3]);
        }
        fence_proxy_async_smem();
        named_barrier_sync<3, 128>();
        if (tid == 0) {
          tma_reduce_add_3d(tmW, smem_u32(smem + L::kDqOff), r * 64, row0, bh_q);
          tma_reduce_add_3d(tmW, smem_u32(smem + L::kDqOff + L::kPanelBytes), r * 64 + 32, row0, bh_q);
          tma_commit_group();
        }
      }
    }
  }
  if (tid == 0) tma_wait_group<0>();
}

// ------------------------------------------------------------------ kernels

template <int D, bool CAUSAL, bool ALIBI, bool DBIAS, int KIND>
__global__ void __launch_bounds__(kBwdThreads, 1)
sigattn_bwd_bf16_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                        const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmDo,
                        const __grid_constant__ CUtensorMap tmDk, const __grid_constant__ CUtensorMap tmDv,
                        const __grid_constant__ CUtensorMap tmW, const BwdParams p) {
  constexpr bool GROUPED = KIND >= 1;
  extern __shared__ uint8_t smem_raw[];
  __shared__ BwdBarriers bars;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int cta_err;

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  const int warp = threadIdx.x >> 5;

  if (threadIdx.x == 0) {
    cta_err = 0;
    mbar_init(smem_u32(&bars.kv_full), 1);
    mbar_init(smem_u32(&bars.kv_empty), 2);
    for (int s = 0; s < 3; ++s) {
      mbar_init(smem_u32(&bars.q_full[s]), 1);
      mbar_init(smem_u32(&bars.q_empty[s]), 1);
    }
    mbar_init(smem_u32(&bars.do_full), 1);
    mbar_init(smem_u32(&bars.do_empty), 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&bars.s_full[s]), 1);
      mbar_init(smem_u32(&bars.p_ready[s]), 256);
      mbar_init(smem_u32(&bars.dq_full[s]), 1);
      mbar_init(smem_u32(&bars.dq_empty[s]), 128);
    }
    mbar_init(smem_u32(&bars.dp_full), 1);
    mbar_init(smem_u32(&bars.ds_ready), 256);
    mbar_init(smem_u32(&bars.dkv_full), 1);
    mbar_init(smem_u32(&bars.dkv_empty), 256);
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&bars.sched_full[s]), 1);
      mbar_init(smem_u32(&bars.sched_empty[s]), kBwdSchedConsumers);
    }
    fence_mbar_init();
  }
  if (warp == kBwdLoadWarp && elect_one()) {
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
    tma_prefetch_desc(&tmDo);
    tma_prefetch_desc(&tmDk);
    tma_prefetch_desc(&tmDv);
    tma_prefetch_desc(&tmW);
  }
  if (warp == kBwdMmaWarp) {
    tmem_alloc(smem_u32(&tmem_base_slot), 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_base_slot;

  if (warp == kBwdLoadWarp) {
    if ((threadIdx.x & 31) == 0) bwd_load_role<D, CAUSAL, GROUPED, KIND == 2>(p, &tmQ, &tmK, &tmV, &tmDo, smem_base, &bars, &cta_err);
    __syncwarp();
  } else if (warp == kBwdMmaWarp) {
    if ((threadIdx.x & 31) == 0) bwd_mma_role<D, CAUSAL, GROUPED, KIND == 2>(p, smem_base, tmem, &bars, &cta_err);
    __syncwarp();
  } else if (warp < 8) {
    bwd_act_role<D, CAUSAL, ALIBI, DBIAS, KIND>(p, &tmDk, &tmDv, warp >> 2, smem, tmem, &bars, &cta_err);
  } else {
    bwd_drain_role<D, CAUSAL, GROUPED, KIND == 2>(p, &tmW, smem, tmem, &bars, &cta_err);
  }

  tc_fence_before_sync();
  __syncthreads();
  if (cta_err != 0) {
    if (threadIdx.x == 0) atomicExch(p.status, 200 + cta_err);
    __nanosleep(100000);
  }
  if (warp == kBwdMmaWarp) tmem_dealloc(tmem, 512);
}

// dQ (bf16) = scale * workspace (fp32): the conversion step that follows the main kernel.
__global__ void __launch_bounds__(256)
sigattn_bwd_convert_dq_kernel(const float4* __restrict__ ws, uint2* __restrict__ dq, size_t n_vec4, float scale) {
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n_vec4; i += stride) {
    const float4 v = ws[i];
    uint2 o;
    o.x = pack_bf16x2(scale * v.x, scale * v.y);
    o.y = pack_bf16x2(scale * v.z, scale * v.w);
    dq[i] = o;
  }
}

// The same conversion with the temperature gradient on the side.  With the logits e^t * scale * q k + b
// (the learnable temperature of Section 5 and Appendix G.2.2; the caller passes scale * e^t as the
// scale), dL/dt = sum_ij dS_ij * scale' q_i k_j = sum_i <q_i, dQ_i>, because dQ_i = scale' sum_j dS_ij k_j:
// a reduction of what this pass streams anyway.  grid = (blocks per head, B*H); every block reduces its
// slice of one head and adds it to dtemp[b*H + h] (fp32 atomics: the last bits depend on the order).
__global__ void __launch_bounds__(256)
sigattn_bwd_convert_dq_dtemp_kernel(const float4* __restrict__ ws, const uint2* __restrict__ q, uint2* __restrict__ dq,
                                    size_t vec4_per_head, float scale, float* __restrict__ dtemp) {
  const size_t base = static_cast<size_t>(blockIdx.y) * vec4_per_head;
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  float sum = 0.0f;
  for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < vec4_per_head; i += stride) {
    const float4 v = ws[base + i];
    const uint2 qq = q[base + i];
    const float g0 = scale * v.x, g1 = scale * v.y, g2 = scale * v.z, g3 = scale * v.w;
    dq[base + i] = make_uint2(pack_bf16x2(g0, g1), pack_bf16x2(g2, g3));
    sum = fmaf(g0, __uint_as_float(qq.x << 16), sum);
    sum = fmaf(g1, __uint_as_float(qq.x & 0xffff0000u), sum);
    sum = fmaf(g2, __uint_as_float(qq.y << 16), sum);
    sum = fmaf(g3, __uint_as_float(qq.y & 0xffff0000u), sum);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
  __shared__ float warp_sums[8];
  if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    float total = 0.0f;
#pragma unroll
    for (int w = 0; w < 8; ++w) total += warp_sums[w];
    atomicAdd(dtemp + blockIdx.y, total);
  }
}

// Sequence-length normalisation, O = r (P V) with one factor per query row: the whole backward
// is the plain one on r_i dO_i.  This pass writes bf16(r_i dO_i) for every row ([B*H, N, D]
// row-major, 8 elements per thread); the main kernel then reads it in place of dO.
__device__ __forceinline__ uint32_t scale_bf16x2(uint32_t x, float r) {
  return pack_bf16x2(r * __uint_as_float(x << 16), r * __uint_as_float(x & 0xffff0000u));
}

__global__ void __launch_bounds__(256)
sigattn_bwd_scale_rows_kernel(const uint4* __restrict__ d_o, const float* __restrict__ row_scale,
                              uint4* __restrict__ out, size_t n_vec8, int N, int vec_per_row) {
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n_vec8; i += stride) {
    const float r = __ldg(row_scale + static_cast<int>((i / vec_per_row) % N));
    const uint4 x = d_o[i];
    out[i] = make_uint4(scale_bf16x2(x.x, r), scale_bf16x2(x.y, r), scale_bf16x2(x.z, r), scale_bf16x2(x.w, r));
  }
}

// Work-item counters of the dynamic schedule: one per launch in flight, handed out round robin.
constexpr int kBwdSchedSlots = 1024;
__device__ int g_bwd_sched_counters[kBwdSchedSlots];

template <int D, bool CAUSAL, bool ALIBI, bool DBIAS, int KIND>
int launch_bwd_variant(const CUtensorMap* maps, const BwdParams& bp, int num_sms, cudaStream_t stream,
                       cudaError_t* cuda_err) {
  auto kernel = sigattn_bwd_bf16_kernel<D, CAUSAL, ALIBI, DBIAS, KIND>;
  // The shared-memory opt-in is a per-device attribute of the kernel: one bit per device ordinal
  // (a process may drive several GPUs); ordinals past 63 simply set it on every launch.
  static std::atomic<unsigned long long> configured{0};
  int dev = 0;
  *cuda_err = cudaGetDevice(&dev);
  if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  const unsigned long long bit = (dev >= 0 && dev < 64) ? (1ull << dev) : 0ull;
  if ((configured.load(std::memory_order_relaxed) & bit) == 0) {
    *cuda_err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdSmem<D>::kDynBytes);
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
    configured.fetch_or(bit, std::memory_order_relaxed);
  }
  const int grid = bp.n_items < num_sms ? bp.n_items : num_sms;
  kernel<<<grid, kBwdThreads, BwdSmem<D>::kDynBytes, stream>>>(maps[0], maps[1], maps[2], maps[3], maps[4], maps[5],
                                                                maps[6], bp);
  *cuda_err = cudaGetLastError();
  return *cuda_err == cudaSuccess ? SIGATTN_OK : SIGATTN_ERR_CUDA;
}

}  // namespace

namespace {
thread_local cudaEvent_t t_ev_start = nullptr;
thread_local cudaEvent_t t_ev_stop = nullptr;
}  // namespace

void set_bwd_timing_events(cudaEvent_t start, cudaEvent_t stop) {
  t_ev_start = start;
  t_ev_stop = stop;
}

int launch_acc_to_bf16(const float* acc, void* out, size_t n, float mul, cudaStream_t stream,
                       unsigned long long* launches, cudaError_t* cuda_err) {
  int dev = 0, num_sms = 0;
  *cuda_err = cudaGetDevice(&dev);
  if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  *cuda_err = cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev);
  if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  const size_t n_vec4 = n / 4;
  const size_t want = n_vec4 / 256 + 1, cap = static_cast<size_t>(num_sms) * 8;
  sigattn_bwd_convert_dq_kernel<<<static_cast<int>(want < cap ? want : cap), 256, 0, stream>>>(
      reinterpret_cast<const float4*>(acc), static_cast<uint2*>(out), n_vec4, mul);
  *cuda_err = cudaGetLastError();
  if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  *launches += 1;
  return SIGATTN_OK;
}

size_t bwd_bf16_workspace_bytes(int B, int H, int N, int D) {
  return static_cast<size_t>(B) * H * N * D * sizeof(float);
}

int launch_bwd_bf16(const void* q, const void* k, const void* v, const void* d_o, void* dq, void* dk, void* dv,
                    const Problem& p, void* workspace, int* status, cudaStream_t stream,
                    unsigned long long* launches, cudaError_t* cuda_err) {
  int dev = 0, num_sms = 0;
  *cuda_err = cudaGetDevice(&dev);
  if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  *cuda_err = cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev);
  if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;

  const uint64_t BH = static_cast<uint64_t>(p.B) * p.H;             // query heads: Q, dO, the dQ accumulator
  const uint64_t BH_kv = static_cast<uint64_t>(p.B) * p.kv_heads();  // K, V, dK, dV
  CUtensorMap maps[7];
  // with factors per query row the main kernel reads r dO, staged in the dq buffer: nothing
  // writes dq before the conversion step at the end, which reads only the workspace
  const void* ptrs[6] = {q, k, v, p.row_scale != nullptr ? dq : d_o, dk, dv};
  for (int i = 0; i < 6; ++i) {
    const uint64_t heads = (i == 0 || i == 3) ? BH : BH_kv;
    const uint64_t rows = (i == 0 || i == 3) ? p.N : p.key_rows();
    if (make_map_3d(&maps[i], ptrs[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, heads, rows, p.D, kT, 64) != 0) {
      *cuda_err = cudaErrorInvalidValue;
      return SIGATTN_ERR_CUDA;
    }
  }
  if (make_map_3d(&maps[6], workspace, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, BH, p.N, p.D, kT, 32) != 0) {
    *cuda_err = cudaErrorInvalidValue;
    return SIGATTN_ERR_CUDA;
  }
  BwdParams bp;
  bp.BH = static_cast<int>(BH_kv);
  bp.H = p.H;
  bp.H_kv = p.kv_heads();
  bp.group = p.H / p.kv_heads();
  bp.N = p.N;
  bp.n_tiles = (p.N + kT - 1) / kT;
  bp.n_tiles_k = (p.key_rows() + kT - 1) / kT;
  bp.pos0 = p.query_pos0();
  // Grouped heads with few (batch, key/value head) pairs: split a group's query heads over several
  // work items (the smallest divisor of the group size that yields two items per SM, if any).
  bp.n_sub = 1;
  if (bp.group > 1 && p.seqlens == nullptr && p.cu_seqlens == nullptr) {
    const long long base_items = static_cast<long long>(bp.n_tiles_k) * bp.BH;
    // at most four parts: every part adds one bf16 rounding to dK, dV (sixteen parts measured a
    // relative error of 5.5e-3, four stay near 3e-3)
    for (int d = 1; d <= bp.group && d <= 4; ++d) {
      if (bp.group % d != 0) continue;
      bp.n_sub = d;
      if (base_items * d >= 2ll * num_sms) break;
    }
  }
  bp.heads_per_sub = bp.group / bp.n_sub;
  // One query head per key/value head and at most one round of items: the first key tiles, which
  // meet every query tile, set the time.  Divide the query tiles of every key tile over two items
  // (two shares add up the same in either order, so dK, dV stay bit-reproducible).
  bp.i_split = 1;
  {
    const long long base_items = static_cast<long long>(bp.n_tiles_k) * bp.BH;
    const bool square = p.key_rows() == p.N && p.query_pos0() == 0;
    if (bp.group == 1 && square && p.seqlens == nullptr && p.cu_seqlens == nullptr && bp.n_tiles >= 4 &&
        (2 * base_items <= num_sms || (p.causal && base_items <= num_sms && bp.n_tiles >= 16)))
      bp.i_split = 2;
  }
  bp.dkv_add = p.acc_only == 2 ? 1 : 0;
  bp.n_items = bp.n_tiles_k * bp.BH * bp.n_sub * bp.i_split;
  bp.scale = p.scale;
  bp.scale_log2e = p.scale * kLog2eB;
  bp.bias_log2e = p.bias * kLog2eB;
  bp.bias_vec = p.bias_vec;
  bp.dbias = p.dbias;
  bp.slopes = p.slopes;
  bp.seqlens = p.seqlens;
  bp.cu_seqlens = p.cu_seqlens;
  bp.n_seqs = p.n_seqs;
  bp.sched_counter = nullptr;
  bp.status = status;

  const size_t n_elems = static_cast<size_t>(BH) * p.N * p.D;
  if ((bp.n_sub > 1 || bp.i_split > 1) && !bp.dkv_add) {   // dK, dV are summed over the parts: clear them first
    const size_t kv_bytes = static_cast<size_t>(BH_kv) * p.key_rows() * p.D * 2;
    *cuda_err = cudaMemsetAsync(dk, 0, kv_bytes, stream);
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
    *cuda_err = cudaMemsetAsync(dv, 0, kv_bytes, stream);
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  }
  // step 1: clear the fp32 dQ accumulator (and the bias gradient, which the kernel adds into);
  // with acc_only the accumulator is the caller's running sum over key/value shards: not cleared
  if (!p.acc_only) {
    *cuda_err = cudaMemsetAsync(workspace, 0, n_elems * sizeof(float), stream);
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  }
  if (p.dbias != nullptr) {
    const size_t n_bias = p.cu_seqlens != nullptr ? static_cast<size_t>(p.n_seqs) * p.H : BH;
    *cuda_err = cudaMemsetAsync(p.dbias, 0, n_bias * sizeof(float), stream);
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  }

  if (p.cu_seqlens != nullptr) {
    static std::atomic<unsigned> next_slot{0};
    int* counters = nullptr;
    *cuda_err = cudaGetSymbolAddress(reinterpret_cast<void**>(&counters), g_bwd_sched_counters);
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
    bp.sched_counter = counters + next_slot.fetch_add(1) % kBwdSchedSlots;
    *cuda_err = cudaMemsetAsync(bp.sched_counter, 0, sizeof(int), stream);
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  }
  if (p.row_scale != nullptr) {
    const size_t n_vec8 = n_elems / 8;
    const size_t want = n_vec8 / 256 + 1, cap = static_cast<size_t>(num_sms) * 8;
    sigattn_bwd_scale_rows_kernel<<<static_cast<int>(want < cap ? want : cap), 256, 0, stream>>>(
        static_cast<const uint4*>(d_o), p.row_scale, static_cast<uint4*>(dq), n_vec8, p.N, p.D / 8);
    *cuda_err = cudaGetLastError();
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
    *launches += 1;
  }

  // step 2: main kernel
  const bool timed = (t_ev_start != nullptr && t_ev_stop != nullptr);
  if (timed) cudaEventRecord(t_ev_start, stream);
  int rc;
  const bool alibi = p.slopes != nullptr;
  // the bias gradient costs the activation groups a running sum (4-5 % of the kernel), so it
  // is compiled in only where it is asked for; likewise the loop over a group's query heads and
  // the per-sequence lengths (kind 1) and the lookups of a batch without padding (kind 2)
#define SIGATTN_BWD_KIND(DD, CC, AA, KK)                                                                   \
  ((p.dbias != nullptr) ? launch_bwd_variant<DD, CC, AA, true, KK>(maps, bp, num_sms, stream, cuda_err)    \
                        : launch_bwd_variant<DD, CC, AA, false, KK>(maps, bp, num_sms, stream, cuda_err))
#define SIGATTN_BWD_CASE(DD, CC, AA)                                                                       \
  rc = (bp.cu_seqlens != nullptr)                  ? SIGATTN_BWD_KIND(DD, CC, AA, 2)                        \
       : (bp.group > 1 || bp.seqlens != nullptr || bp.i_split > 1 || bp.dkv_add) ? SIGATTN_BWD_KIND(DD, CC, AA, 1) \
                                                   : SIGATTN_BWD_KIND(DD, CC, AA, 0)
  if (p.D == 128) {
    if (p.causal) { if (alibi) SIGATTN_BWD_CASE(128, true, true); else SIGATTN_BWD_CASE(128, true, false); }
    else          { if (alibi) SIGATTN_BWD_CASE(128, false, true); else SIGATTN_BWD_CASE(128, false, false); }
  } else {
    if (p.causal) { if (alibi) SIGATTN_BWD_CASE(64, true, true); else SIGATTN_BWD_CASE(64, true, false); }
    else          { if (alibi) SIGATTN_BWD_CASE(64, false, true); else SIGATTN_BWD_CASE(64, false, false); }
  }
#undef SIGATTN_BWD_CASE
#undef SIGATTN_BWD_KIND
  if (rc != SIGATTN_OK) return rc;
  if (timed) cudaEventRecord(t_ev_stop, stream);
  *launches += 1;

  if (p.acc_only) return SIGATTN_OK;   // the owner of the accumulator converts once every shard has added

  // step 3: dQ = scale * accumulator, as bf16 (and, on request, the temperature gradient from the same pass)
  const size_t n_vec4 = n_elems / 4;  // D is a multiple of 64
  if (p.dtemp != nullptr) {
    *cuda_err = cudaMemsetAsync(p.dtemp, 0, BH * sizeof(float), stream);
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
    const size_t per_head = static_cast<size_t>(p.N) * p.D / 4;
    const size_t want = per_head / 256 + 1, cap = (static_cast<size_t>(num_sms) * 8 + BH - 1) / BH;
    dim3 grid(static_cast<unsigned>(want < cap ? want : (cap < 1 ? 1 : cap)), static_cast<unsigned>(BH));
    sigattn_bwd_convert_dq_dtemp_kernel<<<grid, 256, 0, stream>>>(static_cast<const float4*>(workspace),
                                                                  static_cast<const uint2*>(q), static_cast<uint2*>(dq),
                                                                  per_head, p.scale, p.dtemp);
    *cuda_err = cudaGetLastError();
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
    *launches += 1;
    return SIGATTN_OK;
  }
  const int blocks = static_cast<int>(n_vec4 / 256 + 1 < static_cast<size_t>(num_sms) * 8 ? n_vec4 / 256 + 1
                                                                                            : static_cast<size_t>(num_sms) * 8);
  sigattn_bwd_convert_dq_kernel<<<blocks, 256, 0, stream>>>(static_cast<const float4*>(workspace),
                                                            static_cast<uint2*>(dq), n_vec4, p.scale);
  *cuda_err = cudaGetLastError();
  if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  *launches += 1;
  return SIGATTN_OK;
}

}  // namespace sigattn
