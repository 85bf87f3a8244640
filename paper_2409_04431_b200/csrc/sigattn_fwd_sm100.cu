// bf16 forward of sigmoid attention for sm_100a (Algorithm 1 of Appendix F.1, redesigned
// for Blackwell): O = sigmoid(scale * Q K^T + b - slope * |i - j|) [causal-masked] V.
//
// One persistent CTA per SM walks a list of work items (batch*head, pair of 128-row query
// tiles), heaviest first when causal.  Inside a CTA the work is split by warp role:
//
//   warp 16     TMA producer: Q tiles once per item, then K_0, V_0, K_1, V_1, ... through a
//               ring of shared-memory stages (128-byte swizzle, zero fill beyond row N).
//   warp 17     MMA issuer (one thread): S_t = Q_t K_j^T into tensor memory, then
//               O_t += P_t V_j with P read from tensor memory.  The two query tiles are
//               interleaved so the tensor pipe works on one while the other is activated.
//   warps 0-15  activation: threads read S from tensor memory (one row each), evaluate
//               P = sigmoid(.) in registers and write bf16 P back over S.  All 512 threads
//               work on one query tile (32 key columns each) and alternate between the two
//               tiles, so the MUFU pipe and the tensor pipe take turns on a tile.  Sixteen
//               warps rather than eight: the activation is bound by the latency of its
//               dependent chain (tensor-memory load, exponential, polynomial, store), and
//               four warps per scheduler hide it better than two (measured +3 % at D = 128,
//               +15 % at D = 64).  At the end of an item they convert the O accumulators to
//               bf16 and store them with TMA (rows >= N are clipped).
//
// Sigmoid needs no row maximum, no row sum and no rescaling of O (Section 4), so there is
// no correction step and O is touched once, at the end.
//
// Activation: P = u / (1 + u) with u = 2^(log2(e) x), one MUFU op per element in the
// common case; see sigattn_activation.cuh for the evaluation and for why the paper's
// tanh form is not used.
#include <atomic>

#include "sigattn_internal.h"
#include "sigattn_activation.cuh"
#include "sm100_primitives.cuh"
#include "tensor_map.h"
#include "../../include/sigattn.h"

namespace sigattn {
namespace {

using namespace sm100;

constexpr int kBM = 128;        // query rows per tile (= TMEM lanes)
constexpr int kBN = 128;        // keys per tile
// This file is compiled in two shapes.  The default is the one described above (two query tiles per work
// item, sixteen activation warps, one thread block per SM).  With SIGATTN_FWD_TILES = 1 a work item is a
// single query tile, there are eight activation warps, and two thread blocks share an SM (256 columns of
// tensor memory and under half of the shared memory each): the tile's own steps run one after the other
// (logits, activation, P V), and the overlap of tensor and MUFU work comes from the other thread block,
// which also hides a work item's start and end.  That shape serves short sequences (see the launcher).
#ifndef SIGATTN_FWD_TILES
#define SIGATTN_FWD_TILES 2
#endif
constexpr int kTiles = SIGATTN_FWD_TILES;
static_assert(kTiles == 1 || kTiles == 2, "query tiles per work item");
#ifndef SIGATTN_FWD_ACT_WARPS
#define SIGATTN_FWD_ACT_WARPS (SIGATTN_FWD_TILES == 2 ? 16 : 8)
#endif
constexpr int kActWarps = SIGATTN_FWD_ACT_WARPS;   // 8 or 16
constexpr int kActThreads = 32 * kActWarps;
constexpr int kGroups = kActWarps / 4;             // column groups of a tile
constexpr int kCols = kBN / kGroups;               // key columns per activation thread
constexpr int kRun = kCols > 32 ? 32 : kCols;      // of which it holds this many in registers at a time
constexpr int kFwdThreads = kActThreads + 64;
constexpr int kLoadWarp = kActWarps;
constexpr int kMmaWarp = kActWarps + 1;
constexpr float kLog2e = 1.4426950408889634f;
constexpr uint32_t kTmemCols = 256 * kTiles;       // per tile: 128 columns of logits / P, up to 128 of O
constexpr int kCtasPerSm = (kTiles == 1) ? 2 : 1;

// Share of the forward's exponentials evaluated on the FMA pipe (every m-th, 0 = none).
// At D = 128 the shorter instruction stream wins (emulating every 4th measured -6 %); at
// D = 64, where a tile step has half the tensor work per exponential, unloading the MUFU
// pipe gains 1-3 % with a causal mask (N = 2048 and 8192) and loses 3-5 % without one
// (N = 2048 and 8100), so only the causal instantiations do it.
#ifndef SIGATTN_FWD_EMULATE_D64
#define SIGATTN_FWD_EMULATE_D64 8
#endif
#ifndef SIGATTN_FWD_EMULATE_D64_UNMASKED
#define SIGATTN_FWD_EMULATE_D64_UNMASKED 0
#endif
#ifndef SIGATTN_FWD_EMULATE_D128
#define SIGATTN_FWD_EMULATE_D128 0
#endif


template <int D>
struct FwdSmem {
  static constexpr int kPanels = D / 64;
  static constexpr int kPanelBytes = kBM * 128;           // 128 rows x 128 B
  static constexpr int kTileBytes = kPanels * kPanelBytes;  // one Q, K or V tile
  // K/V ring; the single-tile shape must fit two thread blocks into an SM's shared memory
  static constexpr int kStages = (kTiles == 2) ? ((D == 128) ? 4 : 8) : ((D == 128) ? 2 : 4);
  static constexpr int kQOff = 0;
  static constexpr int kKvOff = kTiles * kTileBytes;
  // At D = 64 there is room for a staging buffer of O of its own: the Q buffer is then free as soon
  // as the item's last logits are computed, and the next item's Q load runs under the last activation,
  // the last P V and the epilogue.  At D = 128 O is staged in the Q buffer (shared memory is full).
  static constexpr bool kOStaged = (D == 64);
  static constexpr int kOOff = kKvOff + kStages * kTileBytes;
  static constexpr int kTotal = kOOff + (kOStaged ? kTiles * kTileBytes : 0);
  static constexpr int kDynBytes = kTotal + 1024;  // slack to align the base to 1024 B
};

struct FwdBarriers {
  uint64_t q_full[2], q_empty[2];
  uint64_t s_full[2], p_full[2];
  uint64_t o_full[2], o_empty[2];
  uint64_t kv_full[8], kv_empty[8];
  // dynamic schedule (batches without padding): the TMA thread draws the next work item from a
  // global counter and hands it to the other roles through this two-slot ring
  uint64_t sched_full[2], sched_empty[2];
  int sched_item[2];
};

struct FwdParams {
  int BH, H, N;     // N counts query rows
  int pos0;         // position of query row 0 relative to key row 0: rows of K, V minus N when the
                    // queries are the last positions (0 for self-attention); any value for a shard
  int H_kv, group;  // heads of K, V and query heads per key/value head (H = H_kv * group)
  // Packed grouped heads (few queries per head, e.g. decoding): the rows of all `pack_group`
  // query heads of one key/value head form ONE sequence of pack_group * pack_rows rows, row r
  // belonging to head r / pack_rows, query r % pack_rows, so that K and V are streamed once per
  // group instead of once per query head.  Then BH counts (batch, key/value head) pairs, N is
  // pack_group * pack_rows and H = H_kv, group = 1 for the producer.  0 = not packed.
  int pack_rows, pack_group;
  const int* seqlens;   // padded batch: valid length per batch entry (keys and queries), or nullptr
  const float* row_scale;   // one factor per query row applied to O, or nullptr
  // Batch stored without padding (B = 1): sequence s owns rows [cu_seqlens[s], cu_seqlens[s + 1]) of
  // Q, K and V and attends only within them; bias_vec then holds one bias per (sequence, head).
  const int* cu_seqlens;    // n_seqs + 1 row offsets, or nullptr
  int n_seqs;
  int* sched_counter;       // dynamic schedule: next work item to hand out (zero at launch), or nullptr
  int n_pairs;     // work items per head: ceil(N / (128 kTiles))
  int n_kv_total;  // ceil(N / 128)
  // Keys split over several work items (packed mode only; decoding has too few (batch, head)
  // pairs to fill the GPU): split s of a (head, pair) visits key tiles [s, s + 1) * tiles_per_split
  // and adds its partial O, in fp32, into split_ws [BH, N, D]; there is no row normalisation, so
  // the partial results simply add up.  n_splits = 1: off.
  int n_splits, tiles_per_split;
  float* split_ws;
  int o_reduce;    // 1: split items of the unpacked general mode add bf16 tiles into O instead of storing them
  int n_items;
  float scale_log2e, bias_log2e;
  const float* bias_vec;   // one bias per (batch, head) instead of the scalar, or nullptr
  const float* slopes;
  int* status;
};

struct Item {
  int bh, row0, n_kv, n[2];
  int j0;        // first key tile of the item (0 unless the keys are split)
  int n_valid;   // rows of this sequence that count (N unless the batch is padded)
};

// Work items are ranked by decreasing cost (causal: later query tiles see more keys).
// Round r of the persistent loop hands ranks [r G, (r + 1) G) to the G CTAs, forwards in
// even rounds and backwards in odd rounds, so a CTA that drew an expensive item in one
// round draws a cheap one in the next (a static stand-in for longest-first scheduling).
__device__ __forceinline__ int snake_rank(int round, int n_items) {
  const int g = gridDim.x;
  const int c = (round & 1) ? (g - 1 - static_cast<int>(blockIdx.x)) : static_cast<int>(blockIdx.x);
  const int rank = round * g + c;
  return rank < n_items ? rank : -1;
}

__device__ __forceinline__ int num_rounds(int n_items) { return (n_items + gridDim.x - 1) / gridDim.x; }

// Dynamic schedule.  The static snake order balances the CTAs only if the items' costs fall with
// their rank.  In a padded batch the cost of an item also depends on the length of its sequence,
// and in a batch without padding the cost of a causal item follows its position inside its own
// sequence, a sawtooth over the rows.  The general instantiations therefore draw their items from
// a global counter instead, in row order from the last row down (every sequence then hands out
// its expensive items first, and the cheap starts come last).  One thread per CTA draws; the other
// roles read the item from a two-slot ring in shared memory.  Returns false when a bounded wait
// expired; *item < 0 means no items are left.
constexpr int kSchedConsumers = 32 + kActThreads;   // the MMA warp and the activation threads
__device__ __forceinline__ bool sched_draw(const FwdParams& p, FwdBarriers* bars, int round, int* item,
                                           volatile int* cta_err) {
  const uint32_t slot = round & 1, phase = (round >> 1) & 1;
  if (!mbar_wait(smem_u32(&bars->sched_empty[slot]), phase ^ 1, cta_err, 40)) return false;
  int it = atomicAdd(p.sched_counter, 1);
  // every thread block draws until its first value >= n_items, so one launch draws n_items + gridDim.x
  // values in all; a larger value means another launch in flight shares the counter (more launches
  // overlapping than the library has counters): report it instead of silently skipping or repeating items
  if (it >= p.n_items + static_cast<int>(gridDim.x)) *cta_err = 46;
  if (it >= p.n_items) it = -1;
  *reinterpret_cast<volatile int*>(&bars->sched_item[slot]) = it;
  mbar_arrive(smem_u32(&bars->sched_full[slot]));
  *item = it;
  return true;
}
__device__ __forceinline__ bool sched_take(FwdBarriers* bars, int round, int* item, volatile int* cta_err) {
  const uint32_t slot = round & 1, phase = (round >> 1) & 1;
  if (!mbar_wait(smem_u32(&bars->sched_full[slot]), phase, cta_err, 41)) return false;
  *item = *reinterpret_cast<volatile int*>(&bars->sched_item[slot]);
  mbar_arrive(smem_u32(&bars->sched_empty[slot]));
  return true;
}

// Sequence that owns `row` in a batch stored without padding: the largest s with cu[s] <= row
// (0 <= row < cu[n_seqs]; empty sequences own no row).
__device__ __forceinline__ int seq_of_row(const int* __restrict__ cu, int n_seqs, int row) {
  int lo = 0, hi = n_seqs;   // cu[lo] <= row < cu[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (__ldg(cu + mid) <= row) lo = mid; else hi = mid;
  }
  return lo;
}

template <bool CAUSAL>
__device__ __forceinline__ Item decode_item(const FwdParams& p, int item) {
  Item w;
  int rank = item / p.BH;
  w.bh = item - rank * p.BH;
  const int split = rank / p.n_pairs;   // 0 unless the keys are split
  rank -= split * p.n_pairs;
  const int pair = CAUSAL ? (p.n_pairs - 1 - rank) : rank;
  w.row0 = pair * kTiles * kBM;
  w.n_valid = p.seqlens ? max(0, min(p.N, __ldg(p.seqlens + w.bh / p.H))) : p.N;
  const int n_kv_valid = p.seqlens ? max(1, (w.n_valid + kBN - 1) / kBN) : p.n_kv_total;
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    const int r = w.row0 + t * kBM;
    // causal: the tile's last row, at position r + 127 + pos0, sees keys up to that position
    // (packed rows: every tile holds last queries of some head, so every key tile is visited)
    w.n[t] = (t >= kTiles || r >= p.N) ? 0
             : ((CAUSAL && p.pack_rows == 0)
                    // (a tile that lies before every key still visits one key tile, fully masked: zeros)
                    ? ((r + kBM - 1 + p.pos0 < 0) ? 1 : min(n_kv_valid, (r + kBM - 1 + p.pos0) / kBN + 1))
                    : n_kv_valid);
    // (a tile of a padded batch that lies past the sequence's end visits one key tile, fully masked)
    if (p.seqlens && r < p.N && r >= w.n_valid) w.n[t] = 1;
  }
  w.j0 = 0;
  if (p.cu_seqlens != nullptr) {
    // Batch without padding: a tile's rows see keys from the start of its first row's sequence to
    // the end of its last row's sequence (causal: to its last row).  Both tiles of the item walk
    // the same key tiles, starting where tile 0's keys start; what lies outside a row's own
    // sequence is masked row by row.
    // (offsets that do not rise from 0 to N give wrong results, but the clamps keep every loop bounded)
    w.j0 = max(0, min(p.n_kv_total - 1, __ldg(p.cu_seqlens + seq_of_row(p.cu_seqlens, p.n_seqs, w.row0)) / kBN));
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      const int r_first = w.row0 + t * kBM;
      if (t >= kTiles || r_first >= p.N) { w.n[t] = 0; continue; }
      const int r_last = min(p.N, r_first + kBM) - 1;
      const int key_end = CAUSAL ? r_last + 1 : __ldg(p.cu_seqlens + seq_of_row(p.cu_seqlens, p.n_seqs, r_last) + 1);
      w.n[t] = max(1, min(p.n_kv_total, (key_end + kBN - 1) / kBN) - w.j0);
    }
  }
  if (p.n_splits > 1 && p.pack_rows > 0) {   // packed mode: every valid tile visits all key tiles; this item takes its share
    w.j0 = split * p.tiles_per_split;
    const int n = min(p.tiles_per_split, p.n_kv_total - w.j0);
#pragma unroll
    for (int t = 0; t < 2; ++t) w.n[t] = w.n[t] > 0 ? n : 0;
  } else if (p.n_splits > 1) {
    // Few work items (one long causal sequence, few heads): the key tiles of an item are divided
    // over n_splits items that add their shares of O.  Tile 1 of a pair sees as many key tiles as
    // tile 0 or one more; both must stay non-empty in every part, so the parts are cut by tile 0's
    // count.  Items too short to cut go to part 0 whole; their other parts visit one key tile past
    // the diagonal, which is fully masked (or out of range and read as zeros), and add zeros.
    const int n0 = w.n[0], n1 = w.n[1];
    if (n0 >= 2 * p.n_splits && (n1 == 0 || n1 >= n0)) {
      // part s takes key tiles [s n0 / S, (s + 1) n0 / S): never empty since n0 >= 2 S; the last
      // part of tile 1 runs on to n1
      const int first = split * n0 / p.n_splits, end = (split + 1) * n0 / p.n_splits;
      const bool last = split == p.n_splits - 1;
      w.j0 = first;
      w.n[0] = end - first;
      w.n[1] = n1 == 0 ? 0 : (last ? n1 : end) - first;
    } else if (split > 0) {
      w.j0 = max(n0, n1);
      w.n[0] = n0 > 0 ? 1 : 0;
      w.n[1] = n1 > 0 ? 1 : 0;
    }
  }
  w.n_kv = max(w.n[0], w.n[1]);
  return w;
}

// ------------------------------------------------------------------ producer

template <int D, bool CAUSAL, bool DYNAMIC>
__device__ void fwd_load_role(const FwdParams& p, const CUtensorMap* tmQ, const CUtensorMap* tmK,
                              const CUtensorMap* tmV, uint32_t smem_base, FwdBarriers* bars, volatile int* cta_err) {
  using L = FwdSmem<D>;
  uint32_t kv_cnt = 0;
  uint32_t q_iter[2] = {0, 0};
  for (int round = 0, rounds = num_rounds(p.n_items); DYNAMIC || round < rounds; ++round) {
    int item;
    if (DYNAMIC) {
      if (!sched_draw(p, bars, round, &item, cta_err)) return;
      if (item < 0) break;
    } else {
      item = snake_rank(round, p.n_items);
      if (item < 0) continue;
    }
    const Item w = decode_item<CAUSAL>(p, item);
    const int bh_kv = (w.bh / p.H) * p.H_kv + (w.bh % p.H) / p.group;   // the key/value head this query head reads
    auto load_q = [&](int t) -> bool {
      if (w.n[t] == 0) return true;
      if (!mbar_wait(smem_u32(&bars->q_empty[t]), (q_iter[t] & 1) ^ 1, cta_err, 10 + t)) return false;
      const uint32_t bar = smem_u32(&bars->q_full[t]);
      mbar_arrive_expect_tx(bar, L::kTileBytes);
#pragma unroll
      for (int pn = 0; pn < L::kPanels; ++pn)
        tma_load_3d(smem_base + L::kQOff + t * L::kTileBytes + pn * L::kPanelBytes, tmQ, bar, pn * 64,
                    w.row0 + t * kBM, w.bh);
      ++q_iter[t];
      return true;
    };
    auto load_kv = [&](const CUtensorMap* tm, int j) -> bool {
      const uint32_t stage = kv_cnt % L::kStages;
      const uint32_t phase = (kv_cnt / L::kStages) & 1;
      if (!mbar_wait(smem_u32(&bars->kv_empty[stage]), phase ^ 1, cta_err, 12)) return false;
      const uint32_t bar = smem_u32(&bars->kv_full[stage]);
      mbar_arrive_expect_tx(bar, L::kTileBytes);
#pragma unroll
      for (int pn = 0; pn < L::kPanels; ++pn)
        tma_load_3d(smem_base + L::kKvOff + stage * L::kTileBytes + pn * L::kPanelBytes, tm, bar, pn * 64,
                    (w.j0 + j) * kBN, bh_kv);
      ++kv_cnt;
      return true;
    };
    if (!load_q(0)) return;
    if (!load_kv(tmK, 0)) return;
    if (!load_q(1)) return;
    for (int j = 0; j < w.n_kv; ++j) {
      if (!load_kv(tmV, j)) return;
      if (j + 1 < w.n_kv && !load_kv(tmK, j + 1)) return;
    }
  }
}

// ------------------------------------------------------------------ MMA issuer

template <int D, bool CAUSAL, bool DYNAMIC>
__device__ void fwd_mma_role(const FwdParams& p, uint32_t smem_base, uint32_t tmem, FwdBarriers* bars,
                             volatile int* cta_err) {
  using L = FwdSmem<D>;
  constexpr uint32_t kIdescS = make_idesc_bf16(kBM, kBN, 0, 0);
  constexpr uint32_t kIdescPV = make_idesc_bf16(kBM, D, 0, 1);
  const uint32_t leader = (threadIdx.x & 31) == 0;   // the lane that issues; all lanes run the loop
  uint32_t kv_cnt = 0;
  uint32_t it[2] = {0, 0};      // items seen per query tile
  uint32_t p_cnt[2] = {0, 0};   // P tiles consumed per query tile

  // Descriptors are built once per operand tile; each k-step only advances the start address.
  const uint64_t q_desc[2] = {make_smem_desc_sw128(smem_base + L::kQOff, 16, 1024),
                              make_smem_desc_sw128(smem_base + L::kQOff + L::kTileBytes, 16, 1024)};
  // S_t = Q_t K^T : both operands K-major, 128-byte swizzle.
  auto issue_s = [&](int t, uint32_t k_smem) {
    const uint64_t qd = q_desc[t];
    const uint64_t kd = make_smem_desc_sw128(k_smem, 16, 1024);
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
      const uint32_t off = (ks >> 2) * L::kPanelBytes + (ks & 3) * 32;
      umma_ss_warp(leader, tmem + t * kBN, desc_advance(qd, off), desc_advance(kd, off), kIdescS, ks > 0);
    }
  };
  // O_t (+)= P_t V : A = bf16 P in tensor memory (aliasing S_t), B = V, MN-major.
  auto issue_pv = [&](int t, uint32_t v_smem, bool accumulate) {
    const uint64_t vd = make_smem_desc_sw128(v_smem, L::kPanelBytes, 1024);
#pragma unroll
    for (int ks = 0; ks < kBN / 16; ++ks) {
      // column group c wrote its bf16 P over the first half of its own logits columns:
      // [c kCols, c kCols + kCols / 2), one k-step of 16 keys per 8 columns
      const uint32_t p_col = (ks / (kCols / 16)) * kCols + (ks % (kCols / 16)) * 8;
      umma_ts_warp(leader, tmem + kTiles * kBN + t * D, tmem + t * kBN + p_col, desc_advance(vd, ks * 2048), kIdescPV,
              (accumulate || ks > 0));
    }
  };
  auto kv_wait = [&](uint32_t cnt) -> bool {
    const uint32_t stage = cnt % L::kStages, phase = (cnt / L::kStages) & 1;
    return mbar_wait(smem_u32(&bars->kv_full[stage]), phase, cta_err, 20);
  };
  auto kv_addr = [&](uint32_t cnt) { return smem_base + L::kKvOff + (cnt % L::kStages) * L::kTileBytes; };
  auto kv_release = [&](uint32_t cnt) { umma_commit_warp(leader, smem_u32(&bars->kv_empty[cnt % L::kStages])); };

  for (int round = 0, rounds = num_rounds(p.n_items); DYNAMIC || round < rounds; ++round) {
    int item;
    if (DYNAMIC) {
      if (!sched_take(bars, round, &item, cta_err)) return;
      if (item < 0) break;
    } else {
      item = snake_rank(round, p.n_items);
      if (item < 0) continue;
    }
    const Item w = decode_item<CAUSAL>(p, item);
    // ring positions: K_j at kv_cnt + 2 j (j > 0: 2 j), V_j right after K_j ... order K0 V0 K1 V1 ...
    const uint32_t base_cnt = kv_cnt;
    auto k_cnt = [&](int j) { return base_cnt + 2 * j; };
    auto v_cnt = [&](int j) { return base_cnt + 2 * j + 1; };

    // first logits
    if (!mbar_wait(smem_u32(&bars->q_full[0]), it[0] & 1, cta_err, 21)) return;
    if (!kv_wait(k_cnt(0))) return;
    tc_fence_after_sync();
    issue_s(0, kv_addr(k_cnt(0)));
    umma_commit_warp(leader, smem_u32(&bars->s_full[0]));
    if (L::kOStaged && w.n[0] == 1) umma_commit_warp(leader, smem_u32(&bars->q_empty[0]));   // Q_0 no longer needed
    if (w.n[1] > 0) {
      if (!mbar_wait(smem_u32(&bars->q_full[1]), it[1] & 1, cta_err, 22)) return;
      tc_fence_after_sync();
      issue_s(1, kv_addr(k_cnt(0)));
      umma_commit_warp(leader, smem_u32(&bars->s_full[1]));
      if (L::kOStaged && w.n[1] == 1) umma_commit_warp(leader, smem_u32(&bars->q_empty[1]));
    }
    kv_release(k_cnt(0));
    // accumulators of the previous item must have been read out before the first PV overwrites them
    if (!mbar_wait(smem_u32(&bars->o_empty[0]), (it[0] & 1) ^ 1, cta_err, 23)) return;
    if (w.n[1] > 0 && !mbar_wait(smem_u32(&bars->o_empty[1]), (it[1] & 1) ^ 1, cta_err, 24)) return;

    for (int j = 0; j < w.n_kv; ++j) {
      if (!kv_wait(v_cnt(j))) return;
      const bool more = (j + 1 < w.n_kv);
      if (j < w.n[0]) {
        if (!mbar_wait(smem_u32(&bars->p_full[0]), p_cnt[0] & 1, cta_err, 25)) return;
        ++p_cnt[0];
        tc_fence_after_sync();
        issue_pv(0, kv_addr(v_cnt(j)), j > 0);
        if (j == w.n[0] - 1) umma_commit_warp(leader, smem_u32(&bars->o_full[0]));
      }
      if (more && !kv_wait(k_cnt(j + 1))) return;
      if (j + 1 < w.n[0]) {
        tc_fence_after_sync();
        issue_s(0, kv_addr(k_cnt(j + 1)));
        umma_commit_warp(leader, smem_u32(&bars->s_full[0]));
        if (L::kOStaged && j + 2 == w.n[0]) umma_commit_warp(leader, smem_u32(&bars->q_empty[0]));
      }
      if (j < w.n[1]) {
        if (!mbar_wait(smem_u32(&bars->p_full[1]), p_cnt[1] & 1, cta_err, 26)) return;
        ++p_cnt[1];
        tc_fence_after_sync();
        issue_pv(1, kv_addr(v_cnt(j)), j > 0);
        if (j == w.n[1] - 1) umma_commit_warp(leader, smem_u32(&bars->o_full[1]));
      }
      kv_release(v_cnt(j));
      if (j + 1 < w.n[1]) {
        issue_s(1, kv_addr(k_cnt(j + 1)));
        umma_commit_warp(leader, smem_u32(&bars->s_full[1]));
        if (L::kOStaged && j + 2 == w.n[1]) umma_commit_warp(leader, smem_u32(&bars->q_empty[1]));
      }
      if (more) kv_release(k_cnt(j + 1));
    }
    kv_cnt = base_cnt + 2 * w.n_kv;
    ++it[0];
    if (w.n[1] > 0) ++it[1];
  }
}

// ------------------------------------------------------------------ activation + epilogue

template <int N>
__device__ __forceinline__ void tmem_ld_cols(uint32_t addr, uint32_t (&v)[N]) {
  static_assert(N == 16 || N == 32 || N == 64, "columns per thread");
  if constexpr (N == 16) {
    tmem_ld16(addr, v);
  } else {
#pragma unroll
    for (int c = 0; c < N / 32; ++c) tmem_ld32(addr + c * 32, *reinterpret_cast<uint32_t (*)[32]>(&v[c * 32]));
  }
}
template <int N>
__device__ __forceinline__ void tmem_st_cols(uint32_t addr, uint32_t (&v)[N]) {
  static_assert(N == 16 || N == 32, "packed columns per thread");
  if constexpr (N == 16) tmem_st16(addr, v); else tmem_st32(addr, v);
}

// NC logits of one row -> NC / 2 packed bf16x2 sigmoid values.
//   a = s * scale_log2e + c0   (c0 carries the bias and, with ALiBi, the position term)
// CAUSAL: every key that keeps its weight sits at or before the query, so |i - j| = i - j there and the
// position term is linear in the column: one FMA per logit from a per-call constant instead of a
// difference and an FMA with |.| (what a masked key gets instead is blanked afterwards).
template <int NC, bool ALIBI, bool CAUSAL, int EMULATE_EVERY, bool TWO_SIDED = false>
__device__ __forceinline__ void sigmoid_cols(const uint32_t (&s)[NC], uint32_t (&out)[NC / 2],
                                             float scale_log2e, float bias_log2e, float slope_log2e, float row_rel,
                                             int col_base, bool masked, float mask_limit, float mask_first = 0.0f) {
  float a[NC];
  const float c_first = fmaf(-slope_log2e, row_rel - static_cast<float>(col_base), bias_log2e);   // column col_base
#pragma unroll
  for (int i = 0; i < NC; ++i) {
    float c0 = bias_log2e;
    if (ALIBI && CAUSAL) {
      c0 = fmaf(slope_log2e, static_cast<float>(i), c_first);
    } else if (ALIBI) {
      const float dist = row_rel - static_cast<float>(col_base + i);
      c0 = fmaf(-slope_log2e, fabsf(dist), bias_log2e);
    }
    a[i] = fmaf(__uint_as_float(s[i]), scale_log2e, c0);
  }
  float pr[NC];
  sigmoid_block<NC, false, EMULATE_EVERY>(a, pr, nullptr);
  if (masked) {  // keys after the query (and, in a padded batch, past the sequence's end) get weight 0
#pragma unroll
    for (int i = 0; i < NC; ++i)
      if (static_cast<float>(col_base + i) > mask_limit ||
          (TWO_SIDED && static_cast<float>(col_base + i) < mask_first))   // keys before the row's own sequence
        pr[i] = 0.0f;
  }
#pragma unroll
  for (int i = 0; i < NC / 2; ++i) out[i] = pack_bf16x2(pr[2 * i], pr[2 * i + 1]);
}

// All activation threads work on the same query tile at a time, alternating between the
// two tiles of the item: thread (g, r) owns row r and key columns [kCols g, kCols g + kCols)
// of the tile.  While the groups evaluate one tile, the tensor pipe runs
// P V and the next logits of the other one, so the MUFU pipe and the tensor pipe take turns
// on a tile instead of competing for it.
// MODE: 0 plain (the benchmarked path), 1 packed grouped heads, 2 general: padded batch with
// per-sequence lengths, one output factor per query row, accumulation into an fp32 buffer, each
// asked for at run time; 3 = 2 plus a batch stored without padding (row offsets per sequence)
template <int D, bool CAUSAL, bool ALIBI, int MODE>
__device__ void fwd_act_role(const FwdParams& p, const CUtensorMap* tmO, uint8_t* smem, uint32_t tmem,
                             FwdBarriers* bars, volatile int* cta_err) {
  using L = FwdSmem<D>;
  constexpr bool PACKED = (MODE == 1), GENERAL = (MODE >= 2);
  const bool varlen = GENERAL && p.seqlens != nullptr;
  constexpr bool ragged = (MODE == 3);
  const int g = threadIdx.x >> 7;            // column group of the tile
  const int tid = threadIdx.x & 127;         // row of the tile
  const uint32_t lane_off = static_cast<uint32_t>(((threadIdx.x >> 5) & 3) * 32) << 16;
  uint32_t s_cnt0 = 0, s_cnt1 = 0, it[2] = {0, 0};

  constexpr bool DYNAMIC = (MODE >= 2);
  for (int round = 0, rounds = num_rounds(p.n_items); DYNAMIC || round < rounds; ++round) {
    int item;
    if (DYNAMIC) {
      if (!sched_take(bars, round, &item, cta_err)) return;
      if (item < 0) break;
    } else {
      item = snake_rank(round, p.n_items);
      if (item < 0) continue;
    }
    const Item w = decode_item<CAUSAL>(p, item);
    // Slope, bias and the position of this thread's query row: per item, or with packed heads
    // per row and tile (index 1 of the arrays is only used then).
    float slope_t[2] = {0.0f, 0.0f}, bias_t[2];
    int pos_t[2];   // positions stay integers: shards of very long sequences put them beyond 2^24
    if (PACKED) {
#pragma unroll
      for (int t = 0; t < kTiles; ++t) {
        const int r = w.row0 + t * kBM + tid;
        const int g_head = min(r / p.pack_rows, p.pack_group - 1);   // rows past the end only fill the tile
        const int head = w.bh * p.pack_group + g_head;               // (b * H_kv + h_kv) * group + g = b * H + h
        if (ALIBI) slope_t[t] = p.slopes[head % (p.H * p.pack_group)] * kLog2e;
        bias_t[t] = p.bias_vec ? __ldg(p.bias_vec + head) * kLog2e : p.bias_log2e;
        pos_t[t] = r - g_head * p.pack_rows + p.pos0;
      }
    } else {
      if (ALIBI) slope_t[0] = p.slopes[w.bh % p.H] * kLog2e;
      bias_t[0] = p.bias_vec ? __ldg(p.bias_vec + w.bh) * kLog2e : p.bias_log2e;
      pos_t[0] = w.row0 + tid + p.pos0;
    }
    // Batch without padding: the keys [key_lo, key_hi) this thread's row may see in each tile (its own
    // sequence, cut at the row itself when causal) and the bias of its sequence and head.
    int key_lo[2] = {0, 0}, key_hi[2] = {0, 0};
    if (ragged) {
#pragma unroll
      for (int t = 0; t < kTiles; ++t) {
        const int r = w.row0 + t * kBM + tid;
        bias_t[t] = p.bias_log2e;
        if (r < p.N) {
          const int sq = seq_of_row(p.cu_seqlens, p.n_seqs, r);
          key_lo[t] = __ldg(p.cu_seqlens + sq);
          key_hi[t] = CAUSAL ? r + 1 : __ldg(p.cu_seqlens + sq + 1);
          if (p.bias_vec) bias_t[t] = __ldg(p.bias_vec + sq * p.H + w.bh) * kLog2e;
        }
      }
    }

    // Tile-steps are visited in the order (j, tile 0), (j, tile 1), (j + 1, tile 0), ...
    for (int j = 0; j < w.n_kv; ++j) {
#pragma unroll
      for (int t = 0; t < kTiles; ++t) {
        if (j >= w.n[t]) continue;
        uint32_t& cnt = t ? s_cnt1 : s_cnt0;
        if (!mbar_wait(smem_u32(&bars->s_full[t]), cnt & 1, cta_err, 30 + t)) return;
        ++cnt;
        tc_fence_after_sync();
        const int jk = (PACKED || GENERAL) ? w.j0 + j : j;   // key tile (split keys, unpadded batches: items start later)
        // position of this thread's query relative to the first key of the tile
        // (formed in integers; only the small tile-relative difference is converted)
        const float row_rel = static_cast<float>((PACKED ? pos_t[t] : pos_t[0] + t * kBM) - jk * kBN);
        // the mask cuts through every key tile that reaches beyond the position of the tile's
        // first row: the last one, and with pos0 not a multiple of 128 also the one before
        // (packed rows: a tile may hold a head's first query, at position pos0)
        bool diag = CAUSAL && ((jk + 1) * kBN - 1 > (PACKED ? 0 : w.row0 + t * kBM) + p.pos0);
        float mask_limit = row_rel;   // last key (relative to the tile's first) that keeps its weight
        if (varlen) {
          // padded batch: keys past the end of the sequence are masked, rows past it are masked whole
          const float key_limit = static_cast<float>(w.n_valid - 1 - j * kBN);
          mask_limit = CAUSAL ? fminf(row_rel, key_limit) : key_limit;
          if (w.row0 + t * kBM + tid >= w.n_valid) mask_limit = -1.0f;
          diag = diag || (j + 1) * kBN > w.n_valid || w.row0 + (t + 1) * kBM > w.n_valid;
        }
        // bf16 P goes back over the first half of the columns this thread reads, 32 logits at a time
        // (the packed values of a later run land on logits that an earlier run has consumed)
        const uint32_t tS = tmem + t * kBN + lane_off + g * kCols;
        constexpr int kEmulateEvery = (D == 128) ? SIGATTN_FWD_EMULATE_D128
                                      : CAUSAL ? SIGATTN_FWD_EMULATE_D64 : SIGATTN_FWD_EMULATE_D64_UNMASKED;
#pragma unroll
        for (int c = 0; c < kCols / kRun; ++c) {
          uint32_t sv[kRun];
          tmem_ld_cols(tS + c * kRun, sv);
          tmem_wait_ld();
          uint32_t pk[kRun / 2];
          const int col0 = g * kCols + c * kRun;
          if (ragged) {
            const int key0 = jk * kBN;
            const bool cut = key0 < key_lo[t] || key0 + kBN > key_hi[t];   // not wholly inside the row's range
            sigmoid_cols<kRun, ALIBI, CAUSAL, kEmulateEvery, true>(sv, pk, p.scale_log2e, bias_t[t], slope_t[0], row_rel, col0,
                                                           cut, static_cast<float>(key_hi[t] - 1 - key0),
                                                           static_cast<float>(key_lo[t] - key0));
          } else {
            sigmoid_cols<kRun, ALIBI, CAUSAL, kEmulateEvery>(sv, pk, p.scale_log2e, bias_t[PACKED ? t : 0],
                                                     slope_t[PACKED ? t : 0], row_rel, col0, diag, mask_limit);
          }
          tmem_st_cols(tS + c * (kRun / 2), pk);
        }
        tmem_wait_st();
        tc_fence_before_sync();
        mbar_arrive(smem_u32(&bars->p_full[t]));
      }
    }

    // epilogue: O_t (fp32, tensor memory) -> bf16 -> swizzled shared memory (at D = 128 the Q_t
    // buffer, free once every logits MMA of the item is done; at D = 64 a buffer of its own) -> TMA store.  Each column group
    // converts its share of the D columns.
#pragma unroll
    for (int t = 0; t < kTiles; ++t) {
      if (w.n[t] == 0) continue;
      if (!mbar_wait(smem_u32(&bars->o_full[t]), it[t] & 1, cta_err, 32 + t)) return;
      ++it[t];
      tc_fence_after_sync();
      uint8_t* stage = smem + (L::kOStaged ? L::kOOff : L::kQOff) + t * L::kTileBytes;
      constexpr int kECols = D / kGroups;                 // accumulator columns per thread
      constexpr int kERun = kECols > 32 ? 32 : kECols;    // converted this many at a time
      // Partial result (split keys, or one shard of the keys): this item's rows are added, in fp32,
      // into the accumulator - local scratch or another GPU's memory, plain vector reductions
      // either way.  Whoever owns the accumulator converts the sums to bf16 afterwards.  The Q
      // buffer is not needed for staging.
      const bool to_acc = (PACKED || GENERAL) && p.split_ws != nullptr;
      const int row = w.row0 + t * kBM + tid;
#pragma unroll
      for (int ec = 0; ec < kECols / kERun; ++ec) {
        const int col = g * kECols + ec * kERun;   // first of this run's columns
        uint32_t o[kERun];
        tmem_ld_cols(tmem + kTiles * kBN + t * D + lane_off + col, o);
        tmem_wait_ld();
        if (GENERAL && p.row_scale != nullptr) {
          // sequence-length normalisation: one factor per query row (rows past the end are not stored)
          const float r = row < p.N ? __ldg(p.row_scale + row) : 0.0f;
#pragma unroll
          for (int e = 0; e < kERun; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * r);
        }
        if (to_acc) {
          if (row < p.N) {
            float* dst = p.split_ws + (static_cast<size_t>(w.bh) * p.N + row) * D + col;
#pragma unroll
            for (int e = 0; e < kERun; e += 4)
              red_add_v4_f32(dst + e, __uint_as_float(o[e]), __uint_as_float(o[e + 1]), __uint_as_float(o[e + 2]),
                             __uint_as_float(o[e + 3]));
          }
        } else {
          uint8_t* row_ptr = stage + (col >> 6) * L::kPanelBytes + tid * 128;
#pragma unroll
          for (int q4 = 0; q4 < kERun / 8; ++q4) {
            uint4 val;
            val.x = pack_bf16x2(__uint_as_float(o[8 * q4 + 0]), __uint_as_float(o[8 * q4 + 1]));
            val.y = pack_bf16x2(__uint_as_float(o[8 * q4 + 2]), __uint_as_float(o[8 * q4 + 3]));
            val.z = pack_bf16x2(__uint_as_float(o[8 * q4 + 4]), __uint_as_float(o[8 * q4 + 5]));
            val.w = pack_bf16x2(__uint_as_float(o[8 * q4 + 6]), __uint_as_float(o[8 * q4 + 7]));
            const int chunk = ((col & 63) >> 3) + q4;
            *reinterpret_cast<uint4*>(row_ptr + ((chunk ^ (tid & 7)) * 16)) = val;
          }
        }
      }
      if (to_acc) {
        tc_fence_before_sync();
        mbar_arrive(smem_u32(&bars->o_empty[t]));
        if (!L::kOStaged && threadIdx.x == 0) mbar_arrive(smem_u32(&bars->q_empty[t]));   // all logits MMAs of the item are done
        continue;
      }
      tc_fence_before_sync();
      mbar_arrive(smem_u32(&bars->o_empty[t]));
      fence_proxy_async_smem();
      named_barrier_sync<1, kActThreads>();
      if (threadIdx.x == 0) {
#pragma unroll
        for (int pn = 0; pn < L::kPanels; ++pn)
          if (GENERAL && p.o_reduce)   // the parts of a split item add their shares of O (cleared before the launch)
            tma_reduce_add_3d(tmO, smem_u32(stage + pn * L::kPanelBytes), pn * 64, w.row0 + t * kBM, w.bh);
          else
            tma_store_3d(tmO, smem_u32(stage + pn * L::kPanelBytes), pn * 64, w.row0 + t * kBM, w.bh);
        tma_commit_group();
        tma_wait_group_read<0>();   // (with a staging buffer of its own: before the next item's rows are written there)
        if (!L::kOStaged) mbar_arrive(smem_u32(&bars->q_empty[t]));
      }
    }
  }
  if (threadIdx.x == 0) tma_wait_group<0>();
}

// ------------------------------------------------------------------ kernel

template <int D, bool CAUSAL, bool ALIBI, int MODE>
__global__ void __launch_bounds__(kFwdThreads, kCtasPerSm)
sigattn_fwd_bf16_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                        const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                        const FwdParams p) {
  using L = FwdSmem<D>;
  extern __shared__ uint8_t smem_raw[];
  __shared__ FwdBarriers bars;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int cta_err;

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  const int warp = threadIdx.x >> 5;

  if (threadIdx.x == 0) {
    cta_err = 0;
    for (int t = 0; t < 2; ++t) {
      mbar_init(smem_u32(&bars.q_full[t]), 1);
      mbar_init(smem_u32(&bars.q_empty[t]), 1);
      mbar_init(smem_u32(&bars.s_full[t]), 1);
      mbar_init(smem_u32(&bars.p_full[t]), kActThreads);
      mbar_init(smem_u32(&bars.o_full[t]), 1);
      mbar_init(smem_u32(&bars.o_empty[t]), kActThreads);
    }
    for (int s = 0; s < L::kStages; ++s) {
      mbar_init(smem_u32(&bars.kv_full[s]), 1);
      mbar_init(smem_u32(&bars.kv_empty[s]), 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&bars.sched_full[s]), 1);
      mbar_init(smem_u32(&bars.sched_empty[s]), kSchedConsumers);
    }
    fence_mbar_init();
  }
  if (warp == kLoadWarp && elect_one()) {
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
    tma_prefetch_desc(&tmO);
  }
  if (warp == kMmaWarp) {
    tmem_alloc(smem_u32(&tmem_base_slot), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_base_slot;

  if (warp == kLoadWarp) {
    if ((threadIdx.x & 31) == 0) fwd_load_role<D, CAUSAL, MODE >= 2>(p, &tmQ, &tmK, &tmV, smem_base, &bars, &cta_err);
    __syncwarp();
  } else if (warp == kMmaWarp) {
    fwd_mma_role<D, CAUSAL, MODE >= 2>(p, smem_base, tmem, &bars, &cta_err);
    __syncwarp();
  } else {
    fwd_act_role<D, CAUSAL, ALIBI, MODE>(p, &tmO, smem, tmem, &bars, &cta_err);
  }

  tc_fence_before_sync();
  __syncthreads();
  if (cta_err != 0) {
    if (threadIdx.x == 0) atomicExch(p.status, 100 + cta_err);
    __nanosleep(100000);  // let copies in flight towards this CTA's shared memory land
  }
  if (warp == kMmaWarp) tmem_dealloc(tmem, kTmemCols);
}

#if SIGATTN_FWD_TILES == 2
// O (bf16) = the fp32 sums of the key splits: the pass that follows a split forward.
__global__ void __launch_bounds__(256)
sigattn_fwd_convert_o_kernel(const float4* __restrict__ ws, uint2* __restrict__ o, size_t n_vec4) {
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n_vec4; i += stride) {
    const float4 v = ws[i];
    o[i] = make_uint2(pack_bf16x2(v.x, v.y), pack_bf16x2(v.z, v.w));
  }
}

// Number of key splits for a problem with `base_items` work items of `n_kv` key tiles each:
// the count that minimises rounds of the persistent grid times tiles per item (plus about two
// tiles' worth of per-item start-up and epilogue), each split keeping at least two key tiles.
// Which shape serves a plain problem (the launcher's tile table).  Measured on B200, forward alone, us:
//   B4 H12 N256 D64 (48 pair items)    one tile 13.3   two tiles 17.4
//   B2 H8 N256 D128 (16)               14.3            17.4
//   B8 H12 N197 D64 (96)               17.4            17.4
//   B16 H12 N197 D64 (192)             23.6            25.6
//   B24 / B32 H12 N197 D64 (288, 384)  27.6 / 34.8     25.6 / 31.7
//   B3 / B8 H12 N577 D64 (108, 288)    23.6 / 42.0     21.5 / 37.8
//   B4 H16 N384 D128 causal (128)      20.5            19.5
// and on the benchmark configurations the two-tile shape is 5-16 % faster.  One tile per item pays when the
// two-tile items leave more than half of the SMs empty and the sequence is too short for the keys of an item
// to be divided (that division serves the long sequences with few heads); with N <= 128 both shapes are the same.
bool fwd_single_tile_shape(const Problem& p, int num_sms) {
  const bool plain_self = p.key_rows() == p.N && p.query_pos0() == 0 && p.kv_heads() == p.H;
  const long long pair_items = static_cast<long long>(p.B) * p.H * ((p.N + 2 * kBM - 1) / (2 * kBM));
  const int n_kv_tiles = (p.N + kBN - 1) / kBN;
  return plain_self && p.N > kBM && n_kv_tiles < 4 && 2 * pair_items <= num_sms;
}

int choose_key_splits(int base_items, int n_kv, int num_sms) {
  int best = 1;
  long long best_cost = -1;
  for (int s = 1; s <= 64 && 2 * s <= n_kv + 1; ++s) {
    const int per = (n_kv + s - 1) / s;
    const int used = (n_kv + per - 1) / per;   // splits that are not empty
    if (used != s) continue;
    const long long rounds = (static_cast<long long>(base_items) * s + num_sms - 1) / num_sms;
    const long long cost = rounds * (per + 2);
    if (best_cost < 0 || cost < best_cost) { best = s; best_cost = cost; }
  }
  return best;
}

// Work-item counters of the dynamic schedule: one per launch in flight, handed out round robin
// (1024 launches may overlap on different streams before two of them share a counter; a kernel that
// sees its counter run past what one launch can draw sets the device status word).
constexpr int kSchedSlots = 1024;
__device__ int g_fwd_sched_counters[kSchedSlots];
#endif

template <int D, bool CAUSAL, bool ALIBI, int MODE>
int launch_fwd_variant(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const CUtensorMap& tmO,
                       const FwdParams& fp, int num_sms, cudaStream_t stream, cudaError_t* cuda_err) {
  auto kernel = sigattn_fwd_bf16_kernel<D, CAUSAL, ALIBI, MODE>;
  // The shared-memory opt-in is a per-device attribute of the kernel: one bit per device ordinal
  // (a process may drive several GPUs); ordinals past 63 simply set it on every launch.
  static std::atomic<unsigned long long> configured{0};
  int dev = 0;
  *cuda_err = cudaGetDevice(&dev);
  if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  const unsigned long long bit = (dev >= 0 && dev < 64) ? (1ull << dev) : 0ull;
  if ((configured.load(std::memory_order_relaxed) & bit) == 0) {
    *cuda_err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem<D>::kDynBytes);
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
    configured.fetch_or(bit, std::memory_order_relaxed);
  }
  const int slots = num_sms * kCtasPerSm;
  const int grid = fp.n_items < slots ? fp.n_items : slots;
  kernel<<<grid, kFwdThreads, FwdSmem<D>::kDynBytes, stream>>>(tmQ, tmK, tmV, tmO, fp);
  *cuda_err = cudaGetLastError();
  return *cuda_err == cudaSuccess ? SIGATTN_OK : SIGATTN_ERR_CUDA;
}

}  // namespace

#if SIGATTN_FWD_TILES == 1
// Plain problems only (no grouped heads, padded or unpadded batches, key shards or split keys).
int launch_fwd_bf16_single(const void* q, const void* k, const void* v, void* o, const Problem& p, int* status,
                           cudaStream_t stream, unsigned long long* launches, cudaError_t* cuda_err) {
  int dev = 0, num_sms = 0;
  *cuda_err = cudaGetDevice(&dev);
  if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  *cuda_err = cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev);
  if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  const uint64_t BH = static_cast<uint64_t>(p.B) * p.H;
  CUtensorMap tmQ, tmK, tmV, tmO;
  const void* ptrs[4] = {q, k, v, o};
  CUtensorMap* maps[4] = {&tmQ, &tmK, &tmV, &tmO};
  for (int i = 0; i < 4; ++i) {
    if (make_map_3d(maps[i], ptrs[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, BH, p.N, p.D, kBM, 64) != 0) {
      *cuda_err = cudaErrorInvalidValue;
      return SIGATTN_ERR_CUDA;
    }
  }
  FwdParams fp = {};
  fp.BH = static_cast<int>(BH);
  fp.H = fp.H_kv = p.H;
  fp.group = 1;
  fp.pack_group = 1;
  fp.N = p.N;
  fp.pos0 = 0;
  fp.n_pairs = (p.N + kBM - 1) / kBM;
  fp.n_kv_total = (p.N + kBN - 1) / kBN;
  fp.n_splits = 1;
  fp.tiles_per_split = fp.n_kv_total;
  fp.n_items = fp.n_pairs * fp.BH;
  fp.scale_log2e = p.scale * kLog2e;
  fp.bias_log2e = p.bias * kLog2e;
  fp.bias_vec = p.bias_vec;
  fp.slopes = p.slopes;
  fp.status = status;
  int rc;
  const bool alibi = p.slopes != nullptr;
#define SIGATTN_FWD_CASE(DD, CC, AA) rc = launch_fwd_variant<DD, CC, AA, 0>(tmQ, tmK, tmV, tmO, fp, num_sms, stream, cuda_err)
  if (p.D == 128) {
    if (p.causal) { if (alibi) SIGATTN_FWD_CASE(128, true, true); else SIGATTN_FWD_CASE(128, true, false); }
    else          { if (alibi) SIGATTN_FWD_CASE(128, false, true); else SIGATTN_FWD_CASE(128, false, false); }
  } else {
    if (p.causal) { if (alibi) SIGATTN_FWD_CASE(64, true, true); else SIGATTN_FWD_CASE(64, true, false); }
    else          { if (alibi) SIGATTN_FWD_CASE(64, false, true); else SIGATTN_FWD_CASE(64, false, false); }
  }
#undef SIGATTN_FWD_CASE
  if (rc == SIGATTN_OK) *launches += 1;
  return rc;
}
#else
int launch_fwd_bf16(const void* q, const void* k, const void* v, void* o, const Problem& p, int* status,
                    cudaStream_t stream, unsigned long long* launches, cudaError_t* cuda_err) {
  int dev = 0, num_sms = 0;
  *cuda_err = cudaGetDevice(&dev);
  if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  *cuda_err = cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev);
  if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;

  const uint64_t BH = static_cast<uint64_t>(p.B) * p.H;
  const uint64_t BH_kv = static_cast<uint64_t>(p.B) * p.kv_heads();
  const int group = p.H / p.kv_heads();
  // Few queries per head and several query heads per key/value head (decoding with grouped
  // heads): pack the group's rows into one sequence so that K and V are streamed once per group.
  const bool small = static_cast<long long>(p.N) * group <= 2 * kBM && p.seqlens == nullptr &&
                     p.row_scale == nullptr && p.cu_seqlens == nullptr;
  // With a scratch buffer for fp32 partial sums, the keys of one head may also be split over
  // several work items (decoding: too few (batch, head) pairs for 148 SMs otherwise).
  const int n_kv_tiles = (p.key_rows() + kBN - 1) / kBN;
  const int n_splits = (small && p.split_ws != nullptr) ? choose_key_splits(static_cast<int>(BH_kv), n_kv_tiles, num_sms) : 1;
  const bool packed = small && (group > 1 || n_splits > 1);
  // acc_only: the caller owns an fp32 accumulator that this call adds its (partial) O into; nothing
  // is cleared, nothing converted, `o` is not written.  Otherwise the accumulator is only used as
  // scratch when the keys are split.
  const bool accumulate = p.split_ws != nullptr && (p.acc_only != 0 || n_splits > 1);
  // One long causal sequence with few heads: the most expensive work item alone takes as long as
  // the whole job should.  Divide the key tiles of every item over two items that add their
  // bf16 shares into O (one extra rounding; the sum of two parts does not depend on their order).
  int o_splits = 1;
  if (!small && p.split_ws == nullptr && p.seqlens == nullptr && p.cu_seqlens == nullptr) {
    const long long base_items = static_cast<long long>((p.N + 2 * kBM - 1) / (2 * kBM)) * BH;
    int by_mask = 1, by_round = 1;
    // (one round of items: the longest one sets the time.  With 149 to 295 items the static pairing of an
    // expensive with a cheap item already balances two rounds, and dividing them measured 2-24 % slower.)
    if (p.causal && base_items <= num_sms && n_kv_tiles >= 32) {
      by_mask = static_cast<int>((2ll * num_sms + base_items - 1) / base_items);
      if (by_mask > n_kv_tiles / 4) by_mask = n_kv_tiles / 4;
    }
    // whatever the mask: while all parts still fit one round of the grid, dividing the items only
    // shortens the longest one (B1 H1 N2048 has 8 items, the last of them 16 key tiles long)
    if (2 * base_items <= num_sms && n_kv_tiles >= 4) {
      by_round = static_cast<int>(num_sms / base_items);
      if (by_round > n_kv_tiles / 2) by_round = n_kv_tiles / 2;
    }
    o_splits = by_mask > by_round ? by_mask : by_round;
    // two parts at most: 0 + a + b does not depend on which part arrives first, so O stays
    // bit-reproducible; three or four parts measured 5-10 % faster still but would give that up
    if (o_splits > 2) o_splits = 2;
  }
  const uint64_t q_heads = packed ? BH_kv : BH;
  const uint64_t q_rows = packed ? static_cast<uint64_t>(p.N) * group : p.N;
  CUtensorMap tmQ, tmK, tmV, tmO;
  const void* ptrs[4] = {q, k, v, (p.acc_only && o == nullptr) ? q : o};   // accumulate only: O is never stored
  CUtensorMap* maps[4] = {&tmQ, &tmK, &tmV, &tmO};
  for (int i = 0; i < 4; ++i) {
    const bool kv = (i == 1 || i == 2);
    if (make_map_3d(maps[i], ptrs[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, kv ? BH_kv : q_heads,
                    kv ? p.key_rows() : q_rows, p.D, kBM, 64) != 0) {
      *cuda_err = cudaErrorInvalidValue;
      return SIGATTN_ERR_CUDA;
    }
  }
  FwdParams fp;
  fp.BH = static_cast<int>(q_heads);
  fp.H = packed ? p.kv_heads() : p.H;
  fp.H_kv = p.kv_heads();
  fp.group = packed ? 1 : group;
  fp.pack_rows = packed ? p.N : 0;
  fp.pack_group = packed ? group : 1;
  fp.N = static_cast<int>(q_rows);
  fp.pos0 = p.query_pos0();
  fp.n_pairs = (fp.N + 2 * kBM - 1) / (2 * kBM);
  fp.n_kv_total = (p.key_rows() + kBN - 1) / kBN;
  fp.n_splits = o_splits > 1 ? o_splits : n_splits;
  fp.o_reduce = o_splits > 1 ? 1 : 0;
  fp.tiles_per_split = (fp.n_kv_total + n_splits - 1) / n_splits;
  fp.split_ws = accumulate ? p.split_ws : nullptr;
  fp.n_items = fp.n_pairs * fp.BH * fp.n_splits;
  fp.scale_log2e = p.scale * kLog2e;
  fp.bias_log2e = p.bias * kLog2e;
  fp.bias_vec = p.bias_vec;
  fp.slopes = p.slopes;
  fp.seqlens = p.seqlens;
  fp.row_scale = p.row_scale;
  fp.cu_seqlens = p.cu_seqlens;
  fp.n_seqs = p.n_seqs;
  fp.status = status;

  fp.sched_counter = nullptr;
  const bool general = !packed && (p.cu_seqlens != nullptr || p.seqlens != nullptr || p.row_scale != nullptr || accumulate ||
                                   o_splits > 1);
  if (!packed && !general && fwd_single_tile_shape(p, num_sms))
    return launch_fwd_bf16_single(q, k, v, o, p, status, stream, launches, cuda_err);
  if (general) {   // the general instantiations draw their work items from a counter
    static std::atomic<unsigned> next_slot{0};
    int* counters = nullptr;
    *cuda_err = cudaGetSymbolAddress(reinterpret_cast<void**>(&counters), g_fwd_sched_counters);
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
    fp.sched_counter = counters + next_slot.fetch_add(1) % kSchedSlots;
    *cuda_err = cudaMemsetAsync(fp.sched_counter, 0, sizeof(int), stream);
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  }
  const size_t n_elems = static_cast<size_t>(BH) * p.N * p.D;
  if (o_splits > 1) {
    *cuda_err = cudaMemsetAsync(o, 0, n_elems * 2, stream);
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  }
  if (accumulate && !p.acc_only) {
    *cuda_err = cudaMemsetAsync(p.split_ws, 0, n_elems * sizeof(float), stream);
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  }

  int rc;
  const bool alibi = p.slopes != nullptr;
#define SIGATTN_FWD_CASE(DD, CC, AA)                                                                       \
  rc = packed ? launch_fwd_variant<DD, CC, AA, 1>(tmQ, tmK, tmV, tmO, fp, num_sms, stream, cuda_err)       \
       : (p.cu_seqlens != nullptr)                                                                         \
           ? launch_fwd_variant<DD, CC, AA, 3>(tmQ, tmK, tmV, tmO, fp, num_sms, stream, cuda_err)          \
       : general                                                                                           \
           ? launch_fwd_variant<DD, CC, AA, 2>(tmQ, tmK, tmV, tmO, fp, num_sms, stream, cuda_err)          \
           : launch_fwd_variant<DD, CC, AA, 0>(tmQ, tmK, tmV, tmO, fp, num_sms, stream, cuda_err)
  if (p.D == 128) {
    if (p.causal) { if (alibi) SIGATTN_FWD_CASE(128, true, true); else SIGATTN_FWD_CASE(128, true, false); }
    else          { if (alibi) SIGATTN_FWD_CASE(128, false, true); else SIGATTN_FWD_CASE(128, false, false); }
  } else {
    if (p.causal) { if (alibi) SIGATTN_FWD_CASE(64, true, true); else SIGATTN_FWD_CASE(64, true, false); }
    else          { if (alibi) SIGATTN_FWD_CASE(64, false, true); else SIGATTN_FWD_CASE(64, false, false); }
  }
#undef SIGATTN_FWD_CASE
  if (rc != SIGATTN_OK) return rc;
  *launches += 1;
  if (accumulate && !p.acc_only) {
    const size_t n_vec4 = n_elems / 4;
    const size_t want = n_vec4 / 256 + 1, cap = static_cast<size_t>(num_sms) * 8;
    sigattn_fwd_convert_o_kernel<<<static_cast<int>(want < cap ? want : cap), 256, 0, stream>>>(
        static_cast<const float4*>(static_cast<const void*>(p.split_ws)), static_cast<uint2*>(o), n_vec4);
    *cuda_err = cudaGetLastError();
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
    *launches += 1;
  }
  return SIGATTN_OK;
}
#endif   // SIGATTN_FWD_TILES

}  // namespace sigattn


