// The fast attention tile kernel, in persistent form: one CTA per SM walks a queue of work items (query tiles)
// and keeps its pipeline running across them.
//
// Against attn_fwd_body (the exact-rescaling kernel, where each softmax group owns one S buffer that P overwrites in
// place and one accumulator that is rescaled when the row maximum grows, so that S for a group's next tile can only
// be issued after the P V of its current tile):
//   * every row keeps ONE reference maximum, the maximum of its first tile.  Probabilities are exp2(s*c - m_ref);
//     they may exceed 1 for later tiles, which fp32 accumulation and bf16 P tolerate (same relative precision at
//     any magnitude) as long as nothing overflows.  No per-tile maximum, no rescaling: both groups add into the
//     same accumulator O and their row sums simply add up;
//   * tensor memory is S0 | S1 | O | P0 | P1.  The groups take alternate key tiles, P has its own buffer: a group
//     releases its S buffer the moment the tile is in registers, so Q K^T of its next tile runs under the
//     exponentials of the current one, and it waits for the P V that read its previous P only at the first store
//     of the new P;
//   * two warps issue MMAs, one the Q K^T products and one the P V products: every MMA and every barrier wait
//     costs the issuing thread tens of cycles, which one warp doing both would serialise;
//   * a CTA that handles one query tile spends about 6 us outside its steady state (launch, barrier and tensor-
//     memory set-up, about 3000 cycles of TMA latency for the first tiles with nothing to hide them behind,
//     pipeline fill, drain, store, teardown), and with one CTA per SM nothing overlaps that.  So the roles loop
//     over work items instead:
//     - warp 3 is scheduler and V producer: it takes the next item from a global counter (through an order array
//       that puts the long lists first), checks its list, and publishes it in a four-slot ring two items ahead of
//       the one whose V tiles it is loading (V is needed last in a tile's life, so this warp has the slack);
//     - warp 0 (Q and K), warp 1 (Q K^T) and warp 2 (P V) follow the published items; the K and V rings simply
//       continue into the next item's tiles, and all ring positions and barrier phases are running counts;
//     - the softmax groups finish an item by exchanging their row sums, reading the accumulator out of tensor
//       memory (which hands it back to the P V warp for the next item) and staging their half rows for one TMA
//       store (the fp32 partials of the range mode go straight to global memory with 32-byte stores); the next
//       item's first S tiles are already waiting by then.
// A row whose sum, relative to m_ref, ends above 2^64 (or not finite) outgrew its reference: its work item is
// appended to `redo_list` (count in the status record) and attn_redo_kernel, a small grid launched behind this
// kernel, recomputes the listed items with exact rescaling.  List validation and bounded waits as in attn_fwd_body.
#pragma once
#include "attn_kernel.cuh"

namespace avsa {

// Largest row sum, relative to the first-tile reference maximum, that the fast path accepts (2^64).
constexpr float kFastRowSumLimit = 1.8446744e19f;
enum FastWhere { kFastSFree = 61, kFastPFree, kFastMref };

// K stages, V stages, Q buffers, slots of the item ring.  On the benchmark shapes (64-256 tiles per item) the splits
// (3,3,1), (3,2,2), (2,3,2), (4,2,1) and (2,4,1) of the seven 32 KB tile slots are within noise of each other; the
// seventh slot is the staging buffer of the output tile.
constexpr int kPKS = 3, kPVS = 2, kPQB = 1, kPRing = 4;

template <int BLK, int D>
struct PersistSmem {
  static constexpr int kTileBytes = BLK * D * 2;
  static constexpr int kQBytes = 128 * D * 2;
  static constexpr int kQ = 0;
  static constexpr int kK = kPQB * kQBytes;
  static constexpr int kV = kK + kPKS * kTileBytes;
  static constexpr int kStage = kV + kPVS * kTileBytes;         // output tile, 128-byte swizzled, for the TMA store
  static constexpr int kBars = kStage + kQBytes;
  static constexpr int kNumBars = 2 * kPQB + 2 * kPKS + 2 * kPVS + 18 + 2 * kPRing;
  static constexpr int kStats = kBars + kNumBars * 8;          // float mref[128], lsum[2][128]
  static constexpr int kItems = kStats + 3 * 128 * 4;          // int {item, cnt}[kPRing], two redo flags
  static constexpr int kMisc = kItems + 8 * kPRing + 16;       // tmem base, stop flag
  static constexpr int kTotal = kMisc + 16;
};

enum PersistWhere { kPersistItem = 71, kPersistItemEmpty, kPersistQEmpty, kPersistOFull, kPersistOFree, kPersistLsum, kPersistStage };

__device__ __forceinline__ void st_global_v8(void* ptr, const uint32_t (&r)[8]) {
  asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(ptr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]),
               "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}

// One work item: which query tile, which key tiles.
struct PersistItem {
  int qt, h, b, kb0;
  const int32_t* list;
};
template <int MODE>
__device__ __forceinline__ PersistItem decode_item(const AttnParams& p, int item) {
  PersistItem it;
  int rest = item;
  it.kb0 = 0;
  it.list = nullptr;
  if (MODE == MODE_LIST) {
    it.list = p.col_idx + static_cast<int64_t>(item) * p.NKB;
  } else {
    it.kb0 = (item % p.n_split) * p.tiles_per_split;
    rest = item / p.n_split;
  }
  it.qt = rest % p.NQT;
  const int bh = rest / p.NQT;
  it.h = bh % p.H;
  it.b = bh / p.H;
  return it;
}

// MODE_LIST: work item = query tile with an explicit list of key tiles, output bf16 rows + optional LSE
// (block-sparse self-attention; `order` maps queue position to item).  MODE_RANGE / MODE_RANGE_DIRECT: work
// item = (query tile, split of the key axis), key tiles kb0 .. kb0+cnt-1; output normalised fp32 partials +
// log2 LSE per split (merge_splits_kernel combines them), or bf16 rows directly when there is one split.
template <int BLK, int D, int MODE>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_persist_kernel(const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
                    const __grid_constant__ CUtensorMap tmv, const __grid_constant__ CUtensorMap tmo,
                    const AttnParams p, int* __restrict__ redo_list, const int* __restrict__ order, int n_items) {
  using L = PersistSmem<BLK, D>;
  constexpr bool kListIn = (MODE == MODE_LIST);
  constexpr bool kDirectOut = (MODE != MODE_RANGE);
  constexpr int NPANEL = D / 64;
  constexpr int PANEL_BYTES = BLK * 128;
  constexpr int QPANEL_BYTES = 128 * 128;
  constexpr unsigned FULLM = 0xffffffffu;
  extern __shared__ __align__(1024) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if ((smem_u32(smem) & 1023u) != 0u) {
    if (tid == 0) report_status(p.status, AVSA_ERR_CUDA, kWhereSmemAlign, blockIdx.x, 0);
    return;
  }
  const uint32_t bar0 = smem_u32(smem + L::kBars);
  auto BAR = [&](int i) { return bar0 + static_cast<uint32_t>(i) * 8u; };
  constexpr int Q_FULL = 0, Q_EMPTY = kPQB, K_FULL = 2 * kPQB, K_EMPTY = K_FULL + kPKS, V_FULL = K_EMPTY + kPKS,
                V_EMPTY = V_FULL + kPVS, S_FULL = V_EMPTY + kPVS /* + group */, S_FREE = S_FULL + 2,
                P_FULL = S_FREE + 2 /* + 2*group + half */, P_FREE = P_FULL + 4, O_FULL = P_FREE + 2,
                O_FREE = O_FULL + 1, MREF = O_FREE + 1, ITEM_FULL = MREF + 1 /* + slot */, ITEM_EMPTY = ITEM_FULL + kPRing,
                QK_DRAIN = ITEM_EMPTY + kPRing, PV_DRAIN = QK_DRAIN + 1, LSUM_A = PV_DRAIN + 1, LSUM_B = LSUM_A + 1,
                STAGE_FULL = LSUM_B + 1;
  static_assert(STAGE_FULL + 1 <= L::kNumBars, "barrier table too small");
  // tensor memory: S of group 0 | S of group 1 | O | P of group 0 | P of group 1
  constexpr uint32_t TM_O = 2 * BLK, TM_P = 2 * BLK + D;
  constexpr int NCH = BLK / 32;
  float* mref_s = reinterpret_cast<float*>(smem + L::kStats);
  float* lsum_s = mref_s + 128;                                              // [2][128]
  volatile int* items = reinterpret_cast<volatile int*>(smem + L::kItems);   // {item, cnt} x kPRing, then two redo flags
  // One redo flag per item parity: the flag of item n is cleared after item n's second row-sum barrier, and the
  // first thread that can set the flag of item n + 2 has passed that barrier itself, so a set never meets a
  // pending clear (with a single flag, a fast warp of the other group could set it for item n + 1 first).
  constexpr int REDO = 2 * kPRing;
  volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + L::kMisc);   // [0] tmem base, [1] stop

  if (tid == 0) {
    for (int s = 0; s < kPQB; s++) {
      mbar_init(BAR(Q_FULL + s), 1);
      mbar_init(BAR(Q_EMPTY + s), 1);
    }
    for (int s = 0; s < kPKS; s++) {
      mbar_init(BAR(K_FULL + s), 1);
      mbar_init(BAR(K_EMPTY + s), 1);
    }
    for (int s = 0; s < kPVS; s++) {
      mbar_init(BAR(V_FULL + s), 1);
      mbar_init(BAR(V_EMPTY + s), 1);
    }
    for (int g = 0; g < 2; g++) {
      mbar_init(BAR(S_FULL + g), 1);
      mbar_init(BAR(S_FREE + g), 128);
      mbar_init(BAR(P_FULL + 2 * g), 128);
      mbar_init(BAR(P_FULL + 2 * g + 1), 128);
      mbar_init(BAR(P_FREE + g), 1);
    }
    for (int r = 0; r < kPRing; r++) {
      mbar_init(BAR(ITEM_FULL + r), 1);
      mbar_init(BAR(ITEM_EMPTY + r), 11);      // one arrival per consumer warp (all but the scheduler)
    }
    mbar_init(BAR(O_FULL), 1);
    mbar_init(BAR(O_FREE), 256);
    mbar_init(BAR(MREF), 128);
    mbar_init(BAR(QK_DRAIN), 1);
    mbar_init(BAR(PV_DRAIN), 1);
    mbar_init(BAR(LSUM_A), 256);
    mbar_init(BAR(LSUM_B), 256);
    mbar_init(BAR(STAGE_FULL), 256);
    misc[1] = 0u;
    items[REDO] = 0;
    items[REDO + 1] = 0;
    fence_mbar_init();
    prefetch_tmap(&tmq);
    prefetch_tmap(&tmk);
    prefetch_tmap(&tmv);
    if (kDirectOut) prefetch_tmap(&tmo);
  }
  if (warp == 2) {
    tmem_alloc(smem_u32(smem + L::kMisc), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = misc[0];

  // A wait that gives up when the CTA has been stopped (a time limit was reached somewhere).
  auto wait_or_stop = [&](int bar, uint32_t parity, int where, int tag) -> bool {
    if (mbar_try_wait(BAR(bar), parity)) return true;
    const long long t0 = clock64();
    while (true) {
      if (misc[1] != 0u) return false;
      if (mbar_try_wait(BAR(bar), parity)) return true;
      if (clock64() - t0 > AVSA_WAIT_LIMIT_CYCLES) {
        report_status(p.status, AVSA_ERR_TIMEOUT, where, blockIdx.x, tag);
        misc[1] = 1u;
        return false;
      }
    }
  };
  auto wait_all = [&](int bar, uint32_t parity, int where, int tag) -> bool {
    return __all_sync(FULLM, wait_or_stop(bar, parity, where, tag));
  };
  // consumer side of the item ring: item n sits in slot n mod kPRing
  auto get_item = [&](int n, int& item, int& cnt) -> bool {     // false: stopped, or the queue is empty
    const int slot = n % kPRing;
    if (!wait_all(ITEM_FULL + slot, (n / kPRing) & 1, kPersistItem, n)) return false;
    item = items[2 * slot];
    cnt = items[2 * slot + 1];
    return item >= 0;
  };
  auto item_done = [&](int n) {
    __syncwarp();
    if (lane == 0) mbar_arrive(BAR(ITEM_EMPTY + n % kPRing));
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer of Q and K
    asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
    int kc = 0;              // K tiles loaded so far, over all items
    int q_loads = 0;
    bool ok = true;
    for (int n = 0; ok; n++) {
      int item, cnt;
      if (!get_item(n, item, cnt)) break;
      const PersistItem it = decode_item<MODE>(p, item);
      const int qt = it.qt, h = it.h, b = it.b;
      const int qb = n % kPQB;
      if (n >= kPQB) {
        // the last Q K^T of the item that used this Q buffer has run
        ok = wait_all(Q_EMPTY + qb, ((n / kPQB) - 1) & 1, kPersistQEmpty, n);
        if (!ok) break;
      }
      if (lane == 0) {
        mbar_expect_tx(BAR(Q_FULL + qb), BLK * D * 2);
        for (int pn = 0; pn < NPANEL; pn++)
          tma_load_4d(smem_u32(smem + L::kQ) + qb * L::kQBytes + pn * QPANEL_BYTES, &tmq, BAR(Q_FULL + qb), pn * 64,
                      qt * BLK, h, b);
        q_loads++;
      }
      for (int t0 = 0; t0 < cnt && ok; t0 += 32) {
        int mine = it.kb0 + t0 + lane;
        if (kListIn) mine = (t0 + lane < cnt) ? it.list[t0 + lane] : 0;
        const int nn = min(32, cnt - t0);
        for (int j = 0; j < nn; j++) {
          const int kb = __shfl_sync(FULLM, mine, j);
          const int s = kc % kPKS;
          int good = 1;
          if (lane == 0) {
            if (kc >= kPKS) good = wait_or_stop(K_EMPTY + s, ((kc / kPKS) - 1) & 1, kWhereKEmpty, t0 + j) ? 1 : 0;
            if (good) {
              mbar_expect_tx(BAR(K_FULL + s), L::kTileBytes);
              for (int pn = 0; pn < NPANEL; pn++)
                tma_load_4d(smem_u32(smem + L::kK) + s * L::kTileBytes + pn * PANEL_BYTES, &tmk, BAR(K_FULL + s), pn * 64,
                            kb * BLK, h, b);
            }
          }
          good = __shfl_sync(FULLM, good, 0);
          if (!good) {
            ok = false;
            break;
          }
          kc++;
        }
      }
      if (ok) item_done(n);
    }
    if (lane == 0 && misc[1] != 0u) {
      // stopped: loads still in flight must land before this CTA's shared memory is given away
      for (int c = max(0, q_loads - kPQB); c < q_loads; c++) mbar_wait(BAR(Q_FULL + c % kPQB), (c / kPQB) & 1);
      for (int c = max(0, kc - kPKS); c < kc; c++) mbar_wait(BAR(K_FULL + c % kPKS), (c / kPKS) & 1);
    }
  } else if (warp == 3) {
    // ------------------------------------------------------------------ scheduler + TMA producer of V
    // V is needed last in a tile's life, so this warp has the slack to fetch work: it keeps the item ring two
    // items ahead of the one whose V tiles it is loading.
    asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
    int pub_item = -1, pub_cnt = 0;
    // takes the next valid work item off the global queue and publishes it as item m of this CTA
    auto publish = [&](int m) -> bool {
      const int slot = m % kPRing;
      if (m >= kPRing && !wait_all(ITEM_EMPTY + slot, ((m / kPRing) - 1) & 1, kPersistItemEmpty, m)) return false;
      while (true) {
        int id = 0;
        if (lane == 0) id = atomicAdd(&p.status->next_item, 1);
        id = __shfl_sync(FULLM, id, 0);
        if (id >= n_items) {
          pub_item = -1;
          pub_cnt = 0;
          break;
        }
        if (!kListIn) {
          const int kb0 = (id % p.n_split) * p.tiles_per_split;
          pub_item = id;
          pub_cnt = min(p.NKB, kb0 + p.tiles_per_split) - kb0;
          break;
        }
        id = order[id];                  // queue position -> query tile (long lists first)
        const int c = p.col_cnt[id];
        bool bad = (c < 1 || c > p.NKB);
        if (!bad) {
          // nothing is loaded through a bad list: entries in range and strictly ascending
          const int32_t* lst = p.col_idx + static_cast<int64_t>(id) * p.NKB;
          int carry = -1;
          for (int t0 = 0; t0 < c; t0 += 32) {
            const bool have = t0 + lane < c;
            const int e = have ? lst[t0 + lane] : 0;
            int prev = __shfl_up_sync(FULLM, e, 1);
            if (lane == 0) prev = carry;
            if (have && (e < 0 || e >= p.NKB || e <= prev)) bad = true;
            carry = __shfl_sync(FULLM, e, 31);
          }
          bad = __any_sync(FULLM, bad);
        }
        if (!bad) {
          pub_item = id;
          pub_cnt = c;
          break;
        }
        if (lane == 0) report_status(p.status, AVSA_ERR_BAD_MASK, kWhereList, id, c);   // refused, not deferred
      }
      if (lane == 0) {
        items[2 * slot] = pub_item;
        items[2 * slot + 1] = pub_cnt;
        mbar_arrive(BAR(ITEM_FULL + slot));     // release: the slot is written before the phase completes
      }
      __syncwarp();
      return true;
    };
    int vc = 0;              // V tiles loaded so far, over all items
    bool ok = publish(0);
    int a_item = pub_item, a_cnt = pub_cnt;       // item n, whose V tiles are loaded next
    int b_item = -1, b_cnt = 0;                   // item n + 1
    if (ok && a_item >= 0) {
      ok = publish(1);
      b_item = pub_item;
      b_cnt = pub_cnt;
    }
    for (int n = 0; ok && a_item >= 0; n++) {
      const PersistItem it = decode_item<MODE>(p, a_item);
      const int h = it.h, b = it.b;
      for (int t0 = 0; t0 < a_cnt && ok; t0 += 32) {
        int mine = it.kb0 + t0 + lane;
        if (kListIn) mine = (t0 + lane < a_cnt) ? it.list[t0 + lane] : 0;
        const int nn = min(32, a_cnt - t0);
        for (int j = 0; j < nn; j++) {
          const int kb = __shfl_sync(FULLM, mine, j);
          const int s = vc % kPVS;
          int good = 1;
          if (lane == 0) {
            if (vc >= kPVS) good = wait_or_stop(V_EMPTY + s, ((vc / kPVS) - 1) & 1, kWhereVEmpty, t0 + j) ? 1 : 0;
            if (good) {
              mbar_expect_tx(BAR(V_FULL + s), L::kTileBytes);
              for (int pn = 0; pn < NPANEL; pn++)
                tma_load_4d(smem_u32(smem + L::kV) + s * L::kTileBytes + pn * PANEL_BYTES, &tmv, BAR(V_FULL + s), pn * 64,
                            kb * BLK, h, b);
            }
          }
          good = __shfl_sync(FULLM, good, 0);
          if (!good) {
            ok = false;
            break;
          }
          vc++;
        }
      }
      if (!ok) break;
      // keep the ring two items ahead (nothing more once the end of the queue has been published)
      int c_item = -1, c_cnt = 0;
      if (b_item >= 0) {
        ok = publish(n + 2);
        c_item = pub_item;
        c_cnt = pub_cnt;
      }
      a_item = b_item;
      a_cnt = b_cnt;
      b_item = c_item;
      b_cnt = c_cnt;
    }
    if (lane == 0 && misc[1] != 0u)
      for (int c = max(0, vc - kPVS); c < vc; c++) mbar_wait(BAR(V_FULL + c % kPVS), (c / kPVS) & 1);
  } else if (warp == 1) {
    // ------------------------------------------------------------------ Q K^T issuer
    asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
    const bool leader = elect_one_sync();
    constexpr uint32_t desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
    constexpr uint32_t idesc_qk = make_idesc_bf16(128, BLK, 0, 0);
    const uint32_t tmem_u = __shfl_sync(FULLM, tmem, 0);
    auto desc64 = [](uint32_t lo) { return (static_cast<uint64_t>(desc_hi) << 32) | lo; };
    const uint32_t q_lo0 = ((smem_u32(smem + L::kQ) & 0x3FFFFu) >> 4) | (1u << 16);
    const uint32_t k_lo0 = ((smem_u32(smem + L::kK) & 0x3FFFFu) >> 4) | (1u << 16);
    int kc = 0;                 // K tiles consumed so far
    int used[2] = {0, 0};       // S tiles written so far into each group's buffer
    bool ok = true;
    for (int n = 0; ok; n++) {
      int item, cnt;
      if (!get_item(n, item, cnt)) break;
      const int qb = n % kPQB;
      const uint32_t q_lo = q_lo0 + qb * (L::kQBytes >> 4);
      ok = wait_all(Q_FULL + qb, (n / kPQB) & 1, kWhereQFull, n);
      for (int t = 0; t < cnt && ok; t++) {
        const int j = t & 1, sk = kc % kPKS;
        ok = wait_all(K_FULL + sk, (kc / kPKS) & 1, kWhereKFull, t);
        if (!ok) break;
        if (used[j] > 0) {
          ok = wait_all(S_FREE + j, (used[j] - 1) & 1, kFastSFree, t);     // the group has taken its last tile out
          if (!ok) break;
        }
        tc_fence_after();
        const uint32_t k_lo = k_lo0 + sk * (L::kTileBytes >> 4);
        const uint32_t tm_s = tmem_u + j * BLK;
        if (leader) {
#pragma unroll
          for (int ks = 0; ks < D / 16; ks++) {
            const uint32_t qoff = ((ks >> 2) * QPANEL_BYTES + (ks & 3) * 32) >> 4;
            const uint32_t koff = ((ks >> 2) * PANEL_BYTES + (ks & 3) * 32) >> 4;
            umma_ss(tm_s, desc64(q_lo + qoff), desc64(k_lo + koff), idesc_qk, ks > 0 ? 1u : 0u);
          }
          umma_commit(BAR(S_FULL + j));
          umma_commit(BAR(K_EMPTY + sk));
          if (t == cnt - 1) umma_commit(BAR(Q_EMPTY + qb));     // Q may be replaced once this product has run
        }
        __syncwarp();
        used[j]++;
        kc++;
      }
      if (ok) item_done(n);
    }
    // tensor memory must not be freed under a running MMA: wait for this warp's own
    if (leader) umma_commit(BAR(QK_DRAIN));
    __syncwarp();
    mbar_wait(BAR(QK_DRAIN), 0);
  } else if (warp == 2) {
    // ------------------------------------------------------------------ P V issuer
    asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
    const bool leader = elect_one_sync();
    constexpr uint32_t desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
    constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, 0, 1);
    const uint32_t tmem_u = __shfl_sync(FULLM, tmem, 0);
    auto desc64 = [](uint32_t lo) { return (static_cast<uint64_t>(desc_hi) << 32) | lo; };
    const uint32_t v_lo0 = ((smem_u32(smem + L::kV) & 0x3FFFFu) >> 4) | (static_cast<uint32_t>(PANEL_BYTES >> 4) << 16);
    // P V over one half of the key axis (k-step ks covers keys [16 ks, 16 ks + 16), 8 columns of P)
    auto issue_pv_phase = [&](uint32_t tm_buf, uint32_t v_lo, int ph_, uint32_t acc_first) {
#pragma unroll
      for (int kk = 0; kk < BLK / 32; kk++) {
        const int ks = ph_ * (BLK / 32) + kk;
        umma_ts(tmem_u + TM_O, tm_buf + ks * 8, desc64(v_lo + ks * (2048 >> 4)), idesc_pv, kk > 0 ? 1u : acc_first);
      }
    };
    int vc = 0;                 // V tiles consumed so far
    int used[2] = {0, 0};       // P tiles read so far from each group's buffer
    bool ok = true;
    for (int n = 0; ok; n++) {
      int item, cnt;
      if (!get_item(n, item, cnt)) break;
      for (int t = 0; t < cnt && ok; t++) {
        const int j = t & 1, sv = vc % kPVS;
        ok = wait_all(V_FULL + sv, (vc / kPVS) & 1, kWhereVFull, t);
        if (!ok) break;
        ok = wait_all(P_FULL + 2 * j, used[j] & 1, kWherePFull, t);
        if (!ok) break;
        if (t == 0 && n > 0) {
          ok = wait_all(O_FREE, (n - 1) & 1, kPersistOFree, n);     // the accumulator of the item before has been read out
          if (!ok) break;
        }
        tc_fence_after();
        const uint32_t v_lo = v_lo0 + sv * (L::kTileBytes >> 4);
        const uint32_t tm_buf = tmem_u + TM_P + j * (BLK / 2);
        if (leader) issue_pv_phase(tm_buf, v_lo, 0, t > 0 ? 1u : 0u);
        __syncwarp();
        ok = wait_all(P_FULL + 2 * j + 1, used[j] & 1, kWherePFull, t);
        if (!ok) break;
        tc_fence_after();
        if (leader) {
          issue_pv_phase(tm_buf, v_lo, 1, 1u);
          umma_commit(BAR(P_FREE + j));
          umma_commit(BAR(V_EMPTY + sv));
          if (t == cnt - 1) umma_commit(BAR(O_FULL));
        }
        __syncwarp();
        used[j]++;
        vc++;
      }
      if (ok) item_done(n);
    }
    if (leader) umma_commit(BAR(PV_DRAIN));
    __syncwarp();
    mbar_wait(BAR(PV_DRAIN), 0);
  } else {
    // ------------------------------------------------------------------ softmax groups + epilogue
    asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
    const int w = (warp - 4) >> 2;               // group
    const int row = ((warp & 3) << 5) + lane;    // row of the tile == TMEM lane
    const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t tm_s = tmem + w * BLK + lane_off;                    // this group's S buffer
    const uint32_t tm_p = tmem + TM_P + w * (BLK / 2) + lane_off;       // and its P buffer
    int used = 0;               // tiles this group has taken so far, over all items
    bool ok = true;
    for (int n = 0; ok; n++) {
      int item, cnt;
      if (!get_item(n, item, cnt)) break;
      const PersistItem it = decode_item<MODE>(p, item);
      const int qt = it.qt, h = it.h, b = it.b;
      const int last_kb = kListIn ? it.list[cnt - 1] : it.kb0 + cnt - 1;
      const int ragged_valid = (last_kb == p.NKB - 1) ? (p.Nk - last_kb * BLK) : BLK;
      float m_ref = 0.f;
      uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};
      for (int t = w; t < cnt && ok; t += 2) {       // the groups take alternate key tiles
        ok = __all_sync(FULLM, wait_or_stop(S_FULL + w, used & 1, kWhereSFull, t));   // warp-uniform: aligned ops follow
        if (!ok) break;
        tc_fence_after();
        uint32_t s[BLK];
#pragma unroll
        for (int c = 0; c < NCH; c++) tmem_ld32(tm_s + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive(BAR(S_FREE + w));     // the tile is in registers: Q K^T of this group's next tile may overwrite it
        if (t == cnt - 1 && ragged_valid < BLK) {
#pragma unroll
          for (int j = 0; j < BLK; j++)
            if (j >= ragged_valid) s[j] = 0xff800000u;
        }
        if (t < 2) {
          if (t == 0) {
            // the first tile's row maximum is the reference of the whole row, for both groups
            float mx8[8];
#pragma unroll
            for (int u = 0; u < 8; u++) mx8[u] = fmaxf(__uint_as_float(s[2 * u]), __uint_as_float(s[2 * u + 1]));
#pragma unroll
            for (int j = 16; j < BLK; j += 16) {
#pragma unroll
              for (int u = 0; u < 8; u++)
                mx8[u] = max3f(mx8[u], __uint_as_float(s[j + 2 * u]), __uint_as_float(s[j + 2 * u + 1]));
            }
            m_ref = p.scale_log2 *
                    fmaxf(max3f(mx8[0], mx8[1], mx8[2]), fmaxf(max3f(mx8[3], mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])));
            mref_s[row] = m_ref;
            mbar_arrive(BAR(MREF));
          } else {
            ok = __all_sync(FULLM, wait_or_stop(MREF, n & 1, kFastMref, t));
            if (!ok) break;
            m_ref = mref_s[row];
          }
        }
        const uint64_t c2 = pack_f32x2(p.scale_log2, p.scale_log2);
        const uint64_t nm2 = pack_f32x2(-m_ref, -m_ref);
#pragma unroll
        for (int c = 0; c < NCH; c++) {
          uint32_t pk[16];
#pragma unroll
          for (int j = 0; j < 16; j++) {
            float x0, x1;
            unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(s[c * 32 + 2 * j]), __uint_as_float(s[c * 32 + 2 * j + 1])),
                                   c2, nm2), x0, x1);
            const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
            sum2[j & 3] = add_f32x2(sum2[j & 3], pack_f32x2(p0, p1));
            pk[j] = pack_bf16x2(p0, p1);
          }
          if (c == 0 && used > 0) {
            // first store of the tile: the P V that read this group's previous P must have finished
            ok = __all_sync(FULLM, wait_or_stop(P_FREE + w, (used - 1) & 1, kFastPFree, t));
            if (!ok) break;
          }
          tmem_st16(tm_p + c * 16, pk);
          if (c == NCH / 2 - 1 || c == NCH - 1) {        // one half of the key axis is in tensor memory
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(BAR(P_FULL + 2 * w + (c == NCH - 1 ? 1 : 0)));
          }
        }
        if (ok) used++;
      }
      if (!ok) break;
      // ---- end of the item: row sums of both groups, accumulator out of tensor memory, rows to global memory
      float l_run;
      {
        float sa, sb;
        unpack_f32x2(add_f32x2(add_f32x2(sum2[0], sum2[1]), add_f32x2(sum2[2], sum2[3])), sa, sb);
        l_run = sa + sb;
      }
      // A row sum beyond 2^64 (or not finite) means the row outgrew its first-tile reference: the item is left
      // to the exact-rescaling kernel.  (With 64-row tiles the upper 64 lanes hold no rows: the 128-row MMA filled
      // them from whatever follows the Q tile in shared memory, and their sums mean nothing.)
      if (row < BLK && !(l_run <= kFastRowSumLimit)) items[REDO + (n & 1)] = 1;
      lsum_s[w * 128 + row] = l_run;
      // the staged output tile of the item before must have been read by its TMA store before anybody writes the
      // staging buffer again; the thread that issued the store makes sure of it before it joins the barrier below
      if (kDirectOut && tid == 128) tma_store_wait_read();
      // (time-limited barriers, not bar.sync: a group that gave up must not leave the other one waiting for ever)
      mbar_arrive(BAR(LSUM_A));
      ok = __all_sync(FULLM, wait_or_stop(LSUM_A, n & 1, kPersistLsum, n));
      if (!ok) break;
      const float Lsum = l_run + lsum_s[(1 - w) * 128 + row];
      const bool redo = items[REDO + (n & 1)] != 0;
      mbar_arrive(BAR(LSUM_B));                           // everyone has read the sums and the flag
      ok = __all_sync(FULLM, wait_or_stop(LSUM_B, n & 1, kPersistLsum, n));
      if (!ok) break;
      if (tid == 128) {
        items[REDO + (n & 1)] = 0;
        if (redo) redo_list[atomicAdd(&p.status->redo_count, 1)] = item;
      }
      ok = __all_sync(FULLM, wait_or_stop(O_FULL, n & 1, kPersistOFull, n));
      if (!ok) break;
      tc_fence_after();
      constexpr int HALF = D / 2;
      uint32_t o0[HALF];
#pragma unroll
      for (int c = 0; c < HALF / 32; c++)
        tmem_ld32(tmem + TM_O + lane_off + w * HALF + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&o0[c * 32]));
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(BAR(O_FREE));           // the accumulator is in registers: the next item's P V may start
      const int64_t grow = static_cast<int64_t>(qt) * BLK + row;
      const float inv = 1.0f / Lsum;
      if (kDirectOut) {
        // The tile goes out through shared memory (128-byte swizzled) and one TMA store.  Rows written straight
        // from registers, even as whole 32-byte sectors, kept these warps busy for about 2000 cycles per item
        // (1024 sector requests at 256-byte stride); the store's read of the staging buffer is only waited for
        // when the next item is about to write it.
        if (row < BLK) {
          uint8_t* stage = smem + L::kStage;
#pragma unroll
          for (int g = 0; g < HALF / 8; g++) {
            const int col = w * HALF + g * 8;
            const int panel = col >> 6, chunk = (col & 63) >> 3;
            uint4 val;
            val.x = pack_bf16x2(__uint_as_float(o0[g * 8 + 0]) * inv, __uint_as_float(o0[g * 8 + 1]) * inv);
            val.y = pack_bf16x2(__uint_as_float(o0[g * 8 + 2]) * inv, __uint_as_float(o0[g * 8 + 3]) * inv);
            val.z = pack_bf16x2(__uint_as_float(o0[g * 8 + 4]) * inv, __uint_as_float(o0[g * 8 + 5]) * inv);
            val.w = pack_bf16x2(__uint_as_float(o0[g * 8 + 6]) * inv, __uint_as_float(o0[g * 8 + 7]) * inv);
            *reinterpret_cast<uint4*>(stage + panel * QPANEL_BYTES + row * 128 + ((chunk ^ (row & 7)) << 4)) = val;
          }
          if (!redo && w == 0 && p.lse != nullptr && grow < p.Nq)
            p.lse[(static_cast<int64_t>(b) * p.H + h) * p.Nq + grow] = (m_ref + log2f(Lsum)) * 0.6931471805599453f;
        }
        fence_proxy_async();
        mbar_arrive(BAR(STAGE_FULL));
        if (tid == 128) {
          if (wait_or_stop(STAGE_FULL, n & 1, kPersistStage, n) && !redo) {
            for (int pn = 0; pn < NPANEL; pn++)
              tma_store_4d(&tmo, smem_u32(smem + L::kStage) + pn * QPANEL_BYTES, pn * 64, qt * BLK, h, b);
            tma_store_commit();
          }
        }
      } else if (!redo && row < BLK) {
        // normalised fp32 partial of this split + its log2 LSE, for merge_splits_kernel
        float* prow = p.part_o + (static_cast<int64_t>(item) * BLK + row) * D + w * HALF;
#pragma unroll
        for (int g = 0; g < HALF / 8; g++) {
          uint32_t r[8];
#pragma unroll
          for (int i = 0; i < 8; i++) r[i] = __float_as_uint(__uint_as_float(o0[g * 8 + i]) * inv);
          st_global_v8(prow + g * 8, r);
        }
        if (w == 0) p.part_lse2[static_cast<int64_t>(item) * BLK + row] = m_ref + log2f(Lsum);
      }
      item_done(n);
    }
    if (kDirectOut && tid == 128) tma_store_wait_read();     // the last store has read the staging buffer
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 2) tmem_dealloc(tmem, 512);
}

}  // namespace avsa
