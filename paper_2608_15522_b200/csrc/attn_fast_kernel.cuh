// Fast variant of the flash-attention tile kernel: no rescaling, one shared output accumulator, S handed
// back as soon as it is in registers, and two MMA-issuing warps.
//
// In attn_fwd_kernel each softmax group owns one S buffer (overwritten in place by P) and one output
// accumulator that is rescaled when the row maximum grows.  S for a group's next tile can only be issued
// after the P V of its current tile, and that per-group cycle (S -> softmax -> P -> P V -> next S) bounds
// the kernel: the groups idle while their next S is made.  Here:
//   * every row keeps ONE reference maximum, the maximum of its first tile.  Probabilities are
//     exp2(s*c - m_ref); they may exceed 1 for later tiles, which fp32 accumulation and bf16 P tolerate
//     (same relative precision at any magnitude) as long as nothing overflows.  No per-tile maximum, no
//     rescaling: both groups add into the same accumulator O and their row sums simply add up;
//   * tensor memory is S0 | S1 | O | P0 | P1.  The groups still take alternate key tiles, but P has its own
//     buffer: a group releases its S buffer the moment the tile is in registers, so Q K^T of its next tile
//     runs under the exponentials of the current one, and it waits for the P V that read its previous P
//     only at the first store of the new P;
//   * two warps issue MMAs, one the Q K^T products and one the P V products: every MMA and every barrier
//     wait costs the issuing thread tens of cycles, which one warp doing both would serialise.
// A row whose sum, relative to m_ref, ends above 2^64 (or not finite) outgrew its reference: the CTA appends
// its work item to `redo_list` (count in the status record), and attn_redo_kernel, a small grid launched
// behind this kernel, recomputes the listed items with exact rescaling.
//
// Producer warps, shared-memory rings, list validation and bounded waits are as in attn_fwd_kernel.
#pragma once
#include "attn_kernel.cuh"

namespace avsa {

// Debug builds only: per-phase cycle accounting of the softmax and MMA warps of CTA (0,0,0).
#ifdef AVSA_TRACE
#define AVSA_PHASE(k) do { const uint32_t now_ = clock(); ph[k] += now_ - ph_t; ph_t = now_; } while (0)
#else
#define AVSA_PHASE(k) do { } while (0)
#endif
constexpr float kFastRowSumLimit = 1.8446744e19f;   // 2^64: largest row sum, relative to the reference, the fast path accepts

template <int BLK, int D>
struct FastSmem {
  static constexpr int kTileBytes = BLK * D * 2;
  static constexpr int kQBytes = 128 * D * 2;
  static constexpr int kQ = 0;
  static constexpr int kK = kQBytes;
  static constexpr int kV = kK + kStages * kTileBytes;
  static constexpr int kBars = kV + kStages * kTileBytes;
  static constexpr int kNumBars = 1 + 4 * kStages + 2 + 2 + 4 + 2 + 1 + 1 + 1;
  static constexpr int kStats = kBars + kNumBars * 8;          // float [2][128]: per group, first-tile maximum, later row sum
  static constexpr int kMisc = kStats + 2 * 128 * 4;           // tmem base, stop flag, redo flag
  static constexpr int kTotal = kMisc + 16;
};

enum FastWhere { kFastSFree = 61, kFastPFree, kFastMref };

// List mode only (the block-sparse self-attention call); the range modes stay with attn_fwd_kernel.
template <int BLK, int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_fast_kernel(const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
                 const __grid_constant__ CUtensorMap tmv, const __grid_constant__ CUtensorMap tmo,
                 const AttnParams p, int* __restrict__ redo_list) {
  using L = FastSmem<BLK, D>;
  constexpr int NPANEL = D / 64;
  constexpr int PANEL_BYTES = BLK * 128;
  constexpr int QPANEL_BYTES = 128 * 128;
  extern __shared__ __align__(1024) uint8_t smem[];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int h = blockIdx.y, b = blockIdx.z;
  const int qt = blockIdx.x;
  const int item = (b * p.H + h) * p.NQT + qt;
  const int32_t* list = p.col_idx + static_cast<int64_t>(item) * p.NKB;
  const int cnt = p.col_cnt[item];

  // ---- validation: nothing is loaded through a bad list entry (the fallback kernel reports it too)
  {
    int bad = (cnt < 1 || cnt > p.NKB) ? 1 : 0;
    const int n = min(max(cnt, 0), p.NKB);
    for (int t = tid; t < n; t += kAttnThreads) {
      const int kb = list[t];
      const int prev = t > 0 ? list[t - 1] : -1;
      if (kb < 0 || kb >= p.NKB || kb <= prev) bad = 1;
    }
    const bool misaligned = (smem_u32(smem) & 1023u) != 0u;
    if (misaligned) bad = 1;
    const int any_bad = __syncthreads_or(bad);
    if (any_bad) {
      if (tid == 0)
        report_status(p.status, misaligned ? AVSA_ERR_CUDA : AVSA_ERR_BAD_MASK, misaligned ? kWhereSmemAlign : kWhereList,
                      item, cnt);
      return;     // nothing to recompute: the item is refused, not deferred
    }
  }

  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBars);
  const uint32_t bar0 = smem_u32(bars);
  auto BAR = [&](int i) { return bar0 + static_cast<uint32_t>(i) * 8u; };
  constexpr int Q_FULL = 0, K_FULL = 1, K_EMPTY = 1 + kStages, V_FULL = 1 + 2 * kStages, V_EMPTY = 1 + 3 * kStages,
                S_FULL = 1 + 4 * kStages /* + group */, S_FREE = S_FULL + 2 /* + group: S is in registers */,
                P_FULL = S_FREE + 2 /* + 2*group + half */, P_FREE = P_FULL + 4 /* + group: its P V has finished */,
                FINAL = P_FREE + 2, MREF = FINAL + 1, QK_DRAIN = MREF + 1;
  // tensor memory: S of group 0 | S of group 1 | O | P of group 0 | P of group 1
  constexpr uint32_t TM_O = 2 * BLK, TM_P = 2 * BLK + D;
  constexpr int NCH = BLK / 32;         // 32-column chunks per thread and tile
  float* stats = reinterpret_cast<float*>(smem + L::kStats);
  volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + L::kMisc);   // [0] tmem base, [1] stop, [2] redo

  if (tid == 0) {
    mbar_init(BAR(Q_FULL), 1);
    for (int s = 0; s < kStages; s++) {
      mbar_init(BAR(K_FULL + s), 1);
      mbar_init(BAR(K_EMPTY + s), 1);
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
    mbar_init(BAR(FINAL), 1);
    mbar_init(BAR(MREF), 128);
    mbar_init(BAR(QK_DRAIN), 1);
    misc[1] = 0u;
    misc[2] = 0u;
    fence_mbar_init();
    prefetch_tmap(&tmq);
    prefetch_tmap(&tmk);
    prefetch_tmap(&tmv);
    prefetch_tmap(&tmo);
  }
  if (warp == 2) {
    tmem_alloc(smem_u32(smem + L::kMisc), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = misc[0];

  // A wait that gives up when the CTA has been stopped (time limit reached somewhere, or the item deferred).
  auto wait_or_stop = [&](int bar, uint32_t parity, int where, int tile) -> bool {
    if (mbar_try_wait(BAR(bar), parity)) return true;
    const long long t0 = clock64();
    while (true) {
      if (misc[1] != 0u) return false;
      if (mbar_try_wait(BAR(bar), parity)) return true;
      if (clock64() - t0 > AVSA_WAIT_LIMIT_CYCLES) {
        report_status(p.status, AVSA_ERR_TIMEOUT, where, item, tile);
        misc[1] = 1u;
        return false;
      }
    }
  };

  if (warp == 0 || warp == 3) {
    // ------------------------------------------------------------------ TMA producers: warp 0 K (and Q), warp 3 V
    asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
    const bool is_k = (warp == 0);
    const CUtensorMap* tm = is_k ? &tmk : &tmv;
    const int FULL = is_k ? K_FULL : V_FULL, EMPTY = is_k ? K_EMPTY : V_EMPTY;
    const uint32_t base = smem_u32(smem + (is_k ? L::kK : L::kV));
    if (is_k && lane == 0) {
      mbar_expect_tx(BAR(Q_FULL), BLK * D * 2);
      for (int pn = 0; pn < NPANEL; pn++)
        tma_load_4d(smem_u32(smem + L::kQ) + pn * QPANEL_BYTES, &tmq, BAR(Q_FULL), pn * 64, qt * BLK, h, b);
    }
    int s = 0, fpar = 0;
    int issued = 0;          // lane 0: number of tiles whose load has been issued
    for (int t0 = 0; t0 < cnt; t0 += 32) {
      const int mine = (t0 + lane < cnt) ? list[t0 + lane] : 0;
      const int nn = min(32, cnt - t0);
      for (int j = 0; j < nn; j++) {
        const int kb = __shfl_sync(0xffffffffu, mine, j);
        const int t = t0 + j;
        if (lane == 0) {
          bool ok = true;
          if (t >= kStages) ok = wait_or_stop(EMPTY + s, fpar, is_k ? kWhereKEmpty : kWhereVEmpty, t);
          if (ok) {
            mbar_expect_tx(BAR(FULL + s), L::kTileBytes);
            for (int pn = 0; pn < NPANEL; pn++)
              tma_load_4d(base + s * L::kTileBytes + pn * PANEL_BYTES, tm, BAR(FULL + s), pn * 64, kb * BLK, h, b);
            issued = t + 1;
          }
        }
        if (++s == kStages) { s = 0; if (t >= kStages) fpar ^= 1; }
      }
      if (__any_sync(0xffffffffu, misc[1] != 0u)) break;
    }
    if (lane == 0 && misc[1] != 0u) {
      // stopped early: loads still in flight must land before this CTA's shared memory is given away
      if (is_k) mbar_wait(BAR(Q_FULL), 0);
      for (int t = max(0, issued - kStages); t < issued; t++) mbar_wait(BAR(FULL + t % kStages), (t / kStages) & 1);
    }
  } else if (warp == 1 || warp == 2) {
    // ------------------------------------------------------------------ MMA issuers: warp 1 Q K^T, warp 2 P V
    // Each MMA costs its issuing thread some tens of cycles, and so does every barrier wait: one warp
    // issuing both products of every tile is a serial bottleneck.  Two warps, each with one elected lane,
    // halve it; the Q K^T warp runs ahead as far as the S buffers and the K ring allow.
    asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
    const bool leader = elect_one_sync();
    constexpr uint32_t desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
    const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem, 0);
    auto desc64 = [](uint32_t lo) { return (static_cast<uint64_t>(desc_hi) << 32) | lo; };
    auto wait_all = [&](int bar, uint32_t parity, int where, int tile) -> bool {
      return __all_sync(0xffffffffu, wait_or_stop(bar, parity, where, tile));
    };
#ifdef AVSA_TRACE
    uint32_t ph[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    uint32_t ph_t = clock();
#endif
    bool ok = true;
    if (warp == 1) {
      constexpr uint32_t idesc_qk = make_idesc_bf16(128, BLK, 0, 0);
      const uint32_t q_lo = ((smem_u32(smem + L::kQ) & 0x3FFFFu) >> 4) | (1u << 16);
      const uint32_t k_lo0 = ((smem_u32(smem + L::kK) & 0x3FFFFu) >> 4) | (1u << 16);
      int sk = 0, fk = 0;      // ring stage / fill parity of the next K tile
      ok = wait_all(Q_FULL, 0, kWhereQFull, 0);
      for (int t = 0; t < cnt && ok; t++) {
        // S of tile t goes into its group's buffer, once the group has taken tile t-2 out of it
        const int j = t & 1, u = t >> 1;
        AVSA_PHASE(7);
        ok = wait_all(K_FULL + sk, fk, kWhereKFull, t);
        if (!ok) break;
        AVSA_PHASE(0);
        if (u > 0) {
          ok = wait_all(S_FREE + j, (u - 1) & 1, kFastSFree, t);
          if (!ok) break;
        }
        AVSA_PHASE(2);
        tc_fence_after();
        const uint32_t k_lo = k_lo0 + sk * (L::kTileBytes >> 4);
        const uint32_t tm_s = tmem_u + j * BLK;
        if (leader) {
          AVSA_STAMP(0, t, 0);
#pragma unroll
          for (int ks = 0; ks < D / 16; ks++) {
            const uint32_t qoff = ((ks >> 2) * QPANEL_BYTES + (ks & 3) * 32) >> 4;
            const uint32_t koff = ((ks >> 2) * PANEL_BYTES + (ks & 3) * 32) >> 4;
            umma_ss(tm_s, desc64(q_lo + qoff), desc64(k_lo + koff), idesc_qk, ks > 0 ? 1u : 0u);
          }
          umma_commit(BAR(S_FULL + j));
          umma_commit(BAR(K_EMPTY + sk));
          AVSA_STAMP(0, t, 1);
        }
        __syncwarp();
        AVSA_PHASE(1);
        if (++sk == kStages) { sk = 0; fk ^= 1; }
      }
      // On a stop, tensor memory must not be freed under a running MMA: wait for this warp's own.
      if (!ok) {
        if (leader) umma_commit(BAR(QK_DRAIN));
        __syncwarp();
        mbar_wait(BAR(QK_DRAIN), 0);
      }
    } else {
      constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, 0, 1);
      const uint32_t v_lo0 = ((smem_u32(smem + L::kV) & 0x3FFFFu) >> 4) | (static_cast<uint32_t>(PANEL_BYTES >> 4) << 16);
      int sv = 0, fv = 0;      // ring stage / fill parity of the next V tile
      // P V over one half of the key axis (k-step ks covers keys [16 ks, 16 ks + 16), 8 columns of P)
      auto issue_pv_phase = [&](uint32_t tm_buf, uint32_t v_lo, int ph_, uint32_t acc_first) {
#pragma unroll
        for (int kk = 0; kk < BLK / 32; kk++) {
          const int ks = ph_ * (BLK / 32) + kk;
          umma_ts(tmem_u + TM_O, tm_buf + ks * 8, desc64(v_lo + ks * (2048 >> 4)), idesc_pv, kk > 0 ? 1u : acc_first);
        }
      };
      for (int t = 0; t < cnt && ok; t++) {
        const int j = t & 1, u = t >> 1;
        AVSA_PHASE(7);
        ok = wait_all(V_FULL + sv, fv, kWhereVFull, t);
        if (!ok) break;
        AVSA_PHASE(2);
        // P arrives in two halves of the key axis: the first half of the product starts while the
        // softmax group is still exponentiating the second half
        ok = wait_all(P_FULL + 2 * j, u & 1, kWherePFull, t);
        if (!ok) break;
        AVSA_PHASE(3);
        tc_fence_after();
        const uint32_t v_lo = v_lo0 + sv * (L::kTileBytes >> 4);
        const uint32_t tm_buf = tmem_u + TM_P + j * (BLK / 2);
        if (leader) issue_pv_phase(tm_buf, v_lo, 0, t > 0 ? 1u : 0u);
        __syncwarp();
        AVSA_PHASE(4);
        ok = wait_all(P_FULL + 2 * j + 1, u & 1, kWherePFull, t);
        if (!ok) break;
        AVSA_PHASE(5);
        tc_fence_after();
        if (leader) {
          issue_pv_phase(tm_buf, v_lo, 1, 1u);
          umma_commit(BAR(P_FREE + j));
          umma_commit(BAR(V_EMPTY + sv));
        }
        __syncwarp();
        AVSA_PHASE(6);
        if (++sv == kStages) { sv = 0; fv ^= 1; }
      }
      // FINAL completes when every P V issued above has finished (every Q K^T finished before the P that
      // depends on it was made) -- also on the stop path, where the warp itself waits for it
      if (leader) umma_commit(BAR(FINAL));
      __syncwarp();
      if (!ok) mbar_wait(BAR(FINAL), 0);
    }
#ifdef AVSA_TRACE
    if (p.trace != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && lane == 0)
      for (int k = 0; k < 8; k++) p.trace[1536 + 64 + (warp - 1) * 8 + k] = ph[k];
#endif
  } else {
    // ------------------------------------------------------------------ softmax groups + epilogue
    asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
    const int w = (warp - 4) >> 2;               // group
    const int row = ((warp & 3) << 5) + lane;    // row of the tile == TMEM lane
    const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const int last_kb = list[cnt - 1];
    const int ragged_valid = (last_kb == p.NKB - 1) ? (p.Nk - last_kb * BLK) : BLK;
    float m_ref = 0.f, l_run = 0.f;
    uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};
    bool ok = true;
#ifdef AVSA_TRACE
    uint32_t ph[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    uint32_t ph_t = clock();
#endif
    const uint32_t tm_s = tmem + w * BLK + lane_off;                    // this group's S buffer
    const uint32_t tm_p = tmem + TM_P + w * (BLK / 2) + lane_off;       // and its P buffer
    for (int t = w, i = 0; t < cnt && ok; t += 2, i++) {       // the groups take alternate key tiles
      AVSA_PHASE(7);
      ok = __all_sync(0xffffffffu, wait_or_stop(S_FULL + w, i & 1, kWhereSFull, t));   // warp-uniform: aligned ops follow
      if (!ok) break;
      AVSA_PHASE(0);
      tc_fence_after();
      uint32_t s[BLK];
#pragma unroll
      for (int c = 0; c < NCH; c++) tmem_ld32(tm_s + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(BAR(S_FREE + w));     // the tile is in registers: Q K^T of this group's next tile may overwrite it
      AVSA_PHASE(1);
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
          stats[row] = m_ref;
          mbar_arrive(BAR(MREF));
        } else {
          ok = __all_sync(0xffffffffu, wait_or_stop(MREF, 0, kFastMref, t));
          if (!ok) break;
          m_ref = stats[row];
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
        if (c == 0 && i > 0) {
          // first store of the tile: the P V that read this group's previous P must have finished
          AVSA_PHASE(2);
          ok = __all_sync(0xffffffffu, wait_or_stop(P_FREE + w, (i - 1) & 1, kFastPFree, t));
          if (!ok) break;
          AVSA_PHASE(6);
        }
        tmem_st16(tm_p + c * 16, pk);
        if (c == NCH / 2 - 1 || c == NCH - 1) {        // one half of the key axis is in tensor memory
          AVSA_PHASE(c == NCH - 1 ? 4 : 2);
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(BAR(P_FULL + 2 * w + (c == NCH - 1 ? 1 : 0)));
          AVSA_PHASE(c == NCH - 1 ? 5 : 3);
        }
      }
    }
#ifdef AVSA_TRACE
    if (p.trace != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && lane == 0)
      for (int k = 0; k < 8; k++) p.trace[1536 + (warp - 4) * 8 + k] = ph[k];
#endif
    {
      float sa, sb;
      unpack_f32x2(add_f32x2(add_f32x2(sum2[0], sum2[1]), add_f32x2(sum2[2], sum2[3])), sa, sb);
      l_run = sa + sb;
    }
    // Probabilities are relative to the first tile's maximum and can exceed 1.  A row sum beyond 2^64 (or
    // not finite) means the row outgrew that reference: the item is left to the exact-rescaling kernel.
    if (ok && !(l_run <= kFastRowSumLimit)) misc[2] = 1u;
    // both groups share the reference, so their row sums just add up
    asm volatile("bar.sync 1, 256;" ::: "memory");     // everyone is past the first-tile exchange
    stats[w * 128 + row] = l_run;
    asm volatile("bar.sync 1, 256;" ::: "memory");
    const float l_other = stats[(1 - w) * 128 + row];
    // a stopped CTA writes nothing (FINAL completes on the stop path as well, so the flag is what decides)
    // (on a stop the MMA warp itself waits for FINAL; otherwise the wait here also keeps tensor memory alive
    // until the last MMA has finished, whether or not the result is used)
    ok = misc[1] == 0u && wait_or_stop(FINAL, 0, kWhereFinal, cnt) && misc[1] == 0u && misc[2] == 0u;
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after();
      const float mr = m_ref;
      const float Lsum = l_run + l_other;
      const float inv = 1.0f / Lsum;
      constexpr int HALF = D / 2;
      uint8_t* stage = smem + L::kQ;     // the Q tile is dead once every MMA has finished
#pragma unroll
      for (int c = 0; c < HALF / 32; c++) {
        const int col0 = w * HALF + c * 32;
        uint32_t o0[32];
        tmem_ld32(tmem + TM_O + lane_off + col0, o0);
        tmem_wait_ld();
        float v[32];
#pragma unroll
        for (int j = 0; j < 32; j++) v[j] = __uint_as_float(o0[j]) * inv;
        if (row < BLK) {
#pragma unroll
          for (int g = 0; g < 4; g++) {
            const int col = col0 + g * 8;
            const int panel = col >> 6, chunk = (col & 63) >> 3;
            uint4 val;
            val.x = pack_bf16x2(v[g * 8 + 0], v[g * 8 + 1]);
            val.y = pack_bf16x2(v[g * 8 + 2], v[g * 8 + 3]);
            val.z = pack_bf16x2(v[g * 8 + 4], v[g * 8 + 5]);
            val.w = pack_bf16x2(v[g * 8 + 6], v[g * 8 + 7]);
            *reinterpret_cast<uint4*>(stage + panel * QPANEL_BYTES + row * 128 + ((chunk ^ (row & 7)) << 4)) = val;
          }
        }
      }
      if (w == 0 && row < BLK && p.lse != nullptr && qt * BLK + row < p.Nq)
        p.lse[(static_cast<int64_t>(b) * p.H + h) * p.Nq + qt * BLK + row] = (mr + log2f(Lsum)) * 0.6931471805599453f;
      fence_proxy_async();
    }
    tc_fence_before();
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (ok && warp == 4 && lane == 0) {
      for (int pn = 0; pn < NPANEL; pn++)
        tma_store_4d(&tmo, smem_u32(smem + L::kQ) + pn * QPANEL_BYTES, pn * 64, qt * BLK, h, b);
      tma_store_commit();
      tma_store_wait_read();
    }
  }
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && misc[2] != 0u) redo_list[atomicAdd(&p.status->redo_count, 1)] = item;
  if (warp == 2) tmem_dealloc(tmem, 512);
}

}  // namespace avsa
