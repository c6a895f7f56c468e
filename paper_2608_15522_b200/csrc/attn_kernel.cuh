// Flash-attention forward tile kernel for sm_100a, shared by the block-sparse self-attention
// (Eq. 10) and the first pass of the cross-attention (Eq. 1).
//
// One CTA per work item = one query tile and a list of key tiles.  Warp roles:
//   warp 0      TMA producer: Q tile once, then the listed K tiles through a 3-stage ring
//   warp 3      TMA producer: the listed V tiles through a 3-stage ring
//   warp 1      MMA issuer: S = Q K^T (operands in shared memory) and O += P V (P in tensor memory)
//   warp 2      tensor-memory allocation
//   warps 4-7   softmax group 0: even tiles of the list, accumulator O0
//   warps 8-11  softmax group 1: odd tiles of the list, accumulator O1
// The two groups keep independent running maxima / sums; the epilogue merges (O0, m0, l0) and
// (O1, m1, l1) exactly as a two-way split of the key axis.
// Tensor memory: S0 | S1 | O0 | O1, 128 columns each; P (bf16) overwrites the front of its S buffer.
//
// MODE_LIST   key tiles come from an explicit ascending list; the output tile is converted to bf16
//             and TMA-stored; optional natural-log LSE.
// MODE_RANGE  key tiles are a contiguous range (one split of the key axis); the output is a partial
//             result (fp32 rows normalised by their own sum, plus the log2-domain LSE of the split).
// MODE_RANGE_DIRECT  the whole key axis as one range (few keys): output written like MODE_LIST.
#pragma once
#include "avsa_common.cuh"
#include "sm100_ptx.cuh"

namespace avsa {

constexpr int kAttnThreads = 384;
// Register reallocation between the roles (setmaxnreg): a CTA is launched with 384 x 168 = 64512 registers; afterwards
// its four service warps hold 64 each and its eight softmax warps 216: 128 x 64 + 256 x 216 = 63488.  A request
// beyond what the CTA holds makes setmaxnreg.inc wait for ever, which no time-limited barrier catches: the sum has
// to stay below the launch figure.
constexpr int kLaunchRegs = 168, kServiceRegs = 64, kSoftmaxRegs = 216;
static_assert(4 * 32 * kServiceRegs + 8 * 32 * kSoftmaxRegs <= kAttnThreads * kLaunchRegs, "setmaxnreg budget exceeded");
constexpr int kStages = 3;
constexpr float kRescaleThreshold = 8.0f;   // log2 units: O is rescaled only when a row max grew by more

enum { MODE_LIST = 0, MODE_RANGE = 1, MODE_RANGE_DIRECT = 2 };

enum AttnWhere {
  kWhereQFull = 1, kWhereKEmpty, kWhereVEmpty, kWhereKFull, kWhereVFull, kWherePFull, kWhereSFull, kWhereFinal,
  kWhereSmemAlign, kWhereList
};

template <int BLK, int D>
struct AttnSmem {
  static constexpr int kTileBytes = BLK * D * 2;
  static constexpr int kQBytes = 128 * D * 2;        // 128 MMA rows; only BLK of them are loaded
  static constexpr int kQ = 0;
  static constexpr int kK = kQBytes;
  static constexpr int kV = kK + kStages * kTileBytes;
  static constexpr int kBars = kV + kStages * kTileBytes;
  static constexpr int kNumBars = 1 + 4 * kStages + 2 + 4 + 1;
  static constexpr int kStats = kBars + kNumBars * 8;          // float [2][2][128]: m, l per group and row
  static constexpr int kMisc = kStats + 2 * 2 * 128 * 4;       // tmem base, abort flag
  static constexpr int kTotal = kMisc + 16;
};

struct AttnParams {
  // MODE_LIST
  const int32_t* col_idx;   // [B,H,NB,NB]
  const int32_t* col_cnt;   // [B,H,NB]
  float* lse;               // [B,H,Nq] natural log, optional
  // MODE_RANGE
  float* part_o;            // [items][BLK][D] fp32
  float* part_lse2;         // [items][BLK]
  int n_split, tiles_per_split;
  // both
  StatusRecord* status;
  int H;
  int Nq, NQT;              // query rows and query tiles
  int Nk, NKB;              // key rows and key tiles
  float scale_log2;         // softmax_scale * log2(e)
};

// One work item of the tile kernel: query tile `bx` (MODE_LIST) or query tile / key split `bx`
// (range modes) of head `by`, batch item `bz`.  Called once per flagged work item by attn_redo_kernel;
// every thread of the CTA must call it.
template <int BLK, int D, int MODE>
__device__ __forceinline__ void attn_fwd_body(const CUtensorMap* tmq, const CUtensorMap* tmk, const CUtensorMap* tmv,
                                              const CUtensorMap* tmo, const AttnParams& p, int bx, int by, int bz) {
  using L = AttnSmem<BLK, D>;
  constexpr bool kListIn = (MODE == MODE_LIST);          // explicit list of key tiles (else a contiguous range)
  constexpr bool kDirectOut = (MODE != MODE_RANGE);      // final bf16 tile + LSE (else a partial result)
  constexpr int NPANEL = D / 64;
  constexpr int PANEL_BYTES = BLK * 128;        // one 64-channel panel of a K/V tile
  constexpr int QPANEL_BYTES = 128 * 128;
  extern __shared__ __align__(1024) uint8_t smem[];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int h = by, b = bz;
  int qt, split = 0, kb0 = 0, cnt;
  const int32_t* list = nullptr;
  if (kListIn) {
    qt = bx;
    const int row_id = (b * p.H + h) * p.NQT + qt;
    list = p.col_idx + static_cast<int64_t>(row_id) * p.NKB;
    cnt = p.col_cnt[row_id];
  } else {
    qt = bx / p.n_split;
    split = bx % p.n_split;
    kb0 = split * p.tiles_per_split;
    cnt = min(p.NKB, kb0 + p.tiles_per_split) - kb0;
  }
  const int item = ((b * p.H + h) * p.NQT + qt) * (kListIn ? 1 : p.n_split) + split;
  // ---- validation: nothing is loaded through a bad list entry
  {
    int bad = (cnt < 1 || cnt > p.NKB) ? 1 : 0;
    if (kListIn) {
      const int n = min(max(cnt, 0), p.NKB);
      for (int t = tid; t < n; t += kAttnThreads) {
        const int kb = list[t];
        const int prev = t > 0 ? list[t - 1] : -1;
        if (kb < 0 || kb >= p.NKB || kb <= prev) bad = 1;
      }
    }
    const bool misaligned = (smem_u32(smem) & 1023u) != 0u;
    if (misaligned) bad = 1;
    const int any_bad = __syncthreads_or(bad);
    if (any_bad) {
      if (tid == 0)
        report_status(p.status, misaligned ? AVSA_ERR_CUDA : AVSA_ERR_BAD_MASK, misaligned ? kWhereSmemAlign : kWhereList,
                      item, cnt);
      return;
    }
  }

  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBars);
  const uint32_t bar0 = smem_u32(bars);
  auto BAR = [&](int i) { return bar0 + static_cast<uint32_t>(i) * 8u; };
  constexpr int Q_FULL = 0, K_FULL = 1, K_EMPTY = 1 + kStages, V_FULL = 1 + 2 * kStages, V_EMPTY = 1 + 3 * kStages,
                S_FULL = 1 + 4 * kStages, P_FULL = S_FULL + 2, FINAL = P_FULL + 4;   // P_FULL + 2*group + half
  float* stats = reinterpret_cast<float*>(smem + L::kStats);
  volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + L::kMisc);   // [0] tmem base, [1] abort

  if (tid == 0) {
    mbar_init(BAR(Q_FULL), 1);
    for (int s = 0; s < kStages; s++) {
      mbar_init(BAR(K_FULL + s), 1);
      mbar_init(BAR(K_EMPTY + s), 1);
      mbar_init(BAR(V_FULL + s), 1);
      mbar_init(BAR(V_EMPTY + s), 1);
    }
    for (int w = 0; w < 2; w++) {
      mbar_init(BAR(S_FULL + w), 1);
      mbar_init(BAR(P_FULL + 2 * w), 128);
      mbar_init(BAR(P_FULL + 2 * w + 1), 128);
    }
    mbar_init(BAR(FINAL), 1);
    misc[1] = 0u;
    fence_mbar_init();
    prefetch_tmap(tmq);
    prefetch_tmap(tmk);
    prefetch_tmap(tmv);
    if (kDirectOut) prefetch_tmap(tmo);
  }
  if (warp == 2) {
    // (the allocation permit is kept: attn_redo_kernel runs this body several times in one CTA, and with one
    // CTA per SM nobody else is waiting for it)
    tmem_alloc(smem_u32(smem + L::kMisc), 512);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = misc[0];
  const uint32_t TM_S[2] = {tmem + 0u, tmem + 128u};
  const uint32_t TM_O[2] = {tmem + 256u, tmem + 384u};

  // A wait that gives up: records where, raises the CTA-wide abort flag, and lets every role unwind.
  // The fast path is a single try_wait (the issuing thread's waits sit between MMA batches, so their
  // latency shows up as tensor-pipe bubbles).
  auto wait_or_abort = [&](int bar, uint32_t parity, int where, int tile) -> bool {
    if (mbar_try_wait(BAR(bar), parity)) return true;
    if (misc[1] != 0u) return false;
    if (mbar_wait(BAR(bar), parity)) return true;
    report_status(p.status, AVSA_ERR_TIMEOUT, where, item, tile);
    misc[1] = 1u;
    return false;
  };

  const int n_tiles[2] = {(cnt + 1) >> 1, cnt >> 1};

  // The four service warps (0-3) give registers to the eight softmax warps (4-11); each role
  // changes its own budget as the first thing it does.
  if (warp == 0 || warp == 3) {
    // ------------------------------------------------------------------ TMA producers: warp 0 K (and Q), warp 3 V
    asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
    const bool is_k = (warp == 0);
    const CUtensorMap* tm = is_k ? tmk : tmv;
    const int FULL = is_k ? K_FULL : V_FULL, EMPTY = is_k ? K_EMPTY : V_EMPTY;
    const uint32_t base = smem_u32(smem + (is_k ? L::kK : L::kV));
    if (is_k && lane == 0) {
      mbar_expect_tx(BAR(Q_FULL), BLK * D * 2);
      for (int pn = 0; pn < NPANEL; pn++)
        tma_load_4d(smem_u32(smem + L::kQ) + pn * QPANEL_BYTES, tmq, BAR(Q_FULL), pn * 64, qt * BLK, h, b);
    }
    int s = 0, fpar = 0;     // stage, and the parity of the "empty" phase to wait for once the ring has wrapped
    for (int t0 = 0; t0 < cnt; t0 += 32) {
      int mine = kb0 + t0 + lane;
      if (kListIn) mine = (t0 + lane < cnt) ? list[t0 + lane] : 0;
      const int nn = min(32, cnt - t0);
      for (int j = 0; j < nn; j++) {
        const int kb = __shfl_sync(0xffffffffu, mine, j);
        const int t = t0 + j;
        if (lane == 0) {
          bool ok = true;
          if (t >= kStages) ok = wait_or_abort(EMPTY + s, fpar, is_k ? kWhereKEmpty : kWhereVEmpty, t);
          if (ok) {
            mbar_expect_tx(BAR(FULL + s), L::kTileBytes);
            for (int pn = 0; pn < NPANEL; pn++)
              tma_load_4d(base + s * L::kTileBytes + pn * PANEL_BYTES, tm, BAR(FULL + s), pn * 64, kb * BLK, h, b);
          }
        }
        if (++s == kStages) { s = 0; if (t >= kStages) fpar ^= 1; }
      }
      if (__any_sync(0xffffffffu, misc[1] != 0u)) break;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
    {
      // The whole warp runs this loop (uniform control flow keeps stage indices, addresses and descriptors in
      // the uniform datapath); one elected lane issues the MMAs and commits.  The issuing lane must keep the
      // tensor pipe's queue full (one MMA retires every 64 cycles), so per-MMA scalar work is kept minimal.
      const bool leader = elect_one_sync();
      constexpr uint32_t idesc_qk = make_idesc_bf16(128, BLK, 0, 0);
      constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, 0, 1);
      constexpr uint32_t desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);            // SBO 1024 B, version, 128B swizzle
      const uint32_t q_lo = ((smem_u32(smem + L::kQ) & 0x3FFFFu) >> 4) | (1u << 16);  // LBO field unused for K-major
      const uint32_t k_lo0 = ((smem_u32(smem + L::kK) & 0x3FFFFu) >> 4) | (1u << 16);
      const uint32_t v_lo0 = ((smem_u32(smem + L::kV) & 0x3FFFFu) >> 4) | (static_cast<uint32_t>(PANEL_BYTES >> 4) << 16);
      const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem, 0);
      auto desc64 = [](uint32_t lo) { return (static_cast<uint64_t>(desc_hi) << 32) | lo; };
      auto wait_all = [&](int bar, uint32_t parity, int where, int tile) -> bool {
        const bool r = wait_or_abort(bar, parity, where, tile);
        return __all_sync(0xffffffffu, r);
      };
      bool ok = wait_all(Q_FULL, 0, kWhereQFull, 0);
      int sk = 0, fk = 0;      // stage / fill parity of the tile whose S is issued
      int sv = 0, fv = 0;      // same for the tile whose P V is issued
      if (ok) ok = wait_all(K_FULL + 0, 0, kWhereKFull, 0);
      for (int t = 0; t <= cnt && ok; t++) {
        if (t < cnt) {
          // K tile t has been waited for already (end of the previous iteration): issue at once
          const int w = t & 1;
          tc_fence_after();
          const uint32_t k_lo = k_lo0 + sk * (L::kTileBytes >> 4);
          const uint32_t tm_s = tmem_u + (w << 7);
          if (leader) {
#pragma unroll
            for (int ks = 0; ks < D / 16; ks++) {
              const uint32_t qoff = ((ks >> 2) * QPANEL_BYTES + (ks & 3) * 32) >> 4;
              const uint32_t koff = ((ks >> 2) * PANEL_BYTES + (ks & 3) * 32) >> 4;
              umma_ss(tm_s, desc64(q_lo + qoff), desc64(k_lo + koff), idesc_qk, ks > 0 ? 1u : 0u);
            }
            umma_commit(BAR(S_FULL + w));
            umma_commit(BAR(K_EMPTY + sk));
          }
          __syncwarp();
          if (++sk == kStages) { sk = 0; fk ^= 1; }
        }
        // Waits whose data arrived long ago are taken here, in the shadow of the running softmax, so that
        // nothing but the wait for P stands between P's arrival and the next two MMA batches.
        if (t >= 1) {
          ok = wait_all(V_FULL + sv, fv, kWhereVFull, t - 1);
          if (!ok) break;
        }
        if (t + 1 < cnt) {
          ok = wait_all(K_FULL + sk, fk, kWhereKFull, t + 1);
          if (!ok) break;
        }
        if (t >= 1) {
          const int u = t - 1, w = u & 1, i = u >> 1;
          // P arrives in two halves of the key axis: the first half of the product starts while the
          // softmax group is still exponentiating the second half
          ok = wait_all(P_FULL + 2 * w, i & 1, kWherePFull, u);
          if (!ok) break;
          tc_fence_after();
          const uint32_t v_lo = v_lo0 + sv * (L::kTileBytes >> 4);
          const uint32_t tm_p = tmem_u + (w << 7), tm_o = tmem_u + 256u + (w << 7);
          const uint32_t acc0 = i > 0 ? 1u : 0u;
          if (leader) {
#pragma unroll
            for (int ks = 0; ks < BLK / 32; ks++)
              umma_ts(tm_o, tm_p + ks * 8, desc64(v_lo + ks * (2048 >> 4)), idesc_pv, ks > 0 ? 1u : acc0);
          }
          __syncwarp();
          ok = wait_all(P_FULL + 2 * w + 1, i & 1, kWherePFull, u);
          if (!ok) break;
          tc_fence_after();
          if (leader) {
#pragma unroll
            for (int ks = BLK / 32; ks < BLK / 16; ks++)
              umma_ts(tm_o, tm_p + ks * 8, desc64(v_lo + ks * (2048 >> 4)), idesc_pv, 1u);
            umma_commit(BAR(V_EMPTY + sv));
          }
          __syncwarp();
          if (++sv == kStages) { sv = 0; fv ^= 1; }
        }
      }
      if (ok && leader) umma_commit(BAR(FINAL));
      __syncwarp();
    }
  } else if (warp == 2) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
  } else {
    // ------------------------------------------------------------------ softmax groups + epilogue
    asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
    const int w = (warp - 4) >> 2;               // group
    const int row = ((warp & 3) << 5) + lane;    // row of the tile == TMEM lane
    const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const int nw = n_tiles[w];
    const int last_kb = (kListIn) ? list[cnt - 1] : kb0 + cnt - 1;
    const int ragged_valid = (last_kb == p.NKB - 1) ? (p.Nk - last_kb * BLK) : BLK;   // valid keys of the last tile
    float m_run = -INFINITY, l_run = 0.f;
    bool ok = true;
    for (int i = 0; i < nw && ok; i++) {
      const int t = 2 * i + w;
      ok = wait_or_abort(S_FULL + w, i & 1, kWhereSFull, t);
      if (!ok) break;
      tc_fence_after();
      uint32_t s[BLK];
#pragma unroll
      for (int c = 0; c < BLK / 32; c++)
        tmem_ld32(TM_S[w] + lane_off + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
      tmem_wait_ld();
      if (t == cnt - 1 && ragged_valid < BLK) {
#pragma unroll
        for (int j = 0; j < BLK; j++)
          if (j >= ragged_valid) s[j] = 0xff800000u;
      }
      float mx8[8];                                                  // eight independent chains
#pragma unroll
      for (int u = 0; u < 8; u++) mx8[u] = fmaxf(__uint_as_float(s[2 * u]), __uint_as_float(s[2 * u + 1]));
#pragma unroll
      for (int j = 16; j < BLK; j += 16) {
#pragma unroll
        for (int u = 0; u < 8; u++)
          mx8[u] = max3f(mx8[u], __uint_as_float(s[j + 2 * u]), __uint_as_float(s[j + 2 * u + 1]));
      }
      const float mx = fmaxf(max3f(mx8[0], mx8[1], mx8[2]), fmaxf(max3f(mx8[3], mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])));
      const float m_new = fmaxf(m_run, mx * p.scale_log2);
      const bool need = (m_new - m_run) > kRescaleThreshold;     // true on the first tile (m_run = -inf)
      float factor = 1.f;
      if (need) {
        factor = fast_exp2(m_run - m_new);
        m_run = m_new;
      }
      if (i > 0 && __any_sync(0xffffffffu, need)) {
        // the previous P V of this group has finished (its completion precedes this S): O is stable
#pragma unroll
        for (int c = 0; c < D / 32; c++) {
          uint32_t o[32];
          tmem_ld32(TM_O[w] + lane_off + c * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; j++) o[j] = __float_as_uint(__uint_as_float(o[j]) * factor);
          tmem_st32(TM_O[w] + lane_off + c * 32, o);
        }
      }
      l_run *= factor;
      // p = exp2(s * c - m) on pairs: one packed FMA, two EX2, one packed add, one bf16x2 convert per pair
      const uint64_t c2 = pack_f32x2(p.scale_log2, p.scale_log2);
      const uint64_t nm2 = pack_f32x2(-m_run, -m_run);
      uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
      for (int c = 0; c < BLK / 32; c++) {
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
        tmem_st16(TM_S[w] + lane_off + c * 16, pk);
        if (c == BLK / 64 - 1) {          // first half of the keys is in tensor memory: let the MMA warp start on it
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(BAR(P_FULL + 2 * w));
        }
      }
      float sa, sb;
      unpack_f32x2(add_f32x2(add_f32x2(sum2[0], sum2[1]), add_f32x2(sum2[2], sum2[3])), sa, sb);
      const float sum = sa + sb;
      l_run += sum;
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(BAR(P_FULL + 2 * w + 1));
    }
    // publish this group's statistics, then merge the two halves of the key axis
    stats[(w * 2 + 0) * 128 + row] = m_run;
    stats[(w * 2 + 1) * 128 + row] = l_run;
    asm volatile("bar.sync 1, 256;" ::: "memory");
    ok = wait_or_abort(FINAL, 0, kWhereFinal, cnt);
    if (ok) {
      tc_fence_after();
      const float m0 = stats[0 * 128 + row], l0 = stats[1 * 128 + row];
      const bool have1 = n_tiles[1] > 0;
      const float m1 = have1 ? stats[2 * 128 + row] : -INFINITY;
      const float l1 = have1 ? stats[3 * 128 + row] : 0.f;
      const float m = fmaxf(m0, m1);
      const float a0 = fast_exp2(m0 - m), a1 = have1 ? fast_exp2(m1 - m) : 0.f;
      const float Lsum = a0 * l0 + a1 * l1;
      const float f0 = a0 / Lsum, f1 = a1 / Lsum;
      // group w handles channels [w*D/2, (w+1)*D/2) of every row
      constexpr int HALF = D / 2;
      uint8_t* stage = smem + L::kQ;     // the Q tile is dead once every MMA has finished
#pragma unroll
      for (int c = 0; c < HALF / 32; c++) {
        const int col0 = w * HALF + c * 32;
        uint32_t o0[32], o1[32];
        tmem_ld32(TM_O[0] + lane_off + col0, o0);
        if (have1) tmem_ld32(TM_O[1] + lane_off + col0, o1);
        tmem_wait_ld();
        float v[32];
#pragma unroll
        for (int j = 0; j < 32; j++) {
          v[j] = __uint_as_float(o0[j]) * f0;
          if (have1) v[j] = fmaf(__uint_as_float(o1[j]), f1, v[j]);
        }
        if (row < BLK) {
          if (kDirectOut) {
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
          } else {
            float4* dst = reinterpret_cast<float4*>(p.part_o + (static_cast<int64_t>(item) * BLK + row) * D + col0);
#pragma unroll
            for (int g = 0; g < 8; g++) dst[g] = make_float4(v[g * 4], v[g * 4 + 1], v[g * 4 + 2], v[g * 4 + 3]);
          }
        }
      }
      if (w == 0 && row < BLK) {
        const float lse2 = m + log2f(Lsum);
        if (kDirectOut) {
          if (p.lse != nullptr && qt * BLK + row < p.Nq)
            p.lse[(static_cast<int64_t>(b) * p.H + h) * p.Nq + qt * BLK + row] = lse2 * 0.6931471805599453f;
        } else {
          p.part_lse2[static_cast<int64_t>(item) * BLK + row] = lse2;
        }
      }
      if (kDirectOut) fence_proxy_async();
    }
    tc_fence_before();
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (kDirectOut && ok && warp == 4 && lane == 0) {
      for (int pn = 0; pn < NPANEL; pn++)
        tma_store_4d(tmo, smem_u32(smem + L::kQ) + pn * QPANEL_BYTES, pn * 64, qt * BLK, h, b);
      tma_store_commit();
      tma_store_wait_read();
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 2) tmem_dealloc(tmem, 512);
}

// Exact-rescaling pass behind the fast kernels: recomputes the work items they listed (normally none: then
// every CTA of this small grid returns at once).  CTA c takes entries c, c + gridDim.x, ...
template <int BLK, int D, int MODE = MODE_LIST>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_redo_kernel(const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
                 const __grid_constant__ CUtensorMap tmv, const __grid_constant__ CUtensorMap tmo,
                 const AttnParams p, const int* __restrict__ redo_list) {
  using L = AttnSmem<BLK, D>;
  extern __shared__ __align__(1024) uint8_t smem[];
  const int n_redo = p.status->redo_count;
  const int warp = threadIdx.x >> 5;
  for (int k = blockIdx.x; k < n_redo; k += gridDim.x) {
    const int item = redo_list[k];                     // list mode: (b*H + h)*NQT + qt; range modes: that * n_split + split
    const int per_bh = p.NQT * (MODE == MODE_LIST ? 1 : p.n_split);
    const int bx = item % per_bh, bh = item / per_bh;
    attn_fwd_body<BLK, D, MODE>(&tmq, &tmk, &tmv, &tmo, p, bx, bh % p.H, bh / p.H);
    // back to the launch state for the next item: every warp at the launch register count, barriers invalidated
    if (warp < 4) {
      asm volatile("setmaxnreg.inc.sync.aligned.u32 168;");
    } else {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 168;");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int i = 0; i < L::kNumBars; i++) mbar_inval(smem_u32(smem + L::kBars) + i * 8);
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------------------------------------
// Merge of the key-axis splits written by MODE_RANGE: for every query row, combine the normalised
// partial outputs with weights exp2(lse2_split - max) and write bf16 rows and the natural-log LSE.
// With a row map the result of compact row r goes to row row_map[b][r] of the output (rows mapped to
// a negative index are skipped): that is how recomputed protected rows are scattered back.
// ------------------------------------------------------------------------------------------------
// (`block`, `tid`: index of a group of 128 threads and the thread's place in it, so that another kernel can run
// this work in part of its grid)
template <int BLK, int D>
__device__ __forceinline__ void merge_splits_rows(int block, int tid, const float* __restrict__ part_o,
                                                  const float* __restrict__ part_lse2, int n_split, int NQT, int Nq,
                                                  int H, int total_rows, __nv_bfloat16* __restrict__ o, int64_t o_sb,
                                                  int64_t o_sh, int64_t o_sn, float* __restrict__ lse,
                                                  const int32_t* __restrict__ row_map, int row_map_stride, int n_out) {
  constexpr int TPR = D / 4;
  const int rg = block * (128 / TPR) + tid / TPR;
  const int c4 = tid % TPR;
  if (rg >= total_rows) return;
  const int bh = rg / Nq, qrow = rg % Nq;
  const int b = bh / H, h = bh % H;
  int out_row = qrow;
  if (row_map != nullptr) {
    out_row = row_map[static_cast<int64_t>(b) * row_map_stride + qrow];
    if (out_row < 0 || out_row >= n_out) return;
  }
  const int qt = qrow / BLK, r = qrow % BLK;
  const int64_t item0 = (static_cast<int64_t>(bh) * NQT + qt) * n_split;
  float M = -INFINITY;
  for (int s = 0; s < n_split; s++) M = fmaxf(M, part_lse2[(item0 + s) * BLK + r]);
  float W = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s = 0; s < n_split; s++) {
    const float w = exp2f(part_lse2[(item0 + s) * BLK + r] - M);
    const float4 v = *reinterpret_cast<const float4*>(part_o + ((item0 + s) * BLK + r) * D + c4 * 4);
    W += w;
    acc.x = fmaf(w, v.x, acc.x);
    acc.y = fmaf(w, v.y, acc.y);
    acc.z = fmaf(w, v.z, acc.z);
    acc.w = fmaf(w, v.w, acc.w);
  }
  const float inv = 1.0f / W;
  if (o != nullptr) {
    uint2 pk;
    pk.x = pack_bf16x2(acc.x * inv, acc.y * inv);
    pk.y = pack_bf16x2(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(o + b * o_sb + h * o_sh + out_row * o_sn + c4 * 4) = pk;
  }
  if (c4 == 0 && lse != nullptr) lse[static_cast<int64_t>(bh) * n_out + out_row] = (M + log2f(W)) * 0.6931471805599453f;
}

template <int BLK, int D>
__global__ void __launch_bounds__(128) merge_splits_kernel(const float* __restrict__ part_o,
                                                           const float* __restrict__ part_lse2, int n_split, int NQT,
                                                           int Nq, int H, int total_rows, __nv_bfloat16* __restrict__ o,
                                                           int64_t o_sb, int64_t o_sh, int64_t o_sn,
                                                           float* __restrict__ lse, const int32_t* __restrict__ row_map,
                                                           int row_map_stride, int n_out) {
  merge_splits_rows<BLK, D>(blockIdx.x, threadIdx.x, part_o, part_lse2, n_split, NQT, Nq, H, total_rows, o, o_sb, o_sh,
                            o_sn, lse, row_map, row_map_stride, n_out);
}

}  // namespace avsa
