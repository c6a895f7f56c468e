// avsa_cross_attn_scores: audio->video cross-attention (Eq. 1) that also emits the per-video-token
// response scores (Eq. 2), in two passes over the keys.
//   pass 1  flash attention, key axis split across CTAs -> partial (O, LSE) -> merge -> O, row LSE
//   pass 2  for every key tile: S^T = K Q^T on the tensor cores, p = exp2(S^T c - lse_j), summed over
//           the queries -> per-head column sums -> fixed-order head sum with the beta/gamma blend
#include "attn_persist_kernel.cuh"

namespace avsa {

// ------------------------------------------------------------------------------------------------
// pass 2: column sums of the attention map.  One CTA keeps the queries of one (batch, head) in
// shared memory and walks a range of 128-key tiles.  S^T[key, query] accumulates in tensor memory
// (two buffers of up to 256 columns); two groups of 128 threads (one thread per key row) turn
// alternate buffers into row sums of exp2(S^T c - lse2[query]).
//   warp 0 TMA producer, warp 1 MMA issuer, warp 2 tensor-memory allocation,
//   warps 4-7 / 8-11 the two reduction groups.
// ------------------------------------------------------------------------------------------------
constexpr int kColThreads = 384;
constexpr int kColStages = 3;

struct ColsumParams {
  const float* lse;        // [B,H,Nq] natural log; used when part_lse2 is null
  const float* part_lse2;  // or the log2-domain LSEs of pass 1's key splits, [B,H,NQT,n_split,blk], merged here
  int n_split, NQT, blk;
  float* partial;          // [NCH][B,H,Nk]
  StatusRecord* status;
  int H, Nq, Nk, NKT;      // NKT = key tiles of 128
  int NCH, W;              // query chunks and their width (multiple of 16, <= 256)
  int n_range, tiles_per_range;
  float scale_log2;
};

template <int D>
struct ColsumSmem {
  static constexpr int kKTile = 128 * D * 2;
  static constexpr int kK = 0;
  static constexpr int kQ = kColStages * kKTile;      // NCH * W * D * 2 bytes follow
  static int bars_offset(int NCH, int W) { return kQ + NCH * W * D * 2; }
  static constexpr int kNumBars = 1 + 2 * kColStages + 4;
  static constexpr int kBarBytes = 128;               // keeps the lse table behind it 16-byte aligned
  static_assert(kNumBars * 8 <= kBarBytes, "barrier area too small");
  static int total(int NCH, int W) { return bars_offset(NCH, W) + kBarBytes + 512 * 4 + 16; }
};

enum ColWhere { kColQFull = 21, kColKEmpty, kColKFull, kColSEmpty, kColSFull };

template <int D>
__global__ void __launch_bounds__(kColThreads, 1)
colsum_kernel(const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk, const ColsumParams p) {
  using L = ColsumSmem<D>;
  constexpr int NPANEL = D / 64;
  constexpr int KPANEL_BYTES = 128 * 128;
  extern __shared__ __align__(1024) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int range = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int kt0 = range * p.tiles_per_range;
  const int ntile = min(p.NKT, kt0 + p.tiles_per_range) - kt0;
  const int item = (b * p.H + h) * p.n_range + range;
  const int W = p.W, NCH = p.NCH;
  const int q_chunk_bytes = W * D * 2, q_panel_bytes = W * 128;
  if (ntile <= 0) return;
  if ((smem_u32(smem) & 1023u) != 0u) {
    if (tid == 0) report_status(p.status, AVSA_ERR_CUDA, kWhereSmemAlign, item, 0);
    return;
  }
  const int bars_off = L::kQ + NCH * q_chunk_bytes;
  const uint32_t bar0 = smem_u32(smem + bars_off);
  auto BAR = [&](int i) { return bar0 + static_cast<uint32_t>(i) * 8u; };
  constexpr int Q_FULL = 0, K_FULL = 1, K_EMPTY = 1 + kColStages, S_FULL = 1 + 2 * kColStages, S_EMPTY = S_FULL + 2;
  float* lse2 = reinterpret_cast<float*>(smem + bars_off + L::kBarBytes);
  volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + bars_off + L::kBarBytes + 512 * 4);

  if (tid == 0) {
    mbar_init(BAR(Q_FULL), 1);
    for (int s = 0; s < kColStages; s++) {
      mbar_init(BAR(K_FULL + s), 1);
      mbar_init(BAR(K_EMPTY + s), 1);
    }
    for (int g = 0; g < 2; g++) {
      mbar_init(BAR(S_FULL + g), 1);
      mbar_init(BAR(S_EMPTY + g), 128);
    }
    misc[1] = 0u;
    fence_mbar_init();
    prefetch_tmap(&tmq);
    prefetch_tmap(&tmk);
  }
  // negated log2-domain LSEs (one packed FMA then gives s*c - lse2); queries beyond Nq get -inf: exp2 = 0
  // (straight from the splits' partial LSEs when pass 1 left its merge for later: the same maximum-and-sum as the
  // merge kernel, in the log2 domain)
  for (int j = tid; j < NCH * W; j += kColThreads) {
    float v = -INFINITY;
    if (j < p.Nq) {
      if (p.part_lse2 != nullptr) {
        const int64_t item0 = ((static_cast<int64_t>(b) * p.H + h) * p.NQT + j / p.blk) * p.n_split;
        const float* pl = p.part_lse2 + item0 * p.blk + j % p.blk;
        float M = -INFINITY;
        for (int s = 0; s < p.n_split; s++) M = fmaxf(M, pl[s * p.blk]);
        float Wsum = 0.f;
        for (int s = 0; s < p.n_split; s++) Wsum += exp2f(pl[s * p.blk] - M);
        v = -(M + log2f(Wsum));
      } else {
        v = -p.lse[(static_cast<int64_t>(b) * p.H + h) * p.Nq + j] * 1.4426950408889634f;
      }
    }
    lse2[j] = v;
  }
  if (warp == 2) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(misc)), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = misc[0];

  auto wait_or_abort = [&](int bar, uint32_t parity, int where, int aux) -> bool {
    if (misc[1] != 0u) return false;
    if (mbar_wait(BAR(bar), parity)) return true;
    report_status(p.status, AVSA_ERR_TIMEOUT, where, item, aux);
    misc[1] = 1u;
    return false;
  };

  const int n_units = ntile * NCH;
  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(BAR(Q_FULL), NCH * q_chunk_bytes);
      for (int ch = 0; ch < NCH; ch++)
        for (int pn = 0; pn < NPANEL; pn++)
          tma_load_4d(smem_u32(smem + L::kQ) + ch * q_chunk_bytes + pn * q_panel_bytes, &tmq, BAR(Q_FULL), pn * 64,
                      ch * W, h, b);
      bool ok = true;
      for (int t = 0; t < ntile && ok; t++) {
        const int s = t % kColStages, f = t / kColStages;
        if (f > 0) ok = wait_or_abort(K_EMPTY + s, (f - 1) & 1, kColKEmpty, t);
        if (!ok) break;
        mbar_expect_tx(BAR(K_FULL + s), L::kKTile);
        for (int pn = 0; pn < NPANEL; pn++)
          tma_load_4d(smem_u32(smem + L::kK) + s * L::kKTile + pn * KPANEL_BYTES, &tmk, BAR(K_FULL + s), pn * 64,
                      (kt0 + t) * 128, h, b);
      }
    }
  } else if (warp == 1) {
    // The whole warp runs the loop (uniform control flow), one elected lane issues; descriptor words are
    // prepared ahead so that the issuing lane does little besides issuing.
    const bool leader = elect_one_sync();
    const uint32_t idesc = make_idesc_bf16(128, W, 0, 0);
    constexpr uint32_t desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
    auto desc64 = [](uint32_t lo) { return (static_cast<uint64_t>(desc_hi) << 32) | lo; };
    const uint32_t k_lo0 = ((smem_u32(smem + L::kK) & 0x3FFFFu) >> 4) | (1u << 16);
    const uint32_t q_lo0 = ((smem_u32(smem + L::kQ) & 0x3FFFFu) >> 4) | (1u << 16);
    auto wait_all = [&](int bar, uint32_t parity, int where, int aux) -> bool {
      return __all_sync(0xffffffffu, wait_or_abort(bar, parity, where, aux));
    };
    bool ok = wait_all(Q_FULL, 0, kColQFull, 0);
    for (int t = 0; t < ntile && ok; t++) {
      const int s = t % kColStages, f = t / kColStages;
      ok = wait_all(K_FULL + s, f & 1, kColKFull, t);
      if (!ok) break;
      const uint32_t k_lo = k_lo0 + s * (L::kKTile >> 4);
      for (int ch = 0; ch < NCH && ok; ch++) {
        const int u = t * NCH + ch, g = u & 1, i = u >> 1;
        if (i > 0) ok = wait_all(S_EMPTY + g, (i - 1) & 1, kColSEmpty, u);
        if (!ok) break;
        tc_fence_after();
        const uint32_t q_lo = q_lo0 + ch * (q_chunk_bytes >> 4);
        if (leader) {
#pragma unroll
          for (int ks = 0; ks < D / 16; ks++) {
            const uint32_t koff = ((ks >> 2) * KPANEL_BYTES + (ks & 3) * 32) >> 4;
            const uint32_t qoff = ((ks >> 2) * q_panel_bytes + (ks & 3) * 32) >> 4;
            umma_ss(tmem + g * 256, desc64(k_lo + koff), desc64(q_lo + qoff), idesc, ks > 0 ? 1u : 0u);
          }
          umma_commit(BAR(S_FULL + g));
          if (ch == NCH - 1) umma_commit(BAR(K_EMPTY + s));
        }
        __syncwarp();
      }
    }
  } else if (warp >= 4) {
    const int g = (warp - 4) >> 2;
    const int row = ((warp & 3) << 5) + lane;
    const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
    bool ok = true;
    for (int u = g; u < n_units && ok; u += 2) {
      const int i = u >> 1, t = u / NCH, ch = u % NCH;
      ok = wait_or_abort(S_FULL + g, i & 1, kColSFull, u);
      if (!ok) break;
      tc_fence_after();
      const float* l2 = lse2 + ch * W;
      const uint32_t base = tmem + g * 256 + lane_off;
      const uint64_t c2 = pack_f32x2(p.scale_log2, p.scale_log2);
      uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};
      // sum over 32 (or 16) queries of exp2(s*c - lse2), two values per packed FMA / add
      auto reduce32 = [&](const uint32_t (&sv)[32], const float* nl) {
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          const ulonglong2 nv = *reinterpret_cast<const ulonglong2*>(nl + j);      // four negated LSEs
          float x0, x1, x2, x3;
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sv[j]), __uint_as_float(sv[j + 1])), c2, nv.x), x0, x1);
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sv[j + 2]), __uint_as_float(sv[j + 3])), c2, nv.y), x2, x3);
          acc[(j >> 2) & 3] = add_f32x2(acc[(j >> 2) & 3], pack_f32x2(fast_exp2(x0), fast_exp2(x1)));
          acc[((j >> 2) + 2) & 3] = add_f32x2(acc[((j >> 2) + 2) & 3], pack_f32x2(fast_exp2(x2), fast_exp2(x3)));
        }
      };
      const int n32 = W / 32;           // whole 32-column pieces; W is a multiple of 16, so 16 columns may remain
      uint32_t sa[32], sb[32];
      if (n32 > 0) tmem_ld32(base, sa);
      for (int c = 0; c < n32; c += 2) {
        tmem_wait_ld();
        if (c + 1 < n32) tmem_ld32(base + (c + 1) * 32, sb);      // in flight under the exponentials of piece c
        reduce32(sa, l2 + c * 32);
        if (c + 1 < n32) {
          tmem_wait_ld();
          if (c + 2 < n32) tmem_ld32(base + (c + 2) * 32, sa);
          reduce32(sb, l2 + (c + 1) * 32);
        }
      }
      if (n32 * 32 < W) {
        uint32_t st[16];
        tmem_ld16(base + n32 * 32, st);
        tmem_wait_ld();
        const float* nl = l2 + n32 * 32;
#pragma unroll
        for (int j = 0; j < 16; j += 2) {
          float x0, x1;
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(st[j]), __uint_as_float(st[j + 1])), c2,
                                 *reinterpret_cast<const uint64_t*>(nl + j)), x0, x1);
          acc[(j >> 1) & 3] = add_f32x2(acc[(j >> 1) & 3], pack_f32x2(fast_exp2(x0), fast_exp2(x1)));
        }
      }
      float sum0, sum1;
      unpack_f32x2(add_f32x2(add_f32x2(acc[0], acc[1]), add_f32x2(acc[2], acc[3])), sum0, sum1);
      tc_fence_before();
      mbar_arrive(BAR(S_EMPTY + g));
      const int key = (kt0 + t) * 128 + row;
      if (key < p.Nk)
        p.partial[(static_cast<int64_t>(ch) * gridDim.z * p.H + static_cast<int64_t>(b) * p.H + h) * p.Nk + key] =
            sum0 + sum1;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 2) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------------------------------------
// pass 2, many queries / few keys (the reverse, video->audio direction): the key tiles of one (batch, head)
// stay in shared memory (at most 4 x 128 keys) and the queries stream through a 3-stage ring in chunks of
// 128 together with their slice of log2-domain LSEs.  Units (query chunk, key tile) alternate between two
// tensor-memory buffers and two groups of 128 threads (one thread per key row), each thread accumulating
// the column sum of its key over the CTA's range of query chunks.
//   partial[(range*2 + group)][b,h,key]; the head-sum kernel adds ranges, groups and heads in a fixed order.
// ------------------------------------------------------------------------------------------------
constexpr int kRevStages = 3;
constexpr int kRevLseSlots = 5;      // LSE slices outlive their query stage by up to two units of exponentials

struct ColsumRevParams {
  const float* lse2;       // [B,H,NQC*128] negated log2-domain LSE, -inf beyond Nq
  float* partial;          // [n_range*2][B,H,Nk]
  StatusRecord* status;
  int H, Nk, NKT, NQC;     // key tiles (<= 4) and query chunks of 128
  int n_range, chunks_per_range;
  float scale_log2;
};

template <int D>
struct ColsumRevSmem {
  static constexpr int kTile = 128 * D * 2;
  static constexpr int kQ = 0;                              // ring of query chunks
  __host__ __device__ static int k_offset() { return kRevStages * kTile; }      // NKT resident key tiles follow
  __host__ __device__ static int lse_offset(int NKT) { return k_offset() + NKT * kTile; }
  __host__ __device__ static int bars_offset(int NKT) { return lse_offset(NKT) + kRevLseSlots * 512; }
  static constexpr int kNumBars = 1 + 2 * kRevStages + 4;
  static int total(int NKT) { return bars_offset(NKT) + 128 + 16; }
};

enum ColRevWhere { kRevKFull = 51, kRevQEmpty, kRevQFull, kRevSEmpty, kRevSFull };

template <int D>
__global__ void __launch_bounds__(kColThreads, 1)
colsum_rev_kernel(const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
                  const ColsumRevParams p) {
  using L = ColsumRevSmem<D>;
  constexpr int NPANEL = D / 64;
  constexpr int PANEL_BYTES = 128 * 128;
  extern __shared__ __align__(1024) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int range = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int c_begin = range * p.chunks_per_range;
  const int nchunk = min(p.NQC, c_begin + p.chunks_per_range) - c_begin;
  const int item = (b * p.H + h) * p.n_range + range;
  const int NKT = p.NKT;
  if (nchunk <= 0) return;
  if ((smem_u32(smem) & 1023u) != 0u) {
    if (tid == 0) report_status(p.status, AVSA_ERR_CUDA, kWhereSmemAlign, item, 0);
    return;
  }
  const int bars_off = L::bars_offset(NKT);
  const uint32_t bar0 = smem_u32(smem + bars_off);
  auto BAR = [&](int i) { return bar0 + static_cast<uint32_t>(i) * 8u; };
  constexpr int K_FULL = 0, Q_FULL = 1, Q_EMPTY = 1 + kRevStages, S_FULL = 1 + 2 * kRevStages, S_EMPTY = S_FULL + 2;
  const float* lse_slots = reinterpret_cast<const float*>(smem + L::lse_offset(NKT));
  volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + bars_off + 128);
  const float* lse2_bh = p.lse2 + (static_cast<int64_t>(b) * p.H + h) * (static_cast<int64_t>(p.NQC) * 128);

  if (tid == 0) {
    mbar_init(BAR(K_FULL), 1);
    for (int s = 0; s < kRevStages; s++) {
      mbar_init(BAR(Q_FULL + s), 1);
      mbar_init(BAR(Q_EMPTY + s), 1);
    }
    for (int g = 0; g < 2; g++) {
      mbar_init(BAR(S_FULL + g), 1);
      mbar_init(BAR(S_EMPTY + g), 128);
    }
    misc[1] = 0u;
    fence_mbar_init();
    prefetch_tmap(&tmq);
    prefetch_tmap(&tmk);
  }
  if (warp == 2) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(misc)), 256);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = misc[0];

  auto wait_or_abort = [&](int bar, uint32_t parity, int where, int aux) -> bool {
    if (mbar_try_wait(BAR(bar), parity)) return true;
    if (misc[1] != 0u) return false;
    if (mbar_wait(BAR(bar), parity)) return true;
    report_status(p.status, AVSA_ERR_TIMEOUT, where, item, aux);
    misc[1] = 1u;
    return false;
  };

  const int n_units = nchunk * NKT;
  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(BAR(K_FULL), NKT * L::kTile);
      for (int kt = 0; kt < NKT; kt++)
        for (int pn = 0; pn < NPANEL; pn++)
          tma_load_4d(smem_u32(smem) + L::k_offset() + kt * L::kTile + pn * PANEL_BYTES, &tmk, BAR(K_FULL), pn * 64,
                      kt * 128, h, b);
      bool ok = true;
      for (int c = 0; c < nchunk && ok; c++) {
        const int s = c % kRevStages, f = c / kRevStages;
        if (f > 0) ok = wait_or_abort(Q_EMPTY + s, (f - 1) & 1, kRevQEmpty, c);
        if (!ok) break;
        mbar_expect_tx(BAR(Q_FULL + s), L::kTile + 512);
        for (int pn = 0; pn < NPANEL; pn++)
          tma_load_4d(smem_u32(smem) + L::kQ + s * L::kTile + pn * PANEL_BYTES, &tmq, BAR(Q_FULL + s), pn * 64,
                      (c_begin + c) * 128, h, b);
        bulk_load_1d(smem_u32(smem) + L::lse_offset(NKT) + (c % kRevLseSlots) * 512,
                     lse2_bh + static_cast<int64_t>(c_begin + c) * 128, 512, BAR(Q_FULL + s));
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = make_idesc_bf16(128, 128, 0, 0);
      bool ok = wait_or_abort(K_FULL, 0, kRevKFull, 0);
      for (int c = 0; c < nchunk && ok; c++) {
        const int s = c % kRevStages, f = c / kRevStages;
        ok = wait_or_abort(Q_FULL + s, f & 1, kRevQFull, c);
        if (!ok) break;
        const uint32_t q_addr = smem_u32(smem) + L::kQ + s * L::kTile;
        for (int kt = 0; kt < NKT && ok; kt++) {
          const int u = c * NKT + kt, g = u & 1, i = u >> 1;
          if (i > 0) ok = wait_or_abort(S_EMPTY + g, (i - 1) & 1, kRevSEmpty, u);
          if (!ok) break;
          tc_fence_after();
          const uint32_t k_addr = smem_u32(smem) + L::k_offset() + kt * L::kTile;
#pragma unroll
          for (int ks = 0; ks < D / 16; ks++) {
            const uint64_t ad = make_sdesc(k_addr + (ks >> 2) * PANEL_BYTES + (ks & 3) * 32, 16, 1024);
            const uint64_t bd = make_sdesc(q_addr + (ks >> 2) * PANEL_BYTES + (ks & 3) * 32, 16, 1024);
            umma_ss(tmem + g * 128, ad, bd, idesc, ks > 0 ? 1u : 0u);
          }
          umma_commit(BAR(S_FULL + g));
        }
        if (ok) umma_commit(BAR(Q_EMPTY + s));
      }
    }
  } else if (warp >= 4) {
    const int g = (warp - 4) >> 2;
    const int row = ((warp & 3) << 5) + lane;
    const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    bool ok = true;
    for (int u = g; u < n_units && ok; u += 2) {
      const int i = u >> 1, c = u / NKT, kt = u % NKT;
      ok = wait_or_abort(S_FULL + g, i & 1, kRevSFull, u);
      if (!ok) break;
      tc_fence_after();
      const float* l2 = lse_slots + (c % kRevLseSlots) * 128;       // negated log2-domain LSEs of the chunk's queries
      const uint32_t base = tmem + g * 128 + lane_off;
      const uint64_t c2 = pack_f32x2(p.scale_log2, p.scale_log2);
      uint64_t acc2[4] = {0ull, 0ull, 0ull, 0ull};
      auto reduce32 = [&](const uint32_t (&sv)[32], const float* nl) {
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          const ulonglong2 nv = *reinterpret_cast<const ulonglong2*>(nl + j);
          float x0, x1, x2, x3;
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sv[j]), __uint_as_float(sv[j + 1])), c2, nv.x), x0, x1);
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sv[j + 2]), __uint_as_float(sv[j + 3])), c2, nv.y), x2, x3);
          acc2[(j >> 2) & 3] = add_f32x2(acc2[(j >> 2) & 3], pack_f32x2(fast_exp2(x0), fast_exp2(x1)));
          acc2[((j >> 2) + 2) & 3] = add_f32x2(acc2[((j >> 2) + 2) & 3], pack_f32x2(fast_exp2(x2), fast_exp2(x3)));
        }
      };
      // the next 32 columns are in flight under the exponentials of the current ones
      uint32_t sa[32], sb[32];
      tmem_ld32(base, sa);
      tmem_wait_ld();
      tmem_ld32(base + 32, sb);
      reduce32(sa, l2);
      tmem_wait_ld();
      tmem_ld32(base + 64, sa);
      reduce32(sb, l2 + 32);
      tmem_wait_ld();
      tmem_ld32(base + 96, sb);
      reduce32(sa, l2 + 64);
      tmem_wait_ld();
      reduce32(sb, l2 + 96);
      float sum0, sum1;
      unpack_f32x2(add_f32x2(add_f32x2(acc2[0], acc2[1]), add_f32x2(acc2[2], acc2[3])), sum0, sum1);
      tc_fence_before();
      mbar_arrive(BAR(S_EMPTY + g));
      const float tot = sum0 + sum1;
      if (kt == 0) acc[0] += tot; else if (kt == 1) acc[1] += tot; else if (kt == 2) acc[2] += tot; else acc[3] += tot;
    }
    const int64_t slot = static_cast<int64_t>(range) * 2 + g;
    float* dst = p.partial + (slot * gridDim.z * p.H + static_cast<int64_t>(b) * p.H + h) * p.Nk;
#pragma unroll
    for (int kt = 0; kt < 4; kt++) {
      const int key = kt * 128 + row;
      if (kt < NKT && key < p.Nk) dst[key] = acc[kt];
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 2) tmem_dealloc(tmem, 256);
}

// lse2[bh][i] = -lse[bh][i] * log2(e) for i < Nq (negated: one FMA gives s*c - lse2), -inf up to the padded length
__global__ void __launch_bounds__(256) lse_to_log2_kernel(const float* __restrict__ lse, int Nq, int Nq_pad, int BH,
                                                          float* __restrict__ lse2) {
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
  if (idx >= static_cast<int64_t>(BH) * Nq_pad) return;
  const int bh = static_cast<int>(idx / Nq_pad), i = static_cast<int>(idx % Nq_pad);
  lse2[idx] = i < Nq ? -lse[static_cast<int64_t>(bh) * Nq + i] * 1.4426950408889634f : -INFINITY;
}

// scores[b,i] = beta * scores[b,i] + gamma * sum_h sum_ch partial[ch][b,h,i], heads in ascending order
__device__ __forceinline__ void head_sum_keys(int block, int tid, const float* __restrict__ partial, int NCH, int B,
                                              int H, int Nk, float beta, float gamma, float* __restrict__ scores) {
  const int64_t idx = static_cast<int64_t>(block) * 256 + tid;
  if (idx >= static_cast<int64_t>(B) * Nk) return;
  const int b = static_cast<int>(idx / Nk), i = static_cast<int>(idx % Nk);
  // Fixed summation order: head major, partial slot minor.  Eight loads are issued together (a plain loop made
  // each thread wait for H dependent round trips), the adds stay in order.
  const int J = H * NCH;
  float acc = 0.f;
  for (int j0 = 0; j0 < J; j0 += 8) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; u++) {
      const int j = j0 + u, h = j / NCH, ch = j % NCH;
      v[u] = (j < J) ? partial[(static_cast<int64_t>(ch) * B * H + static_cast<int64_t>(b) * H + h) * Nk + i] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 8; u++)
      if (j0 + u < J) acc += v[u];
  }
  float out = gamma * acc;
  if (beta != 0.f) out = fmaf(beta, scores[idx], out);
  scores[idx] = out;
}
__global__ void __launch_bounds__(256) head_sum_kernel(const float* __restrict__ partial, int NCH, int B, int H,
                                                       int Nk, float beta, float gamma, float* __restrict__ scores) {
  head_sum_keys(blockIdx.x, threadIdx.x, partial, NCH, B, H, Nk, beta, gamma, scores);
}

// End of the forward call in one grid: the first `hs_blocks` CTAs sum the score partials over heads, the rest merge
// the key splits of pass 1 into O and the LSE (two groups of 128 threads per CTA).  The score pass merged the LSEs
// it needs by itself, so nothing waits for this merge.
template <int BLK, int D>
__global__ void __launch_bounds__(256) cross_finalize_kernel(int hs_blocks, const float* __restrict__ partial, int NCH, int B,
                                                             int H, int Nk, float beta, float gamma,
                                                             float* __restrict__ scores, const float* __restrict__ part_o,
                                                             const float* __restrict__ part_lse2, int n_split, int NQT,
                                                             int Nq, int total_rows, __nv_bfloat16* __restrict__ o,
                                                             int64_t o_sb, int64_t o_sh, int64_t o_sn,
                                                             float* __restrict__ lse) {
  if (static_cast<int>(blockIdx.x) < hs_blocks) {
    head_sum_keys(blockIdx.x, threadIdx.x, partial, NCH, B, H, Nk, beta, gamma, scores);
  } else {
    const int block = (static_cast<int>(blockIdx.x) - hs_blocks) * 2 + (threadIdx.x >> 7);
    merge_splits_rows<BLK, D>(block, threadIdx.x & 127, part_o, part_lse2, n_split, NQT, Nq, H, total_rows, o, o_sb, o_sh,
                              o_sn, lse, nullptr, 0, Nq);
  }
}

// The same sum for few keys and many partial slots (the reverse direction: at most 512 keys, two slots per CTA of the
// score pass): one warp per key.  Lane l adds the terms j = l, l + 32, ... in ascending order, then the 32 lane sums
// are combined by a fixed butterfly, so the result is reproducible bit for bit (the order differs from the kernel
// above, which serves the other direction).
__global__ void __launch_bounds__(256) head_sum_wide_kernel(const float* __restrict__ partial, int NCH, int B, int H,
                                                            int Nk, float beta, float gamma, float* __restrict__ scores) {
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (idx >= static_cast<int64_t>(B) * Nk) return;
  const int b = static_cast<int>(idx / Nk), i = static_cast<int>(idx % Nk);
  const int J = H * NCH;
  float acc = 0.f;
  for (int j0 = lane; j0 < J; j0 += 32 * 4) {
    float v[4];
#pragma unroll
    for (int u = 0; u < 4; u++) {
      const int j = j0 + 32 * u, h = j / NCH, ch = j % NCH;
      v[u] = (j < J) ? partial[(static_cast<int64_t>(ch) * B * H + static_cast<int64_t>(b) * H + h) * Nk + i] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 4; u++) acc += v[u];
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
  if (lane == 0) {
    float out = gamma * acc;
    if (beta != 0.f) out = fmaf(beta, scores[idx], out);
    scores[idx] = out;
  }
}

struct CrossPlan {
  int blk, NQT, NKB, n_split, tps;           // pass 1 (key tiles of blk)
  int NKT, NCH, W, n_range, tpr;             // pass 2 (key tiles of 128)
  bool reverse;                              // pass 2 with the keys resident (Nq > 512, Nk <= 512)
  int NQC, rev_ranges, rev_cpr, rev_slots;   // query chunks of 128, CTAs per (b,h), chunks per CTA, partial slots
  size_t off_part_o, off_part_lse, off_lse, off_lse2, off_partial, off_redo, total;
};

static CrossPlan make_cross_plan(int B, int H, int Nq, int Nk, int d) {
  CrossPlan c;
  c.blk = d;   // (blk, d) = (128,128) or (64,64)
  c.NQT = (Nq + c.blk - 1) / c.blk;
  c.NKB = (Nk + c.blk - 1) / c.blk;
  // One work item per SM (one CTA each): a single wave.  Two items per SM were measured slower on the
  // Ovi-class shape (210 vs 196 us for the call): every item pays its own pipeline fill, partial-result
  // write-out and merge work.
  const int target = persistent_grid(1 << 30);
  int want_split = target / (B * H * c.NQT);
  if (want_split < 1) want_split = 1;
  if (want_split > c.NKB) want_split = c.NKB;
  c.tps = (c.NKB + want_split - 1) / want_split;
  c.n_split = (c.NKB + c.tps - 1) / c.tps;
  c.NKT = (Nk + 127) / 128;
  c.NCH = Nq > 256 ? 2 : 1;
  c.W = (((Nq + c.NCH - 1) / c.NCH) + 15) / 16 * 16;
  int want_range = target / (B * H);
  if (want_range < 1) want_range = 1;
  if (want_range > c.NKT) want_range = c.NKT;
  c.tpr = (c.NKT + want_range - 1) / want_range;
  c.n_range = (c.NKT + c.tpr - 1) / c.tpr;
  c.reverse = Nq > 512;
  c.NQC = (Nq + 127) / 128;
  int want_rev = target / (B * H);
  if (want_rev < 1) want_rev = 1;
  if (want_rev > c.NQC) want_rev = c.NQC;
  c.rev_cpr = (c.NQC + want_rev - 1) / want_rev;
  c.rev_ranges = (c.NQC + c.rev_cpr - 1) / c.rev_cpr;
  c.rev_slots = c.rev_ranges * 2;
  size_t off = kStatusBytes;
  const size_t items = static_cast<size_t>(B) * H * c.NQT * c.n_split;
  c.off_part_o = off; off += align_up(items * c.blk * d * sizeof(float), 256);
  c.off_part_lse = off; off += align_up(items * c.blk * sizeof(float), 256);
  c.off_lse = off; off += align_up(static_cast<size_t>(B) * H * Nq * sizeof(float), 256);
  c.off_lse2 = off; off += c.reverse ? align_up(static_cast<size_t>(B) * H * c.NQC * 128 * sizeof(float), 256) : 0;
  const size_t slots = c.reverse ? static_cast<size_t>(c.rev_slots) : static_cast<size_t>(c.NCH);
  c.off_partial = off; off += align_up(slots * B * H * Nk * sizeof(float), 256);
  c.off_redo = off; off += align_up(items * sizeof(int), 256);
  c.total = off;
  return c;
}

template <int BLK, int D>
static int run_cross(int B, int H, int Nq, int Nk, const avsa_bf16_4d& q, const avsa_bf16_4d& k, const avsa_bf16_4d& v,
                     void* o, float* lse_out, float* scores, float beta, float gamma, float scale, uint8_t* ws,
                     const CrossPlan& c, cudaStream_t st) {
  StatusRecord* status = reinterpret_cast<StatusRecord*>(ws);
  float* part_o = reinterpret_cast<float*>(ws + c.off_part_o);
  float* part_lse = reinterpret_cast<float*>(ws + c.off_part_lse);
  float* lse = lse_out != nullptr ? lse_out : reinterpret_cast<float*>(ws + c.off_lse);
  float* partial = reinterpret_cast<float*>(ws + c.off_partial);
  clear_status_kernel<<<1, 1, 0, st>>>(status);
  bool merge_late = false;
  // ---- pass 1
  {
    using L = AttnSmem<BLK, D>;
    CUtensorMap tq, tk, tv;
    if (!encode_bf16_tile_map(&tq, q.ptr, B, H, Nq, D, q.stride_b, q.stride_h, q.stride_n, BLK)) return AVSA_ERR_CUDA;
    if (!encode_bf16_tile_map(&tk, k.ptr, B, H, Nk, D, k.stride_b, k.stride_h, k.stride_n, BLK)) return AVSA_ERR_CUDA;
    if (!encode_bf16_tile_map(&tv, v.ptr, B, H, Nk, D, v.stride_b, v.stride_h, v.stride_n, BLK)) return AVSA_ERR_CUDA;
    using LP = PersistSmem<BLK, D>;
    AttnParams prm = {};
    prm.part_o = part_o;
    prm.part_lse2 = part_lse;
    prm.n_split = c.n_split;
    prm.tiles_per_split = c.tps;
    prm.status = status;
    prm.H = H;
    prm.Nq = Nq;
    prm.NQT = c.NQT;
    prm.Nk = Nk;
    prm.NKB = c.NKB;
    prm.scale_log2 = scale * 1.4426950408889634f;
    // Pass 1 runs on the persistent fast kernel (one CTA per SM over the (query tile, key split) items), with the
    // exact-rescaling kernel behind it for the items whose rows outgrow their first-tile reference.
    int* redo = reinterpret_cast<int*>(ws + c.off_redo);
    const long long items = static_cast<long long>(B) * H * c.NQT * c.n_split;
    const int pgrid = persistent_grid(items);
    if (c.n_split == 1 && o != nullptr) {
      // the whole key axis fits one work item (few keys): write O and the LSE directly, no partials to merge
      CUtensorMap to;
      if (!encode_bf16_tile_map(&to, o, B, H, Nq, D, q.stride_b, q.stride_h, q.stride_n, BLK)) return AVSA_ERR_CUDA;
      prm.lse = lse;
      if (cudaFuncSetAttribute(attn_persist_kernel<BLK, D, MODE_RANGE_DIRECT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               LP::kTotal) != cudaSuccess)
        return AVSA_ERR_CUDA;
      if (cudaFuncSetAttribute(attn_redo_kernel<BLK, D, MODE_RANGE_DIRECT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               L::kTotal) != cudaSuccess)
        return AVSA_ERR_CUDA;
      attn_persist_kernel<BLK, D, MODE_RANGE_DIRECT><<<pgrid, kAttnThreads, LP::kTotal, st>>>(
          tq, tk, tv, to, prm, redo, nullptr, static_cast<int>(items));
      attn_redo_kernel<BLK, D, MODE_RANGE_DIRECT><<<pgrid, kAttnThreads, L::kTotal, st>>>(tq, tk, tv, to, prm, redo);
    } else {
      if (cudaFuncSetAttribute(attn_persist_kernel<BLK, D, MODE_RANGE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               LP::kTotal) != cudaSuccess)
        return AVSA_ERR_CUDA;
      if (cudaFuncSetAttribute(attn_redo_kernel<BLK, D, MODE_RANGE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               L::kTotal) != cudaSuccess)
        return AVSA_ERR_CUDA;
      attn_persist_kernel<BLK, D, MODE_RANGE><<<pgrid, kAttnThreads, LP::kTotal, st>>>(tq, tk, tv, tq, prm, redo, nullptr,
                                                                                       static_cast<int>(items));
      attn_redo_kernel<BLK, D, MODE_RANGE><<<pgrid, kAttnThreads, L::kTotal, st>>>(tq, tk, tv, tq, prm, redo);
      merge_late = scores != nullptr && !c.reverse;      // then the merge rides in the call's last grid
      if (!merge_late) {
        const int total_rows = B * H * Nq;
        constexpr int RPB = 128 / (D / 4);
        merge_splits_kernel<BLK, D><<<(total_rows + RPB - 1) / RPB, 128, 0, st>>>(
            part_o, part_lse, c.n_split, c.NQT, Nq, H, total_rows, static_cast<__nv_bfloat16*>(o), q.stride_b, q.stride_h,
            q.stride_n, lse, nullptr, 0, Nq);
      }
    }
  }
  // ---- pass 2, keys resident (many queries, at most 512 keys)
  if (scores != nullptr && c.reverse) {
    using L = ColsumRevSmem<D>;
    float* lse2 = reinterpret_cast<float*>(ws + c.off_lse2);
    const int64_t n2 = static_cast<int64_t>(B) * H * c.NQC * 128;
    lse_to_log2_kernel<<<static_cast<unsigned>((n2 + 255) / 256), 256, 0, st>>>(lse, Nq, c.NQC * 128, B * H, lse2);
    CUtensorMap tq, tk;
    if (!encode_bf16_tile_map(&tq, q.ptr, B, H, Nq, D, q.stride_b, q.stride_h, q.stride_n, 128)) return AVSA_ERR_CUDA;
    if (!encode_bf16_tile_map(&tk, k.ptr, B, H, Nk, D, k.stride_b, k.stride_h, k.stride_n, 128)) return AVSA_ERR_CUDA;
    const int smem = L::total(c.NKT);
    if (cudaFuncSetAttribute(colsum_rev_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
      return AVSA_ERR_CUDA;
    ColsumRevParams rp;
    rp.lse2 = lse2;
    rp.partial = partial;
    rp.status = status;
    rp.H = H;
    rp.Nk = Nk;
    rp.NKT = c.NKT;
    rp.NQC = c.NQC;
    rp.n_range = c.rev_ranges;
    rp.chunks_per_range = c.rev_cpr;
    rp.scale_log2 = scale * 1.4426950408889634f;
    colsum_rev_kernel<D><<<dim3(c.rev_ranges, H, B), kColThreads, smem, st>>>(tq, tk, rp);
    const int64_t n = static_cast<int64_t>(B) * Nk;
    head_sum_wide_kernel<<<static_cast<unsigned>((n + 7) / 8), 256, 0, st>>>(partial, c.rev_slots, B, H, Nk, beta, gamma,
                                                                            scores);
  }
  // ---- pass 2, queries resident (at most 512 queries)
  if (scores != nullptr && !c.reverse) {
    using L = ColsumSmem<D>;
    CUtensorMap tq, tk;
    if (!encode_bf16_tile_map(&tq, q.ptr, B, H, Nq, D, q.stride_b, q.stride_h, q.stride_n, c.W)) return AVSA_ERR_CUDA;
    if (!encode_bf16_tile_map(&tk, k.ptr, B, H, Nk, D, k.stride_b, k.stride_h, k.stride_n, 128)) return AVSA_ERR_CUDA;
    const int smem = L::total(c.NCH, c.W);
    if (cudaFuncSetAttribute(colsum_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
      return AVSA_ERR_CUDA;
    ColsumParams cp;
    cp.lse = lse;
    cp.part_lse2 = merge_late ? part_lse : nullptr;
    cp.n_split = c.n_split;
    cp.NQT = c.NQT;
    cp.blk = c.blk;
    cp.partial = partial;
    cp.status = status;
    cp.H = H;
    cp.Nq = Nq;
    cp.Nk = Nk;
    cp.NKT = c.NKT;
    cp.NCH = c.NCH;
    cp.W = c.W;
    cp.n_range = c.n_range;
    cp.tiles_per_range = c.tpr;
    cp.scale_log2 = scale * 1.4426950408889634f;
    dim3 grid(c.n_range, H, B);
    colsum_kernel<D><<<grid, kColThreads, smem, st>>>(tq, tk, cp);
    const int64_t n = static_cast<int64_t>(B) * Nk;
    const int hs_blocks = static_cast<int>((n + 255) / 256);
    if (merge_late) {
      const int total_rows = B * H * Nq;
      constexpr int RPB = 128 / (D / 4);
      const int merge_blocks = ((total_rows + RPB - 1) / RPB + 1) / 2;
      cross_finalize_kernel<BLK, D><<<hs_blocks + merge_blocks, 256, 0, st>>>(
          hs_blocks, partial, c.NCH, B, H, Nk, beta, gamma, scores, part_o, part_lse, c.n_split, c.NQT, Nq, total_rows,
          static_cast<__nv_bfloat16*>(o), q.stride_b, q.stride_h, q.stride_n, lse);
    } else {
      head_sum_kernel<<<hs_blocks, 256, 0, st>>>(partial, c.NCH, B, H, Nk, beta, gamma, scores);
    }
  }
  return cudaGetLastError() == cudaSuccess ? AVSA_OK : AVSA_ERR_CUDA;
}

}  // namespace avsa

using namespace avsa;

extern "C" size_t avsa_cross_attn_scores_workspace_bytes(int B, int H, int Nq, int Nk, int d) {
  if (B <= 0 || H <= 0 || Nq <= 0 || Nk <= 0 || (d != 64 && d != 128)) return 0;
  return make_cross_plan(B, H, Nq, Nk, d).total;
}

extern "C" int avsa_cross_attn_scores(int B, int H, int Nq, int Nk, int d, avsa_bf16_4d q, avsa_bf16_4d k,
                                      avsa_bf16_4d v, void* o_bf16, float* lse, float* scores, float score_beta,
                                      float score_gamma, float softmax_scale, void* ws, size_t ws_bytes,
                                      void* stream) {
  if (B <= 0 || H <= 0 || Nq <= 0 || Nk <= 0) return AVSA_ERR_INVALID_ARG;
  if (d != 64 && d != 128) return AVSA_ERR_UNSUPPORTED;
  if (H > 65535 || B > 65535) return AVSA_ERR_UNSUPPORTED;
  // the score pass keeps either the queries or the keys of a head on chip
  if (scores != nullptr && Nq > 512 && Nk > 512) return AVSA_ERR_UNSUPPORTED;
  if (!tensor_ok(q, B, H) || !tensor_ok(k, B, H) || !tensor_ok(v, B, H)) return AVSA_ERR_INVALID_ARG;
  if (o_bf16 != nullptr && !aligned16(o_bf16)) return AVSA_ERR_INVALID_ARG;
  if (softmax_scale < 0.f || softmax_scale != softmax_scale) return AVSA_ERR_INVALID_ARG;
  const CrossPlan c = make_cross_plan(B, H, Nq, Nk, d);
  if (ws == nullptr || ws_bytes < c.total) return AVSA_ERR_WORKSPACE;
  if (!device_is_sm100()) return AVSA_ERR_UNSUPPORTED;
  const float scale = softmax_scale != 0.f ? softmax_scale : 1.0f / sqrtf(static_cast<float>(d));
  uint8_t* base = static_cast<uint8_t*>(ws);
  if (d == 128)
    return run_cross<128, 128>(B, H, Nq, Nk, q, k, v, o_bf16, lse, scores, score_beta, score_gamma, scale, base, c,
                               as_stream(stream));
  return run_cross<64, 64>(B, H, Nq, Nk, q, k, v, o_bf16, lse, scores, score_beta, score_gamma, scale, base, c,
                           as_stream(stream));
}
