// Mask construction: protected token set (Eq. 3 / Eq. 8), block mean-pooling and block scores of the
// base sparse pattern, per-(head, query block) top-k, and the protected block mask of Eq. 9 emitted
// as ascending column lists.  CUDA-core kernels: the work is HBM- or latency-bound.
#include <mutex>

#include "avsa_common.cuh"

namespace avsa {

constexpr int kMaxBlocksPerRow = 2048;

// Order-preserving key of an fp32 value: larger float <=> larger key.  NaN ranks as -inf, -0 as +0.
__device__ __forceinline__ uint32_t rank_key(float x) {
  if (x != x) x = __int_as_float(0xff800000);
  if (x == 0.0f) x = 0.0f;
  uint32_t b = __float_as_uint(x);
  if (b == 0x80000000u) b = 0u;
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// ------------------------------------------------------------------------------------------------
// (i) block mean-pooling.  grid (NB, B*H, 2: q|k); 256 threads; each thread owns 8 channels of a
// subset of the block's rows (16-byte loads), then the row groups are summed in a fixed order.
// ------------------------------------------------------------------------------------------------
constexpr unsigned kPoolTailCtas = 296;   // CTAs at the end of the pooling grid that wait for the token select

template <int D>
__global__ void __launch_bounds__(256) pool_kernel(const __nv_bfloat16* __restrict__ q, int64_t q_sb, int64_t q_sh,
                                                   int64_t q_sn, const __nv_bfloat16* __restrict__ k, int64_t k_sb,
                                                   int64_t k_sh, int64_t k_sn, float* __restrict__ qbar,
                                                   float* __restrict__ kbar, int H, int N, int blk) {
  constexpr int TPR = D / 8;          // threads per row
  constexpr int RPP = 256 / TPR;      // rows per pass
  __shared__ float part[RPP][D + 4];
  // lets the block-score grid be staged while this one drains (it waits for this grid before it reads)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const int nb = blockIdx.x, bh = blockIdx.y, which = blockIdx.z;
  const int b = bh / H, h = bh % H;
  const __nv_bfloat16* src = which == 0 ? q + b * q_sb + h * q_sh : k + b * k_sb + h * k_sh;
  const int64_t sn = which == 0 ? q_sn : k_sn;
  float* dst = (which == 0 ? qbar : kbar) + (static_cast<int64_t>(bh) * gridDim.x + nb) * D;
  const int c = threadIdx.x % TPR, g = threadIdx.x / TPR;
  const int row0 = nb * blk;
  const int valid = min(blk, N - row0);
  float acc[8];
#pragma unroll
  for (int i = 0; i < 8; i++) acc[i] = 0.f;
  constexpr int UNROLL = 8;
  for (int r0 = 0; r0 < blk; r0 += RPP * UNROLL) {
    uint4 v[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; u++) {
      const int r = r0 + u * RPP + g;
      v[u] = make_uint4(0u, 0u, 0u, 0u);
      if (r < valid) v[u] = __ldg(reinterpret_cast<const uint4*>(src + (row0 + r) * sn + c * 8));
    }
#pragma unroll
    for (int u = 0; u < UNROLL; u++) {
      const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
      for (int i = 0; i < 4; i++) {
        acc[2 * i] += __uint_as_float(w[i] << 16);
        acc[2 * i + 1] += __uint_as_float(w[i] & 0xffff0000u);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 8; i++) part[g][c * 8 + i] = acc[i];
  __syncthreads();
  if (threadIdx.x < D) {
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < RPP; j++) s += part[j][threadIdx.x];
    dst[threadIdx.x] = s / static_cast<float>(valid);
  }
  // This grid starts while the token select (its predecessor on the stream) is still running.  The last
  // CTAs wait for it before they retire, so that "pooling finished" implies "token select finished" for the
  // kernels behind (which wait for their predecessor only); by then the select is long done, and no
  // earlier CTA ever holds an SM slot waiting.
  const unsigned lin = (blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
  if (lin + kPoolTailCtas >= gridDim.x * gridDim.y * gridDim.z) asm volatile("griddepcontrol.wait;" ::: "memory");
}

// ------------------------------------------------------------------------------------------------
// fp32-accurate products on the warp-level tensor cores: every operand is split into two tf32 halves
// (x = hi + lo exactly to 2^-22) and three products a_lo*b_hi + a_hi*b_lo + a_hi*b_hi are accumulated in
// fp32 (m16n8k8 MMAs; the block-score problem is far too small for the tcgen05 path).
// ------------------------------------------------------------------------------------------------
// hi = x with the 13 mantissa bits cleared that a tf32 operand does not have, lo = x - hi (exact in fp32; the MMA
// reads its leading 10 mantissa bits, which leaves an error of 2^-21 |x|)
__device__ __forceinline__ uint32_t smem_u32_of(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void split_tf32(float x, uint32_t& hi, uint32_t& lo) {
  hi = __float_as_uint(x) & 0xffffe000u;
  lo = __float_as_uint(x - __uint_as_float(hi));
}
__device__ __forceinline__ void mma_tf32(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// Adds one warp's digits to a shared-memory histogram.  When every participating lane holds the same
// digit (the usual case for the leading byte of like-signed scores) one lane adds the whole count;
// otherwise each lane adds its own (the hardware serialises only lanes that really collide).
__device__ __forceinline__ void warp_hist_add(int* bins, bool in, uint32_t dgt, int lane) {
  const unsigned inmask = __ballot_sync(0xffffffffu, in);
  if (inmask == 0u) return;
  const int leader = __ffs(inmask) - 1;
  const uint32_t d0 = __shfl_sync(0xffffffffu, dgt, leader);
  const bool uniform = __all_sync(0xffffffffu, !in || dgt == d0);
  if (uniform) {
    if (lane == leader) atomicAdd(&bins[d0], __popc(inmask));
  } else if (in) {
    atomicAdd(&bins[dgt], 1);
  }
}

// ------------------------------------------------------------------------------------------------
// Radix-select helper: given 256 digit counts (descending scan), find the digit that holds the
// want-th largest element.  One warp; lane l owns digits 255-8l .. 248-8l.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void warp_pick_digit(const int* bins, int want, int lane, int& digit, int& above,
                                                int& in_bin) {
  int local[8];
  int sum = 0;
#pragma unroll
  for (int i = 0; i < 8; i++) {
    local[i] = bins[255 - (lane * 8 + i)];
    sum += local[i];
  }
  int incl = sum;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += t;
  }
  const int excl = incl - sum;
  const bool mine = (excl < want) && (want <= incl);
  int dg = 0, ab = 0, ib = 0;
  if (mine) {
    int run = excl;
#pragma unroll
    for (int i = 0; i < 8; i++) {
      if (run < want && want <= run + local[i]) {
        dg = 255 - (lane * 8 + i);
        ab = run;
        ib = local[i];
      }
      run += local[i];
    }
  }
  const unsigned who = __ballot_sync(0xffffffffu, mine);
  const int src = __ffs(who) - 1;
  digit = __shfl_sync(0xffffffffu, dg, src);
  above = __shfl_sync(0xffffffffu, ab, src);
  in_bin = __shfl_sync(0xffffffffu, ib, src);
}

// ------------------------------------------------------------------------------------------------
// (iii) protected token set: one CTA of 1024 threads per batch item.  The canonical keys are staged
// in shared memory once (global memory is re-read instead when they do not fit); a radix select
// (4 x 8 bits, warp-aggregated histogram) finds the n_protect-th largest key; then every warp walks
// its own contiguous segment in index order, taking every larger key and the lowest-index ties,
// writes the token flags and raises the flag of every block that holds one.  Block 0 also resets
// the status record of the call.
// ------------------------------------------------------------------------------------------------
constexpr int kSelectSmemKeys = 56 * 1024;   // 224 KB of keys at most

template <bool STAGED>
__global__ void __launch_bounds__(1024) token_select_kernel(const float* __restrict__ scores, int N, int n_protect,
                                                            int blk, int NB, int min_tokens,
                                                            uint8_t* __restrict__ prot_tok,
                                                            uint8_t* __restrict__ prot_blk, StatusRecord* status) {
  extern __shared__ uint32_t skeys[];
  __shared__ int bins[256];
  __shared__ int s_digit, s_above, s_in_bin;
  __shared__ int warp_cnt[32];
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* s = scores + static_cast<int64_t>(b) * N;
  uint8_t* ptok = prot_tok + static_cast<int64_t>(b) * N;
  uint8_t* pblk = prot_blk + static_cast<int64_t>(b) * NB;
  // nothing launched next on the stream depends on this kernel until the list emission, so let the
  // pooling kernel start right away (programmatic dependent launch)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (b == 0 && tid == 0) {
    status->code = 0;
    status->where = 0;
    status->item = 0;
    status->aux = 0;
  }
  for (int i = tid; i < NB; i += 1024) pblk[i] = 0;
  if (n_protect <= 0) {
    for (int i = tid; i < N; i += 1024) ptok[i] = 0;
    return;
  }
  if (STAGED) {
#pragma unroll 8
    for (int i = tid; i < N; i += 1024) skeys[i] = rank_key(__ldg(s + i));
  }
  auto key_at = [&](int i) -> uint32_t { return STAGED ? skeys[i] : rank_key(__ldg(s + i)); };
  uint32_t prefix = 0, mask = 0;
  int want = n_protect;
  for (int pass = 0; pass < 4; pass++) {
    const int shift = 24 - 8 * pass;
    if (tid < 256) bins[tid] = 0;
    __syncthreads();     // also orders the staging stores before the first reads
    for (int i0 = 0; i0 < N; i0 += 1024) {
      const int i = i0 + tid;
      const bool valid = i < N;
      const uint32_t key = valid ? key_at(i) : 0u;
      const bool in = valid && ((key & mask) == prefix);
      warp_hist_add(bins, in, (key >> shift) & 255u, lane);
    }
    __syncthreads();
    if (warp == 0) {
      int dg, ab, ib;
      warp_pick_digit(bins, want, lane, dg, ab, ib);
      if (lane == 0) {
        s_digit = dg;
        s_above = ab;
        s_in_bin = ib;
      }
    }
    __syncthreads();
    want -= s_above;
    prefix |= static_cast<uint32_t>(s_digit) << shift;
    mask |= 255u << shift;
    const bool whole_bin = (s_in_bin == want);   // every key of the bin is taken: no need to refine further
    __syncthreads();
    if (whole_bin) break;
  }
  const uint32_t T = prefix;     // the n_protect-th largest key; `want` ties at T are taken, lowest index first
  // contiguous segment per warp, a whole number of blocks (blk is a multiple of 32), so that every block's
  // count of protected tokens is known to one warp
  const int seg = ((N + 31) / 32 + blk - 1) / blk * blk;
  const int lo = min(N, warp * seg), hi = min(N, lo + seg);
  int eq_mine = 0;
  for (int i0 = lo; i0 < hi; i0 += 32) {
    const int i = i0 + lane;
    eq_mine += __popc(__ballot_sync(0xffffffffu, i < hi && key_at(i) == T));
  }
  if (lane == 0) warp_cnt[warp] = eq_mine;
  __syncthreads();
  int eq_seen = 0;
  for (int w2 = 0; w2 < warp; w2++) eq_seen += warp_cnt[w2];
  int in_block = 0;     // protected tokens of the block being walked
  for (int i0 = lo; i0 < hi; i0 += 32) {
    const int i = i0 + lane;
    const bool valid = i < hi;
    const uint32_t key = valid ? key_at(i) : 0u;
    const bool gt = valid && key > T;
    const bool eq = valid && key == T;
    const unsigned eqm = __ballot_sync(0xffffffffu, eq);
    const bool keep = gt || (eq && (eq_seen + __popc(eqm & ((1u << lane) - 1u))) < want);
    eq_seen += __popc(eqm);
    if (valid) ptok[i] = keep ? 1 : 0;
    in_block += __popc(__ballot_sync(0xffffffffu, keep));
    if ((i0 + 32) % blk == 0 || i0 + 32 >= hi) {          // last 32 tokens of the block (or of the sequence)
      if (in_block >= min_tokens && lane == 0) pblk[i0 / blk] = 1;
      in_block = 0;
    }
  }
}

// ------------------------------------------------------------------------------------------------
// (iv) per-(head, query block) top-k_keep of a block-score row, protection OR (Eq. 9), ascending
// list emission.  One warp per row; the row's keys live in registers (KPL per lane, element j*32+lane
// in slot j).  The radix select stops as soon as the bin that holds the k-th key is taken whole.
// `src` is the row of block scores (global or shared memory), `bins` 256 ints of shared memory owned
// by this warp.
// ------------------------------------------------------------------------------------------------
template <int KPL>
__device__ __forceinline__ void select_row(const float* src, const uint8_t* __restrict__ pb, bool row_prot, int NB,
                                           int k_keep, int protect_cols, int* bins, int lane,
                                           int32_t* __restrict__ out, int32_t* __restrict__ cnt_out) {
  const unsigned lt = (1u << lane) - 1u;
  const bool keep_all = row_prot || k_keep >= NB;
  uint32_t keys[KPL];
  uint32_t T = 0;
  int want = 0;
  if (!keep_all) {
#pragma unroll
    for (int j = 0; j < KPL; j++) {
      const int i = j * 32 + lane;
      keys[j] = (i < NB) ? rank_key(src[i]) : 0u;
    }
    uint32_t prefix = 0, mask = 0;
    want = k_keep;
    for (int pass = 0; pass < 4; pass++) {
      const int shift = 24 - 8 * pass;
      // digit range of the keys: when they all share the leading byte (sign and high exponent bits: the usual
      // case) the first pass needs no histogram at all; later bytes hardly ever agree, so only it is checked
      if (pass == 0) {
        uint32_t dmin = 255u, dmax = 0u;
#pragma unroll
        for (int j = 0; j < KPL; j++) {
          const uint32_t dg = keys[j] >> 24;
          if (j * 32 + lane < NB) {
            dmin = min(dmin, dg);
            dmax = max(dmax, dg);
          }
        }
        dmin = __reduce_min_sync(0xffffffffu, dmin);
        dmax = __reduce_max_sync(0xffffffffu, dmax);
        if (dmin == dmax) {
          prefix = dmin << 24;
          mask = 255u << 24;
          continue;
        }
      }
#pragma unroll
      for (int i = 0; i < 8; i++) bins[i * 32 + lane] = 0;
      __syncwarp();
#pragma unroll
      for (int j = 0; j < KPL; j++) {
        const bool in = (j * 32 + lane < NB) && ((keys[j] & mask) == prefix);
        if (in) atomicAdd(&bins[(keys[j] >> shift) & 255u], 1);
      }
      __syncwarp();
      int dg, ab, ib;
      warp_pick_digit(bins, want, lane, dg, ab, ib);
      want -= ab;
      prefix |= static_cast<uint32_t>(dg) << shift;
      mask |= 255u << shift;
      __syncwarp();
      if (ib == want) break;     // the whole bin is taken
    }
    T = prefix;
  }
  int pos = 0, eq_seen = 0;
#pragma unroll
  for (int j = 0; j < KPL; j++) {
    if (j * 32 >= NB) break;
    const int i = j * 32 + lane;
    const bool valid = i < NB;
    bool keep;
    if (keep_all) {
      keep = valid;
    } else {
      const bool gt = valid && keys[j] > T;
      const bool eq = valid && keys[j] == T;
      const unsigned eqm = __ballot_sync(0xffffffffu, eq);
      keep = gt || (eq && (eq_seen + __popc(eqm & lt)) < want);
      eq_seen += __popc(eqm);
      if (protect_cols && valid && pb[i] != 0) keep = true;
    }
    const unsigned km = __ballot_sync(0xffffffffu, keep);
    if (keep) out[pos + __popc(km & lt)] = i;
    pos += __popc(km);
  }
  for (int i = pos + lane; i < NB; i += 32) out[i] = -1;
  if (lane == 0) *cnt_out = pos;
}

// Lists from a block-score tensor that is already in global memory (AVSA_USE_GIVEN_BLOCK_SCORES): one warp
// per row, 4 rows per CTA.
template <int KPL>
__global__ void __launch_bounds__(128) row_select_kernel(const float* __restrict__ bs, const uint8_t* __restrict__ prot_blk,
                                                         int H, int NB, int k_keep, int protect_rows,
                                                         int protect_cols, int total_rows, int32_t* __restrict__ col_idx,
                                                         int32_t* __restrict__ col_cnt) {
  __shared__ int all_bins[4][256];
  asm volatile("griddepcontrol.wait;" ::: "memory");   // the block flags come from the kernel before
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * 4 + warp;      // row = (b*H + h)*NB + qb
  if (row >= total_rows) return;
  const int qb = row % NB;
  const int b = row / (NB * H);
  const uint8_t* pb = prot_blk + static_cast<int64_t>(b) * NB;
  select_row<KPL>(bs + static_cast<int64_t>(row) * NB, pb, protect_rows && pb[qb] != 0, NB, k_keep, protect_cols,
                  all_bins[warp], lane, col_idx + static_cast<int64_t>(row) * NB, col_cnt + row);
}

// ------------------------------------------------------------------------------------------------
// (ii)+(iv) fused: block scores Bs[bh, i, j] = qbar[bh,i,:] . kbar[bh,j,:] * scale for a strip of 16 query
// blocks against every key block, kept in shared memory, then the lists of those 16 rows straight from
// there.  One CTA of 8 warps per strip: each warp computes 32-column chunks of the strip with 3xTF32 m16n8k8 MMAs
// (A = the strip's pooled queries from shared memory, B = pooled keys read from L2 as 16-byte pieces), then takes
// two rows of the strip through the select (about a thousand instructions per row).  Against separate score and list kernels
// this saves a launch, a drain and a round trip of the scores through L2 on the latency chain behind the
// pooling kernel.
//   The channel order inside each group of 16 is permuted identically for both operands (lane t of a
// quad holds channels 4t..4t+3 of the group and feeds them to two k-steps), which leaves every dot
// product the same sum and lets each operand piece be one 16-byte load.
// ------------------------------------------------------------------------------------------------
constexpr int kStripRows = 16;

template <int D>
__host__ __device__ constexpr int strip_pitch(int NB) { return (NB + 31) / 32 * 32 + 4; }

template <int D, int KPL, int WARPS>
__global__ void __launch_bounds__(WARPS * 32) score_select_kernel(const float* __restrict__ qbar, const float* __restrict__ kbar,
                                                                  float* __restrict__ bs, const uint8_t* __restrict__ prot_blk,
                                                                  int H, int NB, float scale, int k_keep, int protect_rows,
                                                                  int protect_cols, int32_t* __restrict__ col_idx,
                                                                  int32_t* __restrict__ col_cnt) {
  constexpr int PITCH = D + 4;
  constexpr int NT = 32 / WARPS;              // 8-column MMA tiles per warp and pass: 4 with 8 warps, 2 with 16
  constexpr int CHUNK = NT * 8;               // columns per warp and pass
  extern __shared__ __align__(16) float strip_smem[];
  uint32_t* sq_hi = reinterpret_cast<uint32_t*>(strip_smem);            // [16][PITCH] pooled queries of the strip,
  uint32_t* sq_lo = sq_hi + kStripRows * PITCH;                          // split into their two tf32 halves once
  const int SP = strip_pitch<D>(NB);
  float* strip = strip_smem + 2 * kStripRows * PITCH;       // [16][SP] block scores of the strip
  int* all_bins = reinterpret_cast<int*>(strip + kStripRows * SP);      // [WARPS][256]
  float4* ring = reinterpret_cast<float4*>(all_bins + WARPS * 256);     // [WARPS][4 slots][2 tiles][32 lanes]
  static_assert(NT == 4, "the key ring holds two tile pairs per 16-channel group");
  // Staged behind the pooling grid (programmatic dependent launch) and waits for it here; the pooling grid in
  // turn retires only after the token select, so the block flags are final too.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int bh = blockIdx.y, i0 = blockIdx.x * kStripRows;
  const float* qb = qbar + static_cast<int64_t>(bh) * NB * D;
  const float* kb = kbar + static_cast<int64_t>(bh) * NB * D;
  // The pooled keys come through a ring of four 16-byte slots per lane and MMA tile pair (cp.async, no registers
  // held): the pieces of three half-steps ahead are in flight under the MMAs of the current one, and the first
  // three of a warp's first chunk already under the load of the strip's queries.  A plain load per step left every
  // step waiting for its own L2 round trip (1500 cycles each, eight in a row).
  constexpr int HS = (D / 16) * 2;            // half-steps: (16-channel group jg, tile pair hp)
  const uint32_t ring_base = smem_u32_of(ring) + (warp * 4 * 2 * 32 + lane) * 16;
  auto issue = [&](int j0, int hs) {
    const int jg = hs >> 1, hp = hs & 1;
#pragma unroll
    for (int n2 = 0; n2 < 2; n2++) {
      const int col = j0 + (hp * 2 + n2) * 8 + g;
      const bool valid = col < NB;                          // beyond the last key block: zero fill
      const float* src = kb + static_cast<int64_t>(valid ? col : 0) * D + 4 * t + 16 * jg;
      const uint32_t dst = ring_base + (((hs & 3) * 2 + n2) * 32) * 16;
      const int bytes = valid ? 16 : 0;
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
    }
  };
  const int j_first = warp * CHUNK;
  if (j_first < NB) {
#pragma unroll
    for (int hs = 0; hs < 3; hs++) {
      issue(j_first, hs);
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
  }
  for (int e = tid; e < kStripRows * (D / 4); e += WARPS * 32) {
    const int r = e / (D / 4), c4 = e % (D / 4);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i0 + r < NB) v = __ldg(reinterpret_cast<const float4*>(qb + static_cast<int64_t>(i0 + r) * D) + c4);
    uint4 vh, vl;
    split_tf32(v.x, vh.x, vl.x);
    split_tf32(v.y, vh.y, vl.y);
    split_tf32(v.z, vh.z, vl.z);
    split_tf32(v.w, vh.w, vl.w);
    *reinterpret_cast<uint4*>(sq_hi + r * PITCH + c4 * 4) = vh;
    *reinterpret_cast<uint4*>(sq_lo + r * PITCH + c4 * 4) = vl;
  }
  __syncthreads();
  for (int j0 = warp * CHUNK; j0 < NB; j0 += WARPS * CHUNK) {
    float acc[NT][4];
#pragma unroll
    for (int ni = 0; ni < NT; ni++)
#pragma unroll
      for (int r = 0; r < 4; r++) acc[ni][r] = 0.f;
    if (j0 != j_first) {
#pragma unroll
      for (int hs = 0; hs < 3; hs++) {
        issue(j0, hs);
        asm volatile("cp.async.commit_group;" ::: "memory");
      }
    }
    uint32_t ah[2][4], al[2][4];
#pragma unroll
    for (int hs = 0; hs < HS; hs++) {
      const int jg = hs >> 1, hp = hs & 1;
      if (hs + 3 < HS) issue(j0, hs + 3);
      asm volatile("cp.async.commit_group;" ::: "memory");      // (an empty group near the end keeps the count uniform)
      asm volatile("cp.async.wait_group 3;" ::: "memory");       // the pieces of half-step hs have landed
      if (hp == 0) {
        const uint4 qah = *reinterpret_cast<const uint4*>(sq_hi + g * PITCH + 16 * jg + 4 * t);
        const uint4 qal = *reinterpret_cast<const uint4*>(sq_lo + g * PITCH + 16 * jg + 4 * t);
        const uint4 qch = *reinterpret_cast<const uint4*>(sq_hi + (g + 8) * PITCH + 16 * jg + 4 * t);
        const uint4 qcl = *reinterpret_cast<const uint4*>(sq_lo + (g + 8) * PITCH + 16 * jg + 4 * t);
        // two k-steps: (x, y) and (z, w) of each piece
        ah[0][0] = qah.x; ah[0][1] = qch.x; ah[0][2] = qah.y; ah[0][3] = qch.y;
        ah[1][0] = qah.z; ah[1][1] = qch.z; ah[1][2] = qah.w; ah[1][3] = qch.w;
        al[0][0] = qal.x; al[0][1] = qcl.x; al[0][2] = qal.y; al[0][3] = qcl.y;
        al[1][0] = qal.z; al[1][1] = qcl.z; al[1][2] = qal.w; al[1][3] = qcl.w;
      }
#pragma unroll
      for (int n2 = 0; n2 < 2; n2++) {
        const int ni = hp * 2 + n2;
        const float4 kvp = ring[(warp * 4 * 2 + (hs & 3) * 2 + n2) * 32 + lane];
        uint32_t bhh[2][2], bl[2][2];
        split_tf32(kvp.x, bhh[0][0], bl[0][0]);
        split_tf32(kvp.y, bhh[0][1], bl[0][1]);
        split_tf32(kvp.z, bhh[1][0], bl[1][0]);
        split_tf32(kvp.w, bhh[1][1], bl[1][1]);
#pragma unroll
        for (int s2 = 0; s2 < 2; s2++) {
          mma_tf32(acc[ni], al[s2], bhh[s2]);     // small terms first
          mma_tf32(acc[ni], ah[s2], bl[s2]);
          mma_tf32(acc[ni], ah[s2], bhh[s2]);
        }
      }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
#pragma unroll
    for (int ni = 0; ni < NT; ni++) {
      const int j = j0 + ni * 8 + 2 * t;
      *reinterpret_cast<float2*>(strip + g * SP + j) = make_float2(acc[ni][0] * scale, acc[ni][1] * scale);
      *reinterpret_cast<float2*>(strip + (g + 8) * SP + j) = make_float2(acc[ni][2] * scale, acc[ni][3] * scale);
    }
  }
  __syncthreads();
  const int b = bh / H;
  const uint8_t* pb = prot_blk + static_cast<int64_t>(b) * NB;
#pragma unroll 1
  for (int rr = 0; rr < kStripRows / WARPS; rr++) {
    const int r = warp * (kStripRows / WARPS) + rr;
    const int qi = i0 + r;
    if (qi >= NB) break;
    const int64_t row = static_cast<int64_t>(bh) * NB + qi;
    const float* src = strip + r * SP;
    float* dst = bs + row * NB;
    for (int i = lane; i < NB; i += 32) dst[i] = src[i];
    select_row<KPL>(src, pb, protect_rows && pb[qi] != 0, NB, k_keep, protect_cols, all_bins + warp * 256, lane,
                    col_idx + row * NB, col_cnt + row);
  }
}

// ------------------------------------------------------------------------------------------------
// Optional block-sum protection (AVSA_PROTECT_BLOCK_SUM): the response of a block is the sum of its tokens'
// scores, accumulated in fp64 (for 128 fp32 terms of like magnitude that sum is exact, so its value does not
// depend on the order of the adds) and rounded to fp32; the top-n blocks are then chosen by the same select
// kernel that chooses tokens.  One warp per block.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) block_sum_kernel(const float* __restrict__ scores, int N, int blk, int NB,
                                                        float* __restrict__ bsum) {
  const int b = blockIdx.y, lane = threadIdx.x & 31;
  const int j = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (j >= NB) return;
  const float* s = scores + static_cast<int64_t>(b) * N;
  const int lo = j * blk, hi = min(N, lo + blk);
  double acc = 0.0;
  for (int i = lo + lane; i < hi; i += 32) acc += static_cast<double>(__ldg(s + i));
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
  if (lane == 0) bsum[static_cast<int64_t>(b) * NB + j] = static_cast<float>(acc);
}

// prot_tok[b,i] = prot_blk[b, i / blk]
__global__ void __launch_bounds__(256) expand_blocks_kernel(const uint8_t* __restrict__ prot_blk, int N, int blk, int NB,
                                                            int64_t total, uint8_t* __restrict__ prot_tok) {
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
  if (idx >= total) return;
  const int64_t b = idx / N;
  const int i = static_cast<int>(idx % N);
  prot_tok[idx] = prot_blk[b * NB + i / blk];
}

// Launches the fused score + list kernel with the key slots per lane that NB needs.  Eight warps per strip (two
// rows each): sixteen warps with one row each shorten a CTA's own latency chain, but the 512-thread CTAs, staged
// while the pooling grid drains, took thread slots from its last CTAs and the call came out slower (0.118 against
// 0.103 ms on the Ovi-class shape).
template <int D, int KPL, int WARPS>
static cudaError_t launch_score_select_as(cudaLaunchConfig_t& cfg, int NB, const float* qbar, const float* kbar,
                                          float* bs, const uint8_t* pblk, int H, float scale, int k_keep, int pr, int pc,
                                          int32_t* col_idx, int32_t* col_cnt) {
  cfg.blockDim = dim3(WARPS * 32, 1, 1);
  cfg.dynamicSmemBytes = (static_cast<size_t>(2 * kStripRows) * (D + 4) + static_cast<size_t>(kStripRows) * strip_pitch<D>(NB)) *
                             sizeof(float) + WARPS * 256 * sizeof(int) + WARPS * 4 * 2 * 32 * 16;
  // always the same limit (the largest NB the call accepts), so concurrent callers never race on its value
  constexpr int kMaxSmem = (2 * kStripRows * (D + 4) + kStripRows * strip_pitch<D>(kMaxBlocksPerRow)) * 4 + WARPS * 256 * 4 + WARPS * 4 * 2 * 32 * 16;
  cudaError_t e = cudaFuncSetAttribute(score_select_kernel<D, KPL, WARPS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kMaxSmem);
  if (e != cudaSuccess) return e;
  return cudaLaunchKernelEx(&cfg, score_select_kernel<D, KPL, WARPS>, qbar, kbar, bs, pblk, H, NB, scale, k_keep, pr, pc,
                            col_idx, col_cnt);
}
template <int D>
static cudaError_t launch_score_select(cudaLaunchConfig_t& cfg, int NB, const float* qbar, const float* kbar, float* bs,
                                       const uint8_t* pblk, int H, float scale, int k_keep, int pr, int pc,
                                       int32_t* col_idx, int32_t* col_cnt) {
  if (NB <= 256)
    return launch_score_select_as<D, 8, 8>(cfg, NB, qbar, kbar, bs, pblk, H, scale, k_keep, pr, pc, col_idx, col_cnt);
  if (NB <= 512)
    return launch_score_select_as<D, 16, 8>(cfg, NB, qbar, kbar, bs, pblk, H, scale, k_keep, pr, pc, col_idx, col_cnt);
  return launch_score_select_as<D, 64, 8>(cfg, NB, qbar, kbar, bs, pblk, H, scale, k_keep, pr, pc, col_idx, col_cnt);
}

// The staged token select may use up to kSelectSmemKeys keys of dynamic shared memory.  The limit is always set
// to that same maximum, so host threads that call with different N never race on the attribute's value.
static bool allow_select_smem() {
  return cudaFuncSetAttribute(token_select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              static_cast<int>(kSelectSmemKeys * sizeof(uint32_t))) == cudaSuccess;
}

struct MaskWorkspace {
  size_t qbar, kbar, ptok, pblk, bsum, junk, total;
};
static MaskWorkspace mask_ws_layout(int B, int H, int N, int d, int blk) {
  MaskWorkspace w;
  const size_t NB = (static_cast<size_t>(N) + blk - 1) / blk;
  size_t off = kStatusBytes;
  w.qbar = off; off += align_up(static_cast<size_t>(B) * H * NB * d * sizeof(float), 256);
  w.kbar = off; off += align_up(static_cast<size_t>(B) * H * NB * d * sizeof(float), 256);
  w.ptok = off; off += align_up(static_cast<size_t>(B) * N, 256);
  w.pblk = off; off += align_up(static_cast<size_t>(B) * NB, 256);
  w.bsum = off; off += align_up(static_cast<size_t>(B) * NB * sizeof(float), 256);      // block-sum protection only
  w.junk = off; off += align_up(static_cast<size_t>(B) * ((NB + 31) / 32), 256);
  w.total = off;
  return w;
}

}  // namespace avsa

using namespace avsa;

extern "C" size_t avsa_build_block_mask_workspace_bytes(int B, int H, int N, int d, int blk) {
  if (B <= 0 || H <= 0 || N <= 0 || d <= 0 || blk <= 0) return 0;
  return mask_ws_layout(B, H, N, d, blk).total;
}

extern "C" int avsa_build_block_mask(int B, int H, int N, int d, int blk, avsa_bf16_4d q, avsa_bf16_4d k,
                                     const float* scores, int n_protect, int k_keep, unsigned flags,
                                     float softmax_scale, float* block_scores, int32_t* col_idx, int32_t* col_cnt,
                                     uint8_t* prot_tok, uint8_t* prot_blk, void* ws, size_t ws_bytes, void* stream) {
  if (B <= 0 || H <= 0 || N <= 0) return AVSA_ERR_INVALID_ARG;
  if (!((blk == 128 && d == 128) || (blk == 64 && d == 64))) return AVSA_ERR_UNSUPPORTED;
  const int NB = (N + blk - 1) / blk;
  if (NB > kMaxBlocksPerRow) return AVSA_ERR_UNSUPPORTED;
  if (k_keep < 1 || k_keep > NB || n_protect < 0 || n_protect > N) return AVSA_ERR_INVALID_ARG;
  const bool by_block_sum = (flags & AVSA_PROTECT_BLOCK_SUM) != 0;      // n_protect counts blocks
  if (by_block_sum && n_protect > NB) return AVSA_ERR_INVALID_ARG;
  if (block_scores == nullptr || col_idx == nullptr || col_cnt == nullptr) return AVSA_ERR_INVALID_ARG;
  if (n_protect > 0 && scores == nullptr) return AVSA_ERR_INVALID_ARG;
  const bool given = (flags & AVSA_USE_GIVEN_BLOCK_SCORES) != 0;
  if (!given && (!tensor_ok(q, B, H) || !tensor_ok(k, B, H))) return AVSA_ERR_INVALID_ARG;
  if ((flags & (AVSA_PROTECT_ROWS | AVSA_PROTECT_COLS | AVSA_PROTECT_TOKENS)) == 0) flags |= AVSA_PROTECT_ROWS;
  const int min_tokens = max(1, static_cast<int>((flags >> 8) & 0xffu));   // AVSA_MIN_TOKENS_PER_BLOCK(n)
  if (min_tokens > blk) return AVSA_ERR_INVALID_ARG;
  const MaskWorkspace w = mask_ws_layout(B, H, N, d, blk);
  if (ws == nullptr || ws_bytes < w.total) return AVSA_ERR_WORKSPACE;
  cudaStream_t st = as_stream(stream);
  uint8_t* base = static_cast<uint8_t*>(ws);
  float* qbar = reinterpret_cast<float*>(base + w.qbar);
  float* kbar = reinterpret_cast<float*>(base + w.kbar);
  uint8_t* ptok = prot_tok != nullptr ? prot_tok : base + w.ptok;
  uint8_t* pblk = prot_blk != nullptr ? prot_blk : base + w.pblk;
  const float scale = softmax_scale != 0.f ? softmax_scale : 1.0f / sqrtf(static_cast<float>(d));

  if (by_block_sum) {
    // block sums, then the token select run over the NB sums: its "token" flags are the block flags (its own
    // block lift goes to a scratch array); the token flags are filled in at the end of the call
    float* bsum = reinterpret_cast<float*>(base + w.bsum);
    if (n_protect > 0) block_sum_kernel<<<dim3((NB + 7) / 8, B), 256, 0, st>>>(scores, N, blk, NB, bsum);
    const size_t key_bytes = static_cast<size_t>(NB) * sizeof(uint32_t);
    if (!allow_select_smem()) return AVSA_ERR_CUDA;
    token_select_kernel<true><<<B, 1024, key_bytes, st>>>(bsum, NB, n_protect, 32, (NB + 31) / 32, 1, pblk,
                                                         base + w.junk, static_cast<StatusRecord*>(ws));
  } else if (N <= kSelectSmemKeys) {
    const size_t key_bytes = static_cast<size_t>(N) * sizeof(uint32_t);
    if (!allow_select_smem()) return AVSA_ERR_CUDA;
    token_select_kernel<true><<<B, 1024, key_bytes, st>>>(scores, N, n_protect, blk, NB, min_tokens, ptok, pblk,
                                                         static_cast<StatusRecord*>(ws));
  } else {
    token_select_kernel<false><<<B, 1024, 0, st>>>(scores, N, n_protect, blk, NB, min_tokens, ptok, pblk,
                                                   static_cast<StatusRecord*>(ws));
  }
  const int total_rows = B * H * NB;
  const int pr = (flags & AVSA_PROTECT_ROWS) ? 1 : 0, pc = (flags & AVSA_PROTECT_COLS) ? 1 : 0;
  const uint8_t* pbc = pblk;
  if (!given) {
    const __nv_bfloat16* qp = static_cast<const __nv_bfloat16*>(q.ptr);
    const __nv_bfloat16* kp = static_cast<const __nv_bfloat16*>(k.ptr);
    // the pooling kernel does not read anything the token select writes: allow it to start early
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(NB, B * H, 2);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int64_t qsb = q.stride_b, qsh = q.stride_h, qsn = q.stride_n, ksb = k.stride_b, ksh = k.stride_h,
                  ksn = k.stride_n;
    cudaError_t e;
    if (d == 128)
      e = cudaLaunchKernelEx(&cfg, pool_kernel<128>, qp, qsb, qsh, qsn, kp, ksb, ksh, ksn, qbar, kbar, H, N, blk);
    else
      e = cudaLaunchKernelEx(&cfg, pool_kernel<64>, qp, qsb, qsh, qsn, kp, ksb, ksh, ksn, qbar, kbar, H, N, blk);
    if (e != cudaSuccess) return AVSA_ERR_CUDA;
    // block scores and lists of 16 query blocks per CTA, staged behind the pooling grid
    cfg.gridDim = dim3((NB + kStripRows - 1) / kStripRows, B * H, 1);
    const float* qbc = qbar;
    const float* kbc = kbar;
    if (d == 128)
      e = launch_score_select<128>(cfg, NB, qbc, kbc, block_scores, pbc, H, scale, k_keep, pr, pc, col_idx, col_cnt);
    else
      e = launch_score_select<64>(cfg, NB, qbc, kbc, block_scores, pbc, H, scale, k_keep, pr, pc, col_idx, col_cnt);
    if (e != cudaSuccess) return AVSA_ERR_CUDA;
  } else {
    const unsigned rgrid = static_cast<unsigned>((total_rows + 3) / 4);
    const float* bsc = block_scores;
    cudaError_t e = cudaSuccess;
    if (NB <= 256)
      row_select_kernel<8><<<rgrid, 128, 0, st>>>(bsc, pbc, H, NB, k_keep, pr, pc, total_rows, col_idx, col_cnt);
    else if (NB <= 512)
      row_select_kernel<16><<<rgrid, 128, 0, st>>>(bsc, pbc, H, NB, k_keep, pr, pc, total_rows, col_idx, col_cnt);
    else
      row_select_kernel<64><<<rgrid, 128, 0, st>>>(bsc, pbc, H, NB, k_keep, pr, pc, total_rows, col_idx, col_cnt);
    e = cudaGetLastError();
    if (e != cudaSuccess) return AVSA_ERR_CUDA;
  }
  if (by_block_sum) {
    const int64_t total = static_cast<int64_t>(B) * N;
    expand_blocks_kernel<<<static_cast<unsigned>((total + 255) / 256), 256, 0, st>>>(pblk, N, blk, NB, total, ptok);
  }
  return cudaGetLastError() == cudaSuccess ? AVSA_OK : AVSA_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------
// Allocation-free variant: the workspace is a fixed array in the library's own device image.
// ------------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_mask_scratch[AVSA_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices] = {};   // device address of the array, per device ordinal
std::mutex g_static_scratch_mutex;

// In host code the array's name is only a handle for the runtime; the address a kernel can use comes
// from cudaGetSymbolAddress, asked once per device with that device current.
int static_scratch_for_current_device(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return AVSA_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return AVSA_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
  if (g_static_scratch_addr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_mask_scratch) != cudaSuccess || ptr == nullptr) return AVSA_ERR_CUDA;
    g_static_scratch_addr[dev] = ptr;
  }
  *out = g_static_scratch_addr[dev];
  return AVSA_OK;
}
}  // namespace

extern "C" int avsa_build_block_mask_static(int B, int H, int N, int d, int blk, avsa_bf16_4d q, avsa_bf16_4d k,
                                            const float* scores, int n_protect, int k_keep, unsigned flags,
                                            float softmax_scale, float* block_scores, int32_t* col_idx,
                                            int32_t* col_cnt, uint8_t* prot_tok, uint8_t* prot_blk, void* stream) {
  if (B <= 0 || H <= 0 || N <= 0 || d <= 0 || blk <= 0) return AVSA_ERR_INVALID_ARG;
  const size_t need = avsa_build_block_mask_workspace_bytes(B, H, N, d, blk);
  if (need == 0 || need > static_cast<size_t>(AVSA_STATIC_SCRATCH_BYTES)) return AVSA_ERR_WORKSPACE;
  void* scratch = nullptr;
  const int rc = static_scratch_for_current_device(&scratch);
  if (rc != AVSA_OK) return rc;
  return avsa_build_block_mask(B, H, N, d, blk, q, k, scores, n_protect, k_keep, flags, softmax_scale, block_scores,
                               col_idx, col_cnt, prot_tok, prot_blk, scratch, AVSA_STATIC_SCRATCH_BYTES, stream);
}
