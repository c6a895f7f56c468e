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
template <int D>
__global__ void __launch_bounds__(256) pool_kernel(const __nv_bfloat16* __restrict__ q, int64_t q_sb, int64_t q_sh,
                                                   int64_t q_sn, const __nv_bfloat16* __restrict__ k, int64_t k_sb,
                                                   int64_t k_sh, int64_t k_sn, float* __restrict__ qbar,
                                                   float* __restrict__ kbar, int H, int N, int blk) {
  constexpr int TPR = D / 8;          // threads per row
  constexpr int RPP = 256 / TPR;      // rows per pass
  __shared__ float part[RPP][D + 4];
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
}

// ------------------------------------------------------------------------------------------------
// (ii) block scores Bs[bh, i, j] = qbar[bh,i,:] . kbar[bh,j,:] * scale.  64x64 tile per CTA,
// 256 threads x (4x4) outputs, channels summed in ascending order.
// ------------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256) block_score_kernel(const float* __restrict__ qbar,
                                                          const float* __restrict__ kbar, float* __restrict__ bs,
                                                          int NB, float scale) {
  constexpr int KC = 32;
  __shared__ float sq[KC][64 + 1];
  __shared__ float sk[KC][64 + 1];
  const int bh = blockIdx.z, i0 = blockIdx.y * 64, j0 = blockIdx.x * 64;
  const float* qb = qbar + static_cast<int64_t>(bh) * NB * D;
  const float* kb = kbar + static_cast<int64_t>(bh) * NB * D;
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; a++)
#pragma unroll
    for (int c = 0; c < 4; c++) acc[a][c] = 0.f;
  for (int k0 = 0; k0 < D; k0 += KC) {
    for (int e = threadIdx.x; e < 64 * KC; e += 256) {
      const int r = e / KC, c = e % KC;
      sq[c][r] = (i0 + r < NB) ? qb[static_cast<int64_t>(i0 + r) * D + k0 + c] : 0.f;
      sk[c][r] = (j0 + r < NB) ? kb[static_cast<int64_t>(j0 + r) * D + k0 + c] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int c = 0; c < KC; c++) {
      float a[4], bq[4];
#pragma unroll
      for (int t = 0; t < 4; t++) {
        a[t] = sq[c][ty * 4 + t];
        bq[t] = sk[c][tx * 4 + t];
      }
#pragma unroll
      for (int t = 0; t < 4; t++)
#pragma unroll
        for (int u = 0; u < 4; u++) acc[t][u] = fmaf(a[t], bq[u], acc[t][u]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int t = 0; t < 4; t++) {
    const int i = i0 + ty * 4 + t;
    if (i >= NB) continue;
#pragma unroll
    for (int u = 0; u < 4; u++) {
      const int j = j0 + tx * 4 + u;
      if (j < NB) bs[(static_cast<int64_t>(bh) * NB + i) * NB + j] = acc[t][u] * scale;
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Radix-select helper: given 256 digit counts (descending scan), find the digit that holds the
// want-th largest element.  One warp; lane l owns digits 255-8l .. 248-8l.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void warp_pick_digit(const int* bins, int want, int lane, int& digit, int& above) {
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
  int dg = 0, ab = 0;
  if (mine) {
    int run = excl;
#pragma unroll
    for (int i = 0; i < 8; i++) {
      if (run < want && want <= run + local[i]) {
        dg = 255 - (lane * 8 + i);
        ab = run;
      }
      run += local[i];
    }
  }
  const unsigned who = __ballot_sync(0xffffffffu, mine);
  const int src = __ffs(who) - 1;
  digit = __shfl_sync(0xffffffffu, dg, src);
  above = __shfl_sync(0xffffffffu, ab, src);
}

// ------------------------------------------------------------------------------------------------
// (iii) protected token set: one CTA of 1024 threads per batch item.  Radix select (4 x 8 bits) of
// the n_protect-th largest key, then an index-ordered pass that takes every larger key and the
// lowest-index ties, writes the token flags and raises the flag of every block that holds one.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) token_select_kernel(const float* __restrict__ scores, int N, int n_protect,
                                                            int blk, int NB, uint8_t* __restrict__ prot_tok,
                                                            uint8_t* __restrict__ prot_blk) {
  __shared__ int bins[256];
  __shared__ int s_digit, s_above;
  __shared__ int warp_cnt[32];
  __shared__ int s_eq_seen;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* s = scores + static_cast<int64_t>(b) * N;
  uint8_t* ptok = prot_tok + static_cast<int64_t>(b) * N;
  uint8_t* pblk = prot_blk + static_cast<int64_t>(b) * NB;
  for (int i = tid; i < NB; i += 1024) pblk[i] = 0;
  if (n_protect <= 0) {
    for (int i = tid; i < N; i += 1024) ptok[i] = 0;
    return;
  }
  uint32_t prefix = 0, mask = 0;
  int want = n_protect;
  for (int pass = 0; pass < 4; pass++) {
    const int shift = 24 - 8 * pass;
    if (tid < 256) bins[tid] = 0;
    __syncthreads();
    for (int i0 = 0; i0 < N; i0 += 1024) {
      const int i = i0 + tid;
      const bool valid = i < N;
      const uint32_t key = valid ? rank_key(s[i]) : 0u;
      const bool in = valid && ((key & mask) == prefix);
      const uint32_t dgt = in ? ((key >> shift) & 255u) : 256u;
      const unsigned peers = __match_any_sync(0xffffffffu, dgt);
      if (in && lane == __ffs(peers) - 1) atomicAdd(&bins[dgt], __popc(peers));
    }
    __syncthreads();
    if (warp == 0) {
      int dg, ab;
      warp_pick_digit(bins, want, lane, dg, ab);
      if (lane == 0) {
        s_digit = dg;
        s_above = ab;
      }
    }
    __syncthreads();
    want -= s_above;
    prefix |= static_cast<uint32_t>(s_digit) << shift;
    mask |= 255u << shift;
    __syncthreads();
  }
  const uint32_t T = prefix;     // the n_protect-th largest key; `want` ties at T are taken, lowest index first
  if (tid == 0) s_eq_seen = 0;
  __syncthreads();
  for (int i0 = 0; i0 < N; i0 += 1024) {
    const int i = i0 + tid;
    const bool valid = i < N;
    const uint32_t key = valid ? rank_key(s[i]) : 0u;
    const bool gt = valid && key > T;
    const bool eq = valid && key == T;
    const unsigned eqm = __ballot_sync(0xffffffffu, eq);
    if (lane == 0) warp_cnt[warp] = __popc(eqm);
    __syncthreads();
    int before = s_eq_seen;
    for (int w = 0; w < warp; w++) before += warp_cnt[w];
    const int rank = before + __popc(eqm & ((1u << lane) - 1u));
    const bool keep = gt || (eq && rank < want);
    if (valid) ptok[i] = keep ? 1 : 0;
    const unsigned km = __ballot_sync(0xffffffffu, keep);
    if (km != 0u && lane == 0) pblk[(i0 + warp * 32) / blk] = 1;   // blk is a multiple of 32
    __syncthreads();
    if (tid == 0) {
      int tot = 0;
      for (int w = 0; w < 32; w++) tot += warp_cnt[w];
      s_eq_seen += tot;
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------------------------------------
// (iv) per-(head, query block) top-k_keep of a block-score row, protection OR (Eq. 9), ascending
// list emission.  One warp per row, 4 rows per CTA.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) row_select_kernel(const float* __restrict__ bs, const uint8_t* __restrict__ prot_blk,
                                                         int H, int NB, int k_keep, int protect_rows,
                                                         int protect_cols, int total_rows, int32_t* __restrict__ col_idx,
                                                         int32_t* __restrict__ col_cnt) {
  extern __shared__ uint32_t dyn[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint32_t* keys = dyn + static_cast<size_t>(warp) * NB;
  int* bins = reinterpret_cast<int*>(dyn + static_cast<size_t>(4) * NB) + warp * 256;
  const int row = blockIdx.x * 4 + warp;      // row = (b*H + h)*NB + qb
  if (row >= total_rows) return;
  const int qb = row % NB;
  const int b = row / (NB * H);
  const float* src = bs + static_cast<int64_t>(row) * NB;
  int32_t* out = col_idx + static_cast<int64_t>(row) * NB;
  const uint8_t* pb = prot_blk + static_cast<int64_t>(b) * NB;
  const bool row_prot = protect_rows && pb[qb] != 0;
  const unsigned lt = (1u << lane) - 1u;

  uint32_t T = 0;
  int want = 0;
  if (!row_prot && k_keep < NB) {
    for (int i = lane; i < NB; i += 32) keys[i] = rank_key(src[i]);
    __syncwarp();
    uint32_t prefix = 0, mask = 0;
    want = k_keep;
    for (int pass = 0; pass < 4; pass++) {
      const int shift = 24 - 8 * pass;
      for (int i = lane; i < 256; i += 32) bins[i] = 0;
      __syncwarp();
      for (int i0 = 0; i0 < NB; i0 += 32) {
        const int i = i0 + lane;
        const bool valid = i < NB;
        const uint32_t key = valid ? keys[i] : 0u;
        const bool in = valid && ((key & mask) == prefix);
        const uint32_t dgt = in ? ((key >> shift) & 255u) : 256u;
        const unsigned peers = __match_any_sync(0xffffffffu, dgt);
        if (in && lane == __ffs(peers) - 1) bins[dgt] += __popc(peers);
        __syncwarp();
      }
      int dg, ab;
      warp_pick_digit(bins, want, lane, dg, ab);
      want -= ab;
      prefix |= static_cast<uint32_t>(dg) << shift;
      mask |= 255u << shift;
      __syncwarp();
    }
    T = prefix;
  }
  const bool keep_all = row_prot || k_keep >= NB;
  int pos = 0, eq_seen = 0;
  for (int i0 = 0; i0 < NB; i0 += 32) {
    const int i = i0 + lane;
    const bool valid = i < NB;
    bool keep;
    if (keep_all) {
      keep = valid;
    } else {
      const uint32_t key = valid ? keys[i] : 0u;
      const bool gt = valid && key > T;
      const bool eq = valid && key == T;
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
  if (lane == 0) col_cnt[row] = pos;
}

struct MaskWorkspace {
  size_t qbar, kbar, ptok, pblk, total;
};
static MaskWorkspace mask_ws_layout(int B, int H, int N, int d, int blk) {
  MaskWorkspace w;
  const size_t NB = (static_cast<size_t>(N) + blk - 1) / blk;
  size_t off = kStatusBytes;
  w.qbar = off; off += align_up(static_cast<size_t>(B) * H * NB * d * sizeof(float), 256);
  w.kbar = off; off += align_up(static_cast<size_t>(B) * H * NB * d * sizeof(float), 256);
  w.ptok = off; off += align_up(static_cast<size_t>(B) * N, 256);
  w.pblk = off; off += align_up(static_cast<size_t>(B) * NB, 256);
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
  if (block_scores == nullptr || col_idx == nullptr || col_cnt == nullptr) return AVSA_ERR_INVALID_ARG;
  if (n_protect > 0 && scores == nullptr) return AVSA_ERR_INVALID_ARG;
  const bool given = (flags & AVSA_USE_GIVEN_BLOCK_SCORES) != 0;
  if (!given && (!tensor_ok(q, B, H) || !tensor_ok(k, B, H))) return AVSA_ERR_INVALID_ARG;
  if ((flags & (AVSA_PROTECT_ROWS | AVSA_PROTECT_COLS)) == 0) flags |= AVSA_PROTECT_ROWS;
  const MaskWorkspace w = mask_ws_layout(B, H, N, d, blk);
  if (ws == nullptr || ws_bytes < w.total) return AVSA_ERR_WORKSPACE;
  cudaStream_t st = as_stream(stream);
  uint8_t* base = static_cast<uint8_t*>(ws);
  float* qbar = reinterpret_cast<float*>(base + w.qbar);
  float* kbar = reinterpret_cast<float*>(base + w.kbar);
  uint8_t* ptok = prot_tok != nullptr ? prot_tok : base + w.ptok;
  uint8_t* pblk = prot_blk != nullptr ? prot_blk : base + w.pblk;
  const float scale = softmax_scale != 0.f ? softmax_scale : 1.0f / sqrtf(static_cast<float>(d));

  clear_status_kernel<<<1, 1, 0, st>>>(static_cast<StatusRecord*>(ws));
  token_select_kernel<<<B, 1024, 0, st>>>(scores, N, n_protect, blk, NB, ptok, pblk);
  if (!given) {
    const __nv_bfloat16* qp = static_cast<const __nv_bfloat16*>(q.ptr);
    const __nv_bfloat16* kp = static_cast<const __nv_bfloat16*>(k.ptr);
    dim3 pg(NB, B * H, 2);
    dim3 sg((NB + 63) / 64, (NB + 63) / 64, B * H);
    if (d == 128) {
      pool_kernel<128><<<pg, 256, 0, st>>>(qp, q.stride_b, q.stride_h, q.stride_n, kp, k.stride_b, k.stride_h,
                                          k.stride_n, qbar, kbar, H, N, blk);
      block_score_kernel<128><<<sg, 256, 0, st>>>(qbar, kbar, block_scores, NB, scale);
    } else {
      pool_kernel<64><<<pg, 256, 0, st>>>(qp, q.stride_b, q.stride_h, q.stride_n, kp, k.stride_b, k.stride_h,
                                         k.stride_n, qbar, kbar, H, N, blk);
      block_score_kernel<64><<<sg, 256, 0, st>>>(qbar, kbar, block_scores, NB, scale);
    }
  }
  const int total_rows = B * H * NB;
  const size_t smem = (static_cast<size_t>(4) * NB + 4 * 256) * sizeof(uint32_t);
  row_select_kernel<<<(total_rows + 3) / 4, 128, smem, st>>>(block_scores, pblk, H, NB, k_keep,
                                                             (flags & AVSA_PROTECT_ROWS) ? 1 : 0,
                                                             (flags & AVSA_PROTECT_COLS) ? 1 : 0, total_rows, col_idx,
                                                             col_cnt);
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
