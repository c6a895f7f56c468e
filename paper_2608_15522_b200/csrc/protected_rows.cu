// avsa_protected_rows_attn: token-exact protection.  Eq. 9 restores full key connectivity for the
// protected *tokens*; Eq. 11 states it row-wise (protected rows are dense attention rows) and the
// paper's implementation notes call it dense-row recomputation.  The protected query rows are
// gathered into compact tiles, run densely through the attention tile kernel with the key axis split
// across CTAs, and the merged rows overwrite the sparse result in place.
#include "attn_persist_kernel.cuh"

namespace avsa {

enum ProtWhere { kProtCount = 41 };

// prot_tok [B,N] flags -> rows [B, n_pad] ascending token indices, -1 beyond the count.
// One CTA of 1024 threads per batch item; every warp owns a contiguous, 32-aligned segment.
__global__ void __launch_bounds__(1024) compact_rows_kernel(const uint8_t* __restrict__ prot_tok, int N, int n_protect,
                                                            int n_pad, int32_t* __restrict__ rows,
                                                            StatusRecord* status) {
  __shared__ int warp_cnt[32];
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint8_t* f = prot_tok + static_cast<int64_t>(b) * N;
  int32_t* out = rows + static_cast<int64_t>(b) * n_pad;
  if (b == 0 && tid == 0) {
    status->code = 0;
    status->where = 0;
    status->item = 0;
    status->aux = 0;
    status->redo_count = 0;
    status->next_item = 0;
  }
  for (int i = tid; i < n_pad; i += 1024) out[i] = -1;
  const int seg = ((N + 31) / 32 + 31) / 32 * 32;
  const int lo = warp * seg, hi = min(N, lo + seg);
  int mine = 0;
  for (int i0 = lo; i0 < hi; i0 += 32) {
    const int i = i0 + lane;
    mine += __popc(__ballot_sync(0xffffffffu, i < hi && f[i] != 0));
  }
  if (lane == 0) warp_cnt[warp] = mine;
  __syncthreads();     // also orders the -1 fill before the index writes below
  int before = 0, total = 0;
  for (int w2 = 0; w2 < 32; w2++) {
    if (w2 < warp) before += warp_cnt[w2];
    total += warp_cnt[w2];
  }
  if (total != n_protect) {
    if (tid == 0) report_status(status, AVSA_ERR_BAD_MASK, kProtCount, b, total);
    return;     // rows stay -1: nothing is gathered or scattered for this batch item
  }
  for (int i0 = lo; i0 < hi; i0 += 32) {
    const int i = i0 + lane;
    const bool on = i < hi && f[i] != 0;
    const unsigned m = __ballot_sync(0xffffffffu, on);
    if (on) out[before + __popc(m & ((1u << lane) - 1u))] = i;
    before += __popc(m);
  }
}

// Qp[b,h,r,:] = Q[b,h,rows[b][r],:]; rows < 0 give zero rows.  16-byte copies.
template <int D>
__global__ void __launch_bounds__(256) gather_rows_kernel(const __nv_bfloat16* __restrict__ q, int64_t sb, int64_t sh,
                                                          int64_t sn, const int32_t* __restrict__ rows, int n_pad,
                                                          __nv_bfloat16* __restrict__ qp) {
  constexpr int TPR = D / 8;
  const int r = blockIdx.x * (256 / TPR) + threadIdx.x / TPR;
  const int c = threadIdx.x % TPR;
  const int h = blockIdx.y, b = blockIdx.z, H = gridDim.y;
  if (r >= n_pad) return;
  const int src = rows[static_cast<int64_t>(b) * n_pad + r];
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (src >= 0) v = __ldg(reinterpret_cast<const uint4*>(q + b * sb + h * sh + src * sn) + c);
  reinterpret_cast<uint4*>(qp + ((static_cast<int64_t>(b) * H + h) * n_pad + r) * D)[c] = v;
}

struct ProtPlan {
  int n_pad, NQT, NKB, n_split, tps;
  size_t off_rows, off_qp, off_part_o, off_part_lse, off_redo, total;
};

static ProtPlan make_prot_plan(int B, int H, int N, int d, int blk, int n_protect) {
  ProtPlan c;
  c.NQT = (n_protect + blk - 1) / blk;
  if (c.NQT < 1) c.NQT = 1;
  c.n_pad = c.NQT * blk;
  c.NKB = (N + blk - 1) / blk;
  // key-axis splits: work items of about 64 tiles, and at least two waves of 148 items when possible
  int want = (c.NKB + 63) / 64;
  const int items1 = B * H * c.NQT;
  while (items1 * want < 296 && want < c.NKB) want++;
  c.tps = (c.NKB + want - 1) / want;
  c.n_split = (c.NKB + c.tps - 1) / c.tps;
  size_t off = kStatusBytes;
  const size_t items = static_cast<size_t>(items1) * c.n_split;
  c.off_rows = off; off += align_up(static_cast<size_t>(B) * c.n_pad * sizeof(int32_t), 256);
  c.off_qp = off; off += align_up(static_cast<size_t>(B) * H * c.n_pad * d * 2, 256);
  c.off_part_o = off; off += align_up(items * blk * d * sizeof(float), 256);
  c.off_part_lse = off; off += align_up(items * blk * sizeof(float), 256);
  c.off_redo = off; off += align_up(items * sizeof(int), 256);
  c.total = off;
  return c;
}

template <int BLK, int D>
static int run_protected(int B, int H, int N, int n_protect, const avsa_bf16_4d& q, const avsa_bf16_4d& k,
                         const avsa_bf16_4d& v, const uint8_t* prot_tok, void* o, float* lse, float scale, uint8_t* ws,
                         const ProtPlan& c, cudaStream_t st) {
  using L = AttnSmem<BLK, D>;
  StatusRecord* status = reinterpret_cast<StatusRecord*>(ws);
  int32_t* rows = reinterpret_cast<int32_t*>(ws + c.off_rows);
  __nv_bfloat16* qp = reinterpret_cast<__nv_bfloat16*>(ws + c.off_qp);
  float* part_o = reinterpret_cast<float*>(ws + c.off_part_o);
  float* part_lse = reinterpret_cast<float*>(ws + c.off_part_lse);
  compact_rows_kernel<<<B, 1024, 0, st>>>(prot_tok, N, n_protect, c.n_pad, rows, status);
  constexpr int RPB = 256 / (D / 8);
  gather_rows_kernel<D><<<dim3((c.n_pad + RPB - 1) / RPB, H, B), 256, 0, st>>>(
      static_cast<const __nv_bfloat16*>(q.ptr), q.stride_b, q.stride_h, q.stride_n, rows, c.n_pad, qp);
  CUtensorMap tq, tk, tv;
  if (!encode_bf16_tile_map(&tq, qp, B, H, c.n_pad, D, static_cast<int64_t>(H) * c.n_pad * D,
                            static_cast<int64_t>(c.n_pad) * D, D, BLK))
    return AVSA_ERR_CUDA;
  if (!encode_bf16_tile_map(&tk, k.ptr, B, H, N, D, k.stride_b, k.stride_h, k.stride_n, BLK)) return AVSA_ERR_CUDA;
  if (!encode_bf16_tile_map(&tv, v.ptr, B, H, N, D, v.stride_b, v.stride_h, v.stride_n, BLK)) return AVSA_ERR_CUDA;
  using LP = PersistSmem<BLK, D>;
  if (cudaFuncSetAttribute(attn_persist_kernel<BLK, D, MODE_RANGE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           LP::kTotal) != cudaSuccess)
    return AVSA_ERR_CUDA;
  if (cudaFuncSetAttribute(attn_redo_kernel<BLK, D, MODE_RANGE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           L::kTotal) != cudaSuccess)
    return AVSA_ERR_CUDA;
  AttnParams prm = {};
  prm.part_o = part_o;
  prm.part_lse2 = part_lse;
  prm.n_split = c.n_split;
  prm.tiles_per_split = c.tps;
  prm.status = status;
  prm.H = H;
  prm.Nq = c.n_pad;
  prm.NQT = c.NQT;
  prm.Nk = N;
  prm.NKB = c.NKB;
  prm.scale_log2 = scale * 1.4426950408889634f;
  // persistent fast kernel over the (row tile, key split) items, then the exact kernel for what it handed over
  int* redo = reinterpret_cast<int*>(ws + c.off_redo);
  const long long items = static_cast<long long>(B) * H * c.NQT * c.n_split;
  const int grid = persistent_grid(items);
  attn_persist_kernel<BLK, D, MODE_RANGE><<<grid, kAttnThreads, LP::kTotal, st>>>(tq, tk, tv, tq, prm, redo, nullptr,
                                                                                  static_cast<int>(items));
  attn_redo_kernel<BLK, D, MODE_RANGE><<<grid, kAttnThreads, L::kTotal, st>>>(tq, tk, tv, tq, prm, redo);
  const int total_rows = B * H * c.n_pad;
  constexpr int MRPB = 128 / (D / 4);
  merge_splits_kernel<BLK, D><<<(total_rows + MRPB - 1) / MRPB, 128, 0, st>>>(
      part_o, part_lse, c.n_split, c.NQT, c.n_pad, H, total_rows, static_cast<__nv_bfloat16*>(o), q.stride_b,
      q.stride_h, q.stride_n, lse, rows, c.n_pad, N);
  return cudaGetLastError() == cudaSuccess ? AVSA_OK : AVSA_ERR_CUDA;
}

}  // namespace avsa

using namespace avsa;

extern "C" size_t avsa_protected_rows_attn_workspace_bytes(int B, int H, int N, int d, int blk, int n_protect) {
  if (B <= 0 || H <= 0 || N <= 0 || n_protect < 0 || n_protect > N) return 0;
  if (!((blk == 128 && d == 128) || (blk == 64 && d == 64))) return 0;
  return make_prot_plan(B, H, N, d, blk, n_protect).total;
}

extern "C" int avsa_protected_rows_attn(int B, int H, int N, int d, int blk, avsa_bf16_4d q, avsa_bf16_4d k,
                                        avsa_bf16_4d v, const uint8_t* prot_tok, int n_protect, void* o_bf16,
                                        float* lse, float softmax_scale, void* ws, size_t ws_bytes, void* stream) {
  if (B <= 0 || H <= 0 || N <= 0 || n_protect < 0 || n_protect > N) return AVSA_ERR_INVALID_ARG;
  if (!((blk == 128 && d == 128) || (blk == 64 && d == 64))) return AVSA_ERR_UNSUPPORTED;
  if (H > 65535 || B > 65535) return AVSA_ERR_UNSUPPORTED;
  if (!tensor_ok(q, B, H) || !tensor_ok(k, B, H) || !tensor_ok(v, B, H)) return AVSA_ERR_INVALID_ARG;
  if (prot_tok == nullptr || o_bf16 == nullptr || !aligned16(o_bf16)) return AVSA_ERR_INVALID_ARG;
  if (softmax_scale < 0.f || softmax_scale != softmax_scale) return AVSA_ERR_INVALID_ARG;
  const ProtPlan c = make_prot_plan(B, H, N, d, blk, n_protect);
  if (ws == nullptr || ws_bytes < c.total) return AVSA_ERR_WORKSPACE;
  if (!device_is_sm100()) return AVSA_ERR_UNSUPPORTED;
  const float scale = softmax_scale != 0.f ? softmax_scale : 1.0f / sqrtf(static_cast<float>(d));
  if (n_protect == 0) {
    clear_status_kernel<<<1, 1, 0, as_stream(stream)>>>(static_cast<StatusRecord*>(ws));
    return cudaGetLastError() == cudaSuccess ? AVSA_OK : AVSA_ERR_CUDA;
  }
  uint8_t* base = static_cast<uint8_t*>(ws);
  if (d == 128)
    return run_protected<128, 128>(B, H, N, n_protect, q, k, v, prot_tok, o_bf16, lse, scale, base, c,
                                   as_stream(stream));
  return run_protected<64, 64>(B, H, N, n_protect, q, k, v, prot_tok, o_bf16, lse, scale, base, c, as_stream(stream));
}
