// avsa_sparse_self_attn: block-sparse video self-attention under the protected block mask
// (Eq. 10 / Eq. 11; Eq. 5 when every list is full).  Host side: argument checks, tensor maps, launch.
#include "attn_persist_kernel.cuh"

namespace avsa {

// First kernel of the call: resets the status record and writes the order in which the persistent kernel's
// work queue hands out the query tiles.  Query tiles go head by head (one head's K and V stay in L2 while its
// tiles are in flight), except for the last heads of the queue, from `tail_start` on: there the long lists
// (more than half the key blocks: the protected, dense rows) come first and the short ones last, each class in
// index order.  With long items at the very end of the queue, the last CTAs to finish would leave the others
// idle for up to a whole dense row; reordering the whole queue that way would read every head's K and V twice
// from DRAM (once per class), which is why only as many heads as fit in L2 together are reordered.
__global__ void __launch_bounds__(1024) prep_sparse_kernel(StatusRecord* st, const int32_t* __restrict__ col_cnt,
                                                           int n_items, int tail_start, int NKB,
                                                           int* __restrict__ order) {
  __shared__ int warp_tot[32];
  __shared__ int total_heavy;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    st->code = 0;
    st->where = 0;
    st->item = 0;
    st->aux = 0;
    st->redo_count = 0;
    st->next_item = 0;
  }
  for (int i = tid; i < tail_start; i += 1024) order[i] = i;
  const int n_tail = n_items - tail_start;
  const int chunk = (n_tail + 1023) / 1024;
  const int lo = tail_start + min(n_tail, tid * chunk), hi = min(n_items, lo + chunk);
  int heavy = 0;
  for (int i = lo; i < hi; i++) heavy += (2 * col_cnt[i] > NKB) ? 1 : 0;
  // exclusive scan of the per-thread counts over the block
  int incl = heavy;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += t;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const int w = warp_tot[lane];
    int wi = w;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, wi, off);
      if (lane >= off) wi += t;
    }
    warp_tot[lane] = wi - w;
    if (lane == 31) total_heavy = wi;
  }
  __syncthreads();
  int h_pos = warp_tot[warp] + incl - heavy;                      // heavy items of the tail before this thread's chunk
  int l_pos = total_heavy + (lo - tail_start) - h_pos;            // light items go behind all heavy ones
  for (int i = lo; i < hi; i++) {
    if (2 * col_cnt[i] > NKB) order[tail_start + h_pos++] = i; else order[tail_start + l_pos++] = i;
  }
}

// Self-test of the time-limited wait used throughout the tile kernels: one warp waits on an mbarrier that nothing
// ever arrives on, gives up after `limit_cycles`, records AVSA_ERR_TIMEOUT in the status record and returns.
constexpr int kWhereSelfTestWait = 99;
__global__ void __launch_bounds__(32) bounded_wait_selftest_kernel(StatusRecord* st, long long limit_cycles) {
  __shared__ __align__(8) uint64_t bar;
  const uint32_t b = smem_u32(&bar);
  if (threadIdx.x == 0) {
    st->code = 0;
    st->where = 0;
    st->item = 0;
    st->aux = 0;
    st->redo_count = 0;
    st->next_item = 0;
    mbar_init(b, 1);
    fence_mbar_init();
  }
  __syncwarp();
  if (threadIdx.x == 0) {
    const long long t0 = clock64();
    while (!mbar_try_wait(b, 0)) {
      const long long waited = clock64() - t0;
      if (waited > limit_cycles) {
        report_status(st, AVSA_ERR_TIMEOUT, kWhereSelfTestWait, 0, static_cast<int>(min(waited >> 10, 0x7fffffffll)));
        break;
      }
    }
  }
  __syncwarp();
  if (threadIdx.x == 0) mbar_inval(b);
}

template <int BLK, int D>
static int launch_sparse_attn(int B, int H, int N, const avsa_bf16_4d& q, const avsa_bf16_4d& k,
                              const avsa_bf16_4d& v, void* o, const AttnParams& prm, int* redo, cudaStream_t st) {
  using L = AttnSmem<BLK, D>;
  CUtensorMap tq, tk, tv, to;
  if (!encode_bf16_tile_map(&tq, q.ptr, B, H, N, D, q.stride_b, q.stride_h, q.stride_n, BLK)) return AVSA_ERR_CUDA;
  if (!encode_bf16_tile_map(&tk, k.ptr, B, H, N, D, k.stride_b, k.stride_h, k.stride_n, BLK)) return AVSA_ERR_CUDA;
  if (!encode_bf16_tile_map(&tv, v.ptr, B, H, N, D, v.stride_b, v.stride_h, v.stride_n, BLK)) return AVSA_ERR_CUDA;
  if (!encode_bf16_tile_map(&to, o, B, H, N, D, q.stride_b, q.stride_h, q.stride_n, BLK)) return AVSA_ERR_CUDA;
  if (cudaFuncSetAttribute(attn_redo_kernel<BLK, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal) !=
      cudaSuccess)
    return AVSA_ERR_CUDA;
  // The persistent fast kernel first; it lists the (rare) work items whose rows outgrow its fixed reference
  // maxima, and the exact-rescaling kernel behind it recomputes exactly those.
  const long long items = static_cast<long long>(prm.NQT) * H * B;
  using LP = PersistSmem<BLK, D>;
  if (cudaFuncSetAttribute(attn_persist_kernel<BLK, D, MODE_LIST>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           LP::kTotal) != cudaSuccess)
    return AVSA_ERR_CUDA;
  attn_persist_kernel<BLK, D, MODE_LIST><<<persistent_grid(items), kAttnThreads, LP::kTotal, st>>>(
      tq, tk, tv, to, prm, redo, redo + items, static_cast<int>(items));
  const int redo_grid = persistent_grid(items);
  attn_redo_kernel<BLK, D><<<redo_grid, kAttnThreads, L::kTotal, st>>>(tq, tk, tv, to, prm, redo);
  return cudaGetLastError() == cudaSuccess ? AVSA_OK : AVSA_ERR_CUDA;
}

}  // namespace avsa

using namespace avsa;

extern "C" int avsa_selftest_bounded_wait(void* ws, size_t ws_bytes, long long limit_cycles, void* stream) {
  if (ws == nullptr || ws_bytes < kStatusBytes) return AVSA_ERR_WORKSPACE;
  if (limit_cycles < 0 || limit_cycles > 2000000000ll) return AVSA_ERR_INVALID_ARG;     // about a second at most
  if (!device_is_sm100()) return AVSA_ERR_UNSUPPORTED;
  bounded_wait_selftest_kernel<<<1, 32, 0, as_stream(stream)>>>(static_cast<StatusRecord*>(ws), limit_cycles);
  return cudaGetLastError() == cudaSuccess ? AVSA_OK : AVSA_ERR_CUDA;
}

extern "C" size_t avsa_sparse_self_attn_workspace_bytes(int B, int H, int N, int d, int blk) {
  if (B <= 0 || H <= 0 || N <= 0 || d <= 0 || blk <= 0) return 0;
  const size_t nb = (static_cast<size_t>(N) + blk - 1) / blk;
  // status record, list of recomputed work items, order of the work queue
  return kStatusBytes + align_up(static_cast<size_t>(B) * H * nb * 2 * sizeof(int), 256);
}

extern "C" int avsa_sparse_self_attn(int B, int H, int N, int d, int blk, avsa_bf16_4d q, avsa_bf16_4d k,
                                     avsa_bf16_4d v, const int32_t* col_idx, const int32_t* col_cnt, void* o_bf16,
                                     float* lse, float softmax_scale, void* ws, size_t ws_bytes, void* stream) {
  if (B <= 0 || H <= 0 || N <= 0) return AVSA_ERR_INVALID_ARG;
  if (!((blk == 128 && d == 128) || (blk == 64 && d == 64))) return AVSA_ERR_UNSUPPORTED;
  if (H > 65535 || B > 65535) return AVSA_ERR_UNSUPPORTED;
  if (!tensor_ok(q, B, H) || !tensor_ok(k, B, H) || !tensor_ok(v, B, H)) return AVSA_ERR_INVALID_ARG;
  if (col_idx == nullptr || col_cnt == nullptr || o_bf16 == nullptr || !aligned16(o_bf16)) return AVSA_ERR_INVALID_ARG;
  if (softmax_scale < 0.f || softmax_scale != softmax_scale) return AVSA_ERR_INVALID_ARG;
  if (ws == nullptr || ws_bytes < avsa_sparse_self_attn_workspace_bytes(B, H, N, d, blk)) return AVSA_ERR_WORKSPACE;
  if (!device_is_sm100()) return AVSA_ERR_UNSUPPORTED;
  cudaStream_t st = as_stream(stream);
  AttnParams prm = {};
  prm.col_idx = col_idx;
  prm.col_cnt = col_cnt;
  prm.lse = lse;
  prm.status = static_cast<StatusRecord*>(ws);
  prm.H = H;
  prm.Nq = N;
  prm.Nk = N;
  prm.NQT = prm.NKB = (N + blk - 1) / blk;
  const float scale = softmax_scale != 0.f ? softmax_scale : 1.0f / sqrtf(static_cast<float>(d));
  prm.scale_log2 = scale * 1.4426950408889634f;
  int* redo = reinterpret_cast<int*>(static_cast<uint8_t*>(ws) + kStatusBytes);
  const long long n_items = static_cast<long long>(B) * H * prm.NQT;
  if (n_items > 0x3fffffff) return AVSA_ERR_UNSUPPORTED;
  // heads whose K and V (2 x N x d bf16 each) fit into about half of the 126 MB L2 together
  const long long kv_bytes = 4ll * N * d;
  long long tail_heads = (64ll << 20) / kv_bytes;
  if (tail_heads < 1) tail_heads = 1;
  if (tail_heads > static_cast<long long>(B) * H) tail_heads = static_cast<long long>(B) * H;
  const int tail_start = static_cast<int>((static_cast<long long>(B) * H - tail_heads) * prm.NQT);
  prep_sparse_kernel<<<1, 1024, 0, st>>>(prm.status, col_cnt, static_cast<int>(n_items), tail_start, prm.NKB,
                                         redo + n_items);
  if (d == 128) return launch_sparse_attn<128, 128>(B, H, N, q, k, v, o_bf16, prm, redo, st);
  return launch_sparse_attn<64, 64>(B, H, N, q, k, v, o_bf16, prm, redo, st);
}
