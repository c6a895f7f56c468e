// avsa_sparse_self_attn: block-sparse video self-attention under the protected block mask
// (Eq. 10 / Eq. 11; Eq. 5 when every list is full).  Host side: argument checks, tensor maps, launch.
#include "attn_persist_kernel.cuh"

namespace avsa {

template <int BLK, int D>
static int launch_sparse_attn(int B, int H, int N, const avsa_bf16_4d& q, const avsa_bf16_4d& k,
                              const avsa_bf16_4d& v, void* o, const AttnParams& prm, int* redo, cudaStream_t st) {
  using L = AttnSmem<BLK, D>;
  CUtensorMap tq, tk, tv, to;
  if (!encode_bf16_tile_map(&tq, q.ptr, B, H, N, D, q.stride_b, q.stride_h, q.stride_n, BLK)) return AVSA_ERR_CUDA;
  if (!encode_bf16_tile_map(&tk, k.ptr, B, H, N, D, k.stride_b, k.stride_h, k.stride_n, BLK)) return AVSA_ERR_CUDA;
  if (!encode_bf16_tile_map(&tv, v.ptr, B, H, N, D, v.stride_b, v.stride_h, v.stride_n, BLK)) return AVSA_ERR_CUDA;
  if (!encode_bf16_tile_map(&to, o, B, H, N, D, q.stride_b, q.stride_h, q.stride_n, BLK)) return AVSA_ERR_CUDA;
  using LF = FastSmem<BLK, D>;
  if (cudaFuncSetAttribute(attn_fast_kernel<BLK, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           LF::kTotal) != cudaSuccess)
    return AVSA_ERR_CUDA;
  if (cudaFuncSetAttribute(attn_redo_kernel<BLK, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal) !=
      cudaSuccess)
    return AVSA_ERR_CUDA;
  dim3 grid(prm.NQT, H, B);
  // Fast kernel first; it lists the (rare) work items whose rows outgrow its fixed reference maxima, and the
  // exact-rescaling kernel behind it recomputes exactly those.
  const long long items = static_cast<long long>(prm.NQT) * H * B;
  // The persistent form stores rows with 32-byte accesses: it needs 32-byte-aligned rows.
  const bool rows_aligned32 = (reinterpret_cast<uintptr_t>(o) & 31u) == 0 && q.stride_b % 16 == 0 &&
                              q.stride_h % 16 == 0 && q.stride_n % 16 == 0;
  if (rows_aligned32 && items <= 0x7fffffff) {
    using LP = PersistSmem<BLK, D>;
    if (cudaFuncSetAttribute(attn_persist_kernel<BLK, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, LP::kTotal) !=
        cudaSuccess)
      return AVSA_ERR_CUDA;
    const int pgrid = static_cast<int>(items < 148 ? items : 148);
    attn_persist_kernel<BLK, D><<<pgrid, kAttnThreads, LP::kTotal, st>>>(tq, tk, tv, prm, redo, static_cast<int>(items));
  } else {
    attn_fast_kernel<BLK, D><<<grid, kAttnThreads, LF::kTotal, st>>>(tq, tk, tv, to, prm, redo);
  }
  const int redo_grid = static_cast<int>(items < 148 ? items : 148);
  attn_redo_kernel<BLK, D><<<redo_grid, kAttnThreads, L::kTotal, st>>>(tq, tk, tv, to, prm, redo);
  return cudaGetLastError() == cudaSuccess ? AVSA_OK : AVSA_ERR_CUDA;
}

}  // namespace avsa

using namespace avsa;

#ifdef AVSA_TRACE
// Debug builds only: device buffer that receives the pipeline time stamps of CTA (0,0,0).
static long long* g_trace_buffer = nullptr;
extern "C" __attribute__((visibility("default"))) void avsa_debug_set_trace(long long* device_buffer) {
  g_trace_buffer = device_buffer;
}
#endif

extern "C" size_t avsa_sparse_self_attn_workspace_bytes(int B, int H, int N, int d, int blk) {
  if (B <= 0 || H <= 0 || N <= 0 || d <= 0 || blk <= 0) return 0;
  const size_t nb = (static_cast<size_t>(N) + blk - 1) / blk;
  return kStatusBytes + align_up(static_cast<size_t>(B) * H * nb * sizeof(int), 256);   // status + one flag per item
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
  prm.o = static_cast<__nv_bfloat16*>(o_bf16);
  prm.o_sb = q.stride_b;
  prm.o_sh = q.stride_h;
  prm.o_sn = q.stride_n;
  prm.status = static_cast<StatusRecord*>(ws);
  prm.H = H;
  prm.Nq = N;
  prm.Nk = N;
  prm.NQT = prm.NKB = (N + blk - 1) / blk;
  const float scale = softmax_scale != 0.f ? softmax_scale : 1.0f / sqrtf(static_cast<float>(d));
  prm.scale_log2 = scale * 1.4426950408889634f;
#ifdef AVSA_TRACE
  prm.trace = g_trace_buffer;
#endif
  clear_status_kernel<<<1, 1, 0, st>>>(prm.status);
  int* redo = reinterpret_cast<int*>(static_cast<uint8_t*>(ws) + kStatusBytes);
  if (d == 128) return launch_sparse_attn<128, 128>(B, H, N, q, k, v, o_bf16, prm, redo, st);
  return launch_sparse_attn<64, 64>(B, H, N, q, k, v, o_bf16, prm, redo, st);
}
