// avsa_cache_indicators: the synchronization-aware cache-reuse indicators of Eq. 12-15.
//   Eq. 12  dv = |Yv - Yv^|_1 / (|Yv|_1 + eps),  da likewise for the audio stream
//   Eq. 13  dp = the same ratio restricted to the rows of the protected video tokens
//   Eq. 14  ds = 1 - <s, s^> / (|s|_2 |s^|_2 + eps)        (saliency drift)
//   Eq. 15  dsync = max(dv, da, lambda_p dp, lambda_s ds);  reuse iff dsync < tau
// HBM-bound: every feature element is read exactly once.  One warp per token row, 16-byte loads, fp32
// partial sums per CTA written to the workspace and combined in a fixed order (bit-reproducible).
#include "avsa_common.cuh"

namespace avsa {

constexpr int kIndThreads = 256;
constexpr int kIndWarps = kIndThreads / 32;

__device__ __forceinline__ void abs_sums_bf16x8(const uint4& y, const uint4& c, float& diff, float& mag) {
  const uint32_t yw[4] = {y.x, y.y, y.z, y.w}, cw[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
  for (int i = 0; i < 4; i++) {
    const float y0 = __uint_as_float(yw[i] << 16), y1 = __uint_as_float(yw[i] & 0xffff0000u);
    const float c0 = __uint_as_float(cw[i] << 16), c1 = __uint_as_float(cw[i] & 0xffff0000u);
    diff += fabsf(y0 - c0) + fabsf(y1 - c1);
    mag += fabsf(y0) + fabsf(y1);
  }
}

// partial[b][cta][4] = (sum |y - yhat|, sum |y|, the same two over protected rows).  One grid covers both
// streams: CTAs [0, gv) take video rows, CTAs [gv, gv+ga) audio rows (which have no protected set).
__global__ void __launch_bounds__(kIndThreads) l1_partials_kernel(const __nv_bfloat16* __restrict__ y_v,
                                                                  const __nv_bfloat16* __restrict__ yhat_v, int Nv,
                                                                  const __nv_bfloat16* __restrict__ y_a,
                                                                  const __nv_bfloat16* __restrict__ yhat_a, int Na,
                                                                  int C, const uint8_t* __restrict__ prot, int gv, int ga,
                                                                  float* __restrict__ part_v, float* __restrict__ part_a) {
  __shared__ float red[kIndWarps][4];
  const int b = blockIdx.y, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool video = static_cast<int>(blockIdx.x) < gv;
  const int cta = video ? blockIdx.x : blockIdx.x - gv, ncta = video ? gv : ga;
  const int N = video ? Nv : Na;
  const int64_t row_stride = C, batch_stride = static_cast<int64_t>(N) * C;
  const __nv_bfloat16* yb = (video ? y_v : y_a) + b * batch_stride;
  const __nv_bfloat16* cb = (video ? yhat_v : yhat_a) + b * batch_stride;
  const uint8_t* pb = (video && prot != nullptr) ? prot + static_cast<int64_t>(b) * N : nullptr;
  float* partial = video ? part_v : part_a;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int chunks = C / 8;
  float d_all = 0.f, m_all = 0.f, d_p = 0.f, m_p = 0.f;
  for (int row = cta * kIndWarps + warp; row < N; row += ncta * kIndWarps) {
    const uint4* yr = reinterpret_cast<const uint4*>(yb + row * row_stride);
    const uint4* cr = reinterpret_cast<const uint4*>(cb + row * row_stride);
    float d = 0.f, m = 0.f;
    constexpr int UNROLL = 4;      // 8 independent 16-byte loads in flight per lane
    for (int c0 = lane; c0 < chunks; c0 += 32 * UNROLL) {
      uint4 yv[UNROLL], cv[UNROLL];
#pragma unroll
      for (int u = 0; u < UNROLL; u++) {
        const int c = c0 + u * 32;
        yv[u] = make_uint4(0u, 0u, 0u, 0u);
        cv[u] = make_uint4(0u, 0u, 0u, 0u);
        if (c < chunks) {
          yv[u] = __ldg(yr + c);
          cv[u] = __ldg(cr + c);
        }
      }
#pragma unroll
      for (int u = 0; u < UNROLL; u++) abs_sums_bf16x8(yv[u], cv[u], d, m);
    }
    d_all += d;
    m_all += m;
    if (pb != nullptr && pb[row] != 0) {
      d_p += d;
      m_p += m;
    }
  }
  float v[4] = {d_all, m_all, d_p, m_p};
#pragma unroll
  for (int i = 0; i < 4; i++)
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v[i] += __shfl_xor_sync(0xffffffffu, v[i], off);
  if (lane == 0)
    for (int i = 0; i < 4; i++) red[warp][i] = v[i];
  __syncthreads();
  if (threadIdx.x < 4) {
    float s = 0.f;
    for (int w = 0; w < kIndWarps; w++) s += red[w][threadIdx.x];
    partial[(static_cast<int64_t>(b) * ncta + cta) * 4 + threadIdx.x] = s;
  }
}

// One CTA per batch item: fixed-order sums of the partials and of the saliency products, then Eq. 12-15.
constexpr int kFinThreads = 1024;
__global__ void __launch_bounds__(kFinThreads) indicators_finalize_kernel(const float* __restrict__ part_v, int gv,
                                                                  const float* __restrict__ part_a, int ga,
                                                                  const float* __restrict__ s_cur,
                                                                  const float* __restrict__ s_anchor, int N,
                                                                  float lambda_p, float lambda_s, float tau, float eps,
                                                                  float* __restrict__ out, StatusRecord* status) {
  __shared__ float red[kFinThreads][9];
  const int b = blockIdx.x, tid = threadIdx.x;
  asm volatile("griddepcontrol.wait;" ::: "memory");      // the partial sums come from the kernel before
  if (b == 0 && tid == 0) {
    status->code = 0;
    status->where = 0;
    status->item = 0;
    status->aux = 0;
  }
  // nine sums at once, each in a fixed order: thread t takes entries t, t+1024, ...; then a fixed tree
  float acc[9];
#pragma unroll
  for (int i = 0; i < 9; i++) acc[i] = 0.f;
  for (int g = tid; g < gv; g += kFinThreads) {
    const float4 v = *reinterpret_cast<const float4*>(part_v + (static_cast<int64_t>(b) * gv + g) * 4);
    acc[0] += v.x; acc[1] += v.y; acc[2] += v.z; acc[3] += v.w;
  }
  for (int g = tid; g < ga; g += kFinThreads) {
    const float4 v = *reinterpret_cast<const float4*>(part_a + (static_cast<int64_t>(b) * ga + g) * 4);
    acc[4] += v.x; acc[5] += v.y;
  }
  if (s_cur != nullptr && s_anchor != nullptr) {
    const float* sc = s_cur + static_cast<int64_t>(b) * N;
    const float* sa = s_anchor + static_cast<int64_t>(b) * N;
    for (int i0 = tid; i0 < N; i0 += kFinThreads * 8) {
      float a[8], c[8];
#pragma unroll
      for (int u = 0; u < 8; u++) {
        const int i = i0 + u * kFinThreads;
        a[u] = i < N ? __ldg(sc + i) : 0.f;
        c[u] = i < N ? __ldg(sa + i) : 0.f;
      }
#pragma unroll
      for (int u = 0; u < 8; u++) {
        acc[6] = fmaf(a[u], c[u], acc[6]);
        acc[7] = fmaf(a[u], a[u], acc[7]);
        acc[8] = fmaf(c[u], c[u], acc[8]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 9; i++) red[tid][i] = acc[i];
  __syncthreads();
  for (int off = kFinThreads / 2; off > 0; off >>= 1) {
    if (tid < off)
#pragma unroll
      for (int i = 0; i < 9; i++) red[tid][i] += red[tid + off][i];
    __syncthreads();
  }
  const float* sums = red[0];
  if (tid == 0) {
    const float dv = sums[0] / (sums[1] + eps);
    const float dp = sums[2] / (sums[3] + eps);
    const float da = sums[4] / (sums[5] + eps);
    const float ds = (s_cur != nullptr && s_anchor != nullptr)
                         ? 1.0f - sums[6] / (sqrtf(sums[7]) * sqrtf(sums[8]) + eps) : 0.0f;
    const float dsync = fmaxf(fmaxf(dv, da), fmaxf(lambda_p * dp, lambda_s * ds));
    float* o = out + static_cast<int64_t>(b) * 8;
    o[0] = dv; o[1] = da; o[2] = dp; o[3] = ds; o[4] = dsync; o[5] = dsync < tau ? 1.0f : 0.0f; o[6] = 0.f; o[7] = 0.f;
  }
}

struct IndPlan {
  int gv, ga;
  size_t off_v, off_a, total;
};
static IndPlan make_ind_plan(int B, int Nv, int Na) {
  IndPlan p;
  const int cap = 148 * 8;     // eight CTAs of 256 threads per SM keep enough 16-byte loads in flight
  p.gv = (Nv + kIndWarps - 1) / kIndWarps; if (p.gv > cap) p.gv = cap; if (p.gv < 1) p.gv = 1;
  p.ga = (Na + kIndWarps - 1) / kIndWarps; if (p.ga > cap) p.ga = cap; if (p.ga < 1) p.ga = 1;
  size_t off = kStatusBytes;
  p.off_v = off; off += align_up(static_cast<size_t>(B) * p.gv * 4 * sizeof(float), 256);
  p.off_a = off; off += align_up(static_cast<size_t>(B) * p.ga * 4 * sizeof(float), 256);
  p.total = off;
  return p;
}

}  // namespace avsa

using namespace avsa;

extern "C" size_t avsa_cache_indicators_workspace_bytes(int B, int Nv, int Na, int C) {
  if (B <= 0 || Nv <= 0 || Na <= 0 || C <= 0) return 0;
  return make_ind_plan(B, Nv, Na).total;
}

extern "C" int avsa_cache_indicators(int B, int Nv, int Na, int C, const void* y_v, const void* yhat_v, const void* y_a,
                                     const void* yhat_a, const uint8_t* prot_tok, const float* s_cur,
                                     const float* s_anchor, float lambda_p, float lambda_s, float tau, float eps,
                                     float* out, void* ws, size_t ws_bytes, void* stream) {
  if (B <= 0 || Nv <= 0 || Na <= 0 || C <= 0 || (C % 8) != 0) return AVSA_ERR_INVALID_ARG;
  if (y_v == nullptr || yhat_v == nullptr || y_a == nullptr || yhat_a == nullptr || out == nullptr)
    return AVSA_ERR_INVALID_ARG;
  if (!aligned16(y_v) || !aligned16(yhat_v) || !aligned16(y_a) || !aligned16(yhat_a)) return AVSA_ERR_INVALID_ARG;
  if ((s_cur == nullptr) != (s_anchor == nullptr)) return AVSA_ERR_INVALID_ARG;
  if (B > 65535) return AVSA_ERR_UNSUPPORTED;
  const IndPlan p = make_ind_plan(B, Nv, Na);
  if (ws == nullptr || ws_bytes < p.total) return AVSA_ERR_WORKSPACE;
  cudaStream_t st = as_stream(stream);
  uint8_t* base = static_cast<uint8_t*>(ws);
  float* pv = reinterpret_cast<float*>(base + p.off_v);
  float* pa = reinterpret_cast<float*>(base + p.off_a);
  l1_partials_kernel<<<dim3(p.gv + p.ga, B), kIndThreads, 0, st>>>(
      static_cast<const __nv_bfloat16*>(y_v), static_cast<const __nv_bfloat16*>(yhat_v), Nv,
      static_cast<const __nv_bfloat16*>(y_a), static_cast<const __nv_bfloat16*>(yhat_a), Na, C, prot_tok, p.gv, p.ga, pv,
      pa);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(B, 1, 1);
  cfg.blockDim = dim3(kFinThreads, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const float* pvc = pv;
  const float* pac = pa;
  if (cudaLaunchKernelEx(&cfg, indicators_finalize_kernel, pvc, p.gv, pac, p.ga, s_cur, s_anchor, Nv, lambda_p,
                         lambda_s, tau, eps, out, static_cast<StatusRecord*>(ws)) != cudaSuccess)
    return AVSA_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? AVSA_OK : AVSA_ERR_CUDA;
}
