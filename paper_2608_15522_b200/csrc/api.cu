// Library-level entry points that are not tied to one subsystem, and the tensor-map encoder.
#include <mutex>

#include "avsa_common.cuh"

namespace avsa {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess) {
      fn = reinterpret_cast<EncodeTiledFn>(p);
    }
  });
  return fn;
}

bool encode_bf16_tile_map(CUtensorMap* map, const void* ptr, int B, int H, int N, int d, int64_t stride_b,
                          int64_t stride_h, int64_t stride_n, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  // A dimension of extent 1 never has its stride used for addressing, but the encoder still wants a
  // multiple of 16 bytes; give it a harmless one.
  const int64_t sn = stride_n;
  const int64_t sh = (H > 1) ? stride_h : sn * N;
  const int64_t sb = (B > 1) ? stride_b : sh * (H > 1 ? H : 1);
  cuuint64_t dims[4] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(H),
                        static_cast<cuuint64_t>(B)};
  cuuint64_t strides[3] = {static_cast<cuuint64_t>(sn) * 2u, static_cast<cuuint64_t>(sh) * 2u,
                           static_cast<cuuint64_t>(sb) * 2u};
  cuuint32_t box[4] = {64u, static_cast<cuuint32_t>(box_rows), 1u, 1u};
  cuuint32_t elem[4] = {1u, 1u, 1u, 1u};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, elem,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool device_is_sm100() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return false;
  return major == 10;
}

// Grid size of the persistent kernels: one CTA per SM of the current device, at most one per work item.
int persistent_grid(long long items) {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
    sms = 148;
  return static_cast<int>(items < sms ? items : sms);
}

}  // namespace avsa

extern "C" {

int avsa_count_from_percent(int pct, int n) {
  if (pct <= 0 || n <= 0) return 0;
  return static_cast<int>((static_cast<long long>(pct) * n + 99) / 100);
}

int avsa_read_status(const void* ws, void* stream, int* detail) {
  if (ws == nullptr) return AVSA_ERR_INVALID_ARG;
  avsa::StatusRecord rec;
  if (cudaStreamSynchronize(avsa::as_stream(stream)) != cudaSuccess) return AVSA_ERR_CUDA;
  if (cudaMemcpy(&rec, ws, sizeof(rec), cudaMemcpyDeviceToHost) != cudaSuccess) return AVSA_ERR_CUDA;
  if (detail != nullptr) {
    detail[0] = rec.where;
    detail[1] = rec.item;
    detail[2] = rec.aux;
  }
  return rec.code;
}

const char* avsa_status_string(int status) {
  switch (status) {
    case AVSA_OK: return "ok";
    case AVSA_ERR_INVALID_ARG: return "invalid argument";
    case AVSA_ERR_UNSUPPORTED: return "unsupported shape or device";
    case AVSA_ERR_WORKSPACE: return "workspace missing or too small";
    case AVSA_ERR_CUDA: return "CUDA call failed";
    case AVSA_ERR_TIMEOUT: return "device-side wait timed out";
    case AVSA_ERR_BAD_MASK: return "malformed column list";
    default: return "unknown status";
  }
}

int avsa_version(void) { return 100; }

}  // extern "C"
