// Shared host/device plumbing of libavsa: status record, argument checks, tensor-map encoding.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/avsa.h"

namespace avsa {

// First bytes of every workspace.  code == 0 means no device-side check failed.
struct StatusRecord {
  int code;       // avsa_status
  int where;      // which wait / check
  int item;       // work item (block index)
  int aux;        // tile index or offending value
  int redo_count; // sparse attention: work items the fast kernel left to the exact kernel in this call
  int next_item;  // sparse attention: head of the work queue of the persistent kernel
};
constexpr size_t kStatusBytes = 256;   // the record, padded so that what follows stays 256-byte aligned

__device__ __forceinline__ void report_status(StatusRecord* st, int code, int where, int item, int aux) {
  if (atomicCAS(&st->code, 0, code) == 0) {
    st->where = where;
    st->item = item;
    st->aux = aux;
  }
}

// Resets the status record at the start of every call (first node of the call's launch sequence).
static __global__ void clear_status_kernel(StatusRecord* st) {
  st->code = 0;
  st->where = 0;
  st->item = 0;
  st->aux = 0;
  st->redo_count = 0;
  st->next_item = 0;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// A bf16 [B,H,N,d] view is usable when its base is 16-byte aligned and its strides are multiples of
// 8 elements (so every row starts on a 16-byte boundary) and positive.
inline bool tensor_ok(const avsa_bf16_4d& t, int B, int H) {
  if (t.ptr == nullptr || !aligned16(t.ptr)) return false;
  if (t.stride_n <= 0 || (t.stride_n % 8) != 0) return false;
  if (H > 1 && (t.stride_h <= 0 || (t.stride_h % 8) != 0)) return false;
  if (B > 1 && (t.stride_b <= 0 || (t.stride_b % 8) != 0)) return false;
  return true;
}

// Encodes a 4-D tiled tensor map over a bf16 [B,H,N,d] view: dims (d, N, H, B), box (64, box_rows, 1, 1),
// 128-byte swizzle, zero fill out of range.  Returns false when the driver entry point is missing
// or the encode fails.
bool encode_bf16_tile_map(CUtensorMap* map, const void* ptr, int B, int H, int N, int d, int64_t stride_b,
                          int64_t stride_h, int64_t stride_n, int box_rows);

// True when the current device is compute capability 10.x.
bool device_is_sm100();

// Grid size of the persistent kernels: one CTA per SM of the current device, at most one per work item.
int persistent_grid(long long items);

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

}  // namespace avsa
