// Per-process and per-device state of the library, and the tensor maps every launch needs.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/b200gemm.h"
#include "gemm_kernel.cuh"

namespace b200gemm {
namespace {

constexpr int MAX_DEVICES = 64;
constexpr int K_LIMIT_INT = 131071;  // 128*128*K and 16384*K stay below 2^31

__device__ int g_device_status = 0;

constexpr int TRACE_MAX_CTAS = 160;
__device__ unsigned long long g_trace[TRACE_MAX_CTAS * TRACE_SLOTS];

struct DeviceState {
  bool ready = false;
  int num_sms = 0;
  int* status_ptr = nullptr;
  unsigned long long* trace_ptr = nullptr;
  void* s4_workspace = nullptr;
  size_t s4_workspace_bytes = 0;
  uint64_t attr_set[3] = {0, 0, 0};  // bit i: dynamic-smem attribute set for kernel variant i
  // clusters of four CTAs (cluster split-K) the device runs at once, per kind and output
  // mode; 0 = not asked yet
  int quad_clusters[2][4] = {};
};

std::mutex g_mutex;
DeviceState g_dev[MAX_DEVICES];
int g_last_cuda_error = 0;
int g_override_bn = 0;
int g_override_group_m = 0;
int g_override_cta_group = 0;
int g_override_splits = 0;
int g_trace_on = 0;
int g_s4_scheme = 0;   // INT4 route: 0 = automatic, 1 = always the pre-pass, 2 = fused wherever built
int g_swap_ab = 0;     // 0 = automatic, 1 = never, 2 = always exchange A and B inside the library
int g_l2_policy = 11;  // keep A, B normal, serpentine K, C stores evict-first

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                   const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

int cuda_fail(cudaError_t e) {
  g_last_cuda_error = static_cast<int>(e);
  return GEMM_ERR_CUDA;
}

// Looks up (once per device) what every launch needs.  Call with the mutex held.
int device_state(DeviceState** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= MAX_DEVICES) return GEMM_ERR_UNSUPPORTED_DEVICE;
  DeviceState& s = g_dev[dev];
  if (!s.ready) {
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (major != 10) return GEMM_ERR_UNSUPPORTED_DEVICE;
    e = cudaDeviceGetAttribute(&s.num_sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&s.status_ptr), g_device_status);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&s.trace_ptr), g_trace);
    if (e != cudaSuccess) return cuda_fail(e);
    if (!g_encode) {
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult q;
      e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
      if (e != cudaSuccess) return cuda_fail(e);
      if (!fn || q != cudaDriverEntryPointSuccess) return cuda_fail(cudaErrorNotSupported);
      g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    s.ready = true;
  }
  *out = &s;
  return GEMM_OK;
}

// Row-major 2-D tensor of `rows` x `cols` elements, pitch in bytes; the box is
// box_rows rows of 128 bytes, written to shared memory with the 128-byte swizzle.
int encode_operand_map(CUtensorMap* map, CUtensorMapDataType type, int elem_bytes, const void* ptr,
                       uint64_t rows, uint64_t cols, uint64_t pitch_bytes, uint32_t box_rows,
                       bool promote_256 = true) {
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {pitch_bytes};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(BK_BYTES / elem_bytes), box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(map, type, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        promote_256 ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B
                                    : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    g_last_cuda_error = static_cast<int>(cudaErrorInvalidValue);
    return GEMM_ERR_CUDA;
  }
  return GEMM_OK;
}

// C (row-major, 32- or 16-bit elements) for the epilogue's TMA stores: boxes of 32 rows x
// 128 bytes, 128-byte swizzle.  Needs a 16-byte aligned base and pitch.
int encode_c_map(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ldc,
                 int elem_bytes,
                 CUtensorMapDataType reduce_type = CU_TENSOR_MAP_DATA_TYPE_UINT32) {
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ldc * static_cast<uint64_t>(elem_bytes)};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(128 / elem_bytes), 32};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(map, elem_bytes == 4 ? reduce_type : CU_TENSOR_MAP_DATA_TYPE_UINT16,
                        2, const_cast<void*>(ptr), dims,
                        strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    g_last_cuda_error = static_cast<int>(cudaErrorInvalidValue);
    return GEMM_ERR_CUDA;
  }
  return GEMM_OK;
}
}  // namespace
}  // namespace b200gemm
