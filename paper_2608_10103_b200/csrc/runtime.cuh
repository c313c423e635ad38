// Per-process and per-device state of the library, the tensor maps every launch needs and the
// scratch buffers of the INT4 pre-pass.
//
// Threads: the entry points may be called from several host threads.  The hot path takes no
// lock: per-device facts are published once (double-checked under g_mutex), tensor maps are
// cached per thread, the measurement switches are atomics that are read once per call (set
// them while no call is in flight), and scratch buffers are leased per stream from a pool with
// a lock of its own.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <atomic>
#include <mutex>

#include "../../include/b200gemm.h"
#include "../../include/b200gemm_debug.h"
#include "gemm_kernel.cuh"
#include "workspace_pool.h"

namespace b200gemm {
namespace {

constexpr int MAX_DEVICES = 64;
constexpr int K_LIMIT_INT = 131071;  // 128*128*K and 16384*K stay below 2^31

__device__ int g_device_status = 0;

constexpr int TRACE_MAX_CTAS = 160;
__device__ unsigned long long g_trace[TRACE_MAX_CTAS * TRACE_SLOTS];

struct DeviceState {
  std::atomic<bool> ready{false};
  int num_sms = 0;
  int* status_ptr = nullptr;
  unsigned long long* trace_ptr = nullptr;
  // bit i: dynamic-smem attribute set for kernel variant i (setting it twice is harmless)
  std::atomic<uint64_t> attr_set[5] = {};
  // clusters of four CTAs (cluster split-K) the device runs at once, per kind and output
  // mode; 0 = not asked yet
  std::atomic<int> quad_clusters[2][4] = {};
};

std::mutex g_mutex;  // first-use initialisation only
DeviceState g_dev[MAX_DEVICES];
std::atomic<int> g_last_cuda_error{0};
std::atomic<int> g_override_bn{0};
std::atomic<int> g_override_group_m{0};
std::atomic<int> g_override_cta_group{0};
std::atomic<int> g_override_splits{0};
std::atomic<int> g_override_stages{0};  // ring depth of the 256 x 256 pair tile (ablation)
std::atomic<int> g_trace_on{0};
// INT4 route: 0 = automatic, 1 = always the pre-pass, 2 = fused wherever built, 4 = the pre-pass,
// done inside the INT8 GEMM kernel ahead of its tiles where that variant applies (3 = 1)
std::atomic<int> g_s4_scheme{0};
bool s4_prepass_forced() { const int v = g_s4_scheme; return v == 1 || v == 3 || v == 4; }
bool s4_fused_forced() { const int v = g_s4_scheme; return v == 2 || v == 5 || v == 6; }
std::atomic<int> g_swap_ab{0};     // 0 = automatic, 1 = never, 2 = always exchange A and B inside the library
std::atomic<int> g_family{0};      // kernel for large problems: 0 = automatic, 1 = 256 x 256 pair tile, 2 = 512 x 256
std::atomic<int> g_l2_policy{11};  // keep A, B normal, serpentine K, C stores evict-first

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                   const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
std::atomic<EncodeTiledFn> g_encode{nullptr};

int cuda_fail(cudaError_t e) {
  g_last_cuda_error = static_cast<int>(e);
  return GEMM_ERR_CUDA;
}

// What every launch needs to know about the current device, looked up once per device.
int device_state(DeviceState** out, int* device = nullptr) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= MAX_DEVICES) return GEMM_ERR_UNSUPPORTED_DEVICE;
  DeviceState& s = g_dev[dev];
  if (!s.ready.load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!s.ready.load(std::memory_order_relaxed)) {
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
      if (!g_encode.load()) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
        if (e != cudaSuccess) return cuda_fail(e);
        if (!fn || q != cudaDriverEntryPointSuccess) return cuda_fail(cudaErrorNotSupported);
        g_encode.store(reinterpret_cast<EncodeTiledFn>(fn));
      }
      s.ready.store(true, std::memory_order_release);
    }
  }
  *out = &s;
  if (device) *device = dev;
  return GEMM_OK;
}

// SM count of the current device if the library has seen it, else of a B200.
int known_sm_count() {
  int dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < MAX_DEVICES &&
      g_dev[dev].ready.load(std::memory_order_acquire))
    return g_dev[dev].num_sms;
  (void)cudaGetLastError();
  int n = 0;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
    return n;
  (void)cudaGetLastError();
  return 148;
}

// ------------------------------------------------------------------ tensor maps
// A tensor map is a pure function of (base, extents, pitch, box, type, flavour), and encoding
// one costs more host time than the rest of a call, so each thread keeps the last few it built.
struct MapKey {
  const void* ptr;
  uint64_t rows, cols, pitch;
  uint32_t box_rows;
  uint32_t flavour;  // operand / C, element type, L2 promotion
  bool operator==(const MapKey& o) const {
    return ptr == o.ptr && rows == o.rows && cols == o.cols && pitch == o.pitch &&
           box_rows == o.box_rows && flavour == o.flavour;
  }
};

struct MapCache {
  static constexpr int SLOTS = 32;
  MapKey key[SLOTS];
  CUtensorMap map[SLOTS];
  int used = 0;
  int next = 0;
  const CUtensorMap* find(const MapKey& k) const {
    for (int i = 0; i < used; ++i)
      if (key[i] == k) return &map[i];
    return nullptr;
  }
  void insert(const MapKey& k, const CUtensorMap& m) {
    const int i = used < SLOTS ? used++ : next;
    if (i == next) next = (next + 1) % SLOTS;
    key[i] = k;
    map[i] = m;
  }
};
thread_local MapCache t_maps;
std::atomic<long long> g_map_encodes{0};  // how many maps were really encoded (for tests)

int encode_cached(CUtensorMap* map, const MapKey& k, CUtensorMapDataType type,
                  const cuuint32_t* box, CUtensorMapL2promotion promo) {
  if (const CUtensorMap* hit = t_maps.find(k)) {
    *map = *hit;
    return GEMM_OK;
  }
  cuuint64_t dims[2] = {k.cols, k.rows};
  cuuint64_t strides[1] = {k.pitch};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode.load()(map, type, 2, const_cast<void*>(k.ptr), dims, strides, box, estr,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, promo,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    g_last_cuda_error = static_cast<int>(cudaErrorInvalidValue);
    return GEMM_ERR_CUDA;
  }
  g_map_encodes.fetch_add(1, std::memory_order_relaxed);
  t_maps.insert(k, *map);
  return GEMM_OK;
}

// Row-major 2-D tensor of `rows` x `cols` elements, pitch in bytes; the box is
// box_rows rows of 128 bytes, written to shared memory with the 128-byte swizzle.
int encode_operand_map(CUtensorMap* map, CUtensorMapDataType type, int elem_bytes, const void* ptr,
                       uint64_t rows, uint64_t cols, uint64_t pitch_bytes, uint32_t box_rows,
                       bool promote_256 = true) {
  const MapKey k{ptr, rows, cols, pitch_bytes, box_rows,
                 static_cast<uint32_t>(type) | (promote_256 ? 0x100u : 0u)};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(BK_BYTES / elem_bytes), box_rows};
  return encode_cached(map, k, type, box,
                       promote_256 ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B
                                   : CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
}

// C (row-major, 32- or 16-bit elements) for the epilogue's TMA stores: boxes of 32 rows x
// 128 bytes, 128-byte swizzle.  Needs a 16-byte aligned base and pitch.
int encode_c_map(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ldc,
                 int elem_bytes,
                 CUtensorMapDataType reduce_type = CU_TENSOR_MAP_DATA_TYPE_UINT32) {
  const CUtensorMapDataType type = elem_bytes == 4 ? reduce_type : CU_TENSOR_MAP_DATA_TYPE_UINT16;
  const MapKey k{ptr, rows, cols, ldc * static_cast<uint64_t>(elem_bytes), 32,
                 static_cast<uint32_t>(type) | 0x200u};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(128 / elem_bytes), 32};
  return encode_cached(map, k, type, box, CU_TENSOR_MAP_L2_PROMOTION_NONE);
}

// ------------------------------------------------------------------ scratch buffers
struct CudaPoolBackend {
  using Stream = cudaStream_t;
  using Event = cudaEvent_t;
  int alloc(void** p, size_t bytes, Stream s) { return cudaMallocAsync(p, bytes, s); }
  int free_after(void* p, Stream s) { return cudaFreeAsync(p, s); }
  int free_now(void* p) { return cudaFree(p); }
  int event_create(Event* e) { return cudaEventCreateWithFlags(e, cudaEventDisableTiming); }
  void event_destroy(Event e) { cudaEventDestroy(e); }
  int event_record(Event e, Stream s) { return cudaEventRecord(e, s); }
  bool event_done(Event e) {
    if (cudaEventQuery(e) == cudaSuccess) return true;
    (void)cudaGetLastError();  // "not ready" is an answer, not an error to keep
    return false;
  }
  bool capturing(Stream s) {
    cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(s, &st) != cudaSuccess) {
      (void)cudaGetLastError();
      return false;
    }
    return st != cudaStreamCaptureStatusNone;
  }
  int clear(void* p, size_t bytes, Stream s) { return cudaMemsetAsync(p, 0, bytes, s); }
};
using ScratchPool = WorkspacePool<CudaPoolBackend>;
ScratchPool g_pool[MAX_DEVICES];

int pool_fail(int rc) {
  if (rc == ScratchPool::kNoAllocInCapture) return cuda_fail(cudaErrorStreamCaptureUnsupported);
  return cuda_fail(static_cast<cudaError_t>(rc));
}
}  // namespace
}  // namespace b200gemm
