// C-ABI of the library: argument validation, tile selection, tensor-map
// encoding and kernel launch.  See include/b200gemm.h for the contract.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <mutex>

#include "../../include/b200gemm.h"
#include "gemm_kernel.cuh"
#include "peak_probe.cuh"
#include "unpack_s4.cuh"

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
  uint64_t attr_set[2] = {0, 0};  // bit i: dynamic-smem attribute set for kernel variant i
};

std::mutex g_mutex;
DeviceState g_dev[MAX_DEVICES];
int g_last_cuda_error = 0;
int g_override_bn = 0;
int g_override_group_m = 0;
int g_override_cta_group = 0;
int g_override_splits = 0;
int g_trace_on = 0;
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

// ------------------------------------------------------------------ selector
struct TileConfig {
  int bn;
  int cta_group;  // 1: one CTA per 128 x bn tile; 2: a CTA pair per 256 x bn tile
  int stages;
  int group_m;
  int splits;     // split-K factor (1 = off)
};

constexpr int kWidths[] = {256, 128, 64, 32};

// Ring depth and 128-byte K atoms per slot of each built shape.
int stages_for(int bn, int cta_group) {
  if (cta_group == 2) return bn == 256 ? 6 : 4;
  switch (bn) {
    case 256: return 4;
    case 128: return 3;
    default: return 4;
  }
}

// 256-wide tiles are bound by the tensor pipe and want many small slots; narrower tiles are
// bound by the issuing thread and get two K atoms per slot (one wait + one commit per 8 MMAs).
int atoms_for(int bn, int) { return bn == 256 ? 1 : 2; }

bool variant_exists(int bn, int cta_group) {
  if (cta_group == 1) return bn == 256 || bn == 128 || bn == 64 || bn == 32;
  if (cta_group == 2) return bn == 256 || bn == 128 || bn == 64;
  return false;
}

int ceil_div(long long a, long long b) { return static_cast<int>((a + b - 1) / b); }

// Picks the C-tile shape and the split-K factor.  The paper fixes one tiling for all
// sizes (Sec. III-A) and lists non-square shapes as future work (Sec. VI); on 148 SMs small
// problems need more work units than they have tiles, and large ones want the CTA-pair
// tile, which halves the B bytes each SM pulls from L2.
// Cost model, in SM cycles, fitted to the cycle accounting of the kernel: a k-block (128
// bytes of K) costs the slowest of the tensor pipe (2*bn: a 128-row MMA of width bn occupies
// it bn/2 cycles, 4 per k-block), the issuing thread (~450) and the SM's L2 port
// ((128 + bn/cta_group) rows x 128 bytes at ~66 bytes/cycle); units run in waves over the SMs
// (or SM pairs); the last epilogue (~16 cycles per column), set-up (~3000) and a pair's
// cluster launch (~2500) are paid once; split-K adds zeroing C and adding into it.
TileConfig select_config(int M, int N, int num_sms, int k_blocks, int min_bn = 32,
                         bool allow_split = false) {
  TileConfig best{256, 2, 6, 8, 1};
  long long best_cost = -1;
  for (int cg = 2; cg >= 1; --cg) {
    if (g_override_cta_group && cg != g_override_cta_group) continue;
    for (int bn : kWidths) {
      if (g_override_bn && bn != g_override_bn) continue;
      if (!variant_exists(bn, cg) || bn < min_bn) continue;
      const long long tiles = static_cast<long long>(ceil_div(M, BM * cg)) * ceil_div(N, bn);
      const long long units = num_sms / cg;
      const int atoms = atoms_for(bn, cg);
      const int slots = ceil_div(k_blocks, atoms);  // K is split in whole ring slots
      int max_split = 1;
      if (allow_split) {
        max_split = static_cast<int>(units / tiles);
        if (max_split > k_blocks / 2) max_split = k_blocks / 2;  // at least 2 k-blocks each
        if (max_split > 32) max_split = 32;
        if (max_split < 1) max_split = 1;
      }
      if (g_override_splits) {
        // forced: the largest factor <= the request that leaves no K range empty
        max_split = g_override_splits < slots ? g_override_splits : slots;
        while (max_split > 1 &&
               static_cast<long long>(max_split - 1) * ceil_div(slots, max_split) >= slots)
          --max_split;
        if (!allow_split) max_split = 1;
      }
      if (max_split > slots) max_split = slots;
      for (int sp = g_override_splits ? max_split : 1; sp <= max_split; ++sp) {
        if (static_cast<long long>(sp - 1) * ceil_div(slots, sp) >= slots) continue;  // empty range
        const int per = ceil_div(slots, sp) * atoms;  // k-blocks per unit
        const long long waves = (tiles * sp + units - 1) / units;
        long long per_kb = 2 * bn;
        if (per_kb < 450) per_kb = 450;
        const long long port = (128 + bn / cg) * 128 / 66;
        if (per_kb < port) per_kb = port;
        long long cost = waves * per * per_kb + 3000 + 16 * bn + (cg == 2 ? 2500 : 0);
        if (sp > 1) cost += 6000 + static_cast<long long>(M) * N / 250;  // zeroing C + adding into it
        if (best_cost < 0 || cost < best_cost) {
          best_cost = cost;
          best.bn = bn;
          best.cta_group = cg;
          best.splits = sp;
        }
      }
    }
  }
  if (best_cost < 0) {  // the override names a shape this output mode does not have
    best.bn = 0;
    return best;
  }
  best.stages = stages_for(best.bn, best.cta_group);
  // Band height: one wave of tiles about twice as tall as wide in operand bytes (measured
  // DRAM traffic at N = 8192 is lowest there: the A band is what later waves re-read).
  int rows_per_tile = BM * best.cta_group;
  int units = num_sms / best.cta_group;
  int g = 1;
  while ((g + 1) * (g + 1) * rows_per_tile <= 2 * units * best.bn) ++g;
  if (g_override_group_m) g = g_override_group_m;
  int tiles_m = ceil_div(M, rows_per_tile);
  if (g > tiles_m) g = tiles_m;
  if (g < 1) g = 1;
  best.group_m = g;
  return best;
}

template <int KIND, int BN, int STAGES, int CTA_GROUP, int KB, int EPI>
int launch_variant(DeviceState* s, int variant, const CUtensorMap& ta, const CUtensorMap& tb,
                   const CUtensorMap& tc, const GemmParams& p, cudaStream_t stream) {
  using L = SmemLayout<BN, STAGES, CTA_GROUP, KB>;
  auto kernel = gemm_kernel<KIND, BN, STAGES, CTA_GROUP, KB, EPI>;
  if (!(s->attr_set[variant >> 6] & (1ull << (variant & 63)))) {
    cudaError_t e =
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L::DYN_BYTES);
    if (e != cudaSuccess) return cuda_fail(e);
    s->attr_set[variant >> 6] |= 1ull << (variant & 63);
  }
  const long long tiles = static_cast<long long>(p.tiles_m) * p.tiles_n * p.splits;
  const long long units = s->num_sms / CTA_GROUP;
  const int grid = static_cast<int>((tiles < units ? tiles : units) * CTA_GROUP);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(NUM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = L::DYN_BYTES;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CTA_GROUP;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, ta, tb, tc, p);
  if (e != cudaSuccess) return cuda_fail(e);
  return GEMM_OK;
}

// Output options of one GEMM call.
struct OutputSpec {
  int epi = EPI_RAW32;
  const float* row_scale = nullptr;
  const float* col_scale = nullptr;
  long long ldc = 0;        // row pitch of C in elements; 0 = dense (N)
  bool no_split = false;    // C is a block of a larger matrix: never zero / add into it
};

// A, B already in the element type of KIND (fp16 or int8), pitches in bytes.
template <int KIND, int EPI>
int launch_gemm_epi(int M, int N, int K, const void* A, size_t a_pitch, const void* B,
                    size_t b_pitch, void* C, const OutputSpec& out, cudaStream_t stream) {
  std::lock_guard<std::mutex> lock(g_mutex);
  DeviceState* s = nullptr;
  int rc = device_state(&s);
  if (rc != GEMM_OK) return rc;
  constexpr int ELEM = (KIND == ptx::KIND_F16) ? 2 : 1;
  constexpr int C_ELEM = (EPI == EPI_OUT16) ? 2 : 4;
  const CUtensorMapDataType type =
      (KIND == ptx::KIND_F16) ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8;
  const int k_blocks = ceil_div(static_cast<long long>(K) * ELEM, BK_BYTES);
  const TileConfig cfg = select_config(M, N, s->num_sms, k_blocks, EPI == EPI_OUT16 ? 64 : 32,
                                       EPI == EPI_RAW32 && !out.no_split);
  const long long ldc = out.ldc ? out.ldc : N;
  if (cfg.bn == 0) return GEMM_ERR_INVALID_ARG;  // override asks for a shape this mode lacks

  CUtensorMap ta, tb;
  const bool promote = !(g_l2_policy & 16);
  rc = encode_operand_map(&ta, type, ELEM, A, M, K, a_pitch, BM, promote);
  if (rc != GEMM_OK) return rc;
  rc = encode_operand_map(&tb, type, ELEM, B, N, K, b_pitch, cfg.bn / cfg.cta_group, promote);
  if (rc != GEMM_OK) return rc;

  GemmParams p;
  p.M = M;
  p.N = N;
  p.K = K;
  p.tiles_m = ceil_div(M, BM * cfg.cta_group);
  p.tiles_n = ceil_div(N, cfg.bn);
  p.group_m = cfg.group_m;
  p.k_blocks = k_blocks;
  p.splits = cfg.splits;
  p.ldc = ldc;
  p.c_vec_ok = (ldc % (16 / C_ELEM) == 0) && (reinterpret_cast<uintptr_t>(C) % 16 == 0);
  CUtensorMap tc;
  if (p.c_vec_ok) {
    // split-K adds into C by TMA reduction, which takes the element type from the map
    rc = encode_c_map(&tc, C, M, N, ldc, C_ELEM,
                      cfg.splits == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT32
                      : KIND == ptx::KIND_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                              : CU_TENSOR_MAP_DATA_TYPE_INT32);
    if (rc != GEMM_OK) return rc;
  } else {
    tc = ta;  // unused by the kernel on the plain-store path
  }
  p.C = static_cast<uint32_t*>(C);
  p.row_scale = out.row_scale;
  p.col_scale = out.col_scale;
  p.status = s->status_ptr;
  p.trace = (g_trace_on & 1) ? s->trace_ptr : nullptr;
  p.ablate = (g_trace_on >> 1) & 15;
  p.l2_policy = g_l2_policy & 3;
  p.serpentine_k = (g_l2_policy & 4) ? 0 : 1;
  p.c_evict_first = (g_l2_policy & 8) ? 1 : 0;

  if (cfg.splits > 1) {  // only with a dense C (no_split is set for blocks of a larger matrix)
    cudaError_t e = cudaMemsetAsync(C, 0, static_cast<size_t>(M) * N * C_ELEM, stream);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  const int vbase = ((KIND == ptx::KIND_F16) ? 0 : 32) + EPI * 8;  // bit index in attr_set
  if (cfg.cta_group == 2) {
    switch (cfg.bn) {
      case 256: return launch_variant<KIND, 256, 6, 2, 1, EPI>(s, vbase + 4, ta, tb, tc, p, stream);
      case 128: return launch_variant<KIND, 128, 4, 2, 2, EPI>(s, vbase + 5, ta, tb, tc, p, stream);
      case 64: return launch_variant<KIND, 64, 4, 2, 2, EPI>(s, vbase + 6, ta, tb, tc, p, stream);
      default: return GEMM_ERR_INVALID_ARG;
    }
  }
  switch (cfg.bn) {
    case 256: return launch_variant<KIND, 256, 4, 1, 1, EPI>(s, vbase + 0, ta, tb, tc, p, stream);
    case 128: return launch_variant<KIND, 128, 3, 1, 2, EPI>(s, vbase + 1, ta, tb, tc, p, stream);
    case 64: return launch_variant<KIND, 64, 4, 1, 2, EPI>(s, vbase + 2, ta, tb, tc, p, stream);
    case 32:
      if constexpr (EPI != EPI_OUT16)
        return launch_variant<KIND, 32, 4, 1, 2, EPI>(s, vbase + 3, ta, tb, tc, p, stream);
      return GEMM_ERR_INVALID_ARG;
    default: return GEMM_ERR_INVALID_ARG;
  }
}

template <int KIND>
int launch_gemm(int M, int N, int K, const void* A, size_t a_pitch, const void* B, size_t b_pitch,
                void* C, cudaStream_t stream, const OutputSpec& out = OutputSpec()) {
  switch (out.epi) {
    case EPI_RAW32:
      return launch_gemm_epi<KIND, EPI_RAW32>(M, N, K, A, a_pitch, B, b_pitch, C, out, stream);
    case EPI_OUT16:
      return launch_gemm_epi<KIND, EPI_OUT16>(M, N, K, A, a_pitch, B, b_pitch, C, out, stream);
    case EPI_F32_SCALED:
      if constexpr (KIND == ptx::KIND_I8)
        return launch_gemm_epi<KIND, EPI_F32_SCALED>(M, N, K, A, a_pitch, B, b_pitch, C, out,
                                                     stream);
      return GEMM_ERR_INVALID_ARG;
    default: return GEMM_ERR_INVALID_ARG;
  }
}

int check_common(int M, int N, int K, const void* A, const void* B, const void* C) {
  if (M <= 0 || N <= 0 || K <= 0 || !A || !B || !C) return GEMM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(B) |
       reinterpret_cast<uintptr_t>(C)) & 15)
    return GEMM_ERR_MISALIGNED;
  return GEMM_OK;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Unpacks one or two packed matrices (rows_b may be 0) with the same K and output pitch.
int launch_unpack(long long rows_a, const uint8_t* packed_a, int8_t* out_a, long long rows_b,
                  const uint8_t* packed_b, int8_t* out_b, int K, size_t out_pitch,
                  cudaStream_t stream) {
  UnpackJob a{reinterpret_cast<const uint4*>(packed_a), out_a, rows_a * (K / 32)};
  UnpackJob b{reinterpret_cast<const uint4*>(packed_b), out_b, rows_b * (K / 32)};
  const long long chunks = a.chunks + b.chunks;
  long long blocks = (chunks + 255) / 256;
  if (blocks > 148 * 32) blocks = 148 * 32;
  if (blocks < 1) blocks = 1;
  unpack_s4_kernel<<<static_cast<int>(blocks), 256, 0, stream>>>(
      a, b, K / 32, static_cast<long long>(out_pitch));
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  return GEMM_OK;
}

int check_s4(int M, int N, int K, const void* A, const void* B, const void* C) {
  int rc = check_common(M, N, K, A, B, C);
  if (rc != GEMM_OK) return rc;
  if (K % 32) return GEMM_ERR_MISALIGNED;
  if (K > K_LIMIT_INT) return GEMM_ERR_K_TOO_LARGE;
  return GEMM_OK;
}

size_t s4_workspace_need(int M, int N, int K) {
  return align_up(static_cast<size_t>(M) * K, 256) + align_up(static_cast<size_t>(N) * K, 256);
}

// INT4 GEMM through caller-visible scratch: unpack A and B to int8, then the INT8 kernel.
int s4_with_workspace(int M, int N, int K, const uint8_t* A, const uint8_t* B, void* C,
                      void* workspace, size_t workspace_bytes, const OutputSpec& out,
                      cudaStream_t st) {
  if (!workspace) return GEMM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < s4_workspace_need(M, N, K))
    return GEMM_ERR_WORKSPACE;
  int8_t* a8 = static_cast<int8_t*>(workspace);
  int8_t* b8 = a8 + align_up(static_cast<size_t>(M) * K, 256);
  int rc;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState* s = nullptr;
    rc = device_state(&s);
    if (rc != GEMM_OK) return rc;
  }
  rc = launch_unpack(M, A, a8, N, B, b8, K, static_cast<size_t>(K), st);
  if (rc != GEMM_OK) return rc;
  return launch_gemm<ptx::KIND_I8>(M, N, K, a8, static_cast<size_t>(K), b8, static_cast<size_t>(K),
                                   C, st, out);
}

// The library's own grow-only scratch for the current device (cudaMalloc on growth).
int s4_internal_workspace(size_t need, void** ws, size_t* ws_bytes) {
  std::lock_guard<std::mutex> lock(g_mutex);
  DeviceState* s = nullptr;
  int rc = device_state(&s);
  if (rc != GEMM_OK) return rc;
  if (s->s4_workspace_bytes < need) {
    // Grow: earlier launches may still read the old buffer.
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(e);
    if (s->s4_workspace) cudaFree(s->s4_workspace);
    s->s4_workspace = nullptr;
    s->s4_workspace_bytes = 0;
    e = cudaMalloc(&s->s4_workspace, need);
    if (e != cudaSuccess) return cuda_fail(e);
    s->s4_workspace_bytes = need;
  }
  *ws = s->s4_workspace;
  *ws_bytes = s->s4_workspace_bytes;
  return GEMM_OK;
}

int check_scales(const float* row_scale, const float* col_scale, const void* C, int c_is_fp16,
                 OutputSpec* out) {
  if (!row_scale || !col_scale || !C || (c_is_fp16 != 0 && c_is_fp16 != 1))
    return GEMM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(row_scale) | reinterpret_cast<uintptr_t>(col_scale)) & 3)
    return GEMM_ERR_MISALIGNED;
  out->epi = c_is_fp16 ? EPI_OUT16 : EPI_F32_SCALED;
  out->row_scale = row_scale;
  out->col_scale = col_scale;
  return GEMM_OK;
}

}  // namespace
}  // namespace b200gemm

using namespace b200gemm;

extern "C" {

int gemm_fp16(int M, int N, int K, const void* A, const void* B, float* C, gemm_stream_t stream) {
  int rc = check_common(M, N, K, A, B, C);
  if (rc != GEMM_OK) return rc;
  if (K % 8) return GEMM_ERR_MISALIGNED;
  return launch_gemm<ptx::KIND_F16>(M, N, K, A, static_cast<size_t>(K) * 2, B,
                                    static_cast<size_t>(K) * 2, C,
                                    reinterpret_cast<cudaStream_t>(stream));
}

int gemm_s8(int M, int N, int K, const int8_t* A, const int8_t* B, int32_t* C,
            gemm_stream_t stream) {
  int rc = check_common(M, N, K, A, B, C);
  if (rc != GEMM_OK) return rc;
  if (K % 16) return GEMM_ERR_MISALIGNED;
  if (K > K_LIMIT_INT) return GEMM_ERR_K_TOO_LARGE;
  return launch_gemm<ptx::KIND_I8>(M, N, K, A, static_cast<size_t>(K), B, static_cast<size_t>(K), C,
                                   reinterpret_cast<cudaStream_t>(stream));
}

size_t gemm_s4_workspace_bytes(int M, int N, int K) {
  if (M <= 0 || N <= 0 || K <= 0) return 0;
  return s4_workspace_need(M, N, K);
}

int gemm_s4_ws(int M, int N, int K, const uint8_t* A, const uint8_t* B, int32_t* C,
               void* workspace, size_t workspace_bytes, gemm_stream_t stream) {
  int rc = check_s4(M, N, K, A, B, C);
  if (rc != GEMM_OK) return rc;
  return s4_with_workspace(M, N, K, A, B, C, workspace, workspace_bytes, OutputSpec(),
                           reinterpret_cast<cudaStream_t>(stream));
}

int gemm_s4(int M, int N, int K, const uint8_t* A, const uint8_t* B, int32_t* C,
            gemm_stream_t stream) {
  int rc = check_s4(M, N, K, A, B, C);
  if (rc != GEMM_OK) return rc;
  void* ws = nullptr;
  size_t ws_bytes = 0;
  rc = s4_internal_workspace(s4_workspace_need(M, N, K), &ws, &ws_bytes);
  if (rc != GEMM_OK) return rc;
  return s4_with_workspace(M, N, K, A, B, C, ws, ws_bytes, OutputSpec(),
                           reinterpret_cast<cudaStream_t>(stream));
}

int gemm_fp16_f16out(int M, int N, int K, const void* A, const void* B, void* C,
                     gemm_stream_t stream) {
  int rc = check_common(M, N, K, A, B, C);
  if (rc != GEMM_OK) return rc;
  if (K % 8) return GEMM_ERR_MISALIGNED;
  OutputSpec out;
  out.epi = EPI_OUT16;
  return launch_gemm<ptx::KIND_F16>(M, N, K, A, static_cast<size_t>(K) * 2, B,
                                    static_cast<size_t>(K) * 2, C,
                                    reinterpret_cast<cudaStream_t>(stream), out);
}

int gemm_s8_dequant(int M, int N, int K, const int8_t* A, const int8_t* B, const float* row_scale,
                    const float* col_scale, void* C, int c_is_fp16, gemm_stream_t stream) {
  int rc = check_common(M, N, K, A, B, C);
  if (rc != GEMM_OK) return rc;
  if (K % 16) return GEMM_ERR_MISALIGNED;
  if (K > K_LIMIT_INT) return GEMM_ERR_K_TOO_LARGE;
  OutputSpec out;
  rc = check_scales(row_scale, col_scale, C, c_is_fp16, &out);
  if (rc != GEMM_OK) return rc;
  return launch_gemm<ptx::KIND_I8>(M, N, K, A, static_cast<size_t>(K), B, static_cast<size_t>(K), C,
                                   reinterpret_cast<cudaStream_t>(stream), out);
}

int gemm_s4_dequant(int M, int N, int K, const uint8_t* A, const uint8_t* B,
                    const float* row_scale, const float* col_scale, void* C, int c_is_fp16,
                    gemm_stream_t stream) {
  int rc = check_s4(M, N, K, A, B, C);
  if (rc != GEMM_OK) return rc;
  OutputSpec out;
  rc = check_scales(row_scale, col_scale, C, c_is_fp16, &out);
  if (rc != GEMM_OK) return rc;
  void* ws = nullptr;
  size_t ws_bytes = 0;
  rc = s4_internal_workspace(s4_workspace_need(M, N, K), &ws, &ws_bytes);
  if (rc != GEMM_OK) return rc;
  return s4_with_workspace(M, N, K, A, B, C, ws, ws_bytes, out,
                           reinterpret_cast<cudaStream_t>(stream));
}

int gemm_release_workspaces(void) {
  std::lock_guard<std::mutex> lock(g_mutex);
  int cur = 0;
  if (cudaGetDevice(&cur) != cudaSuccess) cur = -1;
  int rc = GEMM_OK;
  for (int d = 0; d < MAX_DEVICES; ++d) {
    if (!g_dev[d].s4_workspace) continue;
    cudaError_t e = cudaSetDevice(d);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaFree(g_dev[d].s4_workspace);
    if (e != cudaSuccess) rc = cuda_fail(e);
    g_dev[d].s4_workspace = nullptr;
    g_dev[d].s4_workspace_bytes = 0;
  }
  if (cur >= 0) cudaSetDevice(cur);
  return rc;
}

int gemm_unpack_s4(int rows, int K, const uint8_t* packed, int8_t* out, size_t out_pitch,
                   gemm_stream_t stream) {
  if (rows <= 0 || K <= 0 || !packed || !out) return GEMM_ERR_INVALID_ARG;
  if (K % 32 || out_pitch % 16 || out_pitch < static_cast<size_t>(K) ||
      ((reinterpret_cast<uintptr_t>(packed) | reinterpret_cast<uintptr_t>(out)) & 15))
    return GEMM_ERR_MISALIGNED;
  return launch_unpack(rows, packed, out, 0, nullptr, nullptr, K, out_pitch,
                       reinterpret_cast<cudaStream_t>(stream));
}

int gemm_mma_peak_probe(int precision, int iters, int n_cols, int commit_every, double* ops_out,
                        gemm_stream_t stream) {
  if (iters <= 0 || !ops_out || (precision != GEMM_PREC_FP16 && precision != GEMM_PREC_S8) ||
      n_cols < 16 || n_cols > PROBE_BN || n_cols % 16 || commit_every < 0)
    return GEMM_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_mutex);
  DeviceState* s = nullptr;
  int rc = device_state(&s);
  if (rc != GEMM_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  unsigned long long* trace = (g_trace_on & 1) ? s->trace_ptr : nullptr;
  cudaError_t e;
  int k_per_mma;
  if (precision == GEMM_PREC_FP16) {
    auto kernel = mma_peak_probe_kernel<ptx::KIND_F16>;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PROBE_SMEM);
    if (e != cudaSuccess) return cuda_fail(e);
    kernel<<<s->num_sms, 128, PROBE_SMEM, st>>>(iters, n_cols, commit_every, s->status_ptr, trace);
    k_per_mma = MMA_K_BYTES / 2;
  } else {
    auto kernel = mma_peak_probe_kernel<ptx::KIND_I8>;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PROBE_SMEM);
    if (e != cudaSuccess) return cuda_fail(e);
    kernel<<<s->num_sms, 128, PROBE_SMEM, st>>>(iters, n_cols, commit_every, s->status_ptr, trace);
    k_per_mma = MMA_K_BYTES;
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  *ops_out += 2.0 * BM * n_cols * k_per_mma * static_cast<double>(iters / 4 * 4) * s->num_sms;
  return GEMM_OK;
}

int gemm_query_config(int precision, int M, int N, int K, char* buf, int len) {
  if (!buf || len <= 0 || M <= 0 || N <= 0 || K <= 0 || precision < GEMM_PREC_FP16 ||
      precision > GEMM_PREC_S4)
    return GEMM_ERR_INVALID_ARG;
  int num_sms = 148;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < MAX_DEVICES && g_dev[dev].ready)
      num_sms = g_dev[dev].num_sms;
  }
  const int elem = precision == GEMM_PREC_FP16 ? 2 : 1;
  const TileConfig c =
      select_config(M, N, num_sms, ceil_div(static_cast<long long>(K) * elem, BK_BYTES), 32, true);
  if (c.bn == 0) return GEMM_ERR_INVALID_ARG;
  const long long tiles =
      static_cast<long long>(ceil_div(M, BM * c.cta_group)) * ceil_div(N, c.bn);
  const long long units = num_sms / c.cta_group;
  snprintf(buf, static_cast<size_t>(len),
           "BM=%d BN=%d BK=%d cta_group=%d stages=%d group_m=%d split_k=%d tiles=%lld ctas=%lld "
           "kind=%s%s",
           BM * c.cta_group, c.bn, atoms_for(c.bn, c.cta_group) * BK_BYTES / elem, c.cta_group,
           c.stages, c.group_m, c.splits, tiles,
           (tiles * c.splits < units ? tiles * c.splits : units) * c.cta_group,
           precision == GEMM_PREC_FP16 ? "f16" : "i8",
           precision == GEMM_PREC_S4 ? " prepass=unpack_s4" : "");
  return GEMM_OK;
}

int gemm_set_config_override(int bn, int group_m, int cta_group, int split_k) {
  if (group_m < 0 || cta_group < 0 || cta_group > 2 || split_k < 0 || split_k > 64)
    return GEMM_ERR_INVALID_ARG;
  bool ok = false;
  for (int cg = 1; cg <= 2; ++cg) {
    if (cta_group && cg != cta_group) continue;
    for (int w : kWidths) {
      if (bn && w != bn) continue;
      ok = ok || variant_exists(w, cg);
    }
  }
  if (!ok) return GEMM_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_mutex);
  g_override_bn = bn;
  g_override_group_m = group_m;
  g_override_cta_group = cta_group;
  g_override_splits = split_k;
  return GEMM_OK;
}

int gemm_last_device_status(void) {
  std::lock_guard<std::mutex> lock(g_mutex);
  DeviceState* s = nullptr;
  int rc = device_state(&s);
  if (rc != GEMM_OK) return rc;
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(e);
  int v = 0;
  e = cudaMemcpy(&v, s->status_ptr, sizeof(int), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(e);
  if (v != 0) {
    e = cudaMemset(s->status_ptr, 0, sizeof(int));
    if (e != cudaSuccess) return cuda_fail(e);
  }
  return v;
}

int gemm_set_l2_policy(int policy) {
  if (policy < 0 || policy > 31) return GEMM_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_mutex);
  g_l2_policy = policy;
  return GEMM_OK;
}

int gemm_trace_enable(int on) {
  std::lock_guard<std::mutex> lock(g_mutex);
  g_trace_on = on & 31;
  return GEMM_OK;
}

int gemm_trace_read(unsigned long long* out, int max_ctas) {
  static_assert(TRACE_SLOTS == 12, "header documents 12 words per CTA");
  if (!out || max_ctas <= 0) return GEMM_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_mutex);
  DeviceState* s = nullptr;
  int rc = device_state(&s);
  if (rc != GEMM_OK) return rc;
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(e);
  const int n = max_ctas < TRACE_MAX_CTAS ? max_ctas : TRACE_MAX_CTAS;
  e = cudaMemcpy(out, s->trace_ptr, sizeof(unsigned long long) * TRACE_SLOTS * n,
                 cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(e);
  return n;
}

int gemm_last_cuda_error(void) { return g_last_cuda_error; }

const char* gemm_status_string(int status) {
  switch (status) {
    case GEMM_OK: return "ok";
    case GEMM_ERR_INVALID_ARG: return "invalid argument";
    case GEMM_ERR_MISALIGNED: return "misaligned pointer or K";
    case GEMM_ERR_K_TOO_LARGE: return "K too large: INT32 result could overflow";
    case GEMM_ERR_UNSUPPORTED_DEVICE: return "unsupported device (needs compute capability 10.x)";
    case GEMM_ERR_CUDA: return "CUDA call failed";
    case GEMM_ERR_WORKSPACE: return "workspace too small or misaligned";
    case GEMM_ERR_TOO_LARGE: return "problem exceeds the capacity of this entry point";
    default: return "unknown status";
  }
}

int gemm_version(void) { return 1000; }

}  // extern "C"

// ---------------------------------------------------------------------------
// gemm_s4_static: the INT4 GEMM for callers that must not allocate.
//
// The int8 images of A and B that gemm_s4 keeps in a cudaMalloc'ed workspace
// live here in a fixed array inside the library's device image, so the call
// needs no allocator at all.  Cost: every GPU that loads the library carries
// the array until the process exits.
// ---------------------------------------------------------------------------
namespace b200gemm {
namespace {

constexpr size_t kStaticScratchBytes = 32u << 20;  // 32 MiB: up to M*K + N*K = 2 * 4096 * 4096

static __device__ __align__(256) unsigned char g_s4_static_scratch[kStaticScratchBytes];

// In host code the array's name is only a handle for the runtime, not a device
// address: the address a kernel can use is looked up once per device.
void* g_s4_static_ptr[MAX_DEVICES] = {};
std::mutex g_s4_static_mutex;

int static_scratch_for_current_device(void** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= MAX_DEVICES) return GEMM_ERR_UNSUPPORTED_DEVICE;
  std::lock_guard<std::mutex> lock(g_s4_static_mutex);
  if (!g_s4_static_ptr[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_s4_static_scratch);  // resolves for the current device
    if (e != cudaSuccess) return cuda_fail(e);
    if (!ptr || (reinterpret_cast<uintptr_t>(ptr) & 255)) return cuda_fail(cudaErrorInvalidSymbol);
    g_s4_static_ptr[dev] = ptr;
  }
  *out = g_s4_static_ptr[dev];
  return GEMM_OK;
}

}  // namespace
}  // namespace b200gemm

extern "C" {

size_t gemm_s4_static_capacity(void) { return b200gemm::kStaticScratchBytes; }

int gemm_s4_static(int M, int N, int K, const uint8_t* A, const uint8_t* B, int32_t* C,
                   gemm_stream_t stream) {
  int rc = check_s4(M, N, K, A, B, C);
  if (rc != GEMM_OK) return rc;
  if (gemm_s4_workspace_bytes(M, N, K) > kStaticScratchBytes) return GEMM_ERR_TOO_LARGE;
  void* scratch = nullptr;
  rc = static_scratch_for_current_device(&scratch);
  if (rc != GEMM_OK) return rc;
  // Every byte of the scratch that the GEMM reads is rewritten by the unpack
  // launches of this call, so nothing left over from an earlier call is used.
  return gemm_s4_ws(M, N, K, A, B, C, scratch, kStaticScratchBytes, stream);
}

}  // extern "C"

// ---------------------------------------------------------------------------
// gemm_host: the GEMM for operands and result in HOST memory.
//
// The matrices are cut into blocks of kHostBlock rows of A / rows of B.  Blocks
// travel to the device on one stream in "wavefront" order (A0 B0 B1 A1 B2 A2 ...),
// every C block is multiplied on the caller's stream as soon as its two operand
// blocks have arrived, and finished C blocks travel back on a third stream, so
// both PCIe directions and the tensor cores work at the same time.
// ---------------------------------------------------------------------------
namespace b200gemm {
namespace {

constexpr int kHostBlock = 2048;

struct HostPipe {
  cudaStream_t h2d = nullptr, d2h = nullptr;
  void* buf[4] = {nullptr, nullptr, nullptr, nullptr};  // A, B, C, int8 images (INT4 only)
  size_t cap[4] = {0, 0, 0, 0};
  cudaEvent_t ev[3 + 2 * 64 + 64 * 64] = {};
  int num_ev = 0;
};
HostPipe g_pipe[MAX_DEVICES];
std::mutex g_pipe_mutex;

int pipe_grow(HostPipe& p, int which, size_t need) {
  if (p.cap[which] >= need) return GEMM_OK;
  cudaError_t e = cudaDeviceSynchronize();  // earlier calls may still use the old buffer
  if (e != cudaSuccess) return cuda_fail(e);
  if (p.buf[which]) cudaFree(p.buf[which]);
  p.buf[which] = nullptr;
  p.cap[which] = 0;
  e = cudaMalloc(&p.buf[which], need);
  if (e != cudaSuccess) return cuda_fail(e);
  p.cap[which] = need;
  return GEMM_OK;
}

int pipe_event(HostPipe& p, int index, cudaEvent_t* out) {
  while (p.num_ev <= index) {
    cudaError_t e = cudaEventCreateWithFlags(&p.ev[p.num_ev], cudaEventDisableTiming);
    if (e != cudaSuccess) return cuda_fail(e);
    ++p.num_ev;
  }
  *out = p.ev[index];
  return GEMM_OK;
}

#define GEMM_CUDA_TRY(call)                         \
  do {                                              \
    cudaError_t e_ = (call);                        \
    if (e_ != cudaSuccess) return cuda_fail(e_);    \
  } while (0)

}  // namespace
}  // namespace b200gemm

extern "C" {

int gemm_host(int precision, int M, int N, int K, const void* A, const void* B, void* C,
              gemm_stream_t stream) {
  if (M <= 0 || N <= 0 || K <= 0 || !A || !B || !C) return GEMM_ERR_INVALID_ARG;
  int k_align, kind_i8;
  size_t row_bytes;  // bytes of one operand row as stored by the caller
  switch (precision) {
    case GEMM_PREC_FP16: k_align = 8; kind_i8 = 0; row_bytes = static_cast<size_t>(K) * 2; break;
    case GEMM_PREC_S8: k_align = 16; kind_i8 = 1; row_bytes = static_cast<size_t>(K); break;
    case GEMM_PREC_S4: k_align = 32; kind_i8 = 1; row_bytes = static_cast<size_t>(K) / 2; break;
    default: return GEMM_ERR_INVALID_ARG;
  }
  if (K % k_align) return GEMM_ERR_MISALIGNED;
  if (kind_i8 && K > K_LIMIT_INT) return GEMM_ERR_K_TOO_LARGE;
  const int nba = ceil_div(M, kHostBlock), nbb = ceil_div(N, kHostBlock);
  if (nba > 64 || nbb > 64) return GEMM_ERR_TOO_LARGE;

  int dev = 0;
  GEMM_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= MAX_DEVICES) return GEMM_ERR_UNSUPPORTED_DEVICE;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState* s = nullptr;
    int rc = device_state(&s);
    if (rc != GEMM_OK) return rc;
  }
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  HostPipe& p = g_pipe[dev];
  if (!p.h2d) GEMM_CUDA_TRY(cudaStreamCreateWithFlags(&p.h2d, cudaStreamNonBlocking));
  if (!p.d2h) GEMM_CUDA_TRY(cudaStreamCreateWithFlags(&p.d2h, cudaStreamNonBlocking));
  int rc = pipe_grow(p, 0, align_up(static_cast<size_t>(M) * row_bytes, 256));
  if (rc == GEMM_OK) rc = pipe_grow(p, 1, align_up(static_cast<size_t>(N) * row_bytes, 256));
  if (rc == GEMM_OK) rc = pipe_grow(p, 2, align_up(static_cast<size_t>(M) * N * 4, 256));
  if (rc == GEMM_OK && precision == GEMM_PREC_S4)
    rc = pipe_grow(p, 3, align_up(static_cast<size_t>(M) * K, 256) +
                             align_up(static_cast<size_t>(N) * K, 256));
  if (rc != GEMM_OK) return rc;

  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const uint8_t* hA = static_cast<const uint8_t*>(A);
  const uint8_t* hB = static_cast<const uint8_t*>(B);
  uint8_t* dA = static_cast<uint8_t*>(p.buf[0]);
  uint8_t* dB = static_cast<uint8_t*>(p.buf[1]);
  uint32_t* dC = static_cast<uint32_t*>(p.buf[2]);
  int8_t* a8 = static_cast<int8_t*>(p.buf[3]);
  int8_t* b8 = a8 ? a8 + align_up(static_cast<size_t>(M) * K, 256) : nullptr;

  cudaEvent_t ev_begin, ev_done;
  if ((rc = pipe_event(p, 0, &ev_begin)) != GEMM_OK) return rc;
  if ((rc = pipe_event(p, 1, &ev_done)) != GEMM_OK) return rc;
  // The copies start when the caller's stream gets here (and after the previous call
  // through this pipe has finished with the device buffers, which that stream waited for).
  GEMM_CUDA_TRY(cudaEventRecord(ev_begin, st));
  GEMM_CUDA_TRY(cudaStreamWaitEvent(p.h2d, ev_begin, 0));
  GEMM_CUDA_TRY(cudaStreamWaitEvent(p.d2h, ev_begin, 0));

  bool have_a[64] = {}, have_b[64] = {};
  auto rows_of = [](int total, int blk) {
    const int lo = blk * kHostBlock;
    return (total - lo < kHostBlock) ? total - lo : kHostBlock;
  };
  OutputSpec out;
  out.ldc = N;
  out.no_split = true;
  // Wavefront order: A0 B0 B1 A1 B2 A2 ...
  int ia = 0, ib = 0;
  while (ia < nba || ib < nbb) {
    const bool take_a = (ia < nba) && (ib >= nbb || ia < ib || (ia == 0 && ib == 0));
    const int blk = take_a ? ia : ib;
    const int total = take_a ? M : N;
    const size_t off = static_cast<size_t>(blk) * kHostBlock * row_bytes;
    const size_t bytes = static_cast<size_t>(rows_of(total, blk)) * row_bytes;
    cudaEvent_t ev_in;
    if ((rc = pipe_event(p, 3 + (take_a ? blk : 64 + blk), &ev_in)) != GEMM_OK) return rc;
    GEMM_CUDA_TRY(cudaMemcpyAsync((take_a ? dA : dB) + off, (take_a ? hA : hB) + off, bytes,
                                  cudaMemcpyHostToDevice, p.h2d));
    GEMM_CUDA_TRY(cudaEventRecord(ev_in, p.h2d));
    GEMM_CUDA_TRY(cudaStreamWaitEvent(st, ev_in, 0));
    if (precision == GEMM_PREC_S4) {  // expand the block to int8 once, on the compute stream
      const size_t off8 = static_cast<size_t>(blk) * kHostBlock * K;
      rc = launch_unpack(rows_of(total, blk), (take_a ? dA : dB) + off, (take_a ? a8 : b8) + off8,
                         0, nullptr, nullptr, K, static_cast<size_t>(K), st);
      if (rc != GEMM_OK) return rc;
    }
    if (take_a) have_a[ia++] = true; else have_b[ib++] = true;
    // every C block that this operand block completes
    for (int i = 0; i < nba; ++i) {
      for (int j = 0; j < nbb; ++j) {
        if (!have_a[i] || !have_b[j]) continue;
        if (!((take_a && i == blk) || (!take_a && j == blk))) continue;
        const int mi = rows_of(M, i), nj = rows_of(N, j);
        uint32_t* c_blk = dC + static_cast<size_t>(i) * kHostBlock * N +
                          static_cast<size_t>(j) * kHostBlock;
        if (precision == GEMM_PREC_FP16) {
          rc = launch_gemm<ptx::KIND_F16>(mi, nj, K, dA + static_cast<size_t>(i) * kHostBlock * row_bytes,
                                          row_bytes, dB + static_cast<size_t>(j) * kHostBlock * row_bytes,
                                          row_bytes, c_blk, st, out);
        } else {
          const int8_t* pa = precision == GEMM_PREC_S4
                                 ? a8 + static_cast<size_t>(i) * kHostBlock * K
                                 : reinterpret_cast<const int8_t*>(dA) + static_cast<size_t>(i) * kHostBlock * K;
          const int8_t* pb = precision == GEMM_PREC_S4
                                 ? b8 + static_cast<size_t>(j) * kHostBlock * K
                                 : reinterpret_cast<const int8_t*>(dB) + static_cast<size_t>(j) * kHostBlock * K;
          rc = launch_gemm<ptx::KIND_I8>(mi, nj, K, pa, static_cast<size_t>(K), pb,
                                         static_cast<size_t>(K), c_blk, st, out);
        }
        if (rc != GEMM_OK) return rc;
        cudaEvent_t ev_c;
        if ((rc = pipe_event(p, 3 + 128 + i * 64 + j, &ev_c)) != GEMM_OK) return rc;
        GEMM_CUDA_TRY(cudaEventRecord(ev_c, st));
        GEMM_CUDA_TRY(cudaStreamWaitEvent(p.d2h, ev_c, 0));
        uint8_t* h_blk = static_cast<uint8_t*>(C) +
                         (static_cast<size_t>(i) * kHostBlock * N + static_cast<size_t>(j) * kHostBlock) * 4;
        GEMM_CUDA_TRY(cudaMemcpy2DAsync(h_blk, static_cast<size_t>(N) * 4, c_blk,
                                        static_cast<size_t>(N) * 4, static_cast<size_t>(nj) * 4, mi,
                                        cudaMemcpyDeviceToHost, p.d2h));
      }
    }
  }
  GEMM_CUDA_TRY(cudaEventRecord(ev_done, p.d2h));
  GEMM_CUDA_TRY(cudaStreamWaitEvent(st, ev_done, 0));
  return GEMM_OK;
}

int gemm_host_release(void) {
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  int cur = 0;
  if (cudaGetDevice(&cur) != cudaSuccess) cur = -1;
  int rc = GEMM_OK;
  for (int d = 0; d < MAX_DEVICES; ++d) {
    HostPipe& p = g_pipe[d];
    if (!p.h2d && !p.buf[0]) continue;
    cudaError_t e = cudaSetDevice(d);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { rc = cuda_fail(e); continue; }
    for (int k = 0; k < 4; ++k) {
      if (p.buf[k]) cudaFree(p.buf[k]);
      p.buf[k] = nullptr;
      p.cap[k] = 0;
    }
    for (int k = 0; k < p.num_ev; ++k) cudaEventDestroy(p.ev[k]);
    p.num_ev = 0;
    if (p.h2d) cudaStreamDestroy(p.h2d);
    if (p.d2h) cudaStreamDestroy(p.d2h);
    p.h2d = p.d2h = nullptr;
  }
  if (cur >= 0) cudaSetDevice(cur);
  return rc;
}

}  // extern "C"

