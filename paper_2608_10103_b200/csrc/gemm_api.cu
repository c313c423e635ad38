// C-ABI of the library (see include/b200gemm.h for the contract): the extern "C" entry
// points.  State and tensor maps live in runtime.cuh, shape selection in selector.cuh,
// launch plumbing in launch.cuh, the host-memory pipeline in host_pipeline.cuh.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <mutex>

#include <chrono>
#include "../../include/b200gemm.h"
#include "gemm_kernel.cuh"
#include "launch.cuh"
#include "peak_probe.cuh"
#include "runtime.cuh"
#include "selector.cuh"
#include "unpack_s4.cuh"

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
  return s4_auto(M, N, K, A, B, C, OutputSpec(), reinterpret_cast<cudaStream_t>(stream));
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
  return s4_auto(M, N, K, A, B, C, out, reinterpret_cast<cudaStream_t>(stream));
}

int gemm_release_workspaces(void) {
  int cur = 0;
  if (cudaGetDevice(&cur) != cudaSuccess) cur = -1;
  int rc = GEMM_OK;
  for (int d = 0; d < MAX_DEVICES; ++d) {
    if (g_pool[d].buffers() == 0) continue;
    cudaError_t e = cudaSetDevice(d);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
      rc = cuda_fail(e);
      continue;
    }
    const int r = g_pool[d].release_all();
    if (r != 0) rc = cuda_fail(static_cast<cudaError_t>(r));
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
  const int num_sms = known_sm_count();
  const int elem = precision == GEMM_PREC_FP16 ? 2 : 1;
  const int kb = ceil_div(static_cast<long long>(K) * elem, BK_BYTES);
  if (few_rows_wanted(M, N, K, precision == GEMM_PREC_S4, OutputSpec(), precision == GEMM_PREC_FP16)) {
    const int rows_l = M < N ? N : M;
    const int row_bytes = precision == GEMM_PREC_S4 ? K / 2 : precision == GEMM_PREC_FP16 ? 2 * K : K;
    const FewRowsShape f = few_rows_shape(rows_l, M < N ? M : N, row_bytes, num_sms);
    snprintf(buf, static_cast<size_t>(len),
             "few_rows rows_per_block=%d blocks=%d short_rows=%d warps=%d depth=%d ctas=%d kind=%s%s",
             16 * f.mt, ceil_div(rows_l, 16 * f.mt), M < N ? M : N, f.warps, f.depth, f.grid,
             precision == GEMM_PREC_FP16 ? "f16" : "i8",
             precision == GEMM_PREC_S4 ? " s4=in_registers" : "");
    return GEMM_OK;
  }
  TileConfig c;
  bool fused = false, swap = false;
  const int user_m = M, user_n = N;
  if (precision == GEMM_PREC_S4 && !s4_prepass_forced()) {  // the decisions of s4_auto / launch_gemm_epi
    swap = swap_ab_wanted(M, N, true, OutputSpec());
    const TileConfig i8 =
        swap ? select_config(N, M, num_sms, kb, 32, true) : select_config(M, N, num_sms, kb, 32, true);
    fused = swap ? select_fused_s4(N, M, user_m, user_n, num_sms, kb, 32, true, i8, &c)
                 : select_fused_s4(M, N, user_m, user_n, num_sms, kb, 32, true, i8, &c);
  }
  if (!fused) {
    swap = swap_ab_wanted(M, N, precision != GEMM_PREC_FP16, OutputSpec());
    c = swap ? select_config(N, M, num_sms, kb, 32, true) : select_config(M, N, num_sms, kb, 32, true);
  }
  if (c.bn == 0) return GEMM_ERR_INVALID_ARG;
  if (swap) {  // the tile counts below are the kernel's
    M = user_n;
    N = user_m;
  }
  // (the overlapped INT4 pre-pass, scheme 4, rides on the 256 x 256 kernel: every problem the
  // 512 x 256 kernel would take qualifies for it)
  const bool wide = !(precision == GEMM_PREC_S4 && g_s4_scheme == 4) &&
                    wide_wanted(c, M, N, kb, num_sms, swap, false, fused, precision == GEMM_PREC_FP16);
  if (wide) {
    c.bn = WIDE_BN;
    c.cta_group = 2;
    c.splits = 1;
    c.split_tiles = 0;
    c.stages = WIDE_STAGES;
    c.group_m = band_height(M, WIDE_TILE_M, WIDE_BN, num_sms / 2);
  }
  const int rows_per_cta = wide ? WIDE_CTA_ROWS : BM;
  const long long tiles =
      static_cast<long long>(ceil_div(M, rows_per_cta * c.cta_group)) * ceil_div(N, c.bn);
  const long long units = num_sms / c.cta_group;
  char even[32] = "";
  long long even_ctas = 0;
  if (fused && c.cta_group == 1) {  // one-CTA fused INT4 tiles: equal contiguous shares of K
    const int kb_fused = 2 * ceil_div(K, 2 * BK_BYTES);
    const int share = s4_even_share(tiles, kb_fused, c.splits, c.split_tiles, num_sms);
    if (share) {
      snprintf(even, sizeof(even), " even_share=%d", share);
      even_ctas = (tiles * (kb_fused / 2) + share - 1) / share;
    }
  }
  snprintf(buf, static_cast<size_t>(len),
           "BM=%d BN=%d BK=%d cta_group=%d stages=%d group_m=%d split_k=%d split_tiles=%d "
           "tiles=%lld ctas=%lld kind=%s%s%s%s%s",
           rows_per_cta * c.cta_group, c.bn,
           (wide ? 1 : atoms_for(c.bn, c.cta_group)) * BK_BYTES / elem, c.cta_group,
           c.stages, c.group_m, c.splits, c.splits > 1 ? c.split_tiles : 0, tiles,
           even_ctas ? even_ctas
                     : (tiles + (c.splits > 1 ? static_cast<long long>(c.split_tiles) * (c.splits - 1) : 0) <
                                units
                            ? tiles + (c.splits > 1 ? static_cast<long long>(c.split_tiles) * (c.splits - 1) : 0)
                            : units) *
                           c.cta_group,
           precision == GEMM_PREC_FP16 ? "f16" : "i8",
           precision != GEMM_PREC_S4 ? "" : fused ? " s4=fused_unpack" : " prepass=unpack_s4",
           swap ? " swap_ab" : "",
           // hybrid form of the fused route: A as an int8 image made beforehand, B packed
           // (the raw outputs this function describes never split inside a cluster)
           (fused && !swap && c.cta_group == 2 && s4_hybrid_wanted(M, N, K)) ? " a=int8_image" : "",
           even);
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
  g_override_bn = bn;
  g_override_group_m = group_m;
  g_override_cta_group = cta_group;
  g_override_splits = split_k;
  return GEMM_OK;
}

int gemm_last_device_status(void) {
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

int gemm_set_kernel_family(int family) {
  if (family < 0 || family > 3) return GEMM_ERR_INVALID_ARG;
  g_family = family;
  return GEMM_OK;
}

int gemm_set_s4_scheme(int scheme) {
  if (scheme < 0 || scheme > 6) return GEMM_ERR_INVALID_ARG;
  g_s4_scheme = scheme;
  return GEMM_OK;
}

int gemm_set_swap_ab(int mode) {
  if (mode < 0 || mode > 2) return GEMM_ERR_INVALID_ARG;
  g_swap_ab = mode;
  return GEMM_OK;
}

int gemm_set_l2_policy(int policy) {
  if (policy < 0 || policy > 255) return GEMM_ERR_INVALID_ARG;
  g_l2_policy = policy;
  return GEMM_OK;
}

int gemm_set_stages_override(int stages) {
  if (stages != 0 && (stages < 3 || stages > 6)) return GEMM_ERR_INVALID_ARG;
  g_override_stages = stages;
  return GEMM_OK;
}

int gemm_debug_counters(long long* out, int n) {
  if (!out || n <= 0) return GEMM_ERR_INVALID_ARG;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) dev = 0;
  const long long v[3] = {g_map_encodes.load(), static_cast<long long>(g_pool[dev].buffers()),
                          t_last_s4_overlapped};
  for (int i = 0; i < n; ++i) out[i] = i < 3 ? v[i] : 0;
  return GEMM_OK;
}

int gemm_debug_host_cost(int precision, int M, int N, int K, const void* A, const void* B, void* C,
                         gemm_stream_t stream, int calls, double* ns_per_call) {
  if (!ns_per_call || calls < 1 || calls > 512) return GEMM_ERR_INVALID_ARG;
  if (precision != GEMM_PREC_FP16 && precision != GEMM_PREC_S8 && precision != GEMM_PREC_S4)
    return GEMM_ERR_INVALID_ARG;
  auto one = [&]() {
    switch (precision) {
      case GEMM_PREC_FP16: return gemm_fp16(M, N, K, A, B, static_cast<float*>(C), stream);
      case GEMM_PREC_S8:
        return gemm_s8(M, N, K, static_cast<const int8_t*>(A), static_cast<const int8_t*>(B),
                       static_cast<int32_t*>(C), stream);
      default:
        return gemm_s4(M, N, K, static_cast<const uint8_t*>(A), static_cast<const uint8_t*>(B),
                       static_cast<int32_t*>(C), stream);
    }
  };
  cudaError_t e = cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(e);
  const auto t0 = std::chrono::steady_clock::now();
  for (int i = 0; i < calls; ++i) {
    const int rc = one();
    if (rc != GEMM_OK) return rc;
  }
  const auto t1 = std::chrono::steady_clock::now();
  *ns_per_call = std::chrono::duration<double, std::nano>(t1 - t0).count() / calls;
  return GEMM_OK;
}

int gemm_debug_reset_l2(void) {
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaCtxResetPersistingL2Cache();
  return e == cudaSuccess ? GEMM_OK : cuda_fail(e);
}

int gemm_debug_read_probe(const void* data, size_t bytes, gemm_stream_t stream) {
  if (!data || bytes == 0 || (bytes & 15) || (reinterpret_cast<uintptr_t>(data) & 15))
    return GEMM_ERR_INVALID_ARG;
  DeviceState* s = nullptr;
  int rc = device_state(&s);
  if (rc != GEMM_OK) return rc;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(8 * s->num_sms), 1, 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.stream = reinterpret_cast<cudaStream_t>(stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;  // launched like the GEMMs: may start early, waits for the grid in front
  const cudaError_t e =
      cudaLaunchKernelEx(&cfg, read_probe_kernel, static_cast<const uint8_t*>(data), bytes,
                         reinterpret_cast<unsigned*>(s->status_ptr), 1);
  return e == cudaSuccess ? GEMM_OK : cuda_fail(e);
}

int gemm_read_device_status(int* host_out, gemm_stream_t stream) {
  if (!host_out) return GEMM_ERR_INVALID_ARG;
  DeviceState* s = nullptr;
  int rc = device_state(&s);
  if (rc != GEMM_OK) return rc;
  cudaError_t e = cudaMemcpyAsync(host_out, s->status_ptr, sizeof(int), cudaMemcpyDeviceToHost,
                                  reinterpret_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(e);
  return GEMM_OK;
}

int gemm_trace_enable(int on) {
  if ((on & 1) && !(g_trace_on & 1)) {
    // recording starts: clear the records, so that CTAs a later launch does not have read 0
    DeviceState* s = nullptr;
    int rc = device_state(&s);
    if (rc != GEMM_OK) return rc;
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess)
      e = cudaMemset(s->trace_ptr, 0, sizeof(unsigned long long) * TRACE_SLOTS * TRACE_MAX_CTAS);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  g_trace_on = on & 127;
  return GEMM_OK;
}

int gemm_trace_read(unsigned long long* out, int max_ctas) {
  static_assert(TRACE_SLOTS == 16, "header documents 16 words per CTA");
  if (!out || max_ctas <= 0) return GEMM_ERR_INVALID_ARG;
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

int gemm_last_cuda_error(void) { return g_last_cuda_error.load(); }

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

int gemm_version(void) { return 2000; }

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

#include "host_pipeline.cuh"
