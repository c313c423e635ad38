// gemm_host: the GEMM for operands and result in HOST memory (included by gemm_api.cu,
// whose internal launch functions it uses).
#pragma once

#include "launch.cuh"

namespace b200gemm {
namespace {

constexpr int kHostBlock = 2048;

struct HostPipe {
  cudaStream_t h2d = nullptr, d2h = nullptr;
  void* buf[4] = {nullptr, nullptr, nullptr, nullptr};  // A, B, C, int8 images (INT4 only)
  size_t cap[4] = {0, 0, 0, 0};
  cudaEvent_t ev[3 + 2 * 64 + 64 * 64] = {};
  int num_ev = 0;
  bool used_before = false;  // ev[1] marks the end of the previous call
};
HostPipe g_pipe[MAX_DEVICES];
std::mutex g_pipe_mutex;

// Grows buffer `which`, stream-ordered on `st` (no device-wide synchronisation).  `st` has been
// made to wait for the previous call through this pipe, so nothing uses the old buffer any more
// once `st` gets here.
int pipe_grow(HostPipe& p, int which, size_t need, cudaStream_t st) {
  if (p.cap[which] >= need) return GEMM_OK;
  cudaError_t e;
  if (p.buf[which]) {
    e = cudaFreeAsync(p.buf[which], st);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  p.buf[which] = nullptr;
  p.cap[which] = 0;
  e = cudaMallocAsync(&p.buf[which], need, st);
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
    DeviceState* s = nullptr;
    int rc = device_state(&s);
    if (rc != GEMM_OK) return rc;
  }
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  HostPipe& p = g_pipe[dev];
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (!p.h2d) GEMM_CUDA_TRY(cudaStreamCreateWithFlags(&p.h2d, cudaStreamNonBlocking));
  if (!p.d2h) GEMM_CUDA_TRY(cudaStreamCreateWithFlags(&p.d2h, cudaStreamNonBlocking));
  // The previous call through this pipe (possibly on another stream) must have finished with
  // the device buffers before this one refills -- or frees -- them.
  if (p.used_before) GEMM_CUDA_TRY(cudaStreamWaitEvent(st, p.ev[1], 0));
  int rc = pipe_grow(p, 0, align_up(static_cast<size_t>(M) * row_bytes, 256), st);
  if (rc == GEMM_OK) rc = pipe_grow(p, 1, align_up(static_cast<size_t>(N) * row_bytes, 256), st);
  if (rc == GEMM_OK) rc = pipe_grow(p, 2, align_up(static_cast<size_t>(M) * N * 4, 256), st);
  if (rc == GEMM_OK && precision == GEMM_PREC_S4)
    rc = pipe_grow(p, 3, align_up(static_cast<size_t>(M) * K, 256) +
                             align_up(static_cast<size_t>(N) * K, 256), st);
  if (rc != GEMM_OK) return rc;

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
  p.used_before = true;
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
    p.used_before = false;
    if (p.h2d) cudaStreamDestroy(p.h2d);
    if (p.d2h) cudaStreamDestroy(p.d2h);
    p.h2d = p.d2h = nullptr;
  }
  if (cur >= 0) cudaSetDevice(cur);
  return rc;
}

}  // extern "C"
