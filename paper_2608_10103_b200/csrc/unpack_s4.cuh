// INT4 pre-pass: packed signed 4-bit values -> int8, one value per byte.
//
// The paper's INT4 kernels feed nibbles straight to mma.sync.m16n8k64.s4
// (Listing 2c).  tcgen05.mma has no 4-bit integer kind, so here every operand
// element is sign-extended once, in a streaming pass bound by HBM bandwidth
// (reads 1/2 byte, writes 1 byte per element), and the INT8 tensor-core kernel
// then consumes the result.  Doing it once per operand costs O(N^2) bytes;
// doing it inside the GEMM pipeline would repeat it for every tile that
// re-reads the operand (N/BN resp. M/BM times).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace b200gemm {

// Eight nibbles of `w` (byte b holds element 2b in bits 0-3 and element 2b+1 in
// bits 4-7) -> eight sign-extended bytes in element order: lo = elements 0-3,
// hi = elements 4-7.
__device__ __forceinline__ void unpack8_s4(uint32_t w, uint32_t& lo, uint32_t& hi) {
  uint32_t even = w & 0x0F0F0F0Fu;         // elements 0,2,4,6 (one per byte)
  uint32_t odd = (w >> 4) & 0x0F0F0F0Fu;   // elements 1,3,5,7
  even |= (even & 0x08080808u) * 0x1Eu;    // bit 3 set -> fill bits 4-7 (0x08 * 0x1E = 0xF0)
  odd |= (odd & 0x08080808u) * 0x1Eu;
  lo = __byte_perm(even, odd, 0x5140);     // e0 o0 e1 o1
  hi = __byte_perm(even, odd, 0x7362);     // e2 o2 e3 o3
}

// One thread expands 16 packed bytes (32 elements) into 32 output bytes.
// chunks_per_row = K / 32.  Bytes K .. out_pitch-1 of each output row are zeroed.
// The kernel handles two matrices in one launch (A then B of a GEMM): chunk
// indices [0, chunks_a) belong to the first, the rest to the second.
struct UnpackJob {
  const uint4* packed;
  int8_t* out;
  long long chunks;  // rows * chunks_per_row
};

__global__ void __launch_bounds__(256)
unpack_s4_kernel(UnpackJob a, UnpackJob b, int chunks_per_row, long long out_pitch, int chained) {
  // the GEMM behind this kernel may set up now; it waits for this grid before its first load
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // launched early itself (its launch latency overlaps the tail of the grid in front): that grid
  // may still read the scratch this kernel writes, or produce the packed operands it reads
  if (chained) asm volatile("griddepcontrol.wait;" ::: "memory");
  const long long total = a.chunks + b.chunks;
  const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
  for (long long g = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; g < total;
       g += stride) {
    const bool second = g >= a.chunks;
    const long long idx = second ? g - a.chunks : g;
    const uint4* src = second ? b.packed : a.packed;
    int8_t* out = second ? b.out : a.out;
    const long long row = idx / chunks_per_row;
    const int chunk = static_cast<int>(idx - row * chunks_per_row);
    const uint4 w = ptx::ld_global_stream_v4(src + idx);
    uint4 o0, o1;
    unpack8_s4(w.x, o0.x, o0.y);
    unpack8_s4(w.y, o0.z, o0.w);
    unpack8_s4(w.z, o1.x, o1.y);
    unpack8_s4(w.w, o1.z, o1.w);
    uint4* dst = reinterpret_cast<uint4*>(out + row * out_pitch + static_cast<long long>(chunk) * 32);
    dst[0] = o0;
    dst[1] = o1;
    if (chunk == chunks_per_row - 1) {
      const long long k_end = static_cast<long long>(chunks_per_row) * 32;
      for (long long t = k_end; t < out_pitch; t += 16)
        *reinterpret_cast<uint4*>(out + row * out_pitch + t) = make_uint4(0, 0, 0, 0);
    }
  }
}

// The int8 image of one packed operand in the form the fused INT4 kernel's expansion warps
// produce in shared memory, for its hybrid variant (only the other operand expanded inside the
// kernel): every value times 16 (nibble in the high half of its byte), and inside each run of
// 256 values of K (one packed slot, 128 bytes; two int8 atoms of 128 bytes) the 16-byte packed
// chunk j = 4h + c goes to atom h, its even-k values to chunk c, its odd-k values to chunk c + 4.
// Rows are out_pitch bytes, a multiple of 256 (K rounded up; the excess is written as zeros).
// One thread per packed chunk.
__global__ void __launch_bounds__(256)
expand_s4_slots_kernel(const uint8_t* packed, int8_t* out, long long rows, int k_bytes,
                       long long out_pitch, int chained) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (chained) asm volatile("griddepcontrol.wait;" ::: "memory");
  const int chunks_per_row = static_cast<int>(out_pitch / 32);
  const long long total = rows * chunks_per_row;
  const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
  constexpr uint32_t HI = 0xF0F0F0F0u;
  for (long long g = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; g < total;
       g += stride) {
    const long long row = g / chunks_per_row;
    const int j = static_cast<int>(g - row * chunks_per_row);
    uint4 w = make_uint4(0, 0, 0, 0);
    if (j * 16 < k_bytes)
      w = ptx::ld_global_stream_v4(packed + row * k_bytes + static_cast<long long>(j) * 16);
    const int ps = j >> 3, h = (j >> 2) & 1, c = j & 3;
    int8_t* dst = out + row * out_pitch + static_cast<long long>(ps) * 256 + h * 128 + c * 16;
    *reinterpret_cast<uint4*>(dst) =
        make_uint4((w.x << 4) & HI, (w.y << 4) & HI, (w.z << 4) & HI, (w.w << 4) & HI);
    *reinterpret_cast<uint4*>(dst + 64) = make_uint4(w.x & HI, w.y & HI, w.z & HI, w.w & HI);
  }
}

}  // namespace b200gemm
