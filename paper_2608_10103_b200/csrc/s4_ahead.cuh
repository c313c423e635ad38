// Device side of the overlapped INT4 pre-pass (work list: s4_ahead.h).
//
// The GEMM kernel that multiplies the int8 images of A and B also produces them: four warps of
// their own per CTA claim chunks (32 rows x 512 columns) of the work list, expand the packed
// nibbles to sign-extended int8 (the paper's s4 operand format, Listing 2c, which tcgen05 cannot
// take directly) and publish each chunk with a flag; the TMA producer looks at the flags behind
// a box before it loads it.  Claims are dynamic, so a
// claimed chunk always belongs to a warp that is running and waits for nothing, and every
// wait on a flag is bounded like the kernel's other waits.
//
// Bookkeeping words (zero when the buffer is allocated, never cleared by the host again):
//   [0] epoch: calls completed on this buffer; a flag is "ready" when it holds epoch + 1, so
//       what earlier calls left behind is stale by construction, also in a replayed graph;
//   [1] CTAs that have left; the last one resets [1]..[3] and publishes the new epoch;
//   [2] next chunk to claim;  [3] chunks finished;  [4] epoch + 1 once every chunk is finished;
//   [S4A_SYNC_WORDS ...] one flag per chunk.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx.cuh"
#include "s4_ahead.h"
#include "unpack_s4.cuh"

namespace b200gemm {

struct S4Ahead {
  const uint4* packed_a;  // M rows of K/2 bytes
  const uint4* packed_b;  // N rows of K/2 bytes
  int8_t* a8;             // int8 images, row pitch K
  int8_t* b8;
  uint32_t* sync;
  S4AheadPlan plan;
  int M, N, K;
};

enum { S4A_EPOCH = 0, S4A_EXIT = 1, S4A_CLAIM = 2, S4A_DONE = 3, S4A_ALL_DONE = 4 };

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_u32(uint32_t* p, uint32_t v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Orders this thread's generic-proxy accesses to global memory before later accesses to it
// through the async proxy (TMA): executed by the writer before it publishes what it wrote.
__device__ __forceinline__ void fence_proxy_async_global() {
  asm volatile("fence.proxy.async.global;" ::: "memory");
}
__device__ __forceinline__ uint4 ld_stream_v4(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p)
               : "memory");
  return v;
}

// The epoch this call works under.  Read once per role, after the grid in front has completed.
__device__ __forceinline__ uint32_t s4a_epoch(const S4Ahead& ah) {
  return ld_acquire_u32(ah.sync + S4A_EPOCH) + 1u;
}

// Where one chunk lives: this lane's first packed 16-byte piece and first output byte, and how
// far its rows and columns are valid.
struct S4AChunkRef {
  const uint4* src;   // piece of row `row0` (rows advance by two per step)
  int8_t* dst;
  int row0, rows;     // first row of this lane, row count of the operand
  bool col_ok;
};

__device__ __forceinline__ S4AChunkRef s4a_chunk_ref(const S4Ahead& ah, int i, int lane) {
  int operand, row_chunk, k_chunk;
  s4a_decode(ah.plan, i, &operand, &row_chunk, &k_chunk);
  const int row_u4 = ah.K / 32;              // 16-byte pieces per packed row
  const int u = k_chunk * 16 + (lane & 15);  // this lane's piece in the row
  S4AChunkRef r;
  r.row0 = row_chunk * S4A_CHUNK_ROWS + (lane >> 4);
  r.rows = operand ? ah.N : ah.M;
  r.col_ok = u < row_u4;
  r.src = (operand ? ah.packed_b : ah.packed_a) + static_cast<size_t>(r.row0) * row_u4 + u;
  r.dst = (operand ? ah.b8 : ah.a8) + static_cast<size_t>(r.row0) * ah.K + static_cast<size_t>(u) * 32;
  return r;
}

// Claims and expands chunks, two at a time, until stop() is true or the list is exhausted (then
// returns false: nothing left to claim, ever).  Whole warp; stop() must be warp-uniform.
// One chunk = 32 rows x 256 packed bytes -> 32 rows x 512 int8; a warp instruction reads two
// rows x 256 contiguous bytes and writes two rows x 512.  Inside a busy GEMM a load or an
// atomic takes a thousand cycles and more to come back (the SM's L2 port is full of operand
// tiles), so a warp keeps all 32 loads of two chunks in flight and pays the round trips of
// claiming, draining its stores and publishing once per pair.
template <int CHUNKS = 2, class Stop>
__device__ __forceinline__ bool s4a_work(const S4Ahead& ah, uint32_t epoch, int lane, Stop stop) {
  static_assert(CHUNKS == 1 || CHUNKS == 2, "one or two chunks in flight per warp");
  const int total = s4a_total(ah.plan);
  const int row_u4 = ah.K / 32;
  while (!stop()) {
    int i = 0;
    if (lane == 0) i = static_cast<int>(atomicAdd(ah.sync + S4A_CLAIM, static_cast<uint32_t>(CHUNKS)));
    i = __shfl_sync(0xffffffffu, i, 0);
    if (i >= total) return false;
    const int n = (CHUNKS == 2 && i + 1 < total) ? 2 : 1;
    S4AChunkRef ref[CHUNKS];
    ref[0] = s4a_chunk_ref(ah, i, lane);
    if constexpr (CHUNKS == 2) ref[1] = s4a_chunk_ref(ah, n == 2 ? i + 1 : i, lane);
    uint4 w[CHUNKS][16];
#pragma unroll
    for (int c = 0; c < CHUNKS; ++c) {
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        if (c < n && ref[c].col_ok && ref[c].row0 + 2 * j < ref[c].rows)
          w[c][j] = ld_stream_v4(ref[c].src + static_cast<size_t>(2 * j) * row_u4);
      }
    }
#pragma unroll
    for (int c = 0; c < CHUNKS; ++c) {
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        if (c < n && ref[c].col_ok && ref[c].row0 + 2 * j < ref[c].rows) {
          uint4 o0, o1;
          unpack8_s4(w[c][j].x, o0.x, o0.y);
          unpack8_s4(w[c][j].y, o0.z, o0.w);
          unpack8_s4(w[c][j].z, o1.x, o1.y);
          unpack8_s4(w[c][j].w, o1.z, o1.w);
          uint4* out = reinterpret_cast<uint4*>(ref[c].dst + static_cast<size_t>(2 * j) * ah.K);
          out[0] = o0;
          out[1] = o1;
        }
      }
    }
    // the image is read through the async proxy (TMA), by other SMs
    fence_proxy_async_global();
    __syncwarp();
    if (lane == 0) {
      __threadfence();
      for (int c = 0; c < n; ++c) {
        int operand, row_chunk, k_chunk;
        s4a_decode(ah.plan, i + c, &operand, &row_chunk, &k_chunk);
        st_release_u32(ah.sync + S4A_SYNC_WORDS + s4a_flag_index(ah.plan, operand, row_chunk, k_chunk),
                       epoch);
      }
      if (atomicAdd(ah.sync + S4A_DONE, static_cast<uint32_t>(n)) + n == static_cast<uint32_t>(total))
        st_release_u32(ah.sync + S4A_ALL_DONE, epoch);
    }
  }
  return true;
}

// Producer warp: are the chunks behind A rows [a_row, a_row + 32 * a_chunks) and B rows
// [b_row, b_row + 32 * b_chunks) at k-chunk `kc` there?  Waits (bounded by `limit_ns`) until
// they are; false if it gave up or another role has.  All lanes call it; a_row, b_row multiples
// of 32, a_chunks + b_chunks <= 32.
__device__ __forceinline__ bool s4a_wait_ready(const S4Ahead& ah, uint32_t epoch, int a_row,
                                               int a_chunks, int b_row, int b_chunks, int kc,
                                               int lane, volatile uint32_t* abort_flag,
                                               uint64_t limit_ns) {
  const uint32_t* flag = nullptr;
  if (lane < a_chunks) {
    const int r = a_row / S4A_CHUNK_ROWS + lane;
    if (r < ah.plan.ra) flag = ah.sync + S4A_SYNC_WORDS + s4a_flag_index(ah.plan, 0, r, kc);
  } else if (lane < a_chunks + b_chunks) {
    const int r = b_row / S4A_CHUNK_ROWS + (lane - a_chunks);
    if (r < ah.plan.rb) flag = ah.sync + S4A_SYNC_WORDS + s4a_flag_index(ah.plan, 1, r, kc);
  }
  uint64_t t0 = 0;
  uint32_t spins = 0;
  bool mine = flag == nullptr;
  while (true) {
    if (!mine) mine = ld_acquire_u32(flag) == epoch;
    if (__all_sync(0xffffffffu, mine)) break;
    if ((++spins & 63u) == 0) {
      bool give_up = *abort_flag != 0;
      const uint64_t now = ptx::globaltimer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) give_up = true;
      if (__any_sync(0xffffffffu, give_up)) return false;
    }
  }
  __syncwarp();
  return true;
}

// One thread per CTA, after the CTA's last claim: the last CTA to leave resets the counters
// and publishes the new epoch.
__device__ __forceinline__ void s4a_cta_exit(const S4Ahead& ah) {
  __threadfence();
  const uint32_t epoch = ld_acquire_u32(ah.sync + S4A_EPOCH) + 1u;
  if (atomicAdd(ah.sync + S4A_EXIT, 1u) == gridDim.x - 1u) {
    ah.sync[S4A_EXIT] = 0;
    ah.sync[S4A_CLAIM] = 0;  // (claims run past the end of the list by design)
    ah.sync[S4A_DONE] = 0;
    __threadfence();
    st_release_u32(ah.sync + S4A_EPOCH, epoch);
  }
}

}  // namespace b200gemm
