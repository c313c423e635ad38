/*
 * b200gemm -- dense GEMM  C = A * B^T  on one NVIDIA B200 (sm_100a) in the three
 * precisions of the multi-precision tensor-core study this library follows.
 *
 * Operation (paper Sec. II-A: the tensor-core operation D = A*B + C, used with a
 * zero initial accumulator; Listing 2(c): ".row.col" operands; Listing 1: row i
 * of A starts i*K elements after the base, i*K/2 bytes for 4-bit data; Sec. VI:
 * INT32 results, no dequantisation or scaling inside the kernel):
 *
 *     C[i][j] = sum_{k=0}^{K-1} a(i,k) * b(j,k)      0 <= i < M, 0 <= j < N
 *
 * Layouts, common to all entry points:
 *     A : M rows, K elements each, row-major, leading dimension K  (device memory)
 *     B : N rows, K elements each, K contiguous ("K-major"), leading dimension K
 *     C : M x N row-major, leading dimension N, 32-bit elements, OVERWRITTEN
 *         (no alpha/beta; previous contents are ignored)
 *
 * Every pointer is a DEVICE pointer owned by the caller; it must stay valid
 * until `stream` has passed the call.  Calls are asynchronous on `stream` and
 * never synchronise.  Argument errors are reported by the return value and
 * enqueue nothing.  M and N are arbitrary; K carries an alignment rule because
 * operand rows are fetched by TMA (row pitch must be a multiple of 16 bytes).
 *
 * Split-K.  The study runs squares only and names non-square shapes as future
 * work (Sec. VI).  When a problem has fewer C tiles than the GPU has SMs (small
 * M, as in LLM decoding, or small squares) the selector lets several work units
 * share one tile over disjoint K ranges: C is zeroed on the stream and every
 * unit ADDS its partial tile (TMA reduction).  When the tiles fill more than one
 * wave of SMs but the last wave is at most half full and K is long, only that
 * last wave's tiles are split (and only their part of C is zeroed first).
 * INT32 results stay exact; FP32
 * results then depend on the order the partial sums land, i.e. two runs can
 * differ in the last bits, always inside the stated bound.
 *
 * All functions return GEMM_OK (0) or a negative GEMM_ERR_* code.
 * A process may call from several host threads; calls that share a stream are
 * ordered by it.
 */
#ifndef B200GEMM_H_
#define B200GEMM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Opaque CUDA stream handle (a cudaStream_t); 0 / NULL is the default stream. */
typedef struct CUstream_st* gemm_stream_t;

enum {
  GEMM_OK = 0,
  GEMM_ERR_INVALID_ARG = -1,  /* null pointer, non-positive dimension, unknown enum value */
  GEMM_ERR_MISALIGNED = -2,   /* base pointer or K violates the alignment rule */
  GEMM_ERR_K_TOO_LARGE = -3,  /* integer paths: K > 131071, an INT32 result could overflow */
  GEMM_ERR_UNSUPPORTED_DEVICE = -4, /* current device is not compute capability 10.x */
  GEMM_ERR_CUDA = -5,         /* a CUDA runtime/driver call failed (see gemm_last_cuda_error) */
  GEMM_ERR_WORKSPACE = -6,    /* caller-supplied workspace too small or misaligned */
  GEMM_ERR_TOO_LARGE = -7     /* problem exceeds a fixed capacity of the entry point */
};

enum { GEMM_PREC_FP16 = 0, GEMM_PREC_S8 = 1, GEMM_PREC_S4 = 2 };

/*
 * FP16 inputs, FP32 accumulate, FP32 output (the study's FP16 family, Table VI:
 * f16 operands with f32 accumulators; Sec. IV Run 1 counts a 4-byte C).
 * A, B: IEEE binary16.  Accumulation order inside the tensor core is hardware
 * defined; results satisfy |C - exact| <= 1e-4 * sum_k|a*b| + 1e-6.
 * Alignment: A, B, C 16-byte aligned; K % 8 == 0.
 */
int gemm_fp16(int M, int N, int K, const void* A, const void* B, float* C, gemm_stream_t stream);

/*
 * Signed 8-bit inputs, INT32 accumulate and output, exact (the study's INT8
 * family, Sec. IV Run 2).  Alignment: A, B, C 16-byte aligned; K % 16 == 0;
 * K <= 131071 so that no INT32 sum can overflow.
 */
int gemm_s8(int M, int N, int K, const int8_t* A, const int8_t* B, int32_t* C,
            gemm_stream_t stream);

/*
 * Signed 4-bit inputs, INT32 accumulate and output, exact (the study's INT4
 * family, Sec. IV Runs 3-4; Listing 2(c) ".s4.s4 -> .s32").  A: M rows of K/2
 * bytes, B: N rows of K/2 bytes; element k of a row is bits [4*(k&1), 4*(k&1)+4)
 * of byte k>>1 (low nibble first), two's complement.
 *
 * Blackwell's tcgen05.mma has no 4-bit integer kind.  Large problems: the
 * operands are first sign-extended to int8 by a streaming pre-pass into a
 * workspace of gemm_s4_workspace_bytes(M, N, K) bytes and then multiplied by the
 * INT8 kernel.  Small problems and problems with few rows: a kernel variant
 * expands the nibbles on the way to the MMAs and needs no workspace (see
 * gemm_set_s4_scheme for the rule and the switch).  For the pre-pass gemm_s4
 * keeps one grow-only workspace per device inside the library:
 * the first call on a device (and any call that needs a larger one) allocates
 * with cudaMalloc, which synchronises the device; the buffer is reused by later
 * calls, so concurrent gemm_s4 calls on different streams of one device must be
 * ordered by the caller.  Use gemm_s4_ws to supply the workspace yourself.
 * Alignment: A, B, C 16-byte aligned; K % 32 == 0; K <= 131071.
 */
int gemm_s4(int M, int N, int K, const uint8_t* A, const uint8_t* B, int32_t* C,
            gemm_stream_t stream);

/* Bytes of device scratch gemm_s4_ws needs for this problem (0 on bad sizes). */
size_t gemm_s4_workspace_bytes(int M, int N, int K);

/*
 * gemm_s4 with caller-owned scratch: `workspace` is a device buffer of at least
 * gemm_s4_workspace_bytes(M, N, K) bytes, 256-byte aligned, which the call
 * overwrites; it must not be shared by calls that may overlap on the GPU.
 * Allocates nothing.
 */
int gemm_s4_ws(int M, int N, int K, const uint8_t* A, const uint8_t* B, int32_t* C,
               void* workspace, size_t workspace_bytes, gemm_stream_t stream);

/*
 * FP16 inputs, FP32 accumulate, FP16 OUTPUT: each FP32 sum is rounded once to
 * binary16 (round to nearest even) on the way out, halving the bytes of C.
 * (The study's closest variant, fp16_ptx_fp16acc in Table VI, keeps FP16
 * accumulators; here only the stored result is narrowed, so the error is the
 * FP32 path's plus one half-precision rounding.)  C: M x N binary16, row-major.
 * Alignment as gemm_fp16; rows of C that are not 16-byte multiples (N % 8 != 0)
 * take a slower scalar store path.  A 16-bit (or scaled) result cannot be
 * accumulated in C, so where the plain GEMMs split K over CTAs that add into C,
 * this entry point and the dequantising ones split K between the two or four
 * CTAs of a cluster, which send their partial sums to the first one as bulk
 * copies between shared memories (narrow one-CTA tiles: M = 16, N = 4096,
 * K = 16384: 46 -> 28 us).
 */
int gemm_fp16_f16out(int M, int N, int K, const void* A, const void* B, void* C,
                     gemm_stream_t stream);

/*
 * INT8 / INT4 GEMM with the dequantisation fused into the epilogue -- the step
 * the study leaves to the surrounding inference pipeline (Sec. VI: its kernels
 * stop at INT32 "without in-kernel dequantization or scaling"):
 *
 *     C[i][j] = float(sum_k a(i,k) * b(j,k)) * row_scale[i] * col_scale[j]
 *
 * computed in FP32 from the exact INT32 sum (conversion and the two products
 * each round once), stored as FP32 (c_is_fp16 = 0) or rounded once more to
 * binary16 (c_is_fp16 = 1).  row_scale: M floats, col_scale: N floats, device
 * memory, 4-byte aligned.  Operand layouts, K rules and (for INT4) the internal
 * workspace are those of gemm_s8 / gemm_s4.
 */
int gemm_s8_dequant(int M, int N, int K, const int8_t* A, const int8_t* B, const float* row_scale,
                    const float* col_scale, void* C, int c_is_fp16, gemm_stream_t stream);
int gemm_s4_dequant(int M, int N, int K, const uint8_t* A, const uint8_t* B,
                    const float* row_scale, const float* col_scale, void* C, int c_is_fp16,
                    gemm_stream_t stream);

/*
 * The same GEMM for operands and result in HOST memory (the end-to-end path:
 * the study times kernels only, Sec. III-B; a caller whose data lives on the
 * host also pays the PCIe transfers).  A, B, C are HOST pointers with the
 * layouts above (A: M x K, B: N x K, C: M x N 32-bit; for GEMM_PREC_S4 A and B
 * are packed, K/2 bytes per row).  precision = GEMM_PREC_FP16 / _S8 / _S4.
 *
 * The call cuts A and B into blocks of 2048 rows, sends them to the device in an
 * order that lets C blocks start early, multiplies each C block on `stream` as
 * soon as its two operand blocks have arrived and sends finished C blocks back
 * while later ones are still being multiplied, using two internal copy streams.
 * Everything is enqueued asynchronously: C is complete when `stream` has passed
 * the call.  Use page-locked (pinned) host memory; with pageable memory the
 * copies are staged by the driver, block the calling thread and run slower.
 * The library keeps grow-only device copies of A, B and C per device
 * (cudaMalloc on first use / growth, which synchronises the device);
 * gemm_host_release frees them.  Calls through this entry point on one device
 * share those buffers and must be ordered by the caller (same stream, or
 * events).  K rules as for the device entry points; at most 64 x 64 blocks.
 */
int gemm_host(int precision, int M, int N, int K, const void* A, const void* B, void* C,
              gemm_stream_t stream);

/* Frees the device buffers, streams and events behind gemm_host (synchronises). */
int gemm_host_release(void);

/*
 * gemm_s4 for callers that cannot allocate device memory.  (The paper has no
 * counterpart: its INT4 kernels need no scratch.)
 *
 * Who needs it: a process that hands all device memory to its own pool at
 * start-up (an inference server, a trainer running under a memory cap) cannot
 * let a library call cudaMalloc behind its back -- it may fail, or break the
 * budget -- and has no spare buffer to lend to gemm_s4_ws; and a latency-
 * critical loop cannot afford the device-wide synchronisation that cudaMalloc
 * and cudaFree imply, which gemm_s4 incurs whenever its workspace has to grow.
 *
 * This entry point computes exactly what gemm_s4 computes, but unpacks into a
 * fixed 32 MiB array that is part of the library's device image.  It calls no
 * cudaMalloc, cudaFree or other allocating routine.  Limits and rules:
 *   - gemm_s4_workspace_bytes(M, N, K) must not exceed gemm_s4_static_capacity()
 *     (32 MiB: M*K + N*K <= 2 * 4096 * 4096); larger problems are refused with
 *     GEMM_ERR_TOO_LARGE and enqueue nothing.
 *   - Every GPU on which the library is loaded holds the 32 MiB until the
 *     process exits.
 *   - The first call on each device looks up the array's device address (one
 *     cudaGetSymbolAddress, with that device current).  Make that first call
 *     before starting any stream capture.
 *   - All calls on a device share the one array: calls that may overlap on the
 *     GPU (different streams without an ordering between them) race on it and
 *     give wrong results.  Calls on one stream are safe.  The array keeps the
 *     previous call's bytes; each call rewrites every byte it later reads.
 * Arguments, layouts, alignment (K % 32 == 0, 16-byte pointers, K <= 131071)
 * and error codes are those of gemm_s4.
 */
int gemm_s4_static(int M, int N, int K, const uint8_t* A, const uint8_t* B, int32_t* C,
                   gemm_stream_t stream);

/* Size in bytes of the fixed scratch behind gemm_s4_static. */
size_t gemm_s4_static_capacity(void);

/*
 * Frees the per-device workspaces held for gemm_s4 (synchronises).  Optional;
 * they are otherwise released when the process exits.
 */
int gemm_release_workspaces(void);

/*
 * The INT4 pre-pass on its own (Sec. IV Run 3 discusses why the 4-bit path's
 * cost is the cost of getting nibbles into the MMA's operand format): expands
 * `rows` rows of K packed signed 4-bit values (K/2 bytes per row, pitch K/2)
 * into int8, one value per byte, row pitch `out_pitch` bytes (>= K, multiple of
 * 16; bytes K..out_pitch-1 of each row are set to zero).  K % 32 == 0,
 * `packed` and `out` 16-byte aligned.
 */
int gemm_unpack_s4(int rows, int K, const uint8_t* packed, int8_t* out, size_t out_pitch,
                   gemm_stream_t stream);

/*
 * Measurement aid (Sec. III-B profiles every kernel against the hardware's
 * limits): every SM issues `iters` back-to-back tcgen05.mma instructions of
 * shape 128 x n_cols x (32 bytes of K) on shared-memory operands that are never
 * reloaded, and the operation count performed is added to *ops_out (host
 * pointer).  n_cols: multiple of 16 up to 256 (256 = the production tile).
 * iters is rounded down to a multiple of 4 (MMAs are issued in groups of 4, one
 * k-block of the GEMM kernels).  commit_every: 0 = none inside the loop; c > 0 =
 * a tcgen05.commit after every c groups, as a pipelined GEMM does once per
 * k-block (c = 1).
 * Time it with events on `stream` for the MMA-issue-only rate of the given
 * precision (GEMM_PREC_FP16 or GEMM_PREC_S8); with tracing on, words [0] and
 * [1] of each CTA's trace record hold the cycles and nanoseconds of the loop.
 */
int gemm_mma_peak_probe(int precision, int iters, int n_cols, int commit_every, double* ops_out,
                        gemm_stream_t stream);

/*
 * Writes a human-readable description of the tile configuration the selector
 * picks for this problem ("BM=256 BN=256 BK=64 cta_group=2 stages=6 group_m=12
 * split_k=1 split_tiles=0 tiles=1024 ctas=148 kind=f16") into buf (NUL
 * terminated, truncated to len); for INT4 followed by the route
 * (" prepass=unpack_s4" or " s4=fused_unpack"), and by " swap_ab" when the
 * kernel runs on exchanged operands (the tile is then described in the
 * kernel's orientation).  Describes the raw 32-bit outputs (gemm_fp16,
 * gemm_s8, gemm_s4).  Host only, no GPU work.
 */
int gemm_query_config(int precision, int M, int N, int K, char* buf, int len);

/*
 * Overrides the selector for later calls from this process: tile width BN
 * (0 = automatic), raster band height in tiles (0 = automatic), the number
 * of CTAs that share one tile (0 = automatic, 1 = 128 x BN tile per CTA, 2 =
 * 256 x BN tile per CTA pair) and the split-K factor (0 = automatic, 1 = off,
 * s = every C tile is computed by s work units over disjoint K ranges; capped
 * at the number of 128-byte K blocks; honoured only by gemm_fp16 / gemm_s8 /
 * gemm_s4*, whose 32-bit results can be summed in place).  For ablation sweeps
 * in the spirit of the paper's Run 4.  Returns GEMM_ERR_INVALID_ARG for a shape
 * that is not built.
 */
int gemm_set_config_override(int bn, int group_m, int cta_group, int split_k);

/*
 * Kernels never spin forever: a barrier wait that exceeds its limit makes the
 * kernel record a non-zero code and drain.  This reads that code for the
 * current device (synchronises the device) and clears it.  0 = no event;
 * 1/2/3 = producer / MMA / epilogue wait expired, 5 = a wait of the INT4
 * expansion warps expired.
 */
int gemm_last_device_status(void);

/*
 * Route of later gemm_s4 / gemm_s4_dequant calls.  tcgen05 has no signed 4-bit
 * integer kind (the paper's kernels feed mma.sync m16n8k64 .s4 operands
 * directly, Listing 2c), so the nibbles are expanded to int8 either
 *   - by a streaming pre-pass kernel into an int8 scratch, followed by the
 *     INT8 GEMM ("pre-pass"): each operand element is expanded once; or
 *   - inside the GEMM kernel ("fused"): packed tiles are loaded as they are and
 *     eight extra warps per CTA expand them in shared memory into the slots the
 *     MMAs read.  No scratch, and a quarter of the pre-pass route's HBM bytes
 *     for an operand that is read once; but half as much shared-memory traffic
 *     again per unit of math, which is what bounds the large-tile kernel.
 * Measured: at M = N = K = 8192 the pre-pass route is 1.1-1.35x faster; for
 * M = 16, N = K = 8192 (bound by the bytes of B) the fused route takes 15 us
 * instead of 33.
 * Small problems, bound by launches and latencies, save one launch with the
 * fused route (10-26 % up to 1024 x 1024 outputs).
 * scheme 0 (default, automatic): fused where the selector picks a one-CTA tile
 * and M <= 128 or N <= 128 or both <= 1024, or a single wave of CTA-pair tiles
 * (e.g. 2048^3); also for problems with a short side, where the pre-pass (cost:
 * the bytes of both operands) is dear next to the GEMM: M N / (M + N) <= 384
 * with the best tile the fused kernel has, and up to 1024 rows or columns with
 * its CTA-pair tile if the tiles fill their waves to 75 % (256 x 28672 x 8192:
 * 119 -> 67 us; 512 x 16384 x 4096: 44 -> 35 us); else the pre-pass.  1: always
 * the pre-pass; 2: fused wherever a fused variant is built (every one-CTA tile,
 * and the 256 x 256 and 256 x 128 CTA pairs), else the pre-pass.  gemm_s4_ws and gemm_s4_static
 * always use the pre-pass.  Results are identical, bit for bit.
 * gemm_query_config shows the route.  The paper has no counterpart; its Run 4
 * ablates how the operands reach the tensor cores, of which this is the
 * analogue here.
 */
int gemm_set_s4_scheme(int scheme);

/*
 * Whether later calls run the kernel on exchanged operands: its 128-row tile
 * side then holds rows of B (the caller's N), its narrow side rows of A, and C
 * is written by plain stores that are contiguous along N.  For problems with
 * few rows (M = 1..64, LLM decoding) this keeps 128 - M rows of zero fill out
 * of shared memory, of the ring depth and -- on the fused INT4 route -- of the
 * expansion work.  mode 0 (default, automatic): when N >= 1024 and M <= 32
 * (gemm_fp16) or M <= 64 (INT8, INT4, gemm_fp16_f16out, and gemm_fp16 from
 * N = 16384 on) (measured 2-12 % faster there); 1: never; 2: always
 * (any shape, precision and INT4 route; for tests and measurements).  Results:
 * integers identical; FP16 within the bound; dequantised outputs multiply the
 * two scales in the other order (last-bit differences).  gemm_query_config
 * shows "swap_ab" and then describes the tile in the kernel's orientation.  The
 * paper has no counterpart (square sizes only, Sec. VI).
 */
int gemm_set_swap_ab(int mode);

/*
 * L2 behaviour of later calls, a bit set (the paper's Run 4 ablates the
 * analogous .ca / .cg cache policy of cp.async).  Bits 0-1, eviction priority
 * of the operand loads: 0 = normal for A and B; 1 = A "evict last" (kept), B
 * "evict first" (streamed); 2 = both "evict last"; 3 = A "evict last", B
 * normal.  Bit 2 (4): turn OFF the serpentine K order (by default successive
 * tiles of a CTA walk K forward, backward, forward, ... so that a tile begins
 * on the K range its predecessor, which shares its A rows, read last and still
 * finds in L2).  Bit 3 (8): mark the C stores "evict first" (written once,
 * never re-read).  Bit 4 (16): fetch operands with 128-byte instead of 256-byte
 * L2 promotion.  Bit 5 (32): launch in plain stream order.  By default a GEMM
 * of this library is launched so that it may begin while the kernel in front of
 * it in the stream is still running (programmatic dependent launch): its set-up
 * (barriers, tensor memory, descriptor prefetch) and the launch latency overlap
 * that kernel's tail, and it waits for that kernel to complete before its first
 * load and its first store; a GEMM of this library lets its successor begin as
 * soon as it runs itself.  Stream semantics are unchanged; back-to-back small
 * GEMMs get 15-25 % faster (N = 512: 5.1 -> 4.0 us).  Default 11 = 3 + 8 with
 * the serpentine order on, which gave the lowest DRAM traffic at N = 8192; with
 * the default, problems that are one tile wide or one tile tall (few rows on one
 * side) use 2 for bits 0-1, so that the short operand every CTA re-reads is not
 * pushed out of L2 by the long one streaming past.  Bit 6 (64): no split-K
 * inside a cluster (see gemm_fp16_f16out / the dequantising entry points).
 * Integer results never depend on any of this; FP16 results may differ in the last bits (summation order) within the
 * bound.
 */
int gemm_set_l2_policy(int policy);

/*
 * Cycle accounting, in the spirit of the counter attribution the paper does
 * with its profiler (Sec. III-B).  gemm_trace_enable(1) makes later GEMM
 * launches record, per CTA, 16 unsigned 64-bit words: [0] SM cycles and [1]
 * nanoseconds the CTA ran (their ratio is the SM clock during the kernel),
 * cycles the producer waited for a free slot [2], the MMA issuer waited for
 * operands [3] and for a free accumulator [4], one epilogue warp waited for a
 * finished accumulator [5] and spent draining [6], the tile count [7], and the
 * issuer's cycles inside tcgen05.mma [8] and tcgen05.commit [9], the cycles
 * the CTA spent setting up barriers and tensor memory [10], and the producer's
 * cycles issuing loads [11]; fused INT4 only, one expansion warp: cycles
 * waiting for packed operands [12], for a free int8 slot [13] and spent
 * expanding [14]; [15] is unused.
 * Switching recording on (bit 1 from 0 to 1) synchronises the device and clears
 * all records.  Traced launches run in plain stream order (no early start, see
 * gemm_set_l2_policy bit 5), so that the cycle counts are the kernel's own.
 * gemm_trace_read synchronises the device, copies the words of the first
 * min(max_ctas, 160) CTAs of the last traced launch to `out` (host memory,
 * 16 * max_ctas words) and returns that CTA count.  Off by default; the cost
 * when on is a few clock reads per k-block.
 * `on` is a bit set: 1 = record; 2 = ablation, issue no MMAs (operand loads and
 * barriers only); 4 = ablation, issue no operand loads (MMAs and barriers only,
 * on whatever shared memory holds); 8 = the epilogue's waits back off with
 * nanosleep instead of polling; 16 = failure drill: one operand slot of the
 * first tile is never filled, so the kernel's bounded waits (2 s) must expire,
 * record a code for gemm_last_device_status, drain and return -- the call takes
 * a few seconds, C is garbage and the context stays usable; 32 = the epilogue
 * writes C straight from registers (16 bytes per thread and store) instead of
 * staging it in shared memory for TMA stores (results unchanged).  With bit 2, 4 or
 * 16 set C is garbage; 2 and 4 exist to attribute cycles to the load path or
 * the MMA path.
 */
int gemm_trace_enable(int on);
int gemm_trace_read(unsigned long long* out, int max_ctas);

/* cudaError_t value of the last failed CUDA call made by this library, or 0. */
int gemm_last_cuda_error(void);

/* Text for a GEMM_* return code. */
const char* gemm_status_string(int status);

/* Library version: major * 1000 + minor. */
int gemm_version(void);

#ifdef __cplusplus
}
#endif
#endif /* B200GEMM_H_ */
