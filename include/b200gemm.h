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
 * L2.  The tile kernels fetch the operand they re-read (a band of A, or the
 * long operand of a problem with few rows) with the L2 eviction priority "evict
 * last".  Lines so marked are displaced by other such lines but not by ordinary
 * traffic, so after a call part of L2 stays occupied by operand data until
 * later calls of this library replace it or the application returns the lines
 * to normal status (cudaCtxResetPersistingL2Cache; gemm_debug_reset_l2 in
 * b200gemm_debug.h does that).  A timing harness that "flushes L2" by writing a
 * large buffer does not remove them.
 *
 * All functions return GEMM_OK (0) or a negative GEMM_ERR_* code.
 * A process may call from several host threads (the call path takes no global
 * lock); calls that share a stream are ordered by it, and two threads that
 * enqueue on the same stream at once get an unspecified order, as with any CUDA
 * work.  Tensor-map descriptors are cached per thread, keyed on pointer, extents
 * and pitch, so repeated calls on the same buffers skip their encoding.
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
 * (A problem with at most 16 rows on one side against 512 or more on the
 * other, and at most 32 M elements in the long operand, does not run on tiles:
 * see gemm_set_kernel_family in b200gemm_debug.h.  Same bound.)
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
 * Blackwell's tcgen05.mma has no 4-bit integer kind.  A problem with at most 16
 * rows on one side (M or N) against 512 or more on the other (at most 32 rows
 * against 512 ... 8192) never reaches it:
 * the long operand goes from global memory straight into the fragments of the
 * warp-level integer MMA, its nibbles expanded in registers, in one launch that
 * needs no scratch and zeroes nothing (gemm_s8 does the same with up to 8
 * such rows, and with 9-16 while the long operand has at most 64 MB; see
 * gemm_set_kernel_family in b200gemm_debug.h).
 * Most other problems: a kernel
 * variant expands the nibbles on the way to the MMAs (see gemm_set_s4_scheme in
 * b200gemm_debug.h for the rule and the switch).  The rest (a short K, less than
 * a wave of tiles with more than 1024 rows and columns, a few in-between
 * shapes): the operands are first sign-extended to int8 by a streaming pre-pass
 * into a workspace of gemm_s4_workspace_bytes(M, N, K) bytes and then multiplied
 * by the INT8 kernel.  Where A is re-read by many tile columns -- large problems,
 * a short M against a large N x K -- the expanding variant takes A as an int8 image made by
 * a small kernel in front (M x K rounded up to 256 bytes of scratch).  For
 * the pre-pass and that image the library leases a scratch buffer from a per-device pool for
 * the call's stream: the first call on a stream (and any call that needs a
 * larger one) allocates with cudaMallocAsync on that stream -- no device-wide
 * synchronisation -- and later calls on the stream reuse it, so calls on
 * different streams never share scratch.  A buffer whose last use has finished
 * may move to another stream.  While a stream is being captured into a graph
 * nothing can be allocated: make one call of the same size outside the capture
 * first (a captured call that only wanted the image of A does without it and
 * expands both operands in the kernel instead; one that needs the pre-pass
 * fails); the captured call then keeps using that buffer, and keeping replays of
 * the graph apart from other gemm_s4 calls that may use it is the caller's job.
 * gemm_release_workspaces frees the pool.  Use gemm_s4_ws to supply the scratch
 * yourself.
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
 *     before starting any stream capture.  The array is part of the library's
 *     device code image, which the CUDA runtime places in device memory when the
 *     image is first needed on a device -- by any call of this library there.  A
 *     process that is about to hand all remaining device memory to its own pool
 *     should therefore make one call into the library on each device first (any
 *     entry point that launches, e.g. a tiny gemm_s4_static), so that the image
 *     and its 32 MiB are in place before the memory is gone.
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
 * Frees the scratch buffers the library holds for gemm_s4 / gemm_s4_dequant on
 * every device (synchronises each device that has any).  Optional; they are
 * otherwise released when the process exits.
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
 * Writes a human-readable description of the tile configuration the selector
 * picks for this problem ("BM=256 BN=256 BK=64 cta_group=2 stages=6 group_m=12
 * split_k=1 split_tiles=0 tiles=1024 ctas=148 kind=f16") into buf (NUL
 * terminated, truncated to len); for INT4 followed by the route
 * (" prepass=unpack_s4" or " s4=fused_unpack"), and by " swap_ab" when the
 * kernel runs on exchanged operands (the tile is then described in the
 * kernel's orientation).  A problem that goes to the kernel for a few rows
 * instead of a tile kernel reads "few_rows rows_per_block=32 blocks=256
 * short_rows=16 warps=8 depth=3 ctas=256 kind=i8" (" s4=in_registers" for INT4).
 * Describes the raw 32-bit outputs (gemm_fp16, gemm_s8, gemm_s4).  Host only,
 * no GPU work.
 */
int gemm_query_config(int precision, int M, int N, int K, char* buf, int len);

/*
 * Kernels never spin forever: a barrier wait that exceeds its limit (2 s) makes
 * the kernel record a non-zero code in a status word on the device, drain and
 * return, leaving garbage in C -- the host call has long returned GEMM_OK by
 * then.  A caller that must be sure of C therefore reads the word after the
 * work: gemm_last_device_status reads it for the current device and clears it
 * (it synchronises the device); gemm_read_device_status enqueues a copy of the
 * word to `host_out` (host memory, page-locked for a truly asynchronous copy) on
 * `stream`, in stream order behind the GEMMs enqueued there, without clearing.
 * 0 = no event; 1/2/3 = producer / MMA / epilogue wait expired, 5 = a wait of the
 * INT4 expansion warps expired.
 */
int gemm_last_device_status(void);
int gemm_read_device_status(int* host_out, gemm_stream_t stream);

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
