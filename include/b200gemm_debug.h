/*
 * b200gemm, measurement and ablation switches -- not part of the product interface.
 *
 * The multi-precision study this library follows changes one variable at a time on
 * its best kernel (Sec. IV Run 4, Table XII) and attributes time with profiler
 * counters (Sec. III-B).  The calls below are the corresponding knobs here: they force
 * tile shapes, routes and cache policies, switch the kernels' cycle accounting on,
 * and run a failure drill.  They act on process-wide state that every later call of
 * the library reads once at its start, from whichever thread: set them while no
 * GEMM call is in flight, and put them back (0 / default) afterwards.  Results never
 * depend on them beyond the FP32 summation order, except where a switch says that C
 * is garbage.
 */
#ifndef B200GEMM_DEBUG_H_
#define B200GEMM_DEBUG_H_

#include "b200gemm.h"

#ifdef __cplusplus
extern "C" {
#endif

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
 * Which kernel large problems run on (a measurement switch; results do not
 * depend on it beyond the FP32 summation order): 0 = automatic; 1 = the
 * 256 x 256 tile per CTA pair with two accumulator buffers, whose epilogue
 * overlaps the next tile; 2 = the 512 x 256 tile per CTA pair wherever the
 * problem's layout allows it (plain orientation, no split-K), whose two
 * accumulators fill tensor memory and which moves a quarter fewer operand
 * bytes per unit of math.  The automatic rule takes 2 when its tiles fill at
 * least two waves of CTA pairs to 90 % and K covers at least 96 blocks of 128
 * bytes for FP16 (K >= 6144) or 64 for the integer kinds (K >= 8192; the INT4
 * pre-pass route included).  The paper fixes one tiling for every size
 * (Sec. III-A); this is the corresponding ablation axis here.
 *
 * There is a third kernel, for problems with a few rows on one side, which
 * are bound by reading the long operand once: every thread copies the 16-byte
 * pieces its own warp-level MMA fragments need (mma.sync m16n8k32, s8 x s8 ->
 * s32, or m16n8k16, f16 x f16 -> f32) into a private ring in shared memory
 * (cp.async, several steps ahead), loads them back and, for INT4, expands the
 * nibbles in registers; a CTA owns
 * 32 rows of the long operand over the whole of K, sums its warps'
 * results and writes its part of C once.  Family 0 takes it for a short side
 * of at most 16 rows against at least 512 -- INT4 always (and with 17-32
 * rows against at most 8192), INT8 with up to 8
 * rows always and with 9-16 while the long operand has at most 64 MB, FP16
 * while it has at most 32 M elements (INT8 and FP16 only with at least six
 * 32-row blocks per KB of a row); 3 =
 * wherever it exists (a short side of at most 32 rows); 1 and 2 never, nor do
 * calls with a forced tile shape, operand order or INT4 scheme, or traced ones.
 * gemm_query_config describes such a call as "few_rows rows_per_block=..
 * blocks=.. short_rows=.. warps=.. depth=.. ctas=..".
 */
int gemm_set_kernel_family(int family);

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
 * Measured: for M = 16, N = K = 8192 (bound by the bytes of B) the fused route
 * takes 15 us instead of 33; at M = N = K = 8192 the fused CTA-pair kernel in
 * its hybrid form (below) takes 337 us in a 20-launch loop and 379 us in a
 * sustained one against 359 / 409 us for the pre-pass route -- its kernel needs
 * 12 % more SM cycles but nothing expands B beforehand and it draws less power,
 * which on a power-capped part is clock -- and the INT8 GEMM on int8 operands
 * takes 342 / 385 us.
 * Small problems, bound by launches and latencies, save one launch with the
 * fused route (10-26 % up to 1024 x 1024 outputs).
 * scheme 0 (default, automatic): fused where the selector picks a one-CTA tile
 * and M <= 128 or N <= 128 or both <= 1024, or a single wave of CTA-pair tiles
 * (e.g. 2048^3); for problems with a short side, where the pre-pass (cost:
 * the bytes of both operands) is dear next to the GEMM: M N / (M + N) <= 384
 * with the best tile the fused kernel has, and up to 1024 rows or columns with
 * its CTA-pair tile if the tiles fill their waves to 75 %; and for problems that
 * are large in both dimensions (more than 1024 rows and columns, at least one
 * wave of 256 x 256 pair tiles, K >= 2048: fifteen shapes between 2048 and 16384
 * measured, the pre-pass ahead on none) (256 x 28672 x 8192:
 * 119 -> 67 us; 512 x 16384 x 4096: 44 -> 35 us); else the pre-pass.  1: always
 * the pre-pass; 2: fused wherever a fused variant is built (every one-CTA tile,
 * and the 256 x 256 and 256 x 128 CTA pairs), else the pre-pass.  4: the
 * pre-pass, but where the INT8 GEMM runs on the 256 x 256 CTA-pair tile over at
 * least two waves, four extra warps per CTA of that kernel expand the operands
 * inside it, chunk by chunk ahead of the tiles that read them (no separate
 * launch; measured slower than 1 -- N = 8192: 573 k SM cycles against 495 k plus
 * a 36 us pre-pass -- because that kernel already keeps the SM's L2 port and
 * shared-memory pipe full and runs at ~60 % speed while the expansion is in
 * progress; kept as the ablation's third INT4 route).  3 = 1.
 * On the CTA-pair tiles (plain operand order) the fused route has a hybrid
 * form: B stays packed and is expanded inside the kernel, A -- the short operand
 * there, which every tile column would otherwise expand again -- is turned into
 * an int8 image once, by a small kernel in front, into scratch leased from the
 * pool (gemm_query_config then shows "a=int8_image").  Taken where the 6-8 % it
 * saves in the kernel outweigh that extra launch and the image's bytes, i.e. for
 * large N K against a short M (256 x 28672 x 8192: 66 -> 61 us).  5 = as 2, but
 * never the hybrid form; 6 = as 2, always the hybrid form where it exists.
 * gemm_s4_ws and gemm_s4_static always use the pre-pass launch.  Results are
 * identical, bit for bit.
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
 * Bit 7 (128): no even shares.  By default the one-CTA fused INT4 kernels (few
 * rows on one side, raw output) cut the tiles' K ranges, laid end to end, into
 * equal contiguous shares, one per SM, where that lowers the busiest SM's work by
 * a fifth or more -- 224 tiles on 148 SMs make some SMs do two where the average
 * is 1.5 -- instead of giving every SM whole tiles or equal parts of one tile;
 * each piece is added into a zeroed C (gemm_query_config shows "even_share=").
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
 * expanding [14]; 512 x 256 kernel only: cycles the MMA issuer waited for
 * the tile's second accumulator [15] ([4] is then the first); hybrid fused INT4
 * kernel: [15] is the part of [3] spent waiting for the atom of the A image.
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
 * staging it in shared memory for TMA stores (results unchanged); 64 = the
 * epilogue of the 128/256-row kernels reads the accumulator in the 16x256b shape,
 * in which four neighbouring threads hold 32 contiguous bytes of a row, and
 * stores whole 32-byte sectors straight to C: no staging, no shared-memory
 * traffic beside the mainloop's (raw outputs with rows of whole 32-byte sectors;
 * results unchanged; 2-4 % fewer SM cycles at N = 8192 and the same time, the
 * part being power-capped).  With bit 2, 4 or
 * 16 set C is garbage; 2 and 4 exist to attribute cycles to the load path or
 * the MMA path.
 */
int gemm_trace_enable(int on);
int gemm_trace_read(unsigned long long* out, int max_ctas);

/*
 * Ring depth (shared-memory slots of one k-block each) of the 256 x 256 CTA-pair
 * kernel for gemm_fp16 / gemm_s8: 0 = the shipped depth (6), else 3, 4, 5 or 6.  A
 * seventh slot does not fit beside the epilogue's staging buffers in 227 KB.  The
 * analogue of the paper's 2-stage / 3-stage pipeline comparison (Sec. III-A,
 * Listing 3; Sec. IV Run 4), with depth as the only variable.
 */
int gemm_set_stages_override(int stages);

/*
 * Host-side counters for tests: out[0] = tensor maps encoded so far by this process
 * (calls that find their maps in the per-thread cache do not count), out[1] = scratch
 * buffers the pool of the current device holds, out[2] = 1 if the last gemm_s4-family
 * call on this thread used the overlapped pre-pass.  `n` = entries of `out`.
 */
int gemm_debug_counters(long long* out, int n);

/*
 * Host time of one call of gemm_fp16 / gemm_s8 / gemm_s4 (precision = GEMM_PREC_*), measured
 * inside the library so that no foreign-function dispatch is in it: synchronises `stream`,
 * enqueues `calls` (1..512, below the depth of the launch queue, so that the device never
 * holds the host back) identical calls back to back, and writes the wall time of that loop
 * divided by `calls`, in nanoseconds, to *ns_per_call.  The calls are real: C is written.
 * Returns the first non-zero code of a call, else 0.  A measurement aid (the paper does not
 * discuss host cost; its sizes start at 512, where a call is a few microseconds on the device
 * and the enqueue rate of the host bounds a stream of them).
 */
int gemm_debug_host_cost(int precision, int M, int N, int K, const void* A, const void* B, void* C,
                         gemm_stream_t stream, int calls, double* ns_per_call);

/*
 * Measurement aid for calls that are bound by reading one operand once (the
 * problems with a few rows): enqueues a kernel on `stream` that reads `bytes`
 * bytes (a multiple of 16) at `data` (device memory, 16-byte aligned) with
 * 16-byte loads and keeps nothing.  Launched like the GEMMs (it may start while
 * the grid in front drains and waits for it before its first load), so its
 * time in a given harness -- launch, first-byte latency and tail included -- is
 * what a GEMM call that only had to read that operand could at best take there.
 * Writes nothing.
 */
int gemm_debug_read_probe(const void* data, size_t bytes, gemm_stream_t stream);

/*
 * Measurement aid: waits for the device and returns every L2 line that is held
 * with raised priority to normal status (cudaCtxResetPersistingL2Cache).  The
 * tile kernels load operands they re-read with the L2 priority "evict last",
 * and lines so marked survive any amount of ordinary traffic: a timing harness
 * that flushes L2 by writing a large buffer does not remove them, and whatever
 * it times next may find part of its operands in L2 (measured: a kernel that
 * reads a 128 MB operand once ran 25.1 us from a clean L2 and 23.4 us after a
 * tile kernel had read the same operand).  Call it between the cases of a
 * comparison.
 */
int gemm_debug_reset_l2(void);

#ifdef __cplusplus
}
#endif
#endif /* B200GEMM_DEBUG_H_ */
