/*
 * tman.h -- C ABI of the low-bit-weight x fp16-activation matmul through table lookup
 * (decode: bit-serial LUT mpGEMV; prefill: LUT dequantization fused into a tensor-core GEMM),
 * written for NVIDIA B200 (sm_100a).
 *
 * Conventions for every call
 *   - All data pointers are DEVICE pointers owned by the caller unless a parameter says "host".
 *   - Nothing is allocated, nothing is kept between calls, the device is never synchronised
 *     (except tman_read_status), all work is enqueued on `stream`.
 *   - The return value is a tman_status.  Argument errors are reported before anything is
 *     enqueued.  Errors only the device can see (a packed buffer whose header does not match
 *     the arguments, a bounded wait that ran out) are written to the first 32-bit word of the
 *     workspace ("status word"); read it with tman_read_status after the stream has drained.
 *     A kernel that finds a bad header leaves its outputs untouched.
 *   - Shapes: M tokens (rows of x), K input channels (reduction), N output channels.
 *     W is logically [K x N]:  w[k][n] = s[k/group][n] * (q[k][n] - z[k/group][n])
 *     (paper Sec. 2.2, "Dequantization-based low-bit inference"), q and z unsigned integers
 *     in [0, 2^bits).
 *   - Alignment: packed and workspace 256 bytes, x and y 16 bytes (else TMAN_ERR_SHAPE).
 *   - Legal shapes: bits in {1,2,3,4} for pack/unpack, {2,3,4} for the matmuls;
 *     group in {32,64,128}; K % 128 == 0; N % 8 == 0.  Anything else: TMAN_ERR_SHAPE /
 *     TMAN_ERR_UNSUPPORTED.
 */
#ifndef TMAN_H_
#define TMAN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Same type as the CUDA runtime's cudaStream_t (an opaque CUstream_st pointer). */
typedef struct CUstream_st *tman_stream_t;

typedef enum {
    TMAN_OK = 0,
    TMAN_ERR_NULL = 1,             /* a required pointer is NULL */
    TMAN_ERR_SHAPE = 2,            /* K, N, M, bits or group outside the legal set */
    TMAN_ERR_UNSUPPORTED = 3,      /* legal for the format, not for this call */
    TMAN_ERR_BUFFER_TOO_SMALL = 4, /* packed buffer or workspace smaller than required */
    TMAN_ERR_BAD_PACKED = 5,       /* (device-side) header does not match the arguments */
    TMAN_ERR_CUDA = 6,             /* a CUDA runtime/driver call or a launch failed */
    TMAN_ERR_TIMEOUT = 7,          /* (device-side) a bounded wait ran out */
    TMAN_ERR_LAYOUT = 8            /* (device-side) shared memory does not start where the kernel was built to expect */
} tman_status;

/* Human-readable name of a status code (host pointer to a static string). */
const char *tman_status_string(int status);

/* Library version, 1000*major + minor. */
int tman_version(void);

/* ---- sizes (host only, no GPU touched) ------------------------------------------------ */

/* Bytes of the packed weight buffer (256-byte header + bit-plane words + scales + zeros,
 * each section padded to 256 bytes).  Paper Sec. 4.1: one bit-serial copy of the weights
 * serves both decode and prefill. */
tman_status tman_packed_bytes(int K, int N, int bits, int group, size_t *out_bytes /*host*/);

/* Bytes of scratch a call needs.  op: 0 = tman_mpgemv, 1 = tman_mpgemm, 2 = unpack / debug
 * extractors and the other calls that only need the status word, 3 = tman_mpgemv_ternary.  For op 0 the size depends on M: it is what the fastest plan for M rows wants;
 * tman_mpgemv also accepts any workspace of at least the M = 1 size and then makes more passes over the
 * weights with fewer rows each (see tman_debug_gemv_plan).  The workspace must have been cleared once with tman_workspace_init before its
 * first use; calls leave it ready for the next call.  Two calls that overlap on the GPU must
 * not share a workspace. */
tman_status tman_workspace_bytes(int op, int M, int K, int N, int bits, int group,
                                 size_t *out_bytes /*host*/);

/* Prepare a workspace: status word zero, partial-sum area marked "no sum pending".  After a call
 * reported TMAN_ERR_TIMEOUT the workspace must be prepared again. */
tman_status tman_workspace_init(void *workspace, size_t ws_bytes, tman_stream_t stream);

/* Copy the workspace's status word to *out_status (host) and wait for `stream`. */
tman_status tman_read_status(const void *workspace, int *out_status /*host*/,
                             tman_stream_t stream);

/* ---- offline repack (paper Sec. 4.1 "Unified Layout", Sec. 2.2 bit-serial decomposition) -- */

/* codes  uint8 [K][N], one code per byte, values in [0, 2^bits)
 * scales fp16  [K/group][N]
 * zeros  uint8 [K/group][N], values in [0, 2^bits)
 * packed: output, packed_bytes >= tman_packed_bytes(...), 256-byte aligned.
 * Layout written (little endian):
 *   header (256 B): "TMANB200", u32 version=2, u32 K, N, bits, group, lut_g=4,
 *                   u64 planes_off, scales_off, zeros_off, total_bytes
 *   planes: u32 word[((nb*bits + i)*(K/32) + v)*4 + c], n = 4*nb + c; the word holds bit i of the 32
 *           codes q[32*v .. 32*v+31][n], permuted: weight 32*v + 8*ph + j sits at bit 4*j + ph
 *           (ph < 4, j < 8).  Byte e of the word is an 8-bit table index over the activations
 *           32*v + 8*ph + 2*e + hi (index bit 4*hi + ph); its nibbles are 4-bit indices in the
 *           paper's sense.  The permutation is what lets the prefill path rebuild codes in k order.
 *   scales: fp16 [((nb*(K/group) + B)*4 + c]
 *   zeros : u16  [nb*(K/group) + B], nibble c = z[B][4*nb + c]                              */
tman_status tman_pack_weights(const uint8_t *codes, const void *scales_f16, const uint8_t *zeros,
                              int K, int N, int bits, int group,
                              void *packed, size_t packed_bytes, tman_stream_t stream);

/* Inverse of tman_pack_weights (for round-trip checks).  Header mismatch -> status word. */
tman_status tman_unpack_weights(const void *packed, size_t packed_bytes,
                                int K, int N, int bits, int group,
                                uint8_t *codes, void *scales_f16, uint8_t *zeros,
                                void *workspace, size_t ws_bytes, tman_stream_t stream);

/* ---- the two matmuls:  y[M][N] (fp16, row-major) = x[M][K] (fp16, row-major) . W ----------
 * packed_bytes is the size of the caller's packed allocation; it must be at least
 * tman_packed_bytes(K, N, bits, group) (else TMAN_ERR_BUFFER_TOO_SMALL).  With that guarantee the
 * kernels may start streaming weights before the header check has completed; a header that does
 * not match the arguments still leaves y untouched and sets the status word.
 *
 * Stream order of the packed buffer.  The decode calls are launched so that they may begin while
 * the kernel before them on `stream` is still draining (programmatic dependent launch), and they
 * read the packed buffer in that window.  What is safe without further care: a packed buffer
 * written by tman_pack_weights on the same stream (the library puts the next decode call in plain
 * stream order), by a memory copy, or by any kernel that does not signal early completion.  What
 * is not: a kernel of the caller's own that calls cudaTriggerProgrammaticLaunchCompletion (PTX
 * griddepcontrol.launch_dependents) and then writes the packed buffer, directly followed by a decode
 * call on the same stream -- put an event or another kernel between them.  Activations and the
 * workspace have no such rule: they are read only after the predecessor has completed. */

/* Decode (paper Sec. 2.2 "Bit-serial table lookup", Fig. 2; Sec. 4.3): activation tables are
 * built in shared memory, packed bit-plane bytes index them, partial sums are
 * shift-accumulated per quantization block, scaled, and summed across blocks in fp32.
 * M in [1, 8], normally in one pass over the weights.  Precision: one row -- fp32 table entries and
 * sums.  Two to eight rows -- each row of a K-slice is scaled by a power of two into [1, 2) (exactly
 * undone at the end), table entries are rounded to fp16 and the bits x 4 lookups of a 32-activation word
 * are added in fp16, everything after in fp32 (the paper's 16-bit table entries and low-precision
 * aggregation inside a block, Sec. 4.3, Sec. 5): error at most about 1.5e-3 of the largest output,
 * whatever the activations' magnitude, against 4e-4 for one row. */
tman_status tman_mpgemv(const void *packed, size_t packed_bytes, const void *x_f16, void *y_f16,
                        int M, int K, int N, int bits, int group,
                        void *workspace, size_t ws_bytes, tman_stream_t stream);

/* Decode for `count` (1..4) weight matrices that read the same activations, in one launch (paper
 * Sec. 5 "Implementation", graph optimisation: the table precomputation is shared by the
 * projections with a common input, e.g. Q/K/V or gate/up).  All matrices have the same K, bits and
 * group; matrix g has N[g] output columns and its own packed buffer and output y_f16[g]
 * ([M][N[g]], fp16).  packed, packed_bytes, y_f16 and N are HOST arrays of `count` entries (read
 * during the call); their entries follow the rules of tman_mpgemv.  The workspace must hold
 * tman_workspace_bytes(0, M, K, N[0] + ... + N[count-1], bits, group). */
tman_status tman_mpgemv_grouped(int count, const void *const *packed /*host*/, const size_t *packed_bytes /*host*/,
                                const void *x_f16, void *const *y_f16 /*host*/, int M, int K, const int *N /*host*/,
                                int bits, int group, void *workspace, size_t ws_bytes, tman_stream_t stream);

/* ---- integer path: per-tensor ternary weights with 16-bit integer activations -------------------
 * (paper Sec. 6.1 "Models and Quantization": BitNet's ternary weights, quantized per tensor, are treated
 * as 2-bit, W_INT2 A_INT16; Sec. 4.3: integer aggregation inside the quantization block -- here the whole
 * tensor -- and floating point after it.)
 *
 * Weights: codes q = t + 1 in {0, 1, 2} for t in {-1, 0, +1}, packed by tman_pack_weights with bits = 2
 * (any legal group; the buffer's scales and zero-points are not read: zero-point 1 and the one scale
 * w_scale are implied). */

/* Per-row symmetric quantization of activations: row_scale[m] = max_k |x[m][k]| / qmax (1 for a row of
 * zeros), a[m][k] = round(x[m][k] / row_scale[m]) clamped to +-qmax; division and rounding (to nearest
 * even) in single precision.  qmax = 32767 (decode) or 127.  a_i16: int16 [M][K]; row_scale: fp32 [M].
 * x_f16 and a_i16 are 16-byte aligned (TMAN_ERR_SHAPE otherwise). */
tman_status tman_quantize_rows(const void *x_f16, int M, int K, int qmax, int16_t *a_i16, float *row_scale,
                               tman_stream_t stream);

/* Decode of M rows (1 <= M <= 8, in passes of up to four rows; K <= 16384): the bit-serial table lookup of
 * tman_mpgemv on integers.  Tables hold exact integer sums of activations, lookups are shift-accumulated,
 * the activation sum is subtracted once (zero-point 1), K-slices are added as 32-bit integers;
 *   y[m][n] = fp16( row_scale[m] * w_scale * sum_k a[m][k] * (q[k][n] - 1) ).
 * acc_i32 (device, int32 [M][N], 16-byte aligned, may be NULL) receives the exact integer sums.
 * Workspace: tman_workspace_bytes(3, M, K, N, 2, group), prepared with tman_workspace_init; status word
 * as for tman_mpgemv. */
tman_status tman_mpgemv_ternary(const void *packed, size_t packed_bytes, const int16_t *a_i16,
                                const float *row_scale, float w_scale, void *y_f16, int32_t *acc_i32,
                                int M, int K, int N, int group,
                                void *workspace, size_t ws_bytes, tman_stream_t stream);

/* The same row quantization with 8-bit output (qmax = 127) for the prefill side.  a_i8: int8 [M][K],
 * 16-byte aligned. */
tman_status tman_quantize_rows_i8(const void *x_f16, int M, int K, int8_t *a_i8, float *row_scale,
                                  tman_stream_t stream);

/* Prefill of the integer path (paper Sec. 6.2 "mpGEMM": per-tensor weights are dequantized to INT8 for the
 * matrix unit; Sec. 4.1 / Fig. 7 two-level lookup; Sec. 4.2 / Fig. 9 three pipelined agents): packed
 * ternary tiles are staged by TMA, rebuilt as INT8 tiles by bit repacking and a four-entry conversion
 * table, and multiplied with the 8-bit activations on the tensor cores with 32-bit integer accumulators;
 *   y[m][n] = fp16( row_scale[m] * w_scale * sum_k a[m][k] * (q[k][n] - 1) ),  M >= 1.
 * packed: as for tman_mpgemv_ternary.  workspace: at least 256 bytes (status word). */
tman_status tman_mpgemm_ternary_i8(const void *packed, size_t packed_bytes, const int8_t *a_i8,
                                   const float *row_scale, float w_scale, void *y_f16, int M, int K, int N,
                                   int group, void *workspace, size_t ws_bytes, tman_stream_t stream);

/* Prefill side of the integer path, the dequantization step alone (paper Sec. 6.2 "mpGEMM": per-tensor
 * weights are dequantized to INT8 for the matrix unit; Sec. 4.1 / Fig. 7: by two table lookups, bit
 * repacking and a conversion table, here with the INT8 values -1, 0, +1 as the table's entries).
 * w8_nk: output, int8 [N][K] (channel-major, 16-byte aligned).  workspace: at least 256 bytes (status
 * word: a header that does not match leaves the output untouched).  tman_mpgemm_ternary_i8 does the same
 * lookups inside its pipeline; this call exists to check them bit for bit and to time them alone. */
tman_status tman_dequant_ternary_int8(const void *packed, size_t packed_bytes, int K, int N, int group,
                                      int8_t *w8_nk, void *workspace, size_t ws_bytes, tman_stream_t stream);

/* Prefill (paper Sec. 4.1 two-level LUT dequantization, Fig. 7; Sec. 4.2 three-stage pipeline,
 * Fig. 9): packed tiles are staged in shared memory, rebuilt into fp16 tiles through the
 * repack step and the per-(block, column) conversion table, and multiplied on the tensor
 * cores with fp32 accumulation.  M >= 1.
 *   - The output is cut into tiles dealt to the SMs; when the tiles do not go round evenly, or
 *     are too few to fill the machine, the k-range of tiles is divided among the SMs and summed,
 *     in a fixed order, through fp32 partial tiles in the workspace (tens of MB: ask
 *     tman_workspace_bytes(1, ...)).  The result does not depend on timing: the same call gives
 *     the same bits.
 *   - All CTAs of the call must be able to run at the same time (at most one per SM is
 *     launched); if another kernel holds SMs for longer than a second while this one runs,
 *     the call gives up with TMAN_ERR_TIMEOUT in the status word instead of waiting on. */
tman_status tman_mpgemm(const void *packed, size_t packed_bytes, const void *x_f16, void *y_f16,
                        int M, int K, int N, int bits, int group,
                        void *workspace, size_t ws_bytes, tman_stream_t stream);

/* Decode without a caller-supplied workspace.  (No counterpart in the paper: this call exists for
 * the way the library is embedded, not for the method.)
 *
 * For callers that may not allocate device memory when they need a matmul -- a runtime that fixed
 * its arena at start-up, code running inside another framework's callback, a region where the
 * allocator is locked -- and so cannot produce the workspace tman_mpgemv asks for.  The scratch
 * is a fixed 4 MiB array inside the library image; every GPU that loads the library holds it
 * until the process exits, and this call allocates and frees nothing.
 *
 *   - Same result as tman_mpgemv for the same arguments (same kernels, same summation order).
 *   - A shape whose scratch, tman_workspace_bytes(0, M, K, N, bits, group), exceeds 4 MiB is
 *     refused with TMAN_ERR_BUFFER_TOO_SMALL before anything is enqueued.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents: each
 *     call first clears the part that must start at zero.  Two calls that overlap on the GPU
 *     (different streams without an ordering between them) race on it and give wrong results;
 *     calls on one stream, or ordered by events, are fine.
 *   - status_dev: device pointer to 4 bytes owned by the caller, or NULL.  When given, the
 *     device-side status word (0, TMAN_ERR_BAD_PACKED, ...) is copied there on `stream` after the
 *     kernels. */
tman_status tman_mpgemv_static(const void *packed, size_t packed_bytes, const void *x_f16,
                               void *y_f16, int M, int K, int N, int bits, int group,
                               unsigned int *status_dev, tman_stream_t stream);

/* ---- test-only extractors of the integer / table intermediates -------------------------- */

/* idx uint8 [bits][K/4][N]: the 4-bit table index of every (plane, 4 activations, column)
 * as the kernels read it out of the packed buffer (paper Sec. 4.1 "4-bit LUT index"). */
tman_status tman_debug_indices(const void *packed, int K, int N, int bits, int group,
                               uint8_t *idx, void *workspace, size_t ws_bytes,
                               tman_stream_t stream);

/* lut fp32 [M][K/4][16]: lut[m][t][p] = sum_{j<4} x[m][4t+j] * bit_j(p), computed by the same
 * device routine the decode kernel builds its tables from (paper Sec. 2.2). */
tman_status tman_debug_luts(const void *x_f16, int M, int K, float *lut, tman_stream_t stream);

/* tman_mpgemm with one part of the method replaced, for the ablations of paper Sec. 6.5 ("Efficiency of
 * the LUT-dequant kernel": against converting with floating-point instructions and against loading
 * full-precision weights; "Gain from pipelined execution": against doing load, dequantization and
 * multiplication in turn).  Every variant returns the same y as tman_mpgemm (same bits); only the time
 * differs.  Arguments as tman_mpgemm, plus
 *   variant 0  the product path (two-level lookup dequantization, pipelined)
 *           1  ConvertDQ: every code converted to fp16 with an integer-to-float instruction, zero-point
 *              subtracted, scale multiplied
 *           2  LoadFull: no dequantization; fp16 weights wt_f16 [N][K] (device, 16-byte aligned, row n =
 *              fp16(s * (q - z)) of channel n) are loaded by TMA in place of the packed tiles
 *           3  Sequential: the product's dequantization with a ring of one stage, so that the load, the
 *              dequantization and the multiplication of a k-block follow one another
 *   wt_f16  used by variant 2 only (else may be NULL).
 * Variants 1-3 exist for bits == 4 (TMAN_ERR_UNSUPPORTED otherwise); variant 2 additionally wants N to be a
 * multiple of 32 (TMAN_ERR_UNSUPPORTED otherwise). */
tman_status tman_debug_mpgemm_variant(int variant, const void *packed, size_t packed_bytes, const void *x_f16,
                                      void *y_f16, int M, int K, int N, int bits, int group, const void *wt_f16,
                                      void *workspace, size_t ws_bytes, tman_stream_t stream);

/* Role time stamps of the last tman_mpgemm call on `workspace` (paper Sec. 4.2, Fig. 9: how long each
 * of the three pipeline agents waits for the others).  Only a library built with -DTMAN_ROLE_STAMPS
 * (python -m paper_2511_11248_b200.build --stamps -> libtman_stamps.so) records them: clock readings
 * around every role's barrier waits, nothing else changes and the results are the same bits; the
 * regular library returns TMAN_ERR_UNSUPPORTED.  out_host: ctas x 26 warps x 4 int64 (host): clocks
 * in the warp's first kind of wait, in its second kind, in the whole role, and a tag.  Warp 0 (TMA
 * producer) waits for a free stage; warp 1 (MMA issuer) for free accumulators / for a dequantized stage;
 * warps 2-17 (dequantization) for a loaded stage; warps 18-25 (epilogue) for complete accumulators.
 * Waits for the stream. */
tman_status tman_debug_role_stamps(const void *workspace, size_t ws_bytes, int ctas, long long *out_host /*host*/,
                                   tman_stream_t stream);

/* How tman_mpgemm would cut a call's work on the current device (host-side decision, nothing is
 * launched; no counterpart in the paper).  out8 (host) receives: 1 if pairs of CTAs work on a tile
 * else 0; 128-token row blocks per CTA; row tiles; column tiles; 1 if every tile is dealt whole
 * else 0; workers (CTAs or pairs) launched; number of last tiles whose k-blocks are dealt as equal
 * spans (0: none); pieces every tile's k-blocks are split into (0: not split).  Tests use it to
 * know which path a shape takes. */
tman_status tman_debug_gemm_plan(int M, int K, int N, int bits, int group, int *out8 /*host*/);

/* The same decision for a device described by the caller: `sms` multiprocessors, of which `resident`
 * workers (CTAs, or CTA pairs when pairs are used) of the kernel can run at the same time.  The
 * workers of a call wait for one another's partial tiles, so a call never launches more than
 * `resident` of them; tman_mpgemm takes that number from the occupancy query of the kernel it is about
 * to launch.  Pure host arithmetic: needs no GPU. */
tman_status tman_debug_gemm_plan_for(int M, int K, int N, int bits, int group, int sms, int resident,
                                     int *out8 /*host*/);

/* How tman_mpgemv would serve a call of M rows (paper Sec. 4.3 and Sec. 5 "Implementation": the tiling
 * of the lookup kernel is searched under the hardware's limits; here the searched space is the kernel
 * variants the library carries).  Host arithmetic only, nothing is launched, needs no GPU.  A variant
 * carries 1, 2, 4 or 8 activation rows per pass over the weights (table entries of one fp32 row or of
 * 1, 2 or 4 fp16 row pairs) in K-slices of 16, 32, 16 or 8 plane words.  A variant is admitted when its
 * K-slices can all be resident (`sms` multiprocessors), its tables fit an SM's shared memory and its
 * partial sums fit `ws_limit` bytes (0: no limit); among the admitted ones the passes with the least
 * modelled time (fixed cost per pass + per-megabyte cost of the bit planes, fitted to measurements) are
 * chosen.  out (host, 52 ints): [0] passes (0: none admissible -> TMAN_ERR_UNSUPPORTED), [1] workspace
 * KiB the plan needs, [2] modelled time in ns, then six ints per pass from out[4]: rows carried, rows the
 * variant can carry, plane words per K-slice, K-slices, CTAs launched, shared-memory bytes per CTA. */
tman_status tman_debug_gemv_plan(int M, int K, int N, int bits, int group, int sms, size_t ws_limit,
                                 int *out /*host*/);

/* Lets a bounded wait run out, safely: one warp waits, with the same routine the decode kernel's split-K
 * combine uses, for partial sums that nothing writes (the workspace must be freshly prepared), gives up
 * after `polls` polls (1 .. 2^20, a few hundred nanoseconds each) and reports TMAN_ERR_TIMEOUT in the
 * status word like the decode kernel would.  The kernel always ends by itself.  workspace: at least
 * 256 + 512 bytes.  No counterpart in the paper. */
tman_status tman_debug_wait_timeout(void *workspace, size_t ws_bytes, unsigned int polls, tman_stream_t stream);

/* Microbenchmarks behind the decode kernel's design, the counterpart on this GPU of the paper's
 * instruction study (Sec. 5 "Implementation", Table 1: lookups per instruction x log2(table entries) =
 * "equivalent multiply-adds" of the 16- and 32-entry lookup instructions) and of its load-path study
 * (Table 2: DMA, prefetch and vector loads).  One kernel is enqueued per call; nothing of the product
 * path runs.
 *   kind 0..6  table-lookup loops, one CTA per SM, arg = threads per CTA (0: 512).  Tables: 0 = 256
 *              entries fp32, 1 = 256 entries fp16 with a mixed-precision add, 2 = 16 entries fp32 (the
 *              paper's table shape), 3 = 16 entries held in registers and read with a warp shuffle,
 *              4 / 5 / 6 = 256 entries that carry 2 / 4 / 8 activation rows in fp16.  results receives one
 *              u64 per CTA: the clocks its 64 passes over a 16 KB pool of index words took
 *              (1,048,576 index bytes per CTA: one lookup each for the 256-entry tables, two for the
 *              16-entry ones).
 *   kind 10    every CTA streams its share of buffer once with coalesced 16-byte loads (time it with
 *              events).  kind 11: the same with bulk asynchronous copies of arg bytes into a ring of
 *              shared-memory stages; a wait that runs out sets results[0] (u32) to TMAN_ERR_TIMEOUT.
 *   kind 20    clusters of arg CTAs: results[2i], results[2i+1] (u64) = clocks of a cluster barrier, and
 *              of a store to every peer's shared memory + barrier + read + barrier, for CTA i.
 *   kind 21    one thread follows a chain of dependent loads through arg bytes of buffer (kept in L2
 *              when small): results[0] (u64) = clocks per load.
 * results: device, 256-byte aligned, at least 4096 bytes (its last 256 bytes are scratch); buffer:
 * device, 256-byte aligned, may be NULL for kinds that do not read it. */
tman_status tman_debug_microbench(int kind, int arg, void *results, size_t results_bytes, void *buffer,
                                  size_t buffer_bytes, tman_stream_t stream);

/* How many clusters of `cluster` CTAs (threads, dynamic shared memory each) the current device
 * holds at once (host-side occupancy query, nothing is launched; no counterpart in the paper).  The
 * decode kernel combines its K-slices inside a cluster, so this number bounds its grid. */
tman_status tman_debug_cluster_capacity(int threads, int smem_bytes, int cluster, int *out_clusters /*host*/);

#ifdef __cplusplus
}
#endif
#endif /* TMAN_H_ */
