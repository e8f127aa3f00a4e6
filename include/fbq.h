/*
 * fbq.h -- C ABI of the B200 (sm_100a) FBQuant inference linear.
 *
 * The layer (paper: Algorithm 1 step 6, Z' = Q(W - BA) X^T + B A X^T with the
 * low-rank sub-branch Sigma = B.A of Section 4.2; Section 4.3 "Kernel Fusion"
 * describes the inference kernel this library replaces), for row-major tokens:
 *
 *     y[m][n] = sum_k x[m][k] * s[n][k/group] * ( q[n][k] - z[n][k/group] )
 *             + sum_j ( sum_k x[m][k] * A[j][k] ) * B[n][j]
 *
 *   x  M x K   activations           A  rank x K  down-projection
 *   q  N x K   3- or 4-bit codes     B  N x rank  up-projection
 *   s,z N x (K/group) fp16 scale and (integer-valued) zero point of each group of
 *       `group` consecutive input channels of one output row (Section 5.1: 128)
 *   y  M x N   written once, rounded to nearest even from fp32 accumulators
 *
 * General rules for every entry point
 *   - All matrices are dense row-major.  Unless a comment says HOST, pointers
 *     are DEVICE pointers owned by the caller; the library never frees or keeps
 *     them after the work queued on `stream` has run.  They must be 16-byte
 *     aligned.  y must not overlap any input.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls are asynchronous: the return value reports host-side validation and
 *     launch errors only.  Calls on one stream run in order; calls on different
 *     streams may run concurrently (each stream gets its own scratch space).
 *   - Return value: FBQ_OK or a negative fbq_status.
 *   - The library runs CUDA kernels only.  There is no CPU fallback: without a
 *     usable device every compute entry point returns FBQ_ERR_CUDA.
 *
 * Packed code formats (the paper does not define storage; these are fixed here)
 *   INT4  row n = K/8 consecutive uint32; code k in word k/8, bits 4*(k%8)..+3.
 *   INT3  row n = 3*K/32 consecutive uint32; each run of 32 codes c[0..31] is
 *         three words; word i (0..2): bits 3f..3f+2 = c[10i+f] and bits
 *         16+3f..16+3f+2 = c[10i+5+f] for f = 0..4; bit 15 = bit i of c[30];
 *         bit 31 = bit i of c[31].
 */
#ifndef FBQ_H
#define FBQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FBQ_OK = 0,
    FBQ_ERR_BADARG = -1,      /* NULL pointer, non-positive size, bits not 3/4, ...      */
    FBQ_ERR_UNSUPPORTED = -2, /* shape outside every kernel's domain                     */
    FBQ_ERR_ALIGN = -3,       /* a pointer is not 16-byte aligned                        */
    FBQ_ERR_CUDA = -4,        /* a CUDA runtime call failed (no device, launch error)    */
    FBQ_ERR_TIMEOUT = -5      /* device side: a bounded wait (on a copy, on another CTA's
                                 part of t) expired; read with fbq_poll_status           */
} fbq_status;

typedef enum {
    FBQ_KERNEL_NONE = -1,
    FBQ_KERNEL_GENERIC = 0,   /* any supported shape, CUDA cores, two launches if rank>0 */
    FBQ_KERNEL_DECODE = 1,    /* M <= 16 (chosen for M <= 8, and to 16 at rank 0): fused streaming kernels, one launch */
    FBQ_KERNEL_PREFILL = 2    /* tcgen05 / TMEM tensor-core kernel, one launch (chosen from M = 9, or 7 outside the streaming kernel's domain) */
} fbq_kernel;

/* Number of uint32 words of a packed N x K code matrix: N*K/8 (4 bits) or
 * 3*N*K/32 (3 bits).  Returns 0 for unsupported arguments (bits not 3/4, K not
 * a multiple of 8 resp. 32). */
size_t fbq_packed_words(int N, int K, int bits);

/* Pack one code per byte (codes: N x K uint8, values 0..2^bits-1; higher bits
 * are ignored) into the formats above.  Offline step of the weight-only
 * quantised storage (Section 1: weights kept in INT3/4). */
int fbq_pack_int4(const uint8_t *codes, uint32_t *qweight, int N, int K, void *stream);
int fbq_pack_int3(const uint8_t *codes, uint32_t *qweight, int N, int K, void *stream);

/* Inverse of the packers (test and tooling aid). */
int fbq_unpack(const uint32_t *qweight, uint8_t *codes, int N, int K, int bits, void *stream);

/* Dense fp32 weights W[n][k] = s*(q - z) of the group-wise linear quantiser
 * (Algorithm 1 "linear quantizer").  The product is exact in fp32.  scales and
 * zeros hold fp16 bit patterns.  Test and tooling aid; the linear entry points
 * never materialise W. */
int fbq_dequant(const uint32_t *qweight, const uint16_t *scales, const uint16_t *zeros,
                float *W, int N, int K, int group, int bits, void *stream);

/* The fused layer, fp16 activations: x, A, B, y are fp16; scales, zeros fp16.
 *   rank == 0: A and B are ignored (may be NULL); y is the main path alone.
 *   M == 0: nothing is done.
 * Dispatch (fbq_select_kernel tells which kernel a shape gets): group == 128 and rank a multiple of 8
 * not above 256 are the fast kernels' domain.  The streaming decode kernel ("gemv" option, default on)
 * needs N a multiple of 8, rank a multiple of 16 up to 128 and 16-byte aligned scales and zeros; there
 * it takes M <= 8 for every shape, and M <= 16 while M * K * 2 bytes stay within 136 KB (x of all K in
 * shared memory).  Elsewhere the other decode kernel
 * takes M <= 4 with rank <= 128 and M = 5, 6 with M * rank <= 128.  The prefill kernel (N a multiple of
 * 8) takes the rest of the domain; shapes outside its domain stay with a decode kernel up to M = 16;
 * everything else that is well formed -> generic kernel.
 * Well formed means bits in {3,4}, group a multiple of 8 (4 bits) or 32
 * (3 bits) dividing K, rank >= 0.  Zero points are taken as stored: every kernel accepts
 * integer-valued fp16 zero points of either sign and beyond 2^bits - 1 (what fbq_quantize_feedback
 * produces for groups that do not straddle zero); the decode and generic kernels any fp16 value.
 * Accumulation is fp32; t = x.A^T stays fp32 in the decode and
 * generic kernels (where a decode kernel multiplies it with B on tensor cores it enters as
 * two 16-bit terms, the rounded value and the remainder) and is rounded once to the activation
 * type in the prefill kernel (which also rounds the dequantised weights s*(q-z) once to that
 * type).  At M <= 2 the decode kernels read x in fixed point per group of 128, exact to 2^-17
 * of the group's largest element; a group that holds an Inf or a NaN makes its token's outputs NaN.
 * Summation order is fixed for a given shape and grid size (results are
 * reproducible run to run), except for t in the decode kernel of M >= 3, which is
 * accumulated with floating-point atomics.
 * Scratch and CUDA graphs: the library keeps scratch buffers per (device, stream) and grows them
 * the first time a stream sees a larger shape.  Growing allocates (and, for a buffer that exists,
 * synchronises the stream and frees the old one): a call that would have to grow scratch while
 * `stream` is being captured returns FBQ_ERR_UNSUPPORTED and queues nothing, and a graph captured
 * EARLIER on that stream keeps pointers to a buffer that a later, larger call replaces.  So: run
 * the largest shape of every kind once on a stream, outside capture, before capturing on it.
 * After FBQ_ERR_TIMEOUT the stream's counters are unfinished: call fbq_poll_status (it resets
 * them) before issuing more work on that stream. */
int fbq_linear(const void *x, const uint32_t *qweight, const void *scales, const void *zeros,
               const void *A, const void *B, void *y, int M, int N, int K, int group, int bits,
               int rank, void *stream);

/* Same layer with bf16 x, A, B and y (scales and zeros stay fp16). */
int fbq_linear_bf16(const void *x, const uint32_t *qweight, const void *scales,
                    const void *zeros, const void *A, const void *B, void *y, int M, int N,
                    int K, int group, int bits, int rank, void *stream);

/* End-to-end convenience: x_host (M x K) and y_host (M x N) are HOST buffers
 * (pinned memory makes the copies asynchronous); the weights stay on the
 * device.  Copies x to a per-stream staging buffer, runs the layer, copies y
 * back, all queued on `stream`; the caller synchronises the stream before
 * reading y_host.  act_is_bf16 selects fbq_linear_bf16. */
int fbq_linear_hostio(const void *x_host, const uint32_t *qweight, const void *scales,
                      const void *zeros, const void *A, const void *B, void *y_host, int M,
                      int N, int K, int group, int bits, int rank, int act_is_bf16,
                      void *stream);

/* (The paper has no counterpart: this entry point exists for integration reasons only.)
 * The same fused layer for callers that must not allocate device memory: a process that
 * gave all of it to its own pool at start-up, a latency-critical loop that cannot take the
 * device-wide synchronisation an allocation may imply, a plug-in whose host forbids driver
 * allocations after initialisation.  fbq_linear keeps its scratch space in buffers it
 * allocates per stream on first use; this variant runs the decode kernel with its scratch in
 * one fixed array that is part of the library image (about 2.1 MiB, held by every GPU that
 * loads the library until the process exits), and never calls an allocating routine.
 *   - Domain: the decode kernel's (M <= 16, group == 128, rank a multiple of 8 up to 256),
 *     and the scratch it needs must fit the array: N <= 65536 and roughly M * N * (number
 *     of K slices, 1 unless x is too large for shared memory) <= 524288.  Anything else
 *     returns FBQ_ERR_UNSUPPORTED and runs nothing; use fbq_linear for those.
 *   - The first call on each device looks up the array's device address (a cheap query, no
 *     allocation); make that first call outside any stream capture.
 *   - Every call uses the same array and begins by clearing the part that must start at
 *     zero (a memset queued on `stream`).  Calls that can overlap on the GPU (different
 *     streams, or several host threads) therefore race on it: run them one after another.
 *   - Arguments, layouts, dtypes (act_is_bf16 selects bf16 x, A, B, y) and results are
 *     those of fbq_linear / fbq_linear_bf16 with the "gemv" option off (the streaming kernel
 *     of M <= 2 is not served by the fixed array; the other decode kernel runs every M <= 16).
 *     The process-wide options apply ("pdl", "decode_i8", "decode_t_ctas", ...), except those
 *     that size scratch ("decode_ctas", "decode_sk"), which stay automatic.
 *   - A device-side time-out lands in a status word inside the array; fbq_poll_status(any
 *     stream) of that device returns it once (FBQ_ERR_TIMEOUT), clears it and resets the array.
 *     The per-call clearing leaves that word alone, so a time-out stays readable until polled. */
int fbq_linear_noalloc(const void *x, const uint32_t *qweight, const void *scales,
                       const void *zeros, const void *A, const void *B, void *y, int M, int N,
                       int K, int group, int bits, int rank, int act_is_bf16, void *stream);

/* Feedback quantiser, the offline producer of (codes, s, z) for the main path (Section 4.1:
 * the main path stores Q(W - Sigma) with Sigma = B.A, so that the reconstructed weight
 * W_F = Q(W - Sigma) + Sigma stays within s/2 of W for a round-to-nearest Q).  Per group of
 * `group` consecutive input channels of one output row, with r = W - B.A:
 *     s = max((max r - min r) / (2^bits - 1), 2^-14),  z = rint(-min r / s),
 *     q = clamp(rint(r / s + z), 0, 2^bits - 1),       ties to even
 * (a constant group c gets s = max(|c|, 2^-14), z = 1 if c < 0 else 0).  s and z are rounded
 * to fp16 and the stored values are the ones used for q.  All decisions are single-precision
 * IEEE operations in this order, Sigma accumulated with fused multiply-adds over the rank
 * index ascending.
 *   W      device, [N][K] fp32 (the weights to be quantised)
 *   A, B   device, [rank][K] and [N][rank], fp16 or bf16 (act_is_bf16); NULL when rank == 0
 *   codes  device, [N][K] bytes, one code per byte (feed them to fbq_pack_int3 / fbq_pack_int4)
 *   scales, zeros  device, fp16 [N][K/group]
 *   WF     device, [N][K] fp32 or NULL: receives W_F = s*(q - z) + Sigma
 * group: 1..1024 dividing K (a multiple of 8 (INT4) or 32 (INT3) if the codes are to be packed);
 * K/group <= 65535.  Asynchronous on `stream`; nothing is allocated.  Returns FBQ_OK,
 * FBQ_ERR_BADARG, FBQ_ERR_ALIGN or FBQ_ERR_CUDA. */
int fbq_quantize_feedback(const float *W, const void *A, const void *B, uint8_t *codes, void *scales,
                          void *zeros, float *WF, int N, int K, int group, int bits, int rank,
                          int act_is_bf16, void *stream);

/* Layer-wise reconstruction (Algorithm 1, Section 4.2): the offline loop that fits the sub-branch.
 * With H = X^T X of the layer's calibration activations X [T][K] (fbq_gram), one call of
 * fbq_reconstruct_step performs lines 5-9 of Algorithm 1 once:
 *     Delta_F = W - Q(W - B A) - B A          Q: the quantiser of fbq_quantize_feedback, detached
 *     loss    = tr(Delta_F H Delta_F^T)       = ||W X^T - W_F X^T||_F^2, before the update
 *     G       = -2 Delta_F H                  (the paper's dL/dSigma)
 *     A      <- A - lr B^T G,   B <- B - lr G A^T      (both from the old A and B)
 *   W [N][K], H [K][K], A [rank][K], B [N][rank]: device fp32 (A and B are the master copies and
 *   are updated in place); loss: device float or NULL; workspace: device,
 *   fbq_reconstruct_workspace_floats(N, K, rank) floats, contents meaningless afterwards.
 * The three dense products (and fbq_gram) are this library's own fp32 GEMM kernels (CUDA cores, fixed summation
 * order); no other library is loaded or called.  Initialise as Algorithm 1 says (A ~ N(0, sigma^2), B = 0), iterate, then
 * round A and B to the inference type and call fbq_quantize_feedback once more for (codes, s, z). */
size_t fbq_reconstruct_workspace_floats(int N, int K, int rank);
int fbq_gram(const float *X, float *H, int T, int K, void *stream);
int fbq_reconstruct_step(const float *W, const float *H, float *A, float *B, float lr, float *loss,
                         float *workspace, int N, int K, int group, int bits, int rank, void *stream);

/* Several independent linears of the same kind in one call: the grouped decode of a decoder
 * layer, where q, k, v (and gate, up) read the same x through different weights, or any set
 * of layers whose inputs are ready (Algorithm 1 reconstructs each of the seven projections
 * of a layer on its own; at inference those that do not depend on one another can run
 * together).  Problem i computes
 *     y_i = x_i . dequant(Q_i, s_i, z_i)^T + (x_i . A_i^T) . B_i^T
 * exactly as fbq_linear / fbq_linear_bf16 would with the shared M, group, bits, rank and
 * activation type; N and K are per problem.  No y_i may overlap another problem's inputs.
 *   - `problems` is a HOST array of `count` (<= FBQ_BATCH_MAX) descriptors of DEVICE
 *     pointers (layouts and alignment as for fbq_linear); it is read before the call returns.
 *   - When every problem is decode sized (M <= 16 and the decode kernel's domain) the
 *     problems run concurrently, each with a share of "batch_ctas" CTAs in proportion to its
 *     share of the codes, so that the whole batch is resident at once.  Up to 8 problems run
 *     as ONE launch of the decode kernel over a problem list, on `stream` ("batch_single" = 1,
 *     the default); more problems, or "batch_single" = 0, run one launch per problem on side
 *     streams of the library, forked from and joined to `stream` with events (legal under
 *     stream capture; make the first such call on a device outside a capture: it creates the
 *     side streams and events, which are kept until the process exits).  Either way work
 *     queued on `stream` after the call sees every y_i.
 *   - Otherwise the problems run one after the other on `stream`.
 * Returns the first error, or FBQ_OK. */
#define FBQ_BATCH_MAX 16
typedef struct fbq_problem {
    const void *x;            /* [M][K] */
    const uint32_t *qweight;  /* packed codes of [N][K] */
    const void *scales;       /* fp16 [N][K/group] */
    const void *zeros;        /* fp16 [N][K/group] */
    const void *A;            /* [rank][K] or NULL when rank == 0 */
    const void *B;            /* [N][rank] or NULL when rank == 0 */
    void *y;                  /* [M][N] */
    int N, K;
} fbq_problem;
int fbq_linear_batch(const fbq_problem *problems, int count, int M, int group, int bits, int rank,
                     int act_is_bf16, void *stream);
/* The same with every problem's x and y in HOST memory (pinned for asynchronous copies), the
 * weights on the device as before: per problem the library copies x to a staging buffer it
 * keeps per stream, runs the linear, and copies y back, all on the stream the problem runs on.
 * y is complete once work queued on `stream` after the call has run (synchronise `stream`
 * before reading it).  The end-to-end path of the benchmark. */
int fbq_linear_batch_hostio(const fbq_problem *problems, int count, int M, int group, int bits, int rank,
                            int act_is_bf16, void *stream);

/* Comparator, not a product path: the UNFUSED low-rank sub-branch of the paper's Section 3.2 / Fig. "kernel-fusion"
 * (the quantised main path plus separate launches for the branch), which Section 4.3's fused kernel replaces.
 * After fbq_linear with rank 0 has written y = x.dequant(Q)^T, this call adds the branch with three launches of
 * its own: t = x.A^T (fp32), u = t.B^T (rounded to the activation type, written out), y += u (y read and
 * written once more).  x [M][K], A [rank][K], B [N][rank], y [M][N]: device, fp16 or bf16 (act_is_bf16); rank >= 1.
 * The benchmark times it against the fused call; a test checks that it computes the same layer. */
int fbq_sub_branch_unfused(const void *x, const void *A, const void *B, void *y, int M, int N, int K,
                           int rank, int act_is_bf16, void *stream);

/* Which kernel fbq_linear / fbq_linear_bf16 would run for this shape, or
 * FBQ_KERNEL_NONE when the shape is rejected.  Pure host logic. */
int fbq_select_kernel(int M, int N, int K, int group, int bits, int rank, int act_is_bf16);

/* Tuning and test switches (host side, process wide).  Known names:
 *   "force_kernel"  -1 = automatic, else an fbq_kernel value (shapes outside the
 *                   forced kernel's domain still fall back to the generic one)
 *   "gemv"          1 (default) = M <= 2 runs the streaming decode kernel where its domain allows (see fbq_linear),
 *                   0 = the other decode kernel at every M
 *   "gemv_ctas"     0 = automatic (one main CTA per SM), else an upper bound on the streaming kernel's grid
 *   "t_poll_limit"  0 = default, else the number of looks the streaming kernel takes at the t CTAs' slots
 *                   before it gives up with FBQ_ERR_TIMEOUT
 *   "test_skip_t_arrive", "test_prefill_skip_flag", "prefill_flag_polls"
 *                   test switches of the failure-detection tests: the CTAs that compute t = x.A^T do not
 *                   report it (streaming decode kernel / prefill kernel), and the prefill kernel's number
 *                   of looks at its flag; with them a bounded wait runs out on purpose
 *   "decode_sk"     0 = automatic, else the number of K slices of the decode kernel
 *   "decode_chunk"  0 = automatic, else quantisation groups per smem stage
 *   "decode_depth"  0 = automatic, else stages in flight per warp
 *   "decode_ctas"   0 = automatic, else an upper bound on the decode grid size
 *   "decode_i8"     1 (default) = at M <= 2 the decode kernel takes the codes as unsigned bytes and x as three
 *                   signed base-256 digits per group scale through 8-bit integer MMAs (x exact to 2^-17 of its
 *                   group's largest element); 0 = the 16-bit form (x exact) at every M
 *   "decode_t_ctas" 1 (default) = at M <= 4 (one K slice) t = x.A^T is computed by a few CTAs at the head of the
 *                   grid and the others wait for it (bounded); 0 = every CTA contributes its share
 *   "decode_t_wait" 1 (default) = a finished tile may wait for t in shared memory while that holds nobody up,
 *                   0 = it is parked in scratch at once (only matters without t CTAs)
 *   "batch_ctas"    CTAs shared out among the problems of a decode-sized fbq_linear_batch (default 400)
 *   "prefill_pair"  1 = token tiles of 256 of the prefill kernel run on CTA pairs (cta_group::2 MMAs,
 *                   each CTA staging half of the token tile); 0 (default) = one CTA per tile, which
 *                   measured faster
 *   "prefill_split" the prefill kernel at M <= 128, where a shape has fewer 128-row tiles than SMs: K is cut
 *                   into up to 8 slices, one CTA each, which store fp32 partial tiles to the stream's scratch;
 *                   the CTA that finishes last adds them in slice order and writes y (results do not depend
 *                   on timing).  0 = never, 1 = only for K >= 8192, 2 (default) = whenever the tiles are
 *                   few (faster for linears that run one after another; when several run side by side on
 *                   streams of their own, 1 is faster)
 *   "batch_single"  1 = such a batch of up to 8 problems is one launch (default), 0 = one launch per problem
 *   "hostio_direct_y" 1 (default) = the host-buffer entry points let the kernel write a y of up to 256 KB straight
 *                   into the caller's buffer when that is pinned, GPU-addressable host memory (no copy queued
 *                   behind the kernel); 0 = y always goes through the stream's staging buffer and a copy
 *   "pdl"           1 = launch with programmatic dependent launch (default), 0 = plain.  With 1 a decode or
 *                   prefill kernel may start while the kernel before it on the stream still runs: it sets
 *                   itself up, and the decode kernels already fetch qweight, scales, zeros, A and B, before
 *                   they wait for that kernel; x, y and the scratch are touched only after the wait.  So
 *                   the weight operands must not be written by the launch directly before (x may be)
 *   "decode_t_late" test switch: 1 = contribute to t after the main loop, which drives
 *                   every tile through the parked-tile branch of the combine protocol
 *   "decode_trace"  tuning aid: 1 = the decode kernels record, per CTA and warp, a time stamp at
 *                   their phases, read with fbq_debug_read_trace.  The streaming kernel's marks
 *                   are compiled in only when the library is built with -DFBQ_GEMV_TRACE
 *                   (FBQ_EXTRA_NVCC_FLAGS of the build script); a normal build leaves its part of
 *                   the buffer zero
 * Options are plain process-wide integers read when a call is issued: set them before issuing work, not while
 * other host threads are inside the library.
 * Returns FBQ_OK or FBQ_ERR_BADARG for an unknown name.
 * (Tuning aid outside this interface: with the environment variable FBQ_PLAN set, every plan of the
 * decode kernel is printed to stderr: K slices, CTAs, stage size and count, shared-memory layout, form.) */
int fbq_set_option(const char *name, int value);
int fbq_get_option(const char *name, int *value);

/* Number of kernels the library has launched since load (all streams). */
long long fbq_launch_count(void);

/* Synchronises `stream` and returns the device-side status word of its scratch
 * space (or of the fixed array of fbq_linear_noalloc, if that one is set): FBQ_OK, or
 * FBQ_ERR_TIMEOUT if a bounded wait inside a kernel gave up (the affected outputs are then
 * undefined).  Reading clears the word and resets the counters the kernel left unfinished. */
int fbq_poll_status(void *stream);

/* Tuning aid: copies the phase marks of the last decode launch on `stream` (recorded while
 * "decode_trace" is 1) to host_buf.  The streaming kernel (in a -DFBQ_GEMV_TRACE build) writes uint64 [2][256 CTAs][10 warps][16 marks]
 * of global-timer values (ns), consecutive launches alternating between the two halves; the other
 * decode kernel uint64 [cta][10 warps][16 marks] of SM cycle counts with mark 15 of warp 0 the global
 * timer at kernel entry.  Zero where a mark was not reached.  bytes <= 512*18*16*8.  Synchronises the stream. */
int fbq_debug_read_trace(void *stream, void *host_buf, size_t bytes);

/* Frees every per-stream scratch buffer (synchronises the device first). */
int fbq_release_workspaces(void);

const char *fbq_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* FBQ_H */
