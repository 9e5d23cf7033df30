/* libmtmcfused -- B200 (sm_100a) fused linear layers:  Y = epilogue(X . W^T + b).
 *
 * The operator family is the "GEMM followed by an epilogue" class the paper's
 * Level-2 fused-operator tasks stand for (Table "Details of KernelBench and
 * TritonBench"; the Fusion, Tiling, Pipeline and Reordering principles of section
 * "Optimization Principles"); correctness is the paper's Eq. 1 constraint: the
 * result equals the high-level reference semantics of the operator sequence.
 *
 * Conventions shared by every entry point
 *   - extern "C"; every function returns an int status (MTMC_OK = 0).
 *   - X [M,K], W / Wg / Wu [N,K], out [M,N]: dense row-major.  "bf16" is the upper
 *     16 bits of an IEEE-754 binary32.  b is binary32 [N]; b == NULL means no bias.
 *   - Unless a function name ends in _host, every pointer is a DEVICE pointer on
 *     the current CUDA device, 16-byte aligned, owned by the caller, and must stay
 *     valid until the enqueued work has run.  Outputs must not alias inputs.
 *   - Work is enqueued on the stream set by mtmc_set_stream() (default: the
 *     legacy default stream) and the call returns without synchronising.
 *     Argument errors are reported synchronously and enqueue nothing.  A device
 *     side bounded wait that expires sets a sticky status that
 *     mtmc_check_status() returns after synchronising the stream.
 *   - Shapes: M, N, K >= 1 and K % 8 == 0 (a row of X or W must be a multiple of
 *     16 bytes for the TMA descriptors).  Tails in M, N and K (K % 64 != 0) are
 *     handled by TMA zero fill and predicated stores.  M, N, K < 2^31.
 *   - Only compute capability 10.x is accepted; there is no fallback of any kind.
 *   - Results are bit-reproducible run to run for a fixed shape and device.
 *   - Scratch: split-K partial sums and logsumexp partials live in a workspace.
 *     By default the library owns one per (device, stream) (cudaMalloc, grow-only;
 *     so the first call of a larger shape on a stream allocates and must not run
 *     under stream capture); mtmc_set_workspace() substitutes caller-owned memory.
 *   - Threads and streams: the stream, workspace, tuning and timing settings are
 *     thread-local.  Calls enqueued on different streams, from one host thread or
 *     from several, may overlap on the GPU: their library-owned scratch is
 *     separate (at most 32 streams per device use it; further ones need
 *     mtmc_set_workspace).  Calls on ONE stream run in order and share that
 *     stream's scratch; two host threads that enqueue on the same stream must
 *     order their calls themselves, as for any CUDA stream.
 */
#ifndef MTMC_FUSED_H_
#define MTMC_FUSED_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* status codes */
#define MTMC_OK 0
#define MTMC_ERR_INVALID_ARG 1        /* null / misaligned pointer, M/N/K <= 0, unknown enum */
#define MTMC_ERR_UNSUPPORTED_SHAPE 2  /* K % 8 != 0, or a dimension >= 2^31 */
#define MTMC_ERR_UNSUPPORTED_DEVICE 3 /* not compute capability 10.x */
#define MTMC_ERR_CUDA 4               /* CUDA runtime / driver error; text in mtmc_last_error() */
#define MTMC_ERR_DEVICE_TIMEOUT 5     /* a bounded device-side wait expired */
#define MTMC_ERR_WORKSPACE 6          /* caller-provided workspace too small */
#define MTMC_ERR_DEVICE_CHECK 7       /* -DMTMC_CHECKS builds only: a device-side index check failed (the access was skipped) */

/* activation ids for mtmc_fused_linear */
#define MTMC_ACT_NONE 0
#define MTMC_ACT_RELU 1
#define MTMC_ACT_GELU_TANH 2 /* 0.5 z (1 + tanh(sqrt(2/pi) (z + 0.044715 z^3))) */
#define MTMC_ACT_SILU 3      /* z / (1 + exp(-z)) */

/* output element types for mtmc_fused_linear */
#define MTMC_OUT_FP32 0
#define MTMC_OUT_BF16 1 /* round to nearest even, once, at the final store */

/* operation ids for mtmc_workspace_bytes */
#define MTMC_OP_FUSED_LINEAR 0
#define MTMC_OP_SWIGLU 1
#define MTMC_OP_LINEAR_LSE 2
#define MTMC_OP_LINEAR_ROWMAX 3
#define MTMC_OP_LINEAR_CROSS_ENTROPY 4
#define MTMC_OP_FUSED_LINEAR_MXFP8 5
#define MTMC_OP_SWIGLU_MXFP8 6
#define MTMC_OP_LINEAR_LSE_MXFP8 7
#define MTMC_OP_LINEAR_SOFTMAX 8

/* out[m][n] = act( sum_k X[m][k] W[n][k] + b[n] ).
 * (Fused GEMM + bias + activation: the Fusion principle applied to a linear layer;
 * the bias add and activation happen in fp32 on the fp32 accumulator, with no
 * intermediate rounding.)  X, W bf16; b fp32 or NULL; out fp32 or bf16 [M,N]
 * according to out_dtype.  Shapes with M <= 64 (decode batches) whose W has at
 * least 64 rows per CTA pair take the split-K weight-streaming path (HBM-bound);
 * problems of at most half a wave of 128 x 256 (or 128 x 128) tiles with a long K a
 * cluster split-K kernel (2, 4 or 8 CTAs per tile, reduction through distributed
 * shared memory); all others the tiled tensor-core kernels (CTA pairs on 256 x 256
 * tiles from M > 128 and N >= 256 on, 512 x 256 tiles for very long K, single CTAs
 * otherwise).  Needs workspace only on the ticketed variant of the
 * weight-streaming path (few rows of W, or a forced split; see mtmc_workspace_bytes). */
int mtmc_fused_linear(const void* X, const void* W, const float* b,
                      int64_t M, int64_t N, int64_t K, int act, int out_dtype, void* out);

/* out[m][n] = act( sum_k X[m][k] W[n][k] + b[n] ) + R[m][n].
 * (The layer's skip connection joined to the epilogue, e.g. the MLP down-projection that
 * follows mtmc_swiglu: one more elementwise pass over [M,N] that never happens.)  R is [M,N]
 * in the OUTPUT's element type (fp32 or bf16 according to out_dtype), 16-byte aligned; the
 * sum is formed in fp32 and rounded once.  out may be the same buffer as R (in-place
 * update of the residual stream); any other overlap is not allowed. */
int mtmc_fused_linear_residual(const void* X, const void* W, const float* b, const void* R,
                               int64_t M, int64_t N, int64_t K, int act, int out_dtype, void* out);

/* mtmc_fused_linear on row-major views that are not dense: rows of X, W and out lie ldx, ldw
 * and ldo elements apart (a column slice of a wider matrix, one projection inside a fused
 * QKV weight, an output written straight into a concatenated buffer).  ldx, ldw >= K and
 * multiples of 8 (TMA wants 16-byte row pitches); ldo >= N, any value -- vector stores need
 * ldo % 8 == 0 (bf16) or ldo % 4 == 0 (fp32), otherwise rows are written element by element.
 * Everything else as for mtmc_fused_linear: same kernels, same results.  The paper's operators
 * take framework tensors, which may be such views. */
int mtmc_fused_linear_strided(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* b,
                              int64_t M, int64_t N, int64_t K, int act, int out_dtype, void* out, int64_t ldo);

/* The other operators on row-major views, with the same rules (ldx, ldw... >= K and multiples of 8; ldo >= N,
 * any value): mtmc_swiglu with X, Wg, Wu and out as column slices of wider matrices (the gate and up projections
 * stored side by side in one fused weight, the output written into a concatenated buffer), and the three row
 * reductions with X and W as views (their outputs are dense vectors).  Same kernels, same bits as the dense calls. */
int mtmc_swiglu_strided(const void* X, int64_t ldx, const void* Wg, int64_t ldwg, const void* Wu, int64_t ldwu,
                        int64_t M, int64_t N, int64_t K, void* out, int64_t ldo);
int mtmc_linear_lse_strided(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* b,
                            int64_t M, int64_t N, int64_t K, float* lse_out);
int mtmc_linear_rowmax_strided(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* b,
                               int64_t M, int64_t N, int64_t K, float* max_out, int32_t* argmax_out);
int mtmc_linear_cross_entropy_strided(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* b, const int64_t* targets,
                                      int64_t M, int64_t N, int64_t K, float* loss_out, float* lse_out);

/* The same layer with 8-bit floating-point operands:
 *   out[m][n] = act( scale_x * scale_w * sum_k X8[m][k] W8[n][k] + b[n] ).
 * X8 [M,K] and W8 [N,K] hold E4M3 values (1 sign, 4 exponent bits with bias 7, 3 mantissa
 * bits, no infinities; one byte per element, dense row-major); scale_x, scale_w are the
 * per-tensor scales (real value = scale * stored value), passed by value.  Products are
 * exact and accumulate in fp32 on the tensor cores (tcgen05 kind::f8f6f4, K = 32 per MMA,
 * twice the bf16 rate); the epilogue is the one of mtmc_fused_linear.  K % 16 == 0.  As
 * for bf16, M <= 64 takes the weight-streaming split-K path (half the bytes of bf16
 * weights), larger M the tiled kernels. */
int mtmc_fused_linear_fp8(const void* X8, const void* W8, const float* b, float scale_x, float scale_w,
                          int64_t M, int64_t N, int64_t K, int act, int out_dtype, void* out);

/* The SwiGLU gate and the row logsumexp with E4M3 operands, on the same kernels as their bf16
 * forms (layout, K % 16 == 0 and scale conventions as for mtmc_fused_linear_fp8):
 *   mtmc_swiglu_fp8     : out = silu(scale_x*scale_g * X8.Wg8^T) * (scale_x*scale_u * X8.Wu8^T),
 *                         bf16 [M,N]; gate and up projection carry their own per-tensor scales
 *   mtmc_linear_lse_fp8 : lse_out[m] = log sum_n exp(scale_x*scale_w * X8.W8^T + b), fp32 [M]
 * The paper's operators are bf16/fp16/fp32; these are the lower-precision forms of the same
 * fused epilogues. */
int mtmc_swiglu_fp8(const void* X8, const void* Wg8, const void* Wu8, float scale_x, float scale_g, float scale_u,
                    int64_t M, int64_t N, int64_t K, void* out);
int mtmc_linear_lse_fp8(const void* X8, const void* W8, const float* b, float scale_x, float scale_w,
                        int64_t M, int64_t N, int64_t K, float* lse_out);
/* mtmc_linear_rowmax and mtmc_linear_cross_entropy (below) with E4M3 operands, same conventions:
 * the logits are scale_x*scale_w * X8.W8^T + b. */
int mtmc_linear_rowmax_fp8(const void* X8, const void* W8, const float* b, float scale_x, float scale_w,
                           int64_t M, int64_t N, int64_t K, float* max_out, int32_t* argmax_out);
int mtmc_linear_cross_entropy_fp8(const void* X8, const void* W8, const float* b, float scale_x, float scale_w,
                                  const int64_t* targets, int64_t M, int64_t N, int64_t K, float* loss_out, float* lse_out);

/* Block-scaled 8-bit operands (the MXFP8 format of the OCP microscaling specification): E4M3 elements with one
 * power-of-two scale per 32 consecutive elements of K.  X8 [M,K] and W8 [N,K] hold the elements (one byte each,
 * dense row-major); SX [M, K/32] and SW [N, K/32] hold the scales, one byte each, dense row-major, in UE8M0
 * (a biased exponent: the scale is 2^(byte - 127); 255 is not a number and out of contract):
 *   z[m][n] = sum_k ( 2^(SX[m][k/32] - 127) X8[m][k] ) ( 2^(SW[n][k/32] - 127) W8[n][k] )
 *   mtmc_fused_linear_mxfp8 : out = act(z + b), fp32 or bf16
 *   mtmc_swiglu_mxfp8       : out = silu(z_gate) * z_up, bf16; gate and up weights with their own scales
 *   mtmc_linear_lse_mxfp8   : lse_out[m] = log sum_n exp(z[m][n] + b[n]), fp32
 * The scales differ from k-block to k-block, so they are applied inside the contraction, by the tensor cores
 * (tcgen05.mma kind::mxf8f6f4.block_scale with the scales in tensor memory); accumulation is fp32 and the
 * epilogues are those of the bf16 forms.  K % 32 == 0.  All shapes run on single-CTA tiles of 128 x 128.
 * Workspace: the scales re-arranged for the kernel, mtmc_workspace_bytes(MTMC_OP_..._MXFP8, M, N, K).
 * The paper's operators are bf16/fp16/fp32; these are the block-scaled low-precision forms of the same fused epilogues. */
int mtmc_fused_linear_mxfp8(const void* X8, const void* SX, const void* W8, const void* SW, const float* b,
                            int64_t M, int64_t N, int64_t K, int act, int out_dtype, void* out);
int mtmc_swiglu_mxfp8(const void* X8, const void* SX, const void* Wg8, const void* SG, const void* Wu8, const void* SU,
                      int64_t M, int64_t N, int64_t K, void* out);
int mtmc_linear_lse_mxfp8(const void* X8, const void* SX, const void* W8, const void* SW, const float* b,
                          int64_t M, int64_t N, int64_t K, float* lse_out);

/* out[m][n] = silu(sum_k X[m][k] Wg[n][k]) * (sum_k X[m][k] Wu[n][k]);  no bias;
 * out bf16 [M,N].  (Gated MLP up-projection: two GEMMs sharing X plus the gate
 * product fused in one kernel; neither GEMM result is written to memory.) */
int mtmc_swiglu(const void* X, const void* Wg, const void* Wu,
                int64_t M, int64_t N, int64_t K, void* out);

/* lse_out[m] = log sum_n exp( sum_k X[m][k] W[n][k] + b[n] ),  fp32 [M].
 * (A row reduction fused into a linear layer -- the paper's own example of a
 * semantic action is fusing a linear with a row maximum, section "Training
 * Process".  The M x N logits are never written to memory: each tile keeps an
 * online (max, sum-exp) per row, partials go to the workspace and are merged.)
 * Needs mtmc_workspace_bytes(MTMC_OP_LINEAR_LSE, M, N, K) bytes of workspace. */
int mtmc_linear_lse(const void* X, const void* W, const float* b,
                    int64_t M, int64_t N, int64_t K, float* lse_out);

/* max_out[m] = max_n ( sum_k X[m][k] W[n][k] + b[n] ), fp32 [M]; argmax_out[m] (int32 [M], may
 * be NULL) = the lowest column attaining it.  (The paper's example of a semantic action,
 * fusing a linear with a row maximum, section "Training Process".)  Same machinery as
 * mtmc_linear_lse: per-piece (max, column) partials in the workspace, merged per row.
 * Needs mtmc_workspace_bytes(MTMC_OP_LINEAR_ROWMAX, M, N, K) bytes of workspace. */
int mtmc_linear_rowmax(const void* X, const void* W, const float* b,
                       int64_t M, int64_t N, int64_t K, float* max_out, int32_t* argmax_out);

/* Softmax cross entropy of the never-materialised logits:
 *   loss_out[m] = lse[m] - ( sum_k X[m][k] W[targets[m]][k] + b[targets[m]] ),   fp32 [M];
 * lse_out (fp32 [M], may be NULL) also receives the row logsumexp.  targets is int64 [M] on the
 * device, 8-byte aligned; a target outside [0, N) makes that row's loss NaN.  (Fused LM-head
 * loss: the tile that holds a row's target column sets the logit aside while it accumulates the
 * row's (max, sum-exp).)  Needs mtmc_workspace_bytes(MTMC_OP_LINEAR_CROSS_ENTROPY, M, N, K). */
int mtmc_linear_cross_entropy(const void* X, const void* W, const float* b, const int64_t* targets,
                              int64_t M, int64_t N, int64_t K, float* loss_out, float* lse_out);

/* Row softmax of the logits, written out as probabilities:
 *   prob_out[m][n] = exp( z[m][n] - lse[m] ),  z[m][n] = sum_k X[m][k] W[n][k] + b[n],
 * [M,N] dense row-major, fp32 or bf16 (out_dtype: MTMC_OUT_FP32 / MTMC_OUT_BF16), device, 16-byte
 * aligned; lse_out (fp32 [M], device, may be NULL) also receives the row logsumexp.  (The
 * normalised form of the same row reduction: the logits themselves are never written.  The GEMM's
 * epilogue stores exp(z - max) with the maximum of the row's piece of the tile, which is at most 1
 * whatever the logits' size, and leaves the piece's (max, sum-exp) in the workspace; after the
 * merge (a launch of its own, or the first step of the last pass when a row has few pieces) one
 * pass over prob_out multiplies every piece by exp(max - lse).  A bf16 result therefore
 * carries two roundings of a value in [0, 1]: relative error up to 2^-8.)  N must be below
 * 2^31 - 1024.  bf16 operands.  Needs mtmc_workspace_bytes(MTMC_OP_LINEAR_SOFTMAX, M, N, K). */
int mtmc_linear_softmax(const void* X, const void* W, const float* b,
                        int64_t M, int64_t N, int64_t K, int out_dtype, void* prob_out, float* lse_out);
/* The same on row-major views (X, W rows ldx, ldw elements apart: >= K, multiples of 8; prob_out rows ldo >= N
 * elements apart, any value, e.g. the probabilities written into a wider buffer), and with E4M3 operands and
 * per-tensor scales (as mtmc_linear_lse_fp8: K % 16 == 0, z = scale_x * scale_w * sum_k X8 W8 + b).  Same kernels. */
int mtmc_linear_softmax_strided(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* b,
                                int64_t M, int64_t N, int64_t K, int out_dtype, void* prob_out, int64_t ldo, float* lse_out);
int mtmc_linear_softmax_fp8(const void* X8, const void* W8, const float* b, float scale_x, float scale_w,
                            int64_t M, int64_t N, int64_t K, int out_dtype, void* prob_out, float* lse_out);

/* Allocation-free variant of mtmc_linear_lse: same arguments, same result (same
 * kernels), but the (max, sum-exp) partials live in an 8 MiB array that is part of
 * the library image instead of a workspace from cudaMalloc.  (The paper has no
 * counterpart; this exists for callers that must not allocate.)
 *
 * Who needs it: code that runs where device memory is not theirs to ask for -- an
 * operator called from inside an inference server's request loop, where a
 * cudaMalloc would stall every stream of the device; a plug-in whose host
 * framework has already claimed the whole GPU for its own pool, so a raw
 * allocation fails or fragments it; a job with a fixed memory budget audited at
 * start-up.  This call makes no cudaMalloc / cudaFree and calls no allocating
 * library routine, on any call including the first.
 *
 * Limits and rules:
 *   - ceil(N / 256) * M  (ceil(N / 128) * M when N <= 128 or tile_n = 128 is
 *     forced) must not exceed 1,048,576 partials; larger shapes are rejected with
 *     MTMC_ERR_UNSUPPORTED_SHAPE and the message names mtmc_linear_lse instead.
 *     The benchmark's LM-head shape (M=4096, N=32000) needs 512,000.
 *   - Every GPU that loads the library holds the 8 MiB until the process exits.
 *   - The first call on each device performs a one-time set-up (device attribute
 *     queries, driver entry point lookup, cudaGetSymbolAddress of the scratch,
 *     one 4-byte synchronous copy).  Make that first call before starting any
 *     stream capture.
 *   - All calls on a device share the one array, which keeps whatever the last
 *     call left in it.  Nothing in it needs clearing: every slot a call reads
 *     has been written by that same call first.  Two calls that overlap on the
 *     GPU (different streams, or different host threads) race on it and give
 *     wrong results; serialise them on one stream.
 *   - Device-side timeouts of this path go to a status word of their own, also part
 *     of the library image; mtmc_check_status() reports and clears it like the
 *     regular one (and, in a process that has only ever used this entry point on
 *     the device, does so without creating the regular, allocating state). */
int mtmc_linear_lse_noalloc(const void* X, const void* W, const float* b,
                            int64_t M, int64_t N, int64_t K, float* lse_out);

/* Same three operations with every pointer a HOST pointer (pageable or pinned).
 * The library copies the operands to device buffers it owns (cudaMalloc,
 * grow-only, per device), runs the device entry point on the current stream,
 * copies the result back and waits for it before returning.  These
 * allocate and synchronise; they are a convenience for callers without device
 * memory management and the end-to-end leg of the benchmark.  (No counterpart in
 * the paper: its measurements are device-resident.) */
int mtmc_fused_linear_host(const void* X, const void* W, const float* b,
                           int64_t M, int64_t N, int64_t K, int act, int out_dtype, void* out);
int mtmc_swiglu_host(const void* X, const void* Wg, const void* Wu,
                     int64_t M, int64_t N, int64_t K, void* out);
int mtmc_linear_lse_host(const void* X, const void* W, const float* b,
                         int64_t M, int64_t N, int64_t K, float* lse_out);

/* The same without waiting for the result: the call enqueues the copy in (on a copy stream of
 * the library's), the kernels (on the current stream) and the copy out (on a second copy
 * stream), chained by events, and returns.  Consecutive calls overlap -- the next call's
 * operands travel to the device while this call computes and its result travels back --
 * which is what a host-resident pipeline needs from a PCIe link that is slower than the
 * kernels.  Host buffers should be pinned (pageable memory makes the copies synchronous)
 * and must stay valid, and the result unread, until mtmc_host_sync() returns; at most six
 * calls are in flight (a seventh first waits for the oldest).  mtmc_host_sync() waits for
 * every call issued so far on the current device.  (No counterpart in the paper.) */
int mtmc_fused_linear_host_async(const void* X, const void* W, const float* b,
                                 int64_t M, int64_t N, int64_t K, int act, int out_dtype, void* out);
int mtmc_swiglu_host_async(const void* X, const void* Wg, const void* Wu,
                           int64_t M, int64_t N, int64_t K, void* out);
int mtmc_linear_lse_host_async(const void* X, const void* W, const float* b,
                               int64_t M, int64_t N, int64_t K, float* lse_out);
int mtmc_host_sync(void);

/* Stream on which later calls from this host thread enqueue (a cudaStream_t;
 * NULL = legacy default stream).  Thread-local. */
int mtmc_set_stream(void* cuda_stream);

/* Use caller-owned device scratch instead of the library's own.  dptr must be
 * 256-byte aligned and stay valid while calls are in flight; (NULL, 0) returns to
 * library-owned scratch.  A call whose requirement exceeds `bytes` fails with
 * MTMC_ERR_WORKSPACE.  Calls in flight on different streams must not share one
 * workspace.  Thread-local. */
int mtmc_set_workspace(void* dptr, size_t bytes);

/* Scratch bytes that suffice for the given operation and shape on the current device under this
 * thread's current tuning, whichever kernel and schedule the library picks (0 if none; (size_t)-1 on
 * invalid arguments). */
size_t mtmc_workspace_bytes(int op, int64_t M, int64_t N, int64_t K);

/* Synchronises the current stream, then returns and clears the sticky device
 * status (MTMC_OK, MTMC_ERR_DEVICE_TIMEOUT or MTMC_ERR_CUDA). */
int mtmc_check_status(void);

/* Self-test of the failure-detection path (no counterpart in the paper): enqueues a
 * one-thread kernel that waits, with a one-millisecond limit, on a barrier nothing will
 * ever signal.  The wait gives up, the kernel returns normally, and the next
 * mtmc_check_status() reports MTMC_ERR_DEVICE_TIMEOUT exactly as it would for a stalled
 * pipeline in a real kernel.  Nothing faults or hangs; the context stays usable. */
int mtmc_selftest_timeout(void);

/* Text for the last non-OK status returned on this host thread ("" if none). */
const char* mtmc_last_error(void);

/* Number of kernels this library has launched from this process so far. */
int64_t mtmc_launch_count(void);

/* Number of device allocations (cudaMalloc calls) this library has made from this process so
 * far: status words, tickets, grown workspaces, the device copies behind the _host entry
 * points.  A caller with a memory budget can watch it; mtmc_linear_lse_noalloc never moves it. */
int64_t mtmc_device_alloc_count(void);

/* Name of the main kernel that the most recent compute call of this host thread launched
 * (kernel family, epilogue, and tile or cluster variant), "" before the first call.  Which
 * kernel a shape lands on is decided inside the library; benchmarks and bug reports name it
 * from here instead of guessing. */
const char* mtmc_last_kernel_name(void);

/* Device time, in milliseconds, of the most recent mtmc_* device entry point on
 * this host thread's current device, measured with CUDA events recorded on the
 * launching stream around the library's kernels.  Synchronises on the end event.
 * Timing is recorded only while enabled with mtmc_set_timing(1).
 * Returns a negative value if no timed call has been made. */
int mtmc_set_timing(int enabled);
float mtmc_last_kernel_ms(void);

/* Tuning hooks (0 = automatic).  They select among kernels of this library only; results
 * stay within tolerance of each other.  Thread-local.
 *   split_k  : > 0 forces the ticketed split-K plan of the skinny path (M <= 64) with this
 *              many K splits per 128-row band of W; for larger M it caps the cluster
 *              size of the cluster split-K kernel (1 = never use that kernel)
 *   tile_n   : 128 or 256 forces single-CTA tiles with that accumulator width
 *   cta_pair : 1 forces the CTA-pair (cta_group::2) kernel with 256 x 256 tiles and overlapped
 *              epilogues, 2 the one with 512 x 256 tiles, < 0 forbids both;
 *              automatic = pairs when M > 128 and N >= 256 (and the problem is not tiny);
 *              the large tiles from K = 16384 on (twice that for E4M3), never for SwiGLU */
int mtmc_set_tuning(int split_k, int tile_n, int cta_pair);

/* Device-side trace, for builds of the library compiled with -DMTMC_TRACE (the default build has none:
 * mtmc_trace_enabled() returns 0 and mtmc_set_trace() with a buffer fails with MTMC_ERR_INVALID_ARG).
 * dptr is a zero-filled device buffer of `bytes` bytes, 8-byte aligned, owned by the caller; (NULL, 0)
 * switches tracing off.  Thread-local.  While set, the CTA-pair kernels (bf16 / E4M3 and MXFP8), the cluster
 * split-K kernel and the weight-streaming kernel
 * write one record of 32 uint64 per CTA (launches of more CTAs than the buffer holds are not traced):
 * %globaltimer stamps of set-up, first / last load, first / last MMA, first / last epilogue, clock64 at both
 * ends of the CTA's life, and cycle
 * totals of each role's waits (producer on a free stage, MMA issuer on data and on a drained accumulator,
 * epilogue on an accumulator, stream-K hand-overs, the split-K exchange); word indices are the TR_* constants of
 * paper_2511_20100_b200/csrc/ptx.cuh, decoded by `python -m paper_2511_20100_b200.trace`.  Stall figures
 * quoted for this library come from there.  No counterpart in the paper. */
int mtmc_trace_enabled(void);
int mtmc_set_trace(void* dptr, size_t bytes);

/* Work schedule of the CTA-pair kernel with 256 x 256 tiles (thread-local; default 0).
 *   stream_k : 1 = deal the last full wave of tiles plus the remainder by k-blocks: the flat list of that
 *              region's (tile, k-block) units is cut into one equal, contiguous share per CTA pair, so that
 *              all pairs finish together whatever the tile count (needs at least as many tiles as pairs); a
 *              tile whose k-blocks straddle two shares is finished by whichever of its two holders comes
 *              second, from fp32 accumulator parts kept in the workspace (bit-reproducible: two addends
 *              commute); 0 or negative = whole tiles, the last wave's tiles cut into column pieces (the
 *              default: measured on a par or ahead on this library's benchmark shapes).
 * The schedule needs workspace (mtmc_workspace_bytes includes it while it is switched on).  It follows the
 * paper's Tiling and Reordering principles: the same tiles, dealt differently. */
int mtmc_set_schedule(int stream_k);

/* Static weights (thread-local, default 0 = off).  With enabled != 0 the caller promises, for
 * the calls that follow on this thread, that no work still in flight on the device writes
 * the W operand (the weights of a deployed model: written once, long before).  The
 * weight-streaming path (M <= 64) and the cluster split-K kernel (decode and small
 * prefill batches) then issue their first ring of W loads before they wait
 * for the preceding kernel on the stream to finish, so the start of the weight stream
 * overlaps that kernel's tail; X, the bias, the residual and every output still wait.
 * Results are the same bits as with the switch off.  If the promise is broken (W produced
 * by the kernel just before) the call may read stale weights.  The paper has no counterpart;
 * it follows its "pipeline" principle across a kernel boundary.  The other tiled kernels ignore it. */
int mtmc_set_static_weights(int enabled);

/* Library version: major * 10000 + minor * 100 + patch. */
int mtmc_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MTMC_FUSED_H_ */
