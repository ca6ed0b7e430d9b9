/*
 * qless.h -- C ABI of the QLESS hot path for NVIDIA B200 (sm_100a).
 *
 * QLESS (arXiv 2502.01703) values training examples by the similarity of their
 * projected, quantised LoRA gradients to validation gradients. This library is
 * the data-parallel hot path of that method:
 *
 *   qless_project_quantize  gradient -> Adam direction -> random projection
 *                           -> L2 normalise -> absmax b-bit codes (+ scale)
 *   qless_score             codes x validation codes -> influence scores
 *   qless_select_topk       scores -> indices of the top fraction
 *
 * Naming. The paper projects R^d -> R^k; to avoid a clash this header calls the
 * gradient dimension P and the projected dimension d (d = 8192 in the paper's
 * Sec. 4.1), N / V the numbers of training / validation examples, C the number
 * of checkpoints, T the number of target tasks, b = `bits` the code width.
 *
 * Conventions for every call, unless an argument says otherwise:
 *  - pointers are DEVICE pointers into memory the caller owns; "host" marks the
 *    exceptions. The library allocates nothing that outlives a call; scratch is
 *    the caller's `workspace` (size from the matching *_workspace() query,
 *    256-byte aligned).
 *  - calls enqueue work on `cuda_stream` (a cudaStream_t cast to void*, NULL =
 *    default stream) and return without synchronising. Host arrays are read
 *    before the call returns.
 *  - every precondition is checked before anything is launched; a violation
 *    returns a status and leaves all buffers untouched. Calls with zero rows
 *    succeed and touch nothing. No exception crosses this boundary.
 *  - qless_last_error() gives a thread-local, human readable description of the
 *    last non-OK status returned on this thread.
 */
#ifndef QLESS_H_
#define QLESS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    QLESS_OK = 0,
    QLESS_ERR_INVALID_ARG = 1, /* NULL where a buffer is required, negative size, bad offsets ... */
    QLESS_ERR_UNSUPPORTED = 2, /* bits not in {1,2,4,8}; d or P not a multiple of 128; d > 8192 ... */
    QLESS_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or smaller than the query says */
    QLESS_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed; text in qless_last_error() */
    QLESS_ERR_TIMEOUT = 5      /* a bounded device-side wait gave up (see qless_check) */
} qless_status;

typedef enum { QLESS_F32 = 0, QLESS_BF16 = 1 } qless_dtype;

/* Adam hyper-parameters of the training-gradient prologue. step = 0 switches the bias
 * correction off (it is a uniform factor that normalisation removes, except through eps). */
typedef struct {
    float beta1;  /* 0.9   */
    float beta2;  /* 0.999 */
    float eps;    /* 1e-8  */
    int64_t step; /* 0     */
} qless_adam_cfg;

const char* qless_last_error(void);

/* Reads and clears the device-side timeout flag after synchronising `cuda_stream`. Kernels that
 * wait on asynchronous copies or tensor-core completion give up after a bounded number of polls,
 * set the flag and exit; results of that call are then invalid. Returns QLESS_OK,
 * QLESS_ERR_TIMEOUT or QLESS_ERR_CUDA. */
qless_status qless_check(void* cuda_stream);

/* Self-test of that machinery (no counterpart in the paper). Enqueues a one-block kernel in which one thread waits,
 * with the library's own bounded-wait routine and a limit of `polls` polls (256 .. 65536), on a barrier that nothing
 * ever signals, while a second thread waits on another such barrier with a limit 256 times larger. The first gives
 * up, records the producer code (0x1) in the device timeout word and raises the block-wide abort flag; the second
 * must leave on seeing that flag without recording a code of its own; the kernel then returns normally. The next
 * qless_check on the stream therefore returns QLESS_ERR_TIMEOUT (message: code 0x1) and the one after it QLESS_OK.
 * No tensor memory is touched and no copy is started. Returns QLESS_ERR_INVALID_ARG for polls out of range. */
qless_status qless_selftest_timeout(int32_t polls, void* cuda_stream);

/* Per-kernel timing for benchmarks (no counterpart in the paper; measurement aid). While enabled on the
 * calling thread, every kernel the library launches is bracketed by CUDA events on the call's stream.
 * qless_profile_collect synchronises those events, writes "name=milliseconds*launches;..." (time summed
 * per kernel name since the last collect) into buf (NUL-terminated, truncated to buflen) and clears the
 * record. Enabling costs two event records per launch; leave it off otherwise. */
qless_status qless_profile_enable(int32_t on);
/* Number of kernels this library has launched in this process so far (all threads). */
uint64_t qless_kernel_launches(void);
qless_status qless_profile_collect(char* buf /* host */, size_t buflen);

/* Peak-rate micro-benchmarks (no counterpart in the paper; they give the roofline denominators that no
 * vendor tool has measured on the machine at hand). `what`: 0 / 1 / 2 = back-to-back tcgen05.mma on every SM
 * with operands resident on chip: bf16 with both operands in shared memory / bf16 with A in tensor memory /
 * int8; 3 / 4 / 5 = the same three on CTA pairs (cta_group::2); 6 = the XOR + POPC + IADD mix of 1-bit
 * scoring on the integer pipes (scratch: device buffer of >= 8 KiB per SM); 7 = int8 on CTA pairs with A in
 * tensor memory; 8 = int8 on CTA pairs in the shape 8-bit scoring issues for 448 validation vectors (per K step
 * one MMA of N = 256 and one of N = 192 that re-read the same A from shared memory); 9 = TMA alone streaming
 * 48 KiB stages from an L2-resident buffer into shared memory on every SM, nothing consuming them (scratch:
 * 16-byte aligned device buffer of >= 4 MiB, QLESS_ERR_WORKSPACE otherwise); 10 = 8 and 9 together as 8-bit
 * scoring runs them (the MMAs of one K block committed at once, one 48 KiB stage per K block streamed into other
 * shared memory three stages ahead, the MMAs never waiting for data; same scratch; operations counted are the
 * MMAs'); 11 = the kernel of 10 with the copies switched off; 12 = the MMAs of 8 reading, for every K block, a
 * stage that TMA has just brought from the scratch buffer (same scratch size; the CALLER fills it with the int8
 * values the operands are to take, e.g. pseudo-random ones: the operands then change with every K block, which
 * is what sets the power drawn and so the clock granted under the power cap); 13 = the shape of 8 on e2m1 operands
 * (tcgen05.mma kind::mxf4 with unit scale factors, 64 codes per MMA, both operands in shared memory), which is what
 * 2- and 1-bit scoring issues; 14 = e2m1 on CTA pairs with A in tensor memory, N = 256. Runs the kernel twice and times
 * the second run with CUDA events on `cuda_stream` (synchronises it). *ms_out: milliseconds; *ops_out:
 * operations executed (2 x multiply-accumulates; word operations for 6; bytes moved for 9). Host pointers. */
qless_status qless_microbench(int32_t what, int32_t iters, float* ms_out, double* ops_out, void* scratch,
                              size_t scratch_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Stage 1 + 2: datastore construction (paper Sec. 2.2 Eq. 1-2, Sec. 3.1, Eq. 4-5).
 *
 * For each of the n gradient rows g (row-major [n, P], leading dimension ld_grads elements):
 *   Gamma = Adam direction of g given the checkpoint's moments (the training-side gradient of Sec. 2.2, which
 *           the paper names without a formula):  m' = b1 m + (1-b1) g, v' = b2 v + (1-b2) g^2, (bias-corrected if
 *           step > 0), Gamma = m' / (sqrt(v') + eps), computed in fp32 and rounded to bf16.
 *           adam_m = adam_v = NULL selects the SGD (validation) gradient: Gamma = bf16(g).
 *   y     = R Gamma (Eq. 1), R in {+-1/sqrt(d)}^{d x P} Rademacher. R is never stored: entry
 *           (r, j) is bit t = j mod 128 of the Philox4x32-10 block with counter
 *           (j / 128, r, 0, 0) and key (seed low, seed high); within 32-bit output word t / 32
 *           the bit index is 15 - (u / 2) + 16 (u mod 2), u = t mod 32; bit 1 means -1.
 *           bf16 x bf16 products, fp32 accumulation, one fp32 multiply by 1/sqrt(d).
 *   yhat  = y / ||y||_2 (Eq. 2).
 *   S     = max_m |yhat_m|; alpha = 2^(b-1) - 1; q_m = round_half_even(alpha yhat_m / S) (Eq. 4-5);
 *           b = 1: q_m = -1 if yhat_m < 0 else +1 (sign quantiser). A zero vector gives S = 0 and
 *           all-zero codes.
 * Outputs (all optional except codes and scales):
 *   codes      [n, d*bits/8] bytes, dense little-endian packing: b=8 one int8 per code; b=4 code m in
 *              bits [4(m&1), +4) of byte m>>1; b=2 code m in bits [2(m&3), +2) of byte m>>2 (two's
 *              complement fields); b=1 code m is bit m&7 of byte m>>3, bit 1 <=> -1.
 *   scales     [n] fp32, the absmax S of the normalised vector (the one scale per vector of Sec. 3.1).
 *   code_sumsq [n] int32, sum_m q_m^2 = ||q||^2 of Eq. 6 (NULL to skip).
 *   proj_out   [n, d] fp32, the un-normalised projection y (NULL to skip; test tap).
 * The same seed must be used for every vector that will be scored together.
 * Requirements: d % 128 == 0, 128 <= d <= 8192; P % 128 == 0; P < 2^39; grads 16-byte aligned and
 * ld_grads % 8 == 0; bits in {1,2,4,8}; codes 16-byte aligned.
 * ------------------------------------------------------------------------------------------ */
size_t qless_project_quantize_workspace(int64_t n, int64_t P, int32_t d, int32_t bits);

qless_status qless_project_quantize(
    const void* grads, qless_dtype dtype, int64_t n, int64_t ld_grads,
    const float* adam_m, const float* adam_v, const qless_adam_cfg* adam /* host, NULL = defaults */,
    int64_t P, int32_t d, uint64_t seed, int32_t bits,
    void* codes, float* scales, int32_t* code_sumsq, float* proj_out,
    void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The same computation for callers whose gradients live in HOST memory (pinned memory makes the copies
 * asynchronous). grads [n, P] (ld_grads elements per row), codes, scales, code_sumsq are HOST pointers;
 * adam_m / adam_v stay DEVICE pointers (one copy per checkpoint serves every batch). The call copies the
 * batch to the device workspace, runs qless_project_quantize there and copies the results back, all on
 * `cuda_stream`; the host buffers must stay valid until the stream has drained. Workspace size:
 * qless_project_quantize_host_workspace. Definition of the operation: as qless_project_quantize
 * (Eq. 1-2, Eq. 4-5). */
size_t qless_project_quantize_host_workspace(int64_t n, int64_t P, int32_t d, int32_t bits, qless_dtype dtype);

qless_status qless_project_quantize_host(
    const void* grads_host, qless_dtype dtype, int64_t n, int64_t ld_grads,
    const float* adam_m, const float* adam_v, const qless_adam_cfg* adam /* host, NULL = defaults */,
    int64_t P, int32_t d, uint64_t seed, int32_t bits,
    void* codes_host, float* scales_host, int32_t* code_sumsq_host /* NULL to skip */,
    void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The same two calls with the random matrix R of Eq. 1 chosen per call (Sec. 2.4 leaves its distribution open
 * between Gaussian and Rademacher; R is a property of a datastore, fixed by (seed, matrix) for every vector that
 * will be scored together, so it travels with the call and not in library state: two host threads may build a
 * Rademacher and a Gaussian store at the same time). `projection` is a HOST pointer, NULL = defaults
 * (QLESS_MATRIX_RADEMACHER, which is what qless_project_quantize and qless_project_quantize_host use).
 *   QLESS_MATRIX_RADEMACHER: entries +-1/sqrt(d), entry map above.
 *   QLESS_MATRIX_GAUSSIAN:   entries z/sqrt(d) with z standard normal, rounded to bf16 (the operand type of the
 *     contraction): the four entries of row r in columns 4q .. 4q+3 come from one Philox4x32-10 call with counter
 *     (q mod 2^32, r, q div 2^32, 1) and the same key; output words (w0, w1) give columns 4q, 4q+1 and (w2, w3)
 *     give 4q+2, 4q+3 by the Box-Muller transform z_even = sqrt(-2 ln u1) cos(2 pi u2),
 *     z_odd = sqrt(-2 ln u1) sin(2 pi u2) with u = (floor(w / 2^9) + 1/2) / 2^23. The logarithm, square root, sine
 *     and cosine are evaluated in fp32 on the GPU's approximate units, so an entry may differ from the correctly
 *     rounded one by one bf16 step where it falls next to a rounding boundary. The generator, not the tensor pipe,
 *     bounds this variant.
 * Every other argument, output, requirement and error is that of the call without the suffix; a matrix value other
 * than the two above (or a non-zero reserved field) returns QLESS_ERR_INVALID_ARG. */
enum { QLESS_MATRIX_RADEMACHER = 0, QLESS_MATRIX_GAUSSIAN = 1 };
typedef struct {
    int32_t matrix;      /* QLESS_MATRIX_RADEMACHER */
    int32_t reserved[3]; /* must be 0 */
} qless_projection_cfg;

qless_status qless_project_quantize_ex(
    const void* grads, qless_dtype dtype, int64_t n, int64_t ld_grads,
    const float* adam_m, const float* adam_v, const qless_adam_cfg* adam /* host, NULL = defaults */,
    int64_t P, int32_t d, uint64_t seed, const qless_projection_cfg* projection /* host, NULL = defaults */,
    int32_t bits, void* codes, float* scales, int32_t* code_sumsq, float* proj_out,
    void* workspace, size_t workspace_bytes, void* cuda_stream);

qless_status qless_project_quantize_host_ex(
    const void* grads_host, qless_dtype dtype, int64_t n, int64_t ld_grads,
    const float* adam_m, const float* adam_v, const qless_adam_cfg* adam /* host, NULL = defaults */,
    int64_t P, int32_t d, uint64_t seed, const qless_projection_cfg* projection /* host, NULL = defaults */,
    int32_t bits, void* codes_host, float* scales_host, int32_t* code_sumsq_host /* NULL to skip */,
    void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---- Hooks for tests and measurements only. They select between kernels that compute the SAME result, are
 * process-wide (every thread's later calls take the chosen kernel), and are not meant for production callers:
 * leave them at 0. ---- */

/* Which kernel computes the projection of Eq. 1 in qless_project_quantize. 0 (default): the
 * tcgen05 tensor-core kernel; 1: a plain CUDA-core kernel of the same definition, kept so that the
 * tensor-core result can be cross-checked on the device at sizes the CPU oracle only samples (it is
 * also what runs when P >= 2^31). */
qless_status qless_set_projection_path(int32_t path);

/* As above, for the integer similarity in qless_score and qless_score_dots: 0 (default) the
 * tcgen05 kernel for every code width (used when T <= 8; int8 operands for 8- and 4-bit codes, e2m1 operands with
 * unit scale factors for 2-bit codes and sign bits, whose values e2m1 holds exactly), 1 the CUDA-core kernels (dp4a for 8-, 4- and 2-bit codes, XOR + population count for
 * 1-bit codes). */
qless_status qless_set_score_path(int32_t path);

/* As above, for qless_select_topk. 0 (default): up to 360 448 scores one launch of a thread-block cluster that
 * keeps the keys in shared memory (one read, no workspace used); up to 2^22 the multi-pass radix select (five
 * reads); above, a sampled bracket of the k-th largest key, one gather pass and a radix select on the
 * gathered candidates, with the multi-pass select as the fallback when the bracket misses.
 * 1: multi-pass at every N. 2: as 0, with the bracket forced above every key, so that the fallback does the
 * work. The result is the same in all three. */
qless_status qless_set_select_path(int32_t path);

/* Stage 2 alone (Eq. 2, Eq. 4-5, packing) on fp32 rows x [n, d]; normalize = 0 skips Eq. 2 so that
 * already-normalised rows can be fed. Same outputs and packing as above. Needs no workspace. */
qless_status qless_quantize(
    const float* x, int64_t n, int32_t d, int32_t normalize, int32_t bits,
    void* codes, float* scales, int32_t* code_sumsq, void* cuda_stream);

/* Absmean variant of the same stage (Sec. 6, Table 3). The paper names it without a formula; the reading built
 * here: gamma = mean_m |yhat_m|, Delta = gamma * c_b with c_2 = 1, c_4 = 1/2, c_8 = 1/32,
 * q_m = clamp(round_half_even(yhat_m / Delta), -alpha, alpha); scales[r] = alpha * Delta, so that q * scale / alpha
 * dequantises as for absmax codes and qless_score takes such a store unchanged. bits = 1 is the sign code.
 * Same arguments, packing, limits and errors as qless_quantize. */
qless_status qless_quantize_absmean(const float* x, int64_t n, int32_t d, int32_t normalize, int32_t bits, void* codes,
                                    float* scales, int32_t* code_sumsq, void* cuda_stream);

/* Stage 1a alone: the Adam prologue. gamma_out [n, P] bf16 (raw 16-bit patterns), row-major, leading
 * dimension P. Same reading of Gamma as above. */
qless_status qless_adam_gamma(
    const void* grads, qless_dtype dtype, int64_t n, int64_t ld_grads,
    const float* adam_m, const float* adam_v, const qless_adam_cfg* adam /* host */,
    int64_t P, void* gamma_out, void* cuda_stream);

/* Entries of the projection matrix as the kernels generate them: out [nr, nj] int8 (+1 / -1) for
 * rows r0 .. r0+nr-1 and columns j0 .. j0+nj-1 of sqrt(d) R (entry map above). */
qless_status qless_philox_entries(
    uint64_t seed, int64_t r0, int64_t nr, int64_t j0, int64_t nj, int8_t* out, void* cuda_stream);

/* Entries of the Gaussian matrix as the kernels generate them: out [nr, nj] fp32 (device; bf16-representable
 * values of sqrt(d) R) for rows r0 .. r0+nr-1 and columns j0 .. j0+nj-1; j0 must be a multiple of 4. */
qless_status qless_gaussian_entries(
    uint64_t seed, int64_t r0, int64_t nr, int64_t j0, int64_t nj, float* out, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Stage 3: influence scores over the quantised datastore (paper Eq. 6-7; aggregation as in LESS,
 * which the paper follows when it accumulates influence over the validation data, Sec. 4.1).
 *
 *   D_i[t, v]  = sum_m q_{t,i,m} q_{v,i,m}                 integer, exact (b = 1: d - 2 popcount(xor))
 *   sim_i[t,v] = D_i / (||q_{t,i}|| ||q_{v,i}||)            mode COSINE (Eq. 6-7); a vector whose scale
 *                                                          is 0 is the zero vector and contributes 0
 *              = (S_t/alpha)(S_v/alpha) D_i                mode DEQUANT (alpha := 1 at b = 1): inner
 *                                                          product of the reconstructed vectors (Eq. 3)
 *   A[t, j]    = sum_i eta_i * mean_{v in task j} sim_i[t, v]
 *   score[t]   = max_j A[t, j]
 *
 * train_codes [C][N][d*bits/8] with checkpoint stride train_ckpt_stride_bytes (>= N*d*bits/8, multiple
 * of 16); val_codes likewise with V. train_scales [C][N], val_scales [C][V]. train_sumsq / val_sumsq
 * [C][N] / [C][V] int32 as produced by qless_project_quantize; NULL = recomputed from the codes.
 * lr_weights: host [C] (eta_i, used as given). task_offsets: host [T+1], strictly increasing,
 * [0] = 0, [T] = V. scores [N] fp32; per_task [N, T] fp32 or NULL.
 * The two host arrays reach the device through copies from pageable memory enqueued on `cuda_stream`: the runtime
 * stages them before the call returns (the arrays may be freed at once), but such a copy may wait for earlier work
 * of the stream, so this call (and qless_score_16bit) can block for that long and must not be issued while the
 * stream is being captured into a graph.
 * Requirements: d % 128 == 0, d <= 8192; 1 <= V <= 4096; 1 <= T <= 64; 1 <= C <= 64.
 * ------------------------------------------------------------------------------------------ */
typedef enum { QLESS_SCORE_COSINE = 0, QLESS_SCORE_DEQUANT = 1 } qless_score_mode;

size_t qless_score_workspace(int64_t N, int32_t V, int32_t C, int32_t T, int32_t d, int32_t bits);

qless_status qless_score(
    const void* train_codes, int64_t train_ckpt_stride_bytes,
    const void* val_codes, int64_t val_ckpt_stride_bytes,
    const float* train_scales, const float* val_scales,
    const int32_t* train_sumsq, const int32_t* val_sumsq,
    const float* lr_weights /* host */, const int32_t* task_offsets /* host */,
    int64_t N, int32_t V, int32_t C, int32_t T, int32_t d, int32_t bits, qless_score_mode mode,
    float* scores, float* per_task,
    void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The 16-bit baseline the paper compares against (LESS, Eq. 3 with the aggregation of Sec. 4.1): the store holds
 * the projected gradients themselves as bf16 rows, train_rows [C][N][d] and val_rows [C][V][d] (device,
 * checkpoint strides in bytes, multiples of 16), and
 *   scores[t] = max_j sum_i lr_weights[i] * mean_{v in task j} <x_t,i, x_v,i> / (||x_t,i|| ||x_v,i||)
 * with the inner products accumulated in fp32 on the tensor cores and the norms in fp64; a zero row scores 0.
 * train_inv_norms [C][N] / val_inv_norms [C][V] (device; 1 / ||row||, 0 for a zero row, e.g. from
 * qless_inv_norms_16bit) may be NULL, in which case the call computes them with one more pass over the store.
 * lr_weights [C] and task_offsets [T+1] are host arrays (tasks are consecutive validation rows, T <= 8);
 * per_task (device [N][T]) may be NULL. Same d and V limits as qless_score. Workspace: device, 256-byte
 * aligned, qless_score_16bit_workspace bytes. Errors: the statuses of qless_score. */
size_t qless_score_16bit_workspace(int64_t N, int32_t V, int32_t C, int32_t T);
qless_status qless_inv_norms_16bit(const void* rows, int64_t ckpt_stride_bytes, int64_t nrows, int32_t C, int32_t d,
                                   float* inv_norms /* device [C][nrows] */, void* cuda_stream);
qless_status qless_score_16bit(const void* train_rows, int64_t train_ckpt_stride_bytes, const void* val_rows,
                               int64_t val_ckpt_stride_bytes, const float* train_inv_norms, const float* val_inv_norms,
                               const float* lr_weights, const int32_t* task_offsets,
                               int64_t N, int32_t V, int32_t C, int32_t T, int32_t d, float* scores, float* per_task,
                               void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The integer numerators alone, for one checkpoint: dots [nt, V] int32 = D[t0 + t, v] computed by the
 * same kernels that feed qless_score. train_codes [>= t0+nt, d*bits/8], val_codes [V, d*bits/8]. */
size_t qless_score_dots_workspace(int64_t nt, int32_t V, int32_t d, int32_t bits);

qless_status qless_score_dots(
    const void* train_codes, const void* val_codes, int64_t t0, int64_t nt, int32_t V,
    int32_t d, int32_t bits, int32_t* dots, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Stage 4: top-k selection (the top 5 % of the training data by score, Sec. 4.1).
 *
 *   k = floor(frac * N + 1e-6) clamped to [0, N], written to *k_out (host) before the call returns.
 *   Total order on fp32: by value, -0 below +0, every NaN below -inf; equal scores are admitted by
 *   ascending index. indices [k] int64 receives the selected indices in ascending order.
 * Requirements: 0 <= frac <= 1; N < 2^31.
 * ------------------------------------------------------------------------------------------ */
size_t qless_select_topk_workspace(int64_t N);

qless_status qless_select_topk(
    const float* scores, int64_t N, double frac, int64_t* indices, int64_t* k_out /* host */,
    void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Top-k selection for callers that cannot allocate device memory. (The paper has no counterpart: this
 * is a packaging variant of qless_select_topk, same result, same ordering rules.)
 *
 * Who needs it: code that runs where a cudaMalloc is not an option -- inside a region whose memory is
 * fully budgeted by a pool the caller does not own (a serving process with a fixed arena, a plug-in
 * loaded into somebody else's process), or on a path where an allocation's implicit device
 * synchronisation would stall other streams. qless_select_topk asks such callers for a workspace they
 * cannot produce; this entry point brings its own.
 *
 * The scratch of the radix select (histograms, selection state, per-block counts and offsets) lives in a
 * fixed array in device global memory that is part of the library image: 74 KiB on every GPU that loads
 * the library, held until the process exits. That bounds the input: N <= QLESS_SELECT_STATIC_MAX_N
 * (4 194 304 scores); a larger N is refused with QLESS_ERR_UNSUPPORTED and a message that names the limit.
 * The call makes no cudaMalloc / cudaFree and calls nothing that allocates; inputs and outputs are still
 * the caller's (scores [N] fp32 device, 16-byte aligned; indices [k] int64 device; k_out host).
 *
 * First call on each device: the library looks up the array's device address (once per device, with that
 * device current). Make that first call outside any stream capture; later calls only enqueue kernels and
 * one memset on `cuda_stream`.
 * Sharing: every call on a device uses the same array. The parts that must start at zero are cleared at
 * the start of each call and the rest is overwritten before it is read, so back-to-back calls on one
 * stream are independent. Two calls that overlap on the GPU (different streams, or host threads feeding
 * different streams) race on the array and give undefined results: serialise them.
 */
#define QLESS_SELECT_STATIC_MAX_N (1 << 22)

qless_status qless_select_topk_static(
    const float* scores, int64_t N, double frac, int64_t* indices, int64_t* k_out /* host */,
    void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* QLESS_H_ */
