/*
 * mona.h — C ABI of the B200 (sm_100a) implementation of the MONA matrix-optimizer step.
 *
 * One call of mona_step() performs, for every 2-D weight of a parameter set, the loop body of
 * Algorithm 1 ("MONA Optimizer"):
 *
 *     D_k  = G_k - G_{k-1}                         (Eq. alto_diff,   Algorithm 1 line 4)
 *     A_k  = beta_a A_{k-1} + (1 - beta_a) D_k     (Eq. alto_accel,  line 5)
 *     G~_k = G_k + alpha A_k                       (Eq. alto_grad,   line 6)
 *     M_k  = mu M_{k-1} + G~_k                     (Eq. muon_momentum, line 7)
 *     O_k  = Newton-Schulz(M_k, T)                 (Eq. newton_schulz, line 8)
 *     W   <- W - eta (gamma O_k + lambda W)        (Eq. muon_update,   line 9)
 *     G_{k-1} <- G_k                               (line 10)
 *
 * with X_0 = M_k / (||M_k||_F + eps), X_{t+1} = a X_t + b X_t X_t^T X_t + c X_t X_t^T X_t X_t^T X_t,
 * and gamma = 0.2 sqrt(max(m, n)) unless overridden.
 *
 * Conventions
 *   - All matrix pointers are DEVICE pointers unless a parameter says "host".  Arrays of pointers
 *     (params, grads) and all structs are HOST memory.
 *   - Matrices are row-major with leading dimension = cols.  Parameters are fp32 master weights;
 *     gradients are fp32 or bf16 (per descriptor).
 *   - The caller owns parameters, gradients, the state block and the workspace.  The handle owns only
 *     small host/device tables, one internal stream and a few events.
 *   - Every function returns a mona_status; nothing throws or aborts.  Problems detected on the device
 *     (non-finite norm, a wait that ran out) are latched in a status word read by mona_poll_status().
 *     A step that reported MONA_ERR_TIMEOUT or MONA_ERR_NONFINITE has already advanced M, A and G_prev and
 *     may have written parameters from incomplete iterates: restore state and parameters from the caller's
 *     last checkpoint before stepping again.
 *   - There is no CPU fallback: on a machine without an sm_100 device mona_create() fails with
 *     MONA_ERR_ARCH / MONA_ERR_CUDA.
 *   - One handle is used from one host thread and one stream at a time.
 */
#ifndef MONA_H_
#define MONA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MONA_OK = 0,
    MONA_ERR_INVALID_ARG = 1,        /* null pointer, non-positive size, bad enum                     */
    MONA_ERR_UNSUPPORTED_SHAPE = 2,  /* a shape this build cannot process                             */
    MONA_ERR_ALIGNMENT = 3,          /* a device pointer or stride is not 16-byte aligned             */
    MONA_ERR_CUDA = 4,               /* a CUDA runtime/driver call failed (see mona_last_error)       */
    MONA_ERR_TIMEOUT = 5,            /* a bounded device-side wait ran out                            */
    MONA_ERR_NONFINITE = 6,          /* ||M_k||_F of some matrix was inf/nan                          */
    MONA_ERR_ARCH = 7,               /* device is not compute capability 10.x                         */
    MONA_ERR_BUFFER_TOO_SMALL = 8,   /* state or workspace smaller than mona_query_sizes() reports    */
    MONA_ERR_BOUNDS = 9,             /* debug build (-DMONA_DEBUG) only: a kernel's index check failed */
    MONA_ERR_NOT_BUILT = 10          /* the call needs a build option this library was compiled without */
} mona_status;

typedef enum { MONA_F32 = 0, MONA_BF16 = 1 } mona_dtype;
/* Third value of mona_matrix_desc.state_dtype (see there). */
#define MONA_STATE_COMBINED 2

/* One descriptor = `batch` matrices of identical shape (the experts of one MoE layer, or batch = 1).
 * Matrix b of the descriptor starts `b * batch_stride` ELEMENTS after the descriptor's base pointer,
 * for the parameter and for the gradient alike.  The update scale gamma uses max(rows, cols) of one
 * matrix, never the stacked shape. */
typedef struct {
    int64_t rows, cols;        /* m, n of one matrix                                                  */
    int64_t batch;             /* >= 1                                                                */
    int64_t batch_stride;      /* elements between consecutive matrices, >= rows*cols (0 = rows*cols) */
    int32_t grad_dtype;        /* mona_dtype of the gradient                                          */
    int32_t state_dtype;       /* mona_dtype in which A_k and G_{k-1} are stored: MONA_F32 (0, Algorithm 1 as
                                  printed, "full precision"), or MONA_BF16 = MONA-Lite (section "Efficient
                                  Deployment with Reduced Overhead"): both buffers kept in bfloat16, equations
                                  unchanged.  A_k is formed in fp32, rounded to nearest-even once when stored,
                                  and the stored value is the one G~_k uses; G_{k-1} is the rounded G_k.
                                  M_k is fp32 either way.
                                  MONA_STATE_COMBINED (2): one fp32 buffer Z_k = beta_a A_k - (1-beta_a) G_k in
                                  place of both.  A_k and G_{k-1} enter the next step only through it
                                  (A_{k+1} = Z_k + (1-beta_a) G_{k+1}), so the step is Algorithm 1 unchanged with
                                  8 instead of 12 state bytes per parameter and 22 instead of 30 bytes moved by
                                  the prologue - the counterpart, at this boundary, of the paper's "streaming"
                                  variant that drops the G_{k-1} buffer.  mona_state_layout() then reports Z at
                                  off_A and (size_t)-1 for off_Gprev.                                  */
} mona_matrix_desc;

/* REQUIRE line of Algorithm 1.  Doubles on purpose: (1 - beta_a), eta*gamma and eta*lambda are formed
 * in double on the host and rounded to fp32 once. */
typedef struct {
    double lr;             /* eta                                                                     */
    double momentum;       /* mu                                                                      */
    double accel_beta;     /* beta_a                                                                  */
    double accel_alpha;    /* alpha                                                                   */
    double weight_decay;   /* lambda                                                                  */
    double ns_a, ns_b, ns_c;  /* quintic coefficients (3.4445, -4.7750, 2.0315 in the paper)         */
    double norm_eps;       /* X_0 = M / (||M||_F + eps); the paper has no eps, 1e-7 is a safe default */
    double scale_value;    /* see scale_mode                                                          */
    int32_t ns_steps;      /* T >= 0 (5 in the paper); 0 means O = X_0                                */
    int32_t scale_mode;    /* 0: gamma = scale_value * sqrt(max(m,n)); 1: gamma = scale_value         */
    int32_t ns_precision;  /* 0: bf16 operands on the tensor cores, fp32 accumulate;
                              1: fp32 validation mode (plain FMA, no tensor cores)                    */
    int32_t algorithm;     /* 0: MONA (Algorithm 1).  1: plain Muon, the baseline of Eq. muon_momentum /
                              muon_ns / muon_update: M_k = mu M_{k-1} + G_k, same orthogonalisation and
                              update; accel_beta and accel_alpha are ignored and A, G_prev are neither read
                              nor written (they keep whatever they held).                             */
} mona_hparams;

typedef struct mona_handle mona_handle;

/* Fills *hp with the paper's defaults where it states them (T = 5, the quintic coefficients, the 0.2
 * scale rule, beta_a = 0.99 with alpha = -1/(2(1-beta_a))) and eta = 1e-3, mu = 0.95, lambda = 0.1,
 * eps = 1e-7 where it does not. */
mona_status mona_default_hparams(mona_hparams* hp);

/* Per-handle tuning options.  Obtain the defaults with mona_default_options(), change what you need, and pass
 * the SAME struct to mona_query_sizes_opt() and mona_create_opt(): the workspace size depends on it.  A handle
 * keeps the options it was created with.
 *   chunk_budget_bytes : bytes of bf16 Newton-Schulz iterates (X_t, X_{t+1}, A_t, B'_t) one chunk of same-shape
 *                        matrices may hold (0 = the default, 768 MiB; otherwise at least 1 MiB).  A chunk goes
 *                        through prologue, the whole iteration and the update before the next one starts.
 *                        Chunks are sized to keep every SM pair busy, not to fit a cache: cache-sized chunks
 *                        (tens of MiB) hold too few tiles for the machine and were measured 1.5-2x slower.
 *   chunk_overlap      : 1 (default) pipelines consecutive chunks over two streams - the caller's and one the
 *                        handle owns, joined by events before mona_step*() returns to the caller's stream - so
 *                        that the start and the tail of one chunk's kernels are filled by the other chunk's;
 *                        0 keeps every launch on the caller's stream.  Results are identical either way; the
 *                        workspace holds two chunks.
 *   fuse_update        : 0 (default): O_k is stored in bf16 and a separate elementwise kernel applies Eq. muon_update.
 *                        1: on the tensor-core path the last X' = B' X of a step applies the update in its epilogue
 *                        (fp32 O_k straight from the accumulator, no bf16 copy of O_k written and re-read, one launch
 *                        fewer per chunk).  The two differ by the bf16 rounding of O_k only.  Measured slower on the
 *                        benchmark sets: a thread owns a row of the accumulator, so its fp32 read-modify-write of W
 *                        touches 32 lines per warp instruction and sits, unhidden, in the macro-tile's epilogue.
 *   ns_delay           : how many matrices apart consecutive Newton-Schulz GEMMs of one matrix sit in the kernel's
 *                        work order (0 = the default, 20; at most 1024; a value >= the chunk's matrix count
 *                        runs the chunk GEMM by GEMM).  Larger values hide the dependency latency
 *                        better, smaller ones keep intermediates closer to the cache.  Results do not depend on it.
 *   macro_tile_min_k   : X' = B' X runs as 256 x 512 macro-tiles (two tiles sharing one staged operand slice, both
 *                        accumulators in use, so nothing hides their epilogue) when its inner dimension - the shorter
 *                        side of the weight - is at least this, and as plain 256 x 256 tiles with alternating
 *                        accumulators below it (0 = the default, 1: always macro-tiles.  Plain tiles keep the tensor
 *                        cores busier per clock on short inner dimensions, but the step runs at the power cap and
 *                        macro-tiles move fewer bytes per flop: measured 3-7 % faster on every benchmark set).
 *                        Results do not depend on it. */
typedef struct {
    size_t chunk_budget_bytes;
    int32_t chunk_overlap;
    int32_t fuse_update;
    int32_t ns_delay;
    int32_t macro_tile_min_k;
    int32_t reserved[4];       /* zero */
} mona_options;

/* Fills *opt with the defaults (as changed by the two process-wide setters below, if they were called). */
mona_status mona_default_options(mona_options* opt);

/* Process-wide defaults that seed mona_default_options() and the plain mona_query_sizes()/mona_create():
 * chunk budget in bytes (at least 1 MiB) and chunk overlap (0/1).  They affect handles created later only; an
 * existing handle keeps its own options.  Prefer the options struct: these two exist for callers that create
 * all their handles with one setting, and must not be changed between mona_query_sizes() and mona_create(). */
mona_status mona_set_chunk_budget(size_t bytes);
mona_status mona_set_chunk_overlap(int enabled);

/* Bytes the caller must provide for the optimizer state (M, A, G_prev, Algorithm 1 line 1: 12 bytes per
 * parameter, 8 with bfloat16 storage of A and G_prev) and for the Newton-Schulz workspace.  Host only; no device is touched. */
mona_status mona_query_sizes(const mona_matrix_desc* descs, int64_t n_desc,
                             size_t* state_bytes, size_t* workspace_bytes);
/* The same with explicit options (NULL = defaults). */
mona_status mona_query_sizes_opt(const mona_matrix_desc* descs, int64_t n_desc, const mona_options* options,
                                 size_t* state_bytes, size_t* workspace_bytes);

/* Builds the plan (shape buckets, chunking, tile schedules, TMA descriptors) for `n_desc` descriptors
 * on CUDA device `device`, binds the caller's state and workspace blocks (both 256-byte aligned device
 * memory of at least the queried sizes) and zero-fills the state (M_0 = A_0 = G_0 = 0).
 * Synchronises the device once.  *out receives the handle; destroy it with mona_destroy(). */
mona_status mona_create(mona_handle** out, const mona_matrix_desc* descs, int64_t n_desc,
                        void* state, size_t state_bytes, void* workspace, size_t workspace_bytes,
                        int device);
/* The same with explicit options (NULL = defaults); sizes must come from mona_query_sizes_opt() with the same options. */
mona_status mona_create_opt(mona_handle** out, const mona_matrix_desc* descs, int64_t n_desc,
                            const mona_options* options, void* state, size_t state_bytes, void* workspace,
                            size_t workspace_bytes, int device);

/* One optimizer step for all descriptors, enqueued on `stream` (a cudaStream_t passed as void*;
 * NULL = the legacy default stream).  params[i] / grads[i] are the device base pointers of
 * descriptor i (16-byte aligned).  Reads grads, updates params and the state in place.  Allocates
 * nothing and does not synchronise; work also runs on the handle's internal stream, ordered with
 * `stream` by events, so synchronising `stream` is enough to observe the result. */
mona_status mona_step(mona_handle* h, const mona_hparams* hp,
                      void* const* params, const void* const* grads, void* stream);

/* As mona_step, plus two measurement/verification hooks:
 *   phase_mask : bit 0 prologue (lines 4-7, 10 + norm), bit 1 Newton-Schulz (line 8),
 *                bit 2 parameter update (line 9).  7 = the full step.  A skipped phase leaves its
 *                outputs as they were, so a partial mask is for timing only.
 *   o_out      : NULL, or n_desc device pointers; descriptor i receives O_k in fp32 with the
 *                parameter's own layout (rows x cols, batch_stride).  Entries may be NULL. */
mona_status mona_step_ex(mona_handle* h, const mona_hparams* hp,
                         void* const* params, const void* const* grads, void* const* o_out,
                         uint32_t phase_mask, void* stream);

/* End-to-end variant for callers whose gradients arrive in HOST memory: for every descriptor copies
 * grads_host[i] (pinned host memory, same layout and dtype as the device gradient, batch*batch_stride
 * elements) into grads[i], runs the step, and copies the updated parameters back to params_host[i]
 * (pinned, fp32).  The copies run on two streams the handle owns, pipelined with the step: a chunk starts
 * as soon as the gradients of its descriptors have arrived, and a descriptor is copied back as soon as its
 * last matrix is updated, so both transfer directions overlap the computation.  All of it is ordered after
 * what `stream` held at the call and joined back into `stream` before the call returns; nothing
 * synchronises the host. */
mona_status mona_step_host(mona_handle* h, const mona_hparams* hp,
                           void* const* params, void* const* grads,
                           const void* const* grads_host, void* const* params_host, void* stream);

/* Synchronises `stream` and reads the device status word.  Returns MONA_OK, MONA_ERR_NONFINITE or
 * MONA_ERR_TIMEOUT; *first_bad_matrix (may be NULL) receives the lowest global matrix index that
 * reported a problem, or -1.  The word is cleared by the call. */
mona_status mona_poll_status(mona_handle* h, void* stream, int64_t* first_bad_matrix);

/* Failure-detection self-test: enqueues one Newton-Schulz launch (a single X X^T phase) whose shared-memory stages are made to
 * expect 16 bytes more than their copies deliver.  Nothing faults - every copy completes - but the wait for a
 * full stage can never end, so it must run out after its bound (about half a second), latch the time-out in the
 * status word and leave the kernel cleanly.  Afterwards mona_poll_status() returns MONA_ERR_TIMEOUT once and
 * the handle works as before.  Only the first workspace slot is written (with meaningless values); parameters
 * and state are not touched.  Needs at least one descriptor that takes the tensor-core path. */
mona_status mona_selftest_timeout(mona_handle* h, void* stream);

/* Byte offsets inside the state block of M, A and G_prev of matrix 0 of descriptor `desc`.  Matrix b
 * of the descriptor follows at b * rows * cols * (element size) bytes from each offset: 4 for M, and 4
 * or 2 for A and G_prev according to the descriptor's state_dtype (state is stored densely, whatever
 * batch_stride is).  A checkpoint is the state block plus the caller's own step count. */
mona_status mona_state_layout(const mona_handle* h, int64_t desc,
                              size_t* off_M, size_t* off_A, size_t* off_Gprev);

/* Number of kernels the most recent mona_step*() call launched (for launch accounting). */
int64_t mona_last_launch_count(const mona_handle* h);

/* Counts of executed tensor-core work of the most recent step: bf16 multiply-add flops actually
 * issued (2 * M * N * K summed over issued 256 x 256 tile MMAs: padding and the upper halves of diagonal tiles
 * count) and the dense-equivalent figure (4 s^2 l + 2 s^3 per matrix and iteration).  Either pointer may be NULL. */
mona_status mona_last_ns_flops(const mona_handle* h, double* executed, double* dense_equivalent);
/* The work the iteration itself needs when both symmetric products are computed once per pair of entries:
 * 3 s^2 l + s^3 per matrix and iteration (tensor-core path only). */
mona_status mona_last_ns_useful_flops(const mona_handle* h, double* useful);

/* The order in which the Newton-Schulz kernel hands out its work items (tiles), computed on the HOST with the cursor
 * the kernel's scheduler uses; no device is needed.  The paper has no counterpart: this exposes the property the
 * kernel's freedom from deadlock rests on - every item comes after all items it depends on (GEMM q of a matrix after
 * all items of GEMM q - 1 of that matrix) - so that it can be tested for any launch shape.
 *   n_matrices, n_phases (1..15), delay (>= 1, see mona_options.ns_delay), items_per_phase[n_phases]: items per matrix.
 * Writes (matrix, phase, item) triples of the items start, start + stride, start + 2 stride, ... (one CTA pair sees such
 * a subsequence) into the HOST array out_cqt (3 int32 per item), at most `capacity` items; *n_written receives the
 * count.  MONA_ERR_INVALID_ARG for null pointers or non-positive sizes. */
mona_status mona_work_order(int32_t n_matrices, int32_t n_phases, int32_t delay, const uint32_t* items_per_phase,
                            uint32_t start, uint32_t stride, int32_t* out_cqt, size_t capacity, size_t* n_written);

/* Profiling build only (library compiled with -DMONA_TRACE; every other build returns MONA_ERR_NOT_BUILT and
 * touches nothing).  The paper has no counterpart: this is the instrument behind the per-role wait times quoted
 * for the Newton-Schulz kernel.  In that build every role of the kernel (TMA producer, MMA issuer, scheduler,
 * epilogue warps, store warp) adds up the SM clock cycles its waits took, and the MMA issuer the cycles and
 * k-slices (64 of the inner dimension) per kind of tile; the arithmetic is unchanged, the kernel a few per
 * cent slower.  One row of MONA_TRACE_SLOTS 64-bit words per CTA (row = block index; even rows are the CTAs
 * that issue the MMAs and schedule), summed over all launches since the last reset.
 * mona_trace_read() synchronises the device, copies the first `rows` rows (at most MONA_TRACE_ROWS) to the
 * HOST array `out` (rows * MONA_TRACE_SLOTS words; may be NULL with rows = 0) and clears the table when
 * `reset` is non-zero.  Not thread-safe against running steps of other threads. */
#define MONA_TRACE_ROWS 160
#define MONA_TRACE_SLOTS 64
typedef enum mona_trace_slot {
    MONA_TRACE_KERNEL = 0,            /* launch start to the end of the producer's role                        */
    MONA_TRACE_PRODUCER_EMPTY = 1,    /* producer: waiting for free operand slabs                              */
    MONA_TRACE_PRODUCER_RING = 2,     /* producer: waiting for the next published work item                    */
    MONA_TRACE_PRODUCER_ROLE = 3,     /* producer: whole role                                                  */
    MONA_TRACE_MMA_RING = 4,          /* MMA issuer: waiting for the next published work item                  */
    MONA_TRACE_MMA_ROLE = 5,          /* MMA issuer: whole role                                                */
    MONA_TRACE_SCHED_DEPENDENCY = 6,  /* scheduler: waiting for the previous GEMM of an item's matrix          */
    MONA_TRACE_SCHED_SLOT = 7,        /* scheduler: waiting for a free slot of the item ring (it is ahead)     */
    MONA_TRACE_SCHED_ROLE = 8,        /* scheduler: whole role                                                 */
    MONA_TRACE_EPI_ACC_FULL = 9,      /* epilogue: waiting for a finished accumulator (sum over 8 warps)       */
    MONA_TRACE_EPI_STAGE_EMPTY = 10,  /* epilogue: waiting for the staging buffer (sum over 8 warps)           */
    MONA_TRACE_EPI_RING = 11,         /* epilogue: waiting for the next published item (sum over 8 warps)      */
    MONA_TRACE_EPI_ROLE = 12,         /* epilogue: whole role (sum over 8 warps)                               */
    MONA_TRACE_STORE_STAGED = 13,     /* store warp: waiting for a staged 128-column phase                     */
    MONA_TRACE_STORE_ROLE = 14,       /* store warp: whole role                                                */
    MONA_TRACE_ITEMS = 15,            /* work items completed by this CTA (a count, not cycles)                */
    MONA_TRACE_TILE0 = 16,            /* + 4 * kind + {0: cycles of the MMA issuer inside tiles of the kind, 1: their
                                         k-slices (a count), 2: of the cycles, waiting for operands, 3: waiting for an
                                         accumulator}; kind 0 / 1: X X^T off / on the diagonal, 2 / 3: b A + c A^2 + a I
                                         off / on the diagonal, 4: 256 x 512 macro-tile of X' = B' X, 5: single tile of it */
    MONA_TRACE_EPI_TILE0 = 40         /* + 4 * kind + {0: cycles of an epilogue warp inside items of the kind, 1: items (a
                                         count), 2: of the cycles, waiting for accumulators, 3: waiting for the staging
                                         buffer}, sums over the 8 epilogue warps                                      */
} mona_trace_slot;
mona_status mona_trace_read(unsigned long long* out, size_t rows, int reset);

/* Allocation-free prologue for ONE matrix.  The paper has no counterpart to this entry point; it exists
 * for integration reasons only.  It performs lines 4-7 and 10 of Algorithm 1 on a rows x cols matrix
 * (A, M, G_prev updated in place from `grad`, all device pointers, 16-byte aligned, dense row-major),
 * writes 1 / (||M_k||_F + eps) to inv_norm_out[0] (device) and, when xhat_bf16 is not NULL, the bf16
 * copy of M_k there.  Results equal those of the prologue phase of mona_step_ex().
 *
 * Who needs it: callers that cannot get device memory when they call us - for instance a trainer whose
 * framework allocator already owns all of HBM, or a hook running where the device-wide stall of
 * cudaMalloc/cudaFree is not acceptable.  This function calls no allocator of any kind.  The few hundred
 * scratch words the reduction needs (slab partial sums and an arrival counter) sit in a 2 KiB array
 * compiled into the library, resident on every GPU that loads the library until the process ends.
 *
 * Limits and rules:
 *   - rows * cols <= 16,777,216 (one 4096 x 4096 matrix); larger inputs are refused with
 *     MONA_ERR_UNSUPPORTED_SHAPE and an explanatory message in `err`.
 *   - It works on the CURRENT device; all pointers must belong to it.  The first call on each device
 *     looks up the device address of the built-in array; make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps the previous call's contents (the function
 *     re-zeroes the counter it depends on).  Two calls whose kernels may overlap on the GPU - different
 *     streams, no ordering between them - race on it; order them yourself.
 *   - hp->algorithm must be 0 (the plain-Muon prologue has no acceleration state to update).
 *   - There is no status word to poll here.  A gradient or state holding inf/nan shows in the result itself:
 *     a finite ||M_k||_F always gives a positive finite inv_norm_out[0]; a non-finite one gives 0 (norm = inf)
 *     or nan.  Test inv_norm_out[0] before using M_k.
 *   - A device that is not compute capability 10.x is refused with MONA_ERR_ARCH.
 *   - `err` (may be NULL) receives a NUL-terminated message of at most err_len bytes.
 * Enqueued on `stream`; does not synchronise. */
mona_status mona_prologue_noalloc(const void* grad, int32_t grad_dtype, float* M, float* A, float* G_prev,
                                  void* xhat_bf16, float* inv_norm_out, int64_t rows, int64_t cols,
                                  const mona_hparams* hp, void* stream, char* err, size_t err_len);

/* Human-readable detail of the last failing call on this handle (never NULL). */
const char* mona_last_error(const mona_handle* h);

/* Frees the handle's tables, stream and events.  The caller's buffers are untouched. */
void mona_destroy(mona_handle* h);

#ifdef __cplusplus
}
#endif
#endif /* MONA_H_ */
