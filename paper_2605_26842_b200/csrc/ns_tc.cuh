// Tensor-core Newton-Schulz iteration (definitions in ns_tc.cu): one persistent kernel per chunk runs all
// GEMMs of up to five iterations of Eq. newton_schulz.  tcgen05.mma is issued for a pair of CTAs
// (cta_group::2), operands are TMA-staged bf16 tiles, accumulators are fp32 in tensor memory.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace mona {

constexpr int TC_BM = 256;      // rows of D per tile: one CTA pair, 128 rows per CTA (UMMA M = 256)
constexpr int TC_BN = 256;      // columns of D per tile (UMMA N = 256, each CTA stages 128 of them)
constexpr int TC_BK = 64;       // k-slice per pipeline stage: 64 bf16 = one 128-byte swizzle row
constexpr int TC_BOX = 64;      // every TMA box is 64 bf16 wide (one 128-byte swizzle row) and 64 or 128 rows high
constexpr int NS_MAX_PHASES = 15;   // 3 GEMMs x 5 iterations per launch; longer iterations take several launches
constexpr int NS_TENSORS = 4;       // operand tensors of a chunk: X ping, X pong, A, B'
constexpr int NS_MAPS = 2 * NS_TENSORS;   // each with 64-row boxes (index t) and with 128-row boxes (index t + NS_TENSORS)

// One batched GEMM ("phase") of the iteration of Eq. newton_schulz over the C matrices of a chunk:
//     D = post * (c1 * Cin + c2 * Aop x Bop^T) + diag_add * I,   D, Cin bf16; accumulation fp32.
// Operand tiles are fetched, and D is stored, through tensor maps over [C][rows][cols] bf16 tensors; Cin is
// addressed directly.  An operand is "K-major" when k is its contiguous index and "MN-major" when its row index is
// contiguous; tall weights use the MN-major form so that X^T X and X B' need no transposed copy.
//
// Symmetric matrices (X X^T, b A + c A^2 + a I) are only ever stored in their lower block triangle:
// with `symmetric` set, only the 256 x 256 tiles with tile row >= tile column are computed and
// written (diagonal tiles completely).  A consumer that needs a block above the diagonal fetches the
// stored block below it as an MN-major operand instead (`a_sym` / `b_sym`), so nothing is mirrored.
//
// With `fuse_update` set (the last X' = B' X of a step) D is not stored: the epilogue applies
// Eq. muon_update, W <- (W - eta lambda W) - eta gamma D, to the fp32 parameter of the same matrix
// straight from the fp32 accumulator, and writes D itself (fp32) only where an output pointer is given.
struct NsPhase {
    int M, N, K;                // per-matrix GEMM extents
    int a_map, b_map, d_map;    // which of the chunk's tensors (0 .. NS_TENSORS-1) the operands come from and the output goes to
    int a_mn, b_mn;             // 1: operand is MN-major (ignored for an operand flagged *_sym)
    int a_sym, b_sym;           // 1: operand is a symmetric matrix stored as its lower block triangle
    int symmetric;              // 1: D = D^T, compute lower-triangle tiles only
    int ab_same;                // 1: both operands are the same tensor in the same form (X X^T, A A): a diagonal
                                //    tile stages its operand rows once and uses them on both sides
    int wide;                   // 1 (non-symmetric D only): a work item is a 256 x 512 macro-tile, two tiles that share
                                //    one staged slice of the A operand, one per tensor-memory accumulator
    int tiles_m, tiles_n, items_per_mat;   // filled by ns_phase_plan(); items are macro-tiles when `wide`
    const __nv_bfloat16* cin;   // may be null; [C][M][N] like D; lower-block-stored when D is symmetric
    long long ld, mat_stride;   // leading dimension and per-matrix stride of cin (and of the fp32 parameter when
                                // fuse_update), in elements
    float c1, c2;
    float diag_add;             // added to D(i,i): folds the a*X term of the quintic into B' = b A + c A^2 + a I
    int post_mode;              // 0: post = 1, 1: post = inv_norm[c], 2: post = inv_norm[c]^2
    int fuse_update;            // 1: epilogue applies the parameter update instead of storing D
};

// Everything one launch needs: the phases in execution order and the scheduler state.  Work items are handed
// out through one atomic counter in a fixed order in which every item comes after the items it depends on
// (phase q of matrix c follows phase q - 1 of matrix c by `delay` matrices), so a pair that has taken an item
// only ever waits for items already taken by running pairs; completion of a phase of a matrix is counted in
// done[c * P + q] (two arrivals per item, one from each CTA of the pair).
struct NsProgram {
    int C;                      // matrices in the chunk
    int P;                      // phases in this launch (<= NS_MAX_PHASES)
    int delay;                  // distance, in matrices, between consecutive phases of one matrix in the item order
    unsigned int total_items;
    NsPhase ph[NS_MAX_PHASES];
    const float* inv_norm;      // per-matrix 1/(||M||_F + eps), used when post_mode != 0
    unsigned int* work_counter; // zero at launch
    unsigned int* done;         // C * P words, zero at launch
    float eta_lambda, eta_gamma;    // fuse_update: eta * lambda and eta * gamma
    int selftest_extra_tx;      // 0 in normal use.  The time-out self-test sets it: every stage then expects this many
                                //    bytes more than its copies deliver, so the "full" wait runs out and the kernel must
                                //    report STATUS_TIMEOUT and leave cleanly (all copies still complete; nothing faults)
};

// The kernel's work order, as a cursor that only moves forward (host and device).
//     for tau = 0, 1, ...: for q = 0 .. P-1: the items of phase q of matrix c = tau - delay * q, where that matrix exists,
// i.e. for q_lo(tau) <= q <= q_hi(tau) with q_hi = min(P - 1, tau / delay) (c >= 0) and q_lo = ceil((tau - C + 1) / delay)
// (c < C).  Phase q of matrix c therefore comes `delay` values of tau after phase q - 1 of the same matrix: every item follows
// all items it depends on.  The cursor advances a whole tau at a time and keeps q_lo and q_hi incrementally, so finding an
// item costs a few reads of `first` (no divisions) however many items lie between two calls.
// `first[q]`, q = 0 .. P: items per matrix of the phases before phase q (first[0] = 0).
struct NsItemCursor {
    int C, P, delay;
    int tau = 0, q_lo = 0, q_hi = 0, lo_cnt = 0, hi_cnt = 0;
    unsigned base = 0;                  // index of the first item of the current tau
    __host__ __device__ NsItemCursor(int C_, int P_, int delay_) : C(C_), P(P_), delay(delay_) {}
    // Finds item `idx`, which must not be smaller than any index asked before.  False when the walk runs past the last
    // group without reaching it (idx is not an item of the launch).
    __host__ __device__ bool find(unsigned idx, const volatile unsigned int* first, int& c, int& q, int& t) {
        while (true) {
            const unsigned n_tau = q_lo <= q_hi ? first[q_hi + 1] - first[q_lo] : 0u;
            if (idx < base + n_tau) break;
            if (tau >= C + P * delay) return false;
            base += n_tau;
            ++tau;
            if (++hi_cnt == delay) { hi_cnt = 0; if (q_hi < P - 1) ++q_hi; }
            if (tau == C) { q_lo = 1; lo_cnt = 0; }
            else if (tau > C && ++lo_cnt == delay) { lo_cnt = 0; ++q_lo; }
        }
        const unsigned r = idx - base + first[q_lo];       // counted from phase 0 of this tau
        q = q_lo;
        while (first[q + 1] <= r) ++q;                      // ends at q <= q_hi since r < first[q_hi + 1]
        t = (int)(r - first[q]);
        c = tau - delay * q;
        return true;
    }
};

// Layout of the profiling build's table (-DMONA_TRACE): one row per CTA (blockIdx.x; even rows are the leaders, which
// alone run the MMA issuer and the scheduler), NS_TRACE_SLOTS 64-bit words per row, all in SM clock cycles unless noted,
// summed over the launches since the last reset.
constexpr int NS_TRACE_ROWS = 160;
constexpr int NS_TRACE_SLOTS = 64;
enum NsTraceSlot {
    NS_TRACE_KERNEL = 0,            // launch start to the end of the producer's role
    NS_TRACE_PRODUCER_EMPTY = 1,    // producer: waiting for free operand slabs
    NS_TRACE_PRODUCER_RING = 2,     // producer: waiting for the next published item
    NS_TRACE_PRODUCER_ROLE = 3,     // producer: whole role
    NS_TRACE_MMA_RING = 4,          // MMA issuer: waiting for the next published item
    NS_TRACE_MMA_ROLE = 5,          // MMA issuer: whole role
    NS_TRACE_SCHED_DEPENDENCY = 6,  // scheduler: waiting for the previous phase of an item's matrix
    NS_TRACE_SCHED_SLOT = 7,        // scheduler: waiting for a free slot of the item ring (it is ahead of the pipeline)
    NS_TRACE_SCHED_ROLE = 8,        // scheduler: whole role
    NS_TRACE_EPI_ACC_FULL = 9,      // epilogue: waiting for a finished accumulator (sum over the 8 warps)
    NS_TRACE_EPI_STAGE_EMPTY = 10,  // epilogue: waiting for the staging buffer (sum over the 8 warps)
    NS_TRACE_EPI_RING = 11,         // epilogue: waiting for the next published item (sum over the 8 warps)
    NS_TRACE_EPI_ROLE = 12,         // epilogue: whole role (sum over the 8 warps)
    NS_TRACE_STORE_STAGED = 13,     // store warp: waiting for a staged phase
    NS_TRACE_STORE_ROLE = 14,       // store warp: whole role
    NS_TRACE_ITEMS = 15,            // work items completed by this CTA (a count)
    NS_TRACE_TILE0 = 16,            // 6 kinds of tile x {cycles of the MMA issuer inside the tile, k-slices (a count), of which
                                    // waiting for operands, of which waiting for an accumulator}; kinds: 0/1 X X^T off/on the
                                    // diagonal, 2/3 b A + c A^2 + a I off/on the diagonal, 4 macro-tile and 5 single tile of X' = B' X
    NS_TRACE_EPI_TILE0 = 40         // the same 6 kinds x {cycles of an epilogue warp inside items of the kind, items (a count), of
                                    // which waiting for accumulators, of which waiting for the staging buffer}, sums over the 8 warps
};
static_assert(NS_TRACE_EPI_TILE0 + 4 * 6 <= NS_TRACE_SLOTS, "profiling table");

struct alignas(64) NsMaps {
    CUtensorMap m[NS_MAPS];
};

// Per-matrix parameter and optional fp32 output pointers for a phase with fuse_update: HOST arrays of C device
// pointers (copied into the launch's arguments).  w == nullptr: no phase of the launch fuses the update.
struct NsUpdatePtrs {
    float* const* w;
    float* const* o;            // entries may be null; the array itself may be null
};

// Fills the tile counts of `p` from M, N, symmetric, wide.
void ns_phase_plan(NsPhase& p);
// Tensor-core flops one matrix costs in phase `p`: executed (2*M*N*K per issued 256 x 256 tile MMA, padded
// extents and the upper halves of diagonal tiles included).
double ns_phase_executed_flops(const NsPhase& p);
// Fills total_items from C, P, the phases' item counts.
void ns_program_plan(NsProgram& g);
// Words of scheduler scratch (work counter + done counters) a launch over C matrices and P phases needs zeroed.
inline size_t ns_sched_words(int C, int P) { return 64 + (size_t)C * P; }

// Sets the kernel's shared-memory attribute and finds how many CTA pairs the device holds at once.
// Call once per device before the first launch.
cudaError_t ns_configure(int* max_pairs);
// Host-side walk of the work order of a launch over C matrices and P phases with `items_per_phase[q]` items per matrix:
// writes (c, q, t) of the items start, start + stride, ... into `cqt` (3 ints per item, at most `capacity` items) with the
// cursor the kernel's scheduler uses.  Returns the number written, -1 for bad arguments, -2 if the walk fails.
int ns_work_order(int C, int P, int delay, const unsigned int* items_per_phase, unsigned start, unsigned stride, int* cqt,
                  size_t capacity);
// Copies the first `rows` rows of the profiling table to `out` (host) after synchronising the device, and clears the table
// when `reset` is set.  *available = 0 (and nothing else happens) unless the library was built with -DMONA_TRACE.
cudaError_t ns_trace_read(unsigned long long* out, size_t rows, int reset, int* available);
cudaError_t launch_ns_program(const NsMaps& maps, const NsProgram& g, const NsUpdatePtrs& upd, int max_pairs,
                              DeviceStatus* status, cudaStream_t stream);

}  // namespace mona
