// Tensor-core Newton-Schulz GEMMs (definitions in ns_tc.cu): tcgen05.mma issued for a pair of CTAs
// (cta_group::2), TMA-staged bf16 tiles, fp32 accumulators in tensor memory, TMA-store epilogue.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace mona {

constexpr int TC_BM = 256;      // rows of D per tile: one CTA pair, 128 rows per CTA (UMMA M = 256)
constexpr int TC_BN = 256;      // columns of D per tile (UMMA N = 256, each CTA stages 128 of them)
constexpr int TC_BK = 64;       // k-slice per pipeline stage: 64 bf16 = one 128-byte swizzle row
constexpr int TC_BOX = 64;      // every TMA box is 64 (contiguous) x 64 (strided) bf16 = 8 KiB

// One batched GEMM of the iteration of Eq. newton_schulz over the C matrices of a chunk:
//     D = post * (c1 * Cin + c2 * Aop x Bop^T) + diag_add * I,   D, Cin bf16; accumulation fp32.
// Operand tiles and the output go through tensor maps over [C][rows][cols] bf16 tensors.  An operand
// is "K-major" when k is its contiguous index and "MN-major" when its row index is contiguous; tall
// weights use the MN-major form so that X^T X and B X need no transposed copy.
//
// Symmetric matrices (X X^T, b A + c A^2 + a I) are only ever stored in their lower block triangle:
// with `symmetric` set, only the 256 x 256 tiles with tile row >= tile column are computed and
// written (diagonal tiles completely).  A consumer that needs a block above the diagonal fetches the
// stored block below it as an MN-major operand instead (`a_sym` / `b_sym`), so nothing is mirrored.
struct TcGemm {
    int C;                      // matrices in the launch
    int M, N, K;                // per-matrix GEMM extents
    int a_mn, b_mn;             // 1: operand is MN-major (ignored for an operand flagged *_sym)
    int a_sym, b_sym;           // 1: operand is a symmetric matrix stored as its lower block triangle
    int symmetric;              // 1: D = D^T, compute lower-triangle tiles only
    int ab_same;                // 1: both operands are the same tensor in the same form (X X^T, A A): a diagonal
                                //    tile stages its operand rows once and uses them on both sides
    int wide;                   // 1 (non-symmetric D only): a pair computes 256 x 512 macro-tiles, two tiles that share
                                //    one staged slice of the A operand, one per tensor-memory accumulator
    int tiles_m, tiles_n, tiles_per_mat;   // tiles_per_mat counts macro-tiles when `wide`
    const __nv_bfloat16* cin;   // may be null; when D is symmetric, Cin is lower-block-stored like D
    long long ld, mat_stride;   // leading dimension and per-matrix stride of cin, in elements
    float c1, c2;
    float diag_add;             // added to D(i,i): folds the a*X term of the quintic into B' = b A + c A^2 + a I
    const float* inv_norm;      // per-matrix 1/(||M||_F + eps), used when post_mode != 0
    int post_mode;              // 0: post = 1, 1: post = inv, 2: post = inv^2
    int selftest_extra_tx;      // 0 in normal use.  The time-out self-test sets it: every stage then expects this many
                                //    bytes more than its copies deliver, so the "full" wait runs out and the kernel must
                                //    report STATUS_TIMEOUT and leave cleanly (all copies still complete; nothing faults)
};

// Fills the tile counts of `g` from M, N, symmetric, wide.
void tc_gemm_plan(TcGemm& g);
// Tensor-core flops (2*M*N*K per issued MMA, padded extents included) one launch of `g` executes.
double tc_gemm_executed_flops(const TcGemm& g);

// Sets the kernel's shared-memory attribute and finds how many CTA pairs the device holds at once.
// Call once per device before the first launch.
cudaError_t tc_gemm_configure(int* max_pairs);
// tma_a / tma_b: operand tensors, tma_d: output tensor (all bf16, 64 x 64 boxes, 128-byte swizzle).
cudaError_t launch_tc_gemm(const CUtensorMap& tma_a, const CUtensorMap& tma_b, const CUtensorMap& tma_d,
                           const TcGemm& g, int max_pairs, DeviceStatus* status, cudaStream_t stream);

}  // namespace mona
