// Tensor-core Newton-Schulz GEMMs (definitions in ns_tc.cu): tcgen05.mma with TMA-staged bf16 tiles and
// fp32 accumulators in tensor memory.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace mona {

constexpr int TC_BM = 128;      // rows of D per tile (UMMA M, one CTA)
constexpr int TC_BN = 256;      // max columns of D per tile (UMMA N <= 256)
constexpr int TC_BK = 64;       // k-slice per pipeline stage: 64 bf16 = one 128-byte swizzle row
constexpr int TC_BOX = 64;      // every TMA box is 64 (contiguous) x 64 (strided) bf16 = 8 KiB
constexpr int TC_STAGES = 4;

// One batched GEMM of the iteration of Eq. newton_schulz over the C matrices of a chunk:
//     D = post * (c1 * Cin + c2 * Aop x Bop^T) + diag_add * I,   D, Cin bf16; accumulation fp32.
// Operand tiles come through the two tensor maps.  An operand is "K-major" when k is its contiguous
// index (tensor map dims {K, rows, C}) and "MN-major" when its row index is contiguous (dims {rows, K, C});
// tall weights use the MN-major form so that X^T X and B X need no transposed copy.
// With `symmetric` set only the tiles that touch the lower triangle are computed and the strictly
// lower 128-blocks are mirrored into the upper triangle by the epilogue.
struct TcGemm {
    int C;                      // matrices in the launch
    int M, N, K;                // per-matrix GEMM extents
    int a_mn, b_mn;             // 1: operand is MN-major
    int symmetric;              // 1: D = D^T (X X^T, X^T X, A A)
    int tiles_m, tiles_n, tiles_per_mat;
    const __nv_bfloat16* cin;   // may be null
    __nv_bfloat16* out;
    long long ld, mat_stride;   // leading dimension and per-matrix stride of cin/out, in elements
    float c1, c2;
    float diag_add;             // added to D(i,i): folds the a*X term of the quintic into B' = b A + c A^2 + a I
    const float* inv_norm;      // per-matrix 1/(||M||_F + eps), used when post_mode != 0
    int post_mode;              // 0: post = 1, 1: post = inv, 2: post = inv^2
};

// Fills the tile counts of `g` from M, N, symmetric.
void tc_gemm_plan(TcGemm& g);
// Tensor-core flops (2*M*N*K per issued MMA, padded extents included) one launch of `g` executes.
double tc_gemm_executed_flops(const TcGemm& g);

// Dynamic shared memory the kernel needs; call once per process before the first launch.
cudaError_t tc_gemm_configure();
cudaError_t launch_tc_gemm(const CUtensorMap& tma_a, const CUtensorMap& tma_b, const TcGemm& g, int num_sms,
                           DeviceStatus* status, cudaStream_t stream);

}  // namespace mona
