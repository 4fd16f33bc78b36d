// fp32 validation Newton-Schulz GEMMs on the CUDA cores (definitions in ns_fp32.cu).
#pragma once
#include "common.cuh"

namespace mona {

// Batched D = c1 * Cin + c2 * (A x B) with generic strides, plain fp32 FMA (no tensor cores, no TF32):
//   A(i,k) = a[i*a_si + k*a_sk], B(k,j) = b[k*b_sk + j*b_sj], D(i,j) = d[i*ldd + j], Cin(i,j) = cin[i*ldd + j].
// Matrix z of the batch is offset by z*a_batch / z*b_batch / z*d_batch elements.  cin may be null.
struct SgemmArgs {
    const float* a; long long a_si, a_sk, a_batch;
    const float* b; long long b_sk, b_sj, b_batch;
    const float* cin; float* d; long long ldd, d_batch;
    int M, N, K, batch;
    float c1, c2;
};
cudaError_t launch_sgemm(const SgemmArgs& g, cudaStream_t stream);

// Whole Newton-Schulz iteration (Eq. newton_schulz, T steps, fp32 FMA) of `batch` small matrices, one
// block per matrix with the matrix resident in shared memory: O = NS_T(M * inv_norm).  M and O are dense
// [batch][rows][cols].  Only for shapes small_ns_eligible() accepts (shorter side <= 64 and the matrix
// within 200 KiB of shared memory); call small_ns_configure() once per device first.
bool small_ns_eligible(long long rows, long long cols);
cudaError_t small_ns_configure();
cudaError_t launch_small_ns(const float* M, float* O, const float* inv_norm, int batch, int rows, int cols, int T,
                            float a, float b, float c, cudaStream_t stream);

}  // namespace mona
