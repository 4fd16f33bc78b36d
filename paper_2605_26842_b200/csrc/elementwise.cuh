// Launchers of the elementwise passes (definitions in elementwise.cu).
#pragma once
#include "common.cuh"

namespace mona {

// Fused prologue over a chunk of C same-shape matrices (state stored densely, e elements each):
// updates A, M, G_prev in place from the gradient, optionally writes bf16(M) to `xhat` (null to skip),
// and leaves 1/(||M||_F + eps) of matrix c in inv_norm[c].  `state_kind` says how the acceleration state is kept:
// fp32, bfloat16 (MONA-Lite storage), as the single fp32 buffer Z = beta_a A - (1 - beta_a) G passed in `A`
// (`Gp` ignored), or not at all (plain Muon step, M = mu M + G; A and Gp are ignored).
// M is always fp32.  `partials` holds C*MAX_SLABS floats and
// `counters` C zero-initialised words of scratch.
enum { PROLOGUE_AUX_F32 = 0, PROLOGUE_AUX_BF16 = 1, PROLOGUE_NO_AUX = 2, PROLOGUE_AUX_COMBINED = 3 };
cudaError_t launch_prologue(const ChunkPtrs& ptrs, int C, bool grad_bf16, int state_kind, bool vec4, float* M, void* A, void* Gp,
                            __nv_bfloat16* xhat, float* partials, unsigned int* counters, float* inv_norm,
                            DeviceStatus* status, long long e, long long slab_len, int slabs,
                            const PrologueScalars& k, cudaStream_t stream);

// Parameter update W <- (W - eta*lambda*W) - eta*gamma*O for a chunk; O is bf16 or fp32, dense, e per matrix.
cudaError_t launch_update(const ChunkPtrs& ptrs, int C, bool o_is_bf16, bool vec4, const void* O, long long e,
                          long long slab_len, int slabs, float eta_lambda, float eta_gamma, cudaStream_t stream);

// X_0 = M * inv_norm for the fp32 validation path.
cudaError_t launch_scale(const float* M, float* X, const float* inv_norm, int C, long long e, long long slab_len,
                         int slabs, cudaStream_t stream);

}  // namespace mona
