// fp32 validation path of Eq. newton_schulz: a plain shared-memory tiled SGEMM with generic operand
// strides, so that X X^T, X^T X, A A and B X / X B all go through the same kernel without any
// transposed copy.  Accumulation is sequential fp32 FMA; this path exists to separate algorithmic
// errors from bf16 rounding, and to serve shapes the tensor-core path does not take.
#include "ns_fp32.cuh"

namespace mona {

namespace {

constexpr int TS = 64;   // tile of D per block
constexpr int TK = 16;   // k-slice
// 256 threads, each owns a 4x4 patch of the 64x64 tile.
__global__ void __launch_bounds__(256) sgemm_kernel(SgemmArgs g) {
    __shared__ float As[TK][TS + 4];
    __shared__ float Bs[TK][TS + 4];
    const int z = blockIdx.z;
    const float* __restrict__ A = g.a + (long long)z * g.a_batch;
    const float* __restrict__ B = g.b + (long long)z * g.b_batch;
    const int i0 = blockIdx.y * TS, j0 = blockIdx.x * TS;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    float acc[4][4];
    #pragma unroll
    for (int r = 0; r < 4; ++r)
        #pragma unroll
        for (int c = 0; c < 4; ++c) acc[r][c] = 0.f;

    for (int k0 = 0; k0 < g.K; k0 += TK) {
        // each thread brings 4 elements of each operand slice
        #pragma unroll
        for (int q = 0; q < 4; ++q) {
            int idx = threadIdx.x + q * 256;          // 0..1023 = TK*TS
            int kk, mm;
            if (g.a_sk == 1) { kk = idx % TK; mm = idx / TK; } else { mm = idx % TS; kk = idx / TS; }
            int gi = i0 + mm, gk = k0 + kk;
            As[kk][mm] = (gi < g.M && gk < g.K) ? A[(long long)gi * g.a_si + (long long)gk * g.a_sk] : 0.f;
            int kb, nn;
            if (g.b_sk == 1) { kb = idx % TK; nn = idx / TK; } else { nn = idx % TS; kb = idx / TS; }
            int gj = j0 + nn, gk2 = k0 + kb;
            Bs[kb][nn] = (gj < g.N && gk2 < g.K) ? B[(long long)gk2 * g.b_sk + (long long)gj * g.b_sj] : 0.f;
        }
        __syncthreads();
        #pragma unroll
        for (int kk = 0; kk < TK; ++kk) {
            float a[4], b[4];
            #pragma unroll
            for (int r = 0; r < 4; ++r) a[r] = As[kk][ty * 4 + r];
            #pragma unroll
            for (int c = 0; c < 4; ++c) b[c] = Bs[kk][tx * 4 + c];
            #pragma unroll
            for (int r = 0; r < 4; ++r)
                #pragma unroll
                for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(a[r], b[c], acc[r][c]);
        }
        __syncthreads();
    }
    float* __restrict__ D = g.d + (long long)z * g.d_batch;
    const float* __restrict__ Cin = g.cin ? g.cin + (long long)z * g.d_batch : nullptr;
    #pragma unroll
    for (int r = 0; r < 4; ++r) {
        int gi = i0 + ty * 4 + r;
        if (gi >= g.M) continue;
        #pragma unroll
        for (int c = 0; c < 4; ++c) {
            int gj = j0 + tx * 4 + c;
            if (gj >= g.N) continue;
            long long off = (long long)gi * g.ldd + gj;
            float v = g.c2 * acc[r][c];
            if (Cin) v = fmaf(g.c1, Cin[off], v);
            D[off] = v;
        }
    }
}

}  // namespace

cudaError_t launch_sgemm(const SgemmArgs& g, cudaStream_t stream) {
    dim3 grid((g.N + TS - 1) / TS, (g.M + TS - 1) / TS, g.batch);
    sgemm_kernel<<<grid, 256, 0, stream>>>(g);
    return cudaGetLastError();
}

}  // namespace mona
