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

// ---------------------------------------------------------------------------------------------------
// Small matrices (shorter side <= 64, e.g. a 32 x 1024 router): the whole Newton-Schulz iteration of one
// matrix in ONE block.  The matrix lives in shared memory in its wide orientation Y (s x l, tall inputs
// are transposed while loading), and every iteration forms A = Y Y^T, B' = b A + c A^2 + a I and
// Y <- B' Y there, in plain fp32 FMA.  One launch replaces the scale pass and 3T batched SGEMMs, each of
// which would have had a single block per matrix to work with.
constexpr int SMALL_THREADS = 256;

template <int SMAX>   // upper bound of the shorter side s: 32 or 64 (register arrays are sized by it)
__global__ void __launch_bounds__(SMALL_THREADS)
small_ns_kernel(const float* __restrict__ M, float* __restrict__ O, const float* __restrict__ inv_norm, int rows, int cols,
                int T, float ca, float cb, float cc) {
    extern __shared__ float sm[];
    const bool tall = rows > cols;
    const int s = tall ? cols : rows, l = tall ? rows : cols;
    const int lp = l | 1;                 // odd pitch: the transposing load/store of tall inputs stays conflict-free
    const int sp = s + 1;
    float* Y = sm;
    float* A = Y + (size_t)s * lp;
    float* B = A + s * sp;
    const long long e = (long long)rows * cols;
    const float* Mz = M + (long long)blockIdx.x * e;
    float* Oz = O + (long long)blockIdx.x * e;
    const float scale = inv_norm[blockIdx.x];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    for (long long idx = tid; idx < e; idx += SMALL_THREADS) {          // X_0 = M / (||M||_F + eps)
        const int r = (int)(idx / cols), q = (int)(idx - (long long)r * cols);
        const float v = Mz[idx] * scale;
        if (!tall) Y[r * lp + q] = v; else Y[q * lp + r] = v;
    }
    __syncthreads();

    const int nb = (s + 3) >> 2;          // 4 x 4 blocks of A per side
    const int nblocks = nb * (nb + 1) / 2;
    for (int t = 0; t < T; ++t) {
        // A = Y Y^T: a warp owns a 4 x 4 block on or below the diagonal, its lanes split the l products
        for (int blk = warp; blk < nblocks; blk += SMALL_THREADS / 32) {
            int bi = 0;
            while ((bi + 1) * (bi + 2) / 2 <= blk) ++bi;
            const int bj = blk - bi * (bi + 1) / 2;
            float acc[4][4];
            #pragma unroll
            for (int r = 0; r < 4; ++r)
                #pragma unroll
                for (int q = 0; q < 4; ++q) acc[r][q] = 0.f;
            for (int k = lane; k < l; k += 32) {
                float ya[4], yb[4];
                #pragma unroll
                for (int r = 0; r < 4; ++r) {
                    ya[r] = (4 * bi + r < s) ? Y[(4 * bi + r) * lp + k] : 0.f;
                    yb[r] = (4 * bj + r < s) ? Y[(4 * bj + r) * lp + k] : 0.f;
                }
                #pragma unroll
                for (int r = 0; r < 4; ++r)
                    #pragma unroll
                    for (int q = 0; q < 4; ++q) acc[r][q] = fmaf(ya[r], yb[q], acc[r][q]);
            }
            #pragma unroll
            for (int r = 0; r < 4; ++r)
                #pragma unroll
                for (int q = 0; q < 4; ++q) {
                    float v = acc[r][q];
                    #pragma unroll
                    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                    const int i = 4 * bi + r, j = 4 * bj + q;
                    if (lane == 0 && i < s && j < s) { A[i * sp + j] = v; A[j * sp + i] = v; }
                }
        }
        __syncthreads();
        // B' = b A + c A A + a I
        for (int idx = tid; idx < s * s; idx += SMALL_THREADS) {
            const int i = idx / s, j = idx - i * s;
            float sum = 0.f;
            for (int k = 0; k < s; ++k) sum = fmaf(A[i * sp + k], A[k * sp + j], sum);
            B[i * sp + j] = fmaf(cb, A[i * sp + j], cc * sum) + (i == j ? ca : 0.f);
        }
        __syncthreads();
        // Y <- B' Y: a thread owns NCOL columns, keeps them in registers and overwrites them in place
        constexpr int NCOL = SMAX <= 32 ? 4 : 2;
        for (int c0 = tid * NCOL; c0 < l; c0 += SMALL_THREADS * NCOL) {
            float y[NCOL][SMAX];
            #pragma unroll
            for (int k = 0; k < SMAX; ++k)
                #pragma unroll
                for (int u = 0; u < NCOL; ++u) y[u][k] = (k < s && c0 + u < l) ? Y[k * lp + c0 + u] : 0.f;
            for (int i = 0; i < s; ++i) {
                float o[NCOL];
                #pragma unroll
                for (int u = 0; u < NCOL; ++u) o[u] = 0.f;
                #pragma unroll
                for (int k = 0; k < SMAX; ++k) {
                    const float bik = k < s ? B[i * sp + k] : 0.f;
                    #pragma unroll
                    for (int u = 0; u < NCOL; ++u) o[u] = fmaf(bik, y[u][k], o[u]);
                }
                #pragma unroll
                for (int u = 0; u < NCOL; ++u)
                    if (c0 + u < l) Y[i * lp + c0 + u] = o[u];
            }
        }
        __syncthreads();
    }
    for (long long idx = tid; idx < e; idx += SMALL_THREADS) {          // O = X_T, back in the input's orientation
        const int r = (int)(idx / cols), q = (int)(idx - (long long)r * cols);
        Oz[idx] = !tall ? Y[r * lp + q] : Y[q * lp + r];
    }
}

size_t small_ns_smem(long long s, long long l) { return (size_t)(s * (l | 1) + 2 * s * (s + 1)) * sizeof(float); }

}  // namespace

bool small_ns_eligible(long long rows, long long cols) {
    const long long s = rows < cols ? rows : cols, l = rows < cols ? cols : rows;
    return s <= 64 && small_ns_smem(s, l) <= 200 * 1024;
}

cudaError_t small_ns_configure() {
    cudaError_t e = cudaFuncSetAttribute(small_ns_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(small_ns_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
}

cudaError_t launch_small_ns(const float* M, float* O, const float* inv_norm, int batch, int rows, int cols, int T,
                            float a, float b, float c, cudaStream_t stream) {
    const long long s = rows < cols ? rows : cols, l = rows < cols ? cols : rows;
    const size_t smem = small_ns_smem(s, l);
    if (s <= 32) small_ns_kernel<32><<<batch, SMALL_THREADS, smem, stream>>>(M, O, inv_norm, rows, cols, T, a, b, c);
    else         small_ns_kernel<64><<<batch, SMALL_THREADS, smem, stream>>>(M, O, inv_norm, rows, cols, T, a, b, c);
    return cudaGetLastError();
}

cudaError_t launch_sgemm(const SgemmArgs& g, cudaStream_t stream) {
    dim3 grid((g.N + TS - 1) / TS, (g.M + TS - 1) / TS, g.batch);
    sgemm_kernel<<<grid, 256, 0, stream>>>(g);
    return cudaGetLastError();
}

}  // namespace mona
