// Elementwise passes of the MONA step: the fused prologue (Algorithm 1 lines 4-7 and 10 plus the
// Frobenius norm that Eq. newton_schulz starts from) and the parameter update (line 9).
// Both are single HBM passes over contiguous slabs with 128-bit accesses.
#include "elementwise.cuh"

#include <math.h>

namespace mona {

namespace {

// 128-thread blocks of ~46 registers: small enough to run on an SM beside a resident CTA of the Newton-Schulz kernel
// (which leaves 7168 registers free), so the elementwise passes of one chunk overlap the GEMMs of another.
constexpr int EW_THREADS = 128;

__device__ __forceinline__ float mul_add2(F2 k, float x, float addend) {
    // (k.hi + k.lo) * x + addend with a single rounding on the dominant term
    return fmaf(k.hi, x, fmaf(k.lo, x, addend));
}

template <typename GT>
struct GradLoad;
template <>
struct GradLoad<float> {
    static __device__ __forceinline__ float4 load4(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
    static __device__ __forceinline__ float load1(const float* p) { return __ldcs(p); }
};
template <>
struct GradLoad<__nv_bfloat16> {
    static __device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
        uint2 raw = __ldcs(reinterpret_cast<const uint2*>(p));
        float4 r;
        r.x = __uint_as_float(raw.x << 16);
        r.y = __uint_as_float(raw.x & 0xffff0000u);
        r.z = __uint_as_float(raw.y << 16);
        r.w = __uint_as_float(raw.y & 0xffff0000u);
        return r;
    }
    static __device__ __forceinline__ float load1(const __nv_bfloat16* p) { return __bfloat162float(*p); }
};

// Storage format of the two auxiliary buffers A_k and G_{k-1}: fp32, or bfloat16 (MONA-Lite: the value is
// rounded once, to nearest even, when it is stored, and the stored value is what the step goes on with).
template <typename ST>
struct StateIO;
template <>
struct StateIO<float> {
    using elem = float;
    static constexpr bool has_gp = true;
    static __device__ __forceinline__ float4 load4(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
    static __device__ __forceinline__ void store4(float* p, float4 v) { __stcs(reinterpret_cast<float4*>(p), v); }
    static __device__ __forceinline__ float load1(const float* p) { return *p; }
    static __device__ __forceinline__ void store1(float* p, float v) { *p = v; }
    static __device__ __forceinline__ float round(float v) { return v; }
};
template <>
struct StateIO<__nv_bfloat16> {
    using elem = __nv_bfloat16;
    static constexpr bool has_gp = true;
    static __device__ __forceinline__ float4 load4(const __nv_bfloat16* p) { return GradLoad<__nv_bfloat16>::load4(p); }
    static __device__ __forceinline__ void store4(__nv_bfloat16* p, float4 v) {     // v holds already-rounded values
        __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
        __stcs(reinterpret_cast<uint2*>(p), make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi)));
    }
    static __device__ __forceinline__ float load1(const __nv_bfloat16* p) { return __bfloat162float(*p); }
    static __device__ __forceinline__ void store1(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
    static __device__ __forceinline__ float round(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }
};

// Tag for the single-buffer ("streaming") form of the acceleration state.  A_k and G_{k-1} enter step k+1 only
// through Z_k = beta_a A_k - (1 - beta_a) G_k:  A_{k+1} = beta_a A_k + (1 - beta_a)(G_{k+1} - G_k) = Z_k + (1 - beta_a) G_{k+1}.
// So one fp32 buffer Z replaces the two of Algorithm 1 (Z_0 = 0), and the pass moves 22 bytes per element, not 30.
// The buffer travels through the kernel in the `A` slot; the `G_prev` slot is unused.
struct Combined {};
template <>
struct StateIO<Combined> : StateIO<float> {
    static constexpr bool has_gp = false;
};

// Tag for the plain Muon step (Eq. muon_momentum): there is no acceleration state to read or write.
struct NoAux {};
template <>
struct StateIO<NoAux> {
    using elem = float;
    static constexpr bool has_gp = false;
    static __device__ __forceinline__ float4 load4(const float*) { return make_float4(0.f, 0.f, 0.f, 0.f); }
    static __device__ __forceinline__ void store4(float*, float4) {}
    static __device__ __forceinline__ float load1(const float*) { return 0.f; }
    static __device__ __forceinline__ void store1(float*, float) {}
    static __device__ __forceinline__ float round(float v) { return v; }
};
// The G_{k-1} slot only exists in the two-buffer formats.
template <typename ST>
__device__ __forceinline__ float4 gp_load4(const typename StateIO<ST>::elem* p) {
    if constexpr (StateIO<ST>::has_gp) return StateIO<ST>::load4(p); else return make_float4(0.f, 0.f, 0.f, 0.f);
}
template <typename ST>
__device__ __forceinline__ void gp_store4(typename StateIO<ST>::elem* p, float4 v) {
    if constexpr (StateIO<ST>::has_gp) StateIO<ST>::store4(p, v);
}
template <typename ST>
__device__ __forceinline__ float gp_load1(const typename StateIO<ST>::elem* p) {
    if constexpr (StateIO<ST>::has_gp) return StateIO<ST>::load1(p); else return 0.f;
}
template <typename ST>
__device__ __forceinline__ void gp_store1(typename StateIO<ST>::elem* p, float v) {
    if constexpr (StateIO<ST>::has_gp) StateIO<ST>::store1(p, v);
}

template <typename ST>
__device__ __forceinline__ void mona_elem(float g, float& gp, float& a, float& m, const PrologueScalars& k) {

    float d = g - gp;                                              // D_k = G_k - G_{k-1}
    a = StateIO<ST>::round(mul_add2(k.beta, a, fmaf(k.one_minus_beta.hi, d, k.one_minus_beta.lo * d)));  // A_k as stored
    float gt = mul_add2(k.alpha, a, g);                             // G~_k = G_k + alpha A_k
    m = mul_add2(k.mu, m, gt);                                      // M_k = mu M_{k-1} + G~_k
    gp = StateIO<ST>::round(g);                                     // G_{k-1} <- G_k
}
template <>
__device__ __forceinline__ void mona_elem<Combined>(float g, float&, float& z, float& m, const PrologueScalars& k) {
    const float w = fmaf(k.one_minus_beta.hi, g, k.one_minus_beta.lo * g);   // (1 - beta_a) G_k
    const float a = z + w;                                          // A_k = Z_{k-1} + (1 - beta_a) G_k
    float gt = mul_add2(k.alpha, a, g);                             // G~_k = G_k + alpha A_k
    m = mul_add2(k.mu, m, gt);                                      // M_k = mu M_{k-1} + G~_k
    // Z_k = beta_a A_k - (1 - beta_a) G_k = beta_a Z_{k-1} - (1 - beta_a)^2 G_k; the second form does not cancel
    z = mul_add2(k.beta, z, -fmaf(k.one_minus_beta.hi, w, k.one_minus_beta.lo * w));
}
template <>
__device__ __forceinline__ void mona_elem<NoAux>(float g, float&, float&, float& m, const PrologueScalars& k) {
    m = mul_add2(k.mu, m, g);                                       // Eq. muon_momentum: M_k = mu M_{k-1} + G_k
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ float block_sum(float v, float* smem /* >= 8 floats */) {
    #pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) smem[warp] = v;
    __syncthreads();
    float t = 0.f;
    if (warp == 0) {
        t = (lane < (EW_THREADS >> 5)) ? smem[lane] : 0.f;
        #pragma unroll
        for (int o = 4; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    }
    return t;   // valid in warp 0 (all lanes)
}

// grid = (slabs, C).  Block (p, c) owns elements [p*slab_len, min(e, (p+1)*slab_len)) of matrix c.
// The last block of a matrix to finish adds the slab partials in index order, so ||M||_F does not
// depend on scheduling; it then resets the arrival counter for the next call.
template <typename GT, typename ST, int VEC>
__global__ void __launch_bounds__(EW_THREADS)
prologue_kernel(ChunkPtrs ptrs, float* __restrict__ Mst, void* __restrict__ Ast, void* __restrict__ Gpst,
                __nv_bfloat16* __restrict__ xhat, float* __restrict__ partials, unsigned int* __restrict__ counters,
                float* __restrict__ inv_norm, DeviceStatus* __restrict__ status, long long e, long long slab_len,
                int slabs, PrologueScalars k) {
    __shared__ float red[8];
    __shared__ int is_last;
    const int c = blockIdx.y, p = blockIdx.x;
    const long long lo = (long long)p * slab_len;
    const long long hi = (lo + slab_len < e) ? lo + slab_len : e;
    if (!MONA_IN_BOUNDS(c < MAXC && p < slabs && p < MAX_SLABS && lo < e && (VEC == 1 || (lo % 4 == 0 && e % 4 == 0)), status, 201)) return;
    const GT* __restrict__ g = reinterpret_cast<const GT*>(ptrs.g[c]);
    float* __restrict__ M = Mst + (long long)c * e;
    using AuxT = typename StateIO<ST>::elem;
    AuxT* __restrict__ A = reinterpret_cast<AuxT*>(Ast) + (long long)c * e;      // never dereferenced by formats without it
    AuxT* __restrict__ Gp = reinterpret_cast<AuxT*>(Gpst) + (long long)c * e;
    __nv_bfloat16* __restrict__ X = xhat ? xhat + (long long)c * e : nullptr;

    float acc = 0.f;
    if (VEC == 4) {
        constexpr long long STEP = (long long)EW_THREADS * 4;
        long long i = lo + (long long)threadIdx.x * 4;
        // two independent vectors per trip keep ~128 B per thread in flight
        for (; i + STEP < hi; i += 2 * STEP) {
            float4 g0 = GradLoad<GT>::load4(g + i), g1 = GradLoad<GT>::load4(g + i + STEP);
            float4 p0 = gp_load4<ST>(Gp + i), p1 = gp_load4<ST>(Gp + i + STEP);
            float4 a0 = StateIO<ST>::load4(A + i), a1 = StateIO<ST>::load4(A + i + STEP);
            float4 m0 = __ldcs(reinterpret_cast<const float4*>(M + i)), m1 = __ldcs(reinterpret_cast<const float4*>(M + i + STEP));
            mona_elem<ST>(g0.x, p0.x, a0.x, m0.x, k); mona_elem<ST>(g0.y, p0.y, a0.y, m0.y, k);
            mona_elem<ST>(g0.z, p0.z, a0.z, m0.z, k); mona_elem<ST>(g0.w, p0.w, a0.w, m0.w, k);
            mona_elem<ST>(g1.x, p1.x, a1.x, m1.x, k); mona_elem<ST>(g1.y, p1.y, a1.y, m1.y, k);
            mona_elem<ST>(g1.z, p1.z, a1.z, m1.z, k); mona_elem<ST>(g1.w, p1.w, a1.w, m1.w, k);
            gp_store4<ST>(Gp + i, p0); gp_store4<ST>(Gp + i + STEP, p1);
            StateIO<ST>::store4(A + i, a0);  StateIO<ST>::store4(A + i + STEP, a1);
            __stcs(reinterpret_cast<float4*>(M + i), m0);  __stcs(reinterpret_cast<float4*>(M + i + STEP), m1);
            if (X) {
                *reinterpret_cast<uint2*>(X + i) = make_uint2(pack_bf16x2(m0.x, m0.y), pack_bf16x2(m0.z, m0.w));
                *reinterpret_cast<uint2*>(X + i + STEP) = make_uint2(pack_bf16x2(m1.x, m1.y), pack_bf16x2(m1.z, m1.w));
            }
            acc = fmaf(m0.x, m0.x, acc); acc = fmaf(m0.y, m0.y, acc); acc = fmaf(m0.z, m0.z, acc); acc = fmaf(m0.w, m0.w, acc);
            acc = fmaf(m1.x, m1.x, acc); acc = fmaf(m1.y, m1.y, acc); acc = fmaf(m1.z, m1.z, acc); acc = fmaf(m1.w, m1.w, acc);
        }
        for (; i < hi; i += STEP) {
            float4 g0 = GradLoad<GT>::load4(g + i);
            float4 p0 = gp_load4<ST>(Gp + i);
            float4 a0 = StateIO<ST>::load4(A + i);
            float4 m0 = __ldcs(reinterpret_cast<const float4*>(M + i));
            mona_elem<ST>(g0.x, p0.x, a0.x, m0.x, k); mona_elem<ST>(g0.y, p0.y, a0.y, m0.y, k);
            mona_elem<ST>(g0.z, p0.z, a0.z, m0.z, k); mona_elem<ST>(g0.w, p0.w, a0.w, m0.w, k);
            gp_store4<ST>(Gp + i, p0);
            StateIO<ST>::store4(A + i, a0);
            __stcs(reinterpret_cast<float4*>(M + i), m0);
            if (X) *reinterpret_cast<uint2*>(X + i) = make_uint2(pack_bf16x2(m0.x, m0.y), pack_bf16x2(m0.z, m0.w));
            acc = fmaf(m0.x, m0.x, acc); acc = fmaf(m0.y, m0.y, acc); acc = fmaf(m0.z, m0.z, acc); acc = fmaf(m0.w, m0.w, acc);
        }
    } else {
        for (long long i = lo + threadIdx.x; i < hi; i += EW_THREADS) {
            float gv = GradLoad<GT>::load1(g + i), pv = gp_load1<ST>(Gp + i), av = StateIO<ST>::load1(A + i), mv = M[i];
            mona_elem<ST>(gv, pv, av, mv, k);
            gp_store1<ST>(Gp + i, pv); StateIO<ST>::store1(A + i, av); M[i] = mv;
            if (X) X[i] = __float2bfloat16_rn(mv);
            acc = fmaf(mv, mv, acc);
        }
    }

    float total = block_sum(acc, red);
    if (threadIdx.x == 0) {
        __stcg(partials + (long long)c * MAX_SLABS + p, total);
        __threadfence();
        unsigned int prev = atomicAdd(counters + c, 1u);
        is_last = (prev == (unsigned int)(slabs - 1));
    }
    __syncthreads();
    if (is_last && threadIdx.x < 32) {
        __threadfence();
        double s = 0.0;
        for (int j = threadIdx.x; j < slabs; j += 32) s += (double)__ldcg(partials + (long long)c * MAX_SLABS + j);
        #pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (threadIdx.x == 0) {
            float nrm = (float)sqrt(s);
            inv_norm[c] = 1.0f / (nrm + k.eps);        // X_0 = M / (||M||_F + eps)
            if (!isfinite(nrm)) {
                atomicOr(&status->flags, STATUS_NONFINITE);
                atomicMin(&status->first_bad, ptrs.gid[c]);
            }
            counters[c] = 0u;
        }
    }
}

// W <- W - eta (gamma O + lambda W), evaluated as (W - (eta lambda) W) - (eta gamma) O.
template <typename OT, int VEC>
__global__ void __launch_bounds__(EW_THREADS)
update_kernel(ChunkPtrs ptrs, const OT* __restrict__ O, long long e, long long slab_len, float eta_lambda,
              float eta_gamma) {
    const int c = blockIdx.y, p = blockIdx.x;
    const long long lo = (long long)p * slab_len;
    const long long hi = (lo + slab_len < e) ? lo + slab_len : e;
    float* __restrict__ W = ptrs.w[c];
    float* __restrict__ Oout = ptrs.o[c];
    const OT* __restrict__ Oc = O + (long long)c * e;
    if (VEC == 4) {
        // Four independent vectors per thread and trip, all loads first: when the block runs squeezed beside a resident
        // GEMM CTA (one 128-thread block per SM), the bytes it keeps in flight are all the bandwidth it gets.
        constexpr int UNROLL = 4;
        constexpr long long STEP = (long long)EW_THREADS * 4;
        long long i = lo + (long long)threadIdx.x * 4;
        for (; i + (UNROLL - 1) * STEP < hi; i += UNROLL * STEP) {
            float4 w[UNROLL], o[UNROLL];
            #pragma unroll
            for (int u = 0; u < UNROLL; ++u) w[u] = __ldcs(reinterpret_cast<const float4*>(W + i + u * STEP));
            #pragma unroll
            for (int u = 0; u < UNROLL; ++u) o[u] = GradLoad<OT>::load4(Oc + i + u * STEP);
            #pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                w[u].x = fmaf(-eta_gamma, o[u].x, fmaf(-eta_lambda, w[u].x, w[u].x));
                w[u].y = fmaf(-eta_gamma, o[u].y, fmaf(-eta_lambda, w[u].y, w[u].y));
                w[u].z = fmaf(-eta_gamma, o[u].z, fmaf(-eta_lambda, w[u].z, w[u].z));
                w[u].w = fmaf(-eta_gamma, o[u].w, fmaf(-eta_lambda, w[u].w, w[u].w));
                __stcs(reinterpret_cast<float4*>(W + i + u * STEP), w[u]);
                if (Oout) *reinterpret_cast<float4*>(Oout + i + u * STEP) = o[u];
            }
        }
        for (; i < hi; i += STEP) {
            float4 w = __ldcs(reinterpret_cast<const float4*>(W + i));
            float4 o = GradLoad<OT>::load4(Oc + i);
            w.x = fmaf(-eta_gamma, o.x, fmaf(-eta_lambda, w.x, w.x));
            w.y = fmaf(-eta_gamma, o.y, fmaf(-eta_lambda, w.y, w.y));
            w.z = fmaf(-eta_gamma, o.z, fmaf(-eta_lambda, w.z, w.z));
            w.w = fmaf(-eta_gamma, o.w, fmaf(-eta_lambda, w.w, w.w));
            __stcs(reinterpret_cast<float4*>(W + i), w);
            if (Oout) *reinterpret_cast<float4*>(Oout + i) = o;
        }
    } else {
        for (long long i = lo + threadIdx.x; i < hi; i += EW_THREADS) {
            float w = W[i], o = GradLoad<OT>::load1(Oc + i);
            W[i] = fmaf(-eta_gamma, o, fmaf(-eta_lambda, w, w));
            if (Oout) Oout[i] = o;
        }
    }
}

// X_0 = M * inv_norm (fp32 validation path only).
__global__ void __launch_bounds__(EW_THREADS)
scale_kernel(const float* __restrict__ M, float* __restrict__ X, const float* __restrict__ inv_norm, long long e,
             long long slab_len) {
    const int c = blockIdx.y;
    const long long lo = (long long)blockIdx.x * slab_len;
    const long long hi = (lo + slab_len < e) ? lo + slab_len : e;
    const float s = inv_norm[c];
    for (long long i = lo + threadIdx.x; i < hi; i += EW_THREADS) X[(long long)c * e + i] = M[(long long)c * e + i] * s;
}

}  // namespace

namespace {
template <typename GT, typename ST>
void launch_prologue_t(dim3 grid, dim3 block, cudaStream_t stream, bool vec4, const ChunkPtrs& ptrs, float* M, void* A, void* Gp,
                       __nv_bfloat16* xhat, float* partials, unsigned int* counters, float* inv_norm, DeviceStatus* status,
                       long long e, long long slab_len, int slabs, const PrologueScalars& k) {
    if (vec4) prologue_kernel<GT, ST, 4><<<grid, block, 0, stream>>>(ptrs, M, A, Gp, xhat, partials, counters, inv_norm, status, e, slab_len, slabs, k);
    else      prologue_kernel<GT, ST, 1><<<grid, block, 0, stream>>>(ptrs, M, A, Gp, xhat, partials, counters, inv_norm, status, e, slab_len, slabs, k);
}
}  // namespace

cudaError_t launch_prologue(const ChunkPtrs& ptrs, int C, bool grad_bf16, int state_kind, bool vec4, float* M, void* A, void* Gp,
                            __nv_bfloat16* xhat, float* partials, unsigned int* counters, float* inv_norm,
                            DeviceStatus* status, long long e, long long slab_len, int slabs,
                            const PrologueScalars& k, cudaStream_t stream) {
    dim3 grid(slabs, C), block(EW_THREADS);
#define MONA_PROLOGUE_CASE(GT, ST) launch_prologue_t<GT, ST>(grid, block, stream, vec4, ptrs, M, A, Gp, xhat, partials, counters, inv_norm, status, e, slab_len, slabs, k)
    if (grad_bf16) {
        if (state_kind == PROLOGUE_NO_AUX) MONA_PROLOGUE_CASE(__nv_bfloat16, NoAux);
        else if (state_kind == PROLOGUE_AUX_COMBINED) MONA_PROLOGUE_CASE(__nv_bfloat16, Combined);
        else if (state_kind == PROLOGUE_AUX_BF16) MONA_PROLOGUE_CASE(__nv_bfloat16, __nv_bfloat16);
        else MONA_PROLOGUE_CASE(__nv_bfloat16, float);
    } else {
        if (state_kind == PROLOGUE_NO_AUX) MONA_PROLOGUE_CASE(float, NoAux);
        else if (state_kind == PROLOGUE_AUX_COMBINED) MONA_PROLOGUE_CASE(float, Combined);
        else if (state_kind == PROLOGUE_AUX_BF16) MONA_PROLOGUE_CASE(float, __nv_bfloat16);
        else MONA_PROLOGUE_CASE(float, float);
    }
#undef MONA_PROLOGUE_CASE
    return cudaGetLastError();
}

cudaError_t launch_update(const ChunkPtrs& ptrs, int C, bool o_is_bf16, bool vec4, const void* O, long long e,
                          long long slab_len, int slabs, float eta_lambda, float eta_gamma, cudaStream_t stream) {
    dim3 grid(slabs, C), block(EW_THREADS);
    if (o_is_bf16) {
        if (vec4) update_kernel<__nv_bfloat16, 4><<<grid, block, 0, stream>>>(ptrs, (const __nv_bfloat16*)O, e, slab_len, eta_lambda, eta_gamma);
        else      update_kernel<__nv_bfloat16, 1><<<grid, block, 0, stream>>>(ptrs, (const __nv_bfloat16*)O, e, slab_len, eta_lambda, eta_gamma);
    } else {
        if (vec4) update_kernel<float, 4><<<grid, block, 0, stream>>>(ptrs, (const float*)O, e, slab_len, eta_lambda, eta_gamma);
        else      update_kernel<float, 1><<<grid, block, 0, stream>>>(ptrs, (const float*)O, e, slab_len, eta_lambda, eta_gamma);
    }
    return cudaGetLastError();
}

cudaError_t launch_scale(const float* M, float* X, const float* inv_norm, int C, long long e, long long slab_len,
                         int slabs, cudaStream_t stream) {
    dim3 grid(slabs, C), block(EW_THREADS);
    scale_kernel<<<grid, block, 0, stream>>>(M, X, inv_norm, e, slab_len);
    return cudaGetLastError();
}

}  // namespace mona

// ---------------------------------------------------------------------------------------------------
// Allocation-free single-matrix prologue (mona_prologue_noalloc, declared in include/mona.h).
//
// The fused prologue needs a little global scratch: one partial sum of squares per slab and a counter
// that tells the last slab to finish that it must add them up.  The handle-based path keeps that
// scratch in the caller's workspace.  Some callers have no workspace to give and cannot create one:
// a process whose framework allocator has already claimed the whole device, or a hook that must not
// trigger the device-wide synchronisation that cudaMalloc/cudaFree imply.  For them the scratch below
// lives in the library image itself; every GPU that loads the library carries these 2 KiB until the
// process exits.
#include <mutex>

#include "../../include/mona.h"

namespace mona {
namespace {

constexpr long long NOALLOC_MAX_ELEMS = 1ll << 24;      // one 4096 x 4096 matrix
constexpr int NOALLOC_MAX_DEVICES = 64;

struct NoAllocScratch {
    float partials[MAX_SLABS];     // slab sums of squares (fully rewritten by every call)
    unsigned int counter;          // slab arrival counter; must be 0 when a call starts
    unsigned int pad[3];
    DeviceStatus status;           // sink of the kernel's non-finite flag; the caller reads inv_norm_out instead
};
static_assert(sizeof(NoAllocScratch) <= 2048, "scratch layout");

// In host code this name is only a handle for cudaGetSymbolAddress, never an address to hand to a kernel.
static __device__ __align__(256) unsigned char g_noalloc_scratch[2048];

std::mutex g_noalloc_mutex;
NoAllocScratch* g_noalloc_dev_ptr[NOALLOC_MAX_DEVICES] = {nullptr};
int g_noalloc_dev_major[NOALLOC_MAX_DEVICES] = {0};

void set_msg(char* buf, size_t len, const char* msg) {
    if (buf && len) {
        size_t i = 0;
        for (; msg[i] && i + 1 < len; ++i) buf[i] = msg[i];
        buf[i] = 0;
    }
}

F2 split_double(double v) {
    F2 r;
    r.hi = (float)v;
    r.lo = (float)(v - (double)r.hi);
    return r;
}

}  // namespace
}  // namespace mona

extern "C" mona_status mona_prologue_noalloc(const void* grad, int32_t grad_dtype, float* M, float* A, float* G_prev,
                                             void* xhat_bf16, float* inv_norm_out, int64_t rows, int64_t cols,
                                             const mona_hparams* hp, void* stream_v, char* err, size_t err_len) {
    using namespace mona;
    if (!grad || !M || !A || !G_prev || !inv_norm_out || !hp) { set_msg(err, err_len, "null pointer argument"); return MONA_ERR_INVALID_ARG; }
    if (rows <= 0 || cols <= 0) { set_msg(err, err_len, "rows and cols must be positive"); return MONA_ERR_INVALID_ARG; }
    if (grad_dtype != MONA_F32 && grad_dtype != MONA_BF16) { set_msg(err, err_len, "unknown grad_dtype"); return MONA_ERR_INVALID_ARG; }
    if (hp->algorithm != 0) { set_msg(err, err_len, "this entry point runs the MONA prologue only (hp->algorithm must be 0)"); return MONA_ERR_INVALID_ARG; }
    if (rows > NOALLOC_MAX_ELEMS || cols > NOALLOC_MAX_ELEMS || rows * cols > NOALLOC_MAX_ELEMS) {
        set_msg(err, err_len, "matrix larger than the built-in scratch supports: rows*cols must be <= 16777216 (4096 x 4096)");
        return MONA_ERR_UNSUPPORTED_SHAPE;
    }
    if (((uintptr_t)grad | (uintptr_t)M | (uintptr_t)A | (uintptr_t)G_prev | (uintptr_t)xhat_bf16) & 15) {
        set_msg(err, err_len, "matrix pointers must be 16-byte aligned");
        return MONA_ERR_ALIGNMENT;
    }
    int dev = -1;
    cudaError_t ce = cudaGetDevice(&dev);
    if (ce != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES) { set_msg(err, err_len, "no current CUDA device"); return MONA_ERR_CUDA; }
    NoAllocScratch* scratch = nullptr;
    {
        // once per device, with that device current: resolve the device address of the static array
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (!g_noalloc_dev_ptr[dev]) {
            void* p = nullptr;
            ce = cudaGetSymbolAddress(&p, g_noalloc_scratch);
            if (ce != cudaSuccess || !p) { set_msg(err, err_len, cudaGetErrorString(ce)); return MONA_ERR_CUDA; }
            int major = 0;
            ce = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
            if (ce != cudaSuccess) { set_msg(err, err_len, cudaGetErrorString(ce)); return MONA_ERR_CUDA; }
            g_noalloc_dev_major[dev] = major;
            g_noalloc_dev_ptr[dev] = reinterpret_cast<NoAllocScratch*>(p);
        }
        if (g_noalloc_dev_major[dev] != 10) { set_msg(err, err_len, "the current device is not compute capability 10.x"); return MONA_ERR_ARCH; }
        scratch = g_noalloc_dev_ptr[dev];
    }
    cudaStream_t stream = (cudaStream_t)stream_v;
    const long long e = rows * cols;
    long long slab = 0;
    int slabs = 0;
    slab_plan(e, &slab, &slabs);
    // the array keeps whatever the previous call left: the counter has to start from zero
    ce = cudaMemsetAsync(&scratch->counter, 0, sizeof(unsigned int), stream);
    if (ce != cudaSuccess) { set_msg(err, err_len, cudaGetErrorString(ce)); return MONA_ERR_CUDA; }
    ChunkPtrs ptrs;
    ptrs.g[0] = grad; ptrs.w[0] = nullptr; ptrs.o[0] = nullptr; ptrs.gid[0] = 0;
    PrologueScalars k;
    k.beta = split_double(hp->accel_beta);
    k.one_minus_beta = split_double(1.0 - hp->accel_beta);
    k.alpha = split_double(hp->accel_alpha);
    k.mu = split_double(hp->momentum);
    k.eps = (float)hp->norm_eps;
    ce = launch_prologue(ptrs, 1, grad_dtype == MONA_BF16, PROLOGUE_AUX_F32, e % 4 == 0, M, A, G_prev, (__nv_bfloat16*)xhat_bf16, scratch->partials,
                         &scratch->counter, inv_norm_out, &scratch->status, e, slab, slabs, k, stream);
    if (ce != cudaSuccess) { set_msg(err, err_len, cudaGetErrorString(ce)); return MONA_ERR_CUDA; }
    set_msg(err, err_len, "");
    return MONA_OK;
}
