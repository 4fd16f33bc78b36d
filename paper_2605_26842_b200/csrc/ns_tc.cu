// Tensor-core GEMMs of the Newton-Schulz iteration (Eq. newton_schulz) for sm_100a.
//
// One persistent CTA per SM walks a static list of output tiles (128 x up-to-256) of all matrices of
// a chunk.  Warp 0 stages bf16 operand tiles with TMA into a 4-deep shared-memory ring, warp 1 issues
// tcgen05.mma (fp32 accumulators in tensor memory, two accumulator buffers so the epilogue of one tile
// overlaps the main loop of the next), warps 2-9 read the accumulator back with tcgen05.ld, apply the
// polynomial term (b A + c A^2 + a I) and the deferred 1/||M||_F scale, and store bf16.
//
// Every wait is bounded: a wait that runs out latches STATUS_TIMEOUT, raises a CTA-wide abort flag, and
// all roles fall through to the common exit where tensor memory is released.
#include "ns_tc.cuh"

namespace mona {

namespace {

constexpr int TC_EPI_WARPS = 8;                                   // two warps per tensor-memory lane quadrant
constexpr int TC_THREADS = 64 + 32 * TC_EPI_WARPS;
constexpr uint32_t A_STAGE_BYTES = TC_BM * TC_BK * 2;            // 16 KiB
constexpr uint32_t B_STAGE_BYTES = TC_BN * TC_BK * 2;            // 32 KiB
constexpr uint32_t STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;  // 48 KiB
constexpr uint32_t BOX_BYTES = TC_BOX * TC_BOX * 2;              // 8 KiB
constexpr uint32_t TMEM_COLS = 512;                              // 2 accumulators x 256 fp32 columns
constexpr uint32_t SMEM_CTRL_BYTES = 256;
constexpr uint32_t SMEM_TOTAL = TC_STAGES * STAGE_BYTES + SMEM_CTRL_BYTES + 1024;  // +1024: manual alignment
constexpr long long WAIT_BUDGET_CYCLES = 4000000000ll;           // ~2 s

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---- mbarrier -------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.shared::cta.b64 st, [%0];\n\t}" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n\t}" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the CTA is aborting (this wait or another one ran out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, DeviceStatus* status,
                                          unsigned site) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    unsigned spins = 0;
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > WAIT_BUDGET_CYCLES) {
                *abort_flag = 1;
                atomicOr(&status->flags, STATUS_TIMEOUT);
                status->timeout_site = site;
                return false;
            }
        }
    }
}

// ---- TMA ------------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
        : "memory");
}

// ---- tcgen05 --------------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate; accumulate == 0 overwrites D.
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread t of the warp receives row (lane base + t).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor for a 128-byte-swizzled bf16 tile whose rows are 128 bytes long and
// stacked densely (what a 64-wide TMA box with SWIZZLE_128B produces).
//   K-major : row = m/n index, 128 B = 64 k.  Groups of 8 rows are 1024 B apart (stride byte offset);
//             the leading byte offset is not used by swizzled K-major layouts (encoded 1).
//   MN-major: row = k index, 128 B = 64 m/n.  Groups of 8 k-rows are 1024 B apart (stride byte offset);
//             the next 64 m/n lives in the next 8 KiB box (leading byte offset).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, bool mn_major) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3fffu);                                  // start address, bits [0,14)
    d |= (uint64_t)(mn_major ? (BOX_BYTES >> 4) : 1u) << 16;                 // leading byte offset, bits [16,30)
    d |= (uint64_t)(1024u >> 4) << 32;                                       // stride byte offset, bits [32,46)
    d |= (uint64_t)1 << 46;                                                  // descriptor version for sm_100
    d |= (uint64_t)2 << 61;                                                  // layout: 128-byte swizzle
    return d;
}
// Instruction descriptor, kind::f16: D fp32, A and B bf16, M = 128, N = n.
__device__ __forceinline__ uint32_t instr_desc(int n, int a_mn, int b_mn) {
    return (1u << 4)                      // D format fp32
           | (1u << 7) | (1u << 10)       // A, B format bf16
           | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16)
           | ((uint32_t)(n >> 3) << 17)
           | ((uint32_t)(TC_BM >> 4) << 24);
}

struct TileCoord {
    int c, tm, tn, nw;   // matrix, tile row, tile column, columns of this tile (multiple of 64, <= 256)
};

__device__ __forceinline__ TileCoord decode_tile(const TcGemm& g, int t) {
    TileCoord tc;
    tc.c = t / g.tiles_per_mat;
    int r = t - tc.c * g.tiles_per_mat;
    int n_left;
    if (g.symmetric) {
        // rows come in pairs (2q, 2q+1), each row of the pair owning q+1 tiles of width 256
        int q = 0;
        while ((q + 1) * (q + 2) <= r) ++q;
        int rr = r - q * (q + 1);
        if (rr >= q + 1) { tc.tm = 2 * q + 1; tc.tn = rr - (q + 1); } else { tc.tm = 2 * q; tc.tn = rr; }
        n_left = min(g.N, TC_BM * (tc.tm + 1)) - tc.tn * TC_BN;   // nothing right of the diagonal 128-block
    } else {
        tc.tm = r / g.tiles_n;
        tc.tn = r - tc.tm * g.tiles_n;
        n_left = g.N - tc.tn * TC_BN;
    }
    int nw = (n_left + TC_BOX - 1) / TC_BOX * TC_BOX;
    tc.nw = nw < TC_BN ? nw : TC_BN;
    return tc;
}

__device__ __forceinline__ uint4 pack8(const float* v) {
    uint4 r;
    __nv_bfloat162 t;
    t = __floats2bfloat162_rn(v[0], v[1]); r.x = *reinterpret_cast<uint32_t*>(&t);
    t = __floats2bfloat162_rn(v[2], v[3]); r.y = *reinterpret_cast<uint32_t*>(&t);
    t = __floats2bfloat162_rn(v[4], v[5]); r.z = *reinterpret_cast<uint32_t*>(&t);
    t = __floats2bfloat162_rn(v[6], v[7]); r.w = *reinterpret_cast<uint32_t*>(&t);
    return r;
}

__global__ void __launch_bounds__(TC_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tma_a, const __grid_constant__ CUtensorMap tma_b, TcGemm g,
               DeviceStatus* __restrict__ status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;       // swizzle atoms need 1024-byte alignment
    const uint32_t ctrl = base + TC_STAGES * STAGE_BYTES;
    const uint32_t bar_full = ctrl;                     // TC_STAGES x 8 B
    const uint32_t bar_empty = ctrl + 8 * TC_STAGES;    // TC_STAGES x 8 B
    const uint32_t bar_acc_full = ctrl + 16 * TC_STAGES;        // 2 x 8 B
    const uint32_t bar_acc_empty = bar_acc_full + 16;           // 2 x 8 B
    const uint32_t tmem_slot = bar_acc_empty + 16;              // 4 B
    uint8_t* ctrl_ptr = smem_raw + (ctrl - smem_u32(smem_raw));
    volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(ctrl_ptr + (tmem_slot - ctrl));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl_ptr + (tmem_slot - ctrl) + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_tiles = g.C * g.tiles_per_mat;
    const int num_kb = (g.K + TC_BK - 1) / TC_BK;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < TC_STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(bar_acc_full + 8 * a, 1); mbar_init(bar_acc_empty + 8 * a, TC_EPI_WARPS); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tma_a) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tma_b) : "memory");
    }
    if (warp == 1) {
        __syncwarp();
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_ptr;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                const TileCoord tc = decode_tile(g, t);
                const int m0 = tc.tm * TC_BM, n0 = tc.tn * TC_BN;
                const int nbox_b = tc.nw / TC_BOX;
                const uint32_t tx_bytes = A_STAGE_BYTES + (uint32_t)nbox_b * BOX_BYTES;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!(ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, status, 1))) break;
                    const uint32_t full = bar_full + 8 * stage;
                    const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_STAGE_BYTES;
                    const int k0 = kb * TC_BK;
                    mbar_arrive_expect_tx(full, tx_bytes);
                    #pragma unroll
                    for (int j = 0; j < TC_BM / TC_BOX; ++j) {
                        if (g.a_mn) tma_load_3d(sa + j * BOX_BYTES, &tma_a, full, m0 + j * TC_BOX, k0, tc.c);
                        else        tma_load_3d(sa + j * BOX_BYTES, &tma_a, full, k0, m0 + j * TC_BOX, tc.c);
                    }
                    for (int j = 0; j < nbox_b; ++j) {
                        if (g.b_mn) tma_load_3d(sb + j * BOX_BYTES, &tma_b, full, n0 + j * TC_BOX, k0, tc.c);
                        else        tma_load_3d(sb + j * BOX_BYTES, &tma_b, full, k0, n0 + j * TC_BOX, tc.c);
                    }
                    if (++stage == TC_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            // one k-step of 16 advances 32 B inside the swizzle row (K-major) or 16 rows = 2048 B (MN-major)
            const uint32_t a_kstep = g.a_mn ? (2048u >> 4) : (32u >> 4);
            const uint32_t b_kstep = g.b_mn ? (2048u >> 4) : (32u >> 4);
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                const TileCoord tc = decode_tile(g, t);
                const uint32_t idesc = instr_desc(tc.nw, g.a_mn, g.b_mn);
                if (!(ok = mbar_wait(bar_acc_empty + 8 * acc, acc_phase ^ 1u, abort_flag, status, 2))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * TC_BN;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!(ok = mbar_wait(bar_full + 8 * stage, phase, abort_flag, status, 3))) break;
                    tc_fence_after();
                    const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_STAGE_BYTES;
                    const uint64_t da = smem_desc(sa, g.a_mn), db = smem_desc(sb, g.b_mn);
                    #pragma unroll
                    for (int k = 0; k < TC_BK / 16; ++k)
                        tc_mma_bf16(d_tmem, da + (uint64_t)(k * a_kstep), db + (uint64_t)(k * b_kstep), idesc,
                                    (kb | k) != 0 ? 1u : 0u);
                    tc_commit(bar_empty + 8 * stage);          // frees the stage when these MMAs have read it
                    if (++stage == TC_STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit(bar_acc_full + 8 * acc);             // accumulator complete
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        // ---------------- epilogue (warps 2..9) ----------------
        // A warp may only read the 32 tensor-memory lanes of its quadrant (warp index mod 4); the two warps
        // of a quadrant take alternate 32-column chunks.  Two chunks are in flight per warp so that the
        // tensor-memory load of one overlaps the arithmetic and stores of the other.
        const int quad = warp & 3;
        const int half = (warp - 2) >> 2;
        const int row_in_tile = quad * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        uint32_t acc = 0, acc_phase = 0;
        for (int t = blockIdx.x; t < total_tiles; t += gridDim.x) {
            const TileCoord tc = decode_tile(g, t);
            const int gr = tc.tm * TC_BM + row_in_tile;
            const int n0 = tc.tn * TC_BN;
            const bool row_ok = gr < g.M;
            const long long mat_off = (long long)tc.c * g.mat_stride;
            const long long row_off = mat_off + (long long)gr * g.ld;
            float post = 1.0f;
            if (g.post_mode) { float sc = g.inv_norm[tc.c]; post = g.post_mode == 2 ? sc * sc : sc; }
            const float c1 = g.c1, c2 = g.c2 * post;
            const int nchunks = tc.nw >> 5;
            // operand of the axpy term for the first pair of chunks, requested before the accumulator is ready
            uint4 cin_raw[2][4];
            auto load_cin = [&](int ch, uint4* dst) {
                const int gc0 = n0 + ch * 32;
                #pragma unroll
                for (int q = 0; q < 4; ++q) {
                    if (row_ok && ch < nchunks && gc0 + 8 * q < g.N) dst[q] = *reinterpret_cast<const uint4*>(g.cin + row_off + gc0 + 8 * q);
                    else dst[q] = make_uint4(0u, 0u, 0u, 0u);
                }
            };
            if (g.cin) { load_cin(half, cin_raw[0]); load_cin(half + 2, cin_raw[1]); }
            bool ok = mbar_wait(bar_acc_full + 8 * acc, acc_phase, abort_flag, status, 4);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_base = tmem_base + lane_base + acc * TC_BN;
            for (int ch0 = half; ch0 < nchunks; ch0 += 4) {
                const int ch1 = ch0 + 2;
                float v[2][32];
                tmem_ld32(t_base + ch0 * 32, v[0]);
                if (ch1 < nchunks) tmem_ld32(t_base + ch1 * 32, v[1]);
                tmem_ld_wait();
                #pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int ch = u == 0 ? ch0 : ch1;
                    const int gc0 = n0 + ch * 32;
                    if (ch < nchunks && row_ok && gc0 < g.N) {
                        float* vv = v[u];
                        if (g.cin) {
                            const uint32_t w[16] = {cin_raw[u][0].x, cin_raw[u][0].y, cin_raw[u][0].z, cin_raw[u][0].w,
                                                    cin_raw[u][1].x, cin_raw[u][1].y, cin_raw[u][1].z, cin_raw[u][1].w,
                                                    cin_raw[u][2].x, cin_raw[u][2].y, cin_raw[u][2].z, cin_raw[u][2].w,
                                                    cin_raw[u][3].x, cin_raw[u][3].y, cin_raw[u][3].z, cin_raw[u][3].w};
                            #pragma unroll
                            for (int h = 0; h < 16; ++h) {
                                vv[2 * h] = fmaf(c1 * post, __uint_as_float(w[h] << 16), c2 * vv[2 * h]);
                                vv[2 * h + 1] = fmaf(c1 * post, __uint_as_float(w[h] & 0xffff0000u), c2 * vv[2 * h + 1]);
                            }
                        } else {
                            #pragma unroll
                            for (int j = 0; j < 32; ++j) vv[j] *= c2;
                        }
                        if (g.diag_add != 0.f && gr >= gc0 && gr < gc0 + 32) {
                            #pragma unroll
                            for (int j = 0; j < 32; ++j) vv[j] += (gc0 + j == gr) ? g.diag_add : 0.f;
                        }
                        #pragma unroll
                        for (int q = 0; q < 4; ++q)
                            if (gc0 + 8 * q < g.N) *reinterpret_cast<uint4*>(g.out + row_off + gc0 + 8 * q) = pack8(vv + 8 * q);
                        if (g.symmetric && (gc0 / TC_BM) < tc.tm) {
                            // strictly-lower 128-block: the transposed block is not computed anywhere, write it here
                            __nv_bfloat16* col = g.out + mat_off + (long long)gc0 * g.ld + gr;
                            #pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (gc0 + j < g.N) col[(long long)j * g.ld] = __float2bfloat16_rn(vv[j]);
                        }
                    }
                }
                if (g.cin && ch0 + 4 < nchunks) { load_cin(ch0 + 4, cin_raw[0]); load_cin(ch0 + 6, cin_raw[1]); }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acc_empty + 8 * acc);
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    }

    if (*abort_flag) __nanosleep(200000);      // let copies that are still in flight land before the CTA goes away
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace

void tc_gemm_plan(TcGemm& g) {
    g.tiles_m = (g.M + TC_BM - 1) / TC_BM;
    g.tiles_n = (g.N + TC_BN - 1) / TC_BN;
    if (g.symmetric) {
        int pairs = g.tiles_m / 2;
        g.tiles_per_mat = pairs * (pairs + 1) + ((g.tiles_m & 1) ? pairs + 1 : 0);
    } else {
        g.tiles_per_mat = g.tiles_m * g.tiles_n;
    }
}

double tc_gemm_executed_flops(const TcGemm& g) {
    const double kpad = (double)((g.K + TC_BK - 1) / TC_BK * TC_BK);
    double cols = 0.0;   // sum over tiles of the issued MMA width
    for (int tm = 0; tm < g.tiles_m; ++tm) {
        int ntiles = g.symmetric ? tm / 2 + 1 : g.tiles_n;
        for (int tn = 0; tn < ntiles; ++tn) {
            int n_left = (g.symmetric ? (g.N < TC_BM * (tm + 1) ? g.N : TC_BM * (tm + 1)) : g.N) - tn * TC_BN;
            int nw = (n_left + TC_BOX - 1) / TC_BOX * TC_BOX;
            cols += nw < TC_BN ? nw : TC_BN;
        }
    }
    return 2.0 * TC_BM * cols * kpad * g.C;
}

cudaError_t tc_gemm_configure() {
    return cudaFuncSetAttribute(tc_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_TOTAL);
}

cudaError_t launch_tc_gemm(const CUtensorMap& tma_a, const CUtensorMap& tma_b, const TcGemm& g, int num_sms,
                           DeviceStatus* status, cudaStream_t stream) {
    const int total = g.C * g.tiles_per_mat;
    if (total <= 0) return cudaSuccess;
    const int grid = total < num_sms ? total : num_sms;
    tc_gemm_kernel<<<grid, TC_THREADS, SMEM_TOTAL, stream>>>(tma_a, tma_b, g, status);
    return cudaGetLastError();
}

}  // namespace mona
