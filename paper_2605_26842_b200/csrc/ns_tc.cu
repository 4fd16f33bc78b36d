// Tensor-core GEMMs of the Newton-Schulz iteration (Eq. newton_schulz) for sm_100a.
//
// The kernel is persistent and runs as clusters of two CTAs on neighbouring SMs.  A CTA pair walks a
// static list of 256 x 256 output tiles of all matrices of a chunk; one tcgen05.mma.cta_group::2
// instruction stream, issued by the even CTA (the "leader"), drives the tensor cores of both SMs.
// Each CTA stages its own 128 rows of the A operand and its own 128 rows of the B operand per k-slice,
// so a pair moves 64 KiB from L2 per 256 x 256 x 64 step (half of what two independent 128 x 256 tiles
// would).  Roles inside a CTA:
//   warp 0     TMA producer: operand boxes into a ring of shared-memory stages; the copies of both CTAs
//              complete on the leader's "full" barrier,
//   warp 1     owner of tensor memory; in the leader its lane 0 issues the MMAs and commits them to
//              the "empty" barriers of both CTAs (multicast commit),
//   warps 2-9  epilogue: tcgen05.ld the CTA's 128 x 256 fp32 accumulator, apply the polynomial term
//              (b A + c A^2 + a I) and the deferred 1/||M||_F scale, pack to bf16 into swizzled
//              shared memory and hand the boxes to TMA stores.
// Tensor memory holds two 256-column accumulators.  In the plain configuration they alternate, so the
// epilogue of one tile overlaps the main loop of the next.  In the WIDE configuration (non-symmetric
// products, here X' = B' X) a pair computes a 256 x 512 macro-tile, i.e. two neighbouring tiles at once,
// one per accumulator, from ONE staged slice of the A operand: 96 KiB instead of 128 KiB cross from L2
// per k-slice and pair.  The main loop is bound by that traffic, not by the tensor pipe, so fewer bytes
// per flop is worth more than accumulator double-buffering.  To keep the unhidden part of that epilogue short,
// its warps first read and pack a whole accumulator into registers and hand it back to the MMA issuer, and only
// then stage and store; the operand ring keeps filling meanwhile.
//
// Every wait on an mbarrier is bounded: when one runs out the CTA latches STATUS_TIMEOUT, raises its
// abort flag, and all roles fall through to the common exit, where tensor memory is released.
#include "ns_tc.cuh"

namespace mona {

namespace {

#ifndef MONA_TC_WIDE_STAGES
#define MONA_TC_WIDE_STAGES 4
#endif
#ifndef MONA_TC_WIDE_EPI_BUFS
#define MONA_TC_WIDE_EPI_BUFS 1
#endif
constexpr int TC_EPI_WARPS = 8;                                   // two warps per tensor-memory lane quadrant
constexpr int TC_EPI_THREADS = 32 * TC_EPI_WARPS;
constexpr int TC_THREADS = 64 + TC_EPI_THREADS;
// 320 threads x 160 registers: no spills, and room is left on the SM for one 256-thread block of another kernel
constexpr int TC_MAX_REGS = 160;
constexpr int CTA_M = TC_BM / 2;                                  // accumulator rows held by one CTA
constexpr int CTA_N = TC_BN / 2;                                  // B-operand rows one CTA stages per 256-column tile
constexpr uint32_t BOX_BYTES = TC_BOX * TC_BOX * 2;               // 8 KiB
constexpr uint32_t A_STAGE_BYTES = CTA_M * TC_BK * 2;             // 16 KiB
constexpr uint32_t B_SUB_BYTES = CTA_N * TC_BK * 2;               // 16 KiB per 256-column tile
constexpr int EPI_COLS = 128;                                     // output columns per epilogue phase
constexpr uint32_t EPI_BUF_BYTES = CTA_M * EPI_COLS * 2;          // 32 KiB = 2 x 2 boxes
constexpr uint32_t TMEM_COLS = 512;                               // 2 accumulators x 256 fp32 columns
constexpr uint32_t SMEM_CTRL_BYTES = 256;
constexpr long long WAIT_BUDGET_CYCLES = 1000000000ll;            // ~0.5 s

// Shared-memory plan of the two configurations (per CTA).
template <bool WIDE>
struct Cfg {
    static constexpr int NSUB = WIDE ? 2 : 1;                                   // 256-column tiles per macro-tile
    static constexpr int STAGES = WIDE ? MONA_TC_WIDE_STAGES : 5;               // operand ring depth
    static constexpr int EPI_BUFS = WIDE ? MONA_TC_WIDE_EPI_BUFS : 2;           // staging buffers of the store epilogue
    static constexpr uint32_t STAGE_BYTES = A_STAGE_BYTES + NSUB * B_SUB_BYTES; // 48 / 32 KiB
    static constexpr uint32_t SMEM_TOTAL = STAGES * STAGE_BYTES + EPI_BUFS * EPI_BUF_BYTES + SMEM_CTRL_BYTES + 1024;
    static_assert(SMEM_TOTAL <= 232448, "shared memory budget");
    static_assert(8 * (2 * STAGES + 4) + 8 <= SMEM_CTRL_BYTES, "control block");
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---- cluster --------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// ---- mbarrier -------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n\t}" ::"r"(bar), "r"(bytes)
                 : "memory");
}
// Arrive on a barrier given by its cluster-wide address (own CTA or the peer).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
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

// ---- named barriers among the epilogue warps ------------------------------------------------------
__device__ __forceinline__ void epi_bar_sync(int id) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(TC_EPI_THREADS) : "memory");
}
// Barrier + AND-reduction of a predicate over the epilogue threads (same answer in every thread).
__device__ __forceinline__ bool epi_bar_all(int id, bool pred) {
    uint32_t in = pred ? 1u : 0u, out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "barrier.cta.red.and.pred p, %2, %3, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out)
        : "r"(in), "r"(id), "r"(TC_EPI_THREADS)
        : "memory");
    return out != 0;
}

// ---- TMA ------------------------------------------------------------------------------------------
// Box load into this CTA's shared memory; completion bytes are counted on `bar`, a cluster-wide
// address that may name the barrier of the peer CTA of the pair (cta_group::2 form).
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
        : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int x, int y, int z) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y), "r"(z)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---- tcgen05 --------------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// Arrives (once the MMAs issued so far have completed) on the barrier at offset `bar` in both CTAs.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask)
                 : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T over the CTA pair, bf16 inputs, fp32 accumulate; accumulate == 0 overwrites D.
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
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
// Instruction descriptor, kind::f16: D fp32, A and B bf16, M = 256 over the pair, N = 256.
__device__ __forceinline__ uint32_t instr_desc(int a_mn, int b_mn) {
    return (1u << 4)                      // D format fp32
           | (1u << 7) | (1u << 10)       // A, B format bf16
           | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16)
           | ((uint32_t)(TC_BN >> 3) << 17)
           | ((uint32_t)(TC_BM >> 4) << 24);
}

struct TileCoord {
    int c, tm, tn;   // matrix, tile row, first tile column
    int nsub;        // 256-column tiles in this (macro-)tile: 1 or 2
};

template <bool WIDE>
__device__ __forceinline__ TileCoord decode_tile(const TcGemm& g, int t) {
    TileCoord tc;
    tc.c = t / g.tiles_per_mat;
    const int r = t - tc.c * g.tiles_per_mat;
    tc.nsub = 1;
    if (WIDE) {
        const int macro_n = (g.tiles_n + 1) >> 1;
        tc.tm = r / macro_n;
        tc.tn = 2 * (r - tc.tm * macro_n);
        tc.nsub = tc.tn + 1 < g.tiles_n ? 2 : 1;
    } else if (g.symmetric) {
        int tm = 0;
        while ((tm + 1) * (tm + 2) / 2 <= r) ++tm;     // lower triangle, row by row
        tc.tm = tm;
        tc.tn = r - tm * (tm + 1) / 2;
    } else {
        tc.tm = r / g.tiles_n;
        tc.tn = r - tc.tm * g.tiles_n;
    }
    return tc;
}

// A symmetric operand is stored as its lower block triangle: the k-slice [k0, k0 + 64) of row block
// `blk` lies above the diagonal block exactly when it starts at or beyond the end of that block.
__device__ __forceinline__ int fetch_transposed(int sym, int blk, int k0) { return sym && k0 >= (blk + 1) * TC_BM; }

__device__ __forceinline__ uint4 pack8(const float* v) {
    uint4 r;
    __nv_bfloat162 t;
    t = __floats2bfloat162_rn(v[0], v[1]); r.x = *reinterpret_cast<uint32_t*>(&t);
    t = __floats2bfloat162_rn(v[2], v[3]); r.y = *reinterpret_cast<uint32_t*>(&t);
    t = __floats2bfloat162_rn(v[4], v[5]); r.z = *reinterpret_cast<uint32_t*>(&t);
    t = __floats2bfloat162_rn(v[6], v[7]); r.w = *reinterpret_cast<uint32_t*>(&t);
    return r;
}

template <bool WIDE>
__global__ void __cluster_dims__(2, 1, 1) __maxnreg__(TC_MAX_REGS)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tma_a, const __grid_constant__ CUtensorMap tma_b,
               const __grid_constant__ CUtensorMap tma_d, TcGemm g, DeviceStatus* __restrict__ status) {
    using C = Cfg<WIDE>;
    constexpr int STAGES = C::STAGES;
    constexpr uint32_t STAGE_BYTES = C::STAGE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;       // swizzle atoms need 1024-byte alignment
    const uint32_t epi_base = base + STAGES * STAGE_BYTES;
    const uint32_t ctrl = epi_base + C::EPI_BUFS * EPI_BUF_BYTES;
    const uint32_t bar_full = ctrl;                             // STAGES x 8 B (used in the leader)
    const uint32_t bar_empty = ctrl + 8 * STAGES;               // STAGES x 8 B
    const uint32_t bar_acc_full = ctrl + 16 * STAGES;           // 2 x 8 B, one per accumulator
    const uint32_t bar_acc_empty = bar_acc_full + 16;           // 2 x 8 B (used in the leader)
    const uint32_t tmem_slot = bar_acc_empty + 16;              // 4 B
    uint8_t* ctrl_ptr = smem_raw + (ctrl - smem_u32(smem_raw));
    volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(ctrl_ptr + (tmem_slot - ctrl));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl_ptr + (tmem_slot - ctrl) + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                    // 0: leader, 1: peer
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int total_tiles = g.C * g.tiles_per_mat;
    const int num_kb = (g.K + TC_BK - 1) / TC_BK;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(bar_acc_full + 8 * a, 1); mbar_init(bar_acc_empty + 8 * a, 2 * TC_EPI_WARPS); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tma_a) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tma_b) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tma_d) : "memory");
    }
    if (warp == 1) {
        __syncwarp();
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();                    // both CTAs' barriers exist before either side signals the other
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_ptr;

    // Accumulator of sub-tile j of the n-th (macro-)tile this pair processes: WIDE uses accumulator j,
    // the plain configuration alternates.  Every role keeps one use-parity bit per accumulator.

    if (warp == 0) {
        // ---------------- TMA producer (both CTAs) ----------------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            const uint32_t full_leader = map_to_cta(bar_full, 0);
            for (int t = pair; t < total_tiles && ok; t += num_pairs) {
                const TileCoord tc = decode_tile<WIDE>(g, t);
                const int m0 = tc.tm * TC_BM + (int)rank * CTA_M;      // this CTA's rows of the A operand
                const int n0 = tc.tn * TC_BN + (int)rank * CTA_N;      // this CTA's rows of the B operand (first sub-tile)
                // diagonal tile of X X^T or A A: both operands are the same rows, staged once
                const bool shared_ab = !WIDE && g.ab_same && tc.tm == tc.tn;
                const uint32_t tx_bytes = 2u * (A_STAGE_BYTES + (shared_ab ? 0u : (uint32_t)tc.nsub * B_SUB_BYTES)) + (uint32_t)g.selftest_extra_tx;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!(ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, status, 1))) break;
                    const uint32_t full = full_leader + 8 * stage;
                    const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_STAGE_BYTES;
                    const int k0 = kb * TC_BK;
                    if (rank == 0) mbar_arrive_expect_tx(bar_full + 8 * stage, tx_bytes);   // both CTAs' copies land here
                    const int a_mn = g.a_sym ? fetch_transposed(1, tc.tm, k0) : g.a_mn;
                    #pragma unroll
                    for (int j = 0; j < CTA_M / TC_BOX; ++j) {
                        if (a_mn) tma_load_3d(sa + j * BOX_BYTES, &tma_a, full, m0 + j * TC_BOX, k0, tc.c);
                        else      tma_load_3d(sa + j * BOX_BYTES, &tma_a, full, k0, m0 + j * TC_BOX, tc.c);
                    }
                    if (!shared_ab) {
                        for (int u = 0; u < tc.nsub; ++u) {
                            const int b_mn = g.b_sym ? fetch_transposed(1, tc.tn + u, k0) : g.b_mn;
                            const int nu = n0 + u * TC_BN;
                            const uint32_t sbu = sb + u * B_SUB_BYTES;
                            #pragma unroll
                            for (int j = 0; j < CTA_N / TC_BOX; ++j) {
                                if (b_mn) tma_load_3d(sbu + j * BOX_BYTES, &tma_b, full, nu + j * TC_BOX, k0, tc.c);
                                else      tma_load_3d(sbu + j * BOX_BYTES, &tma_b, full, k0, nu + j * TC_BOX, tc.c);
                            }
                        }
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            // stay until the tensor cores have released every stage: the commits arrive on this CTA's barriers
            for (int s = 0; s < STAGES && ok; ++s) {
                ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, status, 5);
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA only) ----------------
        if (lane == 0 && rank == 0) {
            uint32_t stage = 0, phase = 0, acc_next = 0, acc_par = 0;   // acc_par: one use-parity bit per accumulator
            bool ok = true;
            for (int t = pair; t < total_tiles && ok; t += num_pairs) {
                const TileCoord tc = decode_tile<WIDE>(g, t);
                const bool shared_ab = !WIDE && g.ab_same && tc.tm == tc.tn;
                const uint32_t acc0 = WIDE ? 0u : acc_next;
                for (int kb = 0; kb < num_kb && ok; ++kb) {
                    if (!(ok = mbar_wait(bar_full + 8 * stage, phase, abort_flag, status, 3))) break;
                    tc_fence_after();
                    const int k0 = kb * TC_BK;
                    const int a_mn = g.a_sym ? fetch_transposed(1, tc.tm, k0) : g.a_mn;
                    // one k-step of 16 advances 32 B inside the swizzle row (K-major) or 16 rows = 2048 B (MN-major)
                    const uint32_t a_kstep = a_mn ? (2048u >> 4) : (32u >> 4);
                    const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_STAGE_BYTES;
                    const uint64_t da = smem_desc(sa, a_mn);
                    for (int u = 0; u < tc.nsub; ++u) {
                        const uint32_t acc = acc0 + u;
                        if (kb == 0) {     // the epilogue must have drained this accumulator's previous tile
                            if (!(ok = mbar_wait(bar_acc_empty + 8 * acc, ((acc_par >> acc) & 1u) ^ 1u, abort_flag, status, 2))) break;
                            tc_fence_after();
                        }
                        const int b_mn = shared_ab ? a_mn : (g.b_sym ? fetch_transposed(1, tc.tn + u, k0) : g.b_mn);
                        const uint32_t b_kstep = b_mn ? (2048u >> 4) : (32u >> 4);
                        const uint64_t db = smem_desc(shared_ab ? sa : sb + u * B_SUB_BYTES, b_mn);
                        const uint32_t idesc = instr_desc(a_mn, b_mn);
                        const uint32_t d_tmem = tmem_base + acc * TC_BN;
                        #pragma unroll
                        for (int k = 0; k < TC_BK / 16; ++k)
                            tc_mma_bf16(d_tmem, da + (uint64_t)(k * a_kstep), db + (uint64_t)(k * b_kstep), idesc,
                                        (kb | k) != 0 ? 1u : 0u);
                    }
                    if (!ok) break;
                    tc_commit_pair(bar_empty + 8 * stage);     // frees the stage in both CTAs when these MMAs have read it
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                for (int u = 0; u < tc.nsub; ++u) {
                    const uint32_t acc = acc0 + u;
                    tc_commit_pair(bar_acc_full + 8 * acc);    // accumulator complete, both CTAs' epilogues may read
                    acc_par ^= 1u << acc;
                }
                if (!WIDE) acc_next ^= 1u;
            }
        }
    } else {
        // ---------------- epilogue (warps 2..9, both CTAs) ----------------
        // A warp may only read the 32 tensor-memory lanes of its quadrant (warp index mod 4).  A 256-column
        // tile is written in phases of 128 columns; in a phase the two warps of a quadrant take 64 columns
        // each, i.e. one 64 x 64 store box column.
        const int quad = warp & 3;
        const int half = (warp - 2) >> 2;
        const int row_in_cta = quad * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const bool issuer = threadIdx.x == 64;                 // first epilogue thread: issues and retires TMA stores
        const uint32_t acc_empty_leader = map_to_cta(bar_acc_empty, 0);
        // position of this thread's row inside the staging buffer: box (row half, column half), 128-byte rows
        const uint32_t box_row = (uint32_t)(row_in_cta & 63);
        const uint32_t stage_off = (uint32_t)(((row_in_cta >> 6) * 2 + half)) * BOX_BYTES + box_row * 128u;
        const uint32_t swz = box_row & 7u;
        uint32_t acc_next = 0, acc_par = 0, epi_it = 0;   // acc_par: one use-parity bit per accumulator
        bool alive = true;
        for (int t = pair; t < total_tiles && alive; t += num_pairs) {
            const TileCoord tc = decode_tile<WIDE>(g, t);
            const int m0 = tc.tm * TC_BM + (int)rank * CTA_M;
            const int gr = m0 + row_in_cta;
            const bool row_ok = gr < g.M;
            const long long row_off = (long long)tc.c * g.mat_stride + (long long)gr * g.ld;
            float post = 1.0f;
            if (g.post_mode) { const float sc = g.inv_norm[tc.c]; post = g.post_mode == 2 ? sc * sc : sc; }
            const float c1 = g.c1 * post, c2 = g.c2 * post;
            const uint32_t acc0 = WIDE ? 0u : acc_next;
            for (int u = 0; u < tc.nsub; ++u) {
                const uint32_t acc = acc0 + u;
                const int n0 = (tc.tn + u) * TC_BN;
                const int nphases = (g.N - n0 > EPI_COLS) ? 2 : 1;
                if constexpr (WIDE) {
                    // Macro-tile configuration (no axpy operand, no diagonal term): both accumulators belong to the tile
                    // in flight, so nothing hides this epilogue.  A thread's share of an accumulator (128 values) fits
                    // in 64 packed registers: read and pack all of it first, hand the accumulator back to the MMA issuer,
                    // and only then stage and store.
                    bool ok = mbar_wait(bar_acc_full + 8 * acc, (acc_par >> acc) & 1u, abort_flag, status, 4);
                    ok = epi_bar_all(3, ok);
                    if (!ok) { alive = false; break; }
                    tc_fence_after();
                    acc_par ^= 1u << acc;
                    const uint32_t t_base = tmem_base + lane_base + acc * TC_BN + half * 64;
                    uint4 pk[2][8];
                    #pragma unroll
                    for (int ph = 0; ph < 2; ++ph) {
                        if (ph < nphases) {
                            float v[64];
                            tmem_ld32(t_base + ph * EPI_COLS, v);
                            tmem_ld32(t_base + ph * EPI_COLS + 32, v + 32);
                            tmem_ld_wait();
                            #pragma unroll
                            for (int j = 0; j < 64; ++j) v[j] *= c2;
                            #pragma unroll
                            for (int q = 0; q < 8; ++q) pk[ph][q] = pack8(v + 8 * q);
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(acc_empty_leader + 8 * acc);
                    #pragma unroll
                    for (int ph = 0; ph < 2; ++ph) {
                        if (ph < nphases) {
                            const uint32_t buf = epi_base + (epi_it % C::EPI_BUFS) * EPI_BUF_BYTES;
                            if (issuer) bulk_wait_read<C::EPI_BUFS - 1>();
                            epi_bar_sync(1);
                            #pragma unroll
                            for (int q = 0; q < 8; ++q) {
                                const uint32_t addr = buf + stage_off + (((uint32_t)q ^ swz) << 4);
                                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(pk[ph][q].x), "r"(pk[ph][q].y),
                                             "r"(pk[ph][q].z), "r"(pk[ph][q].w) : "memory");
                            }
                            fence_proxy_async();
                            epi_bar_sync(2);
                            if (issuer) {
                                #pragma unroll
                                for (int b = 0; b < 4; ++b) {
                                    const int x = n0 + ph * EPI_COLS + (b & 1) * TC_BOX, y = m0 + (b >> 1) * TC_BOX;
                                    if (x < g.N && y < g.M) tma_store_3d(&tma_d, buf + b * BOX_BYTES, x, y, tc.c);
                                }
                                bulk_commit();
                            }
                            ++epi_it;
                        }
                    }
                } else {
                // operand of the axpy term, requested before the accumulator is ready
                uint4 cin_raw[8];
                auto load_cin = [&](int ph) {
                    const int gc0 = n0 + ph * EPI_COLS + half * 64;
                    #pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        if (row_ok && gc0 + 8 * q < g.N) cin_raw[q] = *reinterpret_cast<const uint4*>(g.cin + row_off + gc0 + 8 * q);
                        else cin_raw[q] = make_uint4(0u, 0u, 0u, 0u);
                    }
                };
                if (g.cin) load_cin(0);
                bool ok = mbar_wait(bar_acc_full + 8 * acc, (acc_par >> acc) & 1u, abort_flag, status, 4);
                ok = epi_bar_all(3, ok);           // all epilogue threads take the same exit, so no one is left at a barrier
                if (!ok) { alive = false; break; }
                tc_fence_after();
                acc_par ^= 1u << acc;
                const uint32_t t_base = tmem_base + lane_base + acc * TC_BN + half * 64;
                for (int ph = 0; ph < nphases; ++ph) {
                    float v[64];
                    tmem_ld32(t_base + ph * EPI_COLS, v);
                    tmem_ld32(t_base + ph * EPI_COLS + 32, v + 32);
                    tmem_ld_wait();
                    if (ph == nphases - 1) {
                        // this warp has read all it needs from the accumulator: hand it back to the MMA issuer
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(acc_empty_leader + 8 * acc);
                    }
                    const int gc0 = n0 + ph * EPI_COLS + half * 64;
                    if (g.cin) {
                        const uint32_t w[32] = {cin_raw[0].x, cin_raw[0].y, cin_raw[0].z, cin_raw[0].w, cin_raw[1].x, cin_raw[1].y,
                                                cin_raw[1].z, cin_raw[1].w, cin_raw[2].x, cin_raw[2].y, cin_raw[2].z, cin_raw[2].w,
                                                cin_raw[3].x, cin_raw[3].y, cin_raw[3].z, cin_raw[3].w, cin_raw[4].x, cin_raw[4].y,
                                                cin_raw[4].z, cin_raw[4].w, cin_raw[5].x, cin_raw[5].y, cin_raw[5].z, cin_raw[5].w,
                                                cin_raw[6].x, cin_raw[6].y, cin_raw[6].z, cin_raw[6].w, cin_raw[7].x, cin_raw[7].y,
                                                cin_raw[7].z, cin_raw[7].w};
                        #pragma unroll
                        for (int h = 0; h < 32; ++h) {
                            v[2 * h] = fmaf(c1, __uint_as_float(w[h] << 16), c2 * v[2 * h]);
                            v[2 * h + 1] = fmaf(c1, __uint_as_float(w[h] & 0xffff0000u), c2 * v[2 * h + 1]);
                        }
                        if (ph + 1 < nphases) load_cin(ph + 1);
                    } else {
                        #pragma unroll
                        for (int j = 0; j < 64; ++j) v[j] *= c2;
                    }
                    if (g.diag_add != 0.f && gr >= gc0 && gr < gc0 + 64) {
                        #pragma unroll
                        for (int j = 0; j < 64; ++j) v[j] += (gc0 + j == gr) ? g.diag_add : 0.f;
                    }
                    // the staging buffer is free once the stores issued EPI_BUFS phases ago have read it
                    const uint32_t buf = epi_base + (epi_it % C::EPI_BUFS) * EPI_BUF_BYTES;
                    if (issuer) bulk_wait_read<C::EPI_BUFS - 1>();
                    epi_bar_sync(1);
                    #pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const uint4 pk = pack8(v + 8 * q);
                        const uint32_t addr = buf + stage_off + (((uint32_t)q ^ swz) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(pk.x), "r"(pk.y), "r"(pk.z), "r"(pk.w)
                                     : "memory");
                    }
                    fence_proxy_async();           // generic-proxy writes above must be visible to the TMA engine
                    epi_bar_sync(2);
                    if (issuer) {
                        #pragma unroll
                        for (int b = 0; b < 4; ++b) {
                            const int x = n0 + ph * EPI_COLS + (b & 1) * TC_BOX, y = m0 + (b >> 1) * TC_BOX;
                            if (x < g.N && y < g.M) tma_store_3d(&tma_d, buf + b * BOX_BYTES, x, y, tc.c);   // clipped at the extents
                        }
                        bulk_commit();
                    }
                    ++epi_it;
                }
                            }
}
            if (!WIDE) acc_next ^= 1u;
        }
        if (issuer) bulk_wait_all();           // shared memory must outlive the stores that read it
    }

    if (*abort_flag) __nanosleep(200000);      // let copies that are still in flight land before the CTA goes away
    tc_fence_before();
    __syncthreads();
    cluster_sync();                            // neither CTA leaves (or frees tensor memory) while its peer may still signal it
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
    if (g.symmetric) g.wide = 0;
    if (g.wide) g.tiles_per_mat = g.tiles_m * ((g.tiles_n + 1) / 2);
    else g.tiles_per_mat = g.symmetric ? g.tiles_m * (g.tiles_m + 1) / 2 : g.tiles_m * g.tiles_n;
}

double tc_gemm_executed_flops(const TcGemm& g) {
    const double kpad = (double)((g.K + TC_BK - 1) / TC_BK * TC_BK);
    const double tiles256 = g.symmetric ? g.tiles_m * (g.tiles_m + 1) / 2 : g.tiles_m * g.tiles_n;
    return 2.0 * TC_BM * TC_BN * kpad * tiles256 * g.C;
}

namespace {
template <bool WIDE>
cudaError_t configure_one(int sms, int* clusters) {
    cudaError_t e = cudaFuncSetAttribute(tc_gemm_kernel<WIDE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<WIDE>::SMEM_TOTAL);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(sms / 2 * 2));
    cfg.blockDim = dim3(TC_THREADS);
    cfg.dynamicSmemBytes = Cfg<WIDE>::SMEM_TOTAL;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaOccupancyMaxActiveClusters(clusters, tc_gemm_kernel<WIDE>, &cfg);
}
}  // namespace

cudaError_t tc_gemm_configure(int* max_pairs) {
    int dev = 0, sms = 0;
    cudaError_t e;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    int c0 = 0, c1 = 0;
    if ((e = configure_one<false>(sms, &c0)) != cudaSuccess) return e;
    if ((e = configure_one<true>(sms, &c1)) != cudaSuccess) return e;
    const int clusters = c0 < c1 ? c0 : c1;
    if (clusters < 1) return cudaErrorInvalidConfiguration;
    *max_pairs = clusters < sms / 2 ? clusters : sms / 2;
    return cudaSuccess;
}

cudaError_t launch_tc_gemm(const CUtensorMap& tma_a, const CUtensorMap& tma_b, const CUtensorMap& tma_d,
                           const TcGemm& g, int max_pairs, DeviceStatus* status, cudaStream_t stream) {
    const int total = g.C * g.tiles_per_mat;
    if (total <= 0) return cudaSuccess;
    const int pairs = total < max_pairs ? total : max_pairs;
    if (g.wide) tc_gemm_kernel<true><<<2 * pairs, TC_THREADS, Cfg<true>::SMEM_TOTAL, stream>>>(tma_a, tma_b, tma_d, g, status);
    else        tc_gemm_kernel<false><<<2 * pairs, TC_THREADS, Cfg<false>::SMEM_TOTAL, stream>>>(tma_a, tma_b, tma_d, g, status);
    return cudaGetLastError();
}

}  // namespace mona
