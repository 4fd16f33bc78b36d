// Tensor-core Newton-Schulz iteration (Eq. newton_schulz) for sm_100a: ONE persistent kernel per chunk runs
// every GEMM of up to five iterations - A = X X^T, B' = b A + c A^2 + a I, X' = B' X - over all matrices of
// the chunk.
//
// Work items are 256 x 256 output tiles (256 x 512 macro-tiles for X' = B' X).  They are handed out through
// one atomic counter, in an order in which every item follows the items it depends on, and the phase-to-phase
// dependency of a matrix is a counter in global memory: the pair that takes phase q of matrix c waits until
// all items of phase q - 1 of matrix c have been stored.  Because a waiting pair only waits for items that
// running pairs already hold, the scheme cannot deadlock whatever share of the grid is resident.  There is no
// launch boundary, no partial last wave and no static tile assignment between the GEMMs of a chunk; the
// intermediate matrices are consumed a few hundred microseconds after they were produced.
//
// The kernel runs as clusters of two CTAs on neighbouring SMs; one tcgen05.mma.cta_group::2 instruction
// stream, issued by the even CTA (the "leader"), drives the tensor cores of both SMs.  Each CTA stages its own
// 128 rows of the A operand and its own 128 rows of the B operand per k-slice, so a pair moves 64 KiB from L2
// per 256 x 256 x 64 step (half of what two independent 128 x 256 tiles would).  Roles inside a CTA:
//   warp 2     (leader only) scheduler: takes items from the counter, waits for their dependencies and publishes them
//              to both CTAs through a small ring in shared memory, a few items ahead of the pipeline, so that the
//              round trips to the counters never hold up a copy,
//   warp 0     TMA producer: operand boxes into a ring of shared-memory stages; the copies of both CTAs
//              complete on the leader's "full" barrier,
//   warp 1     owner of tensor memory; in the leader its lane 0 issues the MMAs and commits them to
//              the "empty" barriers of both CTAs (multicast commit),
//   warps 4-11 epilogue: tcgen05.ld the CTA's 128 x 256 fp32 accumulator, apply the polynomial term
//              (b A + c A^2 + a I) and the deferred 1/||M||_F scale, pack to bf16 into swizzled shared
//              memory and hand the boxes to TMA stores (a thread owns one row, so storing from registers
//              would touch 32 lines per warp instruction; the TMA writes whole lines);
//              for the last X' = B' X of a step the same warps apply the parameter update of Eq. muon_update
//              to the fp32 weights instead,
//   warp 3     store warp: turns each staged phase into TMA stores, frees the staging buffer, and counts the item as
//              done once its stores have completed, so that no epilogue warp ever waits for global memory.
// Tensor memory holds two 256-column accumulators.  Plain tiles alternate between them, so the epilogue of one
// tile overlaps the main loop of the next.  A macro-tile uses both at once, two neighbouring tiles computed
// from ONE staged slice of the A operand: 96 KiB instead of 128 KiB cross from L2 per k-slice and pair.
//
// Every wait - on an mbarrier or on a dependency counter - is bounded: when one runs out the CTA latches
// STATUS_TIMEOUT, raises its abort flag, and all roles fall through to the common exit, where tensor memory
// is released.
#include "ns_tc.cuh"

namespace mona {

namespace {

constexpr int TC_EPI_WARPS = 8;                                   // two warps per tensor-memory lane quadrant
constexpr int TC_EPI_THREADS = 32 * TC_EPI_WARPS;
constexpr int SCHED_WARP = 2;                                     // the scheduler (leader CTA)
constexpr int STORE_WARP = 3;                                     // issues and retires the TMA stores of the epilogue
constexpr int EPI_WARP0 = 4;                                      // epilogue = warps 4..11, i.e. warpgroups 1 and 2
constexpr int TC_THREADS = 32 * EPI_WARP0 + TC_EPI_THREADS;       // 384
// The kernel starts with 152 registers per thread (12 warps x 32 x 152 = 58368 of the SM's 65536: the rest, together
// with the ~1.5 KiB of shared memory the kernel leaves, lets one 128-thread block of the elementwise kernels of the
// NEXT chunk run beside it, so prologue and update overlap the GEMMs instead of waiting for the SMs).  Then the
// warpgroup of the producer, MMA issuer, scheduler and store warp gives registers back and the two epilogue warpgroups
// take them (setmaxnreg): 128 x 56 + 256 x 200 = 58368.  An epilogue thread can then hold its share of BOTH
// accumulators of a macro-tile.
constexpr int TC_MAX_REGS = 152;
constexpr int REGS_CONTROL = 56;
constexpr int REGS_EPILOGUE = 200;
constexpr int CTA_M = TC_BM / 2;                                  // accumulator rows held by one CTA
constexpr int CTA_N = TC_BN / 2;                                  // B-operand rows one CTA stages per 256-column tile
constexpr uint32_t BOX_BYTES = TC_BOX * TC_BOX * 2;               // 8 KiB
constexpr uint32_t A_STAGE_BYTES = CTA_M * TC_BK * 2;             // 16 KiB
constexpr uint32_t B_SUB_BYTES = CTA_N * TC_BK * 2;               // 16 KiB per 256-column tile
constexpr int EPI_COLS = 128;                                     // output columns per epilogue phase
constexpr uint32_t EPI_BUF_BYTES = CTA_M * EPI_COLS * 2;          // 32 KiB = 2 x 2 boxes: staging buffer of the store epilogue
constexpr uint32_t TMEM_COLS = 512;                               // 2 accumulators x 256 fp32 columns
// Operand staging: a ring of 16 KiB slabs.  A k-slice takes one slab per operand part it stages (1: diagonal tile whose
// operands coincide, 2: plain tile, 3: macro-tile), contiguous (a k-slice that does not fit before the end of the ring
// starts again at slab 0), so plain tiles run six k-slices ahead and macro-tiles four.  Every k-slice in flight owns one
// entry of a ring of "full"/"empty" barriers; producer and MMA issuer derive the same slab positions from the item sequence.
constexpr int NSLAB = 12;
constexpr int NENT = 12;                                          // barrier entries = most k-slices in flight
constexpr uint32_t SLAB_BYTES = 16384;
static_assert(SLAB_BYTES == A_STAGE_BYTES && SLAB_BYTES == B_SUB_BYTES, "one slab per operand part");
constexpr int RING = 4;                                           // published-but-unfinished work items
constexpr uint32_t SMEM_CTRL_BYTES = 512;
constexpr uint32_t SMEM_TOTAL = NSLAB * SLAB_BYTES + EPI_BUF_BYTES + SMEM_CTRL_BYTES + 1024;
constexpr long long WAIT_BUDGET_CYCLES = 1000000000ll;            // ~0.5 s
// readers of a published item: producer, MMA issuer, store warp and epilogue warps in the leader; producer, store warp and
// epilogue warps in the peer
constexpr uint32_t RING_READERS = 3 + TC_EPI_WARPS + 2 + TC_EPI_WARPS;
static_assert(SMEM_TOTAL <= 232448, "shared memory budget");
static_assert(8 * (2 * NENT + 4 + 2 * RING + 4) + 16 + 16 * RING + 4 * (NS_MAX_PHASES + 1) <= SMEM_CTRL_BYTES, "control block");

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---- profiling build (-DMONA_TRACE) ---------------------------------------------------------------
// Every role adds up, in registers, the cycles its waits took and flushes them once per work item into a per-CTA table
// in shared memory; the MMA issuer also counts cycles and k-slices per kind of tile.  The tables are summed into
// g_trace[blockIdx.x] when a launch ends and read back with ns_trace_read().  The arithmetic of the kernel is unchanged;
// the clock reads cost a few per cent of its speed.  Without the flag all of this compiles to nothing.
#ifdef MONA_TRACE
__device__ unsigned long long g_trace[NS_TRACE_ROWS][NS_TRACE_SLOTS];
__device__ __forceinline__ uint32_t trace_clock() {
    uint32_t c;
    asm volatile("mov.u32 %0, %%clock;" : "=r"(c));
    return c;
}
#define TRACE_ONLY(...) __VA_ARGS__
#define TRACE_PTR(x) (&(x))
#else
#define TRACE_ONLY(...)
#define TRACE_PTR(x) nullptr
#endif

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
// Publication of shared-memory data to both CTAs of the pair: ONE release fence at cluster scope, then an arrival without
// semantics of its own per barrier (a release on each arrival would be a second fence of the same cost).
__device__ __forceinline__ void fence_release_cluster() { asm volatile("fence.acq_rel.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive_relaxed_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_arrive_local(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Hand-back of a ring slot whose 16 bytes this thread has loaded into `c, q, t, stop`: nothing is published, so the arrival
// needs no release (at cluster scope that is a fence which waits for everything the thread has in flight - for the MMA issuer
// its queued tensor-core work, a couple of thousand cycles per item); it must only not be issued before the load has returned.
// The loaded words are never negative; folding their sign bit into the address makes the instruction depend on the load.
__device__ __forceinline__ void mbar_arrive_slot_read(uint32_t cluster_addr, uint32_t c, uint32_t q, uint32_t t, uint32_t stop) {
    const uint32_t zero = ((c | q | t | stop) >> 31) << 3;
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr + zero) : "memory");
}
// The same with the default semantics, for hand-overs that carry no shared-memory data (tensor-memory accumulators).
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// CLUSTER: acquire at cluster scope, for barriers through which the peer CTA passes ordinary shared-memory data
// (the item ring); the pipeline barriers (TMA bytes, tcgen05 commits, accumulator hand-over) use the default scope.
template <bool CLUSTER>
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    if (CLUSTER) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
    }
    return ok != 0;
}
__device__ __forceinline__ void latch_timeout(volatile int* abort_flag, DeviceStatus* status, unsigned site) {
    *abort_flag = 1;
    atomicOr(&status->flags, STATUS_TIMEOUT);
    status->timeout_site = site;
}
// Bounded wait.  Returns false when the CTA is aborting (this wait or another one ran out).
// `waited` (profiling build only, may be null) accumulates the cycles spent here, the first attempt included.
template <bool CLUSTER = false>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, DeviceStatus* status,
                                          unsigned site, uint32_t* waited = nullptr) {
    TRACE_ONLY(const uint32_t t_in = trace_clock();)
    if (mbar_try_wait<CLUSTER>(bar, parity)) {
        TRACE_ONLY(if (waited) *waited += trace_clock() - t_in;)
        return true;
    }
    const long long t0 = clock64();
    unsigned spins = 0;
    while (true) {
        if (mbar_try_wait<CLUSTER>(bar, parity)) {
            TRACE_ONLY(if (waited) *waited += trace_clock() - t_in;)
            return true;
        }
        if ((++spins & 63u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > WAIT_BUDGET_CYCLES) {
                latch_timeout(abort_flag, status, site);
                return false;
            }
        }
    }
}
__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned int* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Bounded wait until a dependency counter in global memory has reached `need` (acquire at device scope).
__device__ __forceinline__ bool wait_counter(const unsigned int* ctr, unsigned need, volatile int* abort_flag,
                                             DeviceStatus* status, unsigned site, uint32_t* waited = nullptr) {
    TRACE_ONLY(const uint32_t t_in = trace_clock();)
    if (ld_acquire_gpu(ctr) >= need) {
        TRACE_ONLY(if (waited) *waited += trace_clock() - t_in;)
        return true;
    }
    const long long t0 = clock64();
    unsigned spins = 0;
    while (true) {
        if (ld_acquire_gpu(ctr) >= need) {
            TRACE_ONLY(if (waited) *waited += trace_clock() - t_in;)
            return true;
        }
        __nanosleep(64);
        if ((++spins & 63u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > WAIT_BUDGET_CYCLES) {
                latch_timeout(abort_flag, status, site);
                return false;
            }
        }
    }
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
// all earlier store groups of this thread have finished READING shared memory (the staging buffer may be rewritten)
// (all but the PENDING most recent groups)
template <int PENDING>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(PENDING) : "memory"); }
// all earlier store groups of this thread have completed (their global writes are done)
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// Orders this thread's accesses through the generic proxy against its accesses through the asynchronous proxy (TMA), for
// one state space only: the unqualified fence costs over a thousand cycles wherever it stands.
__device__ __forceinline__ void fence_proxy_async_shared() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }

// Shared-memory matrix descriptor (64 bits) for a 128-byte-swizzled bf16 tile whose rows are 128 bytes long and
// stacked densely (what a 64-wide TMA box with SWIZZLE_128B produces):
//   bits [0,14)  start address >> 4            bits [16,30) leading byte offset >> 4
//   bits [32,46) stride byte offset >> 4       bit 46       descriptor version for sm_100      bits [61,64) layout: 2 = 128-byte swizzle
//   K-major : row = m/n index, 128 B = 64 k.  Groups of 8 rows are 1024 B apart (stride byte offset);
//             the leading byte offset is not used by swizzled K-major layouts (encoded 1).
//   MN-major: row = k index, 128 B = 64 m/n.  Groups of 8 k-rows are 1024 B apart (stride byte offset);
//             the next 64 m/n lives in the next 8 KiB box (leading byte offset).
// Shared-memory addresses are below 256 KiB, so address >> 4 fits its field and the low word is address >> 4 | offset field.
constexpr uint32_t DESC_LBO_K = 1u << 16;
constexpr uint32_t DESC_LBO_MN = (BOX_BYTES >> 4) << 16;
constexpr uint32_t DESC_HI = (1024u >> 4) | (1u << 14) | (2u << 29);
// Instruction descriptor, kind::f16: D fp32 (bit 4), A and B bf16 (bits 7, 10), N >> 3 at bit 17, M >> 4 at bit 24 (M = 256 over
// the pair, N = 256); bits 15 / 16 say that A / B is MN-major.
constexpr uint32_t IDESC_BASE = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TC_BN >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);

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
// The two shared-memory matrix descriptors are given by their low words; the high word is the same for every operand.
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint32_t a_desc_lo, uint32_t b_desc_lo, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "mov.b64 da, {%1, %5};\n\t"
        "mov.b64 db, {%2, %5};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_desc_lo), "r"(b_desc_lo), "r"(idesc), "r"(accumulate), "r"(DESC_HI)
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

// A published work item: item `t` of phase `q` for matrix `c`; stop != 0 ends the role loops.
struct Item {
    int c, q, t, stop;
};

struct TileCoord {
    int tm, tn;      // tile row, first tile column
    int nsub;        // 256-column tiles in this item: 1 or 2
};

__device__ __forceinline__ TileCoord decode_tile(const NsPhase& p, int r) {
    TileCoord tc;
    tc.nsub = 1;
    if (p.wide) {
        const int macro_n = (p.tiles_n + 1) >> 1;
        tc.tm = r / macro_n;
        tc.tn = 2 * (r - tc.tm * macro_n);
        tc.nsub = tc.tn + 1 < p.tiles_n ? 2 : 1;
    } else if (p.symmetric) {
        int tm = 0;
        while ((tm + 1) * (tm + 2) / 2 <= r) ++tm;     // lower triangle, row by row
        tc.tm = tm;
        tc.tn = r - tm * (tm + 1) / 2;
    } else {
        tc.tm = r / p.tiles_n;
        tc.tn = r - tc.tm * p.tiles_n;
    }
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

// 32-byte accesses to fp32 rows (the parameter update of the fused epilogue)
__device__ __forceinline__ void ld8(const float* p, float* v) {
    asm volatile("ld.global.cs.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
                 : "l"(p));
}
// 32 bytes of bf16 data written earlier in this launch by other CTAs: from L2 (.cg), never from a line L1 may still hold
__device__ __forceinline__ void ld8cg(const void* p, uint32_t* w) {
    asm volatile("ld.global.cg.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                 : "l"(p));
}
__device__ __forceinline__ void st8(float* p, const float* v) {
    asm volatile("st.global.cs.v8.f32 [%8], {%0, %1, %2, %3, %4, %5, %6, %7};"
                 ::"f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]), "l"(p)
                 : "memory");
}

// Per-matrix pointers of the fused parameter update, passed by value (all null when no phase fuses it).
struct UpdateTable {
    float* w[MAXC];
    float* o[MAXC];
};

__global__ void __cluster_dims__(2, 1, 1) __maxnreg__(TC_MAX_REGS)
ns_chunk_kernel(const __grid_constant__ NsMaps maps, const __grid_constant__ NsProgram g,
                const __grid_constant__ UpdateTable upd, DeviceStatus* __restrict__ status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;       // swizzle atoms need 1024-byte alignment
    const uint32_t epi_buf = base + NSLAB * SLAB_BYTES;
    const uint32_t ctrl = epi_buf + EPI_BUF_BYTES;
    const uint32_t bar_full = ctrl;                             // NENT x 8 B (used in the leader)
    const uint32_t bar_empty = bar_full + 8 * NENT;             // NENT x 8 B
    const uint32_t bar_acc_full = bar_empty + 8 * NENT;         // 2 x 8 B, one per accumulator
    const uint32_t bar_acc_empty = bar_acc_full + 16;           // 2 x 8 B (used in the leader)
    const uint32_t bar_ring_full = bar_acc_empty + 16;          // RING x 8 B
    const uint32_t bar_ring_empty = bar_ring_full + 8 * RING;   // RING x 8 B (used in the leader)
    const uint32_t bar_stg_full = bar_ring_empty + 8 * RING;    // 2 x 8 B: a 64-column half of the staging buffer written (its 4 warps)
    const uint32_t bar_stg_empty = bar_stg_full + 16;           // 2 x 8 B: that half read by its store (store warp)
    const uint32_t tmem_slot = bar_stg_empty + 16;              // 4 B + abort flag 4 B + 8 B pad
    const uint32_t ring_items = tmem_slot + 16;                 // RING x 16 B
    // items per matrix of the phases before phase q (q = 0 .. P): phase q has phase_first[q + 1] - phase_first[q] items
    volatile unsigned int* phase_first = reinterpret_cast<volatile unsigned int*>(smem_raw + (ring_items + 16 * RING - smem_u32(smem_raw)));   // (NS_MAX_PHASES + 1) x 4 B
    uint8_t* ctrl_ptr = smem_raw + (ctrl - smem_u32(smem_raw));
    volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(ctrl_ptr + (tmem_slot - ctrl));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl_ptr + (tmem_slot - ctrl) + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                    // 0: leader, 1: peer
    const int P = g.P;
#ifdef MONA_TRACE
    __shared__ unsigned long long s_trace[NS_TRACE_SLOTS];
    const uint32_t t_kernel0 = trace_clock();
    if (threadIdx.x < NS_TRACE_SLOTS) s_trace[threadIdx.x] = 0ull;
    auto trace_add = [&](int slot, uint32_t v) { atomicAdd(&s_trace[slot], (unsigned long long)v); };
#endif

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        unsigned first = 0u;
        for (int q = 0; q <= NS_MAX_PHASES; ++q) { phase_first[q] = first; if (q < P) first += (unsigned)g.ph[q].items_per_mat; }
        for (int s = 0; s < NENT; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(bar_acc_full + 8 * a, 1); mbar_init(bar_acc_empty + 8 * a, 2 * TC_EPI_WARPS); }
        for (int r = 0; r < RING; ++r) { mbar_init(bar_ring_full + 8 * r, 1); mbar_init(bar_ring_empty + 8 * r, RING_READERS); }
        for (int b = 0; b < 2; ++b) { mbar_init(bar_stg_full + 8 * b, TC_EPI_WARPS / 2); mbar_init(bar_stg_empty + 8 * b, 1); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        #pragma unroll
        for (int i = 0; i < NS_MAPS; ++i) asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.m[i]) : "memory");
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

    // A reader's view of the item ring: wait for the n-th published item, copy it, hand the slot back.
    const uint32_t ring_empty_leader = map_to_cta(bar_ring_empty, 0);
    auto take_item = [&](unsigned n, Item& it, unsigned site, bool arrive, uint32_t* waited = nullptr) -> bool {
        const uint32_t slot = n % RING, par = (n / RING) & 1u;
        if (!mbar_wait<true>(bar_ring_full + 8 * slot, par, abort_flag, status, site, waited)) return false;
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(it.c), "=r"(it.q), "=r"(it.t), "=r"(it.stop) : "r"(ring_items + 16 * slot) : "memory");
        if (arrive) mbar_arrive_slot_read(ring_empty_leader + 8 * slot, it.c, it.q, it.t, it.stop);
        return true;
    };

    // TMA loads of all k-slices of one item into the stage ring (both CTAs run this, each for its own rows).
    // producer's view of the slab ring: next entry, next slab, oldest entry not yet known to be free, free slabs, and
    // the slabs every entry in flight took (3 bits each, wrap-around gap included)
    uint32_t ent = 0, slab_head = 0, tail_ent = 0, slabs_free = NSLAB;
    uint32_t ent_e = 0, ent_par = 0, tail_e = 0, tail_par = 0;     // entries modulo NENT and their use parities, kept incrementally
    unsigned long long ent_cost = 0ull;
    TRACE_ONLY(uint32_t w_empty = 0;)
    const uint32_t full_leader = map_to_cta(bar_full, 0);
    auto produce = [&](const Item& it) -> bool {
        const NsPhase& p = g.ph[it.q];
        const TileCoord tc = decode_tile(p, it.t);
        // K-major operands come as one box of 128 rows, MN-major ones as two boxes of 64 (the swizzle row is 64 elements)
        const CUtensorMap* a_box64 = &maps.m[p.a_map];
        const CUtensorMap* a_box128 = &maps.m[p.a_map + NS_TENSORS];
        const CUtensorMap* b_box64 = &maps.m[p.b_map];
        const CUtensorMap* b_box128 = &maps.m[p.b_map + NS_TENSORS];
        const int m0 = tc.tm * TC_BM + (int)rank * CTA_M;      // this CTA's rows of the A operand
        const int n0 = tc.tn * TC_BN + (int)rank * CTA_N;      // this CTA's rows of the B operand (first sub-tile)
        // diagonal tile of X X^T or A A: both operands are the same rows, staged once
        const bool shared_ab = p.ab_same && tc.tm == tc.tn && tc.nsub == 1;
        const int nb = shared_ab ? 0 : tc.nsub;
        const uint32_t tx_bytes = 2u * (A_STAGE_BYTES + (uint32_t)nb * B_SUB_BYTES) + (uint32_t)g.selftest_extra_tx;
        const int num_kb = (p.K + TC_BK - 1) / TC_BK;
        // from k-slice `switch` on the operand is MN-major (see the MMA issuer)
        const int a_switch = p.a_sym ? (tc.tm + 1) * (TC_BM / TC_BK) : (p.a_mn ? 0 : num_kb);
        const int b_switch0 = p.b_sym ? (tc.tn + 1) * (TC_BN / TC_BK) : (p.b_mn ? 0 : num_kb);
        const int b_switch1 = p.b_sym ? (tc.tn + 2) * (TC_BN / TC_BK) : (p.b_mn ? 0 : num_kb);
        const uint32_t nslab = 1u + (uint32_t)nb;
        for (int kb = 0; kb < num_kb; ++kb) {
            const uint32_t gap = slab_head + nslab > NSLAB ? NSLAB - slab_head : 0u;     // slabs skipped at the end of the ring
            const uint32_t need = gap + nslab;
            while (slabs_free < need) {        // entries are released in order: take back the oldest one's slabs
                if (!mbar_wait(bar_empty + 8 * tail_e, tail_par, abort_flag, status, 1, TRACE_PTR(w_empty))) return false;
                slabs_free += (uint32_t)(ent_cost >> (3 * tail_e)) & 7u;
                ++tail_ent;
                if (++tail_e == NENT) { tail_e = 0; tail_par ^= 1u; }
            }
            slabs_free -= need;
            const uint32_t e = ent_e;
            ent_cost = (ent_cost & ~(7ull << (3 * e))) | ((unsigned long long)need << (3 * e));
            const uint32_t pos = gap ? 0u : slab_head;
            slab_head = pos + nslab == NSLAB ? 0u : pos + nslab;
            ++ent;
            if (++ent_e == NENT) { ent_e = 0; ent_par ^= 1u; }
            if (!MONA_IN_BOUNDS(pos + nslab <= NSLAB && e < NENT && it.c < g.C, status, 102)) return false;
            const uint32_t full = full_leader + 8 * e;
            const uint32_t sa = base + pos * SLAB_BYTES;
            const int k0 = kb * TC_BK;
            if (rank == 0) mbar_arrive_expect_tx(bar_full + 8 * e, tx_bytes);   // both CTAs' copies land here
            if (kb >= a_switch) {
                tma_load_3d(sa, a_box64, full, m0, k0, it.c);
                tma_load_3d(sa + BOX_BYTES, a_box64, full, m0 + TC_BOX, k0, it.c);
            } else {
                tma_load_3d(sa, a_box128, full, k0, m0, it.c);
            }
            if (nb > 0) {
                const uint32_t sb = sa + A_STAGE_BYTES;
                if (kb >= b_switch0) {
                    tma_load_3d(sb, b_box64, full, n0, k0, it.c);
                    tma_load_3d(sb + BOX_BYTES, b_box64, full, n0 + TC_BOX, k0, it.c);
                } else {
                    tma_load_3d(sb, b_box128, full, k0, n0, it.c);
                }
                if (nb > 1) {
                    if (kb >= b_switch1) {
                        tma_load_3d(sb + B_SUB_BYTES, b_box64, full, n0 + TC_BN, k0, it.c);
                        tma_load_3d(sb + B_SUB_BYTES + BOX_BYTES, b_box64, full, n0 + TC_BN + TC_BOX, k0, it.c);
                    } else {
                        tma_load_3d(sb + B_SUB_BYTES, b_box128, full, k0, n0 + TC_BN, it.c);
                    }
                }
            }
        }
        return true;
    };

    if (warp < EPI_WARP0) {
    // the control warpgroup gives registers back (all four warps execute this together) ...
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_CONTROL));
    if (warp == 0) {
        if (lane == 0) {
            // ---------------- TMA producer (both CTAs) ----------------
            TRACE_ONLY(const uint32_t t_role0 = trace_clock(); uint32_t w_ring = 0;)
            bool ok = true;
            for (unsigned n = 0; ok; ++n) {
                Item it;
                if (!(ok = take_item(n, it, 8, true, TRACE_PTR(w_ring))) || it.stop) break;
                fence_proxy_async_global();       // the scheduler's acquire of the dependency precedes these copies
                ok = produce(it);
                TRACE_ONLY(trace_add(NS_TRACE_PRODUCER_EMPTY, w_empty); trace_add(NS_TRACE_PRODUCER_RING, w_ring); w_empty = w_ring = 0;)
            }
            TRACE_ONLY(trace_add(NS_TRACE_PRODUCER_RING, w_ring); trace_add(NS_TRACE_PRODUCER_ROLE, trace_clock() - t_role0);)
            // stay until the tensor cores have released every k-slice: the commits arrive on this CTA's barriers
            for (; ok && tail_ent < ent; ++tail_ent) {
                ok = mbar_wait(bar_empty + 8 * tail_e, tail_par, abort_flag, status, 5);
                if (++tail_e == NENT) { tail_e = 0; tail_par ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA only) ----------------
        if (lane == 0 && rank == 0) {
            uint32_t ment_e = 0, ment_par = 0, mslab = 0, acc_next = 0, acc_par = 0;   // acc_par: one use-parity bit per accumulator
            TRACE_ONLY(const uint32_t t_role0 = trace_clock(); uint32_t w_ring = 0;)
            bool ok = true;
            for (unsigned n = 0; ok; ++n) {
                Item it;
                if (!(ok = take_item(n, it, 9, true, TRACE_PTR(w_ring))) || it.stop) break;
                TRACE_ONLY(const uint32_t t_item0 = trace_clock(); uint32_t w_full = 0, w_acc = 0;)
                const NsPhase& p = g.ph[it.q];
                const TileCoord tc = decode_tile(p, it.t);
                const bool shared_ab = p.ab_same && tc.tm == tc.tn && tc.nsub == 1;
                const uint32_t acc0 = tc.nsub == 2 ? 0u : acc_next;
                const int num_kb = (p.K + TC_BK - 1) / TC_BK;
                // This one thread feeds both tensor cores, so the loop over k-slices is kept to a few dozen instructions:
                // everything that does not change inside a tile is worked out here.  An operand is MN-major from the k-slice
                // `switch` on (0: always, num_kb: never; a symmetric operand turns MN-major where it crosses its diagonal block).
                const int a_switch = p.a_sym ? (tc.tm + 1) * (TC_BM / TC_BK) : (p.a_mn ? 0 : num_kb);
                int b_switch[2];
                #pragma unroll
                for (int u = 0; u < 2; ++u)
                    b_switch[u] = shared_ab ? a_switch : (p.b_sym ? (tc.tn + u + 1) * (TC_BN / TC_BK) : (p.b_mn ? 0 : num_kb));
                const uint32_t b_off0 = shared_ab ? 0u : (A_STAGE_BYTES >> 4);             // operand offsets inside a stage, in 16-byte units
                const uint32_t b_off1 = (A_STAGE_BYTES + B_SUB_BYTES) >> 4;
                // an accumulator must have been drained by the epilogue of its previous tile before the first MMA into it
                if (!(ok = mbar_wait(bar_acc_empty + 8 * acc0, ((acc_par >> acc0) & 1u) ^ 1u, abort_flag, status, 2, TRACE_PTR(w_acc)))) break;
                tc_fence_after();
                const uint32_t d0 = tmem_base + acc0 * TC_BN, d1 = d0 + TC_BN;
                uint32_t accum = 0u;
                const uint32_t nslab = shared_ab ? 1u : 1u + (uint32_t)tc.nsub;
                for (int kb = 0; kb < num_kb; ++kb) {
                    // same slab walk as the producer's
                    const uint32_t pos = mslab + nslab > NSLAB ? 0u : mslab;
                    mslab = pos + nslab == NSLAB ? 0u : pos + nslab;
                    const uint32_t e = ment_e;
                    if (!MONA_IN_BOUNDS(pos + nslab <= NSLAB && tc.tm < p.tiles_m && tc.tn + tc.nsub <= p.tiles_n, status, 103)) { ok = false; break; }
                    const uint32_t stage_lo = (base + pos * SLAB_BYTES) >> 4;
                    // no tcgen05 fence here: the operands arrive through the asynchronous proxy and the barrier orders them
                    if (!(ok = mbar_wait(bar_full + 8 * e, ment_par, abort_flag, status, 3, TRACE_PTR(w_full)))) break;
                    if (++ment_e == NENT) { ment_e = 0; ment_par ^= 1u; }
                    const uint32_t a_mn = kb >= a_switch ? 1u : 0u, b_mn0 = kb >= b_switch[0] ? 1u : 0u;
                    // one k-step of 16 advances 32 B inside the swizzle row (K-major) or 16 rows = 2048 B (MN-major)
                    const uint32_t a_step = a_mn ? (2048u >> 4) : (32u >> 4), b_step0 = b_mn0 ? (2048u >> 4) : (32u >> 4);
                    const uint32_t a_lo = stage_lo | (a_mn ? DESC_LBO_MN : DESC_LBO_K);
                    const uint32_t b_lo0 = (stage_lo + b_off0) | (b_mn0 ? DESC_LBO_MN : DESC_LBO_K);
                    const uint32_t idesc0 = IDESC_BASE | (a_mn << 15) | (b_mn0 << 16);
                    #pragma unroll
                    for (int k = 0; k < TC_BK / 16; ++k) {
                        tc_mma_bf16(d0, a_lo + k * a_step, b_lo0 + k * b_step0, idesc0, accum);
                        accum = 1u;
                    }
                    if (tc.nsub == 2) {
                        if (kb == 0) {
                            if (!(ok = mbar_wait(bar_acc_empty + 8 * (acc0 + 1), ((acc_par >> (acc0 + 1)) & 1u) ^ 1u, abort_flag, status, 2, TRACE_PTR(w_acc)))) break;
                            tc_fence_after();
                        }
                        const uint32_t b_mn1 = kb >= b_switch[1] ? 1u : 0u;
                        const uint32_t b_step1 = b_mn1 ? (2048u >> 4) : (32u >> 4);
                        const uint32_t b_lo1 = (stage_lo + b_off1) | (b_mn1 ? DESC_LBO_MN : DESC_LBO_K);
                        const uint32_t idesc1 = IDESC_BASE | (a_mn << 15) | (b_mn1 << 16);
                        const uint32_t accum1 = kb != 0 ? 1u : 0u;
                        tc_mma_bf16(d1, a_lo, b_lo1, idesc1, accum1);
                        #pragma unroll
                        for (int k = 1; k < TC_BK / 16; ++k) tc_mma_bf16(d1, a_lo + k * a_step, b_lo1 + k * b_step1, idesc1, 1u);
                    }
                    tc_commit_pair(bar_empty + 8 * e);     // frees the k-slice's slabs in both CTAs when these MMAs have read them
                }
                if (!ok) break;
                for (int u = 0; u < tc.nsub; ++u) {
                    const uint32_t acc = acc0 + u;
                    tc_commit_pair(bar_acc_full + 8 * acc);    // accumulator complete, both CTAs' epilogues may read
                    acc_par ^= 1u << acc;
                }
                if (tc.nsub == 1) acc_next ^= 1u;
#ifdef MONA_TRACE
                {   // kind of tile: 0/1 X X^T off/on the diagonal, 2/3 b A + c A^2 + a I off/on the diagonal, 4 macro-tile, 5 single tile of X' = B' X
                    const int kind = !p.symmetric ? (tc.nsub == 2 ? 4 : 5) : ((p.cin ? 2 : 0) + (shared_ab ? 1 : 0));
                    const int slot = NS_TRACE_TILE0 + 4 * kind;
                    trace_add(slot, trace_clock() - t_item0); trace_add(slot + 1, (uint32_t)num_kb);
                    trace_add(slot + 2, w_full); trace_add(slot + 3, w_acc);
                    trace_add(NS_TRACE_MMA_RING, w_ring); w_ring = 0;
                }
#endif
            }
            TRACE_ONLY(trace_add(NS_TRACE_MMA_RING, w_ring); trace_add(NS_TRACE_MMA_ROLE, trace_clock() - t_role0);)
        }
    } else if (warp == STORE_WARP) {
        if (lane == 0) {
            // ---------------- store warp (both CTAs) ----------------
            // Sends every staged phase of the epilogue to D with TMA stores (this thread owns the bulk-copy groups, so it is
            // the one that can wait for them), frees the staging buffer when a phase has been read, and counts the item as
            // done for its matrix and phase once all of its stores have completed.  The epilogue warps never wait for global
            // memory.  It walks the items and their phases in the epilogue's order.
            uint32_t staged = 0;
            TRACE_ONLY(const uint32_t t_role0 = trace_clock(); uint32_t w_stg = 0;)
            bool ok = true;
            for (unsigned n = 0; ok; ++n) {
                Item it;
                if (!(ok = take_item(n, it, 12, true)) || it.stop) break;
                const NsPhase& p = g.ph[it.q];
                if (p.fuse_update) continue;               // the epilogue writes the parameters itself; nothing is staged
                const CUtensorMap* tma_d = &maps.m[p.d_map + NS_TENSORS];     // 64 columns x 128 rows per store
                const TileCoord tc = decode_tile(p, it.t);
                const int m0 = tc.tm * TC_BM + (int)rank * CTA_M;
                // The two 64-column halves of the staging buffer are separate buffers with their own barriers, filled by
                // different warps: each half is stored as soon as it is full and handed back as soon as its own store has
                // read it, the first half while the second store is still reading.
                for (int u = 0; u < tc.nsub && ok; ++u) {
                    for (int ph = 0; ph < 2 && ok; ++ph) {
                        const int x0 = (tc.tn + u) * TC_BN + ph * EPI_COLS;
                        if (x0 >= p.N) continue;
                        if (!MONA_IN_BOUNDS(m0 < p.M + CTA_M && it.c < g.C && tc.tm < p.tiles_m, status, 106)) { ok = false; break; }
                        #pragma unroll
                        for (int bx = 0; bx < 2; ++bx) {
                            if (!(ok = mbar_wait(bar_stg_full + 8 * bx, staged & 1u, abort_flag, status, 13, TRACE_PTR(w_stg)))) break;
                            const int x = x0 + bx * TC_BOX;
                            if (x < p.N && m0 < p.M) tma_store_3d(tma_d, epi_buf + bx * 2 * BOX_BYTES, x, m0, it.c);   // clipped at the extents
                            bulk_commit();
                        }
                        if (!ok) break;
                        bulk_wait_read<1>();               // the first store has read its half: its warps may refill it
                        mbar_arrive_local(bar_stg_empty);
                        bulk_wait_read<0>();
                        mbar_arrive_local(bar_stg_empty + 8);
                        ++staged;
                    }
                }
                if (!ok) break;
                bulk_wait_all();                           // the item's output is in global memory
                fence_proxy_async_global();
                __threadfence();
                atomicAdd(g.done + (size_t)it.c * P + it.q, 1u);
                TRACE_ONLY(trace_add(NS_TRACE_STORE_STAGED, w_stg); w_stg = 0; trace_add(NS_TRACE_ITEMS, 1u);)
            }
            bulk_wait_all();           // shared memory must outlive the stores that read it
            TRACE_ONLY(trace_add(NS_TRACE_STORE_ROLE, trace_clock() - t_role0);)
        }
    } else if (warp == SCHED_WARP) {
        if (lane == 0 && rank == 0) {
            // ---------------- scheduler (leader CTA only) ----------------
            const uint32_t ring_items_peer = map_to_cta(ring_items, 1), ring_full_peer = map_to_cta(bar_ring_full, 1);
            const uint32_t ring_full_own = map_to_cta(bar_ring_full, 0);
            // The item order and the cursor that walks it are NsItemCursor's (ns_tc.cuh); per-phase item counts come from
            // shared memory.
            NsItemCursor cursor(g.C, P, g.delay);
            auto decode = [&](unsigned idx, Item& it) -> bool {
                it.stop = idx >= g.total_items ? 1 : 0;
                it.c = it.q = it.t = 0;
                if (it.stop) return true;
                return cursor.find(idx, phase_first, it.c, it.q, it.t);      // false: the item count and the walk disagree
            };
            // The phase before an item must be complete for its matrix: its outputs are the item's operands, and the buffers
            // the item overwrites were last read two phases further back.
            auto dependency = [&](const Item& it, const unsigned int*& ctr, unsigned& need) {
                ctr = nullptr; need = 0u;
                if (!it.stop && it.q > 0) { ctr = g.done + (size_t)it.c * P + (it.q - 1); need = 2u * (phase_first[it.q] - phase_first[it.q - 1]); }
            };
            unsigned published = 0;
            TRACE_ONLY(const uint32_t t_role0 = trace_clock(); uint32_t w_slot = 0, w_dep = 0;)
            bool ok = true;
            // The counter is always asked for one item more than has been published, so that its round trip (as long as that
            // of the dependency check) runs beside the dependency wait of the item before.  An item claimed early is still
            // published in order and only after everything it depends on, all of it with smaller indices, is complete.
            unsigned next_idx = atomicAdd(g.work_counter, 1u);
            while (ok) {
                const uint32_t slot = published % RING, par = (published / RING) & 1u;
                if (!(ok = mbar_wait<true>(bar_ring_empty + 8 * slot, par ^ 1u, abort_flag, status, 7, TRACE_PTR(w_slot)))) break;
                const unsigned idx = next_idx;
                if (idx < g.total_items) next_idx = atomicAdd(g.work_counter, 1u);
                Item it;
                const bool found = decode(idx, it);
                if (!found || !it.stop && !MONA_IN_BOUNDS(it.c >= 0 && it.c < g.C && it.q >= 0 && it.q < P && it.t >= 0 && (unsigned)it.t < phase_first[it.q + 1] - phase_first[it.q], status, 101)) {
                    latch_timeout(abort_flag, status, 101);        // an item that does not exist: give up the launch, cleanly
                    break;
                }
                const unsigned int* ctr; unsigned need;
                dependency(it, ctr, need);
                if (ctr && !(ok = wait_counter(ctr, need, abort_flag, status, 6, TRACE_PTR(w_dep)))) break;
                // (no proxy fence here: this thread issues no copy; the producers fence after they have taken the item)
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(ring_items + 16 * slot), "r"(it.c), "r"(it.q), "r"(it.t), "r"(it.stop) : "memory");
                asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(ring_items_peer + 16 * slot), "r"(it.c), "r"(it.q), "r"(it.t), "r"(it.stop) : "memory");
                fence_release_cluster();       // the item, and the acquire of its dependency before it, precede both arrivals
                mbar_arrive_relaxed_cluster(ring_full_own + 8 * slot);
                mbar_arrive_relaxed_cluster(ring_full_peer + 8 * slot);
                ++published;
                TRACE_ONLY(trace_add(NS_TRACE_SCHED_SLOT, w_slot); trace_add(NS_TRACE_SCHED_DEPENDENCY, w_dep); w_slot = w_dep = 0;)
                if (it.stop) break;
            }
            TRACE_ONLY(trace_add(NS_TRACE_SCHED_ROLE, trace_clock() - t_role0);)
        }
    }
    } else {
        // ... and the two epilogue warpgroups take them
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_EPILOGUE));
        // ---------------- epilogue (warps 4..11, both CTAs) ----------------
        // A warp may only read the 32 tensor-memory lanes of its quadrant (warp index mod 4).  A 256-column
        // tile is handled in phases of 128 columns; in a phase the two warps of a quadrant take 64 columns
        // each, so a thread owns 64 consecutive columns of one row: one 128-byte line of the bf16 output.
        // The warps run independently of one another: they meet only at the staging buffer's two barriers.
        const int quad = warp & 3;
        const int half = (warp - EPI_WARP0) >> 2;
        const int row_in_cta = quad * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const uint32_t acc_empty_leader = map_to_cta(bar_acc_empty, 0);
        // position of this thread's row inside the staging buffer: one 128-row box per column half, 128-byte rows
        const uint32_t stage_off = (uint32_t)half * (2u * BOX_BYTES) + (uint32_t)row_in_cta * 128u;
        const uint32_t swz = (uint32_t)row_in_cta & 7u;
        uint32_t acc_next = 0, acc_par = 0;   // acc_par: one use-parity bit per accumulator
        uint32_t staged = 0;                  // staging phases handed to the store warp so far
        TRACE_ONLY(const uint32_t t_role0 = trace_clock(); uint32_t w_ring = 0, w_accf = 0, w_stge = 0;)
        bool alive = true;
        // 128 packed columns of this thread's row go to the staging buffer; the store warp sends them on
        auto put_phase = [&](const uint4* pk) -> bool {
            if (!mbar_wait(bar_stg_empty + 8 * half, (staged & 1u) ^ 1u, abort_flag, status, 11, TRACE_PTR(w_stge))) return false;   // the previous phase of this half has been read
            if (!MONA_IN_BOUNDS(stage_off + 128u <= EPI_BUF_BYTES, status, 104)) return false;
            #pragma unroll
            for (int q = 0; q < 8; ++q) {
                const uint32_t addr = epi_buf + stage_off + (((uint32_t)q ^ swz) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(pk[q].x), "r"(pk[q].y), "r"(pk[q].z), "r"(pk[q].w) : "memory");
            }
            fence_proxy_async_shared();            // generic-proxy writes above must be visible to the TMA engine
            __syncwarp();
            if (lane == 0) mbar_arrive_local(bar_stg_full + 8 * half);
            ++staged;
            return true;
        };
        for (unsigned n = 0; alive; ++n) {
            Item it;
            if (!take_item(n, it, 10, false, TRACE_PTR(w_ring))) break;
            __syncwarp();
            if (lane == 0) mbar_arrive_slot_read(ring_empty_leader + 8 * (n % RING), it.c, it.q, it.t, it.stop);   // every lane has its copy of the item
            if (it.stop) break;
            TRACE_ONLY(const uint32_t t_item0 = trace_clock();)
            const NsPhase& p = g.ph[it.q];
            const TileCoord tc = decode_tile(p, it.t);
            const int m0 = tc.tm * TC_BM + (int)rank * CTA_M;
            const int gr = m0 + row_in_cta;
            const bool row_ok = gr < p.M;
            const long long row_off = (long long)it.c * p.mat_stride + (long long)gr * p.ld;
            float post = 1.0f;
            if (p.post_mode) { const float sc = g.inv_norm[it.c]; post = p.post_mode == 2 ? sc * sc : sc; }
            const float c1 = p.c1 * post, c2 = p.c2 * post;
            const uint32_t acc0 = tc.nsub == 2 ? 0u : acc_next;
            if (!p.cin && !p.fuse_update && p.diag_add == 0.f) {
                // No axpy operand, no diagonal term (X X^T and X' = B' X).  A thread's share of an accumulator is 128 values,
                // 64 registers once packed: read and pack every accumulator of the item first, handing each back to the MMA
                // issuer as soon as it has been read, and only then stage.  Nothing hides the epilogue of a macro-tile, so
                // the time the tensor cores wait is the time of these reads.
                uint4 pk[2][2][8];
                #pragma unroll
                for (int u = 0; u < 2; ++u) {
                    if (u < tc.nsub && alive) {
                        const uint32_t acc = acc0 + u;
                        const int n0 = (tc.tn + u) * TC_BN;
                        if (!mbar_wait(bar_acc_full + 8 * acc, (acc_par >> acc) & 1u, abort_flag, status, 4, TRACE_PTR(w_accf))) { alive = false; break; }
                        tc_fence_after();
                        acc_par ^= 1u << acc;
                        const uint32_t t_base = tmem_base + lane_base + acc * TC_BN + half * 64;
                        #pragma unroll
                        for (int ph = 0; ph < 2; ++ph) {
                            if (n0 + ph * EPI_COLS < p.N) {
                                float v[64];
                                tmem_ld32(t_base + ph * EPI_COLS, v);
                                tmem_ld32(t_base + ph * EPI_COLS + 32, v + 32);
                                tmem_ld_wait();
                                #pragma unroll
                                for (int j = 0; j < 64; ++j) v[j] *= c2;
                                #pragma unroll
                                for (int q = 0; q < 8; ++q) pk[u][ph][q] = pack8(v + 8 * q);
                            }
                        }
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_remote(acc_empty_leader + 8 * acc);
                    }
                }
                #pragma unroll
                for (int u = 0; u < 2; ++u)
                    #pragma unroll
                    for (int ph = 0; ph < 2; ++ph)
                        if (alive && u < tc.nsub && (tc.tn + u) * TC_BN + ph * EPI_COLS < p.N) alive = put_phase(pk[u][ph]);
            } else
            for (int u = 0; u < tc.nsub && alive; ++u) {
                const uint32_t acc = acc0 + u;
                const int n0 = (tc.tn + u) * TC_BN;
                const int nphases = (p.N - n0 > EPI_COLS) ? 2 : 1;
                // Operand of the axpy term: this thread's 64 values of a phase (128 bytes), requested before the accumulator is
                // ready (first phase) or before the previous phase is staged (second), so that the round trip is hidden.  It was written by other CTAs of this
                // launch, so it is read from L2 (.cg), never from a line L1 may still hold from an earlier iteration.  A thread
                // owns a row, so a warp's load touches 32 lines whatever its width: 32-byte accesses halve the requests.
                uint32_t cin_w[32];
                const bool cin_v8 = p.cin && ((p.ld | p.mat_stride | (long long)p.N) & 15) == 0 && (reinterpret_cast<uintptr_t>(p.cin) & 31) == 0;
                auto load_cin = [&](int ph) {
                    const int gc0 = n0 + ph * EPI_COLS + half * 64;
                    if (cin_v8) {
                        #pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            if (row_ok && gc0 + 16 * q < p.N && MONA_IN_BOUNDS(row_off + gc0 + 16 * q + 16 <= (long long)g.C * p.mat_stride, status, 105)) ld8cg(p.cin + row_off + gc0 + 16 * q, cin_w + 8 * q);
                            else {
                                #pragma unroll
                                for (int j = 0; j < 8; ++j) cin_w[8 * q + j] = 0u;
                            }
                        }
                    } else {
                        #pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            uint4 r = make_uint4(0u, 0u, 0u, 0u);
                            if (row_ok && gc0 + 8 * q < p.N && MONA_IN_BOUNDS(row_off + gc0 + 8 * q + 8 <= (long long)g.C * p.mat_stride, status, 105)) r = __ldcg(reinterpret_cast<const uint4*>(p.cin + row_off + gc0 + 8 * q));
                            cin_w[4 * q] = r.x; cin_w[4 * q + 1] = r.y; cin_w[4 * q + 2] = r.z; cin_w[4 * q + 3] = r.w;
                        }
                    }
                };
                if (p.cin) load_cin(0);
                if (!mbar_wait(bar_acc_full + 8 * acc, (acc_par >> acc) & 1u, abort_flag, status, 4, TRACE_PTR(w_accf))) { alive = false; break; }
                tc_fence_after();
                acc_par ^= 1u << acc;
                const uint32_t t_base = tmem_base + lane_base + acc * TC_BN + half * 64;
                for (int ph = 0; ph < nphases && alive; ++ph) {
                    float v[64];
                    tmem_ld32(t_base + ph * EPI_COLS, v);
                    tmem_ld32(t_base + ph * EPI_COLS + 32, v + 32);
                    tmem_ld_wait();
                    if (ph == nphases - 1) {
                        // this warp has read all it needs from the accumulator: hand it back to the MMA issuer
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_remote(acc_empty_leader + 8 * acc);
                    }
                    const int gc0 = n0 + ph * EPI_COLS + half * 64;
                    if (p.cin) {
                        #pragma unroll
                        for (int h = 0; h < 32; ++h) {
                            v[2 * h] = fmaf(c1, __uint_as_float(cin_w[h] << 16), c2 * v[2 * h]);
                            v[2 * h + 1] = fmaf(c1, __uint_as_float(cin_w[h] & 0xffff0000u), c2 * v[2 * h + 1]);
                        }
                        if (ph + 1 < nphases) load_cin(ph + 1);
                    } else {
                        #pragma unroll
                        for (int j = 0; j < 64; ++j) v[j] *= c2;
                    }
                    if (p.diag_add != 0.f && gr >= gc0 && gr < gc0 + 64) {
                        #pragma unroll
                        for (int j = 0; j < 64; ++j) v[j] += (gc0 + j == gr) ? p.diag_add : 0.f;
                    }
                    if (!p.fuse_update) {
                        uint4 pk[8];
                        #pragma unroll
                        for (int q = 0; q < 8; ++q) pk[q] = pack8(v + 8 * q);
                        alive = put_phase(pk);
                    } else if (row_ok) {
                        // Eq. muon_update on this thread's 64 parameters: W <- (W - eta lambda W) - eta gamma O.  Nothing in the
                        // launch reads these stores (the phase is the last one of the step), so they need no completion signal.
                        float* wrow = upd.w[it.c] + (long long)gr * p.ld + gc0;
                        float* orow = upd.o[it.c] ? upd.o[it.c] + (long long)gr * p.ld + gc0 : nullptr;
                        #pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            if (gc0 + 8 * q < p.N) {
                                float w8[8];
                                ld8(wrow + 8 * q, w8);
                                #pragma unroll
                                for (int j = 0; j < 8; ++j) w8[j] = fmaf(-g.eta_gamma, v[8 * q + j], fmaf(-g.eta_lambda, w8[j], w8[j]));
                                st8(wrow + 8 * q, w8);
                                if (orow) st8(orow + 8 * q, v + 8 * q);
                            }
                        }
                    }
                }
            }
            if (tc.nsub == 1) acc_next ^= 1u;
#ifdef MONA_TRACE
            if (lane == 0) {      // one lane per warp: the table holds sums over the eight epilogue warps
                trace_add(NS_TRACE_EPI_RING, w_ring); trace_add(NS_TRACE_EPI_ACC_FULL, w_accf); trace_add(NS_TRACE_EPI_STAGE_EMPTY, w_stge);
                const bool diag = p.ab_same && tc.tm == tc.tn && tc.nsub == 1;
                const int kind = !p.symmetric ? (tc.nsub == 2 ? 4 : 5) : ((p.cin ? 2 : 0) + (diag ? 1 : 0));
                const int slot = NS_TRACE_EPI_TILE0 + 4 * kind;
                trace_add(slot, trace_clock() - t_item0); trace_add(slot + 1, 1u); trace_add(slot + 2, w_accf); trace_add(slot + 3, w_stge);
            }
            w_ring = w_accf = w_stge = 0;
#endif
        }
        TRACE_ONLY(if (lane == 0) trace_add(NS_TRACE_EPI_ROLE, trace_clock() - t_role0);)
    }

    TRACE_ONLY(if (threadIdx.x == 0) trace_add(NS_TRACE_KERNEL, trace_clock() - t_kernel0);)
    if (*abort_flag) __nanosleep(200000);      // let copies that are still in flight land before the CTA goes away
    tc_fence_before();
    __syncthreads();
    TRACE_ONLY(if (threadIdx.x < NS_TRACE_SLOTS) atomicAdd(&g_trace[blockIdx.x % NS_TRACE_ROWS][threadIdx.x], s_trace[threadIdx.x]);)
    cluster_sync();                            // neither CTA leaves (or frees tensor memory) while its peer may still signal it
    tc_fence_after();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace

cudaError_t ns_trace_read(unsigned long long* out, size_t rows, int reset, int* available) {
#ifdef MONA_TRACE
    *available = 1;
    if (rows > (size_t)NS_TRACE_ROWS) rows = NS_TRACE_ROWS;
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess && out && rows) e = cudaMemcpyFromSymbol(out, g_trace, rows * NS_TRACE_SLOTS * sizeof(unsigned long long));
    if (e == cudaSuccess && reset) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_trace);
        if (e == cudaSuccess) e = cudaMemset(p, 0, sizeof(unsigned long long) * NS_TRACE_ROWS * NS_TRACE_SLOTS);
    }
    return e;
#else
    (void)out; (void)rows; (void)reset;
    *available = 0;
    return cudaSuccess;
#endif
}

int ns_work_order(int C, int P, int delay, const unsigned int* items_per_phase, unsigned start, unsigned stride, int* cqt,
                  size_t capacity) {
    if (C <= 0 || P <= 0 || P > NS_MAX_PHASES || delay <= 0 || !items_per_phase || stride == 0 || (capacity && !cqt)) return -1;
    unsigned first[NS_MAX_PHASES + 1];
    first[0] = 0u;
    for (int q = 0; q < P; ++q) first[q + 1] = first[q] + items_per_phase[q];
    const unsigned long long total = (unsigned long long)first[P] * (unsigned long long)C;
    NsItemCursor cursor(C, P, delay);
    size_t n = 0;
    for (unsigned long long idx = start; idx < total && n < capacity; idx += stride, ++n) {
        int c, q, t;
        if (!cursor.find((unsigned)idx, first, c, q, t)) return -2;
        cqt[3 * n] = c; cqt[3 * n + 1] = q; cqt[3 * n + 2] = t;
    }
    return (int)n;
}

void ns_phase_plan(NsPhase& p) {
    p.tiles_m = (p.M + TC_BM - 1) / TC_BM;
    p.tiles_n = (p.N + TC_BN - 1) / TC_BN;
    if (p.symmetric || p.tiles_n < 2) p.wide = 0;      // a macro-tile needs two tile columns to pay
    if (p.wide) p.items_per_mat = p.tiles_m * ((p.tiles_n + 1) / 2);
    else p.items_per_mat = p.symmetric ? p.tiles_m * (p.tiles_m + 1) / 2 : p.tiles_m * p.tiles_n;
}

double ns_phase_executed_flops(const NsPhase& p) {
    const double kpad = (double)((p.K + TC_BK - 1) / TC_BK * TC_BK);
    const double tiles256 = p.symmetric ? p.tiles_m * (p.tiles_m + 1) / 2 : p.tiles_m * p.tiles_n;
    return 2.0 * TC_BM * TC_BN * kpad * tiles256;
}

void ns_program_plan(NsProgram& g) {
    unsigned long long total = 0;
    for (int q = 0; q < g.P; ++q) total += (unsigned long long)g.ph[q].items_per_mat * (unsigned long long)g.C;
    g.total_items = (unsigned int)total;
}

cudaError_t ns_configure(int* max_pairs) {
    int dev = 0, sms = 0;
    cudaError_t e;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(ns_chunk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_TOTAL)) != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(sms / 2 * 2));
    cfg.blockDim = dim3(TC_THREADS);
    cfg.dynamicSmemBytes = SMEM_TOTAL;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    if ((e = cudaOccupancyMaxActiveClusters(&clusters, ns_chunk_kernel, &cfg)) != cudaSuccess) return e;
    if (clusters < 1) return cudaErrorInvalidConfiguration;
    *max_pairs = clusters < sms / 2 ? clusters : sms / 2;
    return cudaSuccess;
}

cudaError_t launch_ns_program(const NsMaps& maps, const NsProgram& g, const NsUpdatePtrs& up, int max_pairs,
                              DeviceStatus* status, cudaStream_t stream) {
    if (g.total_items == 0) return cudaSuccess;
    const int pairs = (long long)g.total_items < (long long)max_pairs ? (int)g.total_items : max_pairs;
    static const UpdateTable no_update = {};
    const UpdateTable* table = &no_update;
    UpdateTable filled;
    if (up.w) {
        for (int c = 0; c < g.C; ++c) { filled.w[c] = up.w[c]; filled.o[c] = up.o ? up.o[c] : nullptr; }
        table = &filled;
    }
    ns_chunk_kernel<<<2 * pairs, TC_THREADS, SMEM_TOTAL, stream>>>(maps, g, *table, status);
    return cudaGetLastError();
}

}  // namespace mona
