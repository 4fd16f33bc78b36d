// Shared device-side declarations of the MONA step library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mona {

// A chunk is the unit that goes through prologue -> Newton-Schulz -> update together: up to MAXC
// same-shape matrices whose bf16 iterates fit the chunk budget (sized for full machine occupancy, not for cache).
constexpr int MAXC = 512;   // the pointer table below travels as a kernel argument (14 KiB of the 32 KiB CUDA 12 allows)
// Each matrix is cut into at most MAX_SLABS contiguous slabs for the elementwise passes; every slab
// owns one partial sum of squares, so the Frobenius norm is reduced in a fixed order.
constexpr int MAX_SLABS = 256;

// Slab decomposition of a matrix of e elements: ~16 K elements per slab, at most MAX_SLABS slabs, slab length a
// multiple of 1024 once the cap binds.
inline void slab_plan(long long e, long long* slab_len, int* slabs) {
    long long slab = 16384;
    if ((e + slab - 1) / slab > MAX_SLABS) slab = ((e + MAX_SLABS - 1) / MAX_SLABS + 1023) / 1024 * 1024;
    *slab_len = slab;
    *slabs = (int)((e + slab - 1) / slab);
}

// Per-chunk pointer table passed by value to the elementwise kernels.
struct ChunkPtrs {
    const void* g[MAXC];   // gradient of matrix c (fp32 or bf16)
    float* w[MAXC];        // parameter of matrix c
    float* o[MAXC];        // optional fp32 copy of O_k (may be null)
    int gid[MAXC];         // global matrix index (descriptor order), for error reports
};

// Device status word, latched by kernels and read by mona_poll_status().
struct DeviceStatus {
    unsigned int flags;        // bit 0: non-finite norm, bit 1: a bounded wait ran out
    int first_bad;             // lowest global matrix index that reported (or INT_MAX)
    unsigned int timeout_site; // which wait gave up (diagnostic)
    unsigned int pad;
};
constexpr unsigned STATUS_NONFINITE = 1u;
constexpr unsigned STATUS_TIMEOUT = 2u;
constexpr unsigned STATUS_BOUNDS = 4u;       // debug build only: an index check failed (site in timeout_site)

// Index checks of the debug build (-DMONA_DEBUG).  compute-sanitizer is not available everywhere this library is
// developed, so the kernels can check their own indices: a failed check latches STATUS_BOUNDS with a site number in the
// status word - it never traps - and the guarded access is skipped.  In the normal build the macro is `true`.
#ifdef MONA_DEBUG
#define MONA_IN_BOUNDS(cond, status, site) \
    ((cond) ? true : (atomicOr(&(status)->flags, ::mona::STATUS_BOUNDS), (status)->timeout_site = (site), false))
#else
#define MONA_IN_BOUNDS(cond, status, site) true
#endif

// A scalar hyper-parameter carried as an unevaluated sum of two floats, hi + lo, so that products with
// it are accurate to ~2^-45 instead of 2^-24: rounding beta_a = 0.99 to one float would by itself
// cost 3e-8 per step in the EMA, which accumulates over its ~1/(1-beta_a) step memory.
struct F2 {
    float hi, lo;
};

struct PrologueScalars {
    F2 beta;            // beta_a
    F2 one_minus_beta;  // 1 - beta_a, formed in double
    F2 alpha;           // alpha
    F2 mu;              // mu
    float eps;          // norm_eps
};

}  // namespace mona
