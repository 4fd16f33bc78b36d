// C ABI of the MONA step library: plan (shape buckets, chunking, state/workspace layout, TMA descriptors)
// and the per-step launch sequence.  See include/mona.h for the contract of every entry point.
#include <cuda.h>
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <algorithm>
#include <atomic>
#include <climits>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <string>
#include <tuple>
#include <vector>

#include "../../include/mona.h"
#include "common.cuh"
#include "elementwise.cuh"
#include "ns_fp32.cuh"
#include "ns_tc.cuh"

using namespace mona;

namespace {

// ---- workspace layout -------------------------------------------------------------------------------
// [status word | control block of slot 0 | control block of slot 1 | iterates of slot 0 | iterates of slot 1]
// Consecutive chunks alternate between two slots (and two streams), so that the last wave of each GEMM
// launch is filled by the other chunk's tiles and launch gaps of one chunk are covered by the other.
constexpr int NSLOTS = 2;
constexpr size_t WS_STATUS_OFF = 0;
constexpr size_t WS_CTRL_OFF = 4096;                 // first control block
constexpr size_t WS_CTRL_BYTES = 1024 * 1024;        // per slot
constexpr size_t CTRL_COUNTERS_OFF = 0;
constexpr size_t CTRL_INVNORM_OFF = 4096;
constexpr size_t CTRL_PARTIALS_OFF = 8192;
constexpr size_t CTRL_SCHED_OFF = CTRL_PARTIALS_OFF + sizeof(float) * MAXC * MAX_SLABS;   // work counter + done counters of the NS kernel
constexpr size_t WS_DATA_OFF = WS_CTRL_OFF + NSLOTS * WS_CTRL_BYTES;
static_assert(CTRL_SCHED_OFF + sizeof(unsigned int) * (64 + (size_t)MAXC * NS_MAX_PHASES) <= WS_CTRL_BYTES, "control block overflow");
static_assert(sizeof(unsigned int) * MAXC <= CTRL_INVNORM_OFF && sizeof(float) * MAXC <= CTRL_PARTIALS_OFF - CTRL_INVNORM_OFF, "control block overflow");

// Process-wide defaults behind mona_set_chunk_budget() / mona_set_chunk_overlap().  They only seed
// mona_default_options(); a handle keeps the options it was created with, so changing a default later
// never reaches an existing handle.
//   overlap: 1 = consecutive chunks are pipelined over two streams; 0 = everything on the caller's stream.
//   budget : bytes of bf16 iterates (X_t, X_{t+1}, A_t, B'_t) one chunk may hold.  Chunks are sized to keep every
//            SM pair busy, not for cache residency: chunks small enough to stay in L2 hold fewer tiles than the
//            device has CTA pairs.
constexpr size_t DEFAULT_CHUNK_BUDGET = 768ull << 20;
std::atomic<int> g_chunk_overlap{1};
std::atomic<size_t> g_chunk_budget_bytes{DEFAULT_CHUNK_BUDGET};

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// NVTX range over the host-side enqueue of a phase (shows up in timeline tools; costs nothing without one attached).
struct NvtxRange {
    explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
    NvtxRange(const NvtxRange&) = delete;
    NvtxRange& operator=(const NvtxRange&) = delete;
};

struct MatRef {
    int desc;
    int64_t b;
};

struct Bucket {
    int64_t rows = 0, cols = 0, s = 0, l = 0, e = 0;
    int grad_dtype = 0, state_dtype = 0;
    bool tall = false, tc_ok = false;
    std::vector<MatRef> mats;
    // bytes from the state base of the three blocks: M (fp32), A and G_prev (fp32, or bf16 with MONA-Lite storage)
    size_t off_M = 0, off_A = 0, off_G = 0;
    int Cb = 1, Cf = 1;         // chunk capacity: bf16 tensor-core mode / fp32 mode
    int slabs = 1;
    int64_t slab_len = 0;
    size_t off_x[2] = {0, 0}, off_a = 0, off_b = 0;          // bf16 mode, bytes from the slot's iterate base
    size_t off32_x[2] = {0, 0}, off32_a = 0, off32_b = 0;    // fp32 mode
    size_t data_bytes = 0;
    NsMaps maps[NSLOTS] = {};      // per workspace slot: X ping, X pong, A, B' of a chunk of this bucket
};
constexpr int MAP_X0 = 0, MAP_A = 2, MAP_B = 3;

struct Plan {
    std::vector<mona_matrix_desc> descs;
    std::vector<Bucket> buckets;
    std::vector<int> desc_bucket;          // bucket of descriptor i
    std::vector<int64_t> desc_pos;         // position of descriptor i's matrix 0 inside its bucket
    std::vector<int64_t> desc_first_gid;   // global matrix index (descriptor order) of matrix 0
    size_t state_bytes = 0, workspace_bytes = 0, slot_bytes = 0;
};

mona_status build_plan(const mona_matrix_desc* descs, int64_t n_desc, size_t chunk_budget, Plan& plan, std::string& err) {
    if (!descs || n_desc <= 0) { err = "descs is null or n_desc <= 0"; return MONA_ERR_INVALID_ARG; }
    plan.descs.assign(descs, descs + n_desc);
    std::map<std::tuple<int64_t, int64_t, int, int>, int> index;
    int64_t gid = 0;
    for (int64_t i = 0; i < n_desc; ++i) {
        mona_matrix_desc& d = plan.descs[i];
        if (d.rows <= 0 || d.cols <= 0 || d.batch <= 0) { err = "descriptor with non-positive rows/cols/batch"; return MONA_ERR_INVALID_ARG; }
        if (d.grad_dtype != MONA_F32 && d.grad_dtype != MONA_BF16) { err = "descriptor with unknown grad_dtype"; return MONA_ERR_INVALID_ARG; }
        if (d.state_dtype != MONA_F32 && d.state_dtype != MONA_BF16 && d.state_dtype != MONA_STATE_COMBINED) { err = "descriptor with unknown state_dtype"; return MONA_ERR_INVALID_ARG; }
        if (d.rows > (1 << 20) || d.cols > (1 << 20) || d.rows * d.cols > (1ll << 31)) { err = "matrix too large"; return MONA_ERR_UNSUPPORTED_SHAPE; }
        if (d.batch_stride == 0) d.batch_stride = d.rows * d.cols;
        if (d.batch_stride < d.rows * d.cols) { err = "batch_stride smaller than rows*cols"; return MONA_ERR_INVALID_ARG; }
        auto key = std::make_tuple(d.rows, d.cols, (int)d.grad_dtype, (int)d.state_dtype);
        auto it = index.find(key);
        int bi;
        if (it == index.end()) {
            bi = (int)plan.buckets.size();
            index[key] = bi;
            Bucket b;
            b.rows = d.rows; b.cols = d.cols; b.grad_dtype = d.grad_dtype; b.state_dtype = d.state_dtype;
            b.tall = d.rows > d.cols;
            b.s = std::min(d.rows, d.cols); b.l = std::max(d.rows, d.cols); b.e = d.rows * d.cols;
            // below 64 rows bf16 iterates of very wide matrices drift past the 2e-2 bound (measured 2.0-2.4e-2 at 32 x 1024),
            // so such matrices keep the fp32 path
            b.tc_ok = (b.s % 8 == 0) && (b.l % 8 == 0) && b.s >= 64;
            plan.buckets.push_back(b);
        } else {
            bi = it->second;
        }
        plan.desc_bucket.push_back(bi);
        plan.desc_pos.push_back((int64_t)plan.buckets[bi].mats.size());
        plan.desc_first_gid.push_back(gid);
        for (int64_t b = 0; b < d.batch; ++b) plan.buckets[bi].mats.push_back({(int)i, b});
        gid += d.batch;
    }
    size_t state_bytes = 0;
    size_t max_data = 0;
    for (Bucket& b : plan.buckets) {
        const int64_t count = (int64_t)b.mats.size();
        const size_t aux = b.state_dtype == MONA_BF16 ? 2 : 4;              // every block starts 256-byte aligned
        b.off_M = state_bytes; state_bytes += align_up((size_t)count * b.e * 4, 256);
        b.off_A = state_bytes; state_bytes += align_up((size_t)count * b.e * aux, 256);
        b.off_G = state_bytes;                                              // the single-buffer form has no G_prev block
        if (b.state_dtype != MONA_STATE_COMBINED) state_bytes += align_up((size_t)count * b.e * aux, 256);
        long long slab = 0;
        slab_plan(b.e, &slab, &b.slabs);
        b.slab_len = slab;
        // chunk capacity
        const size_t per_mat_bf16 = (size_t)(2 * b.e + 2 * b.s * b.s) * 2;
        int64_t cb = (int64_t)(chunk_budget / per_mat_bf16);
        cb = std::max<int64_t>(1, std::min<int64_t>(std::min<int64_t>(cb, MAXC), count));
        b.Cb = (int)cb;
        b.Cf = (int)std::max<int64_t>(1, cb / 2);
        size_t off = 0;
        for (int i = 0; i < 2; ++i) { b.off_x[i] = off; off += align_up((size_t)b.Cb * b.e * 2, 1024); }
        b.off_a = off; off += align_up((size_t)b.Cb * b.s * b.s * 2, 1024);
        b.off_b = off; off += align_up((size_t)b.Cb * b.s * b.s * 2, 1024);
        size_t off32 = 0;
        for (int i = 0; i < 2; ++i) { b.off32_x[i] = off32; off32 += align_up((size_t)b.Cf * b.e * 4, 1024); }
        b.off32_a = off32; off32 += align_up((size_t)b.Cf * b.s * b.s * 4, 1024);
        b.off32_b = off32; off32 += align_up((size_t)b.Cf * b.s * b.s * 4, 1024);
        b.data_bytes = std::max(off, off32);
        max_data = std::max(max_data, b.data_bytes);
    }
    plan.state_bytes = state_bytes;
    plan.slot_bytes = align_up(max_data, 1024);
    plan.workspace_bytes = WS_DATA_OFF + NSLOTS * plan.slot_bytes;
    return MONA_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 tensor [C][outer][inner] (inner contiguous) cut into boxes of 64 x box_rows with the 128-byte swizzle.
bool encode_map(EncodeTiledFn fn, CUtensorMap* map, void* base, int64_t inner, int64_t outer, int64_t C, int box_rows) {
    cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)outer, (cuuint64_t)C};
    cuuint64_t strides[2] = {(cuuint64_t)inner * 2, (cuuint64_t)inner * (cuuint64_t)outer * 2};
    cuuint32_t box[3] = {(cuuint32_t)TC_BOX, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

F2 split(double v) {
    F2 r;
    r.hi = (float)v;
    r.lo = (float)(v - (double)r.hi);
    return r;
}

}  // namespace

struct mona_handle {
    Plan plan;
    mona_options opt = {};      // as resolved at creation; later changes of the process-wide defaults do not reach the handle
    int device = 0, max_pairs = 0;
    uint8_t* state = nullptr;
    uint8_t* ws = nullptr;
    cudaStream_t side = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    // host-to-host pipeline of mona_step_host(): copy streams and per-descriptor events, created on first use
    cudaStream_t h2d = nullptr, d2h = nullptr;
    cudaEvent_t ev_hfork = nullptr, ev_hjoin = nullptr;
    std::vector<cudaEvent_t> ev_in;     // gradient of descriptor i has arrived on the device
    std::vector<cudaEvent_t> ev_out;    // 2 per descriptor: its chunks on slot stream 0 / 1 have been updated
    DeviceStatus* host_status = nullptr;   // pinned
    std::string last_error;
    int64_t launches = 0;
    double flops_exec = 0.0, flops_dense = 0.0, flops_useful = 0.0;

    mona_status fail(mona_status st, const char* fmt, ...) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof buf, fmt, ap);
        va_end(ap);
        last_error = buf;
        return st;
    }
};

#define MONA_CUDA(h, call)                                                                                 \
    do {                                                                                                   \
        cudaError_t e_ = (call);                                                                           \
        if (e_ != cudaSuccess) return (h)->fail(MONA_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_)); \
    } while (0)

extern "C" {

mona_status mona_default_hparams(mona_hparams* hp) {
    if (!hp) return MONA_ERR_INVALID_ARG;
    memset(hp, 0, sizeof *hp);
    hp->lr = 1e-3; hp->momentum = 0.95; hp->accel_beta = 0.99; hp->accel_alpha = -1.0 / (2.0 * (1.0 - 0.99));
    hp->weight_decay = 0.1; hp->ns_a = 3.4445; hp->ns_b = -4.7750; hp->ns_c = 2.0315; hp->norm_eps = 1e-7;
    hp->scale_value = 0.2; hp->ns_steps = 5; hp->scale_mode = 0; hp->ns_precision = 0;
    return MONA_OK;
}

mona_status mona_set_chunk_budget(size_t bytes) {
    if (bytes < (1u << 20)) return MONA_ERR_INVALID_ARG;
    g_chunk_budget_bytes.store(bytes);
    return MONA_OK;
}

mona_status mona_set_chunk_overlap(int enabled) {
    g_chunk_overlap.store(enabled ? 1 : 0);
    return MONA_OK;
}

mona_status mona_default_options(mona_options* opt) {
    if (!opt) return MONA_ERR_INVALID_ARG;
    memset(opt, 0, sizeof *opt);
    opt->chunk_budget_bytes = g_chunk_budget_bytes.load();
    opt->chunk_overlap = g_chunk_overlap.load();
    opt->fuse_update = 0;
    opt->ns_delay = 20;
    opt->macro_tile_min_k = 1;
    return MONA_OK;
}

}  // extern "C"

namespace {
// Options as the plan uses them: NULL means the defaults; a zero budget or delay means the default value.
mona_status resolve_options(const mona_options* in, mona_options& out) {
    mona_default_options(&out);
    if (!in) return MONA_OK;
    if (in->chunk_budget_bytes != 0) {
        if (in->chunk_budget_bytes < (1u << 20)) return MONA_ERR_INVALID_ARG;
        out.chunk_budget_bytes = in->chunk_budget_bytes;
    }
    out.chunk_overlap = in->chunk_overlap ? 1 : 0;
    out.fuse_update = in->fuse_update ? 1 : 0;
    if (in->ns_delay < 0 || in->ns_delay > 1024) return MONA_ERR_INVALID_ARG;
    if (in->ns_delay > 0) out.ns_delay = in->ns_delay;
    if (in->macro_tile_min_k < 0) return MONA_ERR_INVALID_ARG;
    if (in->macro_tile_min_k > 0) out.macro_tile_min_k = in->macro_tile_min_k;
    return MONA_OK;
}
}  // namespace

extern "C" {

mona_status mona_query_sizes_opt(const mona_matrix_desc* descs, int64_t n_desc, const mona_options* options,
                                 size_t* state_bytes, size_t* workspace_bytes) {
    mona_options opt;
    if (resolve_options(options, opt) != MONA_OK) return MONA_ERR_INVALID_ARG;
    Plan plan;
    std::string err;
    mona_status st = build_plan(descs, n_desc, opt.chunk_budget_bytes, plan, err);
    if (st != MONA_OK) return st;
    if (state_bytes) *state_bytes = plan.state_bytes;
    if (workspace_bytes) *workspace_bytes = plan.workspace_bytes;
    return MONA_OK;
}

mona_status mona_query_sizes(const mona_matrix_desc* descs, int64_t n_desc, size_t* state_bytes, size_t* workspace_bytes) {
    return mona_query_sizes_opt(descs, n_desc, nullptr, state_bytes, workspace_bytes);
}

mona_status mona_create(mona_handle** out, const mona_matrix_desc* descs, int64_t n_desc, void* state, size_t state_bytes,
                        void* workspace, size_t workspace_bytes, int device) {
    return mona_create_opt(out, descs, n_desc, nullptr, state, state_bytes, workspace, workspace_bytes, device);
}

mona_status mona_create_opt(mona_handle** out, const mona_matrix_desc* descs, int64_t n_desc, const mona_options* options,
                            void* state, size_t state_bytes, void* workspace, size_t workspace_bytes, int device) {
    if (!out) return MONA_ERR_INVALID_ARG;
    *out = nullptr;
    mona_handle* h = new mona_handle();
    *out = h;     // returned even on failure so that mona_last_error() can be read; destroy it either way
    if (resolve_options(options, h->opt) != MONA_OK)
        return h->fail(MONA_ERR_INVALID_ARG, "options: chunk_budget_bytes must be 0 or at least 1 MiB, ns_delay within 0..1024");
    mona_status st = build_plan(descs, n_desc, h->opt.chunk_budget_bytes, h->plan, h->last_error);
    if (st != MONA_OK) return st;
    if (!state || !workspace) return h->fail(MONA_ERR_INVALID_ARG, "state or workspace is null");
    if (((uintptr_t)state & 255) || ((uintptr_t)workspace & 255)) return h->fail(MONA_ERR_ALIGNMENT, "state/workspace must be 256-byte aligned");
    if (state_bytes < h->plan.state_bytes || workspace_bytes < h->plan.workspace_bytes)
        return h->fail(MONA_ERR_BUFFER_TOO_SMALL, "need state %zu B, workspace %zu B", h->plan.state_bytes, h->plan.workspace_bytes);
    int ndev = 0;
    cudaError_t ce = cudaGetDeviceCount(&ndev);
    if (ce != cudaSuccess || device < 0 || device >= ndev)
        return h->fail(MONA_ERR_CUDA, "no usable CUDA device %d (%s)", device, cudaGetErrorString(ce));
    MONA_CUDA(h, cudaSetDevice(device));
    cudaDeviceProp prop;
    MONA_CUDA(h, cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) return h->fail(MONA_ERR_ARCH, "device %d is sm_%d%d; this library is built for sm_100a only", device, prop.major, prop.minor);
    h->device = device;
    h->state = (uint8_t*)state;
    h->ws = (uint8_t*)workspace;

    EncodeTiledFn encode = nullptr;
    cudaDriverEntryPointQueryResult qres;
    MONA_CUDA(h, cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", (void**)&encode, cudaEnableDefault, &qres));
    if (!encode || qres != cudaDriverEntryPointSuccess) return h->fail(MONA_ERR_CUDA, "cuTensorMapEncodeTiled not available");
    for (Bucket& b : h->plan.buckets) {
        if (!b.tc_ok) continue;
        bool ok = true;
        for (int sl = 0; sl < NSLOTS; ++sl) {
            uint8_t* data = h->ws + WS_DATA_OFF + sl * h->plan.slot_bytes;
            for (int big = 0; big < 2; ++big) {     // 64-row boxes, then 128-row boxes
                const int rows = big ? 2 * TC_BOX : TC_BOX, at = big * NS_TENSORS;
                for (int i = 0; i < 2; ++i) ok = ok && encode_map(encode, &b.maps[sl].m[at + MAP_X0 + i], data + b.off_x[i], b.cols, b.rows, b.Cb, rows);
                ok = ok && encode_map(encode, &b.maps[sl].m[at + MAP_A], data + b.off_a, b.s, b.s, b.Cb, rows);
                ok = ok && encode_map(encode, &b.maps[sl].m[at + MAP_B], data + b.off_b, b.s, b.s, b.Cb, rows);
            }
        }
        if (!ok) return h->fail(MONA_ERR_CUDA, "cuTensorMapEncodeTiled failed for bucket %lldx%lld", (long long)b.rows, (long long)b.cols);
    }
    MONA_CUDA(h, ns_configure(&h->max_pairs));
    MONA_CUDA(h, small_ns_configure());
    MONA_CUDA(h, cudaStreamCreateWithFlags(&h->side, cudaStreamNonBlocking));
    MONA_CUDA(h, cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming));
    MONA_CUDA(h, cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming));
    MONA_CUDA(h, cudaMallocHost((void**)&h->host_status, sizeof(DeviceStatus)));
    // M_0 = A_0 = G_0 = 0; control block cleared
    MONA_CUDA(h, cudaMemset(h->state, 0, h->plan.state_bytes));
    MONA_CUDA(h, cudaMemset(h->ws, 0, WS_DATA_OFF));
    DeviceStatus init = {0u, INT_MAX, 0u, 0u};
    MONA_CUDA(h, cudaMemcpy(h->ws + WS_STATUS_OFF, &init, sizeof init, cudaMemcpyHostToDevice));
    MONA_CUDA(h, cudaDeviceSynchronize());
    return MONA_OK;
}

}  // extern "C"

// One optimizer step.  With `params_host` set (mona_step_host) every chunk first waits for the gradient copies of
// the descriptors it touches, and a descriptor whose last matrix has been updated is copied back right away
// on the handle's device-to-host stream, so transfers in both directions overlap the remaining chunks.
static mona_status step_impl(mona_handle* h, const mona_hparams* hp, void* const* params, const void* const* grads,
                             void* const* o_out, uint32_t phase_mask, void* stream_v, void* const* params_host) {
    if (!h) return MONA_ERR_INVALID_ARG;
    if (!hp || !params || !grads) return h->fail(MONA_ERR_INVALID_ARG, "hp, params or grads is null");
    if (hp->ns_steps < 0 || hp->ns_steps > 64) return h->fail(MONA_ERR_INVALID_ARG, "ns_steps out of range");
    if (hp->ns_precision != 0 && hp->ns_precision != 1) return h->fail(MONA_ERR_INVALID_ARG, "ns_precision must be 0 or 1");
    if (hp->scale_mode != 0 && hp->scale_mode != 1) return h->fail(MONA_ERR_INVALID_ARG, "scale_mode must be 0 or 1");
    if (hp->algorithm != 0 && hp->algorithm != 1) return h->fail(MONA_ERR_INVALID_ARG, "algorithm must be 0 (MONA) or 1 (Muon)");
    const Plan& plan = h->plan;
    const int64_t n_desc = (int64_t)plan.descs.size();
    for (int64_t i = 0; i < n_desc; ++i) {
        if (!params[i] || !grads[i]) return h->fail(MONA_ERR_INVALID_ARG, "params[%lld] or grads[%lld] is null", (long long)i, (long long)i);
        if (((uintptr_t)params[i] & 15) || ((uintptr_t)grads[i] & 15) || (o_out && o_out[i] && ((uintptr_t)o_out[i] & 15)))
            return h->fail(MONA_ERR_ALIGNMENT, "descriptor %lld: pointers must be 16-byte aligned", (long long)i);
    }
    MONA_CUDA(h, cudaSetDevice(h->device));
    NvtxRange step_range("mona_step");

    PrologueScalars ps;
    ps.beta = split(hp->accel_beta);
    ps.one_minus_beta = split(1.0 - hp->accel_beta);
    ps.alpha = split(hp->accel_alpha);
    ps.mu = split(hp->momentum);
    ps.eps = (float)hp->norm_eps;
    const float eta_lambda = (float)(hp->lr * hp->weight_decay);
    const int T = hp->ns_steps;
    const float ns_a = (float)hp->ns_a, ns_b = (float)hp->ns_b, ns_c = (float)hp->ns_c;

    DeviceStatus* dstatus = (DeviceStatus*)(h->ws + WS_STATUS_OFF);
    // chunks alternate between the caller's stream (slot 0) and the handle's own stream (slot 1)
    int64_t total_chunks = 0;
    for (const Bucket& b : plan.buckets) {
        const bool tcb = (hp->ns_precision == 0) && b.tc_ok && T >= 1;
        const int capb = tcb ? b.Cb : b.Cf;
        total_chunks += ((int64_t)b.mats.size() + capb - 1) / capb;
    }
    const bool overlap = h->opt.chunk_overlap && total_chunks > 1;
    cudaStream_t slot_stream[NSLOTS] = {(cudaStream_t)stream_v, overlap ? h->side : (cudaStream_t)stream_v};
    if (overlap) {
        MONA_CUDA(h, cudaEventRecord(h->ev_fork, slot_stream[0]));
        MONA_CUDA(h, cudaStreamWaitEvent(h->side, h->ev_fork, 0));
    }
    int64_t chunk_index = 0;
    std::vector<char> out_recorded(params_host ? 2 * plan.descs.size() : 0, 0);
    std::vector<int> chunk_descs;
    h->launches = 0;
    h->flops_exec = 0.0;
    h->flops_dense = 0.0;
    h->flops_useful = 0.0;

    for (const Bucket& b : plan.buckets) {
        const bool tc = (hp->ns_precision == 0) && b.tc_ok && T >= 1;
        const int cap = tc ? b.Cb : b.Cf;
        const int64_t count = (int64_t)b.mats.size();
        const double gamma = hp->scale_mode == 0 ? hp->scale_value * std::sqrt((double)b.l) : hp->scale_value;
        const float eta_gamma = (float)(hp->lr * gamma);
        const size_t gsz = b.grad_dtype == MONA_BF16 ? 2 : 4;
        const size_t aux = b.state_dtype == MONA_BF16 ? 2 : 4;
        float* Mst = (float*)(h->state + b.off_M);

        for (int64_t start = 0; start < count; start += cap) {
            const int C = (int)std::min<int64_t>(cap, count - start);
            ChunkPtrs ptrs;
            bool vec4 = (b.e % 4 == 0);
            chunk_descs.clear();
            for (int c = 0; c < C; ++c) {
                const MatRef& mr = b.mats[start + c];
                const mona_matrix_desc& d = plan.descs[mr.desc];
                if (chunk_descs.empty() || chunk_descs.back() != mr.desc) chunk_descs.push_back(mr.desc);
                if ((d.batch_stride * (int64_t)gsz) % 16 != 0 || (d.batch_stride * 4) % 16 != 0) vec4 = false;
                ptrs.g[c] = (const uint8_t*)grads[mr.desc] + (size_t)mr.b * d.batch_stride * gsz;
                ptrs.w[c] = (float*)params[mr.desc] + mr.b * d.batch_stride;
                ptrs.o[c] = (o_out && o_out[mr.desc]) ? (float*)o_out[mr.desc] + mr.b * d.batch_stride : nullptr;
                ptrs.gid[c] = (int)(plan.desc_first_gid[mr.desc] + mr.b);
            }
            const int slot = overlap ? (int)(chunk_index % NSLOTS) : 0;
            ++chunk_index;
            cudaStream_t stream = slot_stream[slot];
            uint8_t* ctrl = h->ws + WS_CTRL_OFF + slot * WS_CTRL_BYTES;
            uint8_t* data = h->ws + WS_DATA_OFF + slot * plan.slot_bytes;
            unsigned int* counters = (unsigned int*)(ctrl + CTRL_COUNTERS_OFF);
            float* inv_norm = (float*)(ctrl + CTRL_INVNORM_OFF);
            float* partials = (float*)(ctrl + CTRL_PARTIALS_OFF);
            float* Mc = Mst + start * b.e;
            void* Ac = h->state + b.off_A + (size_t)start * b.e * aux;
            void* Gc = h->state + b.off_G + (size_t)start * b.e * aux;
            __nv_bfloat16* xb[2] = {(__nv_bfloat16*)(data + b.off_x[0]), (__nv_bfloat16*)(data + b.off_x[1])};
            __nv_bfloat16* ab = (__nv_bfloat16*)(data + b.off_a);
            float* xf[2] = {(float*)(data + b.off32_x[0]), (float*)(data + b.off32_x[1])};
            float* af = (float*)(data + b.off32_a);
            float* bf = (float*)(data + b.off32_b);

            if (params_host)
                for (int dsc : chunk_descs) MONA_CUDA(h, cudaStreamWaitEvent(stream, h->ev_in[dsc], 0));
            if (phase_mask & 1u) {
                NvtxRange range("mona.prologue");
                MONA_CUDA(h, launch_prologue(ptrs, C, b.grad_dtype == MONA_BF16,
                                             hp->algorithm == 1 ? PROLOGUE_NO_AUX : (b.state_dtype == MONA_BF16 ? PROLOGUE_AUX_BF16 :
                                                 b.state_dtype == MONA_STATE_COMBINED ? PROLOGUE_AUX_COMBINED : PROLOGUE_AUX_F32), vec4, Mc, Ac, Gc, tc ? xb[0] : nullptr, partials,
                                             counters, inv_norm, dstatus, b.e, b.slab_len, b.slabs, ps, stream));
                ++h->launches;
            }
            const void* o_final = nullptr;
            bool update_fused = false;
            if (tc) {
                if (phase_mask & 2u) {
                    NvtxRange range("mona.newton_schulz");
                    // the last X' = B' X applies the parameter update in its epilogue when this call runs both phases and the
                    // fp32 rows can be accessed 32 bytes at a time
                    update_fused = h->opt.fuse_update && (phase_mask & 4u) != 0u;
                    for (int c = 0; c < C && update_fused; ++c)
                        if (((uintptr_t)ptrs.w[c] & 31) || ((uintptr_t)ptrs.o[c] & 31)) update_fused = false;
                    unsigned int* sched = (unsigned int*)(ctrl + CTRL_SCHED_OFF);
                    for (int t0 = 0; t0 < T; t0 += NS_MAX_PHASES / 3) {
                        const int t1 = std::min(T, t0 + NS_MAX_PHASES / 3);
                        NsProgram g{};
                        g.C = C; g.P = 3 * (t1 - t0); g.delay = h->opt.ns_delay;
                        g.inv_norm = inv_norm; g.work_counter = sched; g.done = sched + 64;
                        g.eta_lambda = eta_lambda; g.eta_gamma = eta_gamma;
                        for (int t = t0; t < t1; ++t) {
                            const int cur = t & 1, nxt = cur ^ 1;
                            NsPhase& g1 = g.ph[3 * (t - t0)];      // A = X X^T (wide) or X^T X (tall): lower-triangle tiles only
                            g1.M = g1.N = (int)b.s; g1.K = (int)b.l; g1.a_map = g1.b_map = MAP_X0 + cur; g1.a_mn = g1.b_mn = b.tall ? 1 : 0;
                            g1.symmetric = 1; g1.ab_same = 1; g1.d_map = MAP_A; g1.ld = b.s; g1.mat_stride = b.s * b.s;
                            g1.c1 = 0.f; g1.c2 = 1.f; g1.post_mode = t == 0 ? 2 : 0;
                            ns_phase_plan(g1);
                            NsPhase& g2 = g.ph[3 * (t - t0) + 1];  // B' = b A + c A A + a I, operands and result lower-block-stored
                            g2.M = g2.N = g2.K = (int)b.s; g2.a_map = g2.b_map = MAP_A; g2.a_sym = g2.b_sym = 1; g2.symmetric = 1; g2.ab_same = 1;
                            g2.cin = ab; g2.d_map = MAP_B; g2.ld = b.s; g2.mat_stride = b.s * b.s; g2.c1 = ns_b; g2.c2 = ns_c; g2.diag_add = ns_a;
                            ns_phase_plan(g2);
                            NsPhase& g3 = g.ph[3 * (t - t0) + 2];  // X' = B' X (wide) or X B' (tall); 256 x 512 macro-tiles when the inner dimension is long
                            g3.K = (int)b.s; g3.wide = b.s >= h->opt.macro_tile_min_k ? 1 : 0; g3.d_map = MAP_X0 + nxt; g3.ld = b.cols; g3.mat_stride = b.e;
                            g3.c1 = 0.f; g3.c2 = 1.f; g3.post_mode = t == 0 ? 1 : 0;
                            g3.fuse_update = (update_fused && t == T - 1) ? 1 : 0;
                            if (!b.tall) {   // B' is the symmetric "A" operand, X the MN-major "B" operand
                                g3.M = (int)b.s; g3.N = (int)b.l; g3.a_map = MAP_B; g3.a_sym = 1; g3.b_map = MAP_X0 + cur; g3.b_mn = 1;
                            } else {         // X is K-major, the symmetric B' serves as its own transpose
                                g3.M = (int)b.l; g3.N = (int)b.s; g3.a_map = MAP_X0 + cur; g3.a_mn = 0; g3.b_map = MAP_B; g3.b_sym = 1;
                            }
                            ns_phase_plan(g3);
                            h->flops_exec += (double)C * (ns_phase_executed_flops(g1) + ns_phase_executed_flops(g2) + ns_phase_executed_flops(g3));
                            h->flops_dense += (double)C * (4.0 * b.s * b.s * b.l + 2.0 * (double)b.s * b.s * b.s);
                            h->flops_useful += (double)C * (3.0 * b.s * b.s * b.l + (double)b.s * b.s * b.s);
                        }
                        ns_program_plan(g);
                        MONA_CUDA(h, cudaMemsetAsync(sched, 0, sizeof(unsigned int) * ns_sched_words(C, g.P), stream));
                        NsUpdatePtrs up{};
                        if (update_fused && t1 == T) { up.w = ptrs.w; up.o = ptrs.o; }
                        MONA_CUDA(h, launch_ns_program(b.maps[slot], g, up, h->max_pairs, dstatus, stream));
                        ++h->launches;
                    }
                }
                o_final = xb[T & 1];
            } else if (small_ns_eligible(b.rows, b.cols)) {
                // short side <= 64 (routers): the whole iteration in one launch, one block per matrix
                if (phase_mask & 2u) {
                    NvtxRange range("mona.newton_schulz.small");
                    MONA_CUDA(h, launch_small_ns(Mc, xf[0], inv_norm, C, (int)b.rows, (int)b.cols, T, ns_a, ns_b, ns_c, stream));
                    ++h->launches;
                    h->flops_dense += (double)T * C * (4.0 * b.s * b.s * b.l + 2.0 * (double)b.s * b.s * b.s);
                }
                o_final = xf[0];
            } else {
                if (phase_mask & 2u) {
                    NvtxRange range("mona.newton_schulz.fp32");
                    MONA_CUDA(h, launch_scale(Mc, xf[0], inv_norm, C, b.e, b.slab_len, b.slabs, stream));
                    ++h->launches;
                    for (int t = 0; t < T; ++t) {
                        const int cur = t & 1, nxt = cur ^ 1;
                        SgemmArgs g1{};   // A = X X^T (wide) or X^T X (tall), s x s
                        g1.a = xf[cur]; g1.b = xf[cur]; g1.a_batch = g1.b_batch = b.e;
                        if (!b.tall) { g1.a_si = b.cols; g1.a_sk = 1; g1.b_sk = 1; g1.b_sj = b.cols; }
                        else         { g1.a_si = 1; g1.a_sk = b.cols; g1.b_sk = b.cols; g1.b_sj = 1; }
                        g1.cin = nullptr; g1.d = af; g1.ldd = b.s; g1.d_batch = b.s * b.s;
                        g1.M = g1.N = (int)b.s; g1.K = (int)b.l; g1.batch = C; g1.c1 = 0.f; g1.c2 = 1.f;
                        MONA_CUDA(h, launch_sgemm(g1, stream));
                        SgemmArgs g2{};   // B = b A + c A A
                        g2.a = af; g2.b = af; g2.a_batch = g2.b_batch = b.s * b.s;
                        g2.a_si = b.s; g2.a_sk = 1; g2.b_sk = b.s; g2.b_sj = 1;
                        g2.cin = af; g2.d = bf; g2.ldd = b.s; g2.d_batch = b.s * b.s;
                        g2.M = g2.N = g2.K = (int)b.s; g2.batch = C; g2.c1 = ns_b; g2.c2 = ns_c;
                        MONA_CUDA(h, launch_sgemm(g2, stream));
                        SgemmArgs g3{};   // X' = a X + B X (wide) or a X + X B (tall)
                        if (!b.tall) {
                            g3.a = bf; g3.a_si = b.s; g3.a_sk = 1; g3.a_batch = b.s * b.s;
                            g3.b = xf[cur]; g3.b_sk = b.cols; g3.b_sj = 1; g3.b_batch = b.e;
                            g3.M = (int)b.s; g3.N = (int)b.l;
                        } else {
                            g3.a = xf[cur]; g3.a_si = b.cols; g3.a_sk = 1; g3.a_batch = b.e;
                            g3.b = bf; g3.b_sk = b.s; g3.b_sj = 1; g3.b_batch = b.s * b.s;
                            g3.M = (int)b.l; g3.N = (int)b.s;
                        }
                        g3.K = (int)b.s; g3.cin = xf[cur]; g3.d = xf[nxt]; g3.ldd = b.cols; g3.d_batch = b.e;
                        g3.batch = C; g3.c1 = ns_a; g3.c2 = 1.f;
                        MONA_CUDA(h, launch_sgemm(g3, stream));
                        h->launches += 3;
                        h->flops_dense += (double)C * (4.0 * b.s * b.s * b.l + 2.0 * (double)b.s * b.s * b.s);
                    }
                }
                o_final = xf[T & 1];
            }
            if ((phase_mask & 4u) && !update_fused) {
                NvtxRange range("mona.update");
                MONA_CUDA(h, launch_update(ptrs, C, tc, vec4, o_final, b.e, b.slab_len, b.slabs, eta_lambda, eta_gamma, stream));
                ++h->launches;
            }
            if (params_host) {
                for (int dsc : chunk_descs) {
                    MONA_CUDA(h, cudaEventRecord(h->ev_out[2 * dsc + slot], stream));
                    out_recorded[2 * dsc + slot] = 1;
                }
                const MatRef& last = b.mats[start + C - 1];
                for (int dsc : chunk_descs) {
                    const mona_matrix_desc& d = plan.descs[dsc];
                    if (dsc == last.desc && last.b != d.batch - 1) continue;    // descriptor continues in the next chunk
                    for (int sl = 0; sl < NSLOTS; ++sl)
                        if (out_recorded[2 * dsc + sl]) MONA_CUDA(h, cudaStreamWaitEvent(h->d2h, h->ev_out[2 * dsc + sl], 0));
                    const size_t bytes = (size_t)((d.batch - 1) * d.batch_stride + d.rows * d.cols) * 4;
                    MONA_CUDA(h, cudaMemcpyAsync(params_host[dsc], params[dsc], bytes, cudaMemcpyDeviceToHost, h->d2h));
                }
            }
        }
    }
    if (overlap) {
        MONA_CUDA(h, cudaEventRecord(h->ev_join, h->side));
        MONA_CUDA(h, cudaStreamWaitEvent(slot_stream[0], h->ev_join, 0));
    }
    return MONA_OK;
}

extern "C" {

mona_status mona_step_ex(mona_handle* h, const mona_hparams* hp, void* const* params, const void* const* grads,
                         void* const* o_out, uint32_t phase_mask, void* stream_v) {
    return step_impl(h, hp, params, grads, o_out, phase_mask, stream_v, nullptr);
}

mona_status mona_step(mona_handle* h, const mona_hparams* hp, void* const* params, const void* const* grads, void* stream) {
    return step_impl(h, hp, params, grads, nullptr, 7u, stream, nullptr);
}

mona_status mona_step_host(mona_handle* h, const mona_hparams* hp, void* const* params, void* const* grads,
                           const void* const* grads_host, void* const* params_host, void* stream_v) {
    if (!h) return MONA_ERR_INVALID_ARG;
    if (!params || !grads || !grads_host || !params_host) return h->fail(MONA_ERR_INVALID_ARG, "null pointer array");
    cudaStream_t stream = (cudaStream_t)stream_v;
    MONA_CUDA(h, cudaSetDevice(h->device));
    const int64_t n_desc = (int64_t)h->plan.descs.size();
    for (int64_t i = 0; i < n_desc; ++i)
        if (!grads_host[i] || !grads[i] || !params_host[i] || !params[i])
            return h->fail(MONA_ERR_INVALID_ARG, "descriptor %lld: a gradient or parameter pointer (host or device) is null", (long long)i);
    if (!h->h2d) {
        MONA_CUDA(h, cudaStreamCreateWithFlags(&h->h2d, cudaStreamNonBlocking));
        MONA_CUDA(h, cudaStreamCreateWithFlags(&h->d2h, cudaStreamNonBlocking));
        MONA_CUDA(h, cudaEventCreateWithFlags(&h->ev_hfork, cudaEventDisableTiming));
        MONA_CUDA(h, cudaEventCreateWithFlags(&h->ev_hjoin, cudaEventDisableTiming));
        h->ev_in.assign((size_t)n_desc, nullptr);
        h->ev_out.assign((size_t)(2 * n_desc), nullptr);
        for (auto& e : h->ev_in) MONA_CUDA(h, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        for (auto& e : h->ev_out) MONA_CUDA(h, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    }
    // both copy streams start after whatever the caller's stream holds so far
    MONA_CUDA(h, cudaEventRecord(h->ev_hfork, stream));
    MONA_CUDA(h, cudaStreamWaitEvent(h->h2d, h->ev_hfork, 0));
    MONA_CUDA(h, cudaStreamWaitEvent(h->d2h, h->ev_hfork, 0));
    // gradients travel in the order in which the chunks will want them: bucket by bucket, descriptor by descriptor
    for (const Bucket& b : h->plan.buckets) {
        int prev = -1;
        for (const MatRef& mr : b.mats) {
            if (mr.desc == prev) continue;
            prev = mr.desc;
            const mona_matrix_desc& d = h->plan.descs[mr.desc];
            const size_t bytes = (size_t)((d.batch - 1) * d.batch_stride + d.rows * d.cols) * (d.grad_dtype == MONA_BF16 ? 2 : 4);
            MONA_CUDA(h, cudaMemcpyAsync(grads[mr.desc], grads_host[mr.desc], bytes, cudaMemcpyHostToDevice, h->h2d));
            MONA_CUDA(h, cudaEventRecord(h->ev_in[mr.desc], h->h2d));
        }
    }
    mona_status st = step_impl(h, hp, params, (const void* const*)grads, nullptr, 7u, stream_v, params_host);
    // join the copy streams back into the caller's stream whether or not the step was enqueued completely
    const std::string step_error = h->last_error;
    MONA_CUDA(h, cudaEventRecord(h->ev_hjoin, h->h2d));
    MONA_CUDA(h, cudaStreamWaitEvent(stream, h->ev_hjoin, 0));
    MONA_CUDA(h, cudaEventRecord(h->ev_hjoin, h->d2h));
    MONA_CUDA(h, cudaStreamWaitEvent(stream, h->ev_hjoin, 0));
    if (st != MONA_OK) h->last_error = step_error;
    return st;
}

mona_status mona_selftest_timeout(mona_handle* h, void* stream_v) {
    if (!h) return MONA_ERR_INVALID_ARG;
    MONA_CUDA(h, cudaSetDevice(h->device));
    for (const Bucket& b : h->plan.buckets) {
        if (!b.tc_ok) continue;
        // one X X^T phase over the first matrix slot of the workspace whose stages expect 16 bytes too many
        uint8_t* ctrl = h->ws + WS_CTRL_OFF;
        unsigned int* sched = (unsigned int*)(ctrl + CTRL_SCHED_OFF);
        NsProgram g{};
        g.C = 1; g.P = 1; g.delay = 1; g.inv_norm = (const float*)(ctrl + CTRL_INVNORM_OFF); g.work_counter = sched; g.done = sched + 64;
        g.selftest_extra_tx = 16;
        NsPhase& p = g.ph[0];
        p.M = p.N = (int)b.s; p.K = (int)b.l; p.a_map = p.b_map = MAP_X0; p.a_mn = p.b_mn = b.tall ? 1 : 0; p.symmetric = 1; p.ab_same = 1;
        p.d_map = MAP_A; p.ld = b.s; p.mat_stride = b.s * b.s; p.c1 = 0.f; p.c2 = 1.f;
        ns_phase_plan(p);
        ns_program_plan(g);
        MONA_CUDA(h, cudaMemsetAsync(sched, 0, sizeof(unsigned int) * ns_sched_words(1, 1), (cudaStream_t)stream_v));
        MONA_CUDA(h, launch_ns_program(b.maps[0], g, NsUpdatePtrs{}, h->max_pairs, (DeviceStatus*)(h->ws + WS_STATUS_OFF), (cudaStream_t)stream_v));
        return MONA_OK;
    }
    return h->fail(MONA_ERR_UNSUPPORTED_SHAPE, "no descriptor of this handle takes the tensor-core path");
}

mona_status mona_poll_status(mona_handle* h, void* stream_v, int64_t* first_bad_matrix) {
    if (!h) return MONA_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)stream_v;
    MONA_CUDA(h, cudaSetDevice(h->device));
    MONA_CUDA(h, cudaMemcpyAsync(h->host_status, h->ws + WS_STATUS_OFF, sizeof(DeviceStatus), cudaMemcpyDeviceToHost, stream));
    static const DeviceStatus cleared = {0u, INT_MAX, 0u, 0u};
    MONA_CUDA(h, cudaMemcpyAsync(h->ws + WS_STATUS_OFF, &cleared, sizeof cleared, cudaMemcpyHostToDevice, stream));
    MONA_CUDA(h, cudaStreamSynchronize(stream));
    const DeviceStatus s = *h->host_status;
    if (first_bad_matrix) *first_bad_matrix = (s.first_bad == INT_MAX) ? -1 : s.first_bad;
    if (s.flags & STATUS_BOUNDS) return h->fail(MONA_ERR_BOUNDS, "an index check of the debug build failed (site %u)", s.timeout_site);
    if (s.flags & STATUS_TIMEOUT) return h->fail(MONA_ERR_TIMEOUT, "a device-side wait ran out (site %u)", s.timeout_site);
    if (s.flags & STATUS_NONFINITE) return h->fail(MONA_ERR_NONFINITE, "non-finite ||M||_F, first at matrix %d", s.first_bad);
    return MONA_OK;
}

mona_status mona_state_layout(const mona_handle* h, int64_t desc, size_t* off_M, size_t* off_A, size_t* off_Gprev) {
    if (!h || desc < 0 || desc >= (int64_t)h->plan.descs.size()) return MONA_ERR_INVALID_ARG;
    const Bucket& b = h->plan.buckets[h->plan.desc_bucket[desc]];
    const size_t aux = b.state_dtype == MONA_BF16 ? 2 : 4;
    const size_t pos = (size_t)h->plan.desc_pos[desc] * (size_t)b.e;
    if (off_M) *off_M = b.off_M + pos * 4;
    if (off_A) *off_A = b.off_A + pos * aux;
    if (off_Gprev) *off_Gprev = b.state_dtype == MONA_STATE_COMBINED ? (size_t)-1 : b.off_G + pos * aux;
    return MONA_OK;
}

int64_t mona_last_launch_count(const mona_handle* h) { return h ? h->launches : 0; }

mona_status mona_last_ns_flops(const mona_handle* h, double* executed, double* dense_equivalent) {
    if (!h) return MONA_ERR_INVALID_ARG;
    if (executed) *executed = h->flops_exec;
    if (dense_equivalent) *dense_equivalent = h->flops_dense;
    return MONA_OK;
}

mona_status mona_last_ns_useful_flops(const mona_handle* h, double* useful) {
    if (!h || !useful) return MONA_ERR_INVALID_ARG;
    *useful = h->flops_useful;
    return MONA_OK;
}

static_assert(MONA_TRACE_ROWS == mona::NS_TRACE_ROWS && MONA_TRACE_SLOTS == mona::NS_TRACE_SLOTS &&
              (int)MONA_TRACE_TILE0 == (int)mona::NS_TRACE_TILE0 && (int)MONA_TRACE_EPI_TILE0 == (int)mona::NS_TRACE_EPI_TILE0 && (int)MONA_TRACE_ITEMS == (int)mona::NS_TRACE_ITEMS &&
              (int)MONA_TRACE_EPI_ROLE == (int)mona::NS_TRACE_EPI_ROLE && (int)MONA_TRACE_SCHED_ROLE == (int)mona::NS_TRACE_SCHED_ROLE,
              "the public description of the profiling table follows the kernel's");

mona_status mona_work_order(int32_t n_matrices, int32_t n_phases, int32_t delay, const uint32_t* items_per_phase,
                            uint32_t start, uint32_t stride, int32_t* out_cqt, size_t capacity, size_t* n_written) {
    if (!n_written) return MONA_ERR_INVALID_ARG;
    const int n = mona::ns_work_order(n_matrices, n_phases, delay, items_per_phase, start, stride, out_cqt, capacity);
    if (n < 0) return MONA_ERR_INVALID_ARG;
    *n_written = (size_t)n;
    return MONA_OK;
}

mona_status mona_trace_read(unsigned long long* out, size_t rows, int reset) {
    if (rows && !out) return MONA_ERR_INVALID_ARG;
    int available = 0;
    const cudaError_t e = mona::ns_trace_read(out, rows, reset, &available);
    if (!available) return MONA_ERR_NOT_BUILT;
    return e == cudaSuccess ? MONA_OK : MONA_ERR_CUDA;
}

const char* mona_last_error(const mona_handle* h) { return h ? h->last_error.c_str() : "null handle"; }

void mona_destroy(mona_handle* h) {
    if (!h) return;
    if (h->side) cudaStreamDestroy(h->side);
    if (h->ev_fork) cudaEventDestroy(h->ev_fork);
    if (h->h2d) cudaStreamDestroy(h->h2d);
    if (h->d2h) cudaStreamDestroy(h->d2h);
    if (h->ev_hfork) cudaEventDestroy(h->ev_hfork);
    if (h->ev_hjoin) cudaEventDestroy(h->ev_hjoin);
    for (cudaEvent_t e : h->ev_in) if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : h->ev_out) if (e) cudaEventDestroy(e);
    if (h->ev_join) cudaEventDestroy(h->ev_join);
    if (h->host_status) cudaFreeHost(h->host_status);
    delete h;
}

}  // extern "C"
