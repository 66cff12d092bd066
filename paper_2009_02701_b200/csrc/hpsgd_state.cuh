// Internal state of libhpsgd: the singleton context, arena plan, index ranges of the
// schedule, grids, profiling events and the small helpers every entry point uses.
// Included by hpsgd_api.cu only (one translation unit).
#pragma once

#include "../../include/hpsgd.h"

#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <vector>

#include "hpsgd_kernels.cuh"
#include "hpsgd_staged.cuh"

namespace {

using namespace hpsgd;

constexpr int64_t kAlignElems = 32;        // tensor starts: multiples of 32 elements
constexpr int64_t kRowAlignElems = 1024;   // w, D and the rows of r / m start on 4 KB boundaries: the 4 KB
                                           // tile a block touches in each array then never straddles one
                                           // (measured +1.2-1.6 % on the merge over 256-byte alignment)
constexpr size_t kAlignBytes = 256;        // what a lent arena must be aligned to
constexpr size_t kPageBytes = 4096;        // what the regions inside it are aligned to
constexpr int kMaxChunks = 1024;
constexpr int kMaxTensors = 4096;
constexpr int64_t kChunkGrain = 1024;      // chunk boundaries: multiples of 1024 groups (8192 elements)
constexpr int kMaxGridX = 0x7FFFFFFF;

char g_err[512] = "";

int fail(int code, const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
    return code;
}

// A failed call is reported once: cudaGetLastError also clears a non-sticky error, so that the
// next, valid call is not blamed for it.
#define CUDA_TRY(expr)                                                                      \
    do {                                                                                    \
        cudaError_t e_ = (expr);                                                            \
        if (e_ != cudaSuccess) {                                                            \
            cudaGetLastError();                                                             \
            return fail(HPSGD_E_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e_));      \
        }                                                                                   \
    } while (0)

#define TRY(expr)                \
    do {                         \
        int rc_ = (expr);        \
        if (rc_) return rc_;     \
    } while (0)

size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct EventPair {
    cudaEvent_t a, b;
    int kind;       // HPSGD_KERNEL_*
};

struct Pending {                // configuration collected before hpsgd_init
    std::vector<int64_t> sizes;
    void* arena = nullptr;
    size_t arena_bytes = 0;
    cudaStream_t main = nullptr, side = nullptr;
    bool have_streams = false;
    int form = HPSGD_FORM_REPLICA_CHANGE;
    int pipeline = 0;
} g_pending;

struct Ctx {
    bool inited = false;
    int64_t P = 0, P_pad = 0, stride = 0;  // stride: floats between consecutive workers' rows
    int K = 0;
    float lr = 0.f, beta = 0.f, lambda = 0.f;
    uint64_t seed = 0, key = 0;
    int staleness = 1, grad_dtype = HPSGD_F32, overlap = 1, chunks = 1, profile = 0;
    std::vector<int64_t> sizes, offsets, starts;
    int64_t* d_table = nullptr;            // offsets | starts | sizes, on the device
    char* arena = nullptr;
    size_t arena_bytes = 0;
    bool own_arena = false;
    float *w = nullptr, *D = nullptr, *r = nullptr, *m = nullptr;
    int32_t* slot = nullptr;               // [K][slot_cap] row -> slot scratch map
    int64_t slot_cap = 0;
    bool own_slot = false;
    cudaStream_t main = nullptr, side = nullptr, copy = nullptr, d2h = nullptr;
    cudaEvent_t ev_w_ready = nullptr, ev_d2h_done = nullptr;   // hpsgd_copy_global_async
    bool d2h_outstanding = false;
    bool own_streams = false;
    std::vector<cudaEvent_t> ev_local, ev_merge;
    std::vector<char> local_recorded, merge_unwaited;
    bool D_valid = false;
    int64_t merges = 0;
    int form = HPSGD_FORM_REPLICA_CHANGE;  // what the workers carry: replica change or accumulated gradients
    int fuse = 0;                          // carry a merge into the next batched local step
    int staging = 0;                       // merges bring their tiles through shared memory with bulk-async copies
    bool staged_ran = false;               //   ... one has been launched since the last look at its time-out count
    bool staged_attr = false;              //   ... its shared-memory size has been opted into on this device
    int pipeline = 0;                      // commit/reduce split on double-buffered replicas
    float* wbuf[2] = {nullptr, nullptr};   // pipeline: global model of the current / other period
    float* rbuf[2] = {nullptr, nullptr};   // pipeline: replica sets of the current / other period
    int cur = 0;                           // pipeline: which buffers the current period trains on
    std::vector<char> touched;             // pipeline: worker has made a local step this period
    cudaEvent_t ev_commit = nullptr, ev_reduce = nullptr;
    bool reduce_outstanding = false;
    bool merge_deferred = false;           // fuse 1: hpsgd_sync_merge was called but its merge not yet enqueued
    int deferred_flags = 0;
    int steps_held = 0;                    // fuse 2: local steps held back for the merge they will run with
    std::vector<char> step_held;           //         which workers have one (at most one each)
    BatchPtrs deferred_gp{};               //         their gradient pointers, indexed by worker
    bool deferred_sparse = false;          //         all of them sparse-row steps, or none
    std::vector<char> at_w;                // replica i equals w: no local step since its last clone
    std::vector<char> row_valid;           // row i of r holds replica i (else it is a lazy clone: read w)
    int64_t launches = 0;
    int sm_count = 148;
    int sp_tensor = -1;                    // sparse-row tensor
    int64_t sp_rows = 0, sp_cols = 0;
    void* stage[2] = {nullptr, nullptr};   // staging of hpsgd_local_step_host
    cudaEvent_t stage_copied[2] = {nullptr, nullptr}, stage_free[2] = {nullptr, nullptr};
    bool stage_used[2] = {false, false};
    int stage_next = 0;
    std::vector<EventPair> prof;           // profiling
    double prof_ms[5] = {0, 0, 0, 0, 0};
    int64_t prof_launches[5] = {0, 0, 0, 0, 0};
    bool debug_stage_stall = false;        // checked build: the staged merge's barrier expects bytes that never arrive
    int64_t debug_limit = -1;              // checked build: groups per flat buffer the kernels test against (< 0: P_pad / 8)
} g;

int check_async()
{
    cudaError_t e = cudaGetLastError();     // reported once, then cleared (a sticky error comes back by itself)
    if (e != cudaSuccess) return fail(HPSGD_E_CUDA, "CUDA error: %s", cudaGetErrorString(e));
    return HPSGD_OK;
}

// Groups of 8 elements in a flat buffer: what the guards of the checked build test against.
int64_t group_limit() { return g.debug_limit >= 0 ? g.debug_limit : g.P_pad / 8; }

// Checked build: fetch and clear the record a kernel guard left behind.  Called where the host
// has just waited for the device, so the copy costs nothing extra.
int debug_poll()
{
#ifdef HPSGD_DEBUG
    DebugReport rep{};
    CUDA_TRY(cudaMemcpyFromSymbol(&rep, g_debug_report, sizeof rep));
    if (rep.code != 0) {
        const DebugReport zero{};
        CUDA_TRY(cudaMemcpyToSymbol(g_debug_report, &zero, sizeof zero));
        static const char* what[] = {"", "group index", "row -> slot entry", "row index"};
        return fail(HPSGD_E_CUDA, "checked build: kernel %d met %s %lld outside [0, %lld); the access was skipped",
                    rep.kernel, what[rep.code < 4 ? rep.code : 0], rep.index, rep.limit);
    }
#endif
    return HPSGD_OK;
}

// The staged merge waits (bounded) for its own bulk loads; blocks whose wait ran out counted
// themselves.  Called where the host has just waited for the device.
int staged_poll()
{
    if (!g.staged_ran) return HPSGD_OK;
    g.staged_ran = false;
    unsigned int n = 0;
    CUDA_TRY(cudaMemcpyFromSymbol(&n, g_stage_timeouts, sizeof n));
    if (n != 0) {
        const unsigned int zero = 0;
        CUDA_TRY(cudaMemcpyToSymbol(g_stage_timeouts, &zero, sizeof zero));
        return fail(HPSGD_E_TIMEOUT, "staged merge: %u blocks gave up waiting for their bulk loads after one second and wrote nothing; "
                                     "the state is no longer consistent", n);
    }
    return HPSGD_OK;
}

int64_t layout_of(const std::vector<int64_t>& sizes, std::vector<int64_t>* offsets, std::vector<int64_t>* starts)
{
    int64_t pos = 0, flat = 0;
    for (int64_t s : sizes) {
        if (offsets) offsets->push_back(pos);
        if (starts) starts->push_back(flat);
        pos += (s + kAlignElems - 1) / kAlignElems * kAlignElems;
        flat += s;
    }
    return pos;
}

// Regions of the arena, in order: w | D | r[K] | m[K] | w2 | r2[K] | table | slot maps (the rest).
struct ArenaPlan {
    size_t w, D, r, m, w2, r2, table, slot, fixed;
};

ArenaPlan plan_arena(int64_t stride, int K, bool momentum, bool pipeline)
{
    ArenaPlan a{};
    const size_t row = (size_t)stride * 4;
    size_t pos = 0;
    a.w = pos; pos += row;
    a.D = pos; pos += row;
    a.r = pos; pos += row * K;
    a.m = pos; if (momentum) pos += row * K;
    a.w2 = pos; if (pipeline) pos += row;
    a.r2 = pos; if (pipeline) pos += row * K;
    a.table = pos; pos += round_up((size_t)kMaxTensors * 3 * 8, kPageBytes);
    a.slot = pos;
    a.fixed = pos;
    return a;
}

// Index range [o_lo, o_hi), in 8-element groups, of schedule chunk c.
void chunk_range(int c, int64_t* o_lo, int64_t* o_hi)
{
    const int64_t n = g.P_pad / 8;
    const int64_t grains = (n + kChunkGrain - 1) / kChunkGrain;
    auto edge = [&](int k) { return std::min(n, grains * k / g.chunks * kChunkGrain); };
    *o_lo = edge(c);
    *o_hi = (c == g.chunks - 1) ? n : edge(c + 1);
}

// Grid of the hot kernels: one block per kHotThreads groups.
int hot_grid(int64_t groups)
{
    return (int)std::min<int64_t>(kMaxGridX, std::max<int64_t>(1, (groups + kHotThreads - 1) / kHotThreads));
}

// Grid of the support kernels: enough blocks to cover `items`, capped at one full wave of
// resident blocks (SM count x blocks the kernel can keep resident per SM).
template <typename Kern>
int grid_for(Kern kern, int64_t items, int64_t per_block)
{
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, kThreads, 0) != cudaSuccess || occ < 1) occ = 1;
    const int64_t need = std::max<int64_t>(1, (items + per_block - 1) / per_block);
    return (int)std::min<int64_t>(need, (int64_t)g.sm_count * occ);
}

// ---------------------------------------------------------------------------- profiling
int prof_begin(cudaStream_t s, int kind, EventPair* ep)
{
    if (!g.profile) return HPSGD_OK;
    ep->kind = kind;
    CUDA_TRY(cudaEventCreate(&ep->a));
    CUDA_TRY(cudaEventCreate(&ep->b));
    CUDA_TRY(cudaEventRecord(ep->a, s));
    return HPSGD_OK;
}

int prof_resolve();

int prof_end(cudaStream_t s, EventPair* ep)
{
    if (!g.profile) return HPSGD_OK;
    CUDA_TRY(cudaEventRecord(ep->b, s));
    g.prof.push_back(*ep);
    if (g.prof.size() >= 8192) return prof_resolve();   // bound the number of live events (waits for them)
    return HPSGD_OK;
}

int prof_resolve()
{
    for (EventPair& ep : g.prof) {
        CUDA_TRY(cudaEventSynchronize(ep.b));
        float ms = 0.f;
        CUDA_TRY(cudaEventElapsedTime(&ms, ep.a, ep.b));
        g.prof_ms[ep.kind] += ms;
        g.prof_launches[ep.kind] += 1;
        cudaEventDestroy(ep.a);
        cudaEventDestroy(ep.b);
    }
    g.prof.clear();
    return HPSGD_OK;
}

int check_grad_ptr(const void* p, const char* what)
{
    if (!p) return fail(HPSGD_E_BADARG, "%s is NULL", what);
    if (reinterpret_cast<uintptr_t>(p) % 32) return fail(HPSGD_E_BADARG, "%s is not 32-byte aligned", what);
    return HPSGD_OK;
}

int check_desc(const hpsgd_grad_desc* d)
{
    if (!d) return fail(HPSGD_E_BADARG, "descriptor is NULL");
    TRY(check_grad_ptr(d->dense, "dense gradient"));
    if (d->n_rows < 0 || d->n_rows > g.sp_rows) return fail(HPSGD_E_BADARG, "n_rows %d out of range", d->n_rows);
    if (d->n_rows > 0 && d->row_idx) TRY(check_grad_ptr(d->row_vals, "row_vals"));
    return HPSGD_OK;
}

// Checked build: the listed rows of a sparse-row gradient are copied to the host and tested
// (ascending, hence unique, and inside [0, rows)) before anything is enqueued for them.  The
// copy is ordered behind the work already on `s`, which may still be producing the list.  The
// normal build trusts the caller, as the contract says, and does nothing here.
int validate_rows(const hpsgd_grad_desc* d, int64_t rows, cudaStream_t s)
{
#ifdef HPSGD_DEBUG
    if (!d->row_idx || d->n_rows <= 0) return HPSGD_OK;
    std::vector<int32_t> idx((size_t)d->n_rows);
    CUDA_TRY(cudaMemcpyAsync(idx.data(), d->row_idx, idx.size() * 4, cudaMemcpyDeviceToHost, s));
    CUDA_TRY(cudaStreamSynchronize(s));
    for (size_t k = 0; k < idx.size(); ++k) {
        if (idx[k] < 0 || idx[k] >= rows)
            return fail(HPSGD_E_BADARG, "row_idx[%zu] = %d is outside [0, %lld)", k, idx[k], (long long)rows);
        if (k > 0 && idx[k] == idx[k - 1])
            return fail(HPSGD_E_BADARG, "row_idx[%zu] = %d is listed twice", k, idx[k]);
        if (k > 0 && idx[k] < idx[k - 1])
            return fail(HPSGD_E_BADARG, "row_idx is not ascending at entry %zu (%d after %d)", k, idx[k], idx[k - 1]);
    }
#else
    (void)d; (void)rows; (void)s;
#endif
    return HPSGD_OK;
}

int need_init()
{
    if (!g.inited) return fail(HPSGD_E_STATE, "hpsgd_init has not been called");
    return HPSGD_OK;
}

int check_worker(int worker)
{
    if (worker < 0 || worker >= g.K) return fail(HPSGD_E_BADARG, "worker %d outside [0, %d)", worker, g.K);
    return HPSGD_OK;
}

int sync_all()
{
    CUDA_TRY(cudaStreamSynchronize(g.main));
    CUDA_TRY(cudaStreamSynchronize(g.side));
    if (g.copy) CUDA_TRY(cudaStreamSynchronize(g.copy));
    if (g.d2h) CUDA_TRY(cudaStreamSynchronize(g.d2h));
    g.d2h_outstanding = false;
    TRY(staged_poll());
    return debug_poll();
}

int reset_state_from_w()     // D = 0, r_i = w, m_i = 0, counters cleared; blocking
{
    const size_t row = (size_t)g.stride * 4;
    CUDA_TRY(cudaMemsetAsync(g.D, 0, row, g.main));
    if (g.m) CUDA_TRY(cudaMemsetAsync(g.m, 0, row * g.K, g.main));
    if (g.pipeline) {
        std::fill(g.touched.begin(), g.touched.end(), 0);      // replicas are w until their first step
        g.reduce_outstanding = false;
    } else {
        const int64_t nvec = g.P_pad / 4;
        clone_kernel<<<grid_for(clone_kernel, nvec, kThreads), kThreads, 0, g.main>>>(g.w, g.r, g.stride, g.K, nvec);
        ++g.launches;
        TRY(check_async());
    }
    CUDA_TRY(cudaStreamSynchronize(g.main));
    g.D_valid = false;
    g.merges = 0;
    std::fill(g.at_w.begin(), g.at_w.end(), 1);
    std::fill(g.row_valid.begin(), g.row_valid.end(), 1);
    std::fill(g.local_recorded.begin(), g.local_recorded.end(), 0);
    std::fill(g.merge_unwaited.begin(), g.merge_unwaited.end(), 0);
    return HPSGD_OK;
}

int make_chunk_events(int chunks)
{
    for (cudaEvent_t e : g.ev_local) cudaEventDestroy(e);
    for (cudaEvent_t e : g.ev_merge) cudaEventDestroy(e);
    g.ev_local.assign(chunks, nullptr);
    g.ev_merge.assign(chunks, nullptr);
    g.local_recorded.assign(chunks, 0);
    g.merge_unwaited.assign(chunks, 0);
    g.chunks = chunks;
    for (int c = 0; c < chunks; ++c) {
        CUDA_TRY(cudaEventCreateWithFlags(&g.ev_local[c], cudaEventDisableTiming));
        CUDA_TRY(cudaEventCreateWithFlags(&g.ev_merge[c], cudaEventDisableTiming));
    }
    return HPSGD_OK;
}

GenParams gen_params(int worker, int step, int kind, double scale)
{
    GenParams gp{};
    gp.key = g.key;
    gp.step = (uint64_t)step;
    gp.worker = (uint64_t)worker;
    gp.kind = kind;
    gp.scale_f = (float)scale;
    gp.scale_d = scale;
    if (g.sp_tensor >= 0) {
        gp.sp_start = g.starts[g.sp_tensor];
        gp.sp_rows = g.sp_rows;
        gp.sp_cols = g.sp_cols;
    }
    return gp;
}

int check_gen_args(const void* out, int worker, int step, int kind)
{
    TRY(need_init());
    TRY(check_grad_ptr(out, "output buffer"));
    if (worker < 0 || worker >= 256) return fail(HPSGD_E_BADARG, "worker must be in [0, 256)");
    if (step < 0 || step >= (1 << 20)) return fail(HPSGD_E_BADARG, "step must be in [0, 2^20)");
    if (kind != HPSGD_GEN_UNIFORM && kind != HPSGD_GEN_GAUSS) return fail(HPSGD_E_BADARG, "unknown generator kind");
    return HPSGD_OK;
}

void release_all()
{
    if (g.main) cudaStreamSynchronize(g.main);
    if (g.side) cudaStreamSynchronize(g.side);
    if (g.copy) cudaStreamSynchronize(g.copy);
    if (g.d2h) { cudaStreamSynchronize(g.d2h); cudaStreamDestroy(g.d2h); }
    if (g.ev_w_ready) cudaEventDestroy(g.ev_w_ready);
    if (g.ev_d2h_done) cudaEventDestroy(g.ev_d2h_done);
    for (EventPair& ep : g.prof) { cudaEventDestroy(ep.a); cudaEventDestroy(ep.b); }
    for (cudaEvent_t e : g.ev_local) if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : g.ev_merge) if (e) cudaEventDestroy(e);
    if (g.ev_commit) cudaEventDestroy(g.ev_commit);
    if (g.ev_reduce) cudaEventDestroy(g.ev_reduce);
    for (int b = 0; b < 2; ++b) {
        if (g.stage[b]) cudaFree(g.stage[b]);
        if (g.stage_copied[b]) cudaEventDestroy(g.stage_copied[b]);
        if (g.stage_free[b]) cudaEventDestroy(g.stage_free[b]);
    }
    if (g.copy) cudaStreamDestroy(g.copy);
    if (g.own_streams) {
        if (g.main) cudaStreamDestroy(g.main);
        if (g.side) cudaStreamDestroy(g.side);
    }
    if (g.own_slot && g.slot) cudaFree(g.slot);
    if (g.own_arena && g.arena) cudaFree(g.arena);
    cudaGetLastError();
    g = Ctx();
}

}  // namespace
