// C ABI of libhpsgd: the entry points.  The contract of every entry point is documented in
// include/hpsgd.h; state and helpers live in hpsgd_state.cuh, the stream/event schedule and the
// kernel launches in hpsgd_schedule.cuh, the device code in hpsgd_kernels.cuh.
#include "hpsgd_schedule.cuh"

// =============================================================================== C ABI
extern "C" {

const char* hpsgd_last_error(void) { return g_err; }

int64_t hpsgd_layout_padded(int n_tensors, const int64_t* sizes, int64_t* offsets_out)
{
    if (n_tensors <= 0 || !sizes) return fail(HPSGD_E_BADARG, "layout: need at least one tensor size");
    if (n_tensors > kMaxTensors) return fail(HPSGD_E_UNSUPPORTED, "layout: at most %d tensors", kMaxTensors);
    std::vector<int64_t> s(sizes, sizes + n_tensors), off;
    for (int64_t x : s)
        if (x <= 0) return fail(HPSGD_E_BADARG, "layout: tensor sizes must be positive");
    const int64_t pad = layout_of(s, &off, nullptr);
    if (offsets_out) std::memcpy(offsets_out, off.data(), sizeof(int64_t) * n_tensors);
    return pad;
}

int hpsgd_set_form(int form)
{
    if (g.inited) return fail(HPSGD_E_STATE, "hpsgd_set_form must precede hpsgd_init");
    if (form != HPSGD_FORM_REPLICA_CHANGE && form != HPSGD_FORM_GRADIENT_ACCUMULATION)
        return fail(HPSGD_E_BADARG, "unknown form %d", form);
    g_pending.form = form;
    return HPSGD_OK;
}

int hpsgd_set_pipeline(int enable)
{
    if (g.inited) return fail(HPSGD_E_STATE, "hpsgd_set_pipeline must precede hpsgd_init");
    if (enable != 0 && enable != 1) return fail(HPSGD_E_BADARG, "enable must be 0 or 1");
    g_pending.pipeline = enable;
    return HPSGD_OK;
}

int hpsgd_set_layout(int n_tensors, const int64_t* sizes)
{
    if (g.inited) return fail(HPSGD_E_STATE, "hpsgd_set_layout must precede hpsgd_init");
    const int64_t pad = hpsgd_layout_padded(n_tensors, sizes, nullptr);
    if (pad < 0) return (int)pad;
    g_pending.sizes.assign(sizes, sizes + n_tensors);
    return HPSGD_OK;
}

size_t hpsgd_arena_bytes(int64_t P_pad, int K, int flags, int64_t sparse_rows)
{
    if (P_pad <= 0 || K <= 0 || sparse_rows < 0) return 0;
    const int64_t stride = (P_pad + kRowAlignElems - 1) / kRowAlignElems * kRowAlignElems;
    const int64_t cap = (sparse_rows + 63) / 64 * 64;
    // kPageBytes of slack: the regions start at the first 4 KB boundary inside the arena
    return plan_arena(stride, K, (flags & HPSGD_ARENA_MOMENTUM) != 0, (flags & HPSGD_ARENA_PIPELINE) != 0).fixed +
           (size_t)cap * 4 * K + kPageBytes;
}

int hpsgd_bind(void* arena, size_t bytes, void* main_stream, void* side_stream)
{
    if (g.inited) return fail(HPSGD_E_STATE, "hpsgd_bind must precede hpsgd_init");
    if (arena && reinterpret_cast<uintptr_t>(arena) % kAlignBytes)
        return fail(HPSGD_E_BADARG, "arena must be 256-byte aligned");
    if ((arena == nullptr) != (bytes == 0))
        return fail(HPSGD_E_BADARG, "arena and bytes must both be given or both be zero");
    if ((main_stream == nullptr) != (side_stream == nullptr))
        return fail(HPSGD_E_BADARG, "give both streams or neither");
    if (main_stream && main_stream == side_stream)
        return fail(HPSGD_E_BADARG, "main and side stream must differ");
    g_pending.arena = arena;
    g_pending.arena_bytes = bytes;
    g_pending.main = static_cast<cudaStream_t>(main_stream);
    g_pending.side = static_cast<cudaStream_t>(side_stream);
    g_pending.have_streams = main_stream != nullptr;
    return HPSGD_OK;
}

int hpsgd_init(int64_t P, int K, float lr, float momentum, uint64_t seed)
{
    if (g.inited) return fail(HPSGD_E_STATE, "already initialised; call hpsgd_destroy first");
    if (P <= 0) return fail(HPSGD_E_BADARG, "P must be positive");
    if (P >= (int64_t)1 << 32) return fail(HPSGD_E_UNSUPPORTED, "P must be below 2^32");
    if (K <= 0 || K > 256) return fail(HPSGD_E_BADARG, "K must be in [1, 256]");
    if (!(lr >= 0.f)) return fail(HPSGD_E_BADARG, "lr must be >= 0");
    if (!(momentum >= 0.f && momentum < 1.f)) return fail(HPSGD_E_BADARG, "momentum must be in [0, 1)");
    if (g_pending.form == HPSGD_FORM_GRADIENT_ACCUMULATION && momentum != 0.f)
        return fail(HPSGD_E_BADARG, "the gradient-accumulation form is the paper's plain SGD: momentum must be 0");
    if (g_pending.pipeline && g_pending.form != HPSGD_FORM_REPLICA_CHANGE)
        return fail(HPSGD_E_BADARG, "the pipelined schedule is implemented for the replica-change form");
    if (g_pending.pipeline && K > kMaxBatch)
        return fail(HPSGD_E_UNSUPPORTED, "the pipelined schedule supports K <= %d", kMaxBatch);
    std::vector<int64_t> sizes = g_pending.sizes;
    if (sizes.empty()) sizes.push_back(P);
    int64_t sum = 0;
    for (int64_t s : sizes) sum += s;
    if (sum != P)
        return fail(HPSGD_E_BADARG, "P = %lld does not match the layout total %lld", (long long)P, (long long)sum);

    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    cudaDeviceProp prop;
    CUDA_TRY(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10)
        return fail(HPSGD_E_CUDA, "built for sm_100a only; device is sm_%d%d", prop.major, prop.minor);

    // a lent arena may still be the target of the caller's own work on other streams
    if (g_pending.arena) CUDA_TRY(cudaDeviceSynchronize());

    g = Ctx();
    g.sm_count = prop.multiProcessorCount;
    g.P = P; g.K = K; g.lr = lr; g.beta = momentum; g.seed = seed;
    g.key = mix64(seed + kM3);
    g.sizes = sizes;
    g.P_pad = layout_of(sizes, &g.offsets, &g.starts);
    g.stride = (g.P_pad + kRowAlignElems - 1) / kRowAlignElems * kRowAlignElems;
    g.form = g_pending.form;
    const bool mom = momentum != 0.f || g.form == HPSGD_FORM_GRADIENT_ACCUMULATION;   // K extra rows: m_i or a_i
    g.pipeline = g_pending.pipeline;
    const ArenaPlan a = plan_arena(g.stride, K, mom, g.pipeline != 0);

    if (g_pending.arena) {
        if (g_pending.arena_bytes < a.fixed + kPageBytes) {
            g = Ctx();
            return fail(HPSGD_E_NOMEM, "arena of %zu bytes is smaller than the %zu needed", g_pending.arena_bytes,
                        a.fixed + kPageBytes);
        }
        // the regions start at the first 4 KB boundary inside the lent memory
        char* lent = static_cast<char*>(g_pending.arena);
        const size_t skip = (kPageBytes - reinterpret_cast<uintptr_t>(lent) % kPageBytes) % kPageBytes;
        g.arena = lent + skip;
        g.arena_bytes = g_pending.arena_bytes - skip;
        g.slot_cap = (int64_t)((g.arena_bytes - a.fixed) / ((size_t)4 * K)) / 64 * 64;
        g.slot = g.slot_cap ? reinterpret_cast<int32_t*>(g.arena + a.slot) : nullptr;
    } else {
        void* p = nullptr;
        cudaError_t e = cudaMalloc(&p, a.fixed);
        if (e != cudaSuccess) {
            cudaGetLastError();
            g = Ctx();
            return fail(HPSGD_E_NOMEM, "cudaMalloc of %zu bytes failed: %s", a.fixed, cudaGetErrorString(e));
        }
        g.arena = static_cast<char*>(p);
        g.arena_bytes = a.fixed;
        g.own_arena = true;
    }
    g.w = reinterpret_cast<float*>(g.arena + a.w);
    g.D = reinterpret_cast<float*>(g.arena + a.D);
    g.r = reinterpret_cast<float*>(g.arena + a.r);
    g.m = mom ? reinterpret_cast<float*>(g.arena + a.m) : nullptr;
    g.d_table = reinterpret_cast<int64_t*>(g.arena + a.table);
    g.at_w.assign(K, 1);
    g.row_valid.assign(K, 1);
    g.step_held.assign(K, 0);
    g.wbuf[0] = g.w;
    g.rbuf[0] = g.r;
    if (g.pipeline) {
        g.wbuf[1] = reinterpret_cast<float*>(g.arena + a.w2);
        g.rbuf[1] = reinterpret_cast<float*>(g.arena + a.r2);
        g.touched.assign(K, 0);
    }

    if (g_pending.have_streams) {
        g.main = g_pending.main;
        g.side = g_pending.side;
    } else {
        g.own_streams = true;
        if (cudaStreamCreateWithFlags(&g.main, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&g.side, cudaStreamNonBlocking) != cudaSuccess) {
            release_all();
            return fail(HPSGD_E_CUDA, "could not create streams");
        }
    }
    g.inited = true;
    int rc = make_chunk_events(1);
    if (rc) { release_all(); return rc; }
    if (g.pipeline && (cudaEventCreateWithFlags(&g.ev_commit, cudaEventDisableTiming) != cudaSuccess ||
                       cudaEventCreateWithFlags(&g.ev_reduce, cudaEventDisableTiming) != cudaSuccess)) {
        release_all();
        return fail(HPSGD_E_CUDA, "could not create events");
    }

    // device table: offsets | starts | sizes
    const size_t n = sizes.size();
    std::vector<int64_t> table(3 * n);
    for (size_t t = 0; t < n; ++t) {
        table[t] = g.offsets[t];
        table[n + t] = g.starts[t];
        table[2 * n + t] = sizes[t];
    }
    cudaError_t e = cudaMemcpyAsync(g.d_table, table.data(), table.size() * 8, cudaMemcpyHostToDevice, g.main);
    if (e == cudaSuccess) e = cudaStreamSynchronize(g.main);
    if (e == cudaSuccess) e = cudaMemsetAsync(g.w, 0, (size_t)g.stride * 4, g.main);
    if (e != cudaSuccess) {
        release_all();
        return fail(HPSGD_E_CUDA, "state set-up failed: %s", cudaGetErrorString(e));
    }
    GenParams gp = gen_params(0, 0, 2, 0.0);
    gen_flat_kernel<false><<<grid_for(gen_flat_kernel<false>, g.P_pad, kThreads), kThreads, 0, g.main>>>(
        g.w, g.P_pad, g.d_table, g.d_table + n, g.d_table + 2 * n, (int)n, gp);
    ++g.launches;
    rc = reset_state_from_w();
    if (rc) { release_all(); return rc; }
    g_pending = Pending();
    return HPSGD_OK;
}

int hpsgd_destroy(void)
{
    release_all();
    g_pending = Pending();
    return HPSGD_OK;
}

int hpsgd_synchronize(void)
{
    TRY(need_init());
    TRY(flush_deferred());
    TRY(sync_all());
    return check_async();
}

int hpsgd_set_option(int key, double value)
{
    TRY(need_init());
    TRY(flush_deferred());
    switch (key) {
    case HPSGD_OPT_WEIGHT_DECAY:
        if (!(value >= 0.0)) return fail(HPSGD_E_BADARG, "weight decay must be >= 0");
        if (value != 0.0 && g.form == HPSGD_FORM_GRADIENT_ACCUMULATION)
            return fail(HPSGD_E_BADARG, "the gradient-accumulation form has no weight decay");
        g.lambda = (float)value;
        return HPSGD_OK;
    case HPSGD_OPT_STALENESS:
        if (value != 0.0 && value != 1.0) return fail(HPSGD_E_BADARG, "staleness must be 0 or 1");
        if (g.merges) return fail(HPSGD_E_STATE, "staleness can only change before the first merge");
        if (value == 0.0 && g.pipeline)
            return fail(HPSGD_E_BADARG, "the pipelined schedule needs the one-synchronisation delay (staleness 1)");
        g.staleness = (int)value;
        return HPSGD_OK;
    case HPSGD_OPT_GRAD_DTYPE:
        if (value != HPSGD_F32 && value != HPSGD_BF16) return fail(HPSGD_E_BADARG, "unknown gradient dtype");
        g.grad_dtype = (int)value;
        return HPSGD_OK;
    case HPSGD_OPT_OVERLAP:
        if (value != 0.0 && value != 1.0) return fail(HPSGD_E_BADARG, "overlap must be 0 or 1");
        TRY(sync_all());                   // the schedule may only change while idle
        g.overlap = (int)value;
        std::fill(g.local_recorded.begin(), g.local_recorded.end(), 0);
        std::fill(g.merge_unwaited.begin(), g.merge_unwaited.end(), 0);
        return HPSGD_OK;
    case HPSGD_OPT_CHUNKS:
        if (!(value >= 1.0 && value <= kMaxChunks && value == (double)(int)value))
            return fail(HPSGD_E_BADARG, "chunks must be an integer in [1, %d]", kMaxChunks);
        if (value != 1.0 && g.pipeline) return fail(HPSGD_E_BADARG, "the pipelined schedule is not cut into chunks");
        TRY(sync_all());
        return make_chunk_events((int)value);
    case HPSGD_OPT_FUSE:
        if (value != 0.0 && value != 1.0 && value != 2.0) return fail(HPSGD_E_BADARG, "fuse must be 0, 1 or 2");
        g.fuse = (int)value;
        if (!lazy_clones() && !g.pipeline) TRY(materialize_clones());   // the other schedules read replica rows
        return HPSGD_OK;
    case HPSGD_OPT_STAGING:
        if (value != 0.0 && value != 1.0) return fail(HPSGD_E_BADARG, "staging must be 0 or 1");
        g.staging = (int)value;
        return HPSGD_OK;
    case HPSGD_OPT_DEBUG_GROUP_LIMIT:
#ifdef HPSGD_DEBUG
        if (!(value >= -1.0 && value <= (double)(g.P_pad / 8) && value == (double)(int64_t)value))
            return fail(HPSGD_E_BADARG, "the limit must be -1 (the real one) or a whole number of groups in [0, P_pad / 8]");
        g.debug_limit = (int64_t)value;
        return HPSGD_OK;
#else
        return fail(HPSGD_E_UNSUPPORTED, "only the checked build (HPSGD_DEBUG) has kernel guards");
#endif
    case HPSGD_OPT_DEBUG_STAGE_STALL:
#ifdef HPSGD_DEBUG
        if (value != 0.0 && value != 1.0) return fail(HPSGD_E_BADARG, "stall must be 0 or 1");
        g.debug_stage_stall = value != 0.0;
        return HPSGD_OK;
#else
        return fail(HPSGD_E_UNSUPPORTED, "only the checked build (HPSGD_DEBUG) can make the staged merge's wait run out");
#endif
    case HPSGD_OPT_PROFILE:
        if (value != 0.0 && value != 1.0) return fail(HPSGD_E_BADARG, "profile must be 0 or 1");
        TRY(prof_resolve());
        g.profile = (int)value;
        return HPSGD_OK;
    default:
        return fail(HPSGD_E_BADARG, "unknown option %d", key);
    }
}

int hpsgd_set_sparse_segment(int tensor_id, int64_t rows, int64_t cols)
{
    TRY(need_init());
    TRY(flush_deferred());
    if (tensor_id < 0) {
        g.sp_tensor = -1;
        g.sp_rows = g.sp_cols = 0;
        return HPSGD_OK;
    }
    if (tensor_id >= (int)g.sizes.size()) return fail(HPSGD_E_BADARG, "tensor %d does not exist", tensor_id);
    if (rows <= 0 || cols <= 0 || cols % 8)
        return fail(HPSGD_E_BADARG, "rows must be positive and cols a positive multiple of 8");
    if (rows > INT32_MAX) return fail(HPSGD_E_UNSUPPORTED, "too many rows");
    if (rows * cols != g.sizes[tensor_id]) return fail(HPSGD_E_BADARG, "rows*cols does not match the tensor size");
    if (rows > g.slot_cap) {
        if (!g.own_arena)
            return fail(HPSGD_E_NOMEM, "arena has room for %lld sparse rows per worker, %lld needed",
                        (long long)g.slot_cap, (long long)rows);
        // library-owned memory: the map is its own allocation, kept until hpsgd_destroy
        TRY(sync_all());
        if (g.own_slot && g.slot) cudaFree(g.slot);
        g.slot = nullptr; g.slot_cap = 0; g.own_slot = false;
        const int64_t cap = (rows + 63) / 64 * 64;
        void* p = nullptr;
        cudaError_t e = cudaMalloc(&p, (size_t)cap * 4 * g.K);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return fail(HPSGD_E_NOMEM, "cudaMalloc of the slot map failed: %s", cudaGetErrorString(e));
        }
        g.slot = static_cast<int32_t*>(p);
        g.slot_cap = cap;
        g.own_slot = true;
    }
    g.sp_tensor = tensor_id;
    g.sp_rows = rows;
    g.sp_cols = cols;
    return HPSGD_OK;
}

// ------------------------------------------------------------------------- local steps
}  // extern "C"

namespace {

// Copy stream, two staging buffers and their events of hpsgd_local_step_host: built into locals
// and handed to the state only when all of it exists, so that a failure half-way leaves nothing
// behind and the next call simply tries again.
int make_host_staging()
{
    cudaStream_t copy = nullptr;
    void* stage[2] = {nullptr, nullptr};
    cudaEvent_t copied[2] = {nullptr, nullptr}, freed[2] = {nullptr, nullptr};
    int rc = HPSGD_OK;
    cudaError_t e = cudaStreamCreateWithFlags(&copy, cudaStreamNonBlocking);
    if (e != cudaSuccess) rc = fail(HPSGD_E_CUDA, "could not create the copy stream: %s", cudaGetErrorString(e));
    for (int b = 0; b < 2 && rc == HPSGD_OK; ++b) {
        e = cudaMalloc(&stage[b], (size_t)g.P_pad * 4);
        if (e != cudaSuccess) {
            rc = fail(HPSGD_E_NOMEM, "cudaMalloc of the staging buffer failed: %s", cudaGetErrorString(e));
            break;
        }
        e = cudaEventCreateWithFlags(&copied[b], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&freed[b], cudaEventDisableTiming);
        if (e != cudaSuccess) rc = fail(HPSGD_E_CUDA, "could not create the staging events: %s", cudaGetErrorString(e));
    }
    if (rc != HPSGD_OK) {
        for (int b = 0; b < 2; ++b) {
            if (stage[b]) cudaFree(stage[b]);
            if (copied[b]) cudaEventDestroy(copied[b]);
            if (freed[b]) cudaEventDestroy(freed[b]);
        }
        if (copy) cudaStreamDestroy(copy);
        cudaGetLastError();
        return rc;
    }
    for (int b = 0; b < 2; ++b) {
        g.stage[b] = stage[b];
        g.stage_copied[b] = copied[b];
        g.stage_free[b] = freed[b];
        g.stage_used[b] = false;
    }
    g.copy = copy;
    return HPSGD_OK;
}

}  // namespace

extern "C" {

int hpsgd_local_step(int worker, const void* grads)
{
    TRY(need_init());
    TRY(check_worker(worker));
    TRY(check_grad_ptr(grads, "grads"));
    BatchPtrs gp{};
    gp.dense[0] = grads;
    if (lazy_clones()) return hold_step(worker, gp, 0, false);     // fuse 2: held back for the merge it will run with
    TRY(flush_deferred());
    return enqueue_local(worker, 1, gp, false);
}

int hpsgd_local_step_ex(int worker, const hpsgd_grad_desc* desc)
{
    TRY(need_init());
    TRY(check_worker(worker));
    if (g.sp_tensor < 0) return fail(HPSGD_E_STATE, "no sparse-row tensor declared");
    TRY(check_desc(desc));
    TRY(validate_rows(desc, g.sp_rows, g.main));
    const bool hold = lazy_clones();
    // a held step of this worker still uses its slot map; held dense steps cannot share a launch with this one
    if (!hold || (g.steps_held && (g.step_held[worker] || !g.deferred_sparse))) TRY(flush_deferred());
    BatchPtrs gp{};
    TRY(enqueue_slot_maps(worker, 1, desc, &gp));
    if (hold) return hold_step(worker, gp, 0, true);
    return enqueue_local(worker, 1, gp, true);
}

int hpsgd_local_step_all(const void* grads, int64_t worker_stride_bytes)
{
    TRY(need_init());
    TRY(check_grad_ptr(grads, "grads"));
    const int64_t esz = g.grad_dtype == HPSGD_BF16 ? 2 : 4;
    if (worker_stride_bytes % 32 || worker_stride_bytes < g.P_pad * esz)
        return fail(HPSGD_E_BADARG, "worker stride must be a multiple of 32 bytes and cover P_pad elements");
    if (g.merge_deferred && g.K <= kMaxBatch) {
        BatchPtrs gp{};
        for (int i = 0; i < g.K; ++i) gp.dense[i] = static_cast<const char*>(grads) + (int64_t)i * worker_stride_bytes;
        return enqueue_fused(gp, false);
    }
    TRY(flush_deferred());
    if (lazy_clones()) {                   // fuse 2: held back for the merge they will run with
        BatchPtrs gp{};
        for (int i = 0; i < g.K; ++i) gp.dense[i] = static_cast<const char*>(grads) + (int64_t)i * worker_stride_bytes;
        for (int i = 0; i < g.K; ++i) TRY(hold_step(i, gp, i, false));
        return HPSGD_OK;
    }
    for (int w0 = 0; w0 < g.K; w0 += kMaxBatch) {
        const int nw = std::min(kMaxBatch, g.K - w0);
        BatchPtrs gp{};
        for (int i = 0; i < nw; ++i) gp.dense[i] = static_cast<const char*>(grads) + (int64_t)(w0 + i) * worker_stride_bytes;
        TRY(enqueue_local(w0, nw, gp, false));
    }
    return HPSGD_OK;
}

int hpsgd_local_step_all_ex(const hpsgd_grad_desc* descs)
{
    TRY(need_init());
    if (g.sp_tensor < 0) return fail(HPSGD_E_STATE, "no sparse-row tensor declared");
    if (g.K > kMaxBatch) return fail(HPSGD_E_UNSUPPORTED, "batched sparse steps support K <= %d", kMaxBatch);
    if (!descs) return fail(HPSGD_E_BADARG, "descriptor array is NULL");
    for (int i = 0; i < g.K; ++i) TRY(check_desc(descs + i));
    for (int i = 0; i < g.K; ++i) TRY(validate_rows(descs + i, g.sp_rows, g.main));
    if (g.steps_held) TRY(flush_deferred());             // held-back steps still use the slot maps
    BatchPtrs gp{};
    TRY(enqueue_slot_maps(0, g.K, descs, &gp));
    if (g.merge_deferred) return enqueue_fused(gp, true);
    if (lazy_clones()) {
        for (int i = 0; i < g.K; ++i) TRY(hold_step(i, gp, i, true));
        return HPSGD_OK;
    }
    return enqueue_local(0, g.K, gp, true);
}

int hpsgd_local_step_host(int worker, const void* host_grads)
{
    TRY(need_init());
    TRY(check_worker(worker));
    if (!host_grads) return fail(HPSGD_E_BADARG, "host_grads is NULL");
    TRY(flush_deferred());
    const size_t bytes = (size_t)g.P_pad * (g.grad_dtype == HPSGD_BF16 ? 2 : 4);
    if (!g.copy) TRY(make_host_staging());
    const int b = g.stage_next;
    g.stage_next ^= 1;
    if (g.stage_used[b]) CUDA_TRY(cudaStreamWaitEvent(g.copy, g.stage_free[b], 0));
    CUDA_TRY(cudaMemcpyAsync(g.stage[b], host_grads, bytes, cudaMemcpyHostToDevice, g.copy));
    CUDA_TRY(cudaEventRecord(g.stage_copied[b], g.copy));
    CUDA_TRY(cudaStreamWaitEvent(g.main, g.stage_copied[b], 0));
    BatchPtrs gp{};
    gp.dense[0] = g.stage[b];
    TRY(enqueue_local(worker, 1, gp, false));
    CUDA_TRY(cudaEventRecord(g.stage_free[b], g.main));
    g.stage_used[b] = true;
    return HPSGD_OK;
}

// ------------------------------------------------------------------------- merge
int hpsgd_sync_merge(void)
{
    TRY(need_init());
    if (g.merge_deferred) TRY(flush_deferred());   // two merges in a row: the earlier one runs on its own
    int flags = 0;
    if (g.staleness == 0) flags |= kMergeImmediate;
    else if (g.D_valid) flags |= kMergeApplyPending;
    g.D_valid = true;
    g.merges += 1;
    if (g.steps_held == g.K) return enqueue_round(flags);   // fuse 2: every worker's held-back step and this merge, one kernel
    if (g.steps_held) TRY(flush_deferred());                // some workers only: their steps run first, on their own
    if (g.pipeline) return enqueue_pipelined_merge(flags);
    if (g.fuse == 1 && g.form == HPSGD_FORM_REPLICA_CHANGE) {
        g.merge_deferred = true;
        g.deferred_flags = flags;
        return HPSGD_OK;
    }
    return enqueue_merge(flags);
}

int hpsgd_flush(void)
{
    TRY(need_init());
    return flush_deferred();
}

const float* hpsgd_get_global(void)
{
    if (need_init()) return nullptr;
    if (flush_deferred()) return nullptr;
    if (sync_all()) return nullptr;
    if (check_async()) return nullptr;
    return g.w;
}

// ------------------------------------------------------------------------- host copies, inspection
int hpsgd_set_global_host(const float* host_w, int64_t n)
{
    TRY(need_init());
    if (!host_w || n != g.P) return fail(HPSGD_E_BADARG, "need a host array of exactly P = %lld floats", (long long)g.P);
    TRY(flush_deferred());
    TRY(sync_all());
    CUDA_TRY(cudaMemsetAsync(g.w, 0, (size_t)g.stride * 4, g.main));
    for (size_t t = 0; t < g.sizes.size(); ++t)
        CUDA_TRY(cudaMemcpyAsync(g.w + g.offsets[t], host_w + g.starts[t], (size_t)g.sizes[t] * 4,
                                 cudaMemcpyHostToDevice, g.main));
    return reset_state_from_w();
}

int hpsgd_fill_global(uint64_t seed)
{
    TRY(need_init());
    TRY(flush_deferred());
    TRY(sync_all());
    g.seed = seed;
    g.key = mix64(seed + kM3);
    const size_t n = g.sizes.size();
    CUDA_TRY(cudaMemsetAsync(g.w, 0, (size_t)g.stride * 4, g.main));
    const GenParams gp = gen_params(0, 0, 2, 0.0);
    gen_flat_kernel<false><<<grid_for(gen_flat_kernel<false>, g.P_pad, kThreads), kThreads, 0, g.main>>>(
        g.w, g.P_pad, g.d_table, g.d_table + n, g.d_table + 2 * n, (int)n, gp);
    ++g.launches;
    TRY(check_async());
    return reset_state_from_w();
}

int hpsgd_copy_global(float* host_out, int64_t n)
{
    TRY(need_init());
    if (!host_out || n != g.P) return fail(HPSGD_E_BADARG, "need a host array of exactly P = %lld floats", (long long)g.P);
    TRY(flush_deferred());
    TRY(sync_all());
    for (size_t t = 0; t < g.sizes.size(); ++t)
        CUDA_TRY(cudaMemcpyAsync(host_out + g.starts[t], g.w + g.offsets[t], (size_t)g.sizes[t] * 4,
                                 cudaMemcpyDeviceToHost, g.main));
    CUDA_TRY(cudaStreamSynchronize(g.main));
    return HPSGD_OK;
}

int hpsgd_copy_global_async(float* host_out, int64_t n)
{
    TRY(need_init());
    if (!host_out || n != g.P) return fail(HPSGD_E_BADARG, "need a host array of exactly P = %lld floats", (long long)g.P);
    TRY(flush_deferred());
    if (!g.d2h) {
        CUDA_TRY(cudaStreamCreateWithFlags(&g.d2h, cudaStreamNonBlocking));
        CUDA_TRY(cudaEventCreateWithFlags(&g.ev_w_ready, cudaEventDisableTiming));
        CUDA_TRY(cudaEventCreateWithFlags(&g.ev_d2h_done, cudaEventDisableTiming));
    }
    // w is last written by a merge on the side stream, or on the main stream (no overlap, a fused
    // merge + step kernel, the commit of the pipelined schedule): the copy waits for both
    CUDA_TRY(cudaEventRecord(g.ev_w_ready, g.main));
    CUDA_TRY(cudaStreamWaitEvent(g.d2h, g.ev_w_ready, 0));
    CUDA_TRY(cudaEventRecord(g.ev_w_ready, g.side));
    CUDA_TRY(cudaStreamWaitEvent(g.d2h, g.ev_w_ready, 0));
    for (size_t t = 0; t < g.sizes.size(); ++t)
        CUDA_TRY(cudaMemcpyAsync(host_out + g.starts[t], g.w + g.offsets[t], (size_t)g.sizes[t] * 4,
                                 cudaMemcpyDeviceToHost, g.d2h));
    CUDA_TRY(cudaEventRecord(g.ev_d2h_done, g.d2h));
    g.d2h_outstanding = true;
    return HPSGD_OK;
}

int hpsgd_get_replica(int worker, const float** r, const float** m)
{
    TRY(need_init());
    TRY(check_worker(worker));
    if (r) *r = g.pipeline ? (g.touched[worker] ? g.r + (int64_t)worker * g.stride : g.w) : replica_src(worker);
    if (m) *m = g.m ? g.m + (int64_t)worker * g.stride : nullptr;
    return HPSGD_OK;
}

int hpsgd_get_pending(const float** D)
{
    TRY(need_init());
    if (D) *D = g.D;
    return HPSGD_OK;
}

// ------------------------------------------------------------------------- checkpoint
namespace {

struct StateHeader {
    uint64_t magic;            // "HPSGDST1"
    int64_t P, P_pad, merges;
    int32_t K, form, has_aux, staleness, D_valid, reserved;
};
constexpr uint64_t kStateMagic = 0x3154534447535048ULL;

size_t state_bytes()
{
    const size_t row = (size_t)g.P_pad * 4;
    return sizeof(StateHeader) + row * (2 + (size_t)g.K * (g.m ? 2 : 1));
}

}  // namespace

size_t hpsgd_state_bytes(void)
{
    if (!g.inited) return 0;
    return state_bytes();
}

int hpsgd_export_state(void* host_out, size_t bytes)
{
    TRY(need_init());
    if (!host_out || bytes < state_bytes()) return fail(HPSGD_E_BADARG, "need a host buffer of hpsgd_state_bytes() = %zu bytes", state_bytes());
    TRY(flush_deferred());
    TRY(sync_all());
    StateHeader h{};
    h.magic = kStateMagic;
    h.P = g.P; h.P_pad = g.P_pad; h.merges = g.merges;
    h.K = g.K; h.form = g.form; h.has_aux = g.m ? 1 : 0; h.staleness = g.staleness; h.D_valid = g.D_valid ? 1 : 0;
    char* out = static_cast<char*>(host_out);
    std::memcpy(out, &h, sizeof h);
    out += sizeof h;
    const size_t row = (size_t)g.P_pad * 4;
    CUDA_TRY(cudaMemcpy(out, g.w, row, cudaMemcpyDeviceToHost)); out += row;
    CUDA_TRY(cudaMemcpy(out, g.D, row, cudaMemcpyDeviceToHost)); out += row;
    for (int i = 0; i < g.K; ++i) {
        // a worker that has not stepped since the last synchronisation may have w itself as its replica
        const float* src = g.pipeline ? (g.touched[i] ? g.r + (int64_t)i * g.stride : g.w) : replica_src(i);
        CUDA_TRY(cudaMemcpy(out, src, row, cudaMemcpyDeviceToHost)); out += row;
    }
    if (g.m)
        for (int i = 0; i < g.K; ++i) {
            CUDA_TRY(cudaMemcpy(out, g.m + (int64_t)i * g.stride, row, cudaMemcpyDeviceToHost)); out += row;
        }
    return HPSGD_OK;
}

int hpsgd_import_state(const void* host_in, size_t bytes)
{
    TRY(need_init());
    if (!host_in || bytes < sizeof(StateHeader)) return fail(HPSGD_E_BADARG, "state blob too short");
    StateHeader h;
    std::memcpy(&h, host_in, sizeof h);
    if (h.magic != kStateMagic) return fail(HPSGD_E_BADARG, "not a state blob of this library");
    if (h.P != g.P || h.P_pad != g.P_pad || h.K != g.K || h.form != g.form || h.has_aux != (g.m ? 1 : 0))
        return fail(HPSGD_E_BADARG, "state blob does not match the initialised sizes, form or optimiser");
    if (bytes < state_bytes()) return fail(HPSGD_E_BADARG, "state blob truncated");
    if (h.staleness != 0 && h.staleness != 1) return fail(HPSGD_E_BADARG, "state blob holds staleness %d", h.staleness);
    if (g.pipeline && h.staleness != 1)
        return fail(HPSGD_E_BADARG, "the pipelined schedule needs the one-synchronisation delay; the blob was written with staleness 0");
    if (h.staleness != g.staleness && g.merges) return fail(HPSGD_E_STATE, "staleness differs and merges have already run");
    TRY(flush_deferred());
    TRY(sync_all());
    const char* in = static_cast<const char*>(host_in) + sizeof h;
    const size_t row = (size_t)g.P_pad * 4;
    CUDA_TRY(cudaMemcpy(g.w, in, row, cudaMemcpyHostToDevice)); in += row;
    CUDA_TRY(cudaMemcpy(g.D, in, row, cudaMemcpyHostToDevice)); in += row;
    for (int i = 0; i < g.K; ++i) {
        CUDA_TRY(cudaMemcpy(g.r + (int64_t)i * g.stride, in, row, cudaMemcpyHostToDevice)); in += row;
    }
    if (g.m)
        for (int i = 0; i < g.K; ++i) {
            CUDA_TRY(cudaMemcpy(g.m + (int64_t)i * g.stride, in, row, cudaMemcpyHostToDevice)); in += row;
        }
    g.staleness = h.staleness;
    g.D_valid = h.D_valid != 0;
    g.merges = h.merges;
    if (g.pipeline) std::fill(g.touched.begin(), g.touched.end(), 1);   // every replica row now holds real data
    std::fill(g.row_valid.begin(), g.row_valid.end(), 1);
    std::fill(g.at_w.begin(), g.at_w.end(), 0);                         // unknown history: the rows are what counts
    g.reduce_outstanding = false;
    std::fill(g.local_recorded.begin(), g.local_recorded.end(), 0);
    std::fill(g.merge_unwaited.begin(), g.merge_unwaited.end(), 0);
    return HPSGD_OK;
}

int hpsgd_get_sizes(int64_t* P, int64_t* P_pad, int* K, int64_t* merges)
{
    TRY(need_init());
    if (P) *P = g.P;
    if (P_pad) *P_pad = g.P_pad;
    if (K) *K = g.K;
    if (merges) *merges = g.merges;
    return HPSGD_OK;
}

int64_t hpsgd_tensor_offset(int tensor_id)
{
    TRY(need_init());
    if (tensor_id < 0 || tensor_id >= (int)g.sizes.size()) return fail(HPSGD_E_BADARG, "tensor %d does not exist", tensor_id);
    return g.offsets[tensor_id];
}

// ------------------------------------------------------------------------- generators
int hpsgd_gen_grads(void* out, int worker, int step, int kind, double scale)
{
    TRY(check_gen_args(out, worker, step, kind));
    if (g.steps_held) TRY(flush_deferred());   // a held-back step may still have to read what `out` holds now
    const GenParams gp = gen_params(worker, step, kind, scale);
    const size_t n = g.sizes.size();
    if (g.grad_dtype == HPSGD_BF16)
        gen_flat_kernel<true><<<grid_for(gen_flat_kernel<true>, g.P_pad, kThreads), kThreads, 0, g.main>>>(
            out, g.P_pad, g.d_table, g.d_table + n, g.d_table + 2 * n, (int)n, gp);
    else
        gen_flat_kernel<false><<<grid_for(gen_flat_kernel<false>, g.P_pad, kThreads), kThreads, 0, g.main>>>(
            out, g.P_pad, g.d_table, g.d_table + n, g.d_table + 2 * n, (int)n, gp);
    ++g.launches;
    return check_async();
}

int hpsgd_gen_row_vals(void* out, int worker, int step, int kind, double scale,
                       const int32_t* row_idx, int32_t n_rows)
{
    TRY(check_gen_args(out, worker, step, kind));
    if (g.sp_tensor < 0) return fail(HPSGD_E_STATE, "no sparse-row tensor declared");
    if (n_rows < 0 || n_rows > g.sp_rows) return fail(HPSGD_E_BADARG, "n_rows out of range");
    if (n_rows == 0) return HPSGD_OK;
    if (!row_idx) return fail(HPSGD_E_BADARG, "row_idx is NULL");
    if (g.steps_held) TRY(flush_deferred());
    const GenParams gp = gen_params(worker, step, kind, scale);
    const int64_t n = (int64_t)n_rows * g.sp_cols;
    if (g.grad_dtype == HPSGD_BF16)
        gen_rows_kernel<true><<<grid_for(gen_rows_kernel<true>, n, kThreads), kThreads, 0, g.main>>>(out, row_idx, n_rows, gp);
    else
        gen_rows_kernel<false><<<grid_for(gen_rows_kernel<false>, n, kThreads), kThreads, 0, g.main>>>(out, row_idx, n_rows, gp);
    ++g.launches;
    return check_async();
}

// ------------------------------------------------------------------------- profiling, counters
int hpsgd_profile_read(int kind, double* ms, int64_t* launches)
{
    TRY(need_init());
    if (kind < 0 || kind > 4) return fail(HPSGD_E_BADARG, "unknown kernel kind %d", kind);
    TRY(flush_deferred());
    TRY(sync_all());
    TRY(prof_resolve());
    if (ms) *ms = g.prof_ms[kind];
    if (launches) *launches = g.prof_launches[kind];
    g.prof_ms[kind] = 0;
    g.prof_launches[kind] = 0;
    return HPSGD_OK;
}

int64_t hpsgd_launch_count(void) { return g.inited ? g.launches : 0; }

// ------------------------------------------------------------------------- bandwidth probe
}  // extern "C"

namespace {

template <int R, int W>
void launch_probe(cudaStream_t s, float* base, int64_t row_floats, int64_t n_groups)
{
    // the W destination rows follow the R source rows; with nothing to write the (never taken) store aims at row 0
    float* dst = W > 0 ? base + (int64_t)R * row_floats : base;
    stream_probe_kernel<R, W><<<hot_grid(n_groups), kHotThreads, 0, s>>>(base, dst, row_floats, n_groups);
}

// The read / write mixes the probe is built for: (16, 0) pure reads ... (0, 16) pure writes.
bool probe_dispatch(int R, int W, cudaStream_t s, float* base, int64_t row_floats, int64_t n_groups)
{
#define HPSGD_PROBE_CASE(r, w) if (R == r && W == w) { launch_probe<r, w>(s, base, row_floats, n_groups); return true; }
    HPSGD_PROBE_CASE(16, 0)
    HPSGD_PROBE_CASE(12, 4)
    HPSGD_PROBE_CASE(16, 4)
    HPSGD_PROBE_CASE(13, 7)
    HPSGD_PROBE_CASE(12, 8)
    HPSGD_PROBE_CASE(8, 8)
    HPSGD_PROBE_CASE(4, 16)
    HPSGD_PROBE_CASE(0, 16)
#undef HPSGD_PROBE_CASE
    return false;
}

}  // namespace

extern "C" {

int hpsgd_probe_hbm(void* scratch, size_t scratch_bytes, int n_read, int n_write, int64_t row_bytes, int iters,
                    double* gb_per_s)
{
    if (!scratch || reinterpret_cast<uintptr_t>(scratch) % kPageBytes)
        return fail(HPSGD_E_BADARG, "scratch must be a 4096-byte aligned device pointer");
    if (row_bytes <= 0 || row_bytes % (int64_t)kPageBytes) return fail(HPSGD_E_BADARG, "row_bytes must be a positive multiple of 4096");
    if (n_read < 0 || n_write < 0 || n_read + n_write <= 0) return fail(HPSGD_E_BADARG, "need at least one stream");
    if (iters <= 0 || iters > 10000) return fail(HPSGD_E_BADARG, "iters must be in [1, 10000]");
    if (!gb_per_s) return fail(HPSGD_E_BADARG, "gb_per_s is NULL");
    const int rows = n_read + n_write;
    if (scratch_bytes / (size_t)row_bytes < (size_t)rows)
        return fail(HPSGD_E_NOMEM, "scratch of %zu bytes is smaller than the %d rows of %lld bytes needed", scratch_bytes,
                    rows, (long long)row_bytes);
    cudaStream_t s = nullptr;
    cudaEvent_t a = nullptr, b = nullptr;
    float* base = static_cast<float*>(scratch);
    const int64_t row_floats = row_bytes / 4, n_groups = row_bytes / 32;
    int rc = HPSGD_OK;
    float ms = 0.f;
    cudaError_t e = cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreate(&a);
    if (e == cudaSuccess) e = cudaEventCreate(&b);
    // zeros: sums stay finite however often the probe runs over the same memory
    if (e == cudaSuccess) e = cudaMemsetAsync(scratch, 0, (size_t)rows * (size_t)row_bytes, s);
    if (e == cudaSuccess) {
        for (int it = -2; it < iters && rc == HPSGD_OK; ++it) {          // two untimed launches first
            if (it == 0) e = cudaEventRecord(a, s);
            if (e != cudaSuccess) break;
            if (!probe_dispatch(n_read, n_write, s, base, row_floats, n_groups))
                rc = fail(HPSGD_E_UNSUPPORTED, "no probe for %d read and %d write streams; built: (16,0) (12,4) (16,4) (13,7) "
                                               "(12,8) (8,8) (4,16) (0,16)", n_read, n_write);
        }
    }
    if (e == cudaSuccess && rc == HPSGD_OK) e = cudaEventRecord(b, s);
    if (e == cudaSuccess && rc == HPSGD_OK) e = cudaEventSynchronize(b);
    if (e == cudaSuccess && rc == HPSGD_OK) e = cudaEventElapsedTime(&ms, a, b);
    if (e == cudaSuccess && rc == HPSGD_OK) e = cudaGetLastError();
    if (s) { cudaStreamSynchronize(s); cudaStreamDestroy(s); }
    if (a) cudaEventDestroy(a);
    if (b) cudaEventDestroy(b);
    if (rc != HPSGD_OK) return rc;
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(HPSGD_E_CUDA, "bandwidth probe failed: %s", cudaGetErrorString(e));
    }
    *gb_per_s = (double)(n_read + n_write) * (double)row_bytes * iters / (ms * 1e-3) / 1e9;
    return HPSGD_OK;
}

}  // extern "C"

// =============================================================================== no-allocation entry
// hpsgd_local_step_sparse_noalloc: the sparse-row local step for callers that cannot
// allocate device memory.  Its row -> slot scratch map is the file-scope array below,
// which every GPU that loads this library holds until the process exits.
static __device__ __align__(256) int32_t g_noalloc_slot[HPSGD_NOALLOC_MAX_ROWS];

namespace {

constexpr int kNoallocMaxDevices = 64;
struct NoallocDevice {
    std::once_flag once;
    cudaError_t status = cudaErrorUnknown;
    int32_t* slot = nullptr;     // device address of g_noalloc_slot on this device
} g_noalloc_dev[kNoallocMaxDevices];

// Once per device, with that device current: g_noalloc_slot names a host-side stand-in in
// host code, so the address a kernel can use has to be asked for.  std::call_once makes the
// look-up safe when several host threads make their first call on a device together.
int noalloc_setup(int dev, int32_t** slot)
{
    if (dev < 0 || dev >= kNoallocMaxDevices) return fail(HPSGD_E_UNSUPPORTED, "device index %d not supported", dev);
    NoallocDevice& d = g_noalloc_dev[dev];
    std::call_once(d.once, [&d] {
        void* p = nullptr;
        d.status = cudaGetSymbolAddress(&p, g_noalloc_slot);
        if (d.status == cudaSuccess) d.slot = static_cast<int32_t*>(p);
        else cudaGetLastError();
    });
    if (d.status != cudaSuccess)
        return fail(HPSGD_E_CUDA, "cudaGetSymbolAddress of the scratch map failed: %s", cudaGetErrorString(d.status));
    *slot = d.slot;
    return HPSGD_OK;
}

template <bool BF16, bool MOM, bool WD>
void noalloc_launch(cudaStream_t s, float* r, float* m, const BatchPtrs& gp, const SparseSeg& seg, int64_t n,
                    const StepParams& p)
{
    local_step_kernel<BF16, MOM, WD, true><<<hot_grid(n), kHotThreads, 0, s>>>(r, m, 0, 0, gp, seg, 0, n, p, n);
}

}  // namespace

extern "C" int hpsgd_local_step_sparse_noalloc(float* replica, float* momentum_buf, int64_t n_elems,
                                               const hpsgd_grad_desc* desc, int grad_dtype,
                                               int64_t seg_offset, int64_t rows, int64_t cols,
                                               float lr, float momentum, float weight_decay, void* stream)
{
    if (!replica || reinterpret_cast<uintptr_t>(replica) % 32) return fail(HPSGD_E_BADARG, "replica must be a 32-byte aligned device pointer");
    if (!(momentum >= 0.f && momentum < 1.f)) return fail(HPSGD_E_BADARG, "momentum must be in [0, 1)");
    if (momentum != 0.f && (!momentum_buf || reinterpret_cast<uintptr_t>(momentum_buf) % 32))
        return fail(HPSGD_E_BADARG, "momentum_buf must be a 32-byte aligned device pointer when momentum != 0");
    if (!(lr >= 0.f) || !(weight_decay >= 0.f)) return fail(HPSGD_E_BADARG, "lr and weight_decay must be >= 0");
    if (n_elems <= 0 || n_elems % 8) return fail(HPSGD_E_BADARG, "n_elems must be a positive multiple of 8");
    if (grad_dtype != HPSGD_F32 && grad_dtype != HPSGD_BF16) return fail(HPSGD_E_BADARG, "unknown gradient dtype");
    if (rows <= 0 || cols <= 0 || cols % 8) return fail(HPSGD_E_BADARG, "rows must be positive and cols a positive multiple of 8");
    if (rows > HPSGD_NOALLOC_MAX_ROWS)
        return fail(HPSGD_E_UNSUPPORTED, "%lld rows exceed the built-in scratch map of %d rows; use hpsgd_local_step_ex",
                    (long long)rows, HPSGD_NOALLOC_MAX_ROWS);
    // tested by division first, so that rows * cols is only formed when it cannot overflow
    if (cols > n_elems || rows > n_elems / cols || seg_offset < 0 || seg_offset % 8 || seg_offset > n_elems - rows * cols)
        return fail(HPSGD_E_BADARG, "the sparse tensor does not fit inside the flat buffer");
    if (!desc) return fail(HPSGD_E_BADARG, "descriptor is NULL");
    TRY(check_grad_ptr(desc->dense, "dense gradient"));
    if (desc->n_rows < 0 || desc->n_rows > rows) return fail(HPSGD_E_BADARG, "n_rows %d out of range", desc->n_rows);
    const bool have_rows = desc->row_idx && desc->n_rows > 0;
    if (have_rows) TRY(check_grad_ptr(desc->row_vals, "row_vals"));

    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    int32_t* slot = nullptr;
    TRY(noalloc_setup(dev, &slot));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    TRY(validate_rows(desc, rows, s));     // checked build only

    // the map keeps the previous call's contents: every row starts again at "no slot" (-1)
    CUDA_TRY(cudaMemsetAsync(slot, 0xFF, (size_t)rows * 4, s));
    if (have_rows) {
        SlotBatch sb{};
        sb.slot[0] = slot;
        sb.row_idx[0] = desc->row_idx;
        sb.n_rows[0] = desc->n_rows;
        scatter_slots_kernel<<<dim3((desc->n_rows + 255) / 256, 1), 256, 0, s>>>(sb, rows);
    }
    BatchPtrs gp{};
    gp.dense[0] = desc->dense;
    gp.row_vals[0] = desc->row_vals;
    gp.slot[0] = slot;
    gp.n_rows[0] = have_rows ? desc->n_rows : 0;
    SparseSeg seg{seg_offset / 8, (seg_offset + rows * cols) / 8, (int32_t)(cols / 8)};
    const StepParams p{-lr, momentum, weight_decay};
    const bool mom = momentum != 0.f, wd = weight_decay != 0.f, bf = grad_dtype == HPSGD_BF16;
    const int64_t nvec = n_elems / 8;
#define HPSGD_NOALLOC_CASE(B, M, W) noalloc_launch<B, M, W>(s, replica, momentum_buf, gp, seg, nvec, p)
    if (bf) {
        if (mom && wd) HPSGD_NOALLOC_CASE(true, true, true);
        else if (mom) HPSGD_NOALLOC_CASE(true, true, false);
        else if (wd) HPSGD_NOALLOC_CASE(true, false, true);
        else HPSGD_NOALLOC_CASE(true, false, false);
    } else {
        if (mom && wd) HPSGD_NOALLOC_CASE(false, true, true);
        else if (mom) HPSGD_NOALLOC_CASE(false, true, false);
        else if (wd) HPSGD_NOALLOC_CASE(false, false, true);
        else HPSGD_NOALLOC_CASE(false, false, false);
    }
#undef HPSGD_NOALLOC_CASE
    return check_async();
}
