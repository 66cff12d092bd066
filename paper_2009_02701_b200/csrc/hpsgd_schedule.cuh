// Stream / event schedule of libhpsgd and the kernel launches behind it: local steps on the
// main stream, merges on the side stream, fused and pipelined variants.
// Included by hpsgd_api.cu only (one translation unit), after hpsgd_state.cuh.
#pragma once

#include "hpsgd_state.cuh"

namespace {

// A host copy of w started by hpsgd_copy_global_async must finish before the stream `s` overwrites w.
int wait_pending_d2h(cudaStream_t s)
{
    if (g.d2h_outstanding) CUDA_TRY(cudaStreamWaitEvent(s, g.ev_d2h_done, 0));
    return HPSGD_OK;
}

// Rebuild replica rows that the implicit-replica kernel left stale: r_i = fma(-mu, m_i, w).
int ensure_replicas()
{
    if (!g.replicas_stale) return HPSGD_OK;
    const int64_t n = g.P_pad / 8;
    dim3 grid(hot_grid(n), g.K);
    materialize_kernel<<<grid, kHotThreads, 0, g.main>>>(g.w, g.m, g.r, g.stride, n, -g.lr);
    ++g.launches;
    g.replicas_stale = false;
    if (g.overlap)
        for (int c = 0; c < g.chunks; ++c) {
            CUDA_TRY(cudaEventRecord(g.ev_local[c], g.main));
            g.local_recorded[c] = 1;
        }
    return check_async();
}

// ---------------------------------------------------------------------------- local step
struct LocalLaunch {
    int w0, nw;
    BatchPtrs gp;
    SparseSeg seg;
    int64_t o0, n;
    StepParams p;
};

template <bool BF16, bool MOM, bool WD, bool SPARSE>
void launch_local(const LocalLaunch& L)
{
    dim3 grid(hot_grid(L.n), L.nw);
    local_step_kernel<BF16, MOM, WD, SPARSE><<<grid, kHotThreads, 0, g.main>>>(g.r, g.m, g.stride, L.w0, L.gp,
                                                                               L.seg, L.o0, L.n, L.p);
}

template <bool BF16, bool MOM, bool WD>
void launch_local_s(bool sparse, const LocalLaunch& L)
{
    if (sparse) launch_local<BF16, MOM, WD, true>(L);
    else launch_local<BF16, MOM, WD, false>(L);
}

template <bool BF16>
void launch_local_d(bool mom, bool wd, bool sparse, const LocalLaunch& L)
{
    if (mom && wd) launch_local_s<BF16, true, true>(sparse, L);
    else if (mom) launch_local_s<BF16, true, false>(sparse, L);
    else if (wd) launch_local_s<BF16, false, true>(sparse, L);
    else launch_local_s<BF16, false, false>(sparse, L);
}

// Gradient-accumulation form: r -= mu*g, a += g (the accumulators live where momentum would).
void launch_accum_step(bool sparse, const LocalLaunch& L)
{
    dim3 grid(hot_grid(L.n), L.nw);
    const bool bf = g.grad_dtype == HPSGD_BF16;
#define HPSGD_ACCUM_CASE(B, S) \
    accum_step_kernel<B, S><<<grid, kHotThreads, 0, g.main>>>(g.r, g.m, g.stride, L.w0, L.gp, L.seg, L.o0, L.n, L.p.neg_mu)
    if (bf && sparse) HPSGD_ACCUM_CASE(true, true);
    else if (bf) HPSGD_ACCUM_CASE(true, false);
    else if (sparse) HPSGD_ACCUM_CASE(false, true);
    else HPSGD_ACCUM_CASE(false, false);
#undef HPSGD_ACCUM_CASE
}

// Enqueue the local step of workers [w0, w0 + nw) on the main stream, chunk by chunk.
int enqueue_local(int w0, int nw, const BatchPtrs& gp, bool sparse)
{
    TRY(ensure_replicas());
    for (int i = 0; i < nw; ++i) g.steps_in_period[w0 + i] += 1;
    LocalLaunch L{};
    L.w0 = w0; L.nw = nw; L.gp = gp;
    if (g.pipeline) {
        // first step of a worker in this period: its replica is still the clone, i.e. w itself
        for (int i = 0; i < nw; ++i) {
            if (!g.touched[w0 + i]) {
                L.gp.r_src[i] = g.w;
                g.touched[w0 + i] = 1;
            }
        }
    }
    L.p = StepParams{-g.lr, g.beta, g.lambda};
    L.seg = SparseSeg{0, 0, 1};
    if (sparse) {
        L.seg.o_begin = g.offsets[g.sp_tensor] / 8;
        L.seg.o_end = L.seg.o_begin + g.sp_rows * g.sp_cols / 8;
        L.seg.cols8 = (int32_t)(g.sp_cols / 8);
    }
    const bool mom = g.beta != 0.f, wd = g.lambda != 0.f;
    for (int c = 0; c < g.chunks; ++c) {
        int64_t lo, hi;
        chunk_range(c, &lo, &hi);
        if (hi <= lo) continue;
        if (g.merge_unwaited[c]) {
            CUDA_TRY(cudaStreamWaitEvent(g.main, g.ev_merge[c], 0));
            g.merge_unwaited[c] = 0;
        }
        L.o0 = lo; L.n = hi - lo;
        EventPair ep{};
        TRY(prof_begin(g.main, HPSGD_KERNEL_LOCAL_STEP, &ep));
        if (g.form == HPSGD_FORM_GRADIENT_ACCUMULATION) launch_accum_step(sparse, L);
        else if (g.grad_dtype == HPSGD_BF16) launch_local_d<true>(mom, wd, sparse, L);
        else launch_local_d<false>(mom, wd, sparse, L);
        ++g.launches;
        TRY(prof_end(g.main, &ep));
        if (g.overlap) {
            CUDA_TRY(cudaEventRecord(g.ev_local[c], g.main));
            g.local_recorded[c] = 1;
        }
    }
    return check_async();
}

// Build the row -> slot maps of workers [w0, w0 + nw) from their descriptors: one (strided)
// memset over the nw maps (every row: no slot, -1) and one scatter launch for all of them.
int enqueue_slot_maps(int w0, int nw, const hpsgd_grad_desc* descs, BatchPtrs* gp)
{
    int32_t* first = g.slot + (int64_t)w0 * g.slot_cap;
    // only the rows in use are reset: the maps are slot_cap entries apart, which can be far more
    CUDA_TRY(cudaMemset2DAsync(first, (size_t)g.slot_cap * 4, 0xFF, (size_t)g.sp_rows * 4, nw, g.main));
    SlotBatch sb{};
    int32_t most = 0;
    for (int i = 0; i < nw; ++i) {
        const hpsgd_grad_desc& d = descs[i];
        sb.slot[i] = first + (int64_t)i * g.slot_cap;
        sb.row_idx[i] = d.row_idx;
        sb.n_rows[i] = (d.row_idx && d.n_rows > 0) ? d.n_rows : 0;
        most = std::max(most, sb.n_rows[i]);
        gp->slot[i] = sb.slot[i];
        gp->row_vals[i] = d.row_vals;
        gp->dense[i] = d.dense;
    }
    if (most > 0) {
        scatter_slots_kernel<<<dim3((most + 255) / 256, nw), 256, 0, g.main>>>(sb, g.sp_rows);
        ++g.launches;
    }
    return HPSGD_OK;
}

template <int KT>
void launch_merge(cudaStream_t s, int64_t o0, int64_t n, int flags)
{
    merge_kernel<KT><<<hot_grid(n), kHotThreads, 0, s>>>(g.w, g.D, g.r, g.stride, g.K, o0, n, flags);
}

template <int KT>
void launch_accum_merge(cudaStream_t s, int64_t o0, int64_t n, int flags)
{
    accum_merge_kernel<KT><<<hot_grid(n), kHotThreads, 0, s>>>(g.w, g.D, g.r, g.m, g.stride, g.K, o0, n, flags, -g.lr);
}

// Enqueue one merge, chunk by chunk, on the side stream (main stream without overlap).
int enqueue_merge(int flags)
{
    TRY(ensure_replicas());
    cudaStream_t s = g.overlap ? g.side : g.main;
    TRY(wait_pending_d2h(s));
    for (int c = 0; c < g.chunks; ++c) {
        int64_t lo, hi;
        chunk_range(c, &lo, &hi);
        if (hi <= lo) continue;
        if (g.overlap && g.local_recorded[c]) {
            CUDA_TRY(cudaStreamWaitEvent(s, g.ev_local[c], 0));
            g.local_recorded[c] = 0;
        }
        EventPair ep{};
        TRY(prof_begin(s, HPSGD_KERNEL_MERGE, &ep));
        if (g.form == HPSGD_FORM_GRADIENT_ACCUMULATION) {
            switch (g.K) {
            case 4: launch_accum_merge<4>(s, lo, hi - lo, flags); break;
            case 8: launch_accum_merge<8>(s, lo, hi - lo, flags); break;
            case 16: launch_accum_merge<16>(s, lo, hi - lo, flags); break;
            default: launch_accum_merge<0>(s, lo, hi - lo, flags); break;
            }
        } else {
            switch (g.K) {
            case 4: launch_merge<4>(s, lo, hi - lo, flags); break;
            case 8: launch_merge<8>(s, lo, hi - lo, flags); break;
            case 16: launch_merge<16>(s, lo, hi - lo, flags); break;
            default: launch_merge<0>(s, lo, hi - lo, flags); break;
            }
        }
        ++g.launches;
        TRY(prof_end(s, &ep));
        if (g.overlap) {
            CUDA_TRY(cudaEventRecord(g.ev_merge[c], s));
            g.merge_unwaited[c] = 1;
        }
    }
    return check_async();
}

template <int KT>
void launch_reduce(const float* w_old, const ReducePtrs& rp, int64_t n)
{
    reduce_kernel<KT><<<hot_grid(n), kHotThreads, 0, g.side>>>(w_old, g.D, rp, g.K, n);
}

// Pipelined synchronisation: the commit w_next = w + D runs on the main stream, in order with
// the local steps; the K-way reduce of the period that just ended runs on the side stream and
// nothing on the main stream waits for it until the NEXT synchronisation needs its result.
int enqueue_pipelined_merge(int flags)
{
    const int64_t n = g.P_pad / 8;
    const int nxt = g.cur ^ 1;
    TRY(wait_pending_d2h(g.main));
    if (g.reduce_outstanding) {
        // the previous reduce still reads the buffers about to be written and produces the D read here
        CUDA_TRY(cudaStreamWaitEvent(g.main, g.ev_reduce, 0));
        g.reduce_outstanding = false;
    }
    EventPair ep{};
    TRY(prof_begin(g.main, HPSGD_KERNEL_MERGE, &ep));
    commit_kernel<<<hot_grid(n), kHotThreads, 0, g.main>>>(g.wbuf[g.cur], g.D, g.wbuf[nxt], n, flags);
    ++g.launches;
    TRY(prof_end(g.main, &ep));
    CUDA_TRY(cudaEventRecord(g.ev_commit, g.main));
    CUDA_TRY(cudaStreamWaitEvent(g.side, g.ev_commit, 0));
    ReducePtrs rp{};
    for (int i = 0; i < g.K; ++i)
        rp.src[i] = g.touched[i] ? g.rbuf[g.cur] + (int64_t)i * g.stride : g.wbuf[g.cur];
    EventPair ep2{};
    TRY(prof_begin(g.side, HPSGD_KERNEL_MERGE, &ep2));
    switch (g.K) {
    case 4: launch_reduce<4>(g.wbuf[g.cur], rp, n); break;
    case 8: launch_reduce<8>(g.wbuf[g.cur], rp, n); break;
    case 16: launch_reduce<16>(g.wbuf[g.cur], rp, n); break;
    default: launch_reduce<0>(g.wbuf[g.cur], rp, n); break;
    }
    ++g.launches;
    TRY(prof_end(g.side, &ep2));
    CUDA_TRY(cudaEventRecord(g.ev_reduce, g.side));
    g.reduce_outstanding = true;
    g.cur = nxt;
    g.w = g.wbuf[nxt];
    g.r = g.rbuf[nxt];
    std::fill(g.touched.begin(), g.touched.end(), 0);
    return check_async();
}

// A merge that hpsgd_sync_merge deferred (fuse option) and that nothing has absorbed yet.
int flush_deferred()
{
    if (!g.merge_deferred) return HPSGD_OK;
    g.merge_deferred = false;
    return enqueue_merge(g.deferred_flags);
}

struct FusedLaunch {
    BatchPtrs gp;
    SparseSeg seg;
    int64_t o0, n;
    int flags;
    StepParams p;
};

template <int KT, bool BF16, bool MOM, bool WD, bool SPARSE>
void launch_fused(const FusedLaunch& L)
{
    merge_step_kernel<KT, BF16, MOM, WD, SPARSE><<<hot_grid(L.n), kHotThreads, 0, g.main>>>(
        g.w, g.D, g.r, g.m, g.stride, g.K, L.gp, L.seg, L.o0, L.n, L.flags, L.p);
}

template <int KT, bool BF16>
void launch_fused_d(bool mom, bool wd, bool sparse, const FusedLaunch& L)
{
#define HPSGD_FUSED_CASE(M, W)                                    \
    do {                                                          \
        if (sparse) launch_fused<KT, BF16, M, W, true>(L);        \
        else launch_fused<KT, BF16, M, W, false>(L);              \
    } while (0)
    if (mom && wd) HPSGD_FUSED_CASE(true, true);
    else if (mom) HPSGD_FUSED_CASE(true, false);
    else if (wd) HPSGD_FUSED_CASE(false, true);
    else HPSGD_FUSED_CASE(false, false);
#undef HPSGD_FUSED_CASE
}

template <bool BF16>
void launch_fused_k(bool mom, bool wd, bool sparse, const FusedLaunch& L)
{
    switch (g.K) {
    case 4: launch_fused_d<4, BF16>(mom, wd, sparse, L); break;
    case 8: launch_fused_d<8, BF16>(mom, wd, sparse, L); break;
    case 16: launch_fused_d<16, BF16>(mom, wd, sparse, L); break;
    default: launch_fused_d<0, BF16>(mom, wd, sparse, L); break;
    }
}

template <int KT>
void launch_implicit(bool sparse, const FusedLaunch& L)
{
    const bool bf = g.grad_dtype == HPSGD_BF16, wd = g.lambda != 0.f;
#define HPSGD_IMPLICIT_CASE(B, W, S)                                                                     \
    merge_step_implicit_kernel<KT, B, W, S><<<hot_grid(L.n), kHotThreads, 0, g.main>>>(                \
        g.w, g.D, g.m, g.stride, L.gp, L.seg, L.o0, L.n, L.flags, L.p)
    if (bf) {
        if (wd) { if (sparse) HPSGD_IMPLICIT_CASE(true, true, true); else HPSGD_IMPLICIT_CASE(true, true, false); }
        else { if (sparse) HPSGD_IMPLICIT_CASE(true, false, true); else HPSGD_IMPLICIT_CASE(true, false, false); }
    } else {
        if (wd) { if (sparse) HPSGD_IMPLICIT_CASE(false, true, true); else HPSGD_IMPLICIT_CASE(false, true, false); }
        else { if (sparse) HPSGD_IMPLICIT_CASE(false, false, true); else HPSGD_IMPLICIT_CASE(false, false, false); }
    }
#undef HPSGD_IMPLICIT_CASE
}

// Can the deferred merge and the coming batched step run with the replicas left implicit?
bool implicit_ok()
{
    return g.fuse == 2 && g.deferred_all_single && g.beta != 0.f && (g.K == 4 || g.K == 8 || g.K == 16);
}

// The deferred merge and the local step of all K workers in one kernel per chunk (main stream).
int enqueue_fused(const BatchPtrs& gp, bool sparse)
{
    const bool implicit = implicit_ok();
    if (!implicit) TRY(ensure_replicas());
    TRY(wait_pending_d2h(g.main));
    for (int i = 0; i < g.K; ++i) g.steps_in_period[i] += 1;
    FusedLaunch L{};
    L.gp = gp;
    L.flags = g.deferred_flags;
    L.p = StepParams{-g.lr, g.beta, g.lambda};
    L.seg = SparseSeg{0, 0, 1};
    if (sparse) {
        L.seg.o_begin = g.offsets[g.sp_tensor] / 8;
        L.seg.o_end = L.seg.o_begin + g.sp_rows * g.sp_cols / 8;
        L.seg.cols8 = (int32_t)(g.sp_cols / 8);
    }
    g.merge_deferred = false;
    const bool mom = g.beta != 0.f, wd = g.lambda != 0.f;
    for (int c = 0; c < g.chunks; ++c) {
        int64_t lo, hi;
        chunk_range(c, &lo, &hi);
        if (hi <= lo) continue;
        if (g.merge_unwaited[c]) {
            CUDA_TRY(cudaStreamWaitEvent(g.main, g.ev_merge[c], 0));
            g.merge_unwaited[c] = 0;
        }
        L.o0 = lo; L.n = hi - lo;
        EventPair ep{};
        TRY(prof_begin(g.main, HPSGD_KERNEL_MERGE_STEP, &ep));
        if (implicit) {
            switch (g.K) {
            case 4: launch_implicit<4>(sparse, L); break;
            case 8: launch_implicit<8>(sparse, L); break;
            default: launch_implicit<16>(sparse, L); break;
            }
        } else if (g.grad_dtype == HPSGD_BF16) launch_fused_k<true>(mom, wd, sparse, L);
        else launch_fused_k<false>(mom, wd, sparse, L);
        ++g.launches;
        TRY(prof_end(g.main, &ep));
        if (g.overlap) {
            CUDA_TRY(cudaEventRecord(g.ev_local[c], g.main));
            g.local_recorded[c] = 1;
        }
    }
    g.replicas_stale = implicit;
    return check_async();
}

}  // namespace
