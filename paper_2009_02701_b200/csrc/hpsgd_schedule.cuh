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

// Lazy clones (HPSGD_OPT_FUSE = 2): a merge does not write the K re-cloned replicas; a replica
// that nothing has stepped since is read from w.  Needs one pointer per worker in the launch.
bool lazy_clones()
{
    return g.fuse == 2 && g.form == HPSGD_FORM_REPLICA_CHANGE && !g.pipeline && g.K <= kMaxBatch;
}

// Where replica i is read from (not for the pipelined schedule, which keeps its own books).
const float* replica_src(int i)
{
    return g.row_valid[i] ? g.r + (int64_t)i * g.stride : g.w;
}

// Write the rows of replicas that are lazy clones (r_i = w), for a schedule that reads rows.
int materialize_clones()
{
    bool any = false;
    for (int i = 0; i < g.K; ++i) any = any || !g.row_valid[i];
    if (!any) return HPSGD_OK;
    for (int c = 0; c < g.chunks; ++c)
        if (g.merge_unwaited[c]) {             // w is last written by a merge on the side stream
            CUDA_TRY(cudaStreamWaitEvent(g.main, g.ev_merge[c], 0));
            g.merge_unwaited[c] = 0;
        }
    for (int i = 0; i < g.K; ++i) {
        if (g.row_valid[i]) continue;
        CUDA_TRY(cudaMemcpyAsync(g.r + (int64_t)i * g.stride, g.w, (size_t)g.P_pad * 4, cudaMemcpyDeviceToDevice, g.main));
        g.row_valid[i] = 1;
    }
    if (g.overlap)
        for (int c = 0; c < g.chunks; ++c) {
            CUDA_TRY(cudaEventRecord(g.ev_local[c], g.main));
            g.local_recorded[c] = 1;
        }
    return HPSGD_OK;
}

SparseSeg sparse_seg(bool sparse)
{
    SparseSeg seg{0, 0, 1};
    if (sparse) {
        seg.o_begin = g.offsets[g.sp_tensor] / 8;
        seg.o_end = seg.o_begin + g.sp_rows * g.sp_cols / 8;
        seg.cols8 = (int32_t)(g.sp_cols / 8);
    }
    return seg;
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
                                                                               L.seg, L.o0, L.n, L.p, group_limit());
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
#define HPSGD_ACCUM_CASE(B, S)                                                                                  \
    accum_step_kernel<B, S><<<grid, kHotThreads, 0, g.main>>>(g.r, g.m, g.stride, L.w0, L.gp, L.seg, L.o0, L.n, \
                                                              L.p.neg_mu, group_limit())
    if (bf && sparse) HPSGD_ACCUM_CASE(true, true);
    else if (bf) HPSGD_ACCUM_CASE(true, false);
    else if (sparse) HPSGD_ACCUM_CASE(false, true);
    else HPSGD_ACCUM_CASE(false, false);
#undef HPSGD_ACCUM_CASE
}

// Enqueue the local step of workers [w0, w0 + nw) on the main stream, chunk by chunk.
int enqueue_local(int w0, int nw, const BatchPtrs& gp, bool sparse)
{
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
    } else {
        for (int i = 0; i < nw; ++i) {
            if (!g.row_valid[w0 + i]) L.gp.r_src[i] = g.w;      // a lazy clone: the step writes its row
            g.row_valid[w0 + i] = 1;
            g.at_w[w0 + i] = 0;
        }
    }
    L.p = StepParams{-g.lr, g.beta, g.lambda};
    L.seg = sparse_seg(sparse);
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
        gp->n_rows[i] = sb.n_rows[i];
        gp->row_vals[i] = d.row_vals;
        gp->dense[i] = d.dense;
    }
    if (most > 0) {
        scatter_slots_kernel<<<dim3((most + 255) / 256, nw), 256, 0, g.main>>>(sb, g.sp_rows);
        ++g.launches;
    }
    return HPSGD_OK;
}

// ---------------------------------------------------------------------------- merge
template <int KT>
void launch_merge(cudaStream_t s, int64_t o0, int64_t n, int flags)
{
    merge_kernel<KT><<<hot_grid(n), kHotThreads, 0, s>>>(g.w, g.D, g.r, g.stride, g.K, o0, n, flags, group_limit());
}

// The same merge with its tiles staged through shared memory by bulk-async copies (HPSGD_OPT_STAGING).
int launch_merge_staged(cudaStream_t s, int64_t o0, int64_t n, int flags)
{
    const size_t smem = (size_t)(g.K + 2) * kStageTileFloats * sizeof(float);
    if (!g.staged_attr) {
        CUDA_TRY(cudaFuncSetAttribute(merge_staged_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)((kMaxBatch + 2) * kStageTileFloats * sizeof(float))));
        g.staged_attr = true;
    }
    const int64_t tiles = (n + kStageGroups - 1) / kStageGroups;
    merge_staged_kernel<<<(unsigned)tiles, kHotThreads, smem, s>>>(g.w, g.D, g.r, g.stride, g.K, o0, n, flags, group_limit(),
                                                                   g.debug_stage_stall ? 16u : 0u);
    g.staged_ran = true;
    return HPSGD_OK;
}

bool staged_merge()
{
    return g.staging && g.form == HPSGD_FORM_REPLICA_CHANGE && !g.pipeline && !lazy_clones() && g.K <= kMaxBatch;
}

template <int KT>
void launch_merge_lazy(cudaStream_t s, const ReducePtrs& rp, int64_t o0, int64_t n, int flags)
{
    merge_lazy_kernel<KT><<<hot_grid(n), kHotThreads, 0, s>>>(g.w, g.D, rp, g.K, o0, n, flags, group_limit());
}

template <int KT>
void launch_accum_merge(cudaStream_t s, int64_t o0, int64_t n, int flags)
{
    accum_merge_kernel<KT><<<hot_grid(n), kHotThreads, 0, s>>>(g.w, g.D, g.r, g.m, g.stride, g.K, o0, n, flags, -g.lr,
                                                               group_limit());
}

// Enqueue one merge, chunk by chunk, on the side stream (main stream without overlap).
int enqueue_merge(int flags)
{
    cudaStream_t s = g.overlap ? g.side : g.main;
    TRY(wait_pending_d2h(s));
    const bool lazy = lazy_clones();
    ReducePtrs rp{};
    if (lazy)
        for (int i = 0; i < g.K; ++i) rp.src[i] = replica_src(i);
    for (int c = 0; c < g.chunks; ++c) {
        int64_t lo, hi;
        chunk_range(c, &lo, &hi);
        if (hi <= lo) continue;
        if (g.overlap && g.local_recorded[c]) {
            CUDA_TRY(cudaStreamWaitEvent(s, g.ev_local[c], 0));
            g.local_recorded[c] = 0;
        }
        EventPair ep{};
        TRY(prof_begin(s, (!lazy && staged_merge()) ? HPSGD_KERNEL_MERGE_STAGED : HPSGD_KERNEL_MERGE, &ep));
        if (g.form == HPSGD_FORM_GRADIENT_ACCUMULATION) {
            switch (g.K) {
            case 1: launch_accum_merge<1>(s, lo, hi - lo, flags); break;
            case 2: launch_accum_merge<2>(s, lo, hi - lo, flags); break;
            case 3: launch_accum_merge<3>(s, lo, hi - lo, flags); break;
            case 4: launch_accum_merge<4>(s, lo, hi - lo, flags); break;
            case 5: launch_accum_merge<5>(s, lo, hi - lo, flags); break;
            case 6: launch_accum_merge<6>(s, lo, hi - lo, flags); break;
            case 7: launch_accum_merge<7>(s, lo, hi - lo, flags); break;
            case 8: launch_accum_merge<8>(s, lo, hi - lo, flags); break;
            case 16: launch_accum_merge<16>(s, lo, hi - lo, flags); break;
            default: launch_accum_merge<0>(s, lo, hi - lo, flags); break;
            }
        } else if (lazy) {
            // K up to 8 and K = 16 have instantiations of their own: with few workers the any-K form
            // (built for many: two blocks per SM, eight loads at a time) keeps too little in flight
            switch (g.K) {
            case 1: launch_merge_lazy<1>(s, rp, lo, hi - lo, flags); break;
            case 2: launch_merge_lazy<2>(s, rp, lo, hi - lo, flags); break;
            case 3: launch_merge_lazy<3>(s, rp, lo, hi - lo, flags); break;
            case 4: launch_merge_lazy<4>(s, rp, lo, hi - lo, flags); break;
            case 5: launch_merge_lazy<5>(s, rp, lo, hi - lo, flags); break;
            case 6: launch_merge_lazy<6>(s, rp, lo, hi - lo, flags); break;
            case 7: launch_merge_lazy<7>(s, rp, lo, hi - lo, flags); break;
            case 8: launch_merge_lazy<8>(s, rp, lo, hi - lo, flags); break;
            case 16: launch_merge_lazy<16>(s, rp, lo, hi - lo, flags); break;
            default: launch_merge_lazy<0>(s, rp, lo, hi - lo, flags); break;
            }
        } else if (staged_merge()) {
            TRY(launch_merge_staged(s, lo, hi - lo, flags));
        } else {
            switch (g.K) {
            case 1: launch_merge<1>(s, lo, hi - lo, flags); break;
            case 2: launch_merge<2>(s, lo, hi - lo, flags); break;
            case 3: launch_merge<3>(s, lo, hi - lo, flags); break;
            case 4: launch_merge<4>(s, lo, hi - lo, flags); break;
            case 5: launch_merge<5>(s, lo, hi - lo, flags); break;
            case 6: launch_merge<6>(s, lo, hi - lo, flags); break;
            case 7: launch_merge<7>(s, lo, hi - lo, flags); break;
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
    std::fill(g.at_w.begin(), g.at_w.end(), 1);
    std::fill(g.row_valid.begin(), g.row_valid.end(), lazy ? 0 : 1);
    return check_async();
}

template <int KT>
void launch_reduce(const float* w_old, const ReducePtrs& rp, int64_t n)
{
    reduce_kernel<KT><<<hot_grid(n), kHotThreads, 0, g.side>>>(w_old, g.D, rp, g.K, n, group_limit());
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
    commit_kernel<<<hot_grid(n), kHotThreads, 0, g.main>>>(g.wbuf[g.cur], g.D, g.wbuf[nxt], n, flags, group_limit());
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
    case 1: launch_reduce<1>(g.wbuf[g.cur], rp, n); break;
    case 2: launch_reduce<2>(g.wbuf[g.cur], rp, n); break;
    case 3: launch_reduce<3>(g.wbuf[g.cur], rp, n); break;
    case 4: launch_reduce<4>(g.wbuf[g.cur], rp, n); break;
    case 5: launch_reduce<5>(g.wbuf[g.cur], rp, n); break;
    case 6: launch_reduce<6>(g.wbuf[g.cur], rp, n); break;
    case 7: launch_reduce<7>(g.wbuf[g.cur], rp, n); break;
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

// Work that an earlier call held back (HPSGD_OPT_FUSE) and that nothing has absorbed: a merge
// (fuse 1) runs on its own, local steps (fuse 2) run as ordinary local steps.
int flush_deferred()
{
    if (g.merge_deferred) {
        g.merge_deferred = false;
        TRY(enqueue_merge(g.deferred_flags));
    }
    if (g.steps_held) {
        // every maximal run of consecutive workers with a held step is one batched launch
        const BatchPtrs all = g.deferred_gp;
        const std::vector<char> held = g.step_held;
        g.steps_held = 0;
        std::fill(g.step_held.begin(), g.step_held.end(), 0);
        for (int a = 0; a < g.K;) {
            if (!held[a]) { ++a; continue; }
            int b = a;
            BatchPtrs gp{};
            for (; b < g.K && held[b]; ++b) {
                gp.dense[b - a] = all.dense[b];
                gp.row_vals[b - a] = all.row_vals[b];
                gp.slot[b - a] = all.slot[b];
                gp.n_rows[b - a] = all.n_rows[b];
            }
            TRY(enqueue_local(a, b - a, gp, g.deferred_sparse));
            a = b;
        }
    }
    return HPSGD_OK;
}

// Hold the local step of `worker` back (fuse 2).  A worker holds at most one step, and the held
// steps are all dense or all sparse-row: anything else first launches what is held.
int hold_step(int worker, const BatchPtrs& gp, int src, bool sparse)
{
    if (g.steps_held && (g.step_held[worker] || g.deferred_sparse != sparse)) TRY(flush_deferred());
    if (!g.steps_held) {
        g.deferred_gp = BatchPtrs{};
        g.deferred_sparse = sparse;
    }
    g.deferred_gp.dense[worker] = gp.dense[src];
    g.deferred_gp.row_vals[worker] = gp.row_vals[src];
    g.deferred_gp.slot[worker] = gp.slot[src];
    g.deferred_gp.n_rows[worker] = gp.n_rows[src];
    g.step_held[worker] = 1;
    ++g.steps_held;
    return HPSGD_OK;
}

struct FusedLaunch {
    BatchPtrs gp;
    SparseSeg seg;
    int64_t o0, n;
    int flags;
    StepParams p;
};

// ---------------------------------------------------------------------------- fuse 1: merge + next local step
template <int KT, bool BF16, bool MOM, bool WD, bool SPARSE>
void launch_fused(const FusedLaunch& L)
{
    merge_step_kernel<KT, BF16, MOM, WD, SPARSE><<<hot_grid(L.n), kHotThreads, 0, g.main>>>(
        g.w, g.D, g.r, g.m, g.stride, g.K, L.gp, L.seg, L.o0, L.n, L.flags, L.p, group_limit());
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

// The deferred merge and the local step of all K workers in one kernel per chunk (main stream).
int enqueue_fused(const BatchPtrs& gp, bool sparse)
{
    TRY(wait_pending_d2h(g.main));
    FusedLaunch L{};
    L.gp = gp;
    L.flags = g.deferred_flags;
    L.p = StepParams{-g.lr, g.beta, g.lambda};
    L.seg = sparse_seg(sparse);
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
        if (g.grad_dtype == HPSGD_BF16) launch_fused_k<true>(mom, wd, sparse, L);
        else launch_fused_k<false>(mom, wd, sparse, L);
        ++g.launches;
        TRY(prof_end(g.main, &ep));
        if (g.overlap) {
            CUDA_TRY(cudaEventRecord(g.ev_local[c], g.main));
            g.local_recorded[c] = 1;
        }
    }
    std::fill(g.at_w.begin(), g.at_w.end(), 0);          // merged, re-cloned and stepped once
    return check_async();
}

// ---------------------------------------------------------------------------- fuse 2: local step + merge, one round
template <int B, bool BF16, bool MOM, bool WD, bool SPARSE, bool FROM_W>
void launch_round_b(const FusedLaunch& L)
{
    round_kernel<B, BF16, MOM, WD, SPARSE, FROM_W><<<hot_grid(L.n), kHotThreads, 0, g.main>>>(
        g.w, g.D, g.m, g.stride, g.K, L.gp, L.seg, L.o0, L.n, L.flags, L.p, group_limit());
}

template <int B, bool BF16, bool MOM, bool WD, bool SPARSE, bool FROM_W>
void launch_round_even(const FusedLaunch& L)
{
    round_kernel<B, BF16, MOM, WD, SPARSE, FROM_W, true><<<hot_grid(L.n), kHotThreads, 0, g.main>>>(
        g.w, g.D, g.m, g.stride, g.K, L.gp, L.seg, L.o0, L.n, L.flags, L.p, group_limit());
}

// The batch size is a template argument because it sizes the register arrays; which instantiation runs
// depends on K.
//   Without a sparse-row tensor: fewer workers than the largest batch holds use the instantiation for
//   exactly K workers - all their loads in flight at once in a single batch, and only the registers of
//   that batch, so more blocks are resident per SM (with the largest batch, K = 1..7 reached 4.0-6.0 TB/s
//   on large models: too little in flight per thread for the few blocks its registers allow).  Where the
//   largest batch divides K, full batches; otherwise batches of as equal a size as possible.
//   With a sparse-row tensor: at least two batches of at most four workers (round_batch_size says why).
template <bool BF16, bool MOM, bool WD, bool SPARSE, bool FROM_W>
void launch_round(const FusedLaunch& L)
{
    constexpr int B = round_batch_size(BF16, MOM, SPARSE, FROM_W);
    const int K = g.K;
    if constexpr (SPARSE) {
        static_assert(B == 4, "the cases below are written for batches of four");
        if (K >= 7) return K % 4 == 0 ? launch_round_b<4, BF16, MOM, WD, SPARSE, FROM_W>(L)
                                      : launch_round_even<4, BF16, MOM, WD, SPARSE, FROM_W>(L);
        switch (K) {                                   // two batches: ceil(K / 2) and the rest
        case 1: return launch_round_b<1, BF16, MOM, WD, SPARSE, FROM_W>(L);
        case 2: return launch_round_b<1, BF16, MOM, WD, SPARSE, FROM_W>(L);
        case 3: return launch_round_even<2, BF16, MOM, WD, SPARSE, FROM_W>(L);
        case 4: return launch_round_b<2, BF16, MOM, WD, SPARSE, FROM_W>(L);
        case 5: return launch_round_even<3, BF16, MOM, WD, SPARSE, FROM_W>(L);
        default: return launch_round_b<3, BF16, MOM, WD, SPARSE, FROM_W>(L);      // 6
        }
    } else {
        if constexpr (FROM_W) {
            switch (K) {
            case 1: return launch_round_b<1, BF16, MOM, WD, SPARSE, FROM_W>(L);
            case 2: return launch_round_b<2, BF16, MOM, WD, SPARSE, FROM_W>(L);
            case 3: return launch_round_b<3, BF16, MOM, WD, SPARSE, FROM_W>(L);
            case 4: return launch_round_b<4, BF16, MOM, WD, SPARSE, FROM_W>(L);
            case 5: return launch_round_b<5, BF16, MOM, WD, SPARSE, FROM_W>(L);
            case 6: return launch_round_b<6, BF16, MOM, WD, SPARSE, FROM_W>(L);
            case 7: return launch_round_b<7, BF16, MOM, WD, SPARSE, FROM_W>(L);
            default: break;
            }
        }
        if (K % B == 0) return launch_round_b<B, BF16, MOM, WD, SPARSE, FROM_W>(L);
        // at most 8 workers per batch in the evenly split form: with 16 the bf16 + momentum variants spill,
        // and the light variants, whose threads have little in flight anyway, gain more from the blocks
        // that fewer registers allow
        constexpr int BE = B == 16 ? 8 : B;
        launch_round_even<BE, BF16, MOM, WD, SPARSE, FROM_W>(L);
    }
}

template <bool BF16, bool MOM, bool WD>
void launch_round_s(bool sparse, bool from_w, const FusedLaunch& L)
{
    if (sparse) {
        if (from_w) launch_round<BF16, MOM, WD, true, true>(L);
        else launch_round<BF16, MOM, WD, true, false>(L);
    } else {
        if (from_w) launch_round<BF16, MOM, WD, false, true>(L);
        else launch_round<BF16, MOM, WD, false, false>(L);
    }
}

template <bool BF16>
void launch_round_d(bool mom, bool wd, bool sparse, bool from_w, const FusedLaunch& L)
{
    if (mom && wd) launch_round_s<BF16, true, true>(sparse, from_w, L);
    else if (mom) launch_round_s<BF16, true, false>(sparse, from_w, L);
    else if (wd) launch_round_s<BF16, false, true>(sparse, from_w, L);
    else launch_round_s<BF16, false, false>(sparse, from_w, L);
}

// The held-back local steps of all K workers and the merge that follows them in one kernel per
// chunk (main stream).  Afterwards every replica is a lazy clone of the new w.
int enqueue_round(int flags)
{
    TRY(wait_pending_d2h(g.main));
    g.steps_held = 0;
    std::fill(g.step_held.begin(), g.step_held.end(), 0);
    FusedLaunch L{};
    L.gp = g.deferred_gp;
    bool from_w = true;
    for (int i = 0; i < g.K; ++i) {
        from_w = from_w && g.at_w[i];
        L.gp.r_src[i] = replica_src(i);
    }
    L.flags = flags;
    L.p = StepParams{-g.lr, g.beta, g.lambda};
    L.seg = sparse_seg(g.deferred_sparse);
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
        TRY(prof_begin(g.main, HPSGD_KERNEL_ROUND, &ep));
        if (g.grad_dtype == HPSGD_BF16) launch_round_d<true>(mom, wd, g.deferred_sparse, from_w, L);
        else launch_round_d<false>(mom, wd, g.deferred_sparse, from_w, L);
        ++g.launches;
        TRY(prof_end(g.main, &ep));
        if (g.overlap) {
            CUDA_TRY(cudaEventRecord(g.ev_local[c], g.main));
            g.local_recorded[c] = 1;
        }
    }
    std::fill(g.at_w.begin(), g.at_w.end(), 1);
    std::fill(g.row_valid.begin(), g.row_valid.end(), 0);
    return check_async();
}

}  // namespace
