// Device code of libhpsgd (sm_100a): replica update, K-way delayed merge, input generators.
//
// Every kernel is element-wise over the flat padded buffers and HBM-bound, so the work
// is organised around memory traffic: 256-bit coalesced accesses (one 8-element group per
// thread per array), all loads of a thread requested before their first use, and grids of
// many short blocks that the hardware scheduler hands to SMs as they free up (measured
// ~10 % faster on B200 than a persistent grid of SM-count x residency blocks, whose
// statically assigned shares finish at different times on the two dies).  No tensor
// cores: there is no contraction anywhere on this path.
//
// Arithmetic is written with explicit round-to-nearest intrinsics (__fmaf_rn, __fadd_rn,
// __fsub_rn, __fdiv_rn) so that the compiler can neither fuse nor split an operation:
// the result is the one IEEE-754 binary32 value the definition in hpsgd.h gives.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

namespace hpsgd {

constexpr int kThreads = 256;      // support kernels (generators, clone)
constexpr int kHotThreads = 128;   // local step and merge: one 8-element group per thread

// ---------------------------------------------------------------------------- checked build
// Compiled with -DHPSGD_DEBUG every hot kernel tests the group index it is about to touch
// against the number of groups of a flat buffer (and a row -> slot entry against the number
// of rows it may name) before any access.  A violation is recorded in g_debug_report (first
// one wins) and that group is skipped: nothing traps, nothing waits, the context stays
// usable, and the host turns the record into an error at its next synchronisation.  In the
// normal build the guards compile to nothing.
enum KernelId { kIdLocalStep = 1, kIdMerge, kIdMergeLazy, kIdMergeStep, kIdRound, kIdCommit, kIdReduce,
                kIdAccumStep, kIdAccumMerge, kIdScatter };

#ifdef HPSGD_DEBUG
struct DebugReport {
    int code;            // 0: nothing recorded; 1: group index out of range; 2: slot out of range; 3: row out of range
    int kernel;          // KernelId
    long long index;     // the offending group / slot / row
    long long limit;     // what it was tested against
};
__device__ DebugReport g_debug_report;

__device__ __forceinline__ bool debug_check(bool ok, int code, int kernel, long long index, long long limit)
{
    if (ok) return true;
    if (atomicCAS(&g_debug_report.code, 0, code) == 0) {
        g_debug_report.kernel = kernel;
        g_debug_report.index = index;
        g_debug_report.limit = limit;
    }
    return false;
}
#define HPSGD_GUARD_GROUP(o, limit, kernel) \
    if (!hpsgd::debug_check((o) >= 0 && (o) < (limit), 1, (kernel), (long long)(o), (long long)(limit))) continue
#define HPSGD_SLOT_OK(s, n_rows, kernel) hpsgd::debug_check((s) < (n_rows), 2, (kernel), (long long)(s), (long long)(n_rows))
#define HPSGD_ROW_OK(row, rows, kernel) hpsgd::debug_check((row) >= 0 && (row) < (rows), 3, (kernel), (long long)(row), (long long)(rows))
#else
#define HPSGD_GUARD_GROUP(o, limit, kernel) do { } while (0)
#define HPSGD_SLOT_OK(s, n_rows, kernel) true
#define HPSGD_ROW_OK(row, rows, kernel) ((row) >= 0 && (row) < (rows))
#endif

// ---------------------------------------------------------------------------- memory ops
// The hot kernels move 8 consecutive fp32 values (32 bytes) per thread with the 256-bit
// global loads/stores of sm_100 (ld/st.global.v8.b32); addresses are 32-byte aligned.
struct f8 {
    float v[8];
};

__device__ __forceinline__ f8 ld8(const float* p)
{
    f8 x;
    asm volatile("ld.global.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(x.v[0]), "=f"(x.v[1]), "=f"(x.v[2]), "=f"(x.v[3]),
                   "=f"(x.v[4]), "=f"(x.v[5]), "=f"(x.v[6]), "=f"(x.v[7])
                 : "l"(p));
    return x;
}

__device__ __forceinline__ void st8(float* p, const f8& x)
{
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "l"(p), "f"(x.v[0]), "f"(x.v[1]), "f"(x.v[2]), "f"(x.v[3]),
                    "f"(x.v[4]), "f"(x.v[5]), "f"(x.v[6]), "f"(x.v[7])
                 : "memory");
}

__device__ __forceinline__ f8 zero8()
{
    f8 x;
#pragma unroll
    for (int q = 0; q < 8; ++q) x.v[q] = 0.f;
    return x;
}

// Eight consecutive gradient values of group o (o counts groups of 8 elements), as stored:
// 32 bytes of fp32 or 16 bytes of bf16.  Loading and widening are separate steps so that a
// thread can request several groups before it touches the first one.
template <bool BF16>
struct GradRaw;
template <>
struct GradRaw<false> {
    f8 x;
};
template <>
struct GradRaw<true> {
    uint4 u;
};

template <bool BF16>
__device__ __forceinline__ GradRaw<BF16> load_grad_raw(const void* g, int64_t o)
{
    GradRaw<BF16> raw;
    if constexpr (BF16) {
        asm volatile("ld.global.v4.b32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(raw.u.x), "=r"(raw.u.y), "=r"(raw.u.z), "=r"(raw.u.w)
                     : "l"(reinterpret_cast<const uint4*>(g) + o));
    } else {
        raw.x = ld8(reinterpret_cast<const float*>(g) + o * 8);
    }
    return raw;
}

template <bool BF16>
__device__ __forceinline__ GradRaw<BF16> zero_grad_raw()
{
    GradRaw<BF16> raw;
    if constexpr (BF16) raw.u = make_uint4(0u, 0u, 0u, 0u);
    else raw.x = zero8();
    return raw;
}

// bf16 -> fp32 is exact: the 16 stored bits become the upper half of the binary32 pattern.
template <bool BF16>
__device__ __forceinline__ f8 widen_grad(const GradRaw<BF16>& raw)
{
    if constexpr (BF16) {
        f8 x;
        x.v[0] = __uint_as_float(raw.u.x << 16); x.v[1] = __uint_as_float(raw.u.x & 0xFFFF0000u);
        x.v[2] = __uint_as_float(raw.u.y << 16); x.v[3] = __uint_as_float(raw.u.y & 0xFFFF0000u);
        x.v[4] = __uint_as_float(raw.u.z << 16); x.v[5] = __uint_as_float(raw.u.z & 0xFFFF0000u);
        x.v[6] = __uint_as_float(raw.u.w << 16); x.v[7] = __uint_as_float(raw.u.w & 0xFFFF0000u);
        return x;
    } else {
        return raw.x;
    }
}

template <bool BF16>
__device__ __forceinline__ f8 load_grad8(const void* g, int64_t o)
{
    return widen_grad<BF16>(load_grad_raw<BF16>(g, o));
}

// ---------------------------------------------------------------------------- local step
// Algorithm 2, "update replica", with the momentum / weight-decay extension:
//   gd = g + lambda*r ; m = beta*m + gd ; r = r - mu*m      (one FMA each)
struct StepParams {
    float neg_mu;
    float beta;
    float lambda;
};

template <bool MOM, bool WD>
__device__ __forceinline__ float step1(float g, float& m, float r, const StepParams& p)
{
    float gd = WD ? __fmaf_rn(p.lambda, r, g) : g;
    float mn = MOM ? __fmaf_rn(p.beta, m, gd) : gd;
    if (MOM) m = mn;
    return __fmaf_rn(p.neg_mu, mn, r);
}

// Sparse-row tensor inside the flat buffer: groups [o_begin, o_end) form a
// [rows x cols] tensor whose gradient comes from row_vals through the row->slot map.
struct SparseSeg {
    int64_t o_begin;       // first group of the tensor (element offset / 8)
    int64_t o_end;         // one past its last group
    int32_t cols8;         // cols / 8
};

constexpr int kMaxBatch = 32;   // most workers one batched launch can address

// Per-worker pointers of a batched launch (blockIdx.y selects the worker).
struct BatchPtrs {
    const void* dense[kMaxBatch];
    const void* row_vals[kMaxBatch];
    const int32_t* slot[kMaxBatch];
    int32_t n_rows[kMaxBatch];       // rows listed for the sparse-row tensor (what a slot may name)
    const float* r_src[kMaxBatch];   // where the worker's replica is READ from; NULL: its own row.
                                     // (a replica that is still the clone of the global model is
                                     // read from w itself when its row has not been written)
};

// One worker per blockIdx.y; workers' replicas/momenta are `stride` floats apart starting
// at worker index w0.  Groups [o0, o0 + n) are processed, one group of 8 elements per
// thread.  The grid normally has one block per 128 groups (no persistent loop: on this
// part many short blocks, handed out by the hardware scheduler as SMs free up, stream
// about 10 % faster than one resident wave striding through memory); the loop only
// matters when n exceeds what a grid can index.
template <bool BF16, bool MOM, bool WD, bool SPARSE>
__global__ void __launch_bounds__(kHotThreads, 8)
local_step_kernel(float* __restrict__ r_base, float* __restrict__ m_base, int64_t stride,
                  int w0, BatchPtrs gp, SparseSeg seg, int64_t o0, int64_t n, StepParams p, int64_t lim)
{
    const int wk = blockIdx.y;
    float* __restrict__ r = r_base + (int64_t)(w0 + wk) * stride;
    float* __restrict__ m = MOM ? m_base + (int64_t)(w0 + wk) * stride : nullptr;
    const void* __restrict__ g = gp.dense[wk];
    const void* __restrict__ rv = SPARSE ? gp.row_vals[wk] : nullptr;
    const int32_t* __restrict__ slot = SPARSE ? gp.slot[wk] : nullptr;

    const int64_t step = (int64_t)gridDim.x * kHotThreads;
    const float* __restrict__ rs = gp.r_src[wk] ? gp.r_src[wk] : r;
    for (int64_t o = o0 + (int64_t)blockIdx.x * kHotThreads + threadIdx.x; o < o0 + n; o += step) {
        HPSGD_GUARD_GROUP(o, lim, kIdLocalStep);
        f8 rr = ld8(rs + o * 8);
        f8 mm;
        if (MOM) mm = ld8(m + o * 8);
        f8 gg;
        bool dense_src = true;
        if (SPARSE) {
            if (o >= seg.o_begin && o < seg.o_end) {
                dense_src = false;
                const int64_t rel = o - seg.o_begin;
                const int64_t row = rel / seg.cols8;
                const int32_t s = __ldg(slot + row);
                if (s >= 0 && HPSGD_SLOT_OK(s, gp.n_rows[wk], kIdLocalStep))
                    gg = load_grad8<BF16>(rv, (int64_t)s * seg.cols8 + (rel - row * seg.cols8));
                else gg = zero8();
            }
        }
        if (dense_src) gg = load_grad8<BF16>(g, o);
#pragma unroll
        for (int q = 0; q < 8; ++q) rr.v[q] = step1<MOM, WD>(gg.v[q], mm.v[q], rr.v[q], p);
        st8(r + o * 8, rr);
        if (MOM) st8(m + o * 8, mm);
    }
}

// Row -> slot maps of the sparse-row tensor: slot_i[row_idx_i[k]] = k for every worker i of
// a batch (blockIdx.y), the maps pre-filled with -1.
struct SlotBatch {
    int32_t* slot[kMaxBatch];
    const int32_t* row_idx[kMaxBatch];
    int32_t n_rows[kMaxBatch];
};

__global__ void scatter_slots_kernel(SlotBatch sb, int64_t rows)
{
    const int i = blockIdx.y;
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k < sb.n_rows[i]) {
        const int32_t row = sb.row_idx[i][k];
        if (HPSGD_ROW_OK(row, rows, kIdScatter)) sb.slot[i][row] = k;
    }
}

// ---------------------------------------------------------------------------- merge
// Algorithm 3 + replica clone, per index:
//   acc = (r_0 - w) + ... + (r_{K-1} - w) left to right ; Dnew = acc / K
//   staleness 1: w += D (if a previous average exists) ; staleness 0: w += Dnew
//   D = Dnew ; r_i = w
// Left-to-right sum of replica changes for a run-time K: workers [i, i + N) are requested
// together and then added in order.  start_changes also takes the first term, which opens the sum.
template <int N>
__device__ __forceinline__ void add_changes(f8& acc, const float* __restrict__ r, int64_t stride, int i,
                                            int64_t e, const f8& wv)
{
    f8 rv[N];
#pragma unroll
    for (int b = 0; b < N; ++b) rv[b] = ld8(r + (int64_t)(i + b) * stride + e);
#pragma unroll
    for (int b = 0; b < N; ++b)
#pragma unroll
        for (int q = 0; q < 8; ++q) acc.v[q] = __fadd_rn(acc.v[q], __fsub_rn(rv[b].v[q], wv.v[q]));
}

template <int N>
__device__ __forceinline__ void start_changes(f8& acc, const float* __restrict__ r, int64_t stride, int64_t e,
                                              const f8& wv)
{
    f8 rv[N];
#pragma unroll
    for (int b = 0; b < N; ++b) rv[b] = ld8(r + (int64_t)b * stride + e);
#pragma unroll
    for (int q = 0; q < 8; ++q) acc.v[q] = __fsub_rn(rv[0].v[q], wv.v[q]);
#pragma unroll
    for (int b = 1; b < N; ++b)
#pragma unroll
        for (int q = 0; q < 8; ++q) acc.v[q] = __fadd_rn(acc.v[q], __fsub_rn(rv[b].v[q], wv.v[q]));
}

// acc = (r_0 - w) + (r_1 - w) + ... + (r_{K-1} - w), eight replicas in flight at a time.
__device__ __forceinline__ void sum_changes(f8& acc, const float* __restrict__ r, int64_t stride, int K,
                                            int64_t e, const f8& wv)
{
    int i;
    if (K >= 8) { start_changes<8>(acc, r, stride, e, wv); i = 8; }
    else if (K >= 4) { start_changes<4>(acc, r, stride, e, wv); i = 4; }
    else { start_changes<1>(acc, r, stride, e, wv); i = 1; }
    for (; i + 8 <= K; i += 8) add_changes<8>(acc, r, stride, i, e, wv);
    for (; i + 4 <= K; i += 4) add_changes<4>(acc, r, stride, i, e, wv);
    for (; i < K; ++i) add_changes<1>(acc, r, stride, i, e, wv);
}

constexpr int kMergeApplyPending = 1;   // flags: a previous average exists (staleness 1)
constexpr int kMergeImmediate = 2;      // flags: staleness 0

// KT > 0: K known at compile time; all K replica groups (K x 32 bytes per thread) are
// requested before the first use.  KT == 0: any K, replicas are loaded four at a time.
template <int KT>
__global__ void __launch_bounds__(kHotThreads, (KT > 8 || KT == 0) ? 2 : 4)
merge_kernel(float* __restrict__ w, float* __restrict__ D, float* __restrict__ r, int64_t stride,
             int K, int64_t o0, int64_t n, int flags, int64_t lim)
{
    const float fK = (float)K;
    const int64_t step = (int64_t)gridDim.x * kHotThreads;
    for (int64_t o = o0 + (int64_t)blockIdx.x * kHotThreads + threadIdx.x; o < o0 + n; o += step) {
        HPSGD_GUARD_GROUP(o, lim, kIdMerge);
        const int64_t e = o * 8;
        const f8 wv = ld8(w + e);
        f8 dv = zero8();
        if (flags & kMergeApplyPending) dv = ld8(D + e);
        f8 acc;
        if constexpr (KT > 0) {
            f8 rv[KT];
#pragma unroll
            for (int i = 0; i < KT; ++i) rv[i] = ld8(r + (int64_t)i * stride + e);
#pragma unroll
            for (int q = 0; q < 8; ++q) acc.v[q] = __fsub_rn(rv[0].v[q], wv.v[q]);
#pragma unroll
            for (int i = 1; i < KT; ++i)
#pragma unroll
                for (int q = 0; q < 8; ++q) acc.v[q] = __fadd_rn(acc.v[q], __fsub_rn(rv[i].v[q], wv.v[q]));
        } else {
            sum_changes(acc, r, stride, K, e, wv);
        }
        f8 dnew, wn;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            dnew.v[q] = __fdiv_rn(acc.v[q], fK);
            wn.v[q] = wv.v[q];
            if (flags & kMergeImmediate) wn.v[q] = __fadd_rn(wv.v[q], dnew.v[q]);
            else if (flags & kMergeApplyPending) wn.v[q] = __fadd_rn(wv.v[q], dv.v[q]);
        }
        st8(w + e, wn);
        st8(D + e, dnew);
        const int Kn = KT > 0 ? KT : K;
#pragma unroll 4
        for (int i = 0; i < Kn; ++i) st8(r + (int64_t)i * stride + e, wn);
    }
}

// ---------------------------------------------------------------------------- pipelined synchronisation
// The paper's timeline (Fig. 1): the synchronising process first commits the previous
// AllReduce result, then all-reduces while the training process already works on replicas
// cloned from the updated global model.  The merge is therefore split in two:
//   commit:  w_next = w + D          (D from the previous synchronisation, if any)
//   reduce:  D = ((r_0 - w) + ... + (r_{K-1} - w)) / K     over the replicas of the period that
//            just ended and the w they were cloned from,
// with replicas and w double-buffered so that the reduce and the next period's local steps
// touch different memory.  Same operations and order as merge_kernel.
__global__ void __launch_bounds__(kHotThreads)
commit_kernel(const float* __restrict__ w, const float* __restrict__ D, float* __restrict__ w_next,
              int64_t n, int flags, int64_t lim)
{
    const int64_t step = (int64_t)gridDim.x * kHotThreads;
    for (int64_t o = (int64_t)blockIdx.x * kHotThreads + threadIdx.x; o < n; o += step) {
        HPSGD_GUARD_GROUP(o, lim, kIdCommit);
        f8 wv = ld8(w + o * 8);
        if (flags & kMergeApplyPending) {
            const f8 dv = ld8(D + o * 8);
#pragma unroll
            for (int q = 0; q < 8; ++q) wv.v[q] = __fadd_rn(wv.v[q], dv.v[q]);
        }
        st8(w_next + o * 8, wv);
    }
}

// Per-worker source of a K-way sum: the worker's replica row, or w itself for a worker whose
// replica is still the clone of w (it made no local step; its change is r - w = 0).
struct ReducePtrs {
    const float* src[kMaxBatch];
};

// acc = (src_0 - w) + (src_1 - w) + ... + (src_{K-1} - w), left to right.  KT > 0: all K groups
// are requested before the first use; KT == 0: any K, four in flight at a time.
template <int KT>
__device__ __forceinline__ void sum_changes_from(f8& acc, const ReducePtrs& rp, int K, int64_t e, const f8& wv)
{
    if constexpr (KT > 0) {
        f8 rv[KT];
#pragma unroll
        for (int i = 0; i < KT; ++i) rv[i] = ld8(rp.src[i] + e);
#pragma unroll
        for (int q = 0; q < 8; ++q) acc.v[q] = __fsub_rn(rv[0].v[q], wv.v[q]);
#pragma unroll
        for (int i = 1; i < KT; ++i)
#pragma unroll
            for (int q = 0; q < 8; ++q) acc.v[q] = __fadd_rn(acc.v[q], __fsub_rn(rv[i].v[q], wv.v[q]));
    } else {
        {
            const f8 r0 = ld8(rp.src[0] + e);
#pragma unroll
            for (int q = 0; q < 8; ++q) acc.v[q] = __fsub_rn(r0.v[q], wv.v[q]);
        }
        int i = 1;
        for (; i + 4 <= K; i += 4) {
            f8 rv[4];
#pragma unroll
            for (int b = 0; b < 4; ++b) rv[b] = ld8(rp.src[i + b] + e);
#pragma unroll
            for (int b = 0; b < 4; ++b)
#pragma unroll
                for (int q = 0; q < 8; ++q) acc.v[q] = __fadd_rn(acc.v[q], __fsub_rn(rv[b].v[q], wv.v[q]));
        }
        for (; i < K; ++i) {
            const f8 ri = ld8(rp.src[i] + e);
#pragma unroll
            for (int q = 0; q < 8; ++q) acc.v[q] = __fadd_rn(acc.v[q], __fsub_rn(ri.v[q], wv.v[q]));
        }
    }
}

template <int KT>
__global__ void __launch_bounds__(kHotThreads, (KT > 8 || KT == 0) ? 2 : 4)
reduce_kernel(const float* __restrict__ w, float* __restrict__ D, ReducePtrs rp, int K, int64_t n, int64_t lim)
{
    const int Kn = KT > 0 ? KT : K;
    const float fK = (float)Kn;
    const int64_t step = (int64_t)gridDim.x * kHotThreads;
    for (int64_t o = (int64_t)blockIdx.x * kHotThreads + threadIdx.x; o < n; o += step) {
        HPSGD_GUARD_GROUP(o, lim, kIdReduce);
        const int64_t e = o * 8;
        const f8 wv = ld8(w + e);
        f8 acc;
        sum_changes_from<KT>(acc, rp, Kn, e, wv);
        f8 dnew;
#pragma unroll
        for (int q = 0; q < 8; ++q) dnew.v[q] = __fdiv_rn(acc.v[q], fK);
        st8(D + e, dnew);
    }
}

// ---------------------------------------------------------------------------- merge with a lazy clone
// The merge without its K replica writes: after it every replica IS w, and whoever reads
// replica i next (a local step, the next merge, an inspection call) reads w instead of a row
// that was never written.  Same operations in the same order as merge_kernel; per index it
// moves (K + 2) * 4 bytes in and 8 out instead of (2K + 4) * 4.  A worker whose replica is
// already such a clone has src = w.
template <int KT>
__global__ void __launch_bounds__(kHotThreads, (KT > 8 || KT == 0) ? 2 : 4)
merge_lazy_kernel(float* __restrict__ w, float* __restrict__ D, ReducePtrs rp, int K, int64_t o0, int64_t n,
                  int flags, int64_t lim)
{
    const int Kn = KT > 0 ? KT : K;
    const float fK = (float)Kn;
    const int64_t step = (int64_t)gridDim.x * kHotThreads;
    for (int64_t o = o0 + (int64_t)blockIdx.x * kHotThreads + threadIdx.x; o < o0 + n; o += step) {
        HPSGD_GUARD_GROUP(o, lim, kIdMergeLazy);
        const int64_t e = o * 8;
        const f8 wv = ld8(w + e);
        f8 dv = zero8();
        if (flags & kMergeApplyPending) dv = ld8(D + e);
        f8 acc;
        sum_changes_from<KT>(acc, rp, Kn, e, wv);
        f8 dnew, wn;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            dnew.v[q] = __fdiv_rn(acc.v[q], fK);
            wn.v[q] = wv.v[q];
            if (flags & kMergeImmediate) wn.v[q] = __fadd_rn(wv.v[q], dnew.v[q]);
            else if (flags & kMergeApplyPending) wn.v[q] = __fadd_rn(wv.v[q], dv.v[q]);
        }
        st8(w + e, wn);
        st8(D + e, dnew);
    }
}

// ---------------------------------------------------------------------------- gradient-accumulation form
// Algorithms 2 and 3 as printed, plain SGD: each worker keeps its accumulated gradients a_i.
//   local step:  r_i = r_i - mu*g (one FMA) ; a_i = a_i + g
//   merge:       w = w - mu*ghat (one FMA, if a previous AllReduce result ghat exists; with
//                staleness 0 the fresh mean is committed instead) ;
//                ghat = (a_0 + ... + a_{K-1}) / K left to right ; a_i = 0 ; r_i = w
template <bool BF16, bool SPARSE>
__global__ void __launch_bounds__(kHotThreads)
accum_step_kernel(float* __restrict__ r_base, float* __restrict__ a_base, int64_t stride,
                  int w0, BatchPtrs gp, SparseSeg seg, int64_t o0, int64_t n, float neg_mu, int64_t lim)
{
    const int wk = blockIdx.y;
    float* __restrict__ r = r_base + (int64_t)(w0 + wk) * stride;
    float* __restrict__ a = a_base + (int64_t)(w0 + wk) * stride;
    const int64_t step = (int64_t)gridDim.x * kHotThreads;
    for (int64_t o = o0 + (int64_t)blockIdx.x * kHotThreads + threadIdx.x; o < o0 + n; o += step) {
        HPSGD_GUARD_GROUP(o, lim, kIdAccumStep);
        f8 rr = ld8(r + o * 8);
        f8 aa = ld8(a + o * 8);
        GradRaw<BF16> raw;
        bool dense_src = true;
        if (SPARSE) {
            if (o >= seg.o_begin && o < seg.o_end) {
                dense_src = false;
                const int64_t rel = o - seg.o_begin;
                const int64_t row = rel / seg.cols8;
                const int32_t s = __ldg(gp.slot[wk] + row);
                if (s >= 0 && HPSGD_SLOT_OK(s, gp.n_rows[wk], kIdAccumStep))
                    raw = load_grad_raw<BF16>(gp.row_vals[wk], (int64_t)s * seg.cols8 + (rel - row * seg.cols8));
                else raw = zero_grad_raw<BF16>();
            }
        }
        if (dense_src) raw = load_grad_raw<BF16>(gp.dense[wk], o);
        const f8 gg = widen_grad<BF16>(raw);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            rr.v[q] = __fmaf_rn(neg_mu, gg.v[q], rr.v[q]);
            aa.v[q] = __fadd_rn(aa.v[q], gg.v[q]);
        }
        st8(r + o * 8, rr);
        st8(a + o * 8, aa);
    }
}

template <int KT>
__global__ void __launch_bounds__(kHotThreads, (KT > 8 || KT == 0) ? 2 : 4)
accum_merge_kernel(float* __restrict__ w, float* __restrict__ ghat, float* __restrict__ r, float* __restrict__ a,
                   int64_t stride, int K, int64_t o0, int64_t n, int flags, float neg_mu, int64_t lim)
{
    const int Kn = KT > 0 ? KT : K;
    const float fK = (float)Kn;
    const f8 zero = zero8();
    const int64_t step = (int64_t)gridDim.x * kHotThreads;
    for (int64_t o = o0 + (int64_t)blockIdx.x * kHotThreads + threadIdx.x; o < o0 + n; o += step) {
        HPSGD_GUARD_GROUP(o, lim, kIdAccumMerge);
        const int64_t e = o * 8;
        const f8 wv = ld8(w + e);
        f8 gv = zero;
        if (flags & kMergeApplyPending) gv = ld8(ghat + e);
        f8 sum;
        if constexpr (KT > 0) {
            f8 av[KT];
#pragma unroll
            for (int i = 0; i < KT; ++i) av[i] = ld8(a + (int64_t)i * stride + e);
            sum = av[0];
#pragma unroll
            for (int i = 1; i < KT; ++i)
#pragma unroll
                for (int q = 0; q < 8; ++q) sum.v[q] = __fadd_rn(sum.v[q], av[i].v[q]);
        } else {
            sum = ld8(a + e);
            int i = 1;
            for (; i + 4 <= K; i += 4) {
                f8 av[4];
#pragma unroll
                for (int b = 0; b < 4; ++b) av[b] = ld8(a + (int64_t)(i + b) * stride + e);
#pragma unroll
                for (int b = 0; b < 4; ++b)
#pragma unroll
                    for (int q = 0; q < 8; ++q) sum.v[q] = __fadd_rn(sum.v[q], av[b].v[q]);
            }
            for (; i < K; ++i) {
                const f8 ai = ld8(a + (int64_t)i * stride + e);
#pragma unroll
                for (int q = 0; q < 8; ++q) sum.v[q] = __fadd_rn(sum.v[q], ai.v[q]);
            }
        }
        f8 gnew, wn;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            gnew.v[q] = __fdiv_rn(sum.v[q], fK);
            wn.v[q] = wv.v[q];
            if (flags & kMergeImmediate) wn.v[q] = __fmaf_rn(neg_mu, gnew.v[q], wv.v[q]);
            else if (flags & kMergeApplyPending) wn.v[q] = __fmaf_rn(neg_mu, gv.v[q], wv.v[q]);
        }
        st8(w + e, wn);
        st8(ghat + e, gnew);
#pragma unroll 4
        for (int i = 0; i < Kn; ++i) {
            st8(a + (int64_t)i * stride + e, zero);
            st8(r + (int64_t)i * stride + e, wn);
        }
    }
}

// ---------------------------------------------------------------------------- merge + next local step
// The merge followed by the first local step of every worker, in one pass: the clone
// r_i = w never goes to memory, it is the starting point of r_i - mu*m_i directly
// (Algorithm 2 makes the replica and updates it in consecutive lines).  Same operations,
// same order, same results as merge_kernel followed by local_step_kernel, but per index
// it moves (K r + w + D) in, (w + D) out, then per worker (g + m) in, (r + m) out:
// (5K + 4) * 4 bytes with fp32 gradients instead of (7K + 4) * 4.
// Position of a group inside the sparse-row tensor.
struct SegPos {
    bool inside;
    int64_t row;
    int64_t col8;
};

__device__ __forceinline__ SegPos seg_pos(const SparseSeg& seg, int64_t o)
{
    SegPos sp{false, 0, 0};
    if (o >= seg.o_begin && o < seg.o_end) {
        // the tensor has fewer than 2^32 groups (P < 2^32): a 32-bit division, far cheaper than a 64-bit one
        const uint32_t rel = (uint32_t)(o - seg.o_begin);
        const uint32_t row = rel / (uint32_t)seg.cols8;
        sp.inside = true;
        sp.row = row;
        sp.col8 = rel - row * (uint32_t)seg.cols8;
    }
    return sp;
}

// Stored gradient group of worker i: from its dense buffer, or, inside the sparse-row tensor,
// from slot `s` of its row values (s < 0: the row has no gradient).
template <bool BF16, bool SPARSE>
__device__ __forceinline__ GradRaw<BF16> fused_grad_raw(const BatchPtrs& gp, const SparseSeg& seg, const SegPos& sp,
                                                        int32_t s, int i, int64_t o)
{
    if (SPARSE && sp.inside) {
        if (s < 0 || !HPSGD_SLOT_OK(s, gp.n_rows[i], kIdRound)) return zero_grad_raw<BF16>();
        return load_grad_raw<BF16>(gp.row_vals[i], (int64_t)s * seg.cols8 + sp.col8);
    }
    return load_grad_raw<BF16>(gp.dense[i], o);
}

template <int KT, bool BF16, bool MOM, bool WD, bool SPARSE>
__global__ void __launch_bounds__(kHotThreads, 2)
merge_step_kernel(float* __restrict__ w, float* __restrict__ D, float* __restrict__ r, float* __restrict__ m,
                  int64_t stride, int K, BatchPtrs gp, SparseSeg seg, int64_t o0, int64_t n, int flags,
                  StepParams p, int64_t lim)
{
    constexpr int B = 4;                         // workers whose g / m are in flight together
    const int Kn = KT > 0 ? KT : K;
    const float fK = (float)Kn;
    const int64_t step = (int64_t)gridDim.x * kHotThreads;
    for (int64_t o = o0 + (int64_t)blockIdx.x * kHotThreads + threadIdx.x; o < o0 + n; o += step) {
        HPSGD_GUARD_GROUP(o, lim, kIdMergeStep);
        const int64_t e = o * 8;
        // every worker's row -> slot entry is requested up front, so that the gradient loads
        // of the step phase do not wait on a dependent lookup
        SegPos sp{false, 0, 0};
        int32_t sl[KT > 0 ? KT : 1];
        if (SPARSE) {
            sp = seg_pos(seg, o);
            if (KT > 0 && sp.inside) {
#pragma unroll
                for (int i = 0; i < (KT > 0 ? KT : 1); ++i) sl[i] = __ldg(gp.slot[i] + sp.row);
            }
        }
        // ---- merge
        const f8 wv = ld8(w + e);
        f8 dv = zero8();
        if (flags & kMergeApplyPending) dv = ld8(D + e);
        f8 acc;
        if constexpr (KT > 0) {
            f8 rv[KT];
#pragma unroll
            for (int i = 0; i < KT; ++i) rv[i] = ld8(r + (int64_t)i * stride + e);
#pragma unroll
            for (int q = 0; q < 8; ++q) acc.v[q] = __fsub_rn(rv[0].v[q], wv.v[q]);
#pragma unroll
            for (int i = 1; i < KT; ++i)
#pragma unroll
                for (int q = 0; q < 8; ++q) acc.v[q] = __fadd_rn(acc.v[q], __fsub_rn(rv[i].v[q], wv.v[q]));
        } else {
            sum_changes(acc, r, stride, K, e, wv);
        }
        f8 dnew, wn;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            dnew.v[q] = __fdiv_rn(acc.v[q], fK);
            wn.v[q] = wv.v[q];
            if (flags & kMergeImmediate) wn.v[q] = __fadd_rn(wv.v[q], dnew.v[q]);
            else if (flags & kMergeApplyPending) wn.v[q] = __fadd_rn(wv.v[q], dv.v[q]);
        }
        st8(w + e, wn);
        st8(D + e, dnew);
        // ---- local step of every worker, starting from the clone r_i = wn
        int i0 = 0;
#pragma unroll
        for (; i0 + B <= Kn; i0 += B) {
            GradRaw<BF16> graw[B];
            f8 mm[B];
            int32_t sb[B];
            if (SPARSE && sp.inside) {
#pragma unroll
                for (int b = 0; b < B; ++b) sb[b] = KT > 0 ? sl[i0 + b] : __ldg(gp.slot[i0 + b] + sp.row);
            }
#pragma unroll
            for (int b = 0; b < B; ++b) {
                graw[b] = fused_grad_raw<BF16, SPARSE>(gp, seg, sp, sb[b], i0 + b, o);
                if (MOM) mm[b] = ld8(m + (int64_t)(i0 + b) * stride + e);
            }
#pragma unroll
            for (int b = 0; b < B; ++b) {
                const f8 gg = widen_grad<BF16>(graw[b]);
                f8 rr;
#pragma unroll
                for (int q = 0; q < 8; ++q) rr.v[q] = step1<MOM, WD>(gg.v[q], mm[b].v[q], wn.v[q], p);
                st8(r + (int64_t)(i0 + b) * stride + e, rr);
                if (MOM) st8(m + (int64_t)(i0 + b) * stride + e, mm[b]);
            }
        }
        for (; i0 < Kn; ++i0) {
            int32_t s1 = -1;
            if (SPARSE && sp.inside) s1 = __ldg(gp.slot[i0] + sp.row);
            const GradRaw<BF16> graw = fused_grad_raw<BF16, SPARSE>(gp, seg, sp, s1, i0, o);
            f8 mm;
            if (MOM) mm = ld8(m + (int64_t)i0 * stride + e);
            const f8 gg = widen_grad<BF16>(graw);
            f8 rr;
#pragma unroll
            for (int q = 0; q < 8; ++q) rr.v[q] = step1<MOM, WD>(gg.v[q], mm.v[q], wn.v[q], p);
            st8(r + (int64_t)i0 * stride + e, rr);
            if (MOM) st8(m + (int64_t)i0 * stride + e, mm);
        }
    }
}

// ---------------------------------------------------------------------------- one round in one kernel
// The local step of all K workers followed by the merge, in one pass over the index range
// (Algorithm 2's "update replica" for every worker, then Algorithm 3 and the re-clone).
// Per index: w and D are read once; for every worker, in the order i = 0..K-1, its gradient
// and momentum are read, the step is taken in registers, the new momentum is stored and the
// replica change r_i - w is added to the running sum; then Dnew = sum / K, w and D are
// written.  The stepped replicas are never stored, because the merge re-clones them: after
// the kernel every replica is w (a lazy clone, see merge_lazy_kernel).
//   FROM_W: every replica is still the clone of w when the round starts (exactly one local
//           step per worker and period, the usual case): the step starts from w in registers
//           and no replica row is read.  Per index the kernel then moves
//           16 + K * (g + 8) bytes with momentum (16 + K * g for plain SGD): w, D, K m, K g in;
//           w, D, K m out.  Otherwise replica i is read from gp.r_src[i] (its row, or w).
// Same operations in the same order as local_step_kernel for every worker followed by
// merge_kernel, so the results are bit-identical.  Workers are handled B at a time: all
// loads of a batch are requested before the first use.
// `first`: worker i0 is worker 0, whose change opens the sum.  `pre`: row -> slot entries of these
// NB workers that the caller requested earlier, or NULL.
template <int NB, bool BF16, bool MOM, bool WD, bool SPARSE, bool FROM_W>
__device__ __forceinline__ void round_batch(f8& acc, bool first, const f8& wv, float* __restrict__ m, int64_t stride,
                                            int i0, const BatchPtrs& gp, const SparseSeg& seg, const SegPos& sp,
                                            int64_t o, const StepParams& p, const int32_t* pre)
{
    const int64_t e = o * 8;
    // Request order matters inside the sparse-row tensor: the row -> slot entries come first (they
    // are short, L2-resident loads that the gradient addresses depend on), then everything that
    // depends on nothing (momentum, replica rows), and only then the gradients, whose addresses
    // need the slots.  The long loads are then in flight while the slots come back.
    int32_t sl[NB];
    if (SPARSE && sp.inside) {
#pragma unroll
        for (int b = 0; b < NB; ++b) sl[b] = pre ? pre[b] : __ldg(gp.slot[i0 + b] + sp.row);
    }
    GradRaw<BF16> graw[NB];
    f8 mm[NB];
    f8 rr[FROM_W ? 1 : NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        if (MOM) mm[b] = ld8(m + (int64_t)(i0 + b) * stride + e);
        if (!FROM_W) rr[b] = ld8(gp.r_src[i0 + b] + e);
    }
#pragma unroll
    for (int b = 0; b < NB; ++b) graw[b] = fused_grad_raw<BF16, SPARSE>(gp, seg, sp, SPARSE ? sl[b] : 0, i0 + b, o);
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        const f8 gg = widen_grad<BF16>(graw[b]);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float r_old = FROM_W ? wv.v[q] : rr[FROM_W ? 0 : b].v[q];
            const float r_new = step1<MOM, WD>(gg.v[q], mm[b].v[q], r_old, p);
            const float change = __fsub_rn(r_new, wv.v[q]);
            acc.v[q] = (b == 0 && first) ? change : __fadd_rn(acc.v[q], change);
        }
        if (MOM) st8(m + (int64_t)(i0 + b) * stride + e, mm[b]);
    }
}

// Workers whose loads are in flight together.  Each costs 8 registers for fp32 gradients (4 for
// bf16), 8 for momentum and 8 for a replica row that has to be read; without a sparse-row tensor the
// batch is as large as fits the 255 registers of a thread without spilling: 8 workers (16 x 32-byte
// loads) for the usual fp32 + momentum case, 16 where a worker needs at most 12 registers.  With a
// sparse-row tensor small batches win: inside that tensor a gradient address waits for a row -> slot
// entry, so what hides the latency is blocks per SM (fewer registers) and the next batch's requests,
// not the width of one batch (batches of 4 against 8 on the GRU-shaped workload: K = 8 6.03 -> 6.81 TB/s,
// K = 12 6.43 -> 6.83, K = 16 6.79 -> 6.83, K = 20 6.57 -> 6.82).
constexpr int round_batch_size(bool bf16, bool mom, bool sparse, bool from_w)
{
    const int per_worker = (bf16 ? 4 : 8) + (mom ? 8 : 0) + (from_w ? 0 : 8);
    if (sparse) return 4;
    if (!from_w) return per_worker >= 24 ? 4 : 8;
    return per_worker <= 12 ? 16 : 8;
}

// Workers [i, K) that do not fill a whole batch: one batch of NB if that many are left, then the
// same with half of it, down to one worker, so that a remainder of n workers takes about log2(n)
// rounds of loads instead of n.
template <int NB, bool BF16, bool MOM, bool WD, bool SPARSE, bool FROM_W>
__device__ __forceinline__ void round_rest(f8& acc, int& i, int K, const f8& wv, float* __restrict__ m, int64_t stride,
                                           const BatchPtrs& gp, const SparseSeg& seg, const SegPos& sp, int64_t o,
                                           const StepParams& p)
{
    if constexpr (NB >= 1) {
        if (i + NB <= K) {
            round_batch<NB, BF16, MOM, WD, SPARSE, FROM_W>(acc, i == 0, wv, m, stride, i, gp, seg, sp, o, p, nullptr);
            i += NB;
        }
        round_rest<NB / 2, BF16, MOM, WD, SPARSE, FROM_W>(acc, i, K, wv, m, stride, gp, seg, sp, o, p);
    }
}

// One batch of `size` workers (1 <= size <= B), `size` the same for every thread of the launch: the
// switch picks the instantiation whose register arrays have exactly that many entries.
template <int B, bool BF16, bool MOM, bool WD, bool SPARSE, bool FROM_W>
__device__ __forceinline__ void round_batch_of(int size, f8& acc, bool first, const f8& wv, float* __restrict__ m,
                                               int64_t stride, int i0, const BatchPtrs& gp, const SparseSeg& seg,
                                               const SegPos& sp, int64_t o, const StepParams& p, const int32_t* pre)
{
#define HPSGD_BATCH_CASE(S)                                                                                          \
    case S:                                                                                                          \
        if constexpr (S <= B) round_batch<S, BF16, MOM, WD, SPARSE, FROM_W>(acc, first, wv, m, stride, i0, gp, seg, sp, o, p, pre); \
        break;
    switch (size) {
        HPSGD_BATCH_CASE(1) HPSGD_BATCH_CASE(2) HPSGD_BATCH_CASE(3) HPSGD_BATCH_CASE(4)
        HPSGD_BATCH_CASE(5) HPSGD_BATCH_CASE(6) HPSGD_BATCH_CASE(7) HPSGD_BATCH_CASE(8)
        HPSGD_BATCH_CASE(9) HPSGD_BATCH_CASE(10) HPSGD_BATCH_CASE(11) HPSGD_BATCH_CASE(12)
        HPSGD_BATCH_CASE(13) HPSGD_BATCH_CASE(14) HPSGD_BATCH_CASE(15) HPSGD_BATCH_CASE(16)
    default: break;
    }
#undef HPSGD_BATCH_CASE
}

// EVEN: K is not a multiple of B; the workers are then cut into ceil(K / B) batches of as equal a
// size as possible (K = 11, B = 8: 6 + 5) instead of full batches and a tail (8 + 2 + 1), whose short
// last batches leave a thread with almost nothing in flight (measured 5-15 % on K = 9, 11, 13, 15).
// Launched only for such K; where B divides K the plain form below is used, unchanged.
template <int B, bool BF16, bool MOM, bool WD, bool SPARSE, bool FROM_W, bool EVEN = false>
__global__ void __launch_bounds__(kHotThreads, 2)
round_kernel(float* __restrict__ w, float* __restrict__ D, float* __restrict__ m, int64_t stride, int K,
             BatchPtrs gp, SparseSeg seg, int64_t o0, int64_t n, int flags, StepParams p, int64_t lim)
{
    const float fK = (float)K;
    const int64_t step = (int64_t)gridDim.x * kHotThreads;
    for (int64_t o = o0 + (int64_t)blockIdx.x * kHotThreads + threadIdx.x; o < o0 + n; o += step) {
        HPSGD_GUARD_GROUP(o, lim, kIdRound);
        const int64_t e = o * 8;
        SegPos sp{false, 0, 0};
        if (SPARSE) sp = seg_pos(seg, o);
        // the slot entries of the first two batches are requested before anything else: by the time
        // the gradient addresses are formed they have arrived (where the registers allow it)
        constexpr bool PRE = SPARSE && FROM_W;
        int32_t sl_pre[PRE ? 2 * B : 1];
        if (PRE && sp.inside && K >= B) {
#pragma unroll
            for (int b = 0; b < (PRE ? 2 * B : 1); ++b) sl_pre[b] = b < K ? __ldg(gp.slot[b] + sp.row) : -1;
        }
        const int32_t* sl = PRE ? sl_pre : nullptr;
        const f8 wv = ld8(w + e);
        f8 dv = zero8();
        if (flags & kMergeApplyPending) dv = ld8(D + e);
        // inside the sparse-row tensor few gradients are read, so a thread has little in flight: the
        // second batch's momentum starts its way from DRAM to L2 now, which costs no registers
        // (measured +2 % there; on dense ranges, where 16 loads are in flight anyway, it costs 2 %)
        if (SPARSE && sp.inside && MOM && K >= 2 * B) {
#pragma unroll
            for (int b = B; b < 2 * B; ++b) asm volatile("prefetch.global.L2 [%0];" :: "l"(m + (int64_t)b * stride + e));
        }
        // ---- local steps and the running sum of replica changes, worker 0 first
        f8 acc;
        int i = 0;
        if constexpr (EVEN) {
            const int batches = (K + B - 1) / B;
            const int small = K / batches, larger = K - small * batches;      // `larger` batches hold small + 1 workers
            for (int b = 0; b < batches; ++b) {
                const int size = small + (b < larger ? 1 : 0);
                // workers 0 .. 2B-1 had their slot entries requested above
                round_batch_of<B, BF16, MOM, WD, SPARSE, FROM_W>(size, acc, i == 0, wv, m, stride, i, gp, seg, sp, o, p,
                                                                 (PRE && i + size <= 2 * B) ? sl + i : nullptr);
                i += size;
            }
        } else {
        if (K >= B) {
            round_batch<B, BF16, MOM, WD, SPARSE, FROM_W>(acc, true, wv, m, stride, 0, gp, seg, sp, o, p, sl);
            i = B;
            if (K >= 2 * B) {
                round_batch<B, BF16, MOM, WD, SPARSE, FROM_W>(acc, false, wv, m, stride, B, gp, seg, sp, o, p, PRE ? sl + B : nullptr);
                i = 2 * B;
            }
        }
        for (; i + B <= K; i += B)
            round_batch<B, BF16, MOM, WD, SPARSE, FROM_W>(acc, false, wv, m, stride, i, gp, seg, sp, o, p, nullptr);
        round_rest<B / 2, BF16, MOM, WD, SPARSE, FROM_W>(acc, i, K, wv, m, stride, gp, seg, sp, o, p);
        }
        // ---- merge
        f8 dnew, wn;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            dnew.v[q] = __fdiv_rn(acc.v[q], fK);
            wn.v[q] = wv.v[q];
            if (flags & kMergeImmediate) wn.v[q] = __fadd_rn(wv.v[q], dnew.v[q]);
            else if (flags & kMergeApplyPending) wn.v[q] = __fadd_rn(wv.v[q], dv.v[q]);
        }
        st8(w + e, wn);
        st8(D + e, dnew);
    }
}

// r_i = w for every worker (used when the state is (re)initialised).
__global__ void __launch_bounds__(kThreads)
clone_kernel(const float* __restrict__ w_, float* __restrict__ r_, int64_t stride, int K, int64_t nvec)
{
    const float4* __restrict__ w = reinterpret_cast<const float4*>(w_);
    float4* __restrict__ r = reinterpret_cast<float4*>(r_);
    const int64_t stride4 = stride >> 2;
    const int64_t step = (int64_t)gridDim.x * kThreads;
    for (int64_t v = (int64_t)blockIdx.x * kThreads + threadIdx.x; v < nvec; v += step) {
        const float4 wv = w[v];
        for (int i = 0; i < K; ++i) r[(int64_t)i * stride4 + v] = wv;
    }
}

// ---------------------------------------------------------------------------- generators
// Counter hash of the synthetic inputs (definition in hpsgd.h, hpsgd_gen_grads).
constexpr uint64_t kM1 = 0x6a09e667f3bcc909ULL;
constexpr uint64_t kM2 = 0xbb67ae8584caa73bULL;
constexpr uint64_t kM3 = 0x3c6ef372fe94f82bULL;
constexpr uint64_t kM4 = 0xa54ff53a5f1d36f1ULL;

__host__ __device__ __forceinline__ uint64_t mix64(uint64_t x)
{
    x ^= x >> 32; x *= kM1;
    x ^= x >> 29; x *= kM2;
    x ^= x >> 32;
    return x;
}

__host__ __device__ __forceinline__ uint64_t hash_ctr(uint64_t key, uint64_t stream, uint64_t step,
                                                      uint64_t worker, uint64_t idx)
{
    const uint64_t ctr = (stream << 60) | (step << 40) | (worker << 32) | idx;
    return mix64(mix64(ctr ^ key) + kM4);
}

__device__ __forceinline__ float uniform_pm1(uint64_t h)
{
    const int32_t u24 = (int32_t)(h >> 40);
    return (float)(u24 - (1 << 23)) * 1.1920928955078125e-07f;   // 2^-23, exact
}

__device__ __forceinline__ double gauss01(uint64_t h)
{
    const uint32_t u24 = (uint32_t)(h >> 40);
    const uint32_t v24 = (uint32_t)((h >> 16) & 0xFFFFFFu);
    const double u1 = ((double)u24 + 1.0) * 5.9604644775390625e-08;      // 2^-24
    const double t = (double)v24 * 5.9604644775390625e-08;
    return sqrt(-2.0 * log(u1)) * cos(6.283185307179586476925286766559 * t);
}

__device__ __forceinline__ uint16_t f32_to_bf16_rne(float f)
{
    const uint32_t u = __float_as_uint(f);
    return (uint16_t)((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
}

struct GenParams {
    uint64_t key;
    uint64_t step;
    uint64_t worker;
    int kind;          // 0 uniform, 1 gauss, 2 initial model (stream 2, scale 0.1f)
    float scale_f;     // uniform: (float)scale
    double scale_d;    // gauss: sigma
    // sparse-row tensor (rows == 0: none): un-padded start, rows, cols
    int64_t sp_start;
    int64_t sp_rows;
    int64_t sp_cols;
};

__device__ __forceinline__ float gen_value(const GenParams& g, uint64_t idx)
{
    if (g.kind == 2) return __fmul_rn(0.1f, uniform_pm1(hash_ctr(g.key, 2, 0, 0, idx)));
    if (g.sp_rows > 0 && (int64_t)idx >= g.sp_start && (int64_t)idx < g.sp_start + g.sp_rows * g.sp_cols) {
        const uint64_t row = (idx - g.sp_start) / g.sp_cols;
        if ((uint32_t)(hash_ctr(g.key, 1, g.step, g.worker, row) >> 40) >= 1677721u) return 0.f;
    }
    const uint64_t h = hash_ctr(g.key, 0, g.step, g.worker, idx);
    if (g.kind == 0) return __fmul_rn(g.scale_f, uniform_pm1(h));
    return (float)(g.scale_d * gauss01(h));
}

// Fill a flat padded buffer: element e of the padded buffer belongs to the tensor t with
// offsets[t] <= e (binary search), and is a pad when e - offsets[t] >= sizes[t].
template <bool BF16>
__global__ void __launch_bounds__(kThreads)
gen_flat_kernel(void* __restrict__ out, int64_t n_pad, const int64_t* __restrict__ offsets,
                const int64_t* __restrict__ starts, const int64_t* __restrict__ sizes, int n_tensors,
                GenParams g)
{
    const int64_t step = (int64_t)gridDim.x * kThreads;
    for (int64_t e = (int64_t)blockIdx.x * kThreads + threadIdx.x; e < n_pad; e += step) {
        int lo = 0, hi = n_tensors - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (offsets[mid] <= e) lo = mid; else hi = mid - 1;
        }
        const int64_t rel = e - offsets[lo];
        float val = 0.f;
        if (rel < sizes[lo]) val = gen_value(g, (uint64_t)(starts[lo] + rel));
        if constexpr (BF16) reinterpret_cast<uint16_t*>(out)[e] = f32_to_bf16_rne(val);
        else reinterpret_cast<float*>(out)[e] = val;
    }
}

// Values of the listed rows of the sparse-row tensor, [n_rows x cols].
template <bool BF16>
__global__ void __launch_bounds__(kThreads)
gen_rows_kernel(void* __restrict__ out, const int32_t* __restrict__ row_idx, int64_t n_rows, GenParams g)
{
    const int64_t n = n_rows * g.sp_cols;
    const int64_t step = (int64_t)gridDim.x * kThreads;
    GenParams dense = g;
    dense.sp_rows = 0;          // listed rows are active by definition: no mask lookup
    for (int64_t e = (int64_t)blockIdx.x * kThreads + threadIdx.x; e < n; e += step) {
        const int64_t k = e / g.sp_cols;
        const int64_t c = e - k * g.sp_cols;
        const float val = gen_value(dense, (uint64_t)(g.sp_start + (int64_t)row_idx[k] * g.sp_cols + c));
        if constexpr (BF16) reinterpret_cast<uint16_t*>(out)[e] = f32_to_bf16_rne(val);
        else reinterpret_cast<float*>(out)[e] = val;
    }
}

}  // namespace hpsgd
