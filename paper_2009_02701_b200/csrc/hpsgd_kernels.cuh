// Device code of libhpsgd (sm_100a): replica update, K-way delayed merge, input generators.
//
// Every kernel is element-wise over the flat padded buffers and HBM-bound, so the work
// is organised around memory traffic: 128-bit coalesced accesses, many independent loads
// in flight per thread before the first use, streaming cache hints for data that is
// touched once, and grids sized as a multiple of the SM count.  No tensor cores: there
// is no contraction anywhere on this path.
//
// Arithmetic is written with explicit round-to-nearest intrinsics (__fmaf_rn, __fadd_rn,
// __fsub_rn, __fdiv_rn) so that the compiler can neither fuse nor split an operation:
// the result is the one IEEE-754 binary32 value the definition in hpsgd.h gives.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

namespace hpsgd {

constexpr int kThreads = 256;

// ---------------------------------------------------------------------------- memory ops
// Streaming (evict-first) accesses for data that is read or written once per kernel.
__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }
__device__ __forceinline__ uint2 ld_stream(const uint2* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(float4* p, float4 v) { __stcs(p, v); }

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

// Four consecutive gradient values at vector index v (v counts groups of 4 elements).
template <bool BF16>
__device__ __forceinline__ float4 load_grad4(const void* g, int64_t v)
{
    if constexpr (BF16) {
        uint2 u = ld_stream(reinterpret_cast<const uint2*>(g) + v);
        return make_float4(bf16_lo(u.x), bf16_hi(u.x), bf16_lo(u.y), bf16_hi(u.y));
    } else {
        return ld_stream(reinterpret_cast<const float4*>(g) + v);
    }
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

template <bool MOM, bool WD>
__device__ __forceinline__ void step4(const float4& g, float4& m, float4& r, const StepParams& p)
{
    r.x = step1<MOM, WD>(g.x, m.x, r.x, p);
    r.y = step1<MOM, WD>(g.y, m.y, r.y, p);
    r.z = step1<MOM, WD>(g.z, m.z, r.z, p);
    r.w = step1<MOM, WD>(g.w, m.w, r.w, p);
}

// Sparse-row tensor inside the flat buffer: vectors [v_begin, v_end) form a
// [rows x cols] tensor whose gradient comes from row_vals through the row->slot map.
struct SparseSeg {
    int64_t v_begin;       // first vector of the tensor (element offset / 4)
    int64_t v_end;         // one past its last vector
    int32_t cols4;         // cols / 4
};

constexpr int kMaxBatch = 32;   // most workers one batched launch can address

// Per-worker pointers of a batched launch (blockIdx.y selects the worker).
struct BatchPtrs {
    const void* dense[kMaxBatch];
    const void* row_vals[kMaxBatch];
    const int32_t* slot[kMaxBatch];
};

// One worker per blockIdx.y; workers' replicas/momenta are `stride` floats apart starting
// at worker index w0.  Vectors [v0, v0 + nvec) are processed, U vectors per thread per
// iteration with all loads issued before the first use.
template <bool BF16, bool MOM, bool WD, bool SPARSE, int U>
__global__ void __launch_bounds__(kThreads)
local_step_kernel(float* __restrict__ r_base, float* __restrict__ m_base, int64_t stride,
                  int w0, BatchPtrs gp, SparseSeg seg, int64_t v0, int64_t nvec, StepParams p)
{
    const int wk = blockIdx.y;
    float4* __restrict__ r = reinterpret_cast<float4*>(r_base + (int64_t)(w0 + wk) * stride);
    float4* __restrict__ m = MOM ? reinterpret_cast<float4*>(m_base + (int64_t)(w0 + wk) * stride) : nullptr;
    const void* __restrict__ g = gp.dense[wk];
    const void* __restrict__ rv = SPARSE ? gp.row_vals[wk] : nullptr;
    const int32_t* __restrict__ slot = SPARSE ? gp.slot[wk] : nullptr;

    const int64_t step = (int64_t)gridDim.x * kThreads * U;
    for (int64_t base = v0 + (int64_t)blockIdx.x * kThreads * U + threadIdx.x; base < v0 + nvec; base += step) {
        float4 gv[U], rvv[U], mv[U];
        bool ok[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t v = base + (int64_t)u * kThreads;
            ok[u] = v < v0 + nvec;
            if (ok[u]) {
                rvv[u] = r[v];
                if (MOM) mv[u] = ld_stream(m + v);
                bool dense_src = true;
                if (SPARSE) {
                    if (v >= seg.v_begin && v < seg.v_end) {
                        dense_src = false;
                        const int64_t rel = v - seg.v_begin;
                        const int64_t row = rel / seg.cols4;
                        const int32_t s = __ldg(slot + row);
                        if (s >= 0) {
                            const int64_t col4 = rel - row * seg.cols4;
                            gv[u] = load_grad4<BF16>(rv, (int64_t)s * seg.cols4 + col4);
                        } else {
                            gv[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                        }
                    }
                }
                if (dense_src) gv[u] = load_grad4<BF16>(g, v);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (ok[u]) {
                const int64_t v = base + (int64_t)u * kThreads;
                step4<MOM, WD>(gv[u], mv[u], rvv[u], p);
                r[v] = rvv[u];
                if (MOM) st_stream(m + v, mv[u]);
            }
        }
    }
}

// Row -> slot map of the sparse-row tensor: slot[row_idx[k]] = k (map pre-filled with -1).
__global__ void scatter_slots_kernel(int32_t* __restrict__ slot, const int32_t* __restrict__ row_idx,
                                     int32_t n_rows, int64_t rows)
{
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k < n_rows) {
        const int32_t row = row_idx[k];
        if (row >= 0 && row < rows) slot[row] = k;
    }
}

// ---------------------------------------------------------------------------- merge
// Algorithm 3 + replica clone, per index:
//   acc = (r_0 - w) + ... + (r_{K-1} - w) left to right ; Dnew = acc / K
//   staleness 1: w += D (if a previous average exists) ; staleness 0: w += Dnew
//   D = Dnew ; r_i = w
constexpr int kMergeApplyPending = 1;   // flags: a previous average exists (staleness 1)
constexpr int kMergeImmediate = 2;      // flags: staleness 0

__device__ __forceinline__ float4 sub4(const float4& a, const float4& b)
{
    return make_float4(__fsub_rn(a.x, b.x), __fsub_rn(a.y, b.y), __fsub_rn(a.z, b.z), __fsub_rn(a.w, b.w));
}
__device__ __forceinline__ float4 add4(const float4& a, const float4& b)
{
    return make_float4(__fadd_rn(a.x, b.x), __fadd_rn(a.y, b.y), __fadd_rn(a.z, b.z), __fadd_rn(a.w, b.w));
}
__device__ __forceinline__ float4 div4(const float4& a, float d)
{
    return make_float4(__fdiv_rn(a.x, d), __fdiv_rn(a.y, d), __fdiv_rn(a.z, d), __fdiv_rn(a.w, d));
}

// KT > 0: K known at compile time, all K replica vectors are loaded before the sum.
// KT == 0: any K, replicas are loaded four at a time.
template <int KT>
__global__ void __launch_bounds__(kThreads)
merge_kernel(float* __restrict__ w_, float* __restrict__ D_, float* __restrict__ r_, int64_t stride,
             int K, int64_t v0, int64_t nvec, int flags)
{
    float4* __restrict__ w = reinterpret_cast<float4*>(w_);
    float4* __restrict__ D = reinterpret_cast<float4*>(D_);
    const int64_t stride4 = stride >> 2;
    float4* __restrict__ r = reinterpret_cast<float4*>(r_);
    const float fK = (float)K;
    const int64_t step = (int64_t)gridDim.x * kThreads;
    for (int64_t v = v0 + (int64_t)blockIdx.x * kThreads + threadIdx.x; v < v0 + nvec; v += step) {
        const float4 wv = ld_stream(w + v);
        float4 dv = make_float4(0.f, 0.f, 0.f, 0.f);
        if (flags & kMergeApplyPending) dv = ld_stream(D + v);
        float4 acc;
        if constexpr (KT > 0) {
            float4 rv[KT];
#pragma unroll
            for (int i = 0; i < KT; ++i) rv[i] = ld_stream(r + i * stride4 + v);
            acc = sub4(rv[0], wv);
#pragma unroll
            for (int i = 1; i < KT; ++i) acc = add4(acc, sub4(rv[i], wv));
        } else {
            acc = sub4(ld_stream(r + v), wv);
            int i = 1;
            for (; i + 4 <= K; i += 4) {
                float4 rv[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) rv[q] = ld_stream(r + (int64_t)(i + q) * stride4 + v);
#pragma unroll
                for (int q = 0; q < 4; ++q) acc = add4(acc, sub4(rv[q], wv));
            }
            for (; i < K; ++i) acc = add4(acc, sub4(ld_stream(r + (int64_t)i * stride4 + v), wv));
        }
        const float4 dnew = div4(acc, fK);
        float4 wn = wv;
        if (flags & kMergeImmediate) wn = add4(wv, dnew);
        else if (flags & kMergeApplyPending) wn = add4(wv, dv);
        st_stream(w + v, wn);
        st_stream(D + v, dnew);
        const int Kn = KT > 0 ? KT : K;
#pragma unroll 4
        for (int i = 0; i < Kn; ++i) r[(int64_t)i * stride4 + v] = wn;
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
