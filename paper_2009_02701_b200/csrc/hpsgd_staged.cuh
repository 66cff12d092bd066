// Two pieces of libhpsgd that exist to measure, not to be the default path:
//
//   merge_staged_kernel   the merge with its K + 2 input tiles brought into shared memory by
//                         bulk asynchronous copies (cp.async.bulk, the untiled form of the TMA
//                         engine) that complete on an mbarrier, and its K + 2 output tiles
//                         written back by bulk stores.  Same arithmetic, same order, same bits
//                         as merge_kernel.  It is the alternative the plain 256-bit load/store
//                         kernel is measured against (HPSGD_OPT_STAGING); no element of the
//                         merge is read by more than one thread, so staging has no reuse to
//                         offer and only changes who issues the memory requests.
//   stream_probe_kernel   R read streams and W write streams of the same access shape as the
//                         hot kernels with no arithmetic to speak of: what HBM gives a kernel
//                         with that share of writes (hpsgd_probe_hbm).
//
// The staged kernel is the one place in the library where device code waits: on the mbarrier
// its own bulk loads complete on.  The wait is a try_wait loop bounded by time (one second); a block
// whose wait runs out counts itself in g_stage_timeouts, waits once more (bounded) so that no copy is still on
// its way into shared memory that the next block will own, writes nothing and returns.  The
// host turns a non-zero count into HPSGD_E_TIMEOUT at its next synchronisation.  Blocks are
// launched without clusters and every copy is between this GPU's global memory and the issuing
// block's own shared memory: nothing is delivered to another block.
#pragma once

#include "hpsgd_kernels.cuh"

namespace hpsgd {

constexpr int kStageGroups = 128;               // 8-element groups per tile: 4 KB per array
constexpr int kStageTileFloats = kStageGroups * 8;
constexpr uint64_t kStageWaitNs = 1000000000ull;   // how long a block waits for its own loads: one second

__device__ unsigned int g_stage_timeouts;       // blocks whose wait for their own loads ran out

__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_u32(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ void bulk_store(void* gmem_dst, const void* smem_src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 :: "l"(gmem_dst), "r"(smem_u32(smem_src)), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ uint64_t global_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait for phase `parity` of the barrier: true when the phase completed, false when
// kStageWaitNs went by first (each try_wait itself returns after a hardware-chosen slice of time).
__device__ __forceinline__ bool bounded_wait(uint64_t* bar, uint32_t parity)
{
    const uint32_t addr = smem_u32(bar);
    const uint64_t t0 = global_ns();
    for (;;) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
        if (global_ns() - t0 > kStageWaitNs) return false;
    }
}

// One block per tile of kStageGroups groups.  Shared memory: [(K + 2)][kStageTileFloats] floats,
// tile 0 = w, tile 1 = D, tile 2 + i = r_i.  Thread t works on the 16-byte pieces t and t + 128
// of every tile (a warp then reads 512 consecutive bytes per instruction: no bank conflicts);
// the operations per element and their order are those of merge_kernel.
__global__ void __launch_bounds__(kHotThreads)
merge_staged_kernel(float* __restrict__ w, float* __restrict__ D, float* __restrict__ r, int64_t stride,
                    int K, int64_t o0, int64_t n, int flags, int64_t lim, uint32_t never_arriving_bytes)
{
    extern __shared__ __align__(128) float tiles[];
    __shared__ __align__(8) uint64_t bar;

    const int64_t t0 = o0 + (int64_t)blockIdx.x * kStageGroups;      // first group of this tile
    if (t0 >= o0 + n) return;
    const int groups = (int)min((int64_t)kStageGroups, o0 + n - t0);
#ifdef HPSGD_DEBUG
    if (!debug_check(t0 >= 0 && t0 + groups <= lim, 1, kIdMerge, t0 + groups - 1, lim)) return;
#else
    (void)lim;
#endif
    const uint32_t bytes = (uint32_t)groups * 32u;
    const bool pending = (flags & kMergeApplyPending) != 0;
    const int64_t e0 = t0 * 8;

    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(&bar)) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        // never_arriving_bytes is 0 except in the checked build's test of the time-out path, where the
        // barrier is told to expect bytes that no copy brings, so that the wait below runs out
        const uint32_t expect = bytes * (uint32_t)(K + 1 + (pending ? 1 : 0)) + never_arriving_bytes;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_u32(&bar)), "r"(expect) : "memory");
        bulk_load(tiles, w + e0, bytes, &bar);
        if (pending) bulk_load(tiles + kStageTileFloats, D + e0, bytes, &bar);
        for (int i = 0; i < K; ++i)
            bulk_load(tiles + (int64_t)(2 + i) * kStageTileFloats, r + (int64_t)i * stride + e0, bytes, &bar);
    }
    // the whole block takes one decision (a barrier that only some threads leave early is its own hang)
    if (!__syncthreads_and(bounded_wait(&bar, 0) ? 1 : 0)) {
        if (threadIdx.x == 0) atomicAdd(&g_stage_timeouts, 1u);
        bounded_wait(&bar, 0);          // once more, so that nothing lands in this memory after the block has gone
        return;
    }

    const float fK = (float)K;
    float4* t4 = reinterpret_cast<float4*>(tiles);
    constexpr int kTile4 = kStageTileFloats / 4;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int p = threadIdx.x + h * kHotThreads;
        if (p >= groups * 2) continue;
        const float4 wv4 = t4[p];
        const float wv[4] = {wv4.x, wv4.y, wv4.z, wv4.w};
        float dv[4] = {0.f, 0.f, 0.f, 0.f};
        if (pending) {
            const float4 d4 = t4[kTile4 + p];
            dv[0] = d4.x; dv[1] = d4.y; dv[2] = d4.z; dv[3] = d4.w;
        }
        float acc[4];
        {
            const float4 r0 = t4[2 * kTile4 + p];
            acc[0] = __fsub_rn(r0.x, wv[0]); acc[1] = __fsub_rn(r0.y, wv[1]);
            acc[2] = __fsub_rn(r0.z, wv[2]); acc[3] = __fsub_rn(r0.w, wv[3]);
        }
#pragma unroll 4
        for (int i = 1; i < K; ++i) {
            const float4 ri = t4[(2 + i) * kTile4 + p];
            acc[0] = __fadd_rn(acc[0], __fsub_rn(ri.x, wv[0]));
            acc[1] = __fadd_rn(acc[1], __fsub_rn(ri.y, wv[1]));
            acc[2] = __fadd_rn(acc[2], __fsub_rn(ri.z, wv[2]));
            acc[3] = __fadd_rn(acc[3], __fsub_rn(ri.w, wv[3]));
        }
        float dn[4], wn[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            dn[q] = __fdiv_rn(acc[q], fK);
            wn[q] = wv[q];
            if (flags & kMergeImmediate) wn[q] = __fadd_rn(wv[q], dn[q]);
            else if (pending) wn[q] = __fadd_rn(wv[q], dv[q]);
        }
        // in place: every piece is read and written by the one thread that owns it
        t4[p] = make_float4(wn[0], wn[1], wn[2], wn[3]);
        t4[kTile4 + p] = make_float4(dn[0], dn[1], dn[2], dn[3]);
    }
    // the writes above went through the generic proxy; the bulk stores read through the async proxy
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0) {
        bulk_store(w + e0, tiles, bytes);
        bulk_store(D + e0, tiles + kStageTileFloats, bytes);
        for (int i = 0; i < K; ++i) bulk_store(r + (int64_t)i * stride + e0, tiles, bytes);   // r_i = w
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        // the block's shared memory must outlive the reads of its stores
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    }
}

// ---------------------------------------------------------------------------- bandwidth probe
// Group o of R source rows is loaded (all R loads requested before the first use), the groups are
// added up, and the sum is stored to group o of W destination rows: the memory traffic of a hot
// kernel that reads R and writes W arrays per index, one block per 128 groups, 256-bit accesses.
template <int R, int W>
__global__ void __launch_bounds__(kHotThreads)
stream_probe_kernel(const float* __restrict__ src, float* __restrict__ dst, int64_t row_floats, int64_t n_groups)
{
    const int64_t o = (int64_t)blockIdx.x * kHotThreads + threadIdx.x;
    if (o >= n_groups) return;
    f8 s = zero8();
    if constexpr (R > 0) {
        f8 x[R];
#pragma unroll
        for (int i = 0; i < R; ++i) x[i] = ld8(src + (int64_t)i * row_floats + o * 8);
#pragma unroll
        for (int i = 0; i < R; ++i)
#pragma unroll
            for (int q = 0; q < 8; ++q) s.v[q] = __fadd_rn(s.v[q], x[i].v[q]);
    }
    if constexpr (W > 0) {
#pragma unroll
        for (int j = 0; j < W; ++j) st8(dst + (int64_t)j * row_floats + o * 8, s);
    } else {
        // nothing to write: the loads still have to happen, so their sum decides a store that the
        // data (zeros) never triggers
        if (s.v[0] == 1.0f && s.v[7] == 2.0f) st8(dst + o * 8, s);
    }
}

}  // namespace hpsgd
