/*
 * Seeded synthetic-input generator (host side).
 *
 * This file produces INPUTS only: initial global models, per-worker gradients and
 * embedding-row masks, all as pure functions of (seed, stream, step, worker, idx).
 * It contains none of the HPSGD update or merge arithmetic, so both the CPU oracle's
 * tests and the CUDA path's tests may be fed from it.
 *
 * Counter-based hash (64-bit, wrap-around arithmetic):
 *   mix(x):  x ^= x>>32; x *= M1; x ^= x>>29; x *= M2; x ^= x>>32
 *   key = mix(seed + M3)
 *   ctr = stream<<60 | step<<40 | worker<<32 | idx     (stream<16, step<2^20, worker<2^8, idx<2^32)
 *   h   = mix(mix(ctr ^ key) + M4)
 *   u24 = h>>40,  v24 = (h>>16) & 0xFFFFFF
 * M1..M4 are the fractional parts of sqrt(2), sqrt(3), sqrt(5), sqrt(7) times 2^64 with
 * the low bit forced to one.
 *
 * Streams: 0 gradient value, 1 embedding-row mask, 2 initial global model, 3 tensor sizes.
 *
 * Derived values:
 *   uniform[-1,1)  = ((int)u24 - 2^23) * 2^-23                       (exact in binary32)
 *   Gaussian       = sqrt(-2 ln u1) * cos(2 pi t),  u1=(u24+1)*2^-24, t=v24*2^-24  (binary64)
 *   gradient       = (float)(sigma * z)
 *   row active     = u24(stream 1) < floor(0.1 * 2^24) = 1677721
 *   w0[j]          = 0.1f * uniform(stream 2, step 0, worker 0, j)
 *
 * Loops are split over OpenMP threads: the generator is input plumbing and may be as
 * fast as it likes; every element depends only on its own counter.
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>

#define HG_M1 0x6a09e667f3bcc909ULL
#define HG_M2 0xbb67ae8584caa73bULL
#define HG_M3 0x3c6ef372fe94f82bULL
#define HG_M4 0xa54ff53a5f1d36f1ULL

static inline uint64_t hg_mix(uint64_t x)
{
    x ^= x >> 32; x *= HG_M1;
    x ^= x >> 29; x *= HG_M2;
    x ^= x >> 32;
    return x;
}

static inline uint64_t hg_key(uint64_t seed) { return hg_mix(seed + HG_M3); }

static inline uint64_t hg_hash_k(uint64_t key, uint64_t stream, uint64_t step,
                                 uint64_t worker, uint64_t idx)
{
    uint64_t ctr = (stream << 60) | (step << 40) | (worker << 32) | idx;
    return hg_mix(hg_mix(ctr ^ key) + HG_M4);
}

uint64_t hg_hash(uint64_t seed, uint64_t stream, uint64_t step, uint64_t worker, uint64_t idx)
{
    return hg_hash_k(hg_key(seed), stream, step, worker, idx);
}

static inline float hg_uniform_from(uint64_t h)
{
    int32_t u24 = (int32_t)(h >> 40);
    return (float)(u24 - (1 << 23)) * 0x1p-23f;
}

static inline double hg_gauss_from(uint64_t h)
{
    uint32_t u24 = (uint32_t)(h >> 40);
    uint32_t v24 = (uint32_t)((h >> 16) & 0xFFFFFFu);
    double u1 = ((double)u24 + 1.0) * 0x1p-24;
    double t = (double)v24 * 0x1p-24;
    return sqrt(-2.0 * log(u1)) * cos(6.283185307179586476925286766559 * t);
}

/* idx == NULL: indices idx0, idx0+1, ... ; otherwise idx[k] (each < 2^32). */
#define HG_INDEX(k) (idx ? (uint64_t)idx[(k)] : (uint64_t)(idx0 + (k)))

/* out[k] = scale * uniform[-1,1) from the gradient stream (stream 0). */
void hg_grad_uniform(uint64_t seed, uint64_t step, uint64_t worker, int64_t idx0,
                     const int64_t* idx, int64_t n, float scale, float* out)
{
    const uint64_t key = hg_key(seed);
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < n; ++k)
        out[k] = scale * hg_uniform_from(hg_hash_k(key, 0, step, worker, HG_INDEX(k)));
}

/* out[k] = (float)(sigma * z), z standard normal by Box-Muller on the gradient stream. */
void hg_grad_gauss(uint64_t seed, uint64_t step, uint64_t worker, int64_t idx0,
                   const int64_t* idx, int64_t n, double sigma, float* out)
{
    const uint64_t key = hg_key(seed);
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < n; ++k)
        out[k] = (float)(sigma * hg_gauss_from(hg_hash_k(key, 0, step, worker, HG_INDEX(k))));
}

/* out[k] = 0.1f * uniform[-1,1) from the initial-model stream (stream 2). */
void hg_init_global(uint64_t seed, int64_t idx0, const int64_t* idx, int64_t n, float* out)
{
    const uint64_t key = hg_key(seed);
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < n; ++k)
        out[k] = 0.1f * hg_uniform_from(hg_hash_k(key, 2, 0, 0, HG_INDEX(k)));
}

/* active[row] = 1 when the row carries a gradient for (worker, step), else 0 (stream 1). */
void hg_row_mask(uint64_t seed, uint64_t step, uint64_t worker, int64_t rows, uint8_t* active)
{
    const uint64_t key = hg_key(seed);
    for (int64_t row = 0; row < rows; ++row)
        active[row] = (uint32_t)(hg_hash_k(key, 1, step, worker, (uint64_t)row) >> 40) < 1677721u;
}

/* 53-bit uniform in [0,1) from the layout stream (stream 3), one per tensor number. */
double hg_layout_u(uint64_t seed, uint64_t tensor)
{
    return (double)(hg_hash(seed, 3, 0, 0, tensor) >> 11) * 0x1p-53;
}

/* Storage conversion binary32 -> bfloat16 bits, round to nearest even (finite inputs). */
void hg_f32_to_bf16(const float* in, int64_t n, uint16_t* out)
{
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < n; ++k) {
        union { float f; uint32_t u; } v;
        v.f = in[k];
        uint32_t lsb = (v.u >> 16) & 1u;
        out[k] = (uint16_t)((v.u + 0x7FFFu + lsb) >> 16);
    }
}

/* Exact widening bfloat16 bits -> binary32. */
void hg_bf16_to_f32(const uint16_t* in, int64_t n, float* out)
{
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < n; ++k) {
        union { float f; uint32_t u; } v;
        v.u = (uint32_t)in[k] << 16;
        out[k] = v.f;
    }
}
