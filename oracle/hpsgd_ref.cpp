/*
 * HPSGD replica update and delayed merge: plain CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file exists to check the CUDA library; it is slow,
 * single-threaded and deliberately unoptimised.  Only tests, the smoke check and the
 * CPU-baseline legs of the benchmark may use it.  It shares no source with the CUDA
 * path and includes nothing from it.
 *
 * What it computes, in the paper's notation (n = K workers, learning rate mu):
 *
 *   Algorithm 2 (training process P_t).  When a synchronisation period begins the
 *   worker clones the global model into a replica r_i; every local gradient is applied
 *   to the replica, r_i <- r_i - mu * g_i, and is also accumulated.  Because the replica
 *   starts as a clone of w, its displacement r_i - w IS -mu times the accumulated
 *   gradient, which is the identity between Eq. 1 and Eq. 2; the accumulated gradient is
 *   therefore carried as the replica change and no separate accumulator is kept.
 *
 *   Algorithm 3 (synchronising process P_s).  (i) If gradients were all-reduced at the
 *   previous synchronisation, commit them to the global model; (ii) all-reduce this
 *   period's accumulated gradients (mean over the n workers, the 1/n of Eq. 1) and keep
 *   the result for the NEXT synchronisation; (iii) the counter is reset, so the next
 *   local step clones the (just updated) global model again.
 *
 *   Section 3.2, last paragraph: the global update therefore always lags the all-reduce
 *   that produced it by one synchronisation, and the very first synchronisation applies
 *   nothing.
 *
 * Readings taken where the paper is silent (the momentum, weight-decay, bf16 and
 * sparse-row variants are workload extensions with no counterpart in the paper):
 *   - AllReduce means the mean over K workers (Eq. 1 divides by n); the sums of Eq. 1/2
 *     run over the K workers 0..K-1.
 *   - Order inside one synchronisation: apply the pending change, then clone replicas
 *     from the UPDATED global model (Section 3.1 has the replica made from the newest
 *     global model).
 *   - Momentum: heavy ball, m <- beta*m + gd, r <- r - mu*m, per worker, zero at start,
 *     untouched by the merge.  Weight decay: coupled L2 at the replica, gd = g + lambda*r.
 *   - What is averaged is the replica change (Eq. 2 form), which under momentum includes
 *     the momentum contribution.
 *   - Every operation is one IEEE-754 binary32 operation, round to nearest even; fused
 *     multiply-adds exactly where written, nowhere else (build with -ffp-contract=off).
 *     The K-way sum runs left to right over i = 0..K-1; the mean is one correctly
 *     rounded division by (float)K.
 *   - staleness = 0 is a test mode that commits the fresh average at once (Eq. 2:
 *     the global model becomes the mean of the replicas, i.e. Local SGD, Algorithm 1).
 *
 * A second, independent set of functions (ref_acc_*) follows Algorithms 2 and 3 in the
 * form they are printed, for the paper's plain SGD: explicit accumulated gradients per
 * worker, AllReduce of those accumulators (mean), and the delayed commit
 * w <- w - mu * (mean gradients all-reduced at the previous synchronisation).
 *
 * Pins (tests/, run without a GPU): hand-worked K=2, P=4 examples; the closed forms of
 * Eq. 1 and Eq. 2 in binary64, also over periods of uneven length; K=1 against a library
 * SGD/momentum optimiser; Local SGD model averaging (Algorithm 1); equal-gradient and
 * first-merge invariants.
 */
#include <cmath>
#include <cstdint>
#include <cstring>
#include <new>
#include <vector>

namespace {

struct RefState {
    int64_t P = 0;
    int K = 0;
    float mu = 0.f, beta = 0.f, lambda = 0.f;
    int staleness = 1;
    bool D_valid = false;      // a pending averaged change from the previous merge exists
    int64_t merges = 0;        // s, the number of merges performed
    std::vector<float> w;      // global model
    std::vector<float> D;      // pending averaged replica change
    std::vector<std::vector<float>> r;   // replicas
    std::vector<std::vector<float>> m;   // momentum buffers
    std::vector<float> scratch;          // widened / expanded gradient
};

inline float widen_bf16(uint16_t bits)
{
    uint32_t u = static_cast<uint32_t>(bits) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return f;
}

/* Algorithm 2, "update replica", with the momentum / weight-decay extension. */
void local_step(RefState* s, int i, const float* g)
{
    float* r = s->r[i].data();
    float* m = s->m[i].data();
    for (int64_t j = 0; j < s->P; ++j) {
        float gd = (s->lambda == 0.f) ? g[j] : std::fmaf(s->lambda, r[j], g[j]);
        float mnew = (s->beta == 0.f) ? gd : std::fmaf(s->beta, m[j], gd);
        if (s->beta != 0.f) m[j] = mnew;   /* plain SGD keeps no momentum state */
        r[j] = std::fmaf(-s->mu, mnew, r[j]);
    }
}

/* Algorithm 3 plus the replica clone of Algorithm 2. */
void sync_merge(RefState* s)
{
    const float fK = static_cast<float>(s->K);
    for (int64_t j = 0; j < s->P; ++j) {
        float acc = s->r[0][j] - s->w[j];
        for (int i = 1; i < s->K; ++i) acc = acc + (s->r[i][j] - s->w[j]);
        float Dnew = acc / fK;
        if (s->staleness == 1) {
            if (s->D_valid) s->w[j] = s->w[j] + s->D[j];   /* commit the previous average */
        } else {
            s->w[j] = s->w[j] + Dnew;                      /* test mode: commit at once */
        }
        s->D[j] = Dnew;                                    /* kept for the next merge */
        for (int i = 0; i < s->K; ++i) s->r[i][j] = s->w[j];
    }
    s->D_valid = true;
    s->merges += 1;
}

/* ---- Algorithms 2 and 3 as printed: gradient-accumulation form, plain SGD ---- */
struct AccState {
    int64_t P = 0;
    int K = 0;
    float mu = 0.f;
    bool synced_valid = false;           // an AllReduce result from the previous synchronisation exists
    int64_t syncs = 0;
    std::vector<float> w;                // global model
    std::vector<float> synced;           // result of the last AllReduce (mean accumulated gradient)
    std::vector<std::vector<float>> r;   // replicas
    std::vector<std::vector<float>> a;   // accumulated gradients
};

/* Algorithm 2: "update replica" r_i = r_i - mu*g and "accumulate gradients" a_i = a_i + g. */
void acc_local_step(AccState* s, int i, const float* g)
{
    float* r = s->r[i].data();
    float* a = s->a[i].data();
    for (int64_t j = 0; j < s->P; ++j) {
        r[j] = std::fmaf(-s->mu, g[j], r[j]);
        a[j] = a[j] + g[j];
    }
}

/* Algorithm 3: commit the previous AllReduce result, AllReduce the accumulators (mean over
 * the K workers, left to right), reset them, and re-clone the replicas (Algorithm 2). */
void acc_sync(AccState* s)
{
    const float fK = static_cast<float>(s->K);
    for (int64_t j = 0; j < s->P; ++j) {
        if (s->synced_valid) s->w[j] = std::fmaf(-s->mu, s->synced[j], s->w[j]);
        float sum = s->a[0][j];
        for (int i = 1; i < s->K; ++i) sum = sum + s->a[i][j];
        s->synced[j] = sum / fK;
        for (int i = 0; i < s->K; ++i) {
            s->a[i][j] = 0.f;
            s->r[i][j] = s->w[j];
        }
    }
    s->synced_valid = true;
    s->syncs += 1;
}

}  // namespace

extern "C" {

void* ref_acc_create(int64_t P, int K, float lr)
{
    if (P <= 0 || K <= 0) return nullptr;
    AccState* s = new (std::nothrow) AccState;
    if (!s) return nullptr;
    s->P = P; s->K = K; s->mu = lr;
    s->w.assign(P, 0.f);
    s->synced.assign(P, 0.f);
    s->r.assign(K, std::vector<float>(P, 0.f));
    s->a.assign(K, std::vector<float>(P, 0.f));
    return s;
}

void ref_acc_destroy(void* h) { delete static_cast<AccState*>(h); }

void ref_acc_set_global(void* h, const float* w0)
{
    AccState* s = static_cast<AccState*>(h);
    s->w.assign(w0, w0 + s->P);
    std::fill(s->synced.begin(), s->synced.end(), 0.f);
    s->synced_valid = false;
    s->syncs = 0;
    for (int i = 0; i < s->K; ++i) {
        s->r[i] = s->w;
        std::fill(s->a[i].begin(), s->a[i].end(), 0.f);
    }
}

int ref_acc_local_step(void* h, int worker, const float* g)
{
    AccState* s = static_cast<AccState*>(h);
    if (worker < 0 || worker >= s->K) return -1;
    acc_local_step(s, worker, g);
    return 0;
}

void ref_acc_sync(void* h) { acc_sync(static_cast<AccState*>(h)); }

const float* ref_acc_get_global(void* h) { return static_cast<AccState*>(h)->w.data(); }
const float* ref_acc_get_synced(void* h) { return static_cast<AccState*>(h)->synced.data(); }
const float* ref_acc_get_replica(void* h, int i) { return static_cast<AccState*>(h)->r[i].data(); }
const float* ref_acc_get_accumulated(void* h, int i) { return static_cast<AccState*>(h)->a[i].data(); }

void* ref_create(int64_t P, int K, float lr, float momentum, float weight_decay, int staleness)
{
    if (P <= 0 || K <= 0 || (staleness != 0 && staleness != 1)) return nullptr;
    RefState* s = new (std::nothrow) RefState;
    if (!s) return nullptr;
    s->P = P; s->K = K; s->mu = lr; s->beta = momentum; s->lambda = weight_decay;
    s->staleness = staleness;
    s->w.assign(P, 0.f);
    s->D.assign(P, 0.f);
    s->r.assign(K, std::vector<float>(P, 0.f));
    s->m.assign(K, std::vector<float>(P, 0.f));
    return s;
}

void ref_destroy(void* h) { delete static_cast<RefState*>(h); }

/* Set the initial global model; replicas become clones, momentum and pending change zero. */
void ref_set_global(void* h, const float* w0)
{
    RefState* s = static_cast<RefState*>(h);
    s->w.assign(w0, w0 + s->P);
    std::fill(s->D.begin(), s->D.end(), 0.f);
    s->D_valid = false;
    s->merges = 0;
    for (int i = 0; i < s->K; ++i) {
        s->r[i] = s->w;
        std::fill(s->m[i].begin(), s->m[i].end(), 0.f);
    }
}

int ref_local_step(void* h, int worker, const float* g)
{
    RefState* s = static_cast<RefState*>(h);
    if (worker < 0 || worker >= s->K) return -1;
    local_step(s, worker, g);
    return 0;
}

/* Gradient stored as bfloat16 bit patterns: widen exactly, then the same step. */
int ref_local_step_bf16(void* h, int worker, const uint16_t* g)
{
    RefState* s = static_cast<RefState*>(h);
    if (worker < 0 || worker >= s->K) return -1;
    s->scratch.resize(s->P);
    for (int64_t j = 0; j < s->P; ++j) s->scratch[j] = widen_bf16(g[j]);
    local_step(s, worker, s->scratch.data());
    return 0;
}

/*
 * Sparse-row gradient for one [rows x cols] tensor that starts at element seg_start:
 * only the listed rows carry values (row_vals is [n_rows x cols]); every other row of
 * that tensor has gradient zero and is stepped exactly like a dense zero.  Outside the
 * tensor the dense gradient applies; inside it the dense buffer is ignored.
 * is_bf16 selects the storage type of both dense and row_vals.
 */
int ref_local_step_sparse(void* h, int worker, const void* dense, int is_bf16,
                          int64_t seg_start, int64_t rows, int64_t cols,
                          const int32_t* row_idx, int32_t n_rows, const void* row_vals)
{
    RefState* s = static_cast<RefState*>(h);
    if (worker < 0 || worker >= s->K) return -1;
    if (seg_start < 0 || seg_start + rows * cols > s->P) return -1;
    s->scratch.resize(s->P);
    float* g = s->scratch.data();
    for (int64_t j = 0; j < s->P; ++j)
        g[j] = is_bf16 ? widen_bf16(static_cast<const uint16_t*>(dense)[j])
                       : static_cast<const float*>(dense)[j];
    for (int64_t j = seg_start; j < seg_start + rows * cols; ++j) g[j] = 0.f;
    for (int32_t k = 0; k < n_rows; ++k) {
        int64_t row = row_idx[k];
        if (row < 0 || row >= rows) return -1;
        for (int64_t c = 0; c < cols; ++c) {
            int64_t src = static_cast<int64_t>(k) * cols + c;
            g[seg_start + row * cols + c] =
                is_bf16 ? widen_bf16(static_cast<const uint16_t*>(row_vals)[src])
                        : static_cast<const float*>(row_vals)[src];
        }
    }
    local_step(s, worker, g);
    return 0;
}

void ref_sync_merge(void* h) { sync_merge(static_cast<RefState*>(h)); }

const float* ref_get_global(void* h) { return static_cast<RefState*>(h)->w.data(); }
const float* ref_get_pending(void* h) { return static_cast<RefState*>(h)->D.data(); }
const float* ref_get_replica(void* h, int i) { return static_cast<RefState*>(h)->r[i].data(); }
const float* ref_get_momentum(void* h, int i) { return static_cast<RefState*>(h)->m[i].data(); }
int64_t ref_merges(void* h) { return static_cast<RefState*>(h)->merges; }

}  // extern "C"
