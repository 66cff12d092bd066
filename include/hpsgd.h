/*
 * libhpsgd: the HPSGD replica update and delayed merge on one NVIDIA B200 (sm_100a).
 *
 * K simulated workers each hold a flat fp32 replica r_i of a P-parameter model.  A local
 * step applies one worker's gradient to its replica (Algorithm 2 of the HPSGD paper); a
 * synchronisation averages the K replica changes in the fixed order i = 0..K-1 (the
 * AllReduce of Algorithm 3, mean as in Eq. 1), commits the average obtained at the
 * PREVIOUS synchronisation to the global model w (Algorithm 3, first step; Section 3.2,
 * last paragraph: the global update lags its all-reduce by one synchronisation) and
 * re-clones every replica from the updated w (Algorithm 2, "make replica").
 *
 * Conventions
 *   - All pointers are DEVICE pointers unless the name or comment says "host".
 *   - Every entry point returns HPSGD_OK (0) or a negative hpsgd_status; nothing throws,
 *     aborts or exits across this boundary.  hpsgd_last_error() gives the text of the
 *     last failure.  Argument errors are detected before any GPU work is issued.
 *   - The library is a process-wide singleton (the four core calls carry no handle) and is
 *     not thread-safe: call it from one host thread.
 *   - hpsgd_local_step* and hpsgd_sync_merge only ENQUEUE work.  An asynchronous CUDA
 *     failure is reported by the next call as HPSGD_E_CUDA.
 *   - Flat layout: tensor t of the parameter set starts at a multiple of 32 elements
 *     (128 bytes) inside every flat buffer; the gaps ("pads") hold zero, must receive
 *     zero gradient, and are not parameters.  P_pad is the padded length.  With a single
 *     tensor P_pad = P rounded up to 32.
 *   - There is no CPU fallback: without a CUDA device every call that needs one fails
 *     with HPSGD_E_CUDA.
 */
#ifndef HPSGD_H_
#define HPSGD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum hpsgd_status {
    HPSGD_OK = 0,
    HPSGD_E_BADARG = -1,      /* invalid argument; nothing was enqueued */
    HPSGD_E_STATE = -2,       /* call not legal in the current state (e.g. before hpsgd_init) */
    HPSGD_E_NOMEM = -3,       /* arena too small or device allocation failed */
    HPSGD_E_CUDA = -4,        /* a CUDA call failed; see hpsgd_last_error() */
    HPSGD_E_TIMEOUT = -5,     /* a bounded device-side wait ran out (only the staged merge of HPSGD_OPT_STAGING has one) */
    HPSGD_E_UNSUPPORTED = -6  /* size beyond a documented limit */
} hpsgd_status;

/* Keys of hpsgd_set_option. */
enum {
    HPSGD_OPT_WEIGHT_DECAY = 1, /* lambda >= 0, coupled L2 at the replica: gd = g + lambda*r. Default 0. */
    HPSGD_OPT_STALENESS = 2,    /* 1 (default): commit the previous average, the paper's schedule.
                                   0: commit the fresh average at once (Eq. 2 / Local SGD). */
    HPSGD_OPT_GRAD_DTYPE = 3,   /* HPSGD_F32 (default) or HPSGD_BF16: storage type of gradients. */
    HPSGD_OPT_OVERLAP = 4,      /* 1 (default): merge on the side stream, ordered against local
                                   steps by events; 0: everything on the main stream. */
    HPSGD_OPT_CHUNKS = 5,       /* number of index ranges the schedule is cut into (1..1024).
                                   Results do not depend on it. Default 1. */
    HPSGD_OPT_PROFILE = 6,      /* 1: bracket every kernel launch of the path with CUDA events
                                   on the stream it runs on (see hpsgd_profile_read). */
    HPSGD_OPT_FUSE = 7,         /* How a round is cut into kernels (replica-change form, K <= 32; otherwise
                                   as 0).  Every setting performs the same operations in the same order,
                                   so results are bit-identical.
                                   0 (default): the paper's two processes.  Every call launches at once:
                                      local steps on the main stream, the merge on the side stream, where it
                                      overlaps whatever the caller does until the next local step.
                                   1: hpsgd_sync_merge holds its merge back; if the next call is a batched
                                      local step (hpsgd_local_step_all[_ex]) both run as ONE kernel in
                                      which the re-cloned replicas never go to memory before they are
                                      stepped; any other call first launches the merge on its own.
                                   2: one kernel per round.  Local steps are held back (hpsgd_local_step[_ex]
                                      and the batched calls alike; at most one per worker, all dense or all
                                      sparse-row); if every worker holds one when hpsgd_sync_merge comes, it
                                      runs them together with the merge: every worker is stepped in
                                      registers, its change enters the K-way sum, and the stepped replica is
                                      never stored, because the merge re-clones it anyway.  Merges also stop writing the K re-cloned replicas: a replica
                                      that nothing has stepped since its clone IS w and is read from w
                                      ("lazy clone"; hpsgd_get_replica then returns w's address).  With one
                                      local step per worker and period no replica row is read or written
                                      at all: per index w, D, K momenta and K gradients come in and w, D,
                                      K momenta go out.  Anything else (a second step of a worker, a merge
                                      while only some workers hold a step, any other call) first launches
                                      the held-back steps on their own.  The gradients of a held-back step
                                      are read when it is launched: leave them alone until hpsgd_sync_merge
                                      (or hpsgd_flush / hpsgd_synchronize) has returned.
                                   For callers whose gradients are already resident (a simulation, a
                                   benchmark) 2 is the fastest; a trainer that computes the next gradients
                                   while the merge runs wants 0. */
    HPSGD_OPT_STAGING = 9,      /* 0 (default): the merge reads and writes global memory directly, one 256-bit
                                   access per thread and array.  1: the stand-alone merge kernel (HPSGD_OPT_FUSE
                                   0 or 1, replica-change form, K <= 32) instead brings the K + 2 tiles of a block
                                   into shared memory with bulk asynchronous copies that complete on an mbarrier,
                                   and writes its K + 2 result tiles back with bulk stores.  Same operations in
                                   the same order: bit-identical.  It exists so that the two ways of issuing the
                                   memory traffic can be timed against each other on the same state; the merge has
                                   no data reuse for shared memory to exploit, and the plain form is as fast or
                                   faster.  The staged kernel is the only device code of this library that waits
                                   (on its own loads, for one second at most): if a wait ever runs out, the
                                   block writes nothing and the next call that waits for the device returns
                                   HPSGD_E_TIMEOUT. */
    HPSGD_OPT_DEBUG_STAGE_STALL = 10, /* Checked build only; HPSGD_E_UNSUPPORTED otherwise.  1: the barrier of the staged
                                   merge (HPSGD_OPT_STAGING) is told to expect 16 bytes more than its copies bring,
                                   so that its wait runs out after one second: the way to see the time-out path
                                   (blocks write nothing, the next synchronisation returns HPSGD_E_TIMEOUT) without
                                   a fault.  The state is not consistent afterwards; destroy it. */
    HPSGD_OPT_DEBUG_GROUP_LIMIT = 8 /* Checked build (compiled with -DHPSGD_DEBUG) only; HPSGD_E_UNSUPPORTED
                                   otherwise.  In that build every hot kernel tests each 8-element group
                                   index against the number of groups of a flat buffer before touching
                                   memory; a group that fails is skipped and recorded, and the next call
                                   that waits for the device (hpsgd_synchronize, hpsgd_get_global, ...)
                                   returns HPSGD_E_CUDA with the record.  This option lowers the number
                                   the kernels test against (value = groups, -1 = the real one), so that
                                   the guard can be seen to work on accesses that are in fact in bounds. */
};

/* Kernel kinds of hpsgd_profile_read. */
enum { HPSGD_KERNEL_LOCAL_STEP = 0, HPSGD_KERNEL_MERGE = 1, HPSGD_KERNEL_MERGE_STEP = 2 /* fuse 1 */,
       HPSGD_KERNEL_ROUND = 3 /* fuse 2: local steps + merge */,
       HPSGD_KERNEL_MERGE_STAGED = 4 /* the merge under HPSGD_OPT_STAGING */ };

enum { HPSGD_F32 = 0, HPSGD_BF16 = 1 };

/* Kinds of synthetic gradient (hpsgd_gen_grads). */
enum { HPSGD_GEN_UNIFORM = 0, HPSGD_GEN_GAUSS = 1 };

/* Flags of hpsgd_arena_bytes. */
enum { HPSGD_ARENA_MOMENTUM = 1, HPSGD_ARENA_PIPELINE = 2 };

/* ------------------------------------------------------------------------------------
 * The four core calls.
 * ---------------------------------------------------------------------------------- */

/*
 * Create the state for K workers and P parameters: global model w, pending averaged
 * change D = 0, replicas r_i = w and (momentum != 0 only) momentum buffers m_i = 0.
 * w is filled with seeded uniform values in [-0.1, 0.1) (counter hash, stream 2; see
 * hpsgd_gen_grads for the hash).  lr is the paper's mu (Algorithm 2 initialisation:
 * mu >= 0); momentum is the heavy-ball factor beta in [0, 1) (0 = the paper's plain SGD).
 * If hpsgd_set_layout was called, P must equal the sum of its sizes; otherwise the
 * parameter set is one tensor of P elements.  If hpsgd_bind supplied an arena it is
 * used (and must be large enough, else HPSGD_E_NOMEM); otherwise the library allocates
 * one with cudaMalloc and frees it in hpsgd_destroy.  A second hpsgd_init without
 * hpsgd_destroy returns HPSGD_E_STATE.  Blocks until the fill has completed.
 */
int hpsgd_init(int64_t P, int K, float lr, float momentum, uint64_t seed);

/*
 * One local step of worker `worker` (Algorithm 2, "update replica"; momentum and weight
 * decay are extensions the paper does not have), element-wise over the flat buffer:
 *     gd = g + lambda*r_i ;  m_i = beta*m_i + gd ;  r_i = r_i - mu*m_i
 * each line one fused multiply-add in binary32, round to nearest even.  `grads` is a
 * device buffer of P_pad elements in the flat layout, fp32 or bf16 per
 * HPSGD_OPT_GRAD_DTYPE, 32-byte aligned, zero in the pads.  It is borrowed: keep it
 * valid and unchanged until the work has run (hpsgd_synchronize, or a stream wait on
 * the main stream).  Its contents must be complete when the call is made, or be produced
 * by work enqueued earlier on the main stream: the library does not wait for other
 * streams.  Several local steps per worker between two merges are legal (Section 3.2:
 * several local trainings per synchronisation); a worker with none contributes a zero
 * change.  Enqueued on the main stream.
 */
int hpsgd_local_step(int worker, const void* grads);

/*
 * One synchronisation (Algorithm 3 + the replica clone of Algorithm 2), per index j:
 *     acc  = (r_0 - w) + (r_1 - w) + ... + (r_{K-1} - w)      left to right
 *     Dnew = acc / (float)K                                    correctly rounded
 *     staleness 1: w = w + D if this is not the first merge ; D = Dnew
 *     staleness 0: w = w + Dnew ; D = Dnew
 *     r_i  = w  for every i
 * in one fused kernel.  m_i is not touched.  Enqueued on the side stream (main stream
 * when HPSGD_OPT_OVERLAP is 0) behind all local steps issued so far; later local steps
 * wait, per index range, for the part of the merge they depend on.  With HPSGD_OPT_FUSE
 * the launch is deferred to the next call (see that option); the result is the same.
 */
int hpsgd_sync_merge(void);

/*
 * Wait for all enqueued work and return the device pointer to w (P_pad floats, flat
 * layout, library-owned, valid until hpsgd_destroy; with hpsgd_set_pipeline the global model
 * alternates between two buffers, so ask again after every hpsgd_sync_merge).  The pending change D is NOT
 * flushed into it: after T merges w holds the changes of rounds 0..T-2 (one-
 * synchronisation delay).  Returns NULL on error.
 */
const float* hpsgd_get_global(void);

/* ------------------------------------------------------------------------------------
 * Layout, memory and streams (all optional; call before hpsgd_init).
 * ---------------------------------------------------------------------------------- */

/*
 * Padded length for a list of tensor sizes (host array); if offsets_out (host, n_tensors
 * entries) is not NULL it receives each tensor's start in the flat buffers.  Pure
 * function, no GPU needed.  Returns a negative hpsgd_status on bad input.
 */
int64_t hpsgd_layout_padded(int n_tensors, const int64_t* sizes, int64_t* offsets_out);

/*
 * What each worker carries between synchronisations, for the next hpsgd_init:
 *   HPSGD_FORM_REPLICA_CHANGE (default): only the replica; its displacement from w stands
 *     for the accumulated gradient (Eq. 2), and the merge averages replica changes.
 *   HPSGD_FORM_GRADIENT_ACCUMULATION: Algorithms 2 and 3 as printed, for the paper's plain
 *     SGD (momentum must be 0, no weight decay).  Local step: r_i = r_i - mu*g (one FMA) and
 *     a_i = a_i + g.  Merge: w = w - mu*ghat (one FMA) if a previous AllReduce result ghat
 *     exists (staleness 0: the fresh mean instead); ghat = (a_0 + ... + a_{K-1}) / K left to
 *     right; a_i = 0; r_i = w.  In this form hpsgd_get_pending returns ghat, the second
 *     pointer of hpsgd_get_replica returns a_i, HPSGD_ARENA_MOMENTUM must be set when sizing
 *     an arena, and HPSGD_OPT_FUSE has no effect.
 */
enum { HPSGD_FORM_REPLICA_CHANGE = 0, HPSGD_FORM_GRADIENT_ACCUMULATION = 1 };
int hpsgd_set_form(int form);

/*
 * Pipelined synchronisation for the next hpsgd_init (replica-change form, staleness 1, K <= 32),
 * the paper's timeline (Fig. 1; Section 3.1: the synchronising process runs beside the training
 * process).  hpsgd_sync_merge is split in two kernels: the commit w_next = w + D on the main
 * stream, and the K-way reduce D = mean(r_i - w) of the period that just ended on the side
 * stream.  Replicas and w are double-buffered (one more w and K more replica rows: set
 * HPSGD_ARENA_PIPELINE when sizing an arena), and a worker's first local step of a period reads
 * the new w instead of a re-cloned replica, so local steps never wait for the reduce; only the
 * next hpsgd_sync_merge does.  Any number of local steps per period.  Same operations in the
 * same order as the plain merge: results are bit-identical.  HPSGD_OPT_FUSE and
 * HPSGD_OPT_CHUNKS do not apply.  The first pointer of hpsgd_get_replica is w itself for a
 * worker that has not stepped since the last synchronisation.
 */
int hpsgd_set_pipeline(int enable);

/* Declare the tensor sizes (host array, each > 0) used by the next hpsgd_init. */
int hpsgd_set_layout(int n_tensors, const int64_t* sizes);

/*
 * Bytes of device memory the state needs: w, D, K replicas, K momentum buffers when
 * flags has HPSGD_ARENA_MOMENTUM, a second w and K more replicas with HPSGD_ARENA_PIPELINE,
 * plus the row->slot scratch map for a sparse-row
 * tensor of up to `sparse_rows` rows per worker (0 if unused) and a small table.
 */
size_t hpsgd_arena_bytes(int64_t P_pad, int K, int flags, int64_t sparse_rows);

/*
 * Lend device memory and streams for the next hpsgd_init.  `arena` (256-byte aligned,
 * `bytes` long) stays owned by the caller and must outlive hpsgd_destroy; pass NULL / 0
 * to let the library allocate.  hpsgd_init waits for all work on the device before it
 * first writes a lent arena (the library works on its own streams, which do not otherwise wait
 * for the caller's); after that the caller must leave the arena alone.  main_stream / side_stream are cudaStream_t handles
 * owned by the caller (e.g. torch streams); pass NULL to let the library create its own.
 */
int hpsgd_bind(void* arena, size_t bytes, void* main_stream, void* side_stream);

/* Set an option (keys above).  Legal after hpsgd_init, between rounds. */
int hpsgd_set_option(int key, double value);

/* ------------------------------------------------------------------------------------
 * Batched and sparse-row local steps.
 * ---------------------------------------------------------------------------------- */

/*
 * Gradient of one worker with one tensor given as sparse rows.  `dense` is as in
 * hpsgd_local_step; inside the span of the sparse tensor its contents are ignored.
 * The sparse tensor (declared by hpsgd_set_sparse_segment) is [rows x cols]; row_idx
 * (device, int32, ascending, unique, each in [0, rows)) lists the n_rows rows that carry
 * a gradient and row_vals (device, [n_rows x cols], same dtype as dense, 32-byte
 * aligned) their values.  Rows not listed have gradient ZERO and are still stepped
 * (momentum decays and moves the replica, weight decay applies): the result equals
 * a dense step with zero rows.  row_idx == NULL or n_rows == 0 means no sparse tensor
 * rows are active.  Unsorted, duplicate or out-of-range rows are the caller's error: the
 * normal build does not look (an out-of-range row is ignored, a duplicate leaves it open
 * which of its values is used).  The checked build (-DHPSGD_DEBUG) copies row_idx to the
 * host, waiting for the main stream, and returns HPSGD_E_BADARG for such a list before
 * anything is enqueued.
 */
typedef struct hpsgd_grad_desc {
    const void* dense;
    const int32_t* row_idx;
    int32_t n_rows;
    const void* row_vals;
} hpsgd_grad_desc;

/* Declare tensor `tensor_id` as the [rows x cols] sparse-row tensor (cols % 8 == 0,
 * rows*cols == its size).  tensor_id < 0 removes the declaration.  After hpsgd_init.
 * The row->slot scratch map lives in the arena; a caller-supplied arena must have been
 * sized with sparse_rows >= rows, else HPSGD_E_NOMEM. */
int hpsgd_set_sparse_segment(int tensor_id, int64_t rows, int64_t cols);

/* hpsgd_local_step with a sparse-row tensor (desc is a host struct, read during the call). */
int hpsgd_local_step_ex(int worker, const hpsgd_grad_desc* desc);

/*
 * One local step of ALL K workers in one launch per index range: worker i reads its
 * dense gradient at (char*)grads + i * worker_stride_bytes (stride a multiple of 32 bytes).
 * Same arithmetic as K calls of hpsgd_local_step; the launches are issued range by
 * range so that, with HPSGD_OPT_CHUNKS > 1, the merge of a range can start while later
 * ranges are still being stepped.
 */
int hpsgd_local_step_all(const void* grads, int64_t worker_stride_bytes);

/* The same for K sparse-row descriptors (host array of K structs).  K <= 32. */
int hpsgd_local_step_all_ex(const hpsgd_grad_desc* descs);

/*
 * (The paper has no counterpart for this call; it exists for deployment reasons only.)
 *
 * A sparse-row local step that allocates nothing.  Some programs that would like to call
 * this library are not in a position to obtain device memory for it: an inference or
 * training server whose own allocator took the whole GPU at start-up and hands out
 * nothing to third parties, a plug-in running inside a latency-critical loop where the
 * implicit device-wide synchronisation of cudaMalloc / cudaFree would stall every other
 * stream, or code running under a memory budget that is accounted to the byte.  For them
 * the row -> slot scratch map of the sparse-row step lives in a fixed array built into
 * the library image (HPSGD_NOALLOC_MAX_ROWS int32 entries = 1 MiB, held by every GPU
 * that loads the library until the process exits), and this call issues no cudaMalloc,
 * cudaFree or other allocating routine.  It does not use or need hpsgd_init: all state is
 * passed in.
 *
 * It performs, on the caller's buffers, exactly the step of hpsgd_local_step_ex:
 *   replica / momentum_buf  device, n_elems floats each (n_elems % 8 == 0), 32-byte aligned,
 *                           updated in place; momentum_buf may be NULL when momentum == 0
 *   desc                    host struct; dense has n_elems elements of grad_dtype, its span
 *                           [seg_offset, seg_offset + rows*cols) is ignored; row_idx / row_vals
 *                           as in hpsgd_grad_desc
 *   seg_offset, rows, cols  the sparse-row tensor inside the flat buffer (seg_offset % 8 == 0,
 *                           cols % 8 == 0, rows <= HPSGD_NOALLOC_MAX_ROWS)
 *   stream                  cudaStream_t the work is enqueued on (NULL = default stream)
 * Errors: HPSGD_E_UNSUPPORTED when rows exceeds HPSGD_NOALLOC_MAX_ROWS (use
 * hpsgd_local_step_ex, which sizes its map from the arena), HPSGD_E_BADARG for the rest.
 *
 * The first call on each device looks up the device address of the built-in array (with
 * that device current) and remembers it; make that first call outside any stream capture.
 * That look-up is safe against several host threads arriving together; everything else
 * about the call follows the rule of this library: one host thread at a time.
 * All calls on one device share the one array, and it keeps whatever the previous call
 * left: each call therefore resets the entries it uses before filling them.  Two calls
 * whose GPU work can overlap (different streams without an ordering between them) race
 * on the array and give undefined results; calls on one stream are safe.
 */
#define HPSGD_NOALLOC_MAX_ROWS 262144
int hpsgd_local_step_sparse_noalloc(float* replica, float* momentum_buf, int64_t n_elems,
                                    const hpsgd_grad_desc* desc, int grad_dtype,
                                    int64_t seg_offset, int64_t rows, int64_t cols,
                                    float lr, float momentum, float weight_decay, void* stream);

/* ------------------------------------------------------------------------------------
 * Host-buffer convenience (end-to-end use) and inspection.
 * ---------------------------------------------------------------------------------- */

/*
 * hpsgd_local_step with `host_grads` in HOST memory (P_pad elements, flat layout;
 * pinned memory gives asynchronous copies).  The library copies it to an internal
 * double-buffered staging area (allocated with cudaMalloc on first use, freed in
 * hpsgd_destroy) and enqueues the step; the host buffer may be reused once the call
 * returns only if it is NOT pinned; for pinned memory keep it unchanged until
 * hpsgd_synchronize.
 */
int hpsgd_local_step_host(int worker, const void* host_grads);

/* Overwrite w from a HOST array of the P parameters (un-padded concatenation of the
 * tensors) and reset D = 0, r_i = w, m_i = 0, merge count 0.  Blocking. */
int hpsgd_set_global_host(const float* host_w, int64_t n);

/*
 * Start again from a freshly seeded model (Algorithm 2, initialisation): `seed` replaces the
 * seed of hpsgd_init for every hash stream, w is filled on the device with the uniform
 * [-0.1, 0.1) values of stream 2 exactly as hpsgd_init fills it, and D = 0, r_i = w, m_i = 0,
 * merge count 0.  Layout, K, options and schedule stay.  Blocking.
 */
int hpsgd_fill_global(uint64_t seed);

/* Wait for all work, then copy the P parameters of w (un-padded concatenation) to a
 * HOST array of n = P floats.  Blocking. */
int hpsgd_copy_global(float* host_out, int64_t n);

/* The same copy, enqueued behind the merges issued so far instead of waited for: it runs on a
 * stream of its own, overlaps later local steps (and their host-to-device copies), and the next
 * merge waits for it before it overwrites w.  host_out (pinned memory, else the call blocks) is
 * complete after hpsgd_synchronize. */
int hpsgd_copy_global_async(float* host_out, int64_t n);

/* Device pointers (P_pad floats each) to worker's replica and momentum buffer (*m = NULL
 * when momentum == 0), and to the pending change D.  Any out pointer may be NULL.
 * Does not synchronise: call hpsgd_synchronize first, which also launches whatever
 * HPSGD_OPT_FUSE held back.  For a replica that is a lazy clone (HPSGD_OPT_FUSE = 2, the
 * pipelined schedule) the pointer is w itself; ask again after the next local step. */
int hpsgd_get_replica(int worker, const float** r, const float** m);
int hpsgd_get_pending(const float** D);

/*
 * Checkpoint of the optimisation state (the paper has none; a long run needs one): a HOST blob
 * holding w, D, every replica, every momentum (or accumulated-gradient) buffer in the flat
 * layout, the merge count and whether a pending change exists.  Hyper-parameters and options
 * are not part of it: import into a state initialised with the same P, layout, K, form and
 * momentum on/off (else HPSGD_E_BADARG), then set the options again.  Both calls wait for all
 * enqueued work (a merge deferred by HPSGD_OPT_FUSE is launched first) and block.  A run of T
 * rounds and a run of T/2 rounds + export + import + T/2 rounds give bit-identical states.
 */
size_t hpsgd_state_bytes(void);                                   /* 0 before hpsgd_init */
int hpsgd_export_state(void* host_out, size_t bytes);
int hpsgd_import_state(const void* host_in, size_t bytes);

/* Current sizes: any out pointer may be NULL. */
int hpsgd_get_sizes(int64_t* P, int64_t* P_pad, int* K, int64_t* merges);

/* Start of tensor t in the flat buffers, or a negative hpsgd_status. */
int64_t hpsgd_tensor_offset(int tensor_id);

/* ------------------------------------------------------------------------------------
 * Synthetic gradients generated on the device (inputs for benchmarks and large tests).
 * ---------------------------------------------------------------------------------- */

/*
 * Fill `out` (device, P_pad elements of the current HPSGD_OPT_GRAD_DTYPE, flat layout,
 * pads zero) with the gradient of (worker, step) from the counter hash seeded by
 * hpsgd_init's seed:
 *   mix(x): x ^= x>>32; x *= M1; x ^= x>>29; x *= M2; x ^= x>>32         (uint64)
 *   key = mix(seed + M3);  ctr = stream<<60 | step<<40 | worker<<32 | idx
 *   h = mix(mix(ctr ^ key) + M4);  u24 = h>>40;  v24 = (h>>16) & 0xFFFFFF
 *   M1..M4 = frac(sqrt 2, 3, 5, 7) * 2^64 with the low bit set
 * with idx the index in the UN-padded concatenation of the tensors (< 2^32), stream 0.
 *   HPSGD_GEN_UNIFORM: g = (float)scale * ((int)u24 - 2^23) * 2^-23
 *   HPSGD_GEN_GAUSS:   g = (float)(scale * sqrt(-2 ln((u24+1) 2^-24)) * cos(2 pi v24 2^-24)), in binary64
 * bf16 storage rounds that fp32 value to nearest even.  If a sparse-row tensor is
 * declared, its rows whose mask hash (stream 1, idx = row) has u24 >= 1677721 are zero.
 * Enqueued on the main stream.  step < 2^20, worker < 256.
 */
int hpsgd_gen_grads(void* out, int worker, int step, int kind, double scale);

/* Values of the listed rows of the sparse-row tensor, [n_rows x cols] into `out`, same
 * generator and dtype as hpsgd_gen_grads.  Enqueued on the main stream. */
int hpsgd_gen_row_vals(void* out, int worker, int step, int kind, double scale,
                       const int32_t* row_idx, int32_t n_rows);

/* ------------------------------------------------------------------------------------
 * Housekeeping.
 * ---------------------------------------------------------------------------------- */

/* Wait for all enqueued work on both streams. */
int hpsgd_synchronize(void);

/*
 * With HPSGD_OPT_PROFILE on: total device milliseconds and number of launches of one kind
 * of kernel (HPSGD_KERNEL_*: local step, merge, merge + next local step, whole round, staged merge) since the last
 * read of that kind, measured with CUDA event pairs recorded around each launch on the
 * stream it ran on.  Launches any deferred merge, synchronises, and resets that kind's
 * totals.  Any out pointer may be NULL.
 */
int hpsgd_profile_read(int kind, double* ms, int64_t* launches);

/*
 * What HBM gives a kernel that reads n_read arrays and writes n_write arrays per index with the
 * access shape of this library's hot kernels (one block per 128 groups of 8 floats, 256-bit
 * loads and stores, all loads requested before the first use) and next to no arithmetic: the
 * ceiling a hot kernel with that share of writes is to be compared with (DRAM loses bandwidth
 * to read/write turnarounds, so the ceiling depends on the mix).  (The paper has no counterpart;
 * this is a measuring aid.)  `scratch` is device memory lent for the duration of the call
 * (4096-byte aligned, at least (n_read + n_write) * row_bytes; it is overwritten with zeros);
 * row_bytes is the length of each array (a multiple of 4096; use arrays that together exceed the
 * L2 cache several times).  Runs two untimed and `iters` timed launches on a stream of its own,
 * waits, and returns (n_read + n_write) * row_bytes * iters / time in *gb_per_s (1e9 bytes/s).
 * Built mixes (n_read, n_write): (16,0) (12,4) (16,4) (13,7) (12,8) (8,8) (4,16) (0,16); others
 * give HPSGD_E_UNSUPPORTED.  Needs no hpsgd_init and touches no state of the library.  Blocking.
 */
int hpsgd_probe_hbm(void* scratch, size_t scratch_bytes, int n_read, int n_write, int64_t row_bytes, int iters,
                    double* gb_per_s);

/* Enqueue what HPSGD_OPT_FUSE held back (a merge, or a batched local step), if anything (does not wait). */
int hpsgd_flush(void);

/* Number of kernels this library has launched since hpsgd_init. */
int64_t hpsgd_launch_count(void);

/* Text of the last error (static storage, never NULL). */
const char* hpsgd_last_error(void);

/* Free everything the library allocated; the state can be created again afterwards. */
int hpsgd_destroy(void);

#ifdef __cplusplus
}
#endif
#endif /* HPSGD_H_ */
