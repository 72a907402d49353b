/*
 * a2cid2.h -- C ABI of the A2CiD2 event-update engine (one NVIDIA B200, sm_100a).
 *
 * The engine holds a population of n simulated asynchronous workers. Worker i owns a
 * parameter row x_i and a continuous-momentum row x~_i (stacked [n, d] device buffers) and a
 * last-event time t_i. Events arrive as a time-sorted stream and are applied as the paper
 * "A2CiD2: Accelerating Asynchronous Communication in Decentralized Deep Learning" defines
 * them (Sec. 3.2 "Training dynamic": the SDE for dx^i_t, dx~^i_t, cited below as Eq. (dynamic) after its
 * label in the paper's source; Algorithm 1):
 *
 *   mixing    before any update of worker w at time t, (x_w, x~_w) is advanced over t - t_w by
 *             the flow dx = eta (x~ - x) dt, dx~ = eta (x - x~) dt, in closed form:
 *             c = (1 - exp(-2 eta (t - t_w))) / 2,  x_w -= c (x_w - x~_w),  x~_w += c (x_w - x~_w).
 *   gradient  x_i -= gamma g,  x~_i -= gamma g,  t_i = t          (g = one row of the gradient buffer)
 *   comm      m = x_i - x_j (taken after both are mixed to t);
 *             x_i -= alpha m,  x~_i -= alpha~ m,  x_j += alpha m,  x~_j += alpha~ m,  t_i = t_j = t.
 *
 * and the consensus distance sum_i |x_i - xbar|^2 (App. A) is reduced on the device.
 *
 * Conventions
 *   - Every function returns an int status (A2_OK = 0, negative on error) unless stated.
 *     No exception, abort or exit crosses this boundary. Invalid input is rejected before any
 *     device work and leaves the state untouched. a2cid2_last_error() gives the text of the
 *     last failure on a handle (or of the last failure in a handle-less call, per thread).
 *   - "host" pointers are ordinary CPU memory, read or written before the call returns.
 *     "device" pointers are CUDA global memory on the current device and are only borrowed.
 *   - Device work is issued on the stream given to a2cid2_bind() and is asynchronous: it is
 *     ordered with other work on that stream. Calls that return results to the host
 *     (consensus distance, read_state) wait for the stream.
 *   - A handle is not thread-safe; use it from one thread at a time.
 *   - There is no CPU path: without a CUDA device every device call fails with A2_ECUDA.
 */
#ifndef A2CID2_H
#define A2CID2_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct a2cid2 a2cid2_t;             /* engine handle; owned by the library            */
typedef struct a2cid2_sched a2cid2_sched_t; /* host-only schedule of an event stream          */
typedef struct a2cid2_plan a2cid2_plan_t;   /* a schedule whose descriptors are on the device  */

enum {
    A2_OK = 0,
    A2_EINVAL = -1, /* bad argument (NULL, size, alignment, non-finite parameter, bad flag)     */
    A2_EORDER = -2, /* times decrease within the call, or an event precedes its worker's t_i   */
    A2_ERANGE = -3, /* worker index or gradient slot out of range, i == j, or both/neither of
                       (wj, slot) given                                                         */
    A2_ENOMEM = -4, /* host or device allocation failed                                         */
    A2_ECUDA = -5,  /* a CUDA call failed (text in a2cid2_last_error)                           */
    A2_ESTATE = -6  /* call out of sequence: not bound, plan does not match the handle's times  */
};

enum { A2_F32 = 0, A2_BF16 = 1 }; /* storage type of x, x~ and the gradient buffer; math is fp32 */

/* Scheduling flags. */
enum {
    A2_SCHED_FUSE = 1u, /* fold the gradient events that directly precede a communication of the
                           same worker into that communication's item, so their rows are read
                           and written once (the arithmetic per element is unchanged)          */
    A2_SCHED_RESIDENT = 2u, /* no batches: one launch walks the whole stream in time order while a
                              column tile of all n workers' x and x~ stays in shared memory, so the
                              state crosses HBM once per call instead of once per batch. Columns
                              never interact, so no thread ever waits for another. Only valid when
                              the gradients of the whole stream are known up front (they are rows
                              of the bound buffer), and only for populations that fit shared
                              memory (2 n + 16 <= 216 rows of 256 floats; A2_EINVAL otherwise).
                              With bf16 storage the tile is kept in fp32 and rounded once, at the
                              end of the call. The schedule then has a single batch holding every
                              event in stream order. Overrides the other flags.                */
    A2_SCHED_CHAIN = 4u, /* A2_SCHED_FUSE, and further: (1) an event whose workers' latest events are
                           all in one item is appended to that item, whose rows then serve one
                           more event without crossing HBM again; (2) a communication between a
                           worker that is free earlier and one whose latest events sit in an item
                           with room joins that item as one more worker, so the shared worker's
                           rows are not written and read again in between. Every worker's own
                           order is kept and the arithmetic per event is unchanged; batches get
                           fewer and items longer (up to four workers with fp32 rows and the
                           momentum buffer, three otherwise)                                    */
    A2_SCHED_ROW_PER_OP = 8u /* with A2_SCHED_FUSE or A2_SCHED_CHAIN: the gradient events an item applies to
                           one worker may each name their own gradient row -- the paper's stochastic
                           gradients are fresh draws at every step (Sec. 3.2; Algorithm 1 computes g_i anew
                           in every iteration of its first loop). The item records the worker's first row
                           (slot_a .. slot_d) and, per gradient operation, the row to fetch next
                           (a2cid2_sched_op_reloads); the event kernel fetches it right after the operation
                           has used the previous one. Without the flag a change of row ends the item, so
                           that one row per worker and item suffices. The engine sets the flag by itself
                           wherever its kernels can follow it (fp32 rows) and clears it elsewhere (bf16
                           rows, whose kernels keep packed rows in registers for the whole item).        */
};

/* Kinds of elementary operation inside an item. */
enum {
    A2_OP_GRAD_A = 0, /* gradient event on the item's worker a                                   */
    A2_OP_GRAD_B = 1,
    A2_OP_COMM = 2,   /* communication between workers a and b                                   */
    A2_OP_MIX_A = 3,  /* mixing only (a2cid2_flush)                                              */
    A2_OP_GRAD_C = 4,
    A2_OP_COMM_AC = 5,
    A2_OP_COMM_BC = 6,
    A2_OP_GRAD_D = 7,
    A2_OP_COMM_AD = 8,
    A2_OP_COMM_BD = 9,
    A2_OP_COMM_CD = 10
};

/* Variants of the dynamic. */
enum {
    A2_MSG_AFTER_MIX = 0,  /* message x_i - x_j taken at the event time, as Eq. (dynamic) states */
    A2_MSG_BEFORE_MIX = 1, /* message taken from the un-mixed buffers, as Algorithm 1 is printed */
    A2_NO_MOMENTUM = 2     /* the asynchronous baseline, Eq. (baselinedynamic) of Sec. 3.2: what
                              Eq. (dynamic) becomes without the method. There is no drift and no
                              momentum buffer: gradient x_i -= gamma g; communication
                              x_i -= alpha (x_i - x_j), x_j += alpha (x_i - x_j). x~ is never read or
                              written (it may be left unbound), eta and alpha~ are ignored, and an
                              event moves half the bytes. a2cid2_flush then only records the time,
                              and the consensus distance at a common time is that of the stored
                              rows. A2_SCHED_RESIDENT is not available (A2_EINVAL).               */
};

/* How a whole event stream (a2cid2_apply_events, a whole a2cid2_plan_run) is put on the GPU. */
enum {
    A2_LAUNCH_AUTO = 0,          /* the library chooses per schedule: column slices when a batch moves less than
                                    1 GiB on average (short launches, where launch gaps and tails weigh), else
                                    one launch per batch                                                     */
    A2_LAUNCH_PER_BATCH = 1,     /* one kernel launch per batch of worker-disjoint items; the CTAs of a launch
                                    share out its (item, column tile) units round robin                      */
    A2_LAUNCH_COLUMN_SLICES = 2  /* launches that hold the items of several consecutive batches: every CTA owns a
                                    contiguous range of columns and applies all items, in schedule order, to
                                    that range alone. Legal because every operation of the method is element-wise
                                    over the parameter dimension (Eq. (dynamic) couples workers, never columns):
                                    what an item needs from an earlier one was written by the same thread. No
                                    CTA ever waits for another. The results are the same bits in all modes.  */
};

/* How often x is rounded to its storage precision (fp32 rows). */
enum {
    A2_ROUND_PER_EVENT = 0, /* every event rounds every value it updates once (the default). This is what an
                               fp32-storage implementation that applies events one by one does, and all
                               schedules and launch modes then give the same bits.                           */
    A2_ROUND_PER_STORE = 1  /* inside an item x is carried as a two-word value (what its roundings have lost
                               is kept beside it) and rounded once, when the item stores the row. Why: at an
                               averaging alpha~ multiplies the rounding errors x has collected into x~
                               (Eq. (dynamic), dM term: x~ moves by alpha~ (x_i - x_j)), so where alpha~ is
                               several times alpha (7.26 against 0.5 on the 64-worker ring) the error of x~ is
                               a random walk of amplified half-ulps of x, and an item that serves ten events
                               can spare nine of ten roundings. Costs about 12 % of the events per second of
                               chained schedules; results then depend on the schedule in the last bits.
                               fp32 rows with the momentum buffer, on 32-byte boundaries, batched schedules
                               (not A2_SCHED_RESIDENT).                                                      */
};

/* One item of a batch: all the work done on one worker (b = c = d = -1) or on two to four workers. */
typedef struct a2cid2_item_info {
    int32_t a, b;           /* worker rows; b = -1 for a gradient-only item                    */
    int32_t slot_a, slot_b; /* gradient row read up front for worker a / b (that of its first gradient
                               operation in the item), or -1                                    */
    int64_t first_op;       /* index of the item's first elementary operation                   */
    int32_t n_ops;          /* operations applied, in order, while the rows sit in registers    */
    int32_t batch;          /* batch (dependency level) the item belongs to                     */
    int32_t c, slot_c;      /* third worker and its gradient row (A2_SCHED_CHAIN), or -1         */
    int32_t d, slot_d;      /* fourth worker and its gradient row, or -1                         */
} a2cid2_item_info;

/* Counters of one a2cid2_apply_events / a2cid2_plan_run call (all device figures are what the
 * descriptors imply, not hardware counters). */
typedef struct a2cid2_stats {
    int64_t n_events, n_comm, n_grad;
    int64_t n_batches;  /* dependency levels                                                    */
    int64_t n_launches; /* event-kernel launches (a batch is split if it exceeds a launch's caps) */
    int64_t n_items;
    int64_t bytes_moved;       /* rows read + rows written by the items (every gradient row fetched counts,
                                  also one fetched in the middle of an item), times d, times element size */
    int64_t bytes_one_by_one;  /* the same stream applied one event per item: comm 8 rows, gradient 5
                                  (4 and 3 under A2_NO_MOMENTUM)                                   */
    int64_t descriptor_bytes;  /* host-to-device bytes of the descriptors                        */
    double host_ms;            /* validation + scheduling + descriptor packing time on the host   */
} a2cid2_stats;

/* ------------------------------------------------------------------------------------------
 * Engine
 * ------------------------------------------------------------------------------------------ */

/* Create an engine for n >= 2 workers of d >= 1 parameters with the hyper-parameters of
 * Eq. (dynamic) (eta >= 0; all finite). storage_dtype is A2_F32 or A2_BF16. Allocates only
 * small host/device bookkeeping; the state buffers come from a2cid2_bind. *out receives the
 * handle, to be released with a2cid2_destroy. Times start at t_i = 0 (Algorithm 1, init). */
int a2cid2_create(int32_t n, int64_t d, double eta, double alpha, double alpha_tilde, double gamma,
                  int32_t storage_dtype, a2cid2_t** out);

/* Select A2_MSG_AFTER_MIX (default), A2_MSG_BEFORE_MIX or A2_NO_MOMENTUM for later events.
 * A2_ESTATE when leaving A2_NO_MOMENTUM while no x~ buffer is bound. */
int a2cid2_set_variant(a2cid2_t* h, int32_t variant);

/* Select how whole streams are launched (A2_LAUNCH_*; default A2_LAUNCH_AUTO). A range of a plan's batches
 * (a2cid2_plan_run with a first batch or a count) is always run with one launch per batch. */
int a2cid2_set_launch_mode(a2cid2_t* h, int32_t mode);

/* Select A2_ROUND_PER_EVENT (default) or A2_ROUND_PER_STORE for later events. A2_EINVAL for bf16 storage; a call
 * that applies events fails with A2_ESTATE, before any launch, if the bound rows do not allow the mode. */
int a2cid2_set_rounding(a2cid2_t* h, int32_t mode);

/* Lend the device buffers: x and x_tilde are [n, row_pitch_elems], grads is
 * [n_grad_slots, row_pitch_elems] (may be NULL with n_grad_slots = 0 if no gradient event is
 * ever applied), all of the storage type, row-major, 16-byte aligned. row_pitch_elems >= d and
 * a multiple of 8; the columns between d and the pitch are padding that the library may
 * overwrite. x_tilde may be NULL only while the variant is A2_NO_MOMENTUM. cuda_stream is a cudaStream_t (NULL = default stream). The caller keeps ownership
 * and must keep the buffers alive until a2cid2_sync/destroy. May be called again to re-bind. */
int a2cid2_bind(a2cid2_t* h, void* x, void* x_tilde, void* grads, int32_t n_grad_slots,
                int64_t row_pitch_elems, void* cuda_stream);

/* Copy a dense host [n, d] array of the storage type into x; x~ from host_x_tilde, or a copy
 * of x when NULL (Algorithm 1: x~ <- x); times from host_t[n], or zeros when NULL. Waits.
 * Without a bound x~ buffer only x is written (host_x_tilde must then be NULL). */
int a2cid2_write_state(a2cid2_t* h, const void* host_x, const void* host_x_tilde, const double* host_t);

/* Copy dense host rows [n_slots, d] into gradient rows first_slot.. . Waits. */
int a2cid2_write_grads(a2cid2_t* h, int32_t first_slot, int32_t n_slots, const void* host_g);

/* Copy x, x~ (dense [n, d], storage type) and t[n] to the host; any pointer may be NULL. Waits.
 * A2_ESTATE if host_x_tilde is given while no x~ buffer is bound. */
int a2cid2_read_state(a2cid2_t* h, void* host_x, void* host_x_tilde, double* host_t);

/* Copy the workers' last-event times t[n] (kept on the host) without touching the device. */
int a2cid2_times(const a2cid2_t* h, double* host_t);

/* Overwrite the workers' last-event times (host array t[n], finite) without touching x, x~:
 * for callers that fill the bound buffers themselves, and for resuming from a checkpoint. */
int a2cid2_set_times(a2cid2_t* h, const double* host_t);

/* Apply n_events events (host arrays, read before return). Event e happens at times[e]
 * (finite, non-decreasing, and >= the stored t of its workers). wj[e] >= 0: communication
 * between wi[e] and wj[e], grad_slot[e] must be -1. wj[e] == -1: gradient event on wi[e]
 * using gradient row grad_slot[e] >= 0. The stream is validated, packed into batches of
 * disjoint workers that keep every worker's own order (flags: A2_SCHED_*), and one fused
 * kernel per batch is queued on the bound stream. stats may be NULL. Asynchronous. */
int a2cid2_apply_events(a2cid2_t* h, int64_t n_events, const double* times, const int32_t* wi,
                        const int32_t* wj, const int32_t* grad_slot, uint32_t flags, a2cid2_stats* stats);

/* Bring every worker to the common time t_flush >= max_i t_i: the mixing flow is applied to each
 * (x_i, x~_i) over t_flush - t_i and t_i = t_flush is recorded; no gradient, no averaging. This is the
 * state Algorithm 1 returns at the end of training (x_T), and the one at which mean(x) = mean(x~)
 * holds (Eq. (mean)). One kernel launch on the bound stream; asynchronous. A2_EORDER if t_flush
 * precedes a worker's time. */
int a2cid2_flush(a2cid2_t* h, double t_flush);

/* Consensus distance sum_i |x_i - xbar|^2, xbar = (1/n) sum_i x_i (App. A). With t_eval = NaN
 * the stored rows are used as they are (each at its own t_i). With a finite
 * t_eval >= max_i t_i every row is first mixed forward to t_eval in registers (nothing is
 * written back). Waits for the stream; *out is a host double. */
int a2cid2_consensus_distance(a2cid2_t* h, double t_eval, double* out);

/* The paper has no counterpart for this call; it exists for callers that must not allocate.
 *
 * Consensus distance of the stored rows (as a2cid2_consensus_distance with t_eval = NaN) for
 * programs in which nothing may call cudaMalloc once they are running: for example a trainer
 * whose own memory pool has already claimed the whole device, so that a raw allocation made by
 * a library would fail or steal from that pool; or a loop with a latency budget, since
 * cudaMalloc and cudaFree can stall the whole device. The call needs no handle and obtains no
 * device or pinned memory, and neither does anything it calls (only a failing call stores an
 * error text on the host). The per-block
 * partial sums, which the handle-based call keeps in memory it allocated at bind time, live here
 * in a fixed array of 4096 doubles (32 KB) inside the library image; every GPU on which the
 * library is used holds that array until the process exits.
 *
 *   x           device, [n, row_pitch_elems] of storage_dtype, 16-byte aligned, only read
 *   n, d        2 <= n <= 4096; 1 <= d <= 67,108,864 for A2_F32 and 134,217,728 for A2_BF16
 *               (4096 partials x 4096 vectors of 16 bytes per row); a larger d is rejected with
 *               A2_ERANGE and a message, nothing is launched
 *   row_pitch_elems  >= d, multiple of 8
 *   cuda_stream a cudaStream_t (NULL = default stream); the work is queued there, not waited for
 *   out_device  device, one double, written by the queued work; the caller owns it
 *
 * The first call on each device looks up the device address of the fixed array (with that
 * device current), remembers it, and has the kernels of both storage types loaded onto the
 * device; make that first call during start-up, outside any stream capture. All calls on one device share the array: a call overwrites every entry it later
 * reads, so nothing has to be cleared between calls, but two calls whose work overlaps on the
 * GPU (different streams, no ordering between them) race on it and give wrong sums. Calls on
 * one stream, or otherwise ordered, are safe. Errors: A2_EINVAL, A2_ERANGE, A2_ECUDA; the text
 * is available from a2cid2_last_error(NULL). */
int a2cid2_consensus_distance_static(const void* x, int32_t n, int64_t d, int64_t row_pitch_elems,
                                     int32_t storage_dtype, void* cuda_stream, double* out_device);

/* Wait for all work queued by this handle; returns the first deferred CUDA error, if any. */
int a2cid2_sync(a2cid2_t* h);

/* Text of the last error on h (h may be NULL: last error of a call that had no handle, for
 * the calling thread). Never NULL; valid until the next call on the same handle/thread. */
const char* a2cid2_last_error(const a2cid2_t* h);

/* Release the handle and everything the library allocated for it (waits for the stream).
 * Plans created from it should be destroyed first; one that is still alive stays valid only as an
 * argument of a2cid2_plan_destroy. NULL is allowed. */
void a2cid2_destroy(a2cid2_t* h);

/* ------------------------------------------------------------------------------------------
 * Plans: schedule once, run later (device-resident descriptors)
 * ------------------------------------------------------------------------------------------ */

/* Validate and schedule an event stream as a2cid2_apply_events does and upload its
 * descriptors, but launch nothing. t_start[n] gives the workers' times the stream starts
 * from (NULL = the handle's current times); a2cid2_plan_run checks them against the handle. A plan of
 * several launches also records them as one CUDA graph (on a private stream), so that running the
 * whole plan is a single submission. */
int a2cid2_plan_create(a2cid2_t* h, const double* t_start, int64_t n_events, const double* times,
                       const int32_t* wi, const int32_t* wj, const int32_t* grad_slot, uint32_t flags,
                       a2cid2_plan_t** out);

/* The plan's schedule, for inspection (owned by the plan). */
const a2cid2_sched_t* a2cid2_plan_sched(const a2cid2_plan_t* p);

/* Queue batches [first_batch, first_batch + n_batches) of the plan; n_batches = -1 means all
 * remaining. Batches must be run in order, each exactly once, and the handle's times must be
 * those the plan expects (A2_ESTATE otherwise). Asynchronous. stats may be NULL. */
int a2cid2_plan_run(a2cid2_t* h, a2cid2_plan_t* p, int64_t first_batch, int64_t n_batches, a2cid2_stats* stats);

void a2cid2_plan_destroy(a2cid2_plan_t* p);

/* ------------------------------------------------------------------------------------------
 * Host scheduler (no device needed)
 * ------------------------------------------------------------------------------------------ */

/* Pack a time-sorted event stream into batches. An event's batch is one more than the latest
 * batch of the workers it touches (greedy, as early as possible), so inside a batch no worker
 * appears in two items and every worker's events keep their order; since an event only
 * touches its own workers' rows (Eq. (dynamic) is local), running the batches in order gives
 * the state of the time-ordered run. With A2_SCHED_FUSE, gradient events of a worker are held
 * back and applied, in order, inside the next communication item of that worker (or in a
 * gradient-only item at the end of the stream, or when max_ops_per_item is reached or the
 * gradient slot changes). With A2_SCHED_CHAIN items also take later events of workers they already
 * hold, and further workers (see the flag). t_last[n] are the workers' times at the start
 * (NULL = zeros). max_ops_per_item <= 0 selects the default; max_workers_per_item is 2, 3 or 4
 * (<= 0: 4) and only matters with A2_SCHED_CHAIN. Validation and error codes as in
 * a2cid2_apply_events. */
int a2cid2_sched_create(int32_t n, int32_t n_grad_slots, const double* t_last, int64_t n_events,
                        const double* times, const int32_t* wi, const int32_t* wj, const int32_t* grad_slot,
                        uint32_t flags, int32_t max_ops_per_item, int32_t max_workers_per_item,
                        a2cid2_sched_t** out);

int64_t a2cid2_sched_num_batches(const a2cid2_sched_t* s);
int64_t a2cid2_sched_num_items(const a2cid2_sched_t* s);
int64_t a2cid2_sched_num_ops(const a2cid2_sched_t* s);

/* Items of batch b are [*first_item, *first_item + *n_items). */
int a2cid2_sched_batch_items(const a2cid2_sched_t* s, int64_t b, int64_t* first_item, int64_t* n_items);

int a2cid2_sched_item(const a2cid2_sched_t* s, int64_t item, a2cid2_item_info* out);

/* Operations [first_op, first_op + n_ops): the index of the event each one applies (into the
 * arrays given to a2cid2_sched_create) and its kind (A2_OP_*). Either output may be NULL. */
int a2cid2_sched_ops(const a2cid2_sched_t* s, int64_t first_op, int64_t n_ops, int64_t* event_index, int32_t* kind);

/* For gradient operations [first_op, first_op + n_ops): the gradient row that is fetched into the worker's
 * gradient registers after the operation (A2_SCHED_ROW_PER_OP), or -1; -1 for every other operation. The row
 * a gradient operation itself uses is the one its event names. */
int a2cid2_sched_op_reloads(const a2cid2_sched_t* s, int64_t first_op, int64_t n_ops, int32_t* reload);

/* Workers' times after the whole schedule has run. */
int a2cid2_sched_t_final(const a2cid2_sched_t* s, double* t_out);

/* Fill the descriptor-derived counters (events, batches, items, launches, bytes for d columns
 * of elem_bytes each, counted for the dynamic with the momentum buffer) for batches
 * [first_batch, first_batch + n_batches); -1 = all remaining. */
int a2cid2_sched_stats(const a2cid2_sched_t* s, int64_t first_batch, int64_t n_batches, int64_t d,
                       int32_t elem_bytes, a2cid2_stats* out);

void a2cid2_sched_destroy(a2cid2_sched_t* s);

/* ------------------------------------------------------------------------------------------
 * Graph quantities and the parameter prescription (host only)
 * ------------------------------------------------------------------------------------------ */

/* For the graph with n nodes and n_edges edges (ei[k], ej[k]) of rates lambda[k] > 0, form the
 * Laplacian as Sec. 3.1 defines it and return chi_1 = 1 / lambda_2(Lambda) (the definition of chi_1 in Sec. 3.1, algebraic
 * connectivity) and chi_2 = 1/2 max over edges of the effective resistance
 * (e_i - e_j)^T Lambda^+ (e_i - e_j) (the definition of chi_2 in Sec. 3.1). A2_EINVAL if the graph is not connected. */
int a2cid2_graph_chi(int32_t n, int64_t n_edges, const int32_t* ei, const int32_t* ej, const double* lambda,
                     double* chi1, double* chi2);

/* Parameters of the convergence proposition of Sec. 3.4: accelerated != 0: eta = 1/(2 sqrt(chi1 chi2)), alpha = 1/2,
 * alpha~ = 1/2 sqrt(chi1/chi2); accelerated == 0: eta = 0, alpha = alpha~ = 1/2. */
int a2cid2_prescribe(double chi1, double chi2, int32_t accelerated, double* eta, double* alpha, double* alpha_tilde);

/* Library version string. */
const char* a2cid2_version(void);

#ifdef __cplusplus
}
#endif
#endif /* A2CID2_H */
