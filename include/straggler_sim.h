/*
 * straggler_sim.h - C ABI of the batched simulator of distributed SGD with straggling workers
 * (K-sync, K-batch-sync, K-async, K-batch-async SGD and a growing-K schedule), after
 * "Slow and Stale Gradients Can Win the Race" (Dutta, Wang, Joshi; arXiv 2003.10579).
 *
 * One handle simulates n_replicas independent parameter servers, each with P workers, on the
 * current CUDA device.  Everything runs in CUDA kernels for sm_100a; there is no CPU path.
 *
 * Conventions
 *   - Every call returns a sim_status and never throws or aborts.  Outputs are defined only on
 *     SIM_OK.  sim_last_error() gives a message for the last failure of a handle
 *     (sim_last_error(NULL): of the last failed sim_create / handle-less call on this thread).
 *   - "device" pointers are CUDA device pointers on the device that was current at sim_create;
 *     "host" pointers are ordinary host memory.  The library never takes ownership of a
 *     caller's buffer.  The data set (X, y / label, w_ref) is borrowed: it must stay valid and
 *     unchanged until sim_destroy.  The library allocates only its own state and trace.
 *   - Work is enqueued on the stream given at sim_create (a cudaStream_t passed as void*, NULL =
 *     the legacy default stream).  sim_run returns after enqueueing; sim_get_* and
 *     sim_trace_size synchronise that stream first and report a device-side error then.
 *   - Random streams are counter-based (Philox4x32-10, key = seed) and keyed by (global replica
 *     id, worker, the worker's task sequence number), so results do not depend on how replicas
 *     are split over handles or GPUs: replica r of a handle has global id replica_base + r.
 */
#ifndef STRAGGLER_SIM_H
#define STRAGGLER_SIM_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SIM_MAX_P 128         /* workers per replica (a warp per replica in the arrival kernel: 1, 2 or 4 workers per lane) */
#define SIM_MAX_CLASSES 16    /* softmax / MLP outputs */

typedef struct sim_handle sim_handle;   /* opaque; owned by the library */

typedef enum {
  SIM_OK = 0,
  SIM_ERR_ARG = 1,       /* invalid argument, detected on the host before any launch */
  SIM_ERR_ALLOC = 2,     /* device or host allocation failed */
  SIM_ERR_CUDA = 3,      /* a CUDA runtime call or a kernel launch failed */
  SIM_ERR_TIMEOUT = 4,   /* a bounded device-side wait ran out; the handle is unusable */
  SIM_ERR_STATE = 5,     /* call not allowed in this state (e.g. sim_set_params after sim_run) */
  SIM_ERR_INTERNAL = 6   /* an internal consistency check failed on the device */
} sim_status;

/* The four variants of Section 2.2 ("Variants of SGD"). */
typedef enum {
  SIM_KSYNC = 0,        /* wait for the first K of P workers, cancel the rest; Eq. 2 */
  SIM_KBATCHSYNC = 1,   /* first K minibatches, finishers start another at the same w_j; Eq. 2 */
  SIM_KASYNC = 2,       /* first K of P workers, others keep their stale parameters; Eq. 3 */
  SIM_KBATCHASYNC = 3   /* every K pushes from anyone, pusher refetches at once; Eq. 3 */
} sim_variant;

/* The per-sample loss f(w, xi) of the empirical risk, Eq. 1. */
typedef enum {
  SIM_NONE = 0,      /* no parameters: arrival process and clock only (the runtime results of Section 3) */
  SIM_LSQ = 1,       /* f = 1/2 (x.w - y)^2,                         n_params = d */
  SIM_LOGISTIC = 2,  /* label b in {0,1}: f = softplus(x.w) - b x.w, n_params = d */
  SIM_SOFTMAX = 3,   /* f = -log softmax(W x)[label], W [n_classes][d] row-major, n_params = n_classes*d */
  SIM_MLP2 = 4       /* relu MLP d-hidden-n_classes with biases, cross-entropy; parameters
                        [W1 (d x hidden row-major), b1, W2 (hidden x n_classes), b2]; the two products
                        over d take bf16 operands (x, W1, delta1) with fp32 accumulation */
} sim_model;

/* Per-minibatch compute time X of a worker, i.i.d. over workers and minibatches (Section 3.1):
 * X = Exp(mu) (rate mu, mean 1/mu), shift + Exp(mu) (Lemma 4's shifted exponential), or the
 * heavy-tailed Pareto law of the runtime simulations of Section 3 (Figs. 4-5) with shape mu = 2
 * (the only shape built) and scale shift > 0: P(X > x) = (shift / x)^2. */
typedef enum { SIM_DELAY_EXP = 0, SIM_DELAY_SHIFTED_EXP = 1, SIM_DELAY_PARETO2 = 2 } sim_delay_kind;
typedef struct { sim_delay_kind kind; double mu; double shift; } sim_delay;

/* The data set S of N samples (Section 2).  All pointers are DEVICE pointers, borrowed. */
typedef struct {
  sim_model model;
  int64_t n;             /* samples, 1 <= n <= 2^32 */
  int32_t d;             /* features per sample, d % 4 == 0 */
  int32_t n_classes;     /* SOFTMAX / MLP2: 2..SIM_MAX_CLASSES; otherwise ignored */
  int32_t hidden;        /* MLP2: hidden width; otherwise ignored */
  const float* X;        /* [n][d] row-major fp32, 16-byte aligned */
  const float* y;        /* LSQ: [n] fp32 targets; otherwise NULL */
  const int32_t* label;  /* LOGISTIC: [n] in {0,1}; SOFTMAX / MLP2: [n] in [0, n_classes); LSQ: NULL */
  const float* w_ref;    /* optional [n_params]: |w_{j+1} - w_ref|^2 is recorded per update; may be NULL */
} sim_problem;

/*
 * Create a simulation: P workers, K of them (or K minibatches) per update, step size eta
 * (Eq. 2 / Eq. 3: w_{j+1} = w_j - (eta/K) sum_l g(w_tau(l,j), xi_l,j)), minibatch size m per
 * worker, drawn with replacement from all n samples.  Initial parameters are zero until
 * sim_set_params.  problem may be NULL or have model SIM_NONE for a clock-only simulation.
 * Errors: SIM_ERR_ARG for P not in [1, SIM_MAX_P], K not in [1, P], m < 1, m > 2^26, an m whose
 * index table does not fit in shared memory beside two tiles of rows of this d, n_replicas < 1,
 * mu <= 0 or NaN, shift < 0 or not finite, d % 4 != 0, misaligned or NULL X, missing y / label,
 * replica ids beyond 2^32; SIM_ERR_ALLOC / SIM_ERR_CUDA otherwise.  *out is NULL on failure.
 */
sim_status sim_create(const sim_problem* problem, int32_t P, int32_t K, sim_variant variant,
                      sim_delay delay, float eta, int32_t m, uint64_t seed, int32_t n_replicas,
                      int64_t replica_base, void* cuda_stream, sim_handle** out);

/* Same w0 (DEVICE, [n_params]) for every replica.  Only before the first sim_run (SIM_ERR_STATE
 * after).  The buffer is read during the call's enqueued work, not kept. */
sim_status sim_set_params(sim_handle* h, const float* w0);

/* Growing-K schedule with the interval structure of Algorithm 1 (Section 6): an update that
 * starts at simulated time t uses K = min(P, K0 * 2^floor(t / t_interval)).  t_interval <= 0
 * switches it off (fixed K from sim_create).  Only before the first sim_run. */
sim_status sim_set_adasync(sim_handle* h, int32_t K0, double t_interval);

/*
 * AdaSync as printed (Algorithm 1; derivation in Section 6 and its appendix): start at K0; whenever
 * an update starts in a later interval of length t_interval than the one K was last set in, and
 * K < P, set K from the full-data risk F (Eq. 1, F* taken as 0) of the parameters at that moment:
 *   K-batch-sync, K-async, K-batch-async:  K = K0 sqrt(F(w_0) / F(w_start))
 *   K-sync:  the positive root of  K^2 / (P - K) = K0^2 / (P - K0) * F(w_0) / F(w_start)
 * rounded half up, never decreasing, at most P.  Replicas pause at different updates, so sim_run
 * proceeds in rounds (one per interval crossing) and synchronises the stream between rounds.  LSQ,
 * LOGISTIC and SOFTMAX only (the MLP's kernels advance all replicas in lock step and cannot pause them one by
 * one).  Only before the first sim_run.
 */
sim_status sim_set_adasync_loss(sim_handle* h, int32_t K0, double t_interval);

/* Optional performance knobs of the linear-model kernels (0 = chosen from d): depth of the
 * shared-memory ring that stages sample rows ahead of the arithmetic (2..8), rows per tile (2 or
 * 4) and threads per replica (256 or 512) where the kernel for that d offers the choice.
 * Left at 0, the block shape also follows the number of replicas (narrow blocks with more columns
 * a thread once there are more than two replicas per SM); setting tile_rows or threads switches
 * that off.  Integer results never depend on any of this; fp32 results can differ in the last
 * bits (summation order). */
sim_status sim_set_tuning(sim_handle* h, int32_t stages, int32_t tile_rows, int32_t threads);

/* Optional: make room for total_updates updates of trace now, so that later sim_run calls
 * allocate nothing. */
sim_status sim_reserve(sim_handle* h, int64_t total_updates);

/* Advance every replica by `iters` server updates.  Resumable: run(a); run(b) gives the same
 * bits as run(a+b).  Enqueues on the handle's stream and returns. */
sim_status sim_run(sim_handle* h, int64_t iters);

/* Updates done so far and the row length K_max of the per-contributor trace arrays
 * (K, or P when the growing-K schedule is on). */
sim_status sim_trace_size(const sim_handle* h, int64_t* n_updates, int32_t* K_max);

/*
 * Copy the trace of all J = n_updates updates of all R = n_replicas replicas into caller-owned
 * DEVICE buffers; any pointer may be NULL to skip that array.  Section 2.3's two metrics are
 * error and wall-clock runtime: t is the simulated clock at update j, loss the minibatch loss
 * (1/(K m)) sum_l sum_q f(w_tau(l,j); xi) of the gradients used, dist2 = |w_{j+1} - w_ref|^2
 * (0 without w_ref).  worker / stale / seq list the K_used[j] contributors in arrival order
 * (staleness j - tau(l,j) of Eq. 3; seq = that worker's task sequence number), padded with
 * 0xFFFF / 0xFFFFFFFF up to K_max.  loss and dist2 are 0 for SIM_NONE.
 */
sim_status sim_get_trace(const sim_handle* h, double* t /*[R][J]*/, float* loss /*[R][J]*/,
                         float* dist2 /*[R][J]*/, uint16_t* K_used /*[R][J]*/,
                         uint16_t* worker /*[R][J][K_max]*/, uint32_t* stale /*[R][J][K_max]*/,
                         uint32_t* seq /*[R][J][K_max]*/);

/* Current parameters w_j of every replica into a DEVICE buffer [R][n_params]. */
sim_status sim_get_params(const sim_handle* h, float* w);

/*
 * Full-data empirical risk F(w_j) = (1/N) sum_n f(w_j, xi_n) (Eq. 1) of every replica's current
 * parameters into a DEVICE buffer [R]: the "error" of Section 2.3, for error-versus-wall-clock
 * curves (call it between sim_run calls; the clock of the same update is in the trace).  Linear
 * models: one dense product over all replicas, fp32 logits, fp64 sums in a fixed order.  MLP2: the
 * tensor-core forward pass (bf16 operands x and W1, as in the gradients) over all rows, fp64 sums in a
 * fixed order.  SIM_ERR_ARG for SIM_NONE.  Enqueued on the handle's stream; does not wait.
 */
sim_status sim_eval_loss(sim_handle* h, float* loss);

/*
 * Error against wall clock, the two metrics of Section 2.3 recorded together inside sim_run: with every > 0 the
 * full-data risk F(w_j) (Eq. 1, as sim_eval_loss computes it) of every replica is recorded before the first update
 * (entry 0: F(w_0) at time 0) and after every `every`-th update (entry i: after i * every updates, at the clock of
 * that update), whatever the lengths of the sim_run calls.  every = 0 switches it off.  Only before the first
 * sim_run; not together with sim_set_adasync_loss (SIM_ERR_STATE); SIM_ERR_ARG for SIM_NONE.  One evaluation reads
 * the whole data set: choose `every` accordingly.
 */
sim_status sim_set_eval_every(sim_handle* h, int64_t every);

/* Number of recorded evaluations E (0 before the first sim_run with a risk trace). */
sim_status sim_risk_trace_size(const sim_handle* h, int64_t* n_evals);

/* The risk trace and its clock into caller-owned DEVICE buffers [R][E] (either may be NULL); synchronises the stream. */
sim_status sim_get_risk_trace(const sim_handle* h, float* risk /*[R][E]*/, double* t /*[R][E]*/);

/*
 * The error-runtime curve of Section 2.3 from the risk trace: for each grid time g (DEVICE [n_grid]) the mean over
 * replicas of F(w) - f_star at the replica's last evaluation completed by g (f_star: the caller's F*, e.g. from the
 * normal equations for LSQ; 0 to get the risk itself) and the number of replicas counted (all of them from g = 0 on,
 * since entry 0 is at time 0).  DEVICE outputs [n_grid]; synchronises.  SIM_ERR_STATE without a risk trace.
 */
sim_status sim_risk_curve(const sim_handle* h, const double* grid, int32_t n_grid, float f_star, float* mean_err, int32_t* count);

/*
 * The trade-off across K that motivates AdaSync (Sections 1, 5 and 6: a small K is ahead early, a large K reaches a
 * lower floor): the lower envelope of the risk curves of several simulations of the same problem (typically one
 * handle per K) on a common grid.  env[g] = the smallest mean error at grid time g among the handles, best[g] = the
 * index of the handle that attains it (lowest index on ties).  grid, env, best are DEVICE arrays [n_grid]; every
 * handle needs a risk trace.  Allocates and frees two temporary arrays; synchronises every handle's stream.
 */
sim_status sim_risk_envelope(sim_handle* const* handles, int32_t n_handles, const double* grid, int32_t n_grid, float f_star,
                             float* env, int32_t* best);

/*
 * Error against simulated wall clock on a common time grid - the error-runtime trade-off picture of
 * Sections 1 and 5: for each grid time g (DEVICE array [n_grid]) the mean over replicas of the
 * minibatch loss recorded at the replica's last update completed by g, and the number of replicas
 * that have completed one by then (DEVICE outputs [n_grid]; mean 0 where the count is 0).
 * Synchronises the handle's stream.  SIM_ERR_STATE before the first update.
 */
sim_status sim_error_curve(const sim_handle* h, const double* grid, int32_t n_grid, float* mean_loss, int32_t* count);

/*
 * Diagnostic (no counterpart in the paper): exercises the path by which a device-side wait that runs out is
 * reported.  Every wait in the library's kernels is bounded; when one gives up, the block votes, sets the handle's
 * error word and drains, and the next synchronising call returns SIM_ERR_TIMEOUT and leaves the handle unusable.
 * This call enqueues a one-block kernel that waits about a thousand polls on a barrier nobody arrives at, so that
 * exactly this happens: sim_trace_size / sim_get_* then return SIM_ERR_TIMEOUT and sim_run SIM_ERR_STATE.  The
 * kernel ends by itself; the device and other handles are unaffected.  Returns SIM_OK after enqueueing.
 */
sim_status sim_selftest_wait_timeout(sim_handle* h);

/* Number of parameters of the handle's model (0 for SIM_NONE). */
int64_t sim_n_params(const sim_handle* h);

const char* sim_last_error(const sim_handle* h);
void sim_destroy(sim_handle* h);

/*
 * The random draws on their own (Section 3.1's X_i and Section 2's minibatches), for checking a
 * stream against another implementation.  DEVICE outputs, enqueued on `cuda_stream`:
 *   sim_draw_delays:  out[(r*P + i)*n_seq + s] = compute time of task s of worker i of global
 *                     replica replica_base + r
 *   sim_draw_indices: out[((r*P + i)*n_seq + s)*m + q] = sample index q of that task's minibatch
 */
sim_status sim_draw_delays(sim_delay delay, uint64_t seed, int64_t replica_base, int32_t n_replicas,
                           int32_t P, int32_t n_seq, double* out, void* cuda_stream);
sim_status sim_draw_indices(uint64_t seed, int64_t replica_base, int32_t n_replicas, int32_t P,
                            int32_t n_seq, int64_t n, int32_t m, uint32_t* out, void* cuda_stream);

/*
 * One-shot call on HOST buffers: copies the data set to the device, creates a simulation,
 * runs `iters` updates, copies the trace (same arrays and layout as sim_get_trace, any may be
 * NULL) and the final parameters ([R][n_params], may be NULL) back to host memory, and frees
 * everything.  `problem` holds HOST pointers here.  w0 (host, [n_params]) may be NULL for zeros;
 * K0 / t_interval as in sim_set_adasync.
 */
sim_status sim_simulate_host(const sim_problem* problem, int32_t P, int32_t K, sim_variant variant,
                             sim_delay delay, float eta, int32_t m, uint64_t seed, int32_t n_replicas,
                             int64_t replica_base, const float* w0, int32_t K0, double t_interval,
                             int64_t iters, double* t, float* loss, float* dist2, uint16_t* K_used,
                             uint16_t* worker, uint32_t* stale, uint32_t* seq, float* w_final);

/*
 * A sweep on HOST buffers: the same data set and delay law under n_runs (variant, K) pairs - the
 * comparison of Section 5's error-runtime trade-offs across K and across variants.  The data set
 * is copied to the device once, the runs are simulated concurrently (one stream each) for `iters`
 * updates from w0 (host, may be NULL for zeros), and the clocks, losses and distances come back
 * as [n_runs][R][iters] host arrays (any may be NULL).  `problem` holds HOST pointers.  Everything
 * allocated is freed before returning.
 */
sim_status sim_sweep_host(const sim_problem* problem, int32_t P, int32_t n_runs, const int32_t* variants,
                          const int32_t* Ks, sim_delay delay, float eta, int32_t m, uint64_t seed,
                          int32_t n_replicas, int64_t replica_base, const float* w0, int64_t iters,
                          double* t, float* loss, float* dist2);

/*
 * Clock-only simulation for callers that cannot allocate device memory.  (The paper has no
 * counterpart for this entry point: it exists for the sake of the library's users, not of the
 * method.)
 *
 * Who needs it: code that must not call cudaMalloc while it runs - a service loop in which an
 * allocation would stall every stream of the device, a process whose device memory is owned by a
 * pool that forbids side allocations, a thread sharing the GPU with a job that has already taken
 * the memory it may use.  sim_create / sim_run allocate worker state and a trace; this call
 * allocates nothing, neither directly nor through any library.  It runs the arrival process of
 * Section 2.2 (same variants, delays, growing-K rule and random streams as a SIM_NONE handle,
 * bit for bit) for `iters` updates from update 0 and writes the schedule straight into the
 * caller's DEVICE buffers, all five required:
 *   t [R][iters], K_used [R][iters], worker / stale / seq [R][iters][K_max],
 *   K_max = K, or P when t_interval > 0 (then K0 is the first K and K is ignored).
 * The per-replica worker state lives in one fixed array inside the library image
 * (SIM_NOALLOC_SCRATCH_BYTES of device memory on every GPU that loads the library, held until the
 * process exits), which bounds the problem: P <= SIM_NOALLOC_MAX_P, n_replicas <= SIM_NOALLOC_MAX_REPLICAS and
 * n_replicas * P <= SIM_NOALLOC_MAX_REPLICA_WORKERS; larger requests return SIM_ERR_ARG and launch
 * nothing.  The first call on each device looks up the array's device address and, with CUDA's lazy
 * module loading, is also the moment the driver loads the library's device code and the array itself
 * onto that device (which takes device memory and can fail if none is left): make that first call at
 * start-up, outside any stream capture and before the memory is claimed by others; the promise of
 * no allocation holds for every later call.  All calls on a device share the array and each call clears
 * the part it uses before it starts, so two calls whose GPU work overlaps (different streams or
 * threads) race: serialise them.  Work is enqueued on `cuda_stream`; the call does not wait for
 * it.  On failure sim_noalloc_last_error() describes the cause (per host thread).
 */
#define SIM_NOALLOC_MAX_P 32   /* sim_schedule_noalloc: one warp lane per worker */
#define SIM_NOALLOC_MAX_REPLICAS 4096
#define SIM_NOALLOC_MAX_REPLICA_WORKERS 65536
#define SIM_NOALLOC_SCRATCH_BYTES (1088 * 1024)
sim_status sim_schedule_noalloc(int32_t P, int32_t K, sim_variant variant, sim_delay delay, uint64_t seed,
                                int64_t replica_base, int32_t n_replicas, int32_t K0, double t_interval,
                                int64_t iters, double* t, uint16_t* K_used, uint16_t* worker,
                                uint32_t* stale, uint32_t* seq, void* cuda_stream);
const char* sim_noalloc_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* STRAGGLER_SIM_H */
