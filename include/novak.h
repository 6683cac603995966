/*
 * novak.h -- C ABI of the B200 (sm_100a) NOVAK per-parameter optimizer step.
 *
 * One handle (novak_opt) = one hyperparameter set = one "parameter group".
 * The caller owns every device buffer (parameters, gradients, the state
 * buffer); the library owns the handle and a small device-side work table
 * (tensor records + chunk table) that lets ONE kernel launch cover every
 * tensor of the group.
 *
 * What a step computes, per element, in fp32 (the paper's phases 2, 4-10;
 * Section 5.1, Table 2):
 *     g~ = g                         (variants none, classical)
 *     g~ = g + beta_N (g - m)        (approximation, Eq. 13)
 *     m  = beta1 m + (1-beta1) g~    (Eq. 1)
 *     v  = beta2 v + (1-beta2) g~^2  (Eq. 2)
 *     m^ = m/(1-beta1^t), v^ = v/(1-beta2^t)              (Eq. 5)
 *     u  = m^/(sqrt(v^)+eps)                               (Eq. 17)
 *     u  = beta1 m^ + (1-beta1) u    (classical only, Eq. 16)
 *     theta_fast = theta (1 - alpha lambda) - alpha r_t u  (Eq. 18, 24, 24a)
 *     lookahead on steps with t mod k == 0                 (Eq. 28-31)
 * The per-step scalars (1-beta^t, rho_t, the branch of Eq. 8, r_t, the decay
 * factor, the sync flag) are computed once per step on the host in double
 * precision and passed to the kernel by value (with NOVAK_OPT_GRAPH_CAPTURABLE:
 * by the same code in a one-thread kernel, from a counter in device memory).
 * Around that step, each behind an option and off by default: gradient clipping
 * and centralization (phase 2), adaptive beta (phase 3), layer adaptation and
 * automatic learning-rate scaling (phase 7), the sparse mask (phase 8), bf16
 * parameter copies, bf16 moment storage, the two parameter passes of true
 * Nesterov momentum, a step in two halves for sharded groups.
 *
 * Threading: a handle is not thread safe; use one handle per host thread.
 * Streams: all work of a handle must be issued on one stream (or on streams
 * the caller orders itself): the device work table is updated in stream order.
 * No call synchronises the device unless its description says so (the calls
 * that read a result back).  Pointers named d_* are device pointers,
 * h_* host pointers; "host array of device pointers" means the array lives in
 * host memory and its entries point to device memory.
 */
#ifndef NOVAK_H
#define NOVAK_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct novak_opt novak_opt;

/* Status codes returned by every int-valued call. */
enum {
    NOVAK_OK = 0,
    NOVAK_EINVAL = 1,  /* bad argument; nothing was changed or enqueued      */
    NOVAK_ESTATE = 2,  /* call not valid in the handle's current state       */
    NOVAK_ECUDA = 3,   /* a CUDA runtime call failed; see novak_last_error() */
    NOVAK_ENOMEM = 4   /* host or device allocation failed                   */
};

/* nesterov_variant (Section 4.4).  TRUE needs a closure that re-evaluates the
 * gradient at the look-ahead point, which stays with the caller: for the first
 * N_taylor = NOVAK_OPT_TRUE_NESTEROV_STEPS steps the caller brackets its closure
 * with novak_nesterov_extrapolate / novak_nesterov_restore and the step takes
 * the gradient it is given as Eq. 11's; afterwards (Section 5.2's fallback), and
 * from the first step while N_taylor = 0 (the default, with
 * NOVAK_WARN_TRUE_DOWNGRADED set: Section 7.3's downgrade rule), the variant
 * is APPROX. */
enum {
    NOVAK_NESTEROV_NONE = 0,
    NOVAK_NESTEROV_APPROX = 1,
    NOVAK_NESTEROV_CLASSICAL = 2,
    NOVAK_NESTEROV_TRUE = 3
};

enum { NOVAK_GRAD_F32 = 0, NOVAK_GRAD_BF16 = 1 };

/* Storage type of the moments m and v (NOVAK_OPT_MOMENT_DTYPE).  BF16 is
 * Section 10's "moments in bfloat16, updates accumulated in float32": a step
 * reads the stored values back, does all of its arithmetic (Eq. 1-2, 5, 17) in
 * fp32 on the unrounded m_t, v_t, and stores each rounded to the nearest
 * bfloat16, ties to even.  20 B per element and step instead of 28 (fp32
 * gradients).  With beta2 = 0.999 a step changes v by about a quarter of the
 * spacing of bfloat16 values, so round-to-nearest can hold v still for long
 * stretches; the paper names that sensitivity and gives no remedy, and none is
 * applied here. */
enum { NOVAK_MOMENT_F32 = 0, NOVAK_MOMENT_BF16 = 1 };

/* Lookahead rule applied on steps with t mod k == 0 (Section 4.7).
 * LAST:      slow += alpha_LA (theta_fast - slow); theta = slow.
 *            The slow weights are read and written on those steps only.
 * TRAJ_MEAN: slow += alpha_LA (mean of the window's k fast iterates - slow),
 *            the rule in the proof of Thm 6.2; keeps a running sum (one more
 *            state array, touched every step). */
enum { NOVAK_LOOKAHEAD_LAST = 0, NOVAK_LOOKAHEAD_TRAJ_MEAN = 1 };

/* Keys of novak_set_option / novak_get_option. */
enum {
    NOVAK_OPT_NESTEROV_BETA = 1,  /* beta_N in [0,1); default beta1 (Eq. 13)          */
    NOVAK_OPT_LOOKAHEAD_MODE = 2, /* NOVAK_LOOKAHEAD_*; only before attach             */
    NOVAK_OPT_RECTIFIED = 3,      /* 1 (default): Eq. 8-9; 0: r_t = 1 on every step    */
    NOVAK_OPT_LR = 4,             /* alpha > 0; may change between steps               */
    NOVAK_OPT_BIAS1_POWER = 5,    /* 1 (default) or 2: divide the step by (1-beta1^t)
                                     once more (Eq. 8 taken together with Eq. 24)      */
    NOVAK_OPT_CHUNK_ELEMS = 6,    /* elements per chunk-table entry (multiple of 1024);
                                     only before the first step                        */
    NOVAK_OPT_CTAS_PER_SM = 7,    /* persistent grid = SMs x this; 0: one CTA per chunk */
    NOVAK_OPT_SERPENTINE = 8,     /* 1: walk the chunk table backwards on even steps so
                                     the tail of one step is still in L2 for the next  */
    NOVAK_OPT_WEIGHT_DECAY = 9,   /* lambda >= 0; may change between steps             */
    NOVAK_OPT_DEPENDENT_LAUNCH = 10, /* 1 (default): launch the step kernel with
                                     programmatic stream serialization, so its CTAs
                                     become resident and fetch their work-table
                                     entries while the previous kernel on the stream
                                     drains; they touch no tensor before that kernel
                                     has completed.  0: plain launch               */
    NOVAK_OPT_HOST_SEGMENT_ELEMS = 11, /* novak_step_host pipelines the step in runs of
                                     about this many elements (default 4 Mi; at most
                                     32 runs per step; 0: one run, nothing overlaps)   */
    NOVAK_OPT_CLIP_THRESHOLD = 12, /* c_clip >= 0 of the global-norm gradient clipping
                                     (Section 5.8; the paper's default is 1.0), 0
                                     (default here): off.  May change between steps  */
    NOVAK_OPT_CENTRALIZE = 13,    /* 1: gradient centralization (Eq. 26) on the tensors
                                     that novak_set_tensor_rows gave rows; 0 (default)  */
    NOVAK_OPT_ADAPTIVE_BETA = 14, /* 1: momentum scheduling (Section 4.2): the moment
                                     updates (Eq. 1-2) use beta1(t), beta2(t) of Eq. 3-4;
                                     bias corrections, rho_t, r_t and the classical
                                     blend keep the base values.  0 (default)          */
    NOVAK_OPT_BETA1_TAU = 15,     /* tau_1 > 0 of Eq. 3 (default 1000)                 */
    NOVAK_OPT_BETA2_TAU = 16,     /* tau_2 > 0 of Eq. 4 (default 5000)                 */
    NOVAK_OPT_LAYER_ADAPTATION = 17, /* 1: layer-wise adaptation (Eq. 19 / 25): each
                                     tensor's step is stretched by its trust ratio
                                     clip(||theta_t|| / ||u_t||, 0.1, 10).  Two more
                                     kernels per step read theta, g, m, v once more
                                     (+16 B per element).  0 (default)               */
    NOVAK_OPT_AUTO_LR = 19,       /* 1: automatic learning-rate scaling (Eq. 20-22): the
                                     step is stretched by clip(g_bar / theta_bar, 0.1,
                                     2), moving averages of the global norms of the
                                     gradient as given and of the parameters before
                                     the step.  Runs the statistics pass and reads
                                     the parameters once more (+4 B per element on top
                                     of clipping's +4).  0 (default)                  */
    NOVAK_OPT_AUTO_LR_GAMMA = 20, /* gamma in (0, 1] of Eq. 20-21 (default 0.1)        */
    NOVAK_OPT_TRUE_NESTEROV_STEPS = 21, /* N_taylor >= 0 (Section 5.2; the paper uses
                                     100-200): steps 1..N_taylor of a handle created
                                     with NOVAK_NESTEROV_TRUE apply no correction of
                                     Eq. 13 to the gradient, which the caller has
                                     evaluated at Eq. 10's point; later steps run
                                     APPROX.  0 (default): APPROX from the first step.
                                     NOVAK_ESTATE for any other variant             */
    NOVAK_OPT_MOMENT_DTYPE = 22,  /* NOVAK_MOMENT_*: storage type of m and v; only
                                     before attach (default NOVAK_MOMENT_F32)          */
    NOVAK_OPT_CENTRALIZE_IN_STEP = 24, /* 1 (default): with centralization on and nothing
                                     else that needs the whole gradient first (no
                                     clipping, no automatic learning-rate scaling, no
                                     layer adaptation), novak_step forms the row means
                                     of Eq. 26 inside the step kernel, whose CTAs then
                                     own whole rows (units of 4096 elements or one
                                     row of up to 32768; longer rows keep the
                                     statistics pass): one launch and 28 B per element
                                     instead of three launches and 32 B.  0: always
                                     the statistics pass                               */
    NOVAK_OPT_LAYER_ADAPTATION_IN_STEP = 25, /* 1 (default): with layer adaptation on,
                                     novak_step runs its statistics and the update as
                                     ONE kernel (behind the gradient's own statistics
                                     pass where clipping, centralization or automatic
                                     learning-rate scaling are on): a CTA advances the moments of one run
                                     of chunk-table entries, leaves the direction of
                                     the update in a scratch array (4 B per element of
                                     the group, allocated at the first such step) and
                                     adds up the norms, then applies the update of an
                                     earlier run whose tensor's ratio is known, from
                                     theta and the direction still in L2: about 30 B
                                     per element from DRAM instead of 44.  0: two
                                     statistics kernels, then the step.  Same results
                                     bit for bit                                      */
    NOVAK_OPT_LAYER_ADAPTATION_LEAD = 26, /* elements by which that kernel's updates trail
                                     the statistics beyond what the longest tensor
                                     needs (default 0); only before the first such
                                     step                                              */
    NOVAK_OPT_LAYER_ADAPTATION_GROUP = 27, /* chunk-table entries one CTA of that kernel
                                     takes, 1..8 (default 4); only before the first
                                     such step                                         */
    NOVAK_OPT_GRAPH_CAPTURABLE = 23, /* Without it every step entry point returns
                                     NOVAK_ESTATE while its stream is being captured (a
                                     replay would repeat ONE step's scalars).
                                     1: novak_step may be captured into a CUDA graph
                                     (stream capture) and replayed: the step counter,
                                     the scalars of Eq. 3-9 / 18 and the lookahead
                                     action then live in device memory, advanced by a
                                     one-thread kernel behind the step kernel (one
                                     launch more per step; it computes the next plan
                                     while the step runs), so that every replay is
                                     the NEXT step.  Take one step outside the
                                     capture first (it allocates and uploads the work
                                     table), keep the captured pointer lists alive,
                                     and change options or import checkpoints outside
                                     a capture only: LR and WEIGHT_DECAY reach the
                                     device at the next novak_step CALL, the other
                                     hyperparameters are part of a captured launch.
                                     novak_get_info and novak_export_meta read the
                                     counters back and SYNCHRONISE the device in this
                                     mode.  Not covered (NOVAK_ESTATE): true
                                     Nesterov steps, novak_step_begin / _host /
                                     _noalloc; NOVAK_OPT_SERPENTINE is ignored.  Only
                                     before the first step.  0 (default)              */
    NOVAK_OPT_SPARSE_THRESHOLD = 18 /* tau >= 0 of the sparse updates (Eq. 27): base
                                     directions with |u| <= tau are set to zero before
                                     the classical blend; 0 (default): no mask.  The
                                     comparison is made in fp32 on the kernel's u     */
};

/* Warning bits (novak_info.warnings). */
enum {
    NOVAK_WARN_TRUE_DOWNGRADED = 1u, /* nesterov_variant TRUE runs as APPROX from the
                                        first step (N_taylor = 0)                      */
    NOVAK_WARN_SCALAR_PATH = 2u,     /* some tensor's parameter, state (or bf16 copy)
                                        pointers do not share 16-byte alignment; it
                                        runs on 4-byte accesses                        */
    NOVAK_WARN_NARROW_GRADIENT = 4u  /* some tensor's gradient sits at another offset
                                        from a 16-byte boundary than its parameter; its
                                        gradient is fetched element by element while
                                        parameter and state keep 128-bit accesses      */
};

/* Read-only view of the handle after the last successful step. */
typedef struct novak_info {
    int64_t t;              /* steps taken (1-based index of the last step)        */
    int64_t n_syncs;        /* lookahead synchronisations so far                   */
    int64_t last_sync_step; /* t of the most recent one, 0 if none                 */
    int64_t total_numel;
    int64_t launches;       /* kernels launched by this handle since creation      */
    int64_t record_uploads; /* times novak_step had to copy the tensor records to
                               the device (a pointer list it did not hold yet)     */
    double bc1, bc2;        /* 1-beta1^t, 1-beta2^t of the last step       (Eq. 5) */
    double rho_inf, rho_t;  /*                                          (Eq. 6-7)  */
    double r_t;             /* Eq. 9, or 1 on the un-rectified branch              */
    double step_size;       /* alpha r_t (divided by bc1 when BIAS1_POWER = 2)     */
    double decay;           /* 1 - alpha lambda                           (Eq. 18) */
    int32_t rect_branch;    /* 1: first case of Eq. 8 (rho_t >= 5) was taken       */
    int32_t is_sync;        /* 1: the last step synchronised                       */
    int32_t nesterov_variant; /* variant of that step: TRUE while t <= N_taylor, else
                                 the configured one (APPROX after the fallback)    */
    int32_t lookahead_mode;
    int32_t lookahead_k;
    int32_t n_tensors;
    int32_t n_chunks;
    int32_t grid, block;    /* launch shape of the last step                       */
    uint32_t warnings;
    int32_t grad_processing; /* phase 2 as configured: 0 none, 1 clipping,
                                2 centralization (with or without clipping)        */
    int32_t reserved;
    double beta1_t, beta2_t; /* coefficients the last step's Eq. 1-2 used: the base
                                values, or Eq. 3-4 with NOVAK_OPT_ADAPTIVE_BETA     */
    int32_t layer_adaptation;
    int32_t moment_dtype;    /* NOVAK_MOMENT_*                                      */
} novak_info;

/* Counters and hyperparameters for checkpoint / resume (Table 3: t and the
 * quantities derived from it).  The state arrays themselves are read and
 * written through novak_state_ptrs. */
typedef struct novak_meta {
    uint64_t magic;
    int64_t t, n_syncs, last_sync_step;
    int64_t total_numel;
    double lr, beta1, beta2, eps, weight_decay, nesterov_beta, lookahead_alpha;
    int32_t nesterov_variant, lookahead_k, lookahead_mode, rectified, bias1_power;
    int32_t n_tensors;
    uint32_t warnings;
    int32_t centralize;
    double clip_threshold;
    double beta1_tau, beta2_tau;
    int32_t adaptive_beta;
    int32_t layer_adaptation;
    double sparse_threshold;
    double auto_lr_gamma;
    int32_t auto_lr;
    int32_t true_nesterov_steps; /* N_taylor; nesterov_variant is TRUE when requested */
    int32_t moment_dtype;    /* NOVAK_MOMENT_*; must match the handle's on import   */
    int32_t reserved;
} novak_meta;

/* Algorithm 1, Input / Section 5.8 "Hyperparameter validation".
 * Creates a handle.  lr > 0; beta1, beta2 in [0,1) and beta2 < 1 - 1e-8;
 * eps > 0; weight_decay >= 0; nesterov_variant one of NOVAK_NESTEROV_*;
 * lookahead_k >= 0 (0 = lookahead off); lookahead_alpha in (0,1) when k > 0.
 * NaN fails every test.  Returns NOVAK_EINVAL (and *out = NULL) otherwise.
 * Does no CUDA work.  The library owns *out; release with novak_destroy. */
int novak_create(novak_opt **out, double lr, double beta1, double beta2,
                 double eps, double weight_decay, int nesterov_variant,
                 int lookahead_k, double lookahead_alpha);

/* Frees the handle and its device work table.  Never touches caller buffers.
 * NULL is allowed. */
void novak_destroy(novak_opt *opt);

/* Options not in novak_create's list (Algorithm 1, Hyperparameters).  Values
 * are validated like novak_create's (NOVAK_EINVAL); keys that change the
 * state layout or the chunk table return NOVAK_ESTATE once state is attached
 * (LOOKAHEAD_MODE, MOMENT_DTYPE) or a step was taken (CHUNK_ELEMS). */
int novak_set_option(novak_opt *opt, int key, double value);
int novak_get_option(const novak_opt *opt, int key, double *value);

/* Table 3: bytes of optimizer state for n tensors of numel[i] fp32 elements:
 * m and v always (fp32, or 2 bytes each under NOVAK_MOMENT_BF16), the slow
 * weights when lookahead_k > 0, the running sum in TRAJ_MEAN mode (both fp32).  Includes per-tensor padding (each tensor's slice may start
 * up to 31 elements into a 128-byte aligned slot so that it shares the
 * parameter's alignment).  Returns 0 on bad arguments. */
size_t novak_state_bytes(const novak_opt *opt, const int64_t *numel, int n);

/* Algorithm 1, Initialize: m_0 = v_0 = 0, t = 0.
 * d_state: caller-allocated device buffer, 256-byte aligned, at least
 * novak_state_bytes() long; the caller keeps ownership and must keep it alive
 * while the handle uses it.  d_params (host array of n device pointers, may be
 * NULL) fixes each slice's alignment phase so that state and parameter share
 * 16-byte alignment; with NULL, slices start at their slot's base.  The whole
 * buffer is zero-filled asynchronously on `stream` (a cudaStream_t); the slow
 * weights are set to theta_0 by the first step's kernel (Eq. 28).
 * The device d_state lives on becomes the handle's device: every later call
 * that touches CUDA makes it current for its own duration and puts the
 * caller's device back, so one process may hold handles on several GPUs (a
 * stream passed to a call must belong to the handle's device).
 * Errors: NOVAK_EINVAL (NULL, n <= 0, numel[i] <= 0, misaligned or short
 * buffer, parameter pointer not 4-byte aligned), NOVAK_ECUDA. */
int novak_attach_state(novak_opt *opt, void *d_state, size_t bytes,
                       void *const *d_params, const int64_t *numel, int n,
                       void *stream);

/* One optimizer step over every tensor of the group: ONE kernel launch on
 * `stream`, no synchronisation, no allocation after the first call.
 * d_params: host array of n device pointers to contiguous fp32 tensors,
 *           updated in place (4-byte aligned at least).
 * d_grads:  host array of n device pointers to contiguous gradients of
 *           grad_dtype (fp32, or bf16 widened exactly), read only.
 * numel:    must equal the attached layout (NOVAK_ESTATE otherwise).
 * Pointers may change between steps: the handle keeps the device tensor records
 * of the 8 most recently used (params, grads) pointer lists, so a caller that
 * cycles through a few gradient buffers enqueues nothing but the kernel; a list
 * it does not hold is uploaded in stream order (novak_info.record_uploads).  Tensors whose parameter, gradient and state
 * addresses are congruent modulo 16 bytes run on 128-bit accesses; where only
 * the gradient is off, it alone is fetched element by element
 * (NOVAK_WARN_NARROW_GRADIENT); where parameter and state disagree the tensor
 * runs on 4-byte accesses (NOVAK_WARN_SCALAR_PATH).
 * Errors: NOVAK_EINVAL (NULL, n mismatch, bad dtype, misaligned pointer),
 * NOVAK_ESTATE (no state attached), NOVAK_ENOMEM, NOVAK_ECUDA.  On any error
 * nothing is enqueued and t is unchanged. */
int novak_step(novak_opt *opt, void *const *d_params,
               const void *const *d_grads, const int64_t *numel, int n,
               int grad_dtype, void *stream);

/* One step in two halves, for a group that is cut across several processes
 * (each owning a range of the flattened parameters and calling the library on
 * its own range) AND uses gradient clipping or the automatic learning-rate
 * scaling, whose norms run over the whole group (Section 5.8: with sharded
 * state the step needs this one exchange):
 *
 *   novak_step_begin(...)          this process's statistics: sums of squares of
 *                                  its gradients (and parameters)
 *   novak_local_sums(opt, &d)      d[0..1]: those two sums, in device memory
 *   <caller: all-reduce (sum) of the two doubles over the group's processes,
 *    e.g. NCCL on the same stream, into any device buffer>
 *   novak_step_finish(opt, d_total_sums, stream)
 *                                  norm, clip factor, Eq. 20-22 from the totals,
 *                                  then the update of this process's range
 *
 * Arguments of begin as novak_step.  d_total_sums: device pointer to the two
 * all-reduced doubles; NULL takes the local ones (then the pair equals
 * novak_step).  Between begin and finish no other step call is allowed on the
 * handle (NOVAK_ESTATE), and the gradients must stay unchanged.  With neither
 * clipping nor auto-LR on, begin enqueues nothing and finish is the plain step.
 * Centralization and layer adaptation work on whole tensors and are refused
 * here (NOVAK_ESTATE).  Both calls enqueue on `stream` and return without
 * synchronising. */
int novak_step_begin(novak_opt *opt, void *const *d_params, const void *const *d_grads,
                     const int64_t *numel, int n, int grad_dtype, void *stream);
int novak_local_sums(novak_opt *opt, double **d_sums);
/* The same two sums copied (device to device, on `stream`) into a buffer of the
 * caller's, e.g. the tensor its collective library reduces; zeros when the open
 * step needed no statistics. */
int novak_copy_local_sums(novak_opt *opt, double *d_dst, void *stream);
int novak_step_finish(novak_opt *opt, const double *d_total_sums, void *stream);

/* The same step for a caller whose gradients arrive in, and whose updated
 * parameters return to, HOST memory (pinned memory, or the copies do not
 * overlap anything).  The chunk table is cut into runs of about
 * NOVAK_OPT_HOST_SEGMENT_ELEMS elements; for each run the gradients go
 * h_grads -> d_grads on an upload stream of the handle, the step kernel runs
 * over that run on `stream` once they have arrived, and the updated
 * parameters go d_params -> h_params on a download stream, so that upload,
 * kernel and download of different runs overlap (one kernel launch per run).
 * Everything is ordered behind the work already on `stream`, and work enqueued
 * on `stream` afterwards sees all copies finished.  The first call creates the
 * two streams and their events.  The device tensors remain the master copy;
 * the state stays on the device.  Ranges adjacent in both host and device
 * memory are merged into one copy.  Errors as novak_step, except that after
 * NOVAK_ECUDA part of the step may already have been enqueued. */
int novak_step_host(novak_opt *opt, void *const *h_params,
                    const void *const *h_grads, void *const *d_params,
                    void *const *d_grads, const int64_t *numel, int n,
                    int grad_dtype, void *stream);

/* The paper has no counterpart of this call; it exists for callers that must
 * not allocate device memory.
 *
 * novak_step with its device work table (tensor records + chunk table) kept in
 * an array that is part of the library image itself instead of memory obtained
 * from cudaMalloc.  It is meant for processes in which a framework's pool owns
 * all device memory up front and a later cudaMalloc would fail or fragment it,
 * and for call sites (real-time loops, callbacks of an allocator) where an
 * allocation may not happen at all.  The call itself, on every invocation, makes
 * no cudaMalloc / cudaFree / cudaHostAlloc / event creation; parameters,
 * gradients and the state buffer are the caller's as in novak_step.
 *
 * Gradient clipping, centralization and layer adaptation need scratch memory
 * that the library allocates, so this call returns NOVAK_ESTATE while any of
 * them is switched on.
 *
 * Limits: at most 4096 tensors and 131072 chunk-table entries (= 268 M
 * elements at the default 2048 elements per entry; raise
 * NOVAK_OPT_CHUNK_ELEMS before the first step for larger groups).  Beyond that
 * the call returns NOVAK_EINVAL with the limit in novak_last_error() and does
 * nothing.  The array costs 2.31 MiB on every GPU that loads the library, until
 * the process exits.
 *
 * The array is ONE per GPU and shared by every handle and every call.  It keeps
 * what the last call wrote; each call rewrites, in stream order, the part it
 * reads whenever another handle used the table in between or this handle's
 * pointers changed (nothing in it needs to start from zero).  Two calls that
 * may overlap on the GPU (different streams, no ordering between them) race on
 * the table: order them yourself.  On the HOST the call may be made from several
 * threads at once, each with a handle of its own: the library keeps track of
 * whose records the table holds under one process-wide lock that covers the
 * upload and the launch, so a kernel is always enqueued behind its own handle's
 * records.  NOVAK_OPT_CTAS_PER_SM caps the grid as in novak_step.
 *
 * The first call on each device looks up the array's device address (with that
 * device current); make that first call outside any stream capture.
 * Arguments, results and errors otherwise as novak_step; both calls may be
 * mixed on one handle and advance the same step counter. */
int novak_step_noalloc(novak_opt *opt, void *const *d_params,
                       const void *const *d_grads, const int64_t *numel, int n,
                       int grad_dtype, void *stream);

/* Phase 2, gradient centralization (Eq. 26; Table 2: "use_gc = true, dim > 1").
 * rows[i] (host array, n entries) is the size of dimension 0 of tensor i when
 * the tensor has more than one dimension, else 0.  With NOVAK_OPT_CENTRALIZE on,
 * a tensor with rows[i] > 0 is treated as rows[i] x (numel[i]/rows[i]) and the
 * mean of each row (all of dimensions 1..d) is subtracted from the row's
 * gradient before the Nesterov approximation; tensors with rows[i] = 0 are left
 * as they are.  Call after novak_attach_state; may be called again between steps.
 * Errors: NOVAK_ESTATE (nothing attached), NOVAK_EINVAL (NULL, n mismatch,
 * negative rows, numel not a multiple of rows, a tensor with rows of 2^31 or more
 * elements).
 *
 * Phase 2 as a whole (Section 5.1, Table 2, Section 5.8), when clipping or
 * centralization is on: novak_step first runs a statistics pass (two kernels)
 * that reads the gradient once and leaves in device memory (a) the global L2
 * norm of the raw gradient over every tensor of the group and the clip factor
 * c_clip/||g|| (1 when ||g|| <= c_clip), (b) the row means; the step kernel
 * then uses g' = factor * (g - row mean).  Clipping acts on the norm of the raw
 * gradient, before any other processing (Section 7.3).  Three launches per
 * step, no host synchronisation, no floating-point atomics (results are
 * bit-identical from run to run); the scratch (about 16 B per chunk-table entry
 * + 8 B per row + 48 B per 16384 elements of tensors with rows) is allocated by
 * the first such step and again when the rows change.
 * novak_step_noalloc refuses to run in this mode (NOVAK_ESTATE). */
int novak_set_tensor_rows(novak_opt *opt, const int64_t *rows, int n);

/* Mixed-precision training keeps fp32 master parameters in the optimizer and a
 * bf16 copy for the forward and backward passes (the paper names reduced
 * precision as future work, Section 10.3, without fixing a rule; this is the
 * part of it that has an exact definition).  d_copies: host array of n device
 * pointers to contiguous bf16 tensors of numel[i] elements, 2-byte aligned,
 * caller-owned.  Every later step (novak_step, novak_step_host,
 * novak_step_noalloc) stores, beside each updated fp32 parameter, its value
 * rounded to nearest even in bf16 (+2 B per element written; no separate cast
 * kernel).  Nothing reads the copies.  A copy whose address is not congruent to
 * half its parameter's address modulo 8 puts the tensor on 4-byte accesses
 * (NOVAK_WARN_SCALAR_PATH).  NULL switches the copies off.
 * Errors: NOVAK_ESTATE (nothing attached), NOVAK_EINVAL (n mismatch, NULL or
 * odd pointer). */
int novak_set_param_copies(novak_opt *opt, void *const *d_copies, int n);

/* Convergence monitoring (Section 5.8 tracks ||g_t||): the global gradient norm
 * and the clip factor of the last step that ran phase 2.  Copies 16 bytes from
 * the device and SYNCHRONISES `stream`.  Either output may be NULL.
 * NOVAK_ESTATE when no such step has run. */
int novak_get_grad_stats(novak_opt *opt, double *norm, double *factor, void *stream);

/* Layer-wise adaptation (Eq. 19 / 25, NOVAK_OPT_LAYER_ADAPTATION): the trust
 * ratio of every tensor as the last step used it, h_out[i] for tensor i (host
 * array of n floats).  The ratio is ||theta_t||_2 / ||u_t||_2 clipped to
 * [0.1, 10], theta_t the parameters before the step, u_t the step's base
 * direction (Eq. 17); 1 where ||u_t|| = 0.  Copies n floats from the device and
 * SYNCHRONISES `stream`.  NOVAK_ESTATE when no such step has run. */
int novak_get_trust_ratios(novak_opt *opt, float *h_out, int n, void *stream);

/* Test hook for the one place where a kernel of this library waits for another
 * CTA (the update part of the one-launch layer adaptation waits for its tensor's
 * ratio; see NOVAK_OPT_LAYER_ADAPTATION_IN_STEP).  Runs that wait, on `stream`, on
 * a word that nothing publishes, and SYNCHRONISES: *gave_up = 1 when the wait
 * returned empty-handed, *seconds = how long it waited on the device (about two
 * seconds: the bound).  Allocates and frees 32 bytes of device memory.  Nothing
 * else on the device is touched; the handle only supplies the device and the
 * error text.  The paper has no counterpart. */
int novak_selftest_bounded_wait(novak_opt *opt, int *gave_up, double *seconds, void *stream);

/* True Nesterov momentum, Section 4.4 (Eq. 10-12) and Section 5.8 ("True
 * Nesterov closure").  The gradient of Eq. 11 is the caller's to compute; these
 * two calls do the parameter traffic around it for a handle created with
 * NOVAK_NESTEROV_TRUE (NOVAK_ESTATE otherwise):
 *
 *   novak_nesterov_extrapolate   save <- theta_{t-1};
 *                                theta <- theta_{t-1} + beta_N m_{t-1}   (Eq. 10)
 *   ... the caller's forward and backward pass at theta~ (Eq. 11) ...
 *   novak_nesterov_restore       theta <- save
 *   novak_step(..., that gradient)      (no Eq. 13 correction while t <= N_taylor)
 *
 * or, one pass and 8 bytes per element less, without the restore:
 *
 *   novak_nesterov_extrapolate
 *   ... the caller's forward and backward pass at theta~ ...
 *   novak_step(..., that gradient)      reads theta_{t-1} from the save buffer and
 *                                       writes theta_t over theta~ in the parameters
 *
 * (novak_step only, with the d_params of the extrapolate call; the result is bit
 * for bit that of the three-call form.  novak_nesterov_restore stays for callers
 * that abandon the step.)
 *
 * One kernel each over the handle's chunk table, enqueued on `stream` (a
 * cudaStream_t; NULL: the default stream); no host synchronisation.  In fp32:
 * one fused multiply-add per element; the restored parameters are bit for bit
 * the saved ones.
 *
 * d_params, numel, n: DEVICE pointers and sizes as in novak_step (fp32, the
 * attached layout).  d_save: DEVICE buffer the CALLER owns, aligned to 16
 * bytes, of at least novak_nesterov_save_bytes() bytes (0 before attach; the
 * size of one state array), laid out like a state array; it must stay valid
 * and unchanged until the restore, which takes the same d_params and d_save.
 * Between extrapolate and restore novak_import_meta,
 * NOVAK_OPT_TRUE_NESTEROV_STEPS and every step entry point other than
 * novak_step return NOVAK_ESTATE.  m_{t-1} = 0 before the
 * first step, so the first look-ahead leaves theta where it is.
 * Errors: NOVAK_EINVAL (NULL, a misaligned or short buffer, restore with other
 * buffers), NOVAK_ESTATE (not attached, wrong variant, a tensor list other
 * than the attached one, extrapolate twice, restore without extrapolate),
 * NOVAK_ENOMEM / NOVAK_ECUDA; the handle and the parameters are unchanged on
 * error. */
size_t novak_nesterov_save_bytes(const novak_opt *opt);
int novak_nesterov_extrapolate(novak_opt *opt, void *const *d_params, void *d_save,
                               size_t save_bytes, const int64_t *numel, int n, void *stream);
int novak_nesterov_restore(novak_opt *opt, void *const *d_params, const void *d_save,
                           size_t save_bytes, const int64_t *numel, int n, void *stream);

/* Automatic learning-rate scaling (Eq. 20-22, NOVAK_OPT_AUTO_LR).  Its two
 * moving averages live in device memory.  get: copies them and the last step's
 * factor (Eq. 22) to the host and SYNCHRONISES `stream` (before the first such
 * step: the initial zeros, or what set put in; any output may be NULL).  set:
 * for resuming from a checkpoint; the values are written to the device in
 * stream order at the next step.  NOVAK_EINVAL for negative or non-finite
 * values. */
int novak_get_auto_lr_state(novak_opt *opt, double *g_bar, double *theta_bar, double *scale,
                            void *stream);
int novak_set_auto_lr_state(novak_opt *opt, double g_bar, double theta_bar);

/* Counters and the last step's scalars (bit-exact step and sync indices). */
int novak_get_info(const novak_opt *opt, novak_info *out);

/* The host-side scalar plan for an arbitrary 1-based step index t, without
 * touching the handle's counters or the device (Eq. 5-9, 18).  Fills bc1, bc2,
 * rho_inf, rho_t, r_t, step_size, decay, rect_branch, is_sync of *out; the
 * other fields are copied from the handle. */
int novak_plan(const novak_opt *opt, int64_t t, novak_info *out);

/* Device pointers of tensor i's state slices (NULL for arrays the mode does
 * not keep): numel[i] elements each, fp32 but for m and v under
 * NOVAK_MOMENT_BF16 (bfloat16).  For checkpointing and for tests; valid after
 * attach. */
int novak_state_ptrs(const novak_opt *opt, int tensor, void **d_m, void **d_v,
                     void **d_slow, void **d_acc);

/* Checkpoint / resume of everything that is not a device array.  Import
 * requires an attached state of the same tensor list and the same
 * layout-relevant hyperparameters (NOVAK_ESTATE otherwise). */
int novak_export_meta(const novak_opt *opt, novak_meta *out);
int novak_import_meta(novak_opt *opt, const novak_meta *in);

/* Host-only helper exposing the chunk-table builder: splits n tensors of
 * numel[i] elements whose first element sits phase[i] (0..31, may be NULL)
 * elements past a 128-byte boundary into entries (tensor, offset, len) with
 * len <= chunk_elems, every entry after a tensor's first starting on a
 * 128-byte boundary.  Writes up to cap entries and returns the number the
 * table needs (negative on bad arguments). */
int64_t novak_build_chunks(const int64_t *numel, const int32_t *phase, int n,
                           int64_t chunk_elems, int32_t *tensor, int64_t *offset,
                           int32_t *len, int64_t cap);

/* Host-only helper exposing how the statistics pass of the centralization cuts
 * tensors with rows into units: groups of whole rows of up to 8192 elements,
 * about 16384 elements per group (part_len = 0), or, for longer rows, slices
 * [part_off, part_off + part_len) of at most 16384 elements of one row
 * (n_rows = 1), consecutive in the table.  rows[i] as in novak_set_tensor_rows.  Writes up to cap entries and
 * returns the number the table needs (negative on bad arguments). */
int64_t novak_build_row_units(const int64_t *numel, const int64_t *rows, int n, int32_t *tensor,
                              int64_t *row0, int64_t *n_rows, int64_t *part_off,
                              int64_t *part_len, int64_t cap);

/* Host-only helper exposing the units of the step kernel that centralizes by
 * itself (NOVAK_OPT_CENTRALIZE_IN_STEP): whole rows [row0, row0 + n_rows) of the
 * tensors whose rows have at most 32768 elements, as many rows as fit in 4096
 * elements (at least one, at most 256) per unit; tensors with longer rows get
 * no unit (they keep the statistics pass).  Arguments and result as in
 * novak_build_row_units. */
int64_t novak_build_own_units(const int64_t *numel, const int64_t *rows, int n, int32_t *tensor,
                              int64_t *row0, int64_t *n_rows, int64_t cap);

/* Host-only helper exposing the work list of the one-launch form of layer
 * adaptation (NOVAK_OPT_LAYER_ADAPTATION_IN_STEP).  The group's chunk table lists
 * tensor i's entries at [tensor_first[i], tensor_first[i+1]) (n + 1 values,
 * non-decreasing, tensor_first[0] = 0).  An item is a run of consecutive entries
 * of one tensor: the tensor's first entry alone, the others in runs of `group`
 * (1..8); items come in tensor order.  out[k] is the k-th item's first chunk-
 * table index, count[k] its number of entries (either array may be NULL).  CTA b
 * of the kernel takes the statistics of item b and the update of item b - *lag:
 * *lag (may be NULL) is the number of items of the tensor that has most, minus
 * one, plus ceil(lead_entries / group).  Writes up to cap items and returns the
 * number of items (negative on bad arguments). */
int64_t novak_build_adapt_order(const int32_t *tensor_first, int n, int64_t lead_entries, int group,
                                int32_t *out, int32_t *count, int64_t cap, int64_t *lag);

/* Text of the last error on this handle ("" if none).  Owned by the handle. */
const char *novak_last_error(const novak_opt *opt);

#ifdef __cplusplus
}
#endif
#endif /* NOVAK_H */
