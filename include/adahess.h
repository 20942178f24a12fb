/*
 * adahess.h - C ABI of the batched AdaHessian + elastic-averaging round on one GPU.
 *
 * The library keeps K simulated workers and one master of a data-parallel system
 * (Xu & Carr, "A Dynamic Weighting Strategy to Mitigate Worker Node Failure in
 * Distributed Deep Learning", Sec. II: one master, several workers, each starting
 * as a copy of the master) as a batched [K, P] binary32 state in device memory:
 *
 *     x[K][P]  worker parameters      m[K][P]  first moment (EMA of the gradient)
 *     c[P]     master parameters      v[K][P]  second moment (EMA of the squared,
 *                                              spatially averaged Hessian diagonal)
 *
 * One *round* is one local AdaHessian step of every active worker
 * (ah_local_step); every tau-th round the caller also runs the elastic exchange
 * with the master (easgd_exchange), with per-worker coefficients from the dynamic
 * weighting rule (dw_weights_next) and a seeded failure mask (dw_mask_next).
 *
 * Conventions
 *   - Every function returns an int status: AH_OK (0) or a negative AH_ERR_* code.
 *     Nothing throws, aborts or traps across this boundary.
 *   - "device pointer" = memory of the handle's CUDA device; "host pointer" =
 *     ordinary host memory.  Host arrays are copied during the call and may be
 *     reused as soon as it returns.
 *   - All kernels are enqueued on the handle's stream and the calls return without
 *     waiting, except where a function is marked "synchronises".
 *   - A handle must not be used from two threads at once.  The handle's CUDA device
 *     must be the calling thread's current device for every call after ah_init.
 *   - Arithmetic: IEEE binary32, round-to-nearest, one rounding per operation in
 *     the order the formulas below are written (no fused multiply-add).
 */
#ifndef ADAHESS_H_
#define ADAHESS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes -------------------------------------------------------- */
#define AH_OK                 0
#define AH_ERR_INVALID_ARG   (-1)  /* null pointer, K/P/period out of range, bad enum      */
#define AH_ERR_ALIGN         (-2)  /* device pointer not 16-byte aligned, or ld % 4 != 0    */
#define AH_ERR_SEGMENTS      (-3)  /* segment table unsorted, overlapping, out of range,
                                      block > AH_MAX_BLOCK, or length % block != 0         */
#define AH_ERR_ALLOC         (-4)  /* device or host allocation failed / workspace too small */
#define AH_ERR_CUDA          (-5)  /* a CUDA runtime call failed; see ah_last_cuda_error    */
#define AH_ERR_STATE         (-6)  /* call out of order (e.g. weights asked for before a
                                      step with want_dist = 1 produced the distances)      */
#define AH_ERR_INTERNAL      (-7)  /* the device status word was set by a kernel            */
#define AH_ERR_TOO_LARGE     (-8)  /* problem exceeds a fixed capacity (ah_distances_static) */

#define AH_MAX_WORKERS  256        /* K <= 256                                              */
#define AH_MAX_BLOCK    128        /* spatial block kh*kw <= 128 (covers 11 x 11 kernels)   */
#define AH_MAX_HIST     32         /* history depth p of the raw score <= 32                */
#define AH_MAX_SAMPLES  8          /* Hutchinson samples per step <= 8                      */
#define AH_ROUND_AUTO   0xFFFFFFFFu
#define AH_STATIC_SCRATCH_ENTRIES (1 << 17)  /* doubles per row of the built-in scratch     */
#define AH_DEVICE_NONE  (-2)       /* ah_alloc.device: bookkeeping-only handle, no GPU      */
/* ah_hyper.want_dist */
#define AH_DIST_NONE      0        /* no distances this round                               */
#define AH_DIST           1        /* also ||x_i - c||^2 for all K workers                  */
#define AH_DIST_AND_RULE  2        /* ... and then the weighting rule of Sec. V-B on the device */

/* ---- types ---------------------------------------------------------------- */
typedef struct ah_ctx ah_ctx;      /* opaque; created by ah_init, freed by ah_destroy       */

/* One parameter tensor inside the flat parameter row: elements
 * [offset, offset + length).  block = kh*kw for a convolution kernel stored
 * [c_out][c_in][kh][kw] (each filter is one run of `block` consecutive entries over
 * which the Hessian diagonal is averaged), 1 for any other tensor.  Segments must
 * be sorted by offset and disjoint; indices covered by no segment behave as
 * block = 1.  length must be a multiple of block.  flags: reserved, 0. */
typedef struct {
    uint64_t offset;
    uint64_t length;
    uint32_t block;
    uint32_t flags;
} ah_segment;

/* Hyper-parameters of one local step. */
typedef struct {
    float lr;             /* eta                                                            */
    float beta1, beta2;   /* EMA rates of the first and second moment                       */
    float eps;            /* added to the denominator                                       */
    float hessian_power;  /* k: denominator is (sqrt(vhat))^k + eps; 1 and 0.5 are exact    */
    float weight_decay;   /* 0 = none; else the step direction gains weight_decay * x       */
    uint32_t round;       /* index t of the Rademacher stream; AH_ROUND_AUTO = the handle's
                             own 1-based count of ah_local_step calls                       */
    const uint8_t *active;/* host pointer, K bytes, or NULL (all active): 0 = worker i
                             skips this step entirely (its x, m, v, step count stay)        */
    int want_dist;        /* AH_DIST: also compute n2_i = ||x_i - c||^2 after the step, for
                             all K workers, into the handle (read by dw_weights_next or by
                             the device forms of the rule).  AH_DIST_AND_RULE: the weighting
                             rule of Sec. V-B is also owed on these distances, on the device,
                             with the moving rate rule_alpha: it runs where the distances
                             are assembled, and the next easgd_exchange_dynamic or
                             easgd_exchange_then_step (dynamic != 0), which must name the
                             same alpha, uses its coefficients.  AH_DIST_NONE: neither.    */
    int n_samples;        /* Hutchinson samples per step, 1 .. AH_MAX_SAMPLES; 0 means 1     */
    uint64_t hvp_sample_stride; /* elements from sample s to sample s + 1 inside hvp (a
                             multiple of 4, at least K * ld); ignored for one sample        */
    float rule_alpha;     /* moving rate alpha of h1 / h2, read with AH_DIST_AND_RULE only  */
} ah_hyper;

/* Hyper-parameters of one first-order local step (sgd_local_step). */
typedef struct {
    float lr;             /* eta                                                            */
    float momentum;       /* delta in [0, 1); 0 = plain SGD, the velocity is not touched     */
    const uint8_t *active;/* host pointer, K bytes, or NULL (all active), as in ah_hyper    */
    int want_dist;        /* AH_DIST = also compute ||x_i - c||^2 after the step, as in
                             ah_hyper (AH_DIST_AND_RULE is not offered here: these methods
                             exchange with a fixed moving rate)                              */
} sgd_hyper;

/* Optional placement: caller-owned device memory and stream.  workspace must be
 * 256-byte aligned, at least ah_workspace_bytes() long, and outlive the handle; the
 * library never frees it.  With opt == NULL the handle allocates its own memory
 * with cudaMalloc on the current device and uses the default stream. */
typedef struct {
    void  *workspace;        /* device pointer or NULL (= allocate)                         */
    size_t workspace_bytes;
    void  *cuda_stream;      /* cudaStream_t, or NULL for the default stream                */
    int    device;           /* CUDA device ordinal, -1 for the current device, or
                                AH_DEVICE_NONE: a handle that holds no device state and
                                makes no CUDA call.  It serves only the host-side
                                bookkeeping (dw_config, dw_mask_next,
                                dw_weights_from_norm2, the host selectors of
                                ah_state_get/set), e.g. on a coordinator without a GPU;
                                every other call returns AH_ERR_STATE.                  */
} ah_alloc;

/* Which part of the state ah_state_get / ah_state_set address. */
enum {
    AH_X = 0,          /* float  [K][P] (worker = -1) or [P] (worker = i)                   */
    AH_M = 1,          /* same shape                                                        */
    AH_V = 2,          /* same shape                                                        */
    AH_CENTER = 3,     /* float  [P]   master parameters (worker ignored)                   */
    AH_NORM2 = 4,      /* double [K]   last ||x_i - c||^2 (host side only)                  */
    AH_STEP = 5,       /* uint32 [K]   steps taken by each worker (host side only)          */
    AH_UHIST = 6,      /* double [K][p+1] ring of u_i, newest first (host side only)        */
    AH_DOWN_UNTIL = 7, /* uint32 [K]   first round at which each worker is up again (host)  */
    AH_ROUND = 8,      /* uint32 [2]   {calls to ah_local_step, ring filled flag} (host)    */
    AH_INFO = 9,       /* uint32 [4]   {tiles, runs, elements per tile, row stride} (get only)  */
    AH_RUNS = 10,      /* uint32 [runs][4]  {start, end, block, reciprocal}: the row cut into
                          maximal runs of equal spatial block (get only, host)              */
    AH_TILES = 11,     /* uint32 [tiles][4] {first run, e0, e1, flags}: each tile's range
                          widened to whole spatial blocks [e0, e1); flags bit 0 = the tile
                          touches a block > 1, bit 1 = every such block is a 3 x 3 kernel
                          (get only, host)                                                  */
    AH_WEIGHTS = 12    /* float  [2K]  h2[0..K) then h1[0..K): the last output of the
                          weighting rule on the device (host side only); part of a
                          checkpoint when lagged one-pass rounds are used                   */
};

/* ---- life cycle ------------------------------------------------------------ */

/* Bytes of device workspace a handle for (K, P) with nseg segments needs.
 * Host-only arithmetic; touches no GPU. */
int ah_workspace_bytes(int K, uint64_t P, int nseg, size_t *out);

/* Create a handle for K workers of P parameters each (Sec. II set-up).
 *   segs/nseg : host pointer to the tensor table (copied); nseg may be 0.
 *   opt       : optional placement, may be NULL.
 * On return m = v = 0, step counts = 0, x and c are zero: load the master with
 * ah_state_set(AH_CENTER) and call ah_broadcast_center.  1 <= K <= AH_MAX_WORKERS,
 * 1 <= P < 2^31.  Errors: INVALID_ARG, SEGMENTS, ALLOC, CUDA. */
int ah_init(ah_ctx **out, int K, uint64_t P, const ah_segment *segs, int nseg,
            const ah_alloc *opt);

/* Free the handle and any memory it allocated itself.  Synchronises. NULL is OK. */
int ah_destroy(ah_ctx *h);

/* Copy state in / out.  `which` is one of the AH_* selectors above; `worker` picks
 * one row of AH_X/AH_M/AH_V or is -1 for all K rows packed as [K][P].  For the
 * float selectors the other side may be a device pointer (on_device = 1) or a
 * host pointer (0); the host-side selectors (AH_NORM2 ... AH_ROUND) take host
 * pointers only.  ah_state_get synchronises the handle's stream; ah_state_set is
 * ordered after earlier work on the stream and returns when the copy is done.
 * Together they give an exact snapshot for checkpoint and resume.  Where an exchange is
 * still to come when the snapshot is taken (its distances measured, the pull deferred to
 * the next step): if the rule has not run yet, AH_NORM2 belongs to the snapshot, and
 * setting it makes those distances pending again on the restored handle, for the host
 * and the device forms of the rule alike; if the rule has run on the device
 * (AH_DIST_AND_RULE), AH_WEIGHTS belongs to it, and the restored run hands those
 * coefficients to that one exchange as caller weights (dynamic == 0): same bits. */
int ah_state_set(ah_ctx *h, int which, int worker, const void *src, int src_on_device);
int ah_state_get(ah_ctx *h, int which, int worker, void *dst, int dst_on_device);

/* x_i <- c for every worker: each worker starts as a copy of the master (Sec. II). */
int ah_broadcast_center(ah_ctx *h);

/* ---- the round --------------------------------------------------------------- */

/* Rademacher vectors of round `round` (Sec. IV-B, Hutchinson's method) as +-1.0f:
 * dst[i*ld + j] = z_{round,i,j}, device pointer, ld >= P.  z is a pure function
 * of (z_seed, round, i, j): Philox4x32-10 with key (z_seed low, z_seed high) and
 * counter (j >> 7, i, round, 0); element j reads bit (j & 31) of output word
 * (j >> 5) & 3; bit 0 -> +1, bit 1 -> -1.  A caller forms the Hessian-vector
 * product Hz with this z and hands it to ah_local_step, which regenerates the same
 * z internally (no z buffer is read there). */
int ah_sample_z(ah_ctx *h, uint64_t z_seed, uint32_t round, float *dst, uint64_t ld);

/* The same for Hutchinson sample `sample` (0 .. AH_MAX_SAMPLES-1) when a step uses
 * several: sample s replaces the last counter word 0 by 256 s.  Sample 0 is
 * ah_sample_z. */
int ah_sample_z_n(ah_ctx *h, uint64_t z_seed, uint32_t round, uint32_t sample, float *dst,
                  uint64_t ld);

/* One local AdaHessian step of every active worker (Sec. IV-B; Eq. 4), fused in
 * one pass over the state.  For worker i with t_i = its step count after this step:
 *     D      = z (.) hvp                     Hutchinson estimate; with n_samples = n > 1
 *                                            D = (sum_s z_s (.) hvp_s) / n, summed in
 *                                            ascending s, hvp_s = hvp + s * stride
 *     Dbar   = block mean of D               spatial averaging inside each tensor,
 *                                            summed in ascending index order
 *     m      = beta1*m + (1-beta1)*grad
 *     v      = beta2*v + ((1-beta2)*Dbar)*Dbar
 *     mhat   = m / (1-beta1^t_i),  vhat = v / (1-beta2^t_i)
 *     x      = x - lr * ( mhat / ((sqrt vhat)^k + eps)  [+ weight_decay * x] )
 * grad, hvp: device pointers, [K][ld] row-major, ld >= P, ld % 4 == 0, 16-byte
 * aligned, read only, must stay valid until the stream has run the step.
 * With hy->want_dist the squared distances ||x_i - c||^2 (binary32 difference,
 * squared and summed in double, pairwise order) are measured by the same kernel: it
 * leaves one sum per worker and tile of 1024 parameters in the workspace (a worker that
 * sits the step out is measured too: only its x is read).  The upper levels of the
 * pairwise tree are formed by whoever needs the K distances next.  An exchange that
 * rides on the next local step with the rule's coefficients (easgd_exchange_then_step,
 * dynamic != 0; ah_local_step_exchange, lagged != 0) does it at the head of its own
 * kernel, runs the weighting rule there (u = log ||x_i - c||, Eqs. 10-11, h1 / h2 of
 * Sec. V-B; same bits as dw_weights_next) and leaves distances, coefficients and history
 * where the other calls find them: between measuring the distances and using the
 * coefficients lies no launch, no copy and no wait of the host.  Every other reader
 * (dw_weights_next, easgd_exchange_dynamic, ah_state_get/set of the distances, the
 * coefficients or the history, dw_config, the next distance round if a rule is still
 * owed) first has a small kernel of its own assemble them.
 * A call that returns an error other than AH_ERR_CUDA leaves the handle unchanged.
 * Errors: INVALID_ARG, ALIGN, CUDA. */
int ah_local_step(ah_ctx *h, const float *grad, const float *hvp, uint64_t ld,
                  uint64_t z_seed, const ah_hyper *hy);

/* One first-order local step of every active worker, the local optimiser of the
 * EASGD and EAMSGD methods the paper compares against (Sec. VI; Sec. VII uses
 * eta = 0.01, delta = 0.5):
 *     momentum == 0 (Eqs. 2-3):   x = x - lr * grad
 *     momentum  > 0:              u = momentum * u - lr * grad;   x = x + u
 * The velocity u lives in the handle's first-moment rows (AH_M); the second-moment
 * rows are not touched.  A handle should be driven by one kind of local step.  grad,
 * ld, active, want_dist and the step counts behave as in ah_local_step; no Rademacher
 * stream is consumed.  Memory traffic: 12 bytes per parameter update, 20 with momentum.
 * Errors: INVALID_ARG, ALIGN, CUDA. */
int sgd_local_step(ah_ctx *h, const float *grad, uint64_t ld, const sgd_hyper *hy);

/* An exchange round in one pass over the state: the local step of ah_local_step
 * followed at once, tile by tile, by the weighted pull of easgd_exchange
 * (asynchronous == 0) or easgd_exchange_async (asynchronous != 0, order as there), so
 * that x is read and written once instead of twice.  The result is bit for bit that of
 * the two calls in sequence with the same coefficients:
 *     for every column j, workers i in arrival order:
 *         x_ij <- local step (if active_i);  n2_i += (x_ij - c_j)^2 (if hy->want_dist)
 *         if worker_mask[i]:  pull of x_ij and the master by h1_i, h2_i   (Eqs. 12-13)
 * The coefficients must be known before the step:
 *   lagged == 0: weights (host, 2K floats: h2 then h1) or, when NULL, alpha for all;
 *   lagged != 0: the dynamic rule of Sec. V-B runs on the device after this round's
 *       distances (hy->want_dist must be 1, weights NULL) and its coefficients serve the
 *       NEXT lagged round: a lagged round pulls with the most recent output of the rule on
 *       the device (from an earlier lagged round or from easgd_exchange_dynamic), or with
 *       alpha while the rule has not yet run there.  This is the
 *       paper's "estimate of the master model": the score follows the distances with a
 *       delay of one communication period, and no call waits for the GPU.
 * Memory traffic: 32 bytes per parameter update (one Hutchinson sample) plus 8
 * per parameter for the master row, 8 per (worker, parameter) less than the two calls.
 * Errors: INVALID_ARG, ALIGN, STATE, CUDA. */
int ah_local_step_exchange(ah_ctx *h, const float *grad, const float *hvp, uint64_t ld,
                           uint64_t z_seed, const ah_hyper *hy, const uint8_t *worker_mask,
                           const float *weights, float alpha, const uint16_t *order,
                           int asynchronous, int lagged);

/* The exchange of the round just finished and the local step of the next round in one
 * pass: tile by tile, each worker first meets the master (easgd_exchange, or
 * easgd_exchange_async with `order` when asynchronous != 0) and then takes its local
 * step (ah_local_step) on the pulled parameters.  Bit for bit the result of the two
 * calls in sequence; x is read and written once instead of twice.  Unlike
 * ah_local_step_exchange nothing lags: the coefficients are those of this exchange,
 *   dynamic == 0: weights (host, 2K floats) or, when NULL, alpha for all;
 *   dynamic != 0: the pass reads the output of the rule of Sec. V-B on the device: what
 *       the last step left there if it ran with AH_DIST_AND_RULE (alpha must be the same,
 *       else INVALID_ARG), else the rule is launched first on the distances that step left
 *       (as easgd_exchange_dynamic; weights must be NULL; STATE if none are pending).
 * worker_mask says who takes part in the exchange; hy->active who takes the step.
 * hy->want_dist must be 0 (the distances to the new master are only defined once every
 * worker has met it): with a communication period of one round use
 * ah_local_step_exchange or the separate calls.  Nothing waits for the GPU.
 * Errors: INVALID_ARG, ALIGN, STATE, CUDA. */
int easgd_exchange_then_step(ah_ctx *h, const float *grad, const float *hvp, uint64_t ld,
                             uint64_t z_seed, const ah_hyper *hy, const uint8_t *worker_mask,
                             const float *weights, float alpha, const uint16_t *order,
                             int asynchronous, int dynamic);

/* The first-order counterpart of easgd_exchange_then_step: the exchange of the round
 * just finished (easgd_exchange, or easgd_exchange_async with `order` when
 * asynchronous != 0; weights host 2K floats or NULL = alpha for all, the fixed moving
 * rate of EASGD / EAMSGD) and the next sgd_local_step in one pass over x; bit for bit
 * the two calls in sequence.  hy->want_dist must be 0.  Traffic: 12 bytes per update
 * (20 with momentum) + 8 per parameter, instead of + 8 per (worker, parameter) + 8.
 * Errors: INVALID_ARG, ALIGN, STATE, CUDA. */
int easgd_exchange_then_sgd_step(ah_ctx *h, const float *grad, uint64_t ld, const sgd_hyper *hy,
                                 const uint8_t *worker_mask, const float *weights, float alpha,
                                 const uint16_t *order, int asynchronous);

/* Parameters of the dynamic weighting rule (Sec. V-B): history depth p, the
 * coefficients c_0..c_{p-1} of Eqs. 10-11 (c_0 weighs the newest difference; they
 * should sum to 1) and the threshold kappa < 0 of h1/h2.  Defaults set by ah_init:
 * p = 4, c = (0.4, 0.3, 0.2, 0.1), kappa = -0.1.  Clears the history. */
int dw_config(ah_ctx *h, int p_hist, const double *c, double kappa);

/* Dynamic weights for the coming exchange (Sec. V-B).  Synchronises (waits for the
 * distances of the last want_dist step).  For each worker: u = log||x_i - c||,
 * pushed into its history ring (the first sample fills the ring);
 *     a  = sum_{j<p} c_j (u_{s-j} - u_{s-j-1})                       Eqs. 10-11
 *     h1 = 1 if a < kappa;  1 + ((1-alpha)/kappa)(a - kappa) if a <= 0;  else alpha
 *     h2 = 0 if a < kappa;  (-alpha/kappa) a + alpha          if a <= 0;  else alpha
 * weights: host pointer, 2K floats: h2[0..K) (master-side coefficients) followed by
 * h1[0..K) (worker-side).  Errors: STATE when no distances are pending. */
int dw_weights_next(ah_ctx *h, float alpha, float *weights);

/* The same rule with the squared distances supplied by the caller (host pointer, K
 * doubles) instead of taken from the last want_dist step: for callers that assemble
 * ||x_i - c||^2 themselves, e.g. from column shards held by several GPUs.
 * Touches no GPU. */
int dw_weights_from_norm2(ah_ctx *h, const double *norm2, float alpha, float *weights);

/* Seeded failure / straggler mask for round `round` (Sec. VI: communication between
 * a worker and the master is suppressed part of the time).  mask[i] = 1: worker i
 * is up.  A worker that is up fails with probability p_fail (Philox draw keyed on
 * (seed; i, round)); a failure lasts 1 round if max_stale == 1, else a uniform
 * 1..max_stale rounds.  mask: host pointer, K bytes.  Host-only; touches no GPU. */
int dw_mask_next(ah_ctx *h, uint64_t seed, uint32_t round, double p_fail, int max_stale,
                 uint8_t *mask);

/* Weighted elastic exchange (Eqs. 12-13; with equal coefficients the EASGD pull of
 * Eqs. 8-9), all workers seeing the same old master value.  For every column j:
 *     c = center_j;  acc = 0
 *     for i = 0..K-1 with worker_mask[i] != 0:
 *         d = x_ij - c;   acc += h2_i * d;   x_ij -= h1_i * d
 *     center_j = c + acc
 * worker_mask: host pointer, K bytes, or NULL (all workers take part).
 * weights: host pointer, 2K floats as written by dw_weights_next, or NULL
 * (h1_i = h2_i = alpha for all i).  alpha is ignored when weights != NULL. */
int easgd_exchange(ah_ctx *h, const uint8_t *worker_mask, const float *weights, float alpha);

/* The exchange of one round with the dynamic weights computed on the device: the same
 * rule as dw_weights_next (Sec. V-B, Eqs. 10-11, h1/h2), same history ring, same bits,
 * fed by the distances of the last want_dist step (if that step ran with
 * AH_DIST_AND_RULE the rule has run already and alpha must be the one given there),
 * followed by the weighted exchange
 * (Eqs. 12-13) of easgd_exchange (asynchronous == 0; order ignored) or
 * easgd_exchange_async (asynchronous != 0; order as there, NULL = ascending).  Nothing
 * is copied to the host and the call does not wait, so a whole communication period
 * can be queued ahead of the GPU.  The coefficients used can be read afterwards with
 * ah_state_get(AH_WEIGHTS); the history with AH_UHIST.  Host and device forms of the
 * rule may be mixed freely on one handle.
 * Errors: STATE when no distances are pending, INVALID_ARG for a bad order, CUDA. */
int easgd_exchange_dynamic(ah_ctx *h, const uint8_t *worker_mask, float alpha,
                           const uint16_t *order, int asynchronous);

/* ---- data overlap -------------------------------------------------------------- */

/* Data-overlap partition (Sec. V-A): n data points, k workers; every worker receives
 * the same `shared` points O plus its own disjoint subset S_j of the rest.
 *   perm   : host pointer, n entries: a seeded uniformly random permutation of 0..n-1
 *            (Fisher-Yates from the top; position q trades places with position
 *            r mod (q+1), r = word1 << 32 | word0 of Philox4x32-10 with key
 *            (seed low, seed high) and counter (q low, q high, 0, 4))
 *   bounds : host pointer, k + 2 entries: O = perm[bounds[0], bounds[1]) with
 *            bounds[0] = 0, bounds[1] = shared;  S_j = perm[bounds[j+1], bounds[j+2])
 * |S_j| = floor((n - shared) / k), one more for the first (n - shared) mod k workers, so
 * that the S_j cover everything outside O.  Worker j trains on O u S_j.
 * Needs no handle and no GPU.  Errors: INVALID_ARG (shared > n, k < 1, n >= 2^32). */
int dw_partition(uint64_t seed, uint64_t n, uint32_t k, uint64_t shared, uint32_t *perm,
                 uint64_t *bounds);

/* ---- asynchronous exchange ---------------------------------------------------- */

/* Seeded arrival order for an asynchronous exchange round (Sec. II: training is
 * asynchronous, so the workers do not reach the master together): a uniformly random
 * permutation of 0..K-1, order[q] = the worker that arrives q-th.  Fisher-Yates shuffle
 * of the identity: for q = K-1 down to 1, entries q and r mod (q+1) trade places,
 * r = first word of Philox4x32-10 with key (seed low, seed high) and counter
 * (q, 0, round, 3).  order: host pointer, K entries.  Host-only; touches no GPU. */
int dw_order_next(ah_ctx *h, uint64_t seed, uint32_t round, uint16_t *order);

/* Weighted elastic exchange with the workers reaching the master one at a time
 * (Eqs. 12-13 applied per worker, as printed): each arrival sees the master as the
 * arrivals before it left it.  For every column j:
 *     c = center_j
 *     for q = 0..K-1, i = order[q], worker_mask[i] != 0:
 *         d = x_ij - c;   x_ij -= h1_i * d;   c += h2_i * d
 *     center_j = c
 * order: host pointer, K entries naming every worker exactly once (else INVALID_ARG),
 * or NULL for 0, 1, ..., K-1.  worker_mask, weights, alpha as in easgd_exchange.
 * Unlike the simultaneous form this stays a contraction for any K (no bound on the
 * sum of the h2_i).  Same memory traffic as easgd_exchange. */
int easgd_exchange_async(ah_ctx *h, const uint8_t *worker_mask, const float *weights, float alpha,
                         const uint16_t *order);

/* ---- diagnostics of the arithmetic --------------------------------------------- */

/* (No counterpart in the paper: a check of the implementation's own premises.)
 * Inside its usual operand range the local step (Eq. 4: the division by (sqrt vhat)^k + eps,
 * the square root) uses branch-free sequences in place of the general IEEE square root and
 * division: a hardware approximation, one Newton step, a fused multiply-add on the exact
 * residual.  They give the correctly rounded result if the refined reciprocal is the
 * correctly rounded one (Markstein's division) and the square-root sequence rounds
 * correctly for every input; both depend on the hardware's approximations, so this call
 * checks them on the current device against the IEEE routines:
 *   mismatches[0]  square root, every binary32 value in [2^-64, 2^90)
 *   mismatches[1]  refined reciprocal, every binary32 value in [2^-33, 2^46)
 *   mismatches[2]  quotient, division_pairs seeded pairs with |a| in [2^-63, 2^88),
 *                  b in [2^-33, 2^46), a quarter of them with divisors next to a power of
 *                  two, a quarter with quotients next to short significands
 * All three must be 0.  mismatches: host pointer, 3 entries.  Synchronises; about a second
 * for 2^32 pairs.  Makes one small cudaMalloc.  Errors: INVALID_ARG, ALLOC, CUDA. */
int ah_check_exact_arithmetic(uint64_t division_pairs, uint64_t *mismatches, void *cuda_stream);

/* ---- without a handle, without allocating ------------------------------------ */

/* (No counterpart in the paper: a deployment convenience.)
 * norm2[i] = ||x_i - c||^2 for i = 0..K-1, the same quantity, summed in the same
 * pairwise order and therefore bit-identical to what a want_dist step leaves in a
 * handle, for callers that hold raw pointers and must not allocate: a hook running
 * inside a job whose framework has already claimed the whole GPU, a
 * latency-critical loop that cannot afford the device-wide synchronisation of an
 * allocation, or a component with no ah_ctx of its own (ah_init allocates).  The
 * call makes no cudaMalloc/cudaFree and uses no workspace: its per-tile partial sums
 * go to a fixed 2 MiB array that is part of the library image on every GPU that
 * loads it.
 *   x      device pointer, [K][ldx] binary32, ldx >= P, ldx % 4 == 0, 16-byte aligned
 *   c      device pointer, [P] binary32, 16-byte aligned, readable up to P rounded up to 4
 *   norm2  device pointer, K doubles, written when the stream reaches the kernels
 *   cuda_stream  cudaStream_t or NULL; the call returns without waiting
 * The device that owns the pointers must be the current device.
 * Capacity: K * (ceil(P / 1024) rounded up to a power of two) <=
 * AH_STATIC_SCRATCH_ENTRIES (for example K = 4 with P up to 33.5 M, or K = 16 with P
 * up to 8.3 M); beyond it the call returns AH_ERR_TOO_LARGE and does nothing.
 * The first call on each device looks up the array's device address (a runtime
 * query, no allocation); make that first call outside any stream capture.
 * All calls share the one array and it keeps the previous call's contents; nothing
 * in it needs clearing, but two calls whose kernels may overlap on the GPU (other
 * streams, other threads) race on it: serialise them.
 * Errors: INVALID_ARG, ALIGN, TOO_LARGE, CUDA. */
int ah_distances_static(const float *x, uint64_t ldx, const float *c, int K, uint64_t P,
                        double *norm2, void *cuda_stream);

/* How long the CTAs of a launch that assembles the distances of a round wait for one
 * another, in polls of an arrival counter (roughly a microsecond each under load), before
 * each of them forms the whole sum by itself (Sec. V-B: the K distances feed the rule).
 * The distances do not depend on it: the sums follow one fixed tree whoever forms them.
 * 0 makes every CTA work alone from the start.  Default 4096.  Host-side setting, takes
 * effect with the next launch; returns AH_ERR_INVALID_ARG for a null handle. */
int ah_set_wait_polls(ah_ctx *h, uint32_t polls);

/* ---- diagnostics ------------------------------------------------------------- */
const char *ah_status_string(int status);
/* cudaError_t of the last failed runtime call on this handle (0 if none). */
int ah_last_cuda_error(const ah_ctx *h);
/* Number of kernel launches this handle has enqueued since ah_init. */
uint64_t ah_launch_count(const ah_ctx *h);

#ifdef __cplusplus
}
#endif
#endif /* ADAHESS_H_ */
