/*
 * CPU oracle for the AdaHessian + elastic-averaging round (test infrastructure).
 *
 * This file is TEST INFRASTRUCTURE.  It is a plain, slow, step-by-step restatement
 * of the update equations of "A Dynamic Weighting Strategy to Mitigate Worker Node
 * Failure in Distributed Deep Learning" (Xu & Carr).  It shares no code, header,
 * table or constant generator with the CUDA library and must never be called from
 * the product path: only the tests, the smoke check and the CPU-baseline leg of the
 * benchmark may load it.
 *
 * Arithmetic contract ("canonical order"): state is IEEE binary32; every written
 * operation is rounded once, to nearest-even, in exactly the order written; no FMA
 * contraction (build with -ffp-contract=off, no -ffast-math).  Building with
 * -DORC_DOUBLE switches the arithmetic type `real` to double while state stays
 * binary32 in memory: that build only measures the binary32 build's own drift.
 *
 * Building with -fopenmp parallelises loops over independent (worker) or (column)
 * items; no per-element operation and no reduction order changes, so both builds
 * give bit-identical results.
 *
 * Parity pins (see tests): Philox known-answer vectors of Salmon et al. (SC'11);
 * Hutchinson identity on a diagonal quadratic (Sec. IV-B); reduction of the step to
 * Adam, also for a worker that sits rounds out; closed forms of h1/h2 (Sec. V-B); the
 * logarithm of u = log ||x_i - c|| against 300-bit arithmetic; EASGD reduction of
 * Eqs. 12-13; a worked two-worker example computed by hand in double precision.
 *
 * Parity unpinned: the history depth p, the coefficients c_j and the threshold
 * (Sec. V-B gives no values) are run-time parameters; only their closed forms are
 * pinned.
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <string.h>

#ifdef ORC_DOUBLE
typedef double real;
#define ORC_SQRT(a) sqrt(a)
#define ORC_POW(a, b) pow((a), (b))
#else
typedef float real;
#define ORC_SQRT(a) sqrtf(a)
#define ORC_POW(a, b) powf((a), (b))
#endif

/* One parameter tensor inside the flat row: elements [offset, offset+length),
 * averaged in consecutive groups of `block` elements (block = kh*kw of a conv
 * kernel; 1 = no averaging).  length % block == 0. */
typedef struct {
    uint64_t offset;
    uint64_t length;
    uint32_t block;
    uint32_t flags;
} orc_segment;

/* ------------------------------------------------------------------------- */
/* S1. Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as
 * easy as 1, 2, 3", SC'11).  Counter-based: out = bijection_key(counter).        */
/* ------------------------------------------------------------------------- */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;   /* round multipliers   */
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;   /* Weyl key increments */
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)M0 * (uint64_t)c0;
        uint64_t p1 = (uint64_t)M1 * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

enum { ORC_DOMAIN_Z = 0, ORC_DOMAIN_FAIL = 1, ORC_DOMAIN_STALE = 2 };

/* Sign bit of the Rademacher entry z_{t,i,j} (Sec. IV-B: "z is a Rademacher
 * vector").  One Philox block covers 128 consecutive indices j of one worker row:
 * counter = (j >> 7, worker, round, domain 0), key = (seed low, seed high).
 * Element j takes bit (j & 31) of output word (j >> 5) & 3.  0 -> +1, 1 -> -1.
 * With several Hutchinson samples per step, sample s = 0, 1, ... uses the counter
 * word 256 s in place of the domain 0 (sample 0 is the single-sample stream). */
static inline uint32_t orc_zbit_s(uint64_t seed, uint32_t t, uint32_t i, uint32_t sample, uint64_t j)
{
    uint32_t ctr[4] = { (uint32_t)(j >> 7), i, t, ORC_DOMAIN_Z + 256u * sample };
    uint32_t key[2] = { (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32) };
    uint32_t r[4];
    orc_philox4x32_10(ctr, key, r);
    return (r[(j >> 5) & 3] >> (j & 31)) & 1u;
}

static inline uint32_t orc_zbit(uint64_t seed, uint32_t t, uint32_t i, uint64_t j)
{
    uint32_t ctr[4] = { (uint32_t)(j >> 7), i, t, ORC_DOMAIN_Z };
    uint32_t key[2] = { (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32) };
    uint32_t r[4];
    orc_philox4x32_10(ctr, key, r);
    return (r[(j >> 5) & 3] >> (j & 31)) & 1u;
}

/* z[K][ld] as +-1.0f. */
void orc_sample_z(uint64_t seed, uint32_t t, int K, uint64_t P, float *z, uint64_t ld)
{
#pragma omp parallel for schedule(static)
    for (int i = 0; i < K; ++i)
        for (uint64_t j = 0; j < P; ++j)
            z[(uint64_t)i * ld + j] = orc_zbit(seed, t, (uint32_t)i, j) ? -1.0f : 1.0f;
}

/* Sign bits of one whole worker row, one Philox call per 128 indices (the same
 * values as orc_zbit; only the repeated calls are saved). sgn[j] in {0,1}. */
static void orc_zbits_row_s(uint64_t seed, uint32_t t, uint32_t i, uint32_t sample, uint64_t P,
                            uint8_t *sgn)
{
    uint32_t key[2] = { (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32) };
    for (uint64_t base = 0; base < P; base += 128) {
        uint32_t ctr[4] = { (uint32_t)(base >> 7), i, t, ORC_DOMAIN_Z + 256u * sample };
        uint32_t r[4];
        orc_philox4x32_10(ctr, key, r);
        uint64_t end = base + 128 < P ? base + 128 : P;
        for (uint64_t j = base; j < end; ++j)
            sgn[j] = (uint8_t)((r[(j >> 5) & 3] >> (j & 31)) & 1u);
    }
}

static void orc_zbits_row(uint64_t seed, uint32_t t, uint32_t i, uint64_t P, uint8_t *sgn)
{
    orc_zbits_row_s(seed, t, i, 0u, P, sgn);
}

/* z of Hutchinson sample `sample`, per element from the definition. */
void orc_sample_z_s(uint64_t seed, uint32_t t, uint32_t sample, int K, uint64_t P, float *z,
                    uint64_t ld)
{
#pragma omp parallel for schedule(static)
    for (int i = 0; i < K; ++i)
        for (uint64_t j = 0; j < P; ++j)
            z[(uint64_t)i * ld + j] = orc_zbit_s(seed, t, (uint32_t)i, sample, j) ? -1.0f : 1.0f;
}

/* z bits as bytes [K][P] (for bit-exact comparison with the device generator). */
void orc_sample_zbits(uint64_t seed, uint32_t t, int K, uint64_t P, uint8_t *bits)
{
#pragma omp parallel for schedule(static)
    for (int i = 0; i < K; ++i)
        orc_zbits_row(seed, t, (uint32_t)i, P, bits + (uint64_t)i * P);
}

/* ------------------------------------------------------------------------- */
/* a3. Spatial average (Sec. IV-B, "taking the average around its neighbours"):
 * inside every tensor, each consecutive group of `block` entries is replaced by
 * the group's mean (sum in ascending index order, then one division).  Indices
 * not covered by any segment, and segments with block 1, are left as they are.  */
/* ------------------------------------------------------------------------- */
void orc_spatial_average(const float *d, uint64_t P, const orc_segment *segs, int nseg,
                         float *dbar)
{
    for (uint64_t j = 0; j < P; ++j) dbar[j] = d[j];
    for (int s = 0; s < nseg; ++s) {
        uint32_t b = segs[s].block;
        if (b <= 1) continue;
        for (uint64_t q = segs[s].offset; q < segs[s].offset + segs[s].length; q += b) {
            real S = (real)d[q];
            for (uint32_t r = 1; r < b; ++r)
                S = S + (real)d[q + r];
            float mean = (float)(S / (real)b);
            for (uint32_t r = 0; r < b; ++r)
                dbar[q + r] = mean;
        }
    }
}

/* a2. Hutchinson diagonal with one sample, D = z (.) Hz (Sec. IV-B): a sign flip. */
void orc_hutchinson_row(const float *hvp, const uint8_t *sgn, uint64_t P, float *d)
{
    for (uint64_t j = 0; j < P; ++j)
        d[j] = sgn[j] ? -hvp[j] : hvp[j];
}

/* ------------------------------------------------------------------------- */
/* S2 (a4 + a5). AdaHessian step of every active worker (Sec. IV-B: Adam-like
 * moments, the second moment built from the spatially averaged Hessian diagonal
 * instead of the gradient; Eq. 4 with D = 1/((sqrt v)^k + eps)).
 *
 * x, m, v: [K][P] state (row stride P).  grad, hvp: [K][ld].  step[K]: per-worker
 * count of steps taken (bias correction uses the worker's own count).
 * active: K bytes or NULL (= all ones); an inactive worker is left untouched.
 * Returns 0, or -1 when scratch memory cannot be had.                           */
/* ------------------------------------------------------------------------- */
#include <stdlib.h>

/* n_samples Hutchinson samples per step (Sec. IV-B: diag(H) ~ (1/n) sum_s z_s (.) H z_s):
 * hvp holds sample s at hvp + s * sample_stride, each [K][ld]; the products are summed
 * in ascending s and divided by n once (n = 1: no division), then averaged spatially. */
int orc_local_step_n(float *x, float *m, float *v, uint32_t *step,
                     const float *grad, const float *hvp, int n_samples, uint64_t sample_stride,
                     int K, uint64_t P, uint64_t ld,
                     const orc_segment *segs, int nseg, uint64_t z_seed, uint32_t t,
                     float lr, float beta1, float beta2, float eps, float hessian_power,
                     float weight_decay, const uint8_t *active)
{
    int err = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int i = 0; i < K; ++i) {
        if (active && !active[i]) continue;
        uint8_t *sgn = (uint8_t *)malloc(P ? P : 1);
        float *d = (float *)malloc((P ? P : 1) * sizeof(float));
        float *dbar = (float *)malloc((P ? P : 1) * sizeof(float));
        if (!sgn || !d || !dbar) {
#pragma omp atomic write
            err = -1;
            free(sgn); free(d); free(dbar);
            continue;
        }
        step[i] += 1;
        const uint32_t ti = step[i];
        /* bias corrections in double on the host, then rounded to the state type */
        /* bias corrections: double on the host, rounded to binary32 (Adam's
         * 1 - beta^t with t the worker's own step count) */
        const real bc1 = (real)(float)(1.0 - pow((double)beta1, (double)ti));
        const real bc2 = (real)(float)(1.0 - pow((double)beta2, (double)ti));
        const real b1 = (real)beta1, b2 = (real)beta2;
        const real omb1 = (real)(1.0f - beta1);      /* binary32 subtraction */
        const real omb2 = (real)(1.0f - beta2);
        const real eta = (real)lr, e = (real)eps, wd = (real)weight_decay;

        const float *g = grad + (uint64_t)i * ld;
        float *xi = x + (uint64_t)i * P, *mi = m + (uint64_t)i * P, *vi = v + (uint64_t)i * P;

        orc_zbits_row(z_seed, t, (uint32_t)i, P, sgn);
        orc_hutchinson_row(hvp + (uint64_t)i * ld, sgn, P, d);
        if (n_samples > 1) {
            for (int sidx = 1; sidx < n_samples; ++sidx) {
                const float *hs = hvp + (uint64_t)sidx * sample_stride + (uint64_t)i * ld;
                orc_zbits_row_s(z_seed, t, (uint32_t)i, (uint32_t)sidx, P, sgn);
                orc_hutchinson_row(hs, sgn, P, dbar);            /* dbar as scratch */
                for (uint64_t j = 0; j < P; ++j)
                    d[j] = (float)((real)d[j] + (real)dbar[j]);
            }
            for (uint64_t j = 0; j < P; ++j)
                d[j] = (float)((real)d[j] / (real)n_samples);
        }
        orc_spatial_average(d, P, segs, nseg, dbar);

        for (uint64_t j = 0; j < P; ++j) {
            const real D = (real)dbar[j];
            const real xo = (real)xi[j];
            /* first moment: EMA of the gradient */
            const real m1 = (b1 * (real)mi[j]) + (omb1 * (real)g[j]);
            /* second moment: EMA of the squared averaged Hessian diagonal */
            const real v1 = (b2 * (real)vi[j]) + ((omb2 * D) * D);
            const real mhat = m1 / bc1;
            const real vhat = v1 / bc2;
            const real r = ORC_SQRT(vhat);
            real pw;
            if (hessian_power == 1.0f) pw = r;
            else if (hessian_power == 0.5f) pw = ORC_SQRT(r);
            else pw = ORC_POW(r, (real)hessian_power);
            const real den = pw + e;
            real xn;
            if (weight_decay != 0.0f)
                xn = xo - (eta * ((mhat / den) + (wd * xo)));
            else
                xn = xo - (eta * (mhat / den));
            xi[j] = (float)xn;
            mi[j] = (float)m1;
            vi[j] = (float)v1;
        }
        free(sgn); free(d); free(dbar);
    }
    return err;
}

int orc_local_step(float *x, float *m, float *v, uint32_t *step,
                   const float *grad, const float *hvp, int K, uint64_t P, uint64_t ld,
                   const orc_segment *segs, int nseg, uint64_t z_seed, uint32_t t,
                   float lr, float beta1, float beta2, float eps, float hessian_power,
                   float weight_decay, const uint8_t *active)
{
    return orc_local_step_n(x, m, v, step, grad, hvp, 1, 0, K, P, ld, segs, nseg, z_seed, t, lr,
                            beta1, beta2, eps, hessian_power, weight_decay, active);
}

/* ------------------------------------------------------------------------- */
/* S3 (a6). Squared distance of worker i to the master, n2_i = sum_j (x_ij-c_j)^2,
 * for u_i = log ||x_i - c|| (Sec. V-B).  The difference is formed in the state
 * type, squared and summed in double.  Summation order: textbook pairwise
 * summation, i.e. the perfect binary tree of adjacent pairs over the index range
 * [0, 2^ceil(log2 P)), indices >= P contributing +0.0.                          */
/* ------------------------------------------------------------------------- */
static double orc_pairwise_sq(const float *x, const float *c, uint64_t lo, uint64_t n, uint64_t P)
{
    if (lo >= P) return 0.0;
    if (n == 1) {
        real d = (real)x[lo] - (real)c[lo];
        double dd = (double)d;
        return dd * dd;
    }
    double left = orc_pairwise_sq(x, c, lo, n / 2, P);
    double right = orc_pairwise_sq(x, c, lo + n / 2, n / 2, P);
    return left + right;
}

void orc_norm2(const float *x, const float *c, int K, uint64_t P, double *n2)
{
    uint64_t n = 1;
    while (n < P) n <<= 1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int i = 0; i < K; ++i)
        n2[i] = orc_pairwise_sq(x + (uint64_t)i * P, c, 0, n, P);
}

/* Natural logarithm of a positive, finite double, rounded to the nearest double.
 * u = log ||x_i - c|| (Sec. V-B) is read as exactly this value: the definition of the
 * function, not one particular library's approximation of it, so that any correct
 * implementation reproduces it bit for bit.  It is obtained here from a library
 * primitive: the logarithm of GNU libquadmath in IEEE binary128 (113 significant
 * bits, error below one unit in the last of them), rounded once to binary64.  The
 * 60 spare bits make that rounding the correct one unless ln x lies within 2^-59
 * units in the last place of the midpoint of two doubles.                         */
#include <quadmath.h>

double orc_ln(double x)
{
    return (double)logq((__float128)x);
}

/* u_i = log ||x_i - c||_2 = 0.5 ln(n2_i), natural log, n2 clamped away from 0
 * (all workers start as copies of the master, Sec. II, so n2 can be exactly 0). */
double orc_u_from_norm2(double n2)
{
    return 0.5 * orc_ln(n2 > 1e-300 ? n2 : 1e-300);
}

/* ------------------------------------------------------------------------- */
/* S4 (a7). Raw score and dynamic weights (Sec. V-B, Eqs. 10-11 and the h1/h2
 * definitions).  uhist[i][0..p] holds worker i's p+1 most recent u values, newest
 * first (uhist[i][0] = u_s).  filled: 0 before the first sample.  The first sample
 * fills the whole ring, so differences that reach before the history are 0.
 *   a = sum_{j=0}^{p-1} c_j (u_{s-j} - u_{s-j-1}),  accumulated j ascending
 *   h1(a) = 1 (a<kappa);  1 + ((1-alpha)/kappa)(a-kappa) (kappa<=a<=0);  alpha (a>0)
 *   h2(a) = 0 (a<kappa);  (-alpha/kappa) a + alpha       (kappa<=a<=0);  alpha (a>0)
 * Outputs: h2[K], h1[K] as binary32, a_out[K] (may be NULL).                    */
/* ------------------------------------------------------------------------- */
double orc_h1(double a, double alpha, double kappa)
{
    if (a < kappa) return 1.0;
    if (a <= 0.0) return 1.0 + ((1.0 - alpha) / kappa) * (a - kappa);
    return alpha;
}

double orc_h2(double a, double alpha, double kappa)
{
    if (a < kappa) return 0.0;
    if (a <= 0.0) return ((-alpha / kappa) * a) + alpha;
    return alpha;
}

void orc_weights_next(double *uhist, int *filled, int K, int p, const double *c, double kappa,
                      float alpha, const double *n2, float *h2, float *h1, double *a_out)
{
    const double al = (double)alpha;
    for (int i = 0; i < K; ++i) {
        double *ring = uhist + (size_t)i * (size_t)(p + 1);
        double u = orc_u_from_norm2(n2[i]);
        if (!*filled) {
            for (int j = 0; j <= p; ++j) ring[j] = u;
        } else {
            for (int j = p; j >= 1; --j) ring[j] = ring[j - 1];
            ring[0] = u;
        }
        double a = 0.0;
        for (int j = 0; j < p; ++j)
            a = a + c[j] * (ring[j] - ring[j + 1]);
        if (a_out) a_out[i] = a;
        h1[i] = (float)orc_h1(a, al, kappa);
        h2[i] = (float)orc_h2(a, al, kappa);
    }
    *filled = 1;
}

/* ------------------------------------------------------------------------- */
/* S5 (a8). Seeded failure / straggler mask (Sec. VI: communication between a
 * worker and the master is suppressed a fixed fraction of the time).
 * For round t and worker i: still down if t < down_until[i]; else draw
 * r = Philox(seed; (0, i, t, 1))[0] and fail iff r < floor(p_fail * 2^32)
 * (always if p_fail >= 1); a failure lasts d rounds, d = 1 if max_stale == 1 else
 * 1 + Philox(seed; (0, i, t, 2))[0] % max_stale.  mask[i] = 1 means "up".        */
/* ------------------------------------------------------------------------- */
void orc_mask_next(uint32_t *down_until, int K, uint64_t seed, uint32_t t, double p_fail,
                   int max_stale, uint8_t *mask)
{
    uint32_t key[2] = { (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32) };
    for (int i = 0; i < K; ++i) {
        if (t < down_until[i]) { mask[i] = 0; continue; }
        uint32_t ctr[4] = { 0u, (uint32_t)i, t, ORC_DOMAIN_FAIL };
        uint32_t r[4];
        orc_philox4x32_10(ctr, key, r);
        int fail;
        if (p_fail >= 1.0) fail = 1;
        else if (p_fail <= 0.0) fail = 0;
        else fail = r[0] < (uint32_t)floor(p_fail * 4294967296.0);
        if (fail) {
            uint32_t d = 1;
            if (max_stale > 1) {
                uint32_t ctr2[4] = { 0u, (uint32_t)i, t, ORC_DOMAIN_STALE };
                uint32_t r2[4];
                orc_philox4x32_10(ctr2, key, r2);
                d = 1u + r2[0] % (uint32_t)max_stale;
            }
            down_until[i] = t + d;
            mask[i] = 0;
        } else {
            mask[i] = 1;
        }
    }
}

/* ------------------------------------------------------------------------- */
/* S6 (a9). Weighted elastic exchange, Eqs. 12-13, all workers seeing the same old
 * master value c (simultaneous form):
 *   for every column j: c = xc_j; acc = 0;
 *     for i ascending with mask_i: d = x_ij - c; acc += h2_i d; x_ij -= h1_i d
 *     xc_j = c + acc
 * With h1_i = h2_i = alpha this is the EASGD pull of Eqs. 8-9, taken in the
 * orientation of Eqs. 12-13 (worker and master move toward each other).         */
/* ------------------------------------------------------------------------- */
void orc_exchange(float *x, float *xc, int K, uint64_t P, const uint8_t *mask,
                  const float *h2, const float *h1)
{
#pragma omp parallel for schedule(static)
    for (uint64_t j = 0; j < P; ++j) {
        const real c = (real)xc[j];
        real acc = (real)0.0f;
        for (int i = 0; i < K; ++i) {
            if (mask && !mask[i]) continue;
            float *xi = x + (uint64_t)i * P;
            const real d = (real)xi[j] - c;
            acc = acc + ((real)h2[i] * d);
            xi[j] = (float)((real)xi[j] - ((real)h1[i] * d));
        }
        xc[j] = (float)(c + acc);
    }
}

/* ------------------------------------------------------------------------- */
/* Asynchronous form of the exchange.  Sec. II assumes asynchronous training and
 * Eqs. 12-13 are written for one worker talking to the master: the workers reach
 * the master one at a time, and each one sees the master as the workers before it
 * left it.  order[0..n_order) lists the workers in the order in which they arrive
 * (NULL = 0, 1, ..., K-1); a worker whose mask byte is 0 does not arrive.  For
 * every column j:
 *   c = xc_j
 *   for q ascending, i = order[q], mask_i: d = x_ij - c; x_ij -= h1_i d; c += h2_i d
 *   xc_j = c                                                                      */
/* ------------------------------------------------------------------------- */
void orc_exchange_async(float *x, float *xc, int K, uint64_t P, const uint8_t *mask,
                        const float *h2, const float *h1, const uint16_t *order, int n_order)
{
    const int n = order ? n_order : K;
#pragma omp parallel for schedule(static)
    for (uint64_t j = 0; j < P; ++j) {
        real c = (real)xc[j];
        for (int q = 0; q < n; ++q) {
            const int i = order ? (int)order[q] : q;
            if (mask && !mask[i]) continue;
            float *xi = x + (uint64_t)i * P;
            const real d = (real)xi[j] - c;
            xi[j] = (float)((real)xi[j] - ((real)h1[i] * d));
            c = (real)(float)(c + ((real)h2[i] * d));
        }
        xc[j] = (float)c;
    }
}

/* Seeded arrival order of round t: a uniformly random permutation of 0..K-1 by the
 * Fisher-Yates shuffle (Durstenfeld's form), driven by the counter-based generator:
 * start from the identity; for q = K-1 down to 1 draw
 * r = Philox(seed; (q, 0, t, 3))[0] and swap entries q and r mod (q+1).           */
enum { ORC_DOMAIN_ORDER = 3 };

void orc_order_next(int K, uint64_t seed, uint32_t t, uint16_t *order)
{
    uint32_t key[2] = { (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32) };
    for (int i = 0; i < K; ++i) order[i] = (uint16_t)i;
    for (int q = K - 1; q >= 1; --q) {
        uint32_t ctr[4] = { (uint32_t)q, 0u, t, ORC_DOMAIN_ORDER };
        uint32_t r[4];
        orc_philox4x32_10(ctr, key, r);
        const uint32_t pick = r[0] % (uint32_t)(q + 1);
        const uint16_t tmp = order[q]; order[q] = order[pick]; order[pick] = tmp;
    }
}

/* ------------------------------------------------------------------------- */
/* First-order local steps of the methods the paper compares against (Sec. VI:
 * EASGD and EAMSGD, "EASGD with Momentum"; Sec. VII: eta = 0.01, delta = 0.5).
 *   plain SGD (Eqs. 2-3, momentum == 0):   x <- x - (eta g)
 *   momentum delta (velocity form):        u <- (delta u) - (eta g);   x <- x + u
 * u[K][P] is the velocity (the paper does not print the momentum rule; this is the
 * classical form of the works it cites for it; with Nesterov's variant only the point
 * where the caller evaluates g changes).  Inactive workers are left untouched; an
 * active worker's step count goes up by one.                                     */
/* ------------------------------------------------------------------------- */
void orc_sgd_step(float *x, float *u, uint32_t *step, const float *grad, int K, uint64_t P,
                  uint64_t ld, float lr, float momentum, const uint8_t *active)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int i = 0; i < K; ++i) {
        if (active && !active[i]) continue;
        step[i] += 1;
        const real eta = (real)lr, delta = (real)momentum;
        const float *g = grad + (uint64_t)i * ld;
        float *xi = x + (uint64_t)i * P, *ui = u + (uint64_t)i * P;
        for (uint64_t j = 0; j < P; ++j) {
            if (momentum == 0.0f) {
                xi[j] = (float)((real)xi[j] - (eta * (real)g[j]));
            } else {
                const real un = (delta * (real)ui[j]) - (eta * (real)g[j]);
                ui[j] = (float)un;
                xi[j] = (float)((real)xi[j] + (real)(float)un);
            }
        }
    }
}

/* ------------------------------------------------------------------------- */
/* Data overlap (Sec. V-A).  n data points, k workers, o shared points.  A seeded,
 * uniformly random permutation perm of 0..n-1 is drawn (Fisher-Yates from the top:
 * for q = n-1 down to 1, entries q and r mod (q+1) trade places, r = the 64-bit
 * value (word1 << 32 | word0) of Philox(seed; (q low, q high, 0, 4))).  Then
 *   O   = perm[0, o)                       the subset every worker receives
 *   S_j = the next |S_j| entries, j = 0..k-1, dealt in order
 *   D_j = O u S_j
 * with |S_j| = floor((n-o)/k), plus one for the first (n-o) mod k workers so that
 * the S_j cover D - O (the text states both; they agree when k divides n-o).
 * bounds[0] = 0, bounds[1] = o, bounds[j+2] = end of S_j in perm.
 * Returns 0, or -1 when o > n or k < 1.                                          */
/* ------------------------------------------------------------------------- */
int orc_partition(uint64_t seed, uint64_t n, uint32_t k, uint64_t o, uint32_t *perm, uint64_t *bounds)
{
    if (o > n || k < 1) return -1;
    uint32_t key[2] = { (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32) };
    for (uint64_t i = 0; i < n; ++i) perm[i] = (uint32_t)i;
    for (uint64_t q = n; q-- > 1;) {
        uint32_t ctr[4] = { (uint32_t)q, (uint32_t)(q >> 32), 0u, 4u };
        uint32_t r[4];
        orc_philox4x32_10(ctr, key, r);
        const uint64_t draw = ((uint64_t)r[1] << 32) | (uint64_t)r[0];
        const uint64_t pick = draw % (q + 1);
        const uint32_t tmp = perm[q]; perm[q] = perm[pick]; perm[pick] = tmp;
    }
    const uint64_t rest = n - o, base = rest / k, extra = rest % k;
    bounds[0] = 0;
    bounds[1] = o;
    for (uint32_t j = 0; j < k; ++j)
        bounds[j + 2] = bounds[j + 1] + base + (j < extra ? 1 : 0);
    return 0;
}

int orc_is_double(void)
{
#ifdef ORC_DOUBLE
    return 1;
#else
    return 0;
#endif
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
