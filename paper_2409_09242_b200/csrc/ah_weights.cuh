// The dynamic weighting rule of Sec. V-B for one worker, written once for the host
// (dw_weights_next, dw_weights_from_norm2) and the device (easgd_exchange_dynamic),
// as a fixed list of IEEE binary64 operations, so that both give the same bits.
// Not installed.
#pragma once

#include "ah_ln.cuh"

namespace ah {

// Pushes the sample u = log ||x_i - c|| into the worker's ring (newest first; the
// first sample fills the whole ring), forms the raw score of Eqs. 10-11 and maps it
// through h1 (worker-side coefficient) and h2 (master-side coefficient).  The ring is read
// from ring_in and the advanced ring goes to ring_out (the same array, another one, or
// null where somebody else stores it).  p, coef and kappa are the rule's setting
// (dw_config), alpha the moving rate.  The ring moves on one entry at a time (entry j is
// read before it is overwritten, also when ring_out is ring_in), so nothing the size of the
// history is held.
__host__ __device__ inline void weight_rule_step(int p_hist, const double *coef, double kappa,
                                                 double alpha, double norm2, const double *ring_in,
                                                 double *ring_out, bool ring_filled,
                                                 float *to_master, float *to_worker)
{
    // The first entries of the ring are fetched before the logarithm is computed, so that
    // from there on only arithmetic is left (on the device every CTA then finishes at the
    // same moment); a deeper history is read as the sum goes.
    constexpr int kAhead = 8;
    double ahead[kAhead];
#if defined(__CUDA_ARCH__)
#pragma unroll
#endif
    for (int j = 0; j < kAhead; ++j) ahead[j] = ring_filled && j < p_hist ? ring_in[j] : 0.0;
    const double u = u_from_norm2(norm2);
    // advanced ring: u, then the old entries 0 .. p-1 (or u throughout, on the first sample);
    // score = sum_j coef[j] * (advanced[j] - advanced[j + 1]), j ascending
    double score = 0.0, newer = u;
#if defined(__CUDA_ARCH__)
#pragma unroll
#endif
    for (int j = 0; j < kAhead; ++j)
        if (j < p_hist) {
            const double older = ring_filled ? ahead[j] : u;        // advanced[j + 1]
            score = AH_DADD(score, AH_DMUL(coef[j], AH_DSUB(newer, older)));
            if (ring_out) ring_out[j] = newer;
            newer = older;
        }
    for (int j = kAhead; j < p_hist; ++j) {
        const double older = ring_filled ? ring_in[j] : u;
        score = AH_DADD(score, AH_DMUL(coef[j], AH_DSUB(newer, older)));
        if (ring_out) ring_out[j] = newer;
        newer = older;
    }
    if (ring_out) ring_out[p_hist] = newer;
    double w_worker, w_master;
    if (score < kappa) {
        w_worker = 1.0;
        w_master = 0.0;
    } else if (score <= 0.0) {
        const double slope_worker = AH_DDIV(AH_DSUB(1.0, alpha), kappa);   // 1 -> alpha on [kappa, 0]
        const double slope_master = AH_DDIV(-alpha, kappa);                // 0 -> alpha on [kappa, 0]
        w_worker = AH_DADD(1.0, AH_DMUL(slope_worker, AH_DSUB(score, kappa)));
        w_master = AH_DADD(AH_DMUL(slope_master, score), alpha);
    } else {
        w_worker = alpha;
        w_master = alpha;
    }
    *to_worker = (float)w_worker;
    *to_master = (float)w_master;
}

}  // namespace ah
