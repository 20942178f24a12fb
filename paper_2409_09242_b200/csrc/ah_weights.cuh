// The dynamic weighting rule of Sec. V-B for one worker, written once for the host
// (dw_weights_next, dw_weights_from_norm2) and the device (easgd_exchange_dynamic),
// as a fixed list of IEEE binary64 operations, so that both give the same bits.
// Not installed.
#pragma once

#include "ah_ln.cuh"

namespace ah {

struct WeightRule {
    int p_hist;                    // history depth p
    double coef[AH_MAX_HIST];      // c_0 .. c_{p-1}, c_0 on the newest difference
    double kappa;                  // threshold of h1 / h2, negative
    double alpha;                  // moving rate, widened from binary32
};

// Pushes the sample u = log ||x_i - c|| into the worker's ring (newest first; the
// first sample fills the whole ring), forms the raw score of Eqs. 10-11 and maps it
// through h1 (worker-side coefficient) and h2 (master-side coefficient).  The ring is read
// from ring_in and the advanced ring goes to ring_out (the same array, another one, or
// null where somebody else stores it).
__host__ __device__ inline void weight_rule_step(const WeightRule &rule, double norm2,
                                                 const double *ring_in, double *ring_out,
                                                 bool ring_filled, float *to_master, float *to_worker)
{
    // the ring is read in one go (the loads do not wait for one another), moved on in
    // registers and written back at the end
    double past[AH_MAX_HIST + 1];
    for (int j = 0; j <= rule.p_hist; ++j) past[j] = ring_in[j];
    const double u = u_from_norm2(norm2);
    if (ring_filled) {
        for (int j = rule.p_hist; j >= 1; --j) past[j] = past[j - 1];
    } else {
        for (int j = 1; j <= rule.p_hist; ++j) past[j] = u;
    }
    past[0] = u;
    double score = 0.0;
    for (int j = 0; j < rule.p_hist; ++j)
        score = AH_DADD(score, AH_DMUL(rule.coef[j], AH_DSUB(past[j], past[j + 1])));
    if (ring_out)
        for (int j = 0; j <= rule.p_hist; ++j) ring_out[j] = past[j];
    double w_worker, w_master;
    if (score < rule.kappa) {
        w_worker = 1.0;
        w_master = 0.0;
    } else if (score <= 0.0) {
        const double slope_worker = AH_DDIV(AH_DSUB(1.0, rule.alpha), rule.kappa);   // 1 -> alpha on [kappa, 0]
        const double slope_master = AH_DDIV(-rule.alpha, rule.kappa);                // 0 -> alpha on [kappa, 0]
        w_worker = AH_DADD(1.0, AH_DMUL(slope_worker, AH_DSUB(score, rule.kappa)));
        w_master = AH_DADD(AH_DMUL(slope_master, score), rule.alpha);
    } else {
        w_worker = rule.alpha;
        w_master = rule.alpha;
    }
    *to_worker = (float)w_worker;
    *to_master = (float)w_master;
}

}  // namespace ah
