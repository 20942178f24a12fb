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
// through h1 (worker-side coefficient) and h2 (master-side coefficient).
__host__ __device__ inline void weight_rule_step(const WeightRule &r, double norm2, double *ring,
                                                 bool ring_filled, float *to_master, float *to_worker)
{
    const double u = u_from_norm2(norm2);
    if (ring_filled) {
        for (int j = r.p_hist; j >= 1; --j) ring[j] = ring[j - 1];
    } else {
        for (int j = 1; j <= r.p_hist; ++j) ring[j] = u;
    }
    ring[0] = u;
    double score = 0.0;
    for (int j = 0; j < r.p_hist; ++j)
        score = AH_DADD(score, AH_DMUL(r.coef[j], AH_DSUB(ring[j], ring[j + 1])));
    double w_worker, w_master;
    if (score < r.kappa) {
        w_worker = 1.0;
        w_master = 0.0;
    } else if (score <= 0.0) {
        const double slope_worker = AH_DDIV(AH_DSUB(1.0, r.alpha), r.kappa);   // 1 -> alpha on [kappa, 0]
        const double slope_master = AH_DDIV(-r.alpha, r.kappa);                // 0 -> alpha on [kappa, 0]
        w_worker = AH_DADD(1.0, AH_DMUL(slope_worker, AH_DSUB(score, r.kappa)));
        w_master = AH_DADD(AH_DMUL(slope_master, score), r.alpha);
    } else {
        w_worker = r.alpha;
        w_master = r.alpha;
    }
    *to_worker = (float)w_worker;
    *to_master = (float)w_master;
}

}  // namespace ah
