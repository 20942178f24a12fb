// Exchange rounds without a host round trip: the dynamic weights of Sec. V-B are
// computed on the device from the distances the preceding local step left there, and
// the exchange kernel reads them from device memory.  The host never waits, so the
// next period's launches can be queued while this one still runs.
#include <string.h>

#include "ah_ctx.h"
#include "ah_weights.cuh"

namespace ah {

// One thread per worker: the weighting rule for worker i (the same function the host
// entry points run), on the device copy of the history ring.
__global__ void __launch_bounds__(AH_MAX_WORKERS)
dynamic_weights_kernel(const __grid_constant__ RuleConfig rule, double alpha, const double *norm2,
                       double *uhist, bool filled, float *weights, int nworkers)
{
    const int i = threadIdx.x;
    if (i < nworkers) {
        double *ring = uhist + (size_t)i * (rule.p_hist + 1);
        weight_rule_step(rule.p_hist, rule.coef, rule.kappa, alpha, norm2[i], ring, ring, filled,
                         &weights[i], &weights[nworkers + i]);
    }
}

}  // namespace ah

using namespace ah;

// The weighting rule on the device, fed by assembled distances that wait in norm2_dev
// (restored from a snapshot, or assembled for another reader before the exchange asked
// for coefficients); its coefficients stay in weights_dev.
int ah::enqueue_weight_rule(ah_ctx *h, float alpha)
{
    const int rc = ring_to_device(h);
    if (rc != AH_OK) return rc;
    const bool filled = h->ring_home == 1 || h->ring_filled != 0;
    RuleConfig rule;
    memset(&rule, 0, sizeof rule);
    rule.p_hist = h->p_hist;
    for (int j = 0; j < h->p_hist; ++j) rule.coef[j] = h->coef[j];
    rule.kappa = h->kappa;
    dynamic_weights_kernel<<<1, AH_MAX_WORKERS, 0, h->stream>>>(rule, (double)alpha, h->norm2_dev + 1,
                                                                 h->ring_dev[h->ring_cur], filled,
                                                                 h->weights_dev, h->K);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return ah_cuda_fail(h, e);
    h->launches += 1;
    h->ring_home = 1;                              // the device copy of the ring leads
    h->norm2_pending = false;                      // these distances have fed the rule
    h->lagged_ready = true;                        // weights_dev now holds coefficients
    return AH_OK;
}

extern "C" int easgd_exchange_dynamic(ah_ctx *h, const uint8_t *worker_mask, float alpha,
                                      const uint16_t *order, int asynchronous)
{
    if (!h) return AH_ERR_INVALID_ARG;
    if (!h->has_device) return AH_ERR_STATE;
    // the rule is either owed on the last distance round (AH_DIST_AND_RULE) or runs now on
    // the pending distances; either way it goes with the assembly of that round's tile
    // sums if they still wait, and its output ends up in weights_dev
    if (h->rule_fresh) {
        if (alpha != h->rule_fresh_alpha) return AH_ERR_INVALID_ARG;
    } else if (!h->norm2_pending) {
        return AH_ERR_STATE;
    }
    ExchangeParams p;
    int rc = fill_exchange(h, worker_mask, nullptr, alpha, asynchronous ? order : nullptr,
                           h->weights_dev, p);
    if (rc != AH_OK) return rc;
    if (h->sums_raw && !h->raw_rule) {
        h->raw_rule = true;
        h->raw_alpha = alpha;
    }
    if ((rc = settle_distances(h)) != AH_OK) return rc;
    if (!h->rule_fresh && h->norm2_pending && (rc = enqueue_weight_rule(h, alpha)) != AH_OK) return rc;
    if (p.nact == 0) {                             // the history advances even if nobody arrives
        h->rule_fresh = false;
        return AH_OK;
    }
    const cudaError_t e = asynchronous ? launch_exchange_in_order(p, h->stream)
                                       : launch_exchange(p, h->stream);
    if (e != cudaSuccess) return ah_cuda_fail(h, e);
    h->rule_fresh = false;
    h->launches += 1;
    return AH_OK;
}
