// The handle behind the opaque ah_ctx of adahess.h: shapes, device views into the
// workspace, and the host-side bookkeeping.  Shared by the translation units that
// implement entry points on a handle.  Not installed.
#pragma once

#include <vector>

#include "ah_internal.h"

struct ah_ctx {
    int K = 0;
    uint32_t P = 0;
    uint64_t lds = 0;              // row stride of x, m, v, c (P rounded up to 4)
    uint32_t ntiles = 0, ntiles_pad = 0;
    int device = 0;
    int sm_count = 0;
    bool has_device = true;        // false: bookkeeping-only handle (AH_DEVICE_NONE)
    std::vector<ah::Run> runs_host;
    std::vector<ah::TileInfo> tiles_host;
    cudaStream_t stream = nullptr;
    bool owns_workspace = false;
    void *workspace = nullptr;
    size_t workspace_bytes = 0;

    // device views into the workspace
    float *x = nullptr, *m = nullptr, *v = nullptr, *c = nullptr;
    double *partials = nullptr;    // level 0 of the distance tree: [K][ntiles_pad]
    ah::DistTree tree;             // the whole tree as the kernels see it (rule fields unset)
    size_t tree_count_bytes = 0;   // arrival counters (+ the finished-rows word) of the tree
    bool tree_dirty = false;       // a distance round failed half way: clear the counters first
    double *norm2_dev = nullptr;   // [0] holds the status word, [1..K] the distances
    uint32_t *sched = nullptr;     // item scheduler of the local-step kernel (2 words)
    uint32_t *ring_flag_dev = nullptr;   // device copy of ring_filled
    double *uhist_dev = nullptr;   // device copy of the history ring, [K][p_hist + 1]
    float *weights_dev = nullptr;  // [2K] coefficients of the last dynamic exchange
    ah::Run *runs = nullptr;
    ah::TileInfo *tiles = nullptr;
    uint32_t nruns = 0;

    // host state
    double *norm2_host = nullptr;  // pinned, mapped copy of norm2_dev (status word + K doubles):
                                   // written by the kernel that completes the last distance
    double *norm2_host_dev = nullptr;   // the same memory as the device addresses it
    cudaEvent_t norm2_ready = nullptr;
    bool norm2_pending = false;    // distances of a want_dist step not yet used by a weight rule
    bool norm2_unread = false;     // ... and not yet copied into norm2_last
    int ring_home = 0;             // 0: the host copy of the ring is current, 1: the device copy
    bool lagged_ready = false;     // weights_dev holds the rule's output of an earlier fused round
    bool rule_fresh = false;       // weights_dev holds the rule's output for the distances of the
                                   // last want_dist step (AH_DIST_AND_RULE), not yet used
    float rule_fresh_alpha = 0.f;  // ... computed with this moving rate
    double norm2_last[AH_MAX_WORKERS];
    uint32_t step[AH_MAX_WORKERS];
    uint32_t down_until[AH_MAX_WORKERS];
    uint32_t calls = 0;            // ah_local_step calls so far
    int p_hist = 4;
    double coef[AH_MAX_HIST];
    double kappa = -0.1;
    std::vector<double> uhist;     // [K][p_hist + 1], newest first
    int ring_filled = 0;

    int last_cuda = 0;
    uint64_t launches = 0;
};

// Records a failed runtime call on the handle and maps it to AH_ERR_CUDA.
inline int ah_cuda_fail(ah_ctx *h, cudaError_t e)
{
    if (h) h->last_cuda = (int)e;
    return AH_ERR_CUDA;
}

namespace ah {
int finish_distances(ah_ctx *h);   // ah_host.cu
int prepare_distance_round(ah_ctx *h, bool run_rule, float alpha, DistTree &tree);
void commit_rule_in_round(ah_ctx *h, float alpha);
int ring_to_host(ah_ctx *h);
int ring_to_device(ah_ctx *h);
int enqueue_weight_rule(ah_ctx *h, float alpha);   // ah_dynamic.cu
int fill_exchange(ah_ctx *h, const uint8_t *worker_mask, const float *weights, float alpha,
                  const uint16_t *order, const float *weights_dev, ExchangeParams &p);
cudaError_t launch_exchange_in_order(const ExchangeParams &p, cudaStream_t s);   // ah_exchange_async.cu
}
