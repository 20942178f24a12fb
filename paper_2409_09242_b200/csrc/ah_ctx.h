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
    double *sums[2] = {nullptr, nullptr};   // level 0 of the distance tree, two copies: [K][ntiles_pad]
    int sums_cur = 0;              // the copy that holds the latest distance round's tile sums
    ah::DistTree tree;             // the tree's shape and fixed addresses (per-launch fields unset)
    uint32_t arrive_total[ah::kTreeMaxLevels + 1] = {};   // what the tree's counters stand at
    bool tree_dirty = false;       // a kernel gave up half way: clear the tree's counters first
    uint32_t wait_polls = 4096;    // how long the CTAs of an assembling launch wait for one another
    double *norm2_dev = nullptr;   // [0] holds the status word, [1..K] the distances
    uint32_t *sched = nullptr;     // item scheduler of the local-step kernel (2 words)
    double *ring_dev[2] = {nullptr, nullptr};   // device copies of the history ring, [K][p_hist + 1]:
    int ring_cur = 0;              //   a rule on the device reads ring_dev[ring_cur] and writes the other
    float *weights_dev = nullptr;  // [2K] coefficients of the last dynamic exchange
    ah::Run *runs = nullptr;
    ah::TileInfo *tiles = nullptr;
    uint32_t nruns = 0;

    // host state
    double *norm2_host = nullptr;  // pinned, mapped copy of norm2_dev (status word + K doubles):
                                   // written by the launch that assembles the distances
    double *norm2_host_dev = nullptr;   // the same memory as the device addresses it
    cudaEvent_t norm2_ready = nullptr;
    bool sums_raw = false;         // the latest distance round's tile sums wait in sums[sums_cur]:
                                   // nobody has assembled them yet
    bool raw_rule = false;         // ... and whoever assembles them also runs the weighting rule,
    float raw_alpha = 0.f;         //     with this moving rate
    bool norm2_pending = false;    // distances of a want_dist step not yet used by a weight rule
    bool norm2_unread = false;     // ... and not yet copied into norm2_last
    int ring_home = 0;             // 0: the host copy of the ring is current, 1: the device copy
    bool lagged_ready = false;     // weights_dev holds the rule's output of an earlier fused round
    bool rule_fresh = false;       // the rule's output for the distances of the last want_dist
                                   // step (AH_DIST_AND_RULE) is owed to the next exchange (it is in
                                   // weights_dev once those distances have been assembled)
    float rule_fresh_alpha = 0.f;  // ... with this moving rate
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
// ah_host.cu: the life of a distance round's tile sums
int begin_distance_store(ah_ctx *h, DistTree &tree);       // a launch is about to store a round's sums
void commit_distance_store(ah_ctx *h, bool rule, float alpha, bool owed_to_exchange);
int begin_assembly(ah_ctx *h, bool run_rule, float alpha, DistTree &tree);
int commit_assembly(ah_ctx *h, const DistTree &tree);
int settle_distances(ah_ctx *h);   // assembles waiting sums with a kernel of its own, if any
int ring_to_host(ah_ctx *h);
int ring_to_device(ah_ctx *h);
int enqueue_weight_rule(ah_ctx *h, float alpha);   // ah_dynamic.cu
int fill_exchange(ah_ctx *h, const uint8_t *worker_mask, const float *weights, float alpha,
                  const uint16_t *order, const float *weights_dev, ExchangeParams &p);
cudaError_t launch_exchange_in_order(const ExchangeParams &p, cudaStream_t s);   // ah_exchange_async.cu
cudaError_t launch_assemble(const DistTree &T, uint32_t ctas, cudaStream_t s);   // ah_kernels.cu
}
