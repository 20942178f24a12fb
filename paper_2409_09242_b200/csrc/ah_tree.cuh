// Assembly of the squared distances ||x_i - c||^2 (Sec. V-B: u = log ||x_i - c||) inside
// the kernels that produce the per-tile sums, with no launch of its own: an arrival tree
// of radix 64 over the tiles of each worker (see DistTree), then, by whoever completes
// the last worker, the copy of the results to pinned host memory and the weighting rule
// of Sec. V-B (Eqs. 10-11, h1 / h2).  The sums follow the same adjacent-pairs binary tree
// whatever the order of arrival, so the result is a pure function of the tile sums.
// Not installed.
#pragma once

#include "ah_device.cuh"
#include "ah_internal.h"
#include "ah_weights.cuh"

namespace ah {

// Orders this thread's earlier writes before its later ones, and its later reads after
// its earlier ones, as seen from anywhere on the GPU (lighter than the sequentially
// consistent __threadfence()).
__device__ __forceinline__ void fence_gpu()
{
    asm volatile("fence.acq_rel.gpu;" ::: "memory");
}

// By one warp, after every root of the round is complete: results and status word to the
// host copy, then the rule for all workers.  Kept out of line: it runs once per round and
// its double-double logarithm would otherwise claim registers in the streaming kernels.
static __device__ __noinline__ void finish_round(const DistTree &T, int lane)
{
    fence_gpu();                                       // the roots other warps wrote
    const bool filled = __ldcg(T.ring_flag) != 0u;
    __syncwarp();
    WeightRule rule;
    if (T.run_rule) {
        rule.p_hist = T.rule.p_hist;
        for (int j = 0; j < AH_MAX_HIST; ++j) rule.coef[j] = T.rule.coef[j];
        rule.kappa = T.rule.kappa;
        rule.alpha = T.rule_alpha;
    }
    for (uint32_t w = (uint32_t)lane; w < T.K; w += 32u) {
        const double n2 = __ldcg(&T.norm2[w]);
        T.norm2_host[1u + w] = n2;
        if (T.run_rule)
            weight_rule_step(rule, n2, T.uhist + (size_t)w * (size_t)(rule.p_hist + 1), filled,
                             &T.weights[w], &T.weights[T.K + w]);
    }
    if (lane == 0) {
        // the status word travels as the bit pattern of the first double, as it sits in
        // device memory in front of the distances
        reinterpret_cast<uint32_t *>(T.norm2_host)[0] = __ldcg(T.status);
        reinterpret_cast<uint32_t *>(T.norm2_host)[1] = 0u;
        if (T.run_rule) *T.ring_flag = 1u;
    }
    // the host reads its copy only behind an event that follows this kernel
}

// Live children of node `parent` of level L (L >= 1): nodes of level L - 1 that exist.
__device__ __forceinline__ uint32_t tree_children(const DistTree &T, uint32_t L, uint32_t parent)
{
    return min(1u << kTreeRadixLog2, T.live[L - 1] - (parent << kTreeRadixLog2));
}

__device__ __forceinline__ uint32_t *tree_counter(const DistTree &T, uint32_t L, uint32_t i,
                                                  uint32_t node)
{
    return T.count + (size_t)T.K * T.off[L] + (size_t)i * T.n[L] + node;
}

// A tile's sum reaches the tree in three steps that a caller may spread over time, so
// that no memory round trip sits on its critical path (each step by itself is correct
// however long after the previous one it runs):
//   1. tree_store_tile  (one lane)   the sum goes to its level-0 slot;
//   2. tree_count_tile  (same lane)  a fence, then the arrival is counted at the tile's
//                                    level-1 node; returns the arrivals before this one;
//   3. tree_after_counts (whole warp, one counted tile per lane) where an arrival was its
//                                    node's last, the node is summed and delivered upwards,
//                                    as far as that completes nodes.
__device__ __forceinline__ void tree_store_tile(const DistTree &T, uint32_t i, uint32_t tile, double v)
{
    T.level0[(size_t)i * T.n[0] + tile] = v;
}

__device__ __forceinline__ uint32_t tree_count_tile(const DistTree &T, uint32_t i, uint32_t tile)
{
    fence_gpu();                                       // the sum is visible before it is counted
    return atomicAdd(tree_counter(T, 1u, i, tile >> kTreeRadixLog2), 1u);
}

// Every lane with `climbing` set has just completed the level-1 node above its tile.  The
// warp sums those nodes one after the other, all 32 lanes on one node at a time (two
// children a lane, then the butterfly: the adjacent-pairs order; the loads of eight nodes
// are issued before the first sum is formed), delivers each to its parent, and repeats
// with the lanes whose delivery completed the parent.  All 32 lanes must call; at the
// top, whoever completes the last worker has the whole warp finish the round.
static __device__ __noinline__ void tree_climb(const DistTree &T, bool climbing, uint32_t i,
                                               uint32_t tile, int lane)
{
    uint32_t node = tile >> kTreeRadixLog2, L = 1u;
    bool last_row = false;
    fence_gpu();                                       // counted children are visible from here on
    for (uint32_t todo = __ballot_sync(0xffffffffu, climbing); todo != 0u;
         todo = __ballot_sync(0xffffffffu, climbing)) {
        // the nodes of this pass, eight at a time: loads first, sums after
        double mine = 0.0;                             // lane e ends up with the sum of its own node
        for (uint32_t rest = todo; rest != 0u;) {
            double pair[8];
            int owner[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                owner[q] = rest ? __ffs(rest) - 1 : -1;
                if (rest) rest &= rest - 1u;
                pair[q] = 0.0;
                if (owner[q] >= 0) {
                    const uint32_t oi = __shfl_sync(0xffffffffu, i, owner[q]);
                    const uint32_t on = __shfl_sync(0xffffffffu, node, owner[q]);
                    const uint32_t oL = __shfl_sync(0xffffffffu, L, owner[q]);
                    const double *below = oL == 1u ? T.level0 + (size_t)oi * T.n[0]
                                                   : T.upper + (size_t)T.K * T.off[oL - 1u] + (size_t)oi * T.n[oL - 1u];
                    const uint32_t children = tree_children(T, oL, on);
                    const double *child = below + ((size_t)on << kTreeRadixLog2);
                    const uint32_t a = 2u * (uint32_t)lane, b = a + 1u;
                    const double va = a < children ? __ldcg(child + a) : 0.0;
                    const double vb = b < children ? __ldcg(child + b) : 0.0;
                    pair[q] = __dadd_rn(va, vb);
                }
            }
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (owner[q] >= 0) {
                    const double sum = warp_tree_sum(pair[q]);
                    if (lane == owner[q]) mine = sum;
                }
        }
        // every owner delivers its node upwards
        if (climbing) {
            *tree_counter(T, L, i, node) = 0u;         // ready for the next round
            if (L == T.levels) {                       // the root of worker i
                T.norm2[i] = mine;
                fence_gpu();
                last_row = atomicAdd(T.rows_done, 1u) + 1u == T.K;
                climbing = false;
            } else {
                T.upper[(size_t)T.K * T.off[L] + (size_t)i * T.n[L] + node] = mine;
                fence_gpu();
                const uint32_t parent = node >> kTreeRadixLog2;
                climbing = atomicAdd(tree_counter(T, L + 1u, i, parent), 1u) + 1u ==
                           tree_children(T, L + 1u, parent);
                node = parent;
                ++L;
            }
        }
        fence_gpu();                                   // what the counters announced is visible
    }
    if (__any_sync(0xffffffffu, last_row)) {
        if (last_row) *T.rows_done = 0u;
        finish_round(T, lane);
    }
}

// Step 3 for a whole warp at once: lane by lane, (valid, i, tile, before) describe one
// counted tile sum.  All 32 lanes, converged.  The common case (no count completed a
// node) costs one vote.
__device__ __forceinline__ void tree_after_counts(const DistTree &T, bool valid, uint32_t i,
                                                  uint32_t tile, uint32_t before, int lane)
{
    const bool climbing = valid && before + 1u == tree_children(T, 1u, tile >> kTreeRadixLog2);
    if (__any_sync(0xffffffffu, climbing)) tree_climb(T, climbing, i, tile, lane);
}

// The three steps at once for one tile sum.  All 32 lanes of a converged warp; `value`
// counts in lane 0.
__device__ __forceinline__ void deliver_tile_sum(const DistTree &T, uint32_t i, uint32_t tile,
                                                 double value, int lane)
{
    uint32_t before = 0;
    if (lane == 0) {
        tree_store_tile(T, i, tile, value);
        before = tree_count_tile(T, i, tile);
    }
    tree_after_counts(T, lane == 0, i, tile, before, lane);
}

}  // namespace ah
