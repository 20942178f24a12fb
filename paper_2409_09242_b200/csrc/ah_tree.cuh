// Assembly of the squared distances ||x_i - c||^2 (Sec. V-B: u = log ||x_i - c||) from
// the per-tile sums that a distance round stores (see DistTree), at the head of the launch
// that needs them, and the weighting rule of Sec. V-B (Eqs. 10-11, h1 / h2) on the result.
// The sums follow the same adjacent-pairs binary tree whoever forms them, so the result
// is a pure function of the tile sums.  Not installed.
#pragma once

#include "ah_device.cuh"
#include "ah_internal.h"
#include "ah_weights.cuh"

namespace ah {

// Orders this thread's earlier writes (and those it has observed) before its later ones,
// and its later reads after its earlier ones, as seen from anywhere on the GPU (lighter
// than the sequentially consistent __threadfence()).
__device__ __forceinline__ void fence_gpu()
{
    asm volatile("fence.acq_rel.gpu;" ::: "memory");
}

__device__ __forceinline__ uint32_t ld_relaxed_gpu(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// A distance round's only contribution: the tile's sum goes to its level-0 slot.
__device__ __forceinline__ void tree_store_tile(const DistTree &T, uint32_t i, uint32_t tile, double v)
{
    T.sums_out[(size_t)i * T.n[0] + tile] = v;
}

// Nodes first, first + stride, ... of level L (numbered worker by worker over the live
// nodes), each by one warp: two children a lane, then the butterfly (the adjacent-pairs
// order).  Four nodes' loads are in flight before the first sum is formed.
__device__ __forceinline__ void tree_sum_nodes(const DistTree &T, uint32_t L, uint32_t first,
                                               uint32_t stride, int lane)
{
    const uint32_t per = T.live[L], total = T.K * per;
    const double *below = L == 1u ? T.sums_in : T.upper + (size_t)T.K * T.off[L - 1u];
    const uint32_t below_n = T.n[L - 1u], below_live = T.live[L - 1u];
    for (uint32_t base = first; base < total; base += 4u * stride) {
        double pair[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint32_t node = base + (uint32_t)q * stride;
            pair[q] = 0.0;
            if (node < total) {
                const uint32_t i = node / per, nd = node - i * per;
                const uint32_t children = min(1u << kTreeRadixLog2, below_live - (nd << kTreeRadixLog2));
                const double *child = below + (size_t)i * below_n + ((size_t)nd << kTreeRadixLog2);
                const uint32_t a = 2u * (uint32_t)lane, b = a + 1u;
                const double va = a < children ? __ldcg(child + a) : 0.0;
                const double vb = b < children ? __ldcg(child + b) : 0.0;
                pair[q] = __dadd_rn(va, vb);
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint32_t node = base + (uint32_t)q * stride;
            if (node < total) {                            // the same for every lane
                const double sum = warp_tree_sum(pair[q]);
                if (lane == 0) {
                    const uint32_t i = node / per, nd = node - i * per;
                    if (L == T.levels) T.norm2[i] = sum;
                    else T.upper[(size_t)T.K * T.off[L] + (size_t)i * T.n[L] + nd] = sum;
                }
            }
        }
    }
}

// The whole assembly, by `nthreads` threads (whole warps) of every CTA of the launch;
// `sync` is a barrier over exactly those threads and `scratch` one word of shared memory.
// Afterwards every calling CTA may read norm2[0 .. K) (with __ldcg), and, if the rule was
// asked for, finds the coefficients of worker w in h1s[w], h2s[w] (shared memory, may be
// null).  Kept out of line: it runs once per launch, and its double-double logarithm
// would otherwise claim registers in the streaming kernels.
template <class Sync>
static __device__ __noinline__ void assemble_distances(const DistTree &T, int tid, int nthreads,
                                                       uint32_t cta, float *h1s, float *h2s,
                                                       uint32_t *scratch, Sync sync)
{
    const int lane = tid & 31, warp = tid >> 5, nwarps = nthreads >> 5;
    for (uint32_t L = 1u; L <= T.levels; ++L) {
        if (L > T.shared_levels) {
            // few inputs: every CTA forms the whole level for itself (the CTAs store the
            // same values to the same places)
            tree_sum_nodes(T, L, (uint32_t)warp, (uint32_t)nwarps, lane);
            sync();
            continue;
        }
        if (cta < T.sync_ctas)
            tree_sum_nodes(T, L, cta * (uint32_t)nwarps + (uint32_t)warp,
                           T.sync_ctas * (uint32_t)nwarps, lane);
        sync();                                            // this CTA's share is stored
        if (tid == 0) {
            if (cta < T.sync_ctas) {
                fence_gpu();                               // ... and visible before it is counted
                atomicAdd(&T.arrive[L], 1u);
            }
            uint32_t polls = 0;
            bool there;
            while (!(there = (int32_t)(ld_relaxed_gpu(&T.arrive[L]) - T.arrive_target) >= 0) &&
                   polls < T.wait_polls) {
                ++polls;
                __nanosleep(64);
            }
            fence_gpu();                                   // what the counter announced is visible
            *scratch = there ? 0u : 1u;
        }
        sync();
        const bool alone = *scratch != 0u;
        sync();                                            // the word may be written again
        if (alone) {                                       // the others are late: the whole level here
            tree_sum_nodes(T, L, (uint32_t)warp, (uint32_t)nwarps, lane);
            sync();
        }
    }
    // ---- results to the host copy, the rule
    WeightRule rule;
    const size_t depth = (size_t)T.rule.p_hist + 1u;
    if (T.run_rule) {
        rule.p_hist = T.rule.p_hist;
        for (int j = 0; j < AH_MAX_HIST; ++j) rule.coef[j] = T.rule.coef[j];
        rule.kappa = T.rule.kappa;
        rule.alpha = T.rule_alpha;
    }
    for (uint32_t w = (uint32_t)tid; w < T.K; w += (uint32_t)nthreads) {
        const double n2 = __ldcg(&T.norm2[w]);
        if (cta == 0u) T.norm2_host[1u + w] = n2;
        if (T.run_rule) {
            float to_master, to_worker;
            weight_rule_step(rule, n2, T.ring_in + (size_t)w * depth,
                             cta == 0u ? T.ring_out + (size_t)w * depth : nullptr,
                             T.ring_filled != 0u, &to_master, &to_worker);
            if (h1s) { h1s[w] = to_worker; h2s[w] = to_master; }
            if (cta == 0u) { T.weights[w] = to_master; T.weights[T.K + w] = to_worker; }
        }
    }
    if (cta == 0u && tid == 0) {
        // the status word travels as the bit pattern of the first double, as it sits in
        // device memory in front of the distances; the host reads its copy only behind an
        // event that follows this kernel
        reinterpret_cast<uint32_t *>(T.norm2_host)[0] = __ldcg(T.status);
        reinterpret_cast<uint32_t *>(T.norm2_host)[1] = 0u;
    }
    sync();
}

}  // namespace ah
