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

// node / per: one mul-hi where the host found that exact for every node of the level
// (magic != 0), nothing at all at the root level.
__device__ __forceinline__ uint32_t tree_worker_of(uint32_t node, uint32_t per, uint32_t magic)
{
    if (per == 1u) return node;
    return magic ? __umulhi(node, magic) : node / per;
}

__device__ __forceinline__ uint32_t ld_relaxed_gpu(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// A distance round's only contribution: the tile's sum goes to its level-0 slot.  The line
// is asked to stay in the L2 cache: it is read once more, at the head of a later launch,
// after gigabytes of state have streamed past.
__device__ __forceinline__ void tree_store_tile(const DistTree &T, uint32_t i, uint32_t tile, double v)
{
    uint64_t keep;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(keep));
    asm volatile("st.global.L2::cache_hint.f64 [%0], %1, %2;"
                 :: "l"(T.sums_out + (size_t)i * T.n[0] + tile), "d"(v), "l"(keep) : "memory");
}

// Nodes first, first + stride, ... of level L (numbered worker by worker over the live
// nodes), each by one warp: two children a lane, then the butterfly (the adjacent-pairs
// order).  Four nodes' loads are in flight before the first sum is formed.  Returns how
// many nodes this warp summed.  Out of line and short: one copy of the code serves every
// level, and it runs once per launch, where fetching the instructions is most of the time.
static __device__ __noinline__ uint32_t tree_sum_nodes(const DistTree &T, uint32_t L, uint32_t first,
                                                       uint32_t stride, int lane)
{
    constexpr int kBatch = 4;
    const uint32_t per = T.live[L], total = T.K * per, magic = T.magic[L];
    const double *below = L == 1u ? T.sums_in : T.upper + (size_t)T.K * T.off[L - 1u];
    const uint32_t below_n = T.n[L - 1u], below_live = T.live[L - 1u];
    uint32_t done = 0;
    for (uint32_t base = first; base < total; base += (uint32_t)kBatch * stride) {
        double pair[kBatch];
#pragma unroll
        for (int q = 0; q < kBatch; ++q) {
            const uint32_t node = base + (uint32_t)q * stride;
            pair[q] = 0.0;
            if (node < total) {
                const uint32_t i = tree_worker_of(node, per, magic), nd = node - i * per;
                const uint32_t children = min(1u << kTreeRadixLog2, below_live - (nd << kTreeRadixLog2));
                const double *child = below + (size_t)i * below_n + ((size_t)nd << kTreeRadixLog2);
                const uint32_t a = 2u * (uint32_t)lane, b = a + 1u;
                const double va = a < children ? __ldcg(child + a) : 0.0;
                const double vb = b < children ? __ldcg(child + b) : 0.0;
                pair[q] = __dadd_rn(va, vb);
            }
        }
#pragma unroll
        for (int q = 0; q < kBatch; ++q) {
            const uint32_t node = base + (uint32_t)q * stride;
            if (node < total) {                            // the same for every lane
                const double sum = warp_tree_sum(pair[q]);
                if (lane == 0) {
                    const uint32_t i = tree_worker_of(node, per, magic), nd = node - i * per;
                    if (L == T.levels) T.norm2[i] = sum;
                    else T.upper[(size_t)T.K * T.off[L] + (size_t)i * T.n[L] + nd] = sum;
                }
                ++done;
            }
        }
    }
    return done;
}

// The whole assembly, by `nthreads` threads (whole warps) of every CTA of the launch (cta
// of nctas); `sync` is a barrier over exactly those threads and `scratch` two words of
// shared memory.  Afterwards every calling CTA may read norm2[0 .. K) (with __ldcg), and,
// if the rule was asked for, finds the coefficients of worker w in h1s[w], h2s[w] (shared
// memory; null where the caller does not use them).  `tree_done` is called by every thread
// when the loads of the tree and of the rule are over: the moment for the caller's bulk
// traffic to start, since those few small loads would otherwise queue behind it.  Kept out of
// line: it runs once per launch, and its double-double logarithm would otherwise claim
// registers in the streaming kernels.
template <class Sync, class TreeDone>
static __device__ __noinline__ void assemble_distances(const DistTree &T, int tid, int nthreads,
                                                       uint32_t cta, uint32_t nctas, float *h1s,
                                                       float *h2s, uint32_t *scratch, Sync sync,
                                                       TreeDone tree_done)
{
    const int lane = tid & 31, warp = tid >> 5, nwarps = nthreads >> 5;
    const size_t depth = (size_t)T.rule.p_hist + 1u;
    if (T.run_rule && T.ring_filled)                       // the rule's history: on its way while
        for (uint32_t w = (uint32_t)tid; w < T.K; w += (uint32_t)nthreads) {      // the sums form
            asm volatile("prefetch.global.L2 [%0];" :: "l"(T.ring_in + (size_t)w * depth));
            asm volatile("prefetch.global.L2 [%0];" :: "l"(T.ring_in + (size_t)w * depth + depth - 1u));
        }
    if (tid == 0) scratch[1] = 0u;
    sync();
    // While the tree is formed (memory is quiet, and the last warp has the least to do), one
    // thread runs the logarithm once for nothing: its instructions and constants are then at
    // hand when the rule needs them, whatever the other CTAs are streaming by that time.
    if (T.run_rule && h1s && warp == nwarps - 1 && lane == 31)
        if (u_from_norm2(T.rule_alpha + 2.0) == -1.0) scratch[0] = 0u;      // never true
    for (uint32_t L = 1u; L <= T.levels; ++L) {
        if (L > T.shared_levels) {
            // few inputs: every CTA forms the whole level for itself (the CTAs store the
            // same values to the same places)
            tree_sum_nodes(T, L, (uint32_t)warp, (uint32_t)nwarps, lane);
            sync();
            continue;
        }
        // this CTA's share of the level, then the count of what it finished
        const uint32_t mine = tree_sum_nodes(T, L, cta * (uint32_t)nwarps + (uint32_t)warp,
                                             nctas * (uint32_t)nwarps, lane);
        if (lane == 0 && mine) atomicAdd(&scratch[1], mine);
        sync();                                            // the share is stored and tallied
        if (tid == 0) {
            const uint32_t finished = scratch[1];
            scratch[1] = 0u;
            if (finished) {
                fence_gpu();                               // the sums are visible before they count
                atomicAdd(&T.arrive[L], finished);
            }
            uint32_t polls = 0;
            bool there;
            while (!(there = (int32_t)(ld_relaxed_gpu(&T.arrive[L]) - T.arrive_target[L]) >= 0) &&
                   polls < T.wait_polls) {
                ++polls;
                __nanosleep(32);
            }
            fence_gpu();                                   // what the counter announced is visible
            scratch[0] = there ? 0u : 1u;
        }
        sync();
        if (scratch[0] != 0u) {                            // the others are late: the whole level here
            tree_sum_nodes(T, L, (uint32_t)warp, (uint32_t)nwarps, lane);
            sync();
        }
    }
    // ---- the rule, in every CTA of a launch that uses the coefficients (all of them finish
    // it at the same moment: from here on nothing but arithmetic separates them from their
    // first tile, and a CTA that fell behind would have to fetch through the others' traffic);
    // CTA 0 stores what the rule leaves behind
    const bool use_here = h1s != nullptr;
    if (T.run_rule && (use_here || cta == 0u))
        for (uint32_t w = (uint32_t)tid; w < T.K; w += (uint32_t)nthreads) {
            const double n2 = __ldcg(&T.norm2[w]);
            float to_master, to_worker;
            weight_rule_step(T.rule.p_hist, T.rule.coef, T.rule.kappa, T.rule_alpha, n2,
                             T.ring_in + (size_t)w * depth,
                             cta == 0u ? T.ring_out + (size_t)w * depth : nullptr,
                             T.ring_filled != 0u, &to_master, &to_worker);
            if (use_here) { h1s[w] = to_worker; h2s[w] = to_master; }
            if (cta == 0u) { T.weights[w] = to_master; T.weights[T.K + w] = to_worker; }
        }
    tree_done();
    if (cta == 0u) {
        // results and status word to the host copy; the word travels as the bit pattern of
        // the first double, as it sits in device memory in front of the distances; the host
        // reads its copy only behind an event that follows this kernel
        for (uint32_t w = (uint32_t)tid; w < T.K; w += (uint32_t)nthreads)
            T.norm2_host[1u + w] = __ldcg(&T.norm2[w]);
        if (tid == 0) {
            reinterpret_cast<uint32_t *>(T.norm2_host)[0] = __ldcg(T.status);
            reinterpret_cast<uint32_t *>(T.norm2_host)[1] = 0u;
        }
    }
    sync();
}

}  // namespace ah
