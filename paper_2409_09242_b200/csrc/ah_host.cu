// Host side of the AdaHessian + elastic-averaging library: the handle, argument
// checks, workspace layout, the per-tile tensor descriptors, and the O(K) weight and
// failure bookkeeping of the dynamic weighting rule.  Kernels live in ah_kernels.cu.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include "ah_ctx.h"
#include "ah_weights.cuh"

using namespace ah;

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

inline uint32_t pow2_at_least(uint32_t n)
{
    uint32_t p = 1;
    while (p < n) p <<= 1;
    return p;
}

int cuda_fail(ah_ctx *h, cudaError_t e)
{
    if (h) h->last_cuda = (int)e;
    return AH_ERR_CUDA;
}

#define AH_CUDA(h, call)                                    \
    do {                                                    \
        cudaError_t e_ = (call);                            \
        if (e_ != cudaSuccess) return cuda_fail((h), e_);   \
    } while (0)

struct Layout {
    size_t x, m, v, c, sums[2], upper, arrive, norm2, sched, ring[2], weights, runs, tiles, total;
};

// Shape of the distance tree over ntp = 2^a tile slots of which ntiles exist: nodes per
// worker at every level, how many of them are live, where each level starts, and which
// levels are large enough (over all K workers) to be shared between CTAs.  Returns the
// nodes per worker above level 0.
uint32_t tree_shape(uint32_t ntiles, uint32_t ntp, uint32_t K, DistTree &T)
{
    T.n[0] = ntp;
    T.live[0] = ntiles;
    T.off[0] = 0;
    uint32_t L = 0, above = 0;
    do {
        ++L;
        T.n[L] = T.n[L - 1] >> kTreeRadixLog2 ? T.n[L - 1] >> kTreeRadixLog2 : 1u;
        T.live[L] = (T.live[L - 1] + (1u << kTreeRadixLog2) - 1u) >> kTreeRadixLog2;
        T.off[L] = above;
        above += T.n[L];
    } while (T.n[L] > 1u);
    T.levels = L;
    for (uint32_t q = L + 1; q <= (uint32_t)kTreeMaxLevels; ++q) T.n[q] = T.live[q] = T.off[q] = 0u;
    T.K = K;
    // node / live[q] == mulhi(node, ceil(2^32 / live[q])) for every node < K * live[q] as long
    // as K * live[q]^2 < 2^32; otherwise (magic 0) the kernels divide
    for (uint32_t q = 0; q <= (uint32_t)kTreeMaxLevels; ++q) {
        const uint64_t d = T.live[q];
        T.magic[q] = d > 1u && (uint64_t)K * d * d < (1ull << 32) ? (uint32_t)(((1ull << 32) + d - 1) / d) : 0u;
    }
    T.shared_levels = 0;
    for (uint32_t q = 1; q <= L; ++q)
        if ((uint64_t)K * T.live[q - 1] > kTreeOwnLevelInputs) T.shared_levels = q;
    return above;
}

// Offsets of every array inside the workspace (each 256-byte aligned).
Layout workspace_layout(int K, uint64_t P, int nruns_max)
{
    const uint64_t lds = (P + 3) / 4 * 4;
    const uint32_t ntiles = (uint32_t)((P + kTile - 1) / kTile);
    const uint32_t ntp = pow2_at_least(ntiles);
    Layout L;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    L.x = take((size_t)K * lds * sizeof(float));
    L.m = take((size_t)K * lds * sizeof(float));
    L.v = take((size_t)K * lds * sizeof(float));
    L.c = take((size_t)lds * sizeof(float));
    L.sums[0] = take((size_t)K * ntp * sizeof(double));
    L.sums[1] = take((size_t)K * ntp * sizeof(double));
    DistTree shape;
    const uint32_t above = tree_shape(ntiles, ntp, (uint32_t)K, shape);
    L.upper = take((size_t)K * above * sizeof(double));
    L.arrive = take((kTreeMaxLevels + 1) * sizeof(uint32_t));
    L.norm2 = take((size_t)(AH_MAX_WORKERS + 1) * sizeof(double));
    L.sched = take(4 * sizeof(uint32_t));                 // item counter, exit counter
    L.ring[0] = take((size_t)K * (AH_MAX_HIST + 1) * sizeof(double));
    L.ring[1] = take((size_t)K * (AH_MAX_HIST + 1) * sizeof(double));
    L.weights = take(2 * (size_t)K * sizeof(float));
    L.runs = take((size_t)nruns_max * sizeof(Run));
    L.tiles = take((size_t)ntiles * sizeof(TileInfo));
    L.total = off;
    return L;
}

// Cut [0, P) into maximal runs of equal spatial block; gaps behave as block 1.
int build_runs(uint64_t P, const ah_segment *segs, int nseg, std::vector<Run> &runs)
{
    runs.clear();
    auto push = [&](uint64_t a, uint64_t b, uint32_t block) {
        if (a >= b) return;
        if (!runs.empty() && runs.back().block == 1 && block == 1 && runs.back().end == a) {
            runs.back().end = (uint32_t)b;
            return;
        }
        Run r;
        r.start = (uint32_t)a;
        r.end = (uint32_t)b;
        r.block = block;
        r.magic = block > 1 ? (uint32_t)(((1ull << 32) + block - 1) / block) : 0u;
        runs.push_back(r);
    };
    uint64_t pos = 0;
    for (int s = 0; s < nseg; ++s) {
        const ah_segment &g = segs[s];
        if (g.block < 1 || g.block > AH_MAX_BLOCK) return AH_ERR_SEGMENTS;
        if (g.offset < pos || g.offset > P || g.length > P - g.offset) return AH_ERR_SEGMENTS;
        if (g.length % g.block != 0) return AH_ERR_SEGMENTS;
        push(pos, g.offset, 1);
        push(g.offset, g.offset + g.length, g.block);
        pos = g.offset + g.length;
    }
    push(pos, P, 1);
    return AH_OK;
}

void build_tiles(uint32_t P, const std::vector<Run> &runs, std::vector<TileInfo> &tiles)
{
    const uint32_t ntiles = (P + kTile - 1) / kTile;
    tiles.resize(ntiles);
    size_t ri = 0;
    for (uint32_t t = 0; t < ntiles; ++t) {
        const uint32_t t0 = t * (uint32_t)kTile;
        const uint32_t t1 = (uint64_t)t0 + kTile < P ? t0 + kTile : P;
        while (runs[ri].end <= t0) ++ri;
        TileInfo ti;
        ti.run0 = (uint32_t)ri;
        const Run &first = runs[ri];
        ti.e0 = first.block > 1 ? first.start + (t0 - first.start) / first.block * first.block : t0;
        size_t rj = ri;
        uint32_t flags = 0;
        bool all9 = true;
        for (;;) {
            if (runs[rj].block > 1) { flags |= 1u; if (runs[rj].block != 9) all9 = false; }
            if (runs[rj].end >= t1) break;
            ++rj;
        }
        if ((flags & 1u) && all9) flags |= 2u;
        const Run &last = runs[rj];
        ti.e1 = last.block > 1
                    ? last.start + ((t1 - 1 - last.start) / last.block + 1) * last.block
                    : t1;
        ti.flags = flags;
        tiles[t] = ti;
    }
}

void reset_history(ah_ctx *h)
{
    h->uhist.assign((size_t)h->K * (size_t)(h->p_hist + 1), 0.0);
    h->ring_filled = 0;
}

}  // namespace

// The history ring of the weighting rule has a host copy and device copies; ring_home
// says which side is current.  These bring the other side up to date.  A rule that is
// still owed on waiting tile sums runs first: it belongs in front of whatever looks at
// the ring next.
int ah::ring_to_host(ah_ctx *h)
{
    if (!h->has_device) return AH_OK;
    const int rc = settle_distances(h);
    if (rc != AH_OK) return rc;
    if (h->ring_home == 0) return AH_OK;
    AH_CUDA(h, cudaStreamSynchronize(h->stream));
    const size_t depth = (size_t)h->p_hist + 1;
    AH_CUDA(h, cudaMemcpy(h->uhist.data(), h->ring_dev[h->ring_cur], (size_t)h->K * depth * sizeof(double),
                          cudaMemcpyDeviceToHost));
    h->ring_filled = 1;           // a rule has run on the device
    h->ring_home = 0;
    return AH_OK;
}

// Uploads the host copy of the ring if it is the current one.  The device copy becomes the
// current one only when a rule has been enqueued behind the upload: the caller sets
// ring_home = 1 after that launch has succeeded.
int ah::ring_to_device(ah_ctx *h)
{
    if (h->ring_home == 1) return AH_OK;
    const size_t depth = (size_t)h->p_hist + 1;
    // pageable source: the call returns once the data has been staged
    AH_CUDA(h, cudaMemcpyAsync(h->ring_dev[h->ring_cur], h->uhist.data(),
                               (size_t)h->K * depth * sizeof(double), cudaMemcpyHostToDevice, h->stream));
    return AH_OK;
}

// A launch is about to store a distance round's tile sums: they go to the copy of level 0
// that holds nothing anybody still needs.
int ah::begin_distance_store(ah_ctx *h, DistTree &tree)
{
    // sums of an earlier round that nobody has assembled: if a rule is owed on them it
    // runs now (the history advances once per such round); otherwise they are superseded
    if (h->sums_raw && h->raw_rule && !tree.assemble) {
        const int rc = settle_distances(h);
        if (rc != AH_OK) return rc;
    }
    tree.sums_out = h->sums[h->sums_cur ^ 1];
    return AH_OK;
}

// ... and has been enqueued.  `rule`: whoever assembles these sums also runs the weighting
// rule with moving rate alpha; `owed_to_exchange`: its output belongs to the next exchange
// (AH_DIST_AND_RULE).
void ah::commit_distance_store(ah_ctx *h, bool rule, float alpha, bool owed_to_exchange)
{
    h->sums_cur ^= 1;
    h->sums_raw = true;
    h->raw_rule = rule;
    h->raw_alpha = alpha;
    h->norm2_pending = true;
    h->norm2_unread = true;
    h->rule_fresh = owed_to_exchange;
    if (owed_to_exchange) h->rule_fresh_alpha = alpha;
}

// A launch is about to assemble the waiting tile sums at its head, and to run the
// weighting rule on the result if asked.
int ah::begin_assembly(ah_ctx *h, bool run_rule, float alpha, DistTree &tree)
{
    if (h->tree_dirty) {          // an earlier kernel stopped half way
        AH_CUDA(h, cudaMemsetAsync(h->tree.arrive, 0, (kTreeMaxLevels + 1) * sizeof(uint32_t), h->stream));
        memset(h->arrive_total, 0, sizeof h->arrive_total);
        h->tree_dirty = false;
    }
    tree.assemble = 1u;
    tree.sums_in = h->sums[h->sums_cur];
    for (uint32_t L = 1; L <= tree.shared_levels; ++L)     // the counters count finished nodes
        tree.arrive_target[L] = h->arrive_total[L] + tree.K * tree.live[L];
    tree.wait_polls = h->wait_polls;
    tree.run_rule = run_rule ? 1u : 0u;
    tree.rule_alpha = (double)alpha;
    if (run_rule) {
        const int rc = ring_to_device(h);
        if (rc != AH_OK) return rc;
        memset(&tree.rule, 0, sizeof tree.rule);
        for (int j = 0; j < h->p_hist; ++j) tree.rule.coef[j] = h->coef[j];
        tree.rule.kappa = h->kappa;
        tree.rule.p_hist = h->p_hist;
        tree.ring_in = h->ring_dev[h->ring_cur];
        tree.ring_out = h->ring_dev[h->ring_cur ^ 1];
        tree.ring_filled = h->ring_home == 1 ? 1u : (uint32_t)(h->ring_filled != 0);
    }
    return AH_OK;
}

// ... and has been enqueued: the K doubles (and the status word in front of them) will be
// in pinned host memory once it has run, so an event behind it is all the host needs to
// wait for; the rule's bookkeeping follows.
int ah::commit_assembly(ah_ctx *h, const DistTree &tree)
{
    for (uint32_t L = 1; L <= tree.shared_levels; ++L) h->arrive_total[L] = tree.arrive_target[L];
    h->sums_raw = false;
    if (tree.run_rule) {
        h->ring_cur ^= 1;
        h->ring_home = 1;         // the device copy of the ring leads
        h->norm2_pending = false; // these distances have fed the rule
        h->lagged_ready = true;   // weights_dev holds coefficients
    }
    AH_CUDA(h, cudaEventRecord(h->norm2_ready, h->stream));
    return AH_OK;
}

// Readers other than a fused exchange: the waiting sums are assembled by a small kernel
// of its own (and the rule that is owed on them runs there).
int ah::settle_distances(ah_ctx *h)
{
    if (!h->has_device || !h->sums_raw) return AH_OK;
    DistTree tree = h->tree;
    // one warp a node of the first level, four warps a CTA, at most two CTAs per SM
    const uint64_t nodes = (uint64_t)h->K * tree.live[1];
    uint32_t ctas = (uint32_t)((nodes + 3) / 4);
    if (ctas > 2u * (uint32_t)h->sm_count) ctas = 2u * (uint32_t)h->sm_count;
    if (ctas < 1u) ctas = 1u;
    const int rc = begin_assembly(h, h->raw_rule, h->raw_alpha, tree);
    if (rc != AH_OK) return rc;
    AH_CUDA(h, launch_assemble(tree, ctas, h->stream));
    h->launches += 1;
    return commit_assembly(h, tree);
}

extern "C" {

int ah_workspace_bytes(int K, uint64_t P, int nseg, size_t *out)
{
    if (!out || K < 1 || K > AH_MAX_WORKERS || P < 1 || P >= (1ull << 31) || nseg < 0)
        return AH_ERR_INVALID_ARG;
    *out = workspace_layout(K, P, 2 * nseg + 1).total;
    return AH_OK;
}

int ah_init(ah_ctx **out, int K, uint64_t P, const ah_segment *segs, int nseg, const ah_alloc *opt)
{
    if (!out) return AH_ERR_INVALID_ARG;
    *out = nullptr;
    if (K < 1 || K > AH_MAX_WORKERS || P < 1 || P >= (1ull << 31) || nseg < 0 || (nseg > 0 && !segs))
        return AH_ERR_INVALID_ARG;

    std::vector<Run> runs;
    int rc = build_runs(P, segs, nseg, runs);
    if (rc != AH_OK) return rc;
    std::vector<TileInfo> tiles;
    build_tiles((uint32_t)P, runs, tiles);

    ah_ctx *h = new (std::nothrow) ah_ctx();
    if (!h) return AH_ERR_ALLOC;
    h->K = K;
    h->P = (uint32_t)P;
    h->lds = (P + 3) / 4 * 4;
    h->ntiles = (uint32_t)tiles.size();
    h->ntiles_pad = pow2_at_least(h->ntiles);
    h->nruns = (uint32_t)runs.size();
    memset(h->step, 0, sizeof(h->step));
    memset(h->down_until, 0, sizeof(h->down_until));
    memset(h->norm2_last, 0, sizeof(h->norm2_last));
    const double c_default[4] = {0.4, 0.3, 0.2, 0.1};
    memcpy(h->coef, c_default, sizeof(c_default));
    reset_history(h);

    h->runs_host = runs;
    h->tiles_host = tiles;
    if (opt && opt->device == AH_DEVICE_NONE) {
        h->has_device = false;
        *out = h;
        return AH_OK;
    }

    auto fail = [&](int code) { ah_destroy(h); return code; };

    cudaError_t e;
    if (opt && opt->device >= 0) {
        h->device = opt->device;
        if ((e = cudaSetDevice(h->device)) != cudaSuccess) { h->last_cuda = (int)e; return fail(AH_ERR_CUDA); }
    } else if ((e = cudaGetDevice(&h->device)) != cudaSuccess) {
        h->last_cuda = (int)e;
        return fail(AH_ERR_CUDA);
    }
    h->stream = opt ? (cudaStream_t)opt->cuda_stream : nullptr;

    const Layout L = workspace_layout(K, P, 2 * nseg + 1);
    h->workspace_bytes = L.total;
    if (opt && opt->workspace) {
        if (((uintptr_t)opt->workspace & 255u) != 0) return fail(AH_ERR_ALIGN);
        if (opt->workspace_bytes < L.total) return fail(AH_ERR_ALLOC);
        h->workspace = opt->workspace;
    } else {
        if ((e = cudaMalloc(&h->workspace, L.total)) != cudaSuccess) {
            h->last_cuda = (int)e;
            h->workspace = nullptr;
            return fail(AH_ERR_ALLOC);
        }
        h->owns_workspace = true;
    }
    char *base = (char *)h->workspace;
    h->x = (float *)(base + L.x);
    h->m = (float *)(base + L.m);
    h->v = (float *)(base + L.v);
    h->c = (float *)(base + L.c);
    h->sums[0] = (double *)(base + L.sums[0]);
    h->sums[1] = (double *)(base + L.sums[1]);
    h->norm2_dev = (double *)(base + L.norm2);
    h->sched = (uint32_t *)(base + L.sched);
    h->ring_dev[0] = (double *)(base + L.ring[0]);
    h->ring_dev[1] = (double *)(base + L.ring[1]);
    h->weights_dev = (float *)(base + L.weights);
    h->runs = (Run *)(base + L.runs);
    h->tiles = (TileInfo *)(base + L.tiles);

    if ((e = cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device)) !=
        cudaSuccess) {
        h->last_cuda = (int)e;
        return fail(AH_ERR_CUDA);
    }
    if ((e = cudaHostAlloc((void **)&h->norm2_host, (AH_MAX_WORKERS + 1) * sizeof(double),
                           cudaHostAllocMapped)) != cudaSuccess ||
        (e = cudaHostGetDevicePointer((void **)&h->norm2_host_dev, h->norm2_host, 0)) != cudaSuccess ||
        (e = cudaEventCreateWithFlags(&h->norm2_ready, cudaEventDisableTiming)) != cudaSuccess) {
        h->last_cuda = (int)e;
        return fail(AH_ERR_ALLOC);
    }
    memset(h->norm2_host, 0, (AH_MAX_WORKERS + 1) * sizeof(double));
    // the distance tree as the kernels see it: shape and fixed addresses
    memset(&h->tree, 0, sizeof h->tree);
    tree_shape(h->ntiles, h->ntiles_pad, (uint32_t)K, h->tree);
    h->tree.upper = (double *)(base + L.upper);
    h->tree.arrive = (uint32_t *)(base + L.arrive);
    h->tree.norm2 = h->norm2_dev + 1;
    h->tree.norm2_host = h->norm2_host_dev;
    h->tree.status = reinterpret_cast<const uint32_t *>(h->norm2_dev);
    h->tree.weights = h->weights_dev;
    // state (and its row padding) starts at zero; descriptors go up once
    if ((e = cudaMemsetAsync(h->workspace, 0, L.runs, h->stream)) != cudaSuccess ||
        (e = cudaMemcpyAsync(h->runs, runs.data(), runs.size() * sizeof(Run), cudaMemcpyHostToDevice,
                             h->stream)) != cudaSuccess ||
        (e = cudaMemcpyAsync(h->tiles, tiles.data(), tiles.size() * sizeof(TileInfo),
                             cudaMemcpyHostToDevice, h->stream)) != cudaSuccess ||
        (e = cudaStreamSynchronize(h->stream)) != cudaSuccess) {
        h->last_cuda = (int)e;
        return fail(AH_ERR_CUDA);
    }
    *out = h;
    return AH_OK;
}

int ah_destroy(ah_ctx *h)
{
    if (!h) return AH_OK;
    int rc = AH_OK;
    if (h->has_device && (h->workspace || h->norm2_host)) {
        cudaError_t e = cudaStreamSynchronize(h->stream);
        if (e != cudaSuccess) rc = AH_ERR_CUDA;
    }
    if (h->norm2_ready) cudaEventDestroy(h->norm2_ready);
    if (h->norm2_host) cudaFreeHost(h->norm2_host);
    if (h->owns_workspace && h->workspace) cudaFree(h->workspace);
    delete h;
    return rc;
}

int ah_broadcast_center(ah_ctx *h)
{
    if (!h) return AH_ERR_INVALID_ARG;
    if (!h->has_device) return AH_ERR_STATE;
    AH_CUDA(h, launch_broadcast(h->x, h->c, h->lds, h->K, h->stream));
    h->launches += 1;
    return AH_OK;
}

int ah_sample_z_n(ah_ctx *h, uint64_t z_seed, uint32_t round, uint32_t sample, float *dst,
                  uint64_t ld)
{
    if (!h || !dst || ld < h->P || sample >= AH_MAX_SAMPLES) return AH_ERR_INVALID_ARG;
    if (!h->has_device) return AH_ERR_STATE;
    AH_CUDA(h, launch_sample_z(dst, ld, h->P, h->K, (uint32_t)(z_seed & 0xffffffffu),
                               (uint32_t)(z_seed >> 32), round, sample, h->stream));
    h->launches += 1;
    return AH_OK;
}

int ah_sample_z(ah_ctx *h, uint64_t z_seed, uint32_t round, float *dst, uint64_t ld)
{
    return ah_sample_z_n(h, z_seed, round, 0u, dst, ld);
}

namespace {

// What a fused round adds to a local step: who meets the master, with which
// coefficients, in which order.
struct FusedExchange {
    const uint8_t *mask;
    const float *weights;     // host, 2K floats, or null
    float alpha;
    const uint16_t *order;    // host, K entries, or null (ascending)
    bool asynchronous;
    bool lagged;              // coefficients come from the device (previous round's rule)
    bool before_step;         // the exchange precedes the local step (it belongs to the
                              // previous round); coefficients from the device if `dynamic`
    bool dynamic;             // run the rule on the pending distances first
};

int local_step_impl(ah_ctx *h, const float *grad, const float *hvp, uint64_t ld, uint64_t z_seed,
                    const ah_hyper *hy, const FusedExchange *fx)
{
    // ---- every check first: a refused call leaves the handle as it was
    if (!h || !grad || !hvp || !hy || ld < h->P) return AH_ERR_INVALID_ARG;
    if (!h->has_device) return AH_ERR_STATE;
    if (!(hy->beta1 >= 0.f && hy->beta1 < 1.f && hy->beta2 >= 0.f && hy->beta2 < 1.f))
        return AH_ERR_INVALID_ARG;
    if ((ld & 3u) != 0 || ((uintptr_t)grad & 15u) != 0 || ((uintptr_t)hvp & 15u) != 0)
        return AH_ERR_ALIGN;
    if (hy->want_dist < AH_DIST_NONE || hy->want_dist > AH_DIST_AND_RULE) return AH_ERR_INVALID_ARG;

    const int nsamp = hy->n_samples > 0 ? hy->n_samples : 1;
    if (nsamp > AH_MAX_SAMPLES) return AH_ERR_INVALID_ARG;
    if (nsamp > 1) {
        if (hy->hvp_sample_stride < (uint64_t)(h->K - 1) * ld + h->P) return AH_ERR_INVALID_ARG;
        if ((hy->hvp_sample_stride & 3u) != 0) return AH_ERR_ALIGN;
    }
    if (fx && fx->order) {                        // must name every worker exactly once
        bool seen[AH_MAX_WORKERS] = {};
        for (int q = 0; q < h->K; ++q) {
            if (fx->order[q] >= h->K || seen[fx->order[q]]) return AH_ERR_INVALID_ARG;
            seen[fx->order[q]] = true;
        }
    }
    const bool dist = hy->want_dist != AH_DIST_NONE;
    // the weighting rule owed on this round's distances: asked for by the caller, or
    // (lagged one-pass rounds) to serve the next exchange round
    const bool rule_here = hy->want_dist == AH_DIST_AND_RULE || (fx && fx->lagged && dist);
    const float rule_alpha = hy->want_dist == AH_DIST_AND_RULE ? hy->rule_alpha : (fx ? fx->alpha : 0.f);
    if (hy->want_dist == AH_DIST_AND_RULE && fx && !fx->lagged) return AH_ERR_INVALID_ARG;
    if (fx && fx->dynamic) {                      // this exchange's coefficients, on the device
        if (h->rule_fresh) {
            if (fx->alpha != h->rule_fresh_alpha) return AH_ERR_INVALID_ARG;
        } else if (!h->norm2_pending) {
            return AH_ERR_STATE;
        }
    }

    StepParams p;
    p.nsamp = (uint32_t)nsamp;
    p.sample_stride = nsamp > 1 ? hy->hvp_sample_stride : 0;
    p.x = h->x; p.m = h->m; p.v = h->v; p.c = h->c;
    p.grad = grad; p.hvp = hvp;
    p.status = reinterpret_cast<uint32_t *>(h->norm2_dev);
    p.sched = h->sched;
    p.runs = h->runs; p.tiles = h->tiles;
    p.lds = h->lds; p.ld = ld;
    p.P = h->P; p.ntiles = h->ntiles;
    p.key0 = (uint32_t)(z_seed & 0xffffffffu);
    p.key1 = (uint32_t)(z_seed >> 32);
    p.lr = hy->lr; p.beta1 = hy->beta1; p.beta2 = hy->beta2;
    p.omb1 = 1.0f - hy->beta1;
    p.omb2 = 1.0f - hy->beta2;
    p.eps = hy->eps; p.hpow = hy->hessian_power; p.wd = hy->weight_decay;
    p.fused = fx ? 1u : 0u;
    p.asynchronous = fx && fx->asynchronous ? 1u : 0u;
    p.pull_first = fx && fx->before_step ? 1u : 0u;
    p.any_exchange = 0u;
    p.nworkers = (uint32_t)h->K;
    p.c_out = h->c;
    // coefficients from the device: read from weights_dev unless this launch forms them
    // itself at its head (see below)
    p.wdev = fx && ((fx->lagged && h->lagged_ready) || fx->dynamic) ? h->weights_dev : nullptr;
    const uint32_t calls = h->calls + 1;
    p.round = hy->round == AH_ROUND_AUTO ? calls : hy->round;
    p.nrows = 0;
    uint32_t step[AH_MAX_WORKERS];                // step counts once this launch is enqueued
    for (int q = 0; q < h->K; ++q) {
        // a fused round walks the workers in their arrival order
        const int i = fx && fx->asynchronous && fx->order ? (int)fx->order[q] : q;
        const bool on = !hy->active || hy->active[i] != 0;
        const bool meets = fx && (!fx->mask || fx->mask[i] != 0);
        p.active[i] = on ? 1 : 0;
        p.exch[i] = meets ? 1 : 0;
        if (meets) p.any_exchange = 1u;
        p.h2w[i] = fx ? (fx->weights && !fx->lagged ? fx->weights[i] : fx->alpha) : 0.f;
        p.h1w[i] = fx ? (fx->weights && !fx->lagged ? fx->weights[h->K + i] : fx->alpha) : 0.f;
        step[i] = h->step[i] + (on ? 1u : 0u);
        // distances cover every worker: one that sits the step out travels through the
        // pipeline as an item of its own that fetches only x and the master tile
        if (on || meets || dist) p.row[p.nrows++] = (uint16_t)i;
        // bias corrections of Adam-type moments, 1 - beta^t with the worker's own t
        // (a worker that sat out steps has taken fewer); double, then one rounding
        const double t = (double)(step[i] ? step[i] : 1u);
        WorkerConst &w = p.w[i];
        w.bc1 = (float)(1.0 - pow((double)hy->beta1, t));
        w.bc2 = (float)(1.0 - pow((double)hy->beta2, t));
        w.rbc1 = 1.0f / w.bc1;
        w.rbc2 = 1.0f / w.bc2;
    }
    p.nitems = fx ? (p.nrows ? h->ntiles : 0u) : p.nrows * h->ntiles;
    // the branch-free exact square root and division of the kernels hold for eps in
    // [0, 2^40] and bias corrections of at least 2^-24 (beta <= 1 - 2^-24 gives that)
    p.narrow_ok = hy->eps >= 0.f && hy->eps <= 0x1p40f ? 1u : 0u;
    for (int i = 0; i < h->K; ++i)
        if (!(p.w[i].bc1 >= 0x1p-24f && p.w[i].bc2 >= 0x1p-24f)) p.narrow_ok = 0u;

    // ---- enqueue; the handle's bookkeeping follows each launch that went in
    // Tile sums of the last distance round may still wait to be assembled.  A fused exchange
    // that takes its coefficients from the device does that at the head of its own kernel
    // (and runs the rule there); every other reader gets a small kernel of its own.
    bool assemble_here = false, rule_at_head = false;
    float head_alpha = 0.f;
    if (fx && h->sums_raw && p.nitems > 0) {
        if (fx->dynamic) {
            assemble_here = rule_at_head = true;
            head_alpha = h->rule_fresh ? h->rule_fresh_alpha : fx->alpha;
        } else if (fx->lagged && h->raw_rule) {
            assemble_here = rule_at_head = true;
            head_alpha = h->raw_alpha;
        }
    }
    if (fx && fx->dynamic && !assemble_here) {
        if (h->sums_raw && !h->raw_rule) {        // the rule goes with the assembly
            h->raw_rule = true;
            h->raw_alpha = fx->alpha;
        }
        int rc = settle_distances(h);
        if (rc != AH_OK) return rc;
        if (!h->rule_fresh && h->norm2_pending && (rc = enqueue_weight_rule(h, fx->alpha)) != AH_OK)
            return rc;
    }
    p.tree = h->tree;
    if (assemble_here) {
        const int rc = begin_assembly(h, rule_at_head, head_alpha, p.tree);
        if (rc != AH_OK) return rc;
    }
    if (dist) {
        const int rc = begin_distance_store(h, p.tree);
        if (rc != AH_OK) return rc;
    }
    AH_CUDA(h, launch_local_step(p, dist, h->sm_count, h->stream));
    h->calls = calls;
    memcpy(h->step, step, (size_t)h->K * sizeof(uint32_t));
    if (p.nitems) h->launches += 1;
    if (assemble_here) {
        const int rc = commit_assembly(h, p.tree);
        if (rc != AH_OK) return rc;
    }
    if (fx && fx->dynamic) h->rule_fresh = false;     // the pending exchange has been made
    if (dist && p.nitems)
        commit_distance_store(h, rule_here, rule_alpha, hy->want_dist == AH_DIST_AND_RULE);
    return AH_OK;
}

}  // namespace

int ah_local_step(ah_ctx *h, const float *grad, const float *hvp, uint64_t ld, uint64_t z_seed,
                  const ah_hyper *hy)
{
    return local_step_impl(h, grad, hvp, ld, z_seed, hy, nullptr);
}

int ah_local_step_exchange(ah_ctx *h, const float *grad, const float *hvp, uint64_t ld,
                           uint64_t z_seed, const ah_hyper *hy, const uint8_t *worker_mask,
                           const float *weights, float alpha, const uint16_t *order,
                           int asynchronous, int lagged)
{
    if (!hy) return AH_ERR_INVALID_ARG;
    if (lagged && (hy->want_dist != AH_DIST || weights)) return AH_ERR_INVALID_ARG;
    FusedExchange fx;
    fx.mask = worker_mask; fx.weights = weights; fx.alpha = alpha; fx.order = order;
    fx.asynchronous = asynchronous != 0; fx.lagged = lagged != 0;
    fx.before_step = false; fx.dynamic = false;
    return local_step_impl(h, grad, hvp, ld, z_seed, hy, &fx);
}

int easgd_exchange_then_step(ah_ctx *h, const float *grad, const float *hvp, uint64_t ld,
                             uint64_t z_seed, const ah_hyper *hy, const uint8_t *worker_mask,
                             const float *weights, float alpha, const uint16_t *order,
                             int asynchronous, int dynamic)
{
    if (!hy) return AH_ERR_INVALID_ARG;
    if (hy->want_dist) return AH_ERR_INVALID_ARG;
    if (dynamic && weights) return AH_ERR_INVALID_ARG;
    FusedExchange fx;
    fx.mask = worker_mask; fx.weights = weights; fx.alpha = alpha; fx.order = order;
    fx.asynchronous = asynchronous != 0; fx.lagged = false;
    fx.before_step = true; fx.dynamic = dynamic != 0;
    return local_step_impl(h, grad, hvp, ld, z_seed, hy, &fx);
}

// ---- state in / out -----------------------------------------------------------
static int state_copy(ah_ctx *h, int which, int worker, void *user, int on_device, bool to_user)
{
    if (!h || !user) return AH_ERR_INVALID_ARG;
    const size_t row = (size_t)h->P * sizeof(float);
    if (which == AH_X || which == AH_M || which == AH_V || which == AH_CENTER) {
        if (!h->has_device) return AH_ERR_STATE;
        float *base = which == AH_X ? h->x : which == AH_M ? h->m : which == AH_V ? h->v : h->c;
        size_t rows = 1;
        if (which != AH_CENTER) {
            if (worker < -1 || worker >= h->K) return AH_ERR_INVALID_ARG;
            if (worker >= 0) base += (size_t)worker * h->lds;
            else rows = (size_t)h->K;
        }
        const size_t pitch = (size_t)h->lds * sizeof(float);
        cudaMemcpyKind kind;
        if (to_user) kind = on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost;
        else         kind = on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
        if (to_user) AH_CUDA(h, cudaMemcpy2DAsync(user, row, base, pitch, row, rows, kind, h->stream));
        else         AH_CUDA(h, cudaMemcpy2DAsync(base, pitch, user, row, row, rows, kind, h->stream));
        AH_CUDA(h, cudaStreamSynchronize(h->stream));
        return AH_OK;
    }
    if (on_device) return AH_ERR_INVALID_ARG;
    if (which == AH_WEIGHTS || which == AH_NORM2 || which == AH_UHIST || which == AH_ROUND) {
        // tile sums that still wait are assembled first (and the rule owed on them runs):
        // these selectors show, or replace, what that leaves behind
        const int rc = settle_distances(h);
        if (rc != AH_OK) return rc;
    }
    if (which == AH_WEIGHTS) {                 // coefficients of the last rule run on the device
        if (!h->has_device) return AH_ERR_STATE;
        if (to_user) {
            AH_CUDA(h, cudaMemcpyAsync(user, h->weights_dev, 2 * (size_t)h->K * sizeof(float),
                                       cudaMemcpyDeviceToHost, h->stream));
        } else {                               // restored from a checkpoint: a lagged round may use them
            AH_CUDA(h, cudaMemcpyAsync(h->weights_dev, user, 2 * (size_t)h->K * sizeof(float),
                                       cudaMemcpyHostToDevice, h->stream));
            h->lagged_ready = true;
            h->rule_fresh = false;
        }
        AH_CUDA(h, cudaStreamSynchronize(h->stream));
        return AH_OK;
    }
    if (which == AH_UHIST || which == AH_ROUND) {
        const int rc = ring_to_host(h);
        if (rc != AH_OK) return rc;
    }
    void *ptr;
    size_t bytes;
    uint32_t round_info[2];
    uint32_t info[4];
    if ((which == AH_INFO || which == AH_RUNS || which == AH_TILES) && !to_user)
        return AH_ERR_INVALID_ARG;
    switch (which) {
    case AH_INFO:
        info[0] = h->ntiles; info[1] = h->nruns; info[2] = (uint32_t)kTile; info[3] = (uint32_t)h->lds;
        ptr = info; bytes = sizeof(info);
        break;
    case AH_RUNS:  ptr = h->runs_host.data(); bytes = h->runs_host.size() * sizeof(Run); break;
    case AH_TILES: ptr = h->tiles_host.data(); bytes = h->tiles_host.size() * sizeof(TileInfo); break;
    case AH_NORM2:      ptr = h->norm2_last; bytes = h->K * sizeof(double); break;
    case AH_STEP:       ptr = h->step; bytes = h->K * sizeof(uint32_t); break;
    case AH_UHIST:      ptr = h->uhist.data(); bytes = h->uhist.size() * sizeof(double); break;
    case AH_DOWN_UNTIL: ptr = h->down_until; bytes = h->K * sizeof(uint32_t); break;
    case AH_ROUND:
        round_info[0] = h->calls;
        round_info[1] = (uint32_t)h->ring_filled;
        ptr = round_info; bytes = sizeof(round_info);
        break;
    default: return AH_ERR_INVALID_ARG;
    }
    if (to_user) {
        if (which == AH_NORM2 && h->norm2_unread) {
            AH_CUDA(h, cudaEventSynchronize(h->norm2_ready));
            memcpy(h->norm2_last, h->norm2_host + 1, h->K * sizeof(double));
            h->norm2_unread = false;
        }
        memcpy(user, ptr, bytes);
    } else {
        memcpy(ptr, user, bytes);
        if (which == AH_ROUND) {
            h->calls = round_info[0];
            h->ring_filled = (int)round_info[1];
        }
        if (which == AH_NORM2) {
            // restored distances: on a handle with a device they are pending again, for
            // either form of the weighting rule (host or device)
            h->norm2_unread = false;
            h->rule_fresh = false;
            h->norm2_pending = false;
            if (h->has_device) {
                AH_CUDA(h, cudaStreamSynchronize(h->stream));     // nobody is writing the pinned copy
                memcpy(h->norm2_host + 1, h->norm2_last, h->K * sizeof(double));
                memset(h->norm2_host, 0, sizeof(double));
                AH_CUDA(h, cudaMemcpyAsync(h->norm2_dev + 1, h->norm2_last, h->K * sizeof(double),
                                           cudaMemcpyHostToDevice, h->stream));
                AH_CUDA(h, cudaEventRecord(h->norm2_ready, h->stream));
                h->norm2_pending = true;
            }
        }
        if (which == AH_UHIST || which == AH_ROUND) h->ring_home = 0;    // the host copy leads again
    }
    return AH_OK;
}

int ah_state_set(ah_ctx *h, int which, int worker, const void *src, int src_on_device)
{
    return state_copy(h, which, worker, const_cast<void *>(src), src_on_device, false);
}

int ah_state_get(ah_ctx *h, int which, int worker, void *dst, int dst_on_device)
{
    if (h && h->has_device) {
        // the device status word is looked at whenever the host waits for the stream anyway
        uint32_t status = 0;
        AH_CUDA(h, cudaMemcpyAsync(&status, h->norm2_dev, sizeof(status), cudaMemcpyDeviceToHost,
                                   h->stream));
        AH_CUDA(h, cudaStreamSynchronize(h->stream));
        if (status != 0u) {
            h->tree_dirty = true;      // a kernel gave up half way: the next distance round starts clean
            return AH_ERR_INTERNAL;
        }
    }
    return state_copy(h, which, worker, dst, dst_on_device, true);
}

// ---- dynamic weights (Sec. V-B) ------------------------------------------------
int dw_config(ah_ctx *h, int p_hist, const double *c, double kappa)
{
    if (!h || !c || p_hist < 1 || p_hist > AH_MAX_HIST || !(kappa < 0.0)) return AH_ERR_INVALID_ARG;
    const int rc = settle_distances(h);        // a rule that is still owed runs with the old setting
    if (rc != AH_OK) return rc;
    h->p_hist = p_hist;
    for (int j = 0; j < p_hist; ++j) h->coef[j] = c[j];
    h->kappa = kappa;
    reset_history(h);
    h->ring_home = 0;
    return AH_OK;
}

int dw_weights_next(ah_ctx *h, float alpha, float *weights)
{
    if (!h || !weights) return AH_ERR_INVALID_ARG;
    if (!h->has_device) return AH_ERR_STATE;
    const int rc = settle_distances(h);
    if (rc != AH_OK) return rc;
    if (!h->norm2_pending) return AH_ERR_STATE;
    AH_CUDA(h, cudaEventSynchronize(h->norm2_ready));
    h->norm2_pending = false;
    h->norm2_unread = false;
    if (*reinterpret_cast<const uint32_t *>(h->norm2_host) != 0u) return AH_ERR_INTERNAL;
    return dw_weights_from_norm2(h, h->norm2_host + 1, alpha, weights);
}

int dw_weights_from_norm2(ah_ctx *h, const double *norm2, float alpha, float *weights)
{
    if (!h || !norm2 || !weights) return AH_ERR_INVALID_ARG;
    const int rc = ring_to_host(h);
    if (rc != AH_OK) return rc;
    memcpy(h->norm2_last, norm2, h->K * sizeof(double));

    const int depth = h->p_hist + 1;
    for (int i = 0; i < h->K; ++i) {
        double *ring = &h->uhist[(size_t)i * depth];
        weight_rule_step(h->p_hist, h->coef, h->kappa, (double)alpha, h->norm2_last[i], ring, ring,
                         h->ring_filled != 0, &weights[i], &weights[h->K + i]);
    }
    h->ring_filled = 1;
    return AH_OK;
}

// ---- failure / straggler mask (Sec. VI) -----------------------------------------
int dw_mask_next(ah_ctx *h, uint64_t seed, uint32_t round, double p_fail, int max_stale,
                 uint8_t *mask)
{
    if (!h || !mask || max_stale < 1 || !(p_fail >= 0.0)) return AH_ERR_INVALID_ARG;
    const uint32_t k0 = (uint32_t)(seed & 0xffffffffu), k1 = (uint32_t)(seed >> 32);
    const bool always = p_fail >= 1.0;
    const uint32_t threshold = always ? 0u : (uint32_t)floor(p_fail * 4294967296.0);
    for (int i = 0; i < h->K; ++i) {
        bool up = round >= h->down_until[i];
        if (up) {
            uint32_t draw[4];
            philox4x32_10(0u, (uint32_t)i, round, kDomainFail, k0, k1, draw);
            if (always || draw[0] < threshold) {
                uint32_t length = 1;
                if (max_stale > 1) {
                    uint32_t d2[4];
                    philox4x32_10(0u, (uint32_t)i, round, kDomainStale, k0, k1, d2);
                    length += d2[0] % (uint32_t)max_stale;
                }
                h->down_until[i] = round + length;
                up = false;
            }
        }
        mask[i] = up ? 1 : 0;
    }
    return AH_OK;
}

// ---- elastic exchange (Eqs. 12-13) -----------------------------------------------
int easgd_exchange(ah_ctx *h, const uint8_t *worker_mask, const float *weights, float alpha)
{
    if (!h) return AH_ERR_INVALID_ARG;
    if (!h->has_device) return AH_ERR_STATE;
    ExchangeParams p;
    const int rc = fill_exchange(h, worker_mask, weights, alpha, nullptr, nullptr, p);
    if (rc != AH_OK) return rc;
    if (p.nact == 0) return AH_OK;     // nobody reaches the master: nothing moves
    AH_CUDA(h, launch_exchange(p, h->stream));
    h->launches += 1;
    return AH_OK;
}

// ---- diagnostics ------------------------------------------------------------------
const char *ah_status_string(int status)
{
    switch (status) {
    case AH_OK: return "ok";
    case AH_ERR_INVALID_ARG: return "invalid argument";
    case AH_ERR_ALIGN: return "pointer or stride not aligned";
    case AH_ERR_SEGMENTS: return "bad segment table";
    case AH_ERR_ALLOC: return "allocation failed or workspace too small";
    case AH_ERR_CUDA: return "CUDA runtime error";
    case AH_ERR_STATE: return "call out of order";
    case AH_ERR_INTERNAL: return "internal device error";
    case AH_ERR_TOO_LARGE: return "problem exceeds the built-in scratch capacity";
    default: return "unknown status";
    }
}

int ah_set_wait_polls(ah_ctx *h, uint32_t polls)
{
    if (!h) return AH_ERR_INVALID_ARG;
    h->wait_polls = polls;
    return AH_OK;
}

int ah_last_cuda_error(const ah_ctx *h) { return h ? h->last_cuda : 0; }

uint64_t ah_launch_count(const ah_ctx *h) { return h ? h->launches : 0; }

}  // extern "C"
