// The fused local step of the AdaHessian + elastic-averaging round (sm_100a): kernel
// template and its launcher.  Included by the translation units that instantiate it
// (ah_step_inst.cu, once per combination of Hessian power and weight decay, so that they
// compile side by side).
//
// Everything here is HBM-bound streaming work: the fused local step reads
// grad, hvp, x, m, v and writes x, m, v once (32 bytes per parameter update), the
// exchange reads and writes x once more (8 bytes per update) plus the master row.
// There is no dense contraction, so no tensor cores; the rules that matter are
// wide coalesced accesses, enough bytes in flight, and not touching a byte twice.
//
// Arithmetic follows one fixed order with one binary32 rounding per operation
// (__fmul_rn / __fadd_rn / __fdiv_rn / __fsqrt_rn are never contracted into FMAs),
// so results do not depend on compiler flags or launch shape.
#pragma once

#include <atomic>

#include "ah_internal.h"
#include "ah_device.cuh"
#include "ah_tree.cuh"

namespace ah {

// ---------------------------------------------------------------------------
// Small PTX wrappers: mbarriers, 1-D bulk copies (TMA), named barriers.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t arrivals)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(arrivals)
                 : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)),
                 "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return done != 0;
}

// Bounded wait: polls the barrier at most kWaitPolls times (backing off after the
// first few), then records `code` in the status word and gives up.  A healthy run
// never comes near the limit (about a second).
constexpr uint32_t kWaitPolls = 1u << 22;

__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, uint32_t *status,
                                          uint32_t code)
{
    for (uint32_t it = 0; it < kWaitPolls; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it > 32) __nanosleep(128);
    }
    atomicOr(status, code);
    return false;
}

// Global -> shared bulk copy of `bytes` (a multiple of 16; both addresses 16-byte
// aligned), completion counted on `bar`.
__device__ __forceinline__ void bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar))
        : "memory");
}

// Orders this thread's earlier generic-proxy accesses to shared memory before later
// async-proxy (bulk copy) writes to the same locations.
__device__ __forceinline__ void fence_generic_to_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void consumer_sync()
{
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory");
}

// ---------------------------------------------------------------------------
// Arithmetic helpers
// ---------------------------------------------------------------------------

// x / b for a divisor b whose correctly rounded reciprocal r is known: one
// multiply, the exact remainder by FMA, one correction (Markstein's sequence).  The
// result is the correctly rounded quotient whenever no intermediate leaves the
// normal range, which holds for 2^-24 < b <= 128 when 2^-63 <= |x| < 2^64 (checked
// exhaustively on the host for every significand of x, for the integer divisors
// 2..128 and for divisors of the form 1 - beta^t).  Callers test the window.
__device__ __forceinline__ float div_by_const_in_window(float x, float b, float r)
{
    const float q = __fmul_rn(x, r);
    const float rem = __fmaf_rn(-b, q, x);
    return __fmaf_rn(rem, r, q);
}

__device__ __forceinline__ bool in_window(float lo_abs, float hi_abs)
{
    return lo_abs >= 0x1p-63f && hi_abs < 0x1p64f;
}

__device__ __forceinline__ float div_by_const(float x, float b, float r)
{
    const float a = fabsf(x);
    return in_window(a, a) ? div_by_const_in_window(x, b, r) : __fdiv_rn(x, b);
}

__device__ __forceinline__ float min_abs4(float4 a)
{
    return fminf(fminf(fabsf(a.x), fabsf(a.y)), fminf(fabsf(a.z), fabsf(a.w)));
}

__device__ __forceinline__ float max_abs4(float4 a)
{
    return fmaxf(fmaxf(fabsf(a.x), fabsf(a.y)), fmaxf(fabsf(a.z), fabsf(a.w)));
}

// Per-element AdaHessian update (Sec. IV-B of the paper; Eq. 4 with the diagonal
// preconditioner 1 / ((sqrt vhat)^k + eps)), split in two so that four elements can
// share one test of the division window.  D is the spatially averaged Hutchinson
// estimate of the Hessian diagonal for this element.
// POWMODE: 0 -> k = 1, 1 -> k = 1/2, 2 -> general k via powf.
__device__ __forceinline__ void moments(float &m, float &v, float g, float D, const StepCommon &p)
{
    m = __fadd_rn(__fmul_rn(p.beta1, m), __fmul_rn(p.omb1, g));
    v = __fadd_rn(__fmul_rn(p.beta2, v), __fmul_rn(__fmul_rn(p.omb2, D), D));
}

template <int POWMODE, bool WD, bool WINDOW>
__device__ __forceinline__ float step_from_moments(float x, float m1, float v1, const StepCommon &p,
                                                   const WorkerConst &w)
{
    // Inside the window (and with eps in [0, 2^40], which the host checks once per launch):
    // |mhat| in [2^-63, 2^88), vhat in [2^-63, 2^88), sqrt vhat in [2^-32, 2^44], the
    // denominator in [2^-32, 2^45): the ranges of the branch-free exact routines.
    const float mhat = WINDOW ? div_by_const_in_window(m1, w.bc1, w.rbc1) : __fdiv_rn(m1, w.bc1);
    const float vhat = WINDOW ? div_by_const_in_window(v1, w.bc2, w.rbc2) : __fdiv_rn(v1, w.bc2);
    const float r = WINDOW ? sqrt_in_range(vhat) : __fsqrt_rn(vhat);
    float pw;
    if (POWMODE == 0) pw = r;
    else if (POWMODE == 1) pw = WINDOW ? sqrt_in_range(r) : __fsqrt_rn(r);
    else pw = powf(r, p.hpow);
    const float den = __fadd_rn(pw, p.eps);
    const float q = WINDOW && POWMODE != 2 ? div_in_range(mhat, den) : __fdiv_rn(mhat, den);
    if (WD) return __fsub_rn(x, __fmul_rn(p.lr, __fadd_rn(q, __fmul_rn(p.wd, x))));
    return __fsub_rn(x, __fmul_rn(p.lr, q));
}

template <int POWMODE, bool WD>
__device__ __forceinline__ void adahessian_update(float &x, float &m, float &v, float g, float D,
                                                  const StepCommon &p, const WorkerConst &w)
{
    moments(m, v, g, D, p);
    const float lo = fminf(fabsf(m), fabsf(v)), hi = fmaxf(fabsf(m), fabsf(v));
    x = in_window(lo, hi) && p.narrow_ok ? step_from_moments<POWMODE, WD, true>(x, m, v, p, w)
                                         : step_from_moments<POWMODE, WD, false>(x, m, v, p, w);
}

// Four consecutive elements at once: one window test for the eight divisions.
template <int POWMODE, bool WD>
__device__ __forceinline__ void adahessian_update4(float4 &x, float4 &m, float4 &v, const float4 g,
                                                   const float4 D, const StepCommon &p,
                                                   const WorkerConst &w)
{
    moments(m.x, v.x, g.x, D.x, p);
    moments(m.y, v.y, g.y, D.y, p);
    moments(m.z, v.z, g.z, D.z, p);
    moments(m.w, v.w, g.w, D.w, p);
    const float lo = fminf(min_abs4(m), min_abs4(v)), hi = fmaxf(max_abs4(m), max_abs4(v));
    if (in_window(lo, hi) && p.narrow_ok) {
        x.x = step_from_moments<POWMODE, WD, true>(x.x, m.x, v.x, p, w);
        x.y = step_from_moments<POWMODE, WD, true>(x.y, m.y, v.y, p, w);
        x.z = step_from_moments<POWMODE, WD, true>(x.z, m.z, v.z, p, w);
        x.w = step_from_moments<POWMODE, WD, true>(x.w, m.w, v.w, p, w);
    } else {
        x.x = step_from_moments<POWMODE, WD, false>(x.x, m.x, v.x, p, w);
        x.y = step_from_moments<POWMODE, WD, false>(x.y, m.y, v.y, p, w);
        x.z = step_from_moments<POWMODE, WD, false>(x.z, m.z, v.z, p, w);
        x.w = step_from_moments<POWMODE, WD, false>(x.w, m.w, v.w, p, w);
    }
}

// a with its sign flipped when bit K of bits is set.
template <int K>
__device__ __forceinline__ float flip_if_bit(float a, uint32_t bits)
{
    return __uint_as_float(__float_as_uint(a) ^ ((bits << (31 - K)) & 0x80000000u));
}

// z (.) h for four consecutive elements; bit k of nib set means z = -1 for lane k.
__device__ __forceinline__ float4 apply_signs(float4 h, uint32_t nib)
{
    h.x = flip_if_bit<0>(h.x, nib);
    h.y = flip_if_bit<1>(h.y, nib);
    h.z = flip_if_bit<2>(h.z, nib);
    h.w = flip_if_bit<3>(h.w, nib);
    return h;
}

// ---------------------------------------------------------------------------
// Fused local step: persistent, warp-specialised, TMA-fed.
//
// An item is one tile of kTile consecutive parameters of one worker.  The grid is
// persistent (one wave of CTAs); each producer draws the next item from a counter in
// global memory whenever one of its stages falls free, so that the tiles in flight
// across the GPU stay one compact, advancing window of the arrays (a fixed
// item-to-CTA assignment lets the CTAs drift apart and was measured 7-20% slower).
//
// Producer warp, per item: waits until the stage is free, computes the Philox
// blocks whose bits are the Rademacher signs of the tile (one lane per group of 128
// parameters), writes the item's header (everything the consumers would otherwise
// work out per thread: which worker, its bias corrections, its exchange coefficients,
// the tile's extent), and issues bulk copies of grad, x, m, v, (c) and of the
// Hessian-vector values of the tile widened to whole spatial blocks.  z costs no
// memory traffic.
//
// Consumers, per item: wait for the stage and agree through one reducing barrier that
// it has arrived (so that they all go on or all leave); where the tile touches a tensor
// with spatial block > 1 they turn hvp into z (.) hvp in place, average each block in
// place (one thread per block, ascending-order sum, one division) and read the means
// back; otherwise the sign is applied in registers.  Tiles whose averaged tensors are
// all 3 x 3 kernels (the common case) skip the separate sign pass: the thread that sums
// a block takes the nine signs from the Philox words as it goes.  Then moments and
// update per element, 128-bit stores of x, m, v, and the stage goes back to the producer.
//
// DIST additionally forms, per item, the pairwise-tree sum of (x_new - c)^2: the
// consumer warps leave their eight partial sums in the stage, and the producer, when it
// takes the stage back, adds them up and stores the tile's sum (level 0 of the distance
// tree of ah_tree.cuh).  A worker that sits the step out contributes its unchanged x
// (only x and c are fetched for it).
//
// A fused exchange whose coefficients come from the weighting rule assembles the
// distances of the preceding distance round from those tile sums at its head and runs
// the rule there (the consumer warps of every CTA, while the producer already fetches the
// first tiles): no launch, no copy and no host round trip lies between measuring the
// distances and using the coefficients.
//
// The kernel may be launched with programmatic stream serialisation: everything before
// griddepcontrol.wait touches only this CTA's shared memory and the launch parameters;
// the first draw from the item counter and every access to state, inputs and workspace
// come after it.
// ---------------------------------------------------------------------------
enum : uint32_t {
    kItemAverage = 1u,        // the tile touches a spatial block > 1
    kItemDistanceOnly = 2u,   // the worker sits the step out: only x (and c) were fetched
    kItemEnd = 4u,            // no item: the producer has left
    kItemFirst = 8u,          // fused exchange: first worker of a tile (c was fetched with it)
    kItemLast = 16u,          // fused exchange: last worker of a tile (the master is written back)
    kItemExchange = 32u,      // fused exchange: this worker meets the master
    kItemAll3x3 = 64u,        // every averaged tensor the tile touches has block 9
};

constexpr int kRed = kPasses * kConsumerWarps;     // per-warp, per-pass sums of a tile
static_assert((kRed & (kRed - 1)) == 0 && kRed <= 32, "the tile's sums form a subtree");

// What the producer tells the consumers about an item: four 16-byte words.
struct __align__(16) ItemHeader {
    uint32_t worker, t0, nvalid, flags;
    uint32_t e0, e1, run0, ea0;
    float bc1, bc2, rbc1, rbc2;            // the worker's bias corrections and reciprocals
    uint32_t tile, reserved[3];
};

template <bool HASC>
struct __align__(128) Stage {
    ItemHeader hdr;
    double red[kRed];                      // DIST: sums of (x - c)^2, one per warp and pass
    uint32_t zw[kStageGroups][4];          // Philox words of groups (ea0 >> 7) ...
    float g[kTile], x[kTile], m[kTile], v[kTile];
    float c[HASC ? kTile : 4];
    float hv[kTile + 2 * kHalo];           // element j lives at hv[j - t0 + kHalo]
};

// With n > 1 Hutchinson samples per step, samples 1 .. n-1 of every stage live behind
// the fixed part of shared memory: their Philox words and their Hessian-vector tile.
struct __align__(128) ExtraSample {
    uint32_t zw[kStageGroups][4];
    float hv[kTile + 2 * kHalo];
};

template <bool HASC, bool FUSE, int MAXW>
struct __align__(128) Shared {
    Stage<HASC> stage[kStages];
    uint64_t full[kStages];                // producer -> consumers (bytes landed)
    uint64_t empty[kStages];               // consumers -> producer (stage drained)
    float h1[FUSE ? MAXW : 1];             // fused exchange: coefficients by worker index
    float h2[FUSE ? MAXW : 1];
    uint32_t words[2];                     // fused exchange: scratch of the distance assembly
};

// All consumers learn whether every one of them saw the stage arrive.
__device__ __forceinline__ bool consumers_agree(bool mine)
{
    uint32_t all;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "barrier.cta.red.and.pred q, 1, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(all)
        : "r"((uint32_t)mine), "n"(kConsumers)
        : "memory");
    return all != 0u;
}

__device__ __forceinline__ uint4 ld_shared_u4(const void *p)
{
    return *reinterpret_cast<const uint4 *>(p);
}

template <int B>
__device__ __forceinline__ void block_means_fixed(float *base, uint32_t nblk, int ctid)
{
    const float fb = (float)B, rb = __frcp_rn(fb);
    for (uint32_t k = ctid; k < nblk; k += kConsumers) {
        float *blk = base + k * B;
        float S = blk[0];
#pragma unroll
        for (int e = 1; e < B; ++e) S = __fadd_rn(S, blk[e]);
        const float mean = div_by_const(S, fb, rb);
#pragma unroll
        for (int e = 0; e < B; ++e) blk[e] = mean;
    }
}

// Block means of 3x3 kernels straight from the raw Hessian-vector values: the signs
// of the nine elements are taken from the Philox words on the fly.
template <bool HASC>
__device__ __forceinline__ void block_means_signed9(Stage<HASC> &st, uint32_t qa, uint32_t nblk,
                                                    uint32_t t0, uint32_t g0, int ctid)
{
    const float rb = __frcp_rn(9.0f);
    for (uint32_t k = ctid; k < nblk; k += kConsumers) {
        const uint32_t j0 = qa + 9u * k;
        float *blk = &st.hv[j0 + kHalo - t0];
        const uint32_t w0 = j0 >> 5, w1 = (j0 + 8u) >> 5;       // words holding the first and last sign
        const uint32_t lo = st.zw[(w0 >> 2) - g0][w0 & 3u];
        const uint32_t hi = st.zw[(w1 >> 2) - g0][w1 & 3u];     // == lo when the block sits in one word
        const uint32_t bits = __funnelshift_r(lo, hi, j0 & 31u);
        float S = flip_if_bit<0>(blk[0], bits);
        S = __fadd_rn(S, flip_if_bit<1>(blk[1], bits));
        S = __fadd_rn(S, flip_if_bit<2>(blk[2], bits));
        S = __fadd_rn(S, flip_if_bit<3>(blk[3], bits));
        S = __fadd_rn(S, flip_if_bit<4>(blk[4], bits));
        S = __fadd_rn(S, flip_if_bit<5>(blk[5], bits));
        S = __fadd_rn(S, flip_if_bit<6>(blk[6], bits));
        S = __fadd_rn(S, flip_if_bit<7>(blk[7], bits));
        S = __fadd_rn(S, flip_if_bit<8>(blk[8], bits));
        const float mean = div_by_const(S, 9.0f, rb);
#pragma unroll
        for (int e = 0; e < 9; ++e) blk[e] = mean;
    }
}

__device__ __forceinline__ void block_means_any(float *base, uint32_t nblk, uint32_t B, int ctid)
{
    const float fb = (float)B, rb = __frcp_rn(fb);
    for (uint32_t k = ctid; k < nblk; k += kConsumers) {
        float *blk = base + k * B;
        float S = blk[0];
        for (uint32_t e = 1; e < B; ++e) S = __fadd_rn(S, blk[e]);
        const float mean = div_by_const(S, fb, rb);
        for (uint32_t e = 0; e < B; ++e) blk[e] = mean;
    }
}

// One worker meets the master on four consecutive columns (Eqs. 12-13), in the operation
// order of the separate exchange kernels.  Simultaneous form: every worker sees the old
// master value c_old and `carry` gathers what the workers add to it, from +0.
// Asynchronous form: `carry` is the master as the arrivals so far left it.
__device__ __forceinline__ void meet_master4(float4 &x, float4 &carry, const float4 &c_old, float h1,
                                             float h2, bool asynchronous)
{
    float *xe = &x.x, *ae = &carry.x;
    const float *ce = &c_old.x;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        if (asynchronous) {
            const float d = __fsub_rn(xe[e], ae[e]);
            xe[e] = __fsub_rn(xe[e], __fmul_rn(h1, d));
            ae[e] = __fadd_rn(ae[e], __fmul_rn(h2, d));
        } else {
            const float d = __fsub_rn(xe[e], ce[e]);
            ae[e] = __fadd_rn(ae[e], __fmul_rn(h2, d));
            xe[e] = __fsub_rn(xe[e], __fmul_rn(h1, d));
        }
    }
}

// Hutchinson estimate of four consecutive elements (Sec. IV-B): z (.) hvp for one
// sample; with MULTI the sum over the samples in ascending order, divided by their
// number.  hidx indexes the stage's hvp arrays, gidx its Philox groups, j is the
// element's index in the row (it selects the word and the bit of the signs).
template <bool MULTI, bool HASC>
__device__ __forceinline__ float4 hutchinson4(const Stage<HASC> &st, const ExtraSample *xs,
                                              uint32_t nsamp, uint32_t hidx, uint32_t gidx,
                                              uint32_t j, float fn, float rn)
{
    const uint32_t wsel = (j >> 5) & 3u, shift = j & 31u;
    float4 D = apply_signs(ld_vec(&st.hv[hidx]), (st.zw[gidx][wsel] >> shift) & 0xFu);
    if constexpr (MULTI) {
        for (uint32_t q = 0; q + 1u < nsamp; ++q) {
            const float4 e = apply_signs(ld_vec(&xs[q].hv[hidx]), (xs[q].zw[gidx][wsel] >> shift) & 0xFu);
            D.x = __fadd_rn(D.x, e.x); D.y = __fadd_rn(D.y, e.y);
            D.z = __fadd_rn(D.z, e.z); D.w = __fadd_rn(D.w, e.w);
        }
        D.x = div_by_const(D.x, fn, rn); D.y = div_by_const(D.y, fn, rn);
        D.z = div_by_const(D.z, fn, rn); D.w = div_by_const(D.w, fn, rn);
    }
    return D;
}

// By the producer warp, on a stage the consumers have handed back: the tile's sum of
// (x - c)^2 from the per-warp, per-pass sums (top levels of the adjacent-pairs tree).
template <bool HASC>
__device__ __forceinline__ double stage_sum(const Stage<HASC> &st, int lane)
{
    double v = st.red[lane & (kRed - 1)];          // every group of kRed lanes forms the same sum
#pragma unroll
    for (int off = 1; off < kRed; off <<= 1)
        v = __dadd_rn(v, __shfl_xor_sync(0xffffffffu, v, off));
    return v;
}

// CTAs per SM an instantiation is built (register bound) and launched for.
constexpr int ctas_per_sm(bool dist, bool multi, bool fuse)
{
    (void)dist;                 // a distance round's stages are those of a plain round
    return multi || fuse ? kCtasPerSm : kCtasPerSmPlain;
}

template <int POWMODE, bool WD, bool DIST, bool MULTI, bool FUSE, int MAXW>
__global__ void __launch_bounds__(kThreads, ctas_per_sm(DIST, MULTI, FUSE))
local_step_kernel(const __grid_constant__ StepParamsT<MAXW> p)
{
    constexpr bool HASC = FUSE;                    // the stages carry a tile of the master row
    extern __shared__ __align__(128) unsigned char smem_raw[];
    using SharedT = Shared<HASC, FUSE, MAXW>;
    SharedT &sh = *reinterpret_cast<SharedT *>(smem_raw);
    ExtraSample *extra = reinterpret_cast<ExtraSample *>(smem_raw + sizeof(SharedT));
    const uint32_t nextra = MULTI ? p.nsamp - 1u : 0u;     // extra samples per stage

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&sh.full[s], 1);
            mbar_init(&sh.empty[s], kConsumerWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // a launch that was allowed to start early waits here for the launches before it
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp == kConsumerWarps) {
        // =============================== producer ===============================
        // Items are drawn from the global counter one ahead of their use, so that the
        // round trip of the atomic overlaps the wait for a free stage.
        uint32_t drawn = 0;
        if (lane == 0) drawn = atomicAdd(&p.sched[0], 1u);
        if constexpr (FUSE) {
            // a launch that assembles distances at its head: the bulk copies start when the
            // consumers have the tree's few small loads behind them (these would otherwise
            // queue behind megabytes of tiles), and land while the rule is computed
            if (p.tree.assemble) asm volatile("bar.sync 2, %0;" ::"n"(kThreads) : "memory");
        }
        uint32_t k = 0;
        uint32_t tile = 0, r = 0, rows_left = 0;   // FUSE: where the producer is in a tile's worker list
        bool healthy = true;
        for (;; ++k) {
            const uint32_t s = k % kStages, use = k / kStages;
            Stage<HASC> &st = sh.stage[s];
            if (use > 0) {
                if (!mbar_wait(&sh.empty[s], (use - 1u) & 1u, p.status, kStatusEmptyTimeout)) {
                    healthy = false;
                    break;
                }
                if constexpr (DIST) {              // the item that just left this stage
                    const double sum = stage_sum(st, lane);
                    if (lane == 0) tree_store_tile(p.tree, st.hdr.worker, st.hdr.tile, sum);
                }
            }
            if (!FUSE || rows_left == 0u) {
                const uint32_t n = __shfl_sync(0xffffffffu, drawn, 0);
                if (n >= p.nitems) {         // nothing left: tell the consumers and leave
                    if (lane == 0) {
                        st.hdr.flags = kItemEnd;
                        mbar_arrive(&sh.full[s]);
                    }
                    break;
                }
                if (lane == 0) drawn = atomicAdd(&p.sched[0], 1u);
                if constexpr (FUSE) {
                    // an item is a tile with all its workers, taken in their arrival order
                    tile = n; r = 0; rows_left = p.nrows;
                } else {
                    // Plain rounds walk one worker's row after the other; distance rounds
                    // walk the workers innermost, so that a tile of the master row is fetched
                    // from HBM once and served from L2 to the other workers.
                    tile = DIST ? n / p.nrows : n % p.ntiles;
                    r = DIST ? n - tile * p.nrows : n / p.ntiles;
                }
            }
            const uint32_t i = p.row[r];
            const bool act = p.active[i] != 0;
            const uint32_t t0 = tile * (uint32_t)kTile;
            const uint32_t nvalid = min((uint32_t)kTile, p.P - t0);
            const uint32_t n4 = (nvalid + 3u) & ~3u;
            const TileInfo ti = p.tiles[tile];
            const bool avg = act && (ti.flags & 1u);
            const uint32_t ea0 = avg ? (ti.e0 & ~3u) : t0;
            const uint32_t ea1 = avg ? ((ti.e1 + 3u) & ~3u) : t0 + n4;
            if (act) {
                const uint32_t g0 = ea0 >> 7;
                const uint32_t ng = ((ea1 - 1u) >> 7) - g0 + 1u;
                if ((uint32_t)lane < ng) {
                    philox4x32_10(g0 + lane, i, p.round, kDomainZ, p.key0, p.key1, st.zw[lane]);
                    if constexpr (MULTI)
                        for (uint32_t q = 0; q < nextra; ++q)
                            philox4x32_10(g0 + lane, i, p.round, kDomainZ + 256u * (q + 1u), p.key0,
                                          p.key1, extra[s * nextra + q].zw[lane]);
                }
            }
            const bool first = FUSE && r == 0u, last = FUSE && rows_left == 1u;
            if (lane == 0) {
                ItemHeader hd;
                hd.worker = i; hd.t0 = t0; hd.nvalid = nvalid;
                hd.flags = (avg ? kItemAverage : 0u) | (act ? 0u : kItemDistanceOnly) |
                           ((ti.flags & 2u) ? kItemAll3x3 : 0u) |
                           (first ? kItemFirst : 0u) | (last ? kItemLast : 0u) |
                           (FUSE && p.exch[i] ? kItemExchange : 0u);
                hd.e0 = ti.e0; hd.e1 = ti.e1; hd.run0 = ti.run0; hd.ea0 = ea0;
                const WorkerConst wc = p.w[i];
                hd.bc1 = wc.bc1; hd.bc2 = wc.bc2; hd.rbc1 = wc.rbc1; hd.rbc2 = wc.rbc2;
                hd.tile = tile;
                hd.reserved[0] = hd.reserved[1] = hd.reserved[2] = 0u;
                st.hdr = hd;
            }
            __syncwarp();
            if (lane == 0) {
                const uint32_t row_bytes = n4 * 4u, hv_bytes = (ea1 - ea0) * 4u;
                const uint64_t so = (uint64_t)i * p.lds + t0;
                uint64_t *bar = &sh.full[s];
                const bool want_c = FUSE && first;            // fused: the master tile, once per tile
                if (act) {
                    mbar_arrive_expect_tx(bar, 4u * row_bytes + (1u + nextra) * hv_bytes +
                                                   (want_c ? row_bytes : 0u));
                    bulk_load(&st.hv[ea0 + kHalo - t0], p.hvp + (uint64_t)i * p.ld + ea0, hv_bytes, bar);
                    if constexpr (MULTI)
                        for (uint32_t q = 0; q < nextra; ++q)
                            bulk_load(&extra[s * nextra + q].hv[ea0 + kHalo - t0],
                                      p.hvp + (uint64_t)(q + 1u) * p.sample_stride +
                                          (uint64_t)i * p.ld + ea0,
                                      hv_bytes, bar);
                    bulk_load(st.g, p.grad + (uint64_t)i * p.ld + t0, row_bytes, bar);
                    bulk_load(st.x, p.x + so, row_bytes, bar);
                    bulk_load(st.m, p.m + so, row_bytes, bar);
                    bulk_load(st.v, p.v + so, row_bytes, bar);
                    if constexpr (HASC) if (want_c) bulk_load(st.c, p.c + t0, row_bytes, bar);
                } else if constexpr (DIST || FUSE) {
                    mbar_arrive_expect_tx(bar, (want_c ? 2u : 1u) * row_bytes);
                    bulk_load(st.x, p.x + so, row_bytes, bar);
                    if constexpr (HASC) if (want_c) bulk_load(st.c, p.c + t0, row_bytes, bar);
                }
            }
            if constexpr (FUSE) { ++r; --rows_left; }
        }
        // this CTA draws no more items: a launch waiting behind this one may move in as the
        // CTAs leave (it still waits for this whole launch before it touches memory)
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        if constexpr (DIST) {
            // the items still with the consumers, in the order in which they finish
            for (uint32_t j = k + 1u; healthy && j < k + (uint32_t)kStages; ++j) {
                const uint32_t s = j % kStages, use = j / kStages;
                if (use == 0u) continue;
                if (!mbar_wait(&sh.empty[s], (use - 1u) & 1u, p.status, kStatusEmptyTimeout)) break;
                const Stage<HASC> &st = sh.stage[s];
                const double sum = stage_sum(st, lane);
                if (lane == 0) tree_store_tile(p.tree, st.hdr.worker, st.hdr.tile, sum);
            }
        }
        // the last producer to leave puts both scheduler words back to zero for the next
        // launch (every producer has made its final fetch before it counts itself out)
        if (lane == 0) {
            __threadfence();
            if (atomicAdd(&p.sched[1], 1u) == gridDim.x - 1u) {
                p.sched[0] = 0u;
                p.sched[1] = 0u;
            }
        }
        return;
    }

    // ================================= consumers =================================
    const int ctid = threadIdx.x;
    if constexpr (FUSE) {
        // exchange coefficients by worker index: from the weighting rule, run here on the
        // distances this launch assembles first, or from device memory, or from the launch
        const bool rule_here = p.tree.assemble != 0u && p.tree.run_rule != 0u;
        if (p.tree.assemble)
            assemble_distances(p.tree, ctid, kConsumers, blockIdx.x, gridDim.x,
                               rule_here ? sh.h1 : nullptr, sh.h2, sh.words, [] { consumer_sync(); },
                               [] { asm volatile("bar.arrive 2, %0;" ::"n"(kThreads) : "memory"); });
        if (!rule_here)
            for (uint32_t w = (uint32_t)ctid; w < p.nworkers; w += (uint32_t)kConsumers) {
                sh.h1[w] = p.wdev ? p.wdev[p.nworkers + w] : p.h1w[w];
                sh.h2[w] = p.wdev ? p.wdev[w] : p.h2w[w];
            }
        consumer_sync();
    }
    float4 c_old[kPasses], c_acc[kPasses];         // FUSE: carried through the workers of a tile
    uint32_t k = 0;
    for (;; ++k) {
        const uint32_t s = k % kStages, use = k / kStages;
        // every consumer polls (bounded); one reducing barrier makes the verdict common, so
        // that nobody is left behind at a later barrier by a warp that gave up
        if (!consumers_agree(mbar_wait(&sh.full[s], use & 1u, p.status, kStatusFullTimeout))) break;
        Stage<HASC> &st = sh.stage[s];
        const uint4 h0 = ld_shared_u4(&st.hdr.worker);
        const uint32_t i = h0.x, t0 = h0.y, nvalid = h0.z, flags = h0.w;
        if (flags & kItemEnd) break;
        const ExtraSample *xs = extra + s * nextra;
        const float fn = (float)p.nsamp, rn = __frcp_rn(fn);
        float4 xn[kPasses];
        // distance rounds without an exchange: the master values of this thread's columns come
        // straight from memory (the L2 cache serves all workers of a tile but the first); asked
        // for now, used after the step
        float4 c_now[kPasses];
        if constexpr (DIST && !FUSE) {
#pragma unroll
            for (int pass = 0; pass < kPasses; ++pass) {
                const uint32_t off = (uint32_t)pass * kPassElems + 4u * ctid;
                if (off < nvalid) c_now[pass] = ld_vec(p.c + t0 + off);
            }
        }
        // fused exchange: does this worker meet the master, with which coefficients, and
        // before its local step (the exchange of the previous round) or after it
        const bool meets = FUSE && (flags & kItemExchange) != 0u;
        const bool meets_first = meets && p.pull_first != 0u;
        float h1 = 0.f, h2 = 0.f;
        if constexpr (FUSE) {
            h1 = sh.h1[i];
            h2 = sh.h2[i];
            if (flags & kItemFirst) {
#pragma unroll
                for (int pass = 0; pass < kPasses; ++pass) {
                    const uint32_t off = (uint32_t)pass * kPassElems + 4u * ctid;
                    if (off < nvalid) {
                        c_old[pass] = ld_vec(&st.c[off]);
                        // simultaneous form: what the workers add to the master, from +0;
                        // asynchronous form: the master as the arrivals so far left it
                        c_acc[pass] = p.asynchronous ? c_old[pass] : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
            }
        }

        if (!(flags & kItemDistanceOnly)) {
            const float4 wcv = ld_vec(&st.hdr.bc1);
            WorkerConst w;
            w.bc1 = wcv.x; w.bc2 = wcv.y; w.rbc1 = wcv.z; w.rbc2 = wcv.w;
            if (flags & kItemAverage) {
                const uint4 h1w = ld_shared_u4(&st.hdr.e0);
                const uint32_t e0 = h1w.x, e1 = h1w.y, run0 = h1w.z, ea0 = h1w.w;
                const uint32_t ea1 = (e1 + 3u) & ~3u, g0 = ea0 >> 7;
                if (!MULTI && (flags & kItemAll3x3)) {
                    // ---- 3x3 kernels only: means from the raw values, signs on the fly;
                    // ranges of unaveraged tensors inside the tile get their signs in place
                    for (uint32_t ri = run0;; ++ri) {
                        const Run rn = p.runs[ri];
                        if (rn.start >= e1) break;
                        const uint32_t qa = max(e0, rn.start), qb = min(e1, rn.end);
                        if (rn.block > 1u) {
                            block_means_signed9(st, qa, __umulhi(qb - qa, rn.magic), t0, g0, ctid);
                        } else {
                            for (uint32_t j = qa + ctid; j < qb; j += kConsumers) {
                                const uint32_t word = st.zw[(j >> 7) - g0][(j >> 5) & 3u];
                                float *ptr = &st.hv[j + kHalo - t0];
                                *ptr = __uint_as_float(__float_as_uint(*ptr) ^ (((word >> (j & 31u)) & 1u) << 31));
                            }
                        }
                        if (rn.end >= e1) break;
                    }
                    consumer_sync();
                } else {
                    // ---- z (.) hvp in place over the widened range
                    for (uint32_t q = ctid; q < (ea1 - ea0) >> 2; q += kConsumers) {
                        const uint32_t j = ea0 + 4u * q, hidx = j + kHalo - t0;
                        st_vec(&st.hv[hidx],
                               hutchinson4<MULTI, HASC>(st, xs, p.nsamp, hidx, (j >> 7) - g0, j, fn, rn));
                    }
                    consumer_sync();
                    // ---- block means in place, one thread per block
                    for (uint32_t ri = run0;; ++ri) {
                        const Run rn = p.runs[ri];
                        if (rn.start >= e1) break;
                        if (rn.block > 1u) {
                            const uint32_t qa = max(e0, rn.start), qb = min(e1, rn.end);
                            const uint32_t nblk = __umulhi(qb - qa, rn.magic);
                            float *base = &st.hv[qa + kHalo - t0];
                            if (rn.block == 9u) block_means_fixed<9>(base, nblk, ctid);
                            else block_means_any(base, nblk, rn.block, ctid);
                        }
                        if (rn.end >= e1) break;
                    }
                    consumer_sync();
                }
            }
            float *xr = p.x + (uint64_t)i * p.lds + t0;
            float *mr = p.m + (uint64_t)i * p.lds + t0;
            float *vr = p.v + (uint64_t)i * p.lds + t0;
#pragma unroll
            for (int pass = 0; pass < kPasses; ++pass) {
                const uint32_t off = (uint32_t)pass * kPassElems + 4u * ctid;
                if (off < nvalid) {
                    const int nv = nvalid - off >= 4u ? 4 : (int)(nvalid - off);
                    const float4 D = (flags & kItemAverage)
                        ? ld_vec(&st.hv[off + kHalo])
                        : hutchinson4<MULTI, HASC>(st, xs, p.nsamp, off + kHalo, off >> 7, off, fn, rn);
                    const float4 g = ld_vec(&st.g[off]);
                    float4 x = ld_vec(&st.x[off]), m = ld_vec(&st.m[off]), v = ld_vec(&st.v[off]);
                    if constexpr (FUSE)
                        if (meets_first)
                            meet_master4(x, c_acc[pass], c_old[pass], h1, h2, p.asynchronous != 0u);
                    if (nv == 4) {
                        adahessian_update4<POWMODE, WD>(x, m, v, g, D, p, w);
                    } else {     // ragged end of the row: lanes past P keep their (zero) state
                        adahessian_update<POWMODE, WD>(x.x, m.x, v.x, g.x, D.x, p, w);
                        if (nv > 1) adahessian_update<POWMODE, WD>(x.y, m.y, v.y, g.y, D.y, p, w);
                        if (nv > 2) adahessian_update<POWMODE, WD>(x.z, m.z, v.z, g.z, D.z, p, w);
                    }
                    if constexpr (!FUSE) st_vec(xr + off, x);     // fused: x is stored after the pull
                    st_vec(mr + off, m);
                    st_vec(vr + off, v);
                    xn[pass] = x;
                }
            }
        } else if constexpr (DIST || FUSE) {
#pragma unroll
            for (int pass = 0; pass < kPasses; ++pass) {
                const uint32_t off = (uint32_t)pass * kPassElems + 4u * ctid;
                if (off < nvalid) {
                    xn[pass] = ld_vec(&st.x[off]);
                    if constexpr (FUSE)
                        if (meets_first)
                            meet_master4(xn[pass], c_acc[pass], c_old[pass], h1, h2, p.asynchronous != 0u);
                }
            }
        }

        if constexpr (DIST) {
            // per warp and pass: the subtree of 128 consecutive (x - c)^2; the producer adds
            // the kRed of them up once the stage is back with it
#pragma unroll
            for (int pass = 0; pass < kPasses; ++pass) {
                const uint32_t off = (uint32_t)pass * kPassElems + 4u * ctid;
                double d = 0.0;
                if (off < nvalid) {
                    const int nv = nvalid - off >= 4u ? 4 : (int)(nvalid - off);
                    d = dist4(xn[pass], FUSE ? c_old[pass] : c_now[pass], nv);
                }
                d = warp_tree_sum(d);
                if (lane == 0) st.red[pass * kConsumerWarps + warp] = d;
            }
        }

        if constexpr (FUSE) {
            // ---- the elastic pull after the step, the stores of x, and the master row
#pragma unroll
            for (int pass = 0; pass < kPasses; ++pass) {
                const uint32_t off = (uint32_t)pass * kPassElems + 4u * ctid;
                if (off < nvalid) {
                    if (meets && !meets_first)
                        meet_master4(xn[pass], c_acc[pass], c_old[pass], h1, h2, p.asynchronous != 0u);
                    if (meets || !(flags & kItemDistanceOnly))
                        st_vec(p.x + (uint64_t)i * p.lds + t0 + off, xn[pass]);
                    if ((flags & kItemLast) && p.any_exchange) {
                        float4 cn = c_acc[pass];
                        if (!p.asynchronous) {
                            cn.x = __fadd_rn(c_old[pass].x, cn.x); cn.y = __fadd_rn(c_old[pass].y, cn.y);
                            cn.z = __fadd_rn(c_old[pass].z, cn.z); cn.w = __fadd_rn(c_old[pass].w, cn.w);
                        }
                        st_vec(p.c_out + t0 + off, cn);
                    }
                }
            }
        }

        // ---- hand the stage back
        fence_generic_to_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.empty[s]);
    }
}

// ---------------------------------------------------------------------------
// Launchers
// ---------------------------------------------------------------------------
template <int POWMODE, bool WD, bool DIST, bool MULTI, bool FUSE, int MAXW>
static cudaError_t launch_step_one(const StepParamsT<MAXW> &p, int sm_count, cudaStream_t s)
{
    auto kernel = local_step_kernel<POWMODE, WD, DIST, MULTI, FUSE, MAXW>;
    constexpr bool HASC = FUSE;
    using SharedT = Shared<HASC, FUSE, MAXW>;
    const size_t smem = sizeof(SharedT) +
                        (MULTI ? (size_t)kStages * (p.nsamp - 1u) * sizeof(ExtraSample) : 0);
    // Shared-memory attributes are per device and per instantiation: one bit per device
    // ordinal.  Setting them twice is harmless, so racing threads need no lock.
    static std::atomic<uint64_t> configured{0};
    static std::atomic<int> ctas_for_nsamp[AH_MAX_SAMPLES + 1] = {};
    int device = 0;
    if (cudaError_t e = cudaGetDevice(&device); e != cudaSuccess) return e;
    const uint64_t device_bit = 1ull << (device & 63);
    if (!(configured.load(std::memory_order_acquire) & device_bit)) {
        const size_t most = sizeof(SharedT) +
                            (MULTI ? (size_t)kStages * (AH_MAX_SAMPLES - 1) * sizeof(ExtraSample) : 0);
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)most);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        configured.fetch_or(device_bit, std::memory_order_release);
    }
    if (p.nitems == 0) return cudaSuccess;
    // resident CTAs per SM of this instantiation (the extra samples take shared memory)
    const uint32_t slot = MULTI ? p.nsamp : 1u;
    if (ctas_for_nsamp[slot].load(std::memory_order_relaxed) == 0) {
        int fit = 0;
        cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&fit, kernel, kThreads, smem);
        if (e != cudaSuccess) return e;
        if (fit < 1) return cudaErrorInvalidConfiguration;
        constexpr int want = ctas_per_sm(DIST, MULTI, FUSE);
        ctas_for_nsamp[slot].store(fit < want ? fit : want, std::memory_order_relaxed);
    }
    const int ctas = ctas_for_nsamp[slot].load(std::memory_order_relaxed);
    const uint32_t resident = (uint32_t)sm_count * (uint32_t)ctas;
    const uint32_t grid = p.nitems < resident ? p.nitems : resident;
    // Programmatic stream serialisation: this launch may begin (set up its barriers, read
    // its parameters) while the kernel before it in the stream drains; it waits for that
    // kernel at griddepcontrol.wait before it touches memory.
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, p);
}

template <int POWMODE, bool WD, int MAXW>
static cudaError_t launch_step_dist(const StepParamsT<MAXW> &p, bool want_dist, int sm_count,
                                    cudaStream_t s)
{
    if (p.fused && p.nsamp > 1u)         // step and exchange in one pass, several samples
        return want_dist ? launch_step_one<POWMODE, WD, true, true, true, MAXW>(p, sm_count, s)
                         : launch_step_one<POWMODE, WD, false, true, true, MAXW>(p, sm_count, s);
    if (p.fused)                         // step and exchange in one pass
        return want_dist ? launch_step_one<POWMODE, WD, true, false, true, MAXW>(p, sm_count, s)
                         : launch_step_one<POWMODE, WD, false, false, true, MAXW>(p, sm_count, s);
    if (p.nsamp > 1u)
        return want_dist ? launch_step_one<POWMODE, WD, true, true, false, MAXW>(p, sm_count, s)
                         : launch_step_one<POWMODE, WD, false, true, false, MAXW>(p, sm_count, s);
    return want_dist ? launch_step_one<POWMODE, WD, true, false, false, MAXW>(p, sm_count, s)
                     : launch_step_one<POWMODE, WD, false, false, false, MAXW>(p, sm_count, s);
}

}  // namespace ah
