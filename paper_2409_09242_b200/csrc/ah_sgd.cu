// First-order local steps on the same batched [K, P] state: plain SGD (Eqs. 2-3 of
// the paper) and SGD with momentum, the local optimisers of the EASGD and EAMSGD
// methods the paper compares against (Sec. VI; eta = 0.01, delta = 0.5 in Sec. VII).
// They share the exchange kernels and the distance / weight machinery with the
// AdaHessian step.
//
// Pure streaming: 12 bytes per parameter update without momentum (read grad and x,
// write x), 20 with it (the velocity is read and written too).  One CTA of 256
// threads covers kTilesPerCta consecutive tiles of 1024 parameters of one worker,
// one float4 per thread and tile, all loads issued before the first use.
#include <string.h>

#include "ah_ctx.h"
#include "ah_device.cuh"
#include "ah_tree.cuh"

namespace ah {

constexpr int kSgdThreads = 256;
constexpr int kSgdTile = 1024;              // = kTile: a subtree of the distance tree
#ifndef AH_SGD_TILES_PER_CTA
#define AH_SGD_TILES_PER_CTA 4
#endif
constexpr int kTilesPerCta = AH_SGD_TILES_PER_CTA;
static_assert(kSgdTile == kTile, "distance partials are indexed by the library's tile");

struct SgdParams {
    float *x, *u;                  // u: velocity (the handle's first-moment rows)
    const float *c;
    const float *grad;
    DistTree tree;                 // DIST: where the tile sums of (x - c)^2 go
    uint64_t lds, ld;
    uint32_t P, ntiles;
    float lr, momentum;
    uint32_t nrows;
    uint16_t row[AH_MAX_WORKERS];
    uint8_t active[AH_MAX_WORKERS];
};

template <bool MOMENTUM, bool DIST>
__global__ void __launch_bounds__(kSgdThreads)
sgd_step_kernel(const __grid_constant__ SgdParams p)
{
    __shared__ double red[kTilesPerCta][kSgdThreads / 32];
    const uint32_t i = p.row[blockIdx.y];
    const bool act = p.active[i] != 0;
    const uint32_t tile0 = blockIdx.x * (uint32_t)kTilesPerCta;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    float4 g[kTilesPerCta], x[kTilesPerCta], u[kTilesPerCta], c[kTilesPerCta];
    uint32_t off[kTilesPerCta];
#pragma unroll
    for (int k = 0; k < kTilesPerCta; ++k) {
        off[k] = (tile0 + k) * (uint32_t)kSgdTile + 4u * threadIdx.x;
        if (off[k] < p.P) {
            const uint64_t so = (uint64_t)i * p.lds + off[k];
            x[k] = ld_vec(p.x + so);
            if (act) g[k] = ld_vec(p.grad + (uint64_t)i * p.ld + off[k]);
            if (MOMENTUM && act) u[k] = ld_vec(p.u + so);
            if (DIST) c[k] = ld_vec(p.c + off[k]);
        }
    }
#pragma unroll
    for (int k = 0; k < kTilesPerCta; ++k) {
        double d = 0.0;
        if (off[k] < p.P) {
            const int nv = p.P - off[k] >= 4u ? 4 : (int)(p.P - off[k]);
            if (act) {
                float *xe = &x[k].x, *ue = &u[k].x;
                const float *ge = &g[k].x;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (e < nv) {            // lanes past P keep their zero state
                        if (MOMENTUM) {
                            ue[e] = __fsub_rn(__fmul_rn(p.momentum, ue[e]), __fmul_rn(p.lr, ge[e]));
                            xe[e] = __fadd_rn(xe[e], ue[e]);
                        } else {
                            xe[e] = __fsub_rn(xe[e], __fmul_rn(p.lr, ge[e]));
                        }
                    }
                }
                const uint64_t so = (uint64_t)i * p.lds + off[k];
                st_vec(p.x + so, x[k]);
                if (MOMENTUM) st_vec(p.u + so, u[k]);
            }
            if (DIST) d = dist4(x[k], c[k], nv);
        }
        if (DIST) {
            d = warp_tree_sum(d);
            if (lane == 0) red[k][warp] = d;
        }
    }
    if (DIST) {
        __syncthreads();
        // the CTA's tile sums go to level 0 of the distance tree; whoever needs the
        // distances assembles them
        if (warp == 0 && lane < kTilesPerCta && tile0 + lane < p.ntiles)
            tree_store_tile(p.tree, i, tile0 + lane, tree8(red[lane]));
    }
}

template <bool MOMENTUM, bool DIST>
static cudaError_t launch_sgd(const SgdParams &p, cudaStream_t s)
{
    const dim3 grid((p.ntiles + kTilesPerCta - 1) / kTilesPerCta, p.nrows);
    if (p.nrows == 0) return cudaSuccess;
    sgd_step_kernel<MOMENTUM, DIST><<<grid, kSgdThreads, 0, s>>>(p);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Exchange, then the first-order step, in one pass (EASGD / EAMSGD periods): one thread
// owns four consecutive columns, keeps their master values in registers and walks the
// workers in arrival order; each worker's x is pulled (Eqs. 12-13), stepped, and stored
// once.  Loads of the next workers are in flight while one is computed.
// ---------------------------------------------------------------------------
struct SgdExchangeParams {
    float *x, *u, *c;
    const float *grad;
    const float *wdev;             // not null: h2 of worker i at wdev[i], h1 at wdev[K + i]
    uint64_t lds, ld;
    uint32_t nvec;                 // float4 columns (= lds / 4)
    uint32_t P;
    float lr, momentum;
    uint32_t nrows, nworkers, asynchronous, any_exchange;
    uint16_t row[AH_MAX_WORKERS];  // workers in arrival order
    uint8_t active[AH_MAX_WORKERS], exch[AH_MAX_WORKERS];   // by worker index
    float h1w[AH_MAX_WORKERS], h2w[AH_MAX_WORKERS];
};

template <bool MOMENTUM>
__global__ void __launch_bounds__(256)
exchange_then_sgd_kernel(const __grid_constant__ SgdExchangeParams p)
{
    constexpr int kDepth = 2;                      // workers whose loads are in flight
    const uint32_t q = blockIdx.x * 256u + threadIdx.x;
    if (q >= p.nvec) return;
    const uint64_t col = 4ull * q;
    const int nv = p.P - (uint32_t)col >= 4u ? 4 : (int)(p.P - (uint32_t)col);   // lanes past P stay zero
    const float4 c_old = ld_vec(p.c + col);
    float4 carry = p.asynchronous ? c_old : make_float4(0.f, 0.f, 0.f, 0.f);
    for (uint32_t r0 = 0; r0 < p.nrows; r0 += kDepth) {
        float4 x[kDepth], g[kDepth], u[kDepth];
#pragma unroll
        for (int k = 0; k < kDepth; ++k) {
            if (r0 + k < p.nrows) {
                const uint32_t i = p.row[r0 + k];
                x[k] = ld_vec(p.x + (uint64_t)i * p.lds + col);
                if (p.active[i]) {
                    g[k] = ld_vec(p.grad + (uint64_t)i * p.ld + col);
                    if (MOMENTUM) u[k] = ld_vec(p.u + (uint64_t)i * p.lds + col);
                }
            }
        }
#pragma unroll
        for (int k = 0; k < kDepth; ++k) {
            if (r0 + k < p.nrows) {
                const uint32_t i = p.row[r0 + k];
                if (p.exch[i]) {
                    const float h1 = p.wdev ? p.wdev[p.nworkers + i] : p.h1w[i];
                    const float h2 = p.wdev ? p.wdev[i] : p.h2w[i];
                    float *xe = &x[k].x, *ae = &carry.x;
                    const float *ce = &c_old.x;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        if (p.asynchronous) {
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
                if (p.active[i]) {
                    float *xe = &x[k].x, *ue = &u[k].x;
                    const float *ge = &g[k].x;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        if (e < nv) {
                            if (MOMENTUM) {
                                ue[e] = __fsub_rn(__fmul_rn(p.momentum, ue[e]), __fmul_rn(p.lr, ge[e]));
                                xe[e] = __fadd_rn(xe[e], ue[e]);
                            } else {
                                xe[e] = __fsub_rn(xe[e], __fmul_rn(p.lr, ge[e]));
                            }
                        }
                    }
                    if (MOMENTUM) st_vec(p.u + (uint64_t)i * p.lds + col, u[k]);
                }
                st_vec(p.x + (uint64_t)i * p.lds + col, x[k]);
            }
        }
    }
    if (p.any_exchange) {
        float4 cn = carry;
        if (!p.asynchronous) {
            cn.x = __fadd_rn(c_old.x, cn.x); cn.y = __fadd_rn(c_old.y, cn.y);
            cn.z = __fadd_rn(c_old.z, cn.z); cn.w = __fadd_rn(c_old.w, cn.w);
        }
        st_vec(p.c + col, cn);
    }
}

}  // namespace ah

using namespace ah;

extern "C" int sgd_local_step(ah_ctx *h, const float *grad, uint64_t ld, const sgd_hyper *hy)
{
    if (!h || !grad || !hy || ld < h->P) return AH_ERR_INVALID_ARG;
    if (!h->has_device) return AH_ERR_STATE;
    if (!(hy->momentum >= 0.f && hy->momentum < 1.f)) return AH_ERR_INVALID_ARG;
    if ((ld & 3u) != 0 || ((uintptr_t)grad & 15u) != 0) return AH_ERR_ALIGN;

    if (hy->want_dist != AH_DIST_NONE && hy->want_dist != AH_DIST) return AH_ERR_INVALID_ARG;
    const bool dist = hy->want_dist != 0;
    SgdParams p;
    p.x = h->x; p.u = h->m; p.c = h->c; p.grad = grad;
    p.lds = h->lds; p.ld = ld;
    p.P = h->P; p.ntiles = h->ntiles;
    p.lr = hy->lr; p.momentum = hy->momentum;
    p.nrows = 0;
    uint32_t step[AH_MAX_WORKERS];                // step counts once the launch is enqueued
    for (int i = 0; i < h->K; ++i) {
        const bool on = !hy->active || hy->active[i] != 0;
        p.active[i] = on ? 1 : 0;
        step[i] = h->step[i] + (on ? 1u : 0u);
        if (on || dist) p.row[p.nrows++] = (uint16_t)i;   // distances cover every worker
    }
    p.tree = h->tree;
    if (dist) {
        const int rc = begin_distance_store(h, p.tree);
        if (rc != AH_OK) return rc;
    }
    cudaError_t e;
    const bool mom = hy->momentum != 0.f;
    if (mom) e = dist ? launch_sgd<true, true>(p, h->stream) : launch_sgd<true, false>(p, h->stream);
    else     e = dist ? launch_sgd<false, true>(p, h->stream) : launch_sgd<false, false>(p, h->stream);
    if (e != cudaSuccess) return ah_cuda_fail(h, e);
    h->calls += 1;
    memcpy(h->step, step, (size_t)h->K * sizeof(uint32_t));
    if (p.nrows) h->launches += 1;
    if (dist && p.nrows) commit_distance_store(h, false, 0.f, false);
    return AH_OK;
}

extern "C" int easgd_exchange_then_sgd_step(ah_ctx *h, const float *grad, uint64_t ld,
                                            const sgd_hyper *hy, const uint8_t *worker_mask,
                                            const float *weights, float alpha, const uint16_t *order,
                                            int asynchronous)
{
    if (!h || !grad || !hy || ld < h->P) return AH_ERR_INVALID_ARG;
    if (!h->has_device) return AH_ERR_STATE;
    if (!(hy->momentum >= 0.f && hy->momentum < 1.f) || hy->want_dist) return AH_ERR_INVALID_ARG;
    if ((ld & 3u) != 0 || ((uintptr_t)grad & 15u) != 0) return AH_ERR_ALIGN;
    if (order) {                                  // must name every worker exactly once
        bool seen[AH_MAX_WORKERS] = {};
        for (int q = 0; q < h->K; ++q) {
            if (order[q] >= h->K || seen[order[q]]) return AH_ERR_INVALID_ARG;
            seen[order[q]] = true;
        }
    }
    SgdExchangeParams p;
    p.x = h->x; p.u = h->m; p.c = h->c; p.grad = grad; p.wdev = nullptr;
    p.lds = h->lds; p.ld = ld;
    p.nvec = (uint32_t)(h->lds / 4); p.P = h->P;
    p.lr = hy->lr; p.momentum = hy->momentum;
    p.nworkers = (uint32_t)h->K;
    p.asynchronous = asynchronous ? 1u : 0u;
    p.any_exchange = 0u;
    p.nrows = 0;
    uint32_t step[AH_MAX_WORKERS];                // step counts once the launch is enqueued
    for (int q = 0; q < h->K; ++q) {
        const int i = asynchronous && order ? (int)order[q] : q;
        const bool on = !hy->active || hy->active[i] != 0;
        const bool meets = !worker_mask || worker_mask[i] != 0;
        p.active[i] = on ? 1 : 0;
        p.exch[i] = meets ? 1 : 0;
        if (meets) p.any_exchange = 1u;
        p.h2w[i] = weights ? weights[i] : alpha;
        p.h1w[i] = weights ? weights[h->K + i] : alpha;
        step[i] = h->step[i] + (on ? 1u : 0u);
        if (on || meets) p.row[p.nrows++] = (uint16_t)i;
    }
    if (p.nrows == 0) {
        h->calls += 1;
        return AH_OK;
    }
    const unsigned blocks = (p.nvec + 255u) / 256u;
    if (hy->momentum != 0.f) exchange_then_sgd_kernel<true><<<blocks, 256, 0, h->stream>>>(p);
    else                     exchange_then_sgd_kernel<false><<<blocks, 256, 0, h->stream>>>(p);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return ah_cuda_fail(h, e);
    h->calls += 1;
    memcpy(h->step, step, (size_t)h->K * sizeof(uint32_t));
    h->launches += 1;
    return AH_OK;
}
