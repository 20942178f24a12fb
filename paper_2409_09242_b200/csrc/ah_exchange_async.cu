// Asynchronous form of the elastic exchange, and the seeded order in which the
// workers reach the master.
//
// The paper assumes asynchronous training (Sec. II) and writes Eqs. 12-13 for one
// worker talking to the master.  Here the workers that take part in an exchange round
// arrive one at a time; each sees the master as the workers before it left it.  Per
// column the master value is carried in a register through all arrivals, so the
// traffic is that of the simultaneous form: one read and one write of every
// arriving worker's row, one read and one write of the master row.
#include "ah_ctx.h"

namespace ah {

__device__ __forceinline__ float4 ldg4(const float *p)
{
    return *reinterpret_cast<const float4 *>(p);
}

__device__ __forceinline__ void stg4(float *p, float4 v)
{
    *reinterpret_cast<float4 *>(p) = v;
}

// One arrival on one column: Eq. 12 for the worker, Eq. 13 for the master, both from
// the same difference.
__device__ __forceinline__ void meet(float &x, float &c, float h1, float h2)
{
    const float d = __fsub_rn(x, c);
    x = __fsub_rn(x, __fmul_rn(h1, d));
    c = __fadd_rn(c, __fmul_rn(h2, d));
}

// One thread owns four consecutive columns.  The row loads do not depend on the
// running master value, so UNROLL of them are in flight while the previous group's
// serial chain of arrivals is computed.
template <int UNROLL>
__global__ void __launch_bounds__(256)
exchange_async_kernel(const __grid_constant__ ExchangeParams p)
{
    const uint32_t q = blockIdx.x * 256u + threadIdx.x;
    if (q >= p.nvec) return;
    const uint64_t col = 4ull * q;
    float4 c = ldg4(p.c + col);
    int a = 0;
    for (; a + UNROLL <= p.nact; a += UNROLL) {
        float4 xv[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
            xv[u] = ldg4(p.x + (uint64_t)p.idx[a + u] * p.lds + col);
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const float h1 = exchange_h1(p, a + u), h2 = exchange_h2(p, a + u);
            meet(xv[u].x, c.x, h1, h2);
            meet(xv[u].y, c.y, h1, h2);
            meet(xv[u].z, c.z, h1, h2);
            meet(xv[u].w, c.w, h1, h2);
            stg4(p.x + (uint64_t)p.idx[a + u] * p.lds + col, xv[u]);
        }
    }
    for (; a < p.nact; ++a) {
        float4 xv = ldg4(p.x + (uint64_t)p.idx[a] * p.lds + col);
        const float h1 = exchange_h1(p, a), h2 = exchange_h2(p, a);
        meet(xv.x, c.x, h1, h2);
        meet(xv.y, c.y, h1, h2);
        meet(xv.z, c.z, h1, h2);
        meet(xv.w, c.w, h1, h2);
        stg4(p.x + (uint64_t)p.idx[a] * p.lds + col, xv);
    }
    stg4(p.c + col, c);
}

static cudaError_t launch_exchange_async(const ExchangeParams &p, cudaStream_t s)
{
    const unsigned blocks = (p.nvec + 255u) / 256u;
    if (blocks == 0) return cudaSuccess;
    if (p.nact >= 4) exchange_async_kernel<4><<<blocks, 256, 0, s>>>(p);
    else             exchange_async_kernel<1><<<blocks, 256, 0, s>>>(p);
    return cudaGetLastError();
}

enum : uint32_t { kDomainOrder = 3 };

}  // namespace ah

using namespace ah;

extern "C" {

int dw_order_next(ah_ctx *h, uint64_t seed, uint32_t round, uint16_t *order)
{
    if (!h || !order) return AH_ERR_INVALID_ARG;
    const uint32_t k0 = (uint32_t)(seed & 0xffffffffu), k1 = (uint32_t)(seed >> 32);
    for (int i = 0; i < h->K; ++i) order[i] = (uint16_t)i;
    // Fisher-Yates from the top: position q trades places with a uniformly drawn
    // position at or below it
    for (int q = h->K - 1; q >= 1; --q) {
        uint32_t draw[4];
        philox4x32_10((uint32_t)q, 0u, round, kDomainOrder, k0, k1, draw);
        const uint32_t pick = draw[0] % (uint32_t)(q + 1);
        const uint16_t held = order[q];
        order[q] = order[pick];
        order[pick] = held;
    }
    return AH_OK;
}

int easgd_exchange_async(ah_ctx *h, const uint8_t *worker_mask, const float *weights, float alpha,
                         const uint16_t *order)
{
    if (!h) return AH_ERR_INVALID_ARG;
    if (!h->has_device) return AH_ERR_STATE;
    ExchangeParams p;
    const int rc = ah::fill_exchange(h, worker_mask, weights, alpha, order, nullptr, p);
    if (rc != AH_OK) return rc;
    if (p.nact == 0) return AH_OK;                // nobody arrives: nothing moves
    const cudaError_t e = launch_exchange_async(p, h->stream);
    if (e != cudaSuccess) return ah_cuda_fail(h, e);
    h->launches += 1;
    return AH_OK;
}

}  // extern "C"

// Arrival list and coefficients of one exchange: the workers that take part, in
// `order` (null: ascending), with coefficients from `weights` (host, 2K floats), from
// `weights_dev` (device, same layout) or all equal to alpha.
int ah::fill_exchange(ah_ctx *h, const uint8_t *worker_mask, const float *weights, float alpha,
                      const uint16_t *order, const float *weights_dev, ExchangeParams &p)
{
    if (order) {                                  // must name every worker exactly once
        bool seen[AH_MAX_WORKERS] = {};
        for (int q = 0; q < h->K; ++q) {
            if (order[q] >= h->K || seen[order[q]]) return AH_ERR_INVALID_ARG;
            seen[order[q]] = true;
        }
    }
    p.x = h->x; p.c = h->c; p.lds = h->lds;
    p.nvec = (uint32_t)(h->lds / 4);
    p.wdev = weights_dev;
    p.nworkers = h->K;
    p.nact = 0;
    for (int q = 0; q < h->K; ++q) {
        const int i = order ? (int)order[q] : q;
        if (worker_mask && !worker_mask[i]) continue;
        p.idx[p.nact] = (uint16_t)i;
        p.h2[p.nact] = weights ? weights[i] : alpha;
        p.h1[p.nact] = weights ? weights[h->K + i] : alpha;
        p.nact += 1;
    }
    return AH_OK;
}

cudaError_t ah::launch_exchange_in_order(const ExchangeParams &p, cudaStream_t s)
{
    return launch_exchange_async(p, s);
}
