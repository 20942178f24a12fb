// CUDA kernels (sm_100a) of the AdaHessian + elastic-averaging round.
//
// Everything here is HBM-bound streaming work: the fused local step reads
// grad, hvp, x, m, v and writes x, m, v once (32 bytes per parameter update), the
// exchange reads and writes x once more (8 bytes per update) plus the master row.
// There is no dense contraction, so no tensor cores; the rules that matter are
// 128-bit coalesced accesses, enough loads in flight, and not touching a byte twice.
//
// Arithmetic follows one fixed order with one binary32 rounding per operation
// (__fmul_rn / __fadd_rn / __fdiv_rn / __fsqrt_rn are never contracted into FMAs),
// so results do not depend on compiler flags or launch shape.
#include "ah_internal.h"

namespace ah {

// ---------------------------------------------------------------------------
// Per-element AdaHessian update (Sec. IV-B of the paper; Eq. 4 with the diagonal
// preconditioner 1 / ((sqrt vhat)^k + eps)).  D is the spatially averaged
// Hutchinson estimate of the Hessian diagonal for this element.
// POWMODE: 0 -> k = 1, 1 -> k = 1/2, 2 -> general k via powf.
// ---------------------------------------------------------------------------
template <int POWMODE, bool WD>
__device__ __forceinline__ void adahessian_update(float &x, float &m, float &v, float g, float D,
                                                  const StepParams &p, float bc1, float bc2)
{
    const float m1 = __fadd_rn(__fmul_rn(p.beta1, m), __fmul_rn(p.omb1, g));
    const float v1 = __fadd_rn(__fmul_rn(p.beta2, v), __fmul_rn(__fmul_rn(p.omb2, D), D));
    const float mhat = __fdiv_rn(m1, bc1);
    const float vhat = __fdiv_rn(v1, bc2);
    const float r = __fsqrt_rn(vhat);
    float pw;
    if (POWMODE == 0) pw = r;
    else if (POWMODE == 1) pw = __fsqrt_rn(r);
    else pw = powf(r, p.hpow);
    const float den = __fadd_rn(pw, p.eps);
    const float q = __fdiv_rn(mhat, den);
    float xn;
    if (WD) xn = __fsub_rn(x, __fmul_rn(p.lr, __fadd_rn(q, __fmul_rn(p.wd, x))));
    else    xn = __fsub_rn(x, __fmul_rn(p.lr, q));
    x = xn; m = m1; v = v1;
}

__device__ __forceinline__ float flip_if(float a, uint32_t bit)
{
    return __uint_as_float(__float_as_uint(a) ^ (bit << 31));
}

__device__ __forceinline__ float4 apply_signs(float4 h, uint32_t nib)
{
    h.x = flip_if(h.x, nib & 1u);
    h.y = flip_if(h.y, (nib >> 1) & 1u);
    h.z = flip_if(h.z, (nib >> 2) & 1u);
    h.w = flip_if(h.w, (nib >> 3) & 1u);
    return h;
}

__device__ __forceinline__ float4 ld_stream(const float *p)
{
    return __ldcs(reinterpret_cast<const float4 *>(p));
}

__device__ __forceinline__ float4 ld_vec(const float *p)
{
    return *reinterpret_cast<const float4 *>(p);
}

__device__ __forceinline__ void st_vec(float *p, float4 v)
{
    *reinterpret_cast<float4 *>(p) = v;
}

// (x - c)^2 of up to four consecutive elements, binary32 difference, double
// square, summed as the 4-leaf subtree (d0 + d1) + (d2 + d3); lanes >= nv give +0.
__device__ __forceinline__ double dist4(float4 x, float4 c, int nv)
{
    const double d0 = nv > 0 ? (double)__fsub_rn(x.x, c.x) : 0.0;
    const double d1 = nv > 1 ? (double)__fsub_rn(x.y, c.y) : 0.0;
    const double d2 = nv > 2 ? (double)__fsub_rn(x.z, c.z) : 0.0;
    const double d3 = nv > 3 ? (double)__fsub_rn(x.w, c.w) : 0.0;
    return __dadd_rn(__dadd_rn(__dmul_rn(d0, d0), __dmul_rn(d1, d1)),
                     __dadd_rn(__dmul_rn(d2, d2), __dmul_rn(d3, d3)));
}

// Adjacent-pairs tree over the 32 lanes of a warp (every lane ends with the total).
__device__ __forceinline__ double warp_tree_sum(double s)
{
#pragma unroll
    for (int off = 1; off < 32; off <<= 1)
        s = __dadd_rn(s, __shfl_xor_sync(0xffffffffu, s, off));
    return s;
}

// ---------------------------------------------------------------------------
// Fused local step.  grid = (tiles, K), one CTA per tile of kTile consecutive
// parameters of one worker.  Element owned by (warp w, pass r, lane l):
//     j = tile*kTile + w*(kGroupsPerWarp*128) + r*128 + 4*l
// so each warp pass is one coalesced 512-byte row per stream, and one row is
// exactly the 128 elements covered by one Philox block.
//
// Rademacher signs: lane l computes the Philox block of group (l mod
// kGroupsPerWarp) of its warp and keeps output word l/8; in pass r every lane
// fetches the word it needs from lane (l & ~7) | r with one shuffle.  z costs no
// memory traffic.
//
// Tiles whose tensors all have spatial block 1 stay in registers.  Tiles that
// touch a tensor with block > 1 stage the signed Hessian-vector values of the tile,
// widened to whole blocks, in shared memory; one thread per block replaces the
// block by its mean in place (ascending-order sum, one division); the update then
// reads the averaged values back.
//
// DIST additionally leaves, per tile, the pairwise-tree sum of (x_new - c)^2 in
// p.partials[worker][tile] (all workers, active or not).
// ---------------------------------------------------------------------------
template <int POWMODE, bool WD, bool DIST>
__global__ void __launch_bounds__(kThreads)
local_step_kernel(const __grid_constant__ StepParams p)
{
    __shared__ __align__(16) float sD[kStageFloats];
    __shared__ uint32_t sZ[kStageGroups][4];
    __shared__ double sRed[kWarps];

    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    const int i = blockIdx.y;
    const uint32_t tile = blockIdx.x;
    const bool active = p.active[i] != 0;
    if (!active && !DIST) return;

    const uint32_t t0 = tile * (uint32_t)kTile;
    const uint32_t jw = t0 + (uint32_t)warp * (kGroupsPerWarp * 128) + 4u * (uint32_t)lane;
    float *xr = p.x + (uint64_t)i * p.lds;

    float4 xv[kGroupsPerWarp];
    int nv[kGroupsPerWarp];            // valid lanes of each float4 (0..4)
#pragma unroll
    for (int r = 0; r < kGroupsPerWarp; ++r) {
        const uint32_t j = jw + 128u * r;
        nv[r] = j >= p.P ? 0 : (p.P - j >= 4u ? 4 : (int)(p.P - j));
    }

    if (active) {
        float *mr = p.m + (uint64_t)i * p.lds;
        float *vr = p.v + (uint64_t)i * p.lds;
        const float *gr = p.grad + (uint64_t)i * p.ld;
        const float *hr = p.hvp + (uint64_t)i * p.ld;
        const float bc1 = p.bc1[i], bc2 = p.bc2[i];
        const TileInfo ti = p.tiles[tile];

        const bool in_registers = (ti.flags & 1u) == 0;

        // issue every global load of the tile up front
        float4 gv[kGroupsPerWarp], mv[kGroupsPerWarp], vv[kGroupsPerWarp], dv[kGroupsPerWarp];
#pragma unroll
        for (int r = 0; r < kGroupsPerWarp; ++r) {
            if (nv[r] > 0) {
                const uint32_t j = jw + 128u * r;
                if (in_registers) dv[r] = ld_stream(hr + j);
                gv[r] = ld_stream(gr + j);
                xv[r] = ld_vec(xr + j);
                mv[r] = ld_vec(mr + j);
                vv[r] = ld_vec(vr + j);
            }
        }

        if (in_registers) {
            // -------- all spatial blocks are 1: signs by shuffle, D stays in registers
            uint32_t w[4];
            const uint32_t grp = (t0 >> 7) + (uint32_t)warp * kGroupsPerWarp
                                 + (uint32_t)(lane & (kGroupsPerWarp - 1));
            philox4x32_10(grp, (uint32_t)i, p.round, kDomainZ, p.key0, p.key1, w);
            const int sel = lane >> 3;
            const uint32_t mine = sel == 0 ? w[0] : sel == 1 ? w[1] : sel == 2 ? w[2] : w[3];
#pragma unroll
            for (int r = 0; r < kGroupsPerWarp; ++r) {
                const uint32_t word = __shfl_sync(0xffffffffu, mine, (lane & ~7) | r);
                if (nv[r] > 0) {
                    const uint32_t nib = (word >> (4 * (lane & 7))) & 0xFu;
                    dv[r] = apply_signs(dv[r], nib);
                }
            }
        } else {
            // -------- stage z (.) hvp for [e0, e1) rounded out to 16 bytes
            const uint32_t ea0 = ti.e0 & ~3u;
            const uint32_t ea1 = (ti.e1 + 3u) & ~3u;
            const uint32_t g0 = ea0 >> 7;
            const uint32_t ng = ((ea1 - 1u) >> 7) - g0 + 1u;
            if ((uint32_t)tid < ng)
                philox4x32_10(g0 + tid, (uint32_t)i, p.round, kDomainZ, p.key0, p.key1, sZ[tid]);
            __syncthreads();
            const uint32_t nvec = (ea1 - ea0) >> 2;
            for (uint32_t q = tid; q < nvec; q += kThreads) {
                const uint32_t j = ea0 + 4u * q;
                const uint32_t word = sZ[(j >> 7) - g0][(j >> 5) & 3u];
                const uint32_t nib = (word >> (j & 31u)) & 0xFu;
                st_vec(&sD[4u * q], apply_signs(ld_stream(hr + j), nib));
            }
            __syncthreads();
            // -------- block means, one thread per block, in place
            for (uint32_t ri = ti.run0; ri < 0xffffffffu; ++ri) {
                const Run rn = p.runs[ri];
                if (rn.start >= ti.e1) break;
                if (rn.block > 1u) {
                    const uint32_t qa = max(ti.e0, rn.start);
                    const uint32_t qb = min(ti.e1, rn.end);
                    const uint32_t nblk = __umulhi(qb - qa, rn.magic);
                    const float fb = (float)rn.block;
                    for (uint32_t k = tid; k < nblk; k += kThreads) {
                        float *blk = &sD[qa - ea0 + k * rn.block];
                        float S = blk[0];
                        for (uint32_t e = 1; e < rn.block; ++e) S = __fadd_rn(S, blk[e]);
                        const float mean = __fdiv_rn(S, fb);
                        for (uint32_t e = 0; e < rn.block; ++e) blk[e] = mean;
                    }
                }
                if (rn.end >= ti.e1) break;
            }
            __syncthreads();
#pragma unroll
            for (int r = 0; r < kGroupsPerWarp; ++r)
                if (nv[r] > 0) dv[r] = ld_vec(&sD[jw + 128u * r - ea0]);
        }

        // -------- moments and update, then store
#pragma unroll
        for (int r = 0; r < kGroupsPerWarp; ++r) {
            if (nv[r] > 0) {
                const uint32_t j = jw + 128u * r;
                float4 x = xv[r], m = mv[r], v = vv[r];
                adahessian_update<POWMODE, WD>(x.x, m.x, v.x, gv[r].x, dv[r].x, p, bc1, bc2);
                if (nv[r] > 1) adahessian_update<POWMODE, WD>(x.y, m.y, v.y, gv[r].y, dv[r].y, p, bc1, bc2);
                if (nv[r] > 2) adahessian_update<POWMODE, WD>(x.z, m.z, v.z, gv[r].z, dv[r].z, p, bc1, bc2);
                if (nv[r] > 3) adahessian_update<POWMODE, WD>(x.w, m.w, v.w, gv[r].w, dv[r].w, p, bc1, bc2);
                st_vec(xr + j, x);
                st_vec(mr + j, m);
                st_vec(vr + j, v);
                xv[r] = x;
            }
        }
    } else {
#pragma unroll
        for (int r = 0; r < kGroupsPerWarp; ++r)
            if (nv[r] > 0) xv[r] = ld_vec(xr + jw + 128u * r);
    }

    if (DIST) {
        double s[kGroupsPerWarp];
#pragma unroll
        for (int r = 0; r < kGroupsPerWarp; ++r) {
            double d = 0.0;
            if (nv[r] > 0) d = dist4(xv[r], ld_vec(p.c + jw + 128u * r), nv[r]);
            s[r] = warp_tree_sum(d);
        }
#pragma unroll
        for (int n = kGroupsPerWarp; n > 1; n >>= 1)
#pragma unroll
            for (int k = 0; k < n / 2; ++k) s[k] = __dadd_rn(s[2 * k], s[2 * k + 1]);
        if (lane == 0) sRed[warp] = s[0];
        __syncthreads();
        if (tid == 0) {
            double t[kWarps];
#pragma unroll
            for (int k = 0; k < kWarps; ++k) t[k] = sRed[k];
#pragma unroll
            for (int n = kWarps; n > 1; n >>= 1)
#pragma unroll
                for (int k = 0; k < n / 2; ++k) t[k] = __dadd_rn(t[2 * k], t[2 * k + 1]);
            p.partials[(uint64_t)i * p.ntiles_pad + tile] = t[0];
        }
    }
}

// ---------------------------------------------------------------------------
// ||x_i - c||^2 from the tile partials: the upper levels of the same pairwise tree,
// one CTA per worker, ping-ponging between two rows of scratch.  Tiles that do not
// exist (index >= ntiles) count as +0.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
norm2_finalize_kernel(double *partials, double *scratch, uint32_t ntiles, uint32_t ntiles_pad,
                      double *norm2)
{
    const int i = blockIdx.x;
    double *a = partials + (uint64_t)i * ntiles_pad;
    double *b = scratch + (uint64_t)i * ntiles_pad;
    uint32_t live = ntiles;
    for (uint32_t n = ntiles_pad; n > 1; n >>= 1) {
        const uint32_t half = n >> 1;
        for (uint32_t k = threadIdx.x; k < half; k += blockDim.x) {
            const double l = 2 * k < live ? a[2 * k] : 0.0;
            const double r = 2 * k + 1 < live ? a[2 * k + 1] : 0.0;
            b[k] = __dadd_rn(l, r);
        }
        __syncthreads();
        double *t = a; a = b; b = t;
        live = half;
    }
    if (threadIdx.x == 0) norm2[i] = a[0];
}

// ---------------------------------------------------------------------------
// Weighted elastic exchange (Eqs. 12-13 of the paper; EASGD pull of Eqs. 8-9 when
// all coefficients are equal).  One thread owns four consecutive columns: it reads
// the master value once, walks the participating workers in ascending order with
// UNROLL row loads in flight, and writes the master once.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void pull4(float4 &x, float4 &acc, const float4 c, float h1, float h2)
{
    float d;
    d = __fsub_rn(x.x, c.x); acc.x = __fadd_rn(acc.x, __fmul_rn(h2, d)); x.x = __fsub_rn(x.x, __fmul_rn(h1, d));
    d = __fsub_rn(x.y, c.y); acc.y = __fadd_rn(acc.y, __fmul_rn(h2, d)); x.y = __fsub_rn(x.y, __fmul_rn(h1, d));
    d = __fsub_rn(x.z, c.z); acc.z = __fadd_rn(acc.z, __fmul_rn(h2, d)); x.z = __fsub_rn(x.z, __fmul_rn(h1, d));
    d = __fsub_rn(x.w, c.w); acc.w = __fadd_rn(acc.w, __fmul_rn(h2, d)); x.w = __fsub_rn(x.w, __fmul_rn(h1, d));
}

template <int UNROLL>
__global__ void __launch_bounds__(256)
exchange_kernel(const __grid_constant__ ExchangeParams p)
{
    const uint32_t q = blockIdx.x * 256u + threadIdx.x;
    if (q >= p.nvec) return;
    const uint64_t col = 4ull * q;
    const float4 c = ld_vec(p.c + col);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    int a = 0;
    for (; a + UNROLL <= p.nact; a += UNROLL) {
        float4 xv[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
            xv[u] = ld_vec(p.x + (uint64_t)p.idx[a + u] * p.lds + col);
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            pull4(xv[u], acc, c, p.h1[a + u], p.h2[a + u]);
            st_vec(p.x + (uint64_t)p.idx[a + u] * p.lds + col, xv[u]);
        }
    }
    for (; a < p.nact; ++a) {
        float4 xv = ld_vec(p.x + (uint64_t)p.idx[a] * p.lds + col);
        pull4(xv, acc, c, p.h1[a], p.h2[a]);
        st_vec(p.x + (uint64_t)p.idx[a] * p.lds + col, xv);
    }
    float4 cn;
    cn.x = __fadd_rn(c.x, acc.x); cn.y = __fadd_rn(c.y, acc.y);
    cn.z = __fadd_rn(c.z, acc.z); cn.w = __fadd_rn(c.w, acc.w);
    st_vec(p.c + col, cn);
}

// Rademacher vectors as +-1.0f (one thread per four consecutive elements).
__global__ void __launch_bounds__(256)
sample_z_kernel(float *dst, uint64_t ld, uint32_t P, uint32_t key0, uint32_t key1, uint32_t round)
{
    const uint32_t q = blockIdx.x * 256u + threadIdx.x;
    const uint32_t j = 4u * q;
    const int i = blockIdx.y;
    if (q >= (P + 3u) / 4u) return;
    uint32_t w[4];
    philox4x32_10(j >> 7, (uint32_t)i, round, kDomainZ, key0, key1, w);
    const uint32_t word = w[(j >> 5) & 3u];
    float *row = dst + (uint64_t)i * ld;
    for (uint32_t e = 0; e < 4u && j + e < P; ++e)
        row[j + e] = ((word >> ((j + e) & 31u)) & 1u) ? -1.0f : 1.0f;
}

// x_i <- c for every worker.
__global__ void __launch_bounds__(256)
broadcast_kernel(float *x, const float *c, uint64_t lds, uint32_t nvec)
{
    const uint32_t q = blockIdx.x * 256u + threadIdx.x;
    if (q >= nvec) return;
    st_vec(x + (uint64_t)blockIdx.y * lds + 4ull * q, ld_vec(c + 4ull * q));
}

// ---------------------------------------------------------------------------
// Launchers
// ---------------------------------------------------------------------------
template <int POWMODE, bool WD>
static cudaError_t launch_step_dist(const StepParams &p, dim3 grid, bool want_dist, cudaStream_t s)
{
    if (want_dist) local_step_kernel<POWMODE, WD, true><<<grid, kThreads, 0, s>>>(p);
    else           local_step_kernel<POWMODE, WD, false><<<grid, kThreads, 0, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_local_step(const StepParams &p, int K, bool want_dist, cudaStream_t s)
{
    const dim3 grid(p.ntiles, (unsigned)K);
    const int mode = p.hpow == 1.0f ? 0 : (p.hpow == 0.5f ? 1 : 2);
    const bool wd = p.wd != 0.0f;
    switch (mode * 2 + (wd ? 1 : 0)) {
    case 0: return launch_step_dist<0, false>(p, grid, want_dist, s);
    case 1: return launch_step_dist<0, true>(p, grid, want_dist, s);
    case 2: return launch_step_dist<1, false>(p, grid, want_dist, s);
    case 3: return launch_step_dist<1, true>(p, grid, want_dist, s);
    case 4: return launch_step_dist<2, false>(p, grid, want_dist, s);
    default: return launch_step_dist<2, true>(p, grid, want_dist, s);
    }
}

cudaError_t launch_norm2_finalize(double *partials, double *scratch, uint32_t ntiles,
                                  uint32_t ntiles_pad, int K, double *norm2, cudaStream_t s)
{
    norm2_finalize_kernel<<<K, 1024, 0, s>>>(partials, scratch, ntiles, ntiles_pad, norm2);
    return cudaGetLastError();
}

cudaError_t launch_exchange(const ExchangeParams &p, cudaStream_t s)
{
    const unsigned blocks = (p.nvec + 255u) / 256u;
    if (blocks == 0) return cudaSuccess;
    if (p.nact >= 4) exchange_kernel<4><<<blocks, 256, 0, s>>>(p);
    else             exchange_kernel<1><<<blocks, 256, 0, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_sample_z(float *dst, uint64_t ld, uint32_t P, int K, uint32_t key0,
                            uint32_t key1, uint32_t round, cudaStream_t s)
{
    const unsigned nvec = (P + 3u) / 4u;
    const dim3 grid((nvec + 255u) / 256u, (unsigned)K);
    sample_z_kernel<<<grid, 256, 0, s>>>(dst, ld, P, key0, key1, round);
    return cudaGetLastError();
}

cudaError_t launch_broadcast(float *x, const float *c, uint64_t lds, int K, cudaStream_t s)
{
    const unsigned nvec = (unsigned)(lds / 4);
    const dim3 grid((nvec + 255u) / 256u, (unsigned)K);
    broadcast_kernel<<<grid, 256, 0, s>>>(x, c, lds, nvec);
    return cudaGetLastError();
}

}  // namespace ah
