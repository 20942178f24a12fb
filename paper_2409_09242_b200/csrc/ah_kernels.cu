// The smaller CUDA kernels (sm_100a) of the AdaHessian + elastic-averaging round: the
// weighted elastic exchange, the Rademacher sampler for callers, the broadcast of the
// master, the assembly of the distances for readers other than a fused exchange; and
// the entry to the fused local step, whose instantiations live in
// ah_step_inst.cu.  All HBM-bound streaming work: wide coalesced accesses, enough bytes
// in flight, no byte touched twice.
#include "ah_internal.h"
#include "ah_device.cuh"
#include "ah_tree.cuh"

namespace ah {

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
            pull4(xv[u], acc, c, exchange_h1(p, a + u), exchange_h2(p, a + u));
            st_vec(p.x + (uint64_t)p.idx[a + u] * p.lds + col, xv[u]);
        }
    }
    for (; a < p.nact; ++a) {
        float4 xv = ld_vec(p.x + (uint64_t)p.idx[a] * p.lds + col);
        pull4(xv, acc, c, exchange_h1(p, a), exchange_h2(p, a));
        st_vec(p.x + (uint64_t)p.idx[a] * p.lds + col, xv);
    }
    float4 cn;
    cn.x = __fadd_rn(c.x, acc.x); cn.y = __fadd_rn(c.y, acc.y);
    cn.z = __fadd_rn(c.z, acc.z); cn.w = __fadd_rn(c.w, acc.w);
    st_vec(p.c + col, cn);
}

// Rademacher vectors as +-1.0f (one thread per four consecutive elements).
__global__ void __launch_bounds__(256)
sample_z_kernel(float *dst, uint64_t ld, uint32_t P, uint32_t key0, uint32_t key1, uint32_t round,
                uint32_t sample)
{
    const uint32_t q = blockIdx.x * 256u + threadIdx.x;
    const uint32_t j = 4u * q;
    const int i = blockIdx.y;
    if (q >= (P + 3u) / 4u) return;
    uint32_t w[4];
    philox4x32_10(j >> 7, (uint32_t)i, round, kDomainZ + 256u * sample, key0, key1, w);
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

// The distances ||x_i - c||^2 from the tile sums of the last distance round (and the
// weighting rule on them, if it is owed), for the host, a snapshot or an exchange kernel:
// a few CTAs of four warps.
constexpr int kAssembleThreads = 128;
__global__ void __launch_bounds__(kAssembleThreads)
assemble_kernel(const __grid_constant__ DistTree T)
{
    __shared__ uint32_t words[2];
    assemble_distances(T, (int)threadIdx.x, kAssembleThreads, blockIdx.x, gridDim.x, nullptr, nullptr,
                       words, [] { __syncthreads(); }, [] {});
}

// ---------------------------------------------------------------------------
// Launchers
// ---------------------------------------------------------------------------
cudaError_t launch_assemble(const DistTree &T, uint32_t ctas, cudaStream_t s)
{
    assemble_kernel<<<ctas, kAssembleThreads, 0, s>>>(T);
    return cudaGetLastError();
}

cudaError_t launch_step_inst_0(const StepParams &p, bool want_dist, int sm_count, cudaStream_t s);
cudaError_t launch_step_inst_1(const StepParams &p, bool want_dist, int sm_count, cudaStream_t s);
cudaError_t launch_step_inst_2(const StepParams &p, bool want_dist, int sm_count, cudaStream_t s);
cudaError_t launch_step_inst_3(const StepParams &p, bool want_dist, int sm_count, cudaStream_t s);
cudaError_t launch_step_inst_4(const StepParams &p, bool want_dist, int sm_count, cudaStream_t s);
cudaError_t launch_step_inst_5(const StepParams &p, bool want_dist, int sm_count, cudaStream_t s);

// The fused local step: Hessian power 1 and 1/2 have exact instantiations of their own,
// any other power goes through powf; weight decay is compiled in or out.
cudaError_t launch_local_step(const StepParams &p, bool want_dist, int sm_count, cudaStream_t s)
{
    const int mode = p.hpow == 1.0f ? 0 : (p.hpow == 0.5f ? 1 : 2);
    const bool wd = p.wd != 0.0f;
    switch (mode * 2 + (wd ? 1 : 0)) {
    case 0: return launch_step_inst_0(p, want_dist, sm_count, s);
    case 1: return launch_step_inst_1(p, want_dist, sm_count, s);
    case 2: return launch_step_inst_2(p, want_dist, sm_count, s);
    case 3: return launch_step_inst_3(p, want_dist, sm_count, s);
    case 4: return launch_step_inst_4(p, want_dist, sm_count, s);
    default: return launch_step_inst_5(p, want_dist, sm_count, s);
    }
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
                            uint32_t key1, uint32_t round, uint32_t sample, cudaStream_t s)
{
    const unsigned nvec = (P + 3u) / 4u;
    const dim3 grid((nvec + 255u) / 256u, (unsigned)K);
    sample_z_kernel<<<grid, 256, 0, s>>>(dst, ld, P, key0, key1, round, sample);
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
