// Internal declarations shared by the host side (ah_host.cu) and the kernels
// (ah_kernels.cu) of the AdaHessian + elastic-averaging library.  Not installed.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "adahess.h"

namespace ah {

// The fused local step is a persistent, warp-specialised pipeline.  One *item* is
// a tile of kTile consecutive parameters of one worker.  A power of two, so that a
// tile is a subtree of the pairwise summation tree used for ||x_i - c||^2.
//   - warp kConsumerWarps (the producer) fills a ring of kStages shared-memory
//     stages: 1-D bulk copies (TMA) of the tile's grad, x, m, v (and c) and of the
//     Hessian-vector tile widened to whole spatial blocks, plus the Philox words of
//     the tile's Rademacher signs;
//   - warps 0..kConsumerWarps-1 (the consumers) take a stage when its mbarrier
//     flips, apply signs, average spatial blocks, update, store, and hand the stage
//     back through a second mbarrier.
// Shape: four consumer warps, each thread taking two float4 per stream and item, so that
// what a thread does once per item (wait, header, addresses, hand-back) is spread over
// eight parameters; five CTAs per SM for the plain round, four where the stages also
// carry a tile of the master row.  Measured against eight warps of one float4 each:
// 16 % fewer instructions per update at the same speed at full clock, 3 % faster where the
// power cap holds the clock down.
#ifndef AH_PASSES
#define AH_PASSES 2
#endif
#ifndef AH_STAGES
#define AH_STAGES 2
#endif
#ifndef AH_CTAS_PER_SM
#define AH_CTAS_PER_SM 4
#endif
#ifndef AH_CTAS_PER_SM_PLAIN
#define AH_CTAS_PER_SM_PLAIN 5
#endif
#ifndef AH_CONSUMER_WARPS
#define AH_CONSUMER_WARPS 4
#endif
constexpr int kPasses = AH_PASSES;                 // float4 per consumer thread per stream
constexpr int kConsumerWarps = AH_CONSUMER_WARPS;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kThreads = kConsumers + 32;
constexpr int kPassElems = kConsumers * 4;         // 1024: one float4 per consumer
constexpr int kTile = kPassElems * kPasses;
constexpr int kStages = AH_STAGES;
constexpr int kCtasPerSm = AH_CTAS_PER_SM;             // resident CTAs per SM the kernels are built for
constexpr int kCtasPerSmPlain = AH_CTAS_PER_SM_PLAIN;   // ... the plain round (smallest stages)
static_assert((kTile & (kTile - 1)) == 0, "tile must be a power of two");

// A spatial block may straddle a tile edge: the Hessian-vector stage holds up to
// kHalo more elements on each side (AH_MAX_BLOCK - 1 rounded out to 16 bytes).
constexpr int kHalo = AH_MAX_BLOCK;
static_assert(kHalo % 4 == 0 && kHalo <= 128, "halo spans at most one Philox group a side");
constexpr int kStageGroups = kTile / 128 + 2;      // Philox groups a stage can touch

// Bits of the device status word (0 = healthy).
enum : uint32_t {
    kStatusFullTimeout = 1u,    // a consumer gave up waiting for a stage to fill
    kStatusEmptyTimeout = 2u,   // the producer gave up waiting for a stage to drain
};

// The row [0, P) cut into maximal runs of equal spatial block (gaps and block-1
// tensors merged).  magic = ceil(2^32 / block) turns r / block into one mul-hi for
// r * block < 2^32; unused when block == 1.
struct Run {
    uint32_t start;
    uint32_t end;
    uint32_t block;
    uint32_t magic;
};

// Per tile: first run that intersects it, and the tile's range widened to whole
// spatial blocks [e0, e1).  flags bit 0: some run with block > 1 intersects the tile;
// bit 1: every such run has block 9 (3 x 3 kernels), the case with its own fast path.
struct TileInfo {
    uint32_t run0;
    uint32_t e0;
    uint32_t e1;
    uint32_t flags;
};

// Per-worker constants of one step: bias corrections 1 - beta^t (t = the worker's
// own step count) and their correctly rounded reciprocals.
struct WorkerConst {
    float bc1, bc2, rbc1, rbc2;
};

// Parameters of the weighting rule of Sec. V-B (dw_config), as the kernels that run the
// rule after assembling the distances receive them.
struct RuleConfig {
    double coef[AH_MAX_HIST];  // c_0 .. c_{p-1}, c_0 on the newest difference
    double kappa;              // threshold of h1 / h2, negative
    int p_hist;                // history depth p
    int reserved;
};

// Where the squared distances ||x_i - c||^2 of a round are assembled.  A kernel that
// measures distances only stores one sum per (worker, tile): level 0 of a tree in which
// every higher level holds, per worker, the adjacent-pairs tree sums of 64 consecutive
// nodes of the level below, up to a single root, norm2[i].  The upper levels are formed at
// the head of the launch that needs the distances (the fused exchange that follows, or a
// small kernel of its own for every other reader): the CTAs share the nodes of the large
// levels and meet at one counter per level, which counts finished nodes; levels with few
// inputs are summed by every CTA for itself.  A CTA that has waited `wait_polls` polls for
// the others sums the whole level itself, so nothing depends on the CTAs running at the
// same time; the values are the same whoever forms them (fixed tree order).  CTA 0 also
// copies the K results (and the status word) to pinned host memory and, when the rule is
// asked for, stores the coefficients and the advanced history ring.  Level 0 has two
// copies, so that a launch may assemble one round's sums while it stores the next one's.
// The counters only ever grow: a launch is told the values they reach with it.
constexpr int kTreeRadixLog2 = 6;
constexpr int kTreeMaxLevels = 4;      // 2^21 tiles at most (P < 2^31, 1024 parameters a tile)
constexpr uint32_t kTreeOwnLevelInputs = 1024;   // a level with at most this many inputs (all
                                                 // workers) is summed by every CTA for itself
struct DistTree {
    double *sums_out;                  // level 0 this launch stores: [K][n[0]], n[0] = tiles
                                       //   rounded up to a power of two
    const double *sums_in;             // level 0 this launch assembles (assemble != 0)
    double *upper;                     // level L >= 1: upper + K * off[L] + i * n[L] + node
    uint32_t *arrive;                  // [L]: nodes of level L finished so far, over all launches
    double *norm2;                     // [K] roots
    double *norm2_host;                // pinned, mapped: [0] status word, [1 .. K] roots
    const uint32_t *status;            // device status word
    RuleConfig rule;                   // the weighting rule after the assembly: its parameters,
    const double *ring_in;             //   the history ring [K][p + 1] it reads,
    double *ring_out;                  //   the advanced ring it writes (another buffer),
    float *weights;                    //   and where the coefficients go: h2[K] then h1[K]
    double rule_alpha;
    uint32_t ring_filled;              // 0: the ring holds no sample yet
    uint32_t run_rule;                 // 1: run the rule on the assembled distances
    uint32_t assemble;                 // 1: this launch assembles sums_in at its head
    uint32_t arrive_target[kTreeMaxLevels + 1];   // what arrive[L] reaches when this launch's
                                       //   nodes of level L are all finished
    uint32_t wait_polls;               // polls before a CTA stops waiting for the others
    uint32_t shared_levels;            // levels 1 .. shared_levels are the large ones
    uint32_t K;
    uint32_t levels;                   // level `levels` is the root (n == 1)
    uint32_t n[kTreeMaxLevels + 1];    // nodes per worker at each level
    uint32_t live[kTreeMaxLevels + 1]; // of which exist (the others count as +0, never read)
    uint32_t off[kTreeMaxLevels + 1];  // nodes per worker in the levels 1 .. L-1
    uint32_t magic[kTreeMaxLevels + 1];// ceil(2^32 / live[L]) where node / live[L] is that mul-hi, else 0
};

// Launch parameters of the fused local step.  The per-worker tables are sized by the
// template argument: a launch for K <= 16 workers carries half a kilobyte of them, not
// the 7 KB that 256 workers need.
struct StepCommon {
    float *x, *m, *v;
    const float *c;
    const float *grad, *hvp;
    uint32_t *status;          // device status word
    uint32_t *sched;           // [0] next item to hand out, [1] producers that have left;
                               // both zero between launches
    const Run *runs;
    const TileInfo *tiles;
    uint64_t lds;              // row stride of x, m, v (elements, multiple of 4)
    uint64_t ld;               // row stride of grad, hvp
    uint32_t P;
    uint32_t ntiles;
    uint32_t key0, key1, round;
    float lr, beta1, beta2, omb1, omb2, eps, hpow, wd;
    uint32_t narrow_ok;        // 1: eps and the bias corrections are where the branch-free exact
                               // square root and division may be used inside the division window
    uint32_t nsamp;            // Hutchinson samples per step (1 .. AH_MAX_SAMPLES)
    uint64_t sample_stride;    // elements between consecutive samples in hvp
    uint32_t nrows;            // worker rows to process (all K when distances are wanted)
    uint32_t nitems;           // nrows * ntiles
    // fused step + exchange (one pass on exchange rounds); unused otherwise
    uint32_t fused;                   // 1: an item is a tile with all its workers, in row order
    uint32_t asynchronous;            // 1: workers meet the master one at a time, in row order
    uint32_t pull_first;              // 1: a worker meets the master before its local step
    uint32_t any_exchange;            // 0: nobody meets the master, it is not written
    uint32_t nworkers;                // K, for the layout of wdev
    float *c_out;                     // the master row, written once per tile
    const float *wdev;                // not null: h2 of worker i at wdev[i], h1 at wdev[K + i]
    DistTree tree;                    // distance rounds only
};

template <int MAXW>
struct StepParamsT : StepCommon {
    WorkerConst w[MAXW];
    float h1w[MAXW];                  // coefficients by worker index when wdev is null
    float h2w[MAXW];
    uint16_t row[MAXW];               // row r -> worker index
    uint8_t active[MAXW];             // by worker index
    uint8_t exch[MAXW];               // by worker index: meets the master this round
};
constexpr int kFewWorkers = 16;
using StepParams = StepParamsT<AH_MAX_WORKERS>;      // what the host fills in
using StepParamsFew = StepParamsT<kFewWorkers>;      // what a launch for K <= 16 carries

struct ExchangeParams {
    float *x;
    float *c;
    uint64_t lds;
    uint32_t nvec;             // float4 columns (= lds / 4)
    int nact;                  // workers taking part
    uint16_t idx[AH_MAX_WORKERS];   // their indices, ascending
    float h1[AH_MAX_WORKERS];       // compacted to the same order
    float h2[AH_MAX_WORKERS];
    const float *wdev;              // not null: coefficients come from device memory instead,
                                    // h2 of worker i at wdev[i], h1 at wdev[nworkers + i]
    int nworkers;
};

#ifdef __CUDACC__
// Coefficients of the a-th arriving worker, from the launch parameters or, when the
// weights were computed on the device, from memory.
__device__ __forceinline__ float exchange_h1(const ExchangeParams &p, int a)
{
    return p.wdev ? p.wdev[p.nworkers + p.idx[a]] : p.h1[a];
}

__device__ __forceinline__ float exchange_h2(const ExchangeParams &p, int a)
{
    return p.wdev ? p.wdev[p.idx[a]] : p.h2[a];
}
#endif

// Kernel launchers (ah_kernels.cu).  Each returns the cudaError_t of the launch.
cudaError_t launch_local_step(const StepParams &p, bool want_dist, int sm_count, cudaStream_t s);
cudaError_t launch_exchange(const ExchangeParams &p, cudaStream_t s);
cudaError_t launch_sample_z(float *dst, uint64_t ld, uint32_t P, int K, uint32_t key0,
                            uint32_t key1, uint32_t round, uint32_t sample, cudaStream_t s);
cudaError_t launch_broadcast(float *x, const float *c, uint64_t lds, int K, cudaStream_t s);

// Philox4x32-10 (Salmon et al., SC'11), usable on both sides.
__host__ __device__ inline void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t out[4])
{
#pragma unroll
    for (int round = 0; round < 10; ++round) {
#ifdef __CUDA_ARCH__
        const uint32_t hiA = __umulhi(0xD2511F53u, c0), loA = 0xD2511F53u * c0;
        const uint32_t hiB = __umulhi(0xCD9E8D57u, c2), loB = 0xCD9E8D57u * c2;
#else
        const uint64_t pa = 0xD2511F53ull * c0, pb = 0xCD9E8D57ull * c2;
        const uint32_t hiA = (uint32_t)(pa >> 32), loA = (uint32_t)pa;
        const uint32_t hiB = (uint32_t)(pb >> 32), loB = (uint32_t)pb;
#endif
        const uint32_t y0 = hiB ^ c1 ^ k0;
        const uint32_t y2 = hiA ^ c3 ^ k1;
        c0 = y0; c1 = loB; c2 = y2; c3 = loA;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

enum : uint32_t { kDomainZ = 0, kDomainFail = 1, kDomainStale = 2 };

}  // namespace ah
