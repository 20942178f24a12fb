// One combination of Hessian power and weight decay of the fused local step, with all its
// variants (distances, several Hutchinson samples, fused exchange, table size).  Compiled
// once per value of AH_STEP_INST = 2 * mode + weight decay (mode 0: k = 1, 1: k = 1/2,
// 2: any k through powf), so that the six sets of instantiations build side by side.
#include "ah_local_step.cuh"

#ifndef AH_STEP_INST
#error "compile with -DAH_STEP_INST=0 .. 5"
#endif

namespace ah {

#define AH_CONCAT2(a, b) a##b
#define AH_CONCAT(a, b) AH_CONCAT2(a, b)

cudaError_t AH_CONCAT(launch_step_inst_, AH_STEP_INST)(const StepParams &p, bool want_dist, int sm_count,
                                                       cudaStream_t s)
{
    constexpr int kMode = AH_STEP_INST / 2;
    constexpr bool kDecay = (AH_STEP_INST % 2) != 0;
    if (p.nworkers > (uint32_t)kFewWorkers)
        return launch_step_dist<kMode, kDecay, AH_MAX_WORKERS>(p, want_dist, sm_count, s);
    // few workers: the launch carries per-worker tables of kFewWorkers entries
    StepParamsFew q;
    static_cast<StepCommon &>(q) = static_cast<const StepCommon &>(p);
    for (int i = 0; i < kFewWorkers; ++i) {
        q.w[i] = p.w[i]; q.h1w[i] = p.h1w[i]; q.h2w[i] = p.h2w[i];
        q.row[i] = p.row[i]; q.active[i] = p.active[i]; q.exch[i] = p.exch[i];
    }
    return launch_step_dist<kMode, kDecay, kFewWorkers>(q, want_dist, sm_count, s);
}

}  // namespace ah
