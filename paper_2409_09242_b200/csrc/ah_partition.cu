// Data-overlap partition of a data set among the workers (Sec. V-A of the paper).
// Host-only integer work: the library offers it so that a caller can build the
// workers' index sets from the same counter-based generator that drives the rest
// of the round.
#include <stdint.h>

#include "ah_internal.h"

using namespace ah;

namespace {
enum : uint32_t { kDomainPartition = 4 };
}

extern "C" int dw_partition(uint64_t seed, uint64_t n, uint32_t k, uint64_t shared, uint32_t *perm,
                            uint64_t *bounds)
{
    if (!perm || !bounds || k < 1 || shared > n || n > 0xffffffffull) return AH_ERR_INVALID_ARG;
    const uint32_t k0 = (uint32_t)(seed & 0xffffffffu), k1 = (uint32_t)(seed >> 32);
    for (uint64_t i = 0; i < n; ++i) perm[i] = (uint32_t)i;
    // uniform shuffle: from the top, each position trades places with a position drawn
    // uniformly at or below it (a 64-bit draw keeps the modulo bias below 2^-32)
    for (uint64_t q = n; q-- > 1;) {
        uint32_t w[4];
        philox4x32_10((uint32_t)q, (uint32_t)(q >> 32), 0u, kDomainPartition, k0, k1, w);
        const uint64_t pick = (((uint64_t)w[1] << 32) | w[0]) % (q + 1);
        const uint32_t held = perm[q];
        perm[q] = perm[pick];
        perm[pick] = held;
    }
    // the shared subset first, then the workers' own subsets in order; the first
    // (n - shared) mod k workers take one point more, so that every point is assigned
    const uint64_t own = (n - shared) / k, longer = (n - shared) % k;
    bounds[0] = 0;
    bounds[1] = shared;
    for (uint32_t j = 0; j < k; ++j) bounds[j + 2] = bounds[j + 1] + own + (j < longer ? 1u : 0u);
    return AH_OK;
}
