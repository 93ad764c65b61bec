// Philox4x32-10 (Salmon et al., SC'11), the counter-based generator behind evo_gen_inputs, for the
// kernels that produce the stream and for the one that regenerates it as a reference.
// Stream element g of seed s is word (g mod 4) of the block with counter (lo32(g/4), hi32(g/4), 0, 0)
// under key (lo32(s), hi32(s)).
#pragma once

#include <stdint.h>

namespace evo {

constexpr uint32_t kPhiloxM0 = 0xD2511F53u;
constexpr uint32_t kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u;
constexpr uint32_t kPhiloxW1 = 0xBB67AE85u;

// The ten round keys (key bumped by the Weyl constants before every round but the first) depend on the seed
// only: the host works them out once and passes them as a kernel argument, so a round reads them as constant
// operands instead of spending two additions.
struct RoundKeys { uint32_t k0[10], k1[10]; };

inline RoundKeys round_keys(uint64_t seed) {
    RoundKeys rk;
    uint32_t k0 = static_cast<uint32_t>(seed), k1 = static_cast<uint32_t>(seed >> 32);
    for (int round = 0; round < 10; ++round) {
        rk.k0[round] = k0; rk.k1[round] = k1;
        k0 += kPhiloxW0; k1 += kPhiloxW1;
    }
    return rk;
}

__device__ __forceinline__ uint4 philox4x32_10(uint64_t block, const RoundKeys& rk) {
    uint32_t c0 = static_cast<uint32_t>(block), c1 = static_cast<uint32_t>(block >> 32), c2 = 0u, c3 = 0u;
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(kPhiloxM0, c0), lo0 = kPhiloxM0 * c0;
        const uint32_t hi1 = __umulhi(kPhiloxM1, c2), lo1 = kPhiloxM1 * c2;
        const uint32_t n0 = hi1 ^ c1 ^ rk.k0[round];
        const uint32_t n2 = hi0 ^ c3 ^ rk.k1[round];
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    }
    return make_uint4(c0, c1, c2, c3);
}

}  // namespace evo
