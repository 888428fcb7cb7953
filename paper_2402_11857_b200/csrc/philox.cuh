// Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC 2011),
// the counter-based generator behind the seeded random-k draw (Def. 3): a pure function of
// (counter, key), so every thread computes the block it needs without any state.
#pragma once
#include <cstdint>

namespace liec {

__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1) {
    constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;   // round multipliers
    constexpr uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;   // key increments (Weyl sequence)
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
        const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += W0;   // the key of the next round
        k1 += W1;
    }
    return make_uint4(c0, c1, c2, c3);
}

// Scores of the seeded subset draw: element j of segment t in the draw (seed, epoch) for row `row`
// takes word j mod 4 of the block with counter (j div 4, t, row, epoch) under key (seed low half,
// seed high half), shifted right by two: a 30-bit integer, which read as a binary32 bit pattern
// is a finite non-negative number with the same order.
struct ScoreStream {
    uint32_t k0, k1, epoch;
    __device__ __forceinline__ uint4 block(uint32_t q, uint32_t t, uint32_t row) const {
        const uint4 w = philox4x32_10(q, t, row, epoch, k0, k1);
        return make_uint4(w.x >> 2, w.y >> 2, w.z >> 2, w.w >> 2);
    }
};

}  // namespace liec
