// Device-side Philox-4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) and the subset
// rule built on it.  The paper asks only for a "randomly sampled subset" per
// stage (Section 2.3) whose elements are chosen independently with probability p
// (Appendix, Lemma 1); a counter-based generator lets every thread decide
// membership of its own coordinates with no memory traffic and no exchanged
// index list.
#pragma once
#include <cstdint>

namespace amk {

struct PhiloxOut { uint32_t x[4]; };

__device__ __forceinline__ PhiloxOut philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2,
                                                   uint32_t c3, uint32_t k0, uint32_t k1)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        const uint32_t n0 = hi1 ^ c1 ^ k0;
        const uint32_t n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    PhiloxOut o;
    o.x[0] = c0; o.x[1] = c1; o.x[2] = c2; o.x[3] = c3;
    return o;
}

// How the subset is drawn: word < thresh, or everything / nothing for p = 1 / 0
// (floor(p * 2^32) = 2^32 does not fit a 32-bit compare).
struct SubsetRule {
    uint32_t key0, key1;   // seed, low and high half
    uint32_t thresh;       // floor(p * 2^32) when 0 < that < 2^32
    uint32_t mode;         // 0: compare, 1: select everything, 2: select nothing
};

// Membership bits of coordinates 4*quad .. 4*quad+3 of `stage` at `step`
// (bit j set: coordinate 4*quad + j is in the subset).
__device__ __forceinline__ uint32_t subset_bits(const SubsetRule &rule, uint32_t stage,
                                                uint32_t step, uint32_t quad)
{
    if (rule.mode == 1u) return 0xFu;
    if (rule.mode == 2u) return 0u;
    const PhiloxOut o = philox4x32_10(quad, stage, step, 0u, rule.key0, rule.key1);
    return (o.x[0] < rule.thresh ? 1u : 0u) | (o.x[1] < rule.thresh ? 2u : 0u) |
           (o.x[2] < rule.thresh ? 4u : 0u) | (o.x[3] < rule.thresh ? 8u : 0u);
}

}  // namespace amk
