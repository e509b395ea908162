// Order-free exact sums of fp32 magnitudes: each term is floor(|v| * 2^64) as an unsigned 128-bit integer, so the
// sum does not depend on the order in which threads, warps and blocks add (the weight scale gamma, Eq. 3, is formed
// this way).
#pragma once

#include <cstdint>

namespace bitlinear {

struct U128 {
    unsigned long long lo, hi;
};

__device__ __forceinline__ void add128(U128 &a, unsigned long long lo, unsigned long long hi)
{
    a.lo += lo;
    a.hi += hi + (a.lo < lo ? 1ull : 0ull);
}

// floor(|v| * 2^64) for an fp32 magnitude given as bits (sign cleared, exponent < 151).
__device__ __forceinline__ void fix64(uint32_t mag, unsigned long long &lo, unsigned long long &hi)
{
    uint32_t e = mag >> 23;
    uint32_t frac = mag & 0x7FFFFFu;
    unsigned long long sig = e ? (frac | 0x800000u) : frac;
    int shift = (int)(e ? e : 1u) - 86; // value = sig * 2^shift
    if (shift >= 0) {
        if (shift == 0) { lo = sig; hi = 0; }
        else if (shift < 64) { lo = sig << shift; hi = sig >> (64 - shift); }
        else { lo = 0; hi = sig << (shift - 64); }
    } else {
        int s = -shift;
        lo = (s < 24) ? (sig >> s) : 0ull;
        hi = 0;
    }
}

} // namespace bitlinear
