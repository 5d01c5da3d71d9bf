// Device evaluation of the AMS hash family over p = 2^61 - 1 (bucket: 2-wise, sign: 4-wise).
// Every residue is brought to canonical form [0, p-1] before `mod m` or the parity test.
#ifndef FDA_HASH_CUH_
#define FDA_HASH_CUH_

#include <stdint.h>

namespace fda {

constexpr uint64_t kP61 = (1ull << 61) - 1;

// (a*x + c) mod p for a, c in [0, p-1] and x < 2^31, without 128-bit arithmetic:
// a = ah*2^32 + al, so a*x = (ah*x)*2^32 + al*x, and 2^61 = 1 (mod p) folds the high bits.
__device__ __forceinline__ uint64_t mul_add_mod_p(uint64_t a, uint32_t x, uint64_t c)
{
    const uint64_t t1 = (a >> 32) * (uint64_t)x;            // < 2^60
    const uint64_t t0 = (a & 0xffffffffull) * (uint64_t)x;  // < 2^63
    // t1*2^32 = (t1 >> 29)*2^61 + (t1 mod 2^29)*2^32  ==  (t1 >> 29) + (t1 mod 2^29)*2^32
    uint64_t s = (t1 >> 29) + ((t1 & ((1ull << 29) - 1)) << 32) + (t0 >> 61) + (t0 & kP61) + c;
    s = (s >> 61) + (s & kP61);                             // s < 2^63  ->  s <= p + 3
    return s >= kP61 ? s - kP61 : s;
}

// y mod m for y < 2^61 with magic = floor((2^64 - 1) / m): one multiply-high, one correction.
__device__ __forceinline__ uint32_t mod_small(uint64_t y, uint32_t m, uint64_t magic)
{
    const uint64_t q = __umul64hi(y, magic);
    uint32_t r = (uint32_t)(y - q * (uint64_t)m);
    return r >= m ? r - m : r;
}

// coefficients of one sketch row: {a, b, c3, c2, c1, c0}
__device__ __forceinline__ uint32_t bucket_of(const uint64_t *c, uint32_t j, uint32_t m,
                                              uint64_t magic)
{
    return mod_small(mul_add_mod_p(c[0], j, c[1]), m, magic);
}

// true when the sign is -1 (odd residue of the cubic)
__device__ __forceinline__ bool sign_is_negative(const uint64_t *c, uint32_t j)
{
    uint64_t g = mul_add_mod_p(c[2], j, c[3]);
    g = mul_add_mod_p(g, j, c[4]);
    g = mul_add_mod_p(g, j, c[5]);
    return (g & 1ull) != 0;
}

}  // namespace fda
#endif
