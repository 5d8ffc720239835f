// Goldilocks field arithmetic for device (and host) code: p = 2^64 - 2^32 + 1.
//
// Elements are canonical uint64 in [0, p).  The reduction rests on 2^64 = 2^32 - 1 (mod p) and
// 2^96 = -1 (mod p): a 128-bit value hi_hi*2^96 + hi_lo*2^64 + lo is congruent to
// lo - hi_hi + hi_lo*(2^32 - 1).
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define GL_HD __host__ __device__ __forceinline__
#define GL_D __device__ __forceinline__
#else
#define GL_HD inline
#endif

namespace gl {

constexpr uint64_t P = 0xFFFFFFFF00000001ULL;
constexpr uint64_t EPS = 0xFFFFFFFFULL;          // 2^64 mod p = 2^32 - 1

GL_HD uint64_t add(uint64_t a, uint64_t b)
{
    uint64_t s = a + b;
    if (s < a) s += EPS;        // wrapped past 2^64: the lost 2^64 is worth 2^32 - 1; stays < p
    if (s >= P) s -= P;
    return s;
}

GL_HD uint64_t sub(uint64_t a, uint64_t b)
{
    uint64_t d = a - b;
    if (a < b) d += P;          // wraps back into [1, p)
    return d;
}

GL_HD uint64_t neg(uint64_t a) { return a == 0 ? 0 : P - a; }

// (hi, lo) = hi*2^64 + lo, any 128-bit value -> canonical
GL_HD uint64_t reduce128(uint64_t hi, uint64_t lo)
{
    uint64_t hi_hi = hi >> 32, hi_lo = hi & EPS;
    uint64_t t0 = lo - hi_hi;
    if (lo < hi_hi) t0 -= EPS;              // borrowed 2^64: add p instead, i.e. subtract 2^32 - 1
    uint64_t t1 = hi_lo * EPS;              // < 2^64
    uint64_t r = t0 + t1;
    if (r < t1) r += EPS;                   // cannot wrap twice
    if (r >= P) r -= P;
    return r;
}

#if defined(__CUDA_ARCH__)
// 64 x 64 -> 128 schoolbook product from 32-bit multiply-low / multiply-high with carry chains.
GL_D void mul_wide(uint64_t a, uint64_t b, uint64_t& hi, uint64_t& lo)
{
    uint32_t a0 = (uint32_t)a, a1 = (uint32_t)(a >> 32);
    uint32_t b0 = (uint32_t)b, b1 = (uint32_t)(b >> 32);
    uint32_t r0, r1, r2, r3;
    asm("{\n\t"
        "mul.lo.u32      %0, %4, %6;\n\t"
        "mul.hi.u32      %1, %4, %6;\n\t"
        "mad.lo.cc.u32   %1, %4, %7, %1;\n\t"
        "madc.hi.u32     %2, %4, %7, 0;\n\t"
        "mad.lo.cc.u32   %1, %5, %6, %1;\n\t"
        "madc.hi.cc.u32  %2, %5, %6, %2;\n\t"
        "addc.u32        %3, 0, 0;\n\t"
        "mad.lo.cc.u32   %2, %5, %7, %2;\n\t"
        "madc.hi.u32     %3, %5, %7, %3;\n\t"
        "}"
        : "=&r"(r0), "=&r"(r1), "=&r"(r2), "=&r"(r3)
        : "r"(a0), "r"(a1), "r"(b0), "r"(b1));
    lo = ((uint64_t)r1 << 32) | r0;
    hi = ((uint64_t)r3 << 32) | r2;
}
#else
inline void mul_wide(uint64_t a, uint64_t b, uint64_t& hi, uint64_t& lo)
{
    unsigned __int128 w = (unsigned __int128)a * b;
    lo = (uint64_t)w;
    hi = (uint64_t)(w >> 64);
}
#endif

GL_HD uint64_t mul(uint64_t a, uint64_t b)
{
    uint64_t hi, lo;
    mul_wide(a, b, hi, lo);
    return reduce128(hi, lo);
}

// signed 64-bit integer (|s| < 2^63 < p) -> canonical element
GL_HD uint64_t from_i64(int64_t s) { return s >= 0 ? (uint64_t)s : (uint64_t)s + P; }

// x * 2^sh for 0 <= sh < 64, x canonical
GL_HD uint64_t shl(uint64_t x, int sh)
{
    if (sh == 0) return x;
    return reduce128(x >> (64 - sh), x << sh);
}

// Representative s of e (s = e or e - p) that splits as s = hi*2^32 + lo with BOTH halves
// signed 32-bit: lets signed 32 x 32 -> 64 multiply-adds consume eq weights directly.
GL_HD void balanced_halves(uint64_t e, int32_t& lo, int32_t& hi)
{
    int64_t s = (e <= 0x7FFFFFFF7FFFFFFFULL) ? (int64_t)e : (int64_t)(e - P);
    lo = (int32_t)(uint32_t)(uint64_t)s;
    hi = (int32_t)((s - (int64_t)lo) >> 32);
}

GL_HD uint64_t mix64(uint64_t z)
{
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

// public-coin challenge: see imm_challenge in imm.h
GL_HD uint64_t challenge(uint64_t seed, uint64_t proof_id, uint32_t domain, uint32_t index)
{
    const uint64_t G = 0x9E3779B97F4A7C15ULL;
    uint64_t key = mix64(mix64(seed + G) + G * (proof_id + 1));
    uint64_t ctr = ((uint64_t)domain << 32) | index;
    uint64_t x = mix64(key + G * (ctr + 1));
    return x >= P ? x - P : x;
}

}  // namespace gl
