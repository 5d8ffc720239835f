// SHA-256 (FIPS 180-4) for device and host code of libimm: the compression function and a helper
// for short messages.  Used by the hash commitments (imm_commit.cu), by the transcript hashing of
// the non-interactive proof (imm_kernels.cu) and by the host verifier (imm_api.cu).
#pragma once

#include <stdint.h>

namespace imm_sha {

// FIPS 180-4, 4.2.2: the first 32 bits of the fractional parts of the cube roots of the first 64 primes
#define IMM_SHA256_K_WORDS                                                                              \
    0x428a2f98u, 0x71374491u, 0xb5c0fbcfu, 0xe9b5dba5u, 0x3956c25bu, 0x59f111f1u, 0x923f82a4u, 0xab1c5ed5u, \
    0xd807aa98u, 0x12835b01u, 0x243185beu, 0x550c7dc3u, 0x72be5d74u, 0x80deb1feu, 0x9bdc06a7u, 0xc19bf174u, \
    0xe49b69c1u, 0xefbe4786u, 0x0fc19dc6u, 0x240ca1ccu, 0x2de92c6fu, 0x4a7484aau, 0x5cb0a9dcu, 0x76f988dau, \
    0x983e5152u, 0xa831c66du, 0xb00327c8u, 0xbf597fc7u, 0xc6e00bf3u, 0xd5a79147u, 0x06ca6351u, 0x14292967u, \
    0x27b70a85u, 0x2e1b2138u, 0x4d2c6dfcu, 0x53380d13u, 0x650a7354u, 0x766a0abbu, 0x81c2c92eu, 0x92722c85u, \
    0xa2bfe8a1u, 0xa81a664bu, 0xc24b8b70u, 0xc76c51a3u, 0xd192e819u, 0xd6990624u, 0xf40e3585u, 0x106aa070u, \
    0x19a4c116u, 0x1e376c08u, 0x2748774cu, 0x34b0bcb5u, 0x391c0cb3u, 0x4ed8aa4au, 0x5b9cca4fu, 0x682e6ff3u, \
    0x748f82eeu, 0x78a5636fu, 0x84c87814u, 0x8cc70208u, 0x90befffau, 0xa4506cebu, 0xbef9a3f7u, 0xc67178f2u

static __constant__ uint32_t K_dev[64] = {IMM_SHA256_K_WORDS};
static const uint32_t K_host[64] = {IMM_SHA256_K_WORDS};

__host__ __device__ __forceinline__ uint32_t kc(int t)
{
#ifdef __CUDA_ARCH__
    return K_dev[t];
#else
    return K_host[t];
#endif
}

__host__ __device__ __forceinline__ uint32_t rotr(uint32_t x, int s)
{
#ifdef __CUDA_ARCH__
    return __funnelshift_r(x, x, s);
#else
    return (x >> s) | (x << (32 - s));
#endif
}

__host__ __device__ __forceinline__ void iv(uint32_t (&h)[8])    // FIPS 180-4, 5.3.3: square roots of the first 8 primes
{
    h[0] = 0x6a09e667u; h[1] = 0xbb67ae85u; h[2] = 0x3c6ef372u; h[3] = 0xa54ff53au;
    h[4] = 0x510e527fu; h[5] = 0x9b05688cu; h[6] = 0x1f83d9abu; h[7] = 0x5be0cd19u;
}

// a + b on the multiply-add pipe: a * one + b with `one` a register the compiler cannot see through
// (it holds 1).  The rotates and three-input logic of SHA-256 fill the integer ALU pipe, which
// issues at half rate; the adds, written as multiply-adds, run beside them on the other pipe.
__host__ __device__ __forceinline__ uint32_t add_m(uint32_t a, uint32_t b, uint32_t one)
{
#ifdef __CUDA_ARCH__
    uint32_t d;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(one), "r"(b));
    return d;
#else
    return a * one + b;
#endif
}

// One round (FIPS 180-4, 6.2.2, step 3) on the working variables, with w + K already added.
#define IMM_SHA_ROUND(kw)                                                          \
    do {                                                                           \
        const uint32_t S1 = rotr(e, 6) ^ rotr(e, 11) ^ rotr(e, 25);                \
        const uint32_t ch = (e & f) ^ (~e & g);                                    \
        const uint32_t t1 = add_m(add_m(add_m(hh, (kw), one), ch, one), S1, one);  \
        const uint32_t S0 = rotr(a, 2) ^ rotr(a, 13) ^ rotr(a, 22);                \
        const uint32_t maj = (a & b) ^ (a & c) ^ (b & c);                          \
        hh = g; g = f; f = e; e = add_m(d, t1, one);                               \
        d = c; c = b; b = a; a = add_m(add_m(S0, maj, one), t1, one);              \
    } while (0)

// One compression (FIPS 180-4, 6.2.2).  w holds the sixteen message words and is overwritten by
// the rolling message schedule.  `one` must hold 1 (see add_m).  Rounds 0..15 are straight-line
// code; rounds 16..63 are three trips through one sixteen-round body, so that the whole function
// stays small enough for the instruction caches close to the schedulers (fully unrolled, the
// warps of an SM stream 24 KB of code per compression and stall on instruction fetch).
__host__ __device__ __forceinline__ void compress(uint32_t (&h)[8], uint32_t (&w)[16], uint32_t one)
{
    uint32_t a = h[0], b = h[1], c = h[2], d = h[3], e = h[4], f = h[5], g = h[6], hh = h[7];
#pragma unroll
    for (int t = 0; t < 16; t++) IMM_SHA_ROUND(add_m(w[t], kc(t), one));
#pragma unroll 1
    for (int base = 16; base < 64; base += 16) {
#pragma unroll
        for (int j = 0; j < 16; j++) {
            const uint32_t w15 = w[(j + 1) & 15], w2 = w[(j + 14) & 15];
            const uint32_t s0 = rotr(w15, 7) ^ rotr(w15, 18) ^ (w15 >> 3);
            const uint32_t s1 = rotr(w2, 17) ^ rotr(w2, 19) ^ (w2 >> 10);
            w[j] = add_m(add_m(w[j], s0, one), add_m(w[(j + 9) & 15], s1, one), one);
            IMM_SHA_ROUND(add_m(w[j], kc(base + j), one));
        }
    }
    h[0] += a; h[1] += b; h[2] += c; h[3] += d; h[4] += e; h[5] += f; h[6] += g; h[7] += hh;
}

#undef IMM_SHA_ROUND

// SHA-256 of a short message held in addressable memory (a few blocks: statement and transcript
// hashes, final commitment hash).  out = the eight state words.
__host__ __device__ inline void sha256_short(const uint8_t* msg, uint32_t len, uint32_t (&out)[8], uint32_t one)
{
    iv(out);
    const uint32_t nblocks = (len + 9 + 63) / 64;          // 0x80 and the 64-bit length must fit
    for (uint32_t blk = 0; blk < nblocks; blk++) {
        uint32_t w[16];
        for (int t = 0; t < 16; t++) {
            uint32_t v = 0;
            for (int q = 0; q < 4; q++) {
                const uint32_t i = blk * 64 + 4 * t + q;
                uint32_t byte = 0;
                if (i < len) byte = msg[i];
                else if (i == len) byte = 0x80;
                v = (v << 8) | byte;
            }
            w[t] = v;
        }
        if (blk == nblocks - 1) w[15] = len * 8;           // (w[14], the high length word, is already 0)
        compress(out, w, one);
    }
}

// digest words -> the usual 32 bytes
__host__ __device__ inline void digest_bytes(const uint32_t (&h)[8], uint8_t* out)
{
    for (int wd = 0; wd < 8; wd++)
        for (int q = 0; q < 4; q++) out[4 * wd + q] = (uint8_t)(h[wd] >> (24 - 8 * q));
}

struct Digest { uint32_t h[8]; };             // the eight state words (big-endian when serialised)

#ifdef __CUDACC__
// Inner node of the Merkle tree of RFC 6962: SHA-256(0x01 || left || right), 65 bytes, two compressions
__device__ __forceinline__ void node_hash(const uint32_t (&l)[8], const uint32_t (&r)[8], uint32_t (&out)[8],
                                          uint32_t one)
{
    uint32_t w[16];
    w[0] = 0x01000000u | (l[0] >> 8);
#pragma unroll
    for (int i = 1; i < 8; i++) w[i] = (l[i - 1] << 24) | (l[i] >> 8);
    w[8] = (l[7] << 24) | (r[0] >> 8);
#pragma unroll
    for (int i = 1; i < 8; i++) w[8 + i] = (r[i - 1] << 24) | (r[i] >> 8);
    iv(out);
    compress(out, w, one);
    w[0] = (r[7] << 24) | 0x00800000u;
#pragma unroll
    for (int i = 1; i < 15; i++) w[i] = 0;
    w[15] = 65 * 8;
    compress(out, w, one);
}

// Folds the `count` digests in sd (shared memory, count <= blockDim.x) to one in sd[0]: neighbours
// pair level by level, an unpaired last digest moves up unchanged (the tree of RFC 6962).  Every
// thread of the block must call it.
__device__ __forceinline__ void fold(Digest* sd, int count, uint32_t one)
{
    const int t = threadIdx.x;
    while (count > 1) {
        const int half = count >> 1;
        uint32_t out[8];
        const bool pair = t < half, lift = (count & 1) && t == half;
        if (pair) node_hash(sd[2 * t].h, sd[2 * t + 1].h, out, one);
        else if (lift) {
#pragma unroll
            for (int i = 0; i < 8; i++) out[i] = sd[count - 1].h[i];
        }
        __syncthreads();
        if (pair || lift) {
#pragma unroll
            for (int i = 0; i < 8; i++) sd[t].h[i] = out[i];
        }
        __syncthreads();
        count = (count + 1) >> 1;
    }
}

#endif  // __CUDACC__

}  // namespace imm_sha
