// Element-wise links between proved products (sm_100a) and their C ABI (declared in imm.h).
//
//   imm_requant_check      H == clamp(floor((C + rnd) / 2^shift), lo, hi), entry by entry
//   imm_gated_link_check   H == clamp(floor((act[q(G)] * q(U) + rnd2) / 2^shift2), lo, hi): the activation table
//                          and gating step between the gate / up and the down projection of an MLP
//
// The sumcheck proofs cover the matrix products of the reference execution one at a time; the map
// that turns one product's int32 output into the next product's int8 input is checked by
// recomputing it over the opened tensors.  That is a single streaming pass: 4 bytes of C (of G and of
// U) and 1 byte of H per entry, each read once, a handful of integer instructions per entry -- bound
// by HBM.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/imm.h"
#include "imm_kernels.h"

namespace imm_glue {

constexpr int THREADS = 256;
constexpr int EPT = 16;                        // entries per thread and row: 64 bytes of C, 16 bytes of H

struct Link {
    const int32_t* C;
    const int8_t* H;
    int64_t ldc, ldh;                          // elements
    int32_t rows, cols;
    int32_t shift, rnd, lo, hi;
    unsigned long long* result;                // [0] differing entries, [1] row-major index of the first
};

struct u32x8 { uint32_t v[8]; };

__device__ __forceinline__ u32x8 ld_stream_v8(const void* p)          // 256-bit streaming load, 32-byte aligned
{
    u32x8 r;
    asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r.v[0]), "=r"(r.v[1]), "=r"(r.v[2]), "=r"(r.v[3]), "=r"(r.v[4]), "=r"(r.v[5]),
                   "=r"(r.v[6]), "=r"(r.v[7])
                 : "l"(p));
    return r;
}

__device__ __forceinline__ uint4 ld_stream_v4(const void* p)          // 128-bit streaming load, 16-byte aligned
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// floor((c + rnd) / 2^shift) without leaving 32 bits: c = q 2^shift + rem with 0 <= rem < 2^shift, and
// rem + rnd < 2^(shift+1) <= 2^31.  The right shift of a negative int32 is arithmetic, i.e. the floor.
__device__ __forceinline__ int32_t requant(int32_t c, int shift, int32_t mask, int32_t rnd, int32_t lo, int32_t hi)
{
    const int32_t q = (c >> shift) + (((c & mask) + rnd) >> shift);
    return max(lo, min(hi, q));
}

// One row's 16 entries of a thread: 16 words of C, 4 words of H (entry e is byte e % 4 of word e / 4).
__device__ __forceinline__ void compare16(const uint32_t (&c)[16], const uint32_t (&h)[4], const Link& L, int32_t mask,
                                          uint64_t base, uint32_t& count, uint64_t& first)
{
#pragma unroll
    for (int w = 0; w < 4; w++) {
        uint32_t packed = 0;
#pragma unroll
        for (int b = 0; b < 4; b++)
            packed |= ((uint32_t)requant((int32_t)c[4 * w + b], L.shift, mask, L.rnd, L.lo, L.hi) & 0xFFu) << (8 * b);
        const uint32_t diff = packed ^ h[w];
        if (diff) {                                        // rare: an honest link never gets here
#pragma unroll
            for (int b = 0; b < 4; b++)
                if ((diff >> (8 * b)) & 0xFFu) {
                    count++;
                    first = min(first, base + 4 * w + b);
                }
        }
    }
}

// VL 2: rows of C 32-byte aligned (256-bit loads); VL 1: 16-byte aligned; both need rows of H 16-byte
// aligned.  VL 0: element-wise loads.  blockDim = (TX, TY), TX * TY = THREADS: TX threads side by
// side cover TX * 16 columns, TY rows at a time; a block walks `rows_per_block` rows.
template <int VL>
__global__ void __launch_bounds__(THREADS) requant_check_kernel(const Link L, int rows_per_block)
{
    const int col = (blockIdx.x * blockDim.x + threadIdx.x) * EPT;
    const int nvalid = min(EPT, L.cols - col);             // <= 0: this thread has no columns
    const int r_begin = blockIdx.y * rows_per_block + threadIdx.y;
    const int r_end = min(L.rows, (int)(blockIdx.y + 1) * rows_per_block);
    const int32_t mask = (int32_t)((1u << L.shift) - 1u);
    uint32_t count = 0;
    uint64_t first = ~0ull;

    if (nvalid == EPT && VL > 0) {
        for (int r = r_begin; r < r_end; r += 2 * blockDim.y) {     // two rows in flight per thread
            uint32_t c[2][16], h[2][4];
#pragma unroll
            for (int u = 0; u < 2; u++) {
                const int row = min(r + u * (int)blockDim.y, r_end - 1);      // clamped: compared only if real
                const char* pc = (const char*)(L.C + (int64_t)row * L.ldc + col);
                if (VL == 2) {
                    const u32x8 a = ld_stream_v8(pc), b = ld_stream_v8(pc + 32);
#pragma unroll
                    for (int i = 0; i < 8; i++) { c[u][i] = a.v[i]; c[u][8 + i] = b.v[i]; }
                } else {
#pragma unroll
                    for (int i = 0; i < 4; i++) {
                        const uint4 v = ld_stream_v4(pc + 16 * i);
                        c[u][4 * i] = v.x; c[u][4 * i + 1] = v.y; c[u][4 * i + 2] = v.z; c[u][4 * i + 3] = v.w;
                    }
                }
                const uint4 hv = ld_stream_v4(L.H + (int64_t)row * L.ldh + col);
                h[u][0] = hv.x; h[u][1] = hv.y; h[u][2] = hv.z; h[u][3] = hv.w;
            }
#pragma unroll
            for (int u = 0; u < 2; u++) {
                const int row = r + u * (int)blockDim.y;
                if (row < r_end) compare16(c[u], h[u], L, mask, (uint64_t)row * (uint64_t)L.cols + (uint64_t)col, count, first);
            }
        }
    } else if (nvalid > 0) {                               // ragged last chunk of a row, or unaligned rows
        for (int r = r_begin; r < r_end; r += blockDim.y) {
            const int32_t* pc = L.C + (int64_t)r * L.ldc + col;
            const int8_t* ph = L.H + (int64_t)r * L.ldh + col;
            for (int e = 0; e < nvalid; e++) {
                const int32_t want = requant(pc[e], L.shift, mask, L.rnd, L.lo, L.hi);
                if (want != (int32_t)ph[e]) {
                    count++;
                    first = min(first, (uint64_t)r * (uint64_t)L.cols + (uint64_t)(col + e));
                }
            }
        }
    }
    // one pair of atomics per warp that saw a difference
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        count += __shfl_xor_sync(0xFFFFFFFFu, count, o);
        const uint64_t other = __shfl_xor_sync(0xFFFFFFFFu, first, o);
        first = min(first, other);
    }
    const int lane = (threadIdx.y * blockDim.x + threadIdx.x) & 31;
    if (lane == 0 && count) {
        atomicAdd(L.result, (unsigned long long)count);
        atomicMin(L.result + 1, (unsigned long long)first);
    }
}

// ---- activation table and gated product (gate, up -> input of the down projection) ----

struct ActTable { int8_t v[256]; };                // v[x + 128] answers x

struct GatedLink {
    const int32_t* G;
    const int32_t* U;                              // nullptr: the activation alone
    const int8_t* H;
    int64_t ldg, ldu, ldh;
    int32_t rows, cols;
    int32_t shift, rnd, shift2, rnd2, lo, hi;
    unsigned long long* result;
};

__device__ __forceinline__ int32_t gated_entry(int32_t g, int32_t u, bool gated, const int8_t* act, const GatedLink& L,
                                               int32_t mask, int32_t mask2)
{
    const int32_t a = (int32_t)act[requant(g, L.shift, mask, L.rnd, -128, 127) + 128];
    if (!gated) return a;
    const int32_t p = a * requant(u, L.shift, mask, L.rnd, -128, 127);      // |p| <= 2^14
    return requant(p, L.shift2, mask2, L.rnd2, L.lo, L.hi);
}

// VEC: rows of G, U and H 16-byte aligned (128-bit loads); otherwise element-wise loads.  Same block
// shape as requant_check_kernel: TX threads side by side cover TX * 16 columns, TY rows at a time.
template <bool VEC, bool GATED>
__global__ void __launch_bounds__(THREADS) gated_link_kernel(const GatedLink L, const ActTable table, int rows_per_block)
{
    __shared__ int8_t act[256];
    const int flat = threadIdx.y * blockDim.x + threadIdx.x;
    act[flat] = table.v[flat];                                                // THREADS == 256
    __syncthreads();
    const int col = (blockIdx.x * blockDim.x + threadIdx.x) * EPT;
    const int nvalid = min(EPT, L.cols - col);
    const int r_begin = blockIdx.y * rows_per_block + threadIdx.y;
    const int r_end = min(L.rows, (int)(blockIdx.y + 1) * rows_per_block);
    const int32_t mask = (int32_t)((1u << L.shift) - 1u), mask2 = (int32_t)((1u << L.shift2) - 1u);
    uint32_t count = 0;
    uint64_t first = ~0ull;

    if (nvalid == EPT && VEC) {
        for (int r = r_begin; r < r_end; r += blockDim.y) {
            const char* pg = (const char*)(L.G + (int64_t)r * L.ldg + col);
            const char* pu = GATED ? (const char*)(L.U + (int64_t)r * L.ldu + col) : nullptr;
            uint4 g[4], u[4];
#pragma unroll
            for (int i = 0; i < 4; i++) g[i] = ld_stream_v4(pg + 16 * i);
            if (GATED) {
#pragma unroll
                for (int i = 0; i < 4; i++) u[i] = ld_stream_v4(pu + 16 * i);
            }
            const uint4 hv = ld_stream_v4(L.H + (int64_t)r * L.ldh + col);
            const uint32_t h[4] = {hv.x, hv.y, hv.z, hv.w};
            const uint64_t base = (uint64_t)r * (uint64_t)L.cols + (uint64_t)col;
#pragma unroll
            for (int w = 0; w < 4; w++) {
                const uint32_t gw[4] = {g[w].x, g[w].y, g[w].z, g[w].w};
                const uint32_t uw[4] = {GATED ? u[w].x : 0u, GATED ? u[w].y : 0u, GATED ? u[w].z : 0u, GATED ? u[w].w : 0u};
                uint32_t packed = 0;
#pragma unroll
                for (int b = 0; b < 4; b++)
                    packed |= ((uint32_t)gated_entry((int32_t)gw[b], (int32_t)uw[b], GATED, act, L, mask, mask2) & 0xFFu) << (8 * b);
                const uint32_t diff = packed ^ h[w];
                if (diff) {
#pragma unroll
                    for (int b = 0; b < 4; b++)
                        if ((diff >> (8 * b)) & 0xFFu) { count++; first = min(first, base + 4 * w + b); }
                }
            }
        }
    } else if (nvalid > 0) {
        for (int r = r_begin; r < r_end; r += blockDim.y) {
            const int32_t* pg = L.G + (int64_t)r * L.ldg + col;
            const int32_t* pu = GATED ? L.U + (int64_t)r * L.ldu + col : nullptr;
            const int8_t* ph = L.H + (int64_t)r * L.ldh + col;
            for (int e = 0; e < nvalid; e++) {
                const int32_t want = gated_entry(pg[e], GATED ? pu[e] : 0, GATED, act, L, mask, mask2);
                if (want != (int32_t)ph[e]) { count++; first = min(first, (uint64_t)r * (uint64_t)L.cols + (uint64_t)(col + e)); }
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        count += __shfl_xor_sync(0xFFFFFFFFu, count, o);
        const uint64_t other = __shfl_xor_sync(0xFFFFFFFFu, first, o);
        first = min(first, other);
    }
    if ((flat & 31) == 0 && count) {
        atomicAdd(L.result, (unsigned long long)count);
        atomicMin(L.result + 1, (unsigned long long)first);
    }
}

}  // namespace imm_glue

extern "C" int imm_requant_check(const int32_t* d_C, const int8_t* d_H, int64_t rows, int64_t cols, int64_t ldc,
                                 int64_t ldh, int shift, int32_t rnd, int32_t lo, int32_t hi, uint64_t* d_result,
                                 void* stream)
{
    using namespace imm_glue;
    if (!d_C || !d_H || !d_result) return IMM_ERR_ARG;
    if (shift < 0 || shift > 30 || rnd < 0 || (int64_t)rnd >= ((int64_t)1 << shift) || lo < -128 || hi > 127 || lo > hi)
        return IMM_ERR_ARG;
    if (rows <= 0 || cols <= 0 || rows > ((int64_t)1 << 20) || cols > ((int64_t)1 << 20) || ldc < cols || ldh < cols)
        return IMM_ERR_SHAPE;
    if ((uintptr_t)d_C % 4 != 0 || (uintptr_t)d_result % 8 != 0) return IMM_ERR_ALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(d_result, 0, 8, st) != cudaSuccess) return IMM_ERR_CUDA;
    if (cudaMemsetAsync(d_result + 1, 0xFF, 8, st) != cudaSuccess) return IMM_ERR_CUDA;

    Link L{d_C, d_H, ldc, ldh, (int32_t)rows, (int32_t)cols, shift, rnd, lo, hi, (unsigned long long*)d_result};
    // block shape: TX threads across the columns (a power of two covering the row if it is short)
    int tx = 4;
    while (tx < THREADS && (int64_t)tx * EPT < cols) tx *= 2;
    const int ty = THREADS / tx;
    const int64_t xtiles = (cols + (int64_t)tx * EPT - 1) / ((int64_t)tx * EPT);
    // rows per block: enough blocks to fill the GPU some 16 times over, each thread at least 4 rows deep
    int64_t rpb = rows * xtiles / ((int64_t)imm::sm_count() * 16);
    const int64_t rpb_min = (int64_t)ty * 4, rpb_max = (int64_t)ty * 64;
    rpb = rpb < rpb_min ? rpb_min : rpb > rpb_max ? rpb_max : rpb;
    rpb = (rpb + ty - 1) / ty * ty;
    const int64_t ytiles = (rows + rpb - 1) / rpb;
    if (ytiles > 65535) return IMM_ERR_SHAPE;              // (cannot happen within the limits above)
    const dim3 grid((unsigned)xtiles, (unsigned)ytiles), block((unsigned)tx, (unsigned)ty);
    const bool h16 = (uintptr_t)d_H % 16 == 0 && ldh % 16 == 0;
    const int vl = !h16 ? 0 : ((uintptr_t)d_C % 32 == 0 && (ldc * 4) % 32 == 0) ? 2
                              : ((uintptr_t)d_C % 16 == 0 && (ldc * 4) % 16 == 0) ? 1 : 0;
    if (vl == 2) requant_check_kernel<2><<<grid, block, 0, st>>>(L, (int)rpb);
    else if (vl == 1) requant_check_kernel<1><<<grid, block, 0, st>>>(L, (int)rpb);
    else requant_check_kernel<0><<<grid, block, 0, st>>>(L, (int)rpb);
    return cudaGetLastError() == cudaSuccess ? IMM_OK : IMM_ERR_CUDA;
}

extern "C" int imm_gated_link_check(const int32_t* d_G, const int32_t* d_U, const int8_t* d_H, int64_t rows, int64_t cols,
                                    int64_t ldg, int64_t ldu, int64_t ldh, const int8_t* act_host, int shift, int32_t rnd,
                                    int shift2, int32_t rnd2, int32_t lo, int32_t hi, uint64_t* d_result, void* stream)
{
    using namespace imm_glue;
    if (!d_G || !d_H || !d_result || !act_host) return IMM_ERR_ARG;
    if (shift < 0 || shift > 30 || rnd < 0 || (int64_t)rnd >= ((int64_t)1 << shift)) return IMM_ERR_ARG;
    const bool gated = d_U != nullptr;
    if (!gated) { shift2 = 0; rnd2 = 0; lo = -128; hi = 127; ldu = ldg; }
    if (shift2 < 0 || shift2 > 14 || rnd2 < 0 || rnd2 >= (1 << shift2) || lo < -128 || hi > 127 || lo > hi) return IMM_ERR_ARG;
    if (rows <= 0 || cols <= 0 || rows > ((int64_t)1 << 20) || cols > ((int64_t)1 << 20) || ldg < cols || ldu < cols || ldh < cols)
        return IMM_ERR_SHAPE;
    if ((uintptr_t)d_G % 4 != 0 || (gated && (uintptr_t)d_U % 4 != 0) || (uintptr_t)d_result % 8 != 0) return IMM_ERR_ALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(d_result, 0, 8, st) != cudaSuccess) return IMM_ERR_CUDA;
    if (cudaMemsetAsync(d_result + 1, 0xFF, 8, st) != cudaSuccess) return IMM_ERR_CUDA;

    GatedLink L{d_G, d_U, d_H, ldg, ldu, ldh, (int32_t)rows, (int32_t)cols, shift, rnd, shift2, rnd2, lo, hi,
                (unsigned long long*)d_result};
    ActTable table;
    for (int i = 0; i < 256; i++) table.v[i] = act_host[i];
    int tx = 4;
    while (tx < THREADS && (int64_t)tx * EPT < cols) tx *= 2;
    const int ty = THREADS / tx;
    const int64_t xtiles = (cols + (int64_t)tx * EPT - 1) / ((int64_t)tx * EPT);
    int64_t rpb = rows * xtiles / ((int64_t)imm::sm_count() * 16);
    const int64_t rpb_min = (int64_t)ty * 4, rpb_max = (int64_t)ty * 64;
    rpb = rpb < rpb_min ? rpb_min : rpb > rpb_max ? rpb_max : rpb;
    rpb = (rpb + ty - 1) / ty * ty;
    const int64_t ytiles = (rows + rpb - 1) / rpb;
    if (ytiles > 65535) return IMM_ERR_SHAPE;              // (cannot happen within the limits above)
    const dim3 grid((unsigned)xtiles, (unsigned)ytiles), block((unsigned)tx, (unsigned)ty);
    const bool vec = (uintptr_t)d_H % 16 == 0 && ldh % 16 == 0 && (uintptr_t)d_G % 16 == 0 && ldg % 4 == 0 &&
                     (!gated || ((uintptr_t)d_U % 16 == 0 && ldu % 4 == 0));
    if (gated) {
        if (vec) gated_link_kernel<true, true><<<grid, block, 0, st>>>(L, table, (int)rpb);
        else gated_link_kernel<false, true><<<grid, block, 0, st>>>(L, table, (int)rpb);
    } else {
        if (vec) gated_link_kernel<true, false><<<grid, block, 0, st>>>(L, table, (int)rpb);
        else gated_link_kernel<false, false><<<grid, block, 0, st>>>(L, table, (int)rpb);
    }
    return cudaGetLastError() == cudaSuccess ? IMM_OK : IMM_ERR_CUDA;
}
