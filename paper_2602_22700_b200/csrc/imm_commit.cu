// Hash commitments of libimm (sm_100a) and their C ABI (declared in imm.h).
//
//   imm_commit   c = Hash(m || r) (Section 2.1 of the paper; the model and response commitments of
//                Algorithm 1) for a batch of device-resident messages.
//
// Hash is SHA-256 (FIPS 180-4) in a tree mode, so that gigabytes hash in parallel: the message is
// cut into 4096-byte leaves and hashed as the Merkle tree of RFC 6962 (leaf = H(0x00 || data),
// node = H(0x01 || left || right), an unpaired last node moves up unchanged), and
// c = H(0x02 || root || le64(length) || r).
//
// SHA-256 is a serial chain of 32-bit adds, rotates and three-input logic per 64-byte block, so
// the work is bound by integer-pipe instruction issue, not by HBM: the rotates and the logic fill
// the integer ALU pipe (one warp instruction per two cycles per SM sub-partition); the adds are
// written as multiply-adds so that they issue on the other pipe.  One thread hashes one leaf
// (65 compressions); the 128 to 512 leaves of a block are then folded to one subtree root in shared
// memory, so the leaf digests never go to global memory.  Later passes fold 1024 digests per block
// until every message has one root, and a last launch forms the commitments.
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <vector>

#include "../../include/imm.h"
#include "imm_kernels.h"
#include "sha256.cuh"

namespace imm_hash {

constexpr int LEAF = IMM_COMMIT_LEAF;         // bytes per leaf
// Leaves per block of the leaf pass.  The pass is bound by the integer pipe, so an SM works through
// its resident warps at a fixed rate and a launch takes (full waves x resident warps + warps of the
// fullest SM in the last, partial wave) units; larger blocks run a few per cent faster per warp
// (measured on 4 GiB: 128 threads 852 GB/s, 256 881, 512 900) but leave a coarser tail.  The
// candidate with the lowest estimate is taken.
struct LeafChoice { int threads, blocks_per_sm; double cost; };    // blocks per SM as the registers allow
constexpr LeafChoice LEAF_CHOICES[3] = {{128, 9, 1.055}, {256, 4, 1.023}, {512, 2, 1.0}};

inline int pick_leaf_threads(const std::vector<uint64_t>& leaves)
{
    const int SM_COUNT = imm::sm_count();
    int best = LEAF_CHOICES[0].threads;
    double best_t = -1;
    for (const LeafChoice& c : LEAF_CHOICES) {
        uint64_t blocks = 0;
        for (uint64_t n : leaves) blocks += (n + c.threads - 1) / c.threads;
        const uint64_t per_wave = (uint64_t)SM_COUNT * c.blocks_per_sm;
        const uint64_t full = blocks / per_wave, rem = blocks % per_wave;
        const double warps = (double)full * c.blocks_per_sm * (c.threads / 32) +
                             (double)((rem + SM_COUNT - 1) / SM_COUNT) * (c.threads / 32);
        const double t = warps * c.cost;
        if (best_t < 0 || t < best_t) { best_t = t; best = c.threads; }
    }
    return best;
}
constexpr int NODE_THREADS = 1024;            // digests per block of a node pass
constexpr size_t ALIGN = 256;

using imm_sha::compress;
using imm_sha::iv;

using imm_sha::Digest;
using imm_sha::fold;

// A full leaf whose data is 16-byte aligned: SHA-256(0x00 || 4096 bytes), 65 compressions.  Message
// word t of a block is the last byte of little-endian data word t-1 followed by the first three
// bytes of data word t (the tag byte shifts everything by one).
__device__ __forceinline__ void leaf_hash_full(const uint4* __restrict__ src, uint32_t (&h)[8], uint32_t one)
{
    iv(h);
    uint32_t prev = 0;                         // the tag 0x00 in the top byte
#pragma unroll 1
    for (int blk = 0; blk < LEAF / 64; blk++) {
        const uint4 v0 = __ldg(src + 4 * blk), v1 = __ldg(src + 4 * blk + 1), v2 = __ldg(src + 4 * blk + 2),
                    v3 = __ldg(src + 4 * blk + 3);
        const uint32_t x[16] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w,
                                v2.x, v2.y, v2.z, v2.w, v3.x, v3.y, v3.z, v3.w};
        uint32_t w[16];
        w[0] = __byte_perm(prev, x[0], 0x3456);
#pragma unroll
        for (int t = 1; t < 16; t++) w[t] = __byte_perm(x[t - 1], x[t], 0x3456);
        prev = x[15];
        compress(h, w, one);
    }
    uint32_t w[16];
    w[0] = (prev & 0xFF000000u) | 0x00800000u;
#pragma unroll
    for (int i = 1; i < 15; i++) w[i] = 0;
    w[15] = (LEAF + 1) * 8;
    compress(h, w, one);
}

// Any leaf, byte by byte: SHA-256(0x00 || len bytes), len in [0, LEAF].  Used for the short last
// leaf of a message and for messages that are not 16-byte aligned.
__device__ __noinline__ void leaf_hash_bytes(const uint8_t* __restrict__ p, uint32_t len, uint32_t (&h)[8],
                                             uint32_t one)
{
    iv(h);
    const uint32_t total = len + 1;                        // tag + data
    const uint32_t nblocks = (total + 9 + 63) / 64;        // 0x80 and the 64-bit length must fit
    for (uint32_t blk = 0; blk < nblocks; blk++) {
        uint32_t w[16];
#pragma unroll
        for (int t = 0; t < 16; t++) {
            uint32_t v = 0;
#pragma unroll
            for (int q = 0; q < 4; q++) {
                const uint32_t i = blk * 64 + 4 * t + q;
                uint32_t byte = 0;
                if (i >= 1 && i < total) byte = p[i - 1];
                else if (i == total) byte = 0x80;
                v = (v << 8) | byte;
            }
            w[t] = v;
        }
        if (blk == nblocks - 1) w[15] = total * 8;         // (w[14], the high length word, is already 0)
        compress(h, w, one);
    }
}

// One message in one pass: `count` inputs (leaves of `msg`, or digests at `in`) in groups of the
// block size; group g of the message is block group0 + g and writes out[g].
struct PassJob {
    const uint8_t* msg;        // leaf pass: the message
    const Digest* in;          // node pass: input digests
    Digest* out;
    uint64_t nbytes;           // leaf pass
    uint64_t count;            // leaves / input digests
    uint32_t group0;
    uint32_t one;              // 1: the multiplier of the multiply-add form of the adds (see add_m)
};

struct FinalJob {
    const Digest* root;
    uint64_t nbytes;
    uint8_t r[32];
    int32_t r_len;
    uint32_t one;              // 1 (see add_m)
};

__device__ __forceinline__ int find_pass_job(const PassJob* jobs, int njobs, uint32_t block)
{
    int lo = 0, hi = njobs - 1;                // last job whose group0 <= block
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (jobs[mid].group0 <= block) lo = mid;
        else hi = mid - 1;
    }
    return lo;
}

template <int LEAF_THREADS>
__global__ void __launch_bounds__(LEAF_THREADS) commit_leaf_kernel(const PassJob* jobs, int njobs)
{
    __shared__ Digest sd[LEAF_THREADS];
    __shared__ int s_job;
    if (threadIdx.x == 0) s_job = find_pass_job(jobs, njobs, blockIdx.x);
    __syncthreads();
    const PassJob jb = jobs[s_job];
    const uint64_t first = (uint64_t)(blockIdx.x - jb.group0) * LEAF_THREADS;
    const uint64_t remaining = jb.count - first;
    const int count = remaining < LEAF_THREADS ? (int)remaining : LEAF_THREADS;
    const uint64_t leaf = first + threadIdx.x;
    if ((int)threadIdx.x < count) {
        const uint64_t off = leaf * LEAF;
        const uint64_t left = jb.nbytes - off;             // (an empty message: one leaf of length 0)
        uint32_t h[8];
        if (left >= LEAF && ((uintptr_t)jb.msg & 15) == 0) leaf_hash_full((const uint4*)(jb.msg + off), h, jb.one);
        else leaf_hash_bytes(jb.msg + off, left < LEAF ? (uint32_t)left : LEAF, h, jb.one);
#pragma unroll
        for (int i = 0; i < 8; i++) sd[threadIdx.x].h[i] = h[i];
    }
    __syncthreads();
    fold(sd, count, jb.one);
    if (threadIdx.x < 8) jb.out[blockIdx.x - jb.group0].h[threadIdx.x] = sd[0].h[threadIdx.x];
}

__global__ void __launch_bounds__(NODE_THREADS) commit_node_kernel(const PassJob* jobs, int njobs)
{
    __shared__ Digest sd[NODE_THREADS];
    __shared__ int s_job;
    if (threadIdx.x == 0) s_job = find_pass_job(jobs, njobs, blockIdx.x);
    __syncthreads();
    const PassJob jb = jobs[s_job];
    const uint64_t first = (uint64_t)(blockIdx.x - jb.group0) * NODE_THREADS;
    const uint64_t remaining = jb.count - first;
    const int count = remaining < NODE_THREADS ? (int)remaining : NODE_THREADS;
    if ((int)threadIdx.x < count) sd[threadIdx.x] = jb.in[first + threadIdx.x];
    __syncthreads();
    fold(sd, count, jb.one);
    if (threadIdx.x < 8) jb.out[blockIdx.x - jb.group0].h[threadIdx.x] = sd[0].h[threadIdx.x];
}

// c = SHA-256(0x02 || root || le64(nbytes) || r): 41 or 73 bytes, one or two compressions.  One thread
// per message.
__global__ void commit_final_kernel(const FinalJob* jobs, int njobs, uint8_t* digests, uint8_t* roots)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= njobs) return;
    const FinalJob& jb = jobs[i];
    uint8_t m[80];
    m[0] = 0x02;
    uint32_t root[8];
    for (int wd = 0; wd < 8; wd++) root[wd] = jb.root->h[wd];
    imm_sha::digest_bytes(root, m + 1);
    for (int q = 0; q < 8; q++) m[33 + q] = (uint8_t)(jb.nbytes >> (8 * q));
    for (int q = 0; q < jb.r_len; q++) m[41 + q] = jb.r[q];
    uint32_t h[8];
    imm_sha::sha256_short(m, 41 + (uint32_t)jb.r_len, h, jb.one);
    for (int wd = 0; wd < 8; wd++)
        for (int q = 0; q < 4; q++) {
            digests[(size_t)i * 32 + 4 * wd + q] = (uint8_t)(h[wd] >> (24 - 8 * q));
            if (roots) roots[(size_t)i * 32 + 4 * wd + q] = (uint8_t)(jb.root->h[wd] >> (24 - 8 * q));
        }
}

// ------------------------------------------------------------------------------ host planning

size_t align_up(size_t v) { return (v + ALIGN - 1) / ALIGN * ALIGN; }

struct Plan {
    int status = IMM_OK;
    // pass 0 is the leaf pass; passes[p] lists the messages that still have more than one digest
    struct Entry { int msg; uint64_t count; uint64_t groups; size_t in_off, out_off; };
    std::vector<std::vector<Entry>> passes;
    std::vector<size_t> root_off;              // where each message's root ends up
    std::vector<size_t> pass_hdr_off;          // PassJob arrays in the header
    int leaf_threads = 128;
    size_t final_hdr_off = 0, header_bytes = 0, total_bytes = 0;
};

Plan make_plan(const imm_commit_desc* descs, int n)
{
    Plan p;
    if (!descs || n <= 0 || n > IMM_COMMIT_MAX_MESSAGES) { p.status = IMM_ERR_ARG; return p; }
    std::vector<uint64_t> count(n);
    std::vector<size_t> cur(n, 0);
    for (int i = 0; i < n; i++) {
        if (descs[i].nbytes > 0 && !descs[i].msg) { p.status = IMM_ERR_ARG; return p; }
        if (descs[i].r_len != 0 && descs[i].r_len != 32) { p.status = IMM_ERR_ARG; return p; }
        if (descs[i].nbytes > IMM_COMMIT_MAX_BYTES) { p.status = IMM_ERR_LIMIT; return p; }
        count[i] = descs[i].nbytes == 0 ? 1 : (descs[i].nbytes + LEAF - 1) / LEAF;
    }
    p.leaf_threads = pick_leaf_threads(count);
    // digest arrays after the header; sizes first, offsets are rebased once the header size is known
    size_t dig = 0;
    p.root_off.assign(n, 0);
    for (int pass = 0;; pass++) {
        const uint64_t per = pass == 0 ? (uint64_t)p.leaf_threads : NODE_THREADS;
        std::vector<Plan::Entry> es;
        uint64_t groups_total = 0;
        for (int i = 0; i < n; i++) {
            if (pass > 0 && count[i] <= 1) continue;
            Plan::Entry e;
            e.msg = i;
            e.count = count[i];
            e.groups = (count[i] + per - 1) / per;
            e.in_off = cur[i];
            e.out_off = dig;
            dig += (size_t)e.groups * sizeof(Digest);
            cur[i] = e.out_off;
            count[i] = e.groups;
            p.root_off[i] = e.out_off;
            groups_total += e.groups;
            es.push_back(e);
        }
        if (es.empty()) break;
        if (groups_total > 0x7FFFFFFFull) { p.status = IMM_ERR_LIMIT; return p; }
        p.passes.push_back(es);
    }
    size_t hdr = 0;
    for (const auto& es : p.passes) {
        p.pass_hdr_off.push_back(hdr);
        hdr = align_up(hdr + es.size() * sizeof(PassJob));
    }
    p.final_hdr_off = hdr;
    hdr = align_up(hdr + (size_t)n * sizeof(FinalJob));
    p.header_bytes = hdr;
    p.total_bytes = hdr + align_up(dig);
    return p;
}

}  // namespace imm_hash

extern "C" {

using namespace imm_hash;

size_t imm_commit_workspace(const imm_commit_desc* descs_host, int n)
{
    Plan p = make_plan(descs_host, n);
    return p.status == IMM_OK ? p.total_bytes : 0;
}

int imm_commit_launches(const imm_commit_desc* descs_host, int n)
{
    Plan p = make_plan(descs_host, n);
    return p.status == IMM_OK ? (int)p.passes.size() + 1 : 0;
}

int imm_commit(const imm_commit_desc* descs_host, int n, uint8_t* d_digests, uint8_t* d_roots,
               void* d_ws, size_t ws_bytes, void* stream)
{
    if (!d_digests || !d_ws) return IMM_ERR_ARG;
    Plan p = make_plan(descs_host, n);
    if (p.status != IMM_OK) return p.status;
    if ((uintptr_t)d_ws % ALIGN != 0) return IMM_ERR_ALIGN;
    if (ws_bytes < p.total_bytes) return IMM_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    char* base = (char*)d_ws;
    char* digs = base + p.header_bytes;

    std::vector<char> hdr(p.header_bytes, 0);
    std::vector<uint32_t> blocks(p.passes.size(), 0);
    for (size_t ps = 0; ps < p.passes.size(); ps++) {
        PassJob* jobs = (PassJob*)(hdr.data() + p.pass_hdr_off[ps]);
        uint32_t g = 0;
        for (size_t j = 0; j < p.passes[ps].size(); j++) {
            const Plan::Entry& e = p.passes[ps][j];
            PassJob& jb = jobs[j];
            jb.msg = (const uint8_t*)descs_host[e.msg].msg;
            jb.in = (const Digest*)(digs + e.in_off);
            jb.out = (Digest*)(digs + e.out_off);
            jb.nbytes = descs_host[e.msg].nbytes;
            jb.count = e.count;
            jb.group0 = g;
            jb.one = 1;
            g += (uint32_t)e.groups;
        }
        blocks[ps] = g;
    }
    FinalJob* fj = (FinalJob*)(hdr.data() + p.final_hdr_off);
    for (int i = 0; i < n; i++) {
        fj[i].root = (const Digest*)(digs + p.root_off[i]);
        fj[i].nbytes = descs_host[i].nbytes;
        fj[i].r_len = descs_host[i].r_len;
        fj[i].one = 1;
        memcpy(fj[i].r, descs_host[i].r, 32);
    }
    if (cudaMemcpyAsync(base, hdr.data(), hdr.size(), cudaMemcpyHostToDevice, st) != cudaSuccess) return IMM_ERR_CUDA;
    for (size_t ps = 0; ps < p.passes.size(); ps++) {
        const PassJob* d_jobs = (const PassJob*)(base + p.pass_hdr_off[ps]);
        const int njobs = (int)p.passes[ps].size();
        if (ps == 0) {
            if (p.leaf_threads == 512) commit_leaf_kernel<512><<<blocks[ps], 512, 0, st>>>(d_jobs, njobs);
            else if (p.leaf_threads == 256) commit_leaf_kernel<256><<<blocks[ps], 256, 0, st>>>(d_jobs, njobs);
            else commit_leaf_kernel<128><<<blocks[ps], 128, 0, st>>>(d_jobs, njobs);
        }
        else commit_node_kernel<<<blocks[ps], NODE_THREADS, 0, st>>>(d_jobs, njobs);
        if (cudaGetLastError() != cudaSuccess) return IMM_ERR_CUDA;
    }
    commit_final_kernel<<<(n + 127) / 128, 128, 0, st>>>((const FinalJob*)(base + p.final_hdr_off), n, d_digests, d_roots);
    return cudaGetLastError() == cudaSuccess ? IMM_OK : IMM_ERR_CUDA;
}

}  // extern "C"
