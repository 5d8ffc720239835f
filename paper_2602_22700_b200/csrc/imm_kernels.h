// Host-callable launch wrappers of the libimm kernels (internal; the C ABI is include/imm.h).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "imm_plan.h"

namespace imm {

// streaming multiprocessors of the current device (cached per device; 148 when no device answers)
int sm_count();

cudaError_t launch_field_binop(int op, const imm_fe* x, const imm_fe* y, imm_fe* out, int64_t n,
                               cudaStream_t st);
cudaError_t launch_eq_direct(const EqDirect& r, int nvars, imm_fe* out, cudaStream_t st);
// max_cover: the most entries any task has to cover (its table, or its limb tables' padded extent)
cudaError_t launch_eq_batch(const EqTask* d_tasks, int ntasks, int64_t max_cover, cudaStream_t st);
// dtype: 0 = int8, 1 = int32.  `point`: dot the bound rows with eq_col, one partial per tile.
cudaError_t launch_rowbind(int dtype, bool point, const MatJob* d_jobs, int njobs, uint32_t ntiles,
                           cudaStream_t st);
cudaError_t launch_colbind(int dtype, const MatJob* d_jobs, int njobs, uint32_t ntiles, cudaStream_t st);
// Tensor-core contractions (their weight limb tables come from launch_eq_batch): the byte-dot
// (contiguous index) and row-binding (strided index, int8 only) kernels.
cudaError_t launch_bytedot(bool i32, bool point, int mt, const MatJob* d_jobs, int njobs, uint32_t ntiles,
                           cudaStream_t st);
cudaError_t launch_rowmma(const MatJob* d_jobs, int njobs, uint32_t ntiles, int warps, cudaStream_t st);
cudaError_t launch_sum_parts(const imm_fe* parts, int nparts, int64_t len, imm_fe* out, cudaStream_t st);
cudaError_t launch_sum_all(const imm_fe* parts, int64_t count, imm_fe* out, cudaStream_t st);
// sum of the partial sums of a tensor-core point evaluation, minus the 2^31 offset of an int32 matrix (nsr > 0)
cudaError_t launch_point_finish(const imm_fe* parts, int64_t count, const imm_fe* sum_row, int nsr,
                                const imm_fe* sum_col, int nsc, imm_fe* out, cudaStream_t st);
// cluster: blocks per proof (1, 2, 4 or 8), or 0 to let the launch choose from the batch size;
// dependent: launched as a programmatic dependent of the kernel before it (reduce_parts_kernel)
cudaError_t launch_sumcheck(const ProofDev* d_proofs, int nproofs, uint64_t seed, imm_fe* transcripts,
                            int64_t stride, int32_t* status, int max_b, int cluster, bool dependent, cudaStream_t st);
// small batches: all three contractions in one persistent launch (a run of segments per block), the eq
// weights built inside the blocks
cudaError_t launch_fused_contract(const FusedJob* d_jobs, const FusedSeg* d_segs, const uint32_t* d_block_first,
                                  uint32_t nblocks, cudaStream_t st);
// the round tables and the claim of every proof from the contractions' partial results
cudaError_t launch_reduce_parts(const ProofDev* d_proofs, int nproofs, int max_b, cudaStream_t st);
// batched transcript (1 + 3b + 3*nproofs words) from per-proof transcripts proved under shared round challenges
cudaError_t launch_combine(const imm_fe* tr, int64_t stride, int nproofs, int b, uint64_t seed, uint64_t batch_id,
                           imm_fe* out, cudaStream_t st);
// non-interactive proof: statement hash and hashed evaluation points; rounds with hashed challenges
cudaError_t launch_fs_points(const ProofDev* d_proofs, const FsProof* d_fs, int nproofs, cudaStream_t st);
cudaError_t launch_sumcheck_fs(const ProofDev* d_proofs, const FsProof* d_fs, int nproofs, imm_fe* transcripts,
                               int64_t stride, int32_t* status, cudaStream_t st);
// the verifier's own (c0, a_fin, b_fin) per proof from the contractions' partial results and E_k
cudaError_t launch_expected(const ProofDev* d_proofs, const ExpectDev* d_ex, int nproofs, imm_fe* expected,
                            int32_t* status, cudaStream_t st);
// batched non-interactive proof: seed and coefficients, members' tables, then per round a combining launch and a
// folding launch (3 + 2b launches in all)
cudaError_t launch_fs_batched_rounds(const ProofDev* d_proofs, const FsProof* d_fs, const FsBatch& fb, imm_fe* transcript,
                                     int32_t* status, cudaStream_t st);

}  // namespace imm
