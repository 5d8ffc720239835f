// Host-callable launch wrappers of the libimm kernels (internal; the C ABI is include/imm.h).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "imm_plan.h"

namespace imm {

cudaError_t launch_field_binop(int op, const imm_fe* x, const imm_fe* y, imm_fe* out, int64_t n,
                               cudaStream_t st);
cudaError_t launch_eq_direct(const EqDirect& r, int nvars, imm_fe* out, cudaStream_t st);
cudaError_t launch_eq_batch(const EqTask* d_tasks, int ntasks, cudaStream_t st);
// dtype: 0 = int8, 1 = int32.  `point`: dot the bound rows with eq_col, one partial per tile.
cudaError_t launch_rowbind(int dtype, bool point, const MatJob* d_jobs, int njobs, uint32_t ntiles,
                           cudaStream_t st);
cudaError_t launch_colbind(int dtype, const MatJob* d_jobs, int njobs, uint32_t ntiles, cudaStream_t st);
// Tensor-core contractions: limb tables of the weights, then the byte-dot (contiguous index) and
// row-binding (strided index, int8 only) kernels.
cudaError_t launch_weights(const WeightTask* d_tasks, int ntasks, int max_words, cudaStream_t st);
cudaError_t launch_bytedot(bool i32, bool point, int mt, const MatJob* d_jobs, int njobs, uint32_t ntiles,
                           cudaStream_t st);
cudaError_t launch_rowmma(const MatJob* d_jobs, int njobs, uint32_t ntiles, cudaStream_t st);
cudaError_t launch_sum_parts(const imm_fe* parts, int nparts, int64_t len, imm_fe* out, cudaStream_t st);
cudaError_t launch_sum_all(const imm_fe* parts, int64_t count, imm_fe* out, cudaStream_t st);
cudaError_t launch_sumcheck(const ProofDev* d_proofs, int nproofs, uint64_t seed, imm_fe* transcripts,
                            int64_t stride, int32_t* status, int max_b, cudaStream_t st);

}  // namespace imm
