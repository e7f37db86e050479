// tcgen05 tensor-core INT8 GEMM (placeholder until the kernel lands in this file).
#include "common.cuh"
namespace ivit {
int launch_gemm_tc(ivit_ctx*, const GemmProblem&) { return IVIT_ERR_UNSUPPORTED; }
}  // namespace ivit
