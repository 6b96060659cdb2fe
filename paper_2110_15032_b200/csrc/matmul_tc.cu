// Tensor-core MatMul kernel (placeholder until the tcgen05 kernel lands in this file).
#include "matmul_plan.h"
#include "sbp_internal.h"

namespace sbp {

size_t matmul_tc_workspace_bytes(const MatmulPlan&) { return 0; }

sbp_status launch_matmul_tc(const MatmulPlan&, void*, size_t, cudaStream_t, bool* taken) {
  *taken = false;
  return SBP_ERR_UNSUPPORTED;
}

}  // namespace sbp
