// bf16 tensor-core GEMM (placeholder until the tcgen05 kernel lands).
#include "common.cuh"

namespace gelo {

bool gemm_tc_supports(const GemmArgs&) { return false; }
int launch_gemm_tc(gelo_ctx*, const GemmArgs&, cudaStream_t) { return GELO_ERR_UNSUPPORTED; }

}  // namespace gelo
