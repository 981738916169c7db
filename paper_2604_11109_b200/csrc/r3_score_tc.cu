// Tensor-core scoring engine (placeholder translation unit until the tcgen05 kernels land).
#include "r3_internal.cuh"

namespace r3 {

bool tc_supported(int, int) { return false; }
r3_status_t tc_prepare(r3_gp*, cudaStream_t) { return R3_OK; }
void tc_release(r3_gp*) {}
size_t score_tc_workspace_bytes(const r3_gp*, long long) { return 0; }
r3_status_t score_tc(r3_gp*, const float*, long long, float*, float*, float*, void*, size_t, cudaStream_t)
{
    set_error("tensor-core engine not built");
    return R3_ERR_UNSUPPORTED;
}

}  // namespace r3
