// Tensor-core LM head (placeholder until the tcgen05 kernel lands).
#include "lm_head_tc.cuh"

namespace ctcsd {

bool lm_head_tc_supported(const Handle*) { return false; }

int launch_lm_head_tc(Handle*, cudaStream_t, int, const void*, const void*, int*, float*) {
    return CTCSD_ERR_UNSUPPORTED;
}

}  // namespace ctcsd
