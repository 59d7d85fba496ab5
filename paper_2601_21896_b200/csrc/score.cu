// Salience head launcher (the kernel is in score_tc.cuh).
#include "common.cuh"
#include "score_tc.cuh"

namespace pafu {

size_t score_workspace_bytes(const pafu_head&) { return 0; }

pafu_status launch_score(const pafu_head& head, const uint16_t* const* X, int n_parts, int64_t n_tokens, int64_t ldx,
                         float* scores, void* ws, size_t, cudaStream_t stream) {
    if (n_tokens == 0) return PAFU_OK;
    return score_tc::launch(head, X, n_parts, n_tokens, ldx, scores,
                            reinterpret_cast<int*>(ws) + kStatusWordTimeout, device_sm_count(), stream);
}

}  // namespace pafu
