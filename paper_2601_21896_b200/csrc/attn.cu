// Chunk attention launcher: picks the kernel for the shape.
#include "common.cuh"
#include "attn_mma.cuh"
#include "attn_tc.cuh"

namespace pafu {

size_t attn_workspace_bytes(const StreamTable&, int32_t, int32_t d_head) {
    return d_head == attn_tc::kD ? attn_tc::workspace_bytes() : 0;
}

pafu_status launch_attn(const uint16_t* Q, const uint16_t* Kc, const uint16_t* Vc,
                        const uint16_t* Kq, const uint16_t* Vq, const StreamTable& st,
                        int32_t n_heads, int32_t d_head, float scale, uint16_t* O, float* LSE,
                        void* ws, size_t, cudaStream_t stream) {
    if (d_head == attn_tc::kD && attn_tc::supports(st, Kq != nullptr)) {
        uint8_t* base = static_cast<uint8_t*>(ws);
        return attn_tc::launch(Q, Kc, Vc, Kq, Vq, st, n_heads, scale, O, LSE,
                               reinterpret_cast<int*>(base) + kStatusWordTimeout,
                               reinterpret_cast<float*>(base + kWsHeaderBytes), stream);
    }
    return attn_mma::launch(Q, Kc, Vc, Kq, Vq, st, n_heads, d_head, scale, O, LSE, stream);
}

}  // namespace pafu
