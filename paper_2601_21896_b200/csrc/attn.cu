// Chunk attention launcher: picks the kernel for the shape.
#include <math.h>
#include <string.h>

#include "common.cuh"
#include "attn_mma.cuh"
#include "attn_tc.cuh"

namespace pafu {

size_t attn_workspace_bytes(const StreamTable&, int32_t, int32_t d_head) {
    return (d_head == attn_tc::kD || d_head == 64) ? attn_tc::workspace_bytes() : 0;
}

pafu_status launch_attn(const uint16_t* Q, const uint16_t* Kc, const uint16_t* Vc,
                        const uint16_t* Kq, const uint16_t* Vq, const StreamTable& st,
                        int32_t n_heads, int32_t d_head, float scale, uint16_t* O, float* LSE,
                        void* ws, size_t, cudaStream_t stream) {
    if ((d_head == attn_tc::kD || d_head == 64) && attn_tc::supports(st, Kq != nullptr)) {
        uint8_t* base = static_cast<uint8_t*>(ws);
        return attn_tc::launch(Q, Kc, Vc, Kq, Vq, st, n_heads, scale, O, LSE,
                               reinterpret_cast<int*>(base) + kStatusWordTimeout,
                               reinterpret_cast<float*>(base + kWsHeaderBytes), stream, 0, nullptr, d_head);
    }
    return attn_mma::launch(Q, Kc, Vc, Kq, Vq, st, n_heads, d_head, scale, O, LSE, stream);
}

// Retained keys/values read through the index list from the uncompacted cache (d_head 128).
pafu_status launch_attn_indexed(const uint16_t* Q, const uint16_t* K, const uint16_t* V, const int32_t* idx,
                                const uint16_t* Kq, const uint16_t* Vq, const StreamTable& st,
                                int32_t n_heads, float scale, uint16_t* O, float* LSE,
                                void* ws, size_t, cudaStream_t stream) {
    uint8_t* base = static_cast<uint8_t*>(ws);
    return attn_tc::launch(Q, K, V, Kq, Vq, st, n_heads, scale, O, LSE,
                           reinterpret_cast<int*>(base) + kStatusWordTimeout,
                           reinterpret_cast<float*>(base + kWsHeaderBytes), stream, 0, idx);
}

bool attn_indexed_supported(const StreamTable& st, int32_t d_head, bool has_chunk) {
    return d_head == attn_tc::kD && attn_tc::supports(st, has_chunk);
}

}  // namespace pafu

// ---------------------------------------------------------------------------------------------
// Chunk attention for callers that cannot allocate device memory.
//
// The tcgen05 attention kernel needs scratch in global memory: a status word and the partial
// results of query blocks whose keys were split across CTAs.  pafu_chunk_attn takes that
// scratch from the caller's workspace.  Here it lives in a file-scope device array that is part
// of the library image, so every GPU that loads the library carries it until the process ends.
// The array holds the partials of kNoAllocCtas CTAs; the kernel is launched with at most that
// many CTAs (fewer than the GPU has SMs, so this entry point trades speed for needing nothing
// from the caller beyond inputs and outputs).
namespace {
constexpr int kNoAllocCtas = 31;
constexpr size_t kNoAllocBytes = pafu::kWsHeaderBytes + (size_t)kNoAllocCtas * 2 * pafu::attn_tc::kPieceBytes;
static_assert(kNoAllocBytes <= (size_t)PAFU_NOALLOC_SCRATCH_BYTES, "scratch array too small");
static __device__ __align__(256) unsigned char g_noalloc_scratch[PAFU_NOALLOC_SCRATCH_BYTES];
void* g_noalloc_ptr[pafu::kMaxDevices] = {nullptr};   // device address of the array, per device
}  // namespace

extern "C" pafu_status pafu_chunk_attn_noalloc(const uint16_t* Q, const uint16_t* Kc, const uint16_t* Vc,
                                               const int64_t* cu_B, const uint16_t* Kq, const uint16_t* Vq,
                                               const pafu_shape* shape, float scale, uint16_t* O, float* LSE,
                                               void* stream) {
    using namespace pafu;
    if (shape == nullptr || cu_B == nullptr || shape->cu_Lq == nullptr) return PAFU_ERR_INVALID_ARG;
    if (shape->n_streams < 1 || shape->n_heads < 1) return PAFU_ERR_INVALID_ARG;
    if (shape->n_streams > PAFU_MAX_STREAMS) return PAFU_ERR_UNSUPPORTED_SHAPE;
    if (shape->d_head != attn_tc::kD) return PAFU_ERR_UNSUPPORTED_SHAPE;
    if (!(scale >= 0.f) || scale > 3.0e38f) return PAFU_ERR_INVALID_ARG;
    StreamTable st;
    memset(&st, 0, sizeof st);
    st.n_streams = shape->n_streams;
    if (cu_B[0] != 0 || shape->cu_Lq[0] != 0) return PAFU_ERR_INVALID_ARG;
    for (int s = 0; s <= shape->n_streams; ++s) {
        if (s > 0 && (cu_B[s] < cu_B[s - 1] || shape->cu_Lq[s] < shape->cu_Lq[s - 1])) return PAFU_ERR_INVALID_ARG;
        st.cu_B[s] = cu_B[s];
        st.cu_Lq[s] = shape->cu_Lq[s];
    }
    const int64_t nQ = st.cu_Lq[st.n_streams], nB = st.cu_B[st.n_streams];
    if (nQ == 0) return PAFU_OK;
    // the size limit: reject before touching the device
    if (nQ * shape->n_heads > (int64_t)PAFU_NOALLOC_MAX_QUERY_HEAD_ROWS) return PAFU_ERR_TOO_LARGE;
    if (Q == nullptr || O == nullptr) return PAFU_ERR_INVALID_ARG;
    if ((Kq == nullptr) != (Vq == nullptr)) return PAFU_ERR_INVALID_ARG;
    if (nB > 0 && (Kc == nullptr || Vc == nullptr)) return PAFU_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(O) || !aligned16(Kc) || !aligned16(Vc) || !aligned16(Kq) ||
        !aligned16(Vq) || !aligned16(LSE)) return PAFU_ERR_MISALIGNED;
    if (!attn_tc::supports(st, Kq != nullptr)) return PAFU_ERR_UNSUPPORTED_SHAPE;
    // set-up, once per device: in host code the array's name is only a handle, the address the
    // kernels need comes from the runtime
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= pafu::kMaxDevices) return PAFU_ERR_CUDA;
    if (g_noalloc_ptr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) return PAFU_ERR_CUDA;
        g_noalloc_ptr[dev] = ptr;
    }
    unsigned char* base = static_cast<unsigned char*>(g_noalloc_ptr[dev]);
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    // the array keeps the previous call's contents; only the status word has to start at zero
    if (cudaMemsetAsync(base, 0, kWsHeaderBytes, cs) != cudaSuccess) return PAFU_ERR_CUDA;
    if (scale == 0.f) scale = 1.0f / sqrtf((float)shape->d_head);
    return attn_tc::launch(Q, Kc, Vc, Kq, Vq, st, shape->n_heads, scale, O, LSE,
                           reinterpret_cast<int*>(base) + kStatusWordTimeout,
                           reinterpret_cast<float*>(base + kWsHeaderBytes), cs, kNoAllocCtas);
}
