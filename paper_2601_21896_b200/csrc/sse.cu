// Teacher-side salience target (Sec. 3.2, Eq. 4 and Eq. 5): C ABI entry and workspace plan.
#include <math.h>
#include <string.h>

#include "common.cuh"
#include "sse_tc.cuh"
#include "sse_meanfirst.cuh"

namespace {
using namespace pafu;

inline size_t up256(size_t v) { return (v + 255) / 256 * 256; }

// Workspace: [status header][attention scratch][LSE N x L][O L x N x D bf16][queries' extra features][maxima].
// The attention scratch, LSE and O parts are only used when the caller passes no LSE.
struct SsePlan {
    size_t attn, lse, o, neglse, maxima, total;
};
SsePlan plan(int64_t L, int32_t n_heads, int32_t d_head, int64_t LB) {
    const sse_tc::Params p = sse_tc::make_params(L, LB, n_heads, 1.0f);
    StreamTable st;
    memset(&st, 0, sizeof st);
    st.n_streams = 1;
    SsePlan pl;
    size_t off = kWsHeaderBytes;
    pl.attn = off; off = up256(off + attn_workspace_bytes(st, n_heads, d_head));
    pl.lse = off; off = up256(off + (size_t)n_heads * L * 4);
    pl.o = off; off = up256(off + (size_t)L * n_heads * d_head * 2);
    pl.neglse = off; off = up256(off + sse_tc::aug_bytes(p));
    pl.maxima = off; off = up256(off + sse_tc::maxima_bytes(p));
    pl.total = off;
    return pl;
}
bool args_ok(int64_t L, int32_t n_heads, int32_t d_head, int64_t LB) {
    return L >= 1 && n_heads >= 1 && LB >= 1 && d_head >= 1;
}
}  // namespace

extern "C" size_t pafu_sse_workspace_bytes(int64_t L, int32_t n_heads, int32_t d_head, int64_t block_len) {
    if (!args_ok(L, n_heads, d_head, block_len) || d_head != sse_tc::kD || L > 0x7fffffffLL) return 0;
    return plan(L, n_heads, d_head, block_len).total;
}

extern "C" pafu_status pafu_sse(const uint16_t* Q, const uint16_t* K, const float* LSE, int64_t L,
                                int32_t n_heads, int32_t d_head, int64_t block_len, float scale,
                                float* s, float* comp, float* gmax, float* gavg, void* ws, size_t ws_bytes, void* stream) {
    if (!args_ok(L, n_heads, d_head, block_len)) return PAFU_ERR_INVALID_ARG;
    if (d_head != sse_tc::kD || L > 0x7fffffffLL) return PAFU_ERR_UNSUPPORTED_SHAPE;
    if (!(scale >= 0.f) || isinf(scale)) return PAFU_ERR_INVALID_ARG;
    if (Q == nullptr || K == nullptr || s == nullptr || ws == nullptr) return PAFU_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(LSE) || !aligned16(s) || !aligned16(comp) || !aligned16(gmax) || !aligned16(gavg)) return PAFU_ERR_MISALIGNED;
    if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return PAFU_ERR_MISALIGNED;
    const SsePlan pl = plan(L, n_heads, d_head, block_len);
    if (ws_bytes < pl.total) return PAFU_ERR_WORKSPACE_TOO_SMALL;
    if (scale == 0.f) scale = 1.0f / sqrtf((float)d_head);
    uint8_t* base = static_cast<uint8_t*>(ws);
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const float* lse = LSE;
    if (lse == nullptr) {
        // row statistics from the attention kernel: keys = the whole sequence, values = the keys
        // (the output is discarded; only the log-sum-exp is kept)
        StreamTable st;
        memset(&st, 0, sizeof st);
        st.n_streams = 1;
        st.cu_B[1] = L; st.cu_Lq[1] = L;
        float* lse_out = reinterpret_cast<float*>(base + pl.lse);
        pafu_status e = launch_attn(Q, K, K, nullptr, nullptr, st, n_heads, d_head, scale,
                                    reinterpret_cast<uint16_t*>(base + pl.o), lse_out, base,
                                    pl.attn + attn_workspace_bytes(st, n_heads, d_head), cs);
        if (e != PAFU_OK) return e;
        lse = lse_out;
    }
    return sse_tc::launch(Q, K, lse, L, block_len, n_heads, scale, s, comp, gmax, gavg,
                          reinterpret_cast<uint16_t*>(base + pl.neglse), reinterpret_cast<float*>(base + pl.maxima),
                          reinterpret_cast<int*>(base) + kStatusWordTimeout, cs);
}

// The same target with the mean over heads taken before the maximum over queries (Algorithm 3's
// order).  Shares the workspace plan of pafu_sse: the row log-sum-exps come from the caller or from
// one attention pass.
extern "C" pafu_status pafu_sse_mean_first(const uint16_t* Q, const uint16_t* K, const float* LSE, int64_t L,
                                           int32_t n_heads, int32_t d_head, int64_t block_len, float scale,
                                           float* s, float* comp, void* ws, size_t ws_bytes, void* stream) {
    if (!args_ok(L, n_heads, d_head, block_len)) return PAFU_ERR_INVALID_ARG;
    if (d_head != sse_tc::kD || L > 0x7fffffffLL) return PAFU_ERR_UNSUPPORTED_SHAPE;
    if (!(scale >= 0.f) || isinf(scale)) return PAFU_ERR_INVALID_ARG;
    if (Q == nullptr || K == nullptr || s == nullptr || ws == nullptr) return PAFU_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(LSE) || !aligned16(s) || !aligned16(comp)) return PAFU_ERR_MISALIGNED;
    if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return PAFU_ERR_MISALIGNED;
    const SsePlan pl = plan(L, n_heads, d_head, block_len);
    if (ws_bytes < pl.total) return PAFU_ERR_WORKSPACE_TOO_SMALL;
    if (scale == 0.f) scale = 1.0f / sqrtf((float)d_head);
    uint8_t* base = static_cast<uint8_t*>(ws);
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const float* lse = LSE;
    if (lse == nullptr) {
        StreamTable st;
        memset(&st, 0, sizeof st);
        st.n_streams = 1;
        st.cu_B[1] = L; st.cu_Lq[1] = L;
        float* lse_out = reinterpret_cast<float*>(base + pl.lse);
        pafu_status e = launch_attn(Q, K, K, nullptr, nullptr, st, n_heads, d_head, scale,
                                    reinterpret_cast<uint16_t*>(base + pl.o), lse_out, base,
                                    pl.attn + attn_workspace_bytes(st, n_heads, d_head), cs);
        if (e != PAFU_OK) return e;
        lse = lse_out;
    }
    return sse_mf::launch(Q, K, lse, L, block_len, n_heads, scale, s, comp, cs);
}
