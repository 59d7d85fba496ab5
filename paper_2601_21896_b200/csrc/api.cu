// C ABI layer: argument validation, launch planning, the fused step driver.
// Every error is detected here, on the host, before anything is enqueued.
#include <math.h>
#include <string.h>

#include "common.cuh"

namespace pafu {

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// true when the byte ranges [a, a + na) and [b, b + nb) share a byte
static bool ranges_overlap(const void* a, size_t na, const void* b, size_t nb) {
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return na > 0 && nb > 0 && a0 < b0 + nb && b0 < a0 + na;
}

static bool prefix_ok(const int64_t* cu, int n) {
    if (cu == nullptr || cu[0] != 0) return false;
    for (int s = 0; s < n; ++s)
        if (cu[s + 1] < cu[s]) return false;
    return true;
}

static pafu_status shape_ok(const pafu_shape* sh, bool need_T, bool need_Lq) {
    if (sh == nullptr) return PAFU_ERR_INVALID_ARG;
    if (sh->n_streams < 1 || sh->n_heads < 1 || sh->d_head < 1) return PAFU_ERR_INVALID_ARG;
    if (sh->n_streams > PAFU_MAX_STREAMS) return PAFU_ERR_UNSUPPORTED_SHAPE;
    if (need_T && !prefix_ok(sh->cu_T, sh->n_streams)) return PAFU_ERR_INVALID_ARG;
    if (need_Lq && !prefix_ok(sh->cu_Lq, sh->n_streams)) return PAFU_ERR_INVALID_ARG;
    return PAFU_OK;
}

// Fills the retention part of the table: clamped sink/recent, k, and cu_B.
static pafu_status fill_policy(const pafu_shape* sh, const pafu_policy* pol, StreamTable* st) {
    if (pol == nullptr) return PAFU_ERR_INVALID_ARG;
    st->cu_B[0] = 0;
    for (int s = 0; s < sh->n_streams; ++s) {
        const int64_t T = sh->cu_T[s + 1] - sh->cu_T[s];
        if (pol[s].budget < 0 || pol[s].n_sink < 0 || pol[s].n_recent < 0) return PAFU_ERR_BAD_BUDGET;
        if (T > 0x7fffffffLL) return PAFU_ERR_UNSUPPORTED_SHAPE;
        int64_t ns = 0, nr = 0, k = 0, B = T;
        if (T > pol[s].budget) {
            B = pol[s].budget;
            nr = pol[s].n_recent < B ? pol[s].n_recent : B;
            ns = pol[s].n_sink < B - nr ? pol[s].n_sink : B - nr;
            k = B - ns - nr;
        }
        st->n_sink[s] = ns;
        st->n_recent[s] = nr;
        st->k[s] = k;
        st->cu_B[s + 1] = st->cu_B[s] + B;
    }
    return PAFU_OK;
}

static void fill_prefix(int64_t* dst, const int64_t* src, int n) {
    for (int s = 0; s <= n; ++s) dst[s] = src ? src[s] : 0;
}

// `device_ptrs`: the weight pointers are device pointers and must be 16-byte aligned
static pafu_status head_ok(const pafu_head* h, bool device_ptrs = true) {
    if (h == nullptr || h->w1 == nullptr || h->w2 == nullptr) return PAFU_ERR_INVALID_ARG;
    if (h->d_in < 1 || h->d_hidden < 1 || h->d_out < 1) return PAFU_ERR_INVALID_ARG;
    if (h->act != PAFU_ACT_GELU && h->act != PAFU_ACT_SILU) return PAFU_ERR_INVALID_ARG;
    if (h->final != PAFU_FINAL_NONE && h->final != PAFU_FINAL_SIGMOID) return PAFU_ERR_INVALID_ARG;
    if (h->d_in % 64 != 0 || h->d_hidden % 16 != 0 || h->d_hidden > 1024) return PAFU_ERR_UNSUPPORTED_SHAPE;
    if (device_ptrs && (!aligned16(h->w1) || !aligned16(h->w2))) return PAFU_ERR_MISALIGNED;
    return PAFU_OK;
}

static size_t workspace_bytes_impl(const StreamTable& st, int n_heads, int d_head, const pafu_head* head) {
    size_t b = kWsHeaderBytes;
    size_t step = 0;
    if (head != nullptr) step = score_workspace_bytes(*head);
    const size_t a = attn_workspace_bytes(st, n_heads, d_head);
    if (a > step) step = a;
    return b + align_up(step, 256);
}

}  // namespace pafu

using namespace pafu;

extern "C" {

int32_t pafu_version(void) { return 1000; }

const char* pafu_status_string(pafu_status s) {
    switch (s) {
        case PAFU_OK: return "ok";
        case PAFU_ERR_INVALID_ARG: return "invalid argument";
        case PAFU_ERR_BAD_BUDGET: return "negative budget, sink or recent length";
        case PAFU_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case PAFU_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case PAFU_ERR_MISALIGNED: return "device pointer not 16-byte aligned";
        case PAFU_ERR_CUDA: return "CUDA call failed";
        case PAFU_ERR_TIMEOUT: return "bounded device wait ran out";
        case PAFU_ERR_TOO_LARGE: return "problem exceeds the built-in scratch of the no-allocation entry point";
        default: return "unknown status";
    }
}

pafu_status pafu_kept_counts(const pafu_shape* shape, const pafu_policy* policy, int64_t* cu_B) {
    pafu_status e = shape_ok(shape, true, false);
    if (e != PAFU_OK) return e;
    if (cu_B == nullptr) return PAFU_ERR_INVALID_ARG;
    StreamTable st;
    e = fill_policy(shape, policy, &st);
    if (e != PAFU_OK) return e;
    for (int s = 0; s <= shape->n_streams; ++s) cu_B[s] = st.cu_B[s];
    return PAFU_OK;
}

size_t pafu_workspace_bytes(const pafu_shape* shape, const pafu_policy* policy, const pafu_head* head) {
    if (shape_ok(shape, false, false) != PAFU_OK) return 0;
    StreamTable st;
    memset(&st, 0, sizeof st);
    st.n_streams = shape->n_streams;
    if (shape->cu_T != nullptr) {
        if (!prefix_ok(shape->cu_T, shape->n_streams)) return 0;
        fill_prefix(st.cu_T, shape->cu_T, shape->n_streams);
        if (policy != nullptr && fill_policy(shape, policy, &st) != PAFU_OK) return 0;
    }
    if (shape->cu_Lq != nullptr) {
        if (!prefix_ok(shape->cu_Lq, shape->n_streams)) return 0;
        fill_prefix(st.cu_Lq, shape->cu_Lq, shape->n_streams);
    }
    if (head != nullptr && head_ok(head) != PAFU_OK) return 0;
    return workspace_bytes_impl(st, shape->n_heads, shape->d_head, head);
}

pafu_status pafu_workspace_status(const void* ws, void* stream) {
    if (ws == nullptr) return PAFU_ERR_INVALID_ARG;
    int32_t word = 0;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&word, ws, sizeof word, cudaMemcpyDeviceToHost, cs) != cudaSuccess) return PAFU_ERR_CUDA;
    if (cudaStreamSynchronize(cs) != cudaSuccess) return PAFU_ERR_CUDA;
    return word == 0 ? PAFU_OK : PAFU_ERR_TIMEOUT;
}

pafu_status pafu_workspace_counters(const void* ws, int64_t* counts, void* stream) {
    if (ws == nullptr || counts == nullptr) return PAFU_ERR_INVALID_ARG;
    int32_t words[3] = {0, 0, 0};
    static_assert(kStatusWordFullSum == kStatusWordFullFirst + 1 && kStatusWordRescale == kStatusWordFullFirst + 2,
                  "the three counters are read with one copy");
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(words, static_cast<const int32_t*>(ws) + kStatusWordFullFirst, sizeof words,
                        cudaMemcpyDeviceToHost, cs) != cudaSuccess) return PAFU_ERR_CUDA;
    if (cudaStreamSynchronize(cs) != cudaSuccess) return PAFU_ERR_CUDA;
    for (int i = 0; i < 3; ++i) counts[i] = words[i];
    return PAFU_OK;
}

namespace {
// shared by the one- and three-matrix entry points; X[i] holds features [i * d_in / n_parts, ...)
pafu_status score_impl(const pafu_head* head, const uint16_t* const* X, int n_parts, int64_t n_tokens, int64_t ldx,
                       float* scores, void* ws, size_t ws_bytes, void* stream) {
    pafu_status e = head_ok(head);
    if (e != PAFU_OK) return e;
    if (head->d_in % (64 * n_parts) != 0) return PAFU_ERR_UNSUPPORTED_SHAPE;
    if (n_tokens < 0) return PAFU_ERR_INVALID_ARG;
    if (n_tokens == 0) return PAFU_OK;
    if (scores == nullptr) return PAFU_ERR_INVALID_ARG;
    for (int i = 0; i < n_parts; ++i)
        if (X[i] == nullptr) return PAFU_ERR_INVALID_ARG;
    if (ldx < head->d_in / n_parts || ldx % 8 != 0) return PAFU_ERR_INVALID_ARG;
    for (int i = 0; i < n_parts; ++i)
        if (!aligned16(X[i])) return PAFU_ERR_MISALIGNED;
    if (!aligned16(scores)) return PAFU_ERR_MISALIGNED;
    const size_t need = kWsHeaderBytes + score_workspace_bytes(*head);
    if (ws == nullptr) return PAFU_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return PAFU_ERR_MISALIGNED;
    if (ws_bytes < need) return PAFU_ERR_WORKSPACE_TOO_SMALL;
    return launch_score(*head, X, n_parts, n_tokens, ldx, scores, ws, ws_bytes, static_cast<cudaStream_t>(stream));
}
}  // namespace

pafu_status pafu_score(const pafu_head* head, const uint16_t* X, int64_t n_tokens, int64_t ldx,
                       float* scores, void* ws, size_t ws_bytes, void* stream) {
    const uint16_t* parts[1] = {X};
    return score_impl(head, parts, 1, n_tokens, ldx, scores, ws, ws_bytes, stream);
}

pafu_status pafu_score_qkv(const pafu_head* head, const uint16_t* Q, const uint16_t* K, const uint16_t* V,
                           int64_t n_tokens, int64_t ld, float* scores, void* ws, size_t ws_bytes, void* stream) {
    const uint16_t* parts[3] = {Q, K, V};
    return score_impl(head, parts, 3, n_tokens, ld, scores, ws, ws_bytes, stream);
}

pafu_status pafu_select(const float* scores, const pafu_shape* shape, const pafu_policy* policy,
                        int32_t* idx, void* ws, size_t ws_bytes, void* stream) {
    (void)ws; (void)ws_bytes;
    pafu_status e = shape_ok(shape, true, false);
    if (e != PAFU_OK) return e;
    StreamTable st;
    memset(&st, 0, sizeof st);
    st.n_streams = shape->n_streams;
    fill_prefix(st.cu_T, shape->cu_T, shape->n_streams);
    e = fill_policy(shape, policy, &st);
    if (e != PAFU_OK) return e;
    if (st.cu_B[st.n_streams] == 0) return PAFU_OK;
    if (scores == nullptr || idx == nullptr) return PAFU_ERR_INVALID_ARG;
    if (!aligned16(scores) || !aligned16(idx)) return PAFU_ERR_MISALIGNED;
    return launch_select(scores, st, idx, static_cast<cudaStream_t>(stream));
}

pafu_status pafu_compact(const uint16_t* K, const uint16_t* V, const float* SL, const int32_t* idx,
                         const pafu_shape* shape, const pafu_policy* policy,
                         uint16_t* Kc, uint16_t* Vc, float* SLc, void* stream) {
    pafu_status e = shape_ok(shape, true, false);
    if (e != PAFU_OK) return e;
    const int64_t dm = (int64_t)shape->n_heads * shape->d_head;
    if (dm % 8 != 0 || dm > 0x7fffffffLL) return PAFU_ERR_UNSUPPORTED_SHAPE;
    StreamTable st;
    memset(&st, 0, sizeof st);
    st.n_streams = shape->n_streams;
    fill_prefix(st.cu_T, shape->cu_T, shape->n_streams);
    e = fill_policy(shape, policy, &st);
    if (e != PAFU_OK) return e;
    if (st.cu_B[st.n_streams] == 0) return PAFU_OK;
    if (K == nullptr || V == nullptr || idx == nullptr || Kc == nullptr || Vc == nullptr) return PAFU_ERR_INVALID_ARG;
    if ((SL == nullptr) != (SLc == nullptr)) return PAFU_ERR_INVALID_ARG;
    if (!aligned16(K) || !aligned16(V) || !aligned16(Kc) || !aligned16(Vc) || !aligned16(idx)) return PAFU_ERR_MISALIGNED;
    {
        const size_t in_b = (size_t)st.cu_T[st.n_streams] * dm * 2, out_b = (size_t)st.cu_B[st.n_streams] * dm * 2;
        if (ranges_overlap(Kc, out_b, K, in_b) || ranges_overlap(Kc, out_b, V, in_b) || ranges_overlap(Vc, out_b, K, in_b) ||
            ranges_overlap(Vc, out_b, V, in_b) || ranges_overlap(Kc, out_b, Vc, out_b)) return PAFU_ERR_INVALID_ARG;
        if (SLc != nullptr && ranges_overlap(SLc, (size_t)st.cu_B[st.n_streams] * 4, SL, (size_t)st.cu_T[st.n_streams] * 4))
            return PAFU_ERR_INVALID_ARG;
    }
    return launch_compact(K, V, SL, idx, st, (int32_t)dm, Kc, Vc, SLc, static_cast<cudaStream_t>(stream));
}

pafu_status pafu_compact_layers(const uint16_t* const* K, const uint16_t* const* V, int32_t n_layers,
                                const float* SL, const int32_t* idx, const pafu_shape* shape,
                                const pafu_policy* policy, uint16_t* const* Kc, uint16_t* const* Vc,
                                float* SLc, void* stream) {
    pafu_status e = shape_ok(shape, true, false);
    if (e != PAFU_OK) return e;
    if (n_layers < 0) return PAFU_ERR_INVALID_ARG;
    if (n_layers > PAFU_MAX_LAYERS) return PAFU_ERR_UNSUPPORTED_SHAPE;
    const int64_t dm = (int64_t)shape->n_heads * shape->d_head;
    if (dm % 8 != 0 || dm > 0x7fffffffLL) return PAFU_ERR_UNSUPPORTED_SHAPE;
    StreamTable st;
    memset(&st, 0, sizeof st);
    st.n_streams = shape->n_streams;
    fill_prefix(st.cu_T, shape->cu_T, shape->n_streams);
    e = fill_policy(shape, policy, &st);
    if (e != PAFU_OK) return e;
    if (st.cu_B[st.n_streams] == 0 || n_layers == 0) return PAFU_OK;
    if (K == nullptr || V == nullptr || Kc == nullptr || Vc == nullptr || idx == nullptr) return PAFU_ERR_INVALID_ARG;
    if ((SL == nullptr) != (SLc == nullptr)) return PAFU_ERR_INVALID_ARG;
    if (!aligned16(idx)) return PAFU_ERR_MISALIGNED;
    for (int l = 0; l < n_layers; ++l) {
        if (K[l] == nullptr || V[l] == nullptr || Kc[l] == nullptr || Vc[l] == nullptr) return PAFU_ERR_INVALID_ARG;
        if (!aligned16(K[l]) || !aligned16(V[l]) || !aligned16(Kc[l]) || !aligned16(Vc[l])) return PAFU_ERR_MISALIGNED;
    }
    {
        // no output may overlap any layer's input or another output
        const size_t in_b = (size_t)st.cu_T[st.n_streams] * dm * 2, out_b = (size_t)st.cu_B[st.n_streams] * dm * 2;
        for (int l = 0; l < n_layers; ++l) {
            const void* outs[2] = {Kc[l], Vc[l]};
            for (const void* o : outs) {
                for (int m = 0; m < n_layers; ++m) {
                    if (ranges_overlap(o, out_b, K[m], in_b) || ranges_overlap(o, out_b, V[m], in_b)) return PAFU_ERR_INVALID_ARG;
                    if (m != l && (ranges_overlap(o, out_b, Kc[m], out_b) || ranges_overlap(o, out_b, Vc[m], out_b))) return PAFU_ERR_INVALID_ARG;
                }
            }
            if (ranges_overlap(Kc[l], out_b, Vc[l], out_b)) return PAFU_ERR_INVALID_ARG;
        }
    }
    return launch_compact_layers(K, V, n_layers, SL, idx, st, (int32_t)dm, Kc, Vc, SLc, static_cast<cudaStream_t>(stream));
}

pafu_status pafu_chunk_attn(const uint16_t* Q, const uint16_t* Kc, const uint16_t* Vc,
                            const int64_t* cu_B, const uint16_t* Kq, const uint16_t* Vq,
                            const pafu_shape* shape, float scale, uint16_t* O, float* LSE,
                            void* ws, size_t ws_bytes, void* stream) {
    pafu_status e = shape_ok(shape, false, true);
    if (e != PAFU_OK) return e;
    if (shape->d_head != 64 && shape->d_head != 128) return PAFU_ERR_UNSUPPORTED_SHAPE;
    if (!prefix_ok(cu_B, shape->n_streams)) return PAFU_ERR_INVALID_ARG;
    if (!(scale >= 0.f) || isinf(scale)) return PAFU_ERR_INVALID_ARG;
    StreamTable st;
    memset(&st, 0, sizeof st);
    st.n_streams = shape->n_streams;
    fill_prefix(st.cu_Lq, shape->cu_Lq, shape->n_streams);
    fill_prefix(st.cu_B, cu_B, shape->n_streams);
    if (st.cu_Lq[st.n_streams] == 0) return PAFU_OK;
    if (Q == nullptr || O == nullptr) return PAFU_ERR_INVALID_ARG;
    if ((Kq == nullptr) != (Vq == nullptr)) return PAFU_ERR_INVALID_ARG;
    if (st.cu_B[st.n_streams] > 0 && (Kc == nullptr || Vc == nullptr)) return PAFU_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(O) || !aligned16(Kc) || !aligned16(Vc) || !aligned16(Kq) ||
        !aligned16(Vq) || !aligned16(LSE)) return PAFU_ERR_MISALIGNED;
    const size_t need = kWsHeaderBytes + attn_workspace_bytes(st, shape->n_heads, shape->d_head);
    if (ws == nullptr) return PAFU_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return PAFU_ERR_MISALIGNED;
    if (ws_bytes < need) return PAFU_ERR_WORKSPACE_TOO_SMALL;
    if (scale == 0.f) scale = 1.0f / sqrtf((float)shape->d_head);
    return launch_attn(Q, Kc, Vc, Kq, Vq, st, shape->n_heads, shape->d_head, scale, O, LSE, ws, ws_bytes,
                       static_cast<cudaStream_t>(stream));
}

pafu_status pafu_chunk_attn_indexed(const uint16_t* Q, const uint16_t* K, const uint16_t* V, const int32_t* idx,
                                    const int64_t* cu_B, const uint16_t* Kq, const uint16_t* Vq,
                                    const pafu_shape* shape, float scale, uint16_t* O, float* LSE,
                                    void* ws, size_t ws_bytes, void* stream) {
    pafu_status e = shape_ok(shape, true, true);
    if (e != PAFU_OK) return e;
    if (shape->d_head != 128) return PAFU_ERR_UNSUPPORTED_SHAPE;
    if (!prefix_ok(cu_B, shape->n_streams)) return PAFU_ERR_INVALID_ARG;
    if (!(scale >= 0.f) || isinf(scale)) return PAFU_ERR_INVALID_ARG;
    StreamTable st;
    memset(&st, 0, sizeof st);
    st.n_streams = shape->n_streams;
    fill_prefix(st.cu_T, shape->cu_T, shape->n_streams);
    fill_prefix(st.cu_Lq, shape->cu_Lq, shape->n_streams);
    fill_prefix(st.cu_B, cu_B, shape->n_streams);
    for (int s = 0; s < st.n_streams; ++s) {
        if (st.cu_B[s + 1] - st.cu_B[s] > st.cu_T[s + 1] - st.cu_T[s]) return PAFU_ERR_INVALID_ARG;
    }
    // the loader addresses cache rows with 32-bit offsets in 16-byte units: K and V below 64 GiB each
    if (st.cu_T[st.n_streams] > 0x7fffffffLL ||
        (uint64_t)st.cu_T[st.n_streams] * (uint64_t)shape->n_heads * 16u >= (1ull << 32)) return PAFU_ERR_UNSUPPORTED_SHAPE;
    if (st.cu_Lq[st.n_streams] == 0) return PAFU_OK;
    if (Q == nullptr || O == nullptr) return PAFU_ERR_INVALID_ARG;
    if ((Kq == nullptr) != (Vq == nullptr)) return PAFU_ERR_INVALID_ARG;
    if (st.cu_B[st.n_streams] > 0 && (K == nullptr || V == nullptr || idx == nullptr)) return PAFU_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(O) || !aligned16(K) || !aligned16(V) || !aligned16(Kq) ||
        !aligned16(Vq) || !aligned16(LSE) || !aligned16(idx)) return PAFU_ERR_MISALIGNED;
    if (!attn_indexed_supported(st, shape->d_head, Kq != nullptr)) return PAFU_ERR_UNSUPPORTED_SHAPE;
    const size_t need = kWsHeaderBytes + attn_workspace_bytes(st, shape->n_heads, shape->d_head);
    if (ws == nullptr) return PAFU_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return PAFU_ERR_MISALIGNED;
    if (ws_bytes < need) return PAFU_ERR_WORKSPACE_TOO_SMALL;
    if (scale == 0.f) scale = 1.0f / sqrtf((float)shape->d_head);
    if (st.cu_B[st.n_streams] == 0)      // nothing retained: the plain kernel over the chunk's own tokens
        return launch_attn(Q, nullptr, nullptr, Kq, Vq, st, shape->n_heads, shape->d_head, scale, O, LSE, ws, ws_bytes,
                           static_cast<cudaStream_t>(stream));
    return launch_attn_indexed(Q, K, V, idx, Kq, Vq, st, shape->n_heads, scale, O, LSE, ws, ws_bytes,
                               static_cast<cudaStream_t>(stream));
}

static pafu_status step_impl(const pafu_step_args* a, void* const* ev, void* stream);

pafu_status pafu_step(const pafu_step_args* a, void* stream) { return step_impl(a, nullptr, stream); }

pafu_status pafu_step_timed(const pafu_step_args* a, void* const* events, void* stream) {
    if (events == nullptr) return PAFU_ERR_INVALID_ARG;
    for (int i = 0; i < 5; ++i)
        if (events[i] == nullptr) return PAFU_ERR_INVALID_ARG;
    return step_impl(a, events, stream);
}

pafu_status pafu_step_indexed(const pafu_step_args* a, void* stream) {
    if (a == nullptr) return PAFU_ERR_INVALID_ARG;
    pafu_status e = shape_ok(&a->shape, true, true);
    if (e != PAFU_OK) return e;
    e = head_ok(a->head);
    if (e != PAFU_OK) return e;
    const int64_t dm = (int64_t)a->shape.n_heads * a->shape.d_head;
    if (a->head->d_in != dm) return PAFU_ERR_INVALID_ARG;
    if (a->shape.d_head != 128) return PAFU_ERR_UNSUPPORTED_SHAPE;
    int64_t cu_B[PAFU_MAX_STREAMS + 1];
    e = pafu_kept_counts(&a->shape, a->policy, cu_B);
    if (e != PAFU_OK) return e;
    const int n = a->shape.n_streams;
    const int64_t nT = a->shape.cu_T[n], nB = cu_B[n], nQ = a->shape.cu_Lq[n];
    if (nT > 0 && (a->K == nullptr || a->V == nullptr || a->scores == nullptr)) return PAFU_ERR_INVALID_ARG;
    if (nB > 0 && a->idx == nullptr) return PAFU_ERR_INVALID_ARG;
    if (nQ > 0 && (a->Q == nullptr || a->O == nullptr)) return PAFU_ERR_INVALID_ARG;
    if ((a->Kq == nullptr) != (a->Vq == nullptr)) return PAFU_ERR_INVALID_ARG;
    if (!(a->scale >= 0.f) || isinf(a->scale)) return PAFU_ERR_INVALID_ARG;
    const void* ptrs[] = {a->K, a->V, a->Q, a->Kq, a->Vq, a->scores, a->idx, a->O, a->LSE};
    for (const void* p : ptrs)
        if (!aligned16(p)) return PAFU_ERR_MISALIGNED;
    StreamTable st;
    memset(&st, 0, sizeof st);
    st.n_streams = n;
    fill_prefix(st.cu_Lq, a->shape.cu_Lq, n);
    fill_prefix(st.cu_B, cu_B, n);
    if (!attn_indexed_supported(st, a->shape.d_head, a->Kq != nullptr)) return PAFU_ERR_UNSUPPORTED_SHAPE;
    const size_t need = pafu_workspace_bytes(&a->shape, a->policy, a->head);
    if (a->ws == nullptr) return PAFU_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(a->ws) & 255u) != 0) return PAFU_ERR_MISALIGNED;
    if (a->ws_bytes < need) return PAFU_ERR_WORKSPACE_TOO_SMALL;
    e = pafu_score(a->head, a->K, nT, dm, a->scores, a->ws, a->ws_bytes, stream);
    if (e != PAFU_OK) return e;
    e = pafu_select(a->scores, &a->shape, a->policy, a->idx, a->ws, a->ws_bytes, stream);
    if (e != PAFU_OK) return e;
    return pafu_chunk_attn_indexed(a->Q, a->K, a->V, a->idx, cu_B, a->Kq, a->Vq, &a->shape, a->scale, a->O, a->LSE,
                                   a->ws, a->ws_bytes, stream);
}

static pafu_status step_impl(const pafu_step_args* a, void* const* ev, void* stream) {
    if (a == nullptr) return PAFU_ERR_INVALID_ARG;
    pafu_status e = shape_ok(&a->shape, true, true);
    if (e != PAFU_OK) return e;
    e = head_ok(a->head);
    if (e != PAFU_OK) return e;
    const int64_t dm = (int64_t)a->shape.n_heads * a->shape.d_head;
    if (a->head->d_in != dm) return PAFU_ERR_INVALID_ARG;
    if (a->shape.d_head != 64 && a->shape.d_head != 128) return PAFU_ERR_UNSUPPORTED_SHAPE;
    int64_t cu_B[PAFU_MAX_STREAMS + 1];
    e = pafu_kept_counts(&a->shape, a->policy, cu_B);
    if (e != PAFU_OK) return e;
    const int n = a->shape.n_streams;
    const int64_t nT = a->shape.cu_T[n], nB = cu_B[n], nQ = a->shape.cu_Lq[n];
    // validate everything the four calls would reject, so that nothing runs on a bad call
    if (nT > 0 && (a->K == nullptr || a->V == nullptr || a->scores == nullptr)) return PAFU_ERR_INVALID_ARG;
    if (nB > 0 && (a->idx == nullptr || a->Kc == nullptr || a->Vc == nullptr)) return PAFU_ERR_INVALID_ARG;
    if (nQ > 0 && (a->Q == nullptr || a->O == nullptr)) return PAFU_ERR_INVALID_ARG;
    if ((a->Kq == nullptr) != (a->Vq == nullptr)) return PAFU_ERR_INVALID_ARG;
    if (!(a->scale >= 0.f) || isinf(a->scale)) return PAFU_ERR_INVALID_ARG;
    const void* ptrs[] = {a->K, a->V, a->Q, a->Kq, a->Vq, a->scores, a->idx, a->Kc, a->Vc, a->SLc, a->O, a->LSE};
    for (const void* p : ptrs)
        if (!aligned16(p)) return PAFU_ERR_MISALIGNED;
    {
        const size_t in_b = (size_t)nT * dm * 2, out_b = (size_t)nB * dm * 2;
        if (ranges_overlap(a->Kc, out_b, a->K, in_b) || ranges_overlap(a->Kc, out_b, a->V, in_b) ||
            ranges_overlap(a->Vc, out_b, a->K, in_b) || ranges_overlap(a->Vc, out_b, a->V, in_b) ||
            ranges_overlap(a->Kc, out_b, a->Vc, out_b)) return PAFU_ERR_INVALID_ARG;
        if (a->SLc != nullptr && ranges_overlap(a->SLc, (size_t)nB * 4, a->scores, (size_t)nT * 4)) return PAFU_ERR_INVALID_ARG;
    }
    const size_t need = pafu_workspace_bytes(&a->shape, a->policy, a->head);
    if (a->ws == nullptr) return PAFU_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(a->ws) & 255u) != 0) return PAFU_ERR_MISALIGNED;
    if (a->ws_bytes < need) return PAFU_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    auto mark = [&](int i) -> bool {
        return ev == nullptr || cudaEventRecord(static_cast<cudaEvent_t>(ev[i]), cs) == cudaSuccess;
    };
    if (!mark(0)) return PAFU_ERR_CUDA;
    e = pafu_score(a->head, a->K, nT, dm, a->scores, a->ws, a->ws_bytes, stream);
    if (e != PAFU_OK) return e;
    if (!mark(1)) return PAFU_ERR_CUDA;
    StreamTable st;
    memset(&st, 0, sizeof st);
    st.n_streams = n;
    fill_prefix(st.cu_T, a->shape.cu_T, n);
    e = fill_policy(&a->shape, a->policy, &st);
    if (e != PAFU_OK) return e;
    if (nB > 0 && dm % 8 == 0) {
        // Top-k and Select(KV; ids) overlapped: the gather is launched as a programmatic dependent of
        // the selection, copies the always-kept rows while the selection runs and the top-k rows
        // once the indices exist.  No event may sit between the two launches, so in the timed
        // variant the "after select" stamp is taken before them.
        if (!mark(2)) return PAFU_ERR_CUDA;
        e = launch_select(a->scores, st, a->idx, cs);
        if (e != PAFU_OK) return e;
        e = launch_compact(a->K, a->V, a->SLc ? a->scores : nullptr, a->idx, st, (int32_t)dm, a->Kc, a->Vc, a->SLc, cs,
                           static_cast<int*>(a->ws) + kStatusWordGatherWork, select_cta_count(st));
        if (e != PAFU_OK) return e;
    } else {
        e = pafu_select(a->scores, &a->shape, a->policy, a->idx, a->ws, a->ws_bytes, stream);
        if (e != PAFU_OK) return e;
        if (!mark(2)) return PAFU_ERR_CUDA;
        e = pafu_compact(a->K, a->V, a->SLc ? a->scores : nullptr, a->idx, &a->shape, a->policy, a->Kc, a->Vc,
                         a->SLc, stream);
        if (e != PAFU_OK) return e;
    }
    if (!mark(3)) return PAFU_ERR_CUDA;
    e = pafu_chunk_attn(a->Q, a->Kc, a->Vc, cu_B, a->Kq, a->Vq, &a->shape, a->scale, a->O, a->LSE,
                        a->ws, a->ws_bytes, stream);
    if (e != PAFU_OK) return e;
    if (!mark(4)) return PAFU_ERR_CUDA;
    return PAFU_OK;
}

// ---- host-buffer variant ------------------------------------------------------------------
namespace {
struct Arena {
    size_t off = 0;
    size_t take(size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; }
};
struct HostPlan {
    size_t K, V, Q, Kq, Vq, w1, b1, w2, b2, scores, idx, Kc, Vc, SLc, O, LSE, ws, ws_bytes, total;
};
HostPlan plan_host(const pafu_shape* sh, const int64_t* cu_B, const pafu_head* h, size_t ws_bytes) {
    const int n = sh->n_streams;
    const size_t dm = (size_t)sh->n_heads * sh->d_head;
    const size_t nT = sh->cu_T[n], nB = cu_B[n], nQ = sh->cu_Lq[n];
    Arena a;
    HostPlan p;
    p.K = a.take(nT * dm * 2); p.V = a.take(nT * dm * 2);
    p.Q = a.take(nQ * dm * 2); p.Kq = a.take(nQ * dm * 2); p.Vq = a.take(nQ * dm * 2);
    p.w1 = a.take((size_t)h->d_hidden * h->d_in * 2); p.b1 = a.take((size_t)h->d_hidden * 2);
    p.w2 = a.take((size_t)h->d_out * h->d_hidden * 2); p.b2 = a.take((size_t)h->d_out * 2);
    p.scores = a.take(nT * 4); p.idx = a.take(nB * 4);
    p.Kc = a.take(nB * dm * 2); p.Vc = a.take(nB * dm * 2); p.SLc = a.take(nB * 4);
    p.O = a.take(nQ * dm * 2); p.LSE = a.take(nQ * sh->n_heads * 4);
    p.ws = a.take(ws_bytes); p.ws_bytes = ws_bytes;
    p.total = a.off;
    return p;
}
}  // namespace

size_t pafu_step_host_arena_bytes(const pafu_shape* shape, const pafu_policy* policy, const pafu_head* head) {
    if (shape_ok(shape, true, true) != PAFU_OK || head == nullptr) return 0;
    int64_t cu_B[PAFU_MAX_STREAMS + 1];
    if (pafu_kept_counts(shape, policy, cu_B) != PAFU_OK) return 0;
    if (head->d_in < 1 || head->d_hidden < 1 || head->d_out < 1) return 0;
    StreamTable st;
    memset(&st, 0, sizeof st);
    st.n_streams = shape->n_streams;
    fill_prefix(st.cu_T, shape->cu_T, shape->n_streams);
    fill_prefix(st.cu_Lq, shape->cu_Lq, shape->n_streams);
    fill_prefix(st.cu_B, cu_B, shape->n_streams);
    const size_t ws = workspace_bytes_impl(st, shape->n_heads, shape->d_head, head);
    return plan_host(shape, cu_B, head, ws).total;
}

static pafu_status step_host_impl(const pafu_step_args* a, void* arena, size_t arena_bytes, void* stream, int32_t* timeout_word);

pafu_status pafu_step_host(const pafu_step_args* a, void* arena, size_t arena_bytes, void* stream) {
    int32_t word = 0;
    pafu_status e = step_host_impl(a, arena, arena_bytes, stream, &word);
    if (e != PAFU_OK) return e;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return PAFU_ERR_CUDA;
    return word == 0 ? PAFU_OK : PAFU_ERR_TIMEOUT;
}

pafu_status pafu_step_host_async(const pafu_step_args* a, void* arena, size_t arena_bytes, void* stream,
                                 int32_t* timeout_word) {
    if (timeout_word == nullptr) return PAFU_ERR_INVALID_ARG;
    return step_host_impl(a, arena, arena_bytes, stream, timeout_word);
}

static pafu_status step_host_impl(const pafu_step_args* a, void* arena, size_t arena_bytes, void* stream, int32_t* timeout_word) {
    if (a == nullptr || arena == nullptr || a->head == nullptr) return PAFU_ERR_INVALID_ARG;
    pafu_status e = shape_ok(&a->shape, true, true);
    if (e != PAFU_OK) return e;
    if ((reinterpret_cast<uintptr_t>(arena) & 255u) != 0) return PAFU_ERR_MISALIGNED;
    int64_t cu_B[PAFU_MAX_STREAMS + 1];
    e = pafu_kept_counts(&a->shape, a->policy, cu_B);
    if (e != PAFU_OK) return e;
    const pafu_head* h = a->head;
    // everything pafu_step would reject is rejected here, before the first copy is enqueued
    e = head_ok(h, /*device_ptrs=*/false);
    if (e != PAFU_OK) return e;
    if (h->d_in != (int64_t)a->shape.n_heads * a->shape.d_head) return PAFU_ERR_INVALID_ARG;
    if (a->shape.d_head != 64 && a->shape.d_head != 128) return PAFU_ERR_UNSUPPORTED_SHAPE;
    if (!(a->scale >= 0.f) || isinf(a->scale)) return PAFU_ERR_INVALID_ARG;
    const size_t total = pafu_step_host_arena_bytes(&a->shape, a->policy, h);
    if (total == 0) return PAFU_ERR_INVALID_ARG;
    if (arena_bytes < total) return PAFU_ERR_WORKSPACE_TOO_SMALL;
    const int n = a->shape.n_streams;
    const size_t dm = (size_t)a->shape.n_heads * a->shape.d_head;
    const size_t nT = a->shape.cu_T[n], nB = cu_B[n], nQ = a->shape.cu_Lq[n];
    if ((nT > 0 && (!a->K || !a->V || !a->scores)) || (nQ > 0 && (!a->Q || !a->O)) || (nB > 0 && !a->idx))
        return PAFU_ERR_INVALID_ARG;
    if ((a->Kq == nullptr) != (a->Vq == nullptr)) return PAFU_ERR_INVALID_ARG;
    StreamTable st;
    memset(&st, 0, sizeof st);
    st.n_streams = n;
    fill_prefix(st.cu_T, a->shape.cu_T, n);
    fill_prefix(st.cu_Lq, a->shape.cu_Lq, n);
    fill_prefix(st.cu_B, cu_B, n);
    const HostPlan p = plan_host(&a->shape, cu_B, h, workspace_bytes_impl(st, a->shape.n_heads, a->shape.d_head, h));
    uint8_t* base = static_cast<uint8_t*>(arena);
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    auto h2d = [&](size_t off, const void* src, size_t bytes) -> bool {
        if (src == nullptr || bytes == 0) return true;
        return cudaMemcpyAsync(base + off, src, bytes, cudaMemcpyHostToDevice, cs) == cudaSuccess;
    };
    auto d2h = [&](void* dst, size_t off, size_t bytes) -> bool {
        if (dst == nullptr || bytes == 0) return true;
        return cudaMemcpyAsync(dst, base + off, bytes, cudaMemcpyDeviceToHost, cs) == cudaSuccess;
    };
    bool ok = cudaMemsetAsync(base + p.ws, 0, kWsHeaderBytes, cs) == cudaSuccess;
    ok = ok && h2d(p.K, a->K, nT * dm * 2) && h2d(p.V, a->V, nT * dm * 2) && h2d(p.Q, a->Q, nQ * dm * 2) &&
         h2d(p.Kq, a->Kq, nQ * dm * 2) && h2d(p.Vq, a->Vq, nQ * dm * 2) &&
         h2d(p.w1, h->w1, (size_t)h->d_hidden * h->d_in * 2) && h2d(p.b1, h->b1, (size_t)h->d_hidden * 2) &&
         h2d(p.w2, h->w2, (size_t)h->d_out * h->d_hidden * 2) && h2d(p.b2, h->b2, (size_t)h->d_out * 2);
    if (!ok) return PAFU_ERR_CUDA;
    pafu_head dh = *h;
    dh.w1 = reinterpret_cast<const uint16_t*>(base + p.w1);
    dh.b1 = h->b1 ? reinterpret_cast<const uint16_t*>(base + p.b1) : nullptr;
    dh.w2 = reinterpret_cast<const uint16_t*>(base + p.w2);
    dh.b2 = h->b2 ? reinterpret_cast<const uint16_t*>(base + p.b2) : nullptr;
    pafu_step_args d = *a;
    d.head = &dh;
    d.K = reinterpret_cast<const uint16_t*>(base + p.K);
    d.V = reinterpret_cast<const uint16_t*>(base + p.V);
    d.Q = reinterpret_cast<const uint16_t*>(base + p.Q);
    d.Kq = a->Kq ? reinterpret_cast<const uint16_t*>(base + p.Kq) : nullptr;
    d.Vq = a->Vq ? reinterpret_cast<const uint16_t*>(base + p.Vq) : nullptr;
    d.scores = reinterpret_cast<float*>(base + p.scores);
    d.idx = reinterpret_cast<int32_t*>(base + p.idx);
    d.Kc = reinterpret_cast<uint16_t*>(base + p.Kc);
    d.Vc = reinterpret_cast<uint16_t*>(base + p.Vc);
    d.SLc = a->SLc ? reinterpret_cast<float*>(base + p.SLc) : nullptr;
    d.O = reinterpret_cast<uint16_t*>(base + p.O);
    d.LSE = a->LSE ? reinterpret_cast<float*>(base + p.LSE) : nullptr;
    d.ws = base + p.ws;
    d.ws_bytes = p.ws_bytes;
    e = pafu_step(&d, stream);
    if (e != PAFU_OK) return e;
    ok = d2h(a->scores, p.scores, nT * 4) && d2h(a->idx, p.idx, nB * 4) && d2h(a->O, p.O, nQ * dm * 2) &&
         d2h(a->Kc, p.Kc, nB * dm * 2) && d2h(a->Vc, p.Vc, nB * dm * 2) && d2h(a->SLc, p.SLc, nB * 4) &&
         d2h(a->LSE, p.LSE, nQ * a->shape.n_heads * 4) && d2h(timeout_word, p.ws, 4);
    return ok ? PAFU_OK : PAFU_ERR_CUDA;
}

pafu_status pafu_cache_update(pafu_cache* c, const pafu_head* head,
                              const uint16_t* Qs, const uint16_t* Ks, const uint16_t* Vs,
                              const uint16_t* const* Knew, const uint16_t* const* Vnew, int64_t chunk,
                              int32_t* pruned, void* ws, size_t ws_bytes, void* stream) {
    if (pruned != nullptr) *pruned = 0;
    if (c == nullptr || chunk < 0) return PAFU_ERR_INVALID_ARG;
    if (c->n_layers < 1 || c->n_heads < 1 || c->d_head < 1 || c->capacity < 1 || c->n_sink < 0) return PAFU_ERR_INVALID_ARG;
    if (c->n_layers > PAFU_MAX_LAYERS) return PAFU_ERR_UNSUPPORTED_SHAPE;
    if (c->cur != 0 && c->cur != 1) return PAFU_ERR_INVALID_ARG;
    if (c->T < 0 || c->T > c->capacity) return PAFU_ERR_INVALID_ARG;
    const int64_t dm = (int64_t)c->n_heads * c->d_head;
    if (dm % 8 != 0 || dm > 0x7fffffffLL || c->capacity > 0x7fffffffLL) return PAFU_ERR_UNSUPPORTED_SHAPE;
    if (chunk > c->capacity) return PAFU_ERR_TOO_LARGE;
    if (chunk == 0) return PAFU_OK;
    pafu_status e = head_ok(head);
    if (e != PAFU_OK) return e;
    if (head->d_in != 3 * dm) return PAFU_ERR_INVALID_ARG;
    if (head->d_in % (64 * 3) != 0) return PAFU_ERR_UNSUPPORTED_SHAPE;
    if (Qs == nullptr || Ks == nullptr || Vs == nullptr || Knew == nullptr || Vnew == nullptr || c->idx == nullptr)
        return PAFU_ERR_INVALID_ARG;
    if (!aligned16(Qs) || !aligned16(Ks) || !aligned16(Vs) || !aligned16(c->idx)) return PAFU_ERR_MISALIGNED;
    const size_t buf_b = (size_t)c->capacity * dm * 2;
    for (int b = 0; b < 2; ++b) {
        if (c->K[b] == nullptr || c->V[b] == nullptr || c->SL[b] == nullptr) return PAFU_ERR_INVALID_ARG;
        if (!aligned16(c->SL[b])) return PAFU_ERR_MISALIGNED;
    }
    if (ranges_overlap(c->SL[0], (size_t)c->capacity * 4, c->SL[1], (size_t)c->capacity * 4)) return PAFU_ERR_INVALID_ARG;
    for (int l = 0; l < c->n_layers; ++l) {
        if (Knew[l] == nullptr || Vnew[l] == nullptr) return PAFU_ERR_INVALID_ARG;
        if (!aligned16(Knew[l]) || !aligned16(Vnew[l])) return PAFU_ERR_MISALIGNED;
        const void* bufs[4] = {c->K[0][l], c->V[0][l], c->K[1][l], c->V[1][l]};
        for (int i = 0; i < 4; ++i) {
            if (bufs[i] == nullptr) return PAFU_ERR_INVALID_ARG;
            if (!aligned16(bufs[i])) return PAFU_ERR_MISALIGNED;
            // a layer's four buffers are distinct, and none of them is where the new rows come from
            for (int j = i + 1; j < 4; ++j)
                if (ranges_overlap(bufs[i], buf_b, bufs[j], buf_b)) return PAFU_ERR_INVALID_ARG;
            if (ranges_overlap(bufs[i], buf_b, Knew[l], (size_t)chunk * dm * 2) ||
                ranges_overlap(bufs[i], buf_b, Vnew[l], (size_t)chunk * dm * 2)) return PAFU_ERR_INVALID_ARG;
        }
    }
    if (ws == nullptr) return PAFU_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return PAFU_ERR_MISALIGNED;
    if (ws_bytes < kWsHeaderBytes + score_workspace_bytes(*head)) return PAFU_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);

    // 1. the chunk does not fit: keep the sink prefix and the Top-k of SL, in every layer
    if (c->T + chunk > c->capacity) {
        const int64_t keep = c->capacity - chunk;
        if (keep > 0) {
            StreamTable st;
            memset(&st, 0, sizeof st);
            st.n_streams = 1;
            st.cu_T[1] = c->T;
            pafu_shape sh;
            memset(&sh, 0, sizeof sh);
            sh.n_streams = 1; sh.n_heads = c->n_heads; sh.d_head = c->d_head; sh.cu_T = st.cu_T;
            pafu_policy pol;
            pol.n_sink = c->n_sink; pol.n_recent = 0; pol.budget = keep;
            e = fill_policy(&sh, &pol, &st);
            if (e != PAFU_OK) return e;
            e = launch_select(c->SL[c->cur], st, c->idx, cs);
            if (e != PAFU_OK) return e;
            const int o = c->cur ^ 1;
            e = launch_compact_layers(c->K[c->cur], c->V[c->cur], c->n_layers, c->SL[c->cur], c->idx, st, (int32_t)dm,
                                      c->K[o], c->V[o], c->SL[o], cs);
            if (e != PAFU_OK) return e;
        }
        c->cur ^= 1;
        c->T = keep;
        if (pruned != nullptr) *pruned = 1;
    }
    // 2. the chunk's salience scores go straight to the tail of SL
    const uint16_t* parts[3] = {Qs, Ks, Vs};
    e = launch_score(*head, parts, 3, chunk, dm, c->SL[c->cur] + c->T, ws, ws_bytes, cs);
    if (e != PAFU_OK) return e;
    // 3. every layer's new rows go to the tail of its K and V
    {
        StreamTable st;
        memset(&st, 0, sizeof st);
        st.n_streams = 1;
        st.cu_T[1] = chunk;
        st.cu_B[1] = chunk;
        const uint16_t* kd[PAFU_MAX_LAYERS]; const uint16_t* vd[PAFU_MAX_LAYERS];
        uint16_t* ko[PAFU_MAX_LAYERS]; uint16_t* vo[PAFU_MAX_LAYERS];
        for (int l = 0; l < c->n_layers; ++l) {
            kd[l] = Knew[l]; vd[l] = Vnew[l];
            ko[l] = c->K[c->cur][l] + c->T * dm;
            vo[l] = c->V[c->cur][l] + c->T * dm;
        }
        e = launch_compact_layers(kd, vd, c->n_layers, nullptr, nullptr, st, (int32_t)dm, ko, vo, nullptr, cs);
        if (e != PAFU_OK) return e;
    }
    c->T += chunk;
    return PAFU_OK;
}

}  // extern "C"
