// Internal declarations shared by the kernels' launchers and the C ABI layer.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/pafu.h"

namespace pafu {

// Per-stream prefix offsets and retention parameters, passed to kernels by value.
struct StreamTable {
    int32_t n_streams;
    int64_t cu_T[PAFU_MAX_STREAMS + 1];   // cache tokens
    int64_t cu_B[PAFU_MAX_STREAMS + 1];   // retained tokens
    int64_t cu_Lq[PAFU_MAX_STREAMS + 1];  // chunk tokens
    int64_t n_sink[PAFU_MAX_STREAMS];     // clamped sink length
    int64_t n_recent[PAFU_MAX_STREAMS];   // clamped recent length
    int64_t k[PAFU_MAX_STREAMS];          // candidates to take by salience
};

// Workspace layout: [0, 256) status header (int32 words), then per-step scratch.
constexpr size_t kWsHeaderBytes = 256;
constexpr int kStatusWordTimeout = 0;   // non-zero: a bounded wait ran out

inline pafu_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? PAFU_OK : PAFU_ERR_CUDA; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// SM count of the current device (148 when no device is visible, e.g. sizing queries on a
// build host); capped so per-CTA tables stay small.
constexpr int kMaxPersistentGrid = 256;
inline int device_sm_count() {
    static int n = 0;
    if (n == 0) {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
            n = v < kMaxPersistentGrid ? v : kMaxPersistentGrid;
        else
            return 148;
    }
    return n;
}

// Every kernel of this library is launched with programmatic stream serialization: its CTAs
// may be scheduled, and run their local set-up, as soon as the preceding kernel's CTAs have
// left the SMs, without waiting for that kernel's completion to be processed first.  In return
// each kernel executes grid_dep_wait() before its first access to global memory; that wait
// returns only when the preceding kernel has completed and its writes are visible.  No kernel
// signals its dependents early: CTAs of a following kernel that sat on the SMs while a
// bandwidth-bound kernel was still in its last wave cost more than the earlier start gained.
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                    cudaStream_t stream, unsigned cluster_x, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = 1;
    if (cluster_x > 1) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = cluster_x;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    cfg.attrs = attr;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Launchers (each enqueues on `stream` and returns the launch status).
pafu_status launch_score(const pafu_head& head, const uint16_t* const* X, int n_parts, int64_t n_tokens, int64_t ldx,
                         float* scores, void* ws, size_t ws_bytes, cudaStream_t stream);
pafu_status launch_select(const float* scores, const StreamTable& st, int32_t* idx,
                          cudaStream_t stream);
pafu_status launch_compact(const uint16_t* K, const uint16_t* V, const float* SL,
                           const int32_t* idx, const StreamTable& st, int32_t d_model,
                           uint16_t* Kc, uint16_t* Vc, float* SLc, cudaStream_t stream);
pafu_status launch_compact_layers(const uint16_t* const* K, const uint16_t* const* V, int32_t n_layers,
                                  const float* SL, const int32_t* idx, const StreamTable& st, int32_t d_model,
                                  uint16_t* const* Kc, uint16_t* const* Vc, float* SLc, cudaStream_t stream);
pafu_status launch_attn(const uint16_t* Q, const uint16_t* Kc, const uint16_t* Vc,
                        const uint16_t* Kq, const uint16_t* Vq, const StreamTable& st,
                        int32_t n_heads, int32_t d_head, float scale, uint16_t* O, float* LSE,
                        void* ws, size_t ws_bytes, cudaStream_t stream);
pafu_status launch_attn_indexed(const uint16_t* Q, const uint16_t* K, const uint16_t* V, const int32_t* idx,
                                const uint16_t* Kq, const uint16_t* Vq, const StreamTable& st,
                                int32_t n_heads, float scale, uint16_t* O, float* LSE,
                                void* ws, size_t ws_bytes, cudaStream_t stream);
bool attn_indexed_supported(const StreamTable& st, int32_t d_head, bool has_chunk);
size_t attn_workspace_bytes(const StreamTable& st, int32_t n_heads, int32_t d_head);
size_t score_workspace_bytes(const pafu_head& head);

}  // namespace pafu
