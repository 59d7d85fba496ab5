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
// Diagnostic counters of the tcgen05 attention kernel, one count per (softmax warp, key tile):
constexpr int kStatusWordFullFirst = 8;    // exact pass on a run's first tile or a segment's ragged last tile
constexpr int kStatusWordFullSum = 9;      // exact pass forced by a row sum that outgrew the running maximum
constexpr int kStatusWordRescale = 10;     // output accumulator and row sum rescaled in tensor memory
// Test hook: while this word is non-zero the attention kernel's loader role issues no copies, so
// every consumer's bounded wait runs out and the kernel unwinds with PAFU_ERR_TIMEOUT.
constexpr int kStatusWordStallLoader = 32;
// Work counters of the row gather inside a layer step (three words; back to zero when it ends).
constexpr int kStatusWordGatherWork = 16;

inline pafu_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? PAFU_OK : PAFU_ERR_CUDA; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// SM count of the current device (148 when no device is visible, e.g. sizing queries on a
// build host); capped so per-CTA tables stay small.
constexpr int kMaxPersistentGrid = 256;
constexpr int kMaxDevices = 64;       // per-device caches below are indexed by the CUDA device ordinal
inline int current_device() {
    int dev = 0;
    return (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices) ? dev : -1;
}
inline int device_sm_count() {
    static int n[kMaxDevices] = {};
    const int dev = current_device();
    if (dev < 0) return 148;
    if (n[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
            n[dev] = v < kMaxPersistentGrid ? v : kMaxPersistentGrid;
        else
            return 148;
    }
    return n[dev];
}
// Runs `set` (the cudaFuncSetAttribute calls of one kernel family) once per device; `done` is
// that family's per-device record.  Function attributes belong to the device's context, so a
// process that uses several GPUs has to opt in on each of them.
template <typename Set>
inline bool once_per_device(bool (&done)[kMaxDevices], Set set) {
    const int dev = current_device();
    if (dev < 0) return false;
    if (!done[dev]) {
        if (!set()) return false;
        done[dev] = true;
    }
    return true;
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
// Lets the kernel launched behind this one (as a programmatic dependent) start now; that kernel
// still sees this one's results only after its own grid_dep_wait().
__device__ __forceinline__ void grid_dep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
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
int select_cta_count(const StreamTable& st);      // CTAs launch_select's kernels occupy for this geometry
// work != nullptr (three zeroed words of the workspace header): the rows that are kept whatever
// the scores say are copied before the kernel waits for its predecessor (only valid when that
// predecessor is launch_select of the same step)
pafu_status launch_compact(const uint16_t* K, const uint16_t* V, const float* SL,
                           const int32_t* idx, const StreamTable& st, int32_t d_model,
                           uint16_t* Kc, uint16_t* Vc, float* SLc, cudaStream_t stream, int* work = nullptr,
                           int select_ctas = 0);
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
