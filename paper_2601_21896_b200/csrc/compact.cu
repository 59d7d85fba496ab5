// KV <- Select(KV; ids), SL <- Select(SL; ids) (Algorithm 2): row gather of the kept tokens.
//
// HBM-bound copy.  One warp moves one kept token: its K row and its V row (d_model bf16 each)
// in 16-byte pieces, all loads of a batch issued before the first store so that each warp
// keeps up to 12 x 512 B in flight.  Rows are contiguous, so every access is fully coalesced;
// the only indirection is one int32 index per row.
#include "common.cuh"

namespace pafu {

constexpr int kCompactWarpsPerBlock = 8;
constexpr int kCompactUnroll = 6;   // 6 x 32 lanes x 16 B = one 3072-byte row (d_model 1536)

__device__ __forceinline__ uint4 ld_nc_v4(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__global__ void __launch_bounds__(kCompactWarpsPerBlock * 32)
compact_rows_kernel(const uint4* __restrict__ K, const uint4* __restrict__ V,
                    const float* __restrict__ SL, const int32_t* __restrict__ idx,
                    StreamTable st, int32_t chunks_per_row,
                    uint4* __restrict__ Kc, uint4* __restrict__ Vc, float* __restrict__ SLc,
                    int64_t n_rows) {
    grid_dep_wait();
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (int64_t)blockIdx.x * kCompactWarpsPerBlock + (threadIdx.x >> 5);
    const int64_t n_warps = (int64_t)gridDim.x * kCompactWarpsPerBlock;
    for (int64_t r = warp0; r < n_rows; r += n_warps) {
        int s = 0;
        while (s + 1 < st.n_streams && r >= st.cu_B[s + 1]) ++s;
        const int64_t src_row = st.cu_T[s] + (int64_t)__ldg(idx + r);
        const uint4* ks = K + src_row * chunks_per_row;
        const uint4* vs = V + src_row * chunks_per_row;
        uint4* kd = Kc + r * chunks_per_row;
        uint4* vd = Vc + r * chunks_per_row;
        for (int c0 = 0; c0 < chunks_per_row; c0 += 32 * kCompactUnroll) {
            uint4 kb[kCompactUnroll], vb[kCompactUnroll];
#pragma unroll
            for (int u = 0; u < kCompactUnroll; ++u) {
                const int c = c0 + u * 32 + lane;
                if (c < chunks_per_row) { kb[u] = ld_nc_v4(ks + c); vb[u] = ld_nc_v4(vs + c); }
            }
#pragma unroll
            for (int u = 0; u < kCompactUnroll; ++u) {
                const int c = c0 + u * 32 + lane;
                if (c < chunks_per_row) { kd[c] = kb[u]; vd[c] = vb[u]; }
            }
        }
        if (SLc != nullptr && lane == 0) SLc[r] = __ldg(SL + src_row);
    }
}

// The same gather for several layers' caches at once: the paper takes the Top-k at the final
// layer only and applies those indices to every layer (Sec. 3.3), so one index list serves
// n_layers K/V pairs.  One warp moves one (layer, kept token) pair of rows; the layer is the
// slowest index, so a warp's accesses stay contiguous and the index list is re-read from L2.
struct LayerPtrs {
    const uint4* K[PAFU_MAX_LAYERS];
    const uint4* V[PAFU_MAX_LAYERS];
    uint4* Kc[PAFU_MAX_LAYERS];
    uint4* Vc[PAFU_MAX_LAYERS];
};

__global__ void __launch_bounds__(kCompactWarpsPerBlock * 32)
compact_layers_kernel(const __grid_constant__ LayerPtrs lp, int32_t n_layers,
                      const float* __restrict__ SL, const int32_t* __restrict__ idx,
                      const __grid_constant__ StreamTable st, int32_t chunks_per_row,
                      float* __restrict__ SLc, int64_t n_rows) {
    grid_dep_wait();
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (int64_t)blockIdx.x * kCompactWarpsPerBlock + (threadIdx.x >> 5);
    const int64_t n_warps = (int64_t)gridDim.x * kCompactWarpsPerBlock;
    for (int64_t w = warp0; w < n_rows * n_layers; w += n_warps) {
        const int layer = (int)(w / n_rows);
        const int64_t r = w - (int64_t)layer * n_rows;
        int s = 0;
        while (s + 1 < st.n_streams && r >= st.cu_B[s + 1]) ++s;
        const int64_t src_row = st.cu_T[s] + (int64_t)__ldg(idx + r);
        const uint4* ks = lp.K[layer] + src_row * chunks_per_row;
        const uint4* vs = lp.V[layer] + src_row * chunks_per_row;
        uint4* kd = lp.Kc[layer] + r * chunks_per_row;
        uint4* vd = lp.Vc[layer] + r * chunks_per_row;
        for (int c0 = 0; c0 < chunks_per_row; c0 += 32 * kCompactUnroll) {
            uint4 kb[kCompactUnroll], vb[kCompactUnroll];
#pragma unroll
            for (int u = 0; u < kCompactUnroll; ++u) {
                const int c = c0 + u * 32 + lane;
                if (c < chunks_per_row) { kb[u] = ld_nc_v4(ks + c); vb[u] = ld_nc_v4(vs + c); }
            }
#pragma unroll
            for (int u = 0; u < kCompactUnroll; ++u) {
                const int c = c0 + u * 32 + lane;
                if (c < chunks_per_row) { kd[c] = kb[u]; vd[c] = vb[u]; }
            }
        }
        if (layer == 0 && SLc != nullptr && lane == 0) SLc[r] = __ldg(SL + src_row);
    }
}

pafu_status launch_compact_layers(const uint16_t* const* K, const uint16_t* const* V, int32_t n_layers,
                                  const float* SL, const int32_t* idx, const StreamTable& st, int32_t d_model,
                                  uint16_t* const* Kc, uint16_t* const* Vc, float* SLc, cudaStream_t stream) {
    const int64_t n_rows = st.cu_B[st.n_streams];
    if (n_rows == 0 || n_layers == 0) return PAFU_OK;
    LayerPtrs lp;
    for (int l = 0; l < PAFU_MAX_LAYERS; ++l) {
        const int i = l < n_layers ? l : 0;
        lp.K[l] = reinterpret_cast<const uint4*>(K[i]); lp.V[l] = reinterpret_cast<const uint4*>(V[i]);
        lp.Kc[l] = reinterpret_cast<uint4*>(Kc[i]); lp.Vc[l] = reinterpret_cast<uint4*>(Vc[i]);
    }
    int64_t blocks = (n_rows * n_layers + kCompactWarpsPerBlock - 1) / kCompactWarpsPerBlock;
    const int64_t max_blocks = 148 * 8 * 4;
    if (blocks > max_blocks) blocks = max_blocks;
    return cuda_ok(launch_dependent(compact_layers_kernel, dim3((unsigned)blocks), dim3(kCompactWarpsPerBlock * 32), 0, stream, 1,
                                    lp, n_layers, SL, idx, st, d_model / 8, SLc, n_rows));
}

pafu_status launch_compact(const uint16_t* K, const uint16_t* V, const float* SL,
                           const int32_t* idx, const StreamTable& st, int32_t d_model,
                           uint16_t* Kc, uint16_t* Vc, float* SLc, cudaStream_t stream) {
    const int64_t n_rows = st.cu_B[st.n_streams];
    if (n_rows == 0) return PAFU_OK;
    const int32_t chunks = d_model / 8;
    int64_t blocks = (n_rows + kCompactWarpsPerBlock - 1) / kCompactWarpsPerBlock;
    const int64_t max_blocks = 148 * 8 * 4;   // a few resident waves; larger inputs loop
    if (blocks > max_blocks) blocks = max_blocks;
    return cuda_ok(launch_dependent(compact_rows_kernel, dim3((unsigned)blocks), dim3(kCompactWarpsPerBlock * 32), 0, stream, 1,
                                    reinterpret_cast<const uint4*>(K), reinterpret_cast<const uint4*>(V), SL, idx, st,
                                    chunks, reinterpret_cast<uint4*>(Kc), reinterpret_cast<uint4*>(Vc), SLc, n_rows));
}

}  // namespace pafu
