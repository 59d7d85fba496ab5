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

// One warp copies row src_row of K and V (and the salience entry) to row dst_row of Kc and Vc.
__device__ __forceinline__ void copy_kv_row(const uint4* __restrict__ K, const uint4* __restrict__ V,
                                            const float* __restrict__ SL, int64_t src_row, int64_t dst_row,
                                            int chunks_per_row, uint4* __restrict__ Kc, uint4* __restrict__ Vc,
                                            float* __restrict__ SLc, int lane) {
    const uint4* ks = K + src_row * chunks_per_row;
    const uint4* vs = V + src_row * chunks_per_row;
    uint4* kd = Kc + dst_row * chunks_per_row;
    uint4* vd = Vc + dst_row * chunks_per_row;
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
    if (SLc != nullptr && lane == 0) SLc[dst_row] = __ldg(SL + src_row);
}

// always_first = 0: wait for the preceding kernel, then copy every kept row through the index list.
// always_first = 1 (inside a layer step, directly behind the selection kernels, which let their
// dependents start at once): the rows that are kept whatever the scores say - sink and recent
// tokens, and all tokens of a stream that keeps everything - are copied first, while the
// selection still runs on its few SMs; only then does the kernel wait for the indices and copy
// the top-k rows.  K and V are not written by the step's earlier kernels, and the outputs are
// not read by them, so the early part touches nothing the predecessor produces.  (SL is the
// score array in a step: all of its entries are copied after the wait.)
// When the selection occupies more than two SMs, rows are handed out through two counters in the
// workspace header (`work`: early rows, late rows, finished blocks), one row per claim with the
// next claim under way during the copy: the blocks that only get an SM when the selection's CTAs
// leave simply find less work left, instead of starting a fixed share late (that tail cost 40 us
// at the batch-4 size); the last block to finish puts the counters back to zero.  With a one- or
// two-CTA selection the grid leaves those SMs out and every block takes a fixed share
// (early_static; 5 us faster at the 28 080-token cache than claiming).
constexpr int kCompactClaim = 1;

// A claim in two halves: lane 0 issues the add; its result is fetched (and shared with the warp)
// only when the rows are needed, so the trip to L2 overlaps the copying in between.
__device__ __forceinline__ int claim_issue(int* counter, int lane) {
    return lane == 0 ? atomicAdd(counter, kCompactClaim) : 0;
}
__device__ __forceinline__ int64_t claim_get(int pending) { return __shfl_sync(0xffffffffu, pending, 0); }

__global__ void __launch_bounds__(kCompactWarpsPerBlock * 32)
compact_rows_kernel(const uint4* __restrict__ K, const uint4* __restrict__ V,
                    const float* __restrict__ SL, const int32_t* __restrict__ idx,
                    const __grid_constant__ StreamTable st, int32_t chunks_per_row,
                    uint4* __restrict__ Kc, uint4* __restrict__ Vc, float* __restrict__ SLc,
                    int64_t n_rows, int* __restrict__ work, int early_static) {
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (int64_t)blockIdx.x * kCompactWarpsPerBlock + (threadIdx.x >> 5);
    const int64_t n_warps = (int64_t)gridDim.x * kCompactWarpsPerBlock;
    if (work == nullptr) {
        grid_dep_wait();
        for (int64_t r = warp0; r < n_rows; r += n_warps) {
            int s = 0;
            while (s + 1 < st.n_streams && r >= st.cu_B[s + 1]) ++s;
            copy_kv_row(K, V, SL, st.cu_T[s] + (int64_t)__ldg(idx + r), r, chunks_per_row, Kc, Vc, SLc, lane);
        }
        return;
    }
    // part 1: always-kept rows, enumerated stream by stream (A_s = n_sink + n_recent of them, or all T)
    int64_t n_always = 0;
    for (int s = 0; s < st.n_streams; ++s) {
        const int64_t T = st.cu_T[s + 1] - st.cu_T[s], B = st.cu_B[s + 1] - st.cu_B[s];
        n_always += B >= T ? T : st.n_sink[s] + st.n_recent[s];
    }
    auto copy_always = [&](int64_t a) {
        int s = 0;
        int64_t p = a;
        for (;; ++s) {
            const int64_t T = st.cu_T[s + 1] - st.cu_T[s], B = st.cu_B[s + 1] - st.cu_B[s];
            const int64_t A = B >= T ? T : st.n_sink[s] + st.n_recent[s];
            if (p < A) break;
            p -= A;
        }
        const int64_t T = st.cu_T[s + 1] - st.cu_T[s], B = st.cu_B[s + 1] - st.cu_B[s];
        const int64_t ns = B >= T ? T : st.n_sink[s], k = B >= T ? 0 : st.k[s], A = B >= T ? T : ns + st.n_recent[s];
        // position p < ns is token p; position ns + k + i is token T - n_recent + i
        const int64_t pos = p < ns ? p : p + k, tok = p < ns ? p : T - A + p;
        copy_kv_row(K, V, nullptr, st.cu_T[s] + tok, st.cu_B[s] + pos, chunks_per_row, Kc, Vc, nullptr, lane);
    };
    auto copy_top = [&](int64_t q) {
        int s = 0;
        int64_t p = q;
        for (; p >= st.k[s]; ++s) p -= st.k[s];
        const int64_t r = st.cu_B[s] + st.n_sink[s] + p;
        copy_kv_row(K, V, SL, st.cu_T[s] + (int64_t)__ldg(idx + r), r, chunks_per_row, Kc, Vc, SLc, lane);
    };
    int64_t n_top = 0;
    for (int s = 0; s < st.n_streams; ++s) n_top += st.k[s];
    auto fill_always_sl = [&]() {
        if (SLc == nullptr) return;
        for (int64_t a = warp0 * 32 + lane; a < n_rows; a += n_warps * 32) {
            int s = 0;
            while (s + 1 < st.n_streams && a >= st.cu_B[s + 1]) ++s;
            const int64_t ns = st.n_sink[s], k = st.k[s], p = a - st.cu_B[s];
            if (k == 0 || p < ns || p >= ns + k) SLc[a] = __ldg(SL + st.cu_T[s] + __ldg(idx + a));
        }
    };
    if (early_static) {
        // every block is resident from the start (the launcher sized the grid for it): fixed shares
        for (int64_t a = warp0; a < n_always; a += n_warps) copy_always(a);
        grid_dep_wait();
        fill_always_sl();
        for (int64_t q = warp0; q < n_top; q += n_warps) copy_top(q);
        return;
    }
    int pending = claim_issue(work + 0, lane);
    for (int64_t base = claim_get(pending); base < n_always; base = claim_get(pending)) {
        pending = claim_issue(work + 0, lane);
        for (int64_t a = base; a < base + kCompactClaim && a < n_always; ++a) copy_always(a);
    }
    // part 2: the selection's result
    grid_dep_wait();
    fill_always_sl();
    pending = claim_issue(work + 1, lane);
    for (int64_t base = claim_get(pending); base < n_top; base = claim_get(pending)) {
        pending = claim_issue(work + 1, lane);
        for (int64_t q = base; q < base + kCompactClaim && q < n_top; ++q) copy_top(q);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(work + 2, 1) == (int)gridDim.x - 1) {      // every block is past its last claim
            work[0] = 0; work[1] = 0; work[2] = 0;
        }
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
        // idx == nullptr: the rows in order (a plain copy of every layer's rows)
        const int64_t src_row = st.cu_T[s] + (idx != nullptr ? (int64_t)__ldg(idx + r) : r - st.cu_B[s]);
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

// `work`: three zeroed 32-bit words of device memory (the step's workspace header) - then the
// always-kept rows are copied before the kernel waits for its predecessor, which must be
// launch_select of the same step and runs on `select_ctas` CTAs; nullptr: plain gather after the
// predecessor.
pafu_status launch_compact(const uint16_t* K, const uint16_t* V, const float* SL,
                           const int32_t* idx, const StreamTable& st, int32_t d_model,
                           uint16_t* Kc, uint16_t* Vc, float* SLc, cudaStream_t stream, int* work, int select_ctas) {
    const int64_t n_rows = st.cu_B[st.n_streams];
    if (n_rows == 0) return PAFU_OK;
    const int32_t chunks = d_model / 8;
    int64_t blocks = (n_rows + kCompactWarpsPerBlock - 1) / kCompactWarpsPerBlock;
    // A few resident waves, larger inputs loop.  With the early part the grid is what the device
    // holds at once (three blocks fit on an SM): a block must not queue behind blocks that are
    // waiting for the selection.  Fixed shares: the selection's SMs are left out of the count.
    const int early_static = work != nullptr && select_ctas <= 2;
    int sms = device_sm_count() - (early_static ? select_ctas : 0);
    if (sms < 1) sms = 1;
    const int64_t max_blocks = work != nullptr ? (int64_t)sms * 3 : 148 * 8 * 4;
    if (blocks > max_blocks) blocks = max_blocks;
    return cuda_ok(launch_dependent(compact_rows_kernel, dim3((unsigned)blocks), dim3(kCompactWarpsPerBlock * 32), 0, stream, 1,
                                    reinterpret_cast<const uint4*>(K), reinterpret_cast<const uint4*>(V), SL, idx, st,
                                    chunks, reinterpret_cast<uint4*>(Kc), reinterpret_cast<uint4*>(Vc), SLc, n_rows, work,
                                    early_static));
}

}  // namespace pafu
