// Retained-token selection (Sec. 3.4 inference paragraph; Algorithm 2 "Top-k"; frame sink
// Sec. 4.1): kept = [0, n_sink) U top-k salient of the middle U [T - n_recent, T), written as
// ascending token indices, ties to the lower index.
//
// The step moves a few hundred KB, so it is latency-bound: one launch, one CTA of 1024
// threads per stream, scores read from L2.
//   1. fp32 scores map to order-preserving 32-bit keys (-0 folded onto +0, NaN lowest).
//   2. MSB-first radix select (4 passes of 8 bits, shared-memory histograms) finds the key of
//      the k-th largest candidate and how many candidates equal to it are still needed.
//   3. Ordered emission: each thread owns a contiguous token range; two block-wide exclusive
//      scans (ties seen so far, tokens kept so far) give every kept token its output slot,
//      so the result is ascending and ties resolve to the lowest indices.
#include "common.cuh"

namespace pafu {

constexpr int kSelThreads = 1024;

__device__ __forceinline__ uint32_t score_key(float f) {
    uint32_t u = __float_as_uint(f);
    if ((u & 0x7fffffffu) > 0x7f800000u) return 0u;      // NaN: below -inf
    if (u == 0x80000000u) u = 0u;                        // -0 == +0
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Exclusive prefix sum of one int per thread over the block; also returns the block total.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums, int* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    __syncthreads();                 // protect warp_sums from the previous use
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int w = warp_sums[lane];
        int winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int n = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += n;
        }
        warp_sums[lane] = winc - w;  // exclusive offset of each warp
        if (lane == 31) warp_sums[32] = winc;
    }
    __syncthreads();
    *total = warp_sums[32];
    return warp_sums[warp] + inc - v;
}

__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ scores, StreamTable st, int32_t* __restrict__ idx) {
    __shared__ int hist[256];
    __shared__ int warp_sums[33];
    __shared__ uint32_t sh_prefix;
    __shared__ int sh_krem;

    const int s = blockIdx.x;
    const int tid = threadIdx.x;
    const int64_t T64 = st.cu_T[s + 1] - st.cu_T[s];
    const int64_t B64 = st.cu_B[s + 1] - st.cu_B[s];
    const float* sc = scores + st.cu_T[s];
    int32_t* out = idx + st.cu_B[s];
    const int T = (int)T64;
    if (B64 >= T64) {                                   // nothing to evict
        for (int t = tid; t < T; t += kSelThreads) out[t] = t;
        return;
    }
    const int ns = (int)st.n_sink[s], nr = (int)st.n_recent[s];
    const int k = (int)st.k[s];
    const int c0 = ns, c1 = T - nr;                     // candidates [c0, c1)

    // ---- radix select: key of the k-th largest candidate
    uint32_t thr = 0xffffffffu;
    int need_eq = 0;
    if (k > 0) {
        uint32_t prefix = 0u, mask = 0u;
        int k_rem = k;
        for (int pass = 0; pass < 4; ++pass) {
            const int shift = 24 - 8 * pass;
            if (tid < 256) hist[tid] = 0;
            __syncthreads();
            for (int t = c0 + tid; t < c1; t += kSelThreads) {
                const uint32_t key = score_key(sc[t]);
                if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
            }
            __syncthreads();
            if (tid < 32) {
                int cnt[8];
                int mine = 0;
#pragma unroll
                for (int b = 0; b < 8; ++b) { cnt[b] = hist[tid * 8 + b]; mine += cnt[b]; }
                // number of matching candidates in bins above this lane's bins
                int suf = mine;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    int n = __shfl_down_sync(0xffffffffu, suf, o);
                    if (tid + o < 32) suf += n;
                }
                int above = suf - mine;
#pragma unroll
                for (int b = 7; b >= 0; --b) {
                    if (above < k_rem && k_rem <= above + cnt[b]) {
                        sh_prefix = prefix | ((uint32_t)(tid * 8 + b) << shift);
                        sh_krem = k_rem - above;
                    }
                    above += cnt[b];
                }
            }
            __syncthreads();
            prefix = sh_prefix;
            k_rem = sh_krem;
            mask |= 0xffu << shift;
        }
        thr = prefix;
        need_eq = k_rem;
    }

    // ---- ordered emission
    const int per = (T + kSelThreads - 1) / kSelThreads;
    const int t0 = min(T, tid * per), t1 = min(T, t0 + per);
    int eqc = 0;
    for (int t = max(t0, c0); t < min(t1, c1); ++t) eqc += (score_key(sc[t]) == thr);
    int total;
    const int eq_before = block_exclusive_scan(eqc, warp_sums, &total);
    int kc = 0, e = eq_before;
    for (int t = t0; t < t1; ++t) {
        bool keep = (t < c0) || (t >= c1);
        if (!keep) {
            const uint32_t key = score_key(sc[t]);
            keep = key > thr;
            if (key == thr) { keep = e < need_eq; ++e; }
        }
        kc += keep;
    }
    int pos = block_exclusive_scan(kc, warp_sums, &total);
    e = eq_before;
    for (int t = t0; t < t1; ++t) {
        bool keep = (t < c0) || (t >= c1);
        if (!keep) {
            const uint32_t key = score_key(sc[t]);
            keep = key > thr;
            if (key == thr) { keep = e < need_eq; ++e; }
        }
        if (keep) out[pos++] = t;
    }
}

pafu_status launch_select(const float* scores, const StreamTable& st, int32_t* idx,
                          cudaStream_t stream) {
    if (st.n_streams == 0 || st.cu_B[st.n_streams] == 0) return PAFU_OK;
    select_kernel<<<st.n_streams, kSelThreads, 0, stream>>>(scores, st, idx);
    return cuda_ok(cudaGetLastError());
}

}  // namespace pafu
