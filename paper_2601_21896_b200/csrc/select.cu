// Retained-token selection (Sec. 3.4 inference paragraph; Algorithm 2 "Top-k"; frame sink
// Sec. 4.1): kept = [0, n_sink) U top-k salient of the middle U [T - n_recent, T), written as
// ascending token indices, ties to the lower index.
//
// The step moves a few hundred KB, so it is latency-bound: a cluster of eight CTAs per stream
// with the candidates in registers (streams up to 131072 candidates), one CTA re-reading L2
// for longer streams.
//   1. fp32 scores map to order-preserving 32-bit keys (-0 folded onto +0, NaN lowest).
//   2. MSB-first radix select (4 passes of 8 bits, shared-memory histograms) finds the key of
//      the k-th largest candidate and how many candidates equal to it are still needed.
//   3. Ordered emission: each thread owns a contiguous token range; two block-wide exclusive
//      scans (ties seen so far, tokens kept so far) give every kept token its output slot,
//      so the result is ascending and ties resolve to the lowest indices.
#include <cooperative_groups.h>

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

constexpr int kSelCluster = 8;                        // CTAs cooperating on one stream
constexpr int kSelRowsSmall = 4, kSelRowsLarge = 16;  // candidates per thread held in registers
constexpr int kSelCapSmall = kSelCluster * kSelRowsSmall * kSelThreads;   // 32768 candidates
constexpr int kSelRegCap = kSelCluster * kSelRowsLarge * kSelThreads;     // 131072 candidates

// Streams with at most kSelRegCap candidates: a cluster of eight CTAs per stream.  Candidate j
// lives in CTA j / (ROWS * 1024), row (j / 1024) % ROWS, thread j % 1024, loaded once and kept in
// registers; ROWS = 4 serves streams up to 32768 candidates, ROWS = 16 those up to 131072 (a
// 93 600-token cache), each stream by exactly one of the two instantiations.
// Every radix pass (12 + 10 + 10 bits) builds one shared-memory histogram per CTA; CTA r then
// sums slice r of the bins over all eight histograms through distributed shared memory, the
// slice totals are exchanged, and the CTA whose slice holds the k-th largest key finds the bin
// and tells the others.  Emission: warp ballots per row, one block scan over the 4 x 32
// (row, warp) counts, and the CTA totals exchanged through distributed shared memory give every
// kept candidate its ascending output slot.
template <int kSelRows>
__global__ void __launch_bounds__(kSelThreads)
select_cluster_kernel(const float* __restrict__ scores, StreamTable st, int32_t* __restrict__ idx) {
    constexpr int kSelPerCta = kSelRows * kSelThreads;
    constexpr int kCap = kSelCluster * kSelPerCta;
    constexpr int kCapBelow = kSelRows == kSelRowsSmall ? 0 : kSelCapSmall;    // smaller streams: the other instantiation
    grid_dep_wait();
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    __shared__ int hist[4096];
    __shared__ int red[512];              // this CTA's slice of the cluster-wide histogram
    __shared__ int slice_tot[kSelCluster];
    __shared__ int cta_cnt[2][kSelCluster];   // per-CTA tie counts / keep counts
    __shared__ int cnt[kSelRows * 32];
    __shared__ int warp_sums[33];
    __shared__ uint32_t sh_prefix;
    __shared__ int sh_krem, sh_bin;

    const int s = blockIdx.x / kSelCluster;
    const int rank = (int)cluster.block_rank();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t T64 = st.cu_T[s + 1] - st.cu_T[s];
    const int64_t B64 = st.cu_B[s + 1] - st.cu_B[s];
    // cluster-uniform exits (before any cluster barrier)
    if (B64 >= T64) return;                               // the streaming kernel writes the identity
    const int T = (int)T64;
    const int ns = (int)st.n_sink[s], nr = (int)st.n_recent[s];
    const int k = (int)st.k[s];
    const int c0 = ns, M = T - nr - ns;
    if (M > kCap || M <= kCapBelow) return;               // another kernel owns this stream
    const float* sc = scores + st.cu_T[s] + c0;
    int32_t* out = idx + st.cu_B[s];
    const int j0 = rank * kSelPerCta;

    uint32_t key[kSelRows];
#pragma unroll
    for (int i = 0; i < kSelRows; ++i) {
        const int j = j0 + i * kSelThreads + tid;
        key[i] = (j < M) ? score_key(__ldg(sc + j)) : 0u;
    }
    // sink and recent tokens are kept as they are (spread over the cluster)
    for (int t = rank * kSelThreads + tid; t < ns; t += kSelCluster * kSelThreads) out[t] = t;
    for (int t = rank * kSelThreads + tid; t < nr; t += kSelCluster * kSelThreads) out[ns + k + t] = T - nr + t;

    uint32_t thr = 0xffffffffu;
    int need_eq = 0, eq_total = 0;
    if (k > 0) {
        uint32_t prefix = 0u, mask = 0u;
        int k_rem = k;
        int shift = 32;
#pragma unroll 1
        for (int pass = 0; pass < 3; ++pass) {
            const int bits = pass == 0 ? 12 : 10;
            const int nb = 1 << bits;
            const int slice = nb / kSelCluster;           // 512 or 128 bins per CTA
            shift -= bits;
            for (int b = tid; b < nb; b += kSelThreads) hist[b] = 0;
            __syncthreads();
#pragma unroll
            for (int i = 0; i < kSelRows; ++i) {
                const bool in = (j0 + i * kSelThreads + tid < M) && ((key[i] & mask) == prefix);
                const uint32_t digit = (key[i] >> shift) & (uint32_t)(nb - 1);
                // a warp whose live lanes all hold one digit (equal or saturated scores) adds once
                const unsigned act = __ballot_sync(0xffffffffu, in);
                if (act != 0u) {
                    const uint32_t d0 = __shfl_sync(0xffffffffu, digit, __ffs(act) - 1);
                    const bool uniform = __all_sync(0xffffffffu, !in || digit == d0);
                    if (uniform) { if (lane == __ffs(act) - 1) atomicAdd(&hist[d0], __popc(act)); }
                    else if (in) atomicAdd(&hist[digit], 1);
                }
            }
            cluster.sync();                                // every CTA's histogram is complete
            // slice `rank` of the bins, summed over the cluster
            int mine = 0;
            if (tid < slice) {
                const int b = rank * slice + tid;
#pragma unroll
                for (int c = 0; c < kSelCluster; ++c) mine += *cluster.map_shared_rank(&hist[b], c);
                red[tid] = mine;
            }
            int total;
            // within the slice, higher bins first: thread t holds bin slice-1-t for the scan below
            const int mine_desc = (tid < slice) ? 0 : 0;
            (void)mine_desc;
            block_exclusive_scan(mine, warp_sums, &total);     // only the total is needed here
            if (tid == 0) {
#pragma unroll
                for (int c = 0; c < kSelCluster; ++c) *cluster.map_shared_rank(&slice_tot[rank], c) = total;
            }
            cluster.sync();                                // slice totals and red[] visible
            // which slice holds the k-th largest matching key (slices scanned from the top)
            int above = 0, q = kSelCluster - 1;
            for (; q > 0; --q) {
                if (k_rem <= above + slice_tot[q]) break;
                above += slice_tot[q];
            }
            if (rank == q) {
                // find the bin inside this slice: descending order, exclusive scan of counts
                const int v = (tid < slice) ? red[slice - 1 - tid] : 0;
                int tt;
                const int ab = above + block_exclusive_scan(v, warp_sums, &tt);
                if (tid < slice && ab < k_rem && k_rem <= ab + v) {
                    const uint32_t bin = (uint32_t)(rank * slice + slice - 1 - tid);
                    const uint32_t np = prefix | (bin << shift);
                    for (int c = 0; c < kSelCluster; ++c) {
                        *cluster.map_shared_rank(&sh_prefix, c) = np;
                        *cluster.map_shared_rank(&sh_krem, c) = k_rem - ab;
                        *cluster.map_shared_rank(&sh_bin, c) = v;
                    }
                }
            }
            cluster.sync();                                // the decision has reached every CTA
            prefix = sh_prefix;
            k_rem = sh_krem;
            eq_total = sh_bin;                             // after the last pass: keys equal to thr
            mask |= (uint32_t)(nb - 1) << shift;
        }
        thr = prefix;
        need_eq = k_rem;
    }

    // ---- ordered emission
    const unsigned lt_mask = (1u << lane) - 1u;
    uint32_t keep_bits = 0u;
    int total;
    if (need_eq == eq_total) {
        // every candidate equal to the threshold is taken: no tie to break
#pragma unroll
        for (int i = 0; i < kSelRows; ++i)
            if ((j0 + i * kSelThreads + tid < M) && k > 0 && key[i] >= thr) keep_bits |= 1u << i;
    } else {
        uint32_t eq_bits = 0u;
#pragma unroll
        for (int i = 0; i < kSelRows; ++i) {
            const bool eq = (j0 + i * kSelThreads + tid < M) && key[i] == thr;
            const unsigned b = __ballot_sync(0xffffffffu, eq);
            if (lane == 0) cnt[i * 32 + warp] = __popc(b);
            if (eq) eq_bits |= 1u << i;
        }
        __syncthreads();
        const int v = (tid < kSelRows * 32) ? cnt[tid] : 0;
        const int ex = block_exclusive_scan(v, warp_sums, &total);
        __syncthreads();
        if (tid < kSelRows * 32) cnt[tid] = ex;
        if (tid == 0)
            for (int c = 0; c < kSelCluster; ++c) *cluster.map_shared_rank(&cta_cnt[0][rank], c) = total;
        cluster.sync();
        int eq_before = 0;
        for (int c = 0; c < rank; ++c) eq_before += cta_cnt[0][c];
#pragma unroll
        for (int i = 0; i < kSelRows; ++i) {
            const bool valid = j0 + i * kSelThreads + tid < M;
            const bool eq = (eq_bits >> i) & 1u;
            const unsigned b = __ballot_sync(0xffffffffu, eq);
            const int rk = eq_before + cnt[i * 32 + warp] + __popc(b & lt_mask);
            const bool keep = valid && (key[i] > thr || (eq && rk < need_eq));
            if (keep) keep_bits |= 1u << i;
        }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kSelRows; ++i) {
        const unsigned b = __ballot_sync(0xffffffffu, (keep_bits >> i) & 1u);
        if (lane == 0) cnt[i * 32 + warp] = __popc(b);
    }
    __syncthreads();
    {
        const int v = (tid < kSelRows * 32) ? cnt[tid] : 0;
        const int ex = block_exclusive_scan(v, warp_sums, &total);
        __syncthreads();
        if (tid < kSelRows * 32) cnt[tid] = ex;
        if (tid == 0)
            for (int c = 0; c < kSelCluster; ++c) *cluster.map_shared_rank(&cta_cnt[1][rank], c) = total;
    }
    cluster.sync();
    int kept_before = 0;
    for (int c = 0; c < rank; ++c) kept_before += cta_cnt[1][c];
#pragma unroll
    for (int i = 0; i < kSelRows; ++i) {
        const bool keep = (keep_bits >> i) & 1u;
        const unsigned b = __ballot_sync(0xffffffffu, keep);
        if (keep) out[ns + kept_before + cnt[i * 32 + warp] + __popc(b & lt_mask)] = c0 + j0 + i * kSelThreads + tid;
    }
    cluster.sync();      // no CTA may exit while another can still write into its shared memory
}

// Streams with more candidates than the register kernel holds: keys are re-read from L2 in
// every pass (4 passes of 8 bits), and each thread emits a contiguous token range.
__global__ void __launch_bounds__(kSelThreads)
select_stream_kernel(const float* __restrict__ scores, StreamTable st, int32_t* __restrict__ idx) {
    grid_dep_wait();
    if (st.cu_T[blockIdx.x + 1] - st.cu_T[blockIdx.x] - st.n_sink[blockIdx.x] - st.n_recent[blockIdx.x] <= kSelRegCap &&
        st.cu_B[blockIdx.x + 1] - st.cu_B[blockIdx.x] < st.cu_T[blockIdx.x + 1] - st.cu_T[blockIdx.x]) return;   // the register kernel owns this stream
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
    // both kernels run over all streams; each stream is handled by exactly one of them
    bool any_small = false, any_large = false, any_stream = false;
    for (int s = 0; s < st.n_streams; ++s) {
        const int64_t T = st.cu_T[s + 1] - st.cu_T[s], B = st.cu_B[s + 1] - st.cu_B[s];
        const int64_t M = T - st.n_sink[s] - st.n_recent[s];
        const bool regs = B < T && M <= kSelRegCap;
        any_small |= regs && M <= kSelCapSmall;
        any_large |= regs && M > kSelCapSmall;
        any_stream |= !regs;
    }
    if (any_small &&
        launch_dependent(select_cluster_kernel<kSelRowsSmall>, dim3((unsigned)(st.n_streams * kSelCluster)), dim3(kSelThreads), 0,
                         stream, kSelCluster, scores, st, idx) != cudaSuccess)
        return PAFU_ERR_CUDA;
    if (any_large &&
        launch_dependent(select_cluster_kernel<kSelRowsLarge>, dim3((unsigned)(st.n_streams * kSelCluster)), dim3(kSelThreads), 0,
                         stream, kSelCluster, scores, st, idx) != cudaSuccess)
        return PAFU_ERR_CUDA;
    if (any_stream &&
        launch_dependent(select_stream_kernel, dim3((unsigned)st.n_streams), dim3(kSelThreads), 0, stream, 1, scores, st,
                         idx) != cudaSuccess)
        return PAFU_ERR_CUDA;
    return cuda_ok(cudaGetLastError());
}

}  // namespace pafu
