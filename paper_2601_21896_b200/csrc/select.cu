// Retained-token selection (Sec. 3.4 inference paragraph; Algorithm 2 "Top-k"; frame sink
// Sec. 4.1): kept = [0, n_sink) U top-k salient of the middle U [T - n_recent, T), written as
// ascending token indices, ties to the lower index.
//
// The step moves a few hundred KB, so it is latency-bound: one CTA of 1024 threads per
// stream, scores read from L2 (once, into registers, when the stream is small enough).
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

constexpr int kSelRows = 32;                          // candidates per thread held in registers
constexpr int kSelRegCap = kSelRows * kSelThreads;    // 32768 candidates
constexpr int kSelList = 2048;                        // survivors of the first pass kept in shared memory

// Streams with at most kSelRegCap candidates: every candidate key is loaded once (all loads in
// flight together) and stays in registers for the three radix passes (12 + 10 + 10 bits) and
// the emission.  Candidate j of the stream sits in row j / 1024 of thread j % 1024, so a warp
// ballot per row plus one block scan over the 32 x 32 (row, warp) counts gives every kept
// candidate its ascending output slot.
__global__ void __launch_bounds__(kSelThreads)
select_regs_kernel(const float* __restrict__ scores, StreamTable st, int32_t* __restrict__ idx) {
    __shared__ int hist[4096];
    __shared__ int cnt[kSelRows * 32];
    __shared__ uint32_t list[kSelList];
    __shared__ int warp_sums[33];
    __shared__ uint32_t sh_prefix;
    __shared__ int sh_krem, sh_bin, sh_nlist;

    const int s = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t T64 = st.cu_T[s + 1] - st.cu_T[s];
    const int64_t B64 = st.cu_B[s + 1] - st.cu_B[s];
    if (B64 >= T64) return;                               // the streaming kernel writes the identity
    const int T = (int)T64;
    const int ns = (int)st.n_sink[s], nr = (int)st.n_recent[s];
    const int k = (int)st.k[s];
    const int c0 = ns, M = T - nr - ns;
    if (M > kSelRegCap) return;                           // the streaming kernel owns this stream
    const float* sc = scores + st.cu_T[s] + c0;
    int32_t* out = idx + st.cu_B[s];

    uint32_t key[kSelRows];
#pragma unroll
    for (int i = 0; i < kSelRows; ++i) {
        const int j = i * kSelThreads + tid;
        key[i] = (j < M) ? score_key(__ldg(sc + j)) : 0u;
    }
    // sink and recent tokens are kept as they are
    for (int t = tid; t < ns; t += kSelThreads) out[t] = t;
    for (int t = tid; t < nr; t += kSelThreads) out[ns + k + t] = T - nr + t;

    uint32_t thr = 0xffffffffu;
    int need_eq = 0, eq_total = 0;
    if (k > 0) {
        uint32_t prefix = 0u, mask = 0u;
        int k_rem = k;
        int shift = 32;
        int n_list = -1;                                  // >= 0: survivors are in list[]
#pragma unroll 1
        for (int pass = 0; pass < 3; ++pass) {
            const int bits = pass == 0 ? 12 : 10;
            const int nb = 1 << bits;
            shift -= bits;
            for (int b = tid; b < nb; b += kSelThreads) hist[b] = 0;
            __syncthreads();
            if (n_list >= 0) {
                // few candidates share the leading digit(s): work on the compacted list
                for (int j = tid; j < n_list; j += kSelThreads) {
                    const uint32_t kv = list[j];
                    if ((kv & mask) == prefix) atomicAdd(&hist[(kv >> shift) & (uint32_t)(nb - 1)], 1);
                }
            } else {
#pragma unroll
                for (int i = 0; i < kSelRows; ++i) {
                    const bool in = (i * kSelThreads + tid < M) && ((key[i] & mask) == prefix);
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
            }
            __syncthreads();
            // thread t owns bins nb-1 - t*bpt ... downwards; the exclusive scan of the per-thread
            // counts is the number of matching candidates in all higher bins
            const int bpt = nb >= kSelThreads ? nb / kSelThreads : 1;
            int mine = 0;
            if (tid * bpt < nb)
                for (int i = 0; i < bpt; ++i) mine += hist[nb - 1 - (tid * bpt + i)];
            int total;
            int above = block_exclusive_scan(mine, warp_sums, &total);
            if (tid * bpt < nb) {
                for (int i = 0; i < bpt; ++i) {
                    const int b = nb - 1 - (tid * bpt + i);
                    const int c = hist[b];
                    if (above < k_rem && k_rem <= above + c) {
                        sh_prefix = prefix | ((uint32_t)b << shift);
                        sh_krem = k_rem - above;
                        sh_bin = c;
                    }
                    above += c;
                }
            }
            if (tid == 0) sh_nlist = 0;
            __syncthreads();
            prefix = sh_prefix;
            k_rem = sh_krem;
            mask |= (uint32_t)(nb - 1) << shift;
            eq_total = sh_bin;                            // after the last pass: keys equal to thr
            if (pass == 0 && sh_bin <= kSelList) {
                // gather the candidates that share the winning leading digit
#pragma unroll
                for (int i = 0; i < kSelRows; ++i)
                    if ((i * kSelThreads + tid < M) && ((key[i] & mask) == prefix))
                        list[atomicAdd(&sh_nlist, 1)] = key[i];
                __syncthreads();
                n_list = sh_nlist;
            }
        }
        thr = prefix;
        need_eq = k_rem;
    }

    // ---- ordered emission.  First the ties: rank of every candidate equal to the threshold.
    const unsigned lt_mask = (1u << lane) - 1u;
    uint32_t keep_bits = 0u;
    int total;
    if (need_eq == eq_total) {
        // every candidate equal to the threshold is taken: no tie to break
#pragma unroll
        for (int i = 0; i < kSelRows; ++i)
            if ((i * kSelThreads + tid < M) && k > 0 && key[i] >= thr) keep_bits |= 1u << i;
    } else {
        uint32_t eq_bits = 0u;                            // bit i: row i equals the threshold
#pragma unroll
        for (int i = 0; i < kSelRows; ++i) {
            const bool eq = (i * kSelThreads + tid < M) && key[i] == thr;
            const unsigned b = __ballot_sync(0xffffffffu, eq);
            if (lane == 0) cnt[i * 32 + warp] = __popc(b);
            if (eq) eq_bits |= 1u << i;
        }
        __syncthreads();
        {
            const int v = cnt[tid];
            const int ex = block_exclusive_scan(v, warp_sums, &total);
            __syncthreads();
            cnt[tid] = ex;
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kSelRows; ++i) {
            const bool valid = i * kSelThreads + tid < M;
            const bool eq = (eq_bits >> i) & 1u;
            const unsigned b = __ballot_sync(0xffffffffu, eq);
            const int rank = cnt[i * 32 + warp] + __popc(b & lt_mask);
            const bool keep = valid && (key[i] > thr || (eq && rank < need_eq));
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
        const int v = cnt[tid];
        const int ex = block_exclusive_scan(v, warp_sums, &total);
        __syncthreads();
        cnt[tid] = ex;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kSelRows; ++i) {
        const bool keep = (keep_bits >> i) & 1u;
        const unsigned b = __ballot_sync(0xffffffffu, keep);
        if (keep) out[ns + cnt[i * 32 + warp] + __popc(b & lt_mask)] = c0 + i * kSelThreads + tid;
    }
}

// Streams with more candidates than the register kernel holds: keys are re-read from L2 in
// every pass (4 passes of 8 bits), and each thread emits a contiguous token range.
__global__ void __launch_bounds__(kSelThreads)
select_stream_kernel(const float* __restrict__ scores, StreamTable st, int32_t* __restrict__ idx) {
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
    bool any_regs = false, any_stream = false;
    for (int s = 0; s < st.n_streams; ++s) {
        const int64_t T = st.cu_T[s + 1] - st.cu_T[s], B = st.cu_B[s + 1] - st.cu_B[s];
        const bool regs = B < T && T - st.n_sink[s] - st.n_recent[s] <= kSelRegCap;
        any_regs |= regs;
        any_stream |= !regs;
    }
    if (any_regs) select_regs_kernel<<<st.n_streams, kSelThreads, 0, stream>>>(scores, st, idx);
    if (any_stream) select_stream_kernel<<<st.n_streams, kSelThreads, 0, stream>>>(scores, st, idx);
    return cuda_ok(cudaGetLastError());
}

}  // namespace pafu
