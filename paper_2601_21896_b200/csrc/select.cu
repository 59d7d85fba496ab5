// Retained-token selection (Sec. 3.4 inference paragraph; Algorithm 2 "Top-k"; frame sink
// Sec. 4.1): kept = [0, n_sink) U top-k salient of the middle U [T - n_recent, T), written as
// ascending token indices, ties to the lower index - and, in the same launch when the caller
// wants it, the cache update that follows it in Algorithm 2: KV <- Select(KV; ids),
// SL <- Select(SL; ids).
//
// Selection moves a few hundred KB, so it is latency-bound; the row gather moves hundreds of MB
// and wants every SM.  One kernel serves both: every CTA that works on a stream repeats that
// stream's selection by itself (the scores are L2-resident; repeating the work costs nothing
// that matters and needs no communication between CTAs), writes its own contiguous share of the
// index list, and then copies exactly those rows.  pafu_select alone runs one CTA per stream.
//   1. fp32 scores map to order-preserving 32-bit keys (-0 folded onto +0, NaN lowest), held
//      in shared memory: whole keys for streams of up to 53 248 candidates, the upper halves
//      for streams of up to 106 496 (the lower halves are then re-read from L2 only for the
//      candidates that share the threshold's upper half).
//   2. MSB-first radix select (11 + 11 + 10 bits, or 11 + 5 per half) over shared-memory
//      histograms finds the key of the k-th largest candidate and how many candidates equal to
//      it are still needed.
//   3. Ordered emission: each thread owns a contiguous candidate range; block-wide exclusive
//      scans (ties seen so far, tokens kept so far) give every kept token its output slot, so
//      the result is ascending and ties resolve to the lowest indices.
// Streams with more candidates than that use one CTA that re-reads L2 in every pass.
#include <type_traits>

#include "common.cuh"

namespace pafu {

constexpr int kSelThreads = 1024;
constexpr int kSelCap32 = 53248;            // candidates whose whole keys fit in shared memory
constexpr int kSelCap16 = 2 * kSelCap32;    // candidates whose upper key halves fit
constexpr int kSelHistBins = 2048;

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

struct SelShared {
    int hist[kSelHistBins];
    int warp_sums[33];
    uint32_t prefix;
    int k_rem, bin_count;
};

// One radix pass over the candidates `get` admits: histogram of `bits` bits at `shift`, then the
// bin that holds the k_rem-th largest admitted key.  get(j, key) returns false for a candidate
// that is out of the running (wrong prefix) and is called with j up to a multiple of the block
// size, so every warp runs the same number of rounds.
template <typename Get>
__device__ __forceinline__ void radix_pass(SelShared& sh, int M, int shift, int bits, uint32_t& prefix,
                                           int& k_rem, int& bin_count, Get get) {
    const int tid = threadIdx.x, lane = tid & 31;
    const int nb = 1 << bits;
    for (int b = tid; b < nb; b += kSelThreads) sh.hist[b] = 0;
    __syncthreads();
    for (int j0 = 0; j0 < M; j0 += kSelThreads) {
        uint32_t key = 0u;
        const bool in = (j0 + tid < M) && get(j0 + tid, key);
        const uint32_t digit = (key >> shift) & (uint32_t)(nb - 1);
        // a warp whose live lanes all hold one digit (equal or saturated scores) adds once
        const unsigned act = __ballot_sync(0xffffffffu, in);
        if (act != 0u) {
            const uint32_t d0 = __shfl_sync(0xffffffffu, digit, __ffs(act) - 1);
            const bool uniform = __all_sync(0xffffffffu, !in || digit == d0);
            if (uniform) { if (lane == __ffs(act) - 1) atomicAdd(&sh.hist[d0], __popc(act)); }
            else if (in) atomicAdd(&sh.hist[digit], 1);
        }
    }
    __syncthreads();
    // bins from the top: thread t holds bins nb-1-2t and nb-2-2t (nb <= 2048 = 2 x block size)
    const int b_hi = nb - 1 - 2 * tid, b_lo = b_hi - 1;
    const int c_hi = b_hi >= 0 ? sh.hist[b_hi] : 0, c_lo = b_lo >= 0 ? sh.hist[b_lo] : 0;
    int total;
    const int above = block_exclusive_scan(c_hi + c_lo, sh.warp_sums, &total);
    if (above < k_rem && k_rem <= above + c_hi) {
        sh.prefix = prefix | ((uint32_t)b_hi << shift); sh.k_rem = k_rem - above; sh.bin_count = c_hi;
    } else if (above + c_hi < k_rem && k_rem <= above + c_hi + c_lo) {
        sh.prefix = prefix | ((uint32_t)b_lo << shift); sh.k_rem = k_rem - above - c_hi; sh.bin_count = c_lo;
    }
    __syncthreads();
    prefix = sh.prefix; k_rem = sh.k_rem; bin_count = sh.bin_count;
}

// Which CTAs work on which stream: stream s owns CTAs [cta0[s], cta0[s + 1]).
struct SelCtaMap {
    int32_t cta0[PAFU_MAX_STREAMS + 1];
};

// WIDE = false: whole 32-bit keys in shared memory.  WIDE = true: upper 16 bits only.
// Writes out[lo, hi) of the stream's ascending index list (lo, hi: this CTA's share of the kept rows).
template <bool WIDE>
__device__ __forceinline__ void select_rows(SelShared& sh, void* key_smem, const float* __restrict__ sc, int M, int k,
                                            int ns, int nr, int T, int32_t* __restrict__ out, int lo, int hi) {
    typedef typename std::conditional<WIDE, uint16_t, uint32_t>::type KeyT;
    KeyT* keys = static_cast<KeyT*>(key_smem);
    const int tid = threadIdx.x;
    for (int j = tid; j < M; j += kSelThreads) {
        const uint32_t kx = score_key(__ldg(sc + j));
        keys[j] = (KeyT)(WIDE ? (kx >> 16) : kx);
    }
    // always-kept tokens of this CTA's share
    const int B = ns + k + nr;
    for (int p = lo + tid; p < hi; p += kSelThreads) {
        if (p < ns) out[p] = p;
        else if (p >= ns + k) out[p] = T - B + p;            // T - nr + (p - ns - k)
    }
    __syncthreads();
    if (k == 0) return;                                      // block-uniform

    // ---- the key of the k-th largest candidate
    uint32_t thr = 0u;         // WIDE: the upper half, then (refined) the whole key
    int need_eq = k, eq_total = 0;
    bool refined = false;      // WIDE only: the lower halves took part
    if (!WIDE) {
        uint32_t mask = 0u;
        const int shifts[3] = {21, 10, 0}, widths[3] = {11, 11, 10};
#pragma unroll 1
        for (int pass = 0; pass < 3; ++pass) {
            const uint32_t m = mask, pf = thr;
            radix_pass(sh, M, shifts[pass], widths[pass], thr, need_eq, eq_total,
                       [&](int j, uint32_t& key) { key = keys[j]; return (key & m) == pf; });
            mask |= ((1u << widths[pass]) - 1u) << shifts[pass];
        }
    } else {
        uint32_t hi16 = 0u;
        {
            radix_pass(sh, M, 5, 11, hi16, need_eq, eq_total,
                       [&](int j, uint32_t& key) { key = keys[j]; return true; });
            const uint32_t pf = hi16;
            radix_pass(sh, M, 0, 5, hi16, need_eq, eq_total,
                       [&](int j, uint32_t& key) { key = keys[j]; return (key & 0xffe0u) == pf; });
        }
        if (need_eq == eq_total) {
            thr = hi16;        // every candidate that shares the upper half is taken: the lower halves do not matter
        } else {
            refined = true;
            uint32_t lo16 = 0u;
            const uint32_t h = hi16;
            radix_pass(sh, M, 5, 11, lo16, need_eq, eq_total, [&](int j, uint32_t& key) {
                if (keys[j] != h) return false;
                key = score_key(__ldg(sc + j)) & 0xffffu;
                return true;
            });
            const uint32_t pf = lo16;
            radix_pass(sh, M, 0, 5, lo16, need_eq, eq_total, [&](int j, uint32_t& key) {
                if (keys[j] != h) return false;
                key = score_key(__ldg(sc + j)) & 0xffffu;
                return (key & 0xffe0u) == pf;
            });
            thr = (hi16 << 16) | lo16;
        }
    }

    // 2: above the threshold, 1: equal to it, 0: below
    auto classify = [&](int j) -> int {
        if (!WIDE) {
            const uint32_t kx = keys[j];
            return kx > thr ? 2 : (kx == thr ? 1 : 0);
        }
        const uint32_t h = keys[j];
        if (!refined) return h > thr ? 2 : (h == thr ? 1 : 0);
        const uint32_t th = thr >> 16;
        if (h != th) return h > th ? 2 : 0;
        const uint32_t l = score_key(__ldg(sc + j)) & 0xffffu, tl = thr & 0xffffu;
        return l > tl ? 2 : (l == tl ? 1 : 0);
    };

    // ---- ordered emission: thread t owns candidates [t * per, (t + 1) * per), per odd (no bank conflicts)
    const int per = ((M + kSelThreads - 1) / kSelThreads) | 1;
    const int j0 = min(M, tid * per), j1 = min(M, j0 + per);
    int gt = 0, eq = 0;
    for (int j = j0; j < j1; ++j) {
        const int c = classify(j);
        gt += (c == 2); eq += (c == 1);
    }
    int total;
    int eq_taken = eq;
    int eq_before = 0;
    if (need_eq != eq_total) {                               // block-uniform: ties to break, lowest indices win
        eq_before = block_exclusive_scan(eq, sh.warp_sums, &total);
        eq_taken = min(eq, max(0, need_eq - eq_before));
    }
    int pos = ns + block_exclusive_scan(gt + eq_taken, sh.warp_sums, &total);
    if (pos < hi && pos + gt + eq_taken > lo) {
        const int c0 = ns;
        int e = 0;
        for (int j = j0; j < j1; ++j) {
            const int c = classify(j);
            const bool keep = c == 2 || (c == 1 && e++ < eq_taken);
            if (keep) {
                if (pos >= lo && pos < hi) out[pos] = c0 + j;
                ++pos;
            }
        }
    }
}

__device__ __forceinline__ uint4 ld_stream_v4(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

constexpr int kSelCopyUnroll = 6;    // 6 x 32 lanes x 16 B = one 3072-byte row (d_model 1536)

// COPY = false: indices only (pafu_select).  COPY = true: each CTA also gathers the K, V (and SL)
// rows of its share of the index list (Algorithm 2's Select(KV; ids) in the same launch).
template <bool COPY>
__global__ void __launch_bounds__(kSelThreads, 1)
select_compact_kernel(const float* __restrict__ scores, const __grid_constant__ StreamTable st,
                      const __grid_constant__ SelCtaMap cm, int32_t* __restrict__ idx,
                      const uint4* __restrict__ K, const uint4* __restrict__ V, const float* __restrict__ SL,
                      int32_t chunks_per_row, uint4* __restrict__ Kc, uint4* __restrict__ Vc, float* __restrict__ SLc) {
    extern __shared__ __align__(16) unsigned char sel_keys[];
    __shared__ SelShared sh;
    grid_dep_wait();
    int s = 0;
    while (s + 1 < st.n_streams && (int)blockIdx.x >= cm.cta0[s + 1]) ++s;
    const int r = (int)blockIdx.x - cm.cta0[s], G = cm.cta0[s + 1] - cm.cta0[s];
    const int64_t T64 = st.cu_T[s + 1] - st.cu_T[s], B64 = st.cu_B[s + 1] - st.cu_B[s];
    if (r < 0 || r >= G || B64 == 0) return;                 // block-uniform
    const int T = (int)T64, B = (int)B64;
    // a stream that keeps everything is one long "sink"
    const bool all = B >= T;
    const int ns = all ? T : (int)st.n_sink[s], nr = all ? 0 : (int)st.n_recent[s], k = all ? 0 : (int)st.k[s];
    const int M = T - ns - nr;
    if (M > kSelCap16) return;                               // the streaming kernel owns this stream
    const int lo = (int)((int64_t)B * r / G), hi = (int)((int64_t)B * (r + 1) / G);
    int32_t* out = idx + st.cu_B[s];
    const float* sc = scores + st.cu_T[s] + ns;
    if (M <= kSelCap32) select_rows<false>(sh, sel_keys, sc, M, k, ns, nr, T, out, lo, hi);
    else select_rows<true>(sh, sel_keys, sc, M, k, ns, nr, T, out, lo, hi);
    if (!COPY) return;
    __syncthreads();                                         // out[lo, hi) was written by this CTA's threads
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int row = lo + warp; row < hi; row += kSelThreads / 32) {
        const int64_t src_row = st.cu_T[s] + (int64_t)__ldcg(out + row);
        const int64_t dst_row = st.cu_B[s] + row;
#pragma unroll 1
        for (int t = 0; t < 2; ++t) {
            const uint4* src = (t ? V : K) + src_row * chunks_per_row;
            uint4* dst = (t ? Vc : Kc) + dst_row * chunks_per_row;
            for (int c0 = 0; c0 < chunks_per_row; c0 += 32 * kSelCopyUnroll) {
                uint4 buf[kSelCopyUnroll];
#pragma unroll
                for (int u = 0; u < kSelCopyUnroll; ++u) {
                    const int c = c0 + u * 32 + lane;
                    if (c < chunks_per_row) buf[u] = ld_stream_v4(src + c);
                }
#pragma unroll
                for (int u = 0; u < kSelCopyUnroll; ++u) {
                    const int c = c0 + u * 32 + lane;
                    if (c < chunks_per_row) dst[c] = buf[u];
                }
            }
        }
        if (SLc != nullptr && lane == 0) SLc[dst_row] = __ldg(SL + src_row);
    }
}

// Streams with more candidates than shared memory holds: keys are re-read from L2 in every pass
// (4 passes of 8 bits), and each thread emits a contiguous token range.
__global__ void __launch_bounds__(kSelThreads)
select_stream_kernel(const float* __restrict__ scores, StreamTable st, int32_t* __restrict__ idx) {
    grid_dep_wait();
    {
        const int64_t T = st.cu_T[blockIdx.x + 1] - st.cu_T[blockIdx.x], B = st.cu_B[blockIdx.x + 1] - st.cu_B[blockIdx.x];
        if (B >= T || T - st.n_sink[blockIdx.x] - st.n_recent[blockIdx.x] <= kSelCap16) return;   // the other kernel owns this stream
    }
    __shared__ int hist[256];
    __shared__ int warp_sums[33];
    __shared__ uint32_t sh_prefix;
    __shared__ int sh_krem;

    const int s = blockIdx.x;
    const int tid = threadIdx.x;
    const int64_t T64 = st.cu_T[s + 1] - st.cu_T[s];
    const float* sc = scores + st.cu_T[s];
    int32_t* out = idx + st.cu_B[s];
    const int T = (int)T64;
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

namespace {
struct SelClass {
    bool any_smem = false, any_stream = false;
    size_t smem_bytes = 0;
};
SelClass classify_streams(const StreamTable& st) {
    SelClass c;
    for (int s = 0; s < st.n_streams; ++s) {
        const int64_t T = st.cu_T[s + 1] - st.cu_T[s], B = st.cu_B[s + 1] - st.cu_B[s];
        if (B == 0) continue;
        const int64_t M = B >= T ? 0 : T - st.n_sink[s] - st.n_recent[s];
        if (M > kSelCap16) { c.any_stream = true; continue; }
        c.any_smem = true;
        const size_t need = M <= kSelCap32 ? (size_t)M * 4 : (size_t)M * 2;
        if (need > c.smem_bytes) c.smem_bytes = need;
    }
    c.smem_bytes = (c.smem_bytes + 15) / 16 * 16;
    return c;
}
bool set_smem_limit() {
    static bool done[kMaxDevices] = {};
    return once_per_device(done, [] {
        const int cap = kSelCap32 * 4;
        return cudaFuncSetAttribute(select_compact_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, cap) == cudaSuccess &&
               cudaFuncSetAttribute(select_compact_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, cap) == cudaSuccess;
    });
}
}  // namespace

pafu_status launch_select(const float* scores, const StreamTable& st, int32_t* idx, cudaStream_t stream) {
    if (st.n_streams == 0 || st.cu_B[st.n_streams] == 0) return PAFU_OK;
    const SelClass c = classify_streams(st);
    if (c.any_smem) {
        if (!set_smem_limit()) return PAFU_ERR_CUDA;
        SelCtaMap cm;
        for (int s = 0; s <= PAFU_MAX_STREAMS; ++s) cm.cta0[s] = s < st.n_streams ? s : st.n_streams;
        if (launch_dependent(select_compact_kernel<false>, dim3((unsigned)st.n_streams), dim3(kSelThreads), c.smem_bytes, stream, 1,
                             scores, st, cm, idx, (const uint4*)nullptr, (const uint4*)nullptr, (const float*)nullptr, 0,
                             (uint4*)nullptr, (uint4*)nullptr, (float*)nullptr) != cudaSuccess)
            return PAFU_ERR_CUDA;
    }
    if (c.any_stream &&
        launch_dependent(select_stream_kernel, dim3((unsigned)st.n_streams), dim3(kSelThreads), 0, stream, 1, scores, st,
                         idx) != cudaSuccess)
        return PAFU_ERR_CUDA;
    return PAFU_OK;
}

// True when selection and row gather of this geometry can run as one launch.
bool select_compact_fusable(const StreamTable& st) {
    const SelClass c = classify_streams(st);
    return c.any_smem && !c.any_stream;
}

// Selection and the gather of the selected rows in one launch: the SMs are shared out among the
// streams in proportion to the rows each keeps.
pafu_status launch_select_compact(const float* scores, const StreamTable& st, int32_t* idx, const uint16_t* K,
                                  const uint16_t* V, const float* SL, int32_t d_model, uint16_t* Kc, uint16_t* Vc,
                                  float* SLc, cudaStream_t stream) {
    const int64_t rows = st.cu_B[st.n_streams];
    if (st.n_streams == 0 || rows == 0) return PAFU_OK;
    const SelClass c = classify_streams(st);
    if (!set_smem_limit()) return PAFU_ERR_CUDA;
    int n_live = 0;
    for (int s = 0; s < st.n_streams; ++s) n_live += st.cu_B[s + 1] > st.cu_B[s];
    const int grid = device_sm_count() > n_live ? device_sm_count() : n_live;
    // every live stream gets one CTA, the rest go where the rows are
    SelCtaMap cm;
    int share[PAFU_MAX_STREAMS], given = 0;
    for (int s = 0; s < st.n_streams; ++s) {
        const int64_t B = st.cu_B[s + 1] - st.cu_B[s];
        share[s] = B > 0 ? 1 + (int)((int64_t)(grid - n_live) * B / rows) : 0;
        given += share[s];
    }
    for (int s = 0; given < grid; s = (s + 1) % st.n_streams)
        if (share[s] > 0) { ++share[s]; ++given; }
    cm.cta0[0] = 0;
    for (int s = 0; s < PAFU_MAX_STREAMS; ++s) cm.cta0[s + 1] = cm.cta0[s] + (s < st.n_streams ? share[s] : 0);
    return cuda_ok(launch_dependent(select_compact_kernel<true>, dim3((unsigned)grid), dim3(kSelThreads), c.smem_bytes, stream, 1,
                                    scores, st, cm, idx, reinterpret_cast<const uint4*>(K), reinterpret_cast<const uint4*>(V), SL,
                                    d_model / 8, reinterpret_cast<uint4*>(Kc), reinterpret_cast<uint4*>(Vc), SLc));
}

}  // namespace pafu
