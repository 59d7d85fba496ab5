// Retained-token selection (Sec. 3.4 inference paragraph; Algorithm 2 "Top-k"; frame sink
// Sec. 4.1): kept = [0, n_sink) U top-k salient of the middle U [T - n_recent, T), written as
// ascending token indices, ties to the lower index - and, in the same launch when the caller
// wants it, the cache update that follows it in Algorithm 2: KV <- Select(KV; ids),
// SL <- Select(SL; ids).
//
// Selection moves a few hundred KB, so it is latency-bound; the row gather moves hundreds of MB
// and wants every SM.  One kernel serves both.  Every CTA that works on a stream repeats that
// stream's selection by itself (the scores are L2-resident; repeating the work costs nothing
// that matters and needs no communication between CTAs), writes its own share of the index list
// and copies exactly those rows.  Inside a CTA half of the warps select while the other half
// already copy the CTA's share of the rows that are kept whatever the scores say (sink and recent
// tokens); when the threshold is known all warps copy the CTA's share of the top-k rows.
// pafu_select alone runs one CTA per stream with every warp selecting.
//   1. fp32 scores map to order-preserving 32-bit keys (-0 folded onto +0, NaN lowest), held in
//      shared memory: whole keys for streams of up to kSelCap32 candidates, the upper halves for
//      streams of up to twice that (the lower halves are then re-read from L2 only for the
//      candidates that share the threshold's upper half).
//   2. MSB-first radix select (11 + 11 + 10 bits, or 11 + 5 per half) over shared-memory
//      histograms finds the key of the k-th largest candidate and how many candidates equal to
//      it are still needed.  The first histogram is kept in several copies (lanes spread over
//      them) because scores crowd into few leading-digit bins and adds to one address are served
//      one after the other; after the first digit the surviving candidates are few and move to
//      a short list that the later passes read instead of the whole array.
//   3. Ordered emission: candidate j belongs to (round, warp, lane) = (j / threads, ...), warp
//      ballots count kept and tied candidates per (round, warp), block-wide scans over those
//      counts give every kept token its output slot, so the result is ascending and ties resolve
//      to the lowest indices.
// Streams with more candidates than that use one CTA that re-reads L2 in every pass.
#include <type_traits>

#include "common.cuh"

namespace pafu {

constexpr int kSelThreads = 1024;
constexpr int kSelCap32 = 45056;            // candidates whose whole keys fit in shared memory (176 KiB)
constexpr int kSelCap16 = 2 * kSelCap32;    // candidates whose upper key halves fit
constexpr int kSelHistBins = 2048;
constexpr int kSelListCap = 4096;           // candidates the later passes can take from the short list
constexpr int kSelBatch = 8;                // independent loads a thread keeps in flight

__device__ __forceinline__ uint32_t score_key(float f) {
    uint32_t u = __float_as_uint(f);
    if ((u & 0x7fffffffu) > 0x7f800000u) return 0u;      // NaN: below -inf
    if (u == 0x80000000u) u = 0u;                        // -0 == +0
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Exclusive prefix sum of one int per thread over the block; also returns the block total.
__device__ __forceinline__ int sel_exclusive_scan(int v, int* warp_sums, int* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    __syncthreads();                // protect warp_sums from the previous use
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
    int warp_sums[33];
    uint32_t prefix;
    int k_rem, bin_count, list_n;
};

// One radix pass over n candidates: histogram of `bits` bits at `shift`, then the bin that holds
// the k_rem-th largest admitted key.  get(j, key) returns false for a candidate that is out of
// the running.  (Spreading the lanes over several copies of the histogram, or grouping equal
// digits with match.any before adding, did not make the adds cheaper: a shared-memory add costs
// about 13 clocks per warp instruction whether or not its lanes collide.)
template <typename Get>
__device__ __forceinline__ void radix_pass(SelShared& sh, int* hist, int n, int shift, int bits,
                                           uint32_t& prefix, int& k_rem, int& bin_count, Get get) {
    constexpr int NTHR = kSelThreads;
    const int tid = threadIdx.x;
    const int nb = 1 << bits;
    for (int b = tid; b < nb; b += NTHR) hist[b] = 0;
    __syncthreads();
    for (int j0 = 0; j0 < n; j0 += NTHR * kSelBatch) {
        uint32_t key[kSelBatch];
        bool in[kSelBatch];
#pragma unroll
        for (int u = 0; u < kSelBatch; ++u) {
            const int j = j0 + u * NTHR + tid;
            key[u] = 0u;
            in[u] = (j < n) && get(j, key[u]);
        }
#pragma unroll
        for (int u = 0; u < kSelBatch; ++u)
            if (in[u]) atomicAdd(&hist[(key[u] >> shift) & (uint32_t)(nb - 1)], 1);
    }
    __syncthreads();
    // bins from the top: thread t holds q consecutive bins nb-1-q*t ... (q = nb / NTHR, at least 1)
    const int q = nb > NTHR ? nb / NTHR : 1;
    int c[4] = {0, 0, 0, 0};      // q <= 4: 2048 bins over 512 threads
    int mine = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int b = nb - 1 - (q * tid + i);
        if (i < q && b >= 0) {
            c[i] = hist[b];
            mine += c[i];
        }
    }
    int total;
    int above = sel_exclusive_scan(mine, sh.warp_sums, &total);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (i < q && above < k_rem && k_rem <= above + c[i]) {
            sh.prefix = prefix | ((uint32_t)(nb - 1 - (q * tid + i)) << shift);
            sh.k_rem = k_rem - above;
            sh.bin_count = c[i];
        }
        above += c[i];
    }
    __syncthreads();
    prefix = sh.prefix; k_rem = sh.k_rem; bin_count = sh.bin_count;
}

// Shared-memory plan of one launch (host-computed, the same for every CTA).
struct SelSmem {
    int32_t keys_bytes;       // key array; the short list and the histogram / pair tables follow it
};

// Selection of one stream by the first NTHR threads of the block.  WIDE = false: whole 32-bit keys
// in shared memory; WIDE = true: upper 16 bits only.  Writes out[ns + q_lo, ns + q_hi): this CTA's
// share of the top-k part of the stream's ascending index list.
template <bool WIDE>
__device__ __forceinline__ void select_rows(SelShared& sh, unsigned char* smem, const SelSmem& plan,
                                            const float* __restrict__ sc, int M, int k, int ns,
                                            int32_t* __restrict__ out, int q_lo, int q_hi) {
    typedef typename std::conditional<WIDE, uint16_t, uint32_t>::type KeyT;
    KeyT* keys = reinterpret_cast<KeyT*>(smem);
    uint32_t* list = reinterpret_cast<uint32_t*>(smem + plan.keys_bytes);
    int* hist = reinterpret_cast<int*>(smem + plan.keys_bytes + kSelListCap * 4);
    constexpr int NTHR = kSelThreads, NW = NTHR / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int j0 = tid; j0 < M; j0 += NTHR * kSelBatch) {
        float v[kSelBatch];
#pragma unroll
        for (int u = 0; u < kSelBatch; ++u) {
            const int j = j0 + u * NTHR;
            v[u] = j < M ? __ldg(sc + j) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < kSelBatch; ++u) {
            const int j = j0 + u * NTHR;
            const uint32_t kx = score_key(v[u]);
            if (j < M) keys[j] = (KeyT)(WIDE ? (kx >> 16) : kx);
        }
    }
    if (tid == 0) sh.list_n = 0;
    __syncthreads();

    // ---- the key of the k-th largest candidate
    uint32_t thr = 0u;         // WIDE: the upper half, then (refined) the whole key
    int need_eq = k, eq_total = 0;
    bool refined = false;      // WIDE only: the lower halves took part
    constexpr int kTopShift = WIDE ? 5 : 21;
    // first digit over all candidates, histogram in several copies
    radix_pass(sh, hist, M, kTopShift, 11, thr, need_eq, eq_total,
                     [&](int j, uint32_t& key) { key = keys[j]; return true; });
    // the survivors go to the short list if they fit (any order: only their values matter now)
    const bool listed = eq_total <= kSelListCap;             // block-uniform
    if (listed) {
        const uint32_t top = thr >> kTopShift;
        for (int j0 = 0; j0 < M; j0 += NTHR) {
            const int j = j0 + tid;
            const uint32_t kx = j < M ? (uint32_t)keys[j] : 0u;
            const bool hit = j < M && (kx >> kTopShift) == top;
            const unsigned b = __ballot_sync(0xffffffffu, hit);
            if (b != 0u) {
                int base = 0;
                if (lane == 0) base = atomicAdd(&sh.list_n, __popc(b));
                base = __shfl_sync(0xffffffffu, base, 0);
                // WIDE: the candidate's index is listed (its lower half may have to be fetched)
                if (hit) list[base + __popc(b & ((1u << lane) - 1u))] = WIDE ? (uint32_t)j : kx;
            }
        }
        __syncthreads();
    }
    const int n_rest = listed ? eq_total : M;
    if (!WIDE) {
        const uint32_t pf1 = thr;
        radix_pass(sh, hist, n_rest, 10, 11, thr, need_eq, eq_total, [&](int j, uint32_t& key) {
            key = listed ? list[j] : keys[j];
            return (key & 0xffe00000u) == pf1;
        });
        const uint32_t pf2 = thr;
        radix_pass(sh, hist, n_rest, 0, 10, thr, need_eq, eq_total, [&](int j, uint32_t& key) {
            key = listed ? list[j] : keys[j];
            return (key & 0xfffffc00u) == pf2;
        });
    } else {
        const uint32_t pf1 = thr;
        radix_pass(sh, hist, n_rest, 0, 5, thr, need_eq, eq_total, [&](int j, uint32_t& key) {
            key = listed ? (uint32_t)keys[list[j]] : (uint32_t)keys[j];
            return (key & 0xffe0u) == pf1;
        });
        if (need_eq != eq_total) {
            // candidates that share the threshold's upper half outnumber what is still needed: their
            // lower halves decide (re-read from the scores; only those candidates are touched)
            refined = true;
            const uint32_t h = thr;
            uint32_t lo16 = 0u;
            auto low_half = [&](int j, uint32_t& key) {
                const int jj = listed ? (int)list[j] : j;
                if ((uint32_t)keys[jj] != h) return false;
                key = score_key(__ldg(sc + jj)) & 0xffffu;
                return true;
            };
            radix_pass(sh, hist, n_rest, 5, 11, lo16, need_eq, eq_total, low_half);
            const uint32_t pf = lo16;
            radix_pass(sh, hist, n_rest, 0, 5, lo16, need_eq, eq_total, [&](int j, uint32_t& key) {
                return low_half(j, key) && (key & 0xffe0u) == pf;
            });
            thr = (h << 16) | lo16;
        }
        // the emission must not wait for memory: the class of every candidate (2 above the threshold,
        // 1 equal, 0 below) replaces its key first, lower halves fetched in batches
        const uint32_t th = refined ? (thr >> 16) : thr, tl = thr & 0xffffu;
        for (int j0 = tid; j0 < M; j0 += NTHR * kSelBatch) {
            uint32_t h[kSelBatch];
            float v[kSelBatch];
#pragma unroll
            for (int u = 0; u < kSelBatch; ++u) {
                const int j = j0 + u * NTHR;
                h[u] = j < M ? (uint32_t)keys[j] : 0u;
                v[u] = (j < M && refined && h[u] == th) ? __ldg(sc + j) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < kSelBatch; ++u) {
                const int j = j0 + u * NTHR;
                int c = h[u] > th ? 2 : (h[u] == th ? 1 : 0);
                if (refined && c == 1) {
                    const uint32_t l = score_key(v[u]) & 0xffffu;
                    c = l > tl ? 2 : (l == tl ? 1 : 0);
                }
                if (j < M) keys[j] = (KeyT)c;
            }
        }
        __syncthreads();
    }
    auto classify = [&](int j) -> int {
        const uint32_t kx = keys[j];
        if (WIDE) return (int)kx;
        return kx > thr ? 2 : (kx == thr ? 1 : 0);
    };

    // ---- ordered emission.  Candidate j = (round * NW + warp) * 32 + lane; per (round, warp) pair
    // the counts of candidates above the threshold and equal to it (one byte each) go to shared
    // memory, scans over the pairs turn them into output slots.
    const bool ties = need_eq != eq_total;                   // block-uniform: some equal candidates stay out
    const int rounds = (M + NTHR - 1) / NTHR, n_pairs = rounds * NW;
    uint16_t* cnt = reinterpret_cast<uint16_t*>(hist);       // [n_pairs]: above | equal << 8
    int* slot = reinterpret_cast<int*>(hist) + 2048;         // [n_pairs]: kept before the pair (hist has >= 2048 ints more)
    // a thread's candidates' classes stay in registers as bit masks (rounds <= 96)
    uint32_t gtb[3], eqb[3];
#pragma unroll
    for (int blk = 0; blk < 3; ++blk) {
        uint32_t g = 0u, e = 0u;
        const int i_end = min(rounds, (blk + 1) * 32);
        for (int i = blk * 32; i < i_end; ++i) {
            const int j = i * NTHR + tid;
            const int c = j < M ? classify(j) : 0;
            const unsigned bg = __ballot_sync(0xffffffffu, c == 2), be = __ballot_sync(0xffffffffu, c == 1);
            if (lane == 0) cnt[i * NW + warp] = (uint16_t)(__popc(bg) | (__popc(be) << 8));
            g |= (uint32_t)(c == 2) << (i & 31);
            e |= (uint32_t)(c == 1) << (i & 31);
        }
        gtb[blk] = g; eqb[blk] = e;
    }
    __syncthreads();
    // thread t owns pairs [t * per, (t + 1) * per)
    const int per = (n_pairs + NTHR - 1) / NTHR;
    const int p0 = min(n_pairs, tid * per), p1 = min(n_pairs, p0 + per);
    int total;
    int eq_before = 0;
    if (ties) {
        int e = 0;
        for (int p = p0; p < p1; ++p) e += cnt[p] >> 8;
        eq_before = sel_exclusive_scan(e, sh.warp_sums, &total);
    }
    {
        int kept = 0, e = eq_before;
        for (int p = p0; p < p1; ++p) {
            const int g = cnt[p] & 0xff, q = cnt[p] >> 8;
            const int take = ties ? min(q, max(0, need_eq - e)) : q;
            e += q;
            kept += g + take;
        }
        int pos = sel_exclusive_scan(kept, sh.warp_sums, &total);
        e = eq_before;
        for (int p = p0; p < p1; ++p) {
            const int g = cnt[p] & 0xff, q = cnt[p] >> 8;
            const int take = ties ? min(q, max(0, need_eq - e)) : q;
            slot[p] = pos | (take << 24);                    // take <= 32; pos < 2^24 (k < 106 496)
            e += q;
            pos += g + take;
        }
    }
    __syncthreads();
    const unsigned lt = (1u << lane) - 1u;
#pragma unroll
    for (int blk = 0; blk < 3; ++blk) {
        const int i_end = min(rounds, (blk + 1) * 32);
        for (int i = blk * 32; i < i_end; ++i) {
            const bool is_gt = (gtb[blk] >> (i & 31)) & 1u, is_eq = (eqb[blk] >> (i & 31)) & 1u;
            const int sl = slot[i * NW + warp];
            bool keep = is_gt || is_eq;
            if (ties) {
                const unsigned be = __ballot_sync(0xffffffffu, is_eq);
                keep = is_gt || (is_eq && __popc(be & lt) < (sl >> 24));
            }
            const unsigned bk = __ballot_sync(0xffffffffu, keep);
            const int pos = (sl & 0xffffff) + __popc(bk & lt);
            if (keep && pos >= q_lo && pos < q_hi) out[ns + pos] = ns + i * NTHR + tid;
        }
    }
}

// Which CTAs work on which stream: stream s owns CTAs [cta0[s], cta0[s + 1]).
struct SelCtaMap {
    int32_t cta0[PAFU_MAX_STREAMS + 1];
};

// One CTA per stream.  A kernel launched behind this one as a programmatic dependent may start at
// once (the trigger below): inside a layer step that is the row gather, which copies the rows that
// are kept whatever the scores say while the selection runs, and waits for the indices after that.
__global__ void __launch_bounds__(kSelThreads, 1)
select_kernel(const float* __restrict__ scores, const __grid_constant__ StreamTable st,
              const __grid_constant__ SelCtaMap cm, const SelSmem plan, int32_t* __restrict__ idx) {
    extern __shared__ __align__(16) unsigned char sel_smem[];
    __shared__ SelShared sh;
    constexpr int NTHR = kSelThreads;
    grid_dep_launch_dependents();
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
    // this CTA's shares: always-kept rows [a_lo, a_hi) of ns + nr, top-k rows [q_lo, q_hi) of k
    const int A = ns + nr;
    const int a_lo = (int)((int64_t)A * r / G), a_hi = (int)((int64_t)A * (r + 1) / G);
    const int q_lo = (int)((int64_t)k * r / G), q_hi = (int)((int64_t)k * (r + 1) / G);
    int32_t* out = idx + st.cu_B[s];
    const float* sc = scores + st.cu_T[s] + ns;
    const int tid = threadIdx.x;
    // always-kept tokens: position p < ns is token p, position ns + k + i is token T - nr + i
    for (int p = a_lo + tid; p < a_hi; p += NTHR) {
        if (p < ns) out[p] = p; else out[p + k] = T - A + p;
    }
    if (k > 0) {                                             // block-uniform
        if (M <= kSelCap32) select_rows<false>(sh, sel_smem, plan, sc, M, k, ns, out, q_lo, q_hi);
        else select_rows<true>(sh, sel_smem, plan, sc, M, k, ns, out, q_lo, q_hi);
    }
}

// Streams with more candidates than shared memory holds: keys are re-read from L2 in every pass
// (4 passes of 8 bits), and each thread emits a contiguous token range.
__global__ void __launch_bounds__(kSelThreads)
select_stream_kernel(const float* __restrict__ scores, StreamTable st, int32_t* __restrict__ idx) {
    grid_dep_launch_dependents();
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
            for (int t0 = c0 + tid; t0 < c1; t0 += kSelThreads * kSelBatch) {
                float v[kSelBatch];                      // the batch's loads are in flight together
#pragma unroll
                for (int u = 0; u < kSelBatch; ++u) v[u] = t0 + u * kSelThreads < c1 ? __ldg(sc + t0 + u * kSelThreads) : 0.f;
#pragma unroll
                for (int u = 0; u < kSelBatch; ++u) {
                    const uint32_t key = score_key(v[u]);
                    if (t0 + u * kSelThreads < c1 && (key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
                }
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
    const int eq_before = sel_exclusive_scan(eqc, warp_sums, &total);
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
    int pos = sel_exclusive_scan(kc, warp_sums, &total);
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
    SelSmem plan = {0};
    size_t smem_bytes = 0;
};
constexpr size_t kSelSmemMax = 227 * 1024 - 1024;            // dynamic shared memory a CTA may ask for (static part left out)
SelClass classify_streams(const StreamTable& st) {
    SelClass c;
    size_t keys = 0;
    for (int s = 0; s < st.n_streams; ++s) {
        const int64_t T = st.cu_T[s + 1] - st.cu_T[s], B = st.cu_B[s + 1] - st.cu_B[s];
        if (B == 0) continue;
        const int64_t M = B >= T ? 0 : T - st.n_sink[s] - st.n_recent[s];
        if (M > kSelCap16) { c.any_stream = true; continue; }
        c.any_smem = true;
        const size_t need = M <= kSelCap32 ? (size_t)M * 4 : (size_t)M * 2;
        if (need > keys) keys = need;
    }
    keys = (keys + 15) / 16 * 16;
    // key array, short list, scratch of four histograms' size (one histogram during the passes,
    // the emission's pair tables after them)
    c.plan.keys_bytes = (int32_t)keys;
    c.smem_bytes = keys + kSelListCap * 4 + (size_t)kSelHistBins * 4 * 4;
    return c;
}
static_assert((size_t)kSelCap32 * 4 + kSelListCap * 4 + kSelHistBins * 4 * 4 <= kSelSmemMax, "largest stream does not fit");
// (round, warp) pairs of the emission: two bytes each in the first 2048 ints, one int each after them
static_assert((kSelCap16 / kSelThreads) * (kSelThreads / 32) * 2 <= 2048 * 4 && 2048 + (kSelCap16 / kSelThreads) * (kSelThreads / 32) <= kSelHistBins * 4,
              "pair tables outgrow the histogram area");
bool set_smem_limit() {
    static bool done[kMaxDevices] = {};
    return once_per_device(done, [] {
        return cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSelSmemMax) == cudaSuccess;
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
        if (launch_dependent(select_kernel, dim3((unsigned)st.n_streams), dim3(kSelThreads), c.smem_bytes, stream, 1,
                             scores, st, cm, c.plan, idx) != cudaSuccess)
            return PAFU_ERR_CUDA;
    }
    if (c.any_stream &&
        launch_dependent(select_stream_kernel, dim3((unsigned)st.n_streams), dim3(kSelThreads), 0, stream, 1, scores, st,
                         idx) != cudaSuccess)
        return PAFU_ERR_CUDA;
    return PAFU_OK;
}

}  // namespace pafu
