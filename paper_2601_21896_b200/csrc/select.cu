// Retained-token selection (Sec. 3.4 inference paragraph; Algorithm 2 "Top-k"; frame sink
// Sec. 4.1): kept = [0, n_sink) U top-k salient of the middle U [T - n_recent, T), written as
// ascending token indices, ties to the lower index.
//
// The step moves a few hundred KB, so it is latency-bound.  One CTA, or a cluster of two, four or
// eight (the host picks by the stream length), works on one stream; CTA r holds the r-th part of
// the candidates in its shared memory.
//   1. fp32 scores map to order-preserving 32-bit keys (-0 folded onto +0, NaN lowest).
//   2. MSB-first radix select (11 + 11 + 10 bits) finds the key of the k-th largest candidate and
//      how many candidates equal to it are still needed.  Per pass every CTA builds the histogram
//      of its own candidates, one cluster barrier later every CTA adds up all eight histograms
//      through distributed shared memory and finds the bin by itself: all eight reach the same
//      decision, so nothing has to be sent back (one barrier per pass; the histograms alternate
//      between two buffers so that a CTA may start the next pass while others still read).  After
//      the first digit a CTA's surviving candidates are few and move to a short list that the
//      later passes read instead of the whole array.
//   3. Ordered emission: candidate j belongs to (CTA, round, warp, lane); warp ballots count
//      kept and tied candidates per (round, warp), the CTAs exchange their totals (one more
//      barrier), and scans over those counts give every kept token its output slot, so the
//      result is ascending and ties resolve to the lowest indices.
// Streams with more candidates than eight CTAs hold (360 448) use one CTA that re-reads L2 in every pass.
// A kernel launched behind these as a programmatic dependent may start at once (the trigger at
// their top): inside a layer step that is the row gather, which copies the rows that are kept
// whatever the scores say while the selection runs, and waits for the indices after that.
#include <cooperative_groups.h>

#include "common.cuh"

namespace pafu {

namespace cg = cooperative_groups;

constexpr int kSelThreads = 1024;
constexpr int kSelCluster = 8;              // at most this many CTAs cooperate on one stream
constexpr int kSelCapCta = 45056;           // candidates one CTA holds (176 KiB of keys)
constexpr int kSelCapCluster = kSelCluster * kSelCapCta;
constexpr int kSelHistBins = 2048;
constexpr int kSelListCap = 4096;           // candidates of a CTA the later passes can take from its short list
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
    int tot[kSelCluster][2];         // every CTA's count of candidates above / equal to the threshold
};

// One radix pass: histogram of `bits` bits at `shift` over this CTA's n candidates that `get`
// admits, into `hist` (this pass's buffer, at the same address in every CTA); then, one cluster
// barrier later, the sum of the eight CTAs' histograms and the bin that holds the k_rem-th largest
// admitted key.  (Spreading the lanes over several copies of the histogram, or grouping equal
// digits with match.any before adding, did not make the adds cheaper: a shared-memory add costs
// about 13 clocks per warp instruction whether or not its lanes collide.)
template <typename Get>
__device__ __forceinline__ void radix_pass(cg::cluster_group& cluster, SelShared& sh, int* hist, int n, int shift,
                                           int bits, uint32_t& prefix, int& k_rem, int& bin_count, Get get) {
    const int tid = threadIdx.x;
    const int nb = 1 << bits, nc = (int)cluster.num_blocks();
    for (int b = tid; b < nb; b += kSelThreads) hist[b] = 0;
    __syncthreads();
    for (int j0 = 0; j0 < n; j0 += kSelThreads * kSelBatch) {
        uint32_t key[kSelBatch];
        bool in[kSelBatch];
#pragma unroll
        for (int u = 0; u < kSelBatch; ++u) {
            const int j = j0 + u * kSelThreads + tid;
            key[u] = 0u;
            in[u] = (j < n) && get(j, key[u]);
        }
#pragma unroll
        for (int u = 0; u < kSelBatch; ++u)
            if (in[u]) atomicAdd(&hist[(key[u] >> shift) & (uint32_t)(nb - 1)], 1);
    }
    cluster.sync();                  // every CTA's histogram is complete (and visible to the cluster)
    // bins from the top: thread t holds bins nb-1-2t and nb-2-2t (nb <= 2048 = 2 x block size)
    int c[2] = {0, 0};
    const int b_hi = nb - 1 - 2 * tid;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int b = b_hi - i;
        if (b >= 0) {
            int v = 0;
            for (int r = 0; r < nc; ++r) v += *cluster.map_shared_rank(hist + b, r);
            c[i] = v;
        }
    }
    int total;
    const int above = sel_exclusive_scan(c[0] + c[1], sh.warp_sums, &total);
    if (above < k_rem && k_rem <= above + c[0]) {
        sh.prefix = prefix | ((uint32_t)b_hi << shift); sh.k_rem = k_rem - above; sh.bin_count = c[0];
    } else if (above + c[0] < k_rem && k_rem <= above + c[0] + c[1]) {
        sh.prefix = prefix | ((uint32_t)(b_hi - 1) << shift); sh.k_rem = k_rem - above - c[0]; sh.bin_count = c[1];
    }
    __syncthreads();
    prefix = sh.prefix; k_rem = sh.k_rem; bin_count = sh.bin_count;
}

__global__ void __launch_bounds__(kSelThreads, 1)
select_cluster_kernel(const float* __restrict__ scores, const __grid_constant__ StreamTable st, int32_t keys_bytes,
                      int32_t* __restrict__ idx) {
    extern __shared__ __align__(16) unsigned char sel_smem[];
    __shared__ SelShared sh;
    grid_dep_launch_dependents();
    grid_dep_wait();
    cg::cluster_group cluster = cg::this_cluster();
    const int nc = (int)cluster.num_blocks();                // 1, 2, 4 or 8: the host's choice for this launch
    const int s = blockIdx.x / nc;
    const int rank = (int)cluster.block_rank();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int NW = kSelThreads / 32;
    const int64_t T64 = st.cu_T[s + 1] - st.cu_T[s], B64 = st.cu_B[s + 1] - st.cu_B[s];
    // cluster-uniform exits (before any cluster barrier)
    if (B64 == 0) return;
    const int T = (int)T64, B = (int)B64;
    // a stream that keeps everything is one long "sink"
    const bool all = B >= T;
    const int ns = all ? T : (int)st.n_sink[s], nr = all ? 0 : (int)st.n_recent[s], k = all ? 0 : (int)st.k[s];
    const int M = T - ns - nr;
    if (M > nc * kSelCapCta) return;                         // the streaming kernel owns this stream
    int32_t* out = idx + st.cu_B[s];
    // always-kept tokens (spread over the cluster): position p < ns is token p, position ns + k + i is token T - nr + i
    for (int p = rank * kSelThreads + tid; p < ns + nr; p += nc * kSelThreads) {
        if (p < ns) out[p] = p; else out[p + k] = T - (ns + nr) + p;
    }
    if (k == 0) return;

    // this CTA's candidates: [j_lo, j_lo + n) of the stream's M, a whole number of rounds per CTA
    const int per_cta = (M + nc * kSelThreads - 1) / (nc * kSelThreads) * kSelThreads;
    const int j_lo = rank * per_cta;
    const int n = max(0, min(M - j_lo, per_cta));
    const float* sc = scores + st.cu_T[s] + ns + j_lo;
    uint32_t* keys = reinterpret_cast<uint32_t*>(sel_smem);
    uint32_t* list = reinterpret_cast<uint32_t*>(sel_smem + keys_bytes);
    int* hist0 = reinterpret_cast<int*>(sel_smem + keys_bytes + kSelListCap * 4);
    int* hist1 = hist0 + kSelHistBins;
    for (int j0 = tid; j0 < n; j0 += kSelThreads * kSelBatch) {
        float v[kSelBatch];
#pragma unroll
        for (int u = 0; u < kSelBatch; ++u) {
            const int j = j0 + u * kSelThreads;
            v[u] = j < n ? __ldg(sc + j) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < kSelBatch; ++u) {
            const int j = j0 + u * kSelThreads;
            if (j < n) keys[j] = score_key(v[u]);
        }
    }
    if (tid == 0) sh.list_n = 0;
    __syncthreads();

    // ---- the key of the k-th largest candidate
    uint32_t thr = 0u;
    int need_eq = k, eq_total = 0;
    radix_pass(cluster, sh, hist0, n, 21, 11, thr, need_eq, eq_total,
               [&](int j, uint32_t& key) { key = keys[j]; return true; });
    // this CTA's survivors go to its short list if they fit (any order: only their values matter now)
    int n_mine = 0;
    {
        const uint32_t top = thr >> 21;
        for (int j0 = 0; j0 < n; j0 += kSelThreads) {
            const int j = j0 + tid;
            const uint32_t kx = j < n ? keys[j] : 0u;
            const bool hit = j < n && (kx >> 21) == top;
            const unsigned b = __ballot_sync(0xffffffffu, hit);
            if (b != 0u) {
                int base = 0;
                if (lane == 0) base = atomicAdd(&sh.list_n, __popc(b));
                base = __shfl_sync(0xffffffffu, base, 0);
                const int slot = base + __popc(b & ((1u << lane) - 1u));
                if (hit && slot < kSelListCap) list[slot] = kx;
            }
        }
        __syncthreads();
        n_mine = sh.list_n;
    }
    const bool listed = n_mine <= kSelListCap;               // block-uniform (each CTA decides for itself)
    const int n_rest = listed ? n_mine : n;
    {
        const uint32_t pf1 = thr;
        radix_pass(cluster, sh, hist1, n_rest, 10, 11, thr, need_eq, eq_total, [&](int j, uint32_t& key) {
            key = listed ? list[j] : keys[j];
            return (key & 0xffe00000u) == pf1;
        });
        const uint32_t pf2 = thr;
        radix_pass(cluster, sh, hist0, n_rest, 0, 10, thr, need_eq, eq_total, [&](int j, uint32_t& key) {
            key = listed ? list[j] : keys[j];
            return (key & 0xfffffc00u) == pf2;
        });
    }

    // ---- ordered emission.  Own candidate j = (round * NW + warp) * 32 + lane; per (round, warp)
    // pair the counts of candidates above the threshold and equal to it (one byte each) go to shared
    // memory, scans over the pairs and the CTAs' totals turn them into output slots.  hist1 and the
    // list are free now (hist0 may still be read by other CTAs).
    const bool ties = need_eq != eq_total;                   // cluster-uniform: some equal candidates stay out
    const int rounds = (n + kSelThreads - 1) / kSelThreads, n_pairs = rounds * NW;
    uint16_t* cnt = reinterpret_cast<uint16_t*>(hist1);      // [n_pairs]: above | equal << 8
    int* slot = reinterpret_cast<int*>(list);                // [n_pairs]: kept before the pair | equal ones taken << 24
    // a thread's candidates' classes stay in registers as bit masks (rounds <= 44)
    uint32_t gtb[2], eqb[2];
#pragma unroll
    for (int blk = 0; blk < 2; ++blk) {
        uint32_t g = 0u, e = 0u;
        const int i_end = min(rounds, (blk + 1) * 32);
        for (int i = blk * 32; i < i_end; ++i) {
            const int j = i * kSelThreads + tid;
            const uint32_t kx = j < n ? keys[j] : 0u;
            const bool is_gt = j < n && kx > thr, is_eq = j < n && kx == thr;
            const unsigned bg = __ballot_sync(0xffffffffu, is_gt), be = __ballot_sync(0xffffffffu, is_eq);
            if (lane == 0) cnt[i * NW + warp] = (uint16_t)(__popc(bg) | (__popc(be) << 8));
            g |= (uint32_t)is_gt << (i & 31);
            e |= (uint32_t)is_eq << (i & 31);
        }
        gtb[blk] = g; eqb[blk] = e;
    }
    __syncthreads();
    // thread t owns pairs [t * per, (t + 1) * per)
    const int per = (n_pairs + kSelThreads - 1) / kSelThreads;
    const int p0 = min(n_pairs, tid * per), p1 = min(n_pairs, p0 + per);
    int my_gt = 0, my_eq = 0;
    for (int p = p0; p < p1; ++p) { my_gt += cnt[p] & 0xff; my_eq += cnt[p] >> 8; }
    int gt_cta, eq_cta;
    const int gt_before_t = sel_exclusive_scan(my_gt, sh.warp_sums, &gt_cta);
    const int eq_before_t = sel_exclusive_scan(my_eq, sh.warp_sums, &eq_cta);
    if (tid < nc) {                                          // this CTA's totals, to every CTA of the cluster
        int* remote = &cluster.map_shared_rank(&sh, tid)->tot[rank][0];
        remote[0] = gt_cta; remote[1] = eq_cta;
    }
    cluster.sync();
    // candidates kept in the CTAs before this one, and equal ones seen there
    int kept_before = 0, eq_before = 0;
    for (int r = 0; r < rank; ++r) {
        const int take = ties ? min(sh.tot[r][1], max(0, need_eq - eq_before)) : sh.tot[r][1];
        kept_before += sh.tot[r][0] + take;
        eq_before += sh.tot[r][1];
    }
    {
        // kept before this thread's pairs inside the CTA: the ones above the threshold, and of the
        // equal ones those that still fit
        int e = eq_before + eq_before_t;
        const int taken_before_t = ties ? min(eq_before_t, max(0, need_eq - eq_before)) : eq_before_t;
        int pos = kept_before + gt_before_t + taken_before_t;
        for (int p = p0; p < p1; ++p) {
            const int g = cnt[p] & 0xff, q = cnt[p] >> 8;
            const int take = ties ? min(q, max(0, need_eq - e)) : q;
            slot[p] = pos | (take << 24);                    // take <= 32; pos < 2^24
            e += q;
            pos += g + take;
        }
    }
    __syncthreads();
    const unsigned lt = (1u << lane) - 1u;
#pragma unroll
    for (int blk = 0; blk < 2; ++blk) {
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
            if (keep) out[ns + (sl & 0xffffff) + __popc(bk & lt)] = ns + j_lo + i * kSelThreads + tid;
        }
    }
}

// Streams with more candidates than a cluster's shared memory holds: keys are re-read from L2 in every pass
// (4 passes of 8 bits), and each thread emits a contiguous token range.
__global__ void __launch_bounds__(kSelThreads)
select_stream_kernel(const float* __restrict__ scores, StreamTable st, int32_t* __restrict__ idx) {
    grid_dep_launch_dependents();
    grid_dep_wait();
    {
        const int64_t T = st.cu_T[blockIdx.x + 1] - st.cu_T[blockIdx.x], B = st.cu_B[blockIdx.x + 1] - st.cu_B[blockIdx.x];
        if (B >= T || T - st.n_sink[blockIdx.x] - st.n_recent[blockIdx.x] <= kSelCapCluster) return;   // the other kernel owns this stream
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
constexpr size_t kSelSmemMax = 227 * 1024 - 1024;            // dynamic shared memory a CTA may ask for (static part left out)
static_assert((size_t)kSelCapCta * 4 + kSelListCap * 4 + kSelHistBins * 4 * 2 <= kSelSmemMax, "a CTA's share does not fit");
// (round, warp) pairs of the emission: two bytes each in one histogram buffer, one int each in the list
static_assert((kSelCapCta / kSelThreads) * (kSelThreads / 32) * 2 <= kSelHistBins * 4 &&
              (kSelCapCta / kSelThreads) * (kSelThreads / 32) <= kSelListCap && kSelCapCta / kSelThreads <= 64,
              "pair tables outgrow their buffers");
}  // namespace

namespace {
struct SelLaunch {
    bool any_cluster = false, any_stream = false;
    int nc = 1;
    int64_t per_cta = 0;
};
SelLaunch plan_select(const StreamTable& st) {
    SelLaunch pl;
    int64_t m_max = 0;
    for (int s = 0; s < st.n_streams; ++s) {
        const int64_t T = st.cu_T[s + 1] - st.cu_T[s], B = st.cu_B[s + 1] - st.cu_B[s];
        if (B == 0) continue;
        const int64_t M = B >= T ? 0 : T - st.n_sink[s] - st.n_recent[s];
        if (M > kSelCapCluster) { pl.any_stream = true; continue; }
        pl.any_cluster = true;
        if (M > m_max) m_max = M;
    }
    // CTAs per stream.  A barrier across CTAs and the trip through distributed shared memory cost
    // more than a few rounds over the candidates: one CTA up to 24 rounds (24 576 candidates: the
    // 28 080-token cache), then as many as keep a CTA's share near 16 rounds.
    while (pl.nc < kSelCluster && m_max > (int64_t)pl.nc * (pl.nc == 1 ? 24576 : 16384)) pl.nc *= 2;
    pl.per_cta = (m_max + pl.nc * kSelThreads - 1) / (pl.nc * kSelThreads) * kSelThreads;
    return pl;
}
}  // namespace

int select_cta_count(const StreamTable& st) {
    const SelLaunch pl = plan_select(st);
    return (pl.any_cluster ? st.n_streams * pl.nc : 0) + (pl.any_stream ? st.n_streams : 0);
}

pafu_status launch_select(const float* scores, const StreamTable& st, int32_t* idx, cudaStream_t stream) {
    if (st.n_streams == 0 || st.cu_B[st.n_streams] == 0) return PAFU_OK;
    const SelLaunch pl = plan_select(st);
    if (pl.any_cluster) {
        static bool done[kMaxDevices] = {};
        if (!once_per_device(done, [] {
                return cudaFuncSetAttribute(select_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSelSmemMax) == cudaSuccess;
            }))
            return PAFU_ERR_CUDA;
        const int32_t keys_bytes = (int32_t)(pl.per_cta * 4);
        const size_t smem = (size_t)keys_bytes + kSelListCap * 4 + kSelHistBins * 4 * 2;
        if (launch_dependent(select_cluster_kernel, dim3((unsigned)(st.n_streams * pl.nc)), dim3(kSelThreads), smem, stream,
                             (unsigned)pl.nc, scores, st, keys_bytes, idx) != cudaSuccess)
            return PAFU_ERR_CUDA;
    }
    if (pl.any_stream &&
        launch_dependent(select_stream_kernel, dim3((unsigned)st.n_streams), dim3(kSelThreads), 0, stream, 1, scores, st,
                         idx) != cudaSuccess)
        return PAFU_ERR_CUDA;
    return PAFU_OK;
}

}  // namespace pafu
