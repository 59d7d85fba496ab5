// Spatialtemporal-balanced Salience Estimation (Sec. 3.2, Eq. 4 and Eq. 5) on the tensor cores.
//
//   P = softmax(Q K^T * scale) per head, full sequence of L tokens, d_head = 128.
//   For key j in block b(j) = j / L_B, the queries fall in three classes by their block:
//     later blocks  -> low_j,   the same block -> diag_j,   earlier blocks -> up_j,
//   each the mean over heads of max_i P[n, i, j] over that class (an empty class gives 0);
//   Eq. 5 averages the classes that exist for the key's block.
//
// Since exp is monotone, max_i P[i, j] = exp(max_i (z_ij - lse_i)) with lse_i the row's
// log-sum-exp: given the row statistics (a by-product of the attention kernel) no exponential is
// needed per element, only one fused multiply-add and one max.  The kernel computes S^T = K Q^T
// tile by tile (keys are the accumulator's rows, so a thread owns one key and runs its maxima
// along the columns) and never writes P.
//
// Tiling.  Keys and queries are tiled per block of L_B tokens (128 per tile, the last tile of
// a block ragged), so every (key tile, query tile) pair lies in exactly one class and the class
// is chosen per tile, not per element.  Columns past a block's end carry -lse = -inf (prepared
// by a small kernel into a padded [head][query tile][128] array that the loader brings in with
// the Q tile), rows past the end are not stored.
//
// An item is one head x one pair of key tiles ("slots") x all query tiles; items go to the
// persistent CTAs round-robin.  Warp roles (320 threads):
//   warps 0-3  read-out of slot 0 (thread = key row = TMEM lane): t = s * scale*log2e - lse*log2e,
//              running maximum per class
//   warps 4-7  read-out of slot 1
//   warp  8    MMA issuer: S^T[slot] = K_slot Q_tile^T, M = N = 128, eight K = 16 steps
//   warp  9    TMA loader: the item's K tiles, then Q tiles (+ their 512 bytes of -lse) through a
//              4-stage ring
// Tensor memory: 2 slots x 2 accumulator buffers x 128 columns = all 512 columns.
// The per-head maxima go to scratch [head][class][key] in the log2 domain; a last kernel takes
// exp2, averages over heads in head order and applies Eq. 5.  Every mbarrier wait is bounded.
#pragma once
#include "common.cuh"
#include "sm100.cuh"

namespace pafu {
namespace sse_tc {

using namespace sm100;

constexpr int kD = 128;
constexpr int kBT = 128;                       // tokens per tile, keys and queries alike
constexpr int kStages = 4;
constexpr int kThreads = 320;
constexpr int kTileBytes = kBT * kD * 2;       // 32 KiB
constexpr int kHalfBytes = kTileBytes / 2;     // one [128 rows x 64 cols] swizzled half
constexpr int kLseBytes = kBT * 4;
constexpr int kStageBytes = kTileBytes + 1024; // Q tile, then -lse (padded to keep 1 KiB alignment)
constexpr int kSmemBytes = 2 * kTileBytes + kStages * kStageBytes + 1024 /*align*/ + 256 /*barriers*/;

struct Params {
    int64_t L, LB;
    int n_heads, n_blocks;
    int tpb, tpb_last;        // tiles per block: full blocks, last block
    int n_qt;                 // query tiles in total = (n_blocks - 1) * tpb + tpb_last
    int pairs, pairs_last;    // key-tile pairs per block
    int items_per_head;       // (n_blocks - 1) * pairs + pairs_last
    float sl2;                // scale * log2(e)
    const float* neg_lse2;    // [n_heads][n_qt][128]: -lse * log2(e), -inf on padding
    float* M;                 // [n_heads][3][L]: per-head class maxima, log2 domain
    int* status;
};

struct Item {
    int head, block, n_slots;
    int64_t key0;             // first key row of slot 0
    int64_t block_end;        // one past the block's last token
};

__device__ __forceinline__ Item decode_item(const Params& p, int item) {
    Item it;
    it.head = item / p.items_per_head;
    const int r = item % p.items_per_head;
    const int full = (p.n_blocks - 1) * p.pairs;
    int pi, tiles;
    if (r < full) { it.block = r / p.pairs; pi = r % p.pairs; tiles = p.tpb; }
    else { it.block = p.n_blocks - 1; pi = r - full; tiles = p.tpb_last; }
    it.n_slots = (2 * pi + 1 < tiles) ? 2 : 1;
    it.key0 = (int64_t)it.block * p.LB + (int64_t)pi * 2 * kBT;
    const int64_t e = (int64_t)(it.block + 1) * p.LB;
    it.block_end = e < p.L ? e : p.L;
    return it;
}
// query tile g -> (block, first row)
__device__ __forceinline__ void decode_qtile(const Params& p, int g, int& qb, int64_t& row) {
    const int full = (p.n_blocks - 1) * p.tpb;
    int t;
    if (g < full) { qb = g / p.tpb; t = g % p.tpb; }
    else { qb = p.n_blocks - 1; t = g - full; }
    row = (int64_t)qb * p.LB + (int64_t)t * kBT;
}

__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// -lse * log2(e) in the padded per-tile layout the main kernel's loader copies.
__global__ void sse_neglse_kernel(const float* __restrict__ lse, Params p, float* __restrict__ out) {
    grid_dep_wait();
    const int64_t n = (int64_t)p.n_heads * p.n_qt * kBT;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % kBT);
        const int g = (int)((i / kBT) % p.n_qt);
        const int head = (int)(i / ((int64_t)kBT * p.n_qt));
        int qb; int64_t row;
        decode_qtile(p, g, qb, row);
        const int64_t e = (int64_t)(qb + 1) * p.LB;
        const int64_t end = e < p.L ? e : p.L;
        const int64_t q = row + c;
        out[i] = q < end ? -lse[(int64_t)head * p.L + q] * 1.4426950408889634f : -INFINITY;
    }
}

__global__ void __launch_bounds__(kThreads, 1)
sse_tc_kernel(const __grid_constant__ CUtensorMap mQ, const __grid_constant__ CUtensorMap mK,
              const __grid_constant__ Params p, int n_items) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sK = smem_u32(smem);                     // 2 slots x 32 KiB
    const uint32_t sQ = sK + 2 * kTileBytes;                // ring of {Q tile, -lse}
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 2 * kTileBytes + kStages * kStageBytes);
    const uint32_t bar0 = smem_u32(bars);
    auto k_full = [&](int s) { return bar0 + 8 * (0 + s); };
    auto k_empty = [&](int s) { return bar0 + 8 * (2 + s); };
    auto s_full = [&](int s, int b) { return bar0 + 8 * (4 + 2 * s + b); };
    auto s_empty = [&](int s, int b) { return bar0 + 8 * (8 + 2 * s + b); };
    auto q_full = [&](int st) { return bar0 + 8 * (12 + st); };
    auto q_empty = [&](int st) { return bar0 + 8 * (12 + kStages + st); };
    __shared__ uint32_t tmem_base_sh;
    __shared__ volatile int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(k_full(s), 1); mbar_init(k_empty(s), 1);
            for (int b = 0; b < 2; ++b) { mbar_init(s_full(s, b), 1); mbar_init(s_empty(s, b), 4); }
        }
        for (int st = 0; st < kStages; ++st) {
            mbar_init(q_full(st), 1);
            mbar_init(q_empty(st), 1 + 8);      // the issuer's commit and every read-out warp
        }
        abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 8) { tmem_alloc(smem_u32(&tmem_base_sh), 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_sh;
    grid_dep_wait();

    auto fail = [&](int code) {
        abort_flag = 1;
        atomicCAS(p.status, 0, code);
    };

    if (warp == 9) {
        // ---------------------------------------------------------------------- TMA loader
        if (elect_one()) {
            prefetch_tmap(&mQ); prefetch_tmap(&mK);
            uint32_t ring = 0, kc0 = 0, kc1 = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                const Item it = decode_item(p, item);
                for (int s = 0; s < it.n_slots && ok; ++s) {
                    const uint32_t kc = s ? kc1 : kc0;
                    if (abort_flag || !mbar_wait(k_empty(s), (kc & 1u) ^ 1u)) { fail(501); ok = false; break; }
                    if (s) ++kc1; else ++kc0;
                    mbar_arrive_expect_tx(k_full(s), kTileBytes);
                    const int row = (int)(it.key0 + s * kBT);
                    tma_load_3d(sK + s * kTileBytes, &mK, k_full(s), 0, it.head, row);
                    tma_load_3d(sK + s * kTileBytes + kHalfBytes, &mK, k_full(s), 64, it.head, row);
                }
                for (int g = 0; g < p.n_qt && ok; ++g, ++ring) {
                    const int st = ring % kStages;
                    if (abort_flag || !mbar_wait(q_empty(st), ((ring / kStages) & 1u) ^ 1u)) { fail(502); ok = false; break; }
                    int qb; int64_t row;
                    decode_qtile(p, g, qb, row);
                    const uint32_t dst = sQ + st * kStageBytes;
                    mbar_arrive_expect_tx(q_full(st), kTileBytes + kLseBytes);
                    tma_load_3d(dst, &mQ, q_full(st), 0, it.head, (int)row);
                    tma_load_3d(dst + kHalfBytes, &mQ, q_full(st), 64, it.head, (int)row);
                    bulk_load(dst + kTileBytes, p.neg_lse2 + ((int64_t)it.head * p.n_qt + g) * kBT, kLseBytes, q_full(st));
                }
            }
            if (!ok)
                for (uint32_t r = ring > (uint32_t)kStages ? ring - kStages : 0; r < ring; ++r)
                    mbar_wait(q_full(r % kStages), (r / kStages) & 1u);
        }
        __syncwarp();
    } else if (warp == 8) {
        // ---------------------------------------------------------------------- MMA issuer
        if (elect_one()) {
            const uint32_t idesc = make_idesc_bf16(kBT, kBT, false, false);
            const uint64_t desc0 = make_smem_desc_sw128(0, 16, 1024);
            uint32_t ring = 0, kc0 = 0, kc1 = 0, tc0 = 0, tc1 = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                const Item it = decode_item(p, item);
                for (int s = 0; s < it.n_slots && ok; ++s) {
                    const uint32_t kc = s ? kc1 : kc0;
                    if (abort_flag || !mbar_wait(k_full(s), kc & 1u)) { fail(511); ok = false; break; }
                    if (s) ++kc1; else ++kc0;
                }
                for (int g = 0; g < p.n_qt && ok; ++g, ++ring) {
                    const int st = ring % kStages;
                    if (abort_flag || !mbar_wait(q_full(st), (ring / kStages) & 1u)) { fail(512); ok = false; break; }
                    const uint64_t b = desc0 + ((sQ + st * kStageBytes) >> 4);
                    for (int s = 0; s < it.n_slots && ok; ++s) {
                        const uint32_t tc = s ? tc1 : tc0;
                        const int buf = tc & 1;
                        if (abort_flag || !mbar_wait(s_empty(s, buf), ((tc >> 1) & 1u) ^ 1u)) { fail(513); ok = false; break; }
                        if (s) ++tc1; else ++tc0;
                        tc_fence_after_sync();
                        const uint64_t a = desc0 + ((sK + s * kTileBytes) >> 4);
#pragma unroll
                        for (int kk = 0; kk < kD / 16; ++kk) {
                            const uint32_t off = ((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4;
                            umma_ss(tmem + (s * 2 + buf) * kBT, a + off, b + off, idesc, kk > 0);
                        }
                        umma_commit(s_full(s, buf));
                    }
                    if (ok) umma_commit(q_empty(st));
                }
                if (ok)
                    for (int s = 0; s < it.n_slots; ++s) umma_commit(k_empty(s));
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------------ read-out
        const int slot = warp >> 2;
        const uint32_t lane_base = ((uint32_t)((warp & 3) * 32)) << 16;
        const int row_in_tile = (warp & 3) * 32 + lane;
        uint32_t ring = 0, tc = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            const Item it = decode_item(p, item);
            const bool active = slot < it.n_slots;
            float m_low = -INFINITY, m_diag = -INFINITY, m_up = -INFINITY;
            for (int g = 0; g < p.n_qt; ++g, ++ring) {
                const int st = ring % kStages;
                {
                    const bool w = mbar_wait(q_full(st), (ring / kStages) & 1u) && !abort_flag;
                    if (!__all_sync(0xffffffffu, w)) { if (lane == 0) fail(521); ok = false; break; }
                }
                if (active) {
                    const int buf = tc & 1;
                    {
                        const bool w = mbar_wait(s_full(slot, buf), (tc >> 1) & 1u) && !abort_flag;
                        if (!__all_sync(0xffffffffu, w)) { if (lane == 0) fail(522); ok = false; break; }
                    }
                    ++tc;
                    tc_fence_after_sync();
                    const float4* nl = reinterpret_cast<const float4*>(smem + 2 * kTileBytes + st * kStageBytes + kTileBytes);
                    const uint32_t tS = tmem + (slot * 2 + buf) * kBT + lane_base;
                    float tm0 = -INFINITY, tm1 = -INFINITY;
#pragma unroll
                    for (int c = 0; c < kBT / 32; ++c) {
                        uint32_t r[32];
                        PAFU_TMEM_LD_X32(tS + c * 32, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            const float4 v = nl[c * 8 + q];
                            const float t0 = fmaf(__uint_as_float(r[4 * q + 0]), p.sl2, v.x);
                            const float t1 = fmaf(__uint_as_float(r[4 * q + 1]), p.sl2, v.y);
                            const float t2 = fmaf(__uint_as_float(r[4 * q + 2]), p.sl2, v.z);
                            const float t3 = fmaf(__uint_as_float(r[4 * q + 3]), p.sl2, v.w);
                            tm0 = fmax3(tm0, t0, t1);
                            tm1 = fmax3(tm1, t2, t3);
                        }
                    }
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(s_empty(slot, buf));
                    const float tm = fmaxf(tm0, tm1);
                    const int qb = g < (p.n_blocks - 1) * p.tpb ? g / p.tpb : p.n_blocks - 1;
                    if (qb > it.block) m_low = fmaxf(m_low, tm);
                    else if (qb == it.block) m_diag = fmaxf(m_diag, tm);
                    else m_up = fmaxf(m_up, tm);
                } else {
                    __syncwarp();
                }
                if (lane == 0) mbar_arrive(q_empty(st));
            }
            if (!ok) break;
            if (active) {
                const int64_t key = it.key0 + slot * kBT + row_in_tile;
                if (key < it.block_end) {
                    float* dst = p.M + (int64_t)it.head * 3 * p.L + key;
                    dst[0] = m_low; dst[p.L] = m_diag; dst[2 * p.L] = m_up;
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem, 512);
}

// exp2 of the per-head maxima, mean over heads (head order), Eq. 5.
__global__ void sse_finish_kernel(Params p, float* __restrict__ s, float* __restrict__ comp) {
    grid_dep_wait();
    for (int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; j < p.L; j += (int64_t)gridDim.x * blockDim.x) {
        float c[3];
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            float acc = 0.f;
            for (int n = 0; n < p.n_heads; ++n) acc += exp2f(p.M[((int64_t)n * 3 + k) * p.L + j]);
            c[k] = acc / (float)p.n_heads;
        }
        float v;
        if (j < p.LB) v = (c[1] + c[0]) * 0.5f;
        else if (j < p.L - p.LB) v = (c[2] + c[1] + c[0]) / 3.0f;
        else v = (c[1] + c[2]) * 0.5f;
        s[j] = v;
        if (comp != nullptr) { comp[j] = c[0]; comp[p.L + j] = c[1]; comp[2 * p.L + j] = c[2]; }
    }
}

inline Params make_params(int64_t L, int64_t LB, int n_heads, float scale) {
    Params p;
    p.L = L; p.LB = LB; p.n_heads = n_heads;
    p.n_blocks = (int)((L + LB - 1) / LB);
    const int64_t last = L - (int64_t)(p.n_blocks - 1) * LB;
    p.tpb = (int)((LB + kBT - 1) / kBT);
    p.tpb_last = (int)((last + kBT - 1) / kBT);
    p.n_qt = (p.n_blocks - 1) * p.tpb + p.tpb_last;
    p.pairs = (p.tpb + 1) / 2;
    p.pairs_last = (p.tpb_last + 1) / 2;
    p.items_per_head = (p.n_blocks - 1) * p.pairs + p.pairs_last;
    p.sl2 = scale * 1.4426950408889634f;
    p.neg_lse2 = nullptr; p.M = nullptr; p.status = nullptr;
    return p;
}

inline size_t neglse_bytes(const Params& p) { return (size_t)p.n_heads * p.n_qt * kBT * 4; }
inline size_t maxima_bytes(const Params& p) { return (size_t)p.n_heads * 3 * p.L * 4; }

inline pafu_status launch(const uint16_t* Q, const uint16_t* K, const float* lse, int64_t L, int64_t LB,
                          int n_heads, float scale, float* s, float* comp, float* neg_lse2, float* M,
                          int* status, cudaStream_t stream) {
    Params p = make_params(L, LB, n_heads, scale);
    p.neg_lse2 = neg_lse2; p.M = M; p.status = status;
    CUtensorMap mQ, mK;
    if (!TmapEncoder::token_tensor(&mQ, Q, (uint64_t)L, n_heads, kD, kBT) ||
        !TmapEncoder::token_tensor(&mK, K, (uint64_t)L, n_heads, kD, kBT)) return PAFU_ERR_CUDA;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(sse_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
            return PAFU_ERR_CUDA;
        attr_set = true;
    }
    const int sms = device_sm_count();
    const int64_t n_pad = (int64_t)n_heads * p.n_qt * kBT;
    const int g0 = (int)((n_pad + 255) / 256 < 4 * sms ? (n_pad + 255) / 256 : 4 * sms);
    if (launch_dependent(sse_neglse_kernel, dim3(g0), dim3(256), 0, stream, 1, lse, p, neg_lse2) != cudaSuccess)
        return PAFU_ERR_CUDA;
    const int n_items = n_heads * p.items_per_head;
    const int grid = n_items < sms ? n_items : sms;
    if (launch_dependent(sse_tc_kernel, dim3(grid), dim3(kThreads), kSmemBytes, stream, 1, mQ, mK, p, n_items) != cudaSuccess)
        return PAFU_ERR_CUDA;
    const int g2 = (int)((L + 255) / 256 < 4 * sms ? (L + 255) / 256 : 4 * sms);
    if (launch_dependent(sse_finish_kernel, dim3(g2), dim3(256), 0, stream, 1, p, s, comp) != cudaSuccess)
        return PAFU_ERR_CUDA;
    return PAFU_OK;
}

}  // namespace sse_tc
}  // namespace pafu
