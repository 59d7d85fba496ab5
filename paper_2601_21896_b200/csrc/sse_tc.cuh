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
// needed per element, only one fused multiply-add and one max.  The kernel computes S = Q K^T
// tile by tile (queries are the accumulator's rows, so -lse is one register per thread, and a
// thread keeps a running maximum for each of its tile's 128 key columns) and never writes P.
//
// Tiling.  Keys and queries are tiled per block of L_B tokens (128 per tile, the last tile of
// a block ragged), so every (key tile, query tile) pair lies in exactly one class and the class
// is chosen per tile, not per element.  Columns past a block's end carry -lse = -inf (prepared
// by a small kernel into a padded [head][query tile][128] array that the loader brings in with
// the Q tile), rows past the end are not stored.
//
// An item is one head x one pair of key tiles ("slots") x all query tiles; items go to the
// persistent CTAs round-robin.  Warp roles (320 threads):
//   warps 0-3  read-out of slot 0 (thread = query row = TMEM lane): t = s * scale*log2e - lse*log2e,
//              running maximum per key column; reduced over the slot's 128 threads per class
//   warps 4-7  read-out of slot 1
//   warp  8    MMA issuer: S[slot] = Q_tile K_slot^T, M = N = 128, eight K = 16 steps
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

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
// barrier among the 128 read-out threads of one slot (hardware barriers 1 and 2)
__device__ __forceinline__ void slot_barrier(int slot) {
    asm volatile("bar.sync %0, 128;" ::"r"(slot + 1) : "memory");
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
    __shared__ float red_sh[2 * 4 * kBT];

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
                    const uint64_t b = desc0 + ((sQ + st * kStageBytes) >> 4);       // Q tile
                    for (int s = 0; s < it.n_slots && ok; ++s) {
                        const uint32_t tc = s ? tc1 : tc0;
                        const int buf = tc & 1;
                        if (abort_flag || !mbar_wait(s_empty(s, buf), ((tc >> 1) & 1u) ^ 1u)) { fail(513); ok = false; break; }
                        if (s) ++tc1; else ++tc0;
                        tc_fence_after_sync();
                        const uint64_t a = desc0 + ((sK + s * kTileBytes) >> 4);     // K tile of this slot
#pragma unroll
                        for (int kk = 0; kk < kD / 16; ++kk) {
                            const uint32_t off = ((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4;
                            umma_ss(tmem + (s * 2 + buf) * kBT, b + off, a + off, idesc, kk > 0);   // rows = queries, columns = keys
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
        // Thread = query row of the streamed tile; it keeps one running maximum per key column
        // (128 registers) for the class in progress, so the per-row -lse is a register scalar
        // and each element costs one multiply-add and one max.  When the class changes (the
        // query tiles pass from earlier blocks to the key's own block to later blocks) and at
        // the item's end, the 128 threads of the slot reduce their maxima per column and store
        // them.  The accumulator is read in 16-column pieces, one piece always in flight.
        const int slot = warp >> 2, wq = warp & 3;
        const uint32_t lane_base = ((uint32_t)(wq * 32)) << 16;
        const int t_in_slot = wq * 32 + lane;
        float* red = red_sh + slot * 4 * kBT;                 // [4 warps][128 columns]
        uint32_t ring = 0, tc = 0;
        bool ok = true;
        auto wait_warp = [&](uint32_t bar, uint32_t ph, int code) {
            const bool w = mbar_wait(bar, ph) && !abort_flag;
            if (!__all_sync(0xffffffffu, w)) { if (lane == 0) fail(code); ok = false; }
        };
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            const Item it = decode_item(p, item);
            const bool active = slot < it.n_slots;
            const int g_diag0 = it.block * p.tpb;                                        // first tile of the key's own block
            const int g_low0 = it.block == p.n_blocks - 1 ? p.n_qt : g_diag0 + p.tpb;    // first tile of the later blocks
            float mx[kBT];
#pragma unroll
            for (int c = 0; c < kBT; ++c) mx[c] = -INFINITY;
            // column maxima of the class that just ended -> scratch; classes: 0 low, 1 diag, 2 up
            auto flush = [&](int cls) {
                float keep[4];
#pragma unroll
                for (int c = 0; c < kBT; ++c) {
                    const float v = warp_max(mx[c]);
                    if ((c & 31) == lane) keep[c >> 5] = v;
                    mx[c] = -INFINITY;
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) red[wq * kBT + k * 32 + lane] = keep[k];
                slot_barrier(slot);
                const float v = fmaxf(fmaxf(red[t_in_slot], red[kBT + t_in_slot]),
                                      fmaxf(red[2 * kBT + t_in_slot], red[3 * kBT + t_in_slot]));
                const int64_t key = it.key0 + slot * kBT + t_in_slot;
                if (key < it.block_end) p.M[((int64_t)it.head * 3 + cls) * p.L + key] = v;
                slot_barrier(slot);
            };
            for (int g = 0; g < p.n_qt; ++g, ++ring) {
                const int st = ring % kStages;
                wait_warp(q_full(st), (ring / kStages) & 1u, 521);
                if (!ok) break;
                if (active) {
                    if (g == g_diag0 && g > 0) flush(2);
                    if (g == g_low0) flush(1);
                    const int buf = tc & 1;
                    wait_warp(s_full(slot, buf), (tc >> 1) & 1u, 522);
                    if (!ok) break;
                    ++tc;
                    tc_fence_after_sync();
                    const uint32_t tS = tmem + (slot * 2 + buf) * kBT + lane_base;
                    const float nl = reinterpret_cast<const float*>(smem + 2 * kTileBytes + st * kStageBytes + kTileBytes)[t_in_slot];
                    uint32_t ra[16], rb[16];
                    PAFU_TMEM_LD_X16(tS, ra);
#pragma unroll
                    for (int c = 0; c < kBT / 32; ++c) {
                        tmem_wait_ld();
                        PAFU_TMEM_LD_X16(tS + c * 32 + 16, rb);
#pragma unroll
                        for (int q = 0; q < 16; ++q)
                            mx[c * 32 + q] = fmaxf(mx[c * 32 + q], fmaf(__uint_as_float(ra[q]), p.sl2, nl));
                        tmem_wait_ld();
                        if (c + 1 < kBT / 32) PAFU_TMEM_LD_X16(tS + c * 32 + 32, ra);
#pragma unroll
                        for (int q = 0; q < 16; ++q)
                            mx[c * 32 + 16 + q] = fmaxf(mx[c * 32 + 16 + q], fmaf(__uint_as_float(rb[q]), p.sl2, nl));
                    }
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(s_empty(slot, buf));
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(q_empty(st));
            }
            if (!ok) break;
            if (active) {
                // the class in progress at the end, then -inf for the classes that have no queries
                flush(it.block == p.n_blocks - 1 ? 1 : 0);
                const int64_t key = it.key0 + slot * kBT + t_in_slot;
                if (key < it.block_end) {
                    if (it.block == 0) p.M[((int64_t)it.head * 3 + 2) * p.L + key] = -INFINITY;
                    if (it.block == p.n_blocks - 1) p.M[((int64_t)it.head * 3 + 0) * p.L + key] = -INFINITY;
                }
            }
        }
        if (!ok) tmem_wait_ld();      // no load may be in flight when tensor memory is released
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
