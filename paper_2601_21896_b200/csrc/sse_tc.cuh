// Spatialtemporal-balanced Salience Estimation (Sec. 3.2, Eq. 4 and Eq. 5) on the tensor cores.
//
//   P = softmax(Q K^T * scale) per head, full sequence of L tokens, d_head = 128.
//   For key j in block b(j) = j / L_B, the queries fall in three classes by their block:
//     later blocks  -> low_j,   the same block -> diag_j,   earlier blocks -> up_j,
//   each the mean over heads of max_i P[n, i, j] over that class (an empty class gives 0);
//   Eq. 5 averages the classes that exist for the key's block.
//
// Since exp is monotone, max_i P[i, j] = exp(max_i (z_ij - lse_i)) with lse_i the row's
// log-sum-exp (a by-product of the attention kernel): no exponential is needed per element.
// The subtraction is folded into the contraction as well: the reduction dimension is extended
// from 128 to 144, every key gets the extra features (1, 1, 1, 0, ...) and query i the extra
// features (h, m, l, 0, ...), h + m + l = -lse_i / scale split into three bf16 terms (24 bits),
// so the accumulator holds q_i.k_j - lse_i / scale and the read-out is a bare running maximum.
// The kernel computes K Q^T tile by tile (keys are the accumulator's rows: a thread owns one
// key) and never writes P.
//
// Tiling.  Keys and queries are tiled per block of L_B tokens (128 per tile, the last tile of
// a block ragged), so every (key tile, query tile) pair lies in exactly one class and the class
// is chosen per tile, not per element.  Query columns past a block's end get -1e30 as their
// extra feature; key rows past the end are not stored.  The extra features of a query tile are
// prepared by a small kernel as a 4 KiB block in the operand layout (no swizzle: 8 x 16-byte
// core matrices) that the loader copies with the tile.
//
// An item is one head x one pair of key tiles ("slots") x all query tiles; items go to the
// persistent CTAs round-robin.  Warp roles (384 threads):
//   warps 0-3  read-out of slot 0 (thread = key row = TMEM lane): running maximum per class
//   warps 4-7  read-out of slot 1
//   warps 8,10 MMA issuers, one per slot: S[slot] = K_slot Q_tile^T, M = N = 128, nine K = 16 steps
//   warp  9    TMA loader: the item's K tiles, then Q tiles (+ extra features) through a 4-stage ring
//   warp  11   idle
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
constexpr int kThreads = 384;
constexpr int kTileBytes = kBT * kD * 2;       // 32 KiB
constexpr int kHalfBytes = kTileBytes / 2;     // one [128 rows x 64 cols] swizzled half
constexpr int kAugBytes = kBT * 16 * 2;        // 4 KiB: 16 extra reduction columns of one tile
constexpr int kStageBytes = kTileBytes + kAugBytes;   // Q tile, then its extra features
constexpr int kSmemBytes = 2 * kTileBytes + kAugBytes + kStages * kStageBytes + 1024 /*align*/ + 256 /*barriers*/;
constexpr int kScratchRows = 4;               // low, diag, up maxima and the column sum, per head and key
constexpr float kMasked = -1.0e30f;            // extra feature of a query column that does not exist

struct Params {
    int64_t L, LB;
    int n_heads, n_blocks;
    int tpb, tpb_last;        // tiles per block: full blocks, last block
    int n_qt;                 // query tiles in total = (n_blocks - 1) * tpb + tpb_last
    int pairs, pairs_last;    // key-tile pairs per block
    int items_per_head;       // (n_blocks - 1) * pairs + pairs_last
    float sl2;                // scale * log2(e)
    float inv_scale;
    const uint16_t* q_aug;    // [n_heads][n_qt][2048] bf16: extra features per query tile, operand layout
    float* M;                 // [n_heads][4][L]: per-head class maxima (log2 domain), then the column sums of P
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

__device__ __forceinline__ float ex2(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }

__device__ __forceinline__ uint16_t bf16_rne(float x) {
    const uint32_t u = __float_as_uint(x);
    return (uint16_t)((u + 0x7fffu + ((u >> 16) & 1u)) >> 16);
}
__device__ __forceinline__ float bf16_val(uint16_t b) { return __uint_as_float(((uint32_t)b) << 16); }

// Extra features of every query tile in the operand's shared-memory layout (K-major, no
// swizzle): element (row r, column c) of a [128 x 16] tile sits at byte
// (r / 8) * 256 + (c / 8) * 128 + (r % 8) * 16 + (c % 8) * 2.  Columns 0..2 carry the three
// bf16 terms of -lse / scale, the rest are zero.
__global__ void sse_aug_kernel(const float* __restrict__ lse, Params p, uint16_t* __restrict__ out) {
    grid_dep_wait();
    const int64_t n = (int64_t)p.n_heads * p.n_qt * (kAugBytes / 2);
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int e = (int)(i % (kAugBytes / 2));
        const int g = (int)((i / (kAugBytes / 2)) % p.n_qt);
        const int head = (int)(i / ((int64_t)(kAugBytes / 2) * p.n_qt));
        const int r = (e / 128) * 8 + (e % 64) / 8;
        const int c = ((e % 128) / 64) * 8 + e % 8;
        uint16_t v = 0;
        if (c < 3) {
            int qb; int64_t row;
            decode_qtile(p, g, qb, row);
            const int64_t end_b = (int64_t)(qb + 1) * p.LB;
            const int64_t end = end_b < p.L ? end_b : p.L;
            const int64_t q = row + r;
            if (q < end) {
                const float a = -lse[(int64_t)head * p.L + q] * p.inv_scale;
                const uint16_t h = bf16_rne(a);
                const uint16_t m = bf16_rne(a - bf16_val(h));
                const uint16_t l = bf16_rne(a - bf16_val(h) - bf16_val(m));
                v = c == 0 ? h : (c == 1 ? m : l);
            } else {
                v = c == 0 ? bf16_rne(kMasked) : (uint16_t)0;
            }
        }
        out[i] = v;
    }
}

// SUM = true additionally accumulates sum_i P[i, j] per key (one exponential per element), for the
// average-pooling output; the default instantiation does no exponentials at all.
template <bool SUM>
__global__ void __launch_bounds__(kThreads, 1)
sse_tc_kernel(const __grid_constant__ CUtensorMap mQ, const __grid_constant__ CUtensorMap mK,
              const __grid_constant__ Params p, int n_items) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sK = smem_u32(smem);                     // 2 slots x 32 KiB
    const uint32_t sKaug = sK + 2 * kTileBytes;             // the keys' extra features (1, 1, 1, 0, ...)
    const uint32_t sQ = sKaug + kAugBytes;                  // ring of {Q tile, its extra features}
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 2 * kTileBytes + kAugBytes + kStages * kStageBytes);
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
            mbar_init(q_empty(st), 2);          // both issuers release a stage
        }
        abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 8) { tmem_alloc(smem_u32(&tmem_base_sh), 512); tmem_relinquish(); }
    // the keys' extra features are the same for every tile: ones in columns 0..2 of each row
    for (int w = tid; w < kAugBytes / 4; w += kThreads) {
        const int off = w * 4, in_group = off % 256;
        uint32_t v = 0;
        if (in_group < 128) {                       // columns 0..7
            const int pair = (in_group % 16) / 4;   // columns 2 * pair, 2 * pair + 1
            v = pair == 0 ? 0x3f803f80u : (pair == 1 ? 0x00003f80u : 0u);
        }
        reinterpret_cast<uint32_t*>(smem + 2 * kTileBytes)[w] = v;
    }
    fence_proxy_async_smem();                       // the tensor core reads it through the async proxy
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
                    mbar_arrive_expect_tx(q_full(st), kTileBytes + kAugBytes);
                    tma_load_3d(dst, &mQ, q_full(st), 0, it.head, (int)row);
                    tma_load_3d(dst + kHalfBytes, &mQ, q_full(st), 64, it.head, (int)row);
                    bulk_load(dst + kTileBytes, p.q_aug + ((int64_t)it.head * p.n_qt + g) * (kAugBytes / 2), kAugBytes, q_full(st));
                }
            }
            if (!ok)
                for (uint32_t r = ring > (uint32_t)kStages ? ring - kStages : 0; r < ring; ++r)
                    mbar_wait(q_full(r % kStages), (r / kStages) & 1u);
        }
        __syncwarp();
    } else if (warp == 11) {
        // idle: completes the third warpgroup
    } else if (warp >= 8) {
        // ------------------------------------------- MMA issuers: warp 8 -> slot 0, warp 10 -> slot 1
        // One issuing thread per slot: with the waits, commits and descriptor arithmetic of its
        // loop a single thread issues roughly one tcgen05.mma per 100 clocks, less than the tensor
        // core consumes (a 128 x 128 x 16 step takes 64).
        if (elect_one()) {
            const int slot = warp == 8 ? 0 : 1;
            const uint32_t idesc = make_idesc_bf16(kBT, kBT, false, false);
            const uint64_t desc0 = make_smem_desc_sw128(0, 16, 1024);
            // extra features: no swizzle, core matrices 128 bytes apart along K, 256 along rows
            const uint64_t desc_aug = make_smem_desc_noswizzle(0, 128, 256);
            const uint64_t a_aug = desc_aug + (sKaug >> 4);
            const uint64_t a = desc0 + ((sK + slot * kTileBytes) >> 4);     // K tile of this slot
            uint32_t ring = 0, kc = 0, tc = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                const Item it = decode_item(p, item);
                const bool active = slot < it.n_slots;
                if (active) {
                    if (abort_flag || !mbar_wait(k_full(slot), kc & 1u)) { fail(511); ok = false; break; }
                    ++kc;
                }
                for (int g = 0; g < p.n_qt && ok; ++g, ++ring) {
                    const int st = ring % kStages;
                    if (abort_flag || !mbar_wait(q_full(st), (ring / kStages) & 1u)) { fail(512); ok = false; break; }
                    if (!active) { mbar_arrive(q_empty(st)); continue; }    // a stage is released by both issuers
                    const int buf = tc & 1;
                    if (abort_flag || !mbar_wait(s_empty(slot, buf), ((tc >> 1) & 1u) ^ 1u)) { fail(513); ok = false; break; }
                    ++tc;
                    tc_fence_after_sync();
                    const uint64_t b = desc0 + ((sQ + st * kStageBytes) >> 4);       // Q tile
                    const uint64_t b_aug = desc_aug + ((sQ + st * kStageBytes + kTileBytes) >> 4);
                    const uint32_t d = tmem + (slot * 2 + buf) * kBT;
#pragma unroll
                    for (int kk = 0; kk < kD / 16; ++kk) {
                        const uint32_t off = ((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4;
                        umma_ss(d, a + off, b + off, idesc, kk > 0);                 // rows = keys, columns = queries
                    }
                    umma_ss(d, a_aug, b_aug, idesc, 1);                              // ... - lse / scale
                    umma_commit(s_full(slot, buf));
                    umma_commit(q_empty(st));
                }
                if (ok && active) umma_commit(k_empty(slot));
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------------ read-out
        // Thread = key row.  The accumulator already holds q.k - lse / scale, so a tile costs
        // each thread 128 values and 64 three-way maxima.  It is read in two halves of 64
        // columns into two register sets: half 1 loads during the arithmetic on half 0, half 0
        // of the next tile during the arithmetic on half 1, and the buffer goes back to the
        // issuer as soon as its second half has landed.
        const int slot = warp >> 2;
        const uint32_t lane_base = ((uint32_t)((warp & 3) * 32)) << 16;
        const int row_in_tile = (warp & 3) * 32 + lane;
        uint32_t tc = 0;
        bool ok = true;
        auto wait_warp = [&](uint32_t bar, uint32_t ph, int code) {
            const bool w = mbar_wait(bar, ph) && !abort_flag;
            if (!__all_sync(0xffffffffu, w)) { if (lane == 0) fail(code); ok = false; }
        };
        float sum0 = 0.f, sum1 = 0.f, sum2 = 0.f, sum3 = 0.f;     // SUM: partial column sums of P for this key
        auto max64 = [&](const uint32_t (&r)[64], float& tm0, float& tm1) {
#pragma unroll
            for (int q = 0; q < 16; ++q) {
                tm0 = fmax3(tm0, __uint_as_float(r[4 * q + 0]), __uint_as_float(r[4 * q + 1]));
                tm1 = fmax3(tm1, __uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3]));
                if (SUM) {
                    sum0 += ex2(__uint_as_float(r[4 * q + 0]) * p.sl2); sum1 += ex2(__uint_as_float(r[4 * q + 1]) * p.sl2);
                    sum2 += ex2(__uint_as_float(r[4 * q + 2]) * p.sl2); sum3 += ex2(__uint_as_float(r[4 * q + 3]) * p.sl2);
                }
            }
        };
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            const Item it = decode_item(p, item);
            if (slot >= it.n_slots) continue;
            float m_low = -INFINITY, m_diag = -INFINITY, m_up = -INFINITY;
            sum0 = sum1 = sum2 = sum3 = 0.f;
            uint32_t ra[64], rb[64];
            wait_warp(s_full(slot, tc & 1), (tc >> 1) & 1u, 522);
            if (!ok) break;
            tc_fence_after_sync();
            {
                const uint32_t tS = tmem + (slot * 2 + (tc & 1)) * kBT + lane_base;
                PAFU_TMEM_LD_X32(tS, ra);
                PAFU_TMEM_LD_X32(tS + 32, ra + 32);
            }
            for (int g = 0; g < p.n_qt; ++g) {
                const int buf = tc & 1;
                const uint32_t tS = tmem + (slot * 2 + buf) * kBT + lane_base;
                float tm0 = -INFINITY, tm1 = -INFINITY;
                tmem_wait_ld();                                   // half 0 in ra
                PAFU_TMEM_LD_X32(tS + 64, rb);
                PAFU_TMEM_LD_X32(tS + 96, rb + 32);
                max64(ra, tm0, tm1);
                tmem_wait_ld();                                   // half 1 in rb: the buffer is free
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(s_empty(slot, buf));
                ++tc;
                if (g + 1 < p.n_qt) {
                    wait_warp(s_full(slot, tc & 1), (tc >> 1) & 1u, 523);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t tN = tmem + (slot * 2 + (tc & 1)) * kBT + lane_base;
                    PAFU_TMEM_LD_X32(tN, ra);
                    PAFU_TMEM_LD_X32(tN + 32, ra + 32);
                }
                max64(rb, tm0, tm1);
                const float tm = fmaxf(tm0, tm1);
                const int qb = g < (p.n_blocks - 1) * p.tpb ? g / p.tpb : p.n_blocks - 1;
                if (qb > it.block) m_low = fmaxf(m_low, tm);
                else if (qb == it.block) m_diag = fmaxf(m_diag, tm);
                else m_up = fmaxf(m_up, tm);
            }
            if (!ok) break;
            const int64_t key = it.key0 + slot * kBT + row_in_tile;
            if (key < it.block_end) {
                // log2 domain; a class without queries stays -inf, a masked column gives about -1e29
                float* dst = p.M + (int64_t)it.head * kScratchRows * p.L + key;
                dst[0] = m_low * p.sl2; dst[p.L] = m_diag * p.sl2; dst[2 * p.L] = m_up * p.sl2;
                if (SUM) dst[3 * p.L] = (sum0 + sum1) + (sum2 + sum3);
            }
        }
        if (!ok) tmem_wait_ld();      // no load may be in flight when tensor memory is released
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem, 512);
}

// exp2 of the per-head maxima, mean over heads (head order), Eq. 5.
__global__ void sse_finish_kernel(Params p, float* __restrict__ s, float* __restrict__ comp, float* __restrict__ gmax,
                                  float* __restrict__ gavg) {
    grid_dep_wait();
    for (int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; j < p.L; j += (int64_t)gridDim.x * blockDim.x) {
        float c[3];
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            float acc = 0.f;
            for (int n = 0; n < p.n_heads; ++n) acc += exp2f(p.M[((int64_t)n * kScratchRows + k) * p.L + j]);
            c[k] = acc / (float)p.n_heads;
        }
        float v;
        if (j < p.LB) v = (c[1] + c[0]) * 0.5f;
        else if (j < p.L - p.LB) v = (c[2] + c[1] + c[0]) / 3.0f;
        else v = (c[1] + c[2]) * 0.5f;
        s[j] = v;
        if (comp != nullptr) { comp[j] = c[0]; comp[p.L + j] = c[1]; comp[2 * p.L + j] = c[2]; }
        if (gmax != nullptr) {          // max over all queries per head, then the mean over heads
            float acc = 0.f;
            for (int n = 0; n < p.n_heads; ++n) {
                const float* m = p.M + (int64_t)n * kScratchRows * p.L + j;
                acc += exp2f(fmaxf(fmaxf(m[0], m[p.L]), m[2 * p.L]));
            }
            gmax[j] = acc / (float)p.n_heads;
        }
        if (gavg != nullptr) {          // mean over all queries per head, then the mean over heads
            float acc = 0.f;
            for (int n = 0; n < p.n_heads; ++n) acc += p.M[((int64_t)n * kScratchRows + 3) * p.L + j];
            gavg[j] = acc / ((float)p.n_heads * (float)p.L);
        }
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
    p.inv_scale = 1.0f / scale;
    p.q_aug = nullptr; p.M = nullptr; p.status = nullptr;
    return p;
}

inline size_t aug_bytes(const Params& p) { return (size_t)p.n_heads * p.n_qt * kAugBytes; }
inline size_t maxima_bytes(const Params& p) { return (size_t)p.n_heads * kScratchRows * p.L * 4; }

inline pafu_status launch(const uint16_t* Q, const uint16_t* K, const float* lse, int64_t L, int64_t LB,
                          int n_heads, float scale, float* s, float* comp, float* gmax, float* gavg, uint16_t* q_aug, float* M,
                          int* status, cudaStream_t stream) {
    Params p = make_params(L, LB, n_heads, scale);
    p.q_aug = q_aug; p.M = M; p.status = status;
    CUtensorMap mQ, mK;
    if (!TmapEncoder::token_tensor(&mQ, Q, (uint64_t)L, n_heads, kD, kBT) ||
        !TmapEncoder::token_tensor(&mK, K, (uint64_t)L, n_heads, kD, kBT)) return PAFU_ERR_CUDA;
    static bool attr_set[kMaxDevices] = {};
    if (!once_per_device(attr_set, [] {
            return cudaFuncSetAttribute(sse_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) == cudaSuccess &&
                   cudaFuncSetAttribute(sse_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) == cudaSuccess;
        }))
        return PAFU_ERR_CUDA;
    const int sms = device_sm_count();
    const int64_t n_pad = (int64_t)n_heads * p.n_qt * (kAugBytes / 2);
    const int g0 = (int)((n_pad + 255) / 256 < 8 * sms ? (n_pad + 255) / 256 : 8 * sms);
    if (launch_dependent(sse_aug_kernel, dim3(g0), dim3(256), 0, stream, 1, lse, p, q_aug) != cudaSuccess)
        return PAFU_ERR_CUDA;
    const int n_items = n_heads * p.items_per_head;
    const int grid = n_items < sms ? n_items : sms;
    if ((gavg != nullptr ? launch_dependent(sse_tc_kernel<true>, dim3(grid), dim3(kThreads), kSmemBytes, stream, 1, mQ, mK, p, n_items)
                         : launch_dependent(sse_tc_kernel<false>, dim3(grid), dim3(kThreads), kSmemBytes, stream, 1, mQ, mK, p, n_items)) != cudaSuccess)
        return PAFU_ERR_CUDA;
    const int g2 = (int)((L + 255) / 256 < 4 * sms ? (L + 255) / 256 : 4 * sms);
    if (launch_dependent(sse_finish_kernel, dim3(g2), dim3(256), 0, stream, 1, p, s, comp, gmax, gavg) != cudaSuccess)
        return PAFU_ERR_CUDA;
    return PAFU_OK;
}

}  // namespace sse_tc
}  // namespace pafu
