// Salience Estimation Head on the tensor cores (Sec. 3.3; Appendix A "S-MLP"):
//   s_t = mean_o( W2 act(W1 x_t + b1) + b2 ),  optionally sigmoid(s_t).
//
// The first layer is a [tokens x d_in] x [d_in x d_hidden] contraction with ~d_hidden flop
// per input byte, i.e. on the tensor-core ridge; it runs as a tcgen05 GEMM and everything
// after it is fused into the accumulator read-out, so HBM traffic is "read X once, write
// 4 bytes per token".  Since the mean over outputs is linear, the second layer folds to
//   w2m[h] = mean_o W2[o, h],  b2m = mean_o b2[o],  s = sum_h w2m[h] act(a_h + b1[h]) + b2m.
//
// Persistent CTAs, one per SM, each taking 128-token tiles round-robin.  Warp roles:
//   warps 0-7  read-out: thread = token row (TMEM lane); warps w and w+4 split the hidden
//              columns of the same 32 rows; bias, activation, dot with w2m, row reduction
//   warp  8    MMA issuer (A = X tile, B = W1 tile, both K-major in shared memory)
//   warp  9    TMA loader, 4-stage ring of {X 128x64, W1 256x64} tiles
// Hidden units are processed in chunks of up to 256 (one accumulator of 256 TMEM columns);
// two accumulators alternate so the read-out of one chunk overlaps the MMAs of the next.
// When the token tiles alone would leave SMs idle (few tokens, a wide head) the kernel is
// launched in clusters of n_chunks CTAs instead: each CTA takes one 256-unit chunk of one tile,
// the partial row sums meet in the first CTA's shared memory (distributed shared memory) and are
// added there in chunk order, so the result does not depend on timing.
// All mbarrier waits are bounded (see sm100.cuh).
#pragma once
#include <cooperative_groups.h>

#include "common.cuh"
#include "sm100.cuh"

namespace pafu {
namespace score_tc {

using namespace sm100;

constexpr int kBM = 128;             // tokens per tile
constexpr int kBK = 64;              // reduction slice per stage (one 128-byte swizzle row)
constexpr int kNMax = 256;           // hidden units per accumulator
constexpr int kStages = 4;
constexpr int kThreads = 384;
constexpr int kXBytes = kBM * kBK * 2;          // 16 KiB
constexpr int kWBytes = kNMax * kBK * 2;        // 32 KiB
constexpr int kStageBytes = kXBytes + kWBytes;
constexpr int kMaxHidden = 1024;
constexpr int kMaxChunks = kMaxHidden / kNMax;
constexpr int kSmemBytes = kStages * kStageBytes + 2 * kMaxHidden * 4 + 2 * kBM * 4 + kMaxChunks * kBM * 4 + 256 + 1024;

struct Params {
    int64_t n_tokens;
    int d_in, d_hidden, d_out, act, final;
    int k_per_part;      // reduction slices (of kBK features) taken from each input matrix
    int split;           // 1: one (tile, chunk) per CTA, clusters of n_chunks CTAs
    int tail_tiles;      // > 0: the last tail_tiles tiles are each split between the two CTAs of a cluster,
    int tail_width;      //      tail_width hidden units per CTA (d_hidden / 2)
    const uint16_t* w2;
    const uint16_t* b1;
    const uint16_t* b2;
    float* scores;
    int* status;
};

__device__ __forceinline__ float bf16_bits(uint16_t b) { return __uint_as_float(((uint32_t)b) << 16); }

__device__ __forceinline__ float ex2f(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float rcpf(float x) { float y; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }

// GELU in its exact form x * Phi(x) = x/2 * (1 + erf(x / sqrt 2)), erf by the rational
// approximation of Abramowitz & Stegun 7.1.26 (absolute error below 1.5e-7).
__device__ __forceinline__ float gelu_erf(float x) {
    const float z = fabsf(x) * 0.70710678118654752f;
    const float t = rcpf(fmaf(0.3275911f, z, 1.0f));
    float poly = fmaf(1.061405429f, t, -1.453152027f);
    poly = fmaf(poly, t, 1.421413741f);
    poly = fmaf(poly, t, -0.284496736f);
    poly = fmaf(poly, t, 0.254829592f);
    const float e = ex2f(-z * z * 1.4426950408889634f);
    const float erf_abs = fmaf(-poly * t, e, 1.0f);
    const float erf_v = copysignf(erf_abs, x);
    return 0.5f * x * (1.0f + erf_v);
}
__device__ __forceinline__ float silu(float x) { return x * rcpf(1.0f + ex2f(-x * 1.4426950408889634f)); }

template <int ACT>
__device__ __forceinline__ float act_fn(float x) { return ACT == PAFU_ACT_GELU ? gelu_erf(x) : silu(x); }

template <int ACT>
__global__ void __launch_bounds__(kThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap mX, const __grid_constant__ CUtensorMap mX1,
                const __grid_constant__ CUtensorMap mX2, const __grid_constant__ CUtensorMap mW,
                const __grid_constant__ CUtensorMap mWt, const __grid_constant__ Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sStage = smem_u32(smem);
    float* w2m = reinterpret_cast<float*>(smem + kStages * kStageBytes);
    float* b1s = w2m + kMaxHidden;
    float* half_sum = b1s + kMaxHidden;                      // [2][kBM]: partial of column-half 1
    float* chunk_sum = half_sum + 2 * kBM;                   // [kMaxChunks][kBM]: per-chunk row sums (split mode, first CTA)
    uint64_t* bars = reinterpret_cast<uint64_t*>(chunk_sum + kMaxChunks * kBM);
    const uint32_t bar0 = smem_u32(bars);
    auto full = [&](int st) { return bar0 + 8 * st; };
    auto empty = [&](int st) { return bar0 + 8 * (kStages + st); };
    auto acc_full = [&](int b) { return bar0 + 8 * (2 * kStages + b); };
    auto acc_empty = [&](int b) { return bar0 + 8 * (2 * kStages + 2 + b); };
    // column-half 1 -> column-half 0, one barrier per half_sum slot: with a single barrier the half-1
    // warps could complete two tiles' arrivals while a half-0 warp still waits for the first
    auto halves_bar = [&](int slot) { return bar0 + 8 * (2 * kStages + 4 + slot); };
    __shared__ uint32_t tmem_base_sh;
    __shared__ volatile int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t n_tiles = (p.n_tokens + kBM - 1) / kBM;
    const int n_chunks = (p.d_hidden + kNMax - 1) / kNMax;
    const int n_k = p.d_in / kBK;
    // Work of this CTA: tiles tile0, tile0 + tile_step, ... below n_main and chunks [ch0, ch1) of each;
    // then, when the tiles do not fill the last round of CTAs, one "tail" unit: half of the hidden
    // units of tile n_main + blockIdx / 2 (the two CTAs of a cluster share a tail tile, so the last
    // round costs about two thirds of a full one instead of leaving half of the SMs idle).
    const int64_t tile0 = p.split ? blockIdx.x / n_chunks : blockIdx.x;
    const int64_t tile_step = p.split ? n_tiles : gridDim.x;
    const int ch0 = p.split ? (int)(blockIdx.x % n_chunks) : 0;
    const int ch1 = p.split ? ch0 + 1 : n_chunks;
    const int64_t n_main = n_tiles - p.tail_tiles;
    const bool has_tail = p.tail_tiles > 0 && (int)(blockIdx.x >> 1) < p.tail_tiles;
    const int tail_half = (int)(blockIdx.x & 1);
    const int64_t tail_tile = n_main + (blockIdx.x >> 1);
    // the i-th tile-level unit of this CTA: false when there is none
    struct Unit { int64_t tile; int c0, c1; bool tail; };
    auto unit_at = [&](int64_t tile_next, bool tail_done, Unit& u) -> bool {
        if (tile_next < n_main) { u.tile = tile_next; u.c0 = ch0; u.c1 = ch1; u.tail = false; return true; }
        if (has_tail && !tail_done) { u.tile = tail_tile; u.c0 = 0; u.c1 = 1; u.tail = true; return true; }
        return false;
    };
    const uint32_t tail_stage_bytes = kXBytes + (uint32_t)p.tail_width * kBK * 2;

    if (tid == 0) {
        for (int st = 0; st < kStages; ++st) { mbar_init(full(st), 1); mbar_init(empty(st), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), 8); }
        mbar_init(halves_bar(0), 4); mbar_init(halves_bar(1), 4);
        abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 8) { tmem_alloc(smem_u32(&tmem_base_sh), 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_sh;
    grid_dep_wait();          // set-up above is local; everything below reads or writes global memory
    // Folded second layer and first-layer bias, fp32 in shared memory: the read-out warps' business
    // (they meet at a barrier of their own below), so the loader and the first MMAs do not wait
    // for these global reads.
    float b2m = 0.f;
    if (warp < 8) {
        for (int h = tid; h < p.d_hidden; h += 256) {
            float m = 0.f;
            for (int o = 0; o < p.d_out; ++o) m += bf16_bits(p.w2[(int64_t)o * p.d_hidden + h]);
            w2m[h] = m / (float)p.d_out;
            b1s[h] = p.b1 ? bf16_bits(p.b1[h]) : 0.f;
        }
        if (p.b2) {
            for (int o = 0; o < p.d_out; ++o) b2m += bf16_bits(p.b2[o]);
            b2m /= (float)p.d_out;
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");    // unconditional and before any wait that can fail
    }

    auto fail = [&](int code) {
        abort_flag = 1;
        atomicCAS(p.status, 0, code);
    };

    if (warp == 9) {
        // ---------------------------------------------------------------------- TMA loader
        if (elect_one()) {
            prefetch_tmap(&mX); prefetch_tmap(&mW);
            if (p.k_per_part < n_k) { prefetch_tmap(&mX1); prefetch_tmap(&mX2); }
            prefetch_tmap(&mWt);
            uint32_t ring = 0;
            bool ok = true;
            Unit u;
            int64_t tile_next = tile0;
            for (bool tail_done = false; ok && unit_at(tile_next, tail_done, u); tile_next += tile_step, tail_done = u.tail) {
                const int64_t tile = u.tile;
                for (int ch = u.c0; ch < u.c1 && ok; ++ch) {
                    for (int k = 0; k < n_k; ++k, ++ring) {
                        const int st = ring % kStages;
                        if (abort_flag || !mbar_wait(empty(st), ((ring / kStages) & 1u) ^ 1u)) { fail(401); ok = false; break; }
                        const uint32_t dst = sStage + st * kStageBytes;
                        mbar_arrive_expect_tx(full(st), u.tail ? tail_stage_bytes : (uint32_t)kStageBytes);
                        // a token's features are the concatenation of its rows in up to three matrices
                        const int part = k / p.k_per_part;
                        const CUtensorMap* mx = part == 0 ? &mX : (part == 1 ? &mX1 : &mX2);
                        tma_load_2d(dst, mx, full(st), (k - part * p.k_per_part) * kBK, (int)(tile * kBM));
                        if (u.tail) tma_load_2d(dst + kXBytes, &mWt, full(st), k * kBK, tail_half * p.tail_width);
                        else tma_load_2d(dst + kXBytes, &mW, full(st), k * kBK, ch * kNMax);
                    }
                }
            }
            if (!ok)
                for (uint32_t r = ring > (uint32_t)kStages ? ring - kStages : 0; r < ring; ++r)
                    mbar_wait(full(r % kStages), (r / kStages) & 1u);
        }
        __syncwarp();
    } else if (warp == 8) {
        // ---------------------------------------------------------------------- MMA issuer
        if (elect_one()) {
            const uint64_t desc0 = make_smem_desc_sw128(0, 16, 1024);
            uint32_t ring = 0, acc_it = 0;
            bool ok = true;
            Unit u;
            int64_t tile_next = tile0;
            for (bool tail_done = false; ok && unit_at(tile_next, tail_done, u); tile_next += tile_step, tail_done = u.tail) {
                for (int ch = u.c0; ch < u.c1 && ok; ++ch, ++acc_it) {
                    const int buf = acc_it & 1;
                    const int nc = u.tail ? p.tail_width : min(kNMax, p.d_hidden - ch * kNMax);
                    const uint32_t idesc = make_idesc_bf16(kBM, nc, false, false);
                    if (abort_flag || !mbar_wait(acc_empty(buf), ((acc_it >> 1) & 1u) ^ 1u)) { fail(402); ok = false; break; }
                    tc_fence_after_sync();
                    for (int k = 0; k < n_k; ++k, ++ring) {
                        const int st = ring % kStages;
                        if (abort_flag || !mbar_wait(full(st), (ring / kStages) & 1u)) { fail(403); ok = false; break; }
                        tc_fence_after_sync();
                        const uint64_t a = desc0 + ((sStage + st * kStageBytes) >> 4);
                        const uint64_t b = desc0 + ((sStage + st * kStageBytes + kXBytes) >> 4);
#pragma unroll
                        for (int kk = 0; kk < kBK / 16; ++kk)
                            umma_ss(tmem + buf * kNMax, a + kk * 2, b + kk * 2, idesc, (k | kk) != 0);
                        umma_commit(empty(st));
                    }
                    if (ok) umma_commit(acc_full(buf));
                }
            }
        }
        __syncwarp();
    } else if (warp < 8) {
        // ------------------------------------------------------------------------ read-out
        const int quad = warp & 3, half = warp >> 2;
        const uint32_t lane_base = ((uint32_t)(quad * 32)) << 16;
        const int row = quad * 32 + lane;
        uint32_t acc_it = 0, tile_it = 0;
        bool ok = true;
        Unit u;
        int64_t tile_next = tile0;
        for (bool tail_done = false; ok && unit_at(tile_next, tail_done, u); tile_next += tile_step, tail_done = u.tail, ++tile_it) {
            const int64_t tile = u.tile;
            float part = 0.f;
            for (int ch = u.c0; ch < u.c1; ++ch, ++acc_it) {
                const int buf = acc_it & 1;
                const int nc = u.tail ? p.tail_width : min(kNMax, p.d_hidden - ch * kNMax);
                const int h_base = u.tail ? tail_half * p.tail_width : ch * kNMax;    // first hidden unit of this accumulator
                {
                    const bool w = mbar_wait(acc_full(buf), (acc_it >> 1) & 1u) && !abort_flag;
                    if (!__all_sync(0xffffffffu, w)) { fail(404); ok = false; break; }
                }
                tc_fence_after_sync();
                // 16-column groups of this chunk alternate between the two warps of a row
                for (int g16 = half; g16 < nc / 16; g16 += 2) {
                    uint32_t r[16];
                    PAFU_TMEM_LD_X16(tmem + buf * kNMax + lane_base + g16 * 16, r);
                    tmem_wait_ld();
                    const int h0 = h_base + g16 * 16;
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        part = fmaf(w2m[h0 + i], act_fn<ACT>(__uint_as_float(r[i]) + b1s[h0 + i]), part);
                }
                tc_fence_before_sync();
                __syncwarp();
                // the column-half-0 warps hand back a tile's last accumulator only after they have
                // taken the other half's partial sums (below): the MMAs that reuse the accumulator, and
                // with them the half-1 warps, can then never run two tiles ahead of a half-0 warp
                if (lane == 0 && (half == 1 || ch + 1 < u.c1)) mbar_arrive(acc_empty(buf));
            }
            if (!ok) break;
            // combine the two column halves of each row
            float* hs = half_sum + (tile_it & 1) * kBM;
            if (half == 1) {
                hs[row] = part;
                __syncwarp();
                if (lane == 0) mbar_arrive(halves_bar(tile_it & 1));
            } else {
                const bool w = mbar_wait(halves_bar(tile_it & 1), (tile_it >> 1) & 1u) && !abort_flag;
                if (!__all_sync(0xffffffffu, w)) { fail(405); ok = false; break; }
                const float other = hs[row];
                __syncwarp();
                if (lane == 0) mbar_arrive(acc_empty((acc_it - 1) & 1));
                const int64_t t = tile * kBM + row;
                if (p.split || u.tail) {
                    // this chunk's (this half's) row sums go to the cluster's first CTA
                    cooperative_groups::this_cluster().map_shared_rank(chunk_sum, 0)[(u.tail ? tail_half : ch0) * kBM + row] = part + other;
                } else if (t < p.n_tokens) {
                    float v = part + other + b2m;
                    if (p.final == PAFU_FINAL_SIGMOID) v = rcpf(1.0f + ex2f(-v * 1.4426950408889634f));
                    p.scores[t] = v;
                }
            }
        }
    }
    if (p.split || p.tail_tiles > 0) {
        // every thread of the cluster gets here (all loops above are bounded)
        cooperative_groups::this_cluster().sync();
        const bool mine = p.split ? ch0 == 0 : (has_tail && tail_half == 0);
        const int n_parts = p.split ? n_chunks : 2;
        if (mine && tid < kBM) {
            const int64_t t = (p.split ? tile0 : tail_tile) * kBM + tid;
            if (t < p.n_tokens) {
                float v = chunk_sum[tid];
                for (int c = 1; c < n_parts; ++c) v += chunk_sum[c * kBM + tid];
                v += b2m;
                if (p.final == PAFU_FINAL_SIGMOID) v = rcpf(1.0f + ex2f(-v * 1.4426950408889634f));
                p.scores[t] = v;
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem, 512);
}

// X[0..n_parts) are the matrices whose rows, side by side, form a token's d_in features
// (n_parts = 1: a plain [n_tokens, d_in] matrix; 3: query, key and value rows of d_in / 3 each).
inline pafu_status launch(const pafu_head& head, const uint16_t* const* X, int n_parts, int64_t n_tokens, int64_t ldx,
                          float* scores, int* status, int sm_count, cudaStream_t stream) {
    CUtensorMap mX[3], mW;
    const int d_part = head.d_in / n_parts;
    for (int i = 0; i < 3; ++i)
        if (!TmapEncoder::matrix(&mX[i], X[i < n_parts ? i : 0], (uint64_t)n_tokens, (uint64_t)d_part, (uint64_t)ldx, kBM))
            return PAFU_ERR_CUDA;
    if (!TmapEncoder::matrix(&mW, head.w1, (uint64_t)head.d_hidden, (uint64_t)head.d_in, (uint64_t)head.d_in, kNMax))
        return PAFU_ERR_CUDA;
    Params p;
    p.n_tokens = n_tokens; p.d_in = head.d_in; p.d_hidden = head.d_hidden; p.d_out = head.d_out;
    p.act = head.act; p.final = head.final; p.w2 = head.w2; p.b1 = head.b1; p.b2 = head.b2;
    p.scores = scores; p.status = status;
    p.k_per_part = d_part / kBK;
    const int64_t n_tiles = (n_tokens + kBM - 1) / kBM;
    const int n_chunks = (head.d_hidden + kNMax - 1) / kNMax;
    // few tokens and a wide head: one CTA per (tile, chunk), clusters of n_chunks CTAs
    p.split = (n_chunks > 1 && n_tiles * n_chunks <= 2 * (int64_t)sm_count) ? 1 : 0;
    // tiles that fill at most half of the last round of CTAs (220 tiles on 148 SMs leave 72): each
    // is shared by the two CTAs of a cluster, half of the hidden units each
    p.tail_tiles = 0; p.tail_width = 0;
    const int64_t rest = n_tiles % sm_count;
    if (!p.split && n_chunks == 1 && head.d_hidden % 32 == 0 && sm_count % 2 == 0 && rest > 0 && 2 * rest <= sm_count) {
        p.tail_tiles = (int)rest;
        p.tail_width = head.d_hidden / 2;
    }
    CUtensorMap mWt = mW;
    if (p.tail_tiles > 0 &&
        !TmapEncoder::matrix(&mWt, head.w1, (uint64_t)head.d_hidden, (uint64_t)head.d_in, (uint64_t)head.d_in, (uint32_t)p.tail_width))
        return PAFU_ERR_CUDA;
    int grid = p.split ? (int)(n_tiles * n_chunks) : (int)(n_tiles < sm_count ? n_tiles : sm_count);
    if (p.tail_tiles > 0 && n_tiles < sm_count) grid = 2 * p.tail_tiles;      // no full round at all
    const unsigned cluster = p.split ? (unsigned)n_chunks : (p.tail_tiles > 0 ? 2u : 1u);
    static bool attr_set[kMaxDevices] = {};
    if (!once_per_device(attr_set, [] {
            return cudaFuncSetAttribute(score_tc_kernel<PAFU_ACT_GELU>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) == cudaSuccess &&
                   cudaFuncSetAttribute(score_tc_kernel<PAFU_ACT_SILU>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) == cudaSuccess;
        }))
        return PAFU_ERR_CUDA;
    return cuda_ok(head.act == PAFU_ACT_GELU
                       ? launch_dependent(score_tc_kernel<PAFU_ACT_GELU>, dim3(grid), dim3(kThreads), kSmemBytes, stream, cluster, mX[0], mX[1], mX[2], mW, mWt, p)
                       : launch_dependent(score_tc_kernel<PAFU_ACT_SILU>, dim3(grid), dim3(kThreads), kSmemBytes, stream, cluster, mX[0], mX[1], mX[2], mW, mWt, p));
}

}  // namespace score_tc
}  // namespace pafu
