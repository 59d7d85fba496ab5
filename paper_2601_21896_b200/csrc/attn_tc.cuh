// Chunk attention on the 5th-generation tensor cores (tcgen05 + TMEM + TMA), d_head = 128 (and 64:
// a second instantiation, see HeadDims; the text below gives the sizes for 128).
//
//   o_i = sum_j softmax_j(scale q_i.k_j) v_j,  j over [retained cache ; chunk tokens]
//   (Sec. 3.2 for the operator; Eq. 2 / Eq. 7 for the key range)
//
// Work decomposition.  An "item" is 256 query rows of one head of one stream, handled as two
// 128-row "slots" that share every K/V tile (each tile is fetched once per 256 rows).  The
// grid is persistent: one CTA per SM.  All items' key tiles are laid end to end and cut into
// equal contiguous shares, one per CTA (a tile with both slots live costs 8 units, with one
// slot 6: a lone slot has no partner to hide its softmax behind), so every SM gets the same
// amount of work whatever the item count.  A CTA whose share covers only
// part of an item's keys writes an unnormalised partial (O, running max, row sum) to the
// workspace; a second small kernel merges the partials of each split item in key order, which
// keeps the result deterministic.
//
// Warp roles inside a CTA (384 threads):
//   warps 0-3  softmax of slot 0 (thread = query row = TMEM lane)
//   warps 4-7  softmax of slot 1
//   warps 8,10 MMA issuers, one per slot: S = Q K^T (both operands in shared memory) and
//              O += P V (P read from tensor memory, V from shared memory, MN-major).  With the
//              waits, commits and descriptor arithmetic of its loop one thread sustains about
//              one tcgen05.mma per 100 clocks while the tensor core finishes a 128x128x16 one
//              in 64, hence an issuing thread per slot
//   warp  9    TMA loader: Q tiles per item, 64-key K/V tiles through a 10-stage ring that
//              runs ahead across item boundaries
//   warp  11   idle (completes the third warpgroup so registers can be re-balanced)
// Tensor memory (512 columns): per slot two S buffers of 64 fp32 columns and one O accumulator
// of 128; the bf16 P tile overwrites the first 32 columns of its S buffer.  S is double
// buffered so that S(j+1) = Q K_{j+1}^T is already finished when the softmax of tile j ends:
// the softmax warps never wait for the tensor core in steady state, and the issuer's order
// "P(j) ready -> O += P(j) V_j -> S(j+2)" keeps the buffer reuse safe without extra barriers.
//
// Online softmax with lazy rescaling: the running maximum only moves when the new tile
// exceeds it by more than 2^8 in the exponent, so the O accumulator is rarely rescaled; when
// it is, the slot's own softmax warps do it after waiting for the previous P V product.
//
// Every mbarrier wait is bounded.  A wait that runs out sets the status word, raises a CTA-wide
// abort flag, and all roles fall through to the common exit where TMEM is released.
#pragma once
#include "common.cuh"
#include "sm100.cuh"

namespace pafu {
namespace attn_tc {

using namespace sm100;

constexpr int kD = 128;
constexpr int kBM = 128;            // query rows per slot
constexpr int kBN = 64;             // keys per tile
constexpr int kStages = 10;         // K/V ring depth (each stage one 64 x 128 bf16 tile)
constexpr int kThreads = 384;       // 3 warpgroups: softmax 0, softmax 1, {2 MMA issuers, loader, 1 idle}
constexpr int kQBytes = kBM * kD * 2;         // 32 KiB: one slot's Q tile
constexpr int kQHalf = kQBytes / 2;           // one [128 rows x 64 cols] swizzled half
constexpr int kTileBytes = kBN * kD * 2;      // 16 KiB: one K or V tile
constexpr int kHalfBytes = kTileBytes / 2;    // one [64 rows x 64 cols] swizzled half
constexpr int kSmemBytes = 2 * kQBytes + kStages * kTileBytes + 1024 /*align*/ + 512 /*barriers*/;
constexpr float kRescaleThresholdLog2 = 8.0f;
constexpr float kSumTrigger = 65536.0f;   // a 64-key row sum this large means some p exceeded 2^10
// Register re-balancing.  With 384 threads the kernel launches with 168 registers per thread.
// setmaxnreg.inc blocks until the registers exist, so what the third warpgroup gives up must
// cover what the two softmax warpgroups take: (168 - kRegsLow) * 128 >= (kRegsHigh - 168) * 256.
constexpr int kRegsLaunch = 168, kRegsLow = 80, kRegsHigh = 208;
static_assert((kRegsLaunch - kRegsLow) * 128 >= (kRegsHigh - kRegsLaunch) * 256,
              "setmaxnreg.inc would wait forever");
constexpr int kMaxGrid = kMaxPersistentGrid;
// one partial: O [256][128] fp32, then m [256], then l [256]
constexpr int kPieceFloats = 2 * kBM * kD + 2 * 2 * kBM;
constexpr size_t kPieceBytes = (size_t)kPieceFloats * 4;

struct Params {
    StreamTable st;
    int n_heads;
    int has_chunk;
    float scale;
    uint16_t* O;
    float* LSE;
    int* status;        // workspace status word (device)
    float* pieces;      // [gridDim][2][kPieceFloats]
    const int32_t* idx; // gather variant: retained token indices, stream-local, [cu_B[n_streams]]
    const uint16_t* Kraw;   // gather variant: the uncompacted cache [cu_T[n_streams], n_heads, 128]
    const uint16_t* Vraw;
    int64_t total_Lq;
    int64_t total_cost;
};

// A contiguous run of key tiles [t0, t1) of one item, as seen by one CTA.
struct Seg {
    int stream, head, n_slots;
    int64_t q0;          // first query row (stream-local)
    int64_t Lq, nB, nC;  // stream's query rows, retained keys, chunk keys
    int nt1, nt, t0, t1; // tiles in the retained segment, tiles in total, this run
    int piece;           // -1: whole item (final output); 0: continues an item begun by an
                         // earlier CTA; 1: begins an item that a later CTA continues
};

constexpr int kCost2 = 8, kCost1 = 6;   // cost of one key tile with two / one live slots (best of 5..7 on every measured workload)

struct StreamCost {
    int64_t nqp, nt, head_cost;
    int tail_slots;
};

__host__ __device__ inline StreamCost stream_cost(const StreamTable& st, int s, int has_chunk) {
    StreamCost c;
    const int64_t lq = st.cu_Lq[s + 1] - st.cu_Lq[s];
    const int64_t nB = st.cu_B[s + 1] - st.cu_B[s];
    c.nqp = (lq + 2 * kBM - 1) / (2 * kBM);
    c.tail_slots = (lq - (c.nqp - 1) * 2 * kBM > kBM) ? 2 : 1;
    c.nt = (nB + kBN - 1) / kBN + (has_chunk ? (lq + kBN - 1) / kBN : 0);
    c.head_cost = (lq > 0) ? c.nt * (kCost2 * (c.nqp - 1) + (c.tail_slots == 2 ? kCost2 : kCost1)) : 0;
    return c;
}

__host__ __device__ inline int64_t total_cost(const StreamTable& st, int n_heads, int has_chunk) {
    int64_t t = 0;
    for (int s = 0; s < st.n_streams; ++s) t += stream_cost(st, s, has_chunk).head_cost * n_heads;
    return t;
}

// Walks the runs of one CTA's share [c0, c1) of the cost line.  Only the first run of a CTA
// can start inside an item (t0 > 0) and only its last run can stop inside one (t1 < nt).
struct SegIter {
    int64_t cur, c1;
    __host__ __device__ SegIter(const Params& p, int cta, int n_cta) {
        cur = p.total_cost * cta / n_cta;
        c1 = p.total_cost * (cta + 1) / n_cta;
    }
    __host__ __device__ bool next(const Params& p, Seg& g) {
        while (cur < c1) {
            int64_t c = cur;
            int s = 0;
            StreamCost sc;
            for (;; ++s) {
                sc = stream_cost(p.st, s, p.has_chunk);
                const int64_t tot = sc.head_cost * p.n_heads;
                if (c < tot) break;
                c -= tot;
            }
            g.stream = s;
            g.head = (int)(c / sc.head_cost);
            const int64_t r = c % sc.head_cost;
            const int64_t full = sc.nt * kCost2 * (sc.nqp - 1);
            int64_t qp, rr;
            if (r < full) { qp = r / (kCost2 * sc.nt); rr = r % (kCost2 * sc.nt); g.n_slots = 2; }
            else { qp = sc.nqp - 1; rr = r - full; g.n_slots = sc.tail_slots; }
            const int unit = g.n_slots == 2 ? kCost2 : kCost1;
            g.q0 = qp * 2 * kBM;
            g.Lq = p.st.cu_Lq[s + 1] - p.st.cu_Lq[s];
            g.nB = p.st.cu_B[s + 1] - p.st.cu_B[s];
            g.nC = p.has_chunk ? g.Lq : 0;
            g.nt1 = (int)((g.nB + kBN - 1) / kBN);
            g.nt = (int)sc.nt;
            const int64_t item_start = cur - rr, item_end = item_start + sc.nt * unit;
            g.t0 = (int)(rr / unit);
            if (c1 >= item_end) { g.t1 = g.nt; cur = item_end; }
            else { g.t1 = (int)((c1 - item_start) / unit); cur = c1; }
            if (g.t1 > g.t0) {
                g.piece = (g.t0 == 0 && g.t1 == g.nt) ? -1 : (g.t0 > 0 ? 0 : 1);
                return true;
            }
        }
        return false;
    }
};

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// packed fp32 pairs (two lanes per instruction on the FMA pipe)
__device__ __forceinline__ uint64_t pack2(uint32_t lo, uint32_t hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t fadd2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// GATHER = false: the retained keys/values are the rows of a compacted cache (mKc, mVc are tiled
// maps of it).  GATHER = true: they are rows idx[.] of the uncompacted cache, fetched by the
// loader warp with 16-byte asynchronous copies (mKc, mVc unused); everything downstream of the
// shared-memory ring is identical.
// Sizes that depend on the head width D (128, or 64: every tile is then a single 64-column
// swizzled block, S = Q K^T takes four slices and O has 64 columns).
template <int D>
struct HeadDims {
    static constexpr int kQBytes = kBM * D * 2;                  // one slot's Q tile
    static constexpr int kQHalf = kBM * 64 * 2;                  // one [128 rows x 64 cols] swizzled block of it
    static constexpr int kHalfBytes = kBN * 64 * 2;              // one [64 rows x 64 cols] swizzled block of a K or V tile
    static constexpr int kTileBytes = kBN * D * 2;
    static constexpr int kSmemBytes = 2 * kQBytes + kStages * kTileBytes + 1024 /*align*/ + 512 /*barriers*/;
    static constexpr int kPieceFloats = 2 * kBM * D + 2 * 2 * kBM;   // one partial: O [256][D], m [256], l [256]
};

template <bool GATHER, int D>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap mQ, const __grid_constant__ CUtensorMap mKc,
               const __grid_constant__ CUtensorMap mVc, const __grid_constant__ CUtensorMap mKq,
               const __grid_constant__ CUtensorMap mVq, const __grid_constant__ Params p) {
    static_assert(D == 128 || (D == 64 && !GATHER), "head widths: 128, or 64 with a compacted cache");
    // this instantiation's sizes (they shadow the D = 128 constants of the namespace)
    constexpr int kD = D;
    constexpr int kQBytes = HeadDims<D>::kQBytes, kQHalf = HeadDims<D>::kQHalf;
    constexpr int kTileBytes = HeadDims<D>::kTileBytes, kHalfBytes = HeadDims<D>::kHalfBytes;
    constexpr int kPieceFloats = HeadDims<D>::kPieceFloats;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sQ = smem_u32(smem);                       // 2 slots x 32 KiB
    const uint32_t sKV = sQ + 2 * kQBytes;                    // ring
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 2 * kQBytes + kStages * kTileBytes);
    const uint32_t bar0 = smem_u32(bars);
    auto q_full = [&](int s) { return bar0 + 8 * (0 + s); };
    auto q_empty = [&](int s) { return bar0 + 8 * (2 + s); };
    auto s_full = [&](int s, int b) { return bar0 + 8 * (4 + 2 * s + b); };
    // P-ready is per S buffer as well: the softmax may finish tile j+1 (whose S was computed
    // early) before the issuer has looked at tile j, and a single barrier would be lapped
    auto p_full = [&](int s, int b) { return bar0 + 8 * (8 + 2 * s + b); };
    auto pv_done = [&](int s) { return bar0 + 8 * (12 + s); };
    auto o_done = [&](int s) { return bar0 + 8 * (14 + s); };
    auto kv_full = [&](int st) { return bar0 + 8 * (16 + st); };
    auto kv_empty = [&](int st) { return bar0 + 8 * (16 + kStages + st); };
    __shared__ uint32_t tmem_base_sh;
    __shared__ volatile int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5;

    if (tid == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(q_full(s), 1); mbar_init(q_empty(s), 1);
            mbar_init(s_full(s, 0), 1); mbar_init(s_full(s, 1), 1);
            mbar_init(p_full(s, 0), 4); mbar_init(p_full(s, 1), 4);   // one arrival per softmax warp
            mbar_init(pv_done(s), 1); mbar_init(o_done(s), 1);
        }
        for (int st = 0; st < kStages; ++st) {
            mbar_init(kv_full(st), GATHER ? 32 : 1);    // gather: every lane of the loader warp arrives
            mbar_init(kv_empty(st), 2);                 // both issuers release a stage
        }
        abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 8) { tmem_alloc(smem_u32(&tmem_base_sh), 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_sh;
    grid_dep_wait();          // set-up above is local; everything below reads or writes global memory

    auto fail = [&](int code) {
        abort_flag = 1;
        atomicCAS(p.status, 0, code);
    };

    if (warp >= 8) {
    // register budget: this warpgroup gives registers up, the softmax warpgroups take them
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsLow));
    if (warp == 11 && !GATHER) {
        // idle
    } else if (warp == 9 || warp == 11) {
        // ------------------------------------------------------------------ TMA loader
        if constexpr (GATHER) {
            // Two loader warps walk the runs together: warp 9 fills the K stages of the ring (and
            // loads Q), warp 11 the V stages.  Lane 0 issues the tiled loads (Q, the chunk's own
            // K/V).  A retained 64-key tile is fetched with 16-byte asynchronous copies: a lane owns
            // 16-byte pieces c and c + 4 of a row in both 64-column halves (4 lanes per row, 8 rows
            // per warp instruction, 4 x 8 instructions per tile) and writes them where the tiled load
            // would have put them (128-byte swizzle: piece c of row r goes to piece c ^ (r mod 8)),
            // so the operand layout is unchanged.  The tile's 64 row offsets (in 16-byte units) sit
            // in two registers per lane, are handed round by shuffles and are fetched one tile
            // ahead of their use.
            const int lane = tid & 31;
            const int kv = warp == 9 ? 0 : 1;
            const int r8 = lane >> 2, piece = lane & 3;           // row within a group of eight; pieces `piece` and `piece + 4`
            if (lane == 0) {
                if (kv == 0) prefetch_tmap(&mQ);
                if (p.has_chunk) prefetch_tmap(kv ? &mVq : &mKq);
            }
            SegIter iter(p, blockIdx.x, gridDim.x);
            Seg g;
            uint32_t ring = (uint32_t)kv, qcnt0 = 0, qcnt1 = 0;     // this warp's stages: every other ring entry
            bool ok = true;
            auto wait_all = [&](uint32_t bar, uint32_t ph, int code) {
                const bool w = !abort_flag && mbar_wait(bar, ph);
                if (!__all_sync(0xffffffffu, w)) { if (lane == 0) fail(code); ok = false; }
            };
            const uint32_t row16 = (uint32_t)p.n_heads * (kD * 2 / 16);          // 16-byte units per token row
            // row = 8 it + r8, so row & 7 = r8: a lane's two swizzled positions never change
            const uint32_t dst_a = (uint32_t)(r8 * 128 + ((piece ^ r8) << 4));
            const uint32_t dst_b = (uint32_t)(r8 * 128 + (((piece + 4) ^ r8) << 4));
            while (ok && iter.next(p, g)) {
                if (kv == 0) {
                    const int qrow = (int)(p.st.cu_Lq[g.stream] + g.q0);
                    for (int s = 0; s < g.n_slots && ok; ++s) {
                        const uint32_t qc = s ? qcnt1 : qcnt0;
                        wait_all(q_empty(s), (qc & 1u) ^ 1u, 100);
                        if (!ok) break;
                        if (s) ++qcnt1; else ++qcnt0;
                        if (lane == 0) {
                            mbar_arrive_expect_tx(q_full(s), kQBytes);
                            tma_load_3d(sQ + s * kQBytes, &mQ, q_full(s), 0, g.head, qrow + s * kBM);
                            if constexpr (D == 128) tma_load_3d(sQ + s * kQBytes + kQHalf, &mQ, q_full(s), 64, g.head, qrow + s * kBM);
                        }
                    }
                }
                const int32_t* sidx = p.idx + p.st.cu_B[g.stream];
                const int row_base = (int)p.st.cu_T[g.stream];
                const uint8_t* base = reinterpret_cast<const uint8_t*>(kv ? p.Vraw : p.Kraw) +
                                      (size_t)g.head * (kD * 2) + piece * 16;
                // row offsets of a retained tile (rows past the segment's end repeat its last row:
                // their logits are masked, and their values must be finite)
                auto tile_offsets = [&](int j, uint32_t& o0, uint32_t& o1) {
                    o0 = o1 = 0;
                    if (j < g.t1 && j < g.nt1) {
                        int64_t pos = (int64_t)j * kBN + lane;
                        o0 = (uint32_t)(row_base + __ldg(sidx + (pos < g.nB ? pos : g.nB - 1))) * row16;
                        pos += 32;
                        o1 = (uint32_t)(row_base + __ldg(sidx + (pos < g.nB ? pos : g.nB - 1))) * row16;
                    }
                };
                uint32_t o0, o1, n0, n1;
                tile_offsets(g.t0, o0, o1);
                for (int j = g.t0; j < g.t1 && ok; ++j, ring += 2) {
                    const bool seg2 = j >= g.nt1;
                    const int st = ring % kStages;
                    tile_offsets(j + 1, n0, n1);                     // the next tile's indices, one tile ahead
                    wait_all(kv_empty(st), ((ring / kStages) & 1u) ^ 1u, 101);
                    if (!ok) break;
                    if (seg2) {
                        if (lane == 0) {
                            const CUtensorMap* m = kv ? &mVq : &mKq;
                            const int row2 = (int)(p.st.cu_Lq[g.stream] + (int64_t)(j - g.nt1) * kBN);
                            mbar_arrive_expect_tx(kv_full(st), kTileBytes);
                            tma_load_3d(sKV + st * kTileBytes, m, kv_full(st), 0, g.head, row2);
                            if constexpr (D == 128) tma_load_3d(sKV + st * kTileBytes + kHalfBytes, m, kv_full(st), 64, g.head, row2);
                        } else {
                            mbar_arrive(kv_full(st));
                        }
                    } else {
                        const uint32_t dst0 = sKV + st * kTileBytes;
#pragma unroll
                        for (int it = 0; it < kBN / 8; ++it) {
                            const uint32_t off16 = __shfl_sync(0xffffffffu, it < 4 ? o0 : o1, (8 * it + r8) & 31);
                            const uint8_t* src = base + (size_t)off16 * 16;
                            const uint32_t d = dst0 + it * 1024;
                            cp_async_16(d + dst_a, src);                                // columns 0..63
                            cp_async_16(d + dst_b, src + 64);
                            cp_async_16(d + dst_a + kHalfBytes, src + 128);             // columns 64..127
                            cp_async_16(d + dst_b + kHalfBytes, src + 192);
                        }
                        cp_async_mbar_arrive_noinc(kv_full(st));
                    }
                    o0 = n0; o1 = n1;
                }
            }
            cp_async_wait_all();
        } else if (elect_one() && p.status[kStatusWordStallLoader] == 0) {
            prefetch_tmap(&mQ); prefetch_tmap(&mKc); prefetch_tmap(&mVc);
            if (p.has_chunk) { prefetch_tmap(&mKq); prefetch_tmap(&mVq); }
            SegIter iter(p, blockIdx.x, gridDim.x);
            Seg g;
            uint32_t ring = 0, qcnt0 = 0, qcnt1 = 0;      // scalars: a runtime-indexed array would live in local memory
            bool ok = true;
            while (ok && iter.next(p, g)) {
                const int qrow = (int)(p.st.cu_Lq[g.stream] + g.q0);
                for (int s = 0; s < g.n_slots && ok; ++s) {
                    const uint32_t qc = s ? qcnt1 : qcnt0;
                    if (abort_flag || !mbar_wait(q_empty(s), (qc & 1u) ^ 1u)) { fail(100); ok = false; break; }
                    if (s) ++qcnt1; else ++qcnt0;
                    mbar_arrive_expect_tx(q_full(s), kQBytes);
                    tma_load_3d(sQ + s * kQBytes, &mQ, q_full(s), 0, g.head, qrow + s * kBM);
                    if constexpr (D == 128) tma_load_3d(sQ + s * kQBytes + kQHalf, &mQ, q_full(s), 64, g.head, qrow + s * kBM);
                }
                for (int j = g.t0; j < g.t1 && ok; ++j) {
                    const bool seg2 = j >= g.nt1;
                    const int row = seg2 ? (int)(p.st.cu_Lq[g.stream] + (int64_t)(j - g.nt1) * kBN)
                                         : (int)(p.st.cu_B[g.stream] + (int64_t)j * kBN);
                    for (int kv = 0; kv < 2; ++kv, ++ring) {
                        const int st = ring % kStages;
                        const uint32_t ph = (ring / kStages) & 1u;
                        if (abort_flag || !mbar_wait(kv_empty(st), ph ^ 1u)) { fail(101); ok = false; break; }
                        const CUtensorMap* m = seg2 ? (kv ? &mVq : &mKq) : (kv ? &mVc : &mKc);
                        mbar_arrive_expect_tx(kv_full(st), kTileBytes);
                        tma_load_3d(sKV + st * kTileBytes, m, kv_full(st), 0, g.head, row);
                        if constexpr (D == 128) tma_load_3d(sKV + st * kTileBytes + kHalfBytes, m, kv_full(st), 64, g.head, row);
                    }
                }
            }
            if (!ok) {
                // let copies already in flight land before the CTA exits
                for (uint32_t r = ring > (uint32_t)kStages ? ring - kStages : 0; r < ring; ++r)
                    mbar_wait(kv_full(r % kStages), (r / kStages) & 1u);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------- MMA issuers: warp 8 -> slot 0, warp 10 -> slot 1
        if (elect_one()) {
            const int slot = warp == 8 ? 0 : 1;
            const uint32_t idesc_qk = make_idesc_bf16(kBM, kBN, false, false);
            const uint32_t idesc_pv = make_idesc_bf16(kBM, kD, false, true);
            // Descriptors differ from tile to tile only in the 14-bit start-address field, so the
            // constant part is built once and the address (in 16-byte units) is added per MMA.
            const uint64_t desc_k = make_smem_desc_sw128(0, 16, 1024);             // K-major Q / K
            const uint64_t desc_v = make_smem_desc_sw128(0, kHalfBytes, 1024);     // MN-major V
            const uint64_t desc_q = desc_k + ((sQ + slot * kQBytes) >> 4);
            const uint32_t tSslot = tmem + slot * 128;
            const uint32_t tOslot = tmem + 256 + slot * kD;
            auto issue_qk = [&](int buf, int stage) {          // S[buf] = Q K^T, N = 64 keys
                const uint64_t b = desc_k + ((sKV + stage * kTileBytes) >> 4);
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk) {
                    const uint32_t qoff = ((kk >> 2) * kQHalf + (kk & 3) * 32) >> 4;
                    const uint32_t koff = ((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4;
                    umma_ss(tSslot + buf * kBN, desc_q + qoff, b + koff, idesc_qk, kk > 0);
                }
            };
            auto issue_pv = [&](int buf, int stage, bool first) {   // O += P[buf] V, K = 64 keys
                const uint64_t b = desc_v + ((sKV + stage * kTileBytes) >> 4);
#pragma unroll
                for (int kk = 0; kk < kBN / 16; ++kk)
                    umma_ts(tOslot, tSslot + buf * kBN + kk * 8, b + kk * (2048 >> 4), idesc_pv,
                            !(first && kk == 0));
            };
            // The issuing thread shares its scheduler with two softmax warps, so its own
            // instruction count per tile matters: ring positions are advanced incrementally (no
            // division), and the abort flag is only looked at when a wait fails.
            bool ok = true;
            auto wait = [&](uint32_t bar, uint32_t ph, int code) {
                if (!mbar_wait(bar, ph)) { fail(code); ok = false; }
            };
            struct Cursor {                      // position of a ring entry: stage and phase bit
                uint32_t st, ph;
                __device__ __forceinline__ void step(uint32_t k) {
                    st += k;
                    if (st >= (uint32_t)kStages) { st -= kStages; ph ^= 1u; }
                }
            };
            SegIter iter(p, blockIdx.x, gridDim.x);
            Seg g;
            Cursor cur{0u, 0u};                  // first ring entry of the next run
            uint32_t qcnt = 0, tc = 0;           // tc: tiles this slot has processed so far
            while (ok && iter.next(p, g)) {
                const int n = g.t1 - g.t0;
                if (slot >= g.n_slots) {
                    // nothing to compute for this slot, but every K/V stage is released by both issuers
                    for (int e = 0; e < 2 * n && ok; ++e) {
                        wait(kv_full(cur.st), cur.ph, 206);
                        if (ok) mbar_arrive(kv_empty(cur.st));
                        cur.step(1);
                    }
                    continue;
                }
                wait(q_full(slot), qcnt & 1u, 201);
                ++qcnt;
                // ring entries of this run: K_i at +2i, V_i at +2i+1
                Cursor ck = cur, cv = cur;
                cv.step(1);
                for (int i = 0; i < 2 && i < n && ok; ++i) {        // S(0), S(1)
                    wait(kv_full(ck.st), ck.ph, 202);
                    if (!ok) break;
                    if constexpr (GATHER) fence_proxy_async_smem();   // the tile came through the generic proxy
                    tc_fence_after_sync();
                    issue_qk((tc + i) & 1, ck.st);
                    umma_commit(s_full(slot, (tc + i) & 1));
                    umma_commit(kv_empty(ck.st));
                    ck.step(2);
                }
                if (n == 1) ck.step(2);                              // keep ck two tiles ahead of cv
#pragma unroll 1
                for (int i = 0; i < n && ok; ++i) {
                    const int buf = (tc + i) & 1;
                    wait(kv_full(cv.st), cv.ph, 203);
                    if (!ok) break;
                    if (!mbar_wait_spin(p_full(slot, buf), ((tc + i) >> 1) & 1u)) { fail(205); ok = false; break; }
                    if constexpr (GATHER) fence_proxy_async_smem();
                    tc_fence_after_sync();
                    issue_pv(buf, cv.st, i == 0);
                    umma_commit(kv_empty(cv.st));
                    if (i + 2 < n) {                                // S(i+2) reuses the buffer P(i) was read from
                        wait(kv_full(ck.st), ck.ph, 204);
                        if (!ok) break;
                        if constexpr (GATHER) fence_proxy_async_smem();
                        issue_qk(buf, ck.st);
                        umma_commit(s_full(slot, buf));
                        umma_commit(kv_empty(ck.st));
                    } else if (i + 2 == n) {
                        umma_commit(pv_done(slot));                 // lets the last tile's softmax know O is at rest
                    }
                    if (i == n - 1) { umma_commit(o_done(slot)); umma_commit(q_empty(slot)); }
                    cv.step(2);
                    ck.step(2);
                }
                tc += (uint32_t)n;
                cur.step((2u * (uint32_t)n) % kStages);
                if (((2u * (uint32_t)n) / kStages) & 1u) cur.ph ^= 1u;
            }
        }
        __syncwarp();
    }
    } else {
        // ------------------------------------------------------------------ softmax warps
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsHigh));
        const int slot = warp >> 2;
        const int row_in_slot = tid & 127;
        const uint32_t lane_base = ((uint32_t)((warp & 3) * 32)) << 16;
        const uint32_t tSslot = tmem + slot * 128 + lane_base;
        const uint32_t tO = tmem + 256 + slot * kD + lane_base;
        const float sl2 = p.scale * 1.4426950408889634f;
        const uint64_t sl2_2 = pack2(__float_as_uint(sl2), __float_as_uint(sl2));
        SegIter iter(p, blockIdx.x, gridDim.x);
        Seg g;
        uint32_t tc = 0, ocnt = 0, pvcnt = 0;     // pvcnt: runs of two or more tiles so far
        bool ok = true;
        while (ok && iter.next(p, g)) {
            if (slot >= g.n_slots) continue;
            float m_used = -INFINITY, l_sum = 0.f;
            const int n = g.t1 - g.t0;
            uint32_t sr[64];
            bool loaded = false;                       // S(i) already requested from tensor memory
            for (int i = 0; i < n; ++i) {
                const int j = g.t0 + i;
                const int buf = (tc + i) & 1;
                const uint32_t tS = tSslot + buf * kBN;
                if (!loaded) {
                    const bool w = mbar_wait_spin(s_full(slot, buf), ((tc + i) >> 1) & 1u) && !abort_flag;
                    if (!__all_sync(0xffffffffu, w)) { fail(301); ok = false; break; }   // warp-uniform
                    tc_fence_after_sync();
                    PAFU_TMEM_LD_X32(tS, sr);
                    PAFU_TMEM_LD_X32(tS + 32, sr + 32);
                }
                loaded = false;
                tmem_wait_ld();
                const bool seg2 = j >= g.nt1;
                const int64_t left = (seg2 ? g.nC - (int64_t)(j - g.nt1) * kBN : g.nB - (int64_t)j * kBN);
                // Fast path (every tile but a run's first and a segment's ragged last): the
                // exponentials use the running maximum as it stands.  Only when the tile's row sum
                // shows that some logit outgrew that maximum by more than 2^10 does the tile take
                // the full pass below (true maximum, rescale of O and of the row sum).
                bool full_pass = (i == 0) || (left < kBN);
                if (!full_pass) {
                    const float mbf = -m_used * sl2;
                    const uint64_t mb_2 = pack2(__float_as_uint(mbf), __float_as_uint(mbf));
                    uint64_t rs2[2] = {0ull, 0ull};
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t pk[16];
#pragma unroll
                        for (int q = 0; q < 16; ++q) {
                            float e0, e1;
                            unpack2(ffma2(pack2(sr[32 * c + 2 * q], sr[32 * c + 2 * q + 1]), sl2_2, mb_2), e0, e1);
                            const float p0 = fast_exp2(e0), p1 = fast_exp2(e1);
                            rs2[q & 1] = fadd2(rs2[q & 1], pack2(__float_as_uint(p0), __float_as_uint(p1)));
                            pk[q] = pack_bf16(p0, p1);
                        }
                        PAFU_TMEM_ST_X16(tS + 16 * c, pk);
                    }
                    float r0, r1, r2, r3;
                    unpack2(rs2[0], r0, r1);
                    unpack2(rs2[1], r2, r3);
                    const float rs = (r0 + r1) + (r2 + r3);
                    full_pass = __any_sync(0xffffffffu, !(rs < kSumTrigger));    // also true for inf / NaN
                    if (!full_pass) l_sum += rs;
                } else if (left < kBN) {               // ragged end of a key segment
#pragma unroll
                    for (int c = 0; c < kBN; ++c)
                        if (c >= left) sr[c] = 0xff800000u;   // -inf
                }
                if (full_pass) {
                    if ((tid & 31) == 0) atomicAdd(p.status + ((i == 0 || left < kBN) ? kStatusWordFullFirst : kStatusWordFullSum), 1);
                    float mx4[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        float m = fmaxf(__uint_as_float(sr[16 * q]), __uint_as_float(sr[16 * q + 1]));
#pragma unroll
                        for (int c = 2; c < 16; c += 2)
                            m = fmax3(m, __uint_as_float(sr[16 * q + c]), __uint_as_float(sr[16 * q + c + 1]));
                        mx4[q] = m;
                    }
                    const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                    if (i == 0) {
                        m_used = mx;
                    } else if (__any_sync(0xffffffffu, (mx - m_used) * sl2 > kRescaleThresholdLog2)) {
                        // The whole warp rescales together (TMEM accesses are warp-collective); rows
                        // whose maximum did not move get alpha = 1.  O must be at rest, i.e. the previous
                        // tile's P V product finished: S(i+1) being ready implies it (it was issued
                        // after that product); the run's last tile has a barrier of its own.
                        const bool w = (i + 1 < n ? mbar_wait(s_full(slot, buf ^ 1), ((tc + i + 1) >> 1) & 1u)
                                                  : mbar_wait(pv_done(slot), pvcnt & 1u)) && !abort_flag;
                        if (!__all_sync(0xffffffffu, w)) { fail(303); ok = false; break; }
                        tc_fence_after_sync();
                        if ((tid & 31) == 0) atomicAdd(p.status + kStatusWordRescale, 1);
                        const float m_new = fmaxf(m_used, mx);
                        const float alpha = fast_exp2((m_used - m_new) * sl2);
                        l_sum *= alpha;
                        m_used = m_new;
#pragma unroll
                        for (int c = 0; c < kD / 32; ++c) {
                            uint32_t orr[32];
                            PAFU_TMEM_LD_X32(tO + c * 32, orr);
                            tmem_wait_ld();
#pragma unroll
                            for (int q = 0; q < 32; ++q) orr[q] = __float_as_uint(__uint_as_float(orr[q]) * alpha);
                            PAFU_TMEM_ST_X32(tO + c * 32, orr);
                        }
                    }
                    const float mb = -m_used * sl2;
                    const uint64_t mb_2 = pack2(__float_as_uint(mb), __float_as_uint(mb));
                    uint64_t rs2[2] = {0ull, 0ull};
                    uint32_t pk[32];
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        float e0, e1;
                        unpack2(ffma2(pack2(sr[2 * c], sr[2 * c + 1]), sl2_2, mb_2), e0, e1);
                        const float p0 = fast_exp2(e0), p1 = fast_exp2(e1);
                        rs2[c & 1] = fadd2(rs2[c & 1], pack2(__float_as_uint(p0), __float_as_uint(p1)));
                        pk[c] = pack_bf16(p0, p1);
                    }
                    PAFU_TMEM_ST_X32(tS, pk);
                    float r0, r1, r2, r3;
                    unpack2(rs2[0], r0, r1);
                    unpack2(rs2[1], r2, r3);
                    l_sum += (r0 + r1) + (r2 + r3);
                }   // full_pass
                if (i + 1 < n && __all_sync(0xffffffffu, mbar_test_wait(s_full(slot, buf ^ 1), ((tc + i + 1) >> 1) & 1u))) {
                    // S(i+1) is already complete: request it now, so that its trip from tensor
                    // memory overlaps the hand-over of P(i)
                    tc_fence_after_sync();
                    PAFU_TMEM_LD_X32(tSslot + (buf ^ 1) * kBN, sr);
                    PAFU_TMEM_LD_X32(tSslot + (buf ^ 1) * kBN + 32, sr + 32);
                    loaded = true;
                }
                tmem_wait_st();
                tc_fence_before_sync();
                __syncwarp();
                if ((tid & 31) == 0) mbar_arrive(p_full(slot, buf));
            }
            if (!ok) break;
            tc += (uint32_t)n;
            if (n >= 2) ++pvcnt;
            {
                const bool w = mbar_wait(o_done(slot), ocnt & 1u) && !abort_flag;
                if (!__all_sync(0xffffffffu, w)) { fail(302); ok = false; break; }
                ++ocnt;
            }
            tc_fence_after_sync();
            const int64_t row = g.q0 + slot * kBM + row_in_slot;
            if (g.piece < 0) {
                // whole item: normalise and store bf16
                const float inv = (l_sum > 0.f) ? 1.0f / l_sum : 0.f;
                uint16_t* dst = p.O + ((p.st.cu_Lq[g.stream] + row) * p.n_heads + g.head) * kD;
#pragma unroll
                for (int c = 0; c < kD / 32; ++c) {
                    uint32_t orr[32];
                    PAFU_TMEM_LD_X32(tO + c * 32, orr);
                    tmem_wait_ld();
                    if (row < g.Lq) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            uint4 v;
                            v.x = pack_bf16(__uint_as_float(orr[8 * q + 0]) * inv, __uint_as_float(orr[8 * q + 1]) * inv);
                            v.y = pack_bf16(__uint_as_float(orr[8 * q + 2]) * inv, __uint_as_float(orr[8 * q + 3]) * inv);
                            v.z = pack_bf16(__uint_as_float(orr[8 * q + 4]) * inv, __uint_as_float(orr[8 * q + 5]) * inv);
                            v.w = pack_bf16(__uint_as_float(orr[8 * q + 6]) * inv, __uint_as_float(orr[8 * q + 7]) * inv);
                            *reinterpret_cast<uint4*>(dst + c * 32 + q * 8) = v;
                        }
                    }
                }
                if (p.LSE != nullptr && row < g.Lq)
                    p.LSE[(int64_t)g.head * p.total_Lq + p.st.cu_Lq[g.stream] + row] =
                        (l_sum > 0.f) ? m_used * p.scale + logf(l_sum) : -INFINITY;
            } else {
                // part of an item: unnormalised fp32 partial for the merge kernel
                float* piece = p.pieces + ((size_t)blockIdx.x * 2 + g.piece) * kPieceFloats;
                const int prow = slot * kBM + row_in_slot;
                float4* dst = reinterpret_cast<float4*>(piece + (size_t)prow * kD);
#pragma unroll
                for (int c = 0; c < kD / 32; ++c) {
                    uint32_t orr[32];
                    PAFU_TMEM_LD_X32(tO + c * 32, orr);
                    tmem_wait_ld();
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        dst[c * 8 + q] = make_float4(__uint_as_float(orr[4 * q]), __uint_as_float(orr[4 * q + 1]),
                                                     __uint_as_float(orr[4 * q + 2]), __uint_as_float(orr[4 * q + 3]));
                }
                piece[2 * kBM * kD + prow] = m_used;
                piece[2 * kBM * kD + 2 * kBM + prow] = l_sum;
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem, 512);
}

// Merges the partials of every item that was split across CTAs.  The host walks the CTAs'
// shares once per launch and passes the work as a table: item i was begun by CTA cta[first]
// (its last run, stored as that CTA's piece 1) and continued by the following entries (each
// CTA's first run, piece 0), in key order, which keeps the result deterministic.  Eight blocks
// of 256 threads per item (two slots x four groups of 32 rows); a warp handles four rows, so
// all loads of a block are in flight together.
constexpr int kMergeRows = 4;
constexpr int kMergeThreads = 256;
constexpr int kMergeBlocksPerItem = 2 * (kBM / (kMergeThreads / 32 * kMergeRows));   // 8
struct MergeItem {
    int32_t o_row;        // row of O (and LSE column) of the item's first query
    int32_t rows;         // valid query rows of the item (<= 256)
    int16_t head, n_slots;
    int16_t first, n_pieces;   // entries [first, first + n_pieces) of MergeTable::cta
};
struct MergeTable {
    int32_t n_items;
    MergeItem item[kMaxGrid];
    int16_t cta[2 * kMaxGrid];
};

template <int D>
__global__ void __launch_bounds__(kMergeThreads)
attn_tc_merge_kernel(const __grid_constant__ MergeTable tb, const float* __restrict__ pieces, float scale,
                     int n_heads, int64_t total_Lq, uint16_t* __restrict__ O, float* __restrict__ LSE) {
    constexpr int kD = D;
    constexpr int kPieceFloats = HeadDims<D>::kPieceFloats;
    grid_dep_wait();
    const MergeItem& it = tb.item[blockIdx.x / kMergeBlocksPerItem];
    const int slot = (blockIdx.x / (kMergeBlocksPerItem / 2)) & 1;
    const int group = blockIdx.x % (kMergeBlocksPerItem / 2);
    if (slot >= it.n_slots) return;                                    // block-uniform
    const int n_pieces = it.n_pieces;
    const float sl2 = scale * 1.4426950408889634f;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;        // 32 float4 per row
    const int r0 = group * (kMergeThreads / 32 * kMergeRows) + warp * kMergeRows;
    float M[kMergeRows], L[kMergeRows];
    float4 acc[kMergeRows];
#pragma unroll
    for (int q = 0; q < kMergeRows; ++q) { M[q] = -INFINITY; L[q] = 0.f; acc[q] = make_float4(0.f, 0.f, 0.f, 0.f); }
    for (int i = 0; i < n_pieces; ++i) {
        const float* piece = pieces + ((size_t)tb.cta[it.first + i] * 2 + (i == 0 ? 1 : 0)) * kPieceFloats;
#pragma unroll
        for (int q = 0; q < kMergeRows; ++q) M[q] = fmaxf(M[q], piece[2 * kBM * kD + slot * kBM + r0 + q]);
    }
    for (int i = 0; i < n_pieces; ++i) {
        const float* piece = pieces + ((size_t)tb.cta[it.first + i] * 2 + (i == 0 ? 1 : 0)) * kPieceFloats;
        float w[kMergeRows], l[kMergeRows];
        float4 v[kMergeRows];
#pragma unroll
        for (int q = 0; q < kMergeRows; ++q) {
            const int r = slot * kBM + r0 + q;
            w[q] = piece[2 * kBM * kD + r];
            l[q] = piece[2 * kBM * kD + 2 * kBM + r];
            v[q] = lane < kD / 4 ? reinterpret_cast<const float4*>(piece + (size_t)r * kD)[lane] : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int q = 0; q < kMergeRows; ++q) {
            const float ww = fast_exp2((w[q] - M[q]) * sl2);
            L[q] += ww * l[q];
            acc[q].x += ww * v[q].x; acc[q].y += ww * v[q].y; acc[q].z += ww * v[q].z; acc[q].w += ww * v[q].w;
        }
    }
#pragma unroll
    for (int q = 0; q < kMergeRows; ++q) {
        const int row = slot * kBM + r0 + q;
        if (row >= it.rows) continue;
        const float inv = (L[q] > 0.f) ? 1.0f / L[q] : 0.f;
        uint16_t* dst = O + (((int64_t)it.o_row + row) * n_heads + it.head) * kD + lane * 4;
        uint2 o;
        o.x = pack_bf16(acc[q].x * inv, acc[q].y * inv);
        o.y = pack_bf16(acc[q].z * inv, acc[q].w * inv);
        if (lane < kD / 4) *reinterpret_cast<uint2*>(dst) = o;
        if (LSE != nullptr && lane == 0)
            LSE[(int64_t)it.head * total_Lq + it.o_row + row] = (L[q] > 0.f) ? M[q] * scale + logf(L[q]) : -INFINITY;
    }
}

// Host side of the merge: which CTAs hold the pieces of which item.
inline void build_merge_table(const Params& p, int n_cta, MergeTable& tb) {
    tb.n_items = 0;
    int n_list = 0;
    Seg g, last;
    for (int b = 0; b < n_cta; ++b) {
        bool have = false;
        {
            SegIter iter(p, b, n_cta);
            while (iter.next(p, g)) { last = g; have = true; }
        }
        if (!have || last.piece != 1) continue;
        MergeItem& it = tb.item[tb.n_items++];
        it.o_row = (int32_t)(p.st.cu_Lq[last.stream] + last.q0);
        const int64_t left = last.Lq - last.q0;
        it.rows = (int32_t)(left < 2 * kBM ? left : 2 * kBM);
        it.head = (int16_t)last.head;
        it.n_slots = (int16_t)last.n_slots;
        it.first = (int16_t)n_list;
        tb.cta[n_list++] = (int16_t)b;
        int t = last.t1;
        for (int c = b + 1; c < n_cta && t < last.nt; ++c) {
            SegIter iter(p, c, n_cta);
            if (!iter.next(p, g)) continue;    // an empty share holds no piece
            t = g.t1;
            tb.cta[n_list++] = (int16_t)c;
        }
        it.n_pieces = (int16_t)(n_list - it.first);
    }
}

inline int sm_count() { return device_sm_count(); }

inline int grid_for(int64_t cost) {
    const int sms = sm_count();
    return (int)(cost < sms ? cost : sms);
}

// True when every stream with queries has at least one key (the cost line has no entry for a
// key-less item).
inline bool supports(const StreamTable& st, bool has_chunk) {
    for (int s = 0; s < st.n_streams; ++s) {
        const int64_t lq = st.cu_Lq[s + 1] - st.cu_Lq[s], nB = st.cu_B[s + 1] - st.cu_B[s];
        if (lq > 0 && nB == 0 && !has_chunk) return false;
    }
    return true;
}

// Scratch for the partials: one pair per CTA.
inline size_t workspace_bytes() { return (size_t)sm_count() * 2 * kPieceBytes; }

// Tensor maps are rebuilt per call (a few microseconds of host work); nothing is cached, so
// the library stays stateless.  D: head width (128; 64 with a compacted cache only).
template <int D>
inline pafu_status launch_d(const uint16_t* Q, const uint16_t* Kc, const uint16_t* Vc,
                            const uint16_t* Kq, const uint16_t* Vq, const StreamTable& st,
                            int32_t n_heads, float scale, uint16_t* O, float* LSE, int* status,
                            float* pieces, cudaStream_t stream, int max_ctas, const int32_t* idx) {
    constexpr int kSmem = HeadDims<D>::kSmemBytes;
    const int n = st.n_streams;
    const int64_t nQ = st.cu_Lq[n], nB = st.cu_B[n];
    const int has_chunk = Kq != nullptr;
    const int64_t cost = total_cost(st, n_heads, has_chunk);
    if (cost == 0) return PAFU_OK;
    CUtensorMap mQ, mKc, mVc, mKq, mVq;
    if (!TmapEncoder::token_tensor(&mQ, Q, (uint64_t)nQ, n_heads, D, kBM)) return PAFU_ERR_CUDA;
    const bool gather = idx != nullptr;      // Kc, Vc are then the uncompacted cache
    if (gather && D != 128) return PAFU_ERR_UNSUPPORTED_SHAPE;
    if (nB > 0 && gather) {
        mKc = mQ; mVc = mQ;                 // the gather loader reads the cache through plain pointers
    } else if (nB > 0) {
        if (!TmapEncoder::token_tensor(&mKc, Kc, (uint64_t)nB, n_heads, D, kBN) ||
            !TmapEncoder::token_tensor(&mVc, Vc, (uint64_t)nB, n_heads, D, kBN)) return PAFU_ERR_CUDA;
    } else { mKc = mQ; mVc = mQ; }
    if (has_chunk) {
        if (!TmapEncoder::token_tensor(&mKq, Kq, (uint64_t)nQ, n_heads, D, kBN) ||
            !TmapEncoder::token_tensor(&mVq, Vq, (uint64_t)nQ, n_heads, D, kBN)) return PAFU_ERR_CUDA;
    } else { mKq = mQ; mVq = mQ; }
    Params p;
    p.st = st; p.n_heads = n_heads; p.has_chunk = has_chunk; p.scale = scale;
    p.O = O; p.LSE = LSE; p.status = status; p.pieces = pieces; p.idx = idx; p.Kraw = gather ? Kc : nullptr; p.Vraw = gather ? Vc : nullptr; p.total_Lq = nQ; p.total_cost = cost;
    static bool attr_set[kMaxDevices] = {};
    if (!once_per_device(attr_set, [] {
            if (cudaFuncSetAttribute(attn_tc_kernel<false, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) != cudaSuccess) return false;
            if constexpr (D == 128)
                return cudaFuncSetAttribute(attn_tc_kernel<true, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) == cudaSuccess;
            return true;
        }))
        return PAFU_ERR_CUDA;
    int grid = grid_for(cost);
    if (max_ctas > 0 && grid > max_ctas) grid = max_ctas;   // caller's scratch holds fewer partials
    cudaError_t le;
    if constexpr (D == 128) {
        le = gather ? launch_dependent(attn_tc_kernel<true, 128>, dim3(grid), dim3(kThreads), kSmem, stream, 1, mQ, mKc, mVc, mKq, mVq, p)
                    : launch_dependent(attn_tc_kernel<false, 128>, dim3(grid), dim3(kThreads), kSmem, stream, 1, mQ, mKc, mVc, mKq, mVq, p);
    } else {
        le = launch_dependent(attn_tc_kernel<false, D>, dim3(grid), dim3(kThreads), kSmem, stream, 1, mQ, mKc, mVc, mKq, mVq, p);
    }
    if (le != cudaSuccess) return PAFU_ERR_CUDA;
    if (grid > 1) {
        MergeTable tb;
        build_merge_table(p, grid, tb);
        if (tb.n_items > 0 &&
            launch_dependent(attn_tc_merge_kernel<D>, dim3(tb.n_items * kMergeBlocksPerItem), dim3(kMergeThreads), 0, stream, 1,
                             tb, (const float*)pieces, scale, (int)n_heads, nQ, O, LSE) != cudaSuccess)
            return PAFU_ERR_CUDA;
    }
    return PAFU_OK;
}

inline pafu_status launch(const uint16_t* Q, const uint16_t* Kc, const uint16_t* Vc,
                          const uint16_t* Kq, const uint16_t* Vq, const StreamTable& st,
                          int32_t n_heads, float scale, uint16_t* O, float* LSE, int* status,
                          float* pieces, cudaStream_t stream, int max_ctas = 0,
                          const int32_t* idx = nullptr, int d_head = kD) {
    if (d_head == 64)
        return launch_d<64>(Q, Kc, Vc, Kq, Vq, st, n_heads, scale, O, LSE, status, pieces, stream, max_ctas, idx);
    return launch_d<128>(Q, Kc, Vc, Kq, Vq, st, n_heads, scale, O, LSE, status, pieces, stream, max_ctas, idx);
}

}  // namespace attn_tc
}  // namespace pafu
