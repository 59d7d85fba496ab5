// Chunk attention on the 5th-generation tensor cores (tcgen05 + TMEM + TMA), d_head = 128.
//
//   o_i = sum_j softmax_j(scale q_i.k_j) v_j,  j over [retained cache ; chunk tokens]
//   (Sec. 3.2 for the operator; Eq. 2 / Eq. 7 for the key range)
//
// One CTA works on 256 query rows of one head as two 128-row "slots" that share every K/V
// tile, so each tile is fetched once per 256 rows.  Warp roles:
//   warps 0-3  softmax of slot 0 (thread = query row = TMEM lane)
//   warps 4-7  softmax of slot 1
//   warp  8    MMA issuer: S = Q K^T (both operands in shared memory) and O += P V
//              (P read from tensor memory, V from shared memory, MN-major)
//   warp  9    TMA loader: Q tiles once, then K/V tiles through a 5-stage ring
//   warps 10-11 idle (they complete the third warpgroup so registers can be re-balanced)
// Tensor memory (512 columns): S0 | S1 | O0 | O1, 128 fp32 columns each; the bf16 P tile
// overwrites the first 64 columns of its S tile.  While one slot runs its softmax the tensor
// core works on the other slot's two products.
//
// Online softmax with lazy rescaling: the running maximum only moves when the new tile
// exceeds it by more than 2^8 in the exponent, so the O accumulator is rarely rescaled; when
// it is, the slot's own softmax warps do it between "S ready" (which implies the previous
// P V product has finished) and "P ready" (which releases the next one).
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
constexpr int kBN = 128;            // keys per tile
constexpr int kStages = 5;          // K/V ring depth (each stage one 128 x 128 bf16 tile)
constexpr int kThreads = 384;           // 3 warpgroups: softmax 0, softmax 1, {MMA, loader, 2 idle}
constexpr int kTileBytes = kBN * kD * 2;      // 32 KiB
constexpr int kHalfBytes = kTileBytes / 2;    // one [128 rows x 64 cols] swizzled half
constexpr int kSmemBytes = 2 * kTileBytes + kStages * kTileBytes + 1024 /*align*/ + 256 /*barriers*/;
constexpr float kRescaleThresholdLog2 = 8.0f;

struct Params {
    StreamTable st;
    int n_heads;
    int has_chunk;
    float scale;
    uint16_t* O;
    float* LSE;
    int* status;        // workspace status word (device)
    int64_t total_Lq;
};

struct Item {            // one CTA's work: 256 query rows of one head of one stream
    int stream, head;
    int64_t q0;          // first query row (stream-local)
    int64_t Lq, nB, nC;  // stream's query rows, retained keys, chunk keys
    int nt1, nt2;        // key tiles in each segment
};

__device__ __forceinline__ Item decode_item(const Params& p, int64_t item) {
    Item it;
    int s = 0;
    for (;; ++s) {
        const int64_t lq = p.st.cu_Lq[s + 1] - p.st.cu_Lq[s];
        const int64_t n = ((lq + 2 * kBM - 1) / (2 * kBM)) * p.n_heads;
        if (item < n) break;
        item -= n;
    }
    it.stream = s;
    it.Lq = p.st.cu_Lq[s + 1] - p.st.cu_Lq[s];
    const int64_t nqp = (it.Lq + 2 * kBM - 1) / (2 * kBM);
    it.head = (int)(item / nqp);
    it.q0 = (item % nqp) * (2 * kBM);
    it.nB = p.st.cu_B[s + 1] - p.st.cu_B[s];
    it.nC = p.has_chunk ? it.Lq : 0;
    it.nt1 = (int)((it.nB + kBN - 1) / kBN);
    it.nt2 = (int)((it.nC + kBN - 1) / kBN);
    return it;
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap mQ, const __grid_constant__ CUtensorMap mKc,
               const __grid_constant__ CUtensorMap mVc, const __grid_constant__ CUtensorMap mKq,
               const __grid_constant__ CUtensorMap mVq, const __grid_constant__ Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sQ = smem_u32(smem);                       // 2 slots x 32 KiB
    const uint32_t sKV = sQ + 2 * kTileBytes;                 // ring
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 2 * kTileBytes + kStages * kTileBytes);
    // barrier map
    const uint32_t bar0 = smem_u32(bars);
    auto q_full = [&](int s) { return bar0 + 8 * (0 + s); };
    auto s_full = [&](int s) { return bar0 + 8 * (2 + s); };
    auto p_full = [&](int s) { return bar0 + 8 * (4 + s); };
    auto o_done = [&](int s) { return bar0 + 8 * (6 + s); };
    auto kv_full = [&](int st) { return bar0 + 8 * (8 + st); };
    auto kv_empty = [&](int st) { return bar0 + 8 * (8 + kStages + st); };
    __shared__ uint32_t tmem_base_sh;
    __shared__ volatile int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5;
    const Item it = decode_item(p, blockIdx.x);
    const int ntiles = it.nt1 + it.nt2;
    const int n_slots = (it.q0 + kBM < it.Lq) ? 2 : 1;

    if (tid == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(q_full(s), 1); mbar_init(s_full(s), 1); mbar_init(p_full(s), kBM); mbar_init(o_done(s), 1);
        }
        for (int st = 0; st < kStages; ++st) { mbar_init(kv_full(st), 1); mbar_init(kv_empty(st), 1); }
        abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 8) { tmem_alloc(smem_u32(&tmem_base_sh), 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_sh;

    auto fail = [&](int code) {
        abort_flag = 1;
        atomicCAS(p.status, 0, code);
    };

    if (warp >= 8) {
    // register budget: this warpgroup gives registers up, the softmax warpgroups (which hold a
    // whole S row per thread) take them
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
    if (warp == 9) {
        // ------------------------------------------------------------------ TMA loader
        if (elect_one()) {
            prefetch_tmap(&mQ); prefetch_tmap(&mKc); prefetch_tmap(&mVc);
            if (p.has_chunk) { prefetch_tmap(&mKq); prefetch_tmap(&mVq); }
            const int qrow = (int)(p.st.cu_Lq[it.stream] + it.q0);
            for (int s = 0; s < n_slots; ++s) {
                mbar_arrive_expect_tx(q_full(s), kTileBytes);
                tma_load_3d(sQ + s * kTileBytes, &mQ, q_full(s), 0, it.head, qrow + s * kBM);
                tma_load_3d(sQ + s * kTileBytes + kHalfBytes, &mQ, q_full(s), 64, it.head, qrow + s * kBM);
            }
            int ring = 0;
            bool ok = true;
            for (int j = 0; j < ntiles && ok; ++j) {
                const bool seg2 = j >= it.nt1;
                const int row = seg2 ? (int)(p.st.cu_Lq[it.stream] + (int64_t)(j - it.nt1) * kBN)
                                     : (int)(p.st.cu_B[it.stream] + (int64_t)j * kBN);
                for (int kv = 0; kv < 2 && ok; ++kv, ++ring) {
                    const int st = ring % kStages;
                    const uint32_t ph = (uint32_t)(ring / kStages) & 1u;
                    if (abort_flag || !mbar_wait(kv_empty(st), ph ^ 1u)) { fail(101); ok = false; break; }
                    const CUtensorMap* m = seg2 ? (kv ? &mVq : &mKq) : (kv ? &mVc : &mKc);
                    mbar_arrive_expect_tx(kv_full(st), kTileBytes);
                    tma_load_3d(sKV + st * kTileBytes, m, kv_full(st), 0, it.head, row);
                    tma_load_3d(sKV + st * kTileBytes + kHalfBytes, m, kv_full(st), 64, it.head, row);
                }
            }
            if (!ok) {
                // let copies already in flight land before the CTA exits
                for (int r = max(0, ring - kStages); r < ring; ++r)
                    mbar_wait(kv_full(r % kStages), (uint32_t)(r / kStages) & 1u);
            }
        }
        __syncwarp();
    } else if (warp == 8) {
        // ------------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            const uint32_t idesc_qk = make_idesc_bf16(kBM, kBN, false, false);
            const uint32_t idesc_pv = make_idesc_bf16(kBM, kD, false, true);
            auto issue_qk = [&](int slot, int stage) {
                const uint32_t a = sQ + slot * kTileBytes, b = sKV + stage * kTileBytes;
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk) {
                    const uint32_t off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
                    umma_ss(tmem + slot * kBN, make_smem_desc_sw128(a + off, 16, 1024),
                            make_smem_desc_sw128(b + off, 16, 1024), idesc_qk, kk > 0);
                }
            };
            auto issue_pv = [&](int slot, int stage, bool first) {
                const uint32_t b = sKV + stage * kTileBytes;
#pragma unroll
                for (int kk = 0; kk < kBN / 16; ++kk)
                    umma_ts(tmem + 256 + slot * kD, tmem + slot * kBN + kk * 8,
                            make_smem_desc_sw128(b + kk * 2048, kHalfBytes, 1024), idesc_pv,
                            !(first && kk == 0));
            };
            bool ok = true;
            auto wait = [&](uint32_t bar, uint32_t ph, int code) {
                if (!ok) return;
                if (abort_flag || !mbar_wait(bar, ph)) { fail(code); ok = false; }
            };
            for (int s = 0; s < n_slots; ++s) wait(q_full(s), 0, 201);
            if (ntiles > 0) {
                wait(kv_full(0), 0, 202);
                if (ok) {
                    tc_fence_after_sync();
                    for (int s = 0; s < n_slots; ++s) { issue_qk(s, 0); umma_commit(s_full(s)); }
                    umma_commit(kv_empty(0));
                }
            }
            for (int j = 0; j < ntiles && ok; ++j) {
                const int rv = 2 * j + 1, rk = 2 * j + 2;          // ring slots of V_j and K_{j+1}
                const int stv = rv % kStages, stk = rk % kStages;
                wait(kv_full(stv), (uint32_t)(rv / kStages) & 1u, 203);
                const bool more = j + 1 < ntiles;
                if (more) wait(kv_full(stk), (uint32_t)(rk / kStages) & 1u, 204);
                for (int s = 0; s < n_slots && ok; ++s) {
                    wait(p_full(s), (uint32_t)j & 1u, 205);
                    if (!ok) break;
                    tc_fence_after_sync();
                    issue_pv(s, stv, j == 0);
                    if (more) { issue_qk(s, stk); umma_commit(s_full(s)); }
                    else umma_commit(o_done(s));
                }
                if (ok) {
                    umma_commit(kv_empty(stv));
                    if (more) umma_commit(kv_empty(stk));
                }
            }
        }
        __syncwarp();
    }
    } else {
        // ------------------------------------------------------------------ softmax warps
        asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
        const int slot = warp >> 2;
        const int row_in_slot = tid & 127;
        const uint32_t lane_base = ((uint32_t)((warp & 3) * 32)) << 16;
        const uint32_t tS = tmem + slot * kBN + lane_base;
        const uint32_t tO = tmem + 256 + slot * kD + lane_base;
        const float sl2 = p.scale * 1.4426950408889634f;
        float m_used = -INFINITY, l_sum = 0.f;
        bool ok = slot < n_slots;
        if (ok) {
            for (int j = 0; j < ntiles; ++j) {
                {
                    const bool w = mbar_wait(s_full(slot), (uint32_t)j & 1u) && !abort_flag;
                    if (!__all_sync(0xffffffffu, w)) { fail(301); ok = false; break; }   // warp-uniform
                }
                tc_fence_after_sync();
                uint32_t sr[128];
                PAFU_TMEM_LD_X32(tS, sr);
                PAFU_TMEM_LD_X32(tS + 32, sr + 32);
                PAFU_TMEM_LD_X32(tS + 64, sr + 64);
                PAFU_TMEM_LD_X32(tS + 96, sr + 96);
                tmem_wait_ld();
                // ragged end of a key segment
                const bool seg2 = j >= it.nt1;
                const int64_t left = (seg2 ? it.nC - (int64_t)(j - it.nt1) * kBN : it.nB - (int64_t)j * kBN);
                if (left < kBN) {
#pragma unroll
                    for (int c = 0; c < 128; ++c)
                        if (c >= left) sr[c] = 0xff800000u;   // -inf
                }
                float mx = __uint_as_float(sr[0]);
#pragma unroll
                for (int c = 1; c < 128; ++c) mx = fmaxf(mx, __uint_as_float(sr[c]));
                if (j == 0) {
                    m_used = mx;
                } else if (__any_sync(0xffffffffu, (mx - m_used) * sl2 > kRescaleThresholdLog2)) {
                    // the whole warp rescales together (TMEM accesses are warp-collective);
                    // rows whose maximum did not move get alpha = 1
                    const float m_new = fmaxf(m_used, mx);
                    const float alpha = fast_exp2((m_used - m_new) * sl2);
                    l_sum *= alpha;
                    m_used = m_new;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t orr[32];
                        PAFU_TMEM_LD_X32(tO + c * 32, orr);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * alpha);
                        PAFU_TMEM_ST_X32(tO + c * 32, orr);
                    }
                }
                const float mb = m_used * sl2;
                float rs = 0.f;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t pk[32];
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        const float p0 = fast_exp2(fmaf(__uint_as_float(sr[64 * h + 2 * c]), sl2, -mb));
                        const float p1 = fast_exp2(fmaf(__uint_as_float(sr[64 * h + 2 * c + 1]), sl2, -mb));
                        rs += p0 + p1;
                        pk[c] = pack_bf16(p0, p1);
                    }
                    PAFU_TMEM_ST_X32(tS + 32 * h, pk);
                }
                l_sum += rs;
                tmem_wait_st();
                tc_fence_before_sync();
                mbar_arrive(p_full(slot));
            }
        }
        if (ok) {
            const int64_t row = it.q0 + slot * kBM + row_in_slot;
            if (ntiles > 0) {
                const bool w = mbar_wait(o_done(slot), 0) && !abort_flag;
                if (!__all_sync(0xffffffffu, w)) { fail(302); ok = false; }
                tc_fence_after_sync();
            }
            if (ok) {
                const float inv = (l_sum > 0.f) ? 1.0f / l_sum : 0.f;
                uint16_t* dst = p.O + ((p.st.cu_Lq[it.stream] + row) * p.n_heads + it.head) * kD;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t orr[32];
                    if (ntiles > 0) {
                        PAFU_TMEM_LD_X32(tO + c * 32, orr);
                        tmem_wait_ld();
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) orr[i] = 0u;
                    }
                    if (row < it.Lq) {
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
                if (p.LSE != nullptr && row < it.Lq)
                    p.LSE[(int64_t)it.head * p.total_Lq + p.st.cu_Lq[it.stream] + row] =
                        (l_sum > 0.f) ? m_used * p.scale + logf(l_sum) : -INFINITY;
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem, 512);
}

// Tensor maps are rebuilt per call (a few microseconds of host work); nothing is cached, so
// the library stays stateless.
inline pafu_status launch(const uint16_t* Q, const uint16_t* Kc, const uint16_t* Vc,
                          const uint16_t* Kq, const uint16_t* Vq, const StreamTable& st,
                          int32_t n_heads, float scale, uint16_t* O, float* LSE, int* status,
                          cudaStream_t stream) {
    const int n = st.n_streams;
    const int64_t nQ = st.cu_Lq[n], nB = st.cu_B[n];
    int64_t items = 0;
    for (int s = 0; s < n; ++s) items += ((st.cu_Lq[s + 1] - st.cu_Lq[s] + 2 * kBM - 1) / (2 * kBM)) * n_heads;
    if (items == 0) return PAFU_OK;
    CUtensorMap mQ, mKc, mVc, mKq, mVq;
    if (!TmapEncoder::token_tensor(&mQ, Q, (uint64_t)nQ, n_heads, kD, kBM)) return PAFU_ERR_CUDA;
    if (nB > 0) {
        if (!TmapEncoder::token_tensor(&mKc, Kc, (uint64_t)nB, n_heads, kD, kBN) ||
            !TmapEncoder::token_tensor(&mVc, Vc, (uint64_t)nB, n_heads, kD, kBN)) return PAFU_ERR_CUDA;
    } else { mKc = mQ; mVc = mQ; }
    if (Kq != nullptr) {
        if (!TmapEncoder::token_tensor(&mKq, Kq, (uint64_t)nQ, n_heads, kD, kBN) ||
            !TmapEncoder::token_tensor(&mVq, Vq, (uint64_t)nQ, n_heads, kD, kBN)) return PAFU_ERR_CUDA;
    } else { mKq = mQ; mVq = mQ; }
    Params p;
    p.st = st; p.n_heads = n_heads; p.has_chunk = Kq != nullptr; p.scale = scale;
    p.O = O; p.LSE = LSE; p.status = status; p.total_Lq = nQ;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
            return PAFU_ERR_CUDA;
        attr_set = true;
    }
    attn_tc_kernel<<<(unsigned)items, kThreads, kSmemBytes, stream>>>(mQ, mKc, mVc, mKq, mVq, p);
    return cuda_ok(cudaGetLastError());
}

}  // namespace attn_tc
}  // namespace pafu
