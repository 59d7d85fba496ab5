// Chunk attention, register-resident variant (mma.sync m16n8k16, cp.async double buffering).
//
// o_i = sum_j softmax_j(scale q_i.k_j) v_j with j over [retained cache ; chunk tokens]
// (Sec. 3.2 for the operator; Eq. 2 / Eq. 7 for the key range).  One CTA of 4 warps owns 64
// query rows of one head and streams 64-key tiles of both key segments through shared memory
// with an online softmax.  It serves the inputs the tcgen05 kernel does not take: a stream that
// has queries but not a single key (no retained cache and no chunk segment), whose rows are zero.
#pragma once
#include "common.cuh"

namespace pafu {
namespace attn_mma {

constexpr int kBM = 64, kBN = 64, kThreads = 128;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;"); }
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
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

// Byte offset of 16-byte chunk `c` of row `r` in a [rows][D] bf16 tile (XOR swizzle).
template <int D>
__device__ __forceinline__ uint32_t tile_off(int r, int c) {
    return (uint32_t)(r * (D * 2) + ((c ^ (r & 7)) << 4));
}

// Copy rows [row0, row0 + 64) of a [n_rows, ld] bf16 matrix (D columns at col0) into a tile;
// rows past n_rows are zero filled.
template <int D>
__device__ __forceinline__ void load_tile(uint32_t tile, const uint16_t* base, int64_t ld,
                                          int64_t row0, int64_t n_rows, int tid) {
    constexpr int kChunks = D / 8;
#pragma unroll
    for (int i = 0; i < 64 * kChunks / kThreads; ++i) {
        const int e = tid + i * kThreads;
        const int r = e / kChunks, c = e % kChunks;
        const int64_t gr = row0 + r;
        const bool ok = gr < n_rows;
        const uint16_t* src = base + (ok ? gr : 0) * ld + c * 8;
        cp_async16(tile + tile_off<D>(r, c), src, ok ? 16 : 0);
    }
}

template <int D>
__global__ void __launch_bounds__(kThreads)
attn_mma_kernel(const uint16_t* __restrict__ Q, const uint16_t* __restrict__ Kc,
                const uint16_t* __restrict__ Vc, const uint16_t* __restrict__ Kq,
                const uint16_t* __restrict__ Vq, StreamTable st, int n_heads, float scale,
                uint16_t* __restrict__ O, float* __restrict__ LSE) {
    grid_dep_wait();
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int kTileBytes = 64 * D * 2;
    const uint32_t sQ = smem_u32(smem);
    const uint32_t sK = sQ + kTileBytes;          // 2 stages
    const uint32_t sV = sK + 2 * kTileBytes;      // 2 stages

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t4 = lane & 3;
    const int head = blockIdx.y;
    const int64_t ld = (int64_t)n_heads * D;

    // which stream / query tile
    int s = 0;
    int64_t tile = blockIdx.x;
    for (;; ++s) {
        const int64_t nt = (st.cu_Lq[s + 1] - st.cu_Lq[s] + kBM - 1) / kBM;
        if (tile < nt) break;
        tile -= nt;
    }
    const int64_t Lq = st.cu_Lq[s + 1] - st.cu_Lq[s];
    const int64_t q0 = tile * kBM;
    const int64_t nB = st.cu_B[s + 1] - st.cu_B[s];
    const int64_t nC = (Kq != nullptr) ? Lq : 0;
    const uint16_t* Qs = Q + st.cu_Lq[s] * ld + head * D;
    const uint16_t* K1 = Kc + st.cu_B[s] * ld + head * D;
    const uint16_t* V1 = Vc + st.cu_B[s] * ld + head * D;
    const uint16_t* K2 = (Kq != nullptr) ? Kq + st.cu_Lq[s] * ld + head * D : nullptr;
    const uint16_t* V2 = (Vq != nullptr) ? Vq + st.cu_Lq[s] * ld + head * D : nullptr;
    const int nt1 = (int)((nB + kBN - 1) / kBN), nt2 = (int)((nC + kBN - 1) / kBN);
    const int ntiles = nt1 + nt2;

    auto issue_kv = [&](int j) {
        const bool seg2 = j >= nt1;
        const int64_t row0 = (int64_t)(seg2 ? j - nt1 : j) * kBN;
        const uint32_t off = (uint32_t)(j & 1) * kTileBytes;
        load_tile<D>(sK + off, seg2 ? K2 : K1, ld, row0, seg2 ? nC : nB, tid);
        load_tile<D>(sV + off, seg2 ? V2 : V1, ld, row0, seg2 ? nC : nB, tid);
    };

    load_tile<D>(sQ, Qs, ld, q0, Lq, tid);
    if (ntiles > 0) issue_kv(0);
    cp_async_commit();

    const float sl2 = scale * 1.4426950408889634f;
    float o[D / 8][4];
#pragma unroll
    for (int i = 0; i < D / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    uint32_t qf[D / 16][4];

    for (int j = 0; j < ntiles; ++j) {
        cp_async_wait_all();
        __syncthreads();
        if (j + 1 < ntiles) issue_kv(j + 1);
        cp_async_commit();
        if (j == 0) {
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const int r = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                const int c = kk * 2 + (lane >> 4);
                ldsm_x4(sQ + tile_off<D>(r, c), qf[kk]);
            }
        }
        const uint32_t kb = sK + (uint32_t)(j & 1) * kTileBytes;
        const uint32_t vb = sV + (uint32_t)(j & 1) * kTileBytes;

        float sacc[8][4];
#pragma unroll
        for (int i = 0; i < 8; ++i) { sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f; }
#pragma unroll
        for (int np = 0; np < 4; ++np) {
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                uint32_t b[4];
                const int r = np * 16 + (lane & 7) + (lane >> 4) * 8;
                const int c = kk * 2 + ((lane >> 3) & 1);
                ldsm_x4(kb + tile_off<D>(r, c), b);
                mma_bf16(sacc[2 * np], qf[kk], b[0], b[1]);
                mma_bf16(sacc[2 * np + 1], qf[kk], b[2], b[3]);
            }
        }
        // mask the ragged end of a segment
        const bool seg2 = j >= nt1;
        const int64_t seg_len = seg2 ? nC : nB;
        const int64_t key0 = (int64_t)(seg2 ? j - nt1 : j) * kBN;
        if (key0 + kBN > seg_len) {
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (key0 + nt * 8 + 2 * t4 + (e & 1) >= seg_len) sacc[nt][e] = -INFINITY;
        }
        // online softmax; rows g (e = 0,1) and g + 8 (e = 2,3)
        float alpha[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            float mx = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) mx = fmaxf(mx, fmaxf(sacc[nt][2 * r], sacc[nt][2 * r + 1]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_run[r], mx);
            alpha[r] = fast_exp2((m_run[r] - m_new) * sl2);
            m_run[r] = m_new;
            const float mb = m_new * sl2;
            float rs = 0.f;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                sacc[nt][2 * r] = fast_exp2(sacc[nt][2 * r] * sl2 - mb);
                sacc[nt][2 * r + 1] = fast_exp2(sacc[nt][2 * r + 1] * sl2 - mb);
                rs += sacc[nt][2 * r] + sacc[nt][2 * r + 1];
            }
            l_run[r] = l_run[r] * alpha[r] + rs;
        }
#pragma unroll
        for (int i = 0; i < D / 8; ++i) {
            o[i][0] *= alpha[0]; o[i][1] *= alpha[0]; o[i][2] *= alpha[1]; o[i][3] *= alpha[1];
        }
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            uint32_t pa[4];
            pa[0] = pack_bf16(sacc[2 * kk][0], sacc[2 * kk][1]);
            pa[1] = pack_bf16(sacc[2 * kk][2], sacc[2 * kk][3]);
            pa[2] = pack_bf16(sacc[2 * kk + 1][0], sacc[2 * kk + 1][1]);
            pa[3] = pack_bf16(sacc[2 * kk + 1][2], sacc[2 * kk + 1][3]);
#pragma unroll
            for (int dp = 0; dp < D / 16; ++dp) {
                uint32_t b[4];
                const int r = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                const int c = dp * 2 + (lane >> 4);
                ldsm_x4_t(vb + tile_off<D>(r, c), b);
                mma_bf16(o[2 * dp], pa, b[0], b[1]);
                mma_bf16(o[2 * dp + 1], pa, b[2], b[3]);
            }
        }
    }
    cp_async_wait_all();

    // finalise: o / l, bf16 store; LSE = m * scale + ln l
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        float l = l_run[r];
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        const int64_t row = q0 + warp * 16 + g + r * 8;
        if (row < Lq) {
            const float inv = (l > 0.f) ? 1.0f / l : 0.f;
            uint16_t* dst = O + (st.cu_Lq[s] + row) * ld + head * D;
#pragma unroll
            for (int nt = 0; nt < D / 8; ++nt) {
                const uint32_t v = pack_bf16(o[nt][2 * r] * inv, o[nt][2 * r + 1] * inv);
                *reinterpret_cast<uint32_t*>(dst + nt * 8 + 2 * t4) = v;
            }
            if (LSE != nullptr && t4 == 0) {
                const int64_t total = st.cu_Lq[st.n_streams];
                LSE[(int64_t)head * total + st.cu_Lq[s] + row] =
                    (l > 0.f) ? m_run[r] * scale + logf(l) : -INFINITY;
            }
        }
    }
}

inline pafu_status launch(const uint16_t* Q, const uint16_t* Kc, const uint16_t* Vc,
                          const uint16_t* Kq, const uint16_t* Vq, const StreamTable& st,
                          int32_t n_heads, int32_t d_head, float scale, uint16_t* O, float* LSE,
                          cudaStream_t stream) {
    int64_t tiles = 0;
    for (int s = 0; s < st.n_streams; ++s) tiles += (st.cu_Lq[s + 1] - st.cu_Lq[s] + kBM - 1) / kBM;
    if (tiles == 0) return PAFU_OK;
    dim3 grid((unsigned)tiles, (unsigned)n_heads);
    cudaError_t e;
    if (d_head == 128) {
        constexpr int smem = 5 * 64 * 128 * 2;
        e = cudaFuncSetAttribute(attn_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return PAFU_ERR_CUDA;
        launch_dependent(attn_mma_kernel<128>, dim3(grid), dim3(kThreads), smem, stream, 1, Q, Kc, Vc, Kq, Vq, st, n_heads, scale, O, LSE);
    } else {
        constexpr int smem = 5 * 64 * 64 * 2;
        e = cudaFuncSetAttribute(attn_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return PAFU_ERR_CUDA;
        launch_dependent(attn_mma_kernel<64>, dim3(grid), dim3(kThreads), smem, stream, 1, Q, Kc, Vc, Kq, Vq, st, n_heads, scale, O, LSE);
    }
    return cuda_ok(cudaGetLastError());
}

}  // namespace attn_mma
}  // namespace pafu
