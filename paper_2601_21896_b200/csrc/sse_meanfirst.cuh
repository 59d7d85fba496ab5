// The teacher-side salience target in Algorithm 3's order of operations: the attention weights
// are averaged over the heads first and the maximum over a block class's queries is taken of
// that average (Eq. 4 as printed takes the per-head maximum first, then the mean; pafu_sse
// follows Eq. 4):
//   a[i,j] = (1/N) sum_n P[n,i,j],  low_j / diag_j / up_j = max of a[i,j] over the queries i of
//   later / the same / earlier blocks than key j's (an empty set gives 0), then Eq. 5.
// The average needs every head's probability of an element at the same place, so the heads are
// the innermost loop and one exponential per (query, key, head) is unavoidable; the per-head
// kernel's trick of taking the maximum in the log domain does not apply.  This variant exists for
// the comparison between the two readings, not for speed: register-resident mma.sync tiles.
// One CTA (4 warps) owns 64 keys and walks all 64-query tiles; per tile and head it forms
// S = Q_n K_n^T (a warp owns 16 query rows), turns it into probabilities with the row's
// log-sum-exp, and adds them up over the heads in registers.  A thread owns 16 key columns and
// keeps three running maxima per column; nothing is exchanged between CTAs and no atomics are
// used, so the result is deterministic.
#pragma once
#include "attn_mma.cuh"
#include "common.cuh"

namespace pafu {
namespace sse_mf {

using namespace attn_mma;     // tile loads, ldmatrix and mma.sync wrappers

constexpr int kD = 128, kT = 64;
constexpr int kTileBytes = kT * kD * 2;
constexpr int kSmemBytes = 4 * kTileBytes + 4 * 3 * kT * 4;

__global__ void __launch_bounds__(kThreads)
sse_meanfirst_kernel(const uint16_t* __restrict__ Q, const uint16_t* __restrict__ K, const float* __restrict__ lse,
                     int64_t L, int64_t LB, int n_heads, float scale, float* __restrict__ s_out,
                     float* __restrict__ comp) {
    grid_dep_wait();
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t sQ = smem_u32(smem);                  // 2 stages
    const uint32_t sK = sQ + 2 * kTileBytes;             // 2 stages
    float* red = reinterpret_cast<float*>(smem + 4 * kTileBytes);     // [4 warps][3 classes][64 keys]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t4 = lane & 3;
    const int64_t j0 = (int64_t)blockIdx.x * kT;
    const int64_t ld = (int64_t)n_heads * kD;
    const int n_qt = (int)((L + kT - 1) / kT);
    const int64_t n_it = (int64_t)n_qt * n_heads;
    const float sl2 = scale * 1.4426950408889634f;
    const float inv_n = 1.0f / (float)n_heads;

    auto issue = [&](int64_t it) {
        const int qt = (int)(it / n_heads), n = (int)(it % n_heads);
        const uint32_t off = (uint32_t)(it & 1) * kTileBytes;
        load_tile<kD>(sQ + off, Q + n * kD, ld, (int64_t)qt * kT, L, tid);
        load_tile<kD>(sK + off, K + n * kD, ld, j0, L, tid);
    };

    // block of each of this thread's 16 key columns; running maxima per class and column
    int64_t bk[16];
    float m_low[16], m_diag[16], m_up[16];
#pragma unroll
    for (int c = 0; c < 16; ++c) {
        bk[c] = (j0 + (c >> 1) * 8 + 2 * t4 + (c & 1)) / LB;
        m_low[c] = m_diag[c] = m_up[c] = 0.f;
    }

    issue(0);
    cp_async_commit();
    for (int qt = 0; qt < n_qt; ++qt) {
        float a[8][4];
#pragma unroll
        for (int i = 0; i < 8; ++i) { a[i][0] = a[i][1] = a[i][2] = a[i][3] = 0.f; }
        const int64_t row[2] = {(int64_t)qt * kT + warp * 16 + g, (int64_t)qt * kT + warp * 16 + g + 8};
        for (int n = 0; n < n_heads; ++n) {
            const int64_t it = (int64_t)qt * n_heads + n;
            cp_async_wait_all();
            __syncthreads();
            if (it + 1 < n_it) issue(it + 1);
            cp_async_commit();
            const uint32_t qb = sQ + (uint32_t)(it & 1) * kTileBytes, kb = sK + (uint32_t)(it & 1) * kTileBytes;
            uint32_t qf[kD / 16][4];
#pragma unroll
            for (int kk = 0; kk < kD / 16; ++kk) {
                const int r = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                const int c = kk * 2 + (lane >> 4);
                ldsm_x4(qb + tile_off<kD>(r, c), qf[kk]);
            }
            float sacc[8][4];
#pragma unroll
            for (int i = 0; i < 8; ++i) { sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f; }
#pragma unroll
            for (int np = 0; np < 4; ++np) {
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk) {
                    uint32_t b[4];
                    const int r = np * 16 + (lane & 7) + (lane >> 4) * 8;
                    const int c = kk * 2 + ((lane >> 3) & 1);
                    ldsm_x4(kb + tile_off<kD>(r, c), b);
                    mma_bf16(sacc[2 * np], qf[kk], b[0], b[1]);
                    mma_bf16(sacc[2 * np + 1], qf[kk], b[2], b[3]);
                }
            }
            // probabilities of this head: exp(scale * s - lse_row), added to the running head sum
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const float nl = row[r] < L ? -__ldg(lse + (int64_t)n * L + row[r]) * 1.4426950408889634f : -INFINITY;
#pragma unroll
                for (int nt = 0; nt < 8; ++nt) {
                    a[nt][2 * r] += fast_exp2(fmaf(sacc[nt][2 * r], sl2, nl));
                    a[nt][2 * r + 1] += fast_exp2(fmaf(sacc[nt][2 * r + 1], sl2, nl));
                }
            }
        }
        // maxima of the head mean over this tile's queries, by block class (rows past L hold zeros)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int64_t bq = row[r] / LB;
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                const float v = a[c >> 1][2 * r + (c & 1)] * inv_n;
                m_low[c] = fmaxf(m_low[c], bq > bk[c] ? v : 0.f);
                m_diag[c] = fmaxf(m_diag[c], bq == bk[c] ? v : 0.f);
                m_up[c] = fmaxf(m_up[c], bq < bk[c] ? v : 0.f);
            }
        }
    }
    cp_async_wait_all();
    // a column's maxima over the eight row groups of the warp, then over the four warps
#pragma unroll
    for (int c = 0; c < 16; ++c) {
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
            m_low[c] = fmaxf(m_low[c], __shfl_xor_sync(0xffffffffu, m_low[c], o));
            m_diag[c] = fmaxf(m_diag[c], __shfl_xor_sync(0xffffffffu, m_diag[c], o));
            m_up[c] = fmaxf(m_up[c], __shfl_xor_sync(0xffffffffu, m_up[c], o));
        }
        if (g == 0) {
            const int col = (c >> 1) * 8 + 2 * t4 + (c & 1);
            red[(warp * 3 + 0) * kT + col] = m_low[c];
            red[(warp * 3 + 1) * kT + col] = m_diag[c];
            red[(warp * 3 + 2) * kT + col] = m_up[c];
        }
    }
    __syncthreads();
    if (tid < kT && j0 + tid < L) {
        float v[3];
#pragma unroll
        for (int cl = 0; cl < 3; ++cl)
            v[cl] = fmaxf(fmaxf(red[(0 * 3 + cl) * kT + tid], red[(1 * 3 + cl) * kT + tid]),
                          fmaxf(red[(2 * 3 + cl) * kT + tid], red[(3 * 3 + cl) * kT + tid]));
        const int64_t j = j0 + tid;
        if (comp != nullptr) { comp[j] = v[0]; comp[L + j] = v[1]; comp[2 * L + j] = v[2]; }
        // Eq. 5
        s_out[j] = j < LB ? (v[1] + v[0]) * 0.5f : (j < L - LB ? (v[2] + v[1] + v[0]) * (1.0f / 3.0f) : (v[1] + v[2]) * 0.5f);
    }
}

inline pafu_status launch(const uint16_t* Q, const uint16_t* K, const float* lse, int64_t L, int64_t LB, int n_heads,
                          float scale, float* s, float* comp, cudaStream_t stream) {
    static bool attr_set[kMaxDevices] = {};
    if (!once_per_device(attr_set, [] {
            return cudaFuncSetAttribute(sse_meanfirst_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) == cudaSuccess;
        }))
        return PAFU_ERR_CUDA;
    const unsigned grid = (unsigned)((L + kT - 1) / kT);
    return cuda_ok(launch_dependent(sse_meanfirst_kernel, dim3(grid), dim3(kThreads), kSmemBytes, stream, 1, Q, K, lse, L, LB,
                                    n_heads, scale, s, comp));
}

}  // namespace sse_mf
}  // namespace pafu
