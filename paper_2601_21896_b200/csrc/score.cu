// Salience Estimation Head (Sec. 3.3; Appendix A "S-MLP"): per token
//   s = mean_o( W2 act(W1 x + b1) + b2 ), optionally sigmoid(s).
//
// Since the mean over outputs is linear, the second layer folds to one vector
//   w2m[h] = mean_o W2[o, h],  b2m = mean_o b2[o],   s = sum_h w2m[h] act(a_h) + b2m,
// so the hidden activations never leave the chip: a tile of tokens x hidden units is
// accumulated in fp32, passed through bias + activation, dotted with w2m and reduced per token.
#include "common.cuh"

namespace pafu {

constexpr int kScTok = 64;      // tokens per block
constexpr int kScHid = 64;      // hidden units per pass
constexpr int kScK = 32;        // reduction slice
constexpr int kScThreads = 256; // 16 x 16 threads, 4 x 4 outputs each

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) {
    return __uint_as_float(((uint32_t)b) << 16);
}

__device__ __forceinline__ float act_apply(float a, int act) {
    if (act == PAFU_ACT_GELU) return 0.5f * a * (1.0f + erff(a * 0.70710678118654752f));
    return a / (1.0f + __expf(-a));
}

__global__ void __launch_bounds__(kScThreads)
score_simt_kernel(const uint16_t* __restrict__ X, int64_t n_tokens, int64_t ldx,
                  int d_in, int d_hidden, int d_out, int act, int final,
                  const uint16_t* __restrict__ w1, const uint16_t* __restrict__ b1,
                  const uint16_t* __restrict__ w2, const uint16_t* __restrict__ b2,
                  float* __restrict__ scores) {
    __shared__ __align__(16) float Xs[kScK][kScTok];
    __shared__ __align__(16) float Ws[kScK][kScHid];
    __shared__ float w2m[kScHid];
    __shared__ float b1s[kScHid];

    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int64_t tok0 = (int64_t)blockIdx.x * kScTok;

    float b2m = 0.f;
    if (b2 != nullptr) {
        for (int o = 0; o < d_out; ++o) b2m += bf16_bits_to_float(b2[o]);
        b2m /= (float)d_out;
    }
    float tok_sum[4] = {0.f, 0.f, 0.f, 0.f};

    for (int h0 = 0; h0 < d_hidden; h0 += kScHid) {
        const int nh = min(kScHid, d_hidden - h0);
        __syncthreads();
        if (tid < kScHid) {
            float m = 0.f, bb = 0.f;
            if (tid < nh) {
                for (int o = 0; o < d_out; ++o) m += bf16_bits_to_float(w2[(int64_t)o * d_hidden + h0 + tid]);
                m /= (float)d_out;
                if (b1 != nullptr) bb = bf16_bits_to_float(b1[h0 + tid]);
            }
            w2m[tid] = m;
            b1s[tid] = bb;
        }
        float acc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

        for (int k0 = 0; k0 < d_in; k0 += kScK) {
            __syncthreads();
            {   // X tile: 64 rows x 32 k, one 16-byte load per thread, stored transposed
                const int row = tid >> 2, kc = (tid & 3) * 8;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (tok0 + row < n_tokens)
                    v = *reinterpret_cast<const uint4*>(X + (tok0 + row) * ldx + k0 + kc);
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    Xs[kc + 2 * i][row] = __uint_as_float(w[i] << 16);
                    Xs[kc + 2 * i + 1][row] = __uint_as_float(w[i] & 0xffff0000u);
                }
                uint4 u = make_uint4(0, 0, 0, 0);
                if (row < nh)
                    u = *reinterpret_cast<const uint4*>(w1 + (int64_t)(h0 + row) * d_in + k0 + kc);
                const uint32_t q[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    Ws[kc + 2 * i][row] = __uint_as_float(q[i] << 16);
                    Ws[kc + 2 * i + 1][row] = __uint_as_float(q[i] & 0xffff0000u);
                }
            }
            __syncthreads();
#pragma unroll
            for (int k = 0; k < kScK; ++k) {
                const float4 xv = *reinterpret_cast<const float4*>(&Xs[k][ty * 4]);
                const float4 wv = *reinterpret_cast<const float4*>(&Ws[k][tx * 4]);
                const float xa[4] = {xv.x, xv.y, xv.z, xv.w};
                const float wa[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(xa[i], wa[j], acc[i][j]);
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int h = tx * 4 + j;
                tok_sum[i] += w2m[h] * act_apply(acc[i][j] + b1s[h], act);   // w2m = 0 past nh
            }
    }
    // reduce over the 16 threads (tx) that share a token row: they are 16 consecutive lanes
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float v = tok_sum[i];
#pragma unroll
        for (int o = 8; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        const int64_t t = tok0 + ty * 4 + i;
        if (tx == 0 && t < n_tokens) {
            v += b2m;
            if (final == PAFU_FINAL_SIGMOID) v = 1.0f / (1.0f + __expf(-v));
            scores[t] = v;
        }
    }
}

size_t score_workspace_bytes(const pafu_head&) { return 0; }

pafu_status launch_score(const pafu_head& head, const uint16_t* X, int64_t n_tokens, int64_t ldx,
                         float* scores, void*, size_t, cudaStream_t stream) {
    if (n_tokens == 0) return PAFU_OK;
    const int64_t blocks = (n_tokens + kScTok - 1) / kScTok;
    score_simt_kernel<<<(unsigned)blocks, kScThreads, 0, stream>>>(
        X, n_tokens, ldx, head.d_in, head.d_hidden, head.d_out, head.act, head.final,
        head.w1, head.b1, head.w2, head.b2, scores);
    return cuda_ok(cudaGetLastError());
}

}  // namespace pafu
