// Multi-row (prefill / catch-up) helpers on the CUDA cores: row-wise RMSNorm and a plain
// shared-memory tiled GEMM  Y[m][n] = sum_k A[m][k] * W[n][k]  (W bf16; fp32 accumulate).
//
// Activations that feed a matrix product are kept as two bf16 planes, A = hi + lo with
// hi = bf16(a) and lo = bf16(a - hi): a single bf16 rounding of the activations (relative error
// 2^-9) costs more than the whole logit tolerance once it has passed through a few layers, the
// pair carries 16 significand bits.  Both planes multiply the same weight tile.
#pragma once
#include "st_common.cuh"

namespace st {

// XN[i] = rmsnorm(X[i]) * gain as a hi/lo bf16 pair, one CTA per row.  With k_splits > 0 the row first
// receives the K-split partial sums of the projection that feeds the residual stream,
// X[i] += sum_s Ws[s][i] (in split order), so that projection needs no reduction pass of its own.
__global__ void __launch_bounds__(1024) rmsnorm_rows_kernel(const StepDesc *desc, float *X, const float *Ws, int k_splits, int ws_rows,
                                                           const float *gain, float eps, int hidden, uint16_t *XN_hi, uint16_t *XN_lo)
{
    pdl_launch();   // the projection that follows may fetch its weights meanwhile
    pdl_wait();     // the row and its partial sums come from the kernels before this one
    const int i = blockIdx.x;
    if (i >= desc->m) return;
    float4 *x4 = reinterpret_cast<float4 *>(X + (size_t)i * hidden);
    const int n4 = hidden >> 2;
    float ss = 0.f;
    for (int j = threadIdx.x; j < n4; j += blockDim.x) {
        float4 v = x4[j];
        if (k_splits > 0) {
            v = add_splits4(v, Ws + (size_t)i * hidden + 4 * (size_t)j, (size_t)ws_rows * hidden, k_splits);
            x4[j] = v;
        }
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
    __shared__ float s_part[32];
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += s_part[w];
    const float inv = rsqrtf(tot / (float)hidden + eps);
    uint2 *hi = reinterpret_cast<uint2 *>(XN_hi + (size_t)i * hidden), *lo = reinterpret_cast<uint2 *>(XN_lo + (size_t)i * hidden);
    for (int j = threadIdx.x; j < n4; j += blockDim.x) {
        const float4 v = x4[j];   // this thread's own values (just written or read above)
        const float4 g = reinterpret_cast<const float4 *>(gain)[j];
        uint16_t h0, h1, h2, h3, l0, l1, l2, l3;
        split_bf16(v.x * inv * g.x, h0, l0);
        split_bf16(v.y * inv * g.y, h1, l1);
        split_bf16(v.z * inv * g.z, h2, l2);
        split_bf16(v.w * inv * g.w, h3, l3);
        hi[j] = make_uint2((uint32_t)h0 | ((uint32_t)h1 << 16), (uint32_t)h2 | ((uint32_t)h3 << 16));
        lo[j] = make_uint2((uint32_t)l0 | ((uint32_t)l1 << 16), (uint32_t)l2 | ((uint32_t)l3 << 16));
    }
}

enum { GEPI_STORE = 0, GEPI_RESADD = 1, GEPI_SILU = 2 };

struct GemmParams {
    const StepDesc *desc;
    const uint16_t *A_hi, *A_lo;  // [m][K] bf16 planes, A = hi + lo
    const uint16_t *W;            // [N][K] bf16
    const float *bias;            // [N] or null
    float *Yf;                    // GEPI_STORE: [m][N]; GEPI_RESADD: [m][N] accumulated
    uint16_t *Yb_hi, *Yb_lo;      // GEPI_SILU: [m][N/2] hi/lo planes of silu(col 2j) * col 2j+1
    int32_t N, K;
};

template <int EPI>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const GemmParams p)
{
    constexpr int BM = 64, BN = 64, BK = 32;
    const int m = p.desc->m;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    if (m0 >= m) return;
    __shared__ float As[BK][BM + 4];
    __shared__ float Ws[BK][BN + 4];
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;  // 16 x 16 threads, 4 x 4 outputs each
    float acc[4][4] = {};
    // loader: 256 threads, each brings 8 consecutive k of one row (64 rows x 32 k = 2048 elements)
    const int lr = tid >> 2, lk = (tid & 3) * 8;
    for (int k0 = 0; k0 < p.K; k0 += BK) {
        {
            uint4 a = make_uint4(0, 0, 0, 0), a2 = make_uint4(0, 0, 0, 0), w = make_uint4(0, 0, 0, 0);
            if (m0 + lr < m && k0 + lk < p.K) {
                a = *reinterpret_cast<const uint4 *>(p.A_hi + (size_t)(m0 + lr) * p.K + k0 + lk);
                a2 = *reinterpret_cast<const uint4 *>(p.A_lo + (size_t)(m0 + lr) * p.K + k0 + lk);
            }
            if (n0 + lr < p.N && k0 + lk < p.K) w = *reinterpret_cast<const uint4 *>(p.W + (size_t)(n0 + lr) * p.K + k0 + lk);
            const uint32_t av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {a2.x, a2.y, a2.z, a2.w}, wv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                As[lk + 2 * j][lr] = bf16_lo(av[j]) + bf16_lo(bv[j]);
                As[lk + 2 * j + 1][lr] = bf16_hi(av[j]) + bf16_hi(bv[j]);
                Ws[lk + 2 * j][lr] = bf16_lo(wv[j]);
                Ws[lk + 2 * j + 1][lr] = bf16_hi(wv[j]);
            }
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            const float4 a = *reinterpret_cast<const float4 *>(&As[kk][ty * 4]);
            const float4 w = *reinterpret_cast<const float4 *>(&Ws[kk][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w}, wv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], wv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = m0 + ty * 4 + i;
        if (r >= m) continue;
        if (EPI == GEPI_SILU) {
#pragma unroll
            for (int j = 0; j < 4; j += 2) {
                const int c = n0 + tx * 4 + j;
                if (c + 1 < p.N) {
                    const float g = acc[i][j], u = acc[i][j + 1];
                    const size_t o = (size_t)r * (p.N >> 1) + (c >> 1);
                    split_bf16(g / (1.f + expf(-g)) * u, p.Yb_hi[o], p.Yb_lo[o]);
                }
            }
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int c = n0 + tx * 4 + j;
                if (c < p.N) {
                    float v = acc[i][j] + (p.bias ? p.bias[c] : 0.f);
                    float *dst = p.Yf + (size_t)r * p.N + c;
                    if (EPI == GEPI_RESADD) v += *dst;
                    *dst = v;
                }
            }
        }
    }
}

}  // namespace st
