// Batch-1 weight-streaming matrix-vector product: y = W x with W bf16 [N][K] row-major, x fp32.
//
// The work is HBM-bound (one FMA per 2 bytes), so it stays on the CUDA cores: each lane streams
// 16-byte pieces of weight rows with non-allocating loads, multiplies them with x held in shared
// memory as fp32 and accumulates in fp32; a warp shuffle closes each row.  A CTA is split into row
// groups of S warps; the S warps of a group share R rows and split K between them in interleaved
// 256-element chunks, so both short-and-wide and tall-and-narrow matrices spread over all SMs.
// CTAs are persistent over row tasks.  Summation order is fixed, so results are reproducible.
//
// Prologues: plain x, or x = rmsnorm(residual) * gain computed redundantly by every CTA (the vector
// is at most 20 KB).  Epilogues: store (+bias), accumulate into the residual stream, or
// silu(gate) * up over interleaved gate/up rows.
#pragma once
#include "st_common.cuh"

namespace st {

enum { PRO_PLAIN = 0, PRO_NORM = 1 };
enum { EPI_STORE = 0, EPI_RESADD = 1, EPI_SILU = 2 };

struct GemvParams {
    const uint16_t *W;     // [N][K] bf16
    const float *x;        // [rows][K]; the row used is x_row (or desc->m - 1 when x_row < 0)
    const float *gain;     // [K] (PRO_NORM)
    const float *bias;     // [N] or null
    float *y;              // EPI_STORE: [N]; EPI_RESADD: [N] accumulated; EPI_SILU: [N/2]
    const StepDesc *desc;  // may be null when x_row >= 0
    int32_t N, K;
    int32_t x_row;
    float eps;
};

template <int NW, int S, int R, int U, int PRO, int EPI>
__global__ void __launch_bounds__(NW * 32) gemv_kernel(const GemvParams p)
{
    static_assert(NW % S == 0, "row groups must tile the CTA");
    constexpr int G = NW / S;
    extern __shared__ float4 smem4[];
    const int K = p.K, K8 = K >> 3;
    float4 *xa = smem4;                       // x[8q .. 8q+3]
    float4 *xb = smem4 + K8;                  // x[8q+4 .. 8q+7]
    float *red = reinterpret_cast<float *>(smem4 + 2 * K8);  // [2][NW][R]
    __shared__ float s_part[32];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int grp = warp / S, ks = warp % S;
    const int n_tasks = (p.N + R - 1) / R;
    const int stride = gridDim.x * G;
    const int n_iter = (n_tasks + stride - 1) / stride;
    const int n_chunks = (K + 255) >> 8;
    const int n_cg = (n_chunks + S * U - 1) / (S * U);   // chunk groups per task, the same for every warp
    const int n_items = n_iter * n_cg;

    // The weight stream is software-pipelined: item j = (task iteration j / n_cg, chunk group j % n_cg);
    // the loads of item j + 1 are in flight while item j is multiplied.
    auto issue = [&](int j, uint4 (&w)[U][R]) {
        const int it = j / n_cg, cg = j - it * n_cg;
        const int task = it * stride + blockIdx.x * G + grp;
        const bool live = j < n_items && task < n_tasks;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int e = ((ks + (cg * U + u) * S) << 8) + (lane << 3);
#pragma unroll
            for (int r = 0; r < R; ++r) {
                int row = task * R + r;
                row = row < p.N ? row : p.N - 1;
                w[u][r] = (live && e < K) ? ldg_nc_v4(p.W + (size_t)row * K + e) : make_uint4(0, 0, 0, 0);
            }
        }
    };

    uint4 wa[U][R], wb[U][R];
    issue(0, wa);   // weights do not depend on the previous kernel: fetch before waiting for it

    pdl_wait();
    pdl_launch();
    if (p.desc && p.desc->m <= 0) return;
    const int xrow = p.x_row >= 0 ? p.x_row : p.desc->m - 1;
    const float4 *xin = reinterpret_cast<const float4 *>(p.x + (size_t)xrow * K);

    // ---- bring x into shared memory (normalised if asked) ----
    // The two halves of each 8-element piece go to separate arrays so that lanes reading
    // consecutive pieces hit consecutive 16-byte slots (no bank conflicts).
    float ss = 0.f;
    for (int q = tid; q < 2 * K8; q += NW * 32) {
        float4 v = xin[q];
        if (PRO == PRO_NORM) ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        ((q & 1) ? xb : xa)[q >> 1] = v;
    }
    if (PRO == PRO_NORM) {
        ss = warp_sum(ss);
        if (lane == 0) s_part[warp] = ss;
        __syncthreads();
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) tot += s_part[w];
        const float inv = rsqrtf(tot / (float)K + p.eps);
        const float4 *g4 = reinterpret_cast<const float4 *>(p.gain);
        for (int q = tid; q < 2 * K8; q += NW * 32) {
            float4 *dst = ((q & 1) ? xb : xa) + (q >> 1);
            float4 v = *dst, g = g4[q];
            v.x *= inv * g.x; v.y *= inv * g.y; v.z *= inv * g.z; v.w *= inv * g.w;
            *dst = v;
        }
    }
    __syncthreads();

    float acc[R];
#pragma unroll
    for (int r = 0; r < R; ++r) acc[r] = 0.f;

    auto consume = [&](int j, const uint4 (&w)[U][R]) {
        if (j >= n_items) return;
        const int it = j / n_cg, cg = j - it * n_cg;
        const int task = it * stride + blockIdx.x * G + grp;
        const bool live = task < n_tasks;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int e = ((ks + (cg * U + u) * S) << 8) + (lane << 3);
            if (e < K) {
                const float4 a = xa[e >> 3], b = xb[e >> 3];
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const uint4 v = w[u][r];
                    float t = acc[r];
                    t = fmaf(bf16_lo(v.x), a.x, t); t = fmaf(bf16_hi(v.x), a.y, t);
                    t = fmaf(bf16_lo(v.y), a.z, t); t = fmaf(bf16_hi(v.y), a.w, t);
                    t = fmaf(bf16_lo(v.z), b.x, t); t = fmaf(bf16_hi(v.z), b.y, t);
                    t = fmaf(bf16_lo(v.w), b.z, t); t = fmaf(bf16_hi(v.w), b.w, t);
                    acc[r] = t;
                }
            }
        }
        if (cg != n_cg - 1) return;
        // ---- the task is complete: close the rows ----
#pragma unroll
        for (int r = 0; r < R; ++r) acc[r] = warp_sum(acc[r]);
        float *rbuf = red + (size_t)(it & 1) * NW * R;
        if (S > 1) {
            if (lane == 0) {
#pragma unroll
                for (int r = 0; r < R; ++r) rbuf[warp * R + r] = acc[r];
            }
            // group-local barrier: the S warps of this row group only
            asm volatile("bar.sync %0, %1;" ::"r"(grp + 1), "r"(S * 32) : "memory");
        }
        if (ks == 0 && lane == 0 && live) {
            float v[R];
#pragma unroll
            for (int r = 0; r < R; ++r) {
                float t = acc[r];
                if (S > 1) {
                    t = 0.f;
#pragma unroll
                    for (int s2 = 0; s2 < S; ++s2) t += rbuf[(grp * S + s2) * R + r];
                }
                v[r] = t;
            }
            if (EPI == EPI_SILU) {
#pragma unroll
                for (int r = 0; r + 1 < R; r += 2) {
                    const int row = task * R + r;
                    if (row + 1 < p.N) {
                        const float g = v[r], u = v[r + 1];
                        p.y[row >> 1] = g / (1.f + expf(-g)) * u;
                    }
                }
            } else {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const int row = task * R + r;
                    if (row < p.N) {
                        float t = v[r] + (p.bias ? p.bias[row] : 0.f);
                        if (EPI == EPI_RESADD) t += p.y[row];
                        p.y[row] = t;
                    }
                }
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) acc[r] = 0.f;
    };

    for (int j = 0; j < n_items; j += 2) {
        issue(j + 1, wb);
        consume(j, wa);
        issue(j + 2, wa);
        consume(j + 1, wb);
    }
}

}  // namespace st
