// Rotary embedding + KV append, and grouped-query attention over the paged KV cache.
//
// KV pages: pool[layer][page][kv_head][slot_in_page][head_dim] in fp16, so the tokens of one
// (page, head) are contiguous.  A sequence's block table maps position / page_size -> page.
//
// Attention is a flash-decoding style split over the keys: one CTA per (key split, kv head, query
// row) processes all G = n_q_heads / n_kv_heads query heads of its kv head against its key range,
// so every K/V byte is read once per kv head.  Lanes are grouped D/8 per key (each lane owns 8
// consecutive channels: one 16-byte load of K and of V), scores close with log2(D/8) shuffles, and
// softmax is kept online in fp32.  Partial results of the splits are merged by the CTA that
// finishes last (a ticket counter; nothing waits on anything).
#pragma once
#include "st_common.cuh"

namespace st {

struct KvView {
    uint16_t *k, *v;          // this layer's pools
    const int32_t *block_tab; // this sequence's block table
    int32_t page_size, page_shift, n_pages, n_kv_heads;
};

__device__ __forceinline__ size_t kv_offset(const KvView &kv, int pos, int head, int D, int32_t *status)
{
    int page = kv.block_tab[pos >> kv.page_shift];
    if ((unsigned)page >= (unsigned)kv.n_pages) {
        atomicOr(status, DEV_BAD_PAGE);
        page = 0;
    }
    return (((size_t)page * kv.n_kv_heads + head) * kv.page_size + (pos & (kv.page_size - 1))) * D;
}

// x[i] = E[token_i] (fp32) and the rotary table of row i: cs[i][j] = (cos, sin)(pos_i * inv_freq[j]),
// evaluated in double so that long positions lose nothing.
// row_pos (nullable): the rows belong to different sequences (batched decode), row i sits at position row_pos[i].
__global__ void embed_rope_kernel(const StepDesc *desc, const int32_t *tok, const uint16_t *E, int hidden, int vocab,
                                  float *X, const double *inv_freq, int half, float2 *cs, int32_t *status,
                                  const int32_t *row_pos = nullptr)
{
    const int i = blockIdx.x;
    if (i >= desc->m) return;
    int t = tok[desc->tok_off + i];
    if ((unsigned)t >= (unsigned)vocab) {
        if (threadIdx.x == 0) atomicOr(status, DEV_BAD_TOKEN);
        t = 0;
    }
    const uint32_t *e = reinterpret_cast<const uint32_t *>(E + (size_t)t * hidden);
    float2 *x2 = reinterpret_cast<float2 *>(X + (size_t)i * hidden);
    for (int j = threadIdx.x; j < hidden / 2; j += blockDim.x) {
        const uint32_t v = e[j];
        x2[j] = make_float2(bf16_lo(v), bf16_hi(v));
    }
    const double pos = (double)(row_pos ? row_pos[i] : desc->pos0 + i);
    for (int j = threadIdx.x; j < half; j += blockDim.x) {
        double s, c;
        sincos(pos * inv_freq[j], &s, &c);
        cs[(size_t)i * half + j] = make_float2((float)c, (float)s);
    }
}

// Rotate q in place (fp32), rotate k and store k, v into the cache (fp16).
// With row_slot / row_pos the rows belong to different sequences (batched decode).
// qkv: [rows][(Hq + 2 Hkv) * D] = q heads, then k heads, then v heads.  With k_splits > 0 the row is not in
// qkv yet: it is bias + the K-split partial sums Ws[s][row] of the QKV projection (summed in split order).
__global__ void __launch_bounds__(512) rope_append_kernel(const StepDesc *desc, float *qkv, const float *Ws, int k_splits, int ws_rows,
                                                          const float *bias, const float2 *cs, int Hq, int Hkv, int D, KvView kv,
                                                          int32_t *status, const int32_t *row_slot = nullptr,
                                                          const int32_t *row_pos = nullptr, int pages_per_seq = 0)
{
    pdl_launch();
    pdl_wait();
    const int i = blockIdx.x;
    if (i >= desc->m) return;
    if (row_slot) kv.block_tab += (size_t)row_slot[i] * pages_per_seq;   // batched decode: kv.block_tab is sequence 0's table
    const int half = D >> 1, pos = row_pos ? row_pos[i] : desc->pos0 + i, N = (Hq + 2 * Hkv) * D;
    float *row = qkv + (size_t)i * N;
    const float2 *c = cs + (size_t)i * half;
    auto val4 = [&](int n) {   // 4 consecutive features of the row, n a multiple of 4
        if (k_splits <= 0) return *reinterpret_cast<const float4 *>(row + n);
        float4 v = bias ? *reinterpret_cast<const float4 *>(bias + n) : make_float4(0.f, 0.f, 0.f, 0.f);
        return add_splits4(v, Ws + (size_t)i * N + n, (size_t)ws_rows * N, k_splits);
    };
    const int q4 = half >> 2;   // groups of 4 channel pairs per head
    for (int idx = threadIdx.x; idx < (Hq + Hkv) * q4; idx += blockDim.x) {
        const int h = idx / q4, j = (idx - h * q4) * 4;
        const float4 a = val4(h * D + j), b = val4(h * D + j + half);
        const float2 t0 = c[j], t1 = c[j + 1], t2 = c[j + 2], t3 = c[j + 3];
        const float4 ra = make_float4(a.x * t0.x - b.x * t0.y, a.y * t1.x - b.y * t1.y, a.z * t2.x - b.z * t2.y, a.w * t3.x - b.w * t3.y);
        const float4 rb = make_float4(b.x * t0.x + a.x * t0.y, b.y * t1.x + a.y * t1.y, b.z * t2.x + a.z * t2.y, b.w * t3.x + a.w * t3.y);
        if (h < Hq) {
            *reinterpret_cast<float4 *>(row + h * D + j) = ra;
            *reinterpret_cast<float4 *>(row + h * D + j + half) = rb;
        } else {
            const size_t o = kv_offset(kv, pos, h - Hq, D, status);
            *reinterpret_cast<uint2 *>(kv.k + o + j) = make_uint2((uint32_t)kv_bits(ra.x) | ((uint32_t)kv_bits(ra.y) << 16),
                                                                  (uint32_t)kv_bits(ra.z) | ((uint32_t)kv_bits(ra.w) << 16));
            *reinterpret_cast<uint2 *>(kv.k + o + j + half) = make_uint2((uint32_t)kv_bits(rb.x) | ((uint32_t)kv_bits(rb.y) << 16),
                                                                         (uint32_t)kv_bits(rb.z) | ((uint32_t)kv_bits(rb.w) << 16));
        }
    }
    const int v0 = (Hq + Hkv) * D;
    for (int idx = threadIdx.x; idx < Hkv * (D >> 2); idx += blockDim.x) {
        const int h = idx / (D >> 2), j = (idx - h * (D >> 2)) * 4;
        const float4 v = val4(v0 + h * D + j);
        *reinterpret_cast<uint2 *>(kv.v + kv_offset(kv, pos, h, D, status) + j) =
            make_uint2((uint32_t)kv_bits(v.x) | ((uint32_t)kv_bits(v.y) << 16), (uint32_t)kv_bits(v.z) | ((uint32_t)kv_bits(v.w) << 16));
    }
}

constexpr int kMaxAttnSplits = 160;   // upper bound of n_splits (the host never asks for more)

struct AttnParams {
    const StepDesc *desc;
    const float *qkv;           // [rows][(Hq + 2 Hkv) * D], q already rotated
    KvView kv;
    float *out_f32;             // [rows][Hq * D] (decode) or null
    uint16_t *out_hi, *out_lo;  // [rows][Hq * D] hi/lo bf16 planes (prefill) or null
    float *part_o;              // [rows][Hq][n_splits][D]     (n_splits > 1)
    float *part_ml;             // [rows][Hq][n_splits][2]
    int32_t *tickets;           // [rows][Hkv], zero between launches
    int32_t *status;
    int32_t Hq, n_splits;
    float scale;
};

__device__ __forceinline__ void attn_store(const AttnParams &p, size_t oi, float r)
{
    if (p.out_f32) p.out_f32[oi] = r;
    if (p.out_hi) split_bf16(r, p.out_hi[oi], p.out_lo[oi]);
}

template <int D, int G>
__global__ void __launch_bounds__(128) attn_kernel(const AttnParams p)
{
    constexpr int LPK = D / 8;       // lanes per key
    constexpr int KPW = 32 / LPK;    // keys per warp step
    constexpr int NWARP = 4;
    constexpr int UK = 4;            // key steps in flight
    const int row = blockIdx.z, hk = blockIdx.y, split = blockIdx.x;
    if (row >= p.desc->m) return;
    const int n_keys = p.desc->pos0 + row + 1;
    const int Hkv = p.kv.n_kv_heads;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int sub = lane / LPK, ch = (lane % LPK) * 8;

    const int per = (n_keys + p.n_splits - 1) / p.n_splits;
    const int k0 = split * per, k1 = min(n_keys, k0 + per);

    float q[G][8];
    {
        const float *qrow = p.qkv + (size_t)row * (p.Hq + 2 * Hkv) * D + (size_t)hk * G * D + ch;
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float4 a = *reinterpret_cast<const float4 *>(qrow + g * D);
            const float4 b = *reinterpret_cast<const float4 *>(qrow + g * D + 4);
            q[g][0] = a.x * p.scale; q[g][1] = a.y * p.scale; q[g][2] = a.z * p.scale; q[g][3] = a.w * p.scale;
            q[g][4] = b.x * p.scale; q[g][5] = b.y * p.scale; q[g][6] = b.z * p.scale; q[g][7] = b.w * p.scale;
        }
    }
    float mx[G], den[G], o[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        mx[g] = -INFINITY;
        den[g] = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) o[g][e] = 0.f;
    }

    for (int base = k0 + (warp * UK) * KPW; base < k1; base += NWARP * UK * KPW) {
        uint4 kf[UK], vf[UK];
        bool ok[UK];
#pragma unroll
        for (int u = 0; u < UK; ++u) {
            const int key = base + u * KPW + sub;
            ok[u] = key < k1;
            if (ok[u]) {
                const size_t off = kv_offset(p.kv, key, hk, D, p.status) + ch;
                kf[u] = *reinterpret_cast<const uint4 *>(p.kv.k + off);
                vf[u] = *reinterpret_cast<const uint4 *>(p.kv.v + off);
            } else {
                kf[u] = make_uint4(0, 0, 0, 0);
                vf[u] = make_uint4(0, 0, 0, 0);
            }
        }
#pragma unroll
        for (int u = 0; u < UK; ++u) {
            float kk[8] = {kv_lo(kf[u].x), kv_hi(kf[u].x), kv_lo(kf[u].y), kv_hi(kf[u].y),
                           kv_lo(kf[u].z), kv_hi(kf[u].z), kv_lo(kf[u].w), kv_hi(kf[u].w)};
            float vv[8] = {kv_lo(vf[u].x), kv_hi(vf[u].x), kv_lo(vf[u].y), kv_hi(vf[u].y),
                           kv_lo(vf[u].z), kv_hi(vf[u].z), kv_lo(vf[u].w), kv_hi(vf[u].w)};
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float s = 0.f;
#pragma unroll
                for (int e = 0; e < 8; ++e) s = fmaf(q[g][e], kk[e], s);
#pragma unroll
                for (int off = LPK / 2; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
                if (ok[u]) {   // uniform within the lane group of a key
                    const float mnew = fmaxf(mx[g], s);
                    const float corr = __expf(mx[g] - mnew), pw = __expf(s - mnew);
                    den[g] = den[g] * corr + pw;
#pragma unroll
                    for (int e = 0; e < 8; ++e) o[g][e] = fmaf(pw, vv[e], o[g][e] * corr);
                    mx[g] = mnew;
                }
            }
        }
    }

    // ---- merge the lane groups of a warp, then the warps of the CTA ----
#pragma unroll
    for (int g = 0; g < G; ++g) {
#pragma unroll
        for (int off = LPK; off < 32; off <<= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, mx[g], off);
            const float d2 = __shfl_xor_sync(0xffffffffu, den[g], off);
            const float mnew = fmaxf(mx[g], m2);
            const float c1 = mx[g] == -INFINITY ? 0.f : __expf(mx[g] - mnew);
            const float c2 = m2 == -INFINITY ? 0.f : __expf(m2 - mnew);
            den[g] = den[g] * c1 + d2 * c2;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float o2 = __shfl_xor_sync(0xffffffffu, o[g][e], off);
                o[g][e] = o[g][e] * c1 + o2 * c2;
            }
            mx[g] = mnew;
        }
    }
    __shared__ float s_o[NWARP][G][D];
    __shared__ float s_m[NWARP][G], s_d[NWARP][G];
    __shared__ int s_last;
    if (sub == 0) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
#pragma unroll
            for (int e = 0; e < 8; ++e) s_o[warp][g][ch + e] = o[g][e];
            if (lane == 0) { s_m[warp][g] = mx[g]; s_d[warp][g] = den[g]; }
        }
    }
    __syncthreads();
    const int hq0 = hk * G;
    for (int idx = tid; idx < G * D; idx += 128) {
        const int g = idx / D, c = idx - g * D;
        float mnew = -INFINITY;
#pragma unroll
        for (int w = 0; w < NWARP; ++w) mnew = fmaxf(mnew, s_m[w][g]);
        float dsum = 0.f, osum = 0.f;
#pragma unroll
        for (int w = 0; w < NWARP; ++w) {
            const float cw = s_m[w][g] == -INFINITY ? 0.f : __expf(s_m[w][g] - mnew);
            dsum += s_d[w][g] * cw;
            osum += s_o[w][g][c] * cw;
        }
        if (p.n_splits == 1) {
            attn_store(p, ((size_t)row * p.Hq + hq0 + g) * D + c, osum / dsum);
        } else {
            const size_t pi = ((size_t)row * p.Hq + hq0 + g) * p.n_splits + split;
            p.part_o[pi * D + c] = osum;
            if (c == 0) { p.part_ml[pi * 2] = mnew; p.part_ml[pi * 2 + 1] = dsum; }
        }
    }
    if (p.n_splits == 1) return;

    // ---- the CTA that finishes last for this (row, kv head) merges the splits ----
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int t = atomicAdd(&p.tickets[row * Hkv + hk], 1);
        s_last = (t == p.n_splits - 1);
        if (s_last) p.tickets[row * Hkv + hk] = 0;   // ready for the next launch
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // weights of the splits: w[g][s] = exp(m_s - max_s m) (0 for empty splits), shared by all channels
    __shared__ float s_w[G][kMaxAttnSplits], s_l[G][kMaxAttnSplits];
    __shared__ float s_den[G];
    for (int idx = tid; idx < G * p.n_splits; idx += 128) {
        const int g = idx / p.n_splits, sp = idx - g * p.n_splits;
        const float2 ml = __ldcg(reinterpret_cast<const float2 *>(p.part_ml) + ((size_t)row * p.Hq + hq0 + g) * p.n_splits + sp);
        s_w[g][sp] = ml.x;
        s_l[g][sp] = ml.y;
    }
    __syncthreads();
    if (tid < G) {
        float mnew = -INFINITY;
        for (int sp = 0; sp < p.n_splits; ++sp) mnew = fmaxf(mnew, s_w[tid][sp]);
        float dsum = 0.f;
        for (int sp = 0; sp < p.n_splits; ++sp) {
            const float ms = s_w[tid][sp];
            const float cw = ms == -INFINITY ? 0.f : __expf(ms - mnew);
            s_w[tid][sp] = cw;
            dsum += s_l[tid][sp] * cw;
        }
        s_den[tid] = dsum;
    }
    __syncthreads();
    for (int idx = tid; idx < G * D; idx += 128) {
        const int g = idx / D, c = idx - g * D;
        const float *po = p.part_o + ((size_t)row * p.Hq + hq0 + g) * p.n_splits * D + c;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        int sp = 0;
        for (; sp + 4 <= p.n_splits; sp += 4) {   // four independent loads in flight
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[j] = fmaf(__ldcg(po + (size_t)(sp + j) * D), s_w[g][sp + j], acc[j]);
        }
        for (; sp < p.n_splits; ++sp) acc[0] = fmaf(__ldcg(po + (size_t)sp * D), s_w[g][sp], acc[0]);
        attn_store(p, ((size_t)row * p.Hq + hq0 + g) * D + c, ((acc[0] + acc[1]) + (acc[2] + acc[3])) / s_den[g]);
    }
}

// Multi-row (prefill / catch-up) attention: the 8 warps of a CTA take 8 consecutive query rows of one kv
// head and walk the keys together, tile by tile through shared memory, so that every K/V byte is read
// from L2 once per 8 rows instead of once per row.  Each warp keeps its row's online softmax for all G
// query heads exactly as the decode kernel does; rows are causal (row i sees keys 0 .. pos0 + i).
template <int D, int G>
__global__ void __launch_bounds__(256, 2) attn_rows_kernel(const AttnParams p)
{
    constexpr int LPK = D / 8, KPW = 32 / LPK, TK = 64, ROWS = 8;
    __shared__ uint4 s_k[TK * D / 8], s_v[TK * D / 8];
    __shared__ float s_w[G][kMaxAttnSplits], s_l[G][kMaxAttnSplits];   // split merge (per warp use, one row at a time)
    __shared__ float s_den[ROWS][G];
    __shared__ int s_last[ROWS];
    const int m = p.desc->m;
    const int row0 = blockIdx.z * ROWS;
    if (row0 >= m) return;
    const int hk = blockIdx.y, split = blockIdx.x;
    const int Hkv = p.kv.n_kv_heads;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int sub = lane / LPK, ch = (lane % LPK) * 8;
    const int row = row0 + warp;
    const bool row_live = row < m;
    const int n_keys = p.desc->pos0 + (row_live ? row : m - 1) + 1;            // keys of this warp's row
    const int n_keys_cta = p.desc->pos0 + min(m, row0 + ROWS);                 // keys of the CTA's last row
    // split the CTA's key range; every row uses the same boundaries (rows with fewer keys stop early)
    const int per = ((n_keys_cta + p.n_splits - 1) / p.n_splits + TK - 1) / TK * TK;
    const int k0 = split * per, k1_cta = min(n_keys_cta, k0 + per);
    const int k1 = min(n_keys, k1_cta);

    float q[G][8];
    {
        const float *qrow = p.qkv + (size_t)(row_live ? row : 0) * (p.Hq + 2 * Hkv) * D + (size_t)hk * G * D + ch;
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float4 a = *reinterpret_cast<const float4 *>(qrow + g * D);
            const float4 b = *reinterpret_cast<const float4 *>(qrow + g * D + 4);
            q[g][0] = a.x * p.scale; q[g][1] = a.y * p.scale; q[g][2] = a.z * p.scale; q[g][3] = a.w * p.scale;
            q[g][4] = b.x * p.scale; q[g][5] = b.y * p.scale; q[g][6] = b.z * p.scale; q[g][7] = b.w * p.scale;
        }
    }
    float mx[G], den[G], o[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        mx[g] = -INFINITY;
        den[g] = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) o[g][e] = 0.f;
    }
    for (int t0 = k0; t0 < k1_cta; t0 += TK) {
        // ---- stage the key tile: TK keys x D channels of K and of V ----
        for (int i = tid; i < TK * LPK; i += 256) {
            const int key = t0 + i / LPK, c8 = (i % LPK) * 8;
            uint4 kq = make_uint4(0, 0, 0, 0), vq = make_uint4(0, 0, 0, 0);
            if (key < k1_cta) {
                const size_t off = kv_offset(p.kv, key, hk, D, p.status) + c8;
                kq = *reinterpret_cast<const uint4 *>(p.kv.k + off);
                vq = *reinterpret_cast<const uint4 *>(p.kv.v + off);
            }
            s_k[i] = kq;
            s_v[i] = vq;
        }
        __syncthreads();
        if (row_live) {
            const int tile_keys = min(TK, k1 - t0);   // may be <= 0 for rows that ended earlier
            constexpr int UB = 4;                      // keys per lane group and softmax update
            for (int j = 0; j < tile_keys; j += KPW * UB) {
                // scores of UB keys first (independent chains), then one rescale per head
                float sc[UB][G];
                bool ok[UB];
#pragma unroll
                for (int u = 0; u < UB; ++u) {
                    const int kj = j + u * KPW + sub;
                    ok[u] = kj < tile_keys;
                    const uint4 kf = s_k[min(kj, TK - 1) * LPK + (lane % LPK)];
                    const float kk[8] = {kv_lo(kf.x), kv_hi(kf.x), kv_lo(kf.y), kv_hi(kf.y),
                                         kv_lo(kf.z), kv_hi(kf.z), kv_lo(kf.w), kv_hi(kf.w)};
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        float t = 0.f;
#pragma unroll
                        for (int e = 0; e < 8; ++e) t = fmaf(q[g][e], kk[e], t);
                        sc[u][g] = t;
                    }
                }
#pragma unroll
                for (int off = LPK / 2; off > 0; off >>= 1)
#pragma unroll
                    for (int u = 0; u < UB; ++u)
#pragma unroll
                        for (int g = 0; g < G; ++g) sc[u][g] += __shfl_xor_sync(0xffffffffu, sc[u][g], off);
                float vv[UB][8];
#pragma unroll
                for (int u = 0; u < UB; ++u) {
                    const int kj = j + u * KPW + sub;
                    const uint4 vf = s_v[min(kj, TK - 1) * LPK + (lane % LPK)];
                    vv[u][0] = kv_lo(vf.x); vv[u][1] = kv_hi(vf.x); vv[u][2] = kv_lo(vf.y); vv[u][3] = kv_hi(vf.y);
                    vv[u][4] = kv_lo(vf.z); vv[u][5] = kv_hi(vf.z); vv[u][6] = kv_lo(vf.w); vv[u][7] = kv_hi(vf.w);
                }
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    float mnew = mx[g];
#pragma unroll
                    for (int u = 0; u < UB; ++u)
                        if (ok[u]) mnew = fmaxf(mnew, sc[u][g]);
                    if (mnew > -INFINITY) {
                        const float corr = mx[g] == -INFINITY ? 0.f : __expf(mx[g] - mnew);
                        den[g] *= corr;
#pragma unroll
                        for (int e = 0; e < 8; ++e) o[g][e] *= corr;
#pragma unroll
                        for (int u = 0; u < UB; ++u) {
                            if (ok[u]) {
                                const float pw = __expf(sc[u][g] - mnew);
                                den[g] += pw;
#pragma unroll
                                for (int e = 0; e < 8; ++e) o[g][e] = fmaf(pw, vv[u][e], o[g][e]);
                            }
                        }
                        mx[g] = mnew;
                    }
                }
            }
        }
        __syncthreads();
    }
    // ---- merge the lane groups of the warp: the row's result for this split ----
#pragma unroll
    for (int g = 0; g < G; ++g) {
#pragma unroll
        for (int off = LPK; off < 32; off <<= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, mx[g], off);
            const float d2 = __shfl_xor_sync(0xffffffffu, den[g], off);
            const float mnew = fmaxf(mx[g], m2);
            const float c1 = mx[g] == -INFINITY ? 0.f : __expf(mx[g] - mnew);
            const float c2 = m2 == -INFINITY ? 0.f : __expf(m2 - mnew);
            den[g] = den[g] * c1 + d2 * c2;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float o2 = __shfl_xor_sync(0xffffffffu, o[g][e], off);
                o[g][e] = o[g][e] * c1 + o2 * c2;
            }
            mx[g] = mnew;
        }
    }
    const int hq0 = hk * G;
    if (p.n_splits == 1) {
        if (row_live && sub == 0) {
#pragma unroll
            for (int g = 0; g < G; ++g)
#pragma unroll
                for (int e = 0; e < 8; ++e) attn_store(p, ((size_t)row * p.Hq + hq0 + g) * D + ch + e, o[g][e] / den[g]);
        }
        return;
    }
    if (row_live && sub == 0) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const size_t pi = ((size_t)row * p.Hq + hq0 + g) * p.n_splits + split;
#pragma unroll
            for (int e = 0; e < 8; ++e) p.part_o[pi * D + ch + e] = o[g][e];
            if (lane == 0) { p.part_ml[pi * 2] = mx[g]; p.part_ml[pi * 2 + 1] = den[g]; }
        }
    }
    // ---- the CTA that finishes a row last (over the splits) merges that row ----
    __threadfence();
    __syncwarp();
    if (lane == 0) {
        int last = 0;
        if (row_live) {
            const int t = atomicAdd(&p.tickets[row * Hkv + hk], 1);
            last = (t == p.n_splits - 1);
            if (last) p.tickets[row * Hkv + hk] = 0;
        }
        s_last[warp] = last;
    }
    __syncthreads();
    for (int r = 0; r < ROWS; ++r) {       // the whole CTA merges each finished row in turn
        if (!s_last[r]) continue;          // uniform: shared flag
        const int rrow = row0 + r;
        __threadfence();
        for (int idx = tid; idx < G * p.n_splits; idx += 256) {
            const int g = idx / p.n_splits, sp = idx - g * p.n_splits;
            const float2 ml = __ldcg(reinterpret_cast<const float2 *>(p.part_ml) + ((size_t)rrow * p.Hq + hq0 + g) * p.n_splits + sp);
            s_w[g][sp] = ml.x;
            s_l[g][sp] = ml.y;
        }
        __syncthreads();
        if (tid < G) {
            float mnew = -INFINITY;
            for (int sp = 0; sp < p.n_splits; ++sp) mnew = fmaxf(mnew, s_w[tid][sp]);
            float dsum = 0.f;
            for (int sp = 0; sp < p.n_splits; ++sp) {
                const float ms = s_w[tid][sp];
                const float cw = ms == -INFINITY ? 0.f : __expf(ms - mnew);
                s_w[tid][sp] = cw;
                dsum += s_l[tid][sp] * cw;
            }
            s_den[r][tid] = dsum;
        }
        __syncthreads();
        for (int idx = tid; idx < G * D; idx += 256) {
            const int g = idx / D, c = idx - g * D;
            const float *po = p.part_o + ((size_t)rrow * p.Hq + hq0 + g) * p.n_splits * D + c;
            float acc = 0.f;
            for (int sp = 0; sp < p.n_splits; ++sp) acc = fmaf(__ldcg(po + (size_t)sp * D), s_w[g][sp], acc);
            attn_store(p, ((size_t)rrow * p.Hq + hq0 + g) * D + c, acc / s_den[r][g]);
        }
        __syncthreads();
    }
}

}  // namespace st
