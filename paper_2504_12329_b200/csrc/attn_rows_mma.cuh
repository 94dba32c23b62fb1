// Causal attention of a multi-row pass (prompt prefill / catch-up) on mma.sync.
//
// A CTA takes the query rows [row0, row0 + RQ) of one kv head, RQ = 64 / G, i.e. up to 64 "query columns"
// (row, head of the group); each of its 8 warps owns 8 of them.  The keys and values of the CTA's key
// range travel through shared memory once, in tiles of 64 keys fetched by TMA (boxes of 16 keys x 64
// channels with the 128-byte swizzle, from the pools of the paged cache viewed as [row][D] matrices; the
// pass has already appended its own rows), four tiles in flight.  Every warp multiplies every tile with
// its own columns in the transposed form the decode kernel uses:
//     S^T[16 keys x 8 columns]  = K[16 x D] . Q^T[D x 8]         (Q as hi + lo fp16 halves)
//     O^T[D x 8 columns]       += V^T[D x 16 keys] . P^T[16 x 8]  (P^T by movmatrix)
// with the causal bound of each column (keys 0 .. pos0 + row) applied to S^T.  Few rows over a long
// context are split over the keys (grid.x); the CTA that finishes a (row tile, kv head) last merges the
// splits, each warp its own columns.
#pragma once
#include "decode_mega.cuh"

namespace st {

constexpr int kArTileKeys = 64;
constexpr int kArStages = 4;
constexpr int kArThreads = 256;

struct AttnRowsMmaParams {
    AttnParams a;
    const CUtensorMap *kmap, *vmap;   // K and V pool: [all rows][D], boxes of 16 rows x 64 channels, 128-byte swizzle
    int32_t row_base;                 // first pool row of this layer
};

template <int D>
__host__ __device__ constexpr int ar_stage_bytes() { return 2 * kArTileKeys * D * 2; }

template <int D, int G>
__global__ void __launch_bounds__(kArThreads, 1) attn_rows_mma_kernel(const AttnRowsMmaParams pp)
{
    static_assert(G >= 1 && G <= 8, "one MMA column per (row, head)");
    constexpr int KS = D / 16, NH = D / 64, RQ = 64 / G, HALF_BYTES = kArTileKeys * 128, STAGE = ar_stage_bytes<D>();
    pdl_launch();
    extern __shared__ uint8_t ar_smem[];
    __shared__ uint64_t s_full[kArStages];
    __shared__ int s_abort, s_last;
    const AttnParams &p = pp.a;
    const int m = p.desc->m, pos0 = p.desc->pos0;
    const int row0 = blockIdx.z * RQ;
    if (row0 >= m) return;   // uniform for the CTA
    const int hk = blockIdx.y, split = blockIdx.x, Hkv = p.kv.n_kv_heads;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int gq = lane >> 2, t = lane & 3;
    const uint32_t base = (smem_u32(ar_smem) + 1023u) & ~1023u;
    uint8_t *base_ptr = ar_smem + (base - smem_u32(ar_smem));

    if (tid == 0) {
        s_abort = 0;
        for (int s = 0; s < kArStages; ++s) mbar_init(smem_u32(&s_full[s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // key range of the CTA (the keys its last row sees), cut into splits of whole tiles
    const int n_keys_cta = pos0 + min(m, row0 + RQ);
    const int per = ((n_keys_cta + p.n_splits - 1) / p.n_splits + kArTileKeys - 1) / kArTileKeys * kArTileKeys;
    const int k0 = split * per, k1 = min(n_keys_cta, k0 + per);
    const int ntiles = k1 > k0 ? (k1 - k0 + kArTileKeys - 1) / kArTileKeys : 0;

    // TMA loads of tile i into its stage (first warp; one box per lane)
    auto issue = [&](int i) {
        const int s = i % kArStages;
        const int key0 = k0 + i * kArTileKeys;
        const int ng = (min(kArTileKeys, k1 - key0) + 15) >> 4;
        const int boxes = ng * NH * 2;
        const uint32_t bar = smem_u32(&s_full[s]);
        if (lane == 0) mbar_expect_tx(bar, (uint32_t)boxes * kMegaKvBoxBytes);
        __syncwarp();
        if (lane < boxes) {
            const int g = lane / (2 * NH), rem = lane - g * (2 * NH);
            const int isv = rem / NH, half = rem - isv * NH;
            const int key = key0 + g * 16;
            int page = p.kv.block_tab[key >> p.kv.page_shift];
            if ((unsigned)page >= (unsigned)p.kv.n_pages) {
                atomicOr(p.status, DEV_BAD_PAGE);
                page = 0;
            }
            const int y = pp.row_base + (page * Hkv + hk) * p.kv.page_size + (key & (p.kv.page_size - 1));
            const uint32_t dst = base + (uint32_t)s * STAGE + (uint32_t)(isv * NH + half) * HALF_BYTES + (uint32_t)g * kMegaKvBoxBytes;
            tma_load_2d(dst, isv ? pp.vmap : pp.kmap, half * 64, y, bar);
        }
    };
    if (warp == 0)
        for (int i = 0; i < min(ntiles, kArStages); ++i) issue(i);

    // this warp's 8 columns: column n = (row, head); the B fragments of Q^T belong to column gq, the
    // accumulators of S^T / O^T to columns 2 t and 2 t + 1
    auto col_row = [&](int n) { return row0 + (warp * 8 + n) / G; };
    auto col_live = [&](int n) { return warp * 8 + n < RQ * G && col_row(n) < m; };
    uint32_t qhi[KS][2], qlo[KS][2];
    {
        const bool live = col_live(gq);
        const int g = (warp * 8 + gq) % G;
        const float *qsrc = p.qkv + (size_t)(live ? col_row(gq) : 0) * (p.Hq + 2 * Hkv) * D + (size_t)(hk * G + g) * D + 2 * t;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                float2 v = make_float2(0.f, 0.f);
                if (live) v = *reinterpret_cast<const float2 *>(qsrc + 16 * ks + 8 * hf);
                const float x = v.x * p.scale, y = v.y * p.scale;
                const uint32_t h = pack_half2(x, y);
                qhi[ks][hf] = h;
                qlo[ks][hf] = pack_half2(x - kv_lo(h), y - kv_hi(h));
            }
    }
    const int lim0 = col_live(2 * t) ? pos0 + col_row(2 * t) : -1;          // last key column 2 t sees
    const int lim1 = col_live(2 * t + 1) ? pos0 + col_row(2 * t + 1) : -1;
    int warp_lim = -1;
#pragma unroll
    for (int n = 0; n < 8; ++n)
        if (col_live(n)) warp_lim = max(warp_lim, pos0 + col_row(n));

    float mrun[2] = {-INFINITY, -INFINITY}, lrun[2] = {0.f, 0.f};
    float oacc[KS][4];
#pragma unroll
    for (int mt = 0; mt < KS; ++mt)
#pragma unroll
        for (int e = 0; e < 4; ++e) oacc[mt][e] = 0.f;

    for (int i = 0; i < ntiles; ++i) {
        const int s = i % kArStages;
        const int key0 = k0 + i * kArTileKeys;
        const int nk = min(kArTileKeys, k1 - key0);
        mbar_wait(smem_u32(&s_full[s]), (uint32_t)(i / kArStages) & 1u, &s_abort, p.status);
        const uint32_t kst = base + (uint32_t)s * STAGE, vst = kst + (uint32_t)NH * HALF_BYTES;
        if (nk < kArTileKeys) {   // last tile of the range: value rows behind the last key must be finite (weight zero)
            uint8_t *vptr = base_ptr + (size_t)s * STAGE + (size_t)NH * HALF_BYTES;
            for (int idx = tid; idx < (kArTileKeys - nk) * (D / 8); idx += kArThreads) {
                const int r = nk + idx / (D / 8), c = idx % (D / 8);
                *reinterpret_cast<uint4 *>(vptr + (size_t)(c >> 3) * HALF_BYTES + (size_t)r * 128 + (c & 7) * 16) = make_uint4(0, 0, 0, 0);
            }
            __syncthreads();
        }
        const int ngroups = (nk + 15) >> 4;
        for (int gi = 0; gi < ngroups; ++gi) {
            const int r0 = gi * 16;
            if (key0 + r0 > warp_lim) break;   // causal: no column of this warp sees these keys
            float sacc[4] = {0.f, 0.f, 0.f, 0.f};
            const int krow = r0 + (lane & 7) + ((lane >> 3) & 1) * 8;
            const uint32_t ka = kst + (uint32_t)krow * 128;
            const uint32_t kx = (uint32_t)(krow & 7);
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                uint32_t a[4];
                ldmatrix_x4(a, ka + (uint32_t)(ks >> 2) * HALF_BYTES + ((((uint32_t)(ks & 3) * 2 + (uint32_t)(lane >> 4)) ^ kx) << 4));
                mma_f16_16816(sacc, a, qhi[ks][0], qhi[ks][1]);
                mma_f16_16816(sacc, a, qlo[ks][0], qlo[ks][1]);
            }
            const int kk0 = key0 + r0 + gq, kk1 = kk0 + 8;
            const bool v00 = kk0 <= lim0 && kk0 < k1, v01 = kk0 <= lim1 && kk0 < k1;
            const bool v10 = kk1 <= lim0 && kk1 < k1, v11 = kk1 <= lim1 && kk1 < k1;
            const float s0 = v00 ? sacc[0] : -INFINITY, s1 = v01 ? sacc[1] : -INFINITY;
            const float s2 = v10 ? sacc[2] : -INFINITY, s3 = v11 ? sacc[3] : -INFINITY;
            float m0 = fmaxf(s0, s2), m1 = fmaxf(s1, s3);
#pragma unroll
            for (int o = 4; o < 32; o <<= 1) {
                m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, o));
                m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, o));
            }
            const float n0 = fmaxf(mrun[0], m0), n1 = fmaxf(mrun[1], m1);   // may still be -inf (no live key yet)
            const float corr0 = mrun[0] == -INFINITY ? 0.f : __expf(mrun[0] - n0);
            const float corr1 = mrun[1] == -INFINITY ? 0.f : __expf(mrun[1] - n1);
            const float p0 = v00 ? __expf(s0 - n0) : 0.f, p1 = v01 ? __expf(s1 - n1) : 0.f;
            const float p2 = v10 ? __expf(s2 - n0) : 0.f, p3 = v11 ? __expf(s3 - n1) : 0.f;
            mrun[0] = n0;
            mrun[1] = n1;
            lrun[0] = lrun[0] * corr0 + p0 + p2;
            lrun[1] = lrun[1] * corr1 + p1 + p3;
            const uint32_t pb0 = movmatrix_trans(pack_half2(p0, p1)), pb1 = movmatrix_trans(pack_half2(p2, p3));
            const int vrow = r0 + (lane & 7) + (lane >> 4) * 8;
            const uint32_t va = vst + (uint32_t)vrow * 128;
            const uint32_t vx = (uint32_t)(vrow & 7);
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) {
                oacc[mt][0] *= corr0; oacc[mt][1] *= corr1; oacc[mt][2] *= corr0; oacc[mt][3] *= corr1;
                uint32_t a[4];
                ldmatrix_x4_trans(a, va + (uint32_t)(mt >> 2) * HALF_BYTES + ((((uint32_t)(mt & 3) * 2 + (uint32_t)((lane >> 3) & 1)) ^ vx) << 4));
                mma_f16_16816(oacc[mt], a, pb0, pb1);
            }
        }
        __syncthreads();   // every warp is done with the stage
        if (warp == 0 && i + kArStages < ntiles) issue(i + kArStages);
    }
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
        lrun[0] += __shfl_xor_sync(0xffffffffu, lrun[0], o);
        lrun[1] += __shfl_xor_sync(0xffffffffu, lrun[1], o);
    }

    const int hq0 = hk * G;
    if (p.n_splits == 1) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int n = 2 * t + e;
            if (!col_live(n)) continue;
            const int row = col_row(n), g = (warp * 8 + n) % G;
            const float inv = 1.f / lrun[e];
            const size_t o0 = ((size_t)row * p.Hq + hq0 + g) * D;
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) {
                attn_store(p, o0 + 16 * mt + gq, oacc[mt][e] * inv);
                attn_store(p, o0 + 16 * mt + gq + 8, oacc[mt][2 + e] * inv);
            }
        }
        return;
    }
    // ---- partial results of this key split ----
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int n = 2 * t + e;
        if (!col_live(n)) continue;
        const int row = col_row(n), g = (warp * 8 + n) % G;
        const size_t pi = ((size_t)row * p.Hq + hq0 + g) * p.n_splits + split;
#pragma unroll
        for (int mt = 0; mt < KS; ++mt) {
            p.part_o[pi * D + 16 * mt + gq] = oacc[mt][e];
            p.part_o[pi * D + 16 * mt + gq + 8] = oacc[mt][2 + e];
        }
        if (gq == 0) { p.part_ml[pi * 2] = mrun[e]; p.part_ml[pi * 2 + 1] = lrun[e]; }
    }
    // ---- the CTA that finishes this (row tile, kv head) last merges the splits ----
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        int *tk = p.tickets + blockIdx.z * Hkv + hk;
        const int tno = atomicAdd(tk, 1);
        s_last = (tno == p.n_splits - 1);
        if (s_last) *tk = 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    for (int n = 0; n < 8; ++n) {
        if (!col_live(n)) continue;   // uniform for the warp
        const int row = col_row(n), g = (warp * 8 + n) % G;
        const size_t pi0 = ((size_t)row * p.Hq + hq0 + g) * p.n_splits;
        float ms = -INFINITY, ls = 0.f;
        if (lane < p.n_splits) {
            const float2 ml = __ldcg(reinterpret_cast<const float2 *>(p.part_ml) + pi0 + lane);
            ms = ml.x;
            ls = ml.y;
        }
        float mmax = ms;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mmax = fmaxf(mmax, __shfl_xor_sync(0xffffffffu, mmax, o));
        const float wgt = ms == -INFINITY ? 0.f : __expf(ms - mmax);
        const float inv = 1.f / warp_sum(ls * wgt);
        constexpr int CPL = D / 32;   // channels per lane
        float acc[CPL];
#pragma unroll
        for (int c = 0; c < CPL; ++c) acc[c] = 0.f;
        for (int sp = 0; sp < p.n_splits; ++sp) {
            const float wsp = __shfl_sync(0xffffffffu, wgt, sp);
            const float *po = p.part_o + (pi0 + sp) * D + lane * CPL;
#pragma unroll
            for (int c = 0; c < CPL; ++c) acc[c] = fmaf(__ldcg(po + c), wsp, acc[c]);
        }
        const size_t o0 = ((size_t)row * p.Hq + hq0 + g) * D + lane * CPL;
#pragma unroll
        for (int c = 0; c < CPL; ++c) attn_store(p, o0 + c, acc[c] * inv);
    }
}

// ---------------------------------------------------------------------------------------------
// Batched decode attention: every row is the newest token of a different sequence.  One CTA per (kv head, row)
// walks that sequence's keys 0 .. pos in tiles of TK keys (TMA, three tiles in flight); warp w of the TK / 16 warps
// takes the w-th group of 16 keys of every tile for the G query heads of the group, and the warps are merged
// through shared memory at the end.  The row's own key/value is already in the cache (the rope kernel appended
// it).  TK = 64 (four warps, two CTAs per SM: one CTA's loads cover the other's prologue, tile hand-overs and
// merge) is what the host launches; TK = 128 (eight warps, one CTA per SM) is kept as an alternative.
// ---------------------------------------------------------------------------------------------
constexpr int kAbStages = 3;

struct AttnBatchParams {
    AttnParams a;                     // a.kv.block_tab: the block table of sequence 0
    const CUtensorMap *kmap, *vmap;
    int32_t row_base;                 // first pool row of this layer
    const int32_t *row_slot, *row_pos;
    int32_t pages_per_seq;
};

template <int D, int TK>
__host__ __device__ constexpr int ab_stage_bytes() { return 2 * TK * D * 2; }

template <int D, int G, int TK>
__global__ void __launch_bounds__(2 * TK, 1) attn_batch_mma_kernel(const AttnBatchParams pp)
{
    static_assert(G >= 1 && G <= 8, "one MMA column per head of the group");
    static_assert(TK == 64 || TK == 128, "one warp per 16 keys of a tile");
    constexpr int kAbTileKeys = TK, NT = 2 * TK, NW = TK / 16;
    constexpr int KS = D / 16, NH = D / 64, HALF_BYTES = kAbTileKeys * 128, STAGE = ab_stage_bytes<D, TK>();
    static_assert(NW * G * (D + 2) * 4 <= kAbStages * STAGE, "the merge area reuses the tile ring");
    pdl_launch();
    extern __shared__ uint8_t ab_smem[];
    __shared__ uint64_t s_full[kAbStages];
    __shared__ int s_abort;
    const AttnParams &p = pp.a;
    const int row = blockIdx.y;
    if (row >= p.desc->m) return;   // uniform for the CTA
    const int hk = blockIdx.x, Hkv = p.kv.n_kv_heads;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int gq = lane >> 2, t = lane & 3;
    const uint32_t base = (smem_u32(ab_smem) + 1023u) & ~1023u;
    uint8_t *base_ptr = ab_smem + (base - smem_u32(ab_smem));
    if (tid == 0) {
        s_abort = 0;
        for (int s = 0; s < kAbStages; ++s) mbar_init(smem_u32(&s_full[s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const int pos = pp.row_pos[row];
    const int n_keys = pos + 1;
    const int32_t *tab = p.kv.block_tab + (size_t)pp.row_slot[row] * pp.pages_per_seq;
    const int ntiles = (n_keys + kAbTileKeys - 1) / kAbTileKeys;

    auto issue = [&](int i) {
        const int s = i % kAbStages;
        const int key0 = i * kAbTileKeys;
        const int ng = (min(kAbTileKeys, n_keys - key0) + 15) >> 4;
        const int boxes = ng * NH * 2;
        const uint32_t bar = smem_u32(&s_full[s]);
        if (lane == 0) mbar_expect_tx(bar, (uint32_t)boxes * kMegaKvBoxBytes);
        __syncwarp();
        if (lane < boxes) {
            const int g = lane / (2 * NH), rem = lane - g * (2 * NH);
            const int isv = rem / NH, half = rem - isv * NH;
            const int key = key0 + g * 16;
            int page = tab[key >> p.kv.page_shift];
            if ((unsigned)page >= (unsigned)p.kv.n_pages) {
                atomicOr(p.status, DEV_BAD_PAGE);
                page = 0;
            }
            const int y = pp.row_base + (page * Hkv + hk) * p.kv.page_size + (key & (p.kv.page_size - 1));
            const uint32_t dst = base + (uint32_t)s * STAGE + (uint32_t)(isv * NH + half) * HALF_BYTES + (uint32_t)g * kMegaKvBoxBytes;
            tma_load_2d(dst, isv ? pp.vmap : pp.kmap, half * 64, y, bar);
        }
    };
    if (warp == 0)
        for (int i = 0; i < min(ntiles, kAbStages); ++i) issue(i);

    uint32_t qhi[KS][2], qlo[KS][2];
    {
        const bool live = gq < G;
        const float *qsrc = p.qkv + (size_t)row * (p.Hq + 2 * Hkv) * D + (size_t)(hk * G + (live ? gq : 0)) * D + 2 * t;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                float2 v = make_float2(0.f, 0.f);
                if (live) v = *reinterpret_cast<const float2 *>(qsrc + 16 * ks + 8 * hf);
                const float x = v.x * p.scale, y = v.y * p.scale;
                const uint32_t h = pack_half2(x, y);
                qhi[ks][hf] = h;
                qlo[ks][hf] = pack_half2(x - kv_lo(h), y - kv_hi(h));
            }
    }
    float mrun[2] = {-INFINITY, -INFINITY}, lrun[2] = {0.f, 0.f};
    float oacc[KS][4];
#pragma unroll
    for (int mt = 0; mt < KS; ++mt)
#pragma unroll
        for (int e = 0; e < 4; ++e) oacc[mt][e] = 0.f;

    for (int i = 0; i < ntiles; ++i) {
        const int s = i % kAbStages;
        const int key0 = i * kAbTileKeys;
        const int nk = min(kAbTileKeys, n_keys - key0);
        mbar_wait(smem_u32(&s_full[s]), (uint32_t)(i / kAbStages) & 1u, &s_abort, p.status);
        const uint32_t kst = base + (uint32_t)s * STAGE, vst = kst + (uint32_t)NH * HALF_BYTES;
        if (nk < kAbTileKeys) {   // last tile: value rows behind the last key of its group must be finite
            uint8_t *vptr = base_ptr + (size_t)s * STAGE + (size_t)NH * HALF_BYTES;
            const int pad = ((nk + 15) & ~15) - nk;
            for (int idx = tid; idx < pad * (D / 8); idx += NT) {
                const int r = nk + idx / (D / 8), c = idx % (D / 8);
                *reinterpret_cast<uint4 *>(vptr + (size_t)(c >> 3) * HALF_BYTES + (size_t)r * 128 + (c & 7) * 16) = make_uint4(0, 0, 0, 0);
            }
            __syncthreads();
        }
        const int r0 = warp * 16;
        if (r0 < nk) {
            float sacc[4] = {0.f, 0.f, 0.f, 0.f};
            const int krow = r0 + (lane & 7) + ((lane >> 3) & 1) * 8;
            const uint32_t ka = kst + (uint32_t)krow * 128;
            const uint32_t kx = (uint32_t)(krow & 7);
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                uint32_t a[4];
                ldmatrix_x4(a, ka + (uint32_t)(ks >> 2) * HALF_BYTES + ((((uint32_t)(ks & 3) * 2 + (uint32_t)(lane >> 4)) ^ kx) << 4));
                mma_f16_16816(sacc, a, qhi[ks][0], qhi[ks][1]);
                mma_f16_16816(sacc, a, qlo[ks][0], qlo[ks][1]);
            }
            const bool v0 = r0 + gq < nk, v1 = r0 + gq + 8 < nk;
            const float s0 = v0 ? sacc[0] : -INFINITY, s1 = v0 ? sacc[1] : -INFINITY;
            const float s2 = v1 ? sacc[2] : -INFINITY, s3 = v1 ? sacc[3] : -INFINITY;
            float m0 = fmaxf(s0, s2), m1 = fmaxf(s1, s3);
#pragma unroll
            for (int o = 4; o < 32; o <<= 1) {
                m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, o));
                m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, o));
            }
            const float n0 = fmaxf(mrun[0], m0), n1 = fmaxf(mrun[1], m1);   // finite: the group holds a live key
            const float corr0 = mrun[0] == -INFINITY ? 0.f : __expf(mrun[0] - n0);
            const float corr1 = mrun[1] == -INFINITY ? 0.f : __expf(mrun[1] - n1);
            const float p0 = v0 ? __expf(s0 - n0) : 0.f, p1 = v0 ? __expf(s1 - n1) : 0.f;
            const float p2 = v1 ? __expf(s2 - n0) : 0.f, p3 = v1 ? __expf(s3 - n1) : 0.f;
            mrun[0] = n0;
            mrun[1] = n1;
            lrun[0] = lrun[0] * corr0 + p0 + p2;
            lrun[1] = lrun[1] * corr1 + p1 + p3;
            const uint32_t pb0 = movmatrix_trans(pack_half2(p0, p1)), pb1 = movmatrix_trans(pack_half2(p2, p3));
            const int vrow = r0 + (lane & 7) + (lane >> 4) * 8;
            const uint32_t va = vst + (uint32_t)vrow * 128;
            const uint32_t vx = (uint32_t)(vrow & 7);
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) {
                oacc[mt][0] *= corr0; oacc[mt][1] *= corr1; oacc[mt][2] *= corr0; oacc[mt][3] *= corr1;
                uint32_t a[4];
                ldmatrix_x4_trans(a, va + (uint32_t)(mt >> 2) * HALF_BYTES + ((((uint32_t)(mt & 3) * 2 + (uint32_t)((lane >> 3) & 1)) ^ vx) << 4));
                mma_f16_16816(oacc[mt], a, pb0, pb1);
            }
        }
        __syncthreads();   // every warp is done with the stage
        if (warp == 0 && i + kAbStages < ntiles) issue(i + kAbStages);
    }
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
        lrun[0] += __shfl_xor_sync(0xffffffffu, lrun[0], o);
        lrun[1] += __shfl_xor_sync(0xffffffffu, lrun[1], o);
    }
    // ---- merge the warps through shared memory (the tiles are no longer needed) ----
    float *so = reinterpret_cast<float *>(base_ptr);                 // [NW warps][G][D]
    float *sm = so + NW * G * D, *sd = sm + NW * G;                  // [NW][G] each
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int head = 2 * t + e;
        if (head < G) {
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) {
                so[(warp * G + head) * D + 16 * mt + gq] = oacc[mt][e];
                so[(warp * G + head) * D + 16 * mt + gq + 8] = oacc[mt][2 + e];
            }
            if (gq == 0) { sm[warp * G + head] = mrun[e]; sd[warp * G + head] = lrun[e]; }
        }
    }
    __syncthreads();
    const int hq0 = hk * G;
    for (int idx = tid; idx < G * D; idx += NT) {
        const int g = idx / D, c = idx - g * D;
        float mnew = -INFINITY;
#pragma unroll
        for (int w = 0; w < NW; ++w) mnew = fmaxf(mnew, sm[w * G + g]);
        float dsum = 0.f, osum = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            const float mw = sm[w * G + g];
            if (mw != -INFINITY) {
                const float cw = __expf(mw - mnew);
                dsum += sd[w * G + g] * cw;
                osum += so[(w * G + g) * D + c] * cw;
            }
        }
        attn_store(p, ((size_t)row * p.Hq + hq0 + g) * D + c, osum / dsum);
    }
}

}  // namespace st
