// One decode step of one model as a single persistent kernel (batch 1).
//
// A batch-1 step is a chain of ~6 dependent phases per layer, each of which moves only a few
// microseconds' worth of HBM traffic on the small model; launched as separate kernels the chain is
// bound by launch/drain latency, not by bandwidth.  Here one CTA per SM stays resident for the whole
// step:
//   * warp 0 (producer) walks the step's weight tiles in order -- every layer's QKV, O, gate/up and
//     down matrices, then the LM head -- and streams them into a shared-memory ring with bulk
//     asynchronous copies (cp.async.bulk + mbarrier).  It never waits for a phase boundary: weights do
//     not depend on activations, so HBM keeps streaming while the other warps synchronise.
//   * warps 1..8 (consumers) multiply the tiles with the phase's input vector (fp32, shared memory),
//     4 rows per warp, fp32 accumulation, and run attention, normalisation, rotary embedding, the
//     residual stream, sampling and the handoff router in between.
//   * phases are separated by a grid-wide barrier (an atomic counter; bounded spin).
// Matrices are cut into tiles of 32 rows x 512 columns; every CTA takes an equal contiguous range of
// the tiles of a phase (so short-and-wide matrices still use all SMs) and adds its partial row sums
// into a zeroed fp32 vector with atomics; the gate/up matrix is split by whole row blocks because
// its epilogue silu(g) * u is not additive.
#pragma once
#include "attention.cuh"
#include "router.cuh"
#include "tc_gemm.cuh"

namespace st {

constexpr int kMegaConsumers = 8;
constexpr int kMegaThreads = 32 * (1 + kMegaConsumers);
constexpr int kMegaCT = 32 * kMegaConsumers;                      // consumer threads
constexpr int kMegaRowsPerWarp = 4;
constexpr int kMegaTileRows = kMegaConsumers * kMegaRowsPerWarp;  // 32
constexpr int kMegaSeg = 512;                                     // K elements per tile
constexpr int kMegaBoxBytes = kMegaTileRows * 256 * 2;            // one TMA box: 32 rows x 256 elements = 16 KB
constexpr int kMegaTileBytes = 2 * kMegaBoxBytes;                 // 32 KB: two boxes side by side in K
constexpr int kMegaMaxStages = 6;
constexpr uint32_t kMegaSpinLimit = 1u << 22;
constexpr int kMegaAttnWarps = kMegaConsumers;                    // all consumer warps work on one attention unit

struct MegaLayer {
    const uint16_t *wqkv, *wo, *wgu, *wd;
    const float *bqkv, *g1, *g2;
    uint16_t *kpool, *vpool;
};

// TMA descriptors of the weight matrices for the decode ring: boxes of 256 elements x 32 rows, no
// swizzle (a tile row is 512 contiguous bytes in shared memory), zero fill outside the matrix.
// Device array: 4 per layer (QKV, O, gate/up, down), then the LM head.
constexpr int kMegaBoxK = 256;

struct MegaParams {
    const MegaLayer *layers;
    const CUtensorMap *maps;   // [4 * n_layers + 1], global memory
    const uint16_t *embed, *lm_head;
    const float *gf;
    const double *inv_freq;
    const StepDesc *desc;
    const int32_t *tok;
    KvView kv;                // block table and page geometry; k/v pools come per layer from `layers`
    float *X0, *X1;           // residual stream before attention / before the FFN
    float *QKV, *ATT, *D1, *D2, *ACT;
    float *logits;            // [vocab]
    float *part_o, *part_ml;  // attention split partials [Hq][n_splits][D], [Hq][n_splits][2]
    int32_t *tickets;         // [Hkv] attention tickets, zero between launches
    unsigned *sync;           // [1] exit tickets, [2] abort flag, [3] argmax tickets, [32 * (1 + i)] barrier counter i < 8
    int32_t *status;
    int32_t n_layers, h, Hq, Hkv, f, vocab, n_splits, stages, xarea_bytes;
    float eps, scale;
    // sampling
    int32_t want_argmax, limit;
    float *part_val;
    int32_t *part_idx;
    int32_t *argmax_out;
    GenState *gen;
    GenBuffers buf;
    StepDesc *desc_small, *desc_large;
};

__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kMegaCT) : "memory"); }
constexpr int kMegaAttnUK = 4;   // key steps in flight per lane

// First batch of cached keys/values of an attention unit, fetched before the grid barrier that
// precedes the attention phase (cached K/V do not depend on this layer's QKV).
struct MegaKvPrefetch {
    uint4 kf[kMegaAttnUK], vf[kMegaAttnUK];
    bool ok[kMegaAttnUK];
};

// The weight matrix of weight phase idx: 4 per layer (QKV, O, gate/up, down), then the LM head.
struct MegaPhase {
    const uint16_t *W;
    int N, K;
    bool whole_blocks;
};
template <int D>
__device__ __forceinline__ MegaPhase mega_phase(const MegaParams &p, int idx)
{
    MegaPhase ph;
    const int qd = p.Hq * D, kd = p.Hkv * D;
    if (idx == 4 * p.n_layers) {
        ph.W = p.lm_head; ph.N = p.vocab; ph.K = p.h; ph.whole_blocks = false;
        return ph;
    }
    const MegaLayer &L = p.layers[idx >> 2];
    switch (idx & 3) {
    case 0: ph.W = L.wqkv; ph.N = qd + 2 * kd; ph.K = p.h; ph.whole_blocks = false; break;
    case 1: ph.W = L.wo; ph.N = p.h; ph.K = qd; ph.whole_blocks = false; break;
    case 2: ph.W = L.wgu; ph.N = 2 * p.f; ph.K = p.h; ph.whole_blocks = true; break;
    default: ph.W = L.wd; ph.N = p.h; ph.K = p.f; ph.whole_blocks = false; break;
    }
    return ph;
}

// Tiles [t0, t1) of a phase for this CTA; tile t = (row block t / nseg, K segment t % nseg).
__device__ __forceinline__ void mega_range(const MegaPhase &ph, int cta, int n_cta, int &t0, int &t1, int &nseg)
{
    const int nblk = (ph.N + kMegaTileRows - 1) / kMegaTileRows;
    nseg = (ph.K + kMegaSeg - 1) / kMegaSeg;
    if (ph.whole_blocks) {
        t0 = (int)((long long)cta * nblk / n_cta) * nseg;
        t1 = (int)((long long)(cta + 1) * nblk / n_cta) * nseg;
    } else {
        const long long T = (long long)nblk * nseg;
        t0 = (int)((long long)cta * T / n_cta);
        t1 = (int)((long long)(cta + 1) * T / n_cta);
    }
}

// Optional phase timeline (compiled in with -DST_MEGA_TRACE): CTA 0 stamps the global timer at every
// phase boundary of the step.
#ifdef ST_MEGA_TRACE
__device__ unsigned long long g_mega_trace[8192];
#define MEGA_MARK()                                                         \
    do {                                                                    \
        if (blockIdx.x == 0 && ctid == 0 && trace_i < 8192) {               \
            unsigned long long t_;                                          \
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));          \
            g_mega_trace[trace_i++] = t_;                                   \
        }                                                                   \
    } while (0)
#else
#define MEGA_MARK() do { } while (0)
#endif

struct MegaShared {
    uint64_t full[kMegaMaxStages], empty[kMegaMaxStages];
    float red[kMegaConsumers];
    float2 cs[64];          // rotary table of this step's position
    float s_v[kMegaConsumers];
    int s_i[kMegaConsumers];
    int last[2];
    int abort;
};

template <int D, int G>
struct MegaAttnScratch {   // per attention unit (4 warps)
    float o[kMegaAttnWarps][G][D];
    float m[kMegaAttnWarps][G], d[kMegaAttnWarps][G];
    float w[G][kMaxAttnSplits], l[G][kMaxAttnSplits];
    float den[G];
};

// Grid-wide barrier over the consumer warps of all CTAs, in two halves so that work which does not depend on
// the other CTAs can be slotted between "I am done" and "everybody is done".  When the bounded wait runs out
// it raises the abort flag (which every later wait honours at once); control flow stays uniform.
// The arrivals are spread over kMegaBarCounters counters on separate 128-byte lines (CTA c adds to counter
// c % 8): same-address atomics are served one after the other, and 148 of them in a row were a visible
// part of the barrier's latency.  Lanes 0..7 of the first consumer warp each watch one counter.
constexpr int kMegaBarCounters = 8;
__device__ __forceinline__ unsigned *mega_bar_counter(const MegaParams &p, int i) { return p.sync + 32 * (1 + i); }

__device__ __forceinline__ void mega_barrier_arrive(const MegaParams &p, int ctid)
{
    consumer_sync();
    // release-add: no return value to wait for
    if (ctid == 0)
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(mega_bar_counter(p, blockIdx.x % kMegaBarCounters)) : "memory");
}
__device__ __forceinline__ bool mega_barrier_wait(const MegaParams &p, MegaShared &sh, unsigned &epoch, int ctid)
{
    ++epoch;
    if (ctid < 32) {
        const int i = ctid < kMegaBarCounters ? ctid : 0;
        // CTAs that add to counter i: those with index congruent to i
        const unsigned members = (gridDim.x - i + kMegaBarCounters - 1) / kMegaBarCounters;
        const unsigned target = epoch * members;
        const unsigned *ctr = mega_bar_counter(p, i);
        bool ok = false;
        for (uint32_t it = 0; it < kMegaSpinLimit; ++it) {
            const bool mine = ctid >= kMegaBarCounters || ld_acquire_u32(ctr) >= target;
            if (__all_sync(0xffffffffu, mine)) { ok = true; break; }
            if ((it & 63) == 63 && __any_sync(0xffffffffu, ld_acquire_u32(&p.sync[2]) != 0)) break;
            if (it > 256) __nanosleep(32);
        }
        if (!ok && ctid == 0) {
            atomicExch(&p.sync[2], 1u);
            atomicOr(p.status, DEV_WAIT_EXPIRED);
            sh.abort = 1;
        }
    }
    consumer_sync();
    return sh.abort == 0;
}
__device__ __forceinline__ bool mega_grid_barrier(const MegaParams &p, MegaShared &sh, unsigned &epoch, int ctid)
{
    mega_barrier_arrive(p, ctid);
    return mega_barrier_wait(p, sh, epoch, ctid);
}

// x (+ add) -> shared memory, optionally normalised; CTA 0 writes the sum back to x_out.
// src_embed: bf16 embedding row (layer 0) instead of fp32 x.
__device__ __forceinline__ void mega_load_x(MegaShared &sh, float4 *xa, float4 *xb, int K, const float *x, const float *add,
                                            const uint16_t *src_embed, float *x_out, const float *gain, float eps, bool norm,
                                            int ctid, int cw, int lane)
{
    const int K8 = K >> 3;
    float ss = 0.f;
    constexpr int XU = 4;   // loads in flight per thread
    for (int q0 = ctid; q0 < 2 * K8; q0 += XU * kMegaCT) {
        float4 v[XU], a[XU];
#pragma unroll
        for (int u = 0; u < XU; ++u) {
            const int q = q0 + u * kMegaCT;
            v[u] = a[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (q < 2 * K8) {
                if (src_embed) {
                    const uint2 e = reinterpret_cast<const uint2 *>(src_embed)[q];
                    v[u] = make_float4(bf16_lo(e.x), bf16_hi(e.x), bf16_lo(e.y), bf16_hi(e.y));
                } else {
                    v[u] = __ldcg(reinterpret_cast<const float4 *>(x) + q);
                }
                if (add) a[u] = __ldcg(reinterpret_cast<const float4 *>(add) + q);
            }
        }
#pragma unroll
        for (int u = 0; u < XU; ++u) {
            const int q = q0 + u * kMegaCT;
            if (q < 2 * K8) {
                float4 t = v[u];
                t.x += a[u].x; t.y += a[u].y; t.z += a[u].z; t.w += a[u].w;
                if (x_out && blockIdx.x == 0) reinterpret_cast<float4 *>(x_out)[q] = t;
                ss += t.x * t.x + t.y * t.y + t.z * t.z + t.w * t.w;
                ((q & 1) ? xb : xa)[q >> 1] = t;
            }
        }
    }
    if (norm) {
        ss = warp_sum(ss);
        if (lane == 0) sh.red[cw] = ss;
        consumer_sync();
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < kMegaConsumers; ++w) tot += sh.red[w];
        const float inv = rsqrtf(tot / (float)K + eps);
        const float4 *g4 = reinterpret_cast<const float4 *>(gain);
        for (int q = ctid; q < 2 * K8; q += kMegaCT) {
            float4 *dst = ((q & 1) ? xb : xa) + (q >> 1);
            float4 v = *dst;
            const float4 g = g4[q];
            v.x *= inv * g.x; v.y *= inv * g.y; v.z *= inv * g.z; v.w *= inv * g.w;
            *dst = v;
        }
    }
    consumer_sync();
}

enum { MEPI_ADD = 0, MEPI_SILU = 1 };

// Consume this CTA's tiles of one weight phase.  out: MEPI_ADD -> out[row] += partial (+ bias with the
// first K segment); MEPI_SILU -> out[row / 2] = silu(row 2j) * row 2j+1 (whole row blocks only).
template <int EPI>
__device__ __forceinline__ bool mega_run_tiles(const MegaParams &p, MegaShared &sh, const MegaPhase &ph, uint32_t ring,
                                               const float4 *xa, const float4 *xb, float *out, const float *bias,
                                               unsigned &it, int cw, int lane)
{
    int t0, t1, nseg;
    mega_range(ph, blockIdx.x, gridDim.x, t0, t1, nseg);
    float acc[kMegaRowsPerWarp], acc2[kMegaRowsPerWarp];
#pragma unroll
    for (int r = 0; r < kMegaRowsPerWarp; ++r) acc[r] = acc2[r] = 0.f;
    bool first_seg_seen = false;
    for (int t = t0; t < t1; ++t, ++it) {
        const int slot = it % p.stages, u = it / p.stages;
        const int rb = t / nseg, seg = t - rb * nseg;
        if (seg == 0 || t == t0) first_seg_seen = (seg == 0);
        const int k0 = seg * kMegaSeg;
        // after an expired wait every later wait returns at once: the step runs to its end (with a
        // status bit set) instead of leaving warps behind at a barrier
        mbar_wait(smem_u32(&sh.full[slot]), u & 1, &sh.abort, p.status);
        const uint32_t tile = ring + (uint32_t)slot * kMegaTileBytes + (uint32_t)(cw * kMegaRowsPerWarp) * (kMegaBoxK * 2);
        // all weight loads of the tile first (8 x 16 bytes per lane), then the multiplies: two
        // independent accumulation chains per row
        uint4 w[kMegaSeg / kMegaBoxK][kMegaRowsPerWarp];
#pragma unroll
        for (int c = 0; c < kMegaSeg / kMegaBoxK; ++c)
#pragma unroll
            for (int r = 0; r < kMegaRowsPerWarp; ++r)
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                             : "=r"(w[c][r].x), "=r"(w[c][r].y), "=r"(w[c][r].z), "=r"(w[c][r].w)
                             : "r"(tile + (uint32_t)c * kMegaBoxBytes + (uint32_t)r * (kMegaBoxK * 2) + (uint32_t)lane * 16));
#pragma unroll
        for (int c = 0; c < kMegaSeg / kMegaBoxK; ++c) {
            const int e = c * kMegaBoxK + lane * 8;
            if (k0 + e < ph.K) {
                const float4 a = xa[(k0 + e) >> 3], b = xb[(k0 + e) >> 3];
#pragma unroll
                for (int r = 0; r < kMegaRowsPerWarp; ++r) {
                    const uint4 v = w[c][r];
                    float s0 = acc[r], s1 = acc2[r];
                    s0 = fmaf(bf16_lo(v.x), a.x, s0); s1 = fmaf(bf16_hi(v.x), a.y, s1);
                    s0 = fmaf(bf16_lo(v.y), a.z, s0); s1 = fmaf(bf16_hi(v.y), a.w, s1);
                    s0 = fmaf(bf16_lo(v.z), b.x, s0); s1 = fmaf(bf16_hi(v.z), b.y, s1);
                    s0 = fmaf(bf16_lo(v.w), b.z, s0); s1 = fmaf(bf16_hi(v.w), b.w, s1);
                    acc[r] = s0;
                    acc2[r] = s1;
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sh.empty[slot]));
        if (seg == nseg - 1 || t == t1 - 1) {
            // close this CTA's share of the row block
#pragma unroll
            for (int r = 0; r < kMegaRowsPerWarp; ++r) acc[r] = warp_sum(acc[r] + acc2[r]);
            const int row0 = rb * kMegaTileRows + cw * kMegaRowsPerWarp;
            if (EPI == MEPI_SILU) {
                if (lane < kMegaRowsPerWarp / 2) {
                    const int row = row0 + 2 * lane;
                    if (row + 1 < ph.N) {
                        const float g = lane == 0 ? acc[0] : acc[2], uu = lane == 0 ? acc[1] : acc[3];
                        out[row >> 1] = g / (1.f + expf(-g)) * uu;
                    }
                }
            } else if (lane < kMegaRowsPerWarp) {
                const int row = row0 + lane;
                if (row < ph.N) {
                    float v = lane == 0 ? acc[0] : lane == 1 ? acc[1] : lane == 2 ? acc[2] : acc[3];
                    if (bias && first_seg_seen) v += bias[row];
                    atomicAdd(out + row, v);
                }
            }
#pragma unroll
            for (int r = 0; r < kMegaRowsPerWarp; ++r) acc[r] = acc2[r] = 0.f;
            first_seg_seen = false;
        }
    }
    return true;
}

// Key range of split `split` of `n_splits` over keys 0..pos.
__device__ __forceinline__ void mega_split_range(int pos, int split, int n_splits, int &k0, int &k1)
{
    const int n_keys = pos + 1;
    const int per = (n_keys + n_splits - 1) / n_splits;
    k0 = split * per;
    k1 = min(n_keys, k0 + per);
}

template <int D>
__device__ __forceinline__ void mega_attention_prefetch(const MegaParams &p, const KvView &kv, int hk, int split, int n_splits,
                                                        int pos, int cw, int lane, MegaKvPrefetch &pf)
{
    constexpr int LPK = D / 8, KPW = 32 / LPK;
    const int sub = lane / LPK, ch = (lane % LPK) * 8;
    int k0, k1;
    mega_split_range(pos, split, n_splits, k0, k1);
    const int k1c = min(k1, pos);
    const int base = k0 + (cw * kMegaAttnUK) * KPW;
#pragma unroll
    for (int u = 0; u < kMegaAttnUK; ++u) {
        const int key = base + u * KPW + sub;
        pf.ok[u] = key < k1c;
        if (pf.ok[u]) {
            const size_t off = kv_offset(kv, key, hk, D, p.status) + ch;
            pf.kf[u] = __ldcg(reinterpret_cast<const uint4 *>(kv.k + off));
            pf.vf[u] = __ldcg(reinterpret_cast<const uint4 *>(kv.v + off));
        } else {
            pf.kf[u] = make_uint4(0, 0, 0, 0);
            pf.vf[u] = make_uint4(0, 0, 0, 0);
        }
    }
}

// Attention of one (kv head, key split) unit by the CTA's consumer warps: rotary embedding of q on the
// fly, cached keys [k0, k1) (the first batch already in registers), and the step's own key/value
// (position pos) taken from the QKV vector by the split that owns it, which also appends them to the
// cache.  Partials go to part_o / part_ml; the unit that finishes last for its kv head merges the
// splits into ATT.
template <int D, int G>
__device__ __forceinline__ void mega_attention_unit(const MegaParams &p, MegaShared &sh, MegaAttnScratch<D, G> &sc,
                                                    const KvView &kv, int hk, int split, int n_splits, int pos, int cw, int lane,
                                                    MegaKvPrefetch &pf)
{
    constexpr int LPK = D / 8, KPW = 32 / LPK, UK = kMegaAttnUK, half = D / 2;
    const int gt = cw * 32 + lane;                  // thread within the unit
    const int sub = lane / LPK, ch = (lane % LPK) * 8;
    int k0, k1;
    mega_split_range(pos, split, n_splits, k0, k1);
    const int k1c = min(k1, pos);                   // cached keys only
    // rotate 8 channels starting at ch of a head vector v (fp32, unrotated) at this step's position
    auto rotated8 = [&](const float *v, float *out8) {
        const int other = ch < half ? ch + half : ch - half;
        const int j0 = ch < half ? ch : ch - half;
        const float4 m0 = __ldcg(reinterpret_cast<const float4 *>(v + ch)), m1 = __ldcg(reinterpret_cast<const float4 *>(v + ch + 4));
        const float4 o0 = __ldcg(reinterpret_cast<const float4 *>(v + other)), o1 = __ldcg(reinterpret_cast<const float4 *>(v + other + 4));
        const float mine[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
        const float oth[8] = {o0.x, o0.y, o0.z, o0.w, o1.x, o1.y, o1.z, o1.w};
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float2 t = sh.cs[j0 + e];
            out8[e] = ch < half ? mine[e] * t.x - oth[e] * t.y : mine[e] * t.x + oth[e] * t.y;
        }
    };
    float q[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        rotated8(p.QKV + (size_t)(hk * G + g) * D, q[g]);
#pragma unroll
        for (int e = 0; e < 8; ++e) q[g][e] *= p.scale;
    }
    float mx[G], den[G], o[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        mx[g] = -INFINITY;
        den[g] = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) o[g][e] = 0.f;
    }
    auto update = [&](const float *kk, const float *vv, bool ok) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float s = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) s = fmaf(q[g][e], kk[e], s);
#pragma unroll
            for (int off = LPK / 2; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
            if (ok) {
                const float mnew = fmaxf(mx[g], s);
                const float corr = __expf(mx[g] - mnew), pw = __expf(s - mnew);
                den[g] = den[g] * corr + pw;
#pragma unroll
                for (int e = 0; e < 8; ++e) o[g][e] = fmaf(pw, vv[e], o[g][e] * corr);
                mx[g] = mnew;
            }
        }
    };
    for (int base = k0 + (cw * UK) * KPW; base < k1c; base += kMegaAttnWarps * UK * KPW) {
        if (base != k0 + (cw * UK) * KPW) {   // later batches; the first one was fetched ahead of the barrier
#pragma unroll
            for (int u = 0; u < UK; ++u) {
                const int key = base + u * KPW + sub;
                pf.ok[u] = key < k1c;
                if (pf.ok[u]) {
                    const size_t off = kv_offset(kv, key, hk, D, p.status) + ch;
                    pf.kf[u] = __ldcg(reinterpret_cast<const uint4 *>(kv.k + off));
                    pf.vf[u] = __ldcg(reinterpret_cast<const uint4 *>(kv.v + off));
                } else {
                    pf.kf[u] = make_uint4(0, 0, 0, 0);
                    pf.vf[u] = make_uint4(0, 0, 0, 0);
                }
            }
        }
        // scores of the whole batch first (independent chains), then one softmax update per head
        float sc_[UK][G];
#pragma unroll
        for (int u = 0; u < UK; ++u) {
            const float kk[8] = {kv_lo(pf.kf[u].x), kv_hi(pf.kf[u].x), kv_lo(pf.kf[u].y), kv_hi(pf.kf[u].y),
                                 kv_lo(pf.kf[u].z), kv_hi(pf.kf[u].z), kv_lo(pf.kf[u].w), kv_hi(pf.kf[u].w)};
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float t = 0.f;
#pragma unroll
                for (int e = 0; e < 8; ++e) t = fmaf(q[g][e], kk[e], t);
                sc_[u][g] = t;
            }
        }
#pragma unroll
        for (int off = LPK / 2; off > 0; off >>= 1)
#pragma unroll
            for (int u = 0; u < UK; ++u)
#pragma unroll
                for (int g = 0; g < G; ++g) sc_[u][g] += __shfl_xor_sync(0xffffffffu, sc_[u][g], off);
        float vv[UK][8];
#pragma unroll
        for (int u = 0; u < UK; ++u) {
            vv[u][0] = kv_lo(pf.vf[u].x); vv[u][1] = kv_hi(pf.vf[u].x); vv[u][2] = kv_lo(pf.vf[u].y); vv[u][3] = kv_hi(pf.vf[u].y);
            vv[u][4] = kv_lo(pf.vf[u].z); vv[u][5] = kv_hi(pf.vf[u].z); vv[u][6] = kv_lo(pf.vf[u].w); vv[u][7] = kv_hi(pf.vf[u].w);
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float mnew = mx[g];
#pragma unroll
            for (int u = 0; u < UK; ++u)
                if (pf.ok[u]) mnew = fmaxf(mnew, sc_[u][g]);
            if (mnew > -INFINITY) {
                const float corr = mx[g] == -INFINITY ? 0.f : __expf(mx[g] - mnew);
                den[g] *= corr;
#pragma unroll
                for (int e = 0; e < 8; ++e) o[g][e] *= corr;
#pragma unroll
                for (int u = 0; u < UK; ++u) {
                    if (pf.ok[u]) {
                        const float pw = __expf(sc_[u][g] - mnew);
                        den[g] += pw;
#pragma unroll
                        for (int e = 0; e < 8; ++e) o[g][e] = fmaf(pw, vv[u][e], o[g][e]);
                    }
                }
                mx[g] = mnew;
            }
        }
    }
    if (k0 <= pos && pos < k1 && cw == 0) {
        // this step's own key/value: rotate k, round both to fp16 (what the cache holds), append, attend
        float kk[8], vv[8];
        rotated8(p.QKV + (size_t)(p.Hq + hk) * D, kk);
        const float *vsrc = p.QKV + (size_t)(p.Hq + p.Hkv + hk) * D + ch;
        const float4 v0 = __ldcg(reinterpret_cast<const float4 *>(vsrc)), v1 = __ldcg(reinterpret_cast<const float4 *>(vsrc + 4));
        const float vraw[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
        uint32_t kb[4], vb[4];
#pragma unroll
        for (int e = 0; e < 8; e += 2) {
            kb[e >> 1] = (uint32_t)kv_bits(kk[e]) | ((uint32_t)kv_bits(kk[e + 1]) << 16);
            vb[e >> 1] = (uint32_t)kv_bits(vraw[e]) | ((uint32_t)kv_bits(vraw[e + 1]) << 16);
            kk[e] = kv_lo(kb[e >> 1]); kk[e + 1] = kv_hi(kb[e >> 1]);
            vv[e] = kv_lo(vb[e >> 1]); vv[e + 1] = kv_hi(vb[e >> 1]);
        }
        if (sub == 0) {
            const size_t off = kv_offset(kv, pos, hk, D, p.status) + ch;
            *reinterpret_cast<uint4 *>(kv.k + off) = make_uint4(kb[0], kb[1], kb[2], kb[3]);
            *reinterpret_cast<uint4 *>(kv.v + off) = make_uint4(vb[0], vb[1], vb[2], vb[3]);
        }
        update(kk, vv, sub == 0);
    }
    // ---- merge lane groups, then the warps ----
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
    if (sub == 0) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
#pragma unroll
            for (int e = 0; e < 8; ++e) sc.o[cw][g][ch + e] = o[g][e];
            if (lane == 0) { sc.m[cw][g] = mx[g]; sc.d[cw][g] = den[g]; }
        }
    }
    consumer_sync();
    const int hq0 = hk * G;
    for (int idx = gt; idx < G * D; idx += kMegaCT) {
        const int g = idx / D, c = idx - g * D;
        float mnew = -INFINITY;
#pragma unroll
        for (int w = 0; w < kMegaAttnWarps; ++w) mnew = fmaxf(mnew, sc.m[w][g]);
        float dsum = 0.f, osum = 0.f;
#pragma unroll
        for (int w = 0; w < kMegaAttnWarps; ++w) {
            const float cw2 = sc.m[w][g] == -INFINITY ? 0.f : __expf(sc.m[w][g] - mnew);
            dsum += sc.d[w][g] * cw2;
            osum += sc.o[w][g][c] * cw2;
        }
        const size_t pi = (size_t)(hq0 + g) * n_splits + split;
        if (n_splits == 1) {
            p.ATT[(size_t)(hq0 + g) * D + c] = osum / dsum;   // a single split is the final result
        } else {
            p.part_o[pi * D + c] = osum;
            if (c == 0) { p.part_ml[pi * 2] = mnew; p.part_ml[pi * 2 + 1] = dsum; }
        }
    }
}

// Merge of the key splits, spread over all CTAs (runs between two grid barriers): CTA c owns a
// contiguous range of the Hq * D output channels; 16 threads share one channel and stride the splits.
template <int D, int G>
__device__ __forceinline__ void mega_attention_merge(const MegaParams &p, MegaAttnScratch<D, G> &sc, int n_splits, int ctid)
{
    constexpr int TPO = 16;
    const int n_out = p.Hq * D;
    const int per = (n_out + gridDim.x - 1) / gridDim.x;
    const int o0 = blockIdx.x * per, o1 = min(n_out, o0 + per);
    if (o0 >= o1) return;   // uniform for the CTA
    float *w = &sc.w[0][0], *l = &sc.l[0][0];
    for (int hq = o0 / D; hq <= (o1 - 1) / D; ++hq) {
        for (int sp = ctid; sp < n_splits; sp += kMegaCT) {
            const float2 ml = __ldcg(reinterpret_cast<const float2 *>(p.part_ml) + (size_t)hq * n_splits + sp);
            w[sp] = ml.x;
            l[sp] = ml.y;
        }
        consumer_sync();
        if (ctid < 32) {
            float mnew = -INFINITY;
            for (int sp = ctid; sp < n_splits; sp += 32) mnew = fmaxf(mnew, w[sp]);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mnew = fmaxf(mnew, __shfl_xor_sync(0xffffffffu, mnew, o));
            float dsum = 0.f;
            for (int sp = ctid; sp < n_splits; sp += 32) {
                const float ms = w[sp];
                const float cw2 = ms == -INFINITY ? 0.f : __expf(ms - mnew);
                w[sp] = cw2;
                dsum += l[sp] * cw2;
            }
            dsum = warp_sum(dsum);
            if (ctid == 0) sc.den[0] = dsum;
        }
        consumer_sync();
        const int lo = max(o0, hq * D), hi = min(o1, (hq + 1) * D);
        const int j = ctid % TPO;
        const int n_pass = (hi - lo + kMegaCT / TPO - 1) / (kMegaCT / TPO);   // the same for every thread
        for (int pass = 0; pass < n_pass; ++pass) {
            const int oi = lo + pass * (kMegaCT / TPO) + ctid / TPO;
            const bool live = oi < hi;
            const int c = (live ? oi : lo) - hq * D;
            const float *po = p.part_o + (size_t)hq * n_splits * D + c;
            float acc = 0.f;
            if (live)
                for (int sp = j; sp < n_splits; sp += TPO) acc = fmaf(__ldcg(po + (size_t)sp * D), w[sp], acc);
#pragma unroll
            for (int o = TPO / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            if (live && j == 0) p.ATT[(size_t)hq * D + c] = acc / sc.den[0];
        }
        consumer_sync();
    }
}

__device__ __forceinline__ void mega_zero(float *buf, int n, int ctid)
{
    // this CTA's share of a vector
    if ((reinterpret_cast<uintptr_t>(buf) & 15) == 0 && (n & 3) == 0) {
        const int n4 = n >> 2;
        const int per = (n4 + gridDim.x - 1) / gridDim.x;
        const int b = blockIdx.x * per, e = min(n4, b + per);
        for (int i = b + ctid; i < e; i += kMegaCT) reinterpret_cast<float4 *>(buf)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    } else {
        const int per = (n + gridDim.x - 1) / gridDim.x;
        const int b = blockIdx.x * per, e = min(n, b + per);
        for (int i = b + ctid; i < e; i += kMegaCT) buf[i] = 0.f;
    }
}

template <int D, int G>
__global__ void __launch_bounds__(kMegaThreads, 1) decode_mega_kernel(const MegaParams p)
{
    extern __shared__ uint8_t mega_smem[];
    __shared__ MegaShared sh;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t base = (smem_u32(mega_smem) + 1023u) & ~1023u;
    uint8_t *base_ptr = mega_smem + (base - smem_u32(mega_smem));
    const uint32_t ring = base + (uint32_t)p.xarea_bytes;
    const int n_phases = 4 * p.n_layers + 1;

    if (tid == 0) {
        sh.abort = 0;
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&sh.full[s]), 1);
            mbar_init(smem_u32(&sh.empty[s]), kMegaConsumers);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == 0) {
        // ------------------------------ producer ------------------------------
        unsigned it = 0;
        bool ok = true;
        for (int idx = 0; idx < n_phases && ok; ++idx) {
            const MegaPhase ph = mega_phase<D>(p, idx);
            int t0, t1, nseg;
            mega_range(ph, blockIdx.x, gridDim.x, t0, t1, nseg);
            for (int t = t0; t < t1 && ok; ++t, ++it) {
                const int slot = it % p.stages, u = it / p.stages;
                if (u > 0) {
                    int w_ok = lane == 0 ? (int)mbar_wait(smem_u32(&sh.empty[slot]), (u - 1) & 1, &sh.abort, p.status) : 1;
                    w_ok = __shfl_sync(0xffffffffu, w_ok, 0);
                    if (!w_ok) { ok = false; break; }
                }
                const int rb = t / nseg, seg = t - rb * nseg;
                const int r0 = rb * kMegaTileRows, k0 = seg * kMegaSeg;
                if (lane == 0) {
                    const uint32_t full = smem_u32(&sh.full[slot]);
                    const uint32_t dst = ring + (uint32_t)slot * kMegaTileBytes;
                    const bool two = k0 + kMegaBoxK < ph.K;     // the second box lies inside the matrix
                    mbar_expect_tx(full, two ? kMegaTileBytes : kMegaBoxBytes);
                    tma_load_2d(dst, p.maps + idx, k0, r0, full);
                    if (two) tma_load_2d(dst + kMegaBoxBytes, p.maps + idx, k0 + kMegaBoxK, r0, full);
                }
                __syncwarp();
            }
        }
        if (!ok && lane == 0) {
            // give copies already in flight a bounded time to land before the CTA leaves
            for (int s = 0; s < p.stages; ++s)
                for (uint32_t w = 0; w < (1u << 14) && !mbar_try(smem_u32(&sh.full[s]), 0) && !mbar_try(smem_u32(&sh.full[s]), 1); ++w)
                    __nanosleep(128);
        }
        return;
    }

    // ------------------------------ consumers ------------------------------
    const int ctid = tid - 32, cw = warp - 1;
    float4 *xa = reinterpret_cast<float4 *>(base_ptr);
    const int pos = p.desc->pos0;
    const int qd = p.Hq * D, kd = p.Hkv * D, qkvd = qd + 2 * kd;
    unsigned epoch = 0, it = 0;
    int trace_i = 0;
    (void)trace_i;
    MEGA_MARK();
    auto xb_of = [&](int K) { return xa + (K >> 3); };

    // step set-up: rotary table, zeroed accumulation vectors
    for (int j = ctid; j < D / 2; j += kMegaCT) {
        double s, c;
        sincos((double)pos * p.inv_freq[j], &s, &c);
        sh.cs[j] = make_float2((float)c, (float)s);
    }
    mega_zero(p.QKV, qkvd, ctid);
    mega_zero(p.D1, p.h, ctid);
    mega_zero(p.D2, p.h, ctid);
    mega_zero(p.logits, p.vocab, ctid);
    mega_grid_barrier(p, sh, epoch, ctid);
    MEGA_MARK();

    int tokid = p.tok[p.desc->tok_off];
    if ((unsigned)tokid >= (unsigned)p.vocab) {
        if (ctid == 0) atomicOr(p.status, DEV_BAD_TOKEN);
        tokid = 0;
    }
    KvView kv = p.kv;
    MegaAttnScratch<D, G> *scratch = reinterpret_cast<MegaAttnScratch<D, G> *>(base_ptr);

    for (int l = 0; l < p.n_layers; ++l) {
        const MegaLayer &L = p.layers[l];
        // ---- QKV: x = (layer 0 ? embedding : x1 + down), normalised ----
        if (l > 0) mega_grid_barrier(p, sh, epoch, ctid);
        MEGA_MARK();
        mega_load_x(sh, xa, xb_of(p.h), p.h, p.X1, l > 0 ? p.D2 : nullptr, l == 0 ? p.embed + (size_t)tokid * p.h : nullptr, p.X0,
                    L.g1, p.eps, true, ctid, cw, lane);
    MEGA_MARK();
        mega_run_tiles<MEPI_ADD>(p, sh, mega_phase<D>(p, 4 * l), ring, xa, xb_of(p.h), p.QKV, L.bqkv, it, cw, lane);
    MEGA_MARK();
        // ---- attention: one (kv head, key split) unit per CTA; its first keys are fetched before the barrier ----
        kv.k = L.kpool;
        kv.v = L.vpool;
        // 64 keys per unit while there are CTAs to spare (every CTA derives the same split count)
        int ns = (pos + 64) / 64;
        ns = min(ns, min(p.n_splits, max(1, (int)gridDim.x / p.Hkv)));
        const bool attn_active = (int)blockIdx.x < p.Hkv * ns;
        const int a_hk = blockIdx.x / ns, a_split = blockIdx.x - a_hk * ns;
        MegaKvPrefetch pf;
        mega_barrier_arrive(p, ctid);
        if (attn_active) mega_attention_prefetch<D>(p, kv, a_hk, a_split, ns, pos, cw, lane, pf);
        mega_barrier_wait(p, sh, epoch, ctid);
    MEGA_MARK();
        mega_zero(p.D2, p.h, ctid);
        if (attn_active) mega_attention_unit<D, G>(p, sh, scratch[0], kv, a_hk, a_split, ns, pos, cw, lane, pf);
        MEGA_MARK();
        if (ns > 1) {   // uniform over the grid: ns depends on the position only
            mega_grid_barrier(p, sh, epoch, ctid);
            MEGA_MARK();
            mega_attention_merge<D, G>(p, scratch[0], ns, ctid);
            MEGA_MARK();
        }
        mega_grid_barrier(p, sh, epoch, ctid);
    MEGA_MARK();
        // ---- O projection into D1 ----
        mega_load_x(sh, xa, xb_of(qd), qd, p.ATT, nullptr, nullptr, nullptr, nullptr, 0.f, false, ctid, cw, lane);
    MEGA_MARK();
        mega_run_tiles<MEPI_ADD>(p, sh, mega_phase<D>(p, 4 * l + 1), ring, xa, xb_of(qd), p.D1, nullptr, it, cw, lane);
    MEGA_MARK();
        mega_grid_barrier(p, sh, epoch, ctid);
    MEGA_MARK();
        // ---- gate/up: x1 = x0 + D1, normalised ----
        mega_load_x(sh, xa, xb_of(p.h), p.h, p.X0, p.D1, nullptr, p.X1, L.g2, p.eps, true, ctid, cw, lane);
    MEGA_MARK();
        mega_zero(p.QKV, qkvd, ctid);
        mega_run_tiles<MEPI_SILU>(p, sh, mega_phase<D>(p, 4 * l + 2), ring, xa, xb_of(p.h), p.ACT, nullptr, it, cw, lane);
    MEGA_MARK();
        mega_grid_barrier(p, sh, epoch, ctid);
    MEGA_MARK();
        // ---- down projection into D2 ----
        mega_load_x(sh, xa, xb_of(p.f), p.f, p.ACT, nullptr, nullptr, nullptr, nullptr, 0.f, false, ctid, cw, lane);
    MEGA_MARK();
        mega_zero(p.D1, p.h, ctid);
        mega_run_tiles<MEPI_ADD>(p, sh, mega_phase<D>(p, 4 * l + 3), ring, xa, xb_of(p.f), p.D2, nullptr, it, cw, lane);
    MEGA_MARK();
    }
    // ---- LM head ----
    mega_grid_barrier(p, sh, epoch, ctid);
    MEGA_MARK();
    mega_load_x(sh, xa, xb_of(p.h), p.h, p.X1, p.D2, nullptr, nullptr, p.gf, p.eps, true, ctid, cw, lane);
    MEGA_MARK();
    mega_run_tiles<MEPI_ADD>(p, sh, mega_phase<D>(p, 4 * p.n_layers), ring, xa, xb_of(p.h), p.logits, nullptr, it, cw, lane);
    MEGA_MARK();
    mega_grid_barrier(p, sh, epoch, ctid);
    MEGA_MARK();

    // ---- sampling + router ----
    if (p.want_argmax) {
        float *trace = nullptr;
        if (p.gen && p.buf.trace && p.gen->trace_n > 0) {
            const int t = p.gen->step - p.gen->trace_first;
            if (t >= 0 && t < p.gen->trace_n) trace = p.buf.trace + (size_t)t * p.limit;
        }
        float v = -INFINITY;
        int idx = 0x7fffffff;
        for (int i = blockIdx.x * kMegaCT + ctid; i < p.limit; i += gridDim.x * kMegaCT) {
            const float z = __ldcg(p.logits + i);
            if (trace) trace[i] = z;
            argmax_merge(v, idx, z, i);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float v2 = __shfl_xor_sync(0xffffffffu, v, o);
            const int i2 = __shfl_xor_sync(0xffffffffu, idx, o);
            argmax_merge(v, idx, v2, i2);
        }
        if (lane == 0) { sh.s_v[cw] = v; sh.s_i[cw] = idx; }
        consumer_sync();
        if (ctid == 0) {
            for (int w = 1; w < kMegaConsumers; ++w) argmax_merge(v, idx, sh.s_v[w], sh.s_i[w]);
            p.part_val[blockIdx.x] = v;
            p.part_idx[blockIdx.x] = idx;
            __threadfence();
            const unsigned t = atomicAdd(&p.sync[3], 1u);
            sh.last[0] = (t == gridDim.x - 1);
            if (sh.last[0]) p.sync[3] = 0;
        }
        consumer_sync();
        if (sh.last[0]) {
            __threadfence();
            v = -INFINITY;
            idx = 0x7fffffff;
            for (int i = ctid; i < (int)gridDim.x; i += kMegaCT) argmax_merge(v, idx, __ldcg(&p.part_val[i]), __ldcg(&p.part_idx[i]));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float v2 = __shfl_xor_sync(0xffffffffu, v, o);
                const int i2 = __shfl_xor_sync(0xffffffffu, idx, o);
                argmax_merge(v, idx, v2, i2);
            }
            consumer_sync();
            if (lane == 0) { sh.s_v[cw] = v; sh.s_i[cw] = idx; }
            consumer_sync();
            if (ctid == 0) {
                for (int w = 1; w < kMegaConsumers; ++w) argmax_merge(v, idx, sh.s_v[w], sh.s_i[w]);
                if (idx == 0x7fffffff) idx = 0;
                if (p.argmax_out) *p.argmax_out = idx;
                if (p.gen) router_step(p.gen, p.buf, idx, p.desc_small, p.desc_large, p.status);
            }
        }
    }
    // ---- exit ticket: the last CTA out re-arms the barrier counter for the next launch ----
    if (ctid == 0) {
        __threadfence();
        const unsigned t = atomicAdd(&p.sync[1], 1u);
        if (t == gridDim.x - 1) {
            for (int i = 0; i < kMegaBarCounters; ++i) *mega_bar_counter(p, i) = 0;
            p.sync[1] = 0;
            __threadfence();
        }
    }
}

}  // namespace st
