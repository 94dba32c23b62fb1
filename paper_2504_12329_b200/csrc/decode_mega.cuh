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
constexpr int kMegaDownSlab = 8;                                  // default K segments per slab of the down projection
constexpr uint32_t kMegaSpinLimit = 1u << 22;
constexpr int kMegaMaxUnitPages = 64;                              // block-table entries of one attention unit kept in shared memory
constexpr int kMegaAttnWarps = kMegaConsumers;                    // all consumer warps work on one attention unit

struct MegaLayer {
    const uint16_t *wqkv, *wo, *wgu, *wd;
    const float *bqkv, *g1, *g2;
    uint16_t *kpool, *vpool;
};

// TMA descriptors of the weight matrices for the decode ring: boxes of 256 elements x 32 rows, no
// swizzle (a tile row is 512 contiguous bytes in shared memory), zero fill outside the matrix.
// Device array: 4 per layer (QKV, O, gate/up, down), then the LM head; behind them the K and V pools of
// the paged cache as [all rows][D] matrices in boxes of 16 rows x 64 channels with the 128-byte swizzle.
constexpr int kMegaBoxK = 256;

struct MegaParams {
    const MegaLayer *layers;
    const CUtensorMap *maps;   // [4 * n_layers + 3], global memory: the weight matrices, then the K and the V pool
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
    int32_t n_layers, h, Hq, Hkv, f, vocab, n_splits, unit_keys, stages, xarea_bytes;
    int32_t down_slab;        // K segments per slab of the down projection (0: the whole input vector is kept)
    int32_t kv_off, kv_cap;   // K/V staging area inside the activation area: byte offset, capacity in keys (multiple of 16)
    uint32_t spin_limit;      // polls of a grid barrier before it gives up (kMegaSpinLimit in normal use)
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
// The weight matrix of weight phase idx: 4 per layer (QKV, O, gate/up, down), then the LM head.
struct MegaPhase {
    const uint16_t *W;
    int N, K;
    bool whole_blocks;   // split by whole row blocks (the epilogue is not additive)
    int slab;            // 0: tiles ordered row block first.  s > 0: K is cut into slabs of s segments, tiles ordered slab first,
                         // then row block, then segment: a CTA's range stays within a slab or two of the input vector
};
template <int D>
__device__ __forceinline__ MegaPhase mega_phase(const MegaParams &p, int idx)
{
    MegaPhase ph;
    const int qd = p.Hq * D, kd = p.Hkv * D;
    if (idx == 4 * p.n_layers) {
        ph.W = p.lm_head; ph.N = p.vocab; ph.K = p.h; ph.whole_blocks = false; ph.slab = 0;
        return ph;
    }
    const MegaLayer &L = p.layers[idx >> 2];
    // O: one segment per slab (its input load merges the key splits of just those heads); down: slabs of 8 segments
    // (the activation vector is wide: only a slab of it is kept in shared memory at a time)
    ph.slab = (idx & 3) == 1 ? 1 : (idx & 3) == 3 ? p.down_slab : 0;
    switch (idx & 3) {
    case 0: ph.W = L.wqkv; ph.N = qd + 2 * kd; ph.K = p.h; ph.whole_blocks = false; break;
    case 1: ph.W = L.wo; ph.N = p.h; ph.K = qd; ph.whole_blocks = false; break;
    case 2: ph.W = L.wgu; ph.N = 2 * p.f; ph.K = p.h; ph.whole_blocks = true; break;
    default: ph.W = L.wd; ph.N = p.h; ph.K = p.f; ph.whole_blocks = false; break;
    }
    return ph;
}

// Tiles [t0, t1) of a phase for this CTA (MegaTileIter maps tile indices to row blocks and K segments).
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

// Walks the tiles of a phase in order without a division per tile.  The order is slab first (a slab is
// ph.slab K segments wide; one slab spanning all of K when ph.slab is 0), then row block, then segment.
struct MegaTileIter {
    int rb, seg;        // current tile
    int s_lo, s_hi;     // segments of the current slab
    int nblk, nseg, slab;
    __device__ __forceinline__ void init(const MegaPhase &ph, int nseg_, int t)
    {
        nseg = nseg_;
        slab = ph.slab > 0 ? ph.slab : nseg_;
        nblk = (ph.N + kMegaTileRows - 1) / kMegaTileRows;
        const int n_slabs = (nseg + slab - 1) / slab;
        const int sl = min(t / (nblk * slab), n_slabs - 1);
        s_lo = sl * slab;
        s_hi = min(nseg, s_lo + slab);   // the last slab may be narrower
        const int r = t - sl * nblk * slab, width = s_hi - s_lo;
        rb = r / width;
        seg = s_lo + (r - rb * width);
    }
    // the next tile belongs to another row block (or slab): partial row sums have to be written out
    __device__ __forceinline__ bool last_of_run() const { return seg + 1 == s_hi; }
    __device__ __forceinline__ void next()
    {
        if (++seg == s_hi) {
            seg = s_lo;
            if (++rb == nblk) {
                rb = 0;
                s_lo = s_hi;
                s_hi = min(nseg, s_lo + slab);
                seg = s_lo;
            }
        }
    }
};

// Position in the shared-memory ring: slot and the parity of the slot's current use.
struct MegaRingPos {
    int slot;
    unsigned par;
    bool wrapped;
    __device__ __forceinline__ void next(int stages)
    {
        if (++slot == stages) {
            slot = 0;
            par ^= 1u;
            wrapped = true;
        }
    }
};

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
#define MEGA_TRACE_PARAM , int &trace_i, const int ctid
#define MEGA_TRACE_ARG , trace_i, ctid
#else
#define MEGA_MARK() do { } while (0)
#define MEGA_TRACE_PARAM
#define MEGA_TRACE_ARG
#endif

struct MegaShared {
    uint64_t full[kMegaMaxStages], empty[kMegaMaxStages];
    uint64_t kvfull[2];        // K/V staging buffers of the attention unit
    int32_t pages[kMegaMaxUnitPages];   // block-table entries of the unit's key range
    float red[kMegaConsumers];
    float2 cs[64];          // rotary table of this step's position
    float s_v[kMegaConsumers];
    int s_i[kMegaConsumers];
    int last[2];
    int abort;
};

template <int D, int G>
struct MegaAttnScratch {   // per-warp partial results of an attention unit
    float o[kMegaAttnWarps][G][D];
    float m[kMegaAttnWarps][G], d[kMegaAttnWarps][G];
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
        for (uint32_t it = 0; it < p.spin_limit; ++it) {
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
    constexpr int XU = 4;   // items in flight per thread
    // The gain is fetched together with x (one trip to L2 instead of two): shared memory first takes x * gain, the
    // second pass only scales by 1 / rms.
    const float4 *g4 = reinterpret_cast<const float4 *>(gain);
    for (int q0 = ctid; q0 < 2 * K8; q0 += XU * kMegaCT) {
        float4 v[XU], a[XU], g[XU];
#pragma unroll
        for (int u = 0; u < XU; ++u) {
            const int q = q0 + u * kMegaCT;
            v[u] = a[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            g[u] = make_float4(1.f, 1.f, 1.f, 1.f);
            if (q < 2 * K8) {
                if (src_embed) {
                    const uint2 e = reinterpret_cast<const uint2 *>(src_embed)[q];
                    v[u] = make_float4(bf16_lo(e.x), bf16_hi(e.x), bf16_lo(e.y), bf16_hi(e.y));
                } else {
                    v[u] = __ldcg(reinterpret_cast<const float4 *>(x) + q);
                }
                if (add) a[u] = __ldcg(reinterpret_cast<const float4 *>(add) + q);
                if (norm) g[u] = g4[q];
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
                ((q & 1) ? xb : xa)[q >> 1] = make_float4(t.x * g[u].x, t.y * g[u].y, t.z * g[u].z, t.w * g[u].w);
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
        for (int q = ctid; q < 2 * K8; q += kMegaCT) {   // each thread rescales what it wrote itself
            float4 *dst = ((q & 1) ? xb : xa) + (q >> 1);
            float4 v = *dst;
            v.x *= inv; v.y *= inv; v.z *= inv; v.w *= inv;
            *dst = v;
        }
    }
    consumer_sync();
}

enum { MEPI_ADD = 0, MEPI_SILU = 1 };

// Consume this CTA's tiles of one weight phase.  out: MEPI_ADD -> out[row] += partial (+ bias with the
// first K segment); MEPI_SILU -> out[row / 2] = silu(row 2j) * row 2j+1 (whole row blocks only).
// xa / xb hold the input from element k_base on (phases ordered segment first keep only their segments).
template <int EPI>
__device__ __forceinline__ bool mega_run_tiles(const MegaParams &p, MegaShared &sh, const MegaPhase &ph, uint32_t ring,
                                               const float4 *xa, const float4 *xb, float *out, const float *bias,
                                               MegaRingPos &it, int cw, int lane, int k_base = 0, int ta = -1, int tb = -1)
{
    int t0, t1, nseg;
    mega_range(ph, blockIdx.x, gridDim.x, t0, t1, nseg);
    if (ta >= 0) {   // a part of this CTA's range
        t0 = ta;
        t1 = tb;
    }
    float acc[kMegaRowsPerWarp], acc2[kMegaRowsPerWarp];
#pragma unroll
    for (int r = 0; r < kMegaRowsPerWarp; ++r) acc[r] = acc2[r] = 0.f;
    bool first_seg_seen = false;
    MegaTileIter ti;
    if (t0 < t1) ti.init(ph, nseg, t0);
    for (int t = t0; t < t1; ++t, ti.next(), it.next(p.stages)) {
        const int slot = it.slot;
        const int rb = ti.rb, seg = ti.seg;
        if (seg == 0) first_seg_seen = true;
        const bool close = t == t1 - 1 || ti.last_of_run();   // the row block's run of tiles ends here
        const int k0 = seg * kMegaSeg;
        // after an expired wait every later wait returns at once: the step runs to its end (with a
        // status bit set) instead of leaving warps behind at a barrier
        mbar_wait(smem_u32(&sh.full[slot]), it.par, &sh.abort, p.status);
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
                const float4 a = xa[(k0 - k_base + e) >> 3], b = xb[(k0 - k_base + e) >> 3];
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
        if (close) {
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

// ---------------------------------------------------------------------------------------------
// Decode attention of one (kv head, key split) unit.
//
// The cached keys and values of the unit are staged in shared memory by TMA loads (boxes of 16 keys x 64
// channels, 128-byte swizzle) that are issued at the very start of the layer (between the arrival at and
// the wait on the barrier that opens it), so that their DRAM latency -- several microseconds while the
// weight ring keeps HBM saturated -- is over by the time the QKV projection has been reduced.  The
// staging rows start at the unit's first key rounded down to a box boundary; with the swizzle ldmatrix reads
// are free of bank conflicts.  The products run on mma.sync (fp16 inputs, fp32 accumulation) in the
// transposed form that wastes no accumulator rows on a handful of query heads:
//     S^T[16 keys x 8 heads]  = K[16 x D] . Q^T[D x 8]        (Q as hi + lo fp16 halves: two MMAs)
//     O^T[D x 8 heads]       += V^T[D x 16 keys] . P^T[16 x 8] (P^T from the S^T accumulators by movmatrix)
// Each warp takes groups of 16 keys and keeps its own running maximum / sum / O^T; the warps are merged
// through shared memory, the key splits by the O projection's input load (mega_load_att).
// ---------------------------------------------------------------------------------------------
struct MegaUnit {
    int hk, split, ns;
    int k0a;           // first key of the unit rounded down to a multiple of 16: row r of the staging area is key k0a + r
    int lead;          // rows before the unit's first key (fetched with the first box, masked)
    int n_rows;        // rows up to and including the unit's last key (this step's own key included)
    int n_cached;      // rows below this bound hold cached keys
    int owner;         // the unit holds this step's position (its last row)
    int CH, nch;       // rows per staging chunk, number of chunks
    int pg0;           // first block-table entry of the unit
    uint32_t kbase, vbase;   // shared-memory addresses of the K and V staging areas
    uint32_t half_bytes;     // one 64-channel half of an area: kv_cap rows of 128 bytes
    uint8_t *kptr, *vptr;
};

constexpr int kMegaKvBoxRows = 16;
constexpr int kMegaKvBoxBytes = kMegaKvBoxRows * 128;

__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a)
{
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ void mma_f16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi)
{
    return (uint32_t)__half_as_ushort(__float2half_rn(lo)) | ((uint32_t)__half_as_ushort(__float2half_rn(hi)) << 16);
}

// Byte offset of channel d of row `row` inside a staging area (two 64-channel halves of 128-byte rows
// with the 128-byte swizzle the tensor map writes: 16-byte chunk index xor row mod 8).
__device__ __forceinline__ uint32_t mega_kv_swz(const MegaUnit &u, int row, int d)
{
    const uint32_t cb = (uint32_t)(d & 63) * 2;
    return (uint32_t)(d >> 6) * u.half_bytes + (uint32_t)row * 128 + (cb ^ ((uint32_t)(row & 7) << 4));
}

// Key splits of a decode step at position pos: unit_keys keys per unit while there are CTAs to spare.
__host__ __device__ __forceinline__ int mega_key_splits(int pos, int n_splits_max, int n_cta, int Hkv, int unit_keys)
{
    int ns = (pos + unit_keys) / unit_keys;
    const int fit = n_cta / Hkv > 1 ? n_cta / Hkv : 1;
    const int cap = n_splits_max < fit ? n_splits_max : fit;
    return ns < cap ? ns : cap;
}

// Rows and staging chunks of key split `split` of `ns` at position pos (kv_cap: staging capacity in keys).
struct MegaUnitShape {
    int k0a, lead, n_rows, n_cached, owner, CH, nch;
};
__host__ __device__ __forceinline__ MegaUnitShape mega_unit_shape(int pos, int ns, int split, int kv_cap)
{
    MegaUnitShape u;
    const int n_keys = pos + 1;
    const int per = (n_keys + ns - 1) / ns;
    const int k0 = split * per;
    const int k1 = n_keys < k0 + per ? n_keys : k0 + per;
    const int n_all = k1 > k0 ? k1 - k0 : 0;
    u.owner = (k0 <= pos && pos < k1) ? 1 : 0;
    u.k0a = k0 & ~15;   // staging boxes hold 16 keys
    u.lead = k0 - u.k0a;
    u.n_rows = n_all > 0 ? u.lead + n_all : 0;
    u.n_cached = n_all > 0 ? u.n_rows - u.owner : 0;
    if (u.n_rows <= kv_cap) {
        u.CH = kv_cap;
        u.nch = u.n_rows > 0 ? 1 : 0;
    } else {
        u.CH = (kv_cap >> 1) & ~15;
        u.nch = (u.n_rows + u.CH - 1) / u.CH;
    }
    return u;
}

// Geometry of this CTA's unit for the whole step (the same in every layer).
template <int D>
__device__ __forceinline__ MegaUnit mega_unit(const MegaParams &p, uint8_t *base_ptr, uint32_t base, int pos, int ns)
{
    static_assert(kMegaKvBoxRows == 16, "mega_unit_shape rounds to boxes of 16 keys");
    MegaUnit u;
    u.ns = ns;
    u.hk = blockIdx.x / ns;
    u.split = blockIdx.x - u.hk * ns;
    const MegaUnitShape sh = mega_unit_shape(pos, ns, u.split, p.kv_cap);
    u.owner = sh.owner;
    u.k0a = sh.k0a;
    u.lead = sh.lead;
    u.n_rows = sh.n_rows;
    u.n_cached = sh.n_cached;
    u.CH = sh.CH;
    u.nch = sh.nch;
    u.pg0 = u.k0a >> p.kv.page_shift;
    u.half_bytes = (uint32_t)p.kv_cap * 128;
    u.kbase = base + (uint32_t)p.kv_off;
    u.vbase = u.kbase + (uint32_t)(D / 64) * u.half_bytes;
    u.kptr = base_ptr + p.kv_off;
    u.vptr = u.kptr + (size_t)(D / 64) * u.half_bytes;
    return u;
}

// TMA loads of the cached keys/values of chunk ci of layer l into its staging buffer: boxes of 16 keys x 64
// channels from the pools viewed as [row][D] matrices (a page holds whole boxes), issued by one warp.
template <int D>
__device__ __forceinline__ void mega_kv_issue(const MegaParams &p, MegaShared &sh, const MegaUnit &u, int l, int ci, int lane)
{
    constexpr int NH = D / 64;
    const int b = ci & 1;
    const int r_begin = ci * u.CH;
    const int r_end = min(u.n_cached, r_begin + u.CH);
    const int ng = r_end > r_begin ? (r_end - r_begin + kMegaKvBoxRows - 1) / kMegaKvBoxRows : 0;
    const int boxes = ng * NH * 2;
    const uint32_t bar = smem_u32(&sh.kvfull[b]);
    if (lane == 0) mbar_expect_tx(bar, (uint32_t)boxes * kMegaKvBoxBytes);
    __syncwarp();
    const CUtensorMap *kmap = p.maps + 4 * p.n_layers + 1;
    for (int idx = lane; idx < boxes; idx += 32) {
        const int g = idx / (2 * NH), rem = idx - g * (2 * NH);
        const int isv = rem / NH, half = rem - isv * NH;
        const int row = r_begin + g * kMegaKvBoxRows;
        const int key = u.k0a + row;
        const int pi = (key >> p.kv.page_shift) - u.pg0;
        int page = pi < kMegaMaxUnitPages ? sh.pages[pi] : p.kv.block_tab[key >> p.kv.page_shift];
        if ((unsigned)page >= (unsigned)p.kv.n_pages) {
            atomicOr(p.status, DEV_BAD_PAGE);
            page = 0;
        }
        const int y = ((l * p.kv.n_pages + page) * p.kv.n_kv_heads + u.hk) * p.kv.page_size + (key & (p.kv.page_size - 1));
        const uint32_t dst = (isv ? u.vbase : u.kbase) + (uint32_t)half * u.half_bytes + (uint32_t)(b * u.CH + row - r_begin) * 128;
        tma_load_2d(dst, kmap + isv, half * 64, y, bar);
    }
}

// The first (up to two) chunks of a layer; called by one consumer warp once the activation area is free.
template <int D>
__device__ __forceinline__ void mega_kv_issue_first(const MegaParams &p, MegaShared &sh, const MegaUnit &u, int l, int lane)
{
    for (int ci = 0; ci < min(u.nch, 2); ++ci) mega_kv_issue<D>(p, sh, u, l, ci, lane);
}

template <int D, int G>
__device__ __forceinline__ void mega_attention_unit(const MegaParams &p, MegaShared &sh, MegaAttnScratch<D, G> &sc, const MegaUnit &u,
                                                    const MegaLayer &L, int l, int pos, unsigned (&kvph)[2], int cw, int lane MEGA_TRACE_PARAM)
{
    static_assert(G <= 8, "one MMA column per query head of the group");
    static_assert(D == 64 || D == 128, "staging rows are one or two 64-channel halves");
    constexpr int KS = D / 16, HALF = D / 2, PER_LANE = (HALF + 31) / 32;
    const int gt = cw * 32 + lane;
    const int gq = lane >> 2, t = lane & 3;
    // ---- Q^T fragments: head gq, channels 16 ks + 2 t + {0, 1, 8, 9}; rotated, scaled, split into hi + lo ----
    uint32_t qhi[KS][2], qlo[KS][2];
    {
        float2 raw[KS][2];
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) raw[ks][hf] = make_float2(0.f, 0.f);
        if (gq < G) {
            const float *qsrc = p.QKV + (size_t)(u.hk * G + gq) * D + 2 * t;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks)
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) raw[ks][hf] = __ldcg(reinterpret_cast<const float2 *>(qsrc + 16 * ks + 8 * hf));
        }
#pragma unroll
        for (int ks = 0; ks < KS / 2; ++ks)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const int d = 16 * ks + 8 * hf + 2 * t;             // channel in the first half; partner d + HALF
                const float2 c0 = sh.cs[d], c1 = sh.cs[d + 1];
                const float2 a = raw[ks][hf], bq = raw[ks + KS / 2][hf];
                const float x0 = (a.x * c0.x - bq.x * c0.y) * p.scale, y0 = (a.y * c1.x - bq.y * c1.y) * p.scale;
                const float x1 = (bq.x * c0.x + a.x * c0.y) * p.scale, y1 = (bq.y * c1.x + a.y * c1.y) * p.scale;
                const uint32_t h0 = pack_half2(x0, y0), h1 = pack_half2(x1, y1);
                qhi[ks][hf] = h0;
                qhi[ks + KS / 2][hf] = h1;
                qlo[ks][hf] = pack_half2(x0 - kv_lo(h0), y0 - kv_hi(h0));
                qlo[ks + KS / 2][hf] = pack_half2(x1 - kv_lo(h1), y1 - kv_hi(h1));
            }
    }
    // ---- this step's own key/value (owner unit, first warp): rotate k, round both to what the cache holds, append ----
    uint16_t own_k[PER_LANE][2], own_v[PER_LANE][2];
    if (u.owner && cw == 0) {
        const float *ksrc = p.QKV + (size_t)(p.Hq + u.hk) * D, *vsrc = p.QKV + (size_t)(p.Hq + p.Hkv + u.hk) * D;
        KvView kv = p.kv;
        const size_t off = kv_offset(kv, pos, u.hk, D, p.status);
#pragma unroll
        for (int i = 0; i < PER_LANE; ++i) {
            const int j = lane + 32 * i;
            if (j < HALF) {
                const float a = __ldcg(ksrc + j), bk = __ldcg(ksrc + j + HALF);
                const float2 c = sh.cs[j];
                own_k[i][0] = kv_bits(a * c.x - bk * c.y);
                own_k[i][1] = kv_bits(bk * c.x + a * c.y);
                own_v[i][0] = kv_bits(__ldcg(vsrc + j));
                own_v[i][1] = kv_bits(__ldcg(vsrc + j + HALF));
                L.kpool[off + j] = own_k[i][0];
                L.kpool[off + j + HALF] = own_k[i][1];
                L.vpool[off + j] = own_v[i][0];
                L.vpool[off + j + HALF] = own_v[i][1];
            }
        }
    }
    MEGA_MARK();
    float mrun[2] = {-INFINITY, -INFINITY}, lrun[2] = {0.f, 0.f};
    float oacc[KS][4];
#pragma unroll
    for (int mt = 0; mt < KS; ++mt)
#pragma unroll
        for (int e = 0; e < 4; ++e) oacc[mt][e] = 0.f;

    for (int ci = 0; ci < u.nch; ++ci) {
        const int b = ci & 1;
        const int nr = min(u.n_rows, (ci + 1) * u.CH) - ci * u.CH;   // rows of the chunk, the own key's included
        mbar_wait(smem_u32(&sh.kvfull[b]), kvph[b] & 1u, &sh.abort, p.status);
        ++kvph[b];
        if (ci == u.nch - 1 && u.owner && cw == 0) {
            const int row = b * u.CH + nr - 1;
#pragma unroll
            for (int i = 0; i < PER_LANE; ++i) {
                const int j = lane + 32 * i;
                if (j < HALF) {
                    *reinterpret_cast<uint16_t *>(u.kptr + mega_kv_swz(u, row, j)) = own_k[i][0];
                    *reinterpret_cast<uint16_t *>(u.kptr + mega_kv_swz(u, row, j + HALF)) = own_k[i][1];
                    *reinterpret_cast<uint16_t *>(u.vptr + mega_kv_swz(u, row, j)) = own_v[i][0];
                    *reinterpret_cast<uint16_t *>(u.vptr + mega_kv_swz(u, row, j + HALF)) = own_v[i][1];
                }
            }
        }
        {   // value rows behind the last key of the last group of 16 must be finite (their weight is zero)
            const int pad = ((nr + 15) & ~15) - nr;
            for (int idx = gt; idx < pad * (D / 8); idx += kMegaCT) {
                const int r = b * u.CH + nr + idx / (D / 8), c = idx % (D / 8);
                *reinterpret_cast<uint4 *>(u.vptr + (size_t)(c >> 3) * u.half_bytes + (size_t)r * 128 + (c & 7) * 16) = make_uint4(0, 0, 0, 0);
            }
        }
        consumer_sync();
        MEGA_MARK();
        const int ngroups = (nr + 15) >> 4;
        for (int gi = cw; gi < ngroups; gi += kMegaConsumers) {
            const int r0 = gi * 16;
            // S^T = K . Q^T
            float s[4] = {0.f, 0.f, 0.f, 0.f};
            const int krow = b * u.CH + r0 + (lane & 7) + ((lane >> 3) & 1) * 8;
            const uint32_t ka = u.kbase + (uint32_t)krow * 128;
            const uint32_t kx = (uint32_t)(krow & 7);
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                uint32_t a[4];
                ldmatrix_x4(a, ka + (uint32_t)(ks >> 2) * u.half_bytes + ((((uint32_t)(ks & 3) * 2 + (uint32_t)(lane >> 4)) ^ kx) << 4));
                mma_f16_16816(s, a, qhi[ks][0], qhi[ks][1]);
                mma_f16_16816(s, a, qlo[ks][0], qlo[ks][1]);
            }
            // online softmax per head (column): this lane holds rows r0 + gq (+ 8) of heads 2 t, 2 t + 1
            const int rr = ci * u.CH + r0 + gq;
            const bool v0 = rr >= u.lead && rr < u.n_rows, v1 = rr + 8 >= u.lead && rr + 8 < u.n_rows;
            const float s0 = v0 ? s[0] : -INFINITY, s1 = v0 ? s[1] : -INFINITY, s2 = v1 ? s[2] : -INFINITY, s3 = v1 ? s[3] : -INFINITY;
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
            // O^T += V^T . P^T
            const int vrow = b * u.CH + r0 + (lane & 7) + (lane >> 4) * 8;
            const uint32_t va = u.vbase + (uint32_t)vrow * 128;
            const uint32_t vx = (uint32_t)(vrow & 7);
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) {
                oacc[mt][0] *= corr0; oacc[mt][1] *= corr1; oacc[mt][2] *= corr0; oacc[mt][3] *= corr1;
                uint32_t a[4];
                ldmatrix_x4_trans(a, va + (uint32_t)(mt >> 2) * u.half_bytes + ((((uint32_t)(mt & 3) * 2 + (uint32_t)((lane >> 3) & 1)) ^ vx) << 4));
                mma_f16_16816(oacc[mt], a, pb0, pb1);
            }
        }
        if (ci + 2 < u.nch) {   // refill this buffer with the chunk after next
            consumer_sync();
            if (cw == 0) mega_kv_issue<D>(p, sh, u, l, ci + 2, lane);
        }
    }
    MEGA_MARK();
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
        lrun[0] += __shfl_xor_sync(0xffffffffu, lrun[0], o);
        lrun[1] += __shfl_xor_sync(0xffffffffu, lrun[1], o);
    }
    // ---- merge the warps (the scratch overlays the staging buffers: every warp must be done reading them) ----
    consumer_sync();
    MEGA_MARK();
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int head = 2 * t + e;
        if (head < G) {
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) {
                sc.o[cw][head][16 * mt + gq] = oacc[mt][e];
                sc.o[cw][head][16 * mt + gq + 8] = oacc[mt][2 + e];
            }
            if (gq == 0) { sc.m[cw][head] = mrun[e]; sc.d[cw][head] = lrun[e]; }
        }
    }
    consumer_sync();
    MEGA_MARK();
    const int hq0 = u.hk * G;
    for (int idx = gt; idx < G * D; idx += kMegaCT) {
        const int g = idx / D, c = idx - g * D;
        // every load first (they do not depend on one another), then the arithmetic
        float mw[kMegaAttnWarps], dw[kMegaAttnWarps], ow[kMegaAttnWarps];
#pragma unroll
        for (int w = 0; w < kMegaAttnWarps; ++w) {
            mw[w] = sc.m[w][g];
            dw[w] = sc.d[w][g];
            ow[w] = sc.o[w][g][c];
        }
        float mnew = -INFINITY;
#pragma unroll
        for (int w = 0; w < kMegaAttnWarps; ++w) mnew = fmaxf(mnew, mw[w]);
        float dsum = 0.f, osum = 0.f;
#pragma unroll
        for (int w = 0; w < kMegaAttnWarps; ++w) {
            const bool live = mw[w] != -INFINITY;   // a warp without keys left its sum and output slots untouched
            const float cw2 = live ? __expf(mw[w] - mnew) : 0.f;
            dsum += live ? dw[w] * cw2 : 0.f;
            osum += live ? ow[w] * cw2 : 0.f;
        }
        const size_t pi = (size_t)(hq0 + g) * u.ns + u.split;
        p.part_o[pi * D + c] = osum;
        if (c == 0) { p.part_ml[pi * 2] = mnew; p.part_ml[pi * 2 + 1] = dsum; }
    }
}

// Input of the O projection: the attention output of the K segments this CTA's tiles cover (the phase is
// ordered segment first, so these are one or two segments = a few heads), merged from the key splits'
// partial results on the fly: att[h][c] = sum_s w_s o_s[c] / sum_s w_s l_s with w_s = exp(m_s - max m).
// Warp i computes the weights of the i-th head of the segment; then 128 threads x 2 halves of the splits
// accumulate 4 channels each.
template <int D>
__device__ __forceinline__ void mega_load_att(const MegaParams &p, const MegaPhase &ph, float4 *xa, float4 *xb, float *wbuf, int ns,
                                              int ctid, int cw, int lane)
{
    constexpr int HPS = kMegaSeg / D;   // heads per K segment
    static_assert(HPS <= kMegaConsumers, "one warp per head of a segment");
    int t0, t1, nseg;
    mega_range(ph, blockIdx.x, gridDim.x, t0, t1, nseg);
    if (t0 >= t1) return;   // uniform for the CTA
    const int nblk = (ph.N + kMegaTileRows - 1) / kMegaTileRows;
    float *w = wbuf;                               // [HPS][ns]
    float *inv_den = wbuf + HPS * kMaxAttnSplits;  // [HPS]
    float4 *tmp = reinterpret_cast<float4 *>(inv_den + 8);   // [128]
    for (int seg = t0 / nblk; seg <= (t1 - 1) / nblk; ++seg) {
        const int hq_first = seg * HPS;
        if (cw < HPS && hq_first + cw < p.Hq) {
            const int hq = hq_first + cw;
            const float2 *ml = reinterpret_cast<const float2 *>(p.part_ml) + (size_t)hq * ns;
            float mmax = -INFINITY;
            for (int sp = lane; sp < ns; sp += 32) mmax = fmaxf(mmax, __ldcg(ml + sp).x);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mmax = fmaxf(mmax, __shfl_xor_sync(0xffffffffu, mmax, o));
            float dsum = 0.f;
            for (int sp = lane; sp < ns; sp += 32) {
                const float2 v = __ldcg(ml + sp);
                const float ws = v.x == -INFINITY ? 0.f : __expf(v.x - mmax);
                w[cw * kMaxAttnSplits + sp] = ws;
                dsum += v.y * ws;
            }
            dsum = warp_sum(dsum);
            if (lane == 0) inv_den[cw] = 1.f / dsum;
        }
        consumer_sync();
        const int col4 = ctid & 127, part = ctid >> 7;
        const int c = seg * kMegaSeg + col4 * 4;    // first of this thread's 4 channels (column of the O matrix)
        const bool live = c < ph.K;
        const int hl = (col4 * 4) / D, hq = hq_first + hl;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (live) {
            const float *po = p.part_o + (size_t)hq * ns * D + (c - hq * D);
            const float *wh = w + hl * kMaxAttnSplits;
            for (int sp = part; sp < ns; sp += 2) {
                const float4 o4 = __ldcg(reinterpret_cast<const float4 *>(po + (size_t)sp * D));
                const float ws = wh[sp];
                acc.x = fmaf(o4.x, ws, acc.x); acc.y = fmaf(o4.y, ws, acc.y);
                acc.z = fmaf(o4.z, ws, acc.z); acc.w = fmaf(o4.w, ws, acc.w);
            }
        }
        if (part == 1) tmp[col4] = acc;
        consumer_sync();
        if (part == 0 && live) {
            const float4 o2 = tmp[col4];
            const float id = inv_den[hl];
            const float4 r = make_float4((acc.x + o2.x) * id, (acc.y + o2.y) * id, (acc.z + o2.z) * id, (acc.w + o2.w) * id);
            const int q = c >> 2;
            ((q & 1) ? xb : xa)[q >> 1] = r;
        }
        consumer_sync();
    }
}

// The piece of this CTA's tile range [t, t1) that lies within one slab: its end and the slab's segments [s0, s1].
__device__ __forceinline__ int mega_slab_piece(const MegaPhase &ph, int nseg, int t, int t1, int &s0, int &s1)
{
    const int slab = ph.slab > 0 ? ph.slab : nseg;   // no slabs: the whole of K is one
    const int nblk = (ph.N + kMegaTileRows - 1) / kMegaTileRows;
    const int n_slabs = (nseg + slab - 1) / slab;
    const int sl = min(t / (nblk * slab), n_slabs - 1);
    s0 = sl * slab;
    s1 = min(nseg, s0 + slab) - 1;
    return sl == n_slabs - 1 ? t1 : min(t1, (sl + 1) * nblk * slab);
}

// Input of a slab-ordered phase taken as is from a global fp32 vector: elements [s0 * 512, (s1 + 1) * 512)
// go to xa / xb (xb = xa + (s1 - s0 + 1) * 64), zero beyond K.
__device__ __forceinline__ void mega_load_segs(float4 *xa, const float *x, int K, int s0, int s1, int ctid)
{
    const int n4 = (s1 - s0 + 1) * (kMegaSeg / 4);
    float4 *xb = xa + (n4 >> 1);
    consumer_sync();   // every warp is done with what the area held before
    const int q_base = s0 * (kMegaSeg / 4);
    for (int q = ctid; q < n4; q += kMegaCT) {
        const int qa = q_base + q;
        const float4 v = qa * 4 < K ? __ldcg(reinterpret_cast<const float4 *>(x) + qa) : make_float4(0.f, 0.f, 0.f, 0.f);
        ((q & 1) ? xb : xa)[q >> 1] = v;
    }
    consumer_sync();
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

// Exercises the grid barrier's bounded wait: one CTA waits for an arrival that never comes (it does not arrive
// itself); the wait must give up after p.spin_limit polls, raise the abort flag and the status bit, and return.
__global__ void __launch_bounds__(kMegaThreads, 1) mega_barrier_selftest_kernel(const MegaParams p, int32_t *returned)
{
    __shared__ MegaShared sh;
    const int tid = threadIdx.x;
    if (tid == 0) sh.abort = 0;
    __syncthreads();
    if (tid < 32) return;   // the producer warp has no part in barriers
    const int ctid = tid - 32;
    unsigned epoch = 0;
    const bool ok = mega_barrier_wait(p, sh, epoch, ctid);
    const bool ok2 = mega_barrier_wait(p, sh, epoch, ctid);   // returns at once: the abort flag is up
    if (ctid == 0) *returned = (ok || ok2) ? 1 : 2;
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
        mbar_init(smem_u32(&sh.kvfull[0]), 1);
        mbar_init(smem_u32(&sh.kvfull[1]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == 0) {
        // ------------------------------ producer ------------------------------
        MegaRingPos it{0, 0u, false};
        bool ok = true;
        for (int idx = 0; idx < n_phases && ok; ++idx) {
            const MegaPhase ph = mega_phase<D>(p, idx);
            int t0, t1, nseg;
            mega_range(ph, blockIdx.x, gridDim.x, t0, t1, nseg);
            MegaTileIter ti;
            if (t0 < t1) ti.init(ph, nseg, t0);
            for (int t = t0; t < t1 && ok; ++t, ti.next(), it.next(p.stages)) {
                const int slot = it.slot;
                if (it.wrapped) {
                    int w_ok = lane == 0 ? (int)mbar_wait(smem_u32(&sh.empty[slot]), it.par ^ 1u, &sh.abort, p.status) : 1;
                    w_ok = __shfl_sync(0xffffffffu, w_ok, 0);
                    if (!w_ok) { ok = false; break; }
                }
                const int r0 = ti.rb * kMegaTileRows, k0 = ti.seg * kMegaSeg;
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
    unsigned epoch = 0;
    MegaRingPos it{0, 0u, false};
    int trace_i = 0;
    (void)trace_i;
    MEGA_MARK();
    auto xb_of = [&](int K) { return xa + (K >> 3); };

    // step set-up: rotary table, zeroed accumulation vectors, this CTA's attention unit
    for (int j = ctid; j < D / 2; j += kMegaCT) {
        double s, c;
        sincos((double)pos * p.inv_freq[j], &s, &c);
        sh.cs[j] = make_float2((float)c, (float)s);
    }
    // every CTA derives the same split count
    const int ns = mega_key_splits(pos, p.n_splits, (int)gridDim.x, p.Hkv, p.unit_keys);
    const bool attn_active = (int)blockIdx.x < p.Hkv * ns;
    const MegaUnit unit = mega_unit<D>(p, base_ptr, base, pos, ns);
    if (attn_active && unit.n_cached > 0) {
        const int npg = ((unit.k0a + unit.n_cached - 1) >> p.kv.page_shift) - unit.pg0 + 1;
        for (int i = ctid; i < min(npg, kMegaMaxUnitPages); i += kMegaCT) sh.pages[i] = p.kv.block_tab[unit.pg0 + i];
    }
    unsigned kvph[2] = {0u, 0u};
    mega_zero(p.QKV, qkvd, ctid);
    mega_zero(p.D1, p.h, ctid);
    mega_zero(p.D2, p.h, ctid);
    mega_zero(p.logits, p.vocab, ctid);
    mega_barrier_arrive(p, ctid);
    if (attn_active && cw == 1) mega_kv_issue_first<D>(p, sh, unit, 0, lane);
    mega_barrier_wait(p, sh, epoch, ctid);
    MEGA_MARK();

    int tokid = p.tok[p.desc->tok_off];
    if ((unsigned)tokid >= (unsigned)p.vocab) {
        if (ctid == 0) atomicOr(p.status, DEV_BAD_TOKEN);
        tokid = 0;
    }
    MegaAttnScratch<D, G> *scratch = reinterpret_cast<MegaAttnScratch<D, G> *>(base_ptr);

    for (int l = 0; l < p.n_layers; ++l) {
        const MegaLayer &L = p.layers[l];
        // ---- QKV: x = (layer 0 ? embedding : x1 + down), normalised ----
        if (l > 0) {
            // the down projection is done with the activation area: the unit's cached K/V can start to land
            fence_proxy_async_smem();
            mega_barrier_arrive(p, ctid);
            if (attn_active && cw == 1) mega_kv_issue_first<D>(p, sh, unit, l, lane);
            mega_barrier_wait(p, sh, epoch, ctid);
        }
        MEGA_MARK();
        mega_load_x(sh, xa, xb_of(p.h), p.h, p.X1, l > 0 ? p.D2 : nullptr, l == 0 ? p.embed + (size_t)tokid * p.h : nullptr, p.X0,
                    L.g1, p.eps, true, ctid, cw, lane);
    MEGA_MARK();
        mega_run_tiles<MEPI_ADD>(p, sh, mega_phase<D>(p, 4 * l), ring, xa, xb_of(p.h), p.QKV, L.bqkv, it, cw, lane);
    MEGA_MARK();
        // ---- attention: one (kv head, key split) unit per CTA ----
        mega_grid_barrier(p, sh, epoch, ctid);
    MEGA_MARK();
        mega_zero(p.D2, p.h, ctid);
        if (attn_active) mega_attention_unit<D, G>(p, sh, scratch[0], unit, L, l, pos, kvph, cw, lane MEGA_TRACE_ARG);
        MEGA_MARK();
        mega_grid_barrier(p, sh, epoch, ctid);
    MEGA_MARK();
        // ---- O projection into D1 (its input load merges the key splits) ----
        {
            const MegaPhase pho = mega_phase<D>(p, 4 * l + 1);
            float *wbuf = reinterpret_cast<float *>(base_ptr) + ((qd + 255) & ~255);
            mega_load_att<D>(p, pho, xa, xb_of(qd), wbuf, ns, ctid, cw, lane);
        }
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
        // ---- down projection into D2, slab by slab of the activation vector ----
        {
            const MegaPhase phd = mega_phase<D>(p, 4 * l + 3);
            int t0, t1, nseg;
            mega_range(phd, blockIdx.x, gridDim.x, t0, t1, nseg);
            mega_zero(p.D1, p.h, ctid);
            for (int t = t0; t < t1;) {
                int s0, s1;
                const int te = mega_slab_piece(phd, nseg, t, t1, s0, s1);
                mega_load_segs(xa, p.ACT, p.f, s0, s1, ctid);
                mega_run_tiles<MEPI_ADD>(p, sh, phd, ring, xa, xa + (s1 - s0 + 1) * (kMegaSeg / 8), p.D2, nullptr, it, cw, lane,
                                         s0 * kMegaSeg, t, te);
                t = te;
            }
        }
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
    if (p.want_argmax && top_p_active(p.gen)) {   // the same decision in every CTA
        // top-p: CTA 0 finds the nucleus' threshold (the ring is free by now), the others learn it after one more barrier
        if (blockIdx.x == 0) {
            unsigned long long *hist = reinterpret_cast<unsigned long long *>(base_ptr + p.xarea_bytes);
            const float tau = nucleus_threshold_cta(p.logits, p.limit, p.gen->inv_temp, p.gen->top_p, hist, hist + kNucleusBins,
                                                    hist + kNucleusBins + 256, ctid, [] { consumer_sync(); });
            if (ctid == 0) p.gen->tau = tau;
        }
        mega_grid_barrier(p, sh, epoch, ctid);
    }
    if (p.want_argmax) {
        float *trace = nullptr;
        if (p.gen && p.buf.trace && p.gen->trace_n > 0) {
            const int t = p.gen->step - p.gen->trace_first;
            if (t >= 0 && t < p.gen->trace_n) trace = p.buf.trace + (size_t)t * p.limit;
        }
        float v = -INFINITY;
        int idx = 0x7fffffff;
        const SampleRule rule = sample_rule(p.gen);   // the step counter changes only after every CTA has taken its ticket
        for (int i = blockIdx.x * kMegaCT + ctid; i < p.limit; i += gridDim.x * kMegaCT) {
            const float z = __ldcg(p.logits + i);
            if (trace) trace[i] = z;
            argmax_merge(v, idx, rule(z, i), i);
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
