// Multi-row (prefill / catch-up) projection on the 5th-generation tensor cores.
//
//   Y[i][n] = sum_k (A_hi[i][k] + A_lo[i][k]) * W[n][k]      i < m <= 256 activation rows
//
// "Swap-AB": the weight tile takes the M side of the MMA (128 weight rows = 128 TMEM lanes), the
// activation rows take the N side (m padded to a multiple of 32 = TMEM columns), so that a pass of a
// few dozen rows still fills the instruction and every weight byte is read from HBM once per pass.
// Both operands are K-major bf16 tiles of 64 elements (128 bytes) per row, brought in by TMA with the
// 128-byte swizzle and consumed from shared memory by tcgen05.mma (kind::f16, fp32 accumulate in
// TMEM).  The hi and lo activation planes are two MMAs on the same weight tile.
//
// One CTA = w_tiles adjacent 128-row weight tiles x one K split.  Warp 0 issues TMA, warp 1 owns TMEM and issues
// the MMAs, warps 2..5 drain the accumulator (tcgen05.ld) into the epilogue.  Stages hand over
// through mbarriers; every wait is bounded and, when it runs out, raises a status bit, lets the CTA
// drain what it armed, frees its TMEM and returns.  Every CTA stands alone: each loads its own tiles.
#pragma once
#include <cuda.h>

#include "st_common.cuh"

namespace st {

enum { TEPI_STORE = 0, TEPI_RESADD = 1, TEPI_SILU = 2 };

struct TcGemmParams {
    const StepDesc *desc;
    const float *bias;        // [N] or null (added by K split 0)
    float *Yf;                // TEPI_STORE / TEPI_RESADD: [rows][N] fp32 when k_splits == 1
    float *Ws;                // k_splits > 1: partial sums [k_splits][ws_rows][N], reduced by splitk_reduce_kernel
    int32_t ws_rows;
    uint16_t *Yb_hi, *Yb_lo;  // TEPI_SILU: [rows][N / 2] hi/lo planes of silu(row 2j) * row 2j+1
    int32_t *status;
    int32_t N, K;
    const CUtensorMap *act_hi, *act_lo;   // global memory, [8] each: the hi / lo activation plane in boxes of 32 (j + 1) rows
    int32_t m_pad;            // upper bound of the MMA N of this launch (multiple of 32, <= 256): shared-memory and TMEM
                              // layout follow it; the rows actually loaded and multiplied are desc->m rounded up to 32
    int32_t stages;           // shared-memory pipeline depth
    int32_t k_splits;
    int32_t tmem_cols;        // power of two >= max(32, w_tiles * m_pad)
    int32_t w_tiles;          // 128-row weight tiles per CTA (each with its own accumulator); they share the
                              // activation tiles of a stage, which cuts the activation re-reads per weight byte
    const CUtensorMap *act_hi_half, *act_lo_half;   // [16] each: the planes in boxes of 16 (j + 1) rows (CTA pairs: each
                                                    // CTA loads half of the activation rows)
};

constexpr int kTcTileW = 128;       // weight rows per CTA
constexpr int kTcBlockK = 64;       // K elements per stage (128 bytes per row)
constexpr int kTcWBytes = kTcTileW * kTcBlockK * 2;
constexpr uint32_t kTcWaitLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false (and a status bit) when the phase does not complete within the limit.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int32_t *status,
                                          uint32_t limit = kTcWaitLimit)
{
    for (uint32_t it = 0; it < limit; ++it) {
        if (mbar_try(bar, parity)) return true;
        if (*abort_flag) return false;
        if (it > 64) __nanosleep(64);
    }
    *abort_flag = 1;
    atomicOr(status, DEV_WAIT_EXPIRED);
    return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

// Shared-memory matrix descriptor of a K-major tile with 128-byte rows and the 128-byte swizzle:
// 8-row groups are 1024 bytes apart (stride byte offset), descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr)
{
    const uint32_t lo = (smem_addr >> 4) & 0x3fffu;
    const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
    return ((uint64_t)hi << 32) | lo;
}

// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t umma_idesc_bf16(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float *v)
{
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Exercises the bounded wait without faulting anything: one CTA waits, with a short limit, on an mbarrier that
// nobody arms; the wait must give up, raise the status bit and let the kernel return normally.
__global__ void wait_expiry_selftest_kernel(int32_t *status, uint32_t limit, int32_t *returned)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    bool ok = true;
    if (threadIdx.x == 0) ok = mbar_wait(smem_u32(&bar), 0, &abort_flag, status, limit);
    __syncthreads();
    // every later wait of the CTA returns at once after the first one gave up
    if (threadIdx.x == 32) ok = mbar_wait(smem_u32(&bar), 0, &abort_flag, status, 1u << 30);
    __syncthreads();
    if (threadIdx.x == 0) *returned = ok ? 1 : 2;
}

// Sum the K-split partials of a projection in a fixed order: Y[i][n] (+)= sum_s Ws[s][i][n] (+ bias[n]).
__global__ void splitk_reduce_kernel(const StepDesc *desc, const float *Ws, int k_splits, int ws_rows, int N, const float *bias,
                                     float *Y, int accumulate)
{
    const int i = blockIdx.y;
    if (i >= desc->m) return;
    const int n4 = N >> 2;
    for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < n4; j += gridDim.x * blockDim.x) {
        float4 acc = bias ? reinterpret_cast<const float4 *>(bias)[j] : make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s = 0; s < k_splits; ++s) {
            const float4 v = __ldcg(reinterpret_cast<const float4 *>(Ws + ((size_t)s * ws_rows + i) * N) + j);
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        float4 *dst = reinterpret_cast<float4 *>(Y + (size_t)i * N) + j;
        if (accumulate) {
            const float4 o = *dst;
            acc.x += o.x; acc.y += o.y; acc.z += o.z; acc.w += o.w;
        }
        *dst = acc;
    }
}

// ---------------------------------------------------------------------------------------------
// The same projection on CTA pairs (tcgen05 cta_group::2).
//
// The single-CTA kernel is bound by what an SM takes in: per 16 KB weight tile it also loads the activation tiles
// of the stage (hi and lo plane of up to 256 rows), and with two or three weight tiles per CTA those are as many
// bytes as the weights.  Two CTAs of a cluster share one MMA: the instruction takes 128 weight rows from each CTA's
// shared memory (M = 256, each CTA's half of the accumulator in its own tensor memory) and HALF of the activation
// rows from each (the N side), so a CTA loads only half of every activation tile.  Protocol:
//   * both CTAs run the same code; rank 0 of the pair (the leader) issues every MMA;
//   * each CTA's TMA thread loads its own weight tiles and its half of the activation rows into its own shared
//     memory, but the loads of BOTH CTAs report their bytes to the leader's "full" barrier of the stage (the
//     barrier address is mapped into the leader's window), which the leader arms with the bytes of both;
//   * the leader's commit after the MMAs of a stage arrives at the "empty" barrier of the stage in both CTAs, the
//     final commit at the accumulator barrier of both; each CTA's epilogue warps drain their own tensor memory;
//   * tensor memory is allocated and freed by the same warp of both CTAs (the pair form of the instructions);
//   * the pair synchronises once, after its barriers are initialised and before any load is issued; every wait is
//     bounded as in the single-CTA kernel, and every path reaches the common exit.
// Every load writes only the issuing CTA's own shared memory (one copy per load).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA load of a CTA of a pair: destination in this CTA's shared memory, completion bytes to `bar`, which may be a
// barrier of either CTA of the pair (cluster address).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrives (once the MMAs issued so far are complete) at the barrier at this address in both CTAs of the pair.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}
// Instruction descriptor of the pair MMA: D fp32, A and B bf16, both K-major, M = 256 (128 rows per CTA), N = n.
__device__ __forceinline__ uint32_t umma_idesc_bf16_pair(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(192) tc_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmW, const TcGemmParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t s_full[8], s_empty[8], s_acc;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    pdl_launch();
    const int m = p.desc->m;
    if (m <= 0) return;   // the same for both CTAs of a pair
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();          // 0: the leader of the pair
    const int n0 = blockIdx.x * kTcTileW * p.w_tiles;   // this CTA's weight rows (the pair holds two adjacent groups)
    const int kb_total = (p.K + kTcBlockK - 1) / kTcBlockK;
    const int kb_per = (kb_total + p.k_splits - 1) / p.k_splits;
    const int kb0 = blockIdx.y * kb_per;
    const int kb1 = min(kb_total, kb0 + kb_per);
    const int n_kb = kb1 - kb0;
    if (n_kb <= 0) return;   // the same for both CTAs of a pair

    const int m_eff = min(p.m_pad, (m + 31) & ~31);   // rows multiplied (both halves): a multiple of 32
    const int half = m_eff >> 1;                      // rows this CTA loads: a multiple of 16
    const uint32_t a_half_bytes = (uint32_t)(p.m_pad >> 1) * kTcBlockK * 2;   // layout follows the launch's bound
    const uint32_t a_half_eff = (uint32_t)half * kTcBlockK * 2;
    const CUtensorMap *tmAhi = p.act_hi_half + (half / 16 - 1), *tmAlo = p.act_lo_half + (half / 16 - 1);
    const uint32_t w_bytes = (uint32_t)p.w_tiles * kTcWBytes;
    const uint32_t stage_bytes = w_bytes + 2 * a_half_bytes;
    const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;

    if (tid == 0) {
        s_abort = 0;
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&s_full[s]), 1);
            mbar_init(smem_u32(&s_empty[s]), 1);
        }
        mbar_init(smem_u32(&s_acc), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {   // the same warp of both CTAs
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)), "r"((uint32_t)p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync_all();   // both CTAs' barriers exist before either issues a load that reports to the leader's
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s_tmem_base;

    if (warp == 0) {
        // ---------------- TMA producer (both CTAs) ----------------
        if (lane == 0) {
            int armed = 0;
            auto full_of = [&](int s) { return map_to_cta(smem_u32(&s_full[s]), 0); };   // the leader's barrier
            auto load_w = [&](int i) {
                const int s = i % p.stages;
                const uint32_t base = tiles + (uint32_t)s * stage_bytes;
                if (rank == 0) mbar_expect_tx(smem_u32(&s_full[s]), 2 * (w_bytes + 2 * a_half_eff));   // bytes of both CTAs
                const int kx = (kb0 + i) * kTcBlockK;
                for (int t = 0; t < p.w_tiles; ++t) tma_load_2d_pair(base + (uint32_t)t * kTcWBytes, &tmW, kx, n0 + t * kTcTileW, full_of(s));
            };
            const int pre = min(n_kb, p.stages);
            for (int i = 0; i < pre; ++i) load_w(i);
            pdl_wait();
            for (int i = 0; i < n_kb; ++i) {
                const int s = i % p.stages, u = i / p.stages;
                if (u > 0) {
                    if (!mbar_wait(smem_u32(&s_empty[s]), (u - 1) & 1, &s_abort, p.status)) break;
                    load_w(i);
                }
                const uint32_t base = tiles + (uint32_t)s * stage_bytes;
                const int kx = (kb0 + i) * kTcBlockK;
                tma_load_2d_pair(base + w_bytes, tmAhi, kx, (int)rank * half, full_of(s));
                tma_load_2d_pair(base + w_bytes + a_half_bytes, tmAlo, kx, (int)rank * half, full_of(s));
                armed = i + 1;
            }
            if (s_abort && rank == 0) {
                for (int i = max(0, armed - p.stages); i < armed; ++i) {
                    const int s = i % p.stages, u = i / p.stages;
                    for (uint32_t it = 0; it < (1u << 16) && !mbar_try(smem_u32(&s_full[s]), u & 1); ++it) __nanosleep(128);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (the leader only) ----------------
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = umma_idesc_bf16_pair(m_eff);
            bool ok = true;
            for (int i = 0; i < n_kb && ok; ++i) {
                const int s = i % p.stages, u = i / p.stages;
                ok = mbar_wait(smem_u32(&s_full[s]), u & 1, &s_abort, p.status);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t base = tiles + (uint32_t)s * stage_bytes;
                const uint64_t dh = umma_desc_sw128(base + w_bytes);
                const uint64_t dl = umma_desc_sw128(base + w_bytes + a_half_bytes);
                for (int t = 0; t < p.w_tiles; ++t) {
                    const uint64_t dw = umma_desc_sw128(base + (uint32_t)t * kTcWBytes);
                    const uint32_t acc = tmem + (uint32_t)(t * p.m_pad);
#pragma unroll
                    for (int k4 = 0; k4 < kTcBlockK / 16; ++k4)
                        umma_bf16_pair(acc, dw + 2 * k4, dh + 2 * k4, idesc, (i > 0 || k4 > 0) ? 1u : 0u);
#pragma unroll
                    for (int k4 = 0; k4 < kTcBlockK / 16; ++k4)
                        umma_bf16_pair(acc, dw + 2 * k4, dl + 2 * k4, idesc, 1u);
                }
                umma_commit_pair(smem_u32(&s_empty[s]));
            }
            // the accumulator barrier of both CTAs; after a failed wait nothing more will complete: release the
            // partner's epilogue through its bounded wait instead
            if (ok) umma_commit_pair(smem_u32(&s_acc));
        }
    } else {
        // ---------------- epilogue (both CTAs, each its own half of the accumulator) ----------------
        const int q = warp & 3;
        pdl_wait();
        int ok_i = lane == 0 ? (int)mbar_wait(smem_u32(&s_acc), 0, &s_abort, p.status) : 1;
        const bool ok = __shfl_sync(0xffffffffu, ok_i, 0) != 0;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok) {
            for (int t = 0; t < p.w_tiles; ++t) {
                const int row = n0 + t * kTcTileW + q * 32 + lane;
                const float bias = (EPI != TEPI_SILU && p.bias && blockIdx.y == 0 && row < p.N) ? p.bias[row] : 0.f;
                for (int c0 = 0; c0 < m; c0 += 16) {
                    float v[16];
                    tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(t * p.m_pad + c0), v);
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int c = c0 + j;
                        if (EPI == TEPI_SILU) {
                            const float other = __shfl_xor_sync(0xffffffffu, v[j], 1);
                            if (c < m && !(lane & 1) && row + 1 < p.N) {
                                const size_t o = (size_t)c * (p.N >> 1) + (row >> 1);
                                split_bf16(v[j] / (1.f + expf(-v[j])) * other, p.Yb_hi[o], p.Yb_lo[o]);
                            }
                        } else if (c < m && row < p.N) {
                            if (p.k_splits > 1) {
                                p.Ws[((size_t)blockIdx.y * p.ws_rows + c) * p.N + row] = v[j];
                            } else {
                                float *dst = p.Yf + (size_t)c * p.N + row;
                                const float tt = v[j] + bias;
                                if (EPI == TEPI_RESADD) *dst += tt;
                                else *dst = tt;
                            }
                        }
                    }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)p.tmem_cols) : "memory");
    }
}

template <int EPI>
__global__ void __launch_bounds__(192) tc_gemm_kernel(const __grid_constant__ CUtensorMap tmW, const TcGemmParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t s_full[8], s_empty[8], s_acc;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    pdl_launch();
    const int m = p.desc->m;   // set before the kernel that precedes this one was launched
    if (m <= 0) return;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n0 = blockIdx.x * kTcTileW * p.w_tiles;
    const int kb_total = (p.K + kTcBlockK - 1) / kTcBlockK;
    const int kb_per = (kb_total + p.k_splits - 1) / p.k_splits;
    const int kb0 = blockIdx.y * kb_per;
    const int kb1 = min(kb_total, kb0 + kb_per);
    const int n_kb = kb1 - kb0;
    if (n_kb <= 0) return;   // uniform for the CTA

    const uint32_t a_bytes = (uint32_t)p.m_pad * kTcBlockK * 2;
    // the pass may hold fewer rows than the launch was sized for: load and multiply only those (rounded up to 32)
    const int m_eff = min(p.m_pad, (m + 31) & ~31);
    const uint32_t a_bytes_eff = (uint32_t)m_eff * kTcBlockK * 2;
    const CUtensorMap *tmAhi = p.act_hi + (m_eff / 32 - 1), *tmAlo = p.act_lo + (m_eff / 32 - 1);
    const uint32_t w_bytes = (uint32_t)p.w_tiles * kTcWBytes;
    const uint32_t stage_bytes = w_bytes + 2 * a_bytes;
    const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;   // 1024-byte aligned tile area

    if (tid == 0) {
        s_abort = 0;
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&s_full[s]), 1);
            mbar_init(smem_u32(&s_empty[s]), 1);
        }
        mbar_init(smem_u32(&s_acc), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)), "r"((uint32_t)p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s_tmem_base;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            int armed = 0;
            auto load_w = [&](int i) {   // arm the stage of K block i and fetch its weight tiles
                const int s = i % p.stages;
                const uint32_t full = smem_u32(&s_full[s]);
                const uint32_t base = tiles + (uint32_t)s * stage_bytes;
                mbar_expect_tx(full, w_bytes + 2 * a_bytes_eff);
                const int kx = (kb0 + i) * kTcBlockK;
                for (int t = 0; t < p.w_tiles; ++t) tma_load_2d(base + (uint32_t)t * kTcWBytes, &tmW, kx, n0 + t * kTcTileW, full);
            };
            // the weights do not depend on the kernel before this one: the first trip round the ring fetches them
            // while that kernel may still be running; the activations follow once it is complete
            const int pre = min(n_kb, p.stages);
            for (int i = 0; i < pre; ++i) load_w(i);
            pdl_wait();
            for (int i = 0; i < n_kb; ++i) {
                const int s = i % p.stages, u = i / p.stages;
                if (u > 0) {
                    if (!mbar_wait(smem_u32(&s_empty[s]), (u - 1) & 1, &s_abort, p.status)) break;
                    load_w(i);
                }
                const uint32_t full = smem_u32(&s_full[s]);
                const uint32_t base = tiles + (uint32_t)s * stage_bytes;
                const int kx = (kb0 + i) * kTcBlockK;
                tma_load_2d(base + w_bytes, tmAhi, kx, 0, full);
                tma_load_2d(base + w_bytes + a_bytes, tmAlo, kx, 0, full);
                armed = i + 1;
            }
            if (s_abort) {
                // give the copies already issued a bounded time to land before the CTA leaves
                for (int i = max(0, armed - p.stages); i < armed; ++i) {
                    const int s = i % p.stages, u = i / p.stages;
                    for (uint32_t it = 0; it < (1u << 16) && !mbar_try(smem_u32(&s_full[s]), u & 1); ++it) __nanosleep(128);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(m_eff);
            bool ok = true;
            for (int i = 0; i < n_kb && ok; ++i) {
                const int s = i % p.stages, u = i / p.stages;
                ok = mbar_wait(smem_u32(&s_full[s]), u & 1, &s_abort, p.status);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t base = tiles + (uint32_t)s * stage_bytes;
                const uint64_t dh = umma_desc_sw128(base + w_bytes);
                const uint64_t dl = umma_desc_sw128(base + w_bytes + a_bytes);
                for (int t = 0; t < p.w_tiles; ++t) {
                    const uint64_t dw = umma_desc_sw128(base + (uint32_t)t * kTcWBytes);
                    const uint32_t acc = tmem + (uint32_t)(t * p.m_pad);   // this tile's accumulator columns
#pragma unroll
                    for (int k4 = 0; k4 < kTcBlockK / 16; ++k4)   // 16 elements = 32 bytes = 2 descriptor units
                        umma_bf16(acc, dw + 2 * k4, dh + 2 * k4, idesc, (i > 0 || k4 > 0) ? 1u : 0u);
#pragma unroll
                    for (int k4 = 0; k4 < kTcBlockK / 16; ++k4)
                        umma_bf16(acc, dw + 2 * k4, dl + 2 * k4, idesc, 1u);
                }
                umma_commit(smem_u32(&s_empty[s]));
            }
            if (ok) umma_commit(smem_u32(&s_acc));
        }
    } else {
        // ---------------- epilogue: TMEM -> registers -> global ----------------
        const int q = warp & 3;                 // TMEM lane quarter this warp may read
        pdl_wait();                             // the residual and the outputs belong to the kernels before this one
        int ok_i = lane == 0 ? (int)mbar_wait(smem_u32(&s_acc), 0, &s_abort, p.status) : 1;
        const bool ok = __shfl_sync(0xffffffffu, ok_i, 0) != 0;   // one poller per warp, uniform outcome
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok) {
            for (int t = 0; t < p.w_tiles; ++t) {
                const int row = n0 + t * kTcTileW + q * 32 + lane;     // weight row = output feature
                const float bias = (EPI != TEPI_SILU && p.bias && blockIdx.y == 0 && row < p.N) ? p.bias[row] : 0.f;
                for (int c0 = 0; c0 < m; c0 += 16) {
                    float v[16];
                    tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(t * p.m_pad + c0), v);
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int c = c0 + j;
                        if (EPI == TEPI_SILU) {
                            const float other = __shfl_xor_sync(0xffffffffu, v[j], 1);
                            if (c < m && !(lane & 1) && row + 1 < p.N) {
                                const size_t o = (size_t)c * (p.N >> 1) + (row >> 1);
                                split_bf16(v[j] / (1.f + expf(-v[j])) * other, p.Yb_hi[o], p.Yb_lo[o]);
                            }
                        } else if (c < m && row < p.N) {
                            if (p.k_splits > 1) {
                                p.Ws[((size_t)blockIdx.y * p.ws_rows + c) * p.N + row] = v[j];
                            } else {
                                float *dst = p.Yf + (size_t)c * p.N + row;
                                const float tt = v[j] + bias;
                                if (EPI == TEPI_RESADD) *dst += tt;
                                else *dst = tt;
                            }
                        }
                    }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)p.tmem_cols) : "memory");
    }
}

}  // namespace st
