// Host side of libst.so: model construction, paged KV bookkeeping, pass scheduling and the C ABI.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/st.h"
#include "attention.cuh"
#include "decode_mega.cuh"
#include "attn_rows_mma.cuh"
#include "gemv.cuh"
#include "prefill_simt.cuh"
#include "router.cuh"
#include "tc_gemm.cuh"
#include "weights.cuh"

#include <cstdlib>
#include <map>

using namespace st;

#define CK(expr)                                                     \
    do {                                                             \
        cudaError_t e_ = (expr);                                     \
        if (e_ != cudaSuccess) {                                     \
            set_error_text(#expr, e_);                               \
            return e_ == cudaErrorMemoryAllocation ? ST_ERR_OOM : ST_ERR_INTERNAL; \
        }                                                            \
    } while (0)
#define TRY(expr)                  \
    do {                           \
        int rc_ = (expr);          \
        if (rc_ != ST_OK) return rc_; \
    } while (0)

static thread_local char g_err_text[256];
static int64_t g_launches = 0;  // kernels launched by this library in this process
static void set_error_text(const char *what, cudaError_t e)
{
    snprintf(g_err_text, sizeof g_err_text, "%s: %s", what, cudaGetErrorString(e));
}

// Layer-local tensor ids of the seeded streams (stream id = 16 * (layer + 1) + id; 0 = embedding,
// 1 = LM head).
enum { TID_WQ = 1, TID_WK = 2, TID_WV = 3, TID_BQ = 4, TID_BK = 5, TID_BV = 6, TID_WO = 7, TID_WG = 9, TID_WU = 10, TID_WD = 11 };

struct LayerMaps {   // TMA descriptors of one layer's weight matrices
    CUtensorMap wqkv, wo, wgu, wd;
};

struct LayerWeights {
    uint16_t *wqkv;  // [(Hq + 2 Hkv) D][h]: q rows, k rows, v rows
    float *bqkv;     // [(Hq + 2 Hkv) D]
    uint16_t *wo;    // [h][Hq D]
    uint16_t *wgu;   // [2 f][h]: row 2j = gate j, row 2j + 1 = up j
    uint16_t *wd;    // [h][f]
    float *g1, *g2;  // norm gains [h]
};

struct GenContext;

struct st_model {
    st_config cfg{};
    uint64_t id = 0;                 // unique per created model
    GenContext *gen_ctx = nullptr;   // generation buffers + graph with this model as the speculative one
    uint64_t seed = 0;
    uint32_t tag = 0;
    cudaStream_t stream = nullptr;
    int device = 0, sm_count = 148;
    std::vector<void *> allocations;

    // weights
    uint16_t *embed = nullptr, *lm_head = nullptr;
    float *gf = nullptr;
    std::vector<LayerWeights> layers;
    std::vector<LayerMaps> maps;
    CUtensorMap map_lm{};                  // LM head in 128-row tiles (batched decode)
    int32_t *row_slot = nullptr, *row_pos = nullptr;   // device [max_rows]: sequence and position of every row of a batched decode pass
    float *batch_logits = nullptr;         // [max_rows][vocab], allocated on first use
    struct BatchGraph {                    // a captured batched decode pass, keyed by everything baked into its nodes
        int m_upper, vlimit, tile;         // tile: keys per attention tile (chosen from the context bound)
        const int32_t *tok;
        const StepDesc *desc;
        float *logits;
        int32_t *argmax;
        cudaGraphExec_t exec;
        int64_t launches;
    };
    std::vector<BatchGraph> batch_graphs;
    cudaStream_t cap_stream = nullptr;     // side stream the batched pass is captured on (the model's own may be the legacy stream)
    CUtensorMap *act_maps = nullptr;       // device [3 buffers][2 planes][8]: activation planes in boxes of 32 (j + 1) rows
    CUtensorMap *act_maps_half = nullptr;  // device [3 buffers][2 planes][16]: the same in boxes of 16 (j + 1) rows (CTA pairs)
    bool simt_gemm = false;                // debugging aid: multi-row projections on the CUDA cores
    bool simt_attn = false;                // debugging aid: multi-row attention on the CUDA cores
    double *inv_freq = nullptr;
    int64_t weight_bytes = 0;

    // paged KV
    int n_pages = 0, pages_per_seq = 0, page_shift = 0;
    uint16_t *kpool = nullptr, *vpool = nullptr;
    size_t pool_layer_stride = 0;  // elements per layer
    int32_t *block_tab = nullptr;  // device [max_seqs][pages_per_seq]
    std::vector<int32_t> free_pages;
    std::vector<std::vector<int32_t>> seq_pages;
    std::vector<int32_t> seq_len;  // host view (explicit prefill/decode calls)
    std::vector<uint8_t> seq_used;

    // scratch
    int max_rows = 0;          // rows per multi-row pass
    int max_splits = 0;
    float *X = nullptr;        // [max_rows][h] residual stream
    uint16_t *XN = nullptr;    // [2][max_rows][h] hi/lo planes
    float *QKV = nullptr;      // [max_rows][(Hq + 2 Hkv) D]
    float *ATT = nullptr;      // [Hq D] (decode)
    uint16_t *ATTb = nullptr;  // [2][max_rows][Hq D]
    float *ACT = nullptr;      // [f] (decode)
    uint16_t *ACTb = nullptr;  // [2][max_rows][f]
    float *splitk_ws = nullptr;  // [kMaxKSplits][max_rows][max(qkv width, h)] partial sums of K-split projections
    float2 *cs = nullptr;      // [max_rows][D / 2]
    float *logits = nullptr;   // [vocab]
    float *part_o = nullptr, *part_ml = nullptr;
    int32_t *tickets = nullptr;  // [max_rows * Hkv + 1]; last entry serves the argmax kernel
    float *amax_val = nullptr;
    int32_t *amax_idx = nullptr;
    int32_t *tokbuf = nullptr;   // [max_rows] staging for explicit calls
    StepDesc *desc = nullptr;    // device
    int32_t *status = nullptr;   // device sticky status word
    // single-kernel decode step
    MegaLayer *mega_layers = nullptr;   // device [n_layers]
    CUtensorMap *mega_maps = nullptr;   // device [4 * n_layers + 1]
    float *X0 = nullptr, *X1 = nullptr, *D1 = nullptr, *D2 = nullptr;   // [h] each
    unsigned *mega_sync = nullptr;      // [4]
    int32_t *mega_tickets = nullptr;    // [Hkv]
    int mega_stages = 0, mega_xarea = 0, mega_splits = 0, mega_kv_off = 0, mega_kv_cap = 0, mega_down_slab = 0, mega_unit_keys = 64;
    size_t mega_smem = 0;
    bool multi_kernel_decode = false;   // debugging aid: one kernel per phase instead

    void *dalloc(size_t bytes)
    {
        void *p = nullptr;
        if (bytes == 0) bytes = 16;
        if (cfg.alloc) p = cfg.alloc(bytes, cfg.alloc_user);
        else if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); p = nullptr; }
        if (p) allocations.push_back(p);
        return p;
    }
};

static constexpr int kArgmaxBlocks = 64;
static constexpr int kGemvWarps = 8;
static constexpr int kMegaSyncWords = 32 * (1 + kMegaBarCounters);   // ticket/abort words + one 128-byte line per barrier counter
static constexpr int kMaxKSplits = 8;  // most K splits of a multi-row projection (add_splits4 holds as many loads)

// Threads of a one-CTA-per-row kernel with `items` independent work items: the fewest passes over the row that
// `cap` threads allow, spread evenly (a row is latency bound, so as many loads as possible should be in flight).
static int row_threads(int items, int cap)
{
    const int passes = (items + cap - 1) / cap;
    const int t = ((items + passes - 1) / passes + 31) / 32 * 32;
    return t < 128 ? 128 : t;
}
static constexpr int kMaxAuxTokens = 64;   // longest auxiliary sentence of takeover (3)
static constexpr int kRowSplits = 8;   // most key splits a multi-row pass uses

// ------------------------------------------------------------------------------------------------
// launch helpers
// ------------------------------------------------------------------------------------------------

// Programmatic dependent launch lets a weight-streaming kernel fetch its first weights while its
// predecessor drains (ST_PDL=0 turns it off for debugging).
static bool use_pdl()
{
    static const bool on = [] { const char *e = getenv("ST_PDL"); return !(e && e[0] == '0'); }();
    return on;
}

template <int S, int PRO, int EPI>
static cudaError_t launch_gemv_s(const GemvParams &p, cudaStream_t s, int sms)
{
    constexpr int NW = kGemvWarps, R = 2, U = 4;
    auto kern = gemv_kernel<NW, S, R, U, PRO, EPI>;
    const size_t smem = (size_t)p.K * 4 + 2 * NW * R * 4;
    const int G = NW / S;
    const int n_tasks = (p.N + R - 1) / R;
    const int ctas_needed = (n_tasks + G - 1) / G;
    // persistent CTAs: as many as are resident at once (at most two per SM, leaving room for the
    // next kernel of the chain to start its prefetch)
    static int occ_cache[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    const int bucket = smem <= 8 * 1024 ? 0 : smem <= 24 * 1024 ? 1 : smem <= 48 * 1024 ? 2 : smem <= 80 * 1024 ? 3 : 4;
    if (!occ_cache[bucket]) {
        int n = 0;
        const cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, NW * 32, smem);
        if (e != cudaSuccess) return e;
        occ_cache[bucket] = n < 1 ? 1 : n > 2 ? 2 : n;
    }
    int grid = sms * occ_cache[bucket];
    if (grid > ctas_needed) grid = ctas_needed;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(NW * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = use_pdl() ? 1 : 0;
    ++g_launches;
    return cudaLaunchKernelEx(&cfg, kern, p);
}

template <int S, int PRO, int EPI>
static cudaError_t gemv_attr()
{
    return cudaFuncSetAttribute(gemv_kernel<kGemvWarps, S, 2, 4, PRO, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
}

template <int PRO, int EPI>
static cudaError_t gemv_attr_all()
{
    cudaError_t e = gemv_attr<1, PRO, EPI>();
    if (e == cudaSuccess) e = gemv_attr<2, PRO, EPI>();
    if (e == cudaSuccess) e = gemv_attr<4, PRO, EPI>();
    if (e == cudaSuccess) e = gemv_attr<8, PRO, EPI>();
    return e;
}

template <int PRO, int EPI>
static cudaError_t launch_gemv(const GemvParams &p, cudaStream_t s, int sms)
{
    const int n_chunks = (p.K + 255) / 256;
    if (n_chunks >= 64) return launch_gemv_s<8, PRO, EPI>(p, s, sms);
    if (n_chunks >= 16) return launch_gemv_s<4, PRO, EPI>(p, s, sms);
    if (n_chunks >= 8) return launch_gemv_s<2, PRO, EPI>(p, s, sms);
    return launch_gemv_s<1, PRO, EPI>(p, s, sms);
}

template <int D>
static cudaError_t launch_attn_d(const AttnParams &p, int G, dim3 grid, cudaStream_t s)
{
    switch (G) {
    case 1: attn_kernel<D, 1><<<grid, 128, 0, s>>>(p); break;
    case 2: attn_kernel<D, 2><<<grid, 128, 0, s>>>(p); break;
    case 3: attn_kernel<D, 3><<<grid, 128, 0, s>>>(p); break;
    case 4: attn_kernel<D, 4><<<grid, 128, 0, s>>>(p); break;
    case 5: attn_kernel<D, 5><<<grid, 128, 0, s>>>(p); break;
    case 6: attn_kernel<D, 6><<<grid, 128, 0, s>>>(p); break;
    case 7: attn_kernel<D, 7><<<grid, 128, 0, s>>>(p); break;
    case 8: attn_kernel<D, 8><<<grid, 128, 0, s>>>(p); break;
    default: return cudaErrorInvalidValue;
    }
    ++g_launches;
    return cudaGetLastError();
}

template <int D>
static cudaError_t launch_attn_rows_d(const AttnParams &p, int G, dim3 grid, cudaStream_t s)
{
    switch (G) {
    case 1: attn_rows_kernel<D, 1><<<grid, 256, 0, s>>>(p); break;
    case 2: attn_rows_kernel<D, 2><<<grid, 256, 0, s>>>(p); break;
    case 3: attn_rows_kernel<D, 3><<<grid, 256, 0, s>>>(p); break;
    case 4: attn_rows_kernel<D, 4><<<grid, 256, 0, s>>>(p); break;
    case 5: attn_rows_kernel<D, 5><<<grid, 256, 0, s>>>(p); break;
    case 6: attn_rows_kernel<D, 6><<<grid, 256, 0, s>>>(p); break;
    case 7: attn_rows_kernel<D, 7><<<grid, 256, 0, s>>>(p); break;
    case 8: attn_rows_kernel<D, 8><<<grid, 256, 0, s>>>(p); break;
    default: return cudaErrorInvalidValue;
    }
    ++g_launches;
    return cudaGetLastError();
}

// grid = (key splits, kv heads, ceil(rows / 8))
static cudaError_t launch_attn_rows(const AttnParams &p, int D, int G, dim3 grid, cudaStream_t s)
{
    if (D == 64) return launch_attn_rows_d<64>(p, G, grid, s);
    if (D == 128) return launch_attn_rows_d<128>(p, G, grid, s);
    return cudaErrorInvalidValue;
}

// Tensor-core multi-row attention: grid = (key splits, kv heads, ceil(rows / (64 / G))).
template <int D, int G>
static cudaError_t launch_attn_rows_mma_dg(const AttnRowsMmaParams &p, dim3 grid, cudaStream_t s, bool attr_only)
{
    auto kern = attn_rows_mma_kernel<D, G>;
    const size_t smem = 1024 + (size_t)kArStages * ar_stage_bytes<D>();
    if (attr_only) return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    kern<<<grid, kArThreads, smem, s>>>(p);
    ++g_launches;
    return cudaGetLastError();
}

template <int D>
static cudaError_t launch_attn_rows_mma_d(const AttnRowsMmaParams &p, int G, dim3 grid, cudaStream_t s, bool attr_only)
{
    switch (G) {
    case 1: return launch_attn_rows_mma_dg<D, 1>(p, grid, s, attr_only);
    case 2: return launch_attn_rows_mma_dg<D, 2>(p, grid, s, attr_only);
    case 3: return launch_attn_rows_mma_dg<D, 3>(p, grid, s, attr_only);
    case 4: return launch_attn_rows_mma_dg<D, 4>(p, grid, s, attr_only);
    case 5: return launch_attn_rows_mma_dg<D, 5>(p, grid, s, attr_only);
    case 6: return launch_attn_rows_mma_dg<D, 6>(p, grid, s, attr_only);
    case 7: return launch_attn_rows_mma_dg<D, 7>(p, grid, s, attr_only);
    case 8: return launch_attn_rows_mma_dg<D, 8>(p, grid, s, attr_only);
    }
    return cudaErrorInvalidValue;
}

static cudaError_t launch_attn_rows_mma(const AttnRowsMmaParams &p, int D, int G, dim3 grid, cudaStream_t s, bool attr_only = false)
{
    if (D == 64) return launch_attn_rows_mma_d<64>(p, G, grid, s, attr_only);
    if (D == 128) return launch_attn_rows_mma_d<128>(p, G, grid, s, attr_only);
    return cudaErrorInvalidValue;
}

// Batched decode attention: grid = (kv heads, rows); tk = keys per tile (64 or 128).
template <int D, int G, int TK>
static cudaError_t launch_attn_batch_dgt(const AttnBatchParams &p, dim3 grid, cudaStream_t s, bool attr_only)
{
    auto kern = attn_batch_mma_kernel<D, G, TK>;
    const size_t smem = 1024 + (size_t)kAbStages * ab_stage_bytes<D, TK>();
    if (attr_only) return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    kern<<<grid, 2 * TK, smem, s>>>(p);
    ++g_launches;
    return cudaGetLastError();
}

template <int D, int G>
static cudaError_t launch_attn_batch_dg(const AttnBatchParams &p, dim3 grid, cudaStream_t s, int tk, bool attr_only)
{
    if (attr_only) {
        const cudaError_t e = launch_attn_batch_dgt<D, G, 64>(p, grid, s, true);
        return e != cudaSuccess ? e : launch_attn_batch_dgt<D, G, 128>(p, grid, s, true);
    }
    return tk == 64 ? launch_attn_batch_dgt<D, G, 64>(p, grid, s, false) : launch_attn_batch_dgt<D, G, 128>(p, grid, s, false);
}

template <int D>
static cudaError_t launch_attn_batch_d(const AttnBatchParams &p, int G, dim3 grid, cudaStream_t s, int tk, bool attr_only)
{
    switch (G) {
    case 1: return launch_attn_batch_dg<D, 1>(p, grid, s, tk, attr_only);
    case 2: return launch_attn_batch_dg<D, 2>(p, grid, s, tk, attr_only);
    case 3: return launch_attn_batch_dg<D, 3>(p, grid, s, tk, attr_only);
    case 4: return launch_attn_batch_dg<D, 4>(p, grid, s, tk, attr_only);
    case 5: return launch_attn_batch_dg<D, 5>(p, grid, s, tk, attr_only);
    case 6: return launch_attn_batch_dg<D, 6>(p, grid, s, tk, attr_only);
    case 7: return launch_attn_batch_dg<D, 7>(p, grid, s, tk, attr_only);
    case 8: return launch_attn_batch_dg<D, 8>(p, grid, s, tk, attr_only);
    }
    return cudaErrorInvalidValue;
}

static cudaError_t launch_attn_batch(const AttnBatchParams &p, int D, int G, dim3 grid, cudaStream_t s, int tk, bool attr_only = false)
{
    if (D == 64) return launch_attn_batch_d<64>(p, G, grid, s, tk, attr_only);
    if (D == 128) return launch_attn_batch_d<128>(p, G, grid, s, tk, attr_only);
    return cudaErrorInvalidValue;
}

// Keys per tile of the batched attention: 64 (two CTAs per SM) was the faster one at every context measured,
// 512 to 4000 keys; ST_AB_TILE=128 selects the 128-key kernel.
static int attn_batch_tile(int ctx_upper)
{
    (void)ctx_upper;
    static const int forced = [] { const char *e = getenv("ST_AB_TILE"); return e ? atoi(e) : 0; }();
    return forced == 128 ? 128 : 64;
}

static cudaError_t launch_attn(const AttnParams &p, int D, int G, dim3 grid, cudaStream_t s)
{
    if (D == 64) return launch_attn_d<64>(p, G, grid, s);
    if (D == 128) return launch_attn_d<128>(p, G, grid, s);
    return cudaErrorInvalidValue;
}

template <int EPI>
static cudaError_t launch_gemm(const GemmParams &p, int m_upper, cudaStream_t s)
{
    dim3 grid((p.N + 63) / 64, (m_upper + 63) / 64);
    gemm_simt_kernel<EPI><<<grid, 256, 0, s>>>(p);
    ++g_launches;
    return cudaGetLastError();
}

// ---- TMA descriptors and the tensor-core GEMM launcher ----

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// 2-D bf16 tensor [rows][K] (K contiguous), boxes of box_k x box_rows elements (64 wide with the
// 128-byte swizzle by default), out-of-range elements read as zero.
static int make_map_bf16(CUtensorMap *map, const void *base, uint64_t rows, uint64_t K, uint32_t box_rows,
                         uint32_t box_k = kTcBlockK, bool swizzle128 = true)
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) {
        snprintf(g_err_text, sizeof g_err_text, "cuTensorMapEncodeTiled is not available");
        return ST_ERR_INTERNAL;
    }
    const cuuint64_t gdim[2] = {K, rows};
    const cuuint64_t gstride[1] = {K * 2};
    const cuuint32_t box[2] = {box_k, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), gdim, gstride, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(g_err_text, sizeof g_err_text, "cuTensorMapEncodeTiled failed (%d)", (int)r);
        return ST_ERR_INTERNAL;
    }
    return ST_OK;
}

// Whether the multi-row projections are launched with programmatic stream serialization: not inside the bodies of
// the generation graph's conditional nodes (g_pdl_off > 0), and never with ST_PDL=0.
static int g_pdl_off = 0;
static bool pdl_enabled() { return use_pdl() && g_pdl_off == 0; }

// Launch of a kernel that begins with pdl_launch(); pdl_wait(): with programmatic stream serialization its CTAs are
// scheduled while the kernel before it drains.
template <typename... KArgs, typename... Args>
static cudaError_t launch_dependent(void (*kern)(KArgs...), dim3 grid, dim3 block, cudaStream_t s, Args... args)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    ++g_launches;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// Passes of at least this many rows run on CTA pairs (0: never): below it the activation tiles are small beside the
// weight tiles and a pair gains nothing.
static int tc_pair_min_rows()
{
    static const int v = [] { const char *e = getenv("ST_TC_PAIR_MIN"); return e ? atoi(e) : 96; }();
    return v;
}

// Shared memory a projection CTA spends on its pipeline stages.  With at most half of an SM's shared memory (and of its
// tensor memory) per CTA two CTAs share an SM: while one drains its accumulators the other -- of the same kernel or,
// launched as a programmatic dependent, of the next -- already streams weights.
// Measured on the 32B: passes of up to 64 rows gain 3 % that way (20 rows 16.3 -> 15.7 ms, 64 rows 19.0 -> 18.4 ms), wider
// ones lose 2 % (their activation tiles leave too few stages in half an SM), so the default halves the budget up to 64 rows.
static int tc_stage_smem(int m_pad)
{
    static const int forced = [] { const char *e = getenv("ST_TC_SMEM_KB"); const int kb = e ? atoi(e) : 0; return kb <= 0 ? 0 : (kb < 64 ? 64 : kb > 220 ? 220 : kb) * 1024; }();
    return forced ? forced : (m_pad <= 64 ? 108 : 220) * 1024;
}

template <int EPI>
// pending_splits: when given, a K-split projection leaves its partial sums in the workspace and reports the split
// count there (0: the output is complete) -- the kernel that consumes the output adds them up.
static int launch_tc_gemm(const CUtensorMap &tw, TcGemmParams p, int m_upper, int sms, cudaStream_t s, int *pending_splits = nullptr)
{
    p.m_pad = (m_upper + 31) / 32 * 32;
    if (p.m_pad > 256) return ST_ERR_INTERNAL;
    const bool pair = tc_pair_min_rows() > 0 && p.m_pad >= tc_pair_min_rows();
    auto kern = pair ? tc_gemm_pair_kernel<EPI> : tc_gemm_kernel<EPI>;
    const int a_rows = pair ? p.m_pad / 2 : p.m_pad;   // activation rows a CTA loads per plane and stage
    // two CTAs per SM when two stages of one weight tile fit the halved budget; the whole SM otherwise
    const int smem_want = tc_stage_smem(p.m_pad);
    const bool shared_sm = smem_want <= 110 * 1024 && 2 * (kTcWBytes + 2 * a_rows * kTcBlockK * 2) <= smem_want && p.m_pad <= 256;
    const int smem_budget = shared_sm ? smem_want : 220 * 1024, tmem_budget = shared_sm ? 256 : 512;
    const int slots = shared_sm ? 2 * sms : sms;   // CTAs resident at a time
    // 128-row weight tiles per CTA (they share the activation tiles of a stage): bounded by TMEM (512 columns) and
    // by two pipeline stages of shared memory; among the candidates take the one whose CTA count fills whole waves
    // of SMs best (a projection with 1.46 waves of CTAs runs as long as one with 2), the larger on a tie.
    int wt = 1;
    {
        double best = -1.0;
        for (int cand = 4; cand >= 1; --cand) {
            if (cand * p.m_pad > tmem_budget) continue;
            if (2 * (cand * kTcWBytes + 2 * a_rows * kTcBlockK * 2) > smem_budget) continue;
            const int tiles = (p.N + kTcTileW * cand - 1) / (kTcTileW * cand);
            // projections that may split K fill the machine through the split; the others only through tiles
            int split = tiles >= slots ? 1 : slots / tiles;   // K splits: as many as still fit one wave
            split = split > kMaxKSplits ? kMaxKSplits : split;
            const int ctas = EPI == TEPI_SILU ? tiles : tiles * split;
            const int waves = (ctas + slots - 1) / slots;
            const double eff = (double)ctas / ((double)waves * slots);
            if (eff > best + 0.03) { best = eff; wt = cand; }
        }
    }
    {   // tuning aid: force the weight tiles per CTA (when the forced count fits tensor and shared memory)
        static const int forced = [] { const char *e = getenv("ST_TC_WT"); return e ? atoi(e) : 0; }();
        if (forced >= 1 && forced <= 4 && forced * p.m_pad <= tmem_budget && 2 * (forced * kTcWBytes + 2 * a_rows * kTcBlockK * 2) <= smem_budget) wt = forced;
    }
    p.w_tiles = wt;
    int cols = wt * p.m_pad;
    p.tmem_cols = cols <= 32 ? 32 : cols <= 64 ? 64 : cols <= 128 ? 128 : cols <= 256 ? 256 : 512;
    const int stage_bytes = wt * kTcWBytes + 2 * a_rows * kTcBlockK * 2;
    int stages = smem_budget / stage_bytes;
    p.stages = stages > 8 ? 8 : stages;
    int n_tiles = (p.N + kTcTileW * wt - 1) / (kTcTileW * wt);
    if (pair) n_tiles = (n_tiles + 1) & ~1;   // whole pairs: a CTA beyond the matrix multiplies zero-filled tiles and stores nothing
    const int kb_total = (p.K + kTcBlockK - 1) / kTcBlockK;
    int ks = 1;
    if (EPI != TEPI_SILU) {
        ks = n_tiles >= slots ? 1 : slots / n_tiles;
        const int ks_max = kb_total / 8 > 1 ? kb_total / 8 : 1;
        ks = ks > ks_max ? ks_max : ks;
        ks = ks > kMaxKSplits ? kMaxKSplits : ks;
        const int per = (kb_total + ks - 1) / ks;   // no empty split
        ks = (kb_total + per - 1) / per;
    }
    if ((p.N & 3) || !p.Ws) ks = 1;
    p.k_splits = ks;
    const size_t smem = (size_t)p.stages * stage_bytes + 1024;
    // programmatic dependent launch: the CTAs may become resident, set up and fetch their first weight tiles while
    // the kernel before this one is still running (it reads that kernel's output only after griddepcontrol.wait)
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(n_tiles, ks);
    cfg.blockDim = dim3(192);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    CK(cudaLaunchKernelEx(&cfg, kern, tw, p));
    ++g_launches;
    if (pending_splits) {
        *pending_splits = ks > 1 ? ks : 0;
        return ST_OK;
    }
    if (ks > 1) {
        int gx = (p.N / 4 + 255) / 256;
        splitk_reduce_kernel<<<dim3(gx, m_upper), 256, 0, s>>>(p.desc, p.Ws, ks, p.ws_rows, p.N, p.bias, p.Yf, EPI == TEPI_RESADD ? 1 : 0);
        ++g_launches;
        CK(cudaGetLastError());
    }
    return ST_OK;
}

// ------------------------------------------------------------------------------------------------
// model construction
// ------------------------------------------------------------------------------------------------

static int fill_rows(st_model *m, uint16_t *out, uint32_t tid, uint64_t rows, uint64_t cols, uint32_t row_mul, uint32_t row_add)
{
    const uint64_t key = tensor_stream_key(m->seed, m->tag, tid);
    const uint64_t n = rows * cols;
    int blocks = (int)((n + 255) / 256 < 148 * 16 ? (n + 255) / 256 : 148 * 16);
    fill_bf16_kernel<<<blocks, 256, 0, m->stream>>>(out, key, 0, rows, cols, row_mul, row_add);
    ++g_launches;
    CK(cudaGetLastError());
    return ST_OK;
}

static int fill_f32(st_model *m, float *out, uint32_t tid, uint64_t n)
{
    const uint64_t key = tensor_stream_key(m->seed, m->tag, tid);
    fill_f32_kernel<<<(int)((n + 255) / 256), 256, 0, m->stream>>>(out, key, n);
    ++g_launches;
    CK(cudaGetLastError());
    return ST_OK;
}

static int fill_const(st_model *m, float *out, float v, uint64_t n)
{
    fill_const_f32_kernel<<<(int)((n + 255) / 256), 256, 0, m->stream>>>(out, v, n);
    ++g_launches;
    CK(cudaGetLastError());
    return ST_OK;
}

static int mega_attr_all();

// Opt every kernel into the shared memory it may ask for (once per device, outside any capture).
static int init_kernel_attributes()
{
    CK((gemv_attr_all<PRO_NORM, EPI_STORE>()));
    CK((gemv_attr_all<PRO_PLAIN, EPI_RESADD>()));
    CK((gemv_attr_all<PRO_NORM, EPI_SILU>()));
    CK(cudaFuncSetAttribute(tc_gemm_kernel<TEPI_STORE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024));
    CK(cudaFuncSetAttribute(tc_gemm_kernel<TEPI_RESADD>, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024));
    CK(cudaFuncSetAttribute(tc_gemm_kernel<TEPI_SILU>, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024));
    CK(cudaFuncSetAttribute(tc_gemm_pair_kernel<TEPI_STORE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024));
    CK(cudaFuncSetAttribute(tc_gemm_pair_kernel<TEPI_RESADD>, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024));
    CK(cudaFuncSetAttribute(tc_gemm_pair_kernel<TEPI_SILU>, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024));
    return mega_attr_all();
}

static size_t mega_scratch_bytes(int D, int G)
{
    // sizeof(MegaAttnScratch<D, G>)
    return sizeof(float) * ((size_t)kMegaAttnWarps * G * D + 2 * (size_t)kMegaAttnWarps * G);
}

static int mega_attr_all();

static int check_config(const st_config *c)
{
    if (!c) return ST_ERR_ARG;
    if (c->n_layers < 1 || c->n_layers > 128 || c->hidden < 8 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->ffn < 8 ||
        c->vocab < 2 || c->max_seqs < 1 || c->max_tokens < 1)
        return ST_ERR_ARG;
    if (c->n_q_heads % c->n_kv_heads) return ST_ERR_ARG;
    if (c->head_dim != 64 && c->head_dim != 128) return ST_ERR_UNSUPPORTED;
    if (c->n_q_heads / c->n_kv_heads > 8) return ST_ERR_UNSUPPORTED;
    if (c->hidden % 8 || c->ffn % 8) return ST_ERR_UNSUPPORTED;
    if ((int64_t)c->hidden * 4 > 160 * 1024 || (int64_t)c->ffn * 4 > 160 * 1024) return ST_ERR_UNSUPPORTED;
    if (c->page_size != 16 && c->page_size != 32 && c->page_size != 64) return ST_ERR_ARG;
    if (!(c->rope_theta > 0.f) || !(c->rms_eps >= 0.f)) return ST_ERR_ARG;
    if ((c->alloc == nullptr) != (c->free == nullptr)) return ST_ERR_ARG;
    return ST_OK;
}

static int model_build(st_model *m)
{
    const st_config &c = m->cfg;
    const int h = c.hidden, D = c.head_dim, qd = c.n_q_heads * D, kd = c.n_kv_heads * D, f = c.ffn;
    const int qkvd = qd + 2 * kd;
    CK(cudaGetDevice(&m->device));
    CK(cudaDeviceGetAttribute(&m->sm_count, cudaDevAttrMultiProcessorCount, m->device));
    TRY(init_kernel_attributes());

#define ALLOC(ptr, type, count)                                      \
    do {                                                             \
        ptr = (type *)m->dalloc((size_t)(count) * sizeof(type));     \
        if (!ptr) return ST_ERR_OOM;                                 \
    } while (0)

    // ---- weights ----
    ALLOC(m->embed, uint16_t, (size_t)c.vocab * h);
    TRY(fill_rows(m, m->embed, 0, c.vocab, h, 1, 0));
    if (c.tie_embeddings) {
        m->lm_head = m->embed;
    } else {
        ALLOC(m->lm_head, uint16_t, (size_t)c.vocab * h);
        TRY(fill_rows(m, m->lm_head, 1, c.vocab, h, 1, 0));
    }
    ALLOC(m->gf, float, h);
    TRY(fill_const(m, m->gf, 1.f, h));
    m->layers.resize(c.n_layers);
    for (int l = 0; l < c.n_layers; ++l) {
        LayerWeights &w = m->layers[l];
        const uint32_t t = 16u * (uint32_t)(l + 1);
        ALLOC(w.wqkv, uint16_t, (size_t)qkvd * h);
        TRY(fill_rows(m, w.wqkv, t + TID_WQ, qd, h, 1, 0));
        TRY(fill_rows(m, w.wqkv + (size_t)qd * h, t + TID_WK, kd, h, 1, 0));
        TRY(fill_rows(m, w.wqkv + (size_t)(qd + kd) * h, t + TID_WV, kd, h, 1, 0));
        ALLOC(w.bqkv, float, qkvd);
        if (c.qkv_bias) {
            TRY(fill_f32(m, w.bqkv, t + TID_BQ, qd));
            TRY(fill_f32(m, w.bqkv + qd, t + TID_BK, kd));
            TRY(fill_f32(m, w.bqkv + qd + kd, t + TID_BV, kd));
        } else {
            TRY(fill_const(m, w.bqkv, 0.f, qkvd));
        }
        ALLOC(w.wo, uint16_t, (size_t)h * qd);
        TRY(fill_rows(m, w.wo, t + TID_WO, h, qd, 1, 0));
        ALLOC(w.wgu, uint16_t, (size_t)2 * f * h);
        TRY(fill_rows(m, w.wgu, t + TID_WG, f, h, 2, 0));
        TRY(fill_rows(m, w.wgu, t + TID_WU, f, h, 2, 1));
        ALLOC(w.wd, uint16_t, (size_t)h * f);
        TRY(fill_rows(m, w.wd, t + TID_WD, h, f, 1, 0));
        ALLOC(w.g1, float, h);
        ALLOC(w.g2, float, h);
        TRY(fill_const(m, w.g1, 1.f, h));
        TRY(fill_const(m, w.g2, 1.f, h));
    }
    m->maps.resize(c.n_layers);
    TRY(make_map_bf16(&m->map_lm, m->lm_head, c.vocab, h, kTcTileW));
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerWeights &w = m->layers[l];
        TRY(make_map_bf16(&m->maps[l].wqkv, w.wqkv, qkvd, h, kTcTileW));
        TRY(make_map_bf16(&m->maps[l].wo, w.wo, h, qd, kTcTileW));
        TRY(make_map_bf16(&m->maps[l].wgu, w.wgu, 2 * f, h, kTcTileW));
        TRY(make_map_bf16(&m->maps[l].wd, w.wd, h, f, kTcTileW));
    }
    {
        const char *e = getenv("ST_SIMT_GEMM");
        m->simt_gemm = e && e[0] == '1';
        const char *ea = getenv("ST_SIMT_ATTN");
        m->simt_attn = ea && ea[0] == '1';
    }
    {
        const int64_t per_layer = 2ll * ((int64_t)qkvd * h + (int64_t)h * qd + 3ll * f * h) + 4ll * qkvd * (c.qkv_bias ? 1 : 0) + 8ll * h;
        m->weight_bytes = c.n_layers * per_layer + 4ll * h + 2ll * (int64_t)c.vocab * h;
    }
    // rotary frequencies theta^(-2j/D), in double
    {
        std::vector<double> fr(D / 2);
        for (int j = 0; j < D / 2; ++j) fr[j] = std::pow((double)c.rope_theta, -2.0 * (double)j / (double)D);
        ALLOC(m->inv_freq, double, D / 2);
        CK(cudaMemcpyAsync(m->inv_freq, fr.data(), fr.size() * sizeof(double), cudaMemcpyHostToDevice, m->stream));
        CK(cudaStreamSynchronize(m->stream));
    }

    // ---- paged KV ----
    m->page_shift = c.page_size == 16 ? 4 : c.page_size == 32 ? 5 : 6;
    m->n_pages = (c.max_tokens + c.page_size - 1) / c.page_size + c.max_seqs;
    m->pages_per_seq = (c.max_tokens + c.page_size - 1) / c.page_size + 1;
    m->pool_layer_stride = (size_t)m->n_pages * c.n_kv_heads * c.page_size * D;
    ALLOC(m->kpool, uint16_t, m->pool_layer_stride * c.n_layers);
    ALLOC(m->vpool, uint16_t, m->pool_layer_stride * c.n_layers);
    ALLOC(m->block_tab, int32_t, (size_t)c.max_seqs * m->pages_per_seq);
    CK(cudaMemsetAsync(m->block_tab, 0, (size_t)c.max_seqs * m->pages_per_seq * sizeof(int32_t), m->stream));
    m->free_pages.resize(m->n_pages);
    for (int i = 0; i < m->n_pages; ++i) m->free_pages[i] = m->n_pages - 1 - i;
    m->seq_pages.assign(c.max_seqs, {});
    m->seq_len.assign(c.max_seqs, 0);
    m->seq_used.assign(c.max_seqs, 0);

    // ---- scratch ----
    m->max_rows = 256;   // rows of one multi-row pass = the MMA N limit
    m->max_splits = (2 * m->sm_count + c.n_kv_heads - 1) / c.n_kv_heads;
    if (m->max_splits > kMaxAttnSplits) m->max_splits = kMaxAttnSplits;
    ALLOC(m->X, float, (size_t)m->max_rows * h);
    ALLOC(m->XN, uint16_t, 2 * (size_t)m->max_rows * h);
    ALLOC(m->QKV, float, (size_t)m->max_rows * qkvd);
    ALLOC(m->ATT, float, qd);
    ALLOC(m->ATTb, uint16_t, 2 * (size_t)m->max_rows * qd);
    ALLOC(m->ACT, float, f);
    ALLOC(m->ACTb, uint16_t, 2 * (size_t)m->max_rows * f);
    ALLOC(m->splitk_ws, float, (size_t)kMaxKSplits * m->max_rows * (qkvd > h ? qkvd : h));
    {   // TMA descriptors of the GEMM inputs: per buffer and plane, boxes of 32, 64, ... 256 rows
        std::vector<CUtensorMap> maps(3 * 2 * 8);
        const uint16_t *bufs[3] = {m->XN, m->ATTb, m->ACTb};
        const int widths[3] = {h, qd, f};
        for (int b = 0; b < 3; ++b)
            for (int plane = 0; plane < 2; ++plane)
                for (int j = 0; j < 8; ++j)
                    TRY(make_map_bf16(&maps[(b * 2 + plane) * 8 + j], bufs[b] + (size_t)plane * m->max_rows * widths[b],
                                      (uint64_t)m->max_rows, (uint64_t)widths[b], (uint32_t)(32 * (j + 1))));
        ALLOC(m->act_maps, CUtensorMap, maps.size());
        CK(cudaMemcpyAsync(m->act_maps, maps.data(), maps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice, m->stream));
        CK(cudaStreamSynchronize(m->stream));
        std::vector<CUtensorMap> halves(3 * 2 * 16);
        for (int b = 0; b < 3; ++b)
            for (int plane = 0; plane < 2; ++plane)
                for (int j = 0; j < 16; ++j)
                    TRY(make_map_bf16(&halves[(b * 2 + plane) * 16 + j], bufs[b] + (size_t)plane * m->max_rows * widths[b],
                                      (uint64_t)m->max_rows, (uint64_t)widths[b], (uint32_t)(16 * (j + 1))));
        ALLOC(m->act_maps_half, CUtensorMap, halves.size());
        CK(cudaMemcpyAsync(m->act_maps_half, halves.data(), halves.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice, m->stream));
        CK(cudaStreamSynchronize(m->stream));
    }
    ALLOC(m->cs, float2, (size_t)m->max_rows * (D / 2));
    ALLOC(m->row_slot, int32_t, m->max_rows);
    ALLOC(m->row_pos, int32_t, m->max_rows);
    ALLOC(m->logits, float, c.vocab);
    {   // split-KV partials: one decode row with up to max_splits splits, or max_rows rows with up to kRowSplits
        size_t n = (size_t)m->max_splits > (size_t)m->max_rows * kRowSplits ? (size_t)m->max_splits : (size_t)m->max_rows * kRowSplits;
        ALLOC(m->part_o, float, (size_t)c.n_q_heads * n * D);
        ALLOC(m->part_ml, float, (size_t)c.n_q_heads * n * 2);
    }
    ALLOC(m->tickets, int32_t, (size_t)m->max_rows * c.n_kv_heads + 1);
    CK(cudaMemsetAsync(m->tickets, 0, ((size_t)m->max_rows * c.n_kv_heads + 1) * sizeof(int32_t), m->stream));
    ALLOC(m->amax_val, float, kArgmaxBlocks > m->sm_count ? kArgmaxBlocks : m->sm_count);
    ALLOC(m->amax_idx, int32_t, kArgmaxBlocks > m->sm_count ? kArgmaxBlocks : m->sm_count);
    ALLOC(m->tokbuf, int32_t, m->max_rows);
    ALLOC(m->desc, StepDesc, 1);
    ALLOC(m->status, int32_t, 1);
    CK(cudaMemsetAsync(m->status, 0, sizeof(int32_t), m->stream));
    // ---- single-kernel decode step ----
    {
        std::vector<MegaLayer> ml(c.n_layers);
        for (int l = 0; l < c.n_layers; ++l) {
            const LayerWeights &w = m->layers[l];
            ml[l] = MegaLayer{w.wqkv, w.wo, w.wgu, w.wd, w.bqkv, w.g1, w.g2,
                              m->kpool + (size_t)l * m->pool_layer_stride, m->vpool + (size_t)l * m->pool_layer_stride};
        }
        ALLOC(m->mega_layers, MegaLayer, c.n_layers);
        CK(cudaMemcpyAsync(m->mega_layers, ml.data(), ml.size() * sizeof(MegaLayer), cudaMemcpyHostToDevice, m->stream));
        CK(cudaStreamSynchronize(m->stream));
        {   // decode-ring TMA descriptors: 256 x 32 boxes without swizzle
            std::vector<CUtensorMap> maps(4 * c.n_layers + 3);
            for (int l = 0; l < c.n_layers; ++l) {
                const LayerWeights &w = m->layers[l];
                TRY(make_map_bf16(&maps[4 * l + 0], w.wqkv, qkvd, h, kMegaTileRows, kMegaBoxK, false));
                TRY(make_map_bf16(&maps[4 * l + 1], w.wo, h, qd, kMegaTileRows, kMegaBoxK, false));
                TRY(make_map_bf16(&maps[4 * l + 2], w.wgu, 2 * f, h, kMegaTileRows, kMegaBoxK, false));
                TRY(make_map_bf16(&maps[4 * l + 3], w.wd, h, f, kMegaTileRows, kMegaBoxK, false));
            }
            TRY(make_map_bf16(&maps[4 * c.n_layers], m->lm_head, c.vocab, h, kMegaTileRows, kMegaBoxK, false));
            // the K and V pools as [layer][page][kv head][slot] rows of D 16-bit values
            const uint64_t kv_rows = (uint64_t)c.n_layers * m->n_pages * c.n_kv_heads * c.page_size;
            if (kv_rows >= (1ull << 31)) return ST_ERR_UNSUPPORTED;   // row coordinates are 32-bit
            TRY(make_map_bf16(&maps[4 * c.n_layers + 1], m->kpool, kv_rows, D, kMegaKvBoxRows, 64, true));
            TRY(make_map_bf16(&maps[4 * c.n_layers + 2], m->vpool, kv_rows, D, kMegaKvBoxRows, 64, true));
            ALLOC(m->mega_maps, CUtensorMap, maps.size());
            CK(cudaMemcpyAsync(m->mega_maps, maps.data(), maps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice, m->stream));
            CK(cudaStreamSynchronize(m->stream));
        }
        ALLOC(m->X0, float, h);
        ALLOC(m->X1, float, h);
        ALLOC(m->D1, float, h);
        ALLOC(m->D2, float, h);
        ALLOC(m->mega_sync, unsigned, kMegaSyncWords);
        ALLOC(m->mega_tickets, int32_t, c.n_kv_heads);
        CK(cudaMemsetAsync(m->mega_sync, 0, kMegaSyncWords * sizeof(unsigned), m->stream));
        CK(cudaMemsetAsync(m->mega_tickets, 0, c.n_kv_heads * sizeof(int32_t), m->stream));
        // Activation area: the input vectors of the QKV / gate-up (h floats) and O (Hq*D floats) projections, the
        // attention scratch, the O projection's merge buffers, and behind the QKV phase's input vector the K/V
        // staging of the attention unit (D 16-bit values per key and pool).  Few KV heads mean many key splits and
        // short units: 64 keys of staging are enough; otherwise 128, and more from whatever shared memory no ring
        // stage can use.
        const int widest = h > qd ? h : qd;
        size_t xarea = (size_t)widest * 4;
        const size_t scratch = mega_scratch_bytes(D, c.n_q_heads / c.n_kv_heads);
        if (scratch > xarea) xarea = scratch;
        const size_t att_area = ((size_t)qd + 256) * 4 + ((size_t)(kMegaSeg / D) * kMaxAttnSplits + 8) * 4 + 2048;
        if (att_area > xarea) xarea = att_area;
        const size_t kv_row = (size_t)D * 2;
        const size_t kv_off = ((size_t)h * 4 + 1023) / 1024 * 1024;
        const size_t kv_min = (size_t)(c.n_kv_heads <= 2 ? 64 : 128) * 2 * kv_row;
        if (kv_off + kv_min > xarea) xarea = kv_off + kv_min;
        // The down projection keeps its whole input vector (ffn floats) when that fits into the area as it is;
        // otherwise it walks K in slabs of 8 segments and keeps one slab at a time.
        m->mega_down_slab = ((size_t)f + kMegaSeg) * 4 <= xarea ? 0 : kMegaDownSlab;
        if (const char *es = getenv("ST_DOWN_SLAB")) m->mega_down_slab = atoi(es) < 0 ? 0 : atoi(es);   // tuning aid
        const size_t down_x = m->mega_down_slab > 0 ? (size_t)m->mega_down_slab * kMegaSeg * 4 : ((size_t)f + kMegaSeg) * 4;
        if (down_x > xarea) xarea = down_x;
        xarea = (xarea + 1023) / 1024 * 1024;
        const long long budget = 226 * 1024 - 1024;
        int stages = (int)((budget - (long long)xarea) / kMegaTileBytes);
        if (stages < 2) return ST_ERR_UNSUPPORTED;
        m->mega_stages = stages > kMegaMaxStages ? kMegaMaxStages : stages;
        // One or two KV heads mean many key splits per head, and merging the splits (every CTA of the O projection
        // reads all partial results of its heads) then costs more than a ring stage buys: give one stage to the K/V
        // staging so that a unit holds 128 keys (measured on the 1.5B shape: -4 % at 3000 cached tokens, -7 % at 6000).
        const bool few_kv_heads = c.n_kv_heads <= 2;
        if (few_kv_heads && m->mega_stages >= 5) m->mega_stages -= 1;
        if (const char *es = getenv("ST_MEGA_STAGES")) {   // tuning aid: fewer ring stages, more K/V staging
            const int want = atoi(es);
            if (want >= 2 && want < m->mega_stages) m->mega_stages = want;
        }
        // shared memory that no ring stage can use enlarges the staging area
        xarea += (size_t)((budget - (long long)xarea - (long long)m->mega_stages * kMegaTileBytes) / 1024 * 1024);
        int cap = (int)((xarea - kv_off) / (2 * kv_row)) & ~15;
        if (cap > 1024) cap = 1024;
        if (const char *ec = getenv("ST_MEGA_KV_CAP")) {   // test aid: a small staging area makes short contexts stream in chunks
            const int want = atoi(ec) & ~15;
            if (want >= 32 && want < cap) cap = want;
        }
        m->mega_kv_off = (int)kv_off;
        m->mega_kv_cap = cap;
        m->mega_xarea = (int)xarea;
        m->mega_smem = 1024 + xarea + (size_t)m->mega_stages * kMegaTileBytes;
        m->mega_splits = m->sm_count / c.n_kv_heads > 0 ? m->sm_count / c.n_kv_heads : 1;
        if (m->mega_splits > kMaxAttnSplits) m->mega_splits = kMaxAttnSplits;
        if (few_kv_heads) {   // as many keys per unit as one staging chunk holds (a unit's first key may sit 15 rows into its first box)
            m->mega_unit_keys = (cap - 16) & ~15;
            if (m->mega_unit_keys > 128) m->mega_unit_keys = 128;
            if (m->mega_unit_keys < 64) m->mega_unit_keys = 64;
        }
        if (const char *eu = getenv("ST_MEGA_UNIT_KEYS")) {   // tuning aid: keys per attention unit while CTAs are to spare
            const int want = atoi(eu) & ~15;
            if (want >= 16 && want + 16 <= cap) m->mega_unit_keys = want;
        }
        const char *e = getenv("ST_MULTI_KERNEL");
        m->multi_kernel_decode = e && e[0] == '1';
    }
#undef ALLOC
    CK(cudaStreamSynchronize(m->stream));
    return ST_OK;
}

// ------------------------------------------------------------------------------------------------
// paged KV bookkeeping (host)
// ------------------------------------------------------------------------------------------------

static int seq_reserve(st_model *m, int slot, int n_tokens)
{
    if (slot < 0 || slot >= m->cfg.max_seqs || !m->seq_used[slot] || n_tokens < 0) return ST_ERR_ARG;
    const int need = (n_tokens + m->cfg.page_size - 1) / m->cfg.page_size;
    if (need > m->pages_per_seq) return ST_ERR_KV_FULL;
    std::vector<int32_t> &pg = m->seq_pages[slot];
    const int have = (int)pg.size();
    if (need <= have) return ST_OK;
    if ((int)m->free_pages.size() < need - have) return ST_ERR_KV_FULL;
    for (int i = have; i < need; ++i) {
        pg.push_back(m->free_pages.back());
        m->free_pages.pop_back();
    }
    CK(cudaMemcpyAsync(m->block_tab + (size_t)slot * m->pages_per_seq + have, pg.data() + have,
                       (size_t)(need - have) * sizeof(int32_t), cudaMemcpyHostToDevice, m->stream));
    return ST_OK;
}

// ------------------------------------------------------------------------------------------------
// one pass of one model
// ------------------------------------------------------------------------------------------------

struct SampleCtx {          // what follows the LM head of an emitting pass
    float *logits_out;      // where the logits go (model scratch when null)
    int32_t *argmax_out;    // plain decode
    int32_t vlimit;         // 0 = whole vocabulary
    GenState *gen;          // generation state (device) or null
    GenBuffers buf;
    StepDesc *desc_small, *desc_large;
    bool want_argmax;
};

static KvView kv_view(st_model *m, int layer, int slot)
{
    KvView kv;
    kv.k = m->kpool + (size_t)layer * m->pool_layer_stride;
    kv.v = m->vpool + (size_t)layer * m->pool_layer_stride;
    kv.block_tab = m->block_tab + (size_t)slot * m->pages_per_seq;
    kv.page_size = m->cfg.page_size;
    kv.page_shift = m->page_shift;
    kv.n_pages = m->n_pages;
    kv.n_kv_heads = m->cfg.n_kv_heads;
    return kv;
}

static int sample_tail(st_model *m, const StepDesc *desc, const SampleCtx &sc)
{
    const st_config &c = m->cfg;
    GemvParams g{};
    g.W = m->lm_head; g.x = m->X; g.gain = m->gf; g.bias = nullptr;
    g.y = sc.logits_out ? sc.logits_out : m->logits;
    g.desc = desc; g.N = c.vocab; g.K = c.hidden; g.x_row = -1; g.eps = c.rms_eps;
    CK((launch_gemv<PRO_NORM, EPI_STORE>(g, m->stream, m->sm_count)));
    if (sc.want_argmax) {
        ArgmaxParams a{};
        a.logits = g.y;
        a.limit = sc.vlimit > 0 ? sc.vlimit : c.vocab;
        a.part_val = m->amax_val; a.part_idx = m->amax_idx;
        a.ticket = m->tickets + (size_t)m->max_rows * c.n_kv_heads;
        a.argmax_out = sc.argmax_out;
        a.gen = sc.gen; a.buf = sc.buf; a.desc_small = sc.desc_small; a.desc_large = sc.desc_large;
        a.status = m->status;
        if (sc.gen) {   // top-p sampling: the nucleus' threshold first (the kernel returns at once when it is off)
            nucleus_kernel<<<1, 256, 0, m->stream>>>(a.logits, a.limit, sc.gen);
            ++g_launches;
            CK(cudaGetLastError());
        }
        argmax_router_kernel<<<kArgmaxBlocks, 256, 0, m->stream>>>(a);
        ++g_launches;
        CK(cudaGetLastError());
    }
    return ST_OK;
}

template <int D, int G>
static cudaError_t mega_launch_dg(const MegaParams &p, int grid, size_t smem, cudaStream_t s, bool attr_only)
{
    auto kern = decode_mega_kernel<D, G>;
    if (attr_only) return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024);
    kern<<<grid, kMegaThreads, smem, s>>>(p);
    return cudaGetLastError();
}

template <int D>
static cudaError_t mega_launch_d(const MegaParams &p, int G, int grid, size_t smem, cudaStream_t s, bool attr_only)
{
    switch (G) {
    case 1: return mega_launch_dg<D, 1>(p, grid, smem, s, attr_only);
    case 2: return mega_launch_dg<D, 2>(p, grid, smem, s, attr_only);
    case 3: return mega_launch_dg<D, 3>(p, grid, smem, s, attr_only);
    case 4: return mega_launch_dg<D, 4>(p, grid, smem, s, attr_only);
    case 5: return mega_launch_dg<D, 5>(p, grid, smem, s, attr_only);
    case 6: return mega_launch_dg<D, 6>(p, grid, smem, s, attr_only);
    case 7: return mega_launch_dg<D, 7>(p, grid, smem, s, attr_only);
    case 8: return mega_launch_dg<D, 8>(p, grid, smem, s, attr_only);
    }
    return cudaErrorInvalidValue;
}

static cudaError_t mega_launch(const MegaParams &p, int D, int G, int grid, size_t smem, cudaStream_t s, bool attr_only)
{
    if (D == 64) return mega_launch_d<64>(p, G, grid, smem, s, attr_only);
    if (D == 128) return mega_launch_d<128>(p, G, grid, smem, s, attr_only);
    return cudaErrorInvalidValue;
}

static int mega_attr_all()
{
    for (int D = 64; D <= 128; D += 64)
        for (int G = 1; G <= 8; ++G) {
            CK(mega_launch(MegaParams{}, D, G, 0, 0, nullptr, true));
            CK(launch_attn_rows_mma(AttnRowsMmaParams{}, D, G, dim3(1, 1, 1), nullptr, true));
            CK(launch_attn_batch(AttnBatchParams{}, D, G, dim3(1, 1, 1), nullptr, 128, true));
        }
    return ST_OK;
}

static int pass_decode_multi(st_model *m, const StepDesc *desc, const int32_t *tok, int slot, int ctx_upper, const SampleCtx &sc);

// Decode pass as one persistent kernel.
static int pass_decode(st_model *m, const StepDesc *desc, const int32_t *tok, int slot, int ctx_upper, const SampleCtx &sc)
{
    if (m->multi_kernel_decode) return pass_decode_multi(m, desc, tok, slot, ctx_upper, sc);
    const st_config &c = m->cfg;
    MegaParams p{};
    p.layers = m->mega_layers;
    p.maps = m->mega_maps;
    p.embed = m->embed; p.lm_head = m->lm_head; p.gf = m->gf; p.inv_freq = m->inv_freq;
    p.desc = desc; p.tok = tok;
    p.kv = kv_view(m, 0, slot);
    p.X0 = m->X0; p.X1 = m->X1; p.QKV = m->QKV; p.ATT = m->ATT; p.D1 = m->D1; p.D2 = m->D2; p.ACT = m->ACT;
    p.logits = sc.logits_out ? sc.logits_out : m->logits;
    p.part_o = m->part_o; p.part_ml = m->part_ml; p.tickets = m->mega_tickets; p.sync = m->mega_sync; p.status = m->status;
    p.n_layers = c.n_layers; p.h = c.hidden; p.Hq = c.n_q_heads; p.Hkv = c.n_kv_heads; p.f = c.ffn; p.vocab = c.vocab;
    p.n_splits = m->mega_splits; p.unit_keys = m->mega_unit_keys; p.stages = m->mega_stages; p.xarea_bytes = m->mega_xarea;
    p.kv_off = m->mega_kv_off; p.kv_cap = m->mega_kv_cap; p.down_slab = m->mega_down_slab;
    p.spin_limit = kMegaSpinLimit;
    p.eps = c.rms_eps; p.scale = 1.f / sqrtf((float)c.head_dim);
    p.want_argmax = sc.want_argmax ? 1 : 0;
    p.limit = sc.vlimit > 0 ? sc.vlimit : c.vocab;
    p.part_val = m->amax_val; p.part_idx = m->amax_idx; p.argmax_out = sc.argmax_out;
    p.gen = sc.gen; p.buf = sc.buf; p.desc_small = sc.desc_small; p.desc_large = sc.desc_large;
    (void)ctx_upper;
    CK(mega_launch(p, c.head_dim, c.n_q_heads / c.n_kv_heads, m->sm_count, m->mega_smem, m->stream, false));
    ++g_launches;
    return ST_OK;
}

// Decode pass, one kernel per phase (debugging aid).  ctx_upper bounds the number of keys (chooses the key split).
static int pass_decode_multi(st_model *m, const StepDesc *desc, const int32_t *tok, int slot, int ctx_upper, const SampleCtx &sc)
{
    const st_config &c = m->cfg;
    const int h = c.hidden, D = c.head_dim, qd = c.n_q_heads * D, kd = c.n_kv_heads * D, f = c.ffn;
    const int G = c.n_q_heads / c.n_kv_heads;
    cudaStream_t s = m->stream;
    embed_rope_kernel<<<1, 256, 0, s>>>(desc, tok, m->embed, h, c.vocab, m->X, m->inv_freq, D / 2, m->cs, m->status);
    ++g_launches;
    CK(cudaGetLastError());
    int n_splits = ctx_upper / 128;
    n_splits = n_splits < 1 ? 1 : n_splits > m->max_splits ? m->max_splits : n_splits;
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerWeights &w = m->layers[l];
        GemvParams g{};
        g.W = w.wqkv; g.x = m->X; g.gain = w.g1; g.bias = w.bqkv; g.y = m->QKV; g.desc = nullptr;
        g.N = qd + 2 * kd; g.K = h; g.x_row = 0; g.eps = c.rms_eps;
        CK((launch_gemv<PRO_NORM, EPI_STORE>(g, s, m->sm_count)));
        const KvView kv = kv_view(m, l, slot);
        rope_append_kernel<<<1, 256, 0, s>>>(desc, m->QKV, nullptr, 0, 0, nullptr, m->cs, c.n_q_heads, c.n_kv_heads, D, kv, m->status);
        ++g_launches;
        CK(cudaGetLastError());
        AttnParams a{};
        a.desc = desc; a.qkv = m->QKV; a.kv = kv; a.out_f32 = m->ATT; a.out_hi = a.out_lo = nullptr;
        a.part_o = m->part_o; a.part_ml = m->part_ml; a.tickets = m->tickets; a.status = m->status;
        a.Hq = c.n_q_heads; a.n_splits = n_splits; a.scale = 1.f / sqrtf((float)D);
        CK(launch_attn(a, D, G, dim3(n_splits, c.n_kv_heads, 1), s));
        g = GemvParams{};
        g.W = w.wo; g.x = m->ATT; g.y = m->X; g.N = h; g.K = qd; g.x_row = 0;
        CK((launch_gemv<PRO_PLAIN, EPI_RESADD>(g, s, m->sm_count)));
        g = GemvParams{};
        g.W = w.wgu; g.x = m->X; g.gain = w.g2; g.y = m->ACT; g.N = 2 * f; g.K = h; g.x_row = 0; g.eps = c.rms_eps;
        CK((launch_gemv<PRO_NORM, EPI_SILU>(g, s, m->sm_count)));
        g = GemvParams{};
        g.W = w.wd; g.x = m->ACT; g.y = m->X; g.N = h; g.K = f; g.x_row = 0;
        CK((launch_gemv<PRO_PLAIN, EPI_RESADD>(g, s, m->sm_count)));
    }
    return sample_tail(m, desc, sc);
}

// One multi-row projection: tensor cores (default) or the CUDA-core tiled GEMM (debugging aid).
template <int EPI>
static int rows_gemm(st_model *m, const StepDesc *desc, int m_upper, int buffer, const uint16_t *A_hi, const uint16_t *A_lo,
                     const CUtensorMap &tw, const uint16_t *W, const float *bias, float *Yf, uint16_t *Yb_hi, uint16_t *Yb_lo,
                     int N, int K, int *pending_splits = nullptr)
{
    if (pending_splits) *pending_splits = 0;
    if (m->simt_gemm) {
        GemmParams g{};
        g.desc = desc; g.A_hi = A_hi; g.A_lo = A_lo; g.W = W; g.bias = bias; g.Yf = Yf; g.Yb_hi = Yb_hi; g.Yb_lo = Yb_lo;
        g.N = N; g.K = K;
        CK(launch_gemm<EPI>(g, m_upper, m->stream));
        return ST_OK;
    }
    (void)A_hi;
    (void)A_lo;
    TcGemmParams p{};
    p.act_hi = m->act_maps + (buffer * 2 + 0) * 8;
    p.act_lo = m->act_maps + (buffer * 2 + 1) * 8;
    p.act_hi_half = m->act_maps_half + (buffer * 2 + 0) * 16;
    p.act_lo_half = m->act_maps_half + (buffer * 2 + 1) * 16;
    p.desc = desc; p.bias = bias; p.Yf = Yf; p.Yb_hi = Yb_hi; p.Yb_lo = Yb_lo; p.status = m->status; p.N = N; p.K = K;
    p.Ws = m->splitk_ws; p.ws_rows = m->max_rows;
    return launch_tc_gemm<EPI>(tw, p, m_upper, m->sm_count, m->stream, pending_splits);
}

// Multi-row pass: up to m_upper rows (the exact count is desc->m on the device).
// batch: the rows are the newest tokens of different sequences (m->row_slot / m->row_pos, `slot` unused); the pass
// then ends with the LM head over all rows (logits [rows][vocab] to sc.logits_out) and one argmax per row.
static int pass_rows(st_model *m, const StepDesc *desc, const int32_t *tok, int slot, int m_upper, int ctx_upper, bool emit, const SampleCtx &sc,
                     bool batch = false)
{
    const st_config &c = m->cfg;
    const int h = c.hidden, D = c.head_dim, qd = c.n_q_heads * D, kd = c.n_kv_heads * D, f = c.ffn;
    const int G = c.n_q_heads / c.n_kv_heads;
    cudaStream_t s = m->stream;
    if (m_upper > m->max_rows) return ST_ERR_INTERNAL;
    uint16_t *XN_lo = m->XN + (size_t)m->max_rows * h, *ATT_lo = m->ATTb + (size_t)m->max_rows * qd,
             *ACT_lo = m->ACTb + (size_t)m->max_rows * f;
    // few rows over a long context: split the keys so that the pass still fills the GPU
    const int rq = m->simt_attn ? 8 : 64 / G;                    // query rows per CTA
    const int row_tiles = (m_upper + rq - 1) / rq;
    const int row_ctas = c.n_kv_heads * row_tiles;
    int row_splits = ((m->simt_attn ? 2 : 1) * m->sm_count + row_ctas - 1) / row_ctas;
    if (row_splits > ctx_upper / 256) row_splits = ctx_upper / 256;
    row_splits = row_splits < 1 ? 1 : row_splits > kRowSplits ? kRowSplits : row_splits;
    static_assert((int)GEPI_STORE == (int)TEPI_STORE && (int)GEPI_RESADD == (int)TEPI_RESADD && (int)GEPI_SILU == (int)TEPI_SILU, "epilogue ids");
    embed_rope_kernel<<<m_upper, 256, 0, s>>>(desc, tok, m->embed, h, c.vocab, m->X, m->inv_freq, D / 2, m->cs, m->status,
                                              batch ? m->row_pos : nullptr);
    ++g_launches;
    CK(cudaGetLastError());
    int pend_down = 0;   // K splits of the previous layer's down projection still to be added to X
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerWeights &w = m->layers[l];
        const LayerMaps &tm = m->maps[l];
        // the previous layer's down projection may have left its K-split partial sums for this kernel to add
        CK(launch_dependent(rmsnorm_rows_kernel, dim3(m_upper), dim3(row_threads(h / 4, 1024)), s, desc, m->X, m->splitk_ws, pend_down, m->max_rows,
                            w.g1, c.rms_eps, h, m->XN, XN_lo));
        int pend = 0;
        TRY((rows_gemm<TEPI_STORE>(m, desc, m_upper, 0, m->XN, XN_lo, tm.wqkv, w.wqkv, w.bqkv, m->QKV, nullptr, nullptr, qd + 2 * kd, h, &pend)));
        const KvView kv = kv_view(m, l, batch ? 0 : slot);
        CK(launch_dependent(rope_append_kernel, dim3(m_upper), dim3(row_threads((c.n_q_heads + c.n_kv_heads) * D / 8, 512)), s, desc, m->QKV,
                            m->splitk_ws, pend, m->max_rows, w.bqkv, m->cs, c.n_q_heads, c.n_kv_heads, D, kv, m->status,
                            batch ? m->row_slot : nullptr, batch ? m->row_pos : nullptr, m->pages_per_seq));
        AttnParams a{};
        a.desc = desc; a.qkv = m->QKV; a.kv = kv; a.out_f32 = nullptr; a.out_hi = m->ATTb; a.out_lo = ATT_lo;
        a.part_o = m->part_o; a.part_ml = m->part_ml; a.tickets = m->tickets; a.status = m->status;
        a.Hq = c.n_q_heads; a.n_splits = row_splits; a.scale = 1.f / sqrtf((float)D);
        if (batch) {
            AttnBatchParams ab{};
            ab.a = a;
            ab.kmap = m->mega_maps + 4 * c.n_layers + 1;
            ab.vmap = m->mega_maps + 4 * c.n_layers + 2;
            ab.row_base = (int32_t)((size_t)l * m->n_pages * c.n_kv_heads * c.page_size);
            ab.row_slot = m->row_slot;
            ab.row_pos = m->row_pos;
            ab.pages_per_seq = m->pages_per_seq;
            CK(launch_attn_batch(ab, D, G, dim3(c.n_kv_heads, m_upper), s, attn_batch_tile(ctx_upper)));
        } else if (m->simt_attn) {
            CK(launch_attn_rows(a, D, G, dim3(row_splits, c.n_kv_heads, row_tiles), s));
        } else {
            AttnRowsMmaParams am{};
            am.a = a;
            am.kmap = m->mega_maps + 4 * c.n_layers + 1;
            am.vmap = m->mega_maps + 4 * c.n_layers + 2;
            am.row_base = (int32_t)((size_t)l * m->n_pages * c.n_kv_heads * c.page_size);
            CK(launch_attn_rows_mma(am, D, G, dim3(row_splits, c.n_kv_heads, row_tiles), s));
        }
        TRY((rows_gemm<TEPI_RESADD>(m, desc, m_upper, 1, m->ATTb, ATT_lo, tm.wo, w.wo, nullptr, m->X, nullptr, nullptr, h, qd, &pend)));
        CK(launch_dependent(rmsnorm_rows_kernel, dim3(m_upper), dim3(row_threads(h / 4, 1024)), s, desc, m->X, m->splitk_ws, pend, m->max_rows,
                            w.g2, c.rms_eps, h, m->XN, XN_lo));
        TRY((rows_gemm<TEPI_SILU>(m, desc, m_upper, 0, m->XN, XN_lo, tm.wgu, w.wgu, nullptr, nullptr, m->ACTb, ACT_lo, 2 * f, h)));
        // the last layer's down projection reduces its own splits: the final norm belongs to the LM head
        TRY((rows_gemm<TEPI_RESADD>(m, desc, m_upper, 2, m->ACTb, ACT_lo, tm.wd, w.wd, nullptr, m->X, nullptr, nullptr, h, f,
                                    l + 1 < c.n_layers ? &pend_down : nullptr)));
    }
    if (batch) {
        // final norm of every row, LM head on the tensor cores, one lowest-id argmax per row
        rmsnorm_rows_kernel<<<m_upper, row_threads(h / 4, 1024), 0, s>>>(desc, m->X, m->splitk_ws, 0, m->max_rows, m->gf, c.rms_eps, h, m->XN, XN_lo);
        ++g_launches;
        CK(cudaGetLastError());
        TRY((rows_gemm<TEPI_STORE>(m, desc, m_upper, 0, m->XN, XN_lo, m->map_lm, m->lm_head, nullptr, sc.logits_out, nullptr, nullptr, c.vocab, h)));
        if (sc.want_argmax) {
            argmax_rows_kernel<<<m_upper, 1024, 0, s>>>(desc, sc.logits_out, c.vocab, sc.vlimit > 0 ? sc.vlimit : c.vocab, sc.argmax_out);
            ++g_launches;
            CK(cudaGetLastError());
        }
        return ST_OK;
    }
    if (emit) return sample_tail(m, desc, sc);
    return ST_OK;
}

// A batched decode pass through a CUDA graph: the pass is ~13 kernels per layer whose arguments depend only on
// device arrays (row tables, descriptor) and on the pointers in the key, so it is captured once per key and
// replayed; the launch gaps between its short kernels go away.
static int pass_rows_batch_graphed(st_model *m, const StepDesc *desc, const int32_t *tok, int m_upper, int ctx_upper, const SampleCtx &sc)
{
    static const bool off = [] { const char *e = getenv("ST_BATCH_GRAPH"); return e && e[0] == '0'; }();
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (off || cudaStreamIsCapturing(m->stream, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone)
        return pass_rows(m, desc, tok, -1, m_upper, ctx_upper, true, sc, true);
    for (auto &g : m->batch_graphs)
        if (g.m_upper == m_upper && g.vlimit == sc.vlimit && g.tile == attn_batch_tile(ctx_upper) && g.tok == tok && g.desc == desc && g.logits == sc.logits_out &&
            g.argmax == (sc.want_argmax ? sc.argmax_out : nullptr)) {
            CK(cudaGraphLaunch(g.exec, m->stream));
            g_launches += g.launches;
            return ST_OK;
        }
    if (m->batch_graphs.size() >= 16) {
        CK(cudaStreamSynchronize(m->stream));
        for (auto &g : m->batch_graphs) cudaGraphExecDestroy(g.exec);
        m->batch_graphs.clear();
    }
    const int64_t before = g_launches;
    // captured on a side stream: the model's own stream may be the legacy default stream, which cannot be captured
    if (!m->cap_stream) CK(cudaStreamCreateWithFlags(&m->cap_stream, cudaStreamNonBlocking));
    if (cudaStreamBeginCapture(m->cap_stream, cudaStreamCaptureModeRelaxed) != cudaSuccess) {
        cudaGetLastError();
        return pass_rows(m, desc, tok, -1, m_upper, ctx_upper, true, sc, true);
    }
    cudaStream_t own = m->stream;
    m->stream = m->cap_stream;
    const int rc = pass_rows(m, desc, tok, -1, m_upper, ctx_upper, true, sc, true);
    m->stream = own;
    cudaGraph_t graph = nullptr;
    const cudaError_t e = cudaStreamEndCapture(m->cap_stream, &graph);
    if (rc != ST_OK) {
        if (graph) cudaGraphDestroy(graph);
        return rc;
    }
    CK(e);
    st_model::BatchGraph g{m_upper, sc.vlimit, attn_batch_tile(ctx_upper), tok, desc, sc.logits_out, sc.want_argmax ? sc.argmax_out : nullptr, nullptr, g_launches - before};
    const cudaError_t ei = cudaGraphInstantiate(&g.exec, graph, 0);
    cudaGraphDestroy(graph);
    CK(ei);
    m->batch_graphs.push_back(g);
    CK(cudaGraphLaunch(g.exec, m->stream));
    return ST_OK;
}

// ------------------------------------------------------------------------------------------------
// C ABI
// ------------------------------------------------------------------------------------------------

static void destroy_gen_context(st_model *m);

extern "C" {

const char *st_strerror(int status)
{
    switch (status) {
    case ST_OK: return "ok";
    case ST_ERR_ARG: return "invalid argument";
    case ST_ERR_OOM: return "out of memory";
    case ST_ERR_KV_FULL: return "KV cache full";
    case ST_ERR_VOCAB: return "vocabulary mismatch or token id out of range";
    case ST_ERR_TIMEOUT: return "device-side wait expired";
    case ST_ERR_UNSUPPORTED: return "unsupported shape or option";
    case ST_ERR_INTERNAL: return g_err_text[0] ? g_err_text : "internal error";
    case ST_ERR_CAPACITY: return "output buffer too small";
    }
    return "unknown status";
}

int st_model_create(const st_config *cfg, uint64_t seed, uint32_t model_tag, void *cuda_stream, st_model **out)
{
    if (!out) return ST_ERR_ARG;
    *out = nullptr;
    TRY(check_config(cfg));
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev < 1) {
        cudaGetLastError();
        snprintf(g_err_text, sizeof g_err_text, "no CUDA device: this library has no CPU path");
        return ST_ERR_INTERNAL;
    }
    st_model *m = new (std::nothrow) st_model();
    if (!m) return ST_ERR_OOM;
    static uint64_t next_id = 0;
    m->id = ++next_id;
    m->cfg = *cfg;
    m->seed = seed;
    m->tag = model_tag;
    m->stream = (cudaStream_t)cuda_stream;
    const int rc = model_build(m);
    if (rc != ST_OK) {
        st_model_destroy(m);
        return rc;
    }
    *out = m;
    return ST_OK;
}

void st_model_destroy(st_model *m)
{
    if (!m) return;
    cudaStreamSynchronize(m->stream);
    destroy_gen_context(m);
    for (auto &g : m->batch_graphs) cudaGraphExecDestroy(g.exec);
    if (m->cap_stream) cudaStreamDestroy(m->cap_stream);
    for (void *p : m->allocations) {
        if (m->cfg.free) m->cfg.free(p, m->cfg.alloc_user);
        else cudaFree(p);
    }
    delete m;
}

int64_t st_weight_bytes(const st_model *m) { return m ? m->weight_bytes : 0; }

int64_t st_kv_bytes_per_token(const st_model *m)
{
    return m ? 4ll * m->cfg.n_layers * m->cfg.n_kv_heads * m->cfg.head_dim : 0;
}

int64_t st_kernel_launches(void) { return g_launches; }

int st_selftest_bounded_wait(st_model *m, int32_t which)
{
    if (!m || which < 0 || which > 1) return ST_ERR_ARG;
    cudaStream_t s = m->stream;
    int32_t *d_ret = (int32_t *)m->tokbuf;   // a device word nobody uses between calls
    CK(cudaMemsetAsync(m->status, 0, sizeof(int32_t), s));
    CK(cudaMemsetAsync(d_ret, 0, sizeof(int32_t), s));
    CK(cudaMemsetAsync(m->mega_sync, 0, kMegaSyncWords * sizeof(unsigned), s));
    if (which == 0) {
        wait_expiry_selftest_kernel<<<1, 64, 0, s>>>(m->status, 1000u, d_ret);
    } else {
        MegaParams p{};
        p.sync = m->mega_sync;
        p.status = m->status;
        p.spin_limit = 1000u;
        mega_barrier_selftest_kernel<<<1, kMegaThreads, 0, s>>>(p, d_ret);
    }
    ++g_launches;
    CK(cudaGetLastError());
    int32_t ret = 0, status = 0;
    CK(cudaMemcpyAsync(&ret, d_ret, sizeof ret, cudaMemcpyDeviceToHost, s));
    CK(cudaMemcpyAsync(&status, m->status, sizeof status, cudaMemcpyDeviceToHost, s));
    CK(cudaStreamSynchronize(s));
    // leave the model clean for the next ordinary call
    CK(cudaMemsetAsync(m->status, 0, sizeof(int32_t), s));
    CK(cudaMemsetAsync(m->mega_sync, 0, kMegaSyncWords * sizeof(unsigned), s));
    if (ret == 0) return ST_ERR_INTERNAL;                          // the kernel did not reach its end
    if (ret == 2 && (status & DEV_WAIT_EXPIRED)) return ST_ERR_TIMEOUT;   // the wait gave up as it should
    return ST_OK;                                                  // the wait did not expire: the check failed
}

int st_decode_geometry(const st_model *m, int32_t ctx, int32_t *n_splits, int32_t *kv_cap, int32_t *max_chunks, int32_t *own_chunk_empty)
{
    if (!m || ctx < 0) return ST_ERR_ARG;
    const int ns = mega_key_splits(ctx, m->mega_splits, m->sm_count, m->cfg.n_kv_heads, m->mega_unit_keys);
    int most = 0, empty = 0;
    for (int sp = 0; sp < ns; ++sp) {
        const MegaUnitShape u = mega_unit_shape(ctx, ns, sp, m->mega_kv_cap);
        if (u.nch > most) most = u.nch;
        if (u.owner && u.nch > 1 && u.n_cached == (u.nch - 1) * u.CH) empty = 1;
    }
    if (n_splits) *n_splits = ns;
    if (kv_cap) *kv_cap = m->mega_kv_cap;
    if (max_chunks) *max_chunks = most;
    if (own_chunk_empty) *own_chunk_empty = empty;
    return ST_OK;
}

#ifdef ST_MEGA_TRACE
int st_debug_trace(unsigned long long *out, int n) { return (int)cudaMemcpyFromSymbol(out, g_mega_trace, (size_t)n * 8); }
#endif

int st_seq_alloc(st_model *m, int32_t *slot_out)
{
    if (!m || !slot_out) return ST_ERR_ARG;
    for (int i = 0; i < m->cfg.max_seqs; ++i)
        if (!m->seq_used[i]) {
            m->seq_used[i] = 1;
            m->seq_len[i] = 0;
            *slot_out = i;
            return ST_OK;
        }
    return ST_ERR_KV_FULL;
}

int st_seq_free(st_model *m, int32_t slot)
{
    if (!m || slot < 0 || slot >= m->cfg.max_seqs || !m->seq_used[slot]) return ST_ERR_ARG;
    for (int32_t p : m->seq_pages[slot]) m->free_pages.push_back(p);
    m->seq_pages[slot].clear();
    m->seq_used[slot] = 0;
    m->seq_len[slot] = 0;
    return ST_OK;
}

int st_seq_reserve(st_model *m, int32_t slot, int32_t n_tokens)
{
    if (!m) return ST_ERR_ARG;
    return seq_reserve(m, slot, n_tokens);
}

int st_kv_len(st_model *m, int32_t slot, int32_t *len_out)
{
    if (!m || !len_out || slot < 0 || slot >= m->cfg.max_seqs || !m->seq_used[slot]) return ST_ERR_ARG;
    CK(cudaStreamSynchronize(m->stream));
    *len_out = m->seq_len[slot];
    return ST_OK;
}

int st_kv_truncate(st_model *m, int32_t slot, int32_t new_len)
{
    if (!m || slot < 0 || slot >= m->cfg.max_seqs || !m->seq_used[slot] || new_len < 0) return ST_ERR_ARG;
    if (new_len < m->seq_len[slot]) m->seq_len[slot] = new_len;
    return ST_OK;
}

int st_last_device_status(st_model *m)
{
    if (!m) return ST_ERR_ARG;
    int32_t v = 0;
    CK(cudaMemcpyAsync(&v, m->status, sizeof v, cudaMemcpyDeviceToHost, m->stream));
    CK(cudaStreamSynchronize(m->stream));
    return v;
}

int st_fill_tensor_bf16(uint64_t seed, uint32_t model_tag, uint32_t tid, uint64_t idx0, uint64_t n, uint16_t *out_dev, void *cuda_stream)
{
    if (!out_dev) return ST_ERR_ARG;
    if (n == 0) return ST_OK;
    const uint64_t key = tensor_stream_key(seed, model_tag, tid);
    // n "rows" of one column starting at row idx0: element index = idx0 + r
    uint64_t blocks = (n + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    fill_bf16_kernel<<<(int)blocks, 256, 0, (cudaStream_t)cuda_stream>>>(out_dev, key, idx0, n, 1, 1, 0);
    ++g_launches;
    CK(cudaGetLastError());
    return ST_OK;
}

int st_time_gemv(st_model *m, int32_t which, int32_t iters, double *seconds_out)
{
    if (!m || !seconds_out || iters < 1 || which < 0 || which > 4) return ST_ERR_ARG;
    const st_config &c = m->cfg;
    const int h = c.hidden, D = c.head_dim, qd = c.n_q_heads * D, kd = c.n_kv_heads * D, f = c.ffn;
    cudaEvent_t e0, e1;
    CK(cudaEventCreate(&e0));
    CK(cudaEventCreate(&e1));
    CK(cudaMemsetAsync(m->X, 0, (size_t)h * sizeof(float), m->stream));
    CK(cudaMemsetAsync(m->ATT, 0, (size_t)qd * sizeof(float), m->stream));
    CK(cudaMemsetAsync(m->ACT, 0, (size_t)f * sizeof(float), m->stream));
    for (int rep = 0; rep < 2; ++rep) {   // the first round warms up
        if (rep == 1) CK(cudaEventRecord(e0, m->stream));
        for (int i = 0; i < iters; ++i) {
            const LayerWeights &w = m->layers[i % c.n_layers];
            GemvParams g{};
            g.x_row = 0; g.eps = c.rms_eps;
            cudaError_t e = cudaSuccess;
            switch (which) {
            case 0: g.W = w.wqkv; g.x = m->X; g.gain = w.g1; g.bias = w.bqkv; g.y = m->QKV; g.N = qd + 2 * kd; g.K = h;
                    e = launch_gemv<PRO_NORM, EPI_STORE>(g, m->stream, m->sm_count); break;
            case 1: g.W = w.wo; g.x = m->ATT; g.y = m->X; g.N = h; g.K = qd;
                    e = launch_gemv<PRO_PLAIN, EPI_RESADD>(g, m->stream, m->sm_count); break;
            case 2: g.W = w.wgu; g.x = m->X; g.gain = w.g2; g.y = m->ACT; g.N = 2 * f; g.K = h;
                    e = launch_gemv<PRO_NORM, EPI_SILU>(g, m->stream, m->sm_count); break;
            case 3: g.W = w.wd; g.x = m->ACT; g.y = m->X; g.N = h; g.K = f;
                    e = launch_gemv<PRO_PLAIN, EPI_RESADD>(g, m->stream, m->sm_count); break;
            default: g.W = m->lm_head; g.x = m->X; g.gain = m->gf; g.y = m->logits; g.N = c.vocab; g.K = h;
                    e = launch_gemv<PRO_NORM, EPI_STORE>(g, m->stream, m->sm_count); break;
            }
            CK(e);
        }
    }
    CK(cudaEventRecord(e1, m->stream));
    CK(cudaEventSynchronize(e1));
    float ms = 0.f;
    CK(cudaEventElapsedTime(&ms, e0, e1));
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    *seconds_out = (double)ms * 1e-3 / iters;
    return ST_OK;
}

int st_prefill(st_model *m, int32_t slot, const int32_t *tokens_host, int32_t n, float *last_logits_dev)
{
    if (!m || !tokens_host || n < 1 || slot < 0 || slot >= m->cfg.max_seqs || !m->seq_used[slot]) return ST_ERR_ARG;
    for (int i = 0; i < n; ++i)
        if ((unsigned)tokens_host[i] >= (unsigned)m->cfg.vocab) return ST_ERR_VOCAB;
    TRY(seq_reserve(m, slot, m->seq_len[slot] + n));
    CK(cudaMemsetAsync(m->mega_sync, 0, kMegaSyncWords * sizeof(unsigned), m->stream));
    for (int done = 0; done < n;) {
        const int rows = n - done < m->max_rows ? n - done : m->max_rows;
        const bool last = done + rows == n;
        StepDesc d{m->seq_len[slot], rows, 0, last ? 1 : 0};
        CK(cudaMemcpyAsync(m->tokbuf, tokens_host + done, (size_t)rows * sizeof(int32_t), cudaMemcpyHostToDevice, m->stream));
        CK(cudaMemcpyAsync(m->desc, &d, sizeof d, cudaMemcpyHostToDevice, m->stream));
        SampleCtx sc{};
        sc.logits_out = last_logits_dev;
        sc.want_argmax = false;
        const bool emit = last && last_logits_dev != nullptr;
        if (rows == 1 && emit) TRY(pass_decode(m, m->desc, m->tokbuf, slot, d.pos0 + 1, sc));
        else TRY(pass_rows(m, m->desc, m->tokbuf, slot, rows, d.pos0 + rows, emit, sc));
        m->seq_len[slot] += rows;
        done += rows;
        // the staging buffer and descriptor are reused by the next chunk
        if (!last) CK(cudaStreamSynchronize(m->stream));
    }
    return ST_OK;
}

int st_decode_step(st_model *m, const int32_t *slots_host, const int32_t *tokens_dev, int32_t batch, float *logits_dev, int32_t *argmax_dev)
{
    if (!m || !slots_host || !tokens_dev || batch < 1) return ST_ERR_ARG;
    for (int i = 0; i < batch; ++i) {
        const int slot = slots_host[i];
        if (slot < 0 || slot >= m->cfg.max_seqs || !m->seq_used[slot]) return ST_ERR_ARG;
        for (int j = 0; j < i; ++j)
            if (slots_host[j] == slot) return ST_ERR_ARG;
    }
    if (batch >= 2 && !m->multi_kernel_decode) {
        // several sequences: one pass over the weights for all of them, projections on the tensor cores
        float *logits = logits_dev;
        if (!logits) {
            if (!m->batch_logits) {
                m->batch_logits = (float *)m->dalloc((size_t)m->max_rows * m->cfg.vocab * sizeof(float));
                if (!m->batch_logits) return ST_ERR_OOM;
            }
            logits = m->batch_logits;
        }
        for (int i0 = 0; i0 < batch; i0 += m->max_rows) {
            const int n = batch - i0 < m->max_rows ? batch - i0 : m->max_rows;
            std::vector<int32_t> rows(2 * (size_t)n);
            int ctx_upper = 1;
            for (int i = 0; i < n; ++i) {
                const int slot = slots_host[i0 + i];
                TRY(seq_reserve(m, slot, m->seq_len[slot] + 1));
                rows[i] = slot;
                rows[n + i] = m->seq_len[slot];
                if (m->seq_len[slot] + 1 > ctx_upper) ctx_upper = m->seq_len[slot] + 1;
            }
            CK(cudaMemcpyAsync(m->row_slot, rows.data(), (size_t)n * sizeof(int32_t), cudaMemcpyHostToDevice, m->stream));
            CK(cudaMemcpyAsync(m->row_pos, rows.data() + n, (size_t)n * sizeof(int32_t), cudaMemcpyHostToDevice, m->stream));
            StepDesc d{0, n, i0, 1};
            CK(cudaMemcpyAsync(m->desc, &d, sizeof d, cudaMemcpyHostToDevice, m->stream));
            SampleCtx sc{};
            sc.logits_out = logits + (logits_dev ? (size_t)i0 * m->cfg.vocab : 0);
            sc.argmax_out = argmax_dev ? argmax_dev + i0 : nullptr;
            sc.want_argmax = argmax_dev != nullptr;
            TRY(pass_rows_batch_graphed(m, m->desc, tokens_dev, (n + 31) / 32 * 32 > m->max_rows ? m->max_rows : (n + 31) / 32 * 32, ctx_upper, sc));
            for (int i = 0; i < n; ++i) m->seq_len[slots_host[i0 + i]] += 1;
            // the row tables and the descriptor are rewritten for the next chunk
            CK(cudaStreamSynchronize(m->stream));
        }
        return ST_OK;
    }
    CK(cudaMemsetAsync(m->mega_sync, 0, kMegaSyncWords * sizeof(unsigned), m->stream));
    for (int i = 0; i < batch; ++i) {
        const int slot = slots_host[i];
        TRY(seq_reserve(m, slot, m->seq_len[slot] + 1));
        StepDesc d{m->seq_len[slot], 1, i, 1};
        CK(cudaMemcpyAsync(m->desc, &d, sizeof d, cudaMemcpyHostToDevice, m->stream));
        SampleCtx sc{};
        sc.logits_out = logits_dev ? logits_dev + (size_t)i * m->cfg.vocab : nullptr;
        sc.argmax_out = argmax_dev ? argmax_dev + i : nullptr;
        sc.want_argmax = argmax_dev != nullptr;
        TRY(pass_decode(m, m->desc, tokens_dev, slot, d.pos0 + 1, sc));
        m->seq_len[slot] += 1;
        // the descriptor is rewritten for the next sequence
        if (i + 1 < batch) CK(cudaStreamSynchronize(m->stream));
    }
    return ST_OK;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// generation
// ------------------------------------------------------------------------------------------------

// Device buffers of a generation and the CUDA graph that runs it.  The graph is one WHILE node whose
// body is a dispatch kernel followed by a SWITCH node with one body per kind of pass (per model:
// decode, multi-row passes of <= 32/64/128/256 rows, ingest-only).  The router kernel at the end of a
// pass plans the next one on the device, the dispatch kernel selects the body: the host launches the
// graph once and waits.  Kernel arguments are baked into the graph, so the buffers live as long as
// the context and the graph is rebuilt only when a capacity grows or a model/slot changes.
struct GenContext {
    st_model *large = nullptr;
    uint64_t large_id = 0;
    int slot_s = -1, slot_l = -1;
    int cap_total = 0, cap_steps = 0, cap_hand = 0, cap_force = 0, vlimit = 0;
    size_t cap_trace = 0;
    GenState *gen = nullptr;
    StepDesc *desc2 = nullptr;
    GenBuffers b{};
    int32_t *d_force = nullptr;
    int32_t *d_aux = nullptr;
    uint8_t *d_cls = nullptr;
    float *d_trace = nullptr;
    std::vector<void *> ptrs;
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    int64_t body_launches[2 * kBodiesPerModel] = {};   // kernels in each captured body

    template <class T>
    T *get(size_t n)
    {
        void *p = nullptr;
        if (cudaMalloc(&p, (n ? n : 1) * sizeof(T)) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        ptrs.push_back(p);
        return (T *)p;
    }
    void release()
    {
        if (exec) cudaGraphExecDestroy(exec);
        if (graph) cudaGraphDestroy(graph);
        for (void *p : ptrs) cudaFree(p);
        ptrs.clear();
        exec = nullptr;
        graph = nullptr;
    }
};

static void destroy_gen_context(st_model *m)
{
    if (m->gen_ctx) {
        m->gen_ctx->release();
        delete m->gen_ctx;
        m->gen_ctx = nullptr;
    }
}

namespace {

struct SlotGuard {
    st_model *m;
    int slot = -1;
    ~SlotGuard()
    {
        if (m && slot >= 0) st_seq_free(m, slot);
    }
};

struct StreamSwap {   // run the pass functions on the capture stream
    st_model *a, *b;
    cudaStream_t sa, sb;
    StreamSwap(st_model *a_, st_model *b_, cudaStream_t cap) : a(a_), b(b_), sa(a_->stream), sb(b_ ? b_->stream : nullptr)
    {
        a->stream = cap;
        if (b) b->stream = cap;
    }
    ~StreamSwap()
    {
        a->stream = sa;
        if (b) b->stream = sb;
    }
};

}  // namespace

static SampleCtx gen_sample_ctx(const GenContext &c)
{
    SampleCtx sc{};
    sc.vlimit = c.vlimit;
    sc.gen = c.gen;
    sc.buf = c.b;
    sc.desc_small = c.desc2;
    sc.desc_large = c.desc2 + 1;
    sc.want_argmax = true;
    return sc;
}

// Capture one pass body into `body`.
static int capture_body(GenContext &c, st_model *small, cudaStream_t cap, cudaGraph_t body, int model, int kind)
{
    static const int kRowsOf[kBodiesPerModel] = {1, 32, 64, 128, 256, 256};
    st_model *m = model ? c.large : small;
    const int slot = model ? c.slot_l : c.slot_s;
    StepDesc *d = c.desc2 + model;
    const SampleCtx sc = gen_sample_ctx(c);
    CK(cudaStreamBeginCaptureToGraph(cap, body, nullptr, nullptr, 0, cudaStreamCaptureModeRelaxed));
    int rc;
    ++g_pdl_off;
    {
        StreamSwap swap(small, c.large, cap);
        int rows = kRowsOf[kind];
        if (rows > m->max_rows) rows = m->max_rows;
        if (kind == 0) rc = pass_decode(m, d, c.b.tokens, slot, c.cap_total, sc);
        else rc = pass_rows(m, d, c.b.tokens, slot, rows, c.cap_total, kind != 5, sc);
        if (rc == ST_OK && kind == 5) {
            advance_ingest_kernel<<<1, 1, 0, cap>>>(c.gen, c.desc2, c.desc2 + 1);
            ++g_launches;
            if (cudaGetLastError() != cudaSuccess) rc = ST_ERR_INTERNAL;
        }
    }
    --g_pdl_off;
    cudaGraph_t g = nullptr;
    const cudaError_t e = cudaStreamEndCapture(cap, &g);
    if (rc != ST_OK) return rc;
    CK(e);
    return ST_OK;
}

static int build_gen_graph(GenContext &c, st_model *small)
{
    if (c.exec) { cudaGraphExecDestroy(c.exec); c.exec = nullptr; }
    if (c.graph) { cudaGraphDestroy(c.graph); c.graph = nullptr; }
    cudaStream_t cap = nullptr;
    CK(cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking));
    int rc = ST_OK;
    do {
        if (cudaGraphCreate(&c.graph, 0) != cudaSuccess) { rc = ST_ERR_INTERNAL; break; }
        cudaGraphConditionalHandle h_loop, h_body;
        if (cudaGraphConditionalHandleCreate(&h_loop, c.graph, 1, cudaGraphCondAssignDefault) != cudaSuccess) { rc = ST_ERR_INTERNAL; break; }
        cudaGraphNodeParams wp = {cudaGraphNodeTypeConditional};
        wp.type = cudaGraphNodeTypeConditional;
        wp.conditional.handle = h_loop;
        wp.conditional.type = cudaGraphCondTypeWhile;
        wp.conditional.size = 1;
        cudaGraphNode_t wnode;
        if (cudaGraphAddNode(&wnode, c.graph, nullptr, 0, &wp) != cudaSuccess) { rc = ST_ERR_INTERNAL; break; }
        cudaGraph_t loop_body = wp.conditional.phGraph_out[0];
        if (cudaGraphConditionalHandleCreate(&h_body, loop_body, 0, 0) != cudaSuccess) { rc = ST_ERR_INTERNAL; break; }
        // dispatch kernel node
        int32_t *status = small->status;
        void *args[4] = {&c.gen, &h_loop, &h_body, &status};
        cudaKernelNodeParams kp;
        memset(&kp, 0, sizeof kp);
        kp.func = (void *)dispatch_kernel;
        kp.gridDim = dim3(1);
        kp.blockDim = dim3(1);
        kp.kernelParams = args;
        cudaGraphNode_t dnode;
        if (cudaGraphAddKernelNode(&dnode, loop_body, nullptr, 0, &kp) != cudaSuccess) { rc = ST_ERR_INTERNAL; break; }
        // switch node with one body per kind of pass
        const int n_bodies = (c.large ? 2 : 1) * kBodiesPerModel;
        cudaGraphNodeParams sp = {cudaGraphNodeTypeConditional};
        sp.type = cudaGraphNodeTypeConditional;
        sp.conditional.handle = h_body;
        sp.conditional.type = cudaGraphCondTypeSwitch;
        sp.conditional.size = (unsigned)n_bodies;
        cudaGraphNode_t snode;
        if (cudaGraphAddNode(&snode, loop_body, &dnode, 1, &sp) != cudaSuccess) { rc = ST_ERR_INTERNAL; break; }
        for (int i = 0; i < n_bodies && rc == ST_OK; ++i) {
            const int64_t before = g_launches;
            rc = capture_body(c, small, cap, sp.conditional.phGraph_out[i], i / kBodiesPerModel, i % kBodiesPerModel);
            c.body_launches[i] = g_launches - before;   // captured, not run
            g_launches = before;
        }
        if (rc != ST_OK) break;
        if (cudaGraphInstantiate(&c.exec, c.graph, 0) != cudaSuccess) { rc = ST_ERR_INTERNAL; break; }
    } while (0);
    if (rc != ST_OK) {
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess || !g_err_text[0]) set_error_text("building the generation graph", e);
    }
    cudaStreamDestroy(cap);
    return rc;
}

// Make sure the speculative model's context fits this call; (re)allocate and rebuild when it does not.
static int ensure_gen_context(st_model *small, st_model *large, int slot_s, int slot_l, int total, int cap_steps, int cap_hand,
                              int n_force, int vlimit, size_t trace_floats, bool want_graph)
{
    GenContext *c = small->gen_ctx;
    const bool fits = c && c->large == large && c->large_id == (large ? large->id : 0) && c->slot_s == slot_s &&
                      c->slot_l == slot_l && c->cap_total >= total && c->cap_steps >= cap_steps && c->cap_hand >= cap_hand &&
                      c->cap_force >= n_force && c->vlimit == vlimit && c->cap_trace >= trace_floats &&
                      (!want_graph || c->exec);
    if (fits) return ST_OK;
    // growing: never shrink a capacity, so that alternating call sizes settle on one graph
    int g_total = total, g_steps = cap_steps, g_hand = cap_hand, g_force = n_force;
    size_t g_trace = trace_floats;
    if (c && c->large == large && c->large_id == (large ? large->id : 0) && c->vlimit == vlimit) {
        g_total = g_total > c->cap_total ? g_total : c->cap_total;
        g_steps = g_steps > c->cap_steps ? g_steps : c->cap_steps;
        g_hand = g_hand > c->cap_hand ? g_hand : c->cap_hand;
        g_force = g_force > c->cap_force ? g_force : c->cap_force;
        g_trace = g_trace > c->cap_trace ? g_trace : c->cap_trace;
    }
    destroy_gen_context(small);
    c = new (std::nothrow) GenContext();
    if (!c) return ST_ERR_OOM;
    small->gen_ctx = c;
    c->large = large;
    c->large_id = large ? large->id : 0;
    c->slot_s = slot_s;
    c->slot_l = slot_l;
    c->cap_total = g_total;
    c->cap_steps = g_steps;
    c->cap_hand = g_hand;
    c->cap_force = g_force;
    c->vlimit = vlimit;
    c->cap_trace = g_trace;
    c->gen = c->get<GenState>(1);
    c->desc2 = c->get<StepDesc>(2);
    c->b.tokens = c->get<int32_t>(g_total);
    c->b.source = c->get<uint8_t>(g_total);
    c->b.em_tok = c->get<int32_t>(g_steps);
    c->b.em_fed = c->get<int32_t>(g_steps);
    c->b.em_arg = c->get<int32_t>(g_steps);
    c->b.em_src = c->get<uint8_t>(g_steps);
    c->b.handoffs = c->get<int32_t>(3 * (size_t)g_hand);
    c->b.hand_kind = c->get<uint8_t>((size_t)g_hand);
    c->d_aux = c->get<int32_t>(kMaxAuxTokens);
    c->b.aux = c->d_aux;
    c->d_force = c->get<int32_t>(g_force);
    c->d_cls = c->get<uint8_t>(vlimit);
    c->d_trace = g_trace ? c->get<float>(g_trace) : nullptr;
    if (!c->gen || !c->desc2 || !c->b.tokens || !c->b.source || !c->b.em_tok || !c->b.em_fed || !c->b.em_arg || !c->b.em_src ||
        !c->b.handoffs || !c->b.hand_kind || !c->d_aux || !c->d_force || !c->d_cls || (g_trace && !c->d_trace)) {
        destroy_gen_context(small);
        return ST_ERR_OOM;
    }
    c->b.force = c->d_force;
    c->b.cls = c->d_cls;
    c->b.trace = c->d_trace;
    if (want_graph) {
        const int rc = build_gen_graph(*c, small);
        if (rc != ST_OK) {
            destroy_gen_context(small);
            return rc;
        }
    }
    return ST_OK;
}

// Takeover parameters beyond the keyword set: ids inside the shared vocabulary, positive segment lengths where a
// rule is on, an auxiliary sentence that fits the device buffer.
static int check_rule_params(const st_spec_params *P, int vlimit)
{
    if (P->n_affirmation < 0 || P->n_verification < 0 || P->n_aux < 0) return ST_ERR_ARG;
    if ((P->n_affirmation > 0 && !P->affirmation_ids) || (P->n_verification > 0 && !P->verification_ids) || (P->n_aux > 0 && !P->aux_ids))
        return ST_ERR_ARG;
    if ((P->n_verification > 0 && P->n2 < 1) || (P->neg_threshold >= 0 && P->n3 < 1)) return ST_ERR_ARG;
    if (P->n_delimiters < 0 || (P->n_delimiters > 0 && !P->delimiter_ids)) return ST_ERR_ARG;
    if (!(P->temperature >= 0.f) || !(P->top_p >= 0.f)) return ST_ERR_ARG;
    for (int i = 0; i < P->n_delimiters; ++i)
        if ((unsigned)P->delimiter_ids[i] >= (unsigned)vlimit) return ST_ERR_VOCAB;
    if (P->n_delimiters == 0 && (unsigned)P->delimiter_id >= (unsigned)vlimit) return ST_ERR_VOCAB;
    if (P->n_aux > kMaxAuxTokens) return ST_ERR_CAPACITY;
    for (int i = 0; i < P->n_affirmation; ++i)
        if ((unsigned)P->affirmation_ids[i] >= (unsigned)vlimit) return ST_ERR_VOCAB;
    for (int i = 0; i < P->n_verification; ++i)
        if ((unsigned)P->verification_ids[i] >= (unsigned)vlimit) return ST_ERR_VOCAB;
    for (int i = 0; i < P->n_aux; ++i)
        if ((unsigned)P->aux_ids[i] >= (unsigned)vlimit) return ST_ERR_VOCAB;
    return ST_OK;
}

static void fill_class_table(const st_spec_params *P, std::vector<uint8_t> &cls)
{
    if (P->n_delimiters > 0)
        for (int i = 0; i < P->n_delimiters; ++i) cls[P->delimiter_ids[i]] |= kClsDelim;
    else
        cls[P->delimiter_id] |= kClsDelim;
    for (int i = 0; i < P->n_keywords; ++i) cls[P->keyword_ids[i]] |= kClsKeyword;
    for (int i = 0; i < P->n_affirmation; ++i) cls[P->affirmation_ids[i]] |= kClsAffirm;
    for (int i = 0; i < P->n_verification; ++i) cls[P->verification_ids[i]] |= kClsVerify;
}

extern "C" int st_generate_spec(st_model *small, st_model *large, const st_spec_params *P, const int32_t *prompt,
                                int32_t prompt_len, const int32_t *force, int32_t n_force, st_spec_result *out)
{
    if (!small || !P || !prompt || !out || prompt_len < 1 || P->max_new_tokens < 0 || P->n1 < 1 || n_force < 0 || P->target_first_n < 0) return ST_ERR_ARG;
    if (P->n_keywords < 0 || (P->n_keywords > 0 && !P->keyword_ids) || (n_force > 0 && !force)) return ST_ERR_ARG;
    if (large && (large->stream != small->stream || large->device != small->device)) return ST_ERR_ARG;
    int vshared = small->cfg.vocab;
    if (large && large->cfg.vocab < vshared) vshared = large->cfg.vocab;
    const int vlimit = P->vocab_limit > 0 ? P->vocab_limit : vshared;
    if (vlimit > vshared) return ST_ERR_VOCAB;
    for (int i = 0; i < prompt_len; ++i)
        if ((unsigned)prompt[i] >= (unsigned)vlimit) return ST_ERR_VOCAB;
    for (int i = 0; i < n_force; ++i)
        if (force[i] >= vlimit) return ST_ERR_VOCAB;
    for (int i = 0; i < P->n_keywords; ++i)
        if ((unsigned)P->keyword_ids[i] >= (unsigned)vlimit) return ST_ERR_VOCAB;
    TRY(check_rule_params(P, vlimit));
    const int max_new = P->max_new_tokens;
    if (out->cap_tokens < max_new || (max_new > 0 && (!out->tokens || !out->source))) return ST_ERR_CAPACITY;
    const int cap_steps = out->cap_steps, cap_handoffs = out->cap_handoffs;
    if ((cap_steps > 0 && (!out->emission_tokens || !out->emission_source)) || (cap_handoffs > 0 && !out->handoffs)) return ST_ERR_ARG;
    if (out->logits_trace && (out->trace_n_steps < 0 || out->trace_first_step < 0)) return ST_ERR_ARG;
    out->n_tokens = out->n_handoffs = out->n_steps = 0;
    out->kv_len_small = out->kv_len_large = 0;
    out->seconds = 0.0;
    out->bytes_algorithmic = 0;
    out->t_prompt_prefill_s = out->t_catchup_s = out->t_decode_s = 0.0;
    out->n_prompt_prefill = out->n_catchup = out->n_decode = 0;

    cudaStream_t s = small->stream;
    CK(cudaMemsetAsync(small->status, 0, sizeof(int32_t), s));
    CK(cudaMemsetAsync(small->mega_sync, 0, kMegaSyncWords * sizeof(unsigned), s));
    CK(cudaMemsetAsync(small->mega_tickets, 0, small->cfg.n_kv_heads * sizeof(int32_t), s));
    if (large) {
        CK(cudaMemsetAsync(large->status, 0, sizeof(int32_t), s));
        CK(cudaMemsetAsync(large->mega_sync, 0, kMegaSyncWords * sizeof(unsigned), s));
        CK(cudaMemsetAsync(large->mega_tickets, 0, large->cfg.n_kv_heads * sizeof(int32_t), s));
    }
    const int total = prompt_len + max_new + 1;
    SlotGuard gs{small}, gl{large};
    TRY(st_seq_alloc(small, &gs.slot));
    TRY(seq_reserve(small, gs.slot, total));
    if (large) {
        TRY(st_seq_alloc(large, &gl.slot));
        TRY(seq_reserve(large, gl.slot, total));
    }
    const int trace_n = out->logits_trace ? out->trace_n_steps : 0;
    static const bool host_loop = [] { const char *e = getenv("ST_HOST_LOOP"); return e && e[0] == '1'; }();
    TRY(ensure_gen_context(small, large, gs.slot, gl.slot, total, cap_steps > 0 ? cap_steps : 1, cap_handoffs > 0 ? cap_handoffs : 1,
                           n_force, vlimit, (size_t)trace_n * vlimit, !host_loop));
    GenContext &C = *small->gen_ctx;
    const GenBuffers &b = C.b;
    GenState *gen = C.gen;
    StepDesc *desc_small = C.desc2, *desc_large = C.desc2 + 1;

    std::vector<uint8_t> cls(vlimit, 0);
    fill_class_table(P, cls);
    GenState g0{};
    g0.wbytes[0] = small->weight_bytes;
    g0.kvb[0] = st_kv_bytes_per_token(small);
    if (large) {
        g0.wbytes[1] = large->weight_bytes;
        g0.kvb[1] = st_kv_bytes_per_token(large);
    }
    g0.has_large = large ? 1 : 0;
    g0.pos = prompt_len;
    g0.delimiter = P->delimiter_id;
    g0.n1 = P->n1;
    g0.keep_probe = P->keep_probe;
    g0.every_delim = P->takeover_every_delimiter ? 1 : 0;
    g0.n2 = P->n2;
    g0.n3 = P->n3;
    g0.neg_threshold = P->neg_threshold;
    g0.n_aux = P->n_aux;
    g0.probe_len = P->probe_len > 1 ? P->probe_len : 1;
    if (P->temperature > 0.f) {
        g0.inv_temp = 1.f / P->temperature;
        g0.sample_seed = P->sample_seed;
        g0.top_p = P->top_p;
    }
    if (large && P->target_first_n > 0) {   // the target opens the answer
        g0.active = 1;
        g0.remaining = P->target_first_n;
    }
    g0.eos = P->eos_id;
    g0.vlimit = vlimit;
    g0.max_new = max_new;
    g0.n_force = n_force;
    g0.prompt_len = prompt_len;
    g0.cap_steps = cap_steps;
    g0.cap_handoffs = cap_handoffs;
    g0.max_chunk = small->max_rows;
    if (large && large->max_rows < g0.max_chunk) g0.max_chunk = large->max_rows;
    g0.trace_first = out->trace_first_step;
    g0.trace_n = trace_n;
    g0.done = max_new == 0 ? 1 : 0;
    // every token costs a pass; a replaced probe sentence costs probe_len passes more per takeover
    const int64_t pass_cap = (1ll + g0.probe_len) * (max_new + 2) + 2ll * (total / g0.max_chunk + 2) * (max_new / P->n1 + 2);
    g0.pass_cap = pass_cap > 0x7fffffff ? 0x7fffffff : (int32_t)pass_cap;
    if (const char *e = getenv("ST_TEST_PASS_CAP")) {   // test aid: makes the device loop's pass bound run out
        const int cap = atoi(e);
        if (cap > 0 && cap < g0.pass_cap) g0.pass_cap = cap;
    }
    CK(cudaMemcpyAsync(gen, &g0, sizeof g0, cudaMemcpyHostToDevice, s));
    CK(cudaMemcpyAsync(b.tokens, prompt, (size_t)prompt_len * sizeof(int32_t), cudaMemcpyHostToDevice, s));
    if (n_force) CK(cudaMemcpyAsync(C.d_force, force, (size_t)n_force * sizeof(int32_t), cudaMemcpyHostToDevice, s));
    CK(cudaMemcpyAsync(C.d_cls, cls.data(), (size_t)vlimit, cudaMemcpyHostToDevice, s));
    if (P->n_aux > 0) CK(cudaMemcpyAsync(C.d_aux, P->aux_ids, (size_t)P->n_aux * sizeof(int32_t), cudaMemcpyHostToDevice, s));
    plan_first_pass_kernel<<<1, 1, 0, s>>>(gen, desc_small, desc_large);
    ++g_launches;
    CK(cudaGetLastError());

    cudaEvent_t ev0, ev1;
    CK(cudaEventCreate(&ev0));
    CK(cudaEventCreate(&ev1));
    CK(cudaEventRecord(ev0, s));
    GenState gh = g0;
    int rc = ST_OK;
    if (!host_loop) {
        // The whole generation is one graph launch; routing happens on the device.
        const int64_t before = g_launches;
        if (cudaGraphLaunch(C.exec, s) != cudaSuccess) {
            set_error_text("cudaGraphLaunch", cudaGetLastError());
            rc = ST_ERR_INTERNAL;
        }
        g_launches = before;   // counted below from the passes that actually ran
    } else {
        // Debugging aid: the same passes launched one by one; the host reads only the shape of the
        // next pass (which model, how many rows, whether it samples), never a token.
        const SampleCtx sc = gen_sample_ctx(C);
        for (int64_t pass = 0; pass < g0.pass_cap; ++pass) {
            if (cudaMemcpyAsync(&gh, gen, sizeof gh, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
                cudaStreamSynchronize(s) != cudaSuccess) {
                set_error_text("generation state readback", cudaGetLastError());
                rc = ST_ERR_INTERNAL;
                break;
            }
            if (gh.done) break;
            st_model *m = gh.next_model ? large : small;
            const int slot = gh.next_model ? gl.slot : gs.slot;
            StepDesc *d = gh.next_model ? desc_large : desc_small;
            const int ctx_after = gh.kv_len[gh.next_model] + gh.next_m;
            if (gh.next_m == 1 && gh.next_emit) rc = pass_decode(m, d, b.tokens, slot, ctx_after, sc);
            else rc = pass_rows(m, d, b.tokens, slot, gh.next_m, ctx_after, gh.next_emit != 0, sc);
            if (rc != ST_OK) break;
            if (!gh.next_emit) {
                advance_ingest_kernel<<<1, 1, 0, s>>>(gen, desc_small, desc_large);
                ++g_launches;
                if (cudaGetLastError() != cudaSuccess) { rc = ST_ERR_INTERNAL; break; }
            }
        }
    }
    cudaEventRecord(ev1, s);
    if (cudaStreamSynchronize(s) != cudaSuccess && rc == ST_OK) {
        set_error_text("generation", cudaGetLastError());
        rc = ST_ERR_INTERNAL;
    }
    float ms = 0.f;
    cudaEventElapsedTime(&ms, ev0, ev1);
    cudaEventDestroy(ev0);
    cudaEventDestroy(ev1);
    if (rc != ST_OK) return rc;
    CK(cudaMemcpy(&gh, gen, sizeof gh, cudaMemcpyDeviceToHost));
    if (!gh.done) return ST_ERR_INTERNAL;
    if (!host_loop) {   // kernels the graph ran: one dispatch per loop turn plus the kernels of every body that ran
        g_launches += (int64_t)gh.passes + 1;
        for (int i = 0; i < 2 * kBodiesPerModel; ++i) g_launches += C.body_launches[i] * gh.body_runs[i];
    }

    // ---- results ----
    out->n_tokens = gh.generated;
    out->n_steps = gh.step;
    out->n_handoffs = gh.n_handoffs;
    out->kv_len_small = gh.kv_len[0];
    out->kv_len_large = gh.kv_len[1];
    out->seconds = ms * 1e-3;
    out->bytes_algorithmic = gh.bytes_algo;
    out->t_prompt_prefill_s = (double)gh.t_kind[0] * 1e-9;
    out->t_catchup_s = (double)gh.t_kind[1] * 1e-9;
    out->t_decode_s = (double)gh.t_kind[2] * 1e-9;
    out->n_prompt_prefill = gh.n_kind[0];
    out->n_catchup = gh.n_kind[1];
    out->n_decode = gh.n_kind[2];
    const int n_steps = gh.step < cap_steps ? gh.step : cap_steps;
    const int n_hand = gh.n_handoffs < cap_handoffs ? gh.n_handoffs : cap_handoffs;
    if (gh.generated > 0) {
        CK(cudaMemcpyAsync(out->tokens, b.tokens + prompt_len, (size_t)gh.generated * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
        CK(cudaMemcpyAsync(out->source, b.source, (size_t)gh.generated, cudaMemcpyDeviceToHost, s));
    }
    if (n_steps > 0) {
        CK(cudaMemcpyAsync(out->emission_tokens, b.em_tok, (size_t)n_steps * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
        CK(cudaMemcpyAsync(out->emission_source, b.em_src, (size_t)n_steps, cudaMemcpyDeviceToHost, s));
        if (out->emission_fed) CK(cudaMemcpyAsync(out->emission_fed, b.em_fed, (size_t)n_steps * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
        if (out->emission_argmax) CK(cudaMemcpyAsync(out->emission_argmax, b.em_arg, (size_t)n_steps * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    }
    if (n_hand > 0) CK(cudaMemcpyAsync(out->handoffs, b.handoffs, (size_t)n_hand * 3 * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    if (n_hand > 0 && out->handoff_kinds) CK(cudaMemcpyAsync(out->handoff_kinds, b.hand_kind, (size_t)n_hand, cudaMemcpyDeviceToHost, s));
    if (trace_n > 0) CK(cudaMemcpyAsync(out->logits_trace, C.d_trace, (size_t)trace_n * vlimit * sizeof(float), cudaMemcpyDeviceToHost, s));
    CK(cudaStreamSynchronize(s));
    int32_t dev_status = 0;
    CK(cudaMemcpy(&dev_status, small->status, sizeof dev_status, cudaMemcpyDeviceToHost));
    if (large) {
        int32_t s2 = 0;
        CK(cudaMemcpy(&s2, large->status, sizeof s2, cudaMemcpyDeviceToHost));
        dev_status |= s2;
    }
    if (dev_status & DEV_LOG_FULL) return ST_ERR_CAPACITY;
    if (dev_status & DEV_BAD_TOKEN) return ST_ERR_VOCAB;
    if (dev_status & DEV_WAIT_EXPIRED) return ST_ERR_TIMEOUT;
    if (dev_status) return ST_ERR_INTERNAL;
    return ST_OK;
}

// Several independent generations advanced together.  Every round a one-thread kernel sorts the live
// sequences: those whose active model lacks exactly one token become rows of that model's batched decode pass
// (one pass over the weights for all of them, projections on the tensor cores), the others (prompt prefill,
// catch-up after a handoff) get a multi-row pass of their own.  The host reads back only the shape of the round
// (row counts, which sequences need a multi-row pass of how many rows), never a token; sampling and the handoff
// rule run on the device per sequence exactly as in st_generate_spec, so the results per sequence are the same.
// Returns ST_OK with *handled = false when the call does not qualify (a logits trace is wanted, more sequences
// than rows of a pass or than free sequence slots / KV pages): the caller then runs the sequences one by one.
static int generate_spec_batch_rounds(st_model *small, st_model *large, const st_spec_params *P, int32_t n, const int32_t *prompts,
                                      const int32_t *prompt_offsets, const int32_t *max_new_per_seq, const int32_t *force,
                                      const int32_t *force_offsets, st_spec_result *outs, bool *handled)
{
    *handled = false;
    static const bool sequential = [] { const char *e = getenv("ST_BATCH_SEQUENTIAL"); return e && e[0] == '1'; }();
    if (sequential || n < 2 || n > small->max_rows || (large && n > large->max_rows)) return ST_OK;
    if (P->temperature > 0.f) return ST_OK;   // the ragged passes' per-row argmax is greedy: sampled runs go one by one
    if (P->max_new_tokens < 0 || P->n1 < 1 || P->n_keywords < 0 || (P->n_keywords > 0 && !P->keyword_ids)) return ST_ERR_ARG;
    if (large && (large->stream != small->stream || large->device != small->device)) return ST_ERR_ARG;
    int vshared = small->cfg.vocab;
    if (large && large->cfg.vocab < vshared) vshared = large->cfg.vocab;
    const int vlimit = P->vocab_limit > 0 ? P->vocab_limit : vshared;
    if (vlimit > vshared) return ST_ERR_VOCAB;
    for (int i = 0; i < P->n_keywords; ++i)
        if ((unsigned)P->keyword_ids[i] >= (unsigned)vlimit) return ST_ERR_VOCAB;
    TRY(check_rule_params(P, vlimit));
    std::vector<int> plen(n), mnew(n), nforce(n), total(n);
    int longest = 0;
    for (int i = 0; i < n; ++i) {
        st_spec_result &o = outs[i];
        if (o.logits_trace && o.trace_n_steps > 0) return ST_OK;   // traces: one sequence at a time
        plen[i] = prompt_offsets[i + 1] - prompt_offsets[i];
        mnew[i] = max_new_per_seq ? max_new_per_seq[i] : P->max_new_tokens;
        nforce[i] = force ? force_offsets[i + 1] - force_offsets[i] : 0;
        total[i] = plen[i] + mnew[i] + 1;
        if (total[i] > longest) longest = total[i];
        if (mnew[i] < 0) return ST_ERR_ARG;
        if (o.cap_tokens < mnew[i] || (mnew[i] > 0 && (!o.tokens || !o.source))) return ST_ERR_CAPACITY;
        if ((o.cap_steps > 0 && (!o.emission_tokens || !o.emission_source)) || (o.cap_handoffs > 0 && !o.handoffs)) return ST_ERR_ARG;
        for (int j = prompt_offsets[i]; j < prompt_offsets[i + 1]; ++j)
            if ((unsigned)prompts[j] >= (unsigned)vlimit) return ST_ERR_VOCAB;
        for (int j = 0; j < nforce[i]; ++j)
            if (force[force_offsets[i] + j] >= vlimit) return ST_ERR_VOCAB;
    }
    // sequence slots and KV pages for every sequence on both models, or the sequential path
    std::vector<int32_t> slots(2 * (size_t)n, -1);
    auto release_slots = [&] {
        for (int i = 0; i < n; ++i) {
            if (slots[2 * i] >= 0) st_seq_free(small, slots[2 * i]);
            if (large && slots[2 * i + 1] >= 0) st_seq_free(large, slots[2 * i + 1]);
        }
    };
    for (int i = 0; i < n; ++i) {
        bool ok = st_seq_alloc(small, &slots[2 * i]) == ST_OK && seq_reserve(small, slots[2 * i], total[i]) == ST_OK;
        if (ok && large) ok = st_seq_alloc(large, &slots[2 * i + 1]) == ST_OK && seq_reserve(large, slots[2 * i + 1], total[i]) == ST_OK;
        if (!ok) {
            release_slots();
            return ST_OK;
        }
    }
    *handled = true;
    cudaStream_t s = small->stream;
    st_model *models[2] = {small, large};
    int rc = ST_OK;
    uint8_t *arena = nullptr;
    BatchPlan *plan_host = nullptr;
    cudaEvent_t ev0 = nullptr, ev1 = nullptr, ev_fork = nullptr, ev_join = nullptr;
    cudaStream_t side = nullptr;   // the speculative model's pass of a round that also has a target pass
    static const bool overlap = [] { const char *e = getenv("ST_BATCH_OVERLAP"); return !(e && e[0] == '0'); }();
    std::vector<GenState> gs(n);
    std::vector<GenBuffers> gb(n);
    GenState *d_gs = nullptr;
    do {
        for (int a = 0; a < 2; ++a) {
            st_model *m = models[a];
            if (!m) continue;
            if (cudaMemsetAsync(m->status, 0, sizeof(int32_t), s) != cudaSuccess) { rc = ST_ERR_INTERNAL; break; }
            if (!m->batch_logits) {
                m->batch_logits = (float *)m->dalloc((size_t)m->max_rows * m->cfg.vocab * sizeof(float));
                if (!m->batch_logits) { rc = ST_ERR_OOM; break; }
            }
        }
        if (rc != ST_OK) break;
        // ---- one device arena for the per-sequence state, buffers and logs ----
        size_t off = 0;
        auto take = [&](size_t bytes) { off = (off + 255) & ~(size_t)255; const size_t o = off; off += bytes; return o; };
        const size_t o_gs = take(n * sizeof(GenState)), o_gb = take(n * sizeof(GenBuffers)), o_slots = take(2 * n * sizeof(int32_t));
        const size_t o_descs = take(2 * n * sizeof(StepDesc)), o_bdesc = take(2 * sizeof(StepDesc));
        int max_chunk = small->max_rows;   // rows of one pass
        if (large && large->max_rows < max_chunk) max_chunk = large->max_rows;
        const size_t o_rtok = take(2 * (size_t)max_chunk * sizeof(int32_t)), o_amax = take(2 * (size_t)max_chunk * sizeof(int32_t));
        const size_t o_pseq = take(2 * n * sizeof(int32_t)), o_plast = take(2 * n * sizeof(int32_t)), o_npass = take(2 * sizeof(int32_t));
        const size_t o_plan = take(sizeof(BatchPlan)), o_cls = take((size_t)vlimit), o_aux = take(kMaxAuxTokens * sizeof(int32_t));
        std::vector<size_t> o_tok(n), o_src(n), o_emt(n), o_emf(n), o_ema(n), o_ems(n), o_hand(n), o_hkind(n), o_force(n);
        for (int i = 0; i < n; ++i) {
            const int cs = outs[i].cap_steps > 0 ? outs[i].cap_steps : 1, ch = outs[i].cap_handoffs > 0 ? outs[i].cap_handoffs : 1;
            o_tok[i] = take((size_t)total[i] * 4);
            o_src[i] = take((size_t)mnew[i] + 1);
            o_emt[i] = take((size_t)cs * 4);
            o_emf[i] = take((size_t)cs * 4);
            o_ema[i] = take((size_t)cs * 4);
            o_ems[i] = take((size_t)cs);
            o_hand[i] = take((size_t)ch * 12);
            o_hkind[i] = take((size_t)ch);
            o_force[i] = take((size_t)(nforce[i] > 0 ? nforce[i] : 1) * 4);
        }
        if (cudaMalloc(&arena, off + 256) != cudaSuccess) { cudaGetLastError(); rc = ST_ERR_OOM; break; }
        if (cudaMallocHost(&plan_host, sizeof(BatchPlan)) != cudaSuccess) { cudaGetLastError(); rc = ST_ERR_OOM; break; }
        d_gs = (GenState *)(arena + o_gs);
        GenBuffers *d_gb = (GenBuffers *)(arena + o_gb);
        int32_t *d_slots = (int32_t *)(arena + o_slots), *d_rtok = (int32_t *)(arena + o_rtok), *d_pseq = (int32_t *)(arena + o_pseq);
        int32_t *d_plast = (int32_t *)(arena + o_plast), *d_npass = (int32_t *)(arena + o_npass);
        int32_t *d_amax = (int32_t *)(arena + o_amax);
        StepDesc *d_descs = (StepDesc *)(arena + o_descs), *d_bdesc = (StepDesc *)(arena + o_bdesc);
        BatchPlan *d_plan = (BatchPlan *)(arena + o_plan);
        uint8_t *d_cls = arena + o_cls;
        std::vector<uint8_t> cls(vlimit, 0);
        fill_class_table(P, cls);
        for (int i = 0; i < n; ++i) {
            GenState &g = gs[i];
            g = GenState{};
            g.wbytes[0] = small->weight_bytes;
            g.kvb[0] = st_kv_bytes_per_token(small);
            if (large) {
                g.wbytes[1] = large->weight_bytes;
                g.kvb[1] = st_kv_bytes_per_token(large);
            }
            g.has_large = large ? 1 : 0;
            g.pos = plen[i];
            g.delimiter = P->delimiter_id;
            g.n1 = P->n1;
            g.keep_probe = P->keep_probe;
            g.every_delim = P->takeover_every_delimiter ? 1 : 0;
            g.n2 = P->n2;
            g.n3 = P->n3;
            g.neg_threshold = P->neg_threshold;
            g.n_aux = P->n_aux;
            g.probe_len = P->probe_len > 1 ? P->probe_len : 1;
            if (large && P->target_first_n > 0) {
                g.active = 1;
                g.remaining = P->target_first_n;
            }
            g.eos = P->eos_id;
            g.vlimit = vlimit;
            g.max_new = mnew[i];
            g.n_force = nforce[i];
            g.prompt_len = plen[i];
            g.cap_steps = outs[i].cap_steps;
            g.cap_handoffs = outs[i].cap_handoffs;
            g.max_chunk = max_chunk;
            g.done = mnew[i] == 0 ? 1 : 0;
            g.pass_cap = 0x7fffffff;
            GenBuffers &b = gb[i];
            b.tokens = (int32_t *)(arena + o_tok[i]);
            b.source = arena + o_src[i];
            b.em_tok = (int32_t *)(arena + o_emt[i]);
            b.em_fed = (int32_t *)(arena + o_emf[i]);
            b.em_arg = (int32_t *)(arena + o_ema[i]);
            b.em_src = arena + o_ems[i];
            b.handoffs = (int32_t *)(arena + o_hand[i]);
            b.hand_kind = arena + o_hkind[i];
            b.aux = (const int32_t *)(arena + o_aux);
            b.force = (const int32_t *)(arena + o_force[i]);
            b.cls = d_cls;
            b.trace = nullptr;
        }
        bool up = cudaMemcpyAsync(d_gs, gs.data(), n * sizeof(GenState), cudaMemcpyHostToDevice, s) == cudaSuccess &&
                  cudaMemcpyAsync(d_gb, gb.data(), n * sizeof(GenBuffers), cudaMemcpyHostToDevice, s) == cudaSuccess &&
                  cudaMemcpyAsync(d_slots, slots.data(), 2 * n * sizeof(int32_t), cudaMemcpyHostToDevice, s) == cudaSuccess &&
                  cudaMemcpyAsync(d_cls, cls.data(), (size_t)vlimit, cudaMemcpyHostToDevice, s) == cudaSuccess &&
                  (P->n_aux == 0 ||
                   cudaMemcpyAsync(arena + o_aux, P->aux_ids, (size_t)P->n_aux * sizeof(int32_t), cudaMemcpyHostToDevice, s) == cudaSuccess);
        for (int i = 0; i < n && up; ++i) {
            up = cudaMemcpyAsync(gb[i].tokens, prompts + prompt_offsets[i], (size_t)plen[i] * 4, cudaMemcpyHostToDevice, s) == cudaSuccess;
            if (up && nforce[i] > 0)
                up = cudaMemcpyAsync(arena + o_force[i], force + force_offsets[i], (size_t)nforce[i] * 4, cudaMemcpyHostToDevice, s) == cudaSuccess;
        }
        if (!up) { set_error_text("batched generation upload", cudaGetLastError()); rc = ST_ERR_INTERNAL; break; }
        if (cudaEventCreate(&ev0) != cudaSuccess || cudaEventCreate(&ev1) != cudaSuccess) { rc = ST_ERR_INTERNAL; break; }
        if (overlap && (cudaStreamCreateWithFlags(&side, cudaStreamNonBlocking) != cudaSuccess ||
                        cudaEventCreateWithFlags(&ev_fork, cudaEventDisableTiming) != cudaSuccess ||
                        cudaEventCreateWithFlags(&ev_join, cudaEventDisableTiming) != cudaSuccess)) { rc = ST_ERR_INTERNAL; break; }
        cudaEventRecord(ev0, s);
        // ---- rounds ----
        int64_t sum_new = 0;
        for (int i = 0; i < n; ++i) sum_new += mnew[i];
        const int64_t round_cap = (3ll + (P->probe_len > 1 ? P->probe_len : 1)) * (sum_new + 4ll * n + 16) + 4ll * n * (longest / max_chunk + 2);
        // rows the target's pass waits for while the speculative model has work: 45 % of the sequences still running
        int min_target_rows = -45;
        if (const char *e = getenv("ST_BATCH_TARGET_MIN")) min_target_rows = atoi(e);   // tuning aid
        bool finished = false;
        for (int64_t round = 0; round < round_cap && rc == ST_OK; ++round) {
            batch_plan_kernel<<<1, 1, 0, s>>>(d_gs, d_gb, n, d_slots, d_descs, small->row_slot, small->row_pos,
                                              large ? large->row_slot : small->row_slot, large ? large->row_pos : small->row_pos,
                                              d_rtok, d_pseq, d_plast, d_npass, d_bdesc, max_chunk, min_target_rows, d_plan);
            ++g_launches;
            if (cudaMemcpyAsync(plan_host, d_plan, sizeof(BatchPlan), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
                cudaStreamSynchronize(s) != cudaSuccess) {
                set_error_text("batched generation round", cudaGetLastError());
                rc = ST_ERR_INTERNAL;
                break;
            }
            const BatchPlan &pl = *plan_host;
            if (pl.all_done) { finished = true; break; }
            // The two models' passes of a round hold different sequences and touch nothing in common: when both
            // have rows, the speculative model's pass and routing run on a side stream beside the target's pass
            // (its short kernels fill the gaps of the target's weight streaming) and join before the next step.
            const bool both = overlap && large && pl.n_dec[0] > 0 && pl.n_dec[1] > 0;
            if (both && (cudaEventRecord(ev_fork, s) != cudaSuccess || cudaStreamWaitEvent(side, ev_fork, 0) != cudaSuccess)) {
                rc = ST_ERR_INTERNAL;
                break;
            }
            for (int a = 0; a < 2 && rc == ST_OK; ++a) {
                const int rows = pl.n_dec[a];
                st_model *m = models[a];
                if (rows <= 0 || !m) continue;
                cudaStream_t ps = both && a == 0 ? side : s;
                SampleCtx sc{};
                sc.logits_out = m->batch_logits;
                sc.argmax_out = d_amax + (size_t)a * max_chunk;
                sc.want_argmax = true;
                sc.vlimit = vlimit;
                int m_upper = (rows + 31) / 32 * 32;
                if (m_upper > m->max_rows) m_upper = m->max_rows;
                m->stream = ps;
                rc = pass_rows_batch_graphed(m, d_bdesc + a, d_rtok + (size_t)a * max_chunk, m_upper, pl.max_ctx[a], sc);
                m->stream = s;
                if (rc != ST_OK) break;
                batch_router_kernel<<<1, 64, 0, ps>>>(d_gs, d_gb, d_pseq + (size_t)a * n, d_plast + (size_t)a * n, d_npass + a,
                                                      d_amax + (size_t)a * max_chunk, d_descs, small->status);
                ++g_launches;
                if (cudaGetLastError() != cudaSuccess) rc = ST_ERR_INTERNAL;
            }
            // joined even after an error, so that nothing is still running on the side stream when the arena is freed
            if (both && (cudaEventRecord(ev_join, side) != cudaSuccess || cudaStreamWaitEvent(s, ev_join, 0) != cudaSuccess)) rc = ST_ERR_INTERNAL;
            for (int k = 0; k < pl.n_cu && rc == ST_OK; ++k) {
                const int i = pl.cu[k][0], a = pl.cu[k][1], rows = pl.cu[k][2], pos0 = pl.cu[k][3], emit = pl.cu[k][4];
                st_model *m = models[a];
                if (i < 0 || i >= n || !m || rows < 1 || rows > m->max_rows) { rc = ST_ERR_INTERNAL; break; }
                SampleCtx sc{};
                sc.vlimit = vlimit;
                sc.gen = d_gs + i;
                sc.buf = gb[i];
                sc.desc_small = d_descs + 2 * i;
                sc.desc_large = d_descs + 2 * i + 1;
                sc.want_argmax = true;
                rc = pass_rows(m, d_descs + 2 * i + a, gb[i].tokens, slots[2 * i + a], rows, pos0 + rows, emit != 0, sc);
                if (rc == ST_OK && !emit) {
                    advance_ingest_kernel<<<1, 1, 0, s>>>(d_gs + i, d_descs + 2 * i, d_descs + 2 * i + 1);
                    ++g_launches;
                    if (cudaGetLastError() != cudaSuccess) rc = ST_ERR_INTERNAL;
                }
            }
        }
        if (rc != ST_OK) break;
        cudaEventRecord(ev1, s);
        if (cudaStreamSynchronize(s) != cudaSuccess) { set_error_text("batched generation", cudaGetLastError()); rc = ST_ERR_INTERNAL; break; }
        if (!finished) { rc = ST_ERR_TIMEOUT; break; }
        float ms = 0.f;
        cudaEventElapsedTime(&ms, ev0, ev1);
        // ---- results ----
        if (cudaMemcpy(gs.data(), d_gs, n * sizeof(GenState), cudaMemcpyDeviceToHost) != cudaSuccess) { rc = ST_ERR_INTERNAL; break; }
        bool dn = true;
        for (int i = 0; i < n && dn; ++i) {
            const GenState &g = gs[i];
            const GenBuffers &b = gb[i];
            st_spec_result &o = outs[i];
            o.n_tokens = g.generated;
            o.n_steps = g.step;
            o.n_handoffs = g.n_handoffs;
            o.kv_len_small = g.kv_len[0];
            o.kv_len_large = g.kv_len[1];
            o.seconds = ms * 1e-3;   // of the whole batch
            o.bytes_algorithmic = g.bytes_algo;
            o.t_prompt_prefill_s = o.t_catchup_s = o.t_decode_s = 0.0;
            o.n_prompt_prefill = g.n_kind[0];
            o.n_catchup = g.n_kind[1];
            o.n_decode = g.n_kind[2];
            const int n_steps = g.step < o.cap_steps ? g.step : o.cap_steps;
            const int n_hand = g.n_handoffs < o.cap_handoffs ? g.n_handoffs : o.cap_handoffs;
            if (g.generated > 0) {
                dn = dn && cudaMemcpyAsync(o.tokens, b.tokens + plen[i], (size_t)g.generated * 4, cudaMemcpyDeviceToHost, s) == cudaSuccess;
                dn = dn && cudaMemcpyAsync(o.source, b.source, (size_t)g.generated, cudaMemcpyDeviceToHost, s) == cudaSuccess;
            }
            if (n_steps > 0) {
                dn = dn && cudaMemcpyAsync(o.emission_tokens, b.em_tok, (size_t)n_steps * 4, cudaMemcpyDeviceToHost, s) == cudaSuccess;
                dn = dn && cudaMemcpyAsync(o.emission_source, b.em_src, (size_t)n_steps, cudaMemcpyDeviceToHost, s) == cudaSuccess;
                if (o.emission_fed) dn = dn && cudaMemcpyAsync(o.emission_fed, b.em_fed, (size_t)n_steps * 4, cudaMemcpyDeviceToHost, s) == cudaSuccess;
                if (o.emission_argmax) dn = dn && cudaMemcpyAsync(o.emission_argmax, b.em_arg, (size_t)n_steps * 4, cudaMemcpyDeviceToHost, s) == cudaSuccess;
            }
            if (n_hand > 0) dn = dn && cudaMemcpyAsync(o.handoffs, b.handoffs, (size_t)n_hand * 12, cudaMemcpyDeviceToHost, s) == cudaSuccess;
            if (n_hand > 0 && o.handoff_kinds)
                dn = dn && cudaMemcpyAsync(o.handoff_kinds, b.hand_kind, (size_t)n_hand, cudaMemcpyDeviceToHost, s) == cudaSuccess;
        }
        if (!dn || cudaStreamSynchronize(s) != cudaSuccess) { set_error_text("batched generation results", cudaGetLastError()); rc = ST_ERR_INTERNAL; break; }
        int32_t dev_status = 0, s2 = 0;
        cudaMemcpy(&dev_status, small->status, sizeof dev_status, cudaMemcpyDeviceToHost);
        if (large) cudaMemcpy(&s2, large->status, sizeof s2, cudaMemcpyDeviceToHost);
        dev_status |= s2;
        if (dev_status & DEV_LOG_FULL) rc = ST_ERR_CAPACITY;
        else if (dev_status & DEV_BAD_TOKEN) rc = ST_ERR_VOCAB;
        else if (dev_status & DEV_WAIT_EXPIRED) rc = ST_ERR_TIMEOUT;
        else if (dev_status) rc = ST_ERR_INTERNAL;
    } while (0);
    cudaStreamSynchronize(s);
    if (side) {
        cudaStreamSynchronize(side);
        cudaStreamDestroy(side);
    }
    if (ev0) cudaEventDestroy(ev0);
    if (ev1) cudaEventDestroy(ev1);
    if (ev_fork) cudaEventDestroy(ev_fork);
    if (ev_join) cudaEventDestroy(ev_join);
    if (plan_host) cudaFreeHost(plan_host);
    if (arena) cudaFree(arena);
    release_slots();
    return rc;
}

extern "C" int st_generate_spec_batch(st_model *small, st_model *large, const st_spec_params *P, int32_t n_seqs,
                                      const int32_t *prompts, const int32_t *prompt_offsets, const int32_t *max_new_per_seq,
                                      const int32_t *force, const int32_t *force_offsets, st_spec_result *outs)
{
    if (!small || !P || n_seqs < 0 || (n_seqs > 0 && (!prompts || !prompt_offsets || !outs))) return ST_ERR_ARG;
    if (force && !force_offsets) return ST_ERR_ARG;
    for (int i = 0; i < n_seqs; ++i) {
        if (prompt_offsets[i + 1] <= prompt_offsets[i]) return ST_ERR_ARG;
        if (force && force_offsets[i + 1] < force_offsets[i]) return ST_ERR_ARG;
    }
    bool handled = false;
    TRY(generate_spec_batch_rounds(small, large, P, n_seqs, prompts, prompt_offsets, max_new_per_seq, force, force_offsets, outs, &handled));
    if (handled) return ST_OK;
    for (int i = 0; i < n_seqs; ++i) {
        st_spec_params pi = *P;
        if (max_new_per_seq) pi.max_new_tokens = max_new_per_seq[i];
        const int32_t *f = force ? force + force_offsets[i] : nullptr;
        const int32_t nf = force ? force_offsets[i + 1] - force_offsets[i] : 0;
        TRY(st_generate_spec(small, large, &pi, prompts + prompt_offsets[i], prompt_offsets[i + 1] - prompt_offsets[i],
                             nf > 0 ? f : nullptr, nf, &outs[i]));
    }
    return ST_OK;
}

// ------------------------------------------------------------------------------------------------
// greedy speculative decoding (the paper's comparison system)
// ------------------------------------------------------------------------------------------------

namespace {
struct DevArena {   // one cudaMalloc for the buffers of a call
    uint8_t *base = nullptr;
    size_t off = 0;
    size_t take(size_t bytes) { off = (off + 255) & ~(size_t)255; const size_t o = off; off += bytes; return o; }
    ~DevArena() { if (base) cudaFree(base); }
};
}  // namespace

// Rounds are driven from the host: the speculative model drafts g tokens (single-kernel decode steps chained on the
// device: each step reads the token the previous one placed), the target scores the pending tokens and the drafts in
// one multi-row pass whose LM head covers every row (the ragged-batch pass with all rows on one sequence), a
// one-thread kernel applies the acceptance rule, and the host reads back how far the text advanced (never a token)
// to size the next round and to cut both caches back to the accepted length.
extern "C" int st_generate_specdec(st_model *small, st_model *large, const st_specdec_params *P, const int32_t *prompt,
                                   int32_t prompt_len, const int32_t *force_draft, int32_t n_force_draft,
                                   const int32_t *force_target, int32_t n_force_target, st_specdec_result *out)
{
    if (!small || !large || !P || !prompt || !out || prompt_len < 1 || P->max_new_tokens < 0 || P->gamma < 1) return ST_ERR_ARG;
    if (n_force_draft < 0 || n_force_target < 0 || (n_force_draft > 0 && !force_draft) || (n_force_target > 0 && !force_target)) return ST_ERR_ARG;
    if (large->stream != small->stream || large->device != small->device) return ST_ERR_ARG;
    const int gamma = P->gamma, max_new = P->max_new_tokens;
    if (gamma + 1 > large->max_rows - 1) return ST_ERR_UNSUPPORTED;
    const int vshared = small->cfg.vocab < large->cfg.vocab ? small->cfg.vocab : large->cfg.vocab;
    const int vlimit = P->vocab_limit > 0 ? P->vocab_limit : vshared;
    if (vlimit > vshared) return ST_ERR_VOCAB;
    for (int i = 0; i < prompt_len; ++i)
        if ((unsigned)prompt[i] >= (unsigned)vlimit) return ST_ERR_VOCAB;
    for (int i = 0; i < n_force_draft; ++i)
        if (force_draft[i] >= vlimit) return ST_ERR_VOCAB;
    for (int i = 0; i < n_force_target; ++i)
        if (force_target[i] >= vlimit) return ST_ERR_VOCAB;
    if (out->cap_tokens < max_new || (max_new > 0 && (!out->tokens || !out->source))) return ST_ERR_CAPACITY;
    if (out->cap_rounds > 0 && (!out->round_drafted || !out->round_accepted)) return ST_ERR_ARG;
    out->n_tokens = out->n_rounds = out->n_drafted = out->n_accepted = 0;
    out->kv_len_small = out->kv_len_large = 0;
    out->seconds = 0.0;
    out->bytes_algorithmic = 0;
    if (max_new == 0) return ST_OK;

    cudaStream_t s = small->stream;
    st_model *models[2] = {small, large};
    for (st_model *m : models) {
        CK(cudaMemsetAsync(m->status, 0, sizeof(int32_t), s));
        CK(cudaMemsetAsync(m->mega_sync, 0, kMegaSyncWords * sizeof(unsigned), s));
    }
    if (!large->batch_logits) {
        large->batch_logits = (float *)large->dalloc((size_t)large->max_rows * large->cfg.vocab * sizeof(float));
        if (!large->batch_logits) return ST_ERR_OOM;
    }
    const int total = prompt_len + max_new + gamma + 2;
    SlotGuard gs{small}, gl{large};
    TRY(st_seq_alloc(small, &gs.slot));
    TRY(seq_reserve(small, gs.slot, total));
    TRY(st_seq_alloc(large, &gl.slot));
    TRY(seq_reserve(large, gl.slot, total));

    const int cap_rounds = out->cap_rounds > 0 ? out->cap_rounds : 1;
    const int cap_drafts = out->cap_drafts > 0 ? out->cap_drafts : 1;
    DevArena A;
    const size_t o_state = A.take(sizeof(SpecDecState)), o_tok = A.take((size_t)total * 4), o_src = A.take((size_t)max_new + 1);
    const size_t o_rd = A.take((size_t)cap_rounds * 4), o_ra = A.take((size_t)cap_rounds * 4);
    const size_t o_dt = A.take((size_t)cap_drafts * 4), o_da = A.take((size_t)cap_drafts * 4), o_ca = A.take(((size_t)max_new + 1) * 4);
    const size_t o_fd = A.take((size_t)(n_force_draft > 0 ? n_force_draft : 1) * 4), o_ft = A.take((size_t)(n_force_target > 0 ? n_force_target : 1) * 4);
    const size_t o_desc = A.take((size_t)(gamma + 8) * sizeof(StepDesc)), o_amax_s = A.take(4), o_amax_l = A.take((size_t)large->max_rows * 4);
    if (cudaMalloc(&A.base, A.off + 256) != cudaSuccess) { cudaGetLastError(); return ST_ERR_OOM; }
    SpecDecState *d_state = (SpecDecState *)(A.base + o_state);
    SpecDecBuffers b{};
    b.tokens = (int32_t *)(A.base + o_tok);
    b.source = A.base + o_src;
    b.round_drafted = (int32_t *)(A.base + o_rd);
    b.round_accepted = (int32_t *)(A.base + o_ra);
    b.draft_tok = (int32_t *)(A.base + o_dt);
    b.draft_arg = (int32_t *)(A.base + o_da);
    b.choice_arg = (int32_t *)(A.base + o_ca);
    b.force_draft = (const int32_t *)(A.base + o_fd);
    b.force_target = (const int32_t *)(A.base + o_ft);
    StepDesc *d_desc = (StepDesc *)(A.base + o_desc);
    int32_t *d_amax_s = (int32_t *)(A.base + o_amax_s), *d_amax_l = (int32_t *)(A.base + o_amax_l);

    SpecDecState st{};
    st.pos = prompt_len;
    st.eos = P->eos_id;
    st.max_new = max_new;
    st.vlimit = vlimit;
    st.n_force_draft = n_force_draft;
    st.n_force_target = n_force_target;
    st.cap_rounds = out->cap_rounds;
    st.cap_drafts = out->cap_drafts;
    st.prompt_len = prompt_len;
    CK(cudaMemcpyAsync(d_state, &st, sizeof st, cudaMemcpyHostToDevice, s));
    CK(cudaMemcpyAsync(b.tokens, prompt, (size_t)prompt_len * 4, cudaMemcpyHostToDevice, s));
    if (n_force_draft) CK(cudaMemcpyAsync(A.base + o_fd, force_draft, (size_t)n_force_draft * 4, cudaMemcpyHostToDevice, s));
    if (n_force_target) CK(cudaMemcpyAsync(A.base + o_ft, force_target, (size_t)n_force_target * 4, cudaMemcpyHostToDevice, s));

    cudaEvent_t ev0, ev1;
    CK(cudaEventCreate(&ev0));
    CK(cudaEventCreate(&ev1));
    CK(cudaEventRecord(ev0, s));
    int kv_s = 0, kv_l = 0;   // cached lengths (host mirrors; the passes take their positions from descriptors)
    int64_t bytes = 0;
    int rc = ST_OK;
    std::vector<StepDesc> descs;
    std::vector<int32_t> rows;
    // a model ingests `pending` tokens starting at position kv (chunks of a pass's rows); the last chunk samples into amax
    auto ingest = [&](st_model *m, int slot, int &kv, int pending, int32_t *amax, bool sample_last) -> int {
        while (pending > 0 && rc == ST_OK) {
            const int rows_now = pending < m->max_rows ? pending : m->max_rows;
            const bool last = rows_now == pending;
            const bool emit = last && sample_last;
            StepDesc d{kv, rows_now, kv, emit ? 1 : 0};
            const int di = (int)descs.size();
            if (di >= gamma + 8) { CK(cudaStreamSynchronize(s)); descs.clear(); }
            descs.push_back(d);
            StepDesc *dd = d_desc + (descs.size() - 1);
            CK(cudaMemcpyAsync(dd, &descs.back(), sizeof d, cudaMemcpyHostToDevice, s));
            SampleCtx sc{};
            sc.argmax_out = amax;
            sc.vlimit = vlimit;
            sc.want_argmax = emit;
            if (rows_now == 1 && emit) rc = pass_decode(m, dd, b.tokens, slot, kv + 1, sc);
            else rc = pass_rows(m, dd, b.tokens, slot, rows_now, kv + rows_now, emit, sc);
            bytes += m->weight_bytes + st_kv_bytes_per_token(m) * (int64_t)(kv + rows_now);
            kv += rows_now;
            pending -= rows_now;
        }
        return rc;
    };
    const int64_t round_cap = (int64_t)max_new + 4;
    int generated = 0, pos = prompt_len;
    for (int64_t round = 0; round < round_cap && rc == ST_OK; ++round) {
        descs.clear();
        descs.reserve(gamma + 8);
        int g = max_new - generated - 1;
        g = g > gamma ? gamma : g;
        CK(cudaMemcpyAsync(&d_state->g, &g, sizeof g, cudaMemcpyHostToDevice, s));
        // ---- drafts ----
        for (int i = 0; i < g && rc == ST_OK; ++i) {
            TRY(ingest(small, gs.slot, kv_s, pos + i - kv_s, d_amax_s, true));
            specdec_take_draft_kernel<<<1, 1, 0, s>>>(d_state, b, d_amax_s, i, small->status);
            ++g_launches;
            CK(cudaGetLastError());
        }
        // ---- the target scores the pending tokens and the drafts: all rows of its last pass get logits ----
        int pending = pos + g - kv_l;
        if (pending > large->max_rows) TRY(ingest(large, gl.slot, kv_l, pending - (g + 1), nullptr, false));   // a long prompt first
        pending = pos + g - kv_l;
        {
            rows.assign(2 * (size_t)pending, 0);
            for (int j = 0; j < pending; ++j) { rows[j] = gl.slot; rows[pending + j] = kv_l + j; }
            CK(cudaMemcpyAsync(large->row_slot, rows.data(), (size_t)pending * 4, cudaMemcpyHostToDevice, s));
            CK(cudaMemcpyAsync(large->row_pos, rows.data() + pending, (size_t)pending * 4, cudaMemcpyHostToDevice, s));
            StepDesc d{0, pending, kv_l, 1};
            descs.push_back(d);
            StepDesc *dd = d_desc + (descs.size() - 1);
            CK(cudaMemcpyAsync(dd, &descs.back(), sizeof d, cudaMemcpyHostToDevice, s));
            SampleCtx sc{};
            sc.logits_out = large->batch_logits;
            sc.argmax_out = d_amax_l;
            sc.vlimit = vlimit;
            sc.want_argmax = true;
            int m_upper = (pending + 31) / 32 * 32;
            if (m_upper > large->max_rows) m_upper = large->max_rows;
            TRY(pass_rows(large, dd, b.tokens, -1, m_upper, kv_l + pending, true, sc, true));
            bytes += large->weight_bytes + st_kv_bytes_per_token(large) * (int64_t)(kv_l + pending);
        }
        specdec_accept_kernel<<<1, 1, 0, s>>>(d_state, b, d_amax_l + (pending - (g + 1)), large->status);
        ++g_launches;
        CK(cudaGetLastError());
        CK(cudaMemcpyAsync(&st, d_state, sizeof st, cudaMemcpyDeviceToHost, s));
        CK(cudaStreamSynchronize(s));   // also makes the staging vectors reusable
        kv_l += pending;
        pos = st.pos;
        generated = st.generated;
        // both caches keep the accepted prefix only (the target's own token has not been fed to anyone)
        if (kv_l > pos - 1) kv_l = pos - 1;
        if (kv_s > pos - 1) kv_s = pos - 1;
        if (st.done) break;
    }
    cudaEventRecord(ev1, s);
    if (cudaStreamSynchronize(s) != cudaSuccess && rc == ST_OK) { set_error_text("speculative decoding", cudaGetLastError()); rc = ST_ERR_INTERNAL; }
    float ms = 0.f;
    cudaEventElapsedTime(&ms, ev0, ev1);
    cudaEventDestroy(ev0);
    cudaEventDestroy(ev1);
    if (rc != ST_OK) return rc;
    if (!st.done) return ST_ERR_TIMEOUT;
    out->n_tokens = st.generated;
    out->n_rounds = st.n_rounds;
    out->n_drafted = st.n_drafted;
    out->n_accepted = st.n_accepted;
    out->kv_len_small = kv_s;
    out->kv_len_large = kv_l;
    out->seconds = ms * 1e-3;
    out->bytes_algorithmic = bytes;
    const int nr = st.n_rounds < out->cap_rounds ? st.n_rounds : out->cap_rounds;
    const int nd = st.k_draft < out->cap_drafts ? st.k_draft : out->cap_drafts;
    CK(cudaMemcpyAsync(out->tokens, b.tokens + prompt_len, (size_t)st.generated * 4, cudaMemcpyDeviceToHost, s));
    CK(cudaMemcpyAsync(out->source, b.source, (size_t)st.generated, cudaMemcpyDeviceToHost, s));
    if (nr > 0) {
        CK(cudaMemcpyAsync(out->round_drafted, b.round_drafted, (size_t)nr * 4, cudaMemcpyDeviceToHost, s));
        CK(cudaMemcpyAsync(out->round_accepted, b.round_accepted, (size_t)nr * 4, cudaMemcpyDeviceToHost, s));
    }
    if (nd > 0 && out->draft_tokens) CK(cudaMemcpyAsync(out->draft_tokens, b.draft_tok, (size_t)nd * 4, cudaMemcpyDeviceToHost, s));
    if (nd > 0 && out->draft_argmax) CK(cudaMemcpyAsync(out->draft_argmax, b.draft_arg, (size_t)nd * 4, cudaMemcpyDeviceToHost, s));
    if (out->choice_argmax) CK(cudaMemcpyAsync(out->choice_argmax, b.choice_arg, (size_t)st.generated * 4, cudaMemcpyDeviceToHost, s));
    CK(cudaStreamSynchronize(s));
    int32_t dev_status = 0, s2 = 0;
    CK(cudaMemcpy(&dev_status, small->status, sizeof dev_status, cudaMemcpyDeviceToHost));
    CK(cudaMemcpy(&s2, large->status, sizeof s2, cudaMemcpyDeviceToHost));
    dev_status |= s2;
    if (dev_status & DEV_LOG_FULL) return ST_ERR_CAPACITY;
    if (dev_status & DEV_BAD_TOKEN) return ST_ERR_VOCAB;
    if (dev_status & DEV_WAIT_EXPIRED) return ST_ERR_TIMEOUT;
    if (dev_status) return ST_ERR_INTERNAL;
    return ST_OK;
}

// ------------------------------------------------------------------------------------------------
// greedy sampling without any allocation
// ------------------------------------------------------------------------------------------------

// Scratch of st_argmax_static: 64 partial maxima, 64 partial indices (int bits) and one ticket word.
// It lives in the library image, so every GPU that loads the library holds these 1 KB until exit.
static constexpr int kStaticArgmaxBlocks = 64;
static constexpr int32_t kStaticArgmaxMaxN = 1 << 22;
static __device__ __align__(256) float g_static_argmax_scratch[256];

extern "C" int st_argmax_static(const float *logits_dev, int32_t n, int32_t *argmax_out_dev, void *cuda_stream)
{
    if (!logits_dev || !argmax_out_dev || n < 1) return ST_ERR_ARG;
    if (n > kStaticArgmaxMaxN) {
        snprintf(g_err_text, sizeof g_err_text, "st_argmax_static: %d elements exceed the built-in scratch limit of %d", n,
                 kStaticArgmaxMaxN);
        return ST_ERR_CAPACITY;
    }
    // The symbol name is only a host-side handle; the kernel needs the device address, looked up once
    // per device with that device current.
    static float *scratch_of_device[64] = {};
    int dev = 0;
    CK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return ST_ERR_UNSUPPORTED;
    if (!scratch_of_device[dev]) {
        float *ptr = nullptr;
        CK(cudaGetSymbolAddress((void **)&ptr, g_static_argmax_scratch));
        scratch_of_device[dev] = ptr;
    }
    float *scratch = scratch_of_device[dev];
    cudaStream_t s = (cudaStream_t)cuda_stream;
    // the array keeps whatever the previous call left: the ticket word must start at zero
    CK(cudaMemsetAsync(scratch + 2 * kStaticArgmaxBlocks, 0, sizeof(int32_t), s));
    ArgmaxParams a{};
    a.logits = logits_dev;
    a.limit = n;
    a.part_val = scratch;
    a.part_idx = reinterpret_cast<int32_t *>(scratch + kStaticArgmaxBlocks);
    a.ticket = reinterpret_cast<int32_t *>(scratch + 2 * kStaticArgmaxBlocks);
    a.argmax_out = argmax_out_dev;
    argmax_router_kernel<<<kStaticArgmaxBlocks, 256, 0, s>>>(a);
    ++g_launches;
    CK(cudaGetLastError());
    return ST_OK;
}
