// Greedy sampling fused with the Speculative Thinking handoff rule (paper Section 3, takeover (1)).
//
// After a model's LM head, one kernel finds the lowest-id argmax of the logits below vocab_limit
// and -- in its last-arriving CTA -- advances the generation state on the device: which model is
// active, how many tokens the target still owes, the write position, each model's cached length,
// the output and the handoff log, and the description of the next pass.  The host only learns the
// kind and size of the next pass; it never sees a token before deciding what to launch.
#pragma once
#include "st_common.cuh"
#include "weights.cuh"

namespace st {

constexpr int kClsDelim = 1;    // class-table bit of a delimiter
constexpr int kClsKeyword = 2;  // ... of a reflection keyword
constexpr int kClsAffirm = 4;   // ... of an affirmation cue
constexpr int kClsVerify = 8;   // ... of a verification cue

struct GenState {
    // --- accounting (64-bit fields first) ---
    int64_t bytes_algo;      // weights + KV bytes the passes so far had to move
    int64_t wbytes[2];       // weight bytes one pass of each model streams
    int64_t kvb[2];          // KV bytes per cached token of each model
    // --- dynamic ---
    int32_t active;      // 0 = speculative (small), 1 = target (large)
    int32_t remaining;   // tokens the target still writes in this takeover
    int32_t pos;         // next position to write (prompt included)
    int32_t step;        // emission steps so far
    int32_t generated;   // tokens written after the prompt
    int32_t kv_len[2];   // cached length of each model
    int32_t done;
    int32_t n_handoffs;
    int32_t next_model;  // the pass to run next ...
    int32_t next_m;      // ... ingests this many tokens ...
    int32_t next_emit;   // ... and samples a token (1) or only ingests (0)
    int32_t ingested;    // tokens already ingested by ingest-only chunks of the catch-up in progress
    int32_t passes;      // passes dispatched so far
    int32_t body_runs[12];  // how often each graph body ran (per model: decode, 4 row buckets, ingest)
    int32_t pass_cap;    // hard bound on passes (the device loop stops there)
    // --- parameters ---
    int32_t has_large, delimiter, n1, keep_probe, eos, vlimit, max_new, n_force;
    int32_t n2, n3, neg_threshold, n_aux;   // takeovers (2) and (3): segment lengths, counter bound (< 0: off), auxiliary tokens
    int32_t probe_len;                      // tokens of the speculative model's sentence after a delimiter that are classified
    int32_t probing, probe_start, probe_n, n_refl, n_aff, n_ver;   // the probe in progress
    int32_t neg_count;                      // reflection cues the speculative model sampled since the last takeover (3)
    int32_t every_delim;   // 1: no keyword test; the target takes over after every delimiter the speculative model writes
    int32_t prompt_len, cap_steps, cap_handoffs, max_chunk;
    int32_t trace_first, trace_n;
    // --- device time by kind of pass: 0 prompt prefill, 1 catch-up, 2 decode ---
    unsigned long long t_last;       // global timer at the end of the previous pass (or at the start)
    unsigned long long t_pending;    // time of the ingest-only chunks of the catch-up in progress
    unsigned long long t_kind[3];    // nanoseconds
    int32_t n_kind[3];
    // --- sampling: inv_temp > 0 draws tokens by the Gumbel-max rule with this seed (0: greedy) ---
    float inv_temp;
    unsigned long long sample_seed;
    // --- top-p: 0 < top_p < 1 restricts every draw to the nucleus; tau is the nucleus' lowest logit of the pass at hand ---
    float top_p, tau;
};

// Standard Gumbel variate number (step, i) of the stream `seed`: u = (k + 0.5) * 2^-23 with k the top 23 bits of
// SplitMix64 output number (step * 2^32 + i + 1), g = -ln(-ln u).  argmax_i (z_i / T + g_i) is a draw from
// softmax(z / T) (Gumbel-max rule), so sampling stays an argmax and keeps its lowest-id tie rule.
__device__ __forceinline__ float gumbel_noise(unsigned long long seed, uint32_t step, uint32_t i)
{
    const uint64_t x = splitmix_out(seed + ((((uint64_t)step << 32) | (uint64_t)i) + 1) * kGamma);
    const float u = ((float)(uint32_t)(x >> 41) + 0.5f) * 1.1920928955078125e-07f;   // * 2^-23, exact
    return -logf(-logf(u));
}

// The value a logit competes with: the logit itself (greedy) or logit / T + Gumbel noise; a logit below the nucleus'
// threshold cannot win.
struct SampleRule {
    float inv_temp;
    unsigned long long seed;
    uint32_t step;
    float tau;
    __device__ __forceinline__ float operator()(float z, int i) const
    {
        if (z < tau) return -INFINITY;
        return inv_temp > 0.f ? fmaf(z, inv_temp, gumbel_noise(seed, step, (uint32_t)i)) : z;
    }
};
__device__ __forceinline__ bool top_p_active(const GenState *g) { return g && g->inv_temp > 0.f && g->top_p > 0.f && g->top_p < 1.f; }
__device__ __forceinline__ SampleRule sample_rule(const GenState *g)
{
    SampleRule r{0.f, 0ull, 0u, -INFINITY};
    if (g && g->inv_temp > 0.f) { r.inv_temp = g->inv_temp; r.seed = g->sample_seed; r.step = (uint32_t)g->step; }
    if (top_p_active(g)) r.tau = __ldcg(&g->tau);
    return r;
}

// ---------------------------------------------------------------------------------------------
// Nucleus (top-p) threshold of softmax(logits / T) over ids < limit, by one CTA of 256 threads.
//
// The nucleus is the shortest prefix of the ids ordered by probability whose probabilities sum to at least top_p,
// plus every id that ties with its last member; the function returns that member's logit.  No sort: the logits'
// bit patterns, mapped to unsigned keys that keep their order, are narrowed down in three histogram passes (11, 11
// and 10 key bits); a bin holds the probability mass of its ids as a 64-bit integer (exp(y - max y) in units of
// 2^-32), so the sums do not depend on the order of the additions and every CTA that runs this gets the same cut.
// hist: 2048 64-bit words of shared memory; part: 256 more; sel: 2.
// ---------------------------------------------------------------------------------------------
constexpr int kNucleusBins = 2048;
__device__ __forceinline__ uint32_t nucleus_key(float z)
{
    const uint32_t b = __float_as_uint(z);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float nucleus_unkey(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
// sync: the barrier of the 256 calling threads.
template <class Sync>
__device__ __noinline__ float nucleus_threshold_cta(const float *logits, int limit, float inv_temp, float top_p, unsigned long long *hist,
                                                    unsigned long long *part, unsigned long long *sel, int tid, Sync sync)
{
    constexpr int NT = 256;
    // ---- max of the scaled logits ----
    float ymax = -INFINITY;
    for (int i = tid; i < limit; i += NT) ymax = fmaxf(ymax, __ldcg(logits + i) * inv_temp);
    float *fred = reinterpret_cast<float *>(part);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ymax = fmaxf(ymax, __shfl_xor_sync(0xffffffffu, ymax, o));
    if ((tid & 31) == 0) fred[tid >> 5] = ymax;
    sync();
    ymax = fred[0];
    for (int w = 1; w < NT / 32; ++w) ymax = fmaxf(ymax, fred[w]);
    sync();
    unsigned long long above = 0, target = 0;   // mass of the keys above the prefix found so far; top_p of the total mass
    uint32_t prefix = 0;
    const int shifts[3] = {21, 10, 0}, bits[3] = {11, 11, 10};
    for (int level = 0; level < 3; ++level) {
        const int sh = shifts[level], nb = 1 << bits[level];
        for (int b = tid; b < kNucleusBins; b += NT) hist[b] = 0ull;
        sync();
        for (int i = tid; i < limit; i += NT) {
            const float z = __ldcg(logits + i);
            const uint32_t k = nucleus_key(z);
            if (level > 0 && (k >> (sh + bits[level])) != (prefix >> (sh + bits[level]))) continue;
            const float m = expf(z * inv_temp - ymax);   // in (0, 1]
            atomicAdd(&hist[(k >> sh) & (uint32_t)(nb - 1)], (unsigned long long)(m * 4294967296.f));
        }
        sync();
        // chunk sums: thread t owns bins [8 t, 8 t + 8)
        unsigned long long mine = 0;
        for (int j = 0; j < kNucleusBins / NT; ++j) mine += hist[tid * (kNucleusBins / NT) + j];
        part[tid] = mine;
        sync();
        if (level == 0) {   // the total mass, identical in every thread
            unsigned long long tot = 0;
            for (int t = 0; t < NT; ++t) tot += part[t];
            target = (unsigned long long)__double2ull_ru((double)top_p * (double)tot);
            if (target > tot) target = tot;
            if (target == 0) target = 1;
        }
        // the bin where the mass counted from the top reaches the target: thread t checks its chunk
        unsigned long long suffix = above;
        for (int t = NT - 1; t > tid; --t) suffix += part[t];   // mass above this thread's chunk
        if (suffix < target && target <= suffix + mine) {
            unsigned long long run = suffix;
            for (int j = kNucleusBins / NT - 1; j >= 0; --j) {
                const unsigned long long h = hist[tid * (kNucleusBins / NT) + j];
                if (run + h >= target) {
                    sel[0] = (unsigned long long)(tid * (kNucleusBins / NT) + j);
                    sel[1] = run;
                    break;
                }
                run += h;
            }
        }
        sync();
        prefix |= (uint32_t)sel[0] << sh;
        above = sel[1];
        sync();
    }
    return nucleus_unkey(prefix);
}

// The threshold for a pass whose sampling runs in a kernel of its own (multi-row passes): one CTA of 256 threads
// writes gen->tau when top-p sampling is on, and does nothing otherwise.
__global__ void __launch_bounds__(256) nucleus_kernel(const float *logits, int limit, GenState *gen)
{
    __shared__ unsigned long long hist[kNucleusBins], part[256], sel[2];
    if (!top_p_active(gen)) return;
    const float tau = nucleus_threshold_cta(logits, limit, gen->inv_temp, gen->top_p, hist, part, sel, (int)threadIdx.x, [] { __syncthreads(); });
    if (threadIdx.x == 0) gen->tau = tau;
}

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

struct GenBuffers {
    int32_t *tokens;           // [prompt_len + max_new + 1] whole sequence
    uint8_t *source;           // [max_new]
    int32_t *em_tok, *em_fed, *em_arg;  // [cap_steps]
    uint8_t *em_src;           // [cap_steps]
    int32_t *handoffs;         // [cap_handoffs][3]
    uint8_t *hand_kind;        // [cap_handoffs] 1 reflection/affirmation, 2 verification, 3 excessive reflection
    const int32_t *aux;        // [n_aux] auxiliary sentence of takeover (3)
    const int32_t *force;      // [n_force]
    const uint8_t *cls;        // [vlimit] class bits per token id
    float *trace;              // [trace_n][vlimit] or null
};

// Describe the pass that has to run next: the active model ingests everything it has not cached,
// at most max_chunk tokens at a time; only the last chunk samples a token.
__device__ __forceinline__ void plan_next_pass(GenState *g, StepDesc *desc_small, StepDesc *desc_large)
{
    const int a = g->active;
    const int pending = g->pos - g->kv_len[a];
    const int m = pending > g->max_chunk ? g->max_chunk : pending;
    g->next_model = a;
    g->next_m = m;
    g->next_emit = (m == pending);
    StepDesc *d = a ? desc_large : desc_small;
    d->pos0 = g->kv_len[a];
    d->m = m;
    d->tok_off = g->kv_len[a];
    d->emit = g->next_emit;
}

// The state transition of one emission step (model `active` sampled `greedy`).
__device__ void router_step(GenState *g, const GenBuffers &b, int greedy, StepDesc *desc_small, StepDesc *desc_large,
                            int32_t *status)
{
    const int a = g->active;
    const int t = g->step;
    const int fed = g->pos - g->kv_len[a] + g->ingested;   // the whole catch-up, however it was chunked
    {   // the pass that just ended, by kind: it began at position pos - fed of this model's cache
        const unsigned long long now = global_timer_ns();
        const int k = fed == 1 ? 2 : (g->pos - fed == 0 ? 0 : 1);
        g->t_kind[k] += now - g->t_last + g->t_pending;
        g->n_kind[k]++;
        g->t_pending = 0;
        g->t_last = now;
    }
    g->ingested = 0;
    g->kv_len[a] = g->pos;
    g->bytes_algo += g->wbytes[a] + g->kvb[a] * (int64_t)g->pos;
    int tok = greedy;
    if (t < g->n_force && b.force[t] >= 0) tok = b.force[t];
    if (t < g->cap_steps) {
        b.em_tok[t] = tok;
        b.em_src[t] = (uint8_t)a;
        b.em_fed[t] = fed;
        b.em_arg[t] = greedy;
    } else {
        atomicOr(status, DEV_LOG_FULL);
    }
    g->step = t + 1;
    if ((unsigned)tok >= (unsigned)g->vlimit) { atomicOr(status, DEV_BAD_TOKEN); tok = 0; }
    // Takeovers of Section 3 in token-id form: the token sampled right after a delimiter stands for the sentence.
    const int cls = b.cls[tok];
    const bool after_delim = (b.cls[b.tokens[g->pos - 1]] & kClsDelim) != 0;
    int kind = 0, len = 0;
    if (g->has_large && a == 0 && !g->every_delim && !g->probing && after_delim) {
        // the speculative model opens a sentence: its next probe_len tokens are classified by cue counts
        g->probing = 1;
        g->probe_start = g->pos;
        g->probe_n = g->n_refl = g->n_aff = g->n_ver = 0;
    }
    if (g->probing) {
        g->n_refl += (cls & kClsKeyword) != 0;
        g->n_aff += (cls & kClsAffirm) != 0;
        g->n_ver += (cls & kClsVerify) != 0;
        g->probe_n++;
        if (g->probe_n >= (g->probe_len > 1 ? g->probe_len : 1)) {
            g->probing = 0;
            // affirmation and reflection cues in one sentence: the majority decides, a tie is a reflection
            const bool reflection = g->n_refl > 0 && g->n_refl >= g->n_aff;
            if (reflection && g->neg_threshold >= 0) g->neg_count++;
            if (g->neg_threshold >= 0 && g->neg_count > g->neg_threshold) { kind = 3; len = g->n3; }   // (3) excessive reflection
            else if (g->n_ver > 0) { kind = 2; len = g->n2; }                                           // (2) verification
            else if (g->n_refl + g->n_aff > 0) { kind = 1; len = g->n1; }                               // (1) reflection / affirmation
        }
    }
    auto log_handoff = [&](int seg_start, int catchup, int k) {
        if (g->n_handoffs < g->cap_handoffs) {
            int32_t *h = b.handoffs + 3 * g->n_handoffs;
            h[0] = seg_start;
            h[1] = t;
            h[2] = catchup;
            if (b.hand_kind) b.hand_kind[g->n_handoffs] = (uint8_t)k;
        } else {
            atomicOr(status, DEV_LOG_FULL);
        }
        g->n_handoffs++;
    };
    if (kind) {
        if (g->keep_probe) {
            b.tokens[g->pos] = tok;
            b.source[g->generated] = 0;
            g->pos++;
            g->generated++;
            if (tok == g->eos) g->done = 1;
        } else {
            // the target's segment replaces the whole probe sentence: the output and the speculative model's cached
            // length go back to where the sentence began (the stale cache rows are overwritten by the next catch-up)
            g->generated -= g->pos - g->probe_start;
            g->pos = g->probe_start;
            g->kv_len[0] = g->probe_start;
        }
        if (kind == 3) {   // the auxiliary sentence goes into the output, then the target continues
            for (int i = 0; i < g->n_aux && g->generated < g->max_new && !g->done; ++i) {
                b.tokens[g->pos] = b.aux[i];
                b.source[g->generated] = 2;
                g->pos++;
                g->generated++;
            }
            g->neg_count = 0;
        }
        log_handoff(g->pos, g->pos - g->kv_len[1], kind);
        g->active = 1;
        g->remaining = len;
    } else {
        if (g->has_large && a == 1 && after_delim && (cls & kClsVerify) && g->remaining < g->n2) {
            // (2) applies to the target's own sentences too: from this token on it writes n2 tokens
            log_handoff(g->pos, 0, 2);
            g->remaining = g->n2;
        }
        b.tokens[g->pos] = tok;
        b.source[g->generated] = (uint8_t)a;
        g->pos++;
        g->generated++;
        if (tok == g->eos) g->done = 1;
        if (a == 1 && --g->remaining == 0) g->active = 0;
        if (g->has_large && a == 0 && g->every_delim && (cls & kClsDelim) && !g->done && g->generated < g->max_new) {
            // the speculative model closed a paragraph: the target writes the next n1 tokens
            log_handoff(g->pos, g->pos - g->kv_len[1], 1);
            g->active = 1;
            g->remaining = g->n1;
        }
    }
    if (g->generated >= g->max_new) g->done = 1;
    plan_next_pass(g, desc_small, desc_large);
}

// After a ragged pass (several independent generations advanced together): the greedy token of a sequence's
// last row advances that sequence's state.
__global__ void batch_router_kernel(GenState *gs, const GenBuffers *gb, const int32_t *pass_seq, const int32_t *pass_last,
                                    const int32_t *n_pass_seq, const int32_t *greedy, StepDesc *descs, int32_t *status)
{
    for (int k = threadIdx.x; k < *n_pass_seq; k += blockDim.x) {
        const int i = pass_seq[k];
        router_step(gs + i, gb[i], greedy[pass_last[k]], descs + 2 * i, descs + 2 * i + 1, status);
    }
}

// An ingest-only chunk finished: advance the cached length and plan the next pass.
__global__ void advance_ingest_kernel(GenState *g, StepDesc *desc_small, StepDesc *desc_large)
{
    const int a = g->next_model;
    {
        const unsigned long long now = global_timer_ns();
        g->t_pending += now - g->t_last;
        g->t_last = now;
    }
    g->kv_len[a] += g->next_m;
    g->ingested += g->next_m;
    g->bytes_algo += g->wbytes[a] + g->kvb[a] * (int64_t)g->kv_len[a];
    plan_next_pass(g, desc_small, desc_large);
}

__global__ void plan_first_pass_kernel(GenState *g, StepDesc *desc_small, StepDesc *desc_large)
{
    g->t_last = global_timer_ns();
    plan_next_pass(g, desc_small, desc_large);
}

// Device-side dispatch of the generation loop (one launch per loop iteration of the graph): picks the
// body that runs the planned pass, or ends the loop.  Bodies per model, in this order: decode,
// multi-row passes of at most 32 / 64 / 128 / 256 rows that sample, ingest-only pass of 256 rows.
constexpr int kBodiesPerModel = 6;

__device__ __forceinline__ int pass_body_index(int model, int m, int emit)
{
    int b;
    if (!emit) b = 5;
    else if (m == 1) b = 0;
    else b = m <= 32 ? 1 : m <= 64 ? 2 : m <= 128 ? 3 : 4;
    return model * kBodiesPerModel + b;
}

__global__ void dispatch_kernel(GenState *g, cudaGraphConditionalHandle loop, cudaGraphConditionalHandle body, int32_t *status)
{
    if (!g->done && g->passes >= g->pass_cap) {
        g->done = 1;
        atomicOr(status, DEV_WAIT_EXPIRED);
    }
    if (g->done) {
        cudaGraphSetConditional(loop, 0);
        cudaGraphSetConditional(body, 0x7fffffffu);   // no such body: nothing runs
        return;
    }
    g->passes++;
    const int b = pass_body_index(g->next_model, g->next_m, g->next_emit);
    g->body_runs[b]++;
    cudaGraphSetConditional(loop, 1);
    cudaGraphSetConditional(body, (unsigned)b);
}

// ---- several independent generations advanced together (batched decode passes) ----

constexpr int kBatchMaxCatchups = 256;

// What the host needs to launch the next round of passes; it never contains a token.
struct BatchPlan {
    int32_t n_dec[2];                       // rows of this round's ragged pass of each model
    int32_t n_cu;                           // sequences that need a multi-row pass of their own this round
    int32_t all_done;
    int32_t max_ctx[2];                     // longest context among the rows of each model
    int32_t cu[kBatchMaxCatchups][5];       // sequence, model, rows, first position, samples (1) or only ingests (0)
};

// One thread builds the round.  Every live sequence lacks `pending` tokens on its active model (1 in steady
// decode, more after a handoff or at the start).  Its tokens become consecutive rows of that model's ragged pass
// -- row j sits at position kv_len + j of the sequence's own cache, the last of them is the one that samples --
// as long as the pass has room; sequences that ingest more than one token are placed first so that the single
// rows cannot crowd them out, and one that does not fit waits for the next round.  More pending tokens than a
// pass has rows (a long prompt) go through the sequence's own chunked multi-row passes instead.
// min_target_rows (r >= 0: r rows; r < 0: |r| percent of the sequences still running): the target's pass is skipped this
// round when it would hold fewer rows and the speculative model has work (sequences do not interact, so the
// order in which they advance does not change any result).
// row_* and bdesc: per model [2]; slots: [n_seqs][2]; descs: [n_seqs][2]; row_tok: [2][max_rows];
// pass_seq / pass_last: [2][n_seqs] sequences of each pass and their sampling rows; n_pass_seq: [2].
__global__ void batch_plan_kernel(GenState *gs, const GenBuffers *gb, int n_seqs, const int32_t *slots, StepDesc *descs,
                                  int32_t *row_slot0, int32_t *row_pos0, int32_t *row_slot1, int32_t *row_pos1,
                                  int32_t *row_tok, int32_t *pass_seq, int32_t *pass_last, int32_t *n_pass_seq, StepDesc *bdesc,
                                  int max_rows, int min_target_rows, BatchPlan *plan)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    int n_rows[2] = {0, 0}, n_in[2] = {0, 0}, n_cu = 0, live = 0, max_ctx[2] = {1, 1};
    for (int round = 0; round < 2; ++round) {   // 0: sequences with several pending tokens, 1: with one
        for (int i = 0; i < n_seqs; ++i) {
            GenState *g = gs + i;
            if (g->done) continue;
            const int a = g->active;
            const int pending = g->pos - g->kv_len[a];
            if ((pending > 1) != (round == 0)) continue;
            ++live;
            if (pending > max_rows) {
                if (n_cu < kBatchMaxCatchups) {
                    plan_next_pass(g, descs + 2 * i, descs + 2 * i + 1);
                    int32_t *c = plan->cu[n_cu++];
                    c[0] = i;
                    c[1] = a;
                    c[2] = g->next_m;
                    c[3] = g->kv_len[a];
                    c[4] = g->next_emit;
                }
                continue;
            }
            if (pending < 1 || n_rows[a] + pending > max_rows) continue;   // no room this round
            const int r0 = n_rows[a];
            int32_t *rs = a ? row_slot1 : row_slot0, *rp = a ? row_pos1 : row_pos0;
            for (int j = 0; j < pending; ++j) {
                rs[r0 + j] = slots[2 * i + a];
                rp[r0 + j] = g->kv_len[a] + j;
                row_tok[a * max_rows + r0 + j] = gb[i].tokens[g->kv_len[a] + j];
            }
            n_rows[a] += pending;
            pass_seq[a * n_seqs + n_in[a]] = i;
            pass_last[a * n_seqs + n_in[a]] = r0 + pending - 1;
            ++n_in[a];
            if (g->pos > max_ctx[a]) max_ctx[a] = g->pos;
        }
    }
    // A pass of the target costs several passes of the speculative model whatever its row count: while the
    // speculative model has rows and the target only a few, the target's sequences wait and their rows accumulate.
    if (min_target_rows < 0) min_target_rows = live * -min_target_rows / 100;   // a share of the sequences still running
    if (n_rows[1] > 0 && n_rows[1] < min_target_rows && n_rows[0] > 0) n_rows[1] = n_in[1] = 0;
    for (int a = 0; a < 2; ++a) {
        bdesc[a].pos0 = 0;
        bdesc[a].m = n_rows[a];
        bdesc[a].tok_off = 0;
        bdesc[a].emit = 1;
        n_pass_seq[a] = n_in[a];
        plan->n_dec[a] = n_rows[a];
        plan->max_ctx[a] = max_ctx[a];
    }
    plan->n_cu = n_cu;
    plan->all_done = live == 0;
}

// ---- greedy speculative decoding (the paper's comparison system): draft bookkeeping and the acceptance rule ----

struct SpecDecState {
    int32_t pos, generated;     // next position to write; tokens written after the prompt
    int32_t k_draft;            // drafts made so far (index into the draft forcing array and logs)
    int32_t g;                  // drafts of the round in progress
    int32_t n_rounds, n_drafted, n_accepted;
    int32_t last_accepted;      // accepted drafts of the round just closed (what the host reads back)
    int32_t done;
    int32_t eos, max_new, vlimit, n_force_draft, n_force_target, cap_rounds, cap_drafts, prompt_len;
};

struct SpecDecBuffers {
    int32_t *tokens;            // [prompt_len + max_new + gamma + 2] whole sequence, drafts written provisionally
    uint8_t *source;            // [max_new + 1] 0 = accepted draft, 1 = written by the target
    int32_t *round_drafted, *round_accepted;   // [cap_rounds]
    int32_t *draft_tok, *draft_arg;            // [cap_drafts] every draft (after forcing) and the greedy choice behind it
    int32_t *choice_arg;                       // [max_new + 1] the target's greedy choice for each generated position it decided
    const int32_t *force_draft, *force_target;
};

// The speculative model sampled draft i of the round: apply the forcing array, log, and place the draft at
// position pos + i, where the next pass of either model reads it.
__global__ void specdec_take_draft_kernel(SpecDecState *s, SpecDecBuffers b, const int32_t *greedy, int i, int32_t *status)
{
    const int k = s->k_draft;
    int d = *greedy;
    if (k < s->n_force_draft && b.force_draft[k] >= 0) d = b.force_draft[k];
    if ((unsigned)d >= (unsigned)s->vlimit) { atomicOr(status, DEV_BAD_TOKEN); d = 0; }
    if (k < s->cap_drafts) {
        b.draft_tok[k] = d;
        b.draft_arg[k] = *greedy;
    }
    b.tokens[s->pos + i] = d;
    s->k_draft = k + 1;
}

// The target scored the round: choices[j] is its greedy token for position pos + j (j <= g).  Keep the longest
// prefix of drafts it would have written itself, then its own token; an end-of-sequence id ends the output.
__global__ void specdec_accept_kernel(SpecDecState *s, SpecDecBuffers b, const int32_t *choices, int32_t *status)
{
    const int g = s->g, pos = s->pos;
    int n = 0, choice = 0;
    for (;;) {
        const int raw = choices[n];
        choice = raw;
        const int gi = s->generated + n;
        if (gi < s->n_force_target && b.force_target[gi] >= 0) choice = b.force_target[gi];
        if ((unsigned)choice >= (unsigned)s->vlimit) { atomicOr(status, DEV_BAD_TOKEN); choice = 0; }
        if (gi <= s->max_new) b.choice_arg[gi] = raw;
        if (n < g && b.tokens[pos + n] == choice) ++n; else break;
    }
    if (s->n_rounds < s->cap_rounds) {
        b.round_drafted[s->n_rounds] = g;
        b.round_accepted[s->n_rounds] = n;
    } else {
        atomicOr(status, DEV_LOG_FULL);
    }
    s->n_rounds++;
    s->n_drafted += g;
    s->n_accepted += n;
    int written = 0;
    for (int i = 0; i <= n && !s->done; ++i) {
        const int tok = i < n ? b.tokens[pos + i] : choice;
        b.tokens[pos + i] = tok;
        b.source[s->generated] = (uint8_t)(i < n ? 0 : 1);
        s->generated++;
        ++written;
        if (tok == s->eos) s->done = 1;
    }
    s->pos = pos + written;
    s->last_accepted = n;
    if (s->generated >= s->max_new) s->done = 1;
}

struct ArgmaxParams {
    const float *logits;   // [vocab]
    int32_t limit;         // ids < limit compete
    float *part_val;       // [gridDim.x]
    int32_t *part_idx;     // [gridDim.x]
    int32_t *ticket;       // zero between launches
    int32_t *argmax_out;   // nullable: plain decode result
    // generation (all null for plain decode)
    GenState *gen;
    GenBuffers buf;
    StepDesc *desc_small, *desc_large;
    int32_t *status;
};

__device__ __forceinline__ void argmax_merge(float &v, int &i, float v2, int i2)
{
    if (v2 > v || (v2 == v && i2 < i)) { v = v2; i = i2; }
}

// Batched decode: lowest-id argmax of every row of logits [rows][vocab] over ids < limit, one CTA per row.
__global__ void __launch_bounds__(1024) argmax_rows_kernel(const StepDesc *desc, const float *logits, int vocab, int limit, int32_t *argmax_out)
{
    __shared__ float s_v[32];
    __shared__ int s_i[32];
    const int row = blockIdx.x;
    if (row >= desc->m) return;
    const float *z = logits + (size_t)row * vocab;
    float v = -INFINITY;
    int idx = 0x7fffffff;
    // 16-byte loads where the rows are 16-byte aligned, four in flight per thread; the ragged end one by one
    const int lim4 = (vocab & 3) == 0 ? limit >> 2 : 0;
    const float4 *z4 = reinterpret_cast<const float4 *>(z);
    for (int i0 = threadIdx.x; i0 < lim4; i0 += 4 * blockDim.x) {
        float4 w[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (i0 + u * (int)blockDim.x < lim4) w[u] = __ldcg(z4 + i0 + u * blockDim.x);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * (int)blockDim.x;
            if (i < lim4) {
                argmax_merge(v, idx, w[u].x, 4 * i);
                argmax_merge(v, idx, w[u].y, 4 * i + 1);
                argmax_merge(v, idx, w[u].z, 4 * i + 2);
                argmax_merge(v, idx, w[u].w, 4 * i + 3);
            }
        }
    }
    for (int i = 4 * lim4 + threadIdx.x; i < limit; i += blockDim.x) argmax_merge(v, idx, __ldcg(z + i), i);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float v2 = __shfl_xor_sync(0xffffffffu, v, o);
        const int i2 = __shfl_xor_sync(0xffffffffu, idx, o);
        argmax_merge(v, idx, v2, i2);
    }
    if ((threadIdx.x & 31) == 0) { s_v[threadIdx.x >> 5] = v; s_i[threadIdx.x >> 5] = idx; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) argmax_merge(v, idx, s_v[w], s_i[w]);
        argmax_out[row] = idx == 0x7fffffff ? 0 : idx;
    }
}

__global__ void __launch_bounds__(256) argmax_router_kernel(const ArgmaxParams p)
{
    __shared__ float s_v[8];
    __shared__ int s_i[8];
    __shared__ int s_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // optional logits trace of this emission step (the step counter only changes after every CTA
    // has taken its ticket, i.e. after all of them have read it here)
    float *trace = nullptr;
    if (p.gen && p.buf.trace && p.gen->trace_n > 0) {
        const int t = p.gen->step - p.gen->trace_first;
        if (t >= 0 && t < p.gen->trace_n) trace = p.buf.trace + (size_t)t * p.limit;
    }
    float v = -INFINITY;
    int idx = 0x7fffffff;
    const SampleRule rule = sample_rule(p.gen);
    for (int i = blockIdx.x * 256 + tid; i < p.limit; i += gridDim.x * 256) {
        const float z = p.logits[i];
        if (trace) trace[i] = z;
        argmax_merge(v, idx, rule(z, i), i);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float v2 = __shfl_xor_sync(0xffffffffu, v, o);
        const int i2 = __shfl_xor_sync(0xffffffffu, idx, o);
        argmax_merge(v, idx, v2, i2);
    }
    if (lane == 0) { s_v[warp] = v; s_i[warp] = idx; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < 8; ++w) argmax_merge(v, idx, s_v[w], s_i[w]);
        p.part_val[blockIdx.x] = v;
        p.part_idx[blockIdx.x] = idx;
        __threadfence();
        const int t = atomicAdd(p.ticket, 1);
        s_last = (t == (int)gridDim.x - 1);
        if (s_last) *p.ticket = 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    v = -INFINITY;
    idx = 0x7fffffff;
    for (int i = tid; i < (int)gridDim.x; i += 256) argmax_merge(v, idx, __ldcg(&p.part_val[i]), __ldcg(&p.part_idx[i]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float v2 = __shfl_xor_sync(0xffffffffu, v, o);
        const int i2 = __shfl_xor_sync(0xffffffffu, idx, o);
        argmax_merge(v, idx, v2, i2);
    }
    __syncthreads();
    if (lane == 0) { s_v[warp] = v; s_i[warp] = idx; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < 8; ++w) argmax_merge(v, idx, s_v[w], s_i[w]);
        if (idx == 0x7fffffff) idx = 0;   // nothing comparable: fall back to id 0
        if (p.argmax_out) *p.argmax_out = idx;
        if (p.gen) router_step(p.gen, p.buf, idx, p.desc_small, p.desc_large, p.status);
    }
}

}  // namespace st
