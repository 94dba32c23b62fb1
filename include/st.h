/*
 * st.h -- C ABI of the Speculative Thinking decode library (libst.so, CUDA, sm_100a).
 *
 * The library runs the hot path of Speculative Thinking (Section 3 of the paper, takeover (1)
 * "Affirmation/Reflection Takeover", hyper-parameters from the appendix "Hyperparameters of
 * Speculative Thinking"): key/value-cached greedy decode of a small "speculative" transformer and a
 * large "target" transformer of the Qwen2 architecture, where the target writes n1 tokens whenever
 * the speculative model samples a reflection keyword right after a delimiter token, and each model
 * ingests the tokens it has not seen (catch-up prefill -- the paper's "prefix" pass, Table
 * "comparison of time") the next time it is asked for a token.
 *
 * Conventions
 *   - Every function returns ST_OK (0) or a negative st_status; nothing throws or aborts.
 *   - "host" pointers are ordinary CPU memory, "dev" pointers are CUDA device memory on the
 *     model's device.  The caller owns every buffer it passes; the library owns weights, KV pages
 *     and scratch, allocated at st_model_create through the allocator in st_config (cudaMalloc when
 *     the callbacks are NULL) and released by st_model_destroy.
 *   - All work is enqueued on the CUDA stream given at creation.  st_generate_spec returns after
 *     the results are in the caller's host buffers; st_prefill / st_decode_step are stream-ordered
 *     and return once the work is enqueued (their host-pointer arguments are consumed before
 *     return).
 *   - Two models used together in st_generate_spec must have been created on the same device and
 *     stream.
 *   - There is no CPU fallback: without a CUDA device every entry point except st_strerror fails.
 */
#ifndef ST_H
#define ST_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ST_OK = 0,
    ST_ERR_ARG = -1,         /* null pointer, size out of range, inconsistent shapes */
    ST_ERR_OOM = -2,         /* device or host allocation failed */
    ST_ERR_KV_FULL = -3,     /* not enough free KV pages / sequence slots */
    ST_ERR_VOCAB = -4,       /* vocab_limit larger than a model's vocabulary, token id out of range */
    ST_ERR_TIMEOUT = -5,     /* a bounded device-side wait expired */
    ST_ERR_UNSUPPORTED = -6, /* shape or option the kernels do not cover */
    ST_ERR_INTERNAL = -7,    /* device status word set, CUDA runtime error */
    ST_ERR_CAPACITY = -8     /* a caller-provided output buffer is too small */
} st_status;

typedef struct st_model st_model; /* opaque: weights, paged KV pool, scratch */

/* Device allocator hooks (e.g. backed by a framework's caching allocator). */
typedef void *(*st_alloc_fn)(uint64_t bytes, void *user);
typedef void (*st_free_fn)(void *ptr, void *user);

/* Architecture of one decoder-only transformer: RMSNorm -> attention (rotary embedding with
 * half-split pairing, grouped-query heads: q head i uses kv head i / (n_q_heads / n_kv_heads)) ->
 * residual -> RMSNorm -> SwiGLU FFN -> residual; final RMSNorm and LM head. */
typedef struct {
    int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab;
    float rope_theta, rms_eps;
    int32_t tie_embeddings; /* LM head shares the embedding matrix */
    int32_t qkv_bias;       /* q/k/v projections carry a bias */
    int32_t max_seqs;       /* sequence slots */
    int32_t max_tokens;     /* total KV capacity in tokens over all slots (rounded up to pages) */
    int32_t page_size;      /* tokens per KV page: 16, 32 or 64 */
    st_alloc_fn alloc;      /* NULL -> cudaMalloc */
    st_free_fn free;        /* NULL -> cudaFree */
    void *alloc_user;
} st_config;

/* Handoff rule parameters (Section 3 (1); appendix "Hyperparameters of Speculative Thinking":
 * n1 = 20).  Keywords and the delimiter are token ids. */
typedef struct {
    int32_t delimiter_id;
    const int32_t *keyword_ids; /* host, n_keywords reflection-keyword ids */
    int32_t n_keywords;
    int32_t n1;             /* tokens the target writes per takeover */
    int32_t keep_probe;     /* 0: the keyword token is dropped and the target writes from its position;
                               1: the keyword stays and the target continues after it */
    int32_t eos_id;         /* -1: none */
    int32_t vocab_limit;    /* tokens are chosen among ids < vocab_limit; 0 = min of the two vocabularies */
    int32_t max_new_tokens;
    /* Variant for a speculative model that emits no reflective cues (Section 4, "Modification for speculative
     * thinking applied to non-reasoning models"); both 0 for the rule above. */
    int32_t takeover_every_delimiter; /* 1: no keyword test -- whenever the speculative model writes the delimiter,
                                         the target writes the next n1 tokens */
    int32_t target_first_n;           /* > 0: the target writes the first target_first_n tokens (paper: 100) */
    /* The other takeovers of Section 3, in token-id form: the token sampled right after a delimiter stands for
     * the sentence that follows it.  All off with empty sets and neg_threshold < 0.  Precedence when several
     * apply to one token: (3), then (2), then (1). */
    const int32_t *affirmation_ids;   /* (1) Affirmation cues: hand over n1 tokens like reflection keywords */
    int32_t n_affirmation;
    const int32_t *verification_ids;  /* (2) Verification cues: sampled after a delimiter by the speculative model -> the
                                         target writes n2 tokens; sampled by the target -> it writes n2 tokens from there */
    int32_t n_verification;
    int32_t n2;                       /* paper: 125; >= 1 when verification_ids is not empty */
    int32_t neg_threshold;            /* (3) Excessive reflection: < 0 off; else, once the speculative model has sampled
                                         more than this many reflection keywords after delimiters (paper: 15), aux_ids
                                         are written into the output (source 2), the target writes n3 tokens and the
                                         count restarts */
    int32_t n3;                       /* paper: 125; >= 1 when neg_threshold >= 0 */
    const int32_t *aux_ids;           /* host, the auxiliary sentence, at most 64 ids */
    int32_t n_aux;
    int32_t probe_len;                /* <= 1: the first token after a delimiter is classified.  k > 1 (paper: n1): the
                                         speculative model writes k tokens after the delimiter, the sentence is classified
                                         by cue counts (affirmation vs reflection: majority, tie = reflection) and on a
                                         takeover the target's segment replaces the whole sentence (keep_probe 0: output
                                         and the speculative model's cached length go back to the sentence's start) or
                                         follows it (keep_probe 1).  Size emission logs for (1 + k) * max_new_tokens steps */
    /* The delimiter as a family of ids (the paper's Table 1 and Appendix B: every token that ends in a blank line
     * closes a paragraph).  n_delimiters == 0: the single delimiter_id above; otherwise delimiter_id is ignored and
     * any of these ids (host array, ids below vocab_limit) counts as the delimiter wherever the rule tests for it. */
    const int32_t *delimiter_ids;
    int32_t n_delimiters;
    /* Sampling.  The paper reports pass@1 and names no sampler; greedy (temperature 0) is the default.  temperature > 0:
     * every token is drawn from softmax(logits / temperature) over ids < vocab_limit by the Gumbel-max rule: the id
     * maximising logit / temperature + g wins, g = -ln(-ln u) a standard Gumbel variate from a counter-based generator
     * (SplitMix64 stream `sample_seed`, output number step * 2^32 + id + 1, u = (top 23 bits + 0.5) * 2^-23), lowest id
     * on ties.  emission_argmax then holds the drawn token.  Not available in st_generate_spec_batch's rounds (the
     * sequences then run one by one). */
    float temperature;
    uint64_t sample_seed;
    /* Top-p (nucleus) sampling, with temperature > 0 only: 0 < top_p < 1 restricts every draw to the nucleus of
     * softmax(logits / temperature) -- the shortest prefix of the ids ordered by probability whose probabilities sum to
     * at least top_p, plus every id tying with its last member -- i.e. draws from the distribution renormalised over
     * it.  0 (or >= 1): no restriction.  The cut is found on the device without a sort (three histogram passes over the
     * logits' bit patterns, probability mass summed as 64-bit integers). */
    float top_p;
} st_spec_params;

typedef struct {
    int32_t seg_start;   /* first position the target writes */
    int32_t step;        /* emission step at which the keyword was sampled */
    int32_t catchup_len; /* tokens the target has to ingest before its first token */
} st_handoff;

/* Results of one generation.  All arrays are caller-allocated host memory; a NULL array with
 * capacity 0 is skipped.  An emission step is one pass of one model that produced one sampled (or
 * forced) token; a dropped keyword still counts as a step. */
typedef struct {
    int32_t *tokens;          /* [cap_tokens] tokens written after the prompt */
    uint8_t *source;          /* [cap_tokens] 0 = speculative model, 1 = target model, 2 = inserted auxiliary token */
    int32_t cap_tokens, n_tokens;
    st_handoff *handoffs;     /* [cap_handoffs] */
    int32_t cap_handoffs, n_handoffs;
    int32_t *emission_tokens; /* [cap_steps] token of every step, dropped ones included */
    uint8_t *emission_source; /* [cap_steps] */
    int32_t *emission_fed;    /* [cap_steps] tokens ingested by the emitting model at that step */
    int32_t *emission_argmax; /* [cap_steps] greedy choice before forcing */
    int32_t cap_steps, n_steps;
    int32_t kv_len_small, kv_len_large;
    float *logits_trace;      /* optional [trace_n_steps][vocab_limit] logits of steps trace_first_step.. */
    int32_t trace_first_step, trace_n_steps;
    double seconds;           /* device time of the generation (CUDA events) */
    int64_t bytes_algorithmic; /* weights + KV bytes the passes had to move (sum over steps) */
    uint8_t *handoff_kinds;   /* optional [cap_handoffs]: which takeover each handoff was (1 reflection / affirmation or
                                 every-delimiter, 2 verification, 3 excessive reflection) */
    /* Device time of the generation by kind of pass (the split of the paper's Table "comparison of time": decode of one
     * token against the "prefix" pass of a handoff), from device timestamps taken at the end of every pass:
     * passes that ingest a model's first tokens (its prompt prefill, for the target inside its first catch-up), other
     * passes of more than one token (catch-up after a handoff), and single-token decode passes.  Zero for
     * st_generate_spec_batch (its passes serve many sequences at once). */
    double t_prompt_prefill_s, t_catchup_s, t_decode_s;
    int32_t n_prompt_prefill, n_catchup, n_decode;   /* passes of each kind (a catch-up cut into chunks counts once) */
} st_spec_result;

/* Create a model with seeded random-init weights: element idx of tensor tid of model `tag` is
 * bf16(0.02 * z), z an Irwin-Hall(12) deviate built from SplitMix64 stream outputs (the N(0, 0.02)
 * initialisation of the workloads; norm gains are 1).  `cuda_stream` is a cudaStream_t (NULL = the
 * legacy default stream).  Blocks until the weights are initialised. */
int st_model_create(const st_config *cfg, uint64_t seed, uint32_t model_tag, void *cuda_stream, st_model **out);
void st_model_destroy(st_model *m);

/* Sequence slots of the paged KV cache.  st_seq_reserve makes sure pages exist for `n_tokens`
 * positions of the slot (ST_ERR_KV_FULL otherwise); prefill/decode reserve what they need themselves. */
int st_seq_alloc(st_model *m, int32_t *slot_out);
int st_seq_free(st_model *m, int32_t slot);
int st_seq_reserve(st_model *m, int32_t slot, int32_t n_tokens);
int st_kv_len(st_model *m, int32_t slot, int32_t *len_out);          /* synchronises the stream */
int st_kv_truncate(st_model *m, int32_t slot, int32_t new_len);      /* drop cached positions >= new_len */

/* Ingest n tokens (host ids) at the slot's next positions -- prompt prefill and catch-up prefill
 * (the paper's "prefix" pass) are the same call.  last_logits_dev (nullable): fp32 [vocab] logits of
 * the last ingested position. */
int st_prefill(st_model *m, int32_t slot, const int32_t *tokens_host, int32_t n, float *last_logits_dev);

/* One KV-cached decode step for `batch` sequences: sequence slots_host[i] ingests tokens_dev[i] at its
 * next position.  logits_dev (nullable): fp32 [batch][vocab]; argmax_dev (nullable): int32 [batch],
 * lowest-id argmax over the whole vocabulary.  batch == 1 runs the single-kernel step; batch >= 2 streams the
 * weights once for all rows (projections and LM head on the tensor cores, attention per sequence over its own
 * pages), in chunks of at most 256 rows; without logits_dev the library keeps the [256][vocab] logits itself
 * (allocated on the first such call). */
int st_decode_step(st_model *m, const int32_t *slots_host, const int32_t *tokens_dev, int32_t batch,
                   float *logits_dev, int32_t *argmax_dev);

/* Speculative Thinking generation at batch 1 (Section 3, takeover (1)).  `large` may be NULL (plain
 * greedy decode of `small`).  prompt: host ids, prompt_len >= 1.  force (nullable): host array,
 * force[t] >= 0 replaces the token sampled at emission step t.  Routing (which model runs next, how
 * much it ingests) is decided on the device from the sampled token; the host never reads a token to
 * choose the next launch. */
int st_generate_spec(st_model *small, st_model *large, const st_spec_params *params,
                     const int32_t *prompt, int32_t prompt_len,
                     const int32_t *force, int32_t n_force, st_spec_result *out);

/* The same for n_seqs independent sequences (the batched workload: ragged prompts, per-sequence token budgets
 * and forcing schedules).  prompts / force are concatenations indexed by prompt_offsets / force_offsets
 * (n_seqs + 1 entries each; force may be NULL); max_new_per_seq (nullable) overrides params->max_new_tokens per
 * sequence; outs[i] receives sequence i's result.  Sequences do not interact, so every outs[i] holds the
 * routing st_generate_spec gives for that sequence alone (its logits differ by rounding: batched rows go
 * through the tensor-core passes).  When both models have a free sequence slot and KV pages for every sequence
 * (st_config.max_seqs >= n_seqs, max_tokens >= the sum of prompt + budget + 1), n_seqs <= 256 and no logits
 * trace is asked for, the sequences advance together in rounds: per round one ragged pass per model whose rows are
 * all the tokens its sequences lack (one per sequence in steady decode, a whole catch-up or prompt of up to 256
 * tokens after a handoff or at the start; each row attends to its own sequence's pages), and chunked passes of
 * its own for a sequence that lacks more than 256; the host reads only the shape of the next round, never a token.  outs[i].seconds is then the
 * time of the whole batch and outs[i].bytes_algorithmic what sequence i would move alone.  Otherwise the
 * sequences run one after the other through st_generate_spec (stops at the first failing one). */
int st_generate_spec_batch(st_model *small, st_model *large, const st_spec_params *params, int32_t n_seqs,
                           const int32_t *prompts, const int32_t *prompt_offsets, const int32_t *max_new_per_seq,
                           const int32_t *force, const int32_t *force_offsets, st_spec_result *outs);

/* Greedy speculative decoding on the same two models: the comparison system of the paper's section "Comparisons
 * between Speculative Decoding and Speculative Thinking" (there with a 7B speculative and the 32B target model, the
 * speculative model drafting 20 tokens per step).  Per round the speculative model drafts `gamma` tokens one by one,
 * the target scores them in ONE multi-row pass, the longest prefix the target would have written itself is kept, and
 * the target's own token follows (its next token when every draft was accepted; acceptance rule of Leviathan et al.
 * 2023 for greedy decoding) -- so the output equals the target's own greedy continuation, and both KV caches are cut
 * back to the accepted length after each round.  Both models must have the token ids below vocab_limit in common.
 * force_draft[k] >= 0 (host, nullable) replaces the k-th draft, counted over all rounds; force_target[i] >= 0 replaces
 * the target's choice for generated position i.  Rounds are host-driven: the host reads back only how far the text
 * advanced, never a token.  All result arrays are caller-allocated host memory (optional ones may be NULL). */
typedef struct {
    int32_t gamma;          /* drafts per round (paper: 20); at most 254 */
    int32_t eos_id;         /* -1: none */
    int32_t vocab_limit;    /* 0 = min of the two vocabularies */
    int32_t max_new_tokens;
} st_specdec_params;

typedef struct {
    int32_t *tokens;         /* [cap_tokens] */
    uint8_t *source;         /* [cap_tokens] 0 = accepted draft, 1 = written by the target */
    int32_t cap_tokens, n_tokens;
    int32_t *round_drafted;  /* [cap_rounds] drafts made in each round */
    int32_t *round_accepted; /* [cap_rounds] drafts kept in each round */
    int32_t cap_rounds, n_rounds;
    int32_t kv_len_small, kv_len_large;
    int32_t n_drafted, n_accepted;
    int32_t *draft_tokens;   /* optional [cap_drafts] every draft, forcing applied */
    int32_t *draft_argmax;   /* optional [cap_drafts] the speculative model's greedy choice behind each draft */
    int32_t cap_drafts;
    int32_t *choice_argmax;  /* optional [cap_tokens] the target's greedy choice (before forcing) for each generated position */
    double seconds;          /* device time (CUDA events) */
    int64_t bytes_algorithmic;
} st_specdec_result;

int st_generate_specdec(st_model *small, st_model *large, const st_specdec_params *params,
                        const int32_t *prompt, int32_t prompt_len,
                        const int32_t *force_draft, int32_t n_force_draft,
                        const int32_t *force_target, int32_t n_force_target, st_specdec_result *out);

/* Fill `out_dev` (bf16 bit patterns, device) with elements idx0.. of seeded tensor `tid`: the
 * generator behind st_model_create, exposed so that it can be compared bit for bit. */
int st_fill_tensor_bf16(uint64_t seed, uint32_t model_tag, uint32_t tid, uint64_t idx0, uint64_t n,
                        uint16_t *out_dev, void *cuda_stream);

/* Bytes of weights one decode step streams, and KV bytes per cached token. */
int64_t st_weight_bytes(const st_model *m);
int64_t st_kv_bytes_per_token(const st_model *m);

/* Measurement aids.  st_kernel_launches: kernels this library has launched in this process.
 * st_time_gemv: average device time (CUDA events on the model's stream, after a warm-up round) of
 * `iters` back-to-back launches of one batch-1 projection kernel, cycling through the layers so that
 * every launch streams different weights: which = 0 QKV, 1 O, 2 gate/up, 3 down, 4 LM head (the
 * weight-streaming matrix-vector products of the decode pass).  Scratch activations are overwritten. */
int64_t st_kernel_launches(void);
int st_time_gemv(st_model *m, int32_t which, int32_t iters, double *seconds_out);

/* Self-test of the bounded device-side waits (the paper has no counterpart; every spin of the kernels -- on an
 * mbarrier, on the decode kernel's grid barrier -- gives up after a fixed number of polls, raises a status bit and
 * lets the kernel run to its end instead of hanging the GPU).  Launches one CTA that waits, with a limit of 1000
 * polls, for something that never happens: which = 0 an mbarrier nobody arms (the waits of the TMA / tensor-core
 * pipelines), which = 1 the decode kernel's grid barrier with no other arrival.  Returns ST_ERR_TIMEOUT when the wait
 * expired and the kernel returned normally (the expected outcome), ST_OK when it did not expire, ST_ERR_INTERNAL
 * when the kernel never reached its end.  The model's status word and barrier state are clean afterwards.
 * Synchronises the model's stream. */
int st_selftest_bounded_wait(st_model *m, int32_t which);

/* How the single-kernel decode step lays out its attention phase (Section 3 names no kernel; this describes the
 * split-KV decode attention of the hot path) when `ctx` tokens are cached: key splits per kv head, the capacity in
 * keys of a CTA's K/V staging area, the most staging chunks any (kv head, split) unit streams through it, and
 * whether the unit that holds the step's own key reaches its last chunk with no cached key left for it.  Host
 * arithmetic only (the same function the kernel evaluates); every output pointer may be NULL.  Tests use it to
 * prove that a case really takes the multi-chunk path. */
int st_decode_geometry(const st_model *m, int32_t ctx, int32_t *n_splits, int32_t *kv_cap, int32_t *max_chunks,
                       int32_t *own_chunk_empty);

/* Greedy sampling that allocates nothing (the paper has no counterpart: this is a service entry point).
 * For callers that must not call cudaMalloc -- code running while another component owns the whole
 * device memory pool, or inside a region where allocation is forbidden or would synchronise the device.
 * Computes the lowest-id argmax of logits_dev[0..n) (fp32, device) into *argmax_out_dev (int32, device),
 * the same selection rule as st_decode_step's argmax_dev, on `cuda_stream`.  Its scratch (partial
 * maxima and a ticket word, 1 KB) is a fixed array inside the library image, present on every GPU
 * that loads the library until the process exits; n may be at most 4,194,304 (1 << 22), larger sizes
 * return ST_ERR_CAPACITY.  The first call on a device looks up the array's device address (no
 * allocation); make that first call outside any stream capture.  `cuda_stream` must be a stream of the device that
 * is current when the call is made (the array's address is looked up for the current device).  All calls share the
 * one array: calls that overlap on the GPU (different streams) race and must be serialised by the caller. */
int st_argmax_static(const float *logits_dev, int32_t n, int32_t *argmax_out_dev, void *cuda_stream);

/* Sticky device status word (0 = clean) and message text. */
int st_last_device_status(st_model *m);
const char *st_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* ST_H */
