/*
 * tandem.h - C boundary of the B200 (sm_100a) Tandem + SPEED greedy decoding library.
 *
 * The library implements the inference loop of "Tandem Transformers for Inference Efficient LLMs"
 * (arXiv 2402.08644): a large decoder M_L that runs in block mode, a per-layer projection FF_Tandem
 * that turns M_L's representations into keys/values of a small decoder M_S, M_S drafting gamma tokens
 * autoregressively over that large-derived context plus its own keys/values, and M_L verifying the
 * drafts (Section 3, Eq. 1 and Eq. 2; Section 3.1).
 *
 * Conventions common to every call
 *  - Plain C types only.  Every pointer argument says whether it is a HOST or a DEVICE pointer.
 *  - Every weight matrix is row-major [out_features][in_features] (y = x W^T), embedding / position
 *    tables are [rows][d_model], the output head is [vocab][d_model].  Matrices and tables are in the
 *    context's dtype (fp32 or bf16); LayerNorm gains and biases are always fp32.
 *  - Model form (the paper leaves it open): pre-LayerNorm blocks with gain and bias, eps 1e-5,
 *    exact GELU, no linear biases, learned absolute position embeddings, untied output head.
 *  - Ownership: the caller owns the weights, the arena and every host buffer.  The library allocates
 *    no device memory: all of its state (both KV caches, workspaces, device-side loop state) lives in
 *    the caller's arena.  Weights and arena must stay valid until tandem_destroy.
 *  - Errors: every call returns a tandem_status; nothing throws or aborts.  Arguments are validated
 *    before any GPU work is launched; on error, out-parameters are left untouched.
 *  - A context is bound to one device and one stream and is not thread-safe.  All GPU work is enqueued
 *    on that stream.
 *  - Greedy decisions: arg-max over fp32 logits, lowest token id on ties.
 *  - bf16 contexts: weights, queries and both KV caches are bf16; everything else between the kernels of a
 *    decode pass (residual stream, normalised rows, attention and GELU outputs) is fp32, and enters each
 *    tensor-core product as the sum of two bf16 numbers.  The prompt pass keeps bf16 activations.
 *  - Two environment variables are read once by tandem_create, for diagnosis only; neither changes a result:
 *    TANDEM_NO_GRAPH (set to anything) launches every kernel of an iteration eagerly instead of replaying a CUDA
 *    graph; TANDEM_NO_PDL orders the kernels by plain stream order instead of programmatic dependent launch.
 */
#ifndef TANDEM_B200_H
#define TANDEM_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define TANDEM_API __attribute__((visibility("default")))
#else
#define TANDEM_API
#endif

typedef struct tandem_ctx tandem_ctx; /* opaque; one per (model pair, device) */

typedef enum {
    TANDEM_OK = 0,
    TANDEM_ERR_INVALID_ARG = 1,     /* null pointer, negative size, unknown enum value */
    TANDEM_ERR_SHAPE = 2,           /* unsupported dims (see tandem_create) */
    TANDEM_ERR_ARENA_TOO_SMALL = 3,
    TANDEM_ERR_CAPACITY = 4,        /* batch > max_batch, or positions would exceed max_seq / max_pos */
    TANDEM_ERR_STATE = 5,           /* call order, e.g. a step before a prefill */
    TANDEM_ERR_CUDA = 6,            /* a CUDA call failed; tandem_last_cuda_error() names it */
    TANDEM_ERR_TIMEOUT = 7,         /* a bounded device-side wait expired */
    TANDEM_ERR_UNIMPLEMENTED = 8
} tandem_status;

enum { TANDEM_DTYPE_FP32 = 0, TANDEM_DTYPE_BF16 = 1 };
enum { TANDEM_FF_LINEAR = 0, TANDEM_FF_MLP = 1 };
/* accept_mode: 0 = compare drafts with M_L's arg-max (Section 3.1); 1 = keep all gamma drafts (equals
 * stand-alone Tandem with the free token, Figure 2); 2 = accept length drawn from a counter-based hash
 * of (mode_seed, sequence, iteration), for tests of ragged accept lengths. */
enum { TANDEM_ACCEPT_NATURAL = 0, TANDEM_ACCEPT_ALL = 1, TANDEM_ACCEPT_HASH = 2,
       /* 3 = a round of stand-alone Tandem without the free token ("Representation Generation Only", Section 3
        * "Inference", Figure 3): M_L reads the pending token and the first gamma-1 drafts as gamma rows and
        * predicts nothing, all gamma drafts are kept, the last one becomes pending.  Needs gamma >= 1; a step
        * result's targets are -1. */
       TANDEM_ACCEPT_REPRESENTATION_ONLY = 3,
       /* 4 = sampled SPEED (Section 3.1 builds on the SPEED / speculative-decoding framework; the paper's latency
        * tables are on sampled responses): draft r is drawn from softmax(logits_S / T_S); it is kept with probability
        * min(1, p(d_r) / q(d_r)) with p = softmax(logits_L / T_L); at the first rejection the token is redrawn from
        * the positive part of p - q; if all drafts are kept one more token is drawn from M_L's next distribution.
        * Temperatures: tandem_set_sampling; mode_seed seeds the counter-based uniform variates, keyed by
        * (seed, sequence, iteration, slot).  A step result's targets then hold, at index accept_len, the token that
        * follows the kept drafts (other entries: M_L's arg-max, for information). */
       TANDEM_ACCEPT_SAMPLE = 4 };
/* variants of tandem_standalone_generate */
enum { TANDEM_STANDALONE_FREE_TOKEN = 0, TANDEM_STANDALONE_REPRESENTATION_ONLY = 1,
       TANDEM_STANDALONE_FREE_TOKEN_FULL_PROMPT = 2 };

#define TANDEM_GAMMA_LIMIT 15 /* largest block length gamma a context can be created for */

typedef struct {
    int32_t n_layers, d_model, n_heads, d_ff, vocab, max_pos;
    int32_t n_kv_heads; /* key/value heads: multi-query (1) or grouped-query attention, which Section 3 allows for
                           either model.  0 = n_heads (multi-head).  Must divide n_heads; query head h reads key/value
                           head h / (n_heads / n_kv_heads); wk and wv are then [n_kv_heads * d_head][d_model] and a
                           cached position holds n_kv_heads * d_head keys (values). */
} tandem_dims;

typedef struct {
    tandem_dims large, small;    /* M_L and M_S; both vocabularies must be equal */
    int32_t ff_tandem_kind;      /* TANDEM_FF_LINEAR (the paper's choice, Section 3) or TANDEM_FF_MLP */
    int32_t ff_tandem_hidden;    /* MLP only: hidden width; 0 = small.d_model */
    const int32_t* layer_map;    /* HOST [small.n_layers]: l(j) of Eq. 2, the number of large layers after
                                    which the residual stream feeds small layer j; 0 = embedding output;
                                    values in [0, large.n_layers] */
    int32_t dtype;               /* TANDEM_DTYPE_* : storage type of weights, activations and KV caches */
    int32_t max_batch;           /* sequences per prefill */
    int32_t max_seq;             /* KV-cache capacity in positions per sequence */
    int32_t gamma_max;           /* largest gamma used with this context, 0..TANDEM_GAMMA_LIMIT */
    int32_t max_prefill_rows;    /* workspace rows for the prompt pass; 0 = max_batch * max_seq */
    int32_t device;              /* CUDA device ordinal */
    void* stream;                /* cudaStream_t to enqueue on; NULL = the legacy default stream */
} tandem_config;

/* DEVICE pointers in this fixed order (n_ptrs must match):
 *   for model in (large, small):  emb[V][d], pos[max_pos][d],
 *       per layer: ln1_g[d], ln1_b[d], wq[d][d], wk[d_kv][d], wv[d_kv][d], wo[d][d], ln2_g[d], ln2_b[d],
 *                  w1[d_ff][d], w2[d][d_ff],
 *       lnf_g[d], lnf_b[d], w_out[V][d]
 *   then per small layer j:  linear: w_t[d_S][d_L]      MLP: w_t1[hidden][d_L], w_t2[d_S][hidden]
 * All pointers 16-byte aligned. */
typedef struct {
    const void* const* ptrs; /* HOST array of DEVICE pointers */
    int32_t n_ptrs;
} tandem_weights;

/* HOST buffers owned by the caller; any member may be NULL (then it is not filled). */
typedef struct {
    int32_t* drafts;      /* [batch][gamma]      the small model's draft tokens d_1..d_gamma */
    int32_t* targets;     /* [batch][gamma+1]    M_L's arg-max for the same positions and the next one */
    int32_t* accept_len;  /* [batch]             number of drafts kept this iteration */
    int32_t* n_committed; /* [batch]             committed tokens (prompt included) after the iteration */
} tandem_step_result;

typedef struct {
    int64_t iterations;   /* draft+verify iterations run by the call */
    int64_t large_runs;   /* M_L passes (one per iteration; the paper's "primary model runs", Table 6) */
    int64_t small_runs;   /* M_S passes (gamma per iteration; "secondary model runs") */
    int64_t emitted;      /* tokens returned over all sequences */
    int64_t accept_hist[TANDEM_GAMMA_LIMIT + 1]; /* iterations of live sequences by accept length */
    int64_t kernel_launches; /* kernels of this library enqueued by the call */
} tandem_stats;

/* Bytes of device memory tandem_create needs for this configuration (KV caches of both models,
 * including the small model's large-derived region; workspaces; loop state). */
TANDEM_API tandem_status tandem_query_arena(const tandem_config* cfg, size_t* bytes /* HOST out */);

/* Builds a context over caller-owned weights and arena (DEVICE, 256-byte aligned, arena_bytes >= the
 * queried size).  Supported shapes: d_model % n_heads == 0; head size 32, 64 or 128; d_model, d_ff and
 * ff_tandem_hidden multiples of 8; max_batch * (gamma_max + 1) <= 256 (up to 64 block rows every weight is
 * read once per pass; beyond that once per group of 64 rows).  Zero-fills the arena's state. */
TANDEM_API tandem_status tandem_create(const tandem_config* cfg, const tandem_weights* weights,
                            void* arena /* DEVICE */, size_t arena_bytes, tandem_ctx** out /* HOST out */);

/* Waits for the context's stream and releases host resources.  Never frees caller memory. */
TANDEM_API tandem_status tandem_destroy(tandem_ctx* ctx);

/* Prompt pass (Section 3 "Inference"; Figure 3): for each sequence b, M_L processes
 * prompt[b][0 .. len_b-2] as a standard causal decoder (Eq. 1) and fills its KV cache; FF_Tandem and the
 * small layers' key/value maps turn x^(l(j)) of those positions into the small model's large-derived
 * keys/values (Eq. 2, first line).  The last prompt token becomes the pending token that M_S starts
 * from.  Resets all per-sequence state.  prompt_ids: HOST, the prompts concatenated; prompt_lens:
 * HOST [batch], each >= 1.  Needs len_b <= max_seq, <= both max_pos, and the total number of processed
 * rows <= max_prefill_rows.  Asynchronous on the context's stream (the host arrays are copied before
 * the call returns). */
TANDEM_API tandem_status tandem_prefill(tandem_ctx* ctx, int32_t batch, const int32_t* prompt_ids,
                             const int32_t* prompt_lens);

/* The same prompt pass for several responses per query ("num-samples" of Section 3.1 and Section 4.2, e.g. 4
 * sampled responses that are ranked afterwards): n_queries prompts, each starting num_samples sequences; query q
 * owns sequences q * num_samples .. (q + 1) * num_samples - 1 of the batch, n_queries * num_samples <= max_batch.
 * M_L reads each prompt ONCE; its keys / values and the small model's large-derived keys / values are then copied
 * to the query's other sequences, which start from the same pending token and diverge through their own random
 * variates (TANDEM_ACCEPT_SAMPLE keys them by sequence).  prompt_ids / prompt_lens as in tandem_prefill, per query.
 * (The copies make the samples ordinary sequences: decode attention reads each sequence's own cache.) */
TANDEM_API tandem_status tandem_prefill_samples(tandem_ctx* ctx, int32_t n_queries, int32_t num_samples,
                                                const int32_t* prompt_ids, const int32_t* prompt_lens);

/* One Tandem + SPEED iteration for every sequence (Section 3.1):
 *   draft   M_S runs gamma times from the pending token; each step attends the large-derived keys/values
 *           of positions M_L has processed plus M_S's own keys/values of the current block (Eq. 2);
 *   verify  M_L processes the pending token and the gamma drafts as one block of gamma+1 rows (Eq. 1 in
 *           block mode), extending its KV cache;
 *   project FF_Tandem writes the small model's keys/values for the block's positions;
 *   accept  per sequence: a = length of the longest prefix of drafts equal to M_L's arg-max; the sequence
 *           gains d_1..d_a and M_L's token for the next position, which becomes pending; both caches
 *           roll back to the kept positions (a length update; no data moves).
 * 0 <= gamma <= gamma_max; accept_mode: TANDEM_ACCEPT_*.  result may be NULL (the call is then asynchronous); filling it waits for
 * the stream.  Fails with TANDEM_ERR_CAPACITY, launching nothing, if a sequence could outgrow max_seq. */
TANDEM_API tandem_status tandem_block_step(tandem_ctx* ctx, int32_t gamma, int32_t accept_mode, uint64_t mode_seed,
                                tandem_step_result* result /* HOST, nullable */);

/* Repeats tandem_block_step until every sequence has max_new_tokens new tokens (surplus tokens of the
 * last iteration are dropped; finished sequences stay frozen).  out_ids: HOST [batch][max_new_tokens];
 * out_lens: HOST [batch] (nullable); stats: HOST, nullable.  Synchronous.  Must follow a prefill; may be
 * called again to continue the same sequences. */
TANDEM_API tandem_status tandem_speculative_generate(tandem_ctx* ctx, int32_t gamma, int32_t max_new_tokens,
                                          int32_t accept_mode, uint64_t mode_seed, int32_t* out_ids,
                                          int32_t* out_lens, tandem_stats* stats);

/* Teacher-forced Tandem forward: Eq. 2 over whole given sequences with block length gamma, as in training (Section 3
 * "Training": the key/value pairs of earlier blocks come from M_L through FF_Tandem, those of the current block from
 * M_S) and in the accuracy / cross-entropy evaluation of Section 4.1.  Blocks of gamma positions are anchored at
 * position 0; the token at position i is M_S's input at i and its logits predict the token at i + 1.
 *   ids: HOST, the sequences concatenated; lens: HOST [batch], each >= 2; max(lens) + gamma <= max_seq and max_pos.
 *   nll:  HOST [sum(lens[b] - 1)], per sequence and position 0 .. len-2 the negative log-likelihood (natural log) of
 *         the true next token under softmax of M_S's logits;  top1: HOST, same shape, M_S's arg-max (nullable).
 * Synchronous.  Replaces the context's sequences (it runs an empty prompt pass and representation-only rounds whose
 * drafts are the given tokens); call tandem_prefill before decoding again. */
TANDEM_API tandem_status tandem_teacher_forced_forward(tandem_ctx* ctx, int32_t gamma, int32_t batch, const int32_t* ids,
                                                       const int32_t* lens, float* nll, int32_t* top1);

/* Temperatures of the two models for accept mode TANDEM_ACCEPT_SAMPLE (both > 0; default 1 and 1).  Applies to the
 * iterations enqueued afterwards; waits for the context's stream when a value changes. */
TANDEM_API tandem_status tandem_set_sampling(tandem_ctx* ctx, float temp_large, float temp_small);

/* Adaptive block length (Section 3.1 "Adaptive Block Length"; Section 4: tau = 0.8; Tables 5-6).  After every
 * draft a router looks at M_S's distribution q = softmax(logits_S) for that draft and decides, per sequence, whether
 * M_S goes on drafting or the drafts made so far are verified.  Features: [entropy of q in nats, the top_k largest
 * probabilities in descending order (lowest id first on ties), M_S's embedding rows of those top_k tokens], length
 * F = 1 + top_k + top_k * d_small.  Router: hidden = relu(w1 x + b1), s = sigmoid(w2 . hidden + b2) = predicted
 * probability that M_L disagrees; drafting continues while 1 - s >= tau and fewer than gamma_max drafts exist.
 *
 * tandem_set_router: w1 [hidden][F], b1 [hidden], w2 [hidden]: DEVICE, fp32, caller-owned, valid until replaced or
 * the context is destroyed; 1 <= top_k <= 8 and F * 4 bytes <= 48 KB (else TANDEM_ERR_SHAPE).  (The paper's router is trained; any weights can be passed.)
 * tandem_adaptive_step: one iteration with the natural (arg-max) comparison.  result arrays are sized by gamma_max
 * ([batch][gamma_max] drafts, [batch][gamma_max+1] targets); entries beyond a sequence's own block are -1.
 * block_len: HOST [batch], drafts each sequence made; confidence: HOST [batch][gamma_max], the router's 1 - s per
 * draft (0 beyond the block); both nullable.  Synchronous: the host reads, after every draft step, how many
 * sequences still draft, launches no further draft step once none does, and sizes M_L's block by the longest block
 * of the batch (rows beyond a sequence's own block are computed and ignored).
 * tandem_adaptive_generate: repeats it until every sequence has max_new_tokens; stats->small_runs counts the draft
 * steps executed, stats->large_runs the verify passes (the two columns of Table 6). */
TANDEM_API tandem_status tandem_set_router(tandem_ctx* ctx, int32_t top_k, int32_t hidden, const void* w1, const void* b1,
                                           const void* w2, float b2, float tau);
TANDEM_API tandem_status tandem_adaptive_step(tandem_ctx* ctx, int32_t gamma_max, tandem_step_result* result,
                                              int32_t* block_len, float* confidence);
TANDEM_API tandem_status tandem_adaptive_generate(tandem_ctx* ctx, int32_t gamma_max, int32_t max_new_tokens,
                                                  int32_t* out_ids, int32_t* out_lens, tandem_stats* stats);

/* Stand-alone Tandem decoding (Section 3 "Inference"; Table 3's latency row): M_S writes the response, M_L only
 * supplies representations (and, with the free token, one token per block); nothing is verified.  Must follow
 * tandem_prefill; same buffers and stop rule as tandem_speculative_generate; 1 <= gamma <= gamma_max.
 *   TANDEM_STANDALONE_FREE_TOKEN              "Representation Generation + Token Prediction" (Figure 2) for the
 *       response blocks after the prompt pass of tandem_prefill (which is Figure 3's): per round M_S appends gamma
 *       tokens, M_L reads the pending token and those gamma tokens and appends its own next token.
 *   TANDEM_STANDALONE_REPRESENTATION_ONLY     "Representation Generation Only" (Figure 3): per round M_S appends
 *       gamma tokens, M_L reads gamma rows (the pending token and the first gamma-1 new ones) without its
 *       output head; the last new token is M_S's next input.
 *   TANDEM_STANDALONE_FREE_TOKEN_FULL_PROMPT  Figure 2 as drawn: M_L first reads the last prompt token too and
 *       its prediction is the first response token; then rounds as in TANDEM_STANDALONE_FREE_TOKEN.
 * stats->accept_hist counts rounds by the number of M_S tokens kept (gamma; 0 for the leading M_L round). */
TANDEM_API tandem_status tandem_standalone_generate(tandem_ctx* ctx, int32_t gamma, int32_t variant,
                                                    int32_t max_new_tokens, int32_t* out_ids, int32_t* out_lens,
                                                    tandem_stats* stats);

/* Baseline and invariant hook: plain greedy decoding of M_L alone, one token per pass (the output that
 * Tandem + SPEED must reproduce; abstract and Section 3.1).  Same buffers as above.  Leaves the small
 * model's keys/values stale: call tandem_prefill again before the next speculative call. */
TANDEM_API tandem_status tandem_large_greedy_generate(tandem_ctx* ctx, int32_t max_new_tokens, int32_t* out_ids,
                                           int32_t* out_lens, tandem_stats* stats);

/* Test hook: copies internal results of the LAST iteration to the host as fp32 / int32.  Synchronous.
 *   what = 0  large logits      [batch][gamma+1][vocab]              (last verify pass)
 *   what = 1  small logits      [gamma][batch][vocab]                (last draft steps)
 *   what = 2  large hidden      [batch][gamma+1][d_large]            (final residual stream, last verify)
 *   what = 3  large keys        [n][d_kv_large]  for (layer, seq), n = positions M_L has processed
 *   what = 4  large values      same
 *   what = 5  small keys        [n][d_kv_small]  for (layer, seq): the large-derived region
 *   what = 6  small values      same
 *   what = 7  committed counts  int32 [batch]
 * bytes must equal the size of the selected item. */
TANDEM_API tandem_status tandem_debug_read(tandem_ctx* ctx, int32_t what, int32_t layer, int32_t seq,
                                void* host_dst, size_t bytes);

/* Test hook for the give-up path of the bounded device-side waits (bf16 contexts).  Enqueues one thread block of
 * the decode GEMM whose weight loads are withheld and whose waits give up after 1024 polls instead of 2^22: its
 * wait for operands runs out, it records the code in the context's error word, frees its tensor memory and
 * returns like any other kernel (nothing faults, nothing is left in flight).  The next tandem_block_step with a
 * result, or the next generate call, then returns TANDEM_ERR_TIMEOUT, leaves the caller's buffers untouched and
 * clears the word; the context stays usable.  The model's state is not touched. */
TANDEM_API tandem_status tandem_debug_expire_wait(tandem_ctx* ctx);

/* Measurement hooks.  tandem_profile_enable(ctx, n > 0) brackets each of the next n kernel launches with a
 * pair of CUDA events on the context's stream (this slows the stream down: never leave it on while timing
 * throughput); n = 0 switches it off.  tandem_profile_read waits for the stream and sums, per kernel class
 * (tandem_profile_class_name(i), i = 0 .. until it returns NULL), the elapsed milliseconds, the launches and
 * the algorithmic work of the recorded launches (bytes for the memory-bound classes, flops for gemm_tiled),
 * then clears the record.  ms, launches, work: HOST [n_classes].  tandem_launch_count: kernels enqueued by
 * the context since tandem_create. */
TANDEM_API tandem_status tandem_profile_enable(tandem_ctx* ctx, int32_t max_launches);
TANDEM_API tandem_status tandem_profile_read(tandem_ctx* ctx, int32_t n_classes, double* ms, int64_t* launches,
                                             double* work);
TANDEM_API const char* tandem_profile_class_name(int32_t cls);
TANDEM_API int64_t tandem_launch_count(tandem_ctx* ctx);

/* Stand-alone kernels of the path (the attention / projection micro-benchmark).
 *
 * tandem_decode_attention: one query per (sequence, head) of the small model attends a mixed context
 * (Eq. 2, second line): `derived_len` positions whose keys/values came from M_L through FF_Tandem,
 * followed by `own_len` positions computed by M_S itself.  All pointers DEVICE, bf16.
 *   q, out           [batch][n_heads][d_head]
 *   k_derived, v_derived  [batch][n_heads][derived_len][d_head]
 *   k_own, v_own     [batch][n_heads][own_len][d_head]
 *   scratch          work space of at least tandem_decode_attention_scratch_bytes(...) bytes (the kernel reads
 *                    every row's sequence and position from two int arrays that the call fills there)
 * d_head in {32, 64, 128}; batch <= 65535.  The context is cut into 128-position chunks by absolute position.
 * A cluster of 1, 2, 4 or 8 CTAs (chosen from batch * n_heads) serves one (sequence, head): CTA r takes every
 * cluster-size-th chunk starting at r, each warp keeps an online-softmax state for its share of the positions,
 * and the states are merged in a fixed order through the cluster's shared memory. */
TANDEM_API size_t tandem_decode_attention_scratch_bytes(int32_t batch, int32_t n_heads, int32_t d_head,
                                             int32_t derived_len, int32_t own_len);
TANDEM_API tandem_status tandem_decode_attention(const void* q, const void* k_derived, const void* v_derived,
                                      const void* k_own, const void* v_own, void* out, void* scratch,
                                      size_t scratch_bytes, int32_t batch, int32_t n_heads, int32_t d_head,
                                      int32_t derived_len, int32_t own_len, void* stream);

/* tandem_decode_attention_static: the same attention for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a packaging variant of the kernel above, not a step of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a host callback or another
 * library's hook, in a process whose memory pool is owned by a framework that hands out no raw buffers,
 * or in a service that must not touch the allocator after start-up because an allocation can block on,
 * or synchronise with, other work on the device.  Such a caller still passes its inputs and its output,
 * but the kernel's work space (the per-row sequence / position arrays) is a buffer built into the library:
 * a file-scope __device__ array of TANDEM_STATIC_SCRATCH_BYTES that every GPU loading the library holds
 * until the process exits.
 *
 * Same arguments, layouts and results as tandem_decode_attention, minus scratch.  Differences:
 *  - Batches whose work space exceeds TANDEM_STATIC_SCRATCH_BYTES (tandem_decode_attention_scratch_bytes
 *    tells; 8 bytes per sequence, so 8192 sequences fit) are refused with TANDEM_ERR_CAPACITY before anything
 *    is launched; tandem_last_cuda_error() then holds a sentence with both sizes.
 *  - The first call on each device looks up the device address of the built-in buffer (with that device
 *    current - make the device that owns the tensors current before calling).  Make that first call before
 *    any stream capture is begun on the device.  Later calls only launch.
 *  - The call itself allocates nothing on host or device and frees nothing.
 *  - All calls on a device share the one buffer, and it keeps whatever the previous call left there.  Each call
 *    rewrites the part it reads, so the caller clears nothing between calls; but two calls that can overlap
 *    on the GPU (different streams, or one stream and a graph) race on it and give wrong results.  Keep calls
 *    to this entry point on one stream, or order them with events. */
#define TANDEM_STATIC_SCRATCH_BYTES (64 * 1024)
TANDEM_API tandem_status tandem_decode_attention_static(const void* q, const void* k_derived, const void* v_derived,
                                                        const void* k_own, const void* v_own, void* out,
                                                        int32_t batch, int32_t n_heads, int32_t d_head,
                                                        int32_t derived_len, int32_t own_len, void* stream);

/* tandem_ff_tandem_project: the linear FF_Tandem of Eq. 2 (first line) followed by the small layer's
 * LayerNorm and key/value maps, written as bf16 keys/values.  All pointers DEVICE, 16-byte aligned.
 *   x [rows][d_large] bf16;  w_t [d_small][d_large] bf16;  ln_g, ln_b [d_small] fp32;
 *   wk, wv [d_small][d_small] bf16;  k_out, v_out [rows][d_small] bf16;
 *   scratch: at least tandem_ff_tandem_project_scratch_bytes(rows, d_small) bytes (the fp32 projection
 *   and its normalised fp32 copy).  rows <= 256; d_large, d_small multiples of 8.
 * The two GEMMs stream their weights on the tensor cores (once up to 64 rows, else once per group of 64 rows)
 * with the key/value write as the second one's epilogue; the LayerNorm is fused into the second one's operand
 * load for up to 8 rows of up to 1024 elements and runs as a kernel of its own otherwise.  Asynchronous; a
 * bounded device-side wait that ran out is reported by tandem_standalone_check. */
TANDEM_API size_t tandem_ff_tandem_project_scratch_bytes(int32_t rows, int32_t d_small);
TANDEM_API tandem_status tandem_ff_tandem_project(const void* x, const void* w_t, const void* ln_g, const void* ln_b,
                                       const void* wk, const void* wv, void* k_out, void* v_out,
                                       void* scratch, size_t scratch_bytes, int32_t rows, int32_t d_large,
                                       int32_t d_small, void* stream);

/* tandem_block_linear: y = x W^T for a block of few token rows, the streaming GEMM behind every projection and
 * feed-forward map of the draft steps and the block pass (Section 3 "Inference": the large model processes the
 * gamma+1 tokens of a block together so that each weight is read once for all of them).  All pointers DEVICE,
 * 16-byte aligned, bf16:  x [rows][in_features];  w [out_features][in_features];  y [rows][out_features].
 * 1 <= rows <= 64; in_features a multiple of 8.  Needs no work space: the K-slices of an output tile are summed
 * through the shared memory of a thread-block cluster.  Asynchronous; see tandem_standalone_check. */
TANDEM_API tandem_status tandem_block_linear(const void* x, const void* w, void* y, int32_t rows, int32_t in_features,
                                             int32_t out_features, void* stream);

/* Waits for `stream` and reports whether a bounded device-side wait ran out in a tandem_ff_tandem_project or
 * tandem_block_linear call on the current device since the last check: TANDEM_ERR_TIMEOUT (the outputs of those
 * calls are then not valid; the record is cleared), else TANDEM_OK. */
TANDEM_API tandem_status tandem_standalone_check(void* stream);

TANDEM_API const char* tandem_status_string(tandem_status s);
/* Name of the last failing CUDA call's error for this thread (valid after TANDEM_ERR_CUDA). */
TANDEM_API const char* tandem_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* TANDEM_B200_H */
