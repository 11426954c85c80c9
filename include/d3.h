/*
 * d3.h -- C ABI of the masked-block denoising path of threshold-based
 * diffusion-LLM decoding on one NVIDIA B200 (sm_100a).
 *
 * The operations follow the paper's statement of the decoding problem:
 *   - a bidirectional transformer predicts every masked position of the
 *     current block at once (Sec. 1; Appendix "Combined with SGLang" (i));
 *   - generation runs block by block, block size fixed (Appendix "More
 *     Implementation Details", inference settings);
 *   - after each forward, tokens whose confidence clears a threshold are
 *     unmasked in parallel (Sec. 2, threshold paragraph) or, in the entropy
 *     variant, tokens whose entropy is below it (Sec. 3.2, first paragraph);
 *   - at least one token is unmasked per forward (Sec. 3.2, Fully-Activated);
 *   - a finished block is cached only after one more forward over its final
 *     tokens (Sec. 3.2, "Completed but Stabilizing"; KV-cache paragraph).
 *
 * Conventions
 *   - C linkage, no exceptions cross the boundary.  Every function returns
 *     D3_OK (0) or a negative D3_ERR_* code; d3_strerror() names it and
 *     d3_last_error() gives a longer per-context message.
 *   - Pointers are marked [host] or [device].  A buffer passed in belongs to
 *     the caller and must stay valid until the context's stream has finished
 *     the call's work; everything the context allocates it frees in
 *     d3_destroy().
 *   - Calls enqueue work on the stream given to d3_create() and return
 *     without waiting, except where stated (d3_generate, d3_load_weights,
 *     d3_get_error_word).
 *   - One context per host thread.  No global state.
 *   - Matrices are row-major [out_features, in_features]; activations are
 *     row-major [rows, features].  Token ids are int32.  Element type is
 *     float (D3_DTYPE_F32) or bfloat16 (D3_DTYPE_BF16) as the config says.
 *   - Visibility: the prompt is segment 0, generation block j is segment j;
 *     a position attends to every position of its own and earlier segments
 *     (no causal mask inside a segment).
 */
#ifndef D3_H_
#define D3_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct d3_ctx d3_ctx;

enum {
  D3_OK = 0,
  D3_ERR_INVALID_ARG = -1,    /* null pointer, non-finite threshold, negative size, ... */
  D3_ERR_SHAPE = -2,          /* sizes exceed the configured maxima or break a divisibility rule */
  D3_ERR_OOM = -3,            /* device allocation failed */
  D3_ERR_CUDA = -4,           /* a CUDA runtime / driver call failed */
  D3_ERR_DEVICE_TIMEOUT = -5, /* a bounded device-side wait gave up (see d3_get_error_word) */
  D3_ERR_STATE = -6,          /* call out of order (e.g. step before prefill / load) */
  D3_ERR_UNSUPPORTED = -7     /* configuration outside what the kernels handle */
};

enum { D3_DTYPE_F32 = 0, D3_DTYPE_BF16 = 1 };
enum { D3_DECIDE_CONFIDENCE = 0, /* commit where max softmax probability > threshold */
       D3_DECIDE_ENTROPY = 1 /* commit where entropy (nats) < threshold */ };
enum { D3_GEMM_AUTO = 0,  /* bf16: tcgen05 tensor-core kernel; f32: SIMT kernel */
       D3_GEMM_SIMT = 1 /* debugging: plain SIMT kernel for every matmul */ };

typedef struct d3_config {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, d_head, d_ffn, vocab;
  int32_t mask_id;      /* excluded from softmax/argmax; fills undecided positions */
  float rope_theta;     /* rotate-half RoPE, angle = position * theta^(-2k/d_head) */
  float rms_eps;        /* RMSNorm: x * rsqrt(mean(x^2) + eps) * gain */
  float logit_scale;    /* logits = scale * (norm(x) . lm_head^T), applied in fp32 */
  int32_t dtype;        /* D3_DTYPE_* : storage type of weights, activations and KV cache */
  int32_t block;        /* block size B (1..128) */
  int32_t max_batch;    /* largest batch any call will use */
  int32_t max_seq;      /* cache slots per sequence: >= longest prompt + generated tokens */
  int32_t max_prefill_rows; /* largest batch * padded prompt length passed to d3_prefill (0: max_batch*max_seq) */
  int32_t decide_mode;  /* D3_DECIDE_* */
  int32_t gemm_impl;    /* D3_GEMM_* */
} d3_config;

/* All pointers [host] or all [device] (see d3_load_weights).  Per-layer arrays have n_layers
 * entries.  Norm gains may be NULL (= all ones).  Shapes: tok_emb, lm_head [vocab, d_model];
 * wq [n_q_heads*d_head, d_model]; wk, wv [n_kv_heads*d_head, d_model]; wo [d_model,
 * n_q_heads*d_head]; w_gate, w_up [d_ffn, d_model]; w_down [d_model, d_ffn]; gains [d_model].
 * On the bfloat16 tensor-core path the gains of each RMSNorm (the paper names no architecture beyond
 * a plain Transformer backbone, appendix on foundation models; the pre-norm layout is that of the
 * model shapes this library is configured with) are multiplied into the columns of the matrix that follows it when the
 * weights are loaded (one extra bfloat16 rounding of those weights), and the row factor
 * rsqrt(mean(x^2) + eps) is applied to the matmul's fp32 accumulator: same function, no separate
 * normalisation kernels (D3_PROF_RMSNORM then stays empty). */
typedef struct d3_weights {
  const void *tok_emb, *lm_head, *final_norm;
  const void *const *attn_norm, *const *wq, *const *wk, *const *wv, *const *wo;
  const void *const *ffn_norm, *const *w_gate, *const *w_up, *const *w_down;
} d3_weights;

typedef struct d3_stats {
  int64_t denoise_forwards;  /* per-sequence denoise forwards, summed over the batch */
  int64_t finalize_forwards; /* per-sequence finalize forwards, summed over the batch */
  int64_t tokens_committed;
  int64_t forced_commits;    /* commits that did not clear the threshold (the >=1 rule) */
  int64_t steps;             /* batched forward passes launched by d3_generate */
  int64_t kernel_launches;   /* kernels of this library launched by the call */
  float prefill_ms, decode_ms; /* not filled by the library unless timing was requested */
} d3_stats;

/* Create a context on the current CUDA device.  cuda_stream is a cudaStream_t (NULL = default
 * stream).  Allocates the KV cache [n_layers][2][max_batch][n_kv_heads][max_seq][d_head] and the
 * activation workspaces.  Errors: INVALID_ARG, UNSUPPORTED (d_head not in {32,64,128}, odd sizes),
 * OOM, CUDA. */
int d3_create(const d3_config *cfg, void *cuda_stream, d3_ctx **out);
void d3_destroy(d3_ctx *ctx);

/* Copy the weights into context-owned device memory, repacked for the kernels (q,k,v rows
 * concatenated with each RoPE pair of a head adjacent; gate/up rows interleaved).  src_is_device: 0 = host pointers,
 * 1 = device pointers.  Synchronises the stream before returning. */
int d3_load_weights(d3_ctx *ctx, const d3_weights *w, int src_is_device);

/* Prefill (KV-cache paragraph of Sec. 3.2): forward over each sequence's prompt alone and store the
 * post-RoPE keys and the values of every layer in cache slots [0, len_i).  prompt_ids: [device]
 * [bs, p_max] right-padded (pad value arbitrary but a valid id); prompt_lens: [device] [bs],
 * 0 <= len_i <= p_max.  Resets the per-sequence prefix length to len_i.  Errors: SHAPE when
 * bs > max_batch or p_max > max_seq or bs*p_max > max_prefill_rows; STATE before d3_load_weights. */
int d3_prefill(d3_ctx *ctx, const int32_t *prompt_ids, const int32_t *prompt_lens, int32_t bs, int32_t p_max);

/* One denoising step (Sec. 2 threshold decoding; Sec. 3.2 at-least-one rule): forward of the bs
 * current blocks against the cached prefixes, softmax statistics over the vocabulary at every row
 * (mask_id excluded), then per sequence commit every masked position with confidence > threshold
 * (or entropy < threshold) and always the most confident masked position (lowest index on ties).
 *   block_ids [device][bs, B] in/out: current ids, masked positions hold mask_id on entry;
 *   mask      [device][bs, B] in/out: 1 = masked;
 *   out_pos, out_ids [device][bs, B]: committed positions (ascending) and their ids, first
 *   out_count[b] entries valid; out_count [device][bs].
 * A block with no masked position commits nothing (count 0) and is left unchanged.  The cache is
 * not modified beyond the scratch slots [prefix, prefix+B).  Errors: INVALID_ARG (NaN threshold,
 * null pointers), SHAPE, STATE (before prefill). */
int d3_denoise_step(d3_ctx *ctx, int32_t *block_ids, uint8_t *mask, float threshold, int32_t bs,
                    int32_t *out_pos, int32_t *out_ids, int32_t *out_count);

/* Finalize (Sec. 3.2 "Completed but Stabilizing", then "store its KV cache"): forward of the fully
 * unmasked blocks without the LM head; their K/V stay in the cache and each prefix length grows
 * by B.  block_ids [device][bs, B].  Errors: SHAPE when a prefix would exceed max_seq. */
int d3_commit_block(d3_ctx *ctx, const int32_t *block_ids, int32_t bs);

/* Whole decoding loop after d3_prefill: gen_len/B blocks per sequence, each starting fully masked;
 * sequences advance independently (a sequence whose block is complete runs its finalize forward
 * while others still denoise).  out_ids [device][bs, gen_len]; commit_step (may be NULL)
 * [device][bs, gen_len]: 1-based step within its block at which each position was committed;
 * host_stats [host] may be NULL.  Waits for the stream.  Errors: SHAPE when gen_len is not a
 * multiple of B or prefix + gen_len > max_seq.
 * While 2 * bs * B <= 64 rows (and the context was created with 2 * max_batch * B <= 64), the finalize
 * forward of a block and the first denoise step of the next block run as one forward of 2B rows per
 * sequence, the finished block unable to see the new one: same results as separate forwards (bit for
 * bit on the fp32 path), one batched forward less per block. */
int d3_generate(d3_ctx *ctx, int32_t gen_len, float threshold, int32_t bs, int32_t *out_ids,
                int32_t *commit_step, d3_stats *host_stats);

/* Multi-block decoding after d3_prefill (Sec. 3.2, "Entropy-Based Multi-Block Parallel Decoding"): up to
 * max_active (1..8) consecutive blocks of a sequence are in flight; every round is one forward over
 * all of them (a block sees the cache, the earlier blocks in flight and itself) followed by the
 * decisions.  A block is opened, fully masked, once the newest block in flight is 10 % unmasked; it
 * commits only what clears the threshold (config decide_mode: confidence > threshold, or entropy <
 * threshold) while its predecessor is less than 95 % unmasked, and at least one token per round
 * afterwards; a block without masks takes part in one more round (cache_delay of them, see
 * d3_set_cache_policy) before its K/V count as cached (blocks enter the cache in order).  States are read from the masks as they stand before a round.
 * max_active = 1 is block-by-block decoding with every finalize forward on its own.
 * out_ids [device][bs, gen_len]; commit_round (may be NULL) [device][bs, gen_len]: 1-based round in
 * which each position was committed.  host_stats (may be NULL): steps = rounds, denoise_forwards =
 * (sequence, block) decisions taken, finalize_forwards = blocks stored in the cache.  Waits for the
 * stream.  Errors: SHAPE when gen_len is not a multiple of B, prefix + gen_len > max_seq, or
 * bs * max_active * B rows exceed the workspaces sized by max_batch. */
int d3_generate_multiblock(d3_ctx *ctx, int32_t gen_len, float threshold, int32_t bs, int32_t max_active,
                           int32_t *out_ids, int32_t *commit_round, d3_stats *host_stats);

/* Commits per decision of the latest d3_generate / d3_generate_multiblock call (the distribution
 * behind tokens per forward, the paper's efficiency measure, Sec. 2 and Sec. 4.1): hist[k], k < n, is
 * the number of (sequence, denoise forward) decisions -- in multi-block decoding (sequence, block,
 * round) decisions -- that committed exactly k tokens.  hist [host][n]; entries beyond the block
 * size are 0.  Waits for the stream. */
int d3_commit_histogram(d3_ctx *ctx, int64_t *hist, int32_t n);

/* Early stopping on the end-of-sequence token (Sec. 3.2, "Early Stopping on EOS Token"): with an id set,
 * d3_generate stops a sequence after the denoise step that commits that id anywhere in its current
 * block.  The block goes out as it stands, undecoded positions (there and in all later blocks) read
 * mask_id, the unfinished block is not added to the cache, and tokens_committed counts what was
 * decoded.  eos_id < 0 switches it off (the default).  INVALID_ARG for ids outside the vocabulary or
 * equal to mask_id.  d3_generate_multiblock stops a sequence after the round that commits the id in any
 * block in flight: all blocks in flight go out as they stand and none of them is added to the cache.
 * d3_early_stops: sequences of the latest generate call that stopped this way. */
int d3_set_eos(d3_ctx *ctx, int32_t eos_id);
int64_t d3_early_stops(d3_ctx *ctx);

/* Temperature sampling (Appendix, inference settings: temperature 0.0 or 0.1).  With temperature T > 0
 * the token of a row is drawn from softmax(l / T) by the Gumbel-max rule: the index of the largest
 * l_v + T * g_v over the vocabulary without the mask token (float32, product and sum rounded
 * separately, lowest index on ties), computed in the LM-head epilogue, logits never stored.  The
 * confidence compared with the threshold is softmax(l) of the drawn token, the entropy that of
 * softmax(l).  Noise: g = -ln(-ln u), u = (top 23 bits of a word + 1/2) * 2^-23; the word for
 * vocabulary index v is word v % 4 of Philox-4x32-10 with counter (v / 4, absolute position of the
 * row, step, sequence index in the batch) and key (low, high half of seed).  step: in d3_generate
 * the 1-based denoise step within the sequence's current block; in d3_denoise_step the number of
 * such calls since the last d3_prefill / d3_commit_block.  T = 0 (default) is greedy decoding.
 * In d3_generate_multiblock the step is the round.  INVALID_ARG for negative or non-finite T. */
int d3_set_sampling(d3_ctx *ctx, float temperature, uint64_t seed);

/* Pseudo-trajectory extraction (Sec. 3.1): a d3_generate run with threshold 1 and no end-of-sequence
 * id unmasks exactly one token per step (no probability exceeds 1, so only the forced commit of the
 * most confident position happens) and decodes the full length; its commit_step output is the
 * trajectory.  d3_trajectory_rank turns commit_step [device][bs, gen_len] (step within the block) into
 * rank [device][bs, gen_len]: the step, counted from 1 over the whole response, at which each position
 * was unmasked (a block's steps follow those of all earlier blocks; positions committed in the same
 * step share a rank).  Asynchronous on the context's stream.  SHAPE when gen_len is not a multiple of B. */
int d3_trajectory_rank(d3_ctx *ctx, const int32_t *commit_step, int32_t bs, int32_t gen_len, int32_t *rank);

/* The noisy training sequence of Sec. 3.1 (displayed equation) for bs responses of n tokens: with
 * positions counted from 1, window start s[b], window length k[b] and m[b] = ceil(k t) for mask ratio
 * t (computed by the caller in integers), out[b, i] = y[b, i] if i <= s, mask_id if i > s + k, and in
 * between y[b, i] if rank[b, i] <= s + m (unmasked in trajectory state T_{s+m}), else mask_id.
 * y, rank, out [device][bs, n]; s, k, m [device][bs].  Asynchronous on the context's stream. */
int d3_noisy_sequence(d3_ctx *ctx, const int32_t *y, const int32_t *rank, const int32_t *s, const int32_t *k,
                      const int32_t *m, int32_t bs, int32_t n, int32_t *out);

/* KV-refresh (Sec. 3.2, "KV-Cache and KV-Refresh Mechanism": previously cached states are recomputed
 * by full forward passes).  One forward over the tokens of the stored prefix of each of the bs
 * sequences (the prompt and every block stored since, as recorded by d3_prefill, d3_commit_block and
 * the generate loops), every position seeing the whole stored prefix; the K/V of positions
 * [0, prefix) are overwritten in place, prefix lengths stay.  Needs bs * (longest stored prefix) rows
 * of workspace (max_prefill_rows at d3_create), else SHAPE.  Waits for the stream once (prefix
 * lengths are read on the host).  After d3_set_state has moved a prefix past what was recorded the
 * recorded ids no longer describe the cache: the caller's business. */
int d3_refresh_cache(d3_ctx *ctx, int32_t bs);

/* Cache policy of the generate loops.  cache_delay (1..16, default 1; the paper's settings: 1-2):
 * rounds of d3_generate_multiblock a complete block takes part in before its K/V count as stored.
 * refresh_every (default 0 = never): d3_generate refreshes a sequence's cache each time the number of
 * its stored blocks reaches a multiple of refresh_every while blocks remain to be decoded (the
 * finalize forward is then never fused with the next block's first step); d3_generate_multiblock
 * refreshes the sequences that are still decoding after every refresh_every-th round.
 * d3_refresh_count: (sequence, refresh) pairs of the latest generate call. */
int d3_set_cache_policy(d3_ctx *ctx, int32_t cache_delay, int32_t refresh_every);
int64_t d3_refresh_count(d3_ctx *ctx);

/* Statistics of the latest denoise forward: conf, entropy [device][bs*B] float, argmax
 * [device][bs*B] int32 (any may be NULL). */
int d3_get_step_stats(d3_ctx *ctx, float *conf, float *entropy, int32_t *argmax, int32_t bs);

/* Parity hooks.  d3_forward_logits runs the same forward as a denoise step but writes the scaled
 * fp32 logits [device][bs*B, vocab] instead of reducing them (mask_id column left as computed).
 * d3_set_tap selects a layer whose residual-stream input and output rows of the next forwards are
 * kept (layer < 0: none); d3_read_tap copies them out as fp32 [rows, d_model].  d3_read_kv copies
 * cache slots [pos0, pos0+n) of one layer and sequence as fp32 [n_kv_heads, n, d_head]. */
int d3_forward_logits(d3_ctx *ctx, const int32_t *block_ids, int32_t bs, float *logits);
/* One round of multi-block decoding without the decisions (Sec. 3.2, multi-block decoding): forward
 * of n_win (1..8) consecutive blocks per sequence, window_ids [device][bs, n_win*B], placed at the
 * sequences' prefixes; block w sees the cache, blocks 0..w-1 of the window and itself.  Writes the
 * softmax statistics of every row, conf / entropy [device][bs*n_win*B] float and argmax
 * [device][bs*n_win*B] int32 (any may be NULL), and leaves the rows' K/V in cache slots
 * [prefix, prefix + n_win*B): advancing the prefix with d3_set_state by k*B afterwards stores the first
 * k blocks exactly as d3_generate_multiblock does after a stabilizing round.  Errors: SHAPE when
 * bs * n_win * B rows exceed the workspaces sized by max_batch, STATE before d3_prefill. */
int d3_denoise_window(d3_ctx *ctx, const int32_t *window_ids, int32_t bs, int32_t n_win, float *conf,
                      float *entropy, int32_t *argmax);
int d3_set_tap(d3_ctx *ctx, int32_t layer);
int d3_read_tap(d3_ctx *ctx, float *resid_in, float *resid_out, int32_t rows);
int d3_read_kv(d3_ctx *ctx, int32_t layer, int32_t seq, int32_t pos0, int32_t n, float *k_out, float *v_out);

/* Per-sequence prefix lengths ([device][bs]).  Setting them rewinds or advances the cache
 * cursor; cache contents are untouched. */
int d3_get_state(d3_ctx *ctx, int32_t *prefix_len, int32_t bs);
int d3_set_state(d3_ctx *ctx, const int32_t *prefix_len, int32_t bs);

/* Single operators through the same kernels the path uses (per-kernel parity tests).
 * d3_op_linear: y = x . w^T.  x [device][m, k], w [device][n, k] in the context dtype;
 *   epilogue 0: y fp32 [m, n];  1: y in context dtype [m, n];  2: y fp32 [m, n] += product
 *   (residual);  3: w holds gate/up rows interleaved (row 2j = gate j, row 2j+1 = up j; n = 2*f), y in
 *   context dtype [m, f] = silu(gate) * up.   splits: number of CTAs the tensor-core kernel deals its
 *   (output tile, K slab) units to (0 = auto: one per SM); any value gives the same result up to the
 *   order of fp32 partial sums.
 * d3_op_lm_head_stats: conf/entropy/argmax [device][m] of scale * x . w^T with mask_id excluded.
 * d3_op_attention: q [device][bs*rows, n_q_heads*d_head]; keys/values are the context's cache of
 *   `layer`; sequence b attends to its slots [0, kv_len[b]); out like q.  kv_len [device][bs].
 * d3_op_unmask: the decision alone on caller-provided statistics. */
int d3_op_linear(d3_ctx *ctx, const void *x, const void *w, void *y, int32_t m, int32_t n, int32_t k,
                 int32_t epilogue, int32_t splits);
/* Tiled weight layout (bfloat16, tensor-core path).  The model's matrices are stored, and streamed by
 * the matmul, as contiguous blocks of 128 rows x 64 columns (16 KB), in the order (row tile, column
 * slab), zero-padded to whole blocks, so that a CTA walking along K reads one contiguous stretch of
 * HBM.  d3_packed_weight_elems: elements of the packed form of an [n, k] matrix (0 on bad sizes).
 * d3_pack_weight: w [device][n, k] row-major -> packed [device][d3_packed_weight_elems(n, k)].
 * d3_op_linear_packed: d3_op_linear with the weights in that form.  Here splits may also be -S: run
 *   the column-strip kernel with strips of S columns (S a multiple of 16, at most 256, dividing n;
 *   m <= 64), D3_ERR_UNSUPPORTED otherwise. */
int64_t d3_packed_weight_elems(int32_t n, int32_t k);
int d3_pack_weight(d3_ctx *ctx, const void *w, int32_t n, int32_t k, void *packed);
int d3_op_linear_packed(d3_ctx *ctx, const void *x, const void *w_packed, void *y, int32_t m, int32_t n, int32_t k,
                        int32_t epilogue, int32_t splits);
int d3_op_lm_head_stats(d3_ctx *ctx, const void *x, const void *w, int32_t m, int32_t vocab, int32_t k,
                        float scale, int32_t mask_id, float *conf, float *entropy, int32_t *argmax);
int d3_op_attention(d3_ctx *ctx, const void *q, int32_t layer, int32_t bs, int32_t rows,
                    const int32_t *kv_len, void *out);
int d3_op_write_kv(d3_ctx *ctx, int32_t layer, int32_t seq, int32_t pos0, int32_t n, const float *k, const float *v);
int d3_op_unmask(d3_ctx *ctx, const float *conf, const float *entropy, const int32_t *argmax,
                 int32_t *block_ids, uint8_t *mask, float threshold, int32_t bs, int32_t *out_pos,
                 int32_t *out_ids, int32_t *out_count);

/* LM-head statistics without any allocation.  (The paper has no counterpart: this entry point exists
 * for the sake of callers, not of the method.)
 *
 * Some callers of this library may not create device memory at the moment they need the
 * statistics: code running between the begin and end of a region in which the allocator is frozen,
 * a plug-in that was handed a fixed memory budget by its host process, or a real-time loop in which
 * a cudaMalloc (which may synchronise the device) is not acceptable.  Those callers cannot use
 * d3_create(), which allocates the cache and the workspaces.  This function needs no context: it
 * computes, for every row of x, the same three numbers as d3_op_lm_head_stats -- confidence = largest
 * softmax probability of scale * (x . w^T) with column mask_id left out, entropy in nats, and the
 * arg max (lowest index on ties) -- and keeps its only intermediate, one partial statistic per
 * (row, 128-column tile of the vocabulary), in an array that is part of the loaded library image.
 *
 *   x [device][m, k], w [device][vocab, k], both of `dtype` (D3_DTYPE_*), row-major;
 *   conf, entropy [device][m] float, argmax [device][m] int32: written by the call;
 *   cuda_stream: a cudaStream_t (NULL = default stream) of the current device; work is enqueued
 *   there and the call returns without waiting.
 *
 * Limits and rules
 *   - m * ceil(vocab / 128) must not exceed D3_STATIC_MAX_PARTIALS (65536 entries, 1 MiB, held by
 *     every GPU that loads the library until the process exits); larger problems return
 *     D3_ERR_SHAPE and nothing is launched.
 *   - The function calls no cudaMalloc / cudaFree and no library routine that allocates.  The first
 *     call on each device looks up the device address of the array (a symbol query, with that
 *     device current); make that first call outside any stream capture.
 *   - All calls on one device share the array.  Two calls whose kernels may overlap on the GPU
 *     (different streams, no ordering between them) race on it: order them on one stream or with
 *     events.  The array keeps what the previous call left; every entry that a call reads it has
 *     written itself first, so nothing needs clearing between calls.
 *   - The matmul inside runs on the plain SIMT kernel of this library for both element types (it is
 *     meant for operator-sized problems, not for streaming a full vocabulary at speed).
 * Errors: INVALID_ARG (null pointer, non-positive size, unknown dtype), SHAPE, CUDA. */
#define D3_STATIC_MAX_PARTIALS 65536
int d3_lm_head_stats_static(const void *x, const void *w, int32_t dtype, int32_t m, int32_t vocab, int32_t k,
                            float scale, int32_t mask_id, float *conf, float *entropy, int32_t *argmax,
                            void *cuda_stream);

/* Kernel overlap.  By default consecutive kernels of a forward are launched with programmatic stream
 * serialization: a kernel may become resident and prefetch its weights while its predecessor drains,
 * and waits (griddepcontrol.wait) before it touches anything the predecessor wrote.  on = 0 launches
 * every kernel fully serialized (for timing kernels in isolation and for debugging); results are
 * identical either way. */
int d3_set_overlap(d3_ctx *ctx, int on);

/* Per-class kernel timing for measurement runs.  While enabled, every launch of the forward pass is
 * bracketed by a CUDA event pair on the context's stream; d3_profile_read waits for the stream and
 * returns, per class, the summed elapsed milliseconds and the number of launches since enabling.
 * ms, launches: [host] arrays of D3_PROF_CLASSES entries.  Off by default (it costs two event
 * records per launch). */
enum { D3_PROF_GEMM_QKV = 0, D3_PROF_GEMM_O = 1, D3_PROF_GEMM_GATE_UP = 2, D3_PROF_GEMM_DOWN = 3,
       D3_PROF_GEMM_HEAD = 4, D3_PROF_GEMM_OTHER = 5, D3_PROF_ATTENTION = 6, D3_PROF_RMSNORM = 7,
       D3_PROF_OTHER = 8, D3_PROF_CHAIN = 9 /* a decode forward's layers as one launch */, D3_PROF_CLASSES = 10 };
int d3_profile_enable(d3_ctx *ctx, int on);
int d3_profile_read(d3_ctx *ctx, double *ms, int64_t *launches);

/* Device error word: 0 when no bounded wait has given up and no kernel saw an invalid index or
 * statistic (bit 0: a wait gave up; 1: token id outside the vocabulary; 2: cache slot outside
 * max_seq; 4: every masked row of a block had a NaN statistic, the lowest one was committed).
 * Synchronises the stream.  Returns D3_OK and writes the word, or D3_ERR_CUDA. */
int d3_get_error_word(d3_ctx *ctx, uint32_t *word);
/* Number of this library's kernels launched on the context since creation. */
int64_t d3_launch_count(d3_ctx *ctx);
/* The same for one kernel, by its name in the source (e.g. "gemm_strip_kernel"); 0 for unknown names. */
int64_t d3_launch_count_of(d3_ctx *ctx, const char *kernel);
/* Bytes of device memory the context holds. */
int64_t d3_device_bytes(d3_ctx *ctx);

const char *d3_strerror(int code);
const char *d3_last_error(d3_ctx *ctx);
const char *d3_version(void);

#ifdef __cplusplus
}
#endif
#endif /* D3_H_ */
