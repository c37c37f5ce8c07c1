/*
 * lacache.h -- C ABI of the B200 (sm_100a) first-layer cached attention path.
 *
 * The path is the first-layer bidirectional attention of a block-wise
 * (semi-autoregressive) diffusion-LLM denoising step with the paper's
 * RoPECache (Sec. 3.3.2, Eq. 1) and FACache (Sec. 3.3.3, Eq. 2-6,
 * Algorithm 1).  Within one block only the tokens of the current block C
 * change; all other tokens U (prompt, earlier blocks, masked suffix) are fixed
 * (Sec. 3.3.1).  `lacache_build` is the cache-filling side of Algorithm 1
 * (GenStep = True): it rotates and stores Q/K/V for every token and stores, for
 * every fixed query, the online-softmax state (m, l, O~) over the fixed keys.
 * `lacache_step` is the reuse pass (GenStep = False): only the block's fresh
 * Q/K/V are rotated, fixed queries attend to the block's keys only and merge
 * the result into their cached state, block queries attend to all keys, and
 * the normalised output O = diag(l)^-1 O~ is written for all positions.
 *
 * General conventions
 *   - Every tensor pointer is a DEVICE pointer owned by the caller unless the
 *     name says `host`.  Tensors are contiguous, 16-byte aligned, token-major
 *     and packed over the batch: q [T, Hq, d], k/v [T, Hkv, d], out
 *     [T, Hq, d], lse [T, Hq]; T = sum_b (prompt_lens[b] + gen_len).  Block
 *     tensors are sequence-major: row b * block_len + r is token r of
 *     sequence b's current block.
 *   - Q/K/V element type is `dtype` (bf16 or fp32).  `out` is fp32 or bf16
 *     (`out_dtype`; the `float* out` parameters point to bf16 data then), `lse`
 *     fp32 in natural-log units (L = m + log l, Algorithm 1).  A bf16 `out` adds
 *     its own rounding, up to 2^-8 |o| per element (0.016 for 4 <= |o| < 8): the
 *     stated tolerances are for fp32.
 *   - Query head h reads KV head h / (Hq / Hkv).  Positions are 0-based
 *     inside each sequence.  RoPE pairs feature c with c + d/2 and uses
 *     frequency theta^(-2c/d); V is not rotated.
 *   - Calls validate on the host, enqueue work on `cuda_stream` (a
 *     cudaStream_t passed as void*, NULL = default stream) and return without
 *     synchronising.  They never throw, abort or print.  The context owns all
 *     caches and scratch; caller tensors are neither retained nor freed.
 *   - There is no CPU fallback: without a CUDA device every call that would
 *     compute returns LACACHE_ERR_CUDA.
 *   - A context is not thread-safe; use one per host thread / stream.
 */
#ifndef LACACHE_H_
#define LACACHE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lacache_ctx lacache_ctx;

typedef enum {
  LACACHE_OK = 0,
  LACACHE_ERR_INVALID_ARG = 1, /* NULL / misaligned pointer, index out of range */
  LACACHE_ERR_SHAPE = 2,       /* inconsistent sizes in the config */
  LACACHE_ERR_STATE = 3,       /* step before build, etc. */
  LACACHE_ERR_UNSUPPORTED = 4, /* head_dim / dtype / mode not implemented */
  LACACHE_ERR_OOM = 5,
  LACACHE_ERR_CUDA = 6,        /* a CUDA runtime call failed; see lacache_last_error */
  LACACHE_ERR_TIMEOUT = 7      /* a bounded device-side wait ran out */
} lacache_status;

enum { LACACHE_DTYPE_BF16 = 0, LACACHE_DTYPE_FP32 = 1 };
/* which kernel family runs the attention: AUTO picks tcgen05 for bf16 with
 * head_dim 128 and the fp32 CUDA-core kernels otherwise */
enum { LACACHE_ENGINE_AUTO = 0, LACACHE_ENGINE_SIMT = 1, LACACHE_ENGINE_TCGEN05 = 2 };
/* element type of `out` (lse is always fp32) */
enum { LACACHE_OUT_BF16 = 0, LACACHE_OUT_FP32 = 1 };
/*
 * How the tcgen05 engine carries the rotated Q', K' into the score product (the paper states no
 * precision for its kernel beyond "the model's"; Sec. 3.4 keeps the first layer at model precision):
 *   PLAIN  one bf16 plane per tensor, one tensor-core product per score tile, 128-key tiles.
 *          Holds the tolerance (2e-2 max / 2e-3 mean abs against an fp64 evaluation) when the
 *          scores are small: |scale * q.k| of order 1 or less, e.g. q, k ~ N(0,1)/sqrt(d) as in
 *          the GQA long-context configuration.  The error grows with the score magnitude:
 *          ~2^-9 * |s| per score, so per-head scales of 2 (scores of order 50) miss it (0.06-0.3).
 *   SPLIT  two bf16 planes hi = bf16(x), lo = bf16(x - hi), three products hi.hi + hi.lo + lo.hi
 *          (16 significant bits): needed for the LLaDA-shaped configurations whose per-head scale
 *          reaches 2 and whose keys carry 4x outliers.  Twice the Q'/K' bytes and twice the
 *          tensor-core work of PLAIN.
 *   FP16   one fp16 plane per tensor (the rotated value rounded once to fp16, saturated to the finite
 *          range), one product per score tile, 128-key tiles: PLAIN's cost with three more significant
 *          bits (~2^-12 * |s| per score).  Holds the tolerance at per-head scales of 2 with a factor of
 *          about two in hand on the maximum and four on the mean (measured against the fp64 evaluation
 *          on the LLaDA-shaped configurations, outlier keys included); SPLIT has a factor of twenty.
 *          Rotated values beyond the fp16 range (|x| > 65504) saturate: inputs of that size need SPLIT.
 * The fp32 CUDA-core engine ignores the mode (its operands are fp32).
 */
enum { LACACHE_PRECISION_PLAIN = 0, LACACHE_PRECISION_SPLIT = 1, LACACHE_PRECISION_FP16 = 3 };
/* (2 is reserved: split planes plus split probabilities, which this library does not offer) */
/*
 * What a build caches (Sec. 3.3.3 last paragraph; Algorithm 1's Q_overlap / K_overlap predicates):
 *   TOKEN  the index sets U and C of Sec. 3.3.1 at token granularity: every fixed row keeps a state
 *          over every fixed key; a step adds exactly the block's keys.
 *   TILE   Algorithm 1 as printed: state is cached only for row tiles (128 rows, counted from the
 *          start of the sequence) that do not overlap the block, over key tiles (128 keys) that do
 *          not overlap it; a step treats every row of a tile that overlaps the block as a block row
 *          (all keys) and adds to the fixed rows every key of the tiles that overlap the block.
 *          Same out / lse; less cached, more work per step.  tcgen05 engine only.
 */
enum { LACACHE_GRANULARITY_TOKEN = 0, LACACHE_GRANULARITY_TILE = 1 };

typedef struct {
  int dtype;          /* LACACHE_DTYPE_*: element type of q/k/v inputs */
  int engine;         /* LACACHE_ENGINE_* */
  int n_q_heads;      /* Hq */
  int n_kv_heads;     /* Hkv, divides Hq */
  int head_dim;       /* d: 64 or 128 */
  float rope_theta;
  float softmax_scale;        /* <= 0 means 1/sqrt(head_dim) */
  int batch;                  /* B >= 1 */
  const int32_t* prompt_lens; /* HOST pointer, B entries, each >= 0; copied */
  int gen_len;                /* G > 0, the same for every sequence */
  int block_len;              /* L_b > 0, divides G */
  int sc_tiles_per_chunk;     /* key tiles per block-query work item; 0 = auto */
  int out_dtype;              /* LACACHE_OUT_*.  NOTE: 0 is bf16; fp32 is what the tolerances are stated for */
  int precision_mode;         /* LACACHE_PRECISION_*.  NOTE: 0 is PLAIN; see above which inputs it suits */
  int cache_granularity;      /* LACACHE_GRANULARITY_* */
} lacache_config;

/* Library version, e.g. 100 = 1.0.0.  No paper counterpart. */
int lacache_version(void);

/*
 * Create a context: validates the config, derives the integer metadata
 * (Sec. 3.3.1 index sets U and C per block; per-token sequence id and
 * position), builds the RoPE cos/sin table in double precision (Eq. 1) and
 * allocates every cache: rotated Q/K/V (RoPECache), (m, l, O~) (FACache;
 * RowMaxcache / RowSumcache / Ocache of Algorithm 1) and scratch.  This is the
 * only call that allocates device memory, with three documented exceptions
 * that allocate once, on their first use: the *_host calls (staging),
 * lacache_build_incremental (the prefix state) and lacache_sample_block (a
 * small scratch).  Uses the current CUDA device.  On failure *out is NULL.
 */
lacache_status lacache_create(const lacache_config* cfg, lacache_ctx** out);

/* Frees everything the context owns.  Synchronises the device first. */
lacache_status lacache_destroy(lacache_ctx* ctx);

/*
 * Algorithm 1 with GenStep = True, cache side (Sec. 3.3.2-3.3.3).  Rotates
 * q_pre/k_pre at each token's position and stores them with v_pre in the
 * rotated cache for all T tokens, then for every fixed query i in U stores
 * (m_i, l_i, O~_i) over the fixed keys j in U of the same sequence
 * (Eq. 2-6).  Rows of the current block are rotated too (so the cache is
 * complete) but get no state.  block_idx in [0, gen_len / block_len).
 * q_pre [T,Hq,d], k_pre / v_pre [T,Hkv,d] of `dtype`.
 */
lacache_status lacache_build(lacache_ctx* ctx, int block_idx, const void* q_pre,
                             const void* k_pre, const void* v_pre, void* cuda_stream);

/*
 * Incremental rebuild across blocks (an extension: the paper refills the cache for every block,
 * Sec. 3.3.1 "recomputed once per block"; the result is the state of Eq. 2-6 over the same key
 * set, reached in another order).  Between block b and block b + 1 of a sequence the fixed set
 * changes by U_{b+1} = U_b + C_b - C_{b+1}, and only the rows of C_b change their Q/K/V (their
 * tokens were decoded).  Online softmax (Eq. 2-6) can add keys to a state but not take them out, so
 * the context keeps a second state per token, the *prefix state*: (m, l, O~) over the keys before
 * the current block.  Then
 *   - prefix state of block b + 1 = prefix state of block b, extended by the keys of C_b (rows of
 *     C_b themselves are computed over all keys before block b + 1 from scratch);
 *   - cached state of block b + 1 = that prefix state, extended by the keys after block b + 1.
 * Work per advance is N x (L_b + suffix length) score columns per row instead of N x (N - L_b).
 *
 * lacache_build_incremental: as lacache_build (same arguments, same cached state up to rounding
 * order), and leaves the prefix state of block_idx behind.  Allocates the prefix state (the size of
 * the (m, l, O~) cache) on first use: LACACHE_ERR_OOM if that fails.
 * lacache_build_advance: from the block the context holds (built by lacache_build_incremental or by
 * an earlier advance; LACACHE_ERR_STATE otherwise, or when it is the last block) to the next one.
 * q_fin [B*L_b,Hq,d], k_fin / v_fin [B*L_b,Hkv,d] of `dtype` are the pre-RoPE rows of the FINISHED
 * block (layout of lacache_step's inputs); all other tokens must be unchanged since the build.
 * Afterwards lacache_step serves the next block.  tcgen05 engine only (LACACHE_ERR_UNSUPPORTED
 * otherwise).  Device pointers, 16-byte aligned, borrowed for the duration of the enqueued work.
 */
lacache_status lacache_build_incremental(lacache_ctx* ctx, int block_idx, const void* q_pre,
                                         const void* k_pre, const void* v_pre, void* cuda_stream);
lacache_status lacache_build_advance(lacache_ctx* ctx, const void* q_fin, const void* k_fin,
                                     const void* v_fin, void* cuda_stream);

/*
 * Algorithm 1 with GenStep = False (Sec. 3.3.3, last paragraph).  Rotates the
 * block's fresh q_blk [B*L_b,Hq,d], k_blk / v_blk [B*L_b,Hkv,d] into the
 * block's cache slots; fixed queries start from the cached state, visit only
 * the block's keys and are normalised; block queries visit all keys.  Writes
 * out [T,Hq,d] fp32 for ALL T rows and, if lse != NULL, lse [T,Hq].  The
 * (m, l, O~) cache is read-only here.  Requires a preceding lacache_build for
 * the same block, else LACACHE_ERR_STATE.
 *
 * Stream semantics: the work is enqueued on `cuda_stream`, is ordered after
 * everything enqueued on that stream before it, and is complete, with out / lse
 * fully written, before any later operation of that stream runs: an ordinary
 * stream-ordered call.  q_blk / k_blk / v_blk must stay unchanged until the
 * call's work has completed.
 *
 * Optional overlap of consecutive steps, lacache_set_step_overlap(ctx, 1): two
 * lacache_step calls in a row on one stream then overlap on the device (the
 * second call's kernels are launched programmatically dependent and store
 * nothing before the first call's kernels have completed).  The price is that
 * such a step reads q_blk / k_blk / v_blk EARLY, possibly before the operation
 * enqueued just ahead of it has flushed its writes.  Switch it on only when
 * the three tensors are complete before the PREVIOUS lacache_step of this
 * context is enqueued (precomputed inputs), or are written by work enqueued on
 * another stream and joined by an event; never when they are written by work
 * enqueued on the same stream between two steps (a projection kernel run
 * before every step).  The results are bit-identical either way.
 * lacache_step_tokens runs such a producer itself and orders its own kernels
 * correctly whatever this setting; what it reads early with the overlap on
 * is blk_token_ids / blk_hidden, to which the same rule applies.
 */
lacache_status lacache_step(lacache_ctx* ctx, const void* q_blk, const void* k_blk,
                            const void* v_blk, float* out, float* lse, void* cuda_stream);

/*
 * Sampling-stage truncation (Sec. 3.4, last paragraph; the caption of the figure of one inference
 * step): the float softmax over the vocabulary is evaluated on the rows of the current block only.
 * logits [T, vocab] of `dtype` (LACACHE_DTYPE_BF16 or _FP32; DEVICE, row-major, every token's row
 * present as the model's head writes them) -- only the B*L_b rows of the block the context was last
 * built for (or advanced to) are read.  Per block row, in the order of lacache_step's inputs
 * (sequence-major): token = the most probable vocabulary entry (the lowest id among entries of
 * exactly equal logit), conf = its probability, lse = log sum_v exp(logit_v) (lse may be NULL).
 * conf / token / lse are DEVICE arrays [B*L_b] (fp32, int32, fp32).  A logit of -inf contributes
 * nothing.  fp32 arithmetic.  LACACHE_ERR_STATE before a build.  Allocates a small scratch on first
 * use.  Calls on one context must not overlap on the GPU (they share that scratch).
 */
lacache_status lacache_sample_block(lacache_ctx* ctx, const void* logits, int dtype, int vocab,
                                    float* conf, int32_t* token, float* lse, void* cuda_stream);

/* Overlap of consecutive lacache_step calls on the device (see lacache_step): off (0, the
 * default: plain stream order) or on (non-zero: the caller vouches that a step's inputs are
 * complete before the previous step is enqueued).  No paper counterpart. */
lacache_status lacache_set_step_overlap(lacache_ctx* ctx, int enable);

/*
 * Plain attention for all rows over all keys (the definition in Sec. 3.3.3 /
 * App. B.2 with the caches ignored): the vanilla full forward the method
 * replaces.  Reads pre-RoPE q/k/v [T,...], writes out/lse.  Uses context
 * scratch only; the caches are neither read nor written.
 */
lacache_status lacache_full_recompute(lacache_ctx* ctx, const void* q_pre, const void* k_pre,
                                      const void* v_pre, float* out, float* lse,
                                      void* cuda_stream);

/*
 * Plain attention for ONE sequence (batch 1, all rows x all keys, the same
 * result as lacache_full_recompute on a one-sequence context) for callers that
 * must not allocate device memory.  The paper has no counterpart.
 *
 * Some callers cannot call cudaMalloc at all: code running inside a memory
 * pool or arena that owns the whole device heap, plugins whose host forbids
 * allocation after start-up, and latency-critical sections where an
 * allocation's implicit device synchronisation is not acceptable.  They cannot
 * create a context either (that allocates the caches).  This entry point needs
 * no context and calls no cudaMalloc, cudaFree or other allocating routine:
 * every piece of scratch (rotated q/k/v planes in fp32, RoPE tables, positions,
 * the work list) lives in one fixed array inside the library's device image --
 * about 18 MiB, held by every GPU that loads the library until the process
 * exits.  The caller passes inputs and outputs only.
 *
 *   - q_pre [n_tokens, n_q_heads, head_dim], k_pre / v_pre [n_tokens,
 *     n_kv_heads, head_dim] of `dtype`; out [n_tokens, n_q_heads, head_dim]
 *     fp32; lse [n_tokens, n_q_heads] fp32 or NULL.  Device pointers, 16-byte
 *     aligned.  softmax_scale <= 0 means 1/sqrt(head_dim).
 *   - Limits: n_tokens <= 4096 and n_tokens * (n_q_heads + 2 * n_kv_heads) *
 *     head_dim <= 4 Mi elements.  Anything larger returns LACACHE_ERR_SHAPE
 *     (text in lacache_last_error(NULL)) and launches nothing.
 *   - The first call on each device resolves the array's device address (with
 *     that device current) and sets kernel attributes; make that first call
 *     before starting any stream capture.
 *   - A call whose (n_tokens, head_dim, rope_theta) differ from the previous
 *     call's on that device recomputes the RoPE tables on the host and copies
 *     them (up to 2 MiB, from pageable memory the library owns, so the call
 *     may wait for the stream's earlier work); a call that repeats them copies
 *     nothing and only enqueues its two kernels.
 *   - All calls share the one array.  Nothing in it has to start at zero: each
 *     call overwrites what it reads, and the previous call's contents are
 *     simply left behind.  Two calls that overlap on the GPU (different
 *     streams, or different host threads) race on it: serialise them.
 *   - Runs the fp32 CUDA-core kernels (any dtype).
 */
lacache_status lacache_full_recompute_static(int dtype, int n_tokens, int n_q_heads, int n_kv_heads,
                                             int head_dim, float rope_theta, float softmax_scale,
                                             const void* q_pre, const void* k_pre, const void* v_pre,
                                             float* out, float* lse, void* cuda_stream);

/*
 * Same operations with HOST buffers: inputs are copied host->device on `cuda_stream` and results
 * device->host inside the call (asynchronously when the host memory is pinned).  Staging, a copy
 * stream and four events are allocated on first use.  No paper counterpart.
 *
 * lacache_step_host copies its result to the host on a stream of the context, so that the copy of one
 * step (the larger transfer by far) runs beside the next step's input copy and kernels; two result
 * buffers alternate on the device.  out_host / lse_host of a call are complete
 *   - once the device is synchronised, or
 *   - once `cuda_stream` is synchronised after lacache_join_host(ctx, cuda_stream), which makes that
 *     stream wait for the latest result copy (a later lacache_step_host call joins the copy of the call
 *     before it in the same way, behind its own kernels).
 * The host buffers of a call must stay valid and untouched until then.
 */
lacache_status lacache_build_host(lacache_ctx* ctx, int block_idx, const void* q_pre_host,
                                  const void* k_pre_host, const void* v_pre_host,
                                  void* cuda_stream);
lacache_status lacache_step_host(lacache_ctx* ctx, const void* q_blk_host, const void* k_blk_host,
                                 const void* v_blk_host, float* out_host, float* lse_host,
                                 void* cuda_stream);
lacache_status lacache_join_host(lacache_ctx* ctx, void* cuda_stream);

/*
 * Token-wise producer (Sec. 3.3.2, EmbedCache and RoPECache; Eq. 1): the operators that act on
 * each token alone in front of the first-layer attention.  For a list of tokens it computes
 * H = Embed(x) (or takes H as given), H^ = RMSNorm(H) and the pre-rotation projections
 * H^ W_Q, H^ W_K, H^ W_V; the rotation of Eq. 1 is applied by lacache_build / lacache_step, which
 * consume the result.  With it a denoising step feeds only the current block's token ids (or
 * hidden states): everything token-wise for the fixed tokens stays in the caches.
 *
 * Arithmetic: bf16 weights and activations; the norm is evaluated in fp32 and rounded once to
 * bf16; the projections accumulate in fp32 on the tensor cores and are rounded once to bf16.
 *
 * Config pointers are DEVICE pointers to bf16 data owned by the caller:
 *   embed        [vocab, d_model]; NULL with vocab == 0 when only hidden states will be fed
 *   norm_weight  [d_model]
 *   w_qkv        [(n_q_heads + 2 n_kv_heads) * head_dim, d_model], one row per output feature
 *                (the layout of a torch Linear weight): Q heads, then K heads, then V heads
 * embed and norm_weight are referenced, not copied: keep them alive and unchanged for the life
 * of the handle.  w_qkv is copied at create into the handle, re-laid out in the tile order the
 * projection kernel streams (same size); the caller's copy may be released afterwards, and a
 * later change to it has no effect.
 * d_model is a multiple of 64, at most 8192; head_dim is 128; max_tokens bounds n_tokens of every
 * later call.  Needs an sm_100 device.  A handle is not thread-safe, and its calls share one
 * workspace: enqueue them on one stream at a time (calls on one stream are ordered and may follow
 * each other without synchronising).
 */
typedef struct lacache_qkv lacache_qkv;
typedef struct {
  int vocab;
  int d_model;
  int n_q_heads;
  int n_kv_heads;
  int head_dim;
  float rms_eps;
  int max_tokens;
  const void* embed;
  const void* norm_weight;
  const void* w_qkv;
} lacache_qkv_config;

/* Allocates the handle's scratch (operand rows, stream-K workspace, projected rows for the
 * *_tokens calls) and encodes the TMA descriptors.  The only allocating call of the producer.
 * On failure *out is NULL and lacache_qkv_last_error(NULL) has the text. */
lacache_status lacache_qkv_create(const lacache_qkv_config* cfg, lacache_qkv** out);
/* Synchronises the device, then frees what the handle owns (not the weights). */
lacache_status lacache_qkv_destroy(lacache_qkv* p);

/*
 * Projects n_tokens tokens (0 <= n_tokens <= max_tokens).  Exactly one of token_ids (DEVICE
 * int32 [n_tokens], each in [0, vocab)) and hidden (DEVICE bf16 [n_tokens, d_model]) is non-NULL.
 * Writes bf16 q [n_tokens, Hq, d], k and v [n_tokens, Hkv, d] (pre-rotation) and, if h_out is
 * non-NULL, the embedding rows H [n_tokens, d_model] bf16 (the EmbedCache content).  Enqueues two
 * kernels on `cuda_stream` and returns without synchronising.  A token id outside the table is
 * reported by lacache_qkv_poll_status (LACACHE_ERR_INVALID_ARG); its rows are zero.
 * The result does not depend on how the work was split over the SMs: equal inputs give equal bits.
 */
lacache_status lacache_qkv_project(lacache_qkv* p, const int32_t* token_ids, const void* hidden,
                                   int n_tokens, void* q, void* k, void* v, void* h_out,
                                   void* cuda_stream);

/*
 * lacache_build / lacache_step fed by the producer: the tokens are projected into the handle's
 * scratch and the attention call consumes it on the same stream.  build takes all T tokens
 * (token_ids [T] or hidden [T, d_model], packed like q_pre), step the block's B * L_b tokens
 * (sequence-major like q_blk).  The context must be bf16 with the same heads and head_dim as
 * the producer, and max_tokens must cover the call (else LACACHE_ERR_SHAPE).  Consecutive
 * calls on one stream are ordered.  A step fed this way does not overlap the previous one, except
 * that its norm kernel runs alongside the previous step's attention kernel when the overlap of
 * lacache_set_step_overlap is on: blk_token_ids / blk_hidden are then read early (see lacache_step).
 */
lacache_status lacache_build_tokens(lacache_ctx* ctx, lacache_qkv* p, int block_idx,
                                    const int32_t* token_ids, const void* hidden,
                                    void* cuda_stream);
/*
 * The incremental rebuild (see lacache_build_incremental / lacache_build_advance) fed by tokens:
 * lacache_build_tokens_incremental projects all T tokens like lacache_build_tokens;
 * lacache_build_advance_tokens projects the B*L_b FINAL tokens of the finished block (ids or hidden
 * rows, layout of lacache_step_tokens' inputs) and advances to the next block.  Same errors as the
 * calls they combine.
 */
lacache_status lacache_build_tokens_incremental(lacache_ctx* ctx, lacache_qkv* p, int block_idx,
                                                const int32_t* token_ids, const void* hidden,
                                                void* cuda_stream);
lacache_status lacache_build_advance_tokens(lacache_ctx* ctx, lacache_qkv* p, const int32_t* fin_token_ids,
                                            const void* fin_hidden, void* cuda_stream);

/*
 * The build of the next block, re-projecting only what changed.  Token-wise results depend on the
 * token alone (Sec. 3.3.2), so from one block to the next only the tokens whose ids changed need
 * the embedding, norm and projections again: as a rule the B * L_b tokens of the block just
 * finished, now decoded.  The producer keeps the pre-rotation rows of all T tokens from the last
 * lacache_build_tokens / _update of this (ctx, p) pair; this call projects the n_changed tokens
 * listed in `rows` (DEVICE int32 [n_changed], distinct packed token indices in [0, T)) from
 * token_ids [n_changed] or hidden [n_changed, d_model], stores them at those rows, and runs
 * lacache_build on the complete set.  Tokens not listed must be unchanged since that call.
 * LACACHE_ERR_STATE without such a preceding call (another context's lacache_build_tokens with the
 * same producer in between invalidates it).  A row outside [0, T) is reported by
 * lacache_qkv_poll_status and dropped.  n_changed == 0 just rebuilds.
 * Rows that are not re-projected keep their bits.  A re-projected row can differ in the last bf16
 * place, in a few elements, from what a projection of all T tokens gives for it: the reduction over
 * d_model is split over the SMs differently for a different token count, so the fp32 sums round
 * differently; both are within one unit of the exactly rounded value.
 */
lacache_status lacache_build_tokens_update(lacache_ctx* ctx, lacache_qkv* p, int block_idx,
                                           const int32_t* rows, const int32_t* token_ids,
                                           const void* hidden, int n_changed, void* cuda_stream);
lacache_status lacache_step_tokens(lacache_ctx* ctx, lacache_qkv* p, const int32_t* blk_token_ids,
                                   const void* blk_hidden, float* out, float* lse,
                                   void* cuda_stream);

/*
 * Every device-side wait of the projection kernel is bounded (about 2 s by default): a wait that runs
 * out sets LACACHE_ERR_TIMEOUT and where it gave up in the producer's status word, the kernel's thread
 * blocks unwind (loads in flight have landed long before; no tensor-core product was issued; TMEM is
 * freed) and return, and the handle stays usable.  lacache_qkv_set_wait_limit sets that bound for later
 * launches (microseconds, approximate; 0 = the default).  No paper counterpart.
 *
 * lacache_qkv_project_without_norm is a TEST HOOK for that path: it launches the projection kernel of
 * lacache_qkv_project on `hidden` rows WITHOUT the norm kernel that would publish them, so the kernel's
 * wait for its operand rows runs out.  Set a short limit first (a millisecond or so).  It writes
 * nothing to q / k / v; lacache_qkv_poll_status then returns LACACHE_ERR_TIMEOUT, and later calls on
 * the handle work as usual.
 */
lacache_status lacache_qkv_set_wait_limit(lacache_qkv* p, double microseconds);
lacache_status lacache_qkv_project_without_norm(lacache_qkv* p, const void* hidden, int n_tokens, void* q,
                                                void* k, void* v, void* cuda_stream);

/* Profiling hook like lacache_set_timing_events, around the projection (GEMM) kernel. */
lacache_status lacache_qkv_set_timing_events(lacache_qkv* p, void* ev_start, void* ev_stop);
/* Kernels launched by the last lacache_qkv_project. */
int lacache_qkv_last_launch_count(const lacache_qkv* p);
/* Synchronises the device and reads the producer's status word (bounded waits, token ids). */
lacache_status lacache_qkv_poll_status(lacache_qkv* p);
/* Text of the last error of this handle; with NULL, of the last failed lacache_qkv_create. */
const char* lacache_qkv_last_error(const lacache_qkv* p);

/*
 * Test hooks.  All outputs are device pointers, token-major fp32.
 *   export_state: the cached triple in natural-log units, m [T,Hq], l [T,Hq],
 *     o_acc [T,Hq,d].  The triple is not unique (any reference m gives the same
 *     merged result); compare o_acc / l and m + log l.  Rows of the current
 *     block are unspecified.
 *   export_rope_cache: rotated q [T,Hq,d], rotated k [T,Hkv,d], v [T,Hkv,d] as
 *     stored (the split bf16 planes summed).
 *   export_index_meta (HOST outputs, any may be NULL): per token sequence id,
 *     0-based position, is-current-block flag [T]; kv head of each q head [Hq].
 */
lacache_status lacache_export_state(lacache_ctx* ctx, float* m, float* l, float* o_acc,
                                    void* cuda_stream);
lacache_status lacache_export_rope_cache(lacache_ctx* ctx, float* q_rot, float* k_rot, float* v,
                                         void* cuda_stream);
lacache_status lacache_export_index_meta(lacache_ctx* ctx, int32_t* seq_of_tok_host,
                                         int32_t* pos_of_tok_host, int32_t* is_block_host,
                                         int32_t* kv_head_of_q_head_host);

/*
 * Profiling hook: when both are non-NULL cudaEvent_t handles, every later
 * build / step / full_recompute records `ev_start` right before and `ev_stop`
 * right after its attention kernel launch, on the call's stream, so a caller
 * can time that kernel alone.  Pass NULLs to switch it off.  The caller owns
 * the events.  No paper counterpart.
 */
lacache_status lacache_set_timing_events(lacache_ctx* ctx, void* ev_start, void* ev_stop);

/*
 * Profiling hook for kernels that overlap their neighbours (an event pair around a launch keeps it
 * from overlapping and adds the launch latency): `ring` is a DEVICE array of n_slots pairs of
 * 64-bit words, initialised by the caller to {UINT64_MAX, 0}.  Every later launch of the tcgen05
 * attention kernel (build, step, full recompute) takes the next slot, in launch order starting at
 * slot 0 and wrapping, and folds the GPU's global nanosecond timer into it: word 0 = the earliest
 * entry of any of its CTAs, word 1 = the latest exit.  The caller reads the ring after
 * synchronising.  Pass NULL, 0 to switch it off.  tcgen05 engine only (other launches leave the
 * ring alone).  No paper counterpart.
 */
lacache_status lacache_set_span_ring(lacache_ctx* ctx, uint64_t* ring, int n_slots);

/* Total packed tokens T, and the number of kernels launched by the last
 * build / step / full_recompute call.  No paper counterpart. */
int lacache_total_tokens(const lacache_ctx* ctx);
int lacache_last_launch_count(const lacache_ctx* ctx);
/* which engine the context runs (LACACHE_ENGINE_SIMT or _TCGEN05) */
int lacache_engine(const lacache_ctx* ctx);

/*
 * Synchronises the device and reads the device status word that bounded waits
 * and self-checks write.  Returns LACACHE_OK, LACACHE_ERR_TIMEOUT, or
 * LACACHE_ERR_CUDA; details in lacache_last_error.
 */
lacache_status lacache_poll_status(lacache_ctx* ctx);

/* Human-readable text for the last error of this context ("" if none).  With
 * ctx == NULL, the text of the last failed lacache_create on this thread. */
const char* lacache_last_error(const lacache_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* LACACHE_H_ */
