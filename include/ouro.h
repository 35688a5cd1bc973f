/* ouro.h - C ABI of the Ouroboros verification path for one NVIDIA B200 (sm_100a).
 *
 * One decoding step of Ouroboros (arXiv 2402.13720): a small draft model proposes d_1..d_gamma
 * (Eq. 1); up to K phrases that start with d_gamma are taken from a phrase pool and appended, giving
 * K lengthened drafts (Section 3.2, Eq. 7); ONE forward of the target model scores all of them under
 * an attention mask in which every phrase suffix sees the prefix, the draft and itself only (Eq. 8);
 * the longest greedily-correct prefix over the candidates is accepted (Eq. 3, Eq. 9); the KV cache is
 * compacted to the accepted path; phrases are harvested from the verification result (Section 3.3).
 *
 * Conventions
 *  - Every function returns an int status (OURO_OK == 0).  Nothing throws or aborts across this ABI.
 *    Out-parameters are written only on OURO_OK.  ouro_last_error() gives a text for the last failure.
 *  - "dev" pointers are device (CUDA global) memory, "host" pointers are host memory.  Token ids and
 *    all integers exchanged are int32_t.
 *  - Ownership: the caller owns ALL device memory (weights, KV caches, workspace) and lends it for the
 *    context's lifetime.  The library never allocates or frees device memory.  It does allocate a few
 *    KB of pinned host memory in ouro_create and frees it in ouro_destroy.
 *  - All GPU work is enqueued on the cudaStream_t given to ouro_create.  Functions that return host
 *    values synchronise that stream; the others are asynchronous.
 *  - A context is not thread safe.  One context drives one decoding stream (the paper's setting is a
 *    single query, see its Limitations section).
 *  - Block rows (query rows of one forward) are limited to OURO_MAX_ROWS.
 */
#ifndef OURO_H
#define OURO_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  OURO_OK = 0,
  OURO_EINVAL = 1,     /* bad argument (null pointer, shape the kernels do not support, ...) */
  OURO_ENOMEM = 2,     /* workspace too small / host allocation failed */
  OURO_ECAPACITY = 3,  /* cache length + block rows would exceed max_seq, or a row limit is exceeded */
  OURO_ECUDA = 4,      /* a CUDA runtime or driver call failed */
  OURO_ETIMEOUT = 5,   /* a bounded device-side wait gave up (the kernel returned normally) */
  OURO_ESTATE = 6      /* call order violated (e.g. verify before assemble) */
};

enum { OURO_F32 = 0, OURO_BF16 = 1 };
enum { OURO_TARGET = 0, OURO_DRAFT = 1 };
enum { OURO_MAX_ROWS = 128, OURO_MAX_BETA = 16, OURO_MAX_K = 16, OURO_MAX_GAMMA = 32, OURO_MAX_WINDOW = 32 };

/* ouro_params.flags */
enum {
  OURO_HARVEST_MATCHED = 1,     /* Section 3.3, first part: matched sub-segments of the discarded draft */
  OURO_HARVEST_CANDIDATES = 2,  /* Section 3.3, second part: tried phrases replaced by their verified version */
  OURO_HARVEST_ACCEPTED = 4,    /* extension: beta-grams ending inside the newly accepted tokens */
  OURO_SEED_PROMPT = 8,         /* extension: beta-grams of the prompt enter the pool at prefill */
  OURO_DRAFT_PHRASES = 16       /* Section 3.1: the draft model drafts phrase by phrase (see ouro_draft) */
};

typedef struct ouro_ctx ouro_ctx;

/* Llama-style decoder: pre-RMSNorm, rotary positions on half-split pairs, grouped-query attention,
 * SwiGLU FFN, no biases, untied LM head.  (The paper runs such checkpoints through a stock library,
 * Section 4.1; it does not define the network itself.)  head_dim must be a multiple of 32, <= 128. */
typedef struct {
  int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab, max_seq;
  int32_t dtype;              /* OURO_F32 or OURO_BF16: type of weights, KV cache and GEMM inputs */
  float rope_theta, rms_eps;
} ouro_model_desc;

/* All device pointers.  Matrices are row-major [out_features, in_features].  The per-layer arrays are
 * HOST arrays of n_layers device pointers (copied at ouro_create).  k_cache / v_cache are
 * [n_layers, max_seq, n_kv_heads, head_dim]; keys are stored already rotated.  Every pointer must be
 * 16-byte aligned. */
typedef struct {
  const void *embed;        /* [vocab, d_model] */
  const void *final_norm;   /* [d_model] */
  const void *lm_head;      /* [vocab, d_model] */
  const void *const *attn_norm; /* [d_model] */
  const void *const *wq;        /* [n_heads*head_dim, d_model] */
  const void *const *wk;        /* [n_kv_heads*head_dim, d_model] */
  const void *const *wv;        /* [n_kv_heads*head_dim, d_model] */
  const void *const *wo;        /* [d_model, n_heads*head_dim] */
  const void *const *ffn_norm;  /* [d_model] */
  const void *const *w_gate;    /* [d_ffn, d_model] */
  const void *const *w_up;      /* [d_ffn, d_model] */
  const void *const *w_down;    /* [d_model, d_ffn] */
  void *k_cache, *v_cache;      /* [n_layers, max_seq, n_kv_heads, head_dim]; ouro_create clears them (unused rows must be finite) */
} ouro_model_mem;

/* gamma: draft length (Eq. 1).  beta: phrase length INCLUDING its first token p_1 = d_gamma (Section
 * 3.2), so each candidate adds beta-1 rows.  K: candidates per step.  The pool is a pool_sets x
 * pool_ways table (pool_sets a power of two); the paper leaves its structure open. */
typedef struct {
  int32_t gamma, beta, K, pool_sets, pool_ways;
  uint32_t flags;
  int32_t eos_token;          /* < 0: none */
  int32_t window;             /* Section 3.1, phrase generation during drafting: width W of the lookahead window that rides
                                 along every forward of the draft model (see ouro_draft); 0: off.  <= OURO_MAX_WINDOW; not
                                 together with OURO_DRAFT_PHRASES. */
} ouro_params;

typedef struct ouro_stats {
  int32_t n_tokens;           /* tokens generated */
  int32_t target_calls;       /* target forwards; block efficiency = n_tokens / target_calls (Appendix C) */
  int32_t draft_calls;        /* draft forwards */
  int32_t full_accepts;       /* steps with A == gamma (Eq. 3) */
  int32_t suffix_tokens;      /* tokens gained from phrase suffixes (sum of hat-A - 1, Eq. 9) */
  int32_t candidates;         /* candidate phrases verified in total */
  float ms_total, ms_target, ms_draft;  /* CUDA-event times of the whole loop / target forwards / drafting */
} ouro_stats;

/* External drafter: fills out[0..gamma) given the whole text so far (seq[n_seq-1] is the pending
 * token).  Used to replay recorded drafts; returns 0 on success. */
typedef int (*ouro_drafter_fn)(void *user, const int32_t *seq_host, int32_t n_seq, int32_t gamma,
                               int32_t step, int32_t *out_host);

const char *ouro_strerror(int status);
const char *ouro_last_error(const ouro_ctx *ctx);   /* ctx may be NULL: error of the last failed ouro_create */

/* Bytes of device workspace ouro_create needs (activations, block descriptors, phrase pool, rotary
 * tables, split-K / split-KV scratch).  draft may be NULL.  Returns 0 on invalid arguments. */
size_t ouro_workspace_bytes(const ouro_model_desc *target, const ouro_model_desc *draft, const ouro_params *params);

/* Creates a context.  draft / draft_mem may both be NULL (then drafts come from ouro_set_drafter or from
 * the caller via ouro_assemble_candidates).  workspace must be 256-byte aligned device memory of at
 * least ouro_workspace_bytes(); cuda_stream is a cudaStream_t (NULL = default stream).  The phrase
 * pool starts empty, both caches start at length 0.  Synchronises the stream once. */
int ouro_create(const ouro_model_desc *target, const ouro_model_mem *target_mem,
                const ouro_model_desc *draft, const ouro_model_mem *draft_mem,
                const ouro_params *params, void *workspace_dev, size_t workspace_bytes,
                void *cuda_stream, ouro_ctx **out);
int ouro_destroy(ouro_ctx *ctx);

/* Forgets the text and both caches.  keep_pool != 0 keeps the phrases of earlier queries (Section 3.4). */
int ouro_reset(ouro_ctx *ctx, int keep_pool);

/* Caches prompt[0..n-2] in the target (causal forwards in chunks) and leaves prompt[n-1] pending;
 * seeds the pool per OURO_SEED_PROMPT.  The draft model catches up lazily at its first drafting. */
int ouro_prefill(ouro_ctx *ctx, const int32_t *prompt_host, int32_t n);

/* Declares both caches to already hold cache_len tokens (contents supplied by the caller) with the given
 * pending token: entry state for stepping from a synthetic cache.  Text positions < cache_len are
 * recorded as token 0. */
int ouro_set_state(ouro_ctx *ctx, int32_t cache_len, int32_t pending_token);
int ouro_get_state(ouro_ctx *ctx, int32_t *target_len, int32_t *draft_len, int32_t *pending_token);

int ouro_set_drafter(ouro_ctx *ctx, ouro_drafter_fn fn, void *user);

/* Phrase pool (Section 3.2: phrases are retrieved by their first token).
 * lookup: up to K most recently inserted phrases whose first token is key; their suffixes p_2..p_beta
 *   go to suffix_dev [K, beta-1] and the number found to count_dev[0].
 * update: n beta-grams ngrams_dev [n, beta] are inserted in order (present -> refreshed; else first
 *   free way of the set; else the least recently inserted entry of the set is overwritten). */
int ouro_phrase_lookup(ouro_ctx *ctx, int32_t key, int32_t K, int32_t *suffix_dev, int32_t *count_dev);
int ouro_phrase_update(ouro_ctx *ctx, const int32_t *ngrams_dev, int32_t n);
/* Host copies of the pool: ngrams_host [cap, beta], stamps_host [cap] with cap = pool_sets*pool_ways,
 * entries sorted by stamp ascending; *n = entries written.  import inserts the phrases in order. */
int ouro_pool_export(ouro_ctx *ctx, int32_t *ngrams_host, uint64_t *stamps_host, int32_t *n);
int ouro_pool_import(ouro_ctx *ctx, const int32_t *ngrams_host, int32_t n);

/* Eq. 7: packs [pending, d_1..d_gamma, p^1_2..beta, .., p^K'_2..beta] into the target's query block with
 * position ids (trunk row b: L+b; suffix row (j,i): L+gamma+i) and the Eq. 8 visibility.  draft_dev
 * [gamma].  suffix_dev / count_dev as written by ouro_phrase_lookup; pass NULL for both to have the
 * pool looked up with key d_gamma here.  Asynchronous when the target runs on the tensor-core kernels (bf16,
 * supported shapes): the block's row count 1 + gamma + K' (beta-1) then stays on the device, the forward is
 * launched for the largest block the parameters allow and ouro_block_get reports the true count.  Otherwise the
 * call synchronises to read the count. */
int ouro_assemble_candidates(ouro_ctx *ctx, const int32_t *draft_dev, const int32_t *suffix_dev,
                             const int32_t *count_dev);
/* Plain causal block of n tokens (tokens_dev [n]) for model `which`: prefill, catch-up, vanilla decoding. */
int ouro_assemble_causal(ouro_ctx *ctx, int which, const int32_t *tokens_dev, int32_t n);
/* Host copies of the current block of model `which`: tokens/pos/group [B], mask [B, 2] (bit c of row r,
 * 128 bits per row: row r may attend block row c), *B rows. */
int ouro_block_get(ouro_ctx *ctx, int which, int32_t *tokens_host, int32_t *pos_host, int32_t *group_host,
                   uint64_t *mask_host, int32_t *B);

/* Section 3.2 / Eq. 8: one forward of model `which` scores every row of its current block (all K
 * lengthened drafts at once, under the candidate mask) against its KV cache.  Appends the block's K/V at cache slots L..L+B-1, writes the
 * greedy next token of every row to argmax_dev [B] (ties -> smallest id) and, if logits_dev is not
 * NULL, the fp32 logits [B, vocab].  Does not change the cache length.  Asynchronous. */
int ouro_verify_forward(ouro_ctx *ctx, int which, int32_t *argmax_dev, float *logits_dev);

/* Eq. 3 / Eq. 9 on the last target verification (argmax_dev [B] as written by ouro_verify_forward):
 * accepted tokens, chosen candidate (-1: none), in-place KV compaction of every layer, pool harvest
 * per flags, new pending token.  accepted_host [gamma+beta].  Host outputs may be NULL. */
int ouro_accept_and_compact(ouro_ctx *ctx, const int32_t *argmax_dev, int32_t *n_accepted_host,
                            int32_t *chosen_host, int32_t *accurate_host, int32_t *accepted_host);
/* The three calls above in one: packs the block for draft_dev [gamma] (pool looked up with key d_gamma), runs the
 * target forward and applies Eq. 3 / Eq. 9, compaction and harvest.  Same host outputs as ouro_accept_and_compact;
 * the only host wait of the step is the one for the acceptance record. */
int ouro_verify_step(ouro_ctx *ctx, const int32_t *draft_dev, int32_t *n_accepted_host, int32_t *chosen_host,
                     int32_t *accurate_host, int32_t *accepted_host);
/* Advances model `which` past the first n rows of its current causal block (they become cached text). */
int ouro_advance(ouro_ctx *ctx, int which, int32_t n);

/* Eq. 1: gamma greedy draft tokens from the draft model (or the external drafter) into draft_dev [gamma].
 * With OURO_DRAFT_PHRASES (and no external drafter) the draft model drafts phrase by phrase (Section 3.1,
 * Eq. 6).  The paper does not give the procedure; here a drafting round is the verification step of Section
 * 3.2 run by the draft model on itself: the text it has not cached yet, followed by the K pool phrases that
 * start with the last known token, go through one draft forward under the mask of Eq. 8; the draft model's
 * greedy outputs accept the longest matching phrase prefix (Eq. 9) and one more token, and its cache is
 * compacted like the target's.  The tokens are those of token-level drafting; only the number of draft
 * forwards (ouro_stats.draft_calls) changes.  The pool is read, not written, while drafting.
 * With ouro_params.window = W > 0 (token-level drafting) every draft forward also carries W guessed tokens for the
 * positions that follow, packed like one candidate suffix (Eq. 8 mask).  The paper says that new phrases are generated
 * in parallel during each forward of the draft model and leaves the procedure to lookahead decoding; here the window
 * rows' greedy outputs (a) become the next forward's guesses (the window slides with the text, one Jacobi step per
 * forward) and (b) give beta-grams along the diagonal - a guess followed by the predictions after it - that enter the
 * pool at once, W - beta + 3 per forward, so that the verification that follows can look them up.  The draft tokens are
 * unchanged. */
int ouro_draft(ouro_ctx *ctx, int32_t *draft_dev);

/* Whole loops.  out_host [max_new]; *n_out tokens written (stops at eos_token).  ouro_generate is the
 * Ouroboros loop; ouro_generate_vanilla is greedy decoding with the target alone through the same
 * kernels, one token per forward.  Both start with ouro_reset(keep_pool) + ouro_prefill. */
int ouro_generate(ouro_ctx *ctx, const int32_t *prompt_host, int32_t n_prompt, int32_t max_new,
                  int32_t keep_pool, int32_t *out_host, int32_t *n_out, ouro_stats *stats_or_null);
int ouro_generate_vanilla(ouro_ctx *ctx, const int32_t *prompt_host, int32_t n_prompt, int32_t max_new,
                          int32_t *out_host, int32_t *n_out, ouro_stats *stats_or_null);

/* Measurement aid (no counterpart in the paper, which reports end-to-end speed only): while enabled,
 * every launch of the kernel class `kernel_class` inside ouro_verify_forward is bracketed by CUDA events
 * on the context's stream.  ouro_profile_read synchronises, adds up the event times and returns the total
 * milliseconds and the number of launches since the last ouro_profile_enable.  Other kernels are not
 * touched; the extra event records cost about a microsecond per launch, so enable it outside timed runs. */
enum {
  OURO_PROF_OFF = -1, OURO_PROF_EMBED = 0, OURO_PROF_NORM = 1, OURO_PROF_QKV = 2, OURO_PROF_ROPE = 3,
  OURO_PROF_ATTENTION = 4, OURO_PROF_WO = 5, OURO_PROF_GATEUP = 6, OURO_PROF_DOWN = 7, OURO_PROF_HEAD = 8,
  OURO_PROF_ARGMAX = 9, OURO_PROF_FORWARD = 10 /* the whole forward */,
  OURO_PROF_GEMM = 11 /* every launch of the weight-streaming GEMM kernel; consecutive GEMMs (output projection, gate/up,
                         down, the next q,k,v or the LM head) run as ONE launch, except while one of the classes
                         QKV..HEAD is being timed: then each GEMM is launched alone so that it can be */
};
/* Number of kernels this library has launched in this process (all contexts), for launch accounting. */
uint64_t ouro_kernel_launches(void);
int ouro_profile_enable(ouro_ctx *ctx, int kernel_class);
/* Test aid for the give-up path of the bounded device-side waits (no counterpart in the paper).  A GEMM tile whose K
 * range is split across CTAs is finished once all contributors have published their partial sums; the waiting thread
 * polls a counter at most `polls` times (default 1 << 22; negative restores the default).  0 makes the wait give up
 * at once: the kernels return normally, the status word is raised, the next call that reads results back
 * (ouro_accept_and_compact, ouro_generate, ouro_generate_vanilla) returns OURO_ETIMEOUT, and ouro_reset makes the
 * context usable again.  OURO_ESTATE when the context does not run the tensor-core kernels. */
int ouro_debug_set_wait_limit(ouro_ctx *ctx, int64_t polls);
int ouro_profile_read(ouro_ctx *ctx, float *ms_total, int32_t *launches);

/* (The paper has no counterpart to this call; it exists for deployment reasons only.)
 * LM-head pass without any caller-provided workspace and without any allocation by the library: for callers
 * that cannot allocate device memory - e.g. a server that gave all of it to its own arena at start-up, or a
 * latency-critical loop that must avoid the device-wide synchronisation an allocation may cause.
 *   x_dev        [rows, d_model] bf16, already normalised activations (device, 16-byte aligned)
 *   lm_head_dev  [vocab, d_model] bf16, row-major (device, 16-byte aligned)
 *   argmax_dev   [rows] int32 out: greedy token per row (ties -> smallest id)
 *   logits_dev   [rows, vocab] fp32 out, or NULL
 * Limits: 1 <= rows <= 128, d_model a multiple of 64, vocab a multiple of 8 and <= 65536; anything else returns
 * OURO_EINVAL with a text in ouro_last_error(NULL).  The split-K scratch, counters and per-tile maxima live in a
 * 5 MiB array inside the library image; every GPU that loads the library holds it until the process exits.
 * The first call on each device resolves that array's device address and sizes the kernel's shared memory;
 * make that first call outside any stream capture, with the device current.  All calls on a device share the
 * array: two calls whose GPU work overlaps (different streams or threads) race on it - serialise them.
 * The call enqueues on cuda_stream (a cudaStream_t, NULL = default), then synchronises that stream and returns
 * OURO_ETIMEOUT if a bounded device-side wait gave up.  It runs on 32 SMs only (the scratch is sized per CTA), so
 * it is slower than ouro_verify_forward's head pass; results agree with it to rounding (another split of K). */
int ouro_lm_head_static(const void *x_dev, const void *lm_head_dev, int32_t rows, int32_t d_model, int32_t vocab,
                        int32_t *argmax_dev, float *logits_dev, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* OURO_H */
