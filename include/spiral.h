/*
 * spiral.h -- C ABI of the rollout-decoding library for one B200 (sm_100a).
 *
 * What it computes.  In the self-play loop of Algorithm 1 every active game asks the shared
 * policy for a multi-token response, y_t ~ pi_theta(. | s_t, p, G_i) (Algorithm 1, response
 * generation line; Section 3 "Self-play": one set of parameters serves both roles and every
 * game).  The state s_t carries the game's history, so the context of a game persists and grows
 * over its turns (Section 3 "Formulation"; Appendix "Training details": past actions are
 * concatenated into the state).  Responses are sampled at temperature 1.0 with top-p 1.0 and
 * top-k -1, i.e. untruncated categorical sampling, up to 8192 tokens (hyperparameter table, Actor
 * block).  This library evaluates that policy one token at a time for a batch of concurrent games:
 * a Qwen/Llama-family pre-norm decoder (RMSNorm, QKV projection, optional per-head q/k RMSNorm,
 * rotate-half RoPE, grouped-query attention over the game's cached keys/values, output projection,
 * SwiGLU MLP, LM head) followed by a Gumbel-max draw  token = argmax_v(logit_v / T + gumbel_v)
 * with caller-supplied noise.  Every step of that computation runs in CUDA kernels of this
 * library; there is no CPU path.
 *
 * Conventions.
 *   - "dev" pointers are CUDA device pointers on the device given to spiral_init, "host" pointers
 *     are ordinary host memory.  The caller owns every buffer it passes in (weights, the KV pool
 *     slab, token / noise / output buffers, the stream).  The library owns host bookkeeping, small
 *     device mirrors of it and a workspace it allocates in spiral_init / spiral_kv_alloc.
 *   - Weights are bf16; the KV pool holds 2-byte floats (fp16 or bf16, chosen in spiral_kv_alloc); tokens, game ids and page ids are int32; noise, logits and
 *     the temperature are fp32.  The residual stream, norms, softmax and all accumulators are fp32.
 *     Activations entering a matrix product are rounded once to fp16 (11-bit mantissa); bf16
 *     weights are exactly representable in fp16 (the tensor-core path re-encodes them once at
 *     init into a private fp16 copy; magnitudes below 2^-24 flush), so products are exact.
 *   - Calls are asynchronous on `cuda_stream` (a cudaStream_t passed as void*, NULL = the legacy
 *     default stream) unless stated otherwise.  Calls on one ctx/kv must be issued from one host
 *     thread at a time and on one stream (or on streams the caller orders).
 *   - Every function returns SPIRAL_OK (0) or a negative error; nothing aborts, throws or traps.
 *     After an error the host state of ctx/kv is unchanged unless stated otherwise.
 */
#ifndef SPIRAL_H
#define SPIRAL_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPIRAL_OK                 0
#define SPIRAL_ERR_INVALID       -1   /* NULL pointer, size out of range, bad or duplicate game id, T <= 0 */
#define SPIRAL_ERR_OOM           -2   /* no free KV page, or a host/device allocation failed */
#define SPIRAL_ERR_CUDA          -3   /* a CUDA runtime/driver call failed (text: spiral_last_cuda_error) */
#define SPIRAL_ERR_TIMEOUT       -4   /* a bounded device-side wait ran out (device status word) */
#define SPIRAL_ERR_DEVICE_CHECK  -5   /* a device-side bounds check tripped (device status word) */
#define SPIRAL_ERR_UNSUPPORTED   -6   /* shape outside what the kernels are built for */
#define SPIRAL_ERR_TOO_LARGE     -7   /* size beyond the fixed capacity of an entry point that cannot allocate */

/* element type of the KV pages */
#define SPIRAL_KV_F16   0   /* IEEE half: 11-bit mantissa; values saturate at +-65504 */
#define SPIRAL_KV_BF16  1   /* bfloat16: 8-bit mantissa */

typedef struct spiral_ctx spiral_ctx;   /* model description, weight pointers, workspace */
typedef struct spiral_kv  spiral_kv;    /* page pool bookkeeping: free list, block tables, lengths */

/* Decoder architecture.  head_dim must be 64 or 128; n_q_heads a multiple of n_kv_heads with
 * n_q_heads / n_kv_heads <= 8; d_model, d_ff and n_q_heads*head_dim multiples of 64. */
typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff, vocab;
    double  rope_theta;      /* RoPE base; angle of pair i at position p is p * theta^(-2i/head_dim) */
    double  rms_eps;         /* epsilon inside the square root of every RMSNorm */
    int32_t qk_norm;         /* 1: RMSNorm over head_dim on every q and k head, before RoPE */
    int32_t qkv_bias;        /* 1: bias added to the q, k, v projections */
    int32_t tied_embed;      /* 1: the LM head is the embedding matrix */
} spiral_model_desc;

/* Device pointers to bf16 weights.  Matrices are [out_features][in_features] row-major.
 * Per-layer members point to host arrays of n_layers device pointers (copied during init).
 *   wqkv      [(n_q_heads + 2 n_kv_heads) * head_dim][d_model]: q heads, then k heads, then v heads
 *   bqkv      same row order, or NULL array when qkv_bias == 0
 *   q_norm, k_norm   [head_dim] gains shared by the heads of a layer, or NULL arrays when qk_norm == 0
 *   wo        [d_model][n_q_heads * head_dim]
 *   w_gate_up [2 d_ff][d_model] with row 2i = gate row i and row 2i+1 = up row i
 *   w_down    [d_model][d_ff]
 *   embed     [vocab][d_model];  lm_head [vocab][d_model] or NULL when tied_embed == 1
 *   ln1, ln2, final_norm   [d_model] RMSNorm gains
 * All matrix base addresses must be 16-byte aligned.  Weights must outlive the ctx. */
typedef struct {
    const void *embed, *lm_head, *final_norm;
    const void *const *ln1, *const *wqkv, *const *bqkv, *const *q_norm, *const *k_norm;
    const void *const *wo, *const *ln2, *const *w_gate_up, *const *w_down;
} spiral_weights;

/* Creates a context on CUDA device `device` for batches of at most max_batch games per step
 * (1..256) and contexts of at most max_ctx tokens (RoPE table size).  Allocates the workspace
 * (activations, split-K pieces, attention partials; tens of MB) with cudaMalloc and builds the
 * RoPE table on the device in fp64.  The kernels are written for sm_100 (tcgen05, TMEM, TMA): on any
 * other device the call returns SPIRAL_ERR_UNSUPPORTED -- there is no second code path.  Synchronous.
 * *out is written only on success. */
int spiral_init(spiral_ctx **out, const spiral_model_desc *desc, const spiral_weights *weights,
                int device, int max_batch, int max_ctx);

/* Bytes of pool one page occupies over all layers: n_layers * n_kv_heads * 2 * page_size * head_dim * 2. */
size_t spiral_kv_page_bytes(const spiral_model_desc *desc, int page_size);

/* Lays a paged KV cache over the caller's slab pool_dev (256-byte aligned, pool_bytes long).
 * Layout: [layer][page][kv_head][K|V][page_size][head_dim] of 2-byte floats, so the K rows of one
 * page and head are contiguous (page_size * head_dim * 2 bytes) and so are its V rows.  n_pages =
 * pool_bytes / spiral_kv_page_bytes.  page_size must be 16.  kv_dtype is SPIRAL_KV_F16 or
 * SPIRAL_KV_BF16: keys and values are rounded once to that type when cached.  (With bf16 pages the
 * rounding of the cache alone costs about 1e-2 relative RMS on the logits of a 36-layer decoder;
 * fp16 pages cost about 1.3e-3 at the same bandwidth.)  Games are numbered 0..max_games-1;
 * each starts empty and may grow to max_ctx tokens (<= the ctx's max_ctx).  A game's cache
 * survives across calls (turns) until spiral_kv_release.  The pool must outlive the kv. */
int spiral_kv_alloc(spiral_ctx *ctx, void *pool_dev, size_t pool_bytes, int page_size, int kv_dtype,
                    int max_games, int max_ctx, spiral_kv **out);

/* Game finished: its pages go back to the free list and its length becomes 0.  Host-only.  The
 * caller must not have work of these games still queued on another stream. */
int spiral_kv_release(spiral_kv *kv, int n, const int32_t *game_ids_host);

/* Rolls games back to shorter cached lengths (new_len_host[i] <= current length of game
 * game_ids_host[i]): pages beyond the new length return to the free list.  Host-only; the cached
 * keys/values of the kept positions are untouched, so decoding can resume from there (a rejected or
 * re-sampled move, or a benchmark replaying the same steps).  Same stream caveat as release. */
int spiral_kv_truncate(spiral_kv *kv, int n, const int32_t *game_ids_host, const int32_t *new_len_host);

/* Host-side queries (no device work): cached length of a game; number of free pages. */
int spiral_kv_seq_len(const spiral_kv *kv, int game_id, int32_t *out);
int spiral_kv_free_pages(const spiral_kv *kv, int32_t *out);

/* Starts game dst_game (which must be empty) from the first n_tokens cached positions of src_game,
 * e.g. a system prompt that many games share (the role conditioning of Section 3 is a prompt).
 * Whole pages are shared by reference -- no copy, no extra memory; a page returns to the free list
 * when its last holder releases it -- and the partly filled last page, if any, is copied on the
 * device (one free page needed: SPIRAL_ERR_OOM otherwise).  Both games then grow independently.
 * spiral_kv_truncate refuses (SPIRAL_ERR_UNSUPPORTED) to cut a game inside a page it shares. */
int spiral_kv_fork(spiral_ctx *ctx, spiral_kv *kv, int src_game, int dst_game, int n_tokens, void *cuda_stream);

/* Test/benchmark aid: sets layer `layer` of an EMPTY or previously loaded game to n_tokens cached
 * positions copied from k_dev, v_dev ([n_tokens][n_kv_heads][head_dim] in the pool's type, already normalised and
 * rotated as a real cache would be).  Pages are allocated on the first layer loaded; every layer
 * must be loaded with the same n_tokens before the game is decoded.  SPIRAL_ERR_OOM leaves the
 * game empty. */
int spiral_kv_load(spiral_ctx *ctx, spiral_kv *kv, int game_id, int layer, int n_tokens,
                   const void *k_dev, const void *v_dev, void *cuda_stream);

/* Appends tokens to n games and caches their keys/values: game game_ids_host[i] receives
 * tokens_dev[offsets_host[i] .. offsets_host[i+1]) at positions len, len+1, ...  May be called
 * again on the same game in a later turn.  If last_logits_dev != NULL it receives the fp32 logits
 * [n][vocab] after each game's last appended token.  All pages needed are reserved up front:
 * SPIRAL_ERR_OOM / SPIRAL_ERR_INVALID leave every game unchanged.  This is the observation every game
 * receives between two turns of Algorithm 1 (the state carries the history).  A call with more than
 * max_batch new tokens in total, on an fp16 cache and a model whose matrices are on the tensor-core
 * path, runs as dense passes of up to 9472 token rows (256-token GEMM tiles, causal block attention);
 * the first such call allocates the passes' workspace (device synchronisation; SPIRAL_ERR_OOM if it
 * does not fit).  Otherwise the new tokens are pushed through the decode kernels in chunks of up to
 * max_batch (game, position) slots; several positions of one game may share a chunk (each attends
 * to positions up to its own only). */
int spiral_prefill(spiral_ctx *ctx, spiral_kv *kv, int n, const int32_t *game_ids_host,
                   const int32_t *tokens_dev, const int32_t *offsets_host, float *last_logits_dev,
                   void *cuda_stream);

/* One token for each of n games.  For game g = game_ids_host[i] with cached length S_g:
 * the input token tok_in_dev[i] is embedded, run through every layer with its k/v written at
 * position S_g, attention covers positions 0..S_g, and
 *     tok_out_dev[i] = argmax_v ( logit_v / temperature + gumbel_dev[i][v] ),  lowest v on ties,
 * computed in fp32 (divide, then add).  S_g becomes S_g + 1.  The caller feeds tok_out back as the
 * next tok_in (or teacher-forces another token).  gumbel_dev is fp32 [n][vocab]; logits_dbg_dev,
 * if not NULL, receives the fp32 logits [n][vocab] (otherwise full-vocabulary logits are never
 * written to memory on the tensor-core path).  game ids must be distinct.  temperature > 0. */
int spiral_decode_step(spiral_ctx *ctx, spiral_kv *kv, int n, const int32_t *game_ids_host,
                       const int32_t *tok_in_dev, const float *gumbel_dev, float temperature,
                       int32_t *tok_out_dev, float *logits_dbg_dev, void *cuda_stream);

/* The same step, which also returns what a policy-gradient learner needs from the actor (the
 * clipped update of Algorithm 1's policy-update line uses the probability the acting policy gave to
 * each sampled token): logprob_dev[i] = log softmax(logits_i / temperature)[tok_out_dev[i]], fp32 [n].
 * The log-sum-exp is accumulated alongside the running argmax in the LM-head epilogue, so the
 * full-vocabulary logits still never go to memory. */
int spiral_decode_step_logprob(spiral_ctx *ctx, spiral_kv *kv, int n, const int32_t *game_ids_host,
                               const int32_t *tok_in_dev, const float *gumbel_dev, float temperature,
                               int32_t *tok_out_dev, float *logprob_dev, float *logits_dbg_dev, void *cuda_stream);

/* spiral_decode_step with nucleus (top-p) sampling -- the evaluation setting of the paper
 * ("Evaluation Settings": temperature 0.6, top-p 0.95; rollouts use top-p 1.0).  With z = logits /
 * temperature and p = softmax(z), token v is kept when the mass of the tokens strictly more
 * probable than v is below top_p (the shortest most-probable-first prefix whose mass reaches top_p,
 * plus ties of its last member; the most probable token is always kept), and
 *     tok_out_dev[i] = argmax over kept v of ( z_v + gumbel_dev[i][v] ),  lowest v on ties,
 * i.e. a draw from the kept tokens' renormalised distribution.  z and the sum are fp32; the mass
 * comparisons use fixed-order fp32 sums of exp(z - max z), so a call is reproducible.  0 < top_p <= 1
 * (1: identical to spiral_decode_step).  The logits of the step pass through an internal fp32
 * [n][vocab] buffer; logits_dbg_dev, if not NULL, receives a copy. */
int spiral_decode_step_nucleus(spiral_ctx *ctx, spiral_kv *kv, int n, const int32_t *game_ids_host,
                               const int32_t *tok_in_dev, const float *gumbel_dev, float temperature,
                               float top_p, int32_t *tok_out_dev, float *logits_dbg_dev,
                               void *cuda_stream);

/* The sampler of spiral_decode_step_nucleus alone, on logits the caller holds: logits_dev and
 * gumbel_dev are fp32 [n][vocab] (gumbel_dev may be NULL: no noise, i.e. the most probable token),
 * tok_out_dev int32 [n]; n <= max_batch.  Component entry point for unit parity. */
int spiral_sample_nucleus(spiral_ctx *ctx, int n, const float *logits_dev, const float *gumbel_dev,
                          float temperature, float top_p, int32_t *tok_out_dev, void *cuda_stream);

/* Role-conditioned advantage estimation (Algorithm 1, policy-optimisation loop; Eq. 2): for
 * trajectory t = 0 .. n_traj-1 in order, of game kind g = game_of_host[t], and role p = 0, 1:
 *     b[g][p] <- alpha * b[g][p] + (1 - alpha) * R_p(t);     A_p(t) = R_p(t) - b[g][p]   (the updated b)
 * baselines_host is [n_games][2] (the caller zeroes it once: Algorithm 1 initialises b = 0),
 * returns_host and advantages_host are [n_traj][2], all fp64, all host memory; alpha in [0, 1]
 * (0.95 in the paper's hyperparameter table).  Host arithmetic only; SPIRAL_ERR_INVALID (bad
 * alpha, game index out of range, NULL) changes nothing. */
int spiral_rae_update(double *baselines_host, int n_games, double alpha, int n_traj,
                      const int32_t *game_of_host, const double *returns_host, double *advantages_host);

/* ---- episode scheduler: continuous batching of multi-turn games ---------------------------------
 * Algorithm 1 plays many games at once; every turn appends an observation to a game's context and
 * generates a response of unknown length, so games start, change turns and finish at different
 * times.  The scheduler keeps the decode batch full from a first-come-first-served queue of waiting
 * turns, on top of spiral_prefill and the decode step of one context and cache (between two ticks
 * the caller may still use them directly, but only on idle games: e.g. to append a shared prompt
 * to a template game that others are then forked from).  Host bookkeeping; one per (ctx, kv).
 *
 * A game is a cache row: spiral_sched_open hands one out (SPIRAL_ERR_OOM when all max_games are
 * taken), spiral_sched_close returns it with its pages (only while no turn of it waits or runs).
 * spiral_sched_turn queues a turn: n_obs >= 1 observation tokens (host memory, copied) to append
 * and a response budget max_new_tokens >= 1; SPIRAL_ERR_INVALID if the game is not idle or the turn
 * cannot fit max_ctx, SPIRAL_ERR_OOM if it cannot fit the pool even when empty.  A response ends
 * with eos_token (given at creation; -1: none) or at its budget.
 *
 * spiral_sched_tick does one round: reads the tokens sampled up to the step before last (the host
 * never waits for the step it launched last), retires finished turns, admits waiting turns in
 * order while the batch has a free slot (max_batch) and the free pages cover the turn's worst case
 * (context + observation + budget) beside what running turns may still claim -- so a running turn
 * never runs out of pages; appends the admitted observations with one spiral_prefill (all but each
 * one's last token, which feeds the game's first step); decodes one token for every running turn
 * with budget left: gumbel_dev is fp32 [max_batch][vocab] fresh noise, row i for the i-th game of
 * the step.  Sampled tokens stay on the device as the next inputs.  Returns the number of games
 * decoded (0: nothing could run -- everything is finished, or the head of the queue waits for
 * pages that only closing games can free), or a negative error.
 *
 * Because an end-of-sequence token is seen one tick late, its game runs one more step; that sample
 * is dropped and the step's only effect is that the final token's key/value is already cached.
 * Otherwise (budget reached) the final token is cached at the start of the game's next turn.
 * Either way the context after a turn is: previous context, observation, full response.
 *
 * spiral_sched_poll returns 1 and one finished turn (game, its response tokens, reason 1 =
 * end-of-sequence, 2 = budget), 0 when none is ready, SPIRAL_ERR_TOO_LARGE if max_tokens is too
 * small.  spiral_sched_policy sets when waiting turns are let in: a small append costs a pass over
 * all weights, so by default they are held until together they bring 1024 observation tokens, or
 * until at most max_batch / 2 turns are still running (admit_tokens = 1, or low_water = max_batch,
 * admits at once).  spiral_sched_stats fills up to 8 counters: turns waiting, running, finished unread, free
 * pages, pages reserved by running turns, tokens decoded, samples dropped, tokens appended. */
typedef struct spiral_sched spiral_sched;
int spiral_sched_create(spiral_ctx *ctx, spiral_kv *kv, int eos_token, spiral_sched **out);
void spiral_sched_free(spiral_sched *sched);
int spiral_sched_open(spiral_sched *sched, int32_t *game_out);
int spiral_sched_close(spiral_sched *sched, int game);
/* a new game whose context starts as a copy-free fork (spiral_kv_fork) of the whole context of an idle game */
int spiral_sched_fork(spiral_sched *sched, int src_game, int32_t *game_out, void *cuda_stream);
int spiral_sched_turn(spiral_sched *sched, int game, int n_obs, const int32_t *obs_host, int max_new_tokens);
int spiral_sched_tick(spiral_sched *sched, const float *gumbel_dev, float temperature, void *cuda_stream);
int spiral_sched_policy(spiral_sched *sched, int admit_tokens, int low_water);
int spiral_sched_poll(spiral_sched *sched, int32_t *game_out, int32_t *tokens_out_host, int max_tokens,
                      int32_t *n_tokens_out, int32_t *reason_out);
/* With spiral_sched_collect_logprob(sched, 1) (only while no turn is running) every later step also
 * records log softmax(logits / temperature)[sampled token], which the policy update of Algorithm 1
 * needs beside the tokens; spiral_sched_poll_logprob is spiral_sched_poll that also copies those
 * values (fp32, one per response token) to logprob_out_host. */
int spiral_sched_collect_logprob(spiral_sched *sched, int on);
int spiral_sched_poll_logprob(spiral_sched *sched, int32_t *game_out, int32_t *tokens_out_host, float *logprob_out_host,
                              int max_tokens, int32_t *n_tokens_out, int32_t *reason_out);
int spiral_sched_stats(const spiral_sched *sched, int64_t *out, int n_out);

/* Same step with HOST token / noise / output buffers (pinned memory recommended): copies
 * tok_in and gumbel to device staging, runs the step, copies tok_out back and waits for it.
 * Synchronous with respect to `cuda_stream`. */
int spiral_decode_step_host(spiral_ctx *ctx, spiral_kv *kv, int n, const int32_t *game_ids_host,
                            const int32_t *tok_in_host, const float *gumbel_host, float temperature,
                            int32_t *tok_out_host, void *cuda_stream);

/* Component entry points (same kernels the step uses), for unit parity and per-kernel timing.
 * spiral_linear:  y_dev[b][r] = sum_k x_dev[b][k] * w_dev[r][k]   (x fp16 [n][k_dim], w bf16
 *   [rows][k_dim], y fp32 [n][rows]); path 0 = automatic, 1 = CUDA-core GEMV, 2 = tcgen05.
 * spiral_attention: q_dev fp32 [n][n_q_heads][head_dim] (already normalised and rotated) against
 *   the first ctx_len_host[i] cached positions of game game_ids_host[i] in layer `layer`;
 *   out_dev fp32 [n][n_q_heads][head_dim]. */
int spiral_linear(spiral_ctx *ctx, const void *w_dev, int rows, int k_dim, const void *x_dev, int n,
                  float *y_dev, int path, void *cuda_stream);
int spiral_attention(spiral_ctx *ctx, spiral_kv *kv, int layer, int n, const int32_t *game_ids_host,
                     const int32_t *ctx_len_host, const float *q_dev, float *out_dev,
                     void *cuda_stream);

/* Host-side query: writes the page ids game `game_id` currently owns, in position order (page i
 * holds positions 16 i .. 16 i + 15), to out_host and returns how many there are; SPIRAL_ERR_INVALID
 * if there are more than max_entries. */
int spiral_kv_block_table(const spiral_kv *kv, int game_id, int32_t *out_host, int max_entries);

/* Paged GQA decode attention for callers that must not allocate device memory.  (The paper has
 * no counterpart to this entry point: it is a packaging variant of the attention kernel above.)
 *
 * Who needs it: code that runs where cudaMalloc is off the table -- a plugin inside a host
 * application that hands every byte of device memory out itself, a real-time loop that may not
 * take the allocator's locks or its implicit device synchronisation, a process that has already
 * given all free memory to one big pool.  Such a caller cannot use spiral_init (which allocates a
 * workspace), so this call takes everything it needs as plain arguments and keeps its scratch --
 * the partial results of the split context, their arrival counters and the small schedule arrays --
 * in one fixed array inside the library image (about 4.3 MB on every GPU that loads the library,
 * until the process exits).  It calls no cudaMalloc / cudaFree and no allocating library routine.
 *
 *   pool_dev         caller's KV pool, 256-byte aligned, laid out as spiral_kv_alloc documents:
 *                    [n_layers][n_pages][n_kv_heads][K|V][16][head_dim], kv_dtype = SPIRAL_KV_F16 / _BF16
 *   block_table_dev  int32 [n][max_pages] on the device: page ids of sequence i in position order
 *   ctx_len_host     host array [n]: positions 0 .. ctx_len_host[i]-1 of sequence i are attended
 *   q_dev, out_dev   fp32 [n][n_q_heads][head_dim], queries already normalised and rotated
 * head_dim is 64 or 128, n_q_heads / n_kv_heads <= 8.  Capacity: n <= SPIRAL_STATIC_ATTN_MAX_SEQS and
 * n * n_kv_heads <= SPIRAL_STATIC_ATTN_MAX_ITEMS; anything larger is refused with SPIRAL_ERR_TOO_LARGE
 * (text in spiral_last_cuda_error) and nothing is launched.  Results equal spiral_attention's up to
 * the order in which partial sums are merged.
 *
 * The first call on a device looks up the device address of the scratch array and configures the
 * kernel (safe against two host threads making that call together).  The call copies its schedule
 * from host arrays of the call, so it cannot be part of a stream capture: while cuda_stream is
 * capturing it returns SPIRAL_ERR_UNSUPPORTED and does nothing.  Every call on a device shares the
 * one array: each call re-zeroes the counters it relies on, but two calls whose GPU work overlaps
 * (two streams, two threads) race on it -- order them.  Asynchronous on cuda_stream.
 *
 * Device-side findings (a page id of the caller's block table outside [0, n_pages): that page is
 * replaced by page 0 and the call's output for that sequence is meaningless; a bounded wait that ran
 * out) are kept in a status word inside the same array until spiral_attention_static_status reads
 * it: that call synchronises the device, returns SPIRAL_OK, SPIRAL_ERR_DEVICE_CHECK or
 * SPIRAL_ERR_TIMEOUT for the first finding since the last read (raw word in *detail_out, optional)
 * and clears it.  It allocates nothing either. */
#define SPIRAL_STATIC_ATTN_MAX_SEQS   256
#define SPIRAL_STATIC_ATTN_MAX_ITEMS  512
int spiral_attention_static(int device, const void *pool_dev, int n_pages, int n_layers, int layer, int kv_dtype,
                            int n_q_heads, int n_kv_heads, int head_dim, const int32_t *block_table_dev,
                            int max_pages, int n, const int32_t *ctx_len_host, const float *q_dev,
                            float *out_dev, void *cuda_stream);
int spiral_attention_static_status(int device, int32_t *detail_out);

/* Per-kernel timing, for roofline reports.  Kernel classes of one decode step: */
#define SPIRAL_KC_ATTN        0   /* split-context paged GQA attention */
#define SPIRAL_KC_ATTN_MERGE  1   /* (unused: the partials are merged inside the attention kernel) */
#define SPIRAL_KC_QKV         2   /* QKV projection */
#define SPIRAL_KC_O           3   /* output projection */
#define SPIRAL_KC_GATE_UP     4   /* gate/up projection */
#define SPIRAL_KC_DOWN        5   /* down projection */
#define SPIRAL_KC_LM_HEAD     6   /* LM head + Gumbel-argmax */
#define SPIRAL_KC_OTHER       7   /* spiral_linear component calls */
#define SPIRAL_KC_COUNT       8
/* spiral_profile: from now on every launch of a class whose bit is set in class_mask is bracketed
 * by two CUDA events on the launch stream (0 switches timing off); earlier records are dropped.
 * Synchronises the device.  The events sit between kernels, so a timed run is slightly slower than
 * an untimed one: time whole steps with the mask at 0.
 * spiral_profile_read: synchronises, then returns the summed device time in milliseconds and the
 * number of launches recorded for one class since the last spiral_profile. */
int spiral_profile(spiral_ctx *ctx, uint32_t class_mask);
int spiral_profile_read(spiral_ctx *ctx, int kernel_class, double *total_ms_out, int64_t *n_launches_out);

/* Read-only bandwidth of the device: streams `bytes` of buf_dev (128-byte aligned, caller-owned; use
 * a buffer several times the L2 size) `passes` times into shared memory with bulk asynchronous
 * copies -- a persistent grid of ctas_per_sm CTAs per SM, each with a ring of `stages` stages of
 * stage_bytes (a multiple of 1024; stages * stage_bytes * ctas_per_sm must fit the SM's shared
 * memory) -- and reports the rate in GB/s.  blocked = 0: CTA c reads chunks c, c + grid, c + 2 grid, ...
 * (at any time the grid reads one contiguous region); blocked = 1: every CTA streams a contiguous
 * share of its own (as many far-apart streams as CTAs); blocked = 2: the chunks of pattern 0 scattered over
 * the buffer by a fixed permutation (cache pages handed out in no particular order).  tiled = 1 fetches every chunk as one tiled TMA box
 * of stage_bytes / 128 rows of 128 bytes with the 128-byte swizzle, the form the GEMM and attention kernels
 * use (stage_bytes <= 32768), instead of one linear bulk copy; tiled = 2 fetches a chunk as two boxes, the left and
 * the right 128-byte halves of its 256-byte rows (the attention kernel's form for 128-element rows).  Nothing is computed and nothing is written: this is the
 * ceiling for the decode step's kernels, which read weights and cached keys/values once per step
 * (the roofline the benchmark spec's metric of the rollout step is stated against; the paper itself gives
 * no kernel figures).  Allocates nothing on the device.  Synchronous; every device-side wait is
 * bounded (SPIRAL_ERR_TIMEOUT). */
int spiral_read_ceiling(int device, const void *buf_dev, size_t bytes, int stage_bytes, int stages,
                        int ctas_per_sm, int blocked, int tiled, int passes, void *cuda_stream, double *gbs_out);

/* Self-test of the device-side bounded waits (no counterpart in the paper: it exists so that the code that
 * unwinds a kernel after a wait ran out -- abort flag, draining of copies in flight, release of tensor memory
 * -- can be exercised without faulting or hanging a GPU).  Lowers the wait bound to about a millisecond,
 * launches one kernel whose producer deliberately leaves a load out -- which = 0: the output projection of
 * layer 0 (tcgen05 GEMM) without its activation loads; which = 1: the attention kernel over game 0's cached
 * context (>= 1 token; kv required) without the first page load of every work range -- waits for it, and
 * restores the bound.  Every access of the kernel stays in bounds and every wait ends.  Returns SPIRAL_OK when
 * the launch went through; the kernel's finding (a timeout) is then in the device status word: the next
 * spiral_last_status returns SPIRAL_ERR_TIMEOUT, re-arms the library's scratch, and the context is usable
 * again.  The kernel's outputs (the pieces buffer / the attention output buffer of the workspace) are
 * garbage.  Synchronous. */
int spiral_selftest_wait_timeout(spiral_ctx *ctx, spiral_kv *kv, int which, void *cuda_stream);

/* Kernel launches issued by this ctx since spiral_init (host counter). */
int64_t spiral_launch_count(const spiral_ctx *ctx);

/* Synchronises the device and returns SPIRAL_OK, SPIRAL_ERR_TIMEOUT or SPIRAL_ERR_DEVICE_CHECK
 * according to the device status word (which it then clears); *detail_out (optional) receives
 * the raw word.  After a finding the results of the steps since the last clean status are not to be
 * trusted (a bad token id was replaced by token 0, a bad page by page 0, a kernel gave up half way):
 * roll the games back with spiral_kv_truncate.  The call re-arms the library's cross-kernel scratch,
 * so the context can be used again. */
int spiral_last_status(spiral_ctx *ctx, int32_t *detail_out);

/* Frees host and device memory owned by the library.  Either argument may be NULL.  Synchronises. */
void spiral_free(spiral_ctx *ctx, spiral_kv *kv);

const char *spiral_strerror(int code);
const char *spiral_last_cuda_error(void);   /* text of the most recent CUDA failure on this thread */

#ifdef __cplusplus
}
#endif
#endif /* SPIRAL_H */
