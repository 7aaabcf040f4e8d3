/*
 * gm.h - C ABI of libgm: one speculative-decoding rollout step on one B200 (sm_100a).
 *
 * The step is the draft-then-verify cycle of the paper's Sec. 2.2: a recurrent one-layer MTP
 * draft head (App. B.1 "MTP Architecture") proposes K tokens, the target decoder verifies all
 * K+1 positions in one batched forward against a paged per-sequence KV cache, and speculative
 * rejection sampling (Eq. 1) accepts a prefix and draws the final token from the corrected
 * distribution norm(max(0, p - q)) or, on full acceptance, from p_{K+1}.
 *
 * Conventions
 *  - Every pointer is a DEVICE pointer owned by the caller unless marked "host".  The library
 *    owns only what gm_init allocates (workspaces, tensor maps, a status word) and frees it in
 *    gm_destroy.  Nothing passed to a call is retained after the call's kernels are enqueued,
 *    except the weight pointers given to gm_init, which must stay valid until gm_destroy.
 *  - All work is enqueued on the CUDA stream given to gm_init.  Calls return after enqueueing;
 *    gm_last_status is the only call that synchronises.
 *  - Matrices are row-major bf16 [out_features, in_features].  Token ids, lengths, page ids are
 *    int32.  Probabilities and debug dumps are fp32.
 *  - Every call returns 0 or a negative GM_ERR_* code.  Arguments are validated on the host
 *    before anything is launched.  Conditions only the device can see (a sequence that runs out
 *    of pages, a page id outside the pool, a bounded wait that expired) set a sticky bit in the
 *    device status word and the offending rows are skipped; gm_last_status reports it.
 *
 * Per-sequence state (struct gm_state).  The committed tokens are x[0..Len-1].  The target
 * cache holds positions 0..Len-2 (kv_len = Len-1): the last committed token has not been fed to
 * the target yet.  The head consumes pairs (H_{i-1}, x_i) - the target hidden state that
 * produced token x_i and that token - and stores pair i at head-cache position i-1, so after
 * the first draft application the head cache also holds positions 0..Len-2.  The pairs the head
 * has not consumed yet are "pending": pending_n[b] of them (1 after a prefill, a+1 after a
 * cycle that accepted a drafts), oldest first; pending_tok[b][pending_n[b]-1] is x[Len-1].
 *
 * KV pool layout: bf16 [layer][2 (K,V)][page][kv_head][16 slots][head_dim]; page_table[b][i] is
 * the physical page of positions 16 i .. 16 i + 15 of sequence b.  Slots that were never
 * written must hold finite values (zero-fill the pool once).
 */
#ifndef GM_H_
#define GM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GM_OK                 0
#define GM_ERR_INVALID_ARG   (-1)   /* null pointer, batch/k out of range, bad shape            */
#define GM_ERR_UNSUPPORTED   (-2)   /* k > max_k, temperature <= 0, page_size != 16, vocab % 8  */
#define GM_ERR_KV_CAPACITY   (-3)   /* a row's pages cannot hold kv_len + k + 1 (device-seen)   */
#define GM_ERR_CUDA          (-4)   /* a CUDA runtime / driver call failed                      */
#define GM_ERR_DEVICE_TIMEOUT (-5)  /* a bounded device-side wait expired (device-seen)         */
#define GM_ERR_BAD_PAGE      (-6)   /* a page id outside the pool (device-seen)                 */
#define GM_ERR_NO_EXTENSION  (-7)   /* not an sm_100 device                                     */
#define GM_ERR_SCRATCH_LIMIT (-8)   /* request larger than the static scratch of a no-alloc call */
#define GM_ERR_OVERRUN       (-9)   /* a guard word behind a library workspace was overwritten   */

#define GM_MAX_K 7
#define GM_PAGE  16

/* gm_config.flags */
#define GM_FLAG_SIMPLE_GEMM 1       /* debug: route every GEMM through the plain mma.sync kernel */
#define GM_FLAG_SAMPLER_CLUSTER 2   /* always map the sampler as one 8-CTA cluster per sequence  */
#define GM_FLAG_SAMPLER_STREAM 4    /* always map the sampler as one CTA per sequence            */
#define GM_FLAG_SAMPLER_FLOW 16     /* always map the sampler as one vocabulary slice of every row per CTA */
#define GM_FLAG_GRAPH 8             /* gm_spec_step, gm_spec_step_host and gm_rollout_run replay a
                                       captured CUDA graph of one cycle (needs a context created on a
                                       stream of its own: on a default stream the flag has no effect) */

typedef struct gm_ctx gm_ctx;       /* opaque */

typedef struct {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
  int32_t page_size;                /* must be 16                                        */
  int32_t max_batch;                /* largest batch any call will use                   */
  int32_t max_k;                    /* largest drafting depth, <= GM_MAX_K               */
  int32_t max_pages_per_seq;        /* row length of both page tables                    */
  int32_t num_pages;                /* physical pages in the target pool                 */
  int32_t head_num_pages;           /* physical pages in the draft-head pool             */
  float   rope_base;                /* rotary base (1e4)                                 */
  float   rms_eps;                  /* RMSNorm epsilon (1e-6)                            */
  int32_t flags;
} gm_config;

/* One decoder layer.  wqkv rows: all query heads, then all key heads, then all value heads.
 * w_gate_up rows are interleaved: row 2i = gate_i, row 2i+1 = up_i.
 * The last three members select the decoder-layer family (App. B.1) and may each be NULL:
 * b_qkv is a bias added to the fused projection (same row order as wqkv); q_norm / k_norm are
 * the weights of an RMSNorm over head_dim applied to every query / key head after the bias and
 * before the rotary embedding (both or neither).                                           */
typedef struct {
  const void *ln1;                  /* [d]                                  */
  const void *wqkv;                 /* [(n_q + 2 n_kv) head_dim, d]         */
  const void *wo;                   /* [d, n_q head_dim]                    */
  const void *ln2;                  /* [d]                                  */
  const void *w_gate_up;            /* [2 d_ffn, d]                         */
  const void *w_down;               /* [d, d_ffn]                           */
  const void *b_qkv;                /* [(n_q + 2 n_kv) head_dim] or NULL    */
  const void *q_norm;               /* [head_dim] or NULL                   */
  const void *k_norm;               /* [head_dim] or NULL                   */
} gm_layer_weights;

/* Model weights (App. B.1: the head has neither embedding nor output projection and takes
 * both from the backbone; its two inputs go through separate RMSNorms, are concatenated
 * [embedding ; hidden] and projected by a bias-free linear layer).  A head trained with the
 * opposite order [hidden ; embedding] is loaded by swapping the two column halves of
 * head_proj, as the paper's own loader does.                                              */
typedef struct {
  const void *embed;                /* [vocab, d]                           */
  const void *lm_head;              /* [vocab, d]                           */
  const void *final_norm;           /* [d]                                  */
  const gm_layer_weights *layers;   /* HOST array [n_layers]                */
  const void *head_enorm;           /* [d]   RMSNorm of the token embedding */
  const void *head_hnorm;           /* [d]   RMSNorm of the hidden state    */
  const void *head_proj;            /* [d, 2 d]                             */
  const void *head_final_norm;      /* [d]                                  */
  gm_layer_weights head_layer;
} gm_weights;

typedef struct {
  int32_t  batch;                   /* B <= max_batch                                   */
  int32_t *kv_len;                  /* [B]   entries in the target cache = Len - 1      */
  int32_t *page_table;              /* [B, max_pages_per_seq]                           */
  void    *kv_pool;                 /* bf16 [n_layers][2][num_pages][n_kv][16][hd]      */
  int32_t *head_page_table;         /* [B, max_pages_per_seq]                           */
  void    *head_kv_pool;            /* bf16 [1][2][head_num_pages][n_kv][16][hd]        */
  int32_t *pending_n;               /* [B]   1 .. max_k+1                               */
  int32_t *pending_tok;             /* [B, max_k+1]                                     */
  void    *pending_hidden;          /* bf16 [B, max_k+1, d]                             */
} gm_state;

/* Create a context.  Validates the configuration, allocates workspaces sized for max_batch and
 * max_k, encodes the weight tensor maps, builds the rotary table.  `cuda_stream` is a
 * cudaStream_t (NULL = the default stream).  Fails with GM_ERR_NO_EXTENSION on a device that is
 * not compute capability 10.x.                                                              */
int gm_init(gm_ctx **out, const gm_config *cfg, const gm_weights *w, void *cuda_stream);
void gm_destroy(gm_ctx *ctx);

/* Prompt prefill: the state a rollout starts from (App. B.2: prompts of at most 1024 tokens; App. D.2:
 * the rollout-time hidden states of the prompt prefill the draft head).  For every sequence b with prompt
 * x[0..L_b-1], L_b = prompt_len[b]:
 *   - the backbone runs causally over the prompt and fills target-cache positions 0..L_b-1;
 *   - the draft head runs over the pairs (H_{i-1}, x_i), i = 1..L_b-1, filling head-cache positions 0..L_b-2;
 *   - the first response token x[L_b] is drawn from softmax(logits(H_{L_b-1}) / T) with the uniform
 *     u24_first[b], or Philox (key = seed, counter = (slot 16 >> 2, row, 0, 0)) when u24_first is NULL;
 *   - kv_len[b] = L_b, pending_n[b] = 1, pending pair = (H_{L_b-1}, x[L_b]).
 * The prompts are processed max_k + 1 positions per sequence and pass, every pass through the kernels of the
 * verify and draft phases; ceil(max_prompt_len / (max_k + 1)) passes.
 *   prompt_tok  device int32 [B, prompt_stride], row b holds L_b tokens;  prompt_len device int32 [B];
 *   max_prompt_len  host value >= every L_b (a longer or empty prompt raises GM_ERR_KV_CAPACITY in
 *                   gm_last_status and its sequence is left untouched);
 *   first_token device int32 [B] out or NULL;  dbg_p fp32 [B, V] out or NULL (the distributions drawn from).
 * The page tables of `st` must cover max_prompt_len + max_k + 1 positions (else GM_ERR_KV_CAPACITY).     */
int gm_prefill(gm_ctx *ctx, gm_state *st, const int32_t *prompt_tok, const int32_t *prompt_len,
               int prompt_stride, int max_prompt_len, float temperature, const uint32_t *u24_first,
               uint64_t seed, int32_t *first_token, float *dbg_p);

/* ---- A whole rollout: cycles until every response has ended (App. B.2: responses capped at 8192 / 16384
 * tokens).  A response is the token the prefill drew followed by what each cycle commits; it ends with the
 * first eos_token (kept) or when it holds max_new tokens; what a cycle commits beyond either is dropped.  A
 * finished row sits out the remaining cycles: it gets no queries and no pages in any phase, the sampler
 * skips it, and its state (kv_len, pending_*, caches) stays as it was.  A row's uniforms depend on seed,
 * step and row only, so its response does not depend on when the others end - up to floating-point
 * rounding in attention at scale: the pages of all running rows are cut into equal ranges over the SMs,
 * so which partial results are merged for a row shifts when another row leaves (with fewer pages than
 * SMs every range is one page and the results are bit-identical).  All pointers are device memory.      */
typedef struct {
  int32_t *out_tok;                 /* [B, out_stride] responses                                         */
  int32_t *out_len;                 /* [B] tokens held by each response                                  */
  int32_t *finished;                /* [B] 0 running, 1 ended with eos_token, 2 reached max_new          */
  int32_t *n_running;               /* [1] rows still running after the last call                        */
  int32_t  out_stride;              /* >= max_new                                                        */
  int32_t  eos_token;               /* < 0: none                                                         */
  int32_t  max_new;                 /* response cap, >= 1                                                */
} gm_rollout;

/* After gm_prefill (or with any state whose pending_tok[b][0] is the first response token): response b =
 * [that token], finished / n_running set by the rules above.                                            */
int gm_rollout_begin(gm_ctx *ctx, const gm_state *st, const gm_rollout *ro);
/* One cycle (gm_spec_step) over the running rows, then the append of what it committed.  With the page
 * allocator on (gm_pages_reset) it first reserves pages for kv_len + k + 1 positions of every running row
 * and afterwards returns the pages of the rows that finished.                                           */
int gm_rollout_step(gm_ctx *ctx, gm_state *st, const gm_rollout *ro, int k, float temperature,
                    uint64_t seed, uint64_t step);
/* Host loop: gm_rollout_step with step = first_step, first_step + 1, ... until no row is running or
 * max_steps cycles ran.  n_running is read back (one stream synchronisation) every check_every cycles, so
 * up to check_every - 1 cycles may run with every row sitting out.  steps_run / rows_running: host
 * outputs, may be NULL.  With GM_FLAG_GRAPH the first call captures one cycle (all its launches,
 * with their programmatic dependencies, the page reserve / release and the append) into a CUDA graph and
 * every cycle is one graph launch; the step index then lives in device memory and is advanced by the
 * append kernel.  The graph is re-captured when the state, the rollout buffers, k, the temperature, the
 * seed, top-p or the hidden-state capture change.  Results are bit-identical to the host-launched loop.  The context must have been
 * created on a stream of its own: the default streams cannot be captured, and the flag is ignored there. */
int gm_rollout_run(gm_ctx *ctx, gm_state *st, const gm_rollout *ro, int k, float temperature,
                   uint64_t seed, uint64_t first_step, int max_steps, int check_every,
                   int32_t *steps_run, int32_t *rows_running);

/* ---- Page allocator (the paper's serving engine allocates cache pages as sequences grow; no passage
 * describes it).  The context keeps one stack of free page ids per pool (target, draft head).
 *   gm_pages_reset    every page free, both page tables of `st` emptied (-1), switches the allocator on;
 *   gm_pages_reserve  every row (finished[b] == 0 when finished is given) receives pages until its two
 *                     tables cover length[b] + extra positions (length NULL = kv_len); a row that needs
 *                     more than max_pages_per_seq pages, or an empty stack, raises GM_ERR_KV_CAPACITY in
 *                     gm_last_status;
 *   gm_pages_release  rows with finished[b] != 0 hand their pages back;
 *   gm_pages_free_count  free pages per pool (host outputs; synchronises the stream).
 * Rows take their slices of the stack in row order (a prefix sum over the rows), so the page assignment
 * is the same on every run.  Batches of at most 1024 rows.  A context serves one state at a time while
 * the allocator is on.                                                                                  */
int gm_pages_reset(gm_ctx *ctx, gm_state *st);
int gm_pages_reserve(gm_ctx *ctx, gm_state *st, const int32_t *length, int extra, const int32_t *finished);
int gm_pages_release(gm_ctx *ctx, gm_state *st, const int32_t *finished);
int gm_pages_free_count(gm_ctx *ctx, int32_t *target_free, int32_t *head_free);

/* Draft phase (App. E, restart equations).  Application 1 runs the head over the pending pairs,
 * overwriting head-cache entries of the previous chain; applications 2..k feed the head its own
 * output and the previous draft.  After each application q_j = softmax(logits / T) and d_j is
 * drawn from q_j by the integer inverse CDF.
 *   u24_draft  [B, k] 24-bit uniforms, or NULL to generate them from Philox4x32-10
 *              (key = seed, counter = (slot >> 2, row, step lo, step hi), slot = j-1).
 *   draft_tok  [B, k] out.   draft_logits bf16 [B, k, V] out.   dbg_q fp32 [B, k, V] out or NULL.
 * Does not change kv_len / pending_*.                                                        */
int gm_draft(gm_ctx *ctx, const gm_state *st, int k, float temperature,
             const uint32_t *u24_draft, uint64_t seed, uint64_t step,
             int32_t *draft_tok, void *draft_logits, float *dbg_q);

/* Verify phase (Sec. 2.2, Eq. 2): target forward over [x[Len-1], d_1..d_k] at positions
 * kv_len .. kv_len+k; appends their keys/values to the pages.
 *   target_logits bf16 [B, k+1, V] out;  target_hidden bf16 [B, k+1, d] out (residual stream
 *   before the final norm: the feature the head consumes).  Does not change kv_len.          */
int gm_verify(gm_ctx *ctx, const gm_state *st, int k, const int32_t *draft_tok,
              void *target_logits, void *target_hidden);

/* Accept phase (Sec. 2.2, Eq. 1).  p_j = softmax(target_logits[j-1] / T), q_j likewise.
 * d_j is accepted iff p_j(d_j) >= q_j(d_j) or fl32(u_j q_j(d_j)) < p_j(d_j), u_j = u24_j 2^-24;
 * a = accepted prefix length; next_token is drawn from max(0, p_{a+1} - q_{a+1}) (a < k) or from
 * p_{k+1} (a == k) through 64-bit integer weights: w[v] = trunc(r[v] 2^44) for r[v] > 0 else 0,
 * W = sum w, t = (u24 W) >> 24, token = the first v whose inclusive prefix sum exceeds t.  If the
 * residual quantises to nothing the draw is repeated on p_{a+1}.
 *   u24_accept [B, k+1]: k accept uniforms then the final one; NULL = Philox slots 8+j-1 and 16.
 *   accept_len [B] out (0..k), next_token [B] out.
 *   dbg_p fp32 [B, k+1, V], dbg_q fp32 [B, k, V]: the probabilities the decisions used, or NULL.
 *   commit_state != 0 (needs st and target_hidden): kv_len += a+1, pending_n = a+1,
 *   pending_tok = d_1..d_a, next_token, pending_hidden = target_hidden rows 0..a.
 *   With commit_state == 0, st and target_hidden may be NULL (sampler-only use).             */
int gm_accept(gm_ctx *ctx, gm_state *st, int batch, int k, float temperature,
              const void *target_logits, const void *draft_logits, const int32_t *draft_tok,
              const uint32_t *u24_accept, uint64_t seed, uint64_t step,
              int32_t *accept_len, int32_t *next_token,
              float *dbg_p, float *dbg_q, const void *target_hidden, int commit_state);

/* One whole cycle: gm_draft, gm_verify, gm_accept(commit_state = 1) on library-owned logit
 * buffers, bit-for-bit the same as the three calls.  draft_tok [B, k] may be NULL.  With
 * GM_FLAG_GRAPH the cycle is captured once per (state, k, temperature, seed, output pointers)
 * and every call is one graph launch plus a one-thread kernel that stores the step index.    */
int gm_spec_step(gm_ctx *ctx, gm_state *st, int k, float temperature, uint64_t seed,
                 uint64_t step, int32_t *accept_len, int32_t *next_token, int32_t *draft_tok);

/* Nucleus (top-p) sampling of the target (the paper's evaluation uses top-p 0.7, its rollouts
 * top-p 1 = none, Sec. 4 / App. B).  gm_set_top_p stores the value in the context (default 1);
 * while it is below 1, gm_accept - and therefore gm_spec_step and its variants - first
 * truncates every target row to its top-p set and renormalises, so the committed tokens
 * follow the truncated target law; the head's distributions are not truncated, and the
 * cycle record still holds the full distribution.  The first call with top_p < 1 allocates a
 * buffer of max_batch (max_k + 1) V bf16.  top_p outside (0, 1] -> GM_ERR_UNSUPPORTED.
 *
 * The set is order-free: with e[v] = 2^((x[v] - max) log2(e) / T) in fp32, w[v] = trunc(e[v] 2^44),
 * W = sum w and tp24 = round(top_p 2^24), v is kept iff
 *     (sum of w over entries whose logit is larger than x[v]) * 2^24  <  tp24 * W,
 * i.e. tokens in decreasing probability while the mass before them is below top_p, every
 * member of a tie at the cut kept.
 *
 * gm_nucleus is the truncation as a stand-alone call: logits bf16 [rows, V] in, out bf16
 * [rows, V] = the same rows with entries outside the set replaced by -inf (out must not alias
 * logits); dbg_weight fp32 [rows, V] receives e or is NULL.  It needs top_p < 1.             */
int gm_set_top_p(gm_ctx *ctx, float top_p);
int gm_nucleus(gm_ctx *ctx, const void *logits, int rows, float temperature, float top_p,
               void *out, float *dbg_weight);

/* Draw one token per row from softmax(logits / T) by the integer inverse CDF (the draw of the
 * draft phase as a stand-alone call).  logits bf16 [rows, V]; u24 [rows]; out_tok [rows];
 * dbg_prob fp32 [rows, V] or NULL.                                                           */
int gm_draw(gm_ctx *ctx, const void *logits, int rows, float temperature, const uint32_t *u24,
            int32_t *out_tok, float *dbg_prob);

/* Host-buffer form of the cycle, for callers that keep no device memory of their own besides the
 * state: copies the uniforms from HOST arrays (u24_draft_host [B, k], u24_accept_host [B, k+1]; both
 * NULL = Philox from seed/step), runs the cycle, copies accept_len [B], next_token [B] and (if not
 * NULL) draft_tok [B, k] back to HOST arrays and waits for the stream.  Pinned host memory makes the
 * copies asynchronous.                                                                        */
int gm_spec_step_host(gm_ctx *ctx, gm_state *st, int k, float temperature, uint64_t seed,
                      uint64_t step, const uint32_t *u24_draft_host, const uint32_t *u24_accept_host,
                      int32_t *accept_len_host, int32_t *next_token_host, int32_t *draft_tok_host);

/* The record a cycle leaves for the head update (App. D.2 "Recording in Rollout"): the backbone hidden state
 * at the cycle's start, the k drafts, the verification distributions kept as the target's top-64
 * log-probabilities in bf16 WITH full-vocabulary normalisation (not renormalised over the retained set), the
 * accepted length with the final token counted, and the absolute position of the start.  Entries of a row
 * are ordered by logit descending, ties by token id ascending; rows with fewer than 64 tokens are padded with
 * index -1 / log-probability -inf.  All pointers are device buffers owned by the caller.                  */
typedef struct {
  void    *start_hidden;            /* bf16 [B, d]      hidden state the first draft application consumed   */
  int32_t *start_pos;               /* [B]              context length at which drafting starts (kv_len+1)  */
  int32_t *drafts;                  /* [B, k]                                                                */
  void    *top_logprob;             /* bf16 [B, k, 64]  log p_j at the target's 64 largest logits, j = 1..k  */
  int32_t *top_index;               /* [B, k, 64]       their token ids                                      */
  int32_t *accepted;                /* [B]              accepted drafts + 1                                  */
} gm_record;
/* gm_record_begin: call before the cycle (fills start_hidden, start_pos from the state).
 * gm_record_end:   call after gm_accept (fills drafts, top_logprob, top_index, accepted from the cycle's
 *                  target logits [B, k+1, V], draft tokens [B, k] and accept_len [B]).
 * gm_spec_step_rec: gm_spec_step with both calls around it; the cycle itself is unchanged bit for bit.       */
int gm_record_begin(gm_ctx *ctx, const gm_state *st, gm_record *rec);
int gm_record_end(gm_ctx *ctx, int batch, int k, float temperature, const void *target_logits,
                  const int32_t *draft_tok, const int32_t *accept_len, gm_record *rec);
int gm_spec_step_rec(gm_ctx *ctx, gm_state *st, int k, float temperature, uint64_t seed, uint64_t step,
                     int32_t *accept_len, int32_t *next_token, int32_t *draft_tok, gm_record *rec);

/* ---- Forward pass of the draft-head update on recorded cycles (Sec. 3.2 Eq. 4; Sec. 3.3-3.4 Eq. 5-9; App. D.2,
 * D.3).  The recorded inputs: per sequence its committed tokens x[0..L-1] and the rollout-time target hidden
 * states H_0..H_{L-2} (H_i produced x_{i+1}); per cycle a gm_record entry.  Forward pass, and the gradient of
 * the objective with respect to the reconstructed logits; the backward pass through the head is not part of it.
 *
 * gm_head_prefill rebuilds the head cache of every sequence from its recorded pairs (H_{i-1}, x_i),
 *   i = 1..L_b-1, at head positions 0..L_b-2 (the shared prefix every chain attends).
 *   seq_hidden bf16 [B, hid_stride, d];  seq_tok int32 [B, tok_stride];  seq_len int32 [B] = L_b (device);
 *   max_len host value >= every L_b;  hid_stride >= max_len - 1, tok_stride >= max_len.
 *
 * gm_reconstruct replays the draft chain of n_cycles recorded cycles (Eq. 4): chain r belongs to sequence
 *   cycle_seq[r], starts at context length rec->start_pos[r] from the hidden rec->start_hidden[r], and feeds
 *   back the recorded drafts rec->drafts[r]; nothing is sampled.  All chains advance together, one draft
 *   application per depth, max_batch chains per pass.  Every chain sees the shared prefix up to its start
 *   and only its own draft entries: it runs as a virtual sequence whose page-table row shares its sequence's
 *   head-cache pages before the page of its first entry and owns the two pages scratch_pages[r][0..1] (ids
 *   in the head pool that no sequence uses) from there on.  draft_logits bf16 [n_cycles, k, V] out.
 *   The state's head cache must have been prefilled (gm_head_prefill, or the rollout that made the record);
 *   it is not modified outside the scratch pages.
 *
 * gm_overlap: alpha[r, j] = sum over the record's 64 retained tokens of min(p, q) + min(1 - sum p, 1 - sum q)
 *   (Eq. 5 on the sparsified record, App. D.2), q = softmax(draft_logits / T) over the full vocabulary.
 *   alpha fp32 [n_cycles, k] out.  lse fp32 [n_cycles, k] out, or NULL: logsumexp(draft_logits / T) of every
 *   row, which gm_dca_grad takes back to skip its own statistics pass.
 *
 * gm_dca_loss: loss[r] = -log sum_{l=1..min(accepted[r], k)} prod_{i<=l} alpha[r, i] (Eq. 9; accepted =
 *   accepted drafts + 1 = the first rejected position, k + 1 if none), evaluated in the log domain (Eq. 7);
 *   mean[0] = their mean, added in a fixed order.  A chain whose first overlap is 0 gives +inf.
 *
 * gm_dca_grad (first step of the backward pass): grad_logits bf16 [n_cycles, k, V] = d mean / d draft_logits.
 *   Per row (r, j): dL/dalpha = -(prod_{i<j} alpha_i) D_j / M with the chain sums cut at min(accepted[r], k)
 *   (Eq. 8 under the gate of Eq. 9), divided by n_cycles; rows at or after the cut, and rows of a chain whose
 *   first overlap is 0, are written as zeros.  alpha is piecewise linear in q: slope 1 on a retained token
 *   where q < p, minus 1 on every retained token when the residual bin of q is the smaller one, 0 on all
 *   other tokens and at ties; the softmax gives d alpha / d logit_v = q_v (slope_v - sum_e q_e slope_e) / T.
 *   alpha and accepted are the arrays gm_overlap and the record produced; lse is gm_overlap's second output
 *   for the same logits and temperature, or NULL (recomputed); draft_logits is only read.                */
/* Rollout-time capture of the target hidden states (App. D.2: every sequence also stores the rollout-time
 * target hidden states of the prompt and of all committed tokens).  While seq_hidden (device bf16
 * [max_batch, stride, d]) is set, gm_prefill writes H_0..H_{L-1} of every prompt and every committing
 * gm_accept / gm_spec_step* / gm_rollout_step writes the hidden states of the positions it commits, so that
 * row b holds H_i at index i - what gm_head_prefill consumes.  Positions >= stride are dropped.  NULL
 * switches the capture off (a cycle captured as a CUDA graph is captured again when the setting changes).  */
int gm_capture_hidden(gm_ctx *ctx, void *seq_hidden, int stride);
int gm_head_prefill(gm_ctx *ctx, gm_state *st, const void *seq_hidden, int hid_stride,
                    const int32_t *seq_tok, int tok_stride, const int32_t *seq_len, int max_len);
int gm_reconstruct(gm_ctx *ctx, gm_state *st, int n_cycles, int k, const int32_t *cycle_seq,
                   const gm_record *rec, const int32_t *seq_tok, int tok_stride,
                   const int32_t *scratch_pages, void *draft_logits);
/* gm_reconstruct that also returns the head states: head_states fp32 [n_cycles, k, d] out (or NULL) receives
 * g_j of every chain and depth, the state the head's final norm and the LM head turn into draft_logits[r, j]
 * (Eq. 4) - the point the backward pass re-enters the head at.                                             */
int gm_reconstruct_states(gm_ctx *ctx, gm_state *st, int n_cycles, int k, const int32_t *cycle_seq,
                          const gm_record *rec, const int32_t *seq_tok, int tok_stride,
                          const int32_t *scratch_pages, void *draft_logits, float *head_states);
int gm_overlap(gm_ctx *ctx, int n_cycles, int k, float temperature, const void *draft_logits,
               const gm_record *rec, float *alpha, float *lse);
int gm_dca_loss(gm_ctx *ctx, int n_cycles, int k, const float *alpha, const int32_t *accepted,
                float *loss, float *mean);
int gm_dca_grad(gm_ctx *ctx, int n_cycles, int k, float temperature, const void *draft_logits,
                const gm_record *rec, const float *alpha, const float *lse, const int32_t *accepted,
                void *grad_logits);
/* Second step of the backward pass (Alg. 1, "update phi"): from the logits back to the head states.  The head's
 * logits are LMhead(RMSNorm(g; head final norm)) with the backbone's LM head (App. B.1), which the head update
 * leaves fixed, so no weight gradient is formed here.
 *   grad_logits  device bf16 [rows, V], rows = n_cycles * k: gm_dca_grad's output
 *   grad_normed  device fp32 [rows, d] out: dL/dy = grad_logits x W_lm for the normed state y (one projection with
 *                the vocabulary as its contraction dimension, fp32 accumulation)
 *   head_states  device fp32 [rows, d] in, grad_states device fp32 [rows, d] out: dL/dg through the norm,
 *                r (w dy) - g r^3 mean(g w dy) with r = (mean(g^2) + eps)^(-1/2); both NULL = skip this step.
 *                This is the derivative through the logits of the state's own position; the terms that reach
 *                g_j through g_{j+1} (Eq. 4) belong to the backward pass of the head layer, which is not built.
 * The projection reads a transposed copy [d, V] of the LM head that the context makes on the first call (d * V
 * bf16 of device memory, kept until gm_destroy); refresh_weights != 0 remakes it, for a caller that has rewritten the
 * LM head's weights in place since.  V % 64 != 0 returns GM_ERR_UNSUPPORTED.                                   */
int gm_head_state_grad(gm_ctx *ctx, int rows, const void *grad_logits, const float *head_states,
                       float *grad_normed, float *grad_states, int refresh_weights);
/* Third step of the backward pass: through the feed-forward half of the head's decoder layer (App. B.1: the head is one
 * more layer of the backbone's shape),  g = x + W_d (silu(W_g u) * (W_u u)),  u = RMSNorm(x; ln2).
 *   x    device fp32 [rows, d]: the block's input (the residual stream after the head layer's attention)
 *   dg   device fp32 [rows, d]: dL/dg (for the rows' own logits: gm_head_state_grad's grad_states)
 *   dx   device fp32 [rows, d] out: dL/dx = dg + the path through the block
 *   dw_gate_up  device fp32 [2 F, d] out, rows interleaved like the packed weight (2f = gate feature f, 2f + 1 = up f);
 *   dw_down     device fp32 [d, F] out;  dln2  device fp32 [d] out: the gradients of the block's parameters, summed
 *               over the rows (the first of the head's own weights the update touches; Alg. 1, "update phi")
 * The forward values it needs (u and the gate / up pre-activations) are recomputed from x in bf16 as the forward pass
 * computes them; products run on the projection kernel (fp32 accumulation, bf16 operands: dg, the activation
 * gradients and the recomputed activations are rounded to bf16 before they enter a product).  Transposed copies of the
 * two weight matrices (3 d F bf16) and scratch for `rows` rounded up to 64 are allocated on first use and kept until
 * gm_destroy; refresh_weights != 0 remakes the copies after the weights have been rewritten in place.
 * d % 64 != 0, F % 64 != 0 or GM_FLAG_SIMPLE_GEMM: GM_ERR_UNSUPPORTED.                                         */
int gm_head_ffn_backward(gm_ctx *ctx, int rows, const float *x, const float *dg, float *dx, float *dw_gate_up,
                         float *dw_down, float *dln2, int refresh_weights);
/* Backward of gm_attention's core (scores, softmax, weighted values) - the operator the attention half of the head's
 * layer needs in the update (Alg. 1, "update phi").  Same query layout, pool, page tables and row conventions as
 * gm_attention; for every valid query row (j < q_count[b]) with output gradient dO and P = softmax(q k^T / sqrt(hd)):
 *   dP_j = dO . v_j,  dS_j = P_j (dP_j - sum_i P_i dP_i),  dq = sum_j dS_j k_j / sqrt(hd),
 *   dk_j += dS_j q / sqrt(hd),  dv_j += P_j dO      (a KV head collects the terms of every query head of its group)
 *   dout     device fp32 [batch * q_stride][n_q * head_dim]: gradient of gm_attention's `out` rows
 *   dq       device fp32 [batch * q_stride][n_q * head_dim] out (rows j >= q_count[b] are zero); with respect to the
 *            queries as gm_attention receives them (rotary embedding already applied)
 *   dk_pool, dv_pool  device fp32 [num_pages][n_kv][16][head_dim]: gradient planes laid out like one layer of the pool,
 *            ACCUMULATED with atomic additions (the caller zeroes them): sequences whose page tables share pages - the
 *            chains of one sequence share its committed prefix - add into the same entries; with respect to the cached
 *            keys (after their rotary embedding) and values, whichever pass wrote them
 * Reads the cache in bf16, computes in fp32; two passes over a row's keys (statistics, then gradients).
 * q_stride > 8, more than 8 query heads per KV head, head_dim other than 64 / 128: GM_ERR_UNSUPPORTED.           */
int gm_attention_backward(gm_ctx *ctx, const void *q, const float *dout, const void *kv_pool, int pool_layers,
                          int num_pages, int layer, const int32_t *page_table, const int32_t *q_count,
                          const int32_t *q_base, int batch, int q_stride, float *dq, float *dk_pool, float *dv_pool);
/* The attention half of the head's decoder layer, backward (App. B.1; Alg. 1, "update phi"):
 *   xmid = x + W_o attention(rope(norm_q(q)), cache),  (q, k, v) = W_qkv RMSNorm(x; ln1) (+ bias),  the rows' own
 *   rope(norm_k(k)), v being the cache entries at their positions.
 * A pass is `batch` sequences of up to q_stride rows, row j of sequence b at position q_base[b] + j, j < q_count[b]
 * (the conventions of gm_attention); passes that share cache entries are walked from the last one written to the first.
 *   x        device fp32 [batch * q_stride, d]: the layer's input rows (the head's projected input z)
 *   dxmid    device fp32 [batch * q_stride, d]: dL/d xmid (gm_head_ffn_backward's dx); zero in rows j >= q_count[b]
 *   kv_pool  device bf16 [1][2][num_pages][n_kv][16][head_dim]: the head's cache as the forward pass left it (read only)
 *   dk_pool, dv_pool  device fp32 [num_pages][n_kv][16][head_dim], IN and OUT: on entry the gradient the rows of LATER
 *            passes left on the cache entries (zero before the first call); these rows' terms are added
 *            (gm_attention_backward), after which the rows' own entries are complete and are read back
 *   dx       device fp32 [batch * q_stride, d] out: dL/dx = dxmid + the path through the attention half
 *   dw_qkv   device fp32 [(n_q + 2 n_kv) head_dim, d] out;  dw_o  device fp32 [d, n_q head_dim] out;  dln1  fp32 [d] out
 *   db_qkv   device fp32 [(n_q + 2 n_kv) head_dim] out - required iff the layer has projection biases, else NULL
 *   dqk_norm device fp32 [2 head_dim] out (query norm, then key norm) - required iff the layer has head norms, else NULL
 * The parameter gradients are this pass's sums over its rows (the caller adds passes up).  Forward values (the normed
 * rows, the projection, the rotated queries, the attention output) are recomputed in bf16 as the forward pass computes
 * them, in the context's own workspaces - not to be interleaved with a cycle in flight on the same context; products run
 * on the projection kernel with bf16 operands and fp32 accumulation.  Transposed copies of W_o and W_qkv and scratch for
 * the rows rounded up to 64 are allocated on first use and kept until gm_destroy; refresh_weights != 0 remakes the copies.
 * GM_ERR_UNSUPPORTED: GM_FLAG_SIMPLE_GEMM, d, n_q head_dim or (n_q + 2 n_kv) head_dim not a multiple of 64, head_dim
 * other than 64 / 128, more than 8 query heads per KV head, q_stride > min(8, max_k + 1), or more rows than a prefill
 * pass of the context holds.  A page outside the pool: the status word reports GM_ERR_BAD_PAGE and the row gets zeros. */
int gm_head_attn_backward(gm_ctx *ctx, const float *x, const float *dxmid, const void *kv_pool, int num_pages,
                          const int32_t *page_table, const int32_t *q_count, const int32_t *q_base, int batch, int q_stride,
                          float *dk_pool, float *dv_pool, float *dx, float *dw_qkv, float *dw_o, float *dln1, float *db_qkv,
                          float *dqk_norm, int refresh_weights);
/* The whole backward pass of the head update over recorded cycles (Alg. 1, "update phi"; Eq. 4-9): the gradient of the
 * mean objective with respect to every parameter of the head, given its gradient with respect to the reconstructed
 * logits.  Call order: gm_head_prefill and gm_reconstruct / gm_reconstruct_states (the head's cache over the committed
 * prefixes, the chains' logits), gm_overlap + gm_dca_grad (grad_logits), then this call with the SAME state, cycles,
 * record, tokens and scratch pages.  It replays the chains a chunk of max_batch at a time (the states they produce are
 * the forward pass's, the kernels being deterministic), takes every application from the last draft back to the
 * first through gm_head_state_grad, gm_head_ffn_backward, gm_head_attn_backward and gm_head_input_backward - a state's
 * gradient collecting the term through its own logits and the term through the next application's input, a cache
 * entry's gradient collecting the terms of every later row that read it - moves what the chains left on the copied
 * part of their private boundary pages to the shared originals, and finishes with the pass over the committed prefixes,
 * whose rows receive gradient only through their cache entries.
 *   grad_logits       device bf16 [n_cycles, k, vocab] (gm_dca_grad)
 *   seq_hidden, hid_stride, seq_len, max_len, seq_tok, tok_stride   as in gm_head_prefill / gm_reconstruct
 *   dk_pool, dv_pool  device fp32 [head_num_pages][n_kv][16][head_dim] out, or both NULL: the gradient of every head-cache
 *                     entry, shared prefix pages and private chain pages alike (a by-product; the update does not need it)
 *   out               device fp32 buffers, overwritten with the sums over all cycles
 * The result does not depend on thread scheduling: the cache entries' gradients are accumulated in 64-bit fixed point
 * (units of 2^-40) inside the call and converted into dk_pool / dv_pool at its end; every other sum runs in a fixed order.
 * Uses the context's cycle workspaces (not to be interleaved with a cycle in flight); scratch for the passes and
 * transposed copies of the head's matrices are allocated on first use and kept until gm_destroy.
 * Limits: those of the four operators (d, q_dim, n_qkv, F multiples of 64; head_dim 64 / 128; group <= 8; no
 * GM_FLAG_SIMPLE_GEMM): GM_ERR_UNSUPPORTED.  An optional output (b_qkv, qk_norm) must be given iff the layer has it.   */
typedef struct {
  float *proj;                      /* [d, 2 d]   packed order [embedding ; hidden]                                     */
  float *enorm, *hnorm, *final_norm;/* [d] each                                                                          */
  float *ln1, *ln2;                 /* [d] each                                                                          */
  float *wqkv;                      /* [(n_q + 2 n_kv) head_dim, d]                                                       */
  float *wo;                        /* [d, n_q head_dim]                                                                  */
  float *w_gate_up;                 /* [2 F, d]   rows interleaved like the packed weight                                 */
  float *w_down;                    /* [d, F]                                                                             */
  float *b_qkv;                     /* [(n_q + 2 n_kv) head_dim] or NULL                                                  */
  float *qk_norm;                   /* [2 head_dim] (query norm, key norm) or NULL                                        */
} gm_head_grads;
int gm_head_update_backward(gm_ctx *ctx, gm_state *st, int n_cycles, int k, const int32_t *cycle_seq, const gm_record *rec,
                            const int32_t *seq_tok, int tok_stride, const int32_t *scratch_pages, const void *grad_logits,
                            const void *seq_hidden, int hid_stride, const int32_t *seq_len, int max_len, float *dk_pool,
                            float *dv_pool, const gm_head_grads *out);
/* One update of the draft head on recorded cycles (Alg. 1, "update phi"), as one call: rebuilds the head's cache over
 * the committed prefixes and replays the chains with the parameters as they are now (gm_head_prefill, gm_reconstruct),
 * evaluates the objective (gm_overlap, gm_dca_loss: Eq. 5-9), takes its gradient with respect to every parameter of the
 * head (gm_dca_grad, gm_head_update_backward) and applies AdamW to every tensor of the head's group (gm_adamw_step;
 * App. B).  Arguments as in those calls, and the same numbers as those calls made one after the other - except that each
 * chunk of max_batch chains is replayed once, its overlaps, logit gradients and backward pass following directly, so no
 * [n_cycles, k, vocab] buffer exists.
 *   step         1, 2, 3, ... - the number of this update; must follow the context's previous one (GM_ERR_INVALID_ARG)
 *   lr           this update's learning rate (the caller applies the schedule: warm-up, cosine decay)
 *   mean_loss    device fp32 [1] out: the mean objective over the cycles BEFORE this update
 * The bf16 tensors the context was created with (head_proj, head_enorm, head_hnorm, head_final_norm and every tensor of
 * head_layer) are REWRITTEN IN PLACE; the backbone's tensors are read only.  fp32 master copies (initialised from the bf16
 * values at the first call), both moments, the gradients and the per-call buffers belong to the context and live until
 * gm_destroy (about 16 bytes per head parameter + 2 bytes x max_batch x max_k x vocab).  The head cache of `st` is left as the
 * rebuild with the parameters BEFORE the update wrote it.                                                               */
int gm_head_update_step(gm_ctx *ctx, gm_state *st, int n_cycles, int k, float temperature, const int32_t *cycle_seq,
                        const gm_record *rec, const int32_t *seq_tok, int tok_stride, const int32_t *scratch_pages,
                        const void *seq_hidden, int hid_stride, const int32_t *seq_len, int max_len, int step, float lr,
                        float beta1, float beta2, float eps, float weight_decay, float *mean_loss);
/* Fourth step of the backward pass: through the head's input (App. B.1),
 *   z = W_p [RMSNorm(E[token]; enorm) ; RMSNorm(hidden; hnorm)]   (the order the packed projection uses).
 *   tokens int32 [rows], hidden fp32 [rows, d]: the pairs that entered;  dz fp32 [rows, d] = dL/dz (device)
 *   dhidden fp32 [rows, d] out: dL/d hidden - for a draft application k >= 2 the hidden state is the head's own previous
 *            output g_{k-1} (Eq. 4), so this is a further term of dL/dg_{k-1}; for the first application it is the
 *            target's hidden state and is dropped
 *   dproj fp32 [d, 2 d], denorm fp32 [d], dhnorm fp32 [d] out: the gradients of the projection and of the two norm
 *            weights, summed over the rows (the embedding table is the backbone's: no gradient)
 * Same conventions as gm_head_ffn_backward: the input rows are recomputed in bf16 as the forward pass computes them, the
 * two products run on the projection kernel over a transposed copy of W_p and transposed operands, scratch is
 * allocated on first use.  d % 64 != 0 or GM_FLAG_SIMPLE_GEMM: GM_ERR_UNSUPPORTED; a token id outside the vocabulary
 * is reported by gm_last_status as GM_ERR_BAD_PAGE (like every out-of-range id) and is treated as token 0.      */
int gm_head_input_backward(gm_ctx *ctx, int rows, const int32_t *tokens, const float *hidden, const float *dz,
                           float *dhidden, float *dproj, float *denorm, float *dhnorm, int refresh_weights);
/* The update of a parameter tensor of the head (Alg. 1, "update phi"; App. B, optimizer and learning rate: AdamW on the
 * head's own parameter group).  All arrays on the device, n elements:
 *   master fp32 in/out (the parameters), param_bf16 out or NULL (the bf16 copy the forward pass reads, rewritten from
 *   the new master values), grad fp32 in, m / v fp32 in/out (first and second moments; zeros before step 1).
 *   m <- b1 m + (1 - b1) g,  v <- b2 v + (1 - b2) g^2,  p <- p (1 - lr wd) - lr (m / (1 - b1^t)) / (sqrt(v / (1 - b2^t)) + eps)
 *   with g = grad_scale * grad (1 for no clipping) and t = step >= 1.  The schedule of lr (warm-up over 10 updates,
 *   cosine decay to a tenth of the peak) is the caller's; the paper gives no moment coefficients, eps or weight decay
 *   for the head: the optimizer's usual defaults are 0.9, 0.999, 1e-8, 0.01.
 * One streaming pass (16 bytes read, 12 + 2 written per element).  beta outside [0, 1), negative lr or eps,
 * non-finite lr or grad_scale: GM_ERR_UNSUPPORTED.                                                             */
int gm_adamw_step(gm_ctx *ctx, int64_t n, float *master, void *param_bf16, const float *grad, float *m, float *v,
                  int step, float lr, float beta1, float beta2, float eps, float weight_decay, float grad_scale);


/* Dense projection out[M, N] = x[M, K] w[N, K]^T on the context's stream (bf16 in, fp32
 * accumulate; the kernel every QKV / O / FFN / LM-head projection of the step uses).
 *   out_fp32 != 0: out is fp32 [M, N]; else bf16 [M, N].  K % 64 == 0, N % 8 == 0, M >= 1.   */
int gm_gemm(gm_ctx *ctx, const void *x, const void *w, void *out, int M, int N, int K,
            int out_fp32);
/* The gate/up projection as the step runs it: y = x w^T with gate and up rows interleaved in w (row 2f = gate
 * feature f, row 2f + 1 = up feature f; the decoder's SwiGLU feed-forward, App. B.1), out bf16 [M, N / 2] = silu(y[:, 2f]) * y[:, 2f + 1],
 * fused into the projection's epilogue.  Same constraints as gm_gemm; N % 16 == 0 (else GM_ERR_UNSUPPORTED).                        */
int gm_gemm_swiglu(gm_ctx *ctx, const void *x, const void *w, void *out, int M, int N, int K);

/* Multi-query paged decode attention as a stand-alone call: the kernel both phases run once per layer
 * (Sec. 2.2: the target verifies all K candidates in a single forward pass; App. B.1: the head keeps a KV
 * cache of its own).  For every sequence b, q_count[b] queries at positions q_base[b] .. q_base[b] +
 * q_count[b] - 1 attend the cached positions <= their own; the caller has already written the new
 * keys/values into the pages.  Grouped-query: query head h reads KV head h / (n_q / n_kv).
 *   q        bf16 [B][n_kv][q_rows][head_dim], q_rows = 16 * ceil(q_stride * group / 16); row j*group + g is
 *            query j of head kv*group + g, rotary embedding already applied; unused rows must be finite
 *   kv_pool  bf16 [pool_layers][2][num_pages][n_kv][16][head_dim]; `layer` selects the slab
 *   page_table [B, max_pages_per_seq];  q_count, q_base [B];  q_stride <= max_k + 1 (rows per sequence in out)
 *   out      bf16 [B * q_stride][n_q * head_dim]; rows j >= q_count[b] are left untouched
 * A sequence whose queries do not fit its page-table row sets GM_ERR_KV_CAPACITY and is skipped.          */
int gm_attention(gm_ctx *ctx, const void *q, const void *kv_pool, int pool_layers, int num_pages, int layer,
                 const int32_t *page_table, const int32_t *q_count, const int32_t *q_base, int batch,
                 int q_stride, void *out);

/* gm_attention for callers that cannot allocate (the paper has no counterpart: this is a packaging
 * variant of the attention kernel, not a step of the method).  Same computation and argument meaning as
 * gm_attention, but it takes no context - the model shape is passed directly - and it calls no cudaMalloc,
 * cudaFree or any other allocating routine: the per-segment partial outputs, the page prefix and a status
 * word live in ONE static device array of GM_NOALLOC_SCRATCH_BYTES (16 MiB) that every GPU loading the
 * library holds until the process exits.  It is meant for callers such as a latency-critical serving
 * thread that must not trigger a device allocation, a plug-in that is given a stream but owns no memory
 * pool, or a process whose device memory is fully managed by another allocator.
 *   Limits: batch <= GM_NOALLOC_MAX_BATCH and
 *   4096 + (SMs + batch) * n_kv * q_rows * (head_dim + 2) * 4 bytes <= GM_NOALLOC_SCRATCH_BYTES
 *   (e.g. 64 sequences, 8 KV heads, 16 query rows, head_dim 128 on 148 SMs need 14.1 MB); anything larger
 *   returns GM_ERR_SCRATCH_LIMIT and launches nothing.
 *   Set-up: the FIRST call on each device resolves the array's device address (cudaGetSymbolAddress) with
 *   that device current; make that first call before any stream capture begins.
 *   Sharing: every call uses the same array, which keeps the previous call's contents; the call clears what
 *   must start at zero itself.  Two calls that overlap on the GPU (different streams, or two host threads)
 *   race on it - serialise them.  Device-seen conditions are not reported (there is no context whose status a
 *   later call could read): a sequence that does not fit its page-table row is skipped (its output rows stay
 *   untouched), an out-of-range page id reads page 0, and should one of the kernels' bounded waits ever run out
 *   the call still returns GM_OK with the rows of the affected segment incomplete - use gm_attention with a
 *   context where such conditions must be seen.
 *   cuda_stream: a cudaStream_t (NULL = the default stream) of the current device.                        */
#define GM_NOALLOC_SCRATCH_BYTES (16u << 20)
#define GM_NOALLOC_MAX_BATCH 256
int gm_attention_noalloc(int n_q_heads, int n_kv_heads, int head_dim, int max_pages_per_seq, const void *q,
                         const void *kv_pool, int pool_layers, int num_pages, int layer,
                         const int32_t *page_table, const int32_t *q_count, const int32_t *q_base, int batch,
                         int q_stride, void *out, void *cuda_stream);

/* Guard words (a stand-in for a memory checker): every workspace the library allocates is followed by 256
 * bytes of a fixed pattern.  With the environment variable GM_CANARY set when the context is created,
 * gm_last_status also reads the guards back and returns GM_ERR_OVERRUN if any byte changed.             */

/* Kernel-class timing.  gm_profile(ctx, mask) makes later calls bracket every launch of the
 * selected classes with CUDA events on the context's stream; gm_profile_read waits for the
 * stream and returns the accumulated device time and launch count of one class since the
 * last gm_profile call.  Independently of that, with the environment variable GM_NVTX set,
 * gm_draft, gm_verify, gm_accept, gm_prefill, gm_head_prefill, gm_rollout_step and
 * gm_reconstruct are wrapped in NVTX ranges of the same names.                              */
#define GM_KC_GEMM       0
#define GM_KC_ATTENTION  1
#define GM_KC_ELEMENTWISE 2
#define GM_KC_SAMPLER    3
#define GM_KC_RECORD     4
#define GM_KC_COUNT      5
int gm_profile(gm_ctx *ctx, int class_mask);
int gm_profile_read(gm_ctx *ctx, int kernel_class, double *total_ms, int64_t *launches);

/* Timeline of the persistent projection-chain kernel (the launch that runs a layer's output projection,
 * feed-forward block and the next layer's QKV projection back to back; a design choice of this library, the
 * paper describes no kernel).  gm_chain_trace(ctx, 1) makes later chain launches write nanosecond stamps of
 * their CTAs' phase transitions into a buffer the context allocates on the first call; gm_chain_trace(ctx, 0)
 * stops it.  gm_chain_trace_read waits for the stream and copies the stamps of the LAST traced launch to
 * `out` (host memory, `capacity` 64-bit words): 64 words per CTA (slot meaning: see csrc/chain.cu); returns
 * the number of words written (2 x CTA pairs x 64), or a negative GM_ERR_*.                               */
int gm_chain_trace(gm_ctx *ctx, int enable);
int gm_chain_trace_read(gm_ctx *ctx, uint64_t *out, int capacity);

/* Number of kernels this library launched since gm_init (all calls).                        */
int64_t gm_launch_count(gm_ctx *ctx);

/* Self-test of the failure path (the paper has no counterpart): every device-side wait of the library is a
 * bounded poll that records GM_ERR_DEVICE_TIMEOUT and returns instead of hanging.  This call launches one tiny
 * kernel whose only thread waits, with a limit of 1024 polls, on a barrier nothing ever arrives on; the wait runs
 * out, the status word is set, the kernel exits normally.  The next gm_last_status returns
 * GM_ERR_DEVICE_TIMEOUT and clears it; the context stays usable.  No GPU fault, trap or unbounded loop is involved. */
int gm_selftest_wait_expiry(gm_ctx *ctx);

/* Waits for the stream and returns 0 or the GM_ERR_* of the first sticky device condition;
 * clears the status word.                                                                   */
int gm_last_status(gm_ctx *ctx);
const char *gm_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* GM_H_ */
