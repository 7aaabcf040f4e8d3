// Internal declarations shared by the kernel files and the C-ABI layer (not part of the public ABI).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

namespace gm {

// Launch with programmatic stream serialisation (the kernel calls pdl_prologue() first) and, if cluster_z > 1, a
// thread-block cluster (launch_k: along z; launch_kc: any shape).  GM_NO_PDL=1 in the environment turns the attribute off (plain serialisation).
bool pdl_enabled();
template <typename... KArgs, typename... Args>
cudaError_t launch_kc(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, dim3 cluster,
                      Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  int n = 0;
  if (pdl_enabled()) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (cluster.x * cluster.y * cluster.z > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster.x; attr[n].val.clusterDim.y = cluster.y; attr[n].val.clusterDim.z = cluster.z;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
template <typename... KArgs, typename... Args>
cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, int cluster_z,
                     Args &&...args) {
  return launch_kc(kernel, grid, block, smem, stream, dim3(1, 1, cluster_z > 1 ? cluster_z : 1), std::forward<Args>(args)...);
}

// The opt-in dynamic shared memory size is an attribute per kernel AND per device: `slot` is a function-local static
// table (one entry per device ordinal) that remembers the largest size already set on each device.
struct SmemConfigured { size_t bytes[64] = {}; };
template <typename K>
cudaError_t ensure_dyn_smem(K kernel, size_t bytes, SmemConfigured &slot) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool tracked = dev >= 0 && dev < 64;
  if (tracked && bytes <= slot.bytes[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes));
  if (e == cudaSuccess && tracked) slot.bytes[dev] = bytes;
  return e;
}

constexpr int GM_MAX_K_ = 7;
constexpr int SAMP_THREADS = 512;
constexpr int SAMP_CLUSTER = 8;

// ---- sampler ------------------------------------------------------------------------------------------
struct SamplerArgs {
  const __nv_bfloat16 *target_logits;   // row (b, r) at target_logits + b*tgt_bstride + r*V, r = 0..K
  const __nv_bfloat16 *draft_logits;    // row (b, r) at draft_logits + b*drf_bstride + r*V, r = 0..K-1 (null if K == 0)
  size_t tgt_bstride, drf_bstride;      // in elements
  const int32_t *draft_tok;             // d_{j+1} of row b at draft_tok[b*tok_in_stride + j]
  int tok_in_stride;
  const uint32_t *u24;                  // [b*u_stride + j], j = 0..K (K accept uniforms, then the final one); null = Philox
  int u_stride;
  uint64_t seed, step;
  uint32_t slot_accept, slot_final;
  float inv_temp;
  int K, V;
  int32_t *accept_len;                  // [b] or null
  int32_t *next_token;                  // [b*tok_out_stride]
  int tok_out_stride;
  float *dbg_p, *dbg_q;                 // same strides as the logits, or null
  int commit;                           // state commit (needs the fields below)
  int32_t *kv_len, *pending_n, *pending_tok;
  __nv_bfloat16 *pending_hidden;
  const __nv_bfloat16 *target_hidden;   // [b, K+1, d_model]
  int d_model, max_k;
  uint32_t *status;
  const uint64_t *step_ptr;             // when set, the step index is read from device memory instead of `step`
  const int32_t *finished;              // [b] non-zero: the row sits out (accept_len 0, next_token -1 (0 from a plain draw), state untouched); or null
};
cudaError_t launch_sampler(const SamplerArgs &A, int batch, cudaStream_t stream);          // cluster of 8 CTAs per sequence
cudaError_t launch_sampler_stream(const SamplerArgs &A, int batch, cudaStream_t stream);   // one CTA per sequence
bool sampler_stream_supported(int V);
// Vocabulary-sliced mapping: every CTA (one per SM) owns the same slice of every row of every sequence; `ws` is device memory
// of sampler_flow_ws_bytes(...) bytes, zeroed once before its first use (the kernel leaves it ready for the next launch).
bool sampler_flow_supported(int V, int batch, int K, int sm_count);
size_t sampler_flow_ws_bytes(int cap_batch, int V, int sm_count);
cudaError_t launch_sampler_flow(const SamplerArgs &A, int batch, void *ws, int cap_batch, int sm_count, cudaStream_t stream);

// ---- cycle record (top-64 target log-probabilities and the other recorded items) ---------------------------------
struct RecordTopkArgs {
  const __nv_bfloat16 *target_logits;   // row (b, k) at target_logits + b*bstride + k*V, k = 0..K-1
  size_t bstride;
  int K, V;
  float inv_temp;
  __nv_bfloat16 *top_logprob;           // [B, K, 64]
  int32_t *top_index;                   // [B, K, 64]
  uint32_t *status;
};
cudaError_t launch_record_topk(const RecordTopkArgs &A, int batch, cudaStream_t stream);
cudaError_t launch_record_begin(const int32_t *kv_len, const int32_t *pending_n, const __nv_bfloat16 *pending_hidden,
                                int batch, int max_k, int d, __nv_bfloat16 *start_hidden, int32_t *start_pos,
                                cudaStream_t stream);
cudaError_t launch_record_end(const int32_t *draft_tok, const int32_t *accept_len, int batch, int k, int32_t *drafts,
                              int32_t *accepted, cudaStream_t stream);

// ---- nucleus (top-p) truncation of logit rows: entries outside the top-p set become -inf ---------------
struct NucleusArgs {
  const __nv_bfloat16 *in;              // [rows][V]
  __nv_bfloat16 *out;                   // [rows][V] (may not alias in)
  float *dbg_e;                         // [rows][V] fp32 weights 2^((x - max) s) or null
  int rows, V;
  float inv_temp;
  uint32_t tp24;                        // round(top_p * 2^24), 1 .. 2^24 - 1
};
cudaError_t launch_nucleus(const NucleusArgs &A, cudaStream_t stream);

// ---- planning: query ranges of a phase and the balanced attention partition --------------------------
enum PhaseMode { PHASE_VERIFY = 0, PHASE_DRAFT_FIRST = 1, PHASE_DRAFT_NEXT = 2, PHASE_CHUNK = 3 };
struct PlanArgs {
  int mode, batch, k_or_j;              // VERIFY: K;  DRAFT_NEXT: application index j (2..K);  CHUNK: first position
  int max_pages_per_seq, n_ctas;
  const int32_t *kv_len, *pending_n;
  const int32_t *finished = nullptr;    // [B] non-zero: the sequence sits the phase out (no queries, no pages); or null
  const int32_t *row_n = nullptr;       // CHUNK: queries per sequence (0 = the sequence sits this pass out)
  const int32_t *row_base = nullptr;    // CHUNK: first position per sequence (null: k_or_j for all)
  int QT = 0;                           // CHUNK: most queries a sequence may have
  int32_t *qn, *qbase;                  // [B] queries of this phase and the position of the first one
  int32_t *page_start;                  // [B+1] exclusive prefix of pages attended per sequence
  uint32_t *status;
};
cudaError_t launch_plan(const PlanArgs &A, cudaStream_t stream);

// ---- prompt prefill in chunks of QT positions per sequence ------------------------------------------------
// Chunk `base / QT` of every prompt: row_n[b] = positions of prompt b inside [base, base + QT) (0 when the prompt
// ended before), head_n[b] = how many of them have a successor token inside the prompt (the pairs the draft head
// is prefilled with), pair_tok[b][j] = token at position base + j + 1.  A prompt shorter than 1 or longer than
// max_len raises ST_KV_CAPACITY and sits out.
// A pass may give every prompt `vr` consecutive chunks ("virtual rows": row v = b * vr + i holds positions
// base + i * QT .. + QT - 1 of prompt b), which the planner and the attention kernel see as vr independent
// sequences sharing a page table; row_base[v] = its first position.
struct ChunkSetupArgs {
  const int32_t *prompt_tok, *prompt_len;
  int batch, stride, base, QT, max_len, pair_stride, vr;
  int32_t *row_n, *head_n, *pair_tok, *row_base;
  uint32_t *status;
};
cudaError_t launch_chunk_setup(const ChunkSetupArgs &A, cudaStream_t stream);
// x[m] = embed[prompt_tok[b][base + j]] (fp32), xn[m] = RMSNorm(x[m]; w) (bf16) for j < row_n[b]; other rows token 0.
cudaError_t launch_embed_chunk(const __nv_bfloat16 *embed, const __nv_bfloat16 *w, const int32_t *prompt_tok, int stride,
                               const int32_t *row_base, const int32_t *row_n, int rows, int vr, int QT, int d, int vocab,
                               float eps, float *x, __nv_bfloat16 *xn, uint32_t *status, cudaStream_t stream);
// dst[v] = src[v / vr] for v < rows * vr: the page-table rows of the virtual rows
cudaError_t launch_dup_table_rows(const int32_t *src, int rows, int vr, int cols, int32_t *dst, cudaStream_t stream);
// For the sequences whose prompt ends inside this chunk: xlast[b] = x[row of the last prompt token] (fp32) and
// pending_hidden[b][0] = the same row of `hidden` (bf16).
cudaError_t launch_prefill_last(const float *x, const __nv_bfloat16 *hidden, const int32_t *row_n,
                                const int32_t *row_base, const int32_t *prompt_len, int rows, int vr, int QT, int d,
                                int pend_stride, float *xlast, __nv_bfloat16 *pending_hidden, cudaStream_t stream);
// kv_len[b] = prompt_len[b], pending_n[b] = 1, pending_tok[b][0] = first_tok[b].
cudaError_t launch_prefill_finish(const int32_t *prompt_len, const int32_t *first_tok, int batch, int pend_stride,
                                  int32_t *kv_len, int32_t *pending_n, int32_t *pending_tok, cudaStream_t stream);

// ---- rollout bookkeeping: responses, stopping, page allocation ------------------------------------------------
struct RolloutArgs {
  int batch, k, out_stride, eos_token, max_new, pend_stride;
  const int32_t *draft_tok;             // [B, k] drafts of the cycle (null for the begin call)
  const int32_t *accept_len, *next_token;   // [B] (null for the begin call: the token is pending_tok[b][0])
  const int32_t *pending_tok;
  int32_t *out_tok, *out_len, *finished, *n_running;
  uint64_t *step_counter = nullptr;     // when set, incremented once per append (the step index of a captured cycle)
};
// begin: response = [first token]; append: response += accepted drafts + final token of the cycle, cut at the first
// end-of-sequence token (kept) or at max_new tokens; finished[b] = 1 / 2 accordingly; n_running = rows still running.
cudaError_t launch_rollout_append(const RolloutArgs &A, bool begin, cudaStream_t stream);
cudaError_t launch_set_step(uint64_t *dst, uint64_t value, cudaStream_t stream);      // *dst = value
// Page allocator: a stack of free page ids per pool.  reserve: every running row gets pages until its table covers
// length[b] + extra positions (ST_KV_CAPACITY when the stack or the table row runs out); release: the pages of
// finished rows go back on the stack.  A row's slice of the stack comes from a prefix sum over the rows in order, so the
// assignment is the one a sequential walk would make and does not depend on scheduling.
struct PageAllocArgs {
  int batch, max_pages_per_seq, num_pages, extra;
  const int32_t *length, *finished;     // finished may be null
  int32_t *page_table, *held, *free_list, *free_top;
  uint32_t *status;
};
cudaError_t launch_page_reset(const PageAllocArgs &A, cudaStream_t stream);
cudaError_t launch_page_reserve(const PageAllocArgs &target, const PageAllocArgs &head, cudaStream_t stream);   // both pools
cudaError_t launch_page_release(const PageAllocArgs &target, const PageAllocArgs &head, cudaStream_t stream);

// ---- forward pass of the head update on recorded cycles ---------------------------------------------------
// A chain = a virtual sequence: shared head-cache pages of its sequence before the page of its first entry, two
// private pages from there (the first a copy of the shared one); pending pair = (start hidden, token at start - 1).
struct ChainSetupArgs {
  const int32_t *cycle_seq, *start_pos;            // [chains] sequence of the cycle; context length at its start
  const __nv_bfloat16 *start_hidden;               // [chains, d]
  const int32_t *seq_tok;                          // [n_seq, tok_stride] committed tokens
  const int32_t *scratch_pages;                    // [chains, 2] private page ids in the head pool
  const int32_t *head_page_table;                  // [n_seq, max_pages_per_seq]
  __nv_bfloat16 *pool;                             // head pool [1][2][num_pages][n_kv][16][hd]
  int n_seq, tok_stride, k, d, vocab, max_pages_per_seq, num_pages, page_elems, pend_stride;
  int32_t *v_kv_len, *v_pending_n, *v_pending_tok, *v_table;
  __nv_bfloat16 *v_pending_hidden;
  uint32_t *status;
};
cudaError_t launch_chain_setup(const ChainSetupArgs &A, int chains, cudaStream_t stream);
// out[v*QT + j] = seq_hidden[v / vr][row_base[v] + j] for j < row_n[v]
cudaError_t launch_gather_chunk_hidden(const __nv_bfloat16 *seq_hidden, int hid_stride, const int32_t *row_base, int rows,
                                       int vr, int QT, int d, const int32_t *row_n, __nv_bfloat16 *out, cudaStream_t stream);
struct OverlapArgs {
  const __nv_bfloat16 *logits;                     // [rows, V] head logits of the reconstructed chains
  const int32_t *top_index;                        // [rows, 64]
  const __nv_bfloat16 *top_logprob;                // [rows, 64]
  float *alpha;                                    // [rows]
  float *lse;                                      // [rows] logsumexp(logits / T) out, or null
  int V;
  float inv_temp;
};
cudaError_t launch_overlap(const OverlapArgs &A, int rows, cudaStream_t stream);
struct DcaGradArgs {
  const __nv_bfloat16 *logits;                     // [n, K, V] head logits of the reconstructed chains
  const int32_t *top_index;                        // [n, K, 64]
  const __nv_bfloat16 *top_logprob;
  const float *alpha;                              // [n, K]
  const int32_t *accepted;                         // [n]
  const float *lse;                                // [n, K] from the overlap pass, or null: recomputed
  __nv_bfloat16 *grad;                             // [n, K, V] out
  int V, K, n;
  float inv_temp;
  int n_total = 0;                                 // cycles the mean runs over when these n are a part of them (0: n)
};
cudaError_t launch_dca_grad(const DcaGradArgs &A, cudaStream_t stream);
// Rollout-time capture of the target hidden states of committed positions (App. D.2: the record keeps, per sequence,
// the hidden states the target computed during the rollout): dst[b][pos] = the hidden state computed at position pos.
//   chunk form (prefill): rows j < row_n[v] of src [rows, QT, d] go to positions row_base[v] + j of sequence v / vr;
//   cycle form: rows l <= accept_len[b] of src [B, k+1, d] go to positions kv_len[b] - (accept_len[b] + 1) + l, with
//   kv_len already advanced by the commit; rows of finished sequences are skipped.
cudaError_t launch_capture_chunk(const __nv_bfloat16 *src, const int32_t *row_n, const int32_t *row_base, int rows, int vr,
                                 int QT, int d, __nv_bfloat16 *dst, int dst_stride, cudaStream_t stream);
cudaError_t launch_capture_cycle(const __nv_bfloat16 *src, const int32_t *accept_len, const int32_t *kv_len,
                                 const int32_t *finished, int batch, int k, int d, __nv_bfloat16 *dst, int dst_stride,
                                 cudaStream_t stream);
cudaError_t launch_dca_loss(const float *alpha, const int32_t *accepted, int n, int K, float *loss, float *mean,
                            cudaStream_t stream);
// Backward through an RMSNorm y = x r w (fp32 rows of d values, bf16 weight): gx = r (w gy) - x r^3 mean(x w gy).
//   res (or null): added to gx (the gradient that reaches x past the norm, e.g. along a residual connection);
//   wterm (or null): fp32 [rows, d], gy x r per row - the rows' terms of dL/dw.
cudaError_t launch_rmsnorm_grad(const float *gy, const float *x, const __nv_bfloat16 *w, float *gx, int rows, int d, float eps,
                                cudaStream_t stream, const float *res = nullptr, float *wterm = nullptr, int gy_ld = 0);
// (gx may be null when only wterm is wanted; gy_ld: row stride of gy when it is a column block of a wider matrix, 0 = d)
// zin bf16 [rows, 2d] = [RMSNorm(embed[tokens]; we) ; RMSNorm(hidden; wh)], e_out fp32 [rows, d] = the embedding rows.
cudaError_t launch_head_input_rows(const __nv_bfloat16 *embed, const int32_t *tokens, const float *hidden, const __nv_bfloat16 *we,
                                   const __nv_bfloat16 *wh, int rows, int d, int vocab, float eps, __nv_bfloat16 *zin, float *e_out,
                                   uint32_t *status, cudaStream_t stream);
// dst [cols, dst_ld] = transpose of src [rows, cols] (bf16, both row-major; dst_ld >= rows, 0 = rows; padding untouched).
cudaError_t launch_transpose_bf16(const __nv_bfloat16 *src, int rows, int cols, __nv_bfloat16 *dst, cudaStream_t stream, int dst_ld = 0);
// out[j] = sum over rows of t[row][j] (fp32, row order).
// scratch (colsum_scratch_floats(d) floats, or null): lets many rows be split into chunks summed by separate CTAs
cudaError_t launch_colsum(const float *t, int rows, int d, float *out, cudaStream_t stream, bool add = false, float *scratch = nullptr);
size_t colsum_scratch_floats(int d);
// Bookkeeping of the backward pass over a reconstruction (chains of recorded cycles; Eq. 4).
struct StepRowsArgs {
  int k, K, d, vocab;                                   // application k (from 1) of K
  const int32_t *start_pos;                             // [chains]
  const __nv_bfloat16 *start_hidden;                    // [chains, d] the pair of application 1
  const int32_t *first_tok; int first_tok_stride;       // token of application 1 at first_tok[c * stride]
  const int32_t *drafts;                                // [chains, K] recorded drafts: application k >= 2 consumes drafts[k - 2]
  const float *states, *dstate;                         // [chains, K, d] head states and their gradients
  float *hidden, *dg;                                   // out [chains, d]
  int32_t *tok, *base, *count;                          // out [chains]: token, position, 1
  uint32_t *status;
};
cudaError_t launch_step_rows(const StepRowsArgs &A, int chains, cudaStream_t stream);
cudaError_t launch_add_state_grad(float *dstate, const float *dhidden, int chains, int K, int k, int d, cudaStream_t stream);
struct FoldArgs {
  const int32_t *cycle_seq, *start_pos, *scratch_pages, *head_page_table;
  int n_seq, max_pages_per_seq, num_pages, n_kv, hd;
  float *dk_pool, *dv_pool;
  long long *dk_fix = nullptr, *dv_fix = nullptr;       // fixed-point planes replacing the two above
};
cudaError_t launch_fold_boundary(const FoldArgs &A, int chains, cudaStream_t stream);
// Fixed point of the gradient accumulators: value * 2^40 rounded to a 64-bit integer.
constexpr float GM_FIX_SCALE = 1099511627776.0f, GM_FIX_INV = 1.0f / 1099511627776.0f;
cudaError_t launch_fix_to_float(const long long *src, float *dst, size_t n, cudaStream_t stream);
cudaError_t launch_widen_bf16(const __nv_bfloat16 *src, float *dst, size_t n, cudaStream_t stream);          // dst[i] = src[i]
cudaError_t launch_rows_to_f32(const __nv_bfloat16 *src, const int32_t *row_n, int rows, int QT, int d, float *dst, cudaStream_t stream);
// AdamW on n fp32 master parameters with fp32 moments; param (bf16 copy the forward pass reads) or null.  decay = 1 - lr wd,
// c1 / c2 = the bias corrections 1 / (1 - b^t), gscale multiplies the gradient (clipping).
cudaError_t launch_adamw(float *master, __nv_bfloat16 *param, const float *grad, float *m, float *v, size_t n, float lr, float b1,
                         float b2, float eps, float decay, float c1, float c2, float gscale, int sm_count, cudaStream_t stream);
cudaError_t launch_cast_bf16(const float *src, __nv_bfloat16 *dst, size_t n, cudaStream_t stream);       // n % 4 == 0
// Backward of h = silu(a) * b on interleaved (a, b) columns: dab bf16 [rows, 2F] (da, db interleaved), h bf16 [rows, F].
// Backward of what lies between the QKV projection and the attention core, for the rows of one pass (App. B.1): takes the
// rows' query gradients and their own cache entries' key / value gradients back through the rotary embedding (the
// rotation by the opposite angle) and the optional per-head RMSNorm, into the packed order of the projection's output.
struct QkvGradArgs {
  const __nv_bfloat16 *qkv;                             // [M][(n_q + 2 n_kv) hd] projection output of the forward, before bias
  const __nv_bfloat16 *bias = nullptr, *qnorm = nullptr, *knorm = nullptr;
  const float *dq;                                      // [M][n_q][hd] gradient of the rotated queries
  const float *dk_pool, *dv_pool;                       // [num_pages][n_kv][16][hd] gradient planes of the cache
  const long long *dk_fix = nullptr, *dv_fix = nullptr, *dq_fix = nullptr;   // fixed-point sources (2^-40) replacing the three above
  const int32_t *qn, *qbase, *page_table;
  const float2 *rope;
  int batch, QT, n_q, n_kv, hd, num_pages, max_pages_per_seq;
  float eps = 0.f;
  float *dqkv;                                          // [M][(n_q + 2 n_kv) hd]; rows beyond a sequence's count are zero
  __nv_bfloat16 *dqkv_bf;                               // the same in bf16 (operand of the projections' backward)
  float *tq = nullptr, *tk = nullptr;                   // per-head terms of the norm weights' gradients [M n_q][hd], [M n_kv][hd]
  uint32_t *status;
};
cudaError_t launch_qkv_grad_rows(const QkvGradArgs &A, cudaStream_t stream);
cudaError_t launch_swiglu_grad(const __nv_bfloat16 *ab, const float *dh, __nv_bfloat16 *dab, __nv_bfloat16 *h, int rows, int F,
                               cudaStream_t stream);

// ---- element-wise --------------------------------------------------------------------------------------
// x[m] = embed[token(m)] (fp32), xn[m] = RMSNorm(x[m]; w) (bf16); rows m = b*QT + j of the verify phase.
cudaError_t launch_embed_norm(const __nv_bfloat16 *embed, const __nv_bfloat16 *w, const int32_t *pending_tok,
                              const int32_t *pending_n, const int32_t *draft_tok, int batch, int K, int max_k, int d,
                              int vocab, float eps, float *x, __nv_bfloat16 *xn, uint32_t *status,
                              cudaStream_t stream);
// zin[m] = [RMSNorm(embed[tok]; we) ; RMSNorm(hidden; wh)] (bf16 [M, 2d]) for the draft head.
struct HeadInputArgs {
  int mode, batch, QT, d, vocab, max_k, k, j;    // j: application index for DRAFT_NEXT
  float eps;
  const __nv_bfloat16 *embed, *we, *wh;
  const int32_t *pending_tok, *pending_n;
  const __nv_bfloat16 *pending_hidden;           // [B, max_k+1, d]
  const int32_t *draft_tok;                      // [B, k]
  const float *g_prev;                           // [B, d] head state of the previous application
  __nv_bfloat16 *zin;                            // [B*QT, 2d]
  uint32_t *status;
};
cudaError_t launch_head_input(const HeadInputArgs &A, cudaStream_t stream);
// xn[m] = RMSNorm(x[m]; w) (bf16) from the fp32 residual stream; optional bf16 copy of x (the hidden state
// handed to the caller).
cudaError_t launch_rmsnorm(const float *x, const __nv_bfloat16 *w, __nv_bfloat16 *xn, __nv_bfloat16 *hidden_out,
                           int M, int d, float eps, cudaStream_t stream);
// Rotary embedding of q and k, KV append into the pages, Q rearranged per (sequence, kv head).
struct RopeAppendArgs {
  const __nv_bfloat16 *qkv;                             // bf16 [M][(n_q + 2 n_kv) hd]
  int batch, QT, n_q, n_kv, hd, layer, num_pages, max_pages_per_seq, qrows;
  const int32_t *qn, *qbase, *page_table;
  const float2 *rope;                                   // [max_pos][hd/2] (cos, sin)
  const __nv_bfloat16 *bias = nullptr;                  // [(n_q + 2 n_kv) hd] added to the projection, or null
  const __nv_bfloat16 *qnorm = nullptr, *knorm = nullptr;  // [hd] RMSNorm weights of the query / key heads, or null
  float eps = 0.f;
  __nv_bfloat16 *qbuf;                                  // [B][n_kv][qrows][hd], row = j*group + g
  __nv_bfloat16 *pool;                                  // [L][2][num_pages][n_kv][16][hd]; null: queries only, nothing appended
  uint32_t *status;
};
cudaError_t launch_rope_append(const RopeAppendArgs &A, cudaStream_t stream);
// g[b] = x[b*QT + qn[b]-1] (fp32), gn[b] = RMSNorm(g[b]; w) (bf16): the head's last valid row per sequence.
cudaError_t launch_head_out(const float *x, const int32_t *qn, int batch, int QT, int d, const __nv_bfloat16 *w,
                            float eps, float *g, __nv_bfloat16 *gn, cudaStream_t stream);

// ---- attention -------------------------------------------------------------------------------------------
struct AttnArgs {
  CUtensorMap kv_map;                   // 2-D view of the pool: [rows of hd elements], box 64 x (heads*16)
  const __nv_bfloat16 *qbuf;            // [B][n_kv][qrows][hd]
  const int32_t *qn, *qbase, *page_start, *page_table;
  int batch, n_kv, group, hd, qrows, layer, num_pages, max_pages_per_seq, n_ctas;
  float scale_log2e;                    // 1/sqrt(hd) * log2(e)
  float *part_o;                        // [n_ctas + B][n_kv][qrows][hd] partial outputs
  float *part_ml;                       // [n_ctas + B][n_kv][qrows][2] partial (max, sum)
  uint32_t *status;
  int rows_used = 0;                    // query rows a sequence can have (q positions x group); 0 = unknown (qrows is assumed)
};
cudaError_t launch_attention(const AttnArgs &A, cudaStream_t stream);
// Backward of the attention core: dq for every query row, and the key / value gradients accumulated (atomically) into fp32
// planes laid out like one layer of the pool.  stats: scratch fp32 [batch * QT][n_q][3].
struct AttnBwdArgs {
  const __nv_bfloat16 *q;               // [B][n_kv][qrows][hd], row j*group + g (the forward kernel's query layout)
  const float *dout;                    // [B * QT][n_q * hd]: gradient of the attention output
  const __nv_bfloat16 *pool;            // [L][2][num_pages][n_kv][16][hd]
  const int32_t *qn, *qbase, *page_table;
  int batch, QT, n_kv, group, hd, qrows, layer, num_pages, max_pages_per_seq;
  float scale;                          // 1 / sqrt(hd)
  float *stats, *dq;                    // dq [B * QT][n_q * hd], zero on entry (the key-split kernels add into it)
  float *dk_pool, *dv_pool;             // [num_pages][n_kv][16][hd], accumulated
  // Fixed-point accumulators (units of 2^-40, 64-bit integer additions: the sums do not depend on the order in which CTAs
  // arrive).  Given, they replace dk_pool / dv_pool / dq, which are then not touched.
  long long *dk_fix = nullptr, *dv_fix = nullptr, *dq_fix = nullptr;
  float *part = nullptr;                // [B][n_kv][nseg][pairs][3] partial softmax statistics per key segment, or null
  int nseg = 0;                         // segments the scratch holds per (sequence, KV head)
  uint32_t *status;
};
cudaError_t launch_attention_backward(const AttnBwdArgs &A, cudaStream_t stream);
constexpr int ATTN_BWD_SEG = 256;       // keys per CTA of the key-split kernels
constexpr int ATTN_BWD_MAX_PAIRS = 16;  // (row, query head of the group) pairs per (sequence, KV head) they hold in registers
struct AttnCombineArgs {
  const float *part_o, *part_ml;
  const int32_t *qn, *page_start;
  int batch, n_kv, group, hd, qrows, QT, n_ctas;
  __nv_bfloat16 *out;                   // [B*QT][n_q*hd]
};
cudaError_t launch_attention_combine(const AttnCombineArgs &A, cudaStream_t stream);
cudaError_t launch_page_prefix(const int32_t *qn, const int32_t *qbase, int batch, int max_pages_per_seq, int q_stride,
                               int32_t *page_start, uint32_t *status, cudaStream_t stream);
int attention_max_ctas(int n_kv, int hd);   // CTAs the attention kernel wants for this shape (<= SM count)
size_t attention_smem_bytes(int n_kv, int hd, int mt);

// ---- GEMM --------------------------------------------------------------------------------------------------
// out = epilogue(x[M, K] * w[N, K]^T) with fp32 accumulation.
enum GemmEpilogue {
  EPI_STORE_BF16 = 0,    // out bf16 [M, ldo]
  EPI_STORE_F32 = 1,     // out fp32 [M, ldo]
  EPI_ADD_F32 = 2,       // out fp32 [M, ldo] += result   (residual stream update)
  EPI_SWIGLU_BF16 = 3,   // rows of w interleaved (gate_i, up_i): out bf16 [M, ldo], column i = silu(gate_i) * up_i
  EPI_QKV_ROPE = 4,      // the QKV projection: rounded to bf16, then bias, head norms, rotary embedding, query rows to qbuf and
                         // keys / values appended to their pages (GemmArgs::rope; `out` unused); head_dim 64 or 128
};
struct GemmArgs {
  CUtensorMap w_map, x_map;             // tcgen05 path only
  CUtensorMap x_half_map;               // CTA-pair kernel only: activation boxes of block_t / 2 rows
  const __nv_bfloat16 *x, *w;
  void *out; int epi;
  int M, N, K;
  int n_base;                           // first output feature of this launch (a projection may be issued as main part + tail)
  int n_tiles;                          // CTAs along N of this launch
  int nsplit;                           // K slices = cluster size along z (1..8); the simple kernel ignores it
  int block_t;                          // tokens per CTA (multiple of 16, <= 256)
  int wtiles;                           // 128-feature sub-tiles per CTA sharing one activation tile (1 or 2)
  size_t ldo;                           // output row stride in elements
  RopeAppendArgs rope;                  // EPI_QKV_ROPE only (qkv unused)
  int early_weights;                    // w is written by no kernel of the stream: its first boxes may be fetched before the dependency wait
  uint32_t *status;
};
cudaError_t launch_gemm_tc(const GemmArgs &A, cudaStream_t stream);
// CTA-pair form (one K slice per tile, an even number of feature tiles, block_t a multiple of 32).
cudaError_t launch_gemm_pair(const GemmArgs &A, cudaStream_t stream);
// CTA pairs with K slices: cluster (2, 1, nsplit), nsplit = 2..8 (above 4: clusters of more than 8 CTAs, an opt-in); n_tiles even,
// one sub-tile per CTA.
cudaError_t launch_gemm_pair_split(const GemmArgs &A, cudaStream_t stream);
cudaError_t gemm_pair_split_max_clusters(int block_t, int nsplit, int *out);
cudaError_t launch_gemm_simple(const GemmArgs &A, cudaStream_t stream);
// How many clusters of `nsplit` CTAs of the tcgen05 kernel can be resident at once (GPC packing).
cudaError_t gemm_tc_max_clusters(int block_t, int nsplit, int *out);

// ---- a chain of dependent projections in one persistent launch (chain.cu) -------------------------------------------
// Phase p computes epilogue_p(x_p[M, K_p] * w_p[N_p, K_p]^T); phase p + 1 may read what phase p wrote.
struct ChainPhase {
  CUtensorMap w_map;                    // weights [N, K] bf16, box 64 x wbox
  CUtensorMap x_map;                    // input rows [M, K] bf16, box 64 x 128
  void *out;                            // EPI_STORE_BF16 / EPI_SWIGLU_BF16: bf16 [M, ldo]; EPI_STORE_F32 / EPI_ADD_F32: fp32 [M, ldo]
  __nv_bfloat16 *xg;                    // fp32 epilogues: also bf16(result * gamma) [M, N], the next norm's input; or null
  const __nv_bfloat16 *gamma;           // [N] norm weight for xg
  float *sq_out;                        // fp32 epilogues: [tiles][m_pad] sums of squares of the result rows per feature tile; or null
  const float *sq_in;                   // [sq_groups][m_pad] sums of squares of this phase's input rows before the norm
                                        // weight was applied: the accumulator rows are scaled by rsqrt(sum * inv_dim + eps); or null
  int sq_groups;
  float inv_dim;                        // 1 / width of the normalised rows
  int epi;
  int N, K;
  int ldo;
  int G, tiles, ns, wbox;               // schedule (chain_schedule): groups of 16 features, feature tiles, K slices per
                                        // tile, weight rows a CTA stages per K block (half of the widest tile)
};
struct ChainArgs {
  ChainPhase ph[4];
  int n_phases;
  int M, mblocks;                       // token rows, blocks of 256 token rows
  int P;                                // CTA pairs of the launch (all resident at once)
  int npw, npa;                         // producer threads for weight / activation boxes
  int m_pad;                            // row stride of the sums of squares
  float eps;
  float *partial;                       // [P][2][128][288] fp32 scratch of the K slices
  unsigned long long *sync;             // monotonic barrier counters: [0] the grid's, [1 + 2 pair + CTA rank] the K-slice groups'
  uint32_t *status;
  unsigned long long *timeline;         // optional trace, [2 P][64] nanosecond stamps (see chain.cu); or null
  int trace_phase;                      // phase whose epilogue detail stamps go to slots 32.. / 48..
};
void chain_schedule(ChainPhase &ph, int mblocks, int P, int force_ns);
size_t chain_partial_floats(int pairs);
cudaError_t chain_max_pairs(int *out);
cudaError_t launch_chain(const ChainArgs &A, cudaStream_t stream);

}  // namespace gm
