// C ABI of libgm: forward pass of the head update on recorded cycles (Sec. 3.2-3.4, App. D.2-D.3) and the first two
// steps of its backward pass (Alg. 1: objective -> head logits -> head states).
// Host code only; the helpers it calls are declared in gm_internal.h.
#include "gm_internal.h"

extern "C" {

int gm_capture_hidden(gm_ctx *c, void *seq_hidden, int stride) {
  if (!c || (seq_hidden && stride < 1)) return GM_ERR_INVALID_ARG;
  c->capture = static_cast<__nv_bfloat16 *>(seq_hidden);
  c->capture_stride = seq_hidden ? stride : 0;
  return GM_OK;
}

int gm_reconstruct(gm_ctx *c, gm_state *st, int n_cycles, int k, const int32_t *cycle_seq, const gm_record *rec,
                   const int32_t *seq_tok, int tok_stride, const int32_t *scratch_pages, void *draft_logits) {
  return gm_reconstruct_states(c, st, n_cycles, k, cycle_seq, rec, seq_tok, tok_stride, scratch_pages, draft_logits, nullptr);
}

int gm_reconstruct_states(gm_ctx *c, gm_state *st, int n_cycles, int k, const int32_t *cycle_seq, const gm_record *rec,
                          const int32_t *seq_tok, int tok_stride, const int32_t *scratch_pages, void *draft_logits,
                          float *head_states) {
  NvtxRange nvtx_range("gm_reconstruct");
  int rc = check_state(c, st, k);
  if (rc) return rc;
  if (n_cycles < 1 || !cycle_seq || !rec || !rec->start_hidden || !rec->start_pos || !rec->drafts || !seq_tok ||
      tok_stride < 2 || !scratch_pages || !draft_logits)
    return GM_ERR_INVALID_ARG;
  const gm_config &cf = c->cfg;
  const int MB = cf.max_batch, PS = cf.max_k + 1;
  if (!c->v_table) {
    if ((rc = dev_alloc(c, &c->v_kv_len, MB)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->v_pending_n, MB)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->v_pending_tok, static_cast<size_t>(MB) * PS)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->v_pending_hidden, static_cast<size_t>(MB) * PS * c->d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->v_table, static_cast<size_t>(MB) * cf.max_pages_per_seq)) != GM_OK) return rc;
  }
  for (int off = 0; off < n_cycles; off += MB) {
    const int m = std::min(MB, n_cycles - off);
    ChainSetupArgs A;
    A.cycle_seq = cycle_seq + off; A.start_pos = rec->start_pos + off;
    A.start_hidden = static_cast<const __nv_bfloat16 *>(rec->start_hidden) + static_cast<size_t>(off) * c->d;
    A.seq_tok = seq_tok; A.scratch_pages = scratch_pages + 2 * static_cast<size_t>(off);
    A.head_page_table = st->head_page_table; A.pool = static_cast<__nv_bfloat16 *>(st->head_kv_pool);
    A.n_seq = st->batch; A.tok_stride = tok_stride; A.k = k; A.d = c->d; A.vocab = c->V;
    A.max_pages_per_seq = cf.max_pages_per_seq; A.num_pages = cf.head_num_pages;
    A.page_elems = cf.n_kv_heads * GM_PAGE * cf.head_dim; A.pend_stride = PS;
    A.v_kv_len = c->v_kv_len; A.v_pending_n = c->v_pending_n; A.v_pending_tok = c->v_pending_tok; A.v_table = c->v_table;
    A.v_pending_hidden = c->v_pending_hidden; A.status = c->status;
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_chain_setup(A, m, c->stream));
    gm_state vs = *st;
    vs.batch = m; vs.kv_len = c->v_kv_len; vs.head_page_table = c->v_table; vs.pending_n = c->v_pending_n;
    vs.pending_tok = c->v_pending_tok; vs.pending_hidden = c->v_pending_hidden;
    c->state_out = head_states ? head_states + static_cast<size_t>(off) * k * c->d : nullptr;
    rc = draft_impl(c, &vs, k, 1.0f, nullptr, 0, 0, rec->drafts + static_cast<size_t>(off) * k,
                    static_cast<__nv_bfloat16 *>(draft_logits) + static_cast<size_t>(off) * k * c->V, nullptr, true);
    c->state_out = nullptr;
    if (rc) return rc;
  }
  return GM_OK;
}

int gm_overlap(gm_ctx *c, int n_cycles, int k, float temperature, const void *draft_logits, const gm_record *rec,
               float *alpha, float *lse) {
  if (!c || n_cycles < 1 || k < 1 || k > GM_MAX_K || !draft_logits || !rec || !rec->top_index || !rec->top_logprob || !alpha)
    return GM_ERR_INVALID_ARG;
  if (!(temperature > 0.f) || !std::isfinite(temperature)) return GM_ERR_UNSUPPORTED;
  OverlapArgs A;
  A.logits = static_cast<const __nv_bfloat16 *>(draft_logits); A.top_index = rec->top_index;
  A.top_logprob = static_cast<const __nv_bfloat16 *>(rec->top_logprob); A.alpha = alpha; A.lse = lse; A.V = c->V;
  A.inv_temp = 1.0f / temperature;
  GM_LAUNCH(c, GM_KC_RECORD, launch_overlap(A, n_cycles * k, c->stream));
  return GM_OK;
}

int gm_dca_loss(gm_ctx *c, int n_cycles, int k, const float *alpha, const int32_t *accepted, float *loss, float *mean) {
  if (!c || n_cycles < 1 || k < 1 || k > GM_MAX_K || !alpha || !accepted || !loss || !mean) return GM_ERR_INVALID_ARG;
  GM_LAUNCH(c, GM_KC_RECORD, launch_dca_loss(alpha, accepted, n_cycles, k, loss, mean, c->stream));
  return GM_OK;
}

int gm_dca_grad(gm_ctx *c, int n_cycles, int k, float temperature, const void *draft_logits, const gm_record *rec,
                const float *alpha, const float *lse, const int32_t *accepted, void *grad_logits) {
  if (!c || n_cycles < 1 || k < 1 || k > GM_MAX_K || !draft_logits || !rec || !rec->top_index || !rec->top_logprob ||
      !alpha || !accepted || !grad_logits)
    return GM_ERR_INVALID_ARG;
  if (!(temperature > 0.f) || !std::isfinite(temperature)) return GM_ERR_UNSUPPORTED;
  DcaGradArgs A;
  A.logits = static_cast<const __nv_bfloat16 *>(draft_logits); A.top_index = rec->top_index;
  A.top_logprob = static_cast<const __nv_bfloat16 *>(rec->top_logprob); A.alpha = alpha; A.lse = lse; A.accepted = accepted;
  A.grad = static_cast<__nv_bfloat16 *>(grad_logits); A.V = c->V; A.K = k; A.n = n_cycles;
  A.inv_temp = 1.0f / temperature;
  GM_LAUNCH(c, GM_KC_RECORD, launch_dca_grad(A, c->stream));
  return GM_OK;
}

int gm_head_state_grad(gm_ctx *c, int rows, const void *grad_logits, const float *head_states, float *grad_normed,
                       float *grad_states, int refresh_weights) {
  if (!c || rows < 1 || !grad_logits || !grad_normed || (grad_states != nullptr) != (head_states != nullptr))
    return GM_ERR_INVALID_ARG;
  if ((c->V % 64) != 0 || (c->d % 8) != 0) return GM_ERR_UNSUPPORTED;
  int rc;
  const bool simple = (c->cfg.flags & GM_FLAG_SIMPLE_GEMM) != 0;
  if (!c->lm_head_t) {
    if ((rc = dev_alloc(c, &c->lm_head_t, static_cast<size_t>(c->d) * c->V, false)) != GM_OK) return rc;
    std::memset(&c->lm_head_t_map, 0, sizeof(c->lm_head_t_map));
    if (!simple && make_map(c, &c->lm_head_t_map, c->lm_head_t, c->d, c->V, 128) != GM_OK) return GM_ERR_CUDA;
    refresh_weights = 1;
  }
  if (refresh_weights)
    GM_LAUNCH(c, GM_KC_ELEMENTWISE,
              launch_transpose_bf16(static_cast<const __nv_bfloat16 *>(c->w.lm_head), c->V, c->d, c->lm_head_t, c->stream));
  // dL/dy [rows, d] = grad_logits [rows, V] x W_lm [V, d]: the projection kernel with the vocabulary as its K
  rc = run_gemm(c, static_cast<const __nv_bfloat16 *>(grad_logits), rows, &c->lm_head_t_map, c->lm_head_t, rows, c->d, c->V,
                grad_normed, EPI_STORE_F32, static_cast<size_t>(c->d), false);
  if (rc) return rc;
  if (grad_states)
    GM_LAUNCH(c, GM_KC_ELEMENTWISE,
              launch_rmsnorm_grad(grad_normed, head_states, static_cast<const __nv_bfloat16 *>(c->w.head_final_norm),
                                  grad_states, rows, c->d, c->cfg.rms_eps, c->stream));
  return GM_OK;
}

}  // extern "C"
