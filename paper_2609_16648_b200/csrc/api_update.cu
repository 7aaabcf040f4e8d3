// C ABI of libgm: forward pass of the head update on recorded cycles (Sec. 3.2-3.4, App. D.2-D.3) and the first two
// steps of its backward pass (Alg. 1: objective -> head logits -> head states).
// Host code only; the helpers it calls are declared in gm_internal.h.
#include "gm_internal.h"

// scratch for column sums split over several CTAs; null (single-chunk sums) if the allocation fails
static float *colsum_ws(gm_ctx *c) {
  if (!c->colsum_ws) {
    const size_t widest = static_cast<size_t>(std::max(std::max(c->n_qkv, 2 * c->d), static_cast<int>(c->cfg.head_dim)));
    if (dev_alloc(c, &c->colsum_ws, gm::colsum_scratch_floats(static_cast<int>(widest))) != GM_OK) c->colsum_ws = nullptr;
  }
  return c->colsum_ws;
}

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

// accum: the parameter gradients are added to what the output buffers hold (a pass among several) instead of stored
static int head_ffn_backward_impl(gm_ctx *c, int rows, const float *x, const float *dg, float *dx, float *dw_gate_up, float *dw_down,
                                  float *dln2, int refresh_weights, bool accum) {
  if (!c || rows < 1 || !x || !dg || !dx || !dw_gate_up || !dw_down || !dln2) return GM_ERR_INVALID_ARG;
  const int wepi = accum ? EPI_ADD_F32 : EPI_STORE_F32;
  const int d = c->d, F = c->F;
  if ((c->cfg.flags & GM_FLAG_SIMPLE_GEMM) || (d % 64) || (F % 64)) return GM_ERR_UNSUPPORTED;
  const gm_layer_weights &lw = c->w.head_layer;
  const __nv_bfloat16 *w_gu = static_cast<const __nv_bfloat16 *>(lw.w_gate_up), *w_d = static_cast<const __nv_bfloat16 *>(lw.w_down);
  const __nv_bfloat16 *ln2 = static_cast<const __nv_bfloat16 *>(lw.ln2);
  int rc;
  if (!c->ffn_wd_t) {
    if ((rc = dev_alloc(c, &c->ffn_wd_t, static_cast<size_t>(F) * d, false)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->ffn_wgu_t, static_cast<size_t>(d) * 2 * F, false)) != GM_OK) return rc;
    if (make_map(c, &c->ffn_wd_t_map, c->ffn_wd_t, F, d, 128) != GM_OK) return GM_ERR_CUDA;
    if (make_map(c, &c->ffn_wgu_t_map, c->ffn_wgu_t, d, 2 * F, 128) != GM_OK) return GM_ERR_CUDA;
    refresh_weights = 1;
  }
  if (refresh_weights) {
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_transpose_bf16(w_d, d, F, c->ffn_wd_t, c->stream));             // [d, F] -> [F, d]
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_transpose_bf16(w_gu, 2 * F, d, c->ffn_wgu_t, c->stream));       // [2F, d] -> [d, 2F]
  }
  const int Mp = (rows + 63) / 64 * 64;              // the weight-gradient products contract over the rows: blocks of 64
  if (Mp > c->ffn_rows_cap) {
    const size_t M = static_cast<size_t>(Mp);
    if ((rc = dev_alloc(c, &c->ffn_u, M * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->ffn_ab, M * 2 * F)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->ffn_dy, M * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->ffn_dab, M * 2 * F)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->ffn_h, M * F)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->ffn_ut, M * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->ffn_dyt, M * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->ffn_dabt, M * 2 * F)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->ffn_ht, M * F)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->ffn_dh, M * F)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->ffn_du, M * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->ffn_t, M * d)) != GM_OK) return rc;
    c->ffn_rows_cap = Mp;
  }
  // forward values the backward needs, recomputed: u = RMSNorm(x; ln2), (a, b) = u W_gu^T (interleaved, bf16)
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_rmsnorm(x, ln2, c->ffn_u, nullptr, rows, d, c->cfg.rms_eps, c->stream));
  if ((rc = run_gemm(c, c->ffn_u, rows, &c->head_maps.wgu, w_gu, rows, 2 * F, d, c->ffn_ab, EPI_STORE_BF16, 2 * static_cast<size_t>(F))) != GM_OK)
    return rc;
  // dh = dg W_d   (the block's output is x + h W_d^T)
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_cast_bf16(dg, c->ffn_dy, static_cast<size_t>(rows) * d, c->stream));
  if ((rc = run_gemm(c, c->ffn_dy, rows, &c->ffn_wd_t_map, c->ffn_wd_t, rows, F, d, c->ffn_dh, EPI_STORE_F32, static_cast<size_t>(F), false)) != GM_OK)
    return rc;
  // through the activation: (da, db) interleaved, and h for the down projection's weight gradient
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_swiglu_grad(c->ffn_ab, c->ffn_dh, c->ffn_dab, c->ffn_h, rows, F, c->stream));
  // du = (da, db) W_gu;  dx = dg + d RMSNorm;  dln2 = sum over rows of du x r
  if ((rc = run_gemm(c, c->ffn_dab, rows, &c->ffn_wgu_t_map, c->ffn_wgu_t, rows, d, 2 * F, c->ffn_du, EPI_STORE_F32, static_cast<size_t>(d), false)) != GM_OK)
    return rc;
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_rmsnorm_grad(c->ffn_du, x, ln2, dx, rows, d, c->cfg.rms_eps, c->stream, dg, c->ffn_t));
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_colsum(c->ffn_t, rows, d, dln2, c->stream, accum, colsum_ws(c)));
  // weight gradients contract over the rows: both operands transposed to [features, rows] (rows padded with zeros to Mp)
  GM_CUDA(c, cudaMemsetAsync(c->ffn_ut, 0, sizeof(__nv_bfloat16) * static_cast<size_t>(Mp) * d, c->stream));
  GM_CUDA(c, cudaMemsetAsync(c->ffn_dyt, 0, sizeof(__nv_bfloat16) * static_cast<size_t>(Mp) * d, c->stream));
  GM_CUDA(c, cudaMemsetAsync(c->ffn_dabt, 0, sizeof(__nv_bfloat16) * static_cast<size_t>(Mp) * 2 * F, c->stream));
  GM_CUDA(c, cudaMemsetAsync(c->ffn_ht, 0, sizeof(__nv_bfloat16) * static_cast<size_t>(Mp) * F, c->stream));
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_transpose_bf16(c->ffn_u, rows, d, c->ffn_ut, c->stream, Mp));
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_transpose_bf16(c->ffn_dy, rows, d, c->ffn_dyt, c->stream, Mp));
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_transpose_bf16(c->ffn_dab, rows, 2 * F, c->ffn_dabt, c->stream, Mp));
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_transpose_bf16(c->ffn_h, rows, F, c->ffn_ht, c->stream, Mp));
  CUtensorMap wm;
  // dW_d [d, F] = dg^T h
  if (make_map(c, &wm, c->ffn_ht, F, Mp, 128) != GM_OK) return GM_ERR_CUDA;
  if ((rc = run_gemm(c, c->ffn_dyt, d, &wm, c->ffn_ht, d, F, Mp, dw_down, wepi, static_cast<size_t>(F), false)) != GM_OK) return rc;
  // dW_gu [2F, d] = (da, db)^T u   (rows interleaved like the packed weight)
  if (make_map(c, &wm, c->ffn_ut, d, Mp, 128) != GM_OK) return GM_ERR_CUDA;
  return run_gemm(c, c->ffn_dabt, 2 * F, &wm, c->ffn_ut, 2 * F, d, Mp, dw_gate_up, wepi, static_cast<size_t>(d), false);
}
int gm_head_ffn_backward(gm_ctx *c, int rows, const float *x, const float *dg, float *dx, float *dw_gate_up, float *dw_down,
                         float *dln2, int refresh_weights) {
  return head_ffn_backward_impl(c, rows, x, dg, dx, dw_gate_up, dw_down, dln2, refresh_weights, false);
}

int gm_adamw_step(gm_ctx *c, int64_t n, float *master, void *param_bf16, const float *grad, float *m, float *v, int step, float lr,
                  float beta1, float beta2, float eps, float weight_decay, float grad_scale) {
  if (!c || n < 1 || !master || !grad || !m || !v || step < 1) return GM_ERR_INVALID_ARG;
  if (!(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(lr >= 0.f) || !(eps >= 0.f) || !std::isfinite(lr) ||
      !std::isfinite(grad_scale))
    return GM_ERR_UNSUPPORTED;
  const double c1 = 1.0 / (1.0 - std::pow(static_cast<double>(beta1), step));
  const double c2 = 1.0 / (1.0 - std::pow(static_cast<double>(beta2), step));
  const double decay = 1.0 - static_cast<double>(lr) * static_cast<double>(weight_decay);
  GM_LAUNCH(c, GM_KC_ELEMENTWISE,
            launch_adamw(master, static_cast<__nv_bfloat16 *>(param_bf16), grad, m, v, static_cast<size_t>(n), lr, beta1, beta2, eps,
                         static_cast<float>(decay), static_cast<float>(c1), static_cast<float>(c2), grad_scale, c->sm_count,
                         c->stream));
  return GM_OK;
}

// dhidden may be null here (rows whose hidden state is a recorded input, not a head state)
static int head_input_backward_impl(gm_ctx *c, int rows, const int32_t *tokens, const float *hidden, const float *dz, float *dhidden,
                                    float *dproj, float *denorm, float *dhnorm, int refresh_weights, bool accum) {
  if (!c || rows < 1 || !tokens || !hidden || !dz || !dproj || !denorm || !dhnorm) return GM_ERR_INVALID_ARG;
  const int d = c->d;
  if ((c->cfg.flags & GM_FLAG_SIMPLE_GEMM) || (d % 64)) return GM_ERR_UNSUPPORTED;
  const __nv_bfloat16 *proj = static_cast<const __nv_bfloat16 *>(c->w.head_proj);
  const __nv_bfloat16 *we = static_cast<const __nv_bfloat16 *>(c->w.head_enorm), *wh = static_cast<const __nv_bfloat16 *>(c->w.head_hnorm);
  int rc;
  if (!c->hin_proj_t) {
    if ((rc = dev_alloc(c, &c->hin_proj_t, static_cast<size_t>(2) * d * d, false)) != GM_OK) return rc;
    if (make_map(c, &c->hin_proj_t_map, c->hin_proj_t, 2 * d, d, 128) != GM_OK) return GM_ERR_CUDA;
    refresh_weights = 1;
  }
  if (refresh_weights)
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_transpose_bf16(proj, d, 2 * d, c->hin_proj_t, c->stream));     // [d, 2d] -> [2d, d]
  const int Mp = (rows + 63) / 64 * 64;
  if (Mp > c->hin_rows_cap) {
    const size_t M = static_cast<size_t>(Mp);
    if ((rc = dev_alloc(c, &c->hin_zin, M * 2 * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hin_dz, M * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hin_zint, M * 2 * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hin_dzt, M * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hin_e, M * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hin_dzin, M * 2 * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hin_t, M * d)) != GM_OK) return rc;
    c->hin_rows_cap = Mp;
  }
  // the forward's input rows, recomputed: [RMSNorm(E[token]) ; RMSNorm(hidden)] in bf16, and the embedding rows in fp32
  GM_LAUNCH(c, GM_KC_ELEMENTWISE,
            launch_head_input_rows(static_cast<const __nv_bfloat16 *>(c->w.embed), tokens, hidden, we, wh, rows, d, c->V, c->cfg.rms_eps,
                                   c->hin_zin, c->hin_e, c->status, c->stream));
  // d zin = dz W_p
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_cast_bf16(dz, c->hin_dz, static_cast<size_t>(rows) * d, c->stream));
  if ((rc = run_gemm(c, c->hin_dz, rows, &c->hin_proj_t_map, c->hin_proj_t, rows, 2 * d, d, c->hin_dzin, EPI_STORE_F32, 2 * static_cast<size_t>(d),
                     false)) != GM_OK)
    return rc;
  // through the two norms: the hidden half gives dL/d hidden and dL/d hnorm, the embedding half only dL/d enorm
  GM_LAUNCH(c, GM_KC_ELEMENTWISE,
            launch_rmsnorm_grad(c->hin_dzin + d, hidden, wh, dhidden, rows, d, c->cfg.rms_eps, c->stream, nullptr, c->hin_t, 2 * d));
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_colsum(c->hin_t, rows, d, dhnorm, c->stream, accum, colsum_ws(c)));
  GM_LAUNCH(c, GM_KC_ELEMENTWISE,
            launch_rmsnorm_grad(c->hin_dzin, c->hin_e, we, nullptr, rows, d, c->cfg.rms_eps, c->stream, nullptr, c->hin_t, 2 * d));
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_colsum(c->hin_t, rows, d, denorm, c->stream, accum, colsum_ws(c)));
  // dW_p [d, 2d] = dz^T zin: both operands transposed to [features, rows] (rows padded with zeros to Mp)
  GM_CUDA(c, cudaMemsetAsync(c->hin_dzt, 0, sizeof(__nv_bfloat16) * static_cast<size_t>(Mp) * d, c->stream));
  GM_CUDA(c, cudaMemsetAsync(c->hin_zint, 0, sizeof(__nv_bfloat16) * static_cast<size_t>(Mp) * 2 * d, c->stream));
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_transpose_bf16(c->hin_dz, rows, d, c->hin_dzt, c->stream, Mp));
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_transpose_bf16(c->hin_zin, rows, 2 * d, c->hin_zint, c->stream, Mp));
  CUtensorMap wm;
  if (make_map(c, &wm, c->hin_zint, 2 * d, Mp, 128) != GM_OK) return GM_ERR_CUDA;
  return run_gemm(c, c->hin_dzt, d, &wm, c->hin_zint, d, 2 * d, Mp, dproj, accum ? EPI_ADD_F32 : EPI_STORE_F32, 2 * static_cast<size_t>(d), false);
}
int gm_head_input_backward(gm_ctx *c, int rows, const int32_t *tokens, const float *hidden, const float *dz, float *dhidden,
                           float *dproj, float *denorm, float *dhnorm, int refresh_weights) {
  if (!dhidden) return GM_ERR_INVALID_ARG;
  return head_input_backward_impl(c, rows, tokens, hidden, dz, dhidden, dproj, denorm, dhnorm, refresh_weights, false);
}

// dk_fix / dv_fix / dq_fix given: the gradients are accumulated there in fixed point (order-independent sums) and the float
// outputs are not touched
static int attention_backward_impl(gm_ctx *c, const void *q, const float *dout, const void *kv_pool, int pool_layers, int num_pages, int layer,
                                   const int32_t *page_table, const int32_t *q_count, const int32_t *q_base, int batch, int q_stride,
                                   float *dq, float *dk_pool, float *dv_pool, long long *dq_fix, long long *dk_fix, long long *dv_fix) {
  const bool fix = dk_fix != nullptr;
  if (!c || !q || !dout || !kv_pool || !page_table || !q_count || !q_base) return GM_ERR_INVALID_ARG;
  if (fix ? (!dq_fix || !dv_fix) : (!dq || !dk_pool || !dv_pool)) return GM_ERR_INVALID_ARG;
  if (batch < 1 || q_stride < 1 || pool_layers < 1 || layer < 0 || layer >= pool_layers || num_pages < 1) return GM_ERR_INVALID_ARG;
  const gm_config &cf = c->cfg;
  if (q_stride > 8 || c->group > 8 || (cf.head_dim != 64 && cf.head_dim != 128)) return GM_ERR_UNSUPPORTED;
  const size_t need = static_cast<size_t>(batch) * q_stride * cf.n_q_heads * 3;
  if (need > c->ab_stats_cap) {
    int rc = dev_alloc(c, &c->ab_stats, need);
    if (rc != GM_OK) return rc;
    c->ab_stats_cap = need;
  }
  const int pairs = q_stride * c->group;
  const int nseg = (cf.max_pages_per_seq * GM_PAGE + ATTN_BWD_SEG - 1) / ATTN_BWD_SEG;
  if (pairs <= ATTN_BWD_MAX_PAIRS) {
    const size_t np = pairs <= 4 ? 4 : (pairs <= 8 ? 8 : 16);
    const size_t want = static_cast<size_t>(batch) * cf.n_kv_heads * nseg * np * 3;
    if (want > c->ab_part_cap) {
      int rc = dev_alloc(c, &c->ab_part, want);
      if (rc != GM_OK) return rc;
      c->ab_part_cap = want;
    }
  }
  AttnBwdArgs A;
  if (pairs <= ATTN_BWD_MAX_PAIRS) { A.part = c->ab_part; A.nseg = nseg; }
  A.q = static_cast<const __nv_bfloat16 *>(q); A.dout = dout; A.pool = static_cast<const __nv_bfloat16 *>(kv_pool);
  A.qn = q_count; A.qbase = q_base; A.page_table = page_table;
  A.batch = batch; A.QT = q_stride; A.n_kv = cf.n_kv_heads; A.group = c->group; A.hd = cf.head_dim;
  A.qrows = round16(q_stride * c->group); A.layer = layer; A.num_pages = num_pages; A.max_pages_per_seq = cf.max_pages_per_seq;
  A.scale = static_cast<float>(1.0 / std::sqrt(static_cast<double>(cf.head_dim)));
  A.stats = c->ab_stats; A.dq = dq; A.dk_pool = dk_pool; A.dv_pool = dv_pool; A.status = c->status;
  A.dq_fix = dq_fix; A.dk_fix = dk_fix; A.dv_fix = dv_fix;
  const size_t nq = static_cast<size_t>(batch) * q_stride * cf.n_q_heads * cf.head_dim;
  if (fix) GM_CUDA(c, cudaMemsetAsync(dq_fix, 0, sizeof(long long) * nq, c->stream));
  else GM_CUDA(c, cudaMemsetAsync(dq, 0, sizeof(float) * nq, c->stream));
  GM_LAUNCH(c, GM_KC_ATTENTION, launch_attention_backward(A, c->stream));
  return GM_OK;
}
int gm_attention_backward(gm_ctx *c, const void *q, const float *dout, const void *kv_pool, int pool_layers, int num_pages, int layer,
                          const int32_t *page_table, const int32_t *q_count, const int32_t *q_base, int batch, int q_stride,
                          float *dq, float *dk_pool, float *dv_pool) {
  return attention_backward_impl(c, q, dout, kv_pool, pool_layers, num_pages, layer, page_table, q_count, q_base, batch, q_stride, dq,
                                 dk_pool, dv_pool, nullptr, nullptr, nullptr);
}

// The attention half's forward values for one pass of rows x [batch * q_stride, d], with the forward pass's own kernels:
// c->xn = RMSNorm(x; ln1), c->qkv = the projection, and - with_attention - c->qbuf = the rotated (normed, biased) queries,
// c->attn_out = the attention output over the given cache, which is only read.  Leaves the plan (c->qn, c->qbase) in place.
static int head_attn_forward(gm_ctx *c, const float *x, const void *kv_pool, int num_pages, const int32_t *page_table,
                             const int32_t *q_count, const int32_t *q_base, int batch, int q_stride, bool with_attention) {
  const gm_config &cf = c->cfg;
  const gm_layer_weights &lw = c->w.head_layer;
  const int d = c->d, hd = cf.head_dim, NQKV = c->n_qkv, rows = batch * q_stride;
  int rc;
  if ((rc = run_plan_chunk(c, batch, q_count, q_base, q_stride)) != GM_OK) return rc;
  GM_LAUNCH(c, GM_KC_ELEMENTWISE,
            launch_rmsnorm(x, static_cast<const __nv_bfloat16 *>(lw.ln1), c->xn, nullptr, rows, d, cf.rms_eps, c->stream));
  if ((rc = run_gemm(c, c->xn, c->Mmax, &c->head_maps.wqkv, static_cast<const __nv_bfloat16 *>(lw.wqkv), rows, NQKV, d, c->qkv,
                     EPI_STORE_BF16, NQKV)) != GM_OK)
    return rc;
  if (!with_attention) return GM_OK;
  const int qrows = round16(q_stride * c->group);
  RopeAppendArgs R;
  R.qkv = c->qkv; R.batch = batch; R.QT = q_stride; R.n_q = cf.n_q_heads; R.n_kv = cf.n_kv_heads; R.hd = hd; R.layer = 0;
  R.num_pages = num_pages; R.max_pages_per_seq = cf.max_pages_per_seq; R.qrows = qrows; R.qn = c->qn; R.qbase = c->qbase;
  R.page_table = page_table; R.rope = c->rope; R.qbuf = c->qbuf; R.pool = nullptr; R.status = c->status;   // the cache is read, not rewritten
  R.bias = static_cast<const __nv_bfloat16 *>(lw.b_qkv);
  R.qnorm = static_cast<const __nv_bfloat16 *>(lw.q_norm); R.knorm = static_cast<const __nv_bfloat16 *>(lw.k_norm);
  R.eps = cf.rms_eps;
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_rope_append(R, c->stream));
  CUtensorMap kvm;
  if ((rc = kv_map(c, kv_pool, 1, num_pages, &kvm)) != GM_OK) return rc;
  AttnArgs T;
  T.kv_map = kvm; T.qbuf = c->qbuf; T.qn = c->qn; T.qbase = c->qbase; T.page_start = c->page_start; T.page_table = page_table;
  T.batch = batch; T.n_kv = cf.n_kv_heads; T.group = c->group; T.hd = hd; T.qrows = qrows; T.layer = 0; T.num_pages = num_pages;
  T.max_pages_per_seq = cf.max_pages_per_seq; T.n_ctas = c->sm_count;
  T.scale_log2e = static_cast<float>(1.4426950408889634 / std::sqrt(static_cast<double>(hd)));
  T.part_o = c->part_o; T.part_ml = c->part_ml; T.status = c->status; T.rows_used = q_stride * c->group;
  GM_LAUNCH(c, GM_KC_ATTENTION, launch_attention(T, c->stream));
  AttnCombineArgs Cb;
  Cb.part_o = c->part_o; Cb.part_ml = c->part_ml; Cb.qn = c->qn; Cb.page_start = c->page_start; Cb.batch = batch;
  Cb.n_kv = cf.n_kv_heads; Cb.group = c->group; Cb.hd = hd; Cb.qrows = qrows; Cb.QT = q_stride; Cb.n_ctas = c->sm_count;
  Cb.out = c->attn_out;
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_attention_combine(Cb, c->stream));
  return GM_OK;
}

// dxmid may be null here: rows whose outputs nothing consumed (the pass over the committed prefix) - only what later rows
// left on their cache entries flows back, the attention core and W_o are skipped and dw_o is left as it is
static int head_attn_backward_impl(gm_ctx *c, const float *x, const float *dxmid, const void *kv_pool, int num_pages,
                                   const int32_t *page_table, const int32_t *q_count, const int32_t *q_base, int batch, int q_stride,
                                   float *dk_pool, float *dv_pool, float *dx, float *dw_qkv, float *dw_o, float *dln1, float *db_qkv,
                                   float *dqk_norm, int refresh_weights, bool accum, bool forward_done = false,
                                   long long *dk_fix = nullptr, long long *dv_fix = nullptr) {
  const int wepi = accum ? EPI_ADD_F32 : EPI_STORE_F32;
  const bool fix = dk_fix != nullptr;                  // key / value gradients in the fixed-point planes instead of dk_pool / dv_pool
  if (!c || !x || !kv_pool || !page_table || !q_count || !q_base || !dx || !dw_qkv || !dw_o || !dln1 || batch < 1 || q_stride < 1 ||
      num_pages < 1 || (fix ? !dv_fix : (!dk_pool || !dv_pool)))
    return GM_ERR_INVALID_ARG;
  const gm_config &cf = c->cfg;
  const gm_layer_weights &lw = c->w.head_layer;
  const int d = c->d, hd = cf.head_dim, NQ = c->q_dim, NQKV = c->n_qkv, rows = batch * q_stride;
  if ((db_qkv != nullptr) != (lw.b_qkv != nullptr) || (dqk_norm != nullptr) != (lw.q_norm != nullptr)) return GM_ERR_INVALID_ARG;
  if ((cf.flags & GM_FLAG_SIMPLE_GEMM) || (d % 64) || (NQ % 64) || (NQKV % 64) || (hd != 64 && hd != 128) || c->group > 8 ||
      q_stride > cf.max_k + 1 || q_stride > 8 || batch > cf.max_batch * c->pf_vr || rows > c->Mmax)
    return GM_ERR_UNSUPPORTED;
  const __nv_bfloat16 *wqkv = static_cast<const __nv_bfloat16 *>(lw.wqkv), *wo = static_cast<const __nv_bfloat16 *>(lw.wo);
  const __nv_bfloat16 *ln1 = static_cast<const __nv_bfloat16 *>(lw.ln1);
  int rc;
  if (!c->hat_wo_t) {
    if ((rc = dev_alloc(c, &c->hat_wo_t, static_cast<size_t>(NQ) * d, false)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hat_wqkv_t, static_cast<size_t>(d) * NQKV, false)) != GM_OK) return rc;
    if (make_map(c, &c->hat_wo_t_map, c->hat_wo_t, NQ, d, 128) != GM_OK) return GM_ERR_CUDA;
    if (make_map(c, &c->hat_wqkv_t_map, c->hat_wqkv_t, d, NQKV, 128) != GM_OK) return GM_ERR_CUDA;
    refresh_weights = 1;
  }
  if (refresh_weights) {
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_transpose_bf16(wo, d, NQ, c->hat_wo_t, c->stream));             // [d, q_dim] -> [q_dim, d]
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_transpose_bf16(wqkv, NQKV, d, c->hat_wqkv_t, c->stream));       // [n_qkv, d] -> [d, n_qkv]
  }
  const int Mp = (rows + 63) / 64 * 64;
  if (Mp > c->hat_rows_cap) {
    const size_t M = static_cast<size_t>(Mp);
    if ((rc = dev_alloc(c, &c->hat_dy, M * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hat_dqkv_bf, M * NQKV)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hat_dyt, M * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hat_ot, M * NQ)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hat_dqkvt, M * NQKV)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hat_ht, M * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hat_do, M * NQ)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hat_dq, M * NQ)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hat_dqkv, M * NQKV)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hat_dh, M * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hat_t, M * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hat_tq, M * NQ)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hat_tk, M * (NQKV - NQ) / 2)) != GM_OK) return rc;
    c->hat_rows_cap = Mp;
  }
  if (fix && static_cast<size_t>(Mp) * NQ > c->hat_dq_fix_cap) {
    if ((rc = dev_alloc(c, &c->hat_dq_fix, static_cast<size_t>(Mp) * NQ)) != GM_OK) return rc;
    c->hat_dq_fix_cap = static_cast<size_t>(Mp) * NQ;
  }
  // ---- the forward's values, recomputed: h = RMSNorm(x; ln1), the projection, the rotated queries, the attention output ----
  if (!forward_done &&
      (rc = head_attn_forward(c, x, kv_pool, num_pages, page_table, q_count, q_base, batch, q_stride, dxmid != nullptr)) != GM_OK)
    return rc;
  const __nv_bfloat16 *bias = static_cast<const __nv_bfloat16 *>(lw.b_qkv);
  const __nv_bfloat16 *qnorm = static_cast<const __nv_bfloat16 *>(lw.q_norm), *knorm = static_cast<const __nv_bfloat16 *>(lw.k_norm);
  if (dxmid) {
  // ---- d(attention output) = dxmid W_o, then the attention core ----
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_cast_bf16(dxmid, c->hat_dy, static_cast<size_t>(rows) * d, c->stream));
  if ((rc = run_gemm(c, c->hat_dy, rows, &c->hat_wo_t_map, c->hat_wo_t, rows, NQ, d, c->hat_do, EPI_STORE_F32, static_cast<size_t>(NQ), false)) != GM_OK)
    return rc;
  if ((rc = attention_backward_impl(c, c->qbuf, c->hat_do, kv_pool, 1, num_pages, 0, page_table, c->qn, c->qbase, batch, q_stride,
                                    c->hat_dq, dk_pool, dv_pool, fix ? c->hat_dq_fix : nullptr, dk_fix, dv_fix)) != GM_OK)
    return rc;
  } else if (fix) {
    GM_CUDA(c, cudaMemsetAsync(c->hat_dq_fix, 0, sizeof(long long) * static_cast<size_t>(rows) * NQ, c->stream));
  } else {
    GM_CUDA(c, cudaMemsetAsync(c->hat_dq, 0, sizeof(float) * static_cast<size_t>(rows) * NQ, c->stream));
  }
  // ---- the rows' own entries are complete now: back through the rotation and the head norms, packed like the projection ----
  QkvGradArgs Q;
  Q.qkv = c->qkv; Q.bias = bias; Q.qnorm = qnorm; Q.knorm = knorm; Q.dq = c->hat_dq; Q.dk_pool = dk_pool; Q.dv_pool = dv_pool;
  if (fix) { Q.dq_fix = c->hat_dq_fix; Q.dk_fix = dk_fix; Q.dv_fix = dv_fix; }
  Q.qn = c->qn; Q.qbase = c->qbase; Q.page_table = page_table; Q.rope = c->rope; Q.batch = batch; Q.QT = q_stride;
  Q.n_q = cf.n_q_heads; Q.n_kv = cf.n_kv_heads; Q.hd = hd; Q.num_pages = num_pages; Q.max_pages_per_seq = cf.max_pages_per_seq;
  Q.eps = cf.rms_eps; Q.dqkv = c->hat_dqkv; Q.dqkv_bf = c->hat_dqkv_bf; Q.status = c->status;
  if (dqk_norm) { Q.tq = c->hat_tq; Q.tk = c->hat_tk; }
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_qkv_grad_rows(Q, c->stream));
  if (dqk_norm) {
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_colsum(c->hat_tq, rows * cf.n_q_heads, hd, dqk_norm, c->stream, accum, colsum_ws(c)));
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_colsum(c->hat_tk, rows * cf.n_kv_heads, hd, dqk_norm + hd, c->stream, accum, colsum_ws(c)));
  }
  if (db_qkv) GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_colsum(c->hat_dqkv, rows, NQKV, db_qkv, c->stream, accum, colsum_ws(c)));
  // ---- dh = dqkv W_qkv;  dx = dxmid + d RMSNorm;  dln1 ----
  if ((rc = run_gemm(c, c->hat_dqkv_bf, rows, &c->hat_wqkv_t_map, c->hat_wqkv_t, rows, d, NQKV, c->hat_dh, EPI_STORE_F32, static_cast<size_t>(d), false)) != GM_OK)
    return rc;
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_rmsnorm_grad(c->hat_dh, x, ln1, dx, rows, d, cf.rms_eps, c->stream, dxmid, c->hat_t));
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_colsum(c->hat_t, rows, d, dln1, c->stream, accum, colsum_ws(c)));
  // ---- weight gradients contract over the rows: operands transposed to [features, rows] (rows padded with zeros to Mp) ----
  GM_CUDA(c, cudaMemsetAsync(c->hat_dqkvt, 0, sizeof(__nv_bfloat16) * static_cast<size_t>(Mp) * NQKV, c->stream));
  GM_CUDA(c, cudaMemsetAsync(c->hat_ht, 0, sizeof(__nv_bfloat16) * static_cast<size_t>(Mp) * d, c->stream));
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_transpose_bf16(c->hat_dqkv_bf, rows, NQKV, c->hat_dqkvt, c->stream, Mp));
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_transpose_bf16(c->xn, rows, d, c->hat_ht, c->stream, Mp));
  CUtensorMap wm;
  if (dxmid) {                                       // dW_o [d, q_dim] = dxmid^T o
    GM_CUDA(c, cudaMemsetAsync(c->hat_dyt, 0, sizeof(__nv_bfloat16) * static_cast<size_t>(Mp) * d, c->stream));
    GM_CUDA(c, cudaMemsetAsync(c->hat_ot, 0, sizeof(__nv_bfloat16) * static_cast<size_t>(Mp) * NQ, c->stream));
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_transpose_bf16(c->hat_dy, rows, d, c->hat_dyt, c->stream, Mp));
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_transpose_bf16(c->attn_out, rows, NQ, c->hat_ot, c->stream, Mp));
    if (make_map(c, &wm, c->hat_ot, NQ, Mp, 128) != GM_OK) return GM_ERR_CUDA;
    if ((rc = run_gemm(c, c->hat_dyt, d, &wm, c->hat_ot, d, NQ, Mp, dw_o, wepi, static_cast<size_t>(NQ), false)) != GM_OK) return rc;
  }
  // dW_qkv [n_qkv, d] = dqkv^T h
  if (make_map(c, &wm, c->hat_ht, d, Mp, 128) != GM_OK) return GM_ERR_CUDA;
  return run_gemm(c, c->hat_dqkvt, NQKV, &wm, c->hat_ht, NQKV, d, Mp, dw_qkv, wepi, static_cast<size_t>(d), false);
}
int gm_head_attn_backward(gm_ctx *c, const float *x, const float *dxmid, const void *kv_pool, int num_pages,
                          const int32_t *page_table, const int32_t *q_count, const int32_t *q_base, int batch, int q_stride,
                          float *dk_pool, float *dv_pool, float *dx, float *dw_qkv, float *dw_o, float *dln1, float *db_qkv,
                          float *dqk_norm, int refresh_weights) {
  if (!dxmid) return GM_ERR_INVALID_ARG;
  return head_attn_backward_impl(c, x, dxmid, kv_pool, num_pages, page_table, q_count, q_base, batch, q_stride, dk_pool, dv_pool, dx,
                                 dw_qkv, dw_o, dln1, db_qkv, dqk_norm, refresh_weights, false);
}

// z = W_p [RMSNorm(E[token]) ; RMSNorm(hidden)] for `rows` pairs, with the forward pass's operand precision
static int head_z_forward(gm_ctx *c, int rows, const int32_t *tokens, const float *hidden, float *z) {
  GM_LAUNCH(c, GM_KC_ELEMENTWISE,
            launch_head_input_rows(static_cast<const __nv_bfloat16 *>(c->w.embed), tokens, hidden,
                                   static_cast<const __nv_bfloat16 *>(c->w.head_enorm), static_cast<const __nv_bfloat16 *>(c->w.head_hnorm),
                                   rows, c->d, c->V, c->cfg.rms_eps, c->zin, c->hub_e, c->status, c->stream));
  return run_gemm(c, c->zin, c->Mmax, &c->head_proj_map, static_cast<const __nv_bfloat16 *>(c->w.head_proj), rows, c->d, 2 * c->d, z,
                  EPI_STORE_F32, c->d);
}

int gm_head_update_backward(gm_ctx *c, gm_state *st, int n_cycles, int k, const int32_t *cycle_seq, const gm_record *rec,
                            const int32_t *seq_tok, int tok_stride, const int32_t *scratch_pages, const void *grad_logits,
                            const void *seq_hidden, int hid_stride, const int32_t *seq_len, int max_len, float *dk_pool,
                            float *dv_pool, const gm_head_grads *out) {
  if (!grad_logits) return GM_ERR_INVALID_ARG;
  return head_update_backward_impl(c, st, n_cycles, k, cycle_seq, rec, seq_tok, tok_stride, scratch_pages, grad_logits, seq_hidden,
                                   hid_stride, seq_len, max_len, dk_pool, dv_pool, out, 1.0f, nullptr, nullptr);
}

}  // extern "C"

int gmh::head_update_backward_impl(gm_ctx *c, gm_state *st, int n_cycles, int k, const int32_t *cycle_seq, const gm_record *rec,
                              const int32_t *seq_tok, int tok_stride, const int32_t *scratch_pages, const void *grad_logits,
                              const void *seq_hidden, int hid_stride, const int32_t *seq_len, int max_len, float *dk_pool,
                              float *dv_pool, const gm_head_grads *out, float temperature, float *alpha, float *lse) {
  NvtxRange nvtx_range("gm_head_update_backward");
  int rc = check_state(c, st, k);
  if (rc) return rc;
  const bool own_grad = grad_logits == nullptr;          // the logit gradients are formed here, chunk by chunk
  if (n_cycles < 1 || !cycle_seq || !rec || !rec->start_hidden || !rec->start_pos || !rec->drafts || !seq_tok || tok_stride < 2 ||
      !scratch_pages || !seq_hidden || !seq_len || max_len < 2 || tok_stride < max_len || hid_stride < max_len - 1 ||
      (dk_pool != nullptr) != (dv_pool != nullptr) || !out)
    return GM_ERR_INVALID_ARG;
  if (own_grad && (!alpha || !lse || !rec->top_index || !rec->top_logprob || !rec->accepted)) return GM_ERR_INVALID_ARG;
  if (own_grad && (!(temperature > 0.f) || !std::isfinite(temperature))) return GM_ERR_UNSUPPORTED;
  const gm_config &cf = c->cfg;
  const gm_layer_weights &lw = c->w.head_layer;
  if (!out->proj || !out->enorm || !out->hnorm || !out->final_norm || !out->ln1 || !out->ln2 || !out->wqkv || !out->wo ||
      !out->w_gate_up || !out->w_down || (out->b_qkv != nullptr) != (lw.b_qkv != nullptr) ||
      (out->qk_norm != nullptr) != (lw.q_norm != nullptr))
    return GM_ERR_INVALID_ARG;
  if (max_len + cf.max_k + 1 > cf.max_pages_per_seq * GM_PAGE) return GM_ERR_KV_CAPACITY;
  const int d = c->d, F = c->F, MB = cf.max_batch, PS = cf.max_k + 1, hd = cf.head_dim;
  const int B = st->batch, QT = cf.max_k + 1, VR = c->pf_vr, R = B * VR;
  if (!c->v_table) {                                   // the chains' virtual state (as gm_reconstruct makes it)
    const size_t MBs = static_cast<size_t>(MB);
    if ((rc = dev_alloc(c, &c->v_kv_len, MBs)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->v_pending_n, MBs)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->v_pending_tok, MBs * PS)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->v_pending_hidden, MBs * PS * c->d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->v_table, MBs * cf.max_pages_per_seq)) != GM_OK) return rc;
  }
  const int cap = std::max(MB, R * QT);
  if (cap > c->hub_rows_cap) {
    const size_t S = static_cast<size_t>(MB) * cf.max_k * d, M = static_cast<size_t>(cap) * d;
    if ((rc = dev_alloc(c, &c->hub_states, S)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hub_gn, S)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hub_dstate, S)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hub_t, S)) != GM_OK) return rc;
    for (float **p : {&c->hub_hidden, &c->hub_z, &c->hub_xmid, &c->hub_dg, &c->hub_dxmid, &c->hub_dz, &c->hub_dhid, &c->hub_e})
      if ((rc = dev_alloc(c, p, M)) != GM_OK) return rc;
    for (int32_t **p : {&c->hub_tok, &c->hub_base, &c->hub_cnt})
      if ((rc = dev_alloc(c, p, static_cast<size_t>(cap))) != GM_OK) return rc;
    c->hub_rows_cap = cap;
  }
  // every output starts at zero; the passes add to them.  The cache entries' gradients are accumulated in fixed point
  // (64-bit integer additions), so that the update does not depend on the order in which the chains' CTAs arrive.
  const size_t NQKV = c->n_qkv, NQ = c->q_dim;
  const size_t plane = static_cast<size_t>(cf.head_num_pages) * cf.n_kv_heads * GM_PAGE * hd;
  if (plane > c->hub_fix_cap) {
    if ((rc = dev_alloc(c, &c->hub_dk_fix, plane, false)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hub_dv_fix, plane, false)) != GM_OK) return rc;
    c->hub_fix_cap = plane;
  }
  GM_CUDA(c, cudaMemsetAsync(c->hub_dk_fix, 0, sizeof(long long) * plane, c->stream));
  GM_CUDA(c, cudaMemsetAsync(c->hub_dv_fix, 0, sizeof(long long) * plane, c->stream));
  struct { float *p; size_t n; } outs[] = {{out->proj, static_cast<size_t>(2) * d * d}, {out->enorm, static_cast<size_t>(d)},
      {out->hnorm, static_cast<size_t>(d)}, {out->final_norm, static_cast<size_t>(d)}, {out->ln1, static_cast<size_t>(d)},
      {out->ln2, static_cast<size_t>(d)}, {out->wqkv, NQKV * d}, {out->wo, NQ * d}, {out->w_gate_up, static_cast<size_t>(2) * F * d},
      {out->w_down, static_cast<size_t>(F) * d}, {out->b_qkv, NQKV}, {out->qk_norm, static_cast<size_t>(2) * hd}};
  for (const auto &o : outs)
    if (o.p) GM_CUDA(c, cudaMemsetAsync(o.p, 0, sizeof(float) * o.n, c->stream));
  const __nv_bfloat16 *fnorm = static_cast<const __nv_bfloat16 *>(c->w.head_final_norm);
  bool refresh = true;                                   // the transposed weight copies are remade once per call

  // ---- the chains, a chunk of max_batch at a time: replay (Eq. 4), then the applications from the last one back ----
  for (int off = 0; off < n_cycles; off += MB) {
    const int m = std::min(MB, n_cycles - off);
    ChainSetupArgs A;
    A.cycle_seq = cycle_seq + off; A.start_pos = rec->start_pos + off;
    A.start_hidden = static_cast<const __nv_bfloat16 *>(rec->start_hidden) + static_cast<size_t>(off) * d;
    A.seq_tok = seq_tok; A.scratch_pages = scratch_pages + 2 * static_cast<size_t>(off);
    A.head_page_table = st->head_page_table; A.pool = static_cast<__nv_bfloat16 *>(st->head_kv_pool);
    A.n_seq = st->batch; A.tok_stride = tok_stride; A.k = k; A.d = d; A.vocab = c->V;
    A.max_pages_per_seq = cf.max_pages_per_seq; A.num_pages = cf.head_num_pages;
    A.page_elems = cf.n_kv_heads * GM_PAGE * hd; A.pend_stride = PS;
    A.v_kv_len = c->v_kv_len; A.v_pending_n = c->v_pending_n; A.v_pending_tok = c->v_pending_tok; A.v_table = c->v_table;
    A.v_pending_hidden = c->v_pending_hidden; A.status = c->status;
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_chain_setup(A, m, c->stream));
    gm_state vs = *st;
    vs.batch = m; vs.kv_len = c->v_kv_len; vs.head_page_table = c->v_table; vs.pending_n = c->v_pending_n;
    vs.pending_tok = c->v_pending_tok; vs.pending_hidden = c->v_pending_hidden;
    c->state_out = c->hub_states;
    rc = draft_impl(c, &vs, k, 1.0f, nullptr, 0, 0, rec->drafts + static_cast<size_t>(off) * k, c->ws_draft_logits, nullptr, true);
    c->state_out = nullptr;
    if (rc) return rc;
    // every state's term through its own logits, and the final norm's weight
    const __nv_bfloat16 *gl = static_cast<const __nv_bfloat16 *>(grad_logits) + static_cast<size_t>(off) * k * c->V;
    if (own_grad) {                                    // overlaps and objective gradient of this chunk, from the replay's logits
      if (!c->hub_glogits && (rc = dev_alloc(c, &c->hub_glogits, static_cast<size_t>(MB) * cf.max_k * c->V, false)) != GM_OK) return rc;
      const size_t ro = static_cast<size_t>(off) * k;
      OverlapArgs O;
      O.logits = c->ws_draft_logits; O.top_index = rec->top_index + ro * 64;
      O.top_logprob = static_cast<const __nv_bfloat16 *>(rec->top_logprob) + ro * 64; O.alpha = alpha + ro; O.lse = lse + ro;
      O.V = c->V; O.inv_temp = 1.0f / temperature;
      GM_LAUNCH(c, GM_KC_RECORD, launch_overlap(O, m * k, c->stream));
      DcaGradArgs G;
      G.logits = c->ws_draft_logits; G.top_index = O.top_index; G.top_logprob = O.top_logprob; G.alpha = alpha + ro; G.lse = lse + ro;
      G.accepted = rec->accepted + off; G.grad = c->hub_glogits; G.V = c->V; G.K = k; G.n = m; G.n_total = n_cycles;
      G.inv_temp = O.inv_temp;
      GM_LAUNCH(c, GM_KC_RECORD, launch_dca_grad(G, c->stream));
      gl = c->hub_glogits;
    }
    if ((rc = gm_head_state_grad(c, m * k, gl, c->hub_states, c->hub_gn, c->hub_dstate, 0)) != GM_OK) return rc;   // the LM head is the backbone's: its copy stays
    GM_LAUNCH(c, GM_KC_ELEMENTWISE,
              launch_rmsnorm_grad(c->hub_gn, c->hub_states, fnorm, nullptr, m * k, d, cf.rms_eps, c->stream, nullptr, c->hub_t));
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_colsum(c->hub_t, m * k, d, out->final_norm, c->stream, true, colsum_ws(c)));
    for (int j = k; j >= 1; --j) {
      StepRowsArgs S;
      S.k = j; S.K = k; S.d = d; S.vocab = c->V; S.start_pos = rec->start_pos + off;
      S.start_hidden = static_cast<const __nv_bfloat16 *>(rec->start_hidden) + static_cast<size_t>(off) * d;
      S.first_tok = c->v_pending_tok; S.first_tok_stride = PS; S.drafts = rec->drafts + static_cast<size_t>(off) * k;
      S.states = c->hub_states; S.dstate = c->hub_dstate; S.hidden = c->hub_hidden; S.dg = c->hub_dg;
      S.tok = c->hub_tok; S.base = c->hub_base; S.count = c->hub_cnt; S.status = c->status;
      GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_step_rows(S, m, c->stream));
      // the application's forward values: z, then xmid = z + W_o attention(...)
      if ((rc = head_z_forward(c, m, c->hub_tok, c->hub_hidden, c->hub_z)) != GM_OK) return rc;
      if ((rc = head_attn_forward(c, c->hub_z, st->head_kv_pool, cf.head_num_pages, c->v_table, c->hub_cnt, c->hub_base, m, 1, true)) != GM_OK)
        return rc;
      GM_CUDA(c, cudaMemcpyAsync(c->hub_xmid, c->hub_z, sizeof(float) * static_cast<size_t>(m) * d, cudaMemcpyDeviceToDevice, c->stream));
      if ((rc = run_gemm(c, c->attn_out, c->Mmax, &c->head_maps.wo, static_cast<const __nv_bfloat16 *>(lw.wo), m, d, c->q_dim, c->hub_xmid,
                         EPI_ADD_F32, d)) != GM_OK)
        return rc;
      if ((rc = head_ffn_backward_impl(c, m, c->hub_xmid, c->hub_dg, c->hub_dxmid, out->w_gate_up, out->w_down, out->ln2, refresh, true)) != GM_OK)
        return rc;
      if ((rc = head_attn_backward_impl(c, c->hub_z, c->hub_dxmid, st->head_kv_pool, cf.head_num_pages, c->v_table, c->hub_cnt, c->hub_base,
                                        m, 1, nullptr, nullptr, c->hub_dz, out->wqkv, out->wo, out->ln1, out->b_qkv, out->qk_norm, refresh,
                                        true, true, c->hub_dk_fix, c->hub_dv_fix)) != GM_OK)
        return rc;
      if ((rc = head_input_backward_impl(c, m, c->hub_tok, c->hub_hidden, c->hub_dz, c->hub_dhid, out->proj, out->enorm, out->hnorm, refresh,
                                         true)) != GM_OK)
        return rc;
      refresh = false;
      // Eq. 4: application j >= 2 consumed the state of application j - 1
      if (j >= 2) GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_add_state_grad(c->hub_dstate, c->hub_dhid, m, k, j - 2, d, c->stream));
    }
  }
  // ---- what the chains left on the copied part of their boundary pages belongs to the shared originals ----
  FoldArgs Fo;
  Fo.cycle_seq = cycle_seq; Fo.start_pos = rec->start_pos; Fo.scratch_pages = scratch_pages; Fo.head_page_table = st->head_page_table;
  Fo.n_seq = st->batch; Fo.max_pages_per_seq = cf.max_pages_per_seq; Fo.num_pages = cf.head_num_pages; Fo.n_kv = cf.n_kv_heads; Fo.hd = hd;
  Fo.dk_pool = nullptr; Fo.dv_pool = nullptr; Fo.dk_fix = c->hub_dk_fix; Fo.dv_fix = c->hub_dv_fix;
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_fold_boundary(Fo, n_cycles, c->stream));
  // ---- the pass over the committed prefixes: nothing consumed these rows' outputs, only their cache entries ----
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_dup_table_rows(st->head_page_table, B, VR, cf.max_pages_per_seq, c->pf_vtable[1], c->stream));
  for (int base = 0; base + 1 < max_len; base += VR * QT) {
    ChunkSetupArgs Cs;
    Cs.prompt_tok = seq_tok; Cs.prompt_len = seq_len; Cs.batch = B; Cs.stride = tok_stride; Cs.base = base; Cs.QT = QT;
    Cs.max_len = max_len; Cs.pair_stride = QT; Cs.vr = VR; Cs.row_n = c->pf_row_n; Cs.head_n = c->pf_head_n;
    Cs.pair_tok = c->pf_pair_tok; Cs.row_base = c->pf_row_base; Cs.status = c->status;
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_chunk_setup(Cs, c->stream));
    GM_LAUNCH(c, GM_KC_ELEMENTWISE,
              launch_gather_chunk_hidden(static_cast<const __nv_bfloat16 *>(seq_hidden), hid_stride, c->pf_row_base, R, VR, QT, d,
                                         c->pf_head_n, c->pf_hidden, c->stream));
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_rows_to_f32(c->pf_hidden, c->pf_head_n, R * QT, QT, d, c->hub_hidden, c->stream));
    if ((rc = head_z_forward(c, R * QT, c->pf_pair_tok, c->hub_hidden, c->hub_z)) != GM_OK) return rc;
    if ((rc = head_attn_backward_impl(c, c->hub_z, nullptr, st->head_kv_pool, cf.head_num_pages, c->pf_vtable[1], c->pf_head_n,
                                      c->pf_row_base, R, QT, nullptr, nullptr, c->hub_dz, out->wqkv, out->wo, out->ln1, out->b_qkv,
                                      out->qk_norm, 0, true, false, c->hub_dk_fix, c->hub_dv_fix)) != GM_OK)
      return rc;
    if ((rc = head_input_backward_impl(c, R * QT, c->pf_pair_tok, c->hub_hidden, c->hub_dz, nullptr, out->proj, out->enorm, out->hnorm, 0,
                                       true)) != GM_OK)
      return rc;
  }
  if (dk_pool) {                                       // the cache entries' gradients, for a caller that wants them
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_fix_to_float(c->hub_dk_fix, dk_pool, plane, c->stream));
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_fix_to_float(c->hub_dv_fix, dv_pool, plane, c->stream));
  }
  return GM_OK;
}
