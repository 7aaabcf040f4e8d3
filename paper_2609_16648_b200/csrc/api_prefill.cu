// C ABI of libgm: prompt prefill (backbone + draft head) and the rebuild of the head cache from recorded pairs.
// Host code only; the helpers it calls are declared in gm_internal.h.
#include "gm_internal.h"

// Virtual rows per sequence for a prefill pass (at most the count the workspaces were sized for).  A pass of m
// 256-token blocks runs every projection as ceil(tiles * m / SMs) waves, and with a few hundred tokens more or less
// a projection can need a whole extra wave (20 feature tiles x 8 blocks = 160 CTAs on 148 SMs); the cost per token of
// each candidate is estimated from the wave counts with the same tiling rules the projections use, and the cheapest
// wins.  GM_PREFILL_VR forces a value.
static int pick_prefill_vr(const gm_ctx *c, int B, int QT) {
  const int vr_max = c->pf_vr;
  if (const char *ov = std::getenv("GM_PREFILL_VR")) {
    const int v = std::atoi(ov);
    if (v >= 1 && v <= vr_max) return v;
  }
  const int sms = c->sm_count;
  const int shape[4][2] = {{c->n_qkv, c->d}, {c->d, c->q_dim}, {2 * c->F, c->d}, {c->d, c->F}};   // (N, K) per projection
  int best = vr_max;
  double best_cost = 0.0;
  for (int vr = vr_max; vr >= 1; --vr) {
    const int rows = B * vr * QT, m = (rows + 255) / 256;
    double cost = 0.0;
    for (const auto &g : shape) {
      const int tiles = (g[0] + 127) / 128, kb = g[1] / 64;
      const int wt = tiles * m >= 2 * sms ? 2 : 1;
      const int ctas = ((tiles + wt - 1) / wt) * m;
      cost += static_cast<double>((ctas + sms - 1) / sms) * kb * wt + 24.0;            // + fixed cost of a launch
    }
    cost /= rows;
    if (vr == vr_max || cost < best_cost * 0.97) { best = vr; best_cost = cost; }
  }
  return best;
}

extern "C" {

int gm_prefill(gm_ctx *c, gm_state *st, const int32_t *prompt_tok, const int32_t *prompt_len, int prompt_stride,
               int max_prompt_len, float temperature, const uint32_t *u24_first, uint64_t seed, int32_t *first_token,
               float *dbg_p) {
  NvtxRange nvtx_range("gm_prefill");
  int rc = check_state(c, st, 1);
  if (rc) return rc;
  if (!prompt_tok || !prompt_len || max_prompt_len < 1 || prompt_stride < max_prompt_len) return GM_ERR_INVALID_ARG;
  const gm_config &cf = c->cfg;
  if (max_prompt_len + cf.max_k + 1 > cf.max_pages_per_seq * GM_PAGE) return GM_ERR_KV_CAPACITY;
  SamplerArgs S;
  if ((rc = fill_sampler(c, S, temperature)) != GM_OK) return rc;
  // Every pass gives each prompt VR consecutive chunks of QT positions: VR "virtual rows" per sequence, which the
  // planner, the rotary/append kernel and attention treat as independent sequences sharing the prompt's page table
  // (all keys of the pass are appended before attention runs, and each row attends only positions up to its own).
  const int B = st->batch, QT = cf.max_k + 1, VR = pick_prefill_vr(c, B, QT), R = B * VR;
  PhaseShape ph;
  ph.B = R; ph.QT = QT; ph.M = R * QT; ph.qrows = round16(QT * c->group);
  CUtensorMap kvm, hkvm;
  if ((rc = kv_map(c, st->kv_pool, cf.n_layers, cf.num_pages, &kvm)) != GM_OK) return rc;
  if ((rc = kv_map(c, st->head_kv_pool, 1, cf.head_num_pages, &hkvm)) != GM_OK) return rc;
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_dup_table_rows(st->page_table, B, VR, cf.max_pages_per_seq, c->pf_vtable[0], c->stream));
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_dup_table_rows(st->head_page_table, B, VR, cf.max_pages_per_seq, c->pf_vtable[1], c->stream));
  for (int base = 0; base < max_prompt_len; base += VR * QT) {
    ChunkSetupArgs Cs;
    Cs.prompt_tok = prompt_tok; Cs.prompt_len = prompt_len; Cs.batch = B; Cs.stride = prompt_stride; Cs.base = base;
    Cs.QT = QT; Cs.max_len = max_prompt_len; Cs.pair_stride = QT; Cs.vr = VR; Cs.row_n = c->pf_row_n; Cs.head_n = c->pf_head_n;
    Cs.pair_tok = c->pf_pair_tok; Cs.row_base = c->pf_row_base; Cs.status = c->status;
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_chunk_setup(Cs, c->stream));
    // the backbone over positions base .. base + VR * QT - 1 of every prompt that reaches them
    if ((rc = run_plan_chunk(c, R, c->pf_row_n, c->pf_row_base, QT)) != GM_OK) return rc;
    GM_LAUNCH(c, GM_KC_ELEMENTWISE,
              launch_embed_chunk(static_cast<const __nv_bfloat16 *>(c->w.embed),
                                 static_cast<const __nv_bfloat16 *>(c->layers[0].ln1), prompt_tok, prompt_stride,
                                 c->pf_row_base, c->pf_row_n, R, VR, QT, c->d, c->V, cf.rms_eps, c->x, c->xn, c->status,
                                 c->stream));
    for (int l = 0; l < cf.n_layers; ++l) {
      const bool last = l + 1 == cf.n_layers;
      rc = run_layer(c, c->layers[l], c->lmaps[l], ph, kvm, static_cast<__nv_bfloat16 *>(st->kv_pool), l, cf.num_pages,
                     c->pf_vtable[0], last ? nullptr : static_cast<const __nv_bfloat16 *>(c->layers[l + 1].ln1),
                     last ? c->pf_hidden : nullptr, last ? nullptr : &c->layers[l + 1], last ? nullptr : &c->lmaps[l + 1],
                     l > 0);
      if (rc) return rc;
    }
    if (c->capture)
      GM_LAUNCH(c, GM_KC_ELEMENTWISE,
                launch_capture_chunk(c->pf_hidden, c->pf_row_n, c->pf_row_base, R, VR, QT, c->d, c->capture,
                                     c->capture_stride, c->stream));
    GM_LAUNCH(c, GM_KC_ELEMENTWISE,
              launch_prefill_last(c->x, c->pf_hidden, c->pf_row_n, c->pf_row_base, prompt_len, R, VR, QT, c->d, QT,
                                  c->pf_xlast, static_cast<__nv_bfloat16 *>(st->pending_hidden), c->stream));
    // the draft head over the pairs (hidden of position t, token t + 1) of the same chunk, at head positions t
    if (base + 1 < max_prompt_len) {
      if ((rc = run_plan_chunk(c, R, c->pf_head_n, c->pf_row_base, QT)) != GM_OK) return rc;
      HeadInputArgs H;
      H.mode = PHASE_DRAFT_FIRST; H.batch = R; H.QT = QT; H.d = c->d; H.vocab = c->V; H.max_k = cf.max_k; H.k = 1; H.j = 1;
      H.eps = cf.rms_eps; H.embed = static_cast<const __nv_bfloat16 *>(c->w.embed);
      H.we = static_cast<const __nv_bfloat16 *>(c->w.head_enorm); H.wh = static_cast<const __nv_bfloat16 *>(c->w.head_hnorm);
      H.pending_tok = c->pf_pair_tok; H.pending_n = c->pf_head_n; H.pending_hidden = c->pf_hidden; H.draft_tok = nullptr;
      H.g_prev = c->g; H.zin = c->zin; H.status = c->status;
      GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_head_input(H, c->stream));
      rc = run_gemm(c, c->zin, c->Mmax, &c->head_proj_map, static_cast<const __nv_bfloat16 *>(c->w.head_proj), ph.M, c->d,
                    2 * c->d, c->x, EPI_STORE_F32, c->d);
      if (rc) return rc;
      GM_LAUNCH(c, GM_KC_ELEMENTWISE,
                launch_rmsnorm(c->x, static_cast<const __nv_bfloat16 *>(c->w.head_layer.ln1), c->xn, nullptr, ph.M, c->d,
                               cf.rms_eps, c->stream));
      // only the pairs' cache entries matter: the head's outputs on prompt rows are read by nothing
      rc = run_layer(c, c->w.head_layer, c->head_maps, ph, hkvm, static_cast<__nv_bfloat16 *>(st->head_kv_pool), 0,
                     cf.head_num_pages, c->pf_vtable[1], nullptr, nullptr, nullptr, nullptr, false, true);
      if (rc) return rc;
    }
  }
  // first response token: final norm + LM head on the hidden state of each prompt's last token, one draw per sequence
  GM_LAUNCH(c, GM_KC_ELEMENTWISE,
            launch_rmsnorm(c->pf_xlast, static_cast<const __nv_bfloat16 *>(c->w.final_norm), c->xn, nullptr, B, c->d,
                           cf.rms_eps, c->stream));
  rc = run_gemm(c, c->xn, c->Mmax, &c->lm_head_map, static_cast<const __nv_bfloat16 *>(c->w.lm_head), B, c->V, c->d,
                c->ws_target_logits, EPI_STORE_BF16, c->V);
  if (rc) return rc;
  S.K = 0; S.target_logits = c->ws_target_logits; S.tgt_bstride = c->V; S.draft_logits = nullptr;
  S.u24 = u24_first; S.u_stride = 1; S.seed = seed; S.step = 0; S.slot_final = SLOT_FINAL;
  S.accept_len = nullptr; S.next_token = c->pf_first; S.tok_out_stride = 1; S.dbg_p = dbg_p; S.dbg_q = nullptr; S.commit = 0;
  GM_LAUNCH(c, GM_KC_SAMPLER, run_sampler(c, S, B));
  GM_LAUNCH(c, GM_KC_ELEMENTWISE,
            launch_prefill_finish(prompt_len, c->pf_first, B, QT, st->kv_len, st->pending_n, st->pending_tok, c->stream));
  if (first_token)
    GM_CUDA(c, cudaMemcpyAsync(first_token, c->pf_first, sizeof(int32_t) * B, cudaMemcpyDeviceToDevice, c->stream));
  return GM_OK;
}

// ---- forward pass of the head update on recorded cycles -------------------------------------------------------------
int gm_head_prefill(gm_ctx *c, gm_state *st, const void *seq_hidden, int hid_stride, const int32_t *seq_tok,
                    int tok_stride, const int32_t *seq_len, int max_len) {
  NvtxRange nvtx_range("gm_head_prefill");
  int rc = check_state(c, st, 1);
  if (rc) return rc;
  if (!seq_hidden || !seq_tok || !seq_len || max_len < 1 || tok_stride < max_len || hid_stride < max_len - 1)
    return GM_ERR_INVALID_ARG;
  const gm_config &cf = c->cfg;
  if (max_len + cf.max_k + 1 > cf.max_pages_per_seq * GM_PAGE) return GM_ERR_KV_CAPACITY;
  const int B = st->batch, QT = cf.max_k + 1, VR = c->pf_vr, R = B * VR;          // virtual rows as in gm_prefill
  PhaseShape ph;
  ph.B = R; ph.QT = QT; ph.M = R * QT; ph.qrows = round16(QT * c->group);
  CUtensorMap hkvm;
  if ((rc = kv_map(c, st->head_kv_pool, 1, cf.head_num_pages, &hkvm)) != GM_OK) return rc;
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_dup_table_rows(st->head_page_table, B, VR, cf.max_pages_per_seq, c->pf_vtable[1], c->stream));
  for (int base = 0; base + 1 < max_len; base += VR * QT) {
    ChunkSetupArgs Cs;
    Cs.prompt_tok = seq_tok; Cs.prompt_len = seq_len; Cs.batch = B; Cs.stride = tok_stride; Cs.base = base; Cs.QT = QT;
    Cs.max_len = max_len; Cs.pair_stride = QT; Cs.vr = VR; Cs.row_n = c->pf_row_n; Cs.head_n = c->pf_head_n;
    Cs.pair_tok = c->pf_pair_tok; Cs.row_base = c->pf_row_base; Cs.status = c->status;
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_chunk_setup(Cs, c->stream));
    GM_LAUNCH(c, GM_KC_ELEMENTWISE,
              launch_gather_chunk_hidden(static_cast<const __nv_bfloat16 *>(seq_hidden), hid_stride, c->pf_row_base, R, VR, QT,
                                         c->d, c->pf_head_n, c->pf_hidden, c->stream));
    if ((rc = run_plan_chunk(c, R, c->pf_head_n, c->pf_row_base, QT)) != GM_OK) return rc;
    HeadInputArgs H;
    H.mode = PHASE_DRAFT_FIRST; H.batch = R; H.QT = QT; H.d = c->d; H.vocab = c->V; H.max_k = cf.max_k; H.k = 1; H.j = 1;
    H.eps = cf.rms_eps; H.embed = static_cast<const __nv_bfloat16 *>(c->w.embed);
    H.we = static_cast<const __nv_bfloat16 *>(c->w.head_enorm); H.wh = static_cast<const __nv_bfloat16 *>(c->w.head_hnorm);
    H.pending_tok = c->pf_pair_tok; H.pending_n = c->pf_head_n; H.pending_hidden = c->pf_hidden; H.draft_tok = nullptr;
    H.g_prev = c->g; H.zin = c->zin; H.status = c->status;
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_head_input(H, c->stream));
    rc = run_gemm(c, c->zin, c->Mmax, &c->head_proj_map, static_cast<const __nv_bfloat16 *>(c->w.head_proj), ph.M, c->d,
                  2 * c->d, c->x, EPI_STORE_F32, c->d);
    if (rc) return rc;
    GM_LAUNCH(c, GM_KC_ELEMENTWISE,
              launch_rmsnorm(c->x, static_cast<const __nv_bfloat16 *>(c->w.head_layer.ln1), c->xn, nullptr, ph.M, c->d,
                             cf.rms_eps, c->stream));
    rc = run_layer(c, c->w.head_layer, c->head_maps, ph, hkvm, static_cast<__nv_bfloat16 *>(st->head_kv_pool), 0,
                   cf.head_num_pages, c->pf_vtable[1], nullptr, nullptr, nullptr, nullptr, false, true);   // cache entries only
    if (rc) return rc;
  }
  return GM_OK;
}

}  // extern "C"
