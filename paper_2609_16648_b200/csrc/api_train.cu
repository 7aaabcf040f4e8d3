// C ABI of libgm: one update of the draft head on recorded cycles (Alg. 1, "update phi"): cache rebuild and draft-path
// reconstruction with the current parameters (Eq. 4), the objective (Eq. 5-9), its gradient with respect to every
// parameter of the head, and AdamW on the head's parameter group (App. B).  Host code only: every step is one of the
// library's own entry points or the driver behind gm_head_update_backward (which replays each chunk of chains once, for
// the objective and for the backward pass alike); this file owns the optimizer state and the order of the calls.
#include "gm_internal.h"

namespace gm {
namespace {

// the head's parameter tensors, in the order of gm_head_grads
struct ParamRef { const void *bf16; float *grad; size_t n; };

int collect_params(gm_ctx *c, const gm_head_grads &g, ParamRef (&out)[13]) {
  const gm_layer_weights &lw = c->w.head_layer;
  const size_t d = c->d, F = c->F, NQKV = c->n_qkv, NQ = c->q_dim, hd = c->cfg.head_dim;
  int n = 0;
  out[n++] = {c->w.head_proj, g.proj, 2 * d * d};
  out[n++] = {c->w.head_enorm, g.enorm, d};
  out[n++] = {c->w.head_hnorm, g.hnorm, d};
  out[n++] = {c->w.head_final_norm, g.final_norm, d};
  out[n++] = {lw.ln1, g.ln1, d};
  out[n++] = {lw.ln2, g.ln2, d};
  out[n++] = {lw.wqkv, g.wqkv, NQKV * d};
  out[n++] = {lw.wo, g.wo, NQ * d};
  out[n++] = {lw.w_gate_up, g.w_gate_up, 2 * F * d};
  out[n++] = {lw.w_down, g.w_down, F * d};
  if (lw.b_qkv) out[n++] = {lw.b_qkv, g.b_qkv, NQKV};
  if (lw.q_norm) {
    out[n++] = {lw.q_norm, g.qk_norm, hd};
    out[n++] = {lw.k_norm, g.qk_norm + hd, hd};
  }
  return n;
}

}  // namespace
}  // namespace gm

extern "C" {

int gm_head_update_step(gm_ctx *c, gm_state *st, int n_cycles, int k, float temperature, const int32_t *cycle_seq,
                        const gm_record *rec, const int32_t *seq_tok, int tok_stride, const int32_t *scratch_pages,
                        const void *seq_hidden, int hid_stride, const int32_t *seq_len, int max_len, int step, float lr,
                        float beta1, float beta2, float eps, float weight_decay, float *mean_loss) {
  using namespace gm;
  NvtxRange nvtx_range("gm_head_update_step");
  int rc = check_state(c, st, k);
  if (rc) return rc;
  if (n_cycles < 1 || !rec || !rec->accepted || !mean_loss || step < 1) return GM_ERR_INVALID_ARG;
  if (step != c->hu_step + 1) return GM_ERR_INVALID_ARG;     // the moments' bias correction counts the updates: 1, 2, 3, ...
  const gm_config &cf = c->cfg;
  const size_t d = c->d, F = c->F, NQKV = c->n_qkv, NQ = c->q_dim, hd = cf.head_dim;
  // ---- state owned by the context: gradients, optimizer state, per-call buffers ----
  if (!c->hu_grads.proj) {
    gm_head_grads &g = c->hu_grads;
    if ((rc = dev_alloc(c, &g.proj, 2 * d * d)) != GM_OK) return rc;
    for (float **p : {&g.enorm, &g.hnorm, &g.final_norm, &g.ln1, &g.ln2})
      if ((rc = dev_alloc(c, p, d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &g.wqkv, NQKV * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &g.wo, NQ * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &g.w_gate_up, 2 * F * d)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &g.w_down, F * d)) != GM_OK) return rc;
    if (c->w.head_layer.b_qkv && (rc = dev_alloc(c, &g.b_qkv, NQKV)) != GM_OK) return rc;
    if (c->w.head_layer.q_norm && (rc = dev_alloc(c, &g.qk_norm, 2 * hd)) != GM_OK) return rc;
    ParamRef ps[13];
    const int np = collect_params(c, g, ps);
    size_t total = 0;
    for (int i = 0; i < np; ++i) total += (ps[i].n + 3) & ~static_cast<size_t>(3);
    if ((rc = dev_alloc(c, &c->hu_master, total, false)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hu_m, total)) != GM_OK) return rc;       // zeroed: the moments start at 0
    if ((rc = dev_alloc(c, &c->hu_v, total)) != GM_OK) return rc;
    // fp32 master copies start from the bf16 parameters the forward pass reads
    size_t o = 0;
    for (int i = 0; i < np; ++i) {
      GM_LAUNCH(c, GM_KC_ELEMENTWISE,
                launch_widen_bf16(static_cast<const __nv_bfloat16 *>(ps[i].bf16), c->hu_master + o, ps[i].n, c->stream));
      o += (ps[i].n + 3) & ~static_cast<size_t>(3);
    }
  }
  if (n_cycles > c->hu_cycles_cap) {
    const size_t rows = static_cast<size_t>(n_cycles) * k;
    if ((rc = dev_alloc(c, &c->hu_alpha, rows)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hu_lse, rows)) != GM_OK) return rc;
    if ((rc = dev_alloc(c, &c->hu_loss, static_cast<size_t>(n_cycles))) != GM_OK) return rc;
    c->hu_cycles_cap = n_cycles;
  }
  // ---- the head's cache over the committed prefixes, with the parameters as they are now ----
  if ((rc = gm_head_prefill(c, st, seq_hidden, hid_stride, seq_tok, tok_stride, seq_len, max_len)) != GM_OK) return rc;
  // ---- chunk by chunk: the chains replayed (Eq. 4), their overlaps and logit gradients, the backward pass; then the prefixes ----
  if ((rc = head_update_backward_impl(c, st, n_cycles, k, cycle_seq, rec, seq_tok, tok_stride, scratch_pages, nullptr, seq_hidden,
                                      hid_stride, seq_len, max_len, nullptr, nullptr, &c->hu_grads, temperature, c->hu_alpha,
                                      c->hu_lse)) != GM_OK)
    return rc;
  if ((rc = gm_dca_loss(c, n_cycles, k, c->hu_alpha, rec->accepted, c->hu_loss, mean_loss)) != GM_OK) return rc;
  // ---- AdamW on every tensor of the group; the bf16 copies the forward pass reads are rewritten in place ----
  ParamRef ps[13];
  const int np = collect_params(c, c->hu_grads, ps);
  size_t o = 0;
  for (int i = 0; i < np; ++i) {
    if ((rc = gm_adamw_step(c, static_cast<int64_t>(ps[i].n), c->hu_master + o, const_cast<void *>(ps[i].bf16), ps[i].grad, c->hu_m + o,
                            c->hu_v + o, step, lr, beta1, beta2, eps, weight_decay, 1.0f)) != GM_OK)
      return rc;
    o += (ps[i].n + 3) & ~static_cast<size_t>(3);
  }
  c->hu_step = step;
  return GM_OK;
}

}  // extern "C"
