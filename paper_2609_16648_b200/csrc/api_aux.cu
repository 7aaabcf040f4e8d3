// C ABI of libgm: top-p truncation, the per-cycle record, and the stand-alone GEMM / attention calls.
// Host code only; the helpers it calls are declared in gm_internal.h.
#include "gm_internal.h"

int gmh::run_nucleus(gm_ctx *c, const void *logits, int rows, float temperature, float top_p, void *out, float *dbg_e) {
  if (!(temperature > 0.f) || !std::isfinite(temperature) || !(top_p > 0.f) || !(top_p < 1.f)) return GM_ERR_UNSUPPORTED;
  NucleusArgs N;
  N.in = static_cast<const __nv_bfloat16 *>(logits); N.out = static_cast<__nv_bfloat16 *>(out); N.dbg_e = dbg_e;
  N.rows = rows; N.V = c->V; N.inv_temp = 1.0f / temperature;
  N.tp24 = static_cast<uint32_t>(std::nearbyint(static_cast<double>(top_p) * 16777216.0));
  if (N.tp24 < 1u) N.tp24 = 1u;
  if (N.tp24 > 16777215u) N.tp24 = 16777215u;
  GM_LAUNCH(c, GM_KC_SAMPLER, launch_nucleus(N, c->stream));
  return GM_OK;
}

namespace gm {
// Self-test of the bounded-wait path: one warp waits on an mbarrier nobody will ever arrive on, gives up after
// `limit` polls, records ST_TIMEOUT like every other wait of the library, and returns.  Nothing spins without a limit.
__global__ void wait_expiry_kernel(uint32_t *status, uint32_t limit) {
  __shared__ uint64_t bar;
  pdl_prologue();
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    mbar_fence_init();
    if (!mbar_wait(&bar, 0, limit)) set_status(status, ST_TIMEOUT);
  }
}
}  // namespace gm

extern "C" {

int gm_nucleus(gm_ctx *c, const void *logits, int rows, float temperature, float top_p, void *out, float *dbg_weight) {
  if (!c || !logits || !out || rows < 1 || logits == out) return GM_ERR_INVALID_ARG;
  return run_nucleus(c, logits, rows, temperature, top_p, out, dbg_weight);
}

int gm_set_top_p(gm_ctx *c, float top_p) {
  if (!c) return GM_ERR_INVALID_ARG;
  if (!(top_p > 0.f) || !(top_p <= 1.f)) return GM_ERR_UNSUPPORTED;
  if (top_p < 1.f && !c->ws_nucleus) {
    const size_t n = static_cast<size_t>(c->cfg.max_batch) * (c->cfg.max_k + 1) * c->V;
    int rc = dev_alloc(c, &c->ws_nucleus, n, false);
    if (rc) return rc;
  }
  c->top_p = top_p;
  return GM_OK;
}

int gm_record_begin(gm_ctx *c, const gm_state *st, gm_record *rec) {
  if (!c || !st || !rec || !rec->start_hidden || !rec->start_pos) return GM_ERR_INVALID_ARG;
  if (st->batch < 1 || st->batch > c->cfg.max_batch || !st->kv_len || !st->pending_n || !st->pending_hidden)
    return GM_ERR_INVALID_ARG;
  GM_LAUNCH(c, GM_KC_ELEMENTWISE,
            launch_record_begin(st->kv_len, st->pending_n, static_cast<const __nv_bfloat16 *>(st->pending_hidden), st->batch,
                                c->cfg.max_k, c->d, static_cast<__nv_bfloat16 *>(rec->start_hidden), rec->start_pos,
                                c->stream));
  return GM_OK;
}

int gm_record_end(gm_ctx *c, int batch, int k, float temperature, const void *target_logits, const int32_t *draft_tok,
                  const int32_t *accept_len, gm_record *rec) {
  if (!c || !rec || !target_logits || !draft_tok || !accept_len || !rec->drafts || !rec->top_logprob || !rec->top_index ||
      !rec->accepted)
    return GM_ERR_INVALID_ARG;
  if (batch < 1 || k < 1) return GM_ERR_INVALID_ARG;
  if (k > GM_MAX_K || !(temperature > 0.f) || !std::isfinite(temperature)) return GM_ERR_UNSUPPORTED;
  RecordTopkArgs R;
  R.target_logits = static_cast<const __nv_bfloat16 *>(target_logits); R.bstride = static_cast<size_t>(k + 1) * c->V;
  R.K = k; R.V = c->V; R.inv_temp = 1.0f / temperature; R.top_logprob = static_cast<__nv_bfloat16 *>(rec->top_logprob);
  R.top_index = rec->top_index; R.status = c->status;
  GM_LAUNCH(c, GM_KC_RECORD, launch_record_topk(R, batch, c->stream));
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_record_end(draft_tok, accept_len, batch, k, rec->drafts, rec->accepted, c->stream));
  return GM_OK;
}

int gm_spec_step_rec(gm_ctx *c, gm_state *st, int k, float temperature, uint64_t seed, uint64_t step, int32_t *accept_len,
                     int32_t *next_token, int32_t *draft_tok, gm_record *rec) {
  int rc = check_state(c, st, k);
  if (rc) return rc;
  if (!accept_len || !next_token || !rec) return GM_ERR_INVALID_ARG;
  if ((rc = gm_record_begin(c, st, rec)) != GM_OK) return rc;
  int32_t *dt = draft_tok ? draft_tok : c->ws_draft_tok;
  if ((rc = spec_step_impl(c, st, k, temperature, nullptr, nullptr, seed, step, accept_len, next_token, dt)) != GM_OK) return rc;
  return gm_record_end(c, st->batch, k, temperature, c->ws_target_logits, dt, accept_len, rec);
}

static int gemm_entry(gm_ctx *c, const void *x, const void *w, void *out, int M, int N, int K, int epi, size_t ldo) {
  if (!c || !x || !w || !out || M < 1 || N < 1 || K < 1) return GM_ERR_INVALID_ARG;
  if ((K % 64) || (N % 8)) return GM_ERR_UNSUPPORTED;
  CUtensorMap wm;
  std::memset(&wm, 0, sizeof(wm));
  if (!(c->cfg.flags & GM_FLAG_SIMPLE_GEMM)) {
    auto key = std::make_tuple(w, N, K);
    auto it = c->w_maps.find(key);
    if (it == c->w_maps.end()) {
      CUtensorMap m;
      if (make_map(c, &m, w, N, K, 128) != GM_OK) return GM_ERR_CUDA;
      it = c->w_maps.emplace(key, m).first;
    }
    wm = it->second;
  }
  return run_gemm(c, static_cast<const __nv_bfloat16 *>(x), M, &wm, static_cast<const __nv_bfloat16 *>(w), M, N, K, out,
                  epi, ldo, false);        // a caller's matrix may have been written by the kernel before
}

int gm_gemm(gm_ctx *c, const void *x, const void *w, void *out, int M, int N, int K, int out_fp32) {
  return gemm_entry(c, x, w, out, M, N, K, out_fp32 ? EPI_STORE_F32 : EPI_STORE_BF16, static_cast<size_t>(N));
}

int gm_gemm_swiglu(gm_ctx *c, const void *x, const void *w, void *out, int M, int N, int K) {
  if (c && N > 0 && (N % 16)) return GM_ERR_UNSUPPORTED;
  return gemm_entry(c, x, w, out, M, N, K, EPI_SWIGLU_BF16, static_cast<size_t>(N / 2));
}

int gm_attention(gm_ctx *c, const void *q, const void *kv_pool, int pool_layers, int num_pages, int layer,
                 const int32_t *page_table, const int32_t *q_count, const int32_t *q_base, int batch, int q_stride,
                 void *out) {
  if (!c || !q || !kv_pool || !page_table || !q_count || !q_base || !out) return GM_ERR_INVALID_ARG;
  if (batch < 1 || batch > c->cfg.max_batch || q_stride < 1 || pool_layers < 1 || layer < 0 || layer >= pool_layers ||
      num_pages < 1)
    return GM_ERR_INVALID_ARG;
  if (q_stride > c->cfg.max_k + 1) return GM_ERR_UNSUPPORTED;
  const gm_config &cf = c->cfg;
  CUtensorMap kvm;
  int rc = kv_map(c, kv_pool, pool_layers, num_pages, &kvm);
  if (rc) return rc;
  GM_LAUNCH(c, GM_KC_ELEMENTWISE,
            launch_page_prefix(q_count, q_base, batch, cf.max_pages_per_seq, q_stride, c->page_start, c->status, c->stream));
  const int qrows = round16(q_stride * c->group);
  AttnArgs T;
  T.kv_map = kvm; T.qbuf = static_cast<const __nv_bfloat16 *>(q); T.qn = q_count; T.qbase = q_base;
  T.page_start = c->page_start; T.page_table = page_table; T.batch = batch; T.n_kv = cf.n_kv_heads; T.group = c->group;
  T.hd = cf.head_dim; T.qrows = qrows; T.layer = layer; T.num_pages = num_pages; T.max_pages_per_seq = cf.max_pages_per_seq;
  T.n_ctas = c->sm_count; T.scale_log2e = static_cast<float>(1.4426950408889634 / std::sqrt(static_cast<double>(cf.head_dim)));
  T.part_o = c->part_o; T.part_ml = c->part_ml; T.status = c->status; T.rows_used = q_stride * c->group;
  GM_LAUNCH(c, GM_KC_ATTENTION, launch_attention(T, c->stream));
  AttnCombineArgs Cb;
  Cb.part_o = c->part_o; Cb.part_ml = c->part_ml; Cb.qn = q_count; Cb.page_start = c->page_start; Cb.batch = batch;
  Cb.n_kv = cf.n_kv_heads; Cb.group = c->group; Cb.hd = cf.head_dim; Cb.qrows = qrows; Cb.QT = q_stride;
  Cb.n_ctas = c->sm_count; Cb.out = static_cast<__nv_bfloat16 *>(out);
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_attention_combine(Cb, c->stream));
  return GM_OK;
}

int gm_chain_trace(gm_ctx *c, int enable) {
  if (!c) return GM_ERR_INVALID_ARG;
  if (!c->chain_on) return GM_ERR_UNSUPPORTED;
  if (enable && !c->chain_trace) {
    int rc = dev_alloc(c, &c->chain_trace, static_cast<size_t>(c->chain_pairs) * 2 * 64);
    if (rc != GM_OK) return rc;
  }
  c->chain_trace_on = enable != 0;
  return GM_OK;
}

int gm_chain_trace_read(gm_ctx *c, uint64_t *out, int capacity) {
  if (!c || !out || capacity < 0) return GM_ERR_INVALID_ARG;
  if (!c->chain_trace) return GM_ERR_UNSUPPORTED;
  const int words = c->chain_pairs * 2 * 64;
  if (capacity < words) return GM_ERR_INVALID_ARG;
  GM_CUDA(c, cudaStreamSynchronize(c->stream));
  GM_CUDA(c, cudaMemcpy(out, c->chain_trace, static_cast<size_t>(words) * sizeof(uint64_t), cudaMemcpyDeviceToHost));
  return words;
}


int gm_selftest_wait_expiry(gm_ctx *c) {
  if (!c) return GM_ERR_INVALID_ARG;
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_k(wait_expiry_kernel, dim3(1), dim3(32), 0, c->stream, 1, c->status, 1024u));
  return GM_OK;
}

}  // extern "C"
