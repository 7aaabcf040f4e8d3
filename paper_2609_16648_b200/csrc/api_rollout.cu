// C ABI of libgm: the rollout driver (cycles until every response ended) and the page allocator.
// Host code only; the helpers it calls are declared in gm_internal.h.
#include "gm_internal.h"

extern "C" {

// ---- rollout driver and page allocator ------------------------------------------------------------------------------
static int rollout_args_ok(const gm_ctx *c, const gm_state *st, const gm_rollout *ro) {
  if (!c || !st || !ro || !ro->out_tok || !ro->out_len || !ro->finished || !ro->n_running) return GM_ERR_INVALID_ARG;
  if (ro->max_new < 1 || ro->out_stride < ro->max_new) return GM_ERR_INVALID_ARG;
  if (st->batch < 1 || st->batch > c->cfg.max_batch) return GM_ERR_INVALID_ARG;
  return GM_OK;
}

static void fill_alloc(gm_ctx *c, gm_state *st, int pool, PageAllocArgs &P) {
  P.batch = st->batch; P.max_pages_per_seq = c->cfg.max_pages_per_seq;
  P.num_pages = pool ? c->cfg.head_num_pages : c->cfg.num_pages; P.extra = 0;
  P.length = nullptr; P.finished = nullptr;
  P.page_table = pool ? st->head_page_table : st->page_table;
  P.held = c->held[pool]; P.free_list = c->free_list[pool]; P.free_top = c->free_top[pool]; P.status = c->status;
}

int gm_pages_reset(gm_ctx *c, gm_state *st) {
  if (!c || !st || !st->page_table || !st->head_page_table || st->batch < 1 || st->batch > c->cfg.max_batch)
    return GM_ERR_INVALID_ARG;
  for (int pool = 0; pool < 2; ++pool) {
    if (!c->free_list[pool]) {
      int rc;
      if ((rc = dev_alloc(c, &c->free_list[pool], pool ? c->cfg.head_num_pages : c->cfg.num_pages, false)) != GM_OK) return rc;
      if ((rc = dev_alloc(c, &c->free_top[pool], 1)) != GM_OK) return rc;
      if ((rc = dev_alloc(c, &c->held[pool], c->cfg.max_batch)) != GM_OK) return rc;
    }
    PageAllocArgs P;
    fill_alloc(c, st, pool, P);
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_page_reset(P, c->stream));
  }
  c->alloc_on = true;
  return GM_OK;
}

int gm_pages_reserve(gm_ctx *c, gm_state *st, const int32_t *length, int extra, const int32_t *finished) {
  if (!c || !st || extra < 0) return GM_ERR_INVALID_ARG;
  if (!c->alloc_on) return GM_ERR_INVALID_ARG;
  PageAllocArgs P[2];
  for (int pool = 0; pool < 2; ++pool) {
    fill_alloc(c, st, pool, P[pool]);
    P[pool].length = length ? length : st->kv_len; P[pool].extra = extra; P[pool].finished = finished;
  }
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_page_reserve(P[0], P[1], c->stream));
  return GM_OK;
}

int gm_pages_release(gm_ctx *c, gm_state *st, const int32_t *finished) {
  if (!c || !st || !finished) return GM_ERR_INVALID_ARG;
  if (!c->alloc_on) return GM_ERR_INVALID_ARG;
  PageAllocArgs P[2];
  for (int pool = 0; pool < 2; ++pool) {
    fill_alloc(c, st, pool, P[pool]);
    P[pool].finished = finished;
  }
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_page_release(P[0], P[1], c->stream));
  return GM_OK;
}

int gm_pages_free_count(gm_ctx *c, int32_t *target_free, int32_t *head_free) {
  if (!c || !c->alloc_on) return GM_ERR_INVALID_ARG;
  int32_t v[2] = {0, 0};
  for (int pool = 0; pool < 2; ++pool)
    GM_CUDA(c, cudaMemcpyAsync(&v[pool], c->free_top[pool], sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream));
  GM_CUDA(c, cudaStreamSynchronize(c->stream));
  if (target_free) *target_free = v[0];
  if (head_free) *head_free = v[1];
  return GM_OK;
}

static void fill_rollout(const gm_ctx *c, const gm_state *st, const gm_rollout *ro, int k, RolloutArgs &R) {
  R.batch = st->batch; R.k = k; R.out_stride = ro->out_stride; R.eos_token = ro->eos_token; R.max_new = ro->max_new;
  R.pend_stride = c->cfg.max_k + 1; R.draft_tok = c->ws_draft_tok; R.accept_len = c->ro_accept; R.next_token = c->ro_next;
  R.pending_tok = st->pending_tok; R.out_tok = ro->out_tok; R.out_len = ro->out_len; R.finished = ro->finished;
  R.n_running = ro->n_running; R.step_counter = c->step_ptr;
}

int gm_rollout_begin(gm_ctx *c, const gm_state *st, const gm_rollout *ro) {
  int rc = rollout_args_ok(c, st, ro);
  if (rc) return rc;
  if (!st->pending_tok) return GM_ERR_INVALID_ARG;
  RolloutArgs R;
  fill_rollout(c, st, ro, 1, R);
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_rollout_append(R, true, c->stream));
  return GM_OK;
}

int gm_rollout_step(gm_ctx *c, gm_state *st, const gm_rollout *ro, int k, float temperature, uint64_t seed, uint64_t step) {
  NvtxRange nvtx_range("gm_rollout_step");
  int rc = rollout_args_ok(c, st, ro);
  if (rc) return rc;
  if ((rc = check_state(c, st, k)) != GM_OK) return rc;
  if (c->alloc_on && (rc = gm_pages_reserve(c, st, nullptr, k + 1, ro->finished)) != GM_OK) return rc;
  c->finished_mask = ro->finished;
  rc = spec_step_impl(c, st, k, temperature, nullptr, nullptr, seed, step, c->ro_accept, c->ro_next, c->ws_draft_tok);
  c->finished_mask = nullptr;
  if (rc) return rc;
  RolloutArgs R;
  fill_rollout(c, st, ro, k, R);
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_rollout_append(R, false, c->stream));
  if (c->alloc_on && (rc = gm_pages_release(c, st, ro->finished)) != GM_OK) return rc;
  return GM_OK;
}

int gm_rollout_run(gm_ctx *c, gm_state *st, const gm_rollout *ro, int k, float temperature, uint64_t seed,
                   uint64_t first_step, int max_steps, int check_every, int32_t *steps_run, int32_t *rows_running) {
  if (max_steps < 0 || check_every < 1) return GM_ERR_INVALID_ARG;
  int rc = rollout_args_ok(c, st, ro);
  if (rc) return rc;
  int done = 0;
  int32_t running = st->batch;
  auto poll = [&]() -> int {
    GM_CUDA(c, cudaMemcpyAsync(&running, ro->n_running, sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream));
    GM_CUDA(c, cudaStreamSynchronize(c->stream));
    return GM_OK;
  };
  if ((rc = poll()) != GM_OK) return rc;
  const bool use_graph = graph_capable(c);
  if (use_graph && running > 0 && max_steps > 0) {
    KeyBytes key;
    key.add(*st); key.add(*ro); key.add(k); key.add(temperature); key.add(seed); key.add(c->alloc_on); key.add(c->top_p);
    key.add(c->capture); key.add(c->capture_stride);
    if ((rc = check_state(c, st, k)) != GM_OK) return rc;
    rc = graph_prepare(c, c->graph_rollout, key.bytes, [&]() { return gm_rollout_step(c, st, ro, k, temperature, seed, 0); });
    if (rc) return rc;
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_set_step(c->dev_step, first_step, c->stream));
  }
  while (done < max_steps && running > 0) {
    if (use_graph) {
      GM_CUDA(c, cudaGraphLaunch(c->graph_rollout.exec, c->stream));
      c->launches += c->graph_rollout.launches;
    } else if ((rc = gm_rollout_step(c, st, ro, k, temperature, seed, first_step + done)) != GM_OK) {
      return rc;
    }
    ++done;
    if (done % check_every == 0 || done == max_steps)
      if ((rc = poll()) != GM_OK) return rc;
  }
  if (steps_run) *steps_run = done;
  if (rows_running) *rows_running = running;
  return GM_OK;
}

}  // extern "C"
