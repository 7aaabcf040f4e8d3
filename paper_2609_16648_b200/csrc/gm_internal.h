// Internals of libgm shared by its host-side translation units: the context, error / launch macros, and the helpers
// that issue the launch sequences.  Not part of the C ABI.
#pragma once

#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <new>
#include <tuple>
#include <vector>

#include <cudaTypedefs.h>
#include <nvtx3/nvToolsExt.h>

#include "../../include/gm.h"
#include "common.cuh"
#include "kernels.h"

using namespace gm;


namespace gmh {

struct LayerMaps { CUtensorMap wqkv, wo, wgu, wdown; };

struct EventPair { cudaEvent_t a, b; };

}  // namespace gmh
using namespace gmh;

struct gm_ctx {
  gm_config cfg;
  gm_weights w;
  std::vector<gm_layer_weights> layers;
  cudaStream_t stream = nullptr;
  int sm_count = 148;
  PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;

  // derived shapes
  int d, q_dim, kv_dim, n_qkv, F, V, group, Mmax;

  // tensor maps
  std::vector<LayerMaps> lmaps;
  LayerMaps head_maps;
  CUtensorMap lm_head_map, head_proj_map;
  std::map<std::tuple<const void *, int, int, int>, CUtensorMap> x_maps;   // (ptr, rows, K, box rows)
  std::map<std::tuple<const void *, int, int>, CUtensorMap> w_maps;        // (ptr, N, K)   (gm_gemm only)
  std::map<std::tuple<const void *, long long>, CUtensorMap> kv_maps;      // (pool, rows)

  // workspaces (device)
  float *x = nullptr, *g = nullptr, *part_o = nullptr, *part_ml = nullptr;
  __nv_bfloat16 *xn = nullptr, *zin = nullptr, *qkv = nullptr, *qbuf = nullptr, *attn_out = nullptr, *act = nullptr, *gn = nullptr;
  bool pair_gemm = true;              // CTA-pair kernel for the full wave of wide projections (GM_NO_PAIR_GEMM: off)
  // persistent chain of a layer's projections (chain.cu); GM_NO_CHAIN: off
  bool chain_on = false;
  int chain_pairs = 0;                // CTA pairs resident at once
  int chain_npw = 4, chain_npa = 2;   // producer threads per CTA for weight / activation boxes
  int chain_mode = 1;                 // 1: only the wide gate/up projection, as a one-phase launch; 2: the whole chain; 0: off
  int chain_max_m = 512;              // phases with more rows than this run as separate launches
  float *chain_partial = nullptr;     // K-slice partial sums, one slot per CTA
  float *chain_sq[2] = {nullptr, nullptr};   // sums of squares per feature tile and row, after the O / down projection
  unsigned long long *chain_sync = nullptr;  // barrier counters
  std::map<std::tuple<const void *, int, int, int>, CUtensorMap> chain_w_maps;   // (weights, N, K, box rows)
  int chain_force_ns[4] = {0, 0, 0, 0};      // GM_CHAIN_NS: K slices per phase position (tuning aid)
  unsigned long long *chain_trace = nullptr;   // gm_chain_trace: [2 pairs][32] stamps
  bool chain_trace_on = false;
  int max_clusters[17][9];            // resident clusters of the GEMM kernel by (block_t / 16, cluster size); -1 = not asked yet
  __nv_bfloat16 *ws_draft_logits = nullptr, *ws_target_logits = nullptr, *ws_target_hidden = nullptr;
  int32_t *ws_draft_tok = nullptr, *ws_accept_len = nullptr, *ws_next_token = nullptr;
  uint32_t *ws_u24 = nullptr;
  int32_t *qn = nullptr, *qbase = nullptr, *page_start = nullptr;
  float2 *rope = nullptr;
  uint32_t *status = nullptr;
  // prompt prefill: per-chunk bookkeeping, the chunk's hidden states, the row of each prompt's last token
  // A prefill pass gives every prompt pf_vr consecutive chunks of max_k + 1 positions ("virtual rows" that share the
  // prompt's page table), so the M-sized workspaces below hold max_batch * pf_vr * (max_k + 1) rows.
  int pf_vr = 1;
  int32_t *pf_row_base = nullptr, *pf_vtable[2] = {nullptr, nullptr};   // first position and page-table row per virtual row
  int32_t *pf_row_n = nullptr, *pf_head_n = nullptr, *pf_pair_tok = nullptr, *pf_first = nullptr;
  __nv_bfloat16 *pf_hidden = nullptr;
  float *pf_xlast = nullptr;
  int32_t *ro_accept = nullptr, *ro_next = nullptr;   // per-step outputs of a rollout step
  // captured cycles (GM_FLAG_GRAPH)
  uint64_t *dev_step = nullptr;             // step index of the captured cycle
  uint64_t *step_ptr = nullptr;             // non-null while a cycle is being captured: kernels read the step from here
  struct GraphSlot {                        // one captured sequence of launches and what it was captured for
    cudaGraphExec_t exec = nullptr;
    int64_t launches = 0;
    std::vector<unsigned char> key;
  } graph_rollout, graph_step;
  const int32_t *finished_mask = nullptr;   // set around the phases of a rollout step: rows that sit out
  // page allocator (gm_pages_*): one stack of free page ids per pool
  bool alloc_on = false;
  int32_t *free_list[2] = {nullptr, nullptr}, *free_top[2] = {nullptr, nullptr}, *held[2] = {nullptr, nullptr};
  // chains of a reconstruction: virtual sequences (allocated on first use)
  int32_t *v_kv_len = nullptr, *v_pending_n = nullptr, *v_pending_tok = nullptr, *v_table = nullptr;
  __nv_bfloat16 *v_pending_hidden = nullptr;
  __nv_bfloat16 *capture = nullptr;         // gm_capture_hidden: [max_batch, capture_stride, d] or null
  int capture_stride = 0;
  void *flow_ws = nullptr;                  // work-queue sampler: counters, per-sequence state, slice partials, queue slots
  size_t flow_ws_bytes = 0;
  int flow_cap = 0;                         // batch the workspace was sized for
  bool fuse_rope = false;                   // GM_FUSED_ROPE: rotary embedding + KV append in the QKV projection's epilogue (measured slower: off)
  int pair_split = 1;                        // CTA pairs with K slices for split projections (GM_GEMM_PAIR_SPLIT: 0 off, 1 when no fewer CTAs run, 2 whenever clusters of <= 8 fit, 3 also larger clusters)
  int pair_split_clusters[9] = {-1, -1, -1, -1, -1, -1, -1, -1, -1};   // resident clusters of 2 x ns CTAs, by ns
  bool pair_blocks = true;                   // CTA pairs for narrow projections over several token blocks (GM_GEMM_PAIR_BLOCKS=0: off)
  bool wide_split = false;                   // split projections with two 128-feature sub-tiles per CTA (GM_GEMM_WIDE_SPLIT=1)
  bool early_weights = true;                // projections fetch their first weight boxes before the dependency wait (GM_NO_EARLY_W switches it off)
  int sampler_mode = 0;                     // 0 = by batch size; 1 cluster, 2 stream, 3 work queue (GM_SAMPLER in the environment)
  float *state_out = nullptr;               // set by the reconstruction while it runs: g_j of chain r -> state_out[(r*k + j-1)*d]
  // head-update backward through the feed-forward block: transposed weight copies and scratch, made on first use
  __nv_bfloat16 *ffn_wd_t = nullptr, *ffn_wgu_t = nullptr;   // [F, d], [d, 2F]
  CUtensorMap ffn_wd_t_map, ffn_wgu_t_map;
  int ffn_rows_cap = 0;
  __nv_bfloat16 *ffn_u = nullptr, *ffn_ab = nullptr, *ffn_dy = nullptr, *ffn_dab = nullptr, *ffn_h = nullptr;
  __nv_bfloat16 *ffn_ut = nullptr, *ffn_dyt = nullptr, *ffn_dabt = nullptr, *ffn_ht = nullptr;
  float *ffn_dh = nullptr, *ffn_du = nullptr, *ffn_t = nullptr;
  // ... and through the head's input projection
  __nv_bfloat16 *hin_proj_t = nullptr;      // [2d, d]
  CUtensorMap hin_proj_t_map;
  int hin_rows_cap = 0;
  __nv_bfloat16 *hin_zin = nullptr, *hin_dz = nullptr, *hin_zint = nullptr, *hin_dzt = nullptr;
  float *hin_e = nullptr, *hin_dzin = nullptr, *hin_t = nullptr;
  float *ab_stats = nullptr;                // attention backward: (max, 1 / sum, D) per (row, query head)
  size_t ab_stats_cap = 0;
  float *ab_part = nullptr;                 // partial statistics per key segment (the key-split kernels)
  size_t ab_part_cap = 0;
  // one update of the head (gm_head_update_step): gradients, optimizer state (fp32 master, first and second moments, the
  // tensors one after the other, each padded to 4 elements), per-call buffers
  gm_head_grads hu_grads = {};
  float *hu_master = nullptr, *hu_m = nullptr, *hu_v = nullptr;
  float *hu_alpha = nullptr, *hu_lse = nullptr, *hu_loss = nullptr;
  int hu_cycles_cap = 0, hu_step = 0;
  long long *hub_dk_fix = nullptr, *hub_dv_fix = nullptr, *hat_dq_fix = nullptr;   // fixed-point gradient accumulators of the driver
  size_t hub_fix_cap = 0, hat_dq_fix_cap = 0;
  float *colsum_ws = nullptr;               // partial column sums (64 chunks x the widest row: n_qkv or 2 d)
  // backward pass over a reconstruction: per-chunk states and their gradients, one pass's rows
  int hub_rows_cap = 0;
  float *hub_states = nullptr, *hub_gn = nullptr, *hub_dstate = nullptr, *hub_t = nullptr;          // [max_batch, max_k, d]
  float *hub_hidden = nullptr, *hub_z = nullptr, *hub_xmid = nullptr, *hub_dg = nullptr, *hub_dxmid = nullptr, *hub_dz = nullptr,
        *hub_dhid = nullptr, *hub_e = nullptr;                                                        // [rows, d]
  int32_t *hub_tok = nullptr, *hub_base = nullptr, *hub_cnt = nullptr;                               // [rows]
  __nv_bfloat16 *hub_glogits = nullptr;                                                              // [max_batch, max_k, V] a chunk's logit gradients
  // attention half of the head's layer, backward: transposed weight copies and per-call scratch
  __nv_bfloat16 *hat_wo_t = nullptr, *hat_wqkv_t = nullptr;      // [q_dim, d], [d, n_qkv]
  CUtensorMap hat_wo_t_map, hat_wqkv_t_map;
  int hat_rows_cap = 0;
  __nv_bfloat16 *hat_dy = nullptr, *hat_dqkv_bf = nullptr, *hat_dyt = nullptr, *hat_ot = nullptr, *hat_dqkvt = nullptr, *hat_ht = nullptr;
  float *hat_do = nullptr, *hat_dq = nullptr, *hat_dqkv = nullptr, *hat_dh = nullptr, *hat_t = nullptr, *hat_tq = nullptr, *hat_tk = nullptr;
  __nv_bfloat16 *lm_head_t = nullptr;       // [d, V]: the LM head transposed, the weight operand of the gradient GEMM
  CUtensorMap lm_head_t_map;
  float top_p = 1.f;                    // nucleus of the target distributions (1 = none)
  __nv_bfloat16 *ws_nucleus = nullptr;  // [max_batch (max_k + 1)][V] filtered target rows, allocated by gm_set_top_p
  std::vector<void *> allocs;
  std::vector<unsigned char *> guards;      // 256 guard bytes behind every workspace
  bool check_guards = false;                // GM_CANARY: gm_last_status verifies them

  // profiling
  int prof_mask = 0;
  std::vector<EventPair> events[GM_KC_COUNT];
  size_t events_used[GM_KC_COUNT] = {};
  int64_t launches = 0;
  cudaError_t last_cuda = cudaSuccess;
};

namespace gmh {

#define GM_CUDA(ctx, call)                                   \
  do {                                                       \
    cudaError_t e__ = (call);                                \
    if (e__ != cudaSuccess) { (ctx)->last_cuda = e__; return GM_ERR_CUDA; } \
  } while (0)

constexpr size_t GM_GUARD_BYTES = 256;
constexpr int GM_GUARD_PATTERN = 0xA5;

template <typename T>
int dev_alloc(gm_ctx *c, T **p, size_t n, bool zero = true) {
  void *q = nullptr;
  const size_t bytes = ((n * sizeof(T) > 0 ? n * sizeof(T) : 16) + 255) & ~static_cast<size_t>(255);
  GM_CUDA(c, cudaMalloc(&q, bytes + GM_GUARD_BYTES));
  c->allocs.push_back(q);
  unsigned char *guard = static_cast<unsigned char *>(q) + bytes;
  GM_CUDA(c, cudaMemsetAsync(guard, GM_GUARD_PATTERN, GM_GUARD_BYTES, c->stream));
  c->guards.push_back(guard);
  if (zero) GM_CUDA(c, cudaMemsetAsync(q, 0, n * sizeof(T), c->stream));
  *p = static_cast<T *>(q);
  return GM_OK;
}

struct Prof {
  gm_ctx *c; int cls; bool on; EventPair ev{};
  Prof(gm_ctx *c_, int cls_) : c(c_), cls(cls_), on((c_->prof_mask >> cls_) & 1) {
    if (!on) return;
    size_t &u = c->events_used[cls];
    if (u == c->events[cls].size()) {
      EventPair e;
      cudaEventCreate(&e.a);
      cudaEventCreate(&e.b);
      c->events[cls].push_back(e);
    }
    ev = c->events[cls][u++];
    cudaEventRecord(ev.a, c->stream);
  }
  ~Prof() {
    if (on) cudaEventRecord(ev.b, c->stream);
    c->launches++;
  }
};
#define GM_LAUNCH(ctx, cls, call)           \
  do {                                      \
    cudaError_t e__;                        \
    { Prof p__(ctx, cls); e__ = (call); }   \
    if (e__ != cudaSuccess) {               \
      (ctx)->last_cuda = e__;               \
      if (std::getenv("GM_DEBUG")) std::fprintf(stderr, "[gm] %s failed: %s\n", #call, cudaGetErrorString(e__)); \
      return GM_ERR_CUDA;                   \
    }                                       \
  } while (0)


// NVTX range around an entry point (GM_NVTX=1): lets a profiler group the launches of a phase.  Off by default.
struct NvtxRange {
  bool on;
  explicit NvtxRange(const char *name) : on(enabled()) { if (on) nvtxRangePushA(name); }
  ~NvtxRange() { if (on) nvtxRangePop(); }
  static bool enabled() {
    static const bool e = std::getenv("GM_NVTX") != nullptr;
    return e;
  }
};

// ---- host helpers shared by the api_*.cu files (defined in gm_api.cu) -------------------------------------------------
int make_map(gm_ctx *c, CUtensorMap *m, const void *ptr, uint64_t rows, uint64_t cols, uint32_t box_rows);
int x_map(gm_ctx *c, const void *ptr, int rows, int K, int box_rows, CUtensorMap *out);
int kv_map(gm_ctx *c, const void *pool, int layers, int num_pages, CUtensorMap *out);
int round16(int v);
int run_gemm(gm_ctx *c, const __nv_bfloat16 *x, int x_rows, const CUtensorMap *wmap, const __nv_bfloat16 *w, int M,
             int N, int K, void *out, int epi, size_t ldo, bool const_w = true,
             const RopeAppendArgs *rope = nullptr);   // const_w: w is a model weight (written by no kernel of the stream)
struct PhaseShape { int B, QT, M, qrows; };
// next_lw / next_lm: the layer whose QKV projection is appended to this layer's chain of projections (its input norm
// is next_norm); qkv_done: this layer's own QKV projection was produced that way by the layer before.
int run_layer(gm_ctx *c, const gm_layer_weights &lw, const LayerMaps &lm, const PhaseShape &ph, const CUtensorMap &kvm,
              __nv_bfloat16 *pool, int layer, int num_pages, const int32_t *page_table,
              const __nv_bfloat16 *next_norm, __nv_bfloat16 *hidden_out, const gm_layer_weights *next_lw = nullptr,
              const LayerMaps *next_lm = nullptr, bool qkv_done = false, bool kv_only = false);
bool chain_usable(const gm_ctx *c, int M);
// One projection of a chain (see ChainPhase); the input is x [x_rows, K] bf16.
struct ChainSpec {
  const void *w; const __nv_bfloat16 *x; int x_rows, N, K; void *out; int epi, ldo;
  __nv_bfloat16 *xg; const __nv_bfloat16 *gamma; float *sq_out;
  const float *sq_in; int sq_from, norm_dim;     // sq_from: the phase of this chain that writes sq_in
};
int run_chain(gm_ctx *c, const ChainSpec *specs, int n, int M);
int run_plan(gm_ctx *c, const gm_state *st, int mode, int k_or_j);
int run_plan_chunk(gm_ctx *c, int batch, const int32_t *row_n, const int32_t *row_base, int QT);
int check_state(const gm_ctx *c, const gm_state *st, int k);
cudaError_t run_sampler(gm_ctx *c, const SamplerArgs &S, int batch);
int fill_sampler(gm_ctx *c, SamplerArgs &S, float temperature);
// forced: draft_tok holds recorded drafts that are fed back instead of sampled ones (Eq. 4); nothing is drawn
// The backward pass over recorded cycles (gm_head_update_backward).  grad_logits null: the logit gradients are formed chunk
// by chunk from the replay's own logits (overlap and objective gradient at `temperature`, the mean over all n_cycles), and
// alpha / lse [n_cycles, k] receive the overlaps and row statistics of every cycle.
int head_update_backward_impl(gm_ctx *c, gm_state *st, int n_cycles, int k, const int32_t *cycle_seq, const gm_record *rec,
                              const int32_t *seq_tok, int tok_stride, const int32_t *scratch_pages, const void *grad_logits,
                              const void *seq_hidden, int hid_stride, const int32_t *seq_len, int max_len, float *dk_pool,
                              float *dv_pool, const gm_head_grads *out, float temperature, float *alpha, float *lse);
int draft_impl(gm_ctx *c, const gm_state *st, int k, float temperature, const uint32_t *u24_draft, uint64_t seed,
               uint64_t step, int32_t *draft_tok, void *draft_logits, float *dbg_q, bool forced);
int spec_step_impl(gm_ctx *c, gm_state *st, int k, float temperature, const uint32_t *u24_draft,
                   const uint32_t *u24_accept, uint64_t seed, uint64_t step, int32_t *accept_len,
                   int32_t *next_token, int32_t *draft_tok);
int run_nucleus(gm_ctx *c, const void *logits, int rows, float temperature, float top_p, void *out, float *dbg_e);

// ---- captured cycles (GM_FLAG_GRAPH) ----------------------------------------------------------------------------------
struct KeyBytes {
  std::vector<unsigned char> bytes;
  template <typename T> void add(const T &v) {
    const unsigned char *p = reinterpret_cast<const unsigned char *>(&v);
    bytes.insert(bytes.end(), p, p + sizeof(T));
  }
};
inline bool graph_capable(const gm_ctx *c) {
  return (c->cfg.flags & GM_FLAG_GRAPH) && c->stream != nullptr && c->stream != cudaStreamLegacy &&
         c->stream != cudaStreamPerThread;
}
// Makes `slot` hold a graph of the launches `body` issues (with the step index read from c->dev_step), re-capturing
// when `key` differs from what the slot was captured for.  Nothing of `body` runs here.
template <typename F>
int graph_prepare(gm_ctx *c, gm_ctx::GraphSlot &slot, const std::vector<unsigned char> &key, F &&body) {
  if (slot.exec && slot.key == key) return GM_OK;
  if (slot.exec) { cudaGraphExecDestroy(slot.exec); slot.exec = nullptr; }
  int rc;
  if (!c->dev_step && (rc = dev_alloc(c, &c->dev_step, 1)) != GM_OK) return rc;
  const int64_t before = c->launches;
  GM_CUDA(c, cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeRelaxed));
  c->step_ptr = c->dev_step;
  rc = body();
  c->step_ptr = nullptr;
  cudaGraph_t graph = nullptr;
  const cudaError_t e = cudaStreamEndCapture(c->stream, &graph);         // always leave capture mode
  const int64_t n = c->launches - before;
  c->launches = before;                                                  // nothing has run yet
  if (rc != GM_OK || e != cudaSuccess || !graph) {
    if (graph) cudaGraphDestroy(graph);
    if (e != cudaSuccess) { c->last_cuda = e; (void)cudaGetLastError(); }
    return rc != GM_OK ? rc : GM_ERR_CUDA;
  }
  const cudaError_t ei = cudaGraphInstantiate(&slot.exec, graph, 0);
  cudaGraphDestroy(graph);
  if (ei != cudaSuccess) { c->last_cuda = ei; slot.exec = nullptr; return GM_ERR_CUDA; }
  slot.launches = n;
  slot.key = key;
  return GM_OK;
}


}  // namespace gmh
