// C ABI of libgm: context, workspaces, tensor maps and the launch sequences of the draft, verify and
// accept phases.  Host code only; every step of the path runs in the kernels of this directory.
#include "gm_internal.h"

namespace gm {
bool pdl_enabled() {
  static const bool on = std::getenv("GM_NO_PDL") == nullptr;
  return on;
}
}  // namespace gm

namespace gmh {

// 2-D bf16 tensor map: inner extent `cols` (contiguous), outer extent `rows`, box 64 x box_rows, 128-byte swizzle.
int make_map(gm_ctx *c, CUtensorMap *m, const void *ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = c->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? GM_OK : GM_ERR_CUDA;
}

int x_map(gm_ctx *c, const void *ptr, int rows, int K, int box_rows, CUtensorMap *out) {
  auto key = std::make_tuple(ptr, rows, K, box_rows);
  auto it = c->x_maps.find(key);
  if (it == c->x_maps.end()) {
    CUtensorMap m;
    if (make_map(c, &m, ptr, rows, K, box_rows) != GM_OK) return GM_ERR_CUDA;
    it = c->x_maps.emplace(key, m).first;
  }
  *out = it->second;
  return GM_OK;
}

int kv_map(gm_ctx *c, const void *pool, int layers, int num_pages, CUtensorMap *out) {
  const long long rows = static_cast<long long>(layers) * 2 * num_pages * c->cfg.n_kv_heads * 16;
  auto key = std::make_tuple(pool, rows);
  auto it = c->kv_maps.find(key);
  if (it == c->kv_maps.end()) {
    const int hpc = c->cfg.n_kv_heads < 8 ? c->cfg.n_kv_heads : 8;
    CUtensorMap m;
    if (make_map(c, &m, pool, rows, c->cfg.head_dim, hpc * 16) != GM_OK) return GM_ERR_CUDA;
    it = c->kv_maps.emplace(key, m).first;
  }
  *out = it->second;
  return GM_OK;
}

int round16(int v) { return (v + 15) & ~15; }

// K slices (= cluster size) for a projection with few output tiles: the largest count whose clusters are all
// resident at once (GPC packing decides), so the slices of a tile run concurrently and the SMs are filled.
int pick_split(gm_ctx *c, int M, int N, int K, int T) {
  const int tiles = ((N + 127) / 128) * ((M + T - 1) / T);
  const int KB = K / 64;
  if (const char *ov = std::getenv("GM_GEMM_SPLIT")) {            // tuning aid: force the K-split of small projections
    const int ns = std::atoi(ov);
    if (ns >= 1 && ns <= 8 && ns <= KB && tiles * 3 < c->sm_count * 2) return ns;
  }
  if (tiles * 3 >= c->sm_count * 2) return 1;
  int best = 1;
  for (int ns = 2; ns <= 8 && ns <= KB; ++ns) {
    int &cap = c->max_clusters[T / 16][ns];
    if (cap < 0) {
      int v = 0;
      cudaError_t e = gemm_tc_max_clusters(T, ns, &v);
      if (e != cudaSuccess) { v = 0; (void)cudaGetLastError(); }
      if (std::getenv("GM_DEBUG")) std::fprintf(stderr, "[gm] resident clusters T=%d size=%d: %d (%s)\n", T, ns, v, cudaGetErrorString(e));
      cap = v;
    }
    if (cap >= tiles) best = ns;
  }
  return best;
}

// out = epilogue(x[M, K] w[N, K]^T) on the tcgen05 kernel (or the plain one under GM_FLAG_SIMPLE_GEMM).
int run_chain(gm_ctx *c, const ChainSpec *specs, int n, int M);
int run_gemm(gm_ctx *c, const __nv_bfloat16 *x, int x_rows, const CUtensorMap *wmap, const __nv_bfloat16 *w, int M,
             int N, int K, void *out, int epi, size_t ldo, bool const_w, const RopeAppendArgs *rope) {
  GemmArgs A;
  std::memset(&A, 0, sizeof(A));
  A.x = x; A.w = w; A.M = M; A.N = N; A.K = K; A.status = c->status;
  A.out = out; A.epi = epi; A.ldo = ldo;
  A.early_weights = (const_w && c->early_weights) ? 1 : 0;
  if (rope) A.rope = *rope;
  const int T = M >= 256 ? 256 : round16(M);
  A.block_t = T;
  A.nsplit = 1;
  A.wtiles = 1;
  if ((c->cfg.flags & GM_FLAG_SIMPLE_GEMM) != 0) {
    GM_LAUNCH(c, GM_KC_GEMM, launch_gemm_simple(A, c->stream));
    return GM_OK;
  }
  if ((K % 64) != 0) return GM_ERR_UNSUPPORTED;      // the tensor-core kernels stage K in blocks of 64
  // A SwiGLU projection wide enough for one tile per CTA pair (gate/up): one wave of the persistent-pair kernel - tiles
  // of 256 / 288 features sized so that the wave is exact - instead of a full wave plus a short tail launch.
  if (c->chain_on && c->chain_mode >= 1 && epi == EPI_SWIGLU_BF16 && M <= c->chain_max_m && N >= c->chain_pairs * 128 &&
      N <= c->chain_pairs * 288 && (N % 16) == 0 && (ldo % 8) == 0) {
    const ChainSpec g = {w, x, x_rows, N, K, out, epi, static_cast<int>(ldo), nullptr, nullptr, nullptr, nullptr, 0, 0};
    return run_chain(c, &g, 1, M);
  }
  int rc = x_map(c, x, x_rows, K, T, &A.x_map);
  if (rc != GM_OK) return rc;
  A.w_map = *wmap;
  const int mblocks = (M + T - 1) / T;
  const int tiles128 = (N + 127) / 128;
  A.nsplit = pick_split(c, M, N, K, T);
  // A split projection whose tiles pair up: two 128-feature sub-tiles per CTA share one activation box, so a CTA moves
  // 2/3 of the bytes per unit of MMA work (the main loops are bound by filling shared memory), with more K slices to
  // keep the SMs filled.  Taken when it does not leave more SMs idle than the one-sub-tile form.
  if (c->wide_split && A.nsplit > 1 && T == 256 && mblocks == 1 && (tiles128 % 2) == 0) {
    const int units2 = tiles128 / 2, KB = K / 64;
    int best = 0;
    for (int ns = 2; ns <= 8 && ns <= KB; ++ns) {
      int &cap = c->max_clusters[T / 16][ns];
      if (cap < 0) { int v = 0; if (gemm_tc_max_clusters(T, ns, &v) != cudaSuccess) { v = 0; (void)cudaGetLastError(); } cap = v; }
      if (cap >= units2) best = ns;
    }
    if (best > 0 && units2 * best >= tiles128 * A.nsplit) { A.wtiles = 2; A.nsplit = best; }
  }
  // CTA pairs with K slices: each CTA stages half of the activation box; taken when all clusters of 2 x slices are
  // resident at once and (unless forced) about as many CTAs run as in the one-CTA form - at 256 rows that is the QKV
  // projection (24 pair tiles x 2 slices); O and down would run on 80 CTAs instead of 120 and gain nothing
  if (c->pair_split && A.nsplit > 1 && A.wtiles == 1 && T == 256 && mblocks == 1 && (tiles128 % 2) == 0 && epi != EPI_QKV_ROPE) {
    const int KB = K / 64;
    int best = 0;
    for (int ns = 2; ns <= (c->pair_split >= 3 ? 8 : 4) && ns <= KB; ++ns) {
      int &cap = c->pair_split_clusters[ns];
      if (cap < 0) {
        int v = 0;
        if (gemm_pair_split_max_clusters(T, ns, &v) != cudaSuccess) { v = 0; (void)cudaGetLastError(); }
        if (std::getenv("GM_DEBUG")) std::fprintf(stderr, "[gm] resident pair clusters T=%d slices=%d: %d\n", T, ns, v);
        cap = v;
      }
      if (cap >= tiles128 / 2) best = ns;
    }
    if (best > 0 && (c->pair_split >= 2 || (tiles128 / 2) * 2 * best >= tiles128 * A.nsplit * 3 / 4)) {
      A.nsplit = best; A.n_base = 0; A.n_tiles = tiles128;
      if (std::getenv("GM_DEBUG")) std::fprintf(stderr, "[gm] pair split: N=%d K=%d slices=%d\n", N, K, best);
      rc = x_map(c, x, x_rows, K, T / 2, &A.x_half_map);
      if (rc != GM_OK) return rc;
      GM_LAUNCH(c, GM_KC_GEMM, launch_gemm_pair_split(A, c->stream));
      return GM_OK;
    }
  }
  // very wide projections: two sub-tiles per CTA halve the activation re-reads from L2
  if (A.nsplit == 1 && tiles128 * mblocks >= 2 * c->sm_count) A.wtiles = 2;
  const int units = (tiles128 + A.wtiles - 1) / A.wtiles;          // CTAs along N
  A.n_base = 0;
  A.n_tiles = units;
  // Wave quantisation: a few CTAs more than a multiple of the SM count would cost a whole extra wave.  Run the full
  // waves as they are and the leftover features as a short launch whose tiles are split along K over clusters.
  const int rem = (units * mblocks) % c->sm_count;
  if (A.nsplit == 1 && mblocks == 1 && units > c->sm_count && rem != 0 && rem * 4 <= c->sm_count) {
    A.n_tiles = units - rem;
    if (c->pair_gemm && A.wtiles == 1 && (T % 32) == 0 && (A.n_tiles % 2) == 0) {
      rc = x_map(c, x, x_rows, K, T / 2, &A.x_half_map);
      if (rc != GM_OK) return rc;
      GM_LAUNCH(c, GM_KC_GEMM, launch_gemm_pair(A, c->stream));
    } else {
      GM_LAUNCH(c, GM_KC_GEMM, launch_gemm_tc(A, c->stream));
    }
    GemmArgs Tl = A;
    Tl.n_base = A.n_tiles * 128 * A.wtiles;
    Tl.wtiles = 1;
    Tl.n_tiles = (N - Tl.n_base + 127) / 128;
    Tl.nsplit = 1;
    const int KB = K / 64;
    for (int ns = 2; ns <= 8 && ns <= KB; ++ns) {
      int &cap = c->max_clusters[T / 16][ns];
      if (cap < 0) { int v = 0; if (gemm_tc_max_clusters(T, ns, &v) != cudaSuccess) { v = 0; (void)cudaGetLastError(); } cap = v; }
      if (cap >= Tl.n_tiles) Tl.nsplit = ns;
    }
    GM_LAUNCH(c, GM_KC_GEMM, launch_gemm_tc(Tl, c->stream));
    return GM_OK;
  }
  // Several token blocks (prefill passes, the head update's prefix passes) on a projection too narrow for two sub-tiles
  // per CTA: CTA pairs, each CTA staging half of the activation box (2/3 of the bytes into shared memory per K block).
  if (c->pair_gemm && c->pair_blocks && A.nsplit == 1 && A.wtiles == 1 && mblocks > 1 && T == 256 && (units % 2) == 0 &&
      epi != EPI_QKV_ROPE) {
    rc = x_map(c, x, x_rows, K, T / 2, &A.x_half_map);
    if (rc != GM_OK) return rc;
    GM_LAUNCH(c, GM_KC_GEMM, launch_gemm_pair(A, c->stream));
    return GM_OK;
  }
  GM_LAUNCH(c, GM_KC_GEMM, launch_gemm_tc(A, c->stream));
  return GM_OK;
}

bool chain_usable(const gm_ctx *c, int M) { return c->chain_on && c->chain_mode == 2 && M <= c->chain_max_m; }

// A chain of dependent projections as one persistent launch.
int run_chain(gm_ctx *c, const ChainSpec *specs, int n, int M) {
  ChainArgs A;
  std::memset(&A, 0, sizeof(A));
  A.n_phases = n; A.M = M; A.mblocks = (M + 255) / 256; A.P = c->chain_pairs; A.m_pad = c->Mmax;
  A.eps = c->cfg.rms_eps; A.partial = c->chain_partial; A.sync = c->chain_sync; A.status = c->status;
  A.timeline = c->chain_trace_on ? c->chain_trace : nullptr;
  A.npw = c->chain_npw; A.npa = c->chain_npa;
  A.trace_phase = std::getenv("GM_CHAIN_TRACE_PHASE") ? std::atoi(std::getenv("GM_CHAIN_TRACE_PHASE")) : 1;
  for (int p = 0; p < n; ++p) {
    const ChainSpec &s = specs[p];
    ChainPhase &ph = A.ph[p];
    ph.out = s.out; ph.xg = s.xg; ph.gamma = s.gamma; ph.sq_out = s.sq_out; ph.sq_in = s.sq_in;
    ph.inv_dim = s.sq_in ? 1.0f / static_cast<float>(s.norm_dim) : 0.f;
    ph.epi = s.epi; ph.N = s.N; ph.K = s.K; ph.ldo = s.ldo;
    chain_schedule(ph, A.mblocks, A.P, n >= 3 ? c->chain_force_ns[p] : 0);
    ph.sq_groups = s.sq_in ? A.ph[s.sq_from].tiles : 0;
    auto key = std::make_tuple(s.w, s.N, s.K, ph.wbox);
    auto it = c->chain_w_maps.find(key);
    if (it == c->chain_w_maps.end()) {
      CUtensorMap m;
      if (make_map(c, &m, s.w, s.N, s.K, ph.wbox) != GM_OK) return GM_ERR_CUDA;
      it = c->chain_w_maps.emplace(key, m).first;
    }
    ph.w_map = it->second;
    // rows beyond M are out of the map's bounds: the copy engine fills them with zeros and fetches nothing
    int rc = x_map(c, s.x, M < s.x_rows ? M : s.x_rows, s.K, 128, &ph.x_map);
    if (rc != GM_OK) return rc;
  }
  GM_LAUNCH(c, GM_KC_GEMM, launch_chain(A, c->stream));
  return GM_OK;
}

// One decoder layer on rows x/xn [M, d] (xn = normed input).  kv_only: stop after the rows' keys and values are in the cache.  `next_norm` is the RMSNorm weight applied to
// the layer's output for whatever consumes it next (null: none); `hidden_out` optionally receives the
// bf16 residual stream.
int run_layer(gm_ctx *c, const gm_layer_weights &lw, const LayerMaps &lm, const PhaseShape &ph, const CUtensorMap &kvm,
              __nv_bfloat16 *pool, int layer, int num_pages, const int32_t *page_table,
              const __nv_bfloat16 *next_norm, __nv_bfloat16 *hidden_out, const gm_layer_weights *next_lw,
              const LayerMaps *next_lm, bool qkv_done, bool kv_only) {
  const gm_config &cf = c->cfg;
  const bool chain = chain_usable(c, ph.M);
  int rc;
  // QKV projection (bf16) -> rotary + KV append + Q rearrangement: in the projection's epilogue where the tensor-core
  // kernel runs it and a 128-feature tile holds whole heads, else as a kernel of its own
  RopeAppendArgs R;
  R.qkv = c->qkv;
  R.batch = ph.B; R.QT = ph.QT; R.n_q = cf.n_q_heads; R.n_kv = cf.n_kv_heads; R.hd = cf.head_dim; R.layer = layer;
  R.num_pages = num_pages; R.max_pages_per_seq = cf.max_pages_per_seq; R.qrows = ph.qrows;
  R.qn = c->qn; R.qbase = c->qbase; R.page_table = page_table; R.rope = c->rope; R.qbuf = c->qbuf; R.pool = pool;
  R.status = c->status;
  R.bias = static_cast<const __nv_bfloat16 *>(lw.b_qkv);
  R.qnorm = static_cast<const __nv_bfloat16 *>(lw.q_norm); R.knorm = static_cast<const __nv_bfloat16 *>(lw.k_norm);
  R.eps = cf.rms_eps;
  const bool fuse_rope = c->fuse_rope && !chain && !(cf.flags & GM_FLAG_SIMPLE_GEMM) && (cf.head_dim == 64 || cf.head_dim == 128) &&
                         (c->d % 64) == 0;
  if (!(chain && qkv_done)) {
    if (chain) {
      const ChainSpec q = {lw.wqkv, c->xn, c->Mmax, c->n_qkv, c->d, c->qkv, EPI_STORE_BF16, c->n_qkv,
                           nullptr, nullptr, nullptr, nullptr, 0, 0};
      rc = run_chain(c, &q, 1, ph.M);
    } else {
      rc = run_gemm(c, c->xn, c->Mmax, &lm.wqkv, static_cast<const __nv_bfloat16 *>(lw.wqkv), ph.M, c->n_qkv, c->d,
                    c->qkv, fuse_rope ? EPI_QKV_ROPE : EPI_STORE_BF16, c->n_qkv, true, fuse_rope ? &R : nullptr);
    }
    if (rc) return rc;
  }
  if (!fuse_rope) GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_rope_append(R, c->stream));
  if (kv_only) return GM_OK;          // the rows' cache entries are all the caller needs (nothing reads their outputs)
  // attention over the pages + merge of the segments
  AttnArgs T;
  T.kv_map = kvm; T.qbuf = c->qbuf; T.qn = c->qn; T.qbase = c->qbase; T.page_start = c->page_start;
  T.page_table = page_table; T.batch = ph.B; T.n_kv = cf.n_kv_heads; T.group = c->group; T.hd = cf.head_dim;
  T.qrows = ph.qrows; T.layer = layer; T.num_pages = num_pages; T.max_pages_per_seq = cf.max_pages_per_seq;
  T.n_ctas = c->sm_count; T.scale_log2e = static_cast<float>(1.4426950408889634 / std::sqrt(static_cast<double>(cf.head_dim)));
  T.part_o = c->part_o; T.part_ml = c->part_ml; T.status = c->status; T.rows_used = ph.QT * c->group;
  GM_LAUNCH(c, GM_KC_ATTENTION, launch_attention(T, c->stream));
  AttnCombineArgs Cb;
  Cb.part_o = c->part_o; Cb.part_ml = c->part_ml; Cb.qn = c->qn; Cb.page_start = c->page_start; Cb.batch = ph.B;
  Cb.n_kv = cf.n_kv_heads; Cb.group = c->group; Cb.hd = cf.head_dim; Cb.qrows = ph.qrows; Cb.QT = ph.QT;
  Cb.n_ctas = c->sm_count; Cb.out = c->attn_out;
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_attention_combine(Cb, c->stream));
  if (chain) {
    // output projection (+ residual), gate/up (+ SwiGLU), down (+ residual) and the next layer's QKV in one launch;
    // the two norms in between are folded around the projections (see chain.cu)
    const bool fuse_next = next_lw && next_lm && next_norm;
    ChainSpec sp[4];
    sp[0] = {lw.wo, c->attn_out, c->Mmax, c->d, c->q_dim, c->x, EPI_ADD_F32, c->d,
             c->xn, static_cast<const __nv_bfloat16 *>(lw.ln2), c->chain_sq[0], nullptr, 0, 0};
    sp[1] = {lw.w_gate_up, c->xn, c->Mmax, 2 * c->F, c->d, c->act, EPI_SWIGLU_BF16, c->F,
             nullptr, nullptr, nullptr, c->chain_sq[0], 0, c->d};
    sp[2] = {lw.w_down, c->act, c->Mmax, c->d, c->F, c->x, EPI_ADD_F32, c->d,
             fuse_next ? c->xn : nullptr, fuse_next ? next_norm : nullptr, fuse_next ? c->chain_sq[1] : nullptr, nullptr, 0, 0};
    if (fuse_next)
      sp[3] = {next_lw->wqkv, c->xn, c->Mmax, c->n_qkv, c->d, c->qkv, EPI_STORE_BF16, c->n_qkv,
               nullptr, nullptr, nullptr, c->chain_sq[1], 2, c->d};
    if ((rc = run_chain(c, sp, fuse_next ? 4 : 3, ph.M)) != GM_OK) return rc;
    if (!fuse_next && (next_norm || hidden_out))
      GM_LAUNCH(c, GM_KC_ELEMENTWISE,
                launch_rmsnorm(c->x, next_norm, next_norm ? c->xn : nullptr, hidden_out, ph.M, c->d, cf.rms_eps,
                               c->stream));
    return GM_OK;
  }
  // output projection added into the residual stream, then the post-attention norm
  rc = run_gemm(c, c->attn_out, c->Mmax, &lm.wo, static_cast<const __nv_bfloat16 *>(lw.wo), ph.M, c->d, c->q_dim,
                c->x, EPI_ADD_F32, c->d);
  if (rc) return rc;
  GM_LAUNCH(c, GM_KC_ELEMENTWISE,
            launch_rmsnorm(c->x, static_cast<const __nv_bfloat16 *>(lw.ln2), c->xn, nullptr, ph.M, c->d, cf.rms_eps,
                           c->stream));
  // SwiGLU feed-forward: gate/up projection with the activation in its epilogue, down projection into the residual
  rc = run_gemm(c, c->xn, c->Mmax, &lm.wgu, static_cast<const __nv_bfloat16 *>(lw.w_gate_up), ph.M, 2 * c->F, c->d,
                c->act, EPI_SWIGLU_BF16, c->F);
  if (rc) return rc;
  rc = run_gemm(c, c->act, c->Mmax, &lm.wdown, static_cast<const __nv_bfloat16 *>(lw.w_down), ph.M, c->d, c->F,
                c->x, EPI_ADD_F32, c->d);
  if (rc) return rc;
  if (next_norm || hidden_out)
    GM_LAUNCH(c, GM_KC_ELEMENTWISE,
              launch_rmsnorm(c->x, next_norm, next_norm ? c->xn : nullptr, hidden_out, ph.M, c->d, cf.rms_eps,
                             c->stream));
  return GM_OK;
}

int run_plan(gm_ctx *c, const gm_state *st, int mode, int k_or_j) {
  PlanArgs P;
  P.mode = mode; P.batch = st->batch; P.k_or_j = k_or_j; P.max_pages_per_seq = c->cfg.max_pages_per_seq;
  P.n_ctas = c->sm_count; P.kv_len = st->kv_len; P.pending_n = st->pending_n; P.qn = c->qn; P.qbase = c->qbase;
  P.page_start = c->page_start; P.status = c->status; P.finished = c->finished_mask;
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_plan(P, c->stream));
  return GM_OK;
}

int run_plan_chunk(gm_ctx *c, int batch, const int32_t *row_n, const int32_t *row_base, int QT) {
  PlanArgs P;
  P.mode = PHASE_CHUNK; P.batch = batch; P.k_or_j = 0; P.row_base = row_base; P.max_pages_per_seq = c->cfg.max_pages_per_seq;
  P.n_ctas = c->sm_count; P.kv_len = row_n; P.pending_n = row_n; P.row_n = row_n; P.QT = QT; P.qn = c->qn; P.qbase = c->qbase;
  P.page_start = c->page_start; P.status = c->status;
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_plan(P, c->stream));
  return GM_OK;
}

int check_state(const gm_ctx *c, const gm_state *st, int k) {
  if (!c || !st) return GM_ERR_INVALID_ARG;
  if (k < 1 || k > c->cfg.max_k) return k > c->cfg.max_k ? GM_ERR_UNSUPPORTED : GM_ERR_INVALID_ARG;
  if (st->batch < 1 || st->batch > c->cfg.max_batch) return GM_ERR_INVALID_ARG;
  if (!st->kv_len || !st->page_table || !st->kv_pool || !st->head_page_table || !st->head_kv_pool || !st->pending_n ||
      !st->pending_tok || !st->pending_hidden)
    return GM_ERR_INVALID_ARG;
  return GM_OK;
}

// Mapping of the sampler: a cluster per sequence while sequences are few, one CTA per sequence once there are enough
// of them to fill the SMs (the flags force one or the other).
cudaError_t run_sampler(gm_ctx *c, const SamplerArgs &S, int batch) {
  int mode = c->sampler_mode;
  if (c->cfg.flags & GM_FLAG_SAMPLER_CLUSTER) mode = 1;
  if (c->cfg.flags & GM_FLAG_SAMPLER_STREAM) mode = 2;
  if (c->cfg.flags & GM_FLAG_SAMPLER_FLOW) mode = 3;
  // by batch size (measured at K = 3, V = 151936): a cluster per sequence while sequences are few, the sliced mapping up
  // to two sequences per SM, one CTA per sequence beyond
  if (mode == 0) mode = batch * 3 < c->sm_count * 2 ? 1 : (batch <= c->sm_count * 2 ? 3 : 2);
  if (mode == 3 && !sampler_flow_supported(S.V, batch, S.K, c->sm_count)) mode = 2;
  if (mode == 3) {
    if (batch > c->flow_cap) {                         // a batch above max_batch (stand-alone gm_accept): grow, outside any capture
      const size_t need = sampler_flow_ws_bytes(batch, S.V, c->sm_count);
      void *q = nullptr;
      if (cudaError_t e = cudaMalloc(&q, need); e != cudaSuccess) return e;
      c->allocs.push_back(q);
      if (cudaError_t e = cudaMemsetAsync(q, 0, need, c->stream); e != cudaSuccess) return e;
      c->flow_ws = q; c->flow_ws_bytes = need; c->flow_cap = batch;
    }
    return launch_sampler_flow(S, batch, c->flow_ws, c->flow_cap, c->sm_count, c->stream);
  }
  if (mode == 2 && sampler_stream_supported(S.V)) return launch_sampler_stream(S, batch, c->stream);
  return launch_sampler(S, batch, c->stream);
}

int fill_sampler(gm_ctx *c, SamplerArgs &S, float temperature) {
  if (!(temperature > 0.f) || !std::isfinite(temperature)) return GM_ERR_UNSUPPORTED;
  std::memset(&S, 0, sizeof(S));
  S.inv_temp = 1.0f / temperature;
  S.V = c->V;
  S.status = c->status;
  S.slot_accept = SLOT_ACCEPT;
  S.slot_final = SLOT_FINAL;
  S.finished = c->finished_mask;
  S.step_ptr = c->step_ptr;
  return GM_OK;
}

}  // namespace gmh

// ======================================================================================================================
extern "C" {

const char *gm_strerror(int code) {
  switch (code) {
    case GM_OK: return "ok";
    case GM_ERR_INVALID_ARG: return "invalid argument";
    case GM_ERR_UNSUPPORTED: return "unsupported configuration";
    case GM_ERR_KV_CAPACITY: return "a sequence's pages cannot hold kv_len + k + 1 positions";
    case GM_ERR_CUDA: return "CUDA call failed";
    case GM_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
    case GM_ERR_BAD_PAGE: return "page id or token id outside its range";
    case GM_ERR_NO_EXTENSION: return "no sm_100 device";
    case GM_ERR_OVERRUN: return "a guard word behind a library workspace was overwritten";
    case GM_ERR_SCRATCH_LIMIT: return "request exceeds the static scratch of the no-alloc entry point (see GM_NOALLOC_SCRATCH_BYTES)";
    default: return "unknown error";
  }
}

int gm_init(gm_ctx **out, const gm_config *cfg, const gm_weights *w, void *cuda_stream) {
  if (!out || !cfg || !w) return GM_ERR_INVALID_ARG;
  *out = nullptr;
  if (cfg->n_layers < 1 || cfg->d_model < 64 || cfg->n_q_heads < 1 || cfg->n_kv_heads < 1 || cfg->d_ffn < 64 ||
      cfg->vocab < 8 || cfg->max_batch < 1 || cfg->max_k < 1 || cfg->max_pages_per_seq < 1 || cfg->num_pages < 1 ||
      cfg->head_num_pages < 1 || !(cfg->rope_base > 1.f) || !(cfg->rms_eps >= 0.f))
    return GM_ERR_INVALID_ARG;
  if (cfg->page_size != GM_PAGE || cfg->max_k > GM_MAX_K || (cfg->vocab % 8) || (cfg->d_model % 64) ||
      (cfg->d_ffn % 64) || (cfg->head_dim != 64 && cfg->head_dim != 128) || (cfg->n_q_heads % cfg->n_kv_heads) ||
      cfg->d_model > 8192 || cfg->max_batch > 1024 || (cfg->n_kv_heads > 8 && cfg->n_kv_heads % 8))
    return GM_ERR_UNSUPPORTED;
  const int group = cfg->n_q_heads / cfg->n_kv_heads;
  if ((cfg->max_k + 1) * group > 32) return GM_ERR_UNSUPPORTED;
  if (!w->embed || !w->lm_head || !w->final_norm || !w->layers || !w->head_enorm || !w->head_hnorm || !w->head_proj ||
      !w->head_final_norm)
    return GM_ERR_INVALID_ARG;
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return GM_ERR_NO_EXTENSION;
  cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  if (major != 10) return GM_ERR_NO_EXTENSION;

  gm_ctx *c = new (std::nothrow) gm_ctx();
  if (!c) return GM_ERR_INVALID_ARG;
  c->cfg = *cfg;
  c->w = *w;
  c->layers.assign(w->layers, w->layers + cfg->n_layers);
  c->w.layers = c->layers.data();
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  c->check_guards = std::getenv("GM_CANARY") != nullptr;
  c->pair_gemm = std::getenv("GM_NO_PAIR_GEMM") == nullptr;
  cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, dev);
  c->d = cfg->d_model; c->q_dim = cfg->n_q_heads * cfg->head_dim; c->kv_dim = cfg->n_kv_heads * cfg->head_dim;
  c->n_qkv = c->q_dim + 2 * c->kv_dim; c->F = cfg->d_ffn; c->V = cfg->vocab; c->group = group;
  c->Mmax = cfg->max_batch * (cfg->max_k + 1);

  auto fail = [&](int code) { gm_destroy(c); return code; };
  {
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn)
      return fail(GM_ERR_CUDA);
    c->encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
  }
  for (int l = 0; l < cfg->n_layers; ++l) {
    const gm_layer_weights &lw = c->layers[l];
    if (!lw.ln1 || !lw.wqkv || !lw.wo || !lw.ln2 || !lw.w_gate_up || !lw.w_down || !lw.q_norm != !lw.k_norm)
      return fail(GM_ERR_INVALID_ARG);
  }
  {
    const gm_layer_weights &lw = w->head_layer;
    if (!lw.ln1 || !lw.wqkv || !lw.wo || !lw.ln2 || !lw.w_gate_up || !lw.w_down || !lw.q_norm != !lw.k_norm)
      return fail(GM_ERR_INVALID_ARG);
  }
  auto layer_maps = [&](const gm_layer_weights &lw, LayerMaps &lm) {
    int rc = make_map(c, &lm.wqkv, lw.wqkv, c->n_qkv, c->d, 128);
    if (!rc) rc = make_map(c, &lm.wo, lw.wo, c->d, c->q_dim, 128);
    if (!rc) rc = make_map(c, &lm.wgu, lw.w_gate_up, 2 * c->F, c->d, 128);
    if (!rc) rc = make_map(c, &lm.wdown, lw.w_down, c->d, c->F, 128);
    return rc;
  };
  c->lmaps.resize(cfg->n_layers);
  for (int l = 0; l < cfg->n_layers; ++l)
    if (layer_maps(c->layers[l], c->lmaps[l])) return fail(GM_ERR_CUDA);
  if (layer_maps(w->head_layer, c->head_maps)) return fail(GM_ERR_CUDA);
  if (make_map(c, &c->lm_head_map, w->lm_head, c->V, c->d, 128)) return fail(GM_ERR_CUDA);
  if (make_map(c, &c->head_proj_map, w->head_proj, c->d, 2 * c->d, 128)) return fail(GM_ERR_CUDA);

  // workspaces
  // Sized for the widest phase: a prefill pass of pf_vr virtual rows per sequence (at most 1024 rows for the planner).
  c->pf_vr = std::max(1, std::min(8, 1024 / cfg->max_batch));
  const size_t B1 = cfg->max_batch, M1 = c->Mmax;                  // rows of a cycle
  const size_t B = B1 * c->pf_vr, M = M1 * c->pf_vr;                // rows of a prefill pass
  c->Mmax = static_cast<int>(M);
  const int qrows = round16((cfg->max_k + 1) * group);
  for (auto &row : c->max_clusters)
    for (int &v : row) v = -1;
  int rc = GM_OK;
  const size_t slots = static_cast<size_t>(c->sm_count) + B;
#define A_(call) if ((rc = (call)) != GM_OK) return fail(rc)
  A_(dev_alloc(c, &c->x, M * c->d));
  A_(dev_alloc(c, &c->xn, M * c->d));
  A_(dev_alloc(c, &c->zin, M * 2 * c->d));
  A_(dev_alloc(c, &c->qkv, M * c->n_qkv));
  A_(dev_alloc(c, &c->qbuf, B * cfg->n_kv_heads * qrows * cfg->head_dim));
  A_(dev_alloc(c, &c->attn_out, M * c->q_dim));
  A_(dev_alloc(c, &c->act, M * c->F));
  A_(dev_alloc(c, &c->g, B1 * c->d));
  A_(dev_alloc(c, &c->gn, B1 * c->d));
  A_(dev_alloc(c, &c->part_o, slots * cfg->n_kv_heads * qrows * cfg->head_dim));
  A_(dev_alloc(c, &c->part_ml, slots * cfg->n_kv_heads * qrows * 2));
  A_(dev_alloc(c, &c->ws_draft_logits, B1 * cfg->max_k * c->V, false));
  A_(dev_alloc(c, &c->ws_target_logits, B1 * (cfg->max_k + 1) * c->V, false));
  A_(dev_alloc(c, &c->ws_target_hidden, M1 * c->d));
  A_(dev_alloc(c, &c->ws_draft_tok, B1 * cfg->max_k));
  A_(dev_alloc(c, &c->ws_accept_len, B1));
  A_(dev_alloc(c, &c->ws_next_token, B1));
  A_(dev_alloc(c, &c->ws_u24, B1 * (2 * cfg->max_k + 1)));
  A_(dev_alloc(c, &c->qn, B));
  A_(dev_alloc(c, &c->qbase, B));
  A_(dev_alloc(c, &c->page_start, B + 1));
  A_(dev_alloc(c, &c->ro_accept, B1));
  A_(dev_alloc(c, &c->ro_next, B1));
  A_(dev_alloc(c, &c->pf_row_n, B));
  A_(dev_alloc(c, &c->pf_head_n, B));
  A_(dev_alloc(c, &c->pf_row_base, B));
  A_(dev_alloc(c, &c->pf_vtable[0], B * cfg->max_pages_per_seq));
  A_(dev_alloc(c, &c->pf_vtable[1], B * cfg->max_pages_per_seq));
  A_(dev_alloc(c, &c->pf_first, B1));
  A_(dev_alloc(c, &c->pf_pair_tok, B * (cfg->max_k + 1)));
  A_(dev_alloc(c, &c->pf_hidden, M * c->d));
  A_(dev_alloc(c, &c->pf_xlast, B1 * c->d));
  A_(dev_alloc(c, &c->status, 1));
  if (sampler_flow_supported(c->V, static_cast<int>(B), cfg->max_k, c->sm_count)) {
    unsigned char *ws = nullptr;
    c->flow_ws_bytes = sampler_flow_ws_bytes(static_cast<int>(B), c->V, c->sm_count);
    c->flow_cap = static_cast<int>(B);
    A_(dev_alloc(c, &ws, c->flow_ws_bytes));
    c->flow_ws = ws;
  }
  if (std::getenv("GM_NO_EARLY_W")) c->early_weights = false;
  if (const char *ws = std::getenv("GM_GEMM_WIDE_SPLIT")) c->wide_split = std::atoi(ws) != 0;
  if (const char *pb = std::getenv("GM_GEMM_PAIR_BLOCKS")) c->pair_blocks = std::atoi(pb) != 0;
  if (const char *ps = std::getenv("GM_GEMM_PAIR_SPLIT")) c->pair_split = std::atoi(ps);
  if (std::getenv("GM_FUSED_ROPE")) c->fuse_rope = true;
  if (const char *ov = std::getenv("GM_SAMPLER")) {     // tuning aid: cluster | stream | flow for every sampler launch
    c->sampler_mode = !std::strcmp(ov, "cluster") ? 1 : !std::strcmp(ov, "stream") ? 2 : !std::strcmp(ov, "flow") ? 3 : 0;
  }
  // persistent chain of a layer's projections: every CTA pair must be resident at once
  if (!(cfg->flags & GM_FLAG_SIMPLE_GEMM) && (c->q_dim % 64) == 0) {
    int pairs = 0;
    if (chain_max_pairs(&pairs) != cudaSuccess) { pairs = 0; (void)cudaGetLastError(); }
    if (pairs > c->sm_count / 2) pairs = c->sm_count / 2;
    if (const char *ov = std::getenv("GM_CHAIN_PAIRS")) { const int v = std::atoi(ov); if (v >= 1 && v < pairs) pairs = v; }
    if (const char *ov = std::getenv("GM_CHAIN_NPW")) { const int v = std::atoi(ov); if (v >= 1 && v <= 4) c->chain_npw = v; }
    if (const char *ov = std::getenv("GM_CHAIN_NPA")) c->chain_npa = std::atoi(ov) == 1 ? 1 : 2;
    if (const char *ov = std::getenv("GM_CHAIN_MODE")) { const int v = std::atoi(ov); if (v >= 0 && v <= 2) c->chain_mode = v; }
    if (const char *ov = std::getenv("GM_CHAIN_MAX_M")) { const int v = std::atoi(ov); if (v >= 1) c->chain_max_m = v; }
    if (pairs >= 1) {
      c->chain_pairs = pairs;
      A_(dev_alloc(c, &c->chain_partial, chain_partial_floats(pairs)));
      A_(dev_alloc(c, &c->chain_sq[0], static_cast<size_t>((c->d + 15) / 16) * M));     // one row per feature tile (at most per 16 features)
      A_(dev_alloc(c, &c->chain_sq[1], static_cast<size_t>((c->d + 15) / 16) * M));
      A_(dev_alloc(c, &c->chain_sync, 1 + static_cast<size_t>(pairs) * 2));
      if (const char *ov = std::getenv("GM_CHAIN_NS"))
        std::sscanf(ov, "%d,%d,%d,%d", &c->chain_force_ns[0], &c->chain_force_ns[1], &c->chain_force_ns[2], &c->chain_force_ns[3]);
      c->chain_on = true;
    }
  }
  // rotary table: cos/sin of pos * base^(-2i/hd), computed in double precision on the host
  {
    const int half = cfg->head_dim / 2;
    const size_t max_pos = static_cast<size_t>(cfg->max_pages_per_seq) * 16;
    std::vector<float2> tab(max_pos * half);
    for (int i = 0; i < half; ++i) {
      const double inv = std::pow(static_cast<double>(cfg->rope_base), -2.0 * i / cfg->head_dim);
      for (size_t p = 0; p < max_pos; ++p) {
        const double a = static_cast<double>(p) * inv;
        tab[p * half + i] = make_float2(static_cast<float>(std::cos(a)), static_cast<float>(std::sin(a)));
      }
    }
    A_(dev_alloc(c, &c->rope, tab.size(), false));
    if (cudaMemcpyAsync(c->rope, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice, c->stream) != cudaSuccess)
      return fail(GM_ERR_CUDA);
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) return fail(GM_ERR_CUDA);
  }
#undef A_
  *out = c;
  return GM_OK;
}

void gm_destroy(gm_ctx *c) {
  if (!c) return;
  cudaStreamSynchronize(c->stream);
  if (c->graph_rollout.exec) cudaGraphExecDestroy(c->graph_rollout.exec);
  if (c->graph_step.exec) cudaGraphExecDestroy(c->graph_step.exec);
  for (void *p : c->allocs) cudaFree(p);
  for (auto &v : c->events)
    for (auto &e : v) { cudaEventDestroy(e.a); cudaEventDestroy(e.b); }
  delete c;
}

int gm_draft(gm_ctx *c, const gm_state *st, int k, float temperature, const uint32_t *u24_draft, uint64_t seed,
             uint64_t step, int32_t *draft_tok, void *draft_logits, float *dbg_q) {
  return draft_impl(c, st, k, temperature, u24_draft, seed, step, draft_tok, draft_logits, dbg_q, false);
}

}  // extern "C"

int gmh::draft_impl(gm_ctx *c, const gm_state *st, int k, float temperature, const uint32_t *u24_draft, uint64_t seed,
                    uint64_t step, int32_t *draft_tok, void *draft_logits, float *dbg_q, bool forced) {
  NvtxRange nvtx_range("gm_draft");
  int rc = check_state(c, st, k);
  if (rc) return rc;
  if (!draft_tok || !draft_logits) return GM_ERR_INVALID_ARG;
  SamplerArgs S;
  if ((rc = fill_sampler(c, S, temperature)) != GM_OK) return rc;
  const gm_config &cf = c->cfg;
  CUtensorMap kvm;
  if ((rc = kv_map(c, st->head_kv_pool, 1, cf.head_num_pages, &kvm)) != GM_OK) return rc;
  __nv_bfloat16 *dl = static_cast<__nv_bfloat16 *>(draft_logits);
  for (int j = 1; j <= k; ++j) {
    const int mode = j == 1 ? PHASE_DRAFT_FIRST : PHASE_DRAFT_NEXT;
    PhaseShape ph;
    ph.B = st->batch; ph.QT = j == 1 ? cf.max_k + 1 : 1; ph.M = ph.B * ph.QT; ph.qrows = round16(ph.QT * c->group);
    if ((rc = run_plan(c, st, mode, j == 1 ? cf.max_k + 1 : j)) != GM_OK) return rc;
    HeadInputArgs H;
    H.mode = mode; H.batch = ph.B; H.QT = ph.QT; H.d = c->d; H.vocab = c->V; H.max_k = cf.max_k; H.k = k; H.j = j;
    H.eps = cf.rms_eps; H.embed = static_cast<const __nv_bfloat16 *>(c->w.embed);
    H.we = static_cast<const __nv_bfloat16 *>(c->w.head_enorm); H.wh = static_cast<const __nv_bfloat16 *>(c->w.head_hnorm);
    H.pending_tok = st->pending_tok; H.pending_n = st->pending_n;
    H.pending_hidden = static_cast<const __nv_bfloat16 *>(st->pending_hidden); H.draft_tok = draft_tok; H.g_prev = c->g;
    H.zin = c->zin; H.status = c->status;
    GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_head_input(H, c->stream));
    rc = run_gemm(c, c->zin, c->Mmax, &c->head_proj_map, static_cast<const __nv_bfloat16 *>(c->w.head_proj), ph.M, c->d,
                  2 * c->d, c->x, EPI_STORE_F32, c->d);
    if (rc) return rc;
    GM_LAUNCH(c, GM_KC_ELEMENTWISE,
              launch_rmsnorm(c->x, static_cast<const __nv_bfloat16 *>(c->w.head_layer.ln1), c->xn, nullptr, ph.M, c->d,
                             cf.rms_eps, c->stream));
    rc = run_layer(c, c->w.head_layer, c->head_maps, ph, kvm, static_cast<__nv_bfloat16 *>(st->head_kv_pool), 0,
                   cf.head_num_pages, st->head_page_table, nullptr, nullptr);
    if (rc) return rc;
    GM_LAUNCH(c, GM_KC_ELEMENTWISE,
              launch_head_out(c->x, c->qn, ph.B, ph.QT, c->d, static_cast<const __nv_bfloat16 *>(c->w.head_final_norm),
                              cf.rms_eps, c->g, c->gn, c->stream));
    if (c->state_out)                      // the update's backward pass wants g_j of every chain (row stride k*d)
      GM_CUDA(c, cudaMemcpy2DAsync(c->state_out + static_cast<size_t>(j - 1) * c->d, sizeof(float) * k * c->d, c->g,
                                   sizeof(float) * c->d, sizeof(float) * c->d, ph.B, cudaMemcpyDeviceToDevice, c->stream));
    // shared LM head -> row j-1 of every sequence's draft logits (row stride k*V)
    rc = run_gemm(c, c->gn, cf.max_batch, &c->lm_head_map, static_cast<const __nv_bfloat16 *>(c->w.lm_head), ph.B, c->V,
                  c->d, dl + static_cast<size_t>(j - 1) * c->V, EPI_STORE_BF16, static_cast<size_t>(k) * c->V);
    if (rc) return rc;
    // d_j ~ softmax(logits / T): the sampler with depth 0
    S.K = 0; S.target_logits = dl + static_cast<size_t>(j - 1) * c->V; S.tgt_bstride = static_cast<size_t>(k) * c->V;
    S.draft_logits = nullptr; S.u24 = u24_draft ? u24_draft + (j - 1) : nullptr; S.u_stride = k;
    S.seed = seed; S.step = step; S.slot_final = SLOT_DRAFT + (j - 1);
    S.accept_len = nullptr; S.next_token = draft_tok + (j - 1); S.tok_out_stride = k;
    S.dbg_p = dbg_q ? dbg_q + static_cast<size_t>(j - 1) * c->V : nullptr; S.dbg_q = nullptr; S.commit = 0;
    if (!forced) GM_LAUNCH(c, GM_KC_SAMPLER, run_sampler(c, S, ph.B));
  }
  return GM_OK;
}

extern "C" {

int gm_verify(gm_ctx *c, const gm_state *st, int k, const int32_t *draft_tok, void *target_logits,
              void *target_hidden) {
  NvtxRange nvtx_range("gm_verify");
  int rc = check_state(c, st, k);
  if (rc) return rc;
  if (!draft_tok || !target_logits || !target_hidden) return GM_ERR_INVALID_ARG;
  const gm_config &cf = c->cfg;
  PhaseShape ph;
  ph.B = st->batch; ph.QT = k + 1; ph.M = ph.B * ph.QT; ph.qrows = round16(ph.QT * c->group);
  CUtensorMap kvm;
  if ((rc = kv_map(c, st->kv_pool, cf.n_layers, cf.num_pages, &kvm)) != GM_OK) return rc;
  if ((rc = run_plan(c, st, PHASE_VERIFY, k)) != GM_OK) return rc;
  GM_LAUNCH(c, GM_KC_ELEMENTWISE,
            launch_embed_norm(static_cast<const __nv_bfloat16 *>(c->w.embed),
                              static_cast<const __nv_bfloat16 *>(c->layers[0].ln1), st->pending_tok, st->pending_n,
                              draft_tok, ph.B, k, cf.max_k, c->d, c->V, cf.rms_eps, c->x, c->xn, c->status, c->stream));
  for (int l = 0; l < cf.n_layers; ++l) {
    const bool last = l + 1 == cf.n_layers;
    const __nv_bfloat16 *next_norm =
        static_cast<const __nv_bfloat16 *>(last ? c->w.final_norm : c->layers[l + 1].ln1);
    rc = run_layer(c, c->layers[l], c->lmaps[l], ph, kvm, static_cast<__nv_bfloat16 *>(st->kv_pool), l, cf.num_pages,
                   st->page_table, next_norm, last ? static_cast<__nv_bfloat16 *>(target_hidden) : nullptr,
                   last ? nullptr : &c->layers[l + 1], last ? nullptr : &c->lmaps[l + 1], l > 0);
    if (rc) return rc;
  }
  return run_gemm(c, c->xn, c->Mmax, &c->lm_head_map, static_cast<const __nv_bfloat16 *>(c->w.lm_head), ph.M, c->V, c->d,
                  target_logits, EPI_STORE_BF16, c->V);
}

int gm_accept(gm_ctx *c, gm_state *st, int batch, int k, float temperature, const void *target_logits,
              const void *draft_logits, const int32_t *draft_tok, const uint32_t *u24_accept, uint64_t seed,
              uint64_t step, int32_t *accept_len, int32_t *next_token, float *dbg_p, float *dbg_q,
              const void *target_hidden, int commit_state) {
  NvtxRange nvtx_range("gm_accept");
  if (!c || !target_logits || !draft_logits || !draft_tok || !accept_len || !next_token) return GM_ERR_INVALID_ARG;
  if (k < 1 || batch < 1) return GM_ERR_INVALID_ARG;
  if (k > GM_MAX_K) return GM_ERR_UNSUPPORTED;
  if (commit_state) {
    int rc = check_state(c, st, k);
    if (rc) return rc;
    if (!target_hidden || batch != st->batch) return GM_ERR_INVALID_ARG;
  }
  SamplerArgs S;
  int rc = fill_sampler(c, S, temperature);
  if (rc) return rc;
  S.K = k;
  if (c->top_p < 1.f) {                 // truncate the target rows to their nucleus first; the head's rows stay as they are
    if (batch > c->cfg.max_batch || k > c->cfg.max_k) return GM_ERR_INVALID_ARG;
    if ((rc = run_nucleus(c, target_logits, batch * (k + 1), temperature, c->top_p, c->ws_nucleus, nullptr)) != GM_OK) return rc;
    target_logits = c->ws_nucleus;
  }
  S.target_logits = static_cast<const __nv_bfloat16 *>(target_logits); S.tgt_bstride = static_cast<size_t>(k + 1) * c->V;
  S.draft_logits = static_cast<const __nv_bfloat16 *>(draft_logits); S.drf_bstride = static_cast<size_t>(k) * c->V;
  S.draft_tok = draft_tok; S.tok_in_stride = k; S.u24 = u24_accept; S.u_stride = k + 1; S.seed = seed; S.step = step;
  S.accept_len = accept_len; S.next_token = next_token; S.tok_out_stride = 1; S.dbg_p = dbg_p; S.dbg_q = dbg_q;
  S.commit = commit_state ? 1 : 0;
  if (commit_state) {
    S.kv_len = st->kv_len; S.pending_n = st->pending_n; S.pending_tok = st->pending_tok;
    S.pending_hidden = static_cast<__nv_bfloat16 *>(st->pending_hidden);
    S.target_hidden = static_cast<const __nv_bfloat16 *>(target_hidden);
    S.d_model = c->d; S.max_k = c->cfg.max_k;
  }
  GM_LAUNCH(c, GM_KC_SAMPLER, run_sampler(c, S, batch));
  if (commit_state && c->capture)
    GM_LAUNCH(c, GM_KC_ELEMENTWISE,
              launch_capture_cycle(static_cast<const __nv_bfloat16 *>(target_hidden), accept_len, st->kv_len,
                                   c->finished_mask, batch, k, c->d, c->capture, c->capture_stride, c->stream));
  return GM_OK;
}

int gm_draw(gm_ctx *c, const void *logits, int rows, float temperature, const uint32_t *u24, int32_t *out_tok,
            float *dbg_prob) {
  if (!c || !logits || !u24 || !out_tok || rows < 1) return GM_ERR_INVALID_ARG;
  SamplerArgs S;
  int rc = fill_sampler(c, S, temperature);
  if (rc) return rc;
  S.K = 0; S.target_logits = static_cast<const __nv_bfloat16 *>(logits); S.tgt_bstride = c->V; S.u24 = u24; S.u_stride = 1;
  S.next_token = out_tok; S.tok_out_stride = 1; S.dbg_p = dbg_prob;
  GM_LAUNCH(c, GM_KC_SAMPLER, run_sampler(c, S, rows));
  return GM_OK;
}

// One cycle, host-launched or (GM_FLAG_GRAPH on a capturable stream) as a replay of the captured cycle.
static int spec_step_run(gm_ctx *c, gm_state *st, int k, float temperature, const uint32_t *u24_draft,
                         const uint32_t *u24_accept, uint64_t seed, uint64_t step, int32_t *accept_len,
                         int32_t *next_token, int32_t *draft_tok) {
  if (!c || !graph_capable(c) || c->prof_mask != 0)          // per-launch timing needs host-launched kernels
    return spec_step_impl(c, st, k, temperature, u24_draft, u24_accept, seed, step, accept_len, next_token, draft_tok);
  int rc = check_state(c, st, k);
  if (rc) return rc;
  if (!accept_len || !next_token) return GM_ERR_INVALID_ARG;
  KeyBytes key;
  key.add(*st); key.add(k); key.add(temperature); key.add(u24_draft); key.add(u24_accept); key.add(seed);
  key.add(accept_len); key.add(next_token); key.add(draft_tok); key.add(c->top_p);
  key.add(c->capture); key.add(c->capture_stride);
  rc = graph_prepare(c, c->graph_step, key.bytes, [&]() {
    return spec_step_impl(c, st, k, temperature, u24_draft, u24_accept, seed, 0, accept_len, next_token, draft_tok);
  });
  if (rc) return rc;
  GM_LAUNCH(c, GM_KC_ELEMENTWISE, launch_set_step(c->dev_step, step, c->stream));
  GM_CUDA(c, cudaGraphLaunch(c->graph_step.exec, c->stream));
  c->launches += c->graph_step.launches;
  return GM_OK;
}

}  // extern "C"

int gmh::spec_step_impl(gm_ctx *c, gm_state *st, int k, float temperature, const uint32_t *u24_draft,
                        const uint32_t *u24_accept, uint64_t seed, uint64_t step, int32_t *accept_len,
                        int32_t *next_token, int32_t *draft_tok) {
  int rc = check_state(c, st, k);
  if (rc) return rc;
  if (!accept_len || !next_token) return GM_ERR_INVALID_ARG;
  int32_t *dt = draft_tok ? draft_tok : c->ws_draft_tok;
  if ((rc = gm_draft(c, st, k, temperature, u24_draft, seed, step, dt, c->ws_draft_logits, nullptr)) != GM_OK) return rc;
  if ((rc = gm_verify(c, st, k, dt, c->ws_target_logits, c->ws_target_hidden)) != GM_OK) return rc;
  return gm_accept(c, st, st->batch, k, temperature, c->ws_target_logits, c->ws_draft_logits, dt, u24_accept, seed, step,
                   accept_len, next_token, nullptr, nullptr, c->ws_target_hidden, 1);
}

extern "C" {

int gm_spec_step(gm_ctx *c, gm_state *st, int k, float temperature, uint64_t seed, uint64_t step, int32_t *accept_len,
                 int32_t *next_token, int32_t *draft_tok) {
  return spec_step_run(c, st, k, temperature, nullptr, nullptr, seed, step, accept_len, next_token, draft_tok);
}

int gm_spec_step_host(gm_ctx *c, gm_state *st, int k, float temperature, uint64_t seed, uint64_t step,
                      const uint32_t *u24_draft_host, const uint32_t *u24_accept_host, int32_t *accept_len_host,
                      int32_t *next_token_host, int32_t *draft_tok_host) {
  int rc = check_state(c, st, k);
  if (rc) return rc;
  if (!accept_len_host || !next_token_host) return GM_ERR_INVALID_ARG;
  if ((u24_draft_host == nullptr) != (u24_accept_host == nullptr)) return GM_ERR_INVALID_ARG;
  const size_t B = static_cast<size_t>(st->batch);
  uint32_t *ud = nullptr, *ua = nullptr;
  if (u24_draft_host) {
    ud = c->ws_u24;
    ua = c->ws_u24 + B * k;
    GM_CUDA(c, cudaMemcpyAsync(ud, u24_draft_host, B * k * sizeof(uint32_t), cudaMemcpyHostToDevice, c->stream));
    GM_CUDA(c, cudaMemcpyAsync(ua, u24_accept_host, B * (k + 1) * sizeof(uint32_t), cudaMemcpyHostToDevice, c->stream));
  }
  rc = spec_step_run(c, st, k, temperature, ud, ua, seed, step, c->ws_accept_len, c->ws_next_token, c->ws_draft_tok);
  if (rc) return rc;
  GM_CUDA(c, cudaMemcpyAsync(accept_len_host, c->ws_accept_len, B * sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream));
  GM_CUDA(c, cudaMemcpyAsync(next_token_host, c->ws_next_token, B * sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream));
  if (draft_tok_host)
    GM_CUDA(c, cudaMemcpyAsync(draft_tok_host, c->ws_draft_tok, B * k * sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream));
  GM_CUDA(c, cudaStreamSynchronize(c->stream));
  return GM_OK;
}

int gm_profile(gm_ctx *c, int class_mask) {
  if (!c) return GM_ERR_INVALID_ARG;
  GM_CUDA(c, cudaStreamSynchronize(c->stream));
  c->prof_mask = class_mask;
  for (int i = 0; i < GM_KC_COUNT; ++i) c->events_used[i] = 0;
  return GM_OK;
}

int gm_profile_read(gm_ctx *c, int kernel_class, double *total_ms, int64_t *launches) {
  if (!c || kernel_class < 0 || kernel_class >= GM_KC_COUNT || !total_ms || !launches) return GM_ERR_INVALID_ARG;
  GM_CUDA(c, cudaStreamSynchronize(c->stream));
  double t = 0;
  for (size_t i = 0; i < c->events_used[kernel_class]; ++i) {
    float ms = 0.f;
    GM_CUDA(c, cudaEventElapsedTime(&ms, c->events[kernel_class][i].a, c->events[kernel_class][i].b));
    t += ms;
  }
  *total_ms = t;
  *launches = static_cast<int64_t>(c->events_used[kernel_class]);
  return GM_OK;
}

int64_t gm_launch_count(gm_ctx *c) { return c ? c->launches : 0; }

int gm_last_status(gm_ctx *c) {
  if (!c) return GM_ERR_INVALID_ARG;
  uint32_t s = 0;
  GM_CUDA(c, cudaStreamSynchronize(c->stream));
  GM_CUDA(c, cudaMemcpy(&s, c->status, sizeof(s), cudaMemcpyDeviceToHost));
  GM_CUDA(c, cudaMemset(c->status, 0, sizeof(s)));
  if (s & ST_TIMEOUT) {                 // a chain launch that gave up may have left its barrier words mid-count
    if (c->flow_ws) GM_CUDA(c, cudaMemset(c->flow_ws, 0, c->flow_ws_bytes));      // likewise the sampler's work queue
    if (c->chain_sync) GM_CUDA(c, cudaMemset(c->chain_sync, 0, (1 + static_cast<size_t>(c->chain_pairs) * 2) * sizeof(unsigned long long)));
    return GM_ERR_DEVICE_TIMEOUT;
  }
  if (s & ST_KV_CAPACITY) return GM_ERR_KV_CAPACITY;
  if (s & (ST_BAD_PAGE | ST_BAD_TOKEN)) return GM_ERR_BAD_PAGE;
  if (c->check_guards) {
    unsigned char host[GM_GUARD_BYTES];
    for (unsigned char *g : c->guards) {
      GM_CUDA(c, cudaMemcpy(host, g, GM_GUARD_BYTES, cudaMemcpyDeviceToHost));
      for (size_t i = 0; i < GM_GUARD_BYTES; ++i)
        if (host[i] != GM_GUARD_PATTERN) return GM_ERR_OVERRUN;
    }
  }
  return GM_OK;
}

}  // extern "C"
