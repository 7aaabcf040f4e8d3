// Forward pass of the draft-head update on recorded cycles (Sec. 3.2 Eq. 4; Sec. 3.3-3.4 Eq. 5-9; App. D.2-D.3).
//
// Draft-path reconstruction replays every recorded chain through the draft phase's own kernels: a chain is a virtual
// sequence whose page-table row shares the pages of its sequence's prefilled head cache up to the page that holds its
// first entry, and owns two private pages from there on (the first one starts as a copy of the shared page).  That is
// the visibility the paper's batched forward gets from its mask - causal over the committed prefix, diagonal over
// the draft entries - expressed in the page table instead of in an additive mask.  The kernels here are the
// bookkeeping around that replay, the overlap alpha_k from the top-64 record, and the objective.
#include "common.cuh"
#include "kernels.h"

namespace gm {
namespace {

__device__ __forceinline__ float bf16_to_float(__nv_bfloat16 v) { return __bfloat162float(v); }

// One CTA per chain of the chunk.
__global__ void __launch_bounds__(128) chain_setup_kernel(const ChainSetupArgs A) {
  const int c = blockIdx.x, tid = threadIdx.x;
  pdl_prologue();
  int seq = A.cycle_seq[c], len = A.start_pos[c];
  const int p0 = A.scratch_pages[2 * c], p1 = A.scratch_pages[2 * c + 1];
  bool ok = seq >= 0 && seq < A.n_seq && len >= 2 && len + A.k - 1 <= A.max_pages_per_seq * 16 && p0 >= 0 &&
            p0 < A.num_pages && p1 >= 0 && p1 < A.num_pages && p0 != p1;
  if (!ok) {                                   // reported; the chain then runs on harmless stand-in values
    if (tid == 0) set_status(A.status, ST_BAD_PAGE);
    seq = 0; len = 2;
  }
  const int pb = (len - 2) >> 4;               // page of the chain's first entry (head position len - 2)
  const int32_t *src_row = A.head_page_table + static_cast<size_t>(seq) * A.max_pages_per_seq;
  int32_t *dst_row = A.v_table + static_cast<size_t>(c) * A.max_pages_per_seq;
  for (int i = tid; i < A.max_pages_per_seq; i += blockDim.x)
    dst_row[i] = i < pb ? src_row[i] : (i == pb ? (ok ? p0 : 0) : (i == pb + 1 ? (ok ? p1 : 0) : 0));
  if (tid == 0) {
    A.v_kv_len[c] = len - 1;
    A.v_pending_n[c] = 1;
    int tok = A.seq_tok[static_cast<size_t>(seq) * A.tok_stride + len - 1];
    if (tok < 0 || tok >= A.vocab) { set_status(A.status, ST_BAD_TOKEN); tok = 0; }
    A.v_pending_tok[static_cast<size_t>(c) * A.pend_stride] = tok;
  }
  const uint4 *hs = reinterpret_cast<const uint4 *>(A.start_hidden + static_cast<size_t>(c) * A.d);
  uint4 *hd = reinterpret_cast<uint4 *>(A.v_pending_hidden + static_cast<size_t>(c) * A.pend_stride * A.d);
  for (int i = tid; i < A.d / 8; i += blockDim.x) hd[i] = hs[i];
  // private copy of the shared boundary page (keys and values)
  const int orig = src_row[pb];
  if (ok && orig >= 0 && orig < A.num_pages) {
    const size_t page_vec = static_cast<size_t>(A.page_elems) / 8;
    for (int plane = 0; plane < 2; ++plane) {
      const uint4 *s = reinterpret_cast<const uint4 *>(A.pool) + (static_cast<size_t>(plane) * A.num_pages + orig) * page_vec;
      uint4 *d = reinterpret_cast<uint4 *>(A.pool) + (static_cast<size_t>(plane) * A.num_pages + p0) * page_vec;
      for (size_t i = tid; i < page_vec; i += blockDim.x) d[i] = s[i];
    }
  } else if (ok && tid == 0) {
    set_status(A.status, ST_BAD_PAGE);
  }
}

__global__ void __launch_bounds__(128)
gather_chunk_hidden_kernel(const __nv_bfloat16 *seq_hidden, int hid_stride, const int32_t *row_base, int vr, int QT, int d,
                           const int32_t *row_n, __nv_bfloat16 *out) {
  const int m = blockIdx.x, v = m / QT, j = m % QT;
  pdl_prologue();
  if (j >= row_n[v]) return;
  const uint4 *s = reinterpret_cast<const uint4 *>(seq_hidden + (static_cast<size_t>(v / vr) * hid_stride + row_base[v] + j) * d);
  uint4 *o = reinterpret_cast<uint4 *>(out + static_cast<size_t>(m) * d);
  for (int i = threadIdx.x; i < d / 8; i += blockDim.x) o[i] = s[i];
}

// Softmax statistics of one row in a single pass: running maximum with the sum rescaled when it moves.  Returns
// logsumexp(x / T) to every thread of the CTA.  NT threads, NT / 32 <= 32.
template <int NT>
__device__ __forceinline__ float row_lse(const uint4 *xv, int nvec, float inv_temp, float *red_m, float *red_z, float *out) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float m = -INFINITY, z = 0.f;
  auto take = [&](const uint4 &v) {
    const uint32_t wds[4] = {v.x, v.y, v.z, v.w};
    const float cm = fmaxf(fmaxf(fmaxf(bf16_lo(v.x), bf16_hi(v.x)), fmaxf(bf16_lo(v.y), bf16_hi(v.y))),
                           fmaxf(fmaxf(bf16_lo(v.z), bf16_hi(v.z)), fmaxf(bf16_lo(v.w), bf16_hi(v.w))));
    if (cm > m) { z *= __expf((m - cm) * inv_temp); m = cm; }
#pragma unroll
    for (int t = 0; t < 4; ++t) z += __expf((bf16_lo(wds[t]) - m) * inv_temp) + __expf((bf16_hi(wds[t]) - m) * inv_temp);
  };
  int i = tid;
  for (; i + 3 * NT < nvec; i += 4 * NT) {                // four loads in flight per thread
    const uint4 v0 = xv[i], v1 = xv[i + NT], v2 = xv[i + 2 * NT], v3 = xv[i + 3 * NT];
    take(v0); take(v1); take(v2); take(v3);
  }
  for (; i < nvec; i += NT) take(xv[i]);
  for (int o = 16; o; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o), z2 = __shfl_xor_sync(0xffffffffu, z, o);
    const float mn = fmaxf(m, m2);
    z = (m == -INFINITY ? 0.f : z * __expf((m - mn) * inv_temp)) + (m2 == -INFINITY ? 0.f : z2 * __expf((m2 - mn) * inv_temp));
    m = mn;
  }
  if (lane == 0) { red_m[warp] = m; red_z[warp] = z; }
  __syncthreads();
  if (tid == 0) {
    float mm = red_m[0];
    for (int w = 1; w < NT / 32; ++w) mm = fmaxf(mm, red_m[w]);
    float t = 0.f;
    for (int w = 0; w < NT / 32; ++w)
      if (red_m[w] != -INFINITY) t += red_z[w] * __expf((red_m[w] - mm) * inv_temp);
    *out = mm * inv_temp + logf(t);
  }
  __syncthreads();
  return *out;
}

// alpha = sum_i min(p_i, q_i) + min(1 - sum p_i, 1 - sum q_i) over the record's retained entries; one CTA per row.
constexpr int OV_THREADS = 512;
__global__ void __launch_bounds__(OV_THREADS) overlap_kernel(const OverlapArgs A) {
  __shared__ float red_m[OV_THREADS / 32], red_z[OV_THREADS / 32];
  __shared__ float sh_lse;
  const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const __nv_bfloat16 *x = A.logits + static_cast<size_t>(row) * A.V;
  pdl_prologue();
  row_lse<OV_THREADS>(reinterpret_cast<const uint4 *>(x), A.V >> 3, A.inv_temp, red_m, red_z, &sh_lse);
  if (tid == 0 && A.lse) A.lse[row] = sh_lse;
  if (warp < 2) {                                          // 64 retained entries: two warps
    const int e = tid;
    const int idx = A.top_index[static_cast<size_t>(row) * 64 + e];
    float p = 0.f, q = 0.f;
    if (idx >= 0 && idx < A.V) {
      p = expf(bf16_to_float(A.top_logprob[static_cast<size_t>(row) * 64 + e]));
      q = expf(bf16_to_float(x[idx]) * A.inv_temp - sh_lse);
    }
    float mn = fminf(p, q), ps = p, qs = q;
    for (int o = 16; o; o >>= 1) {
      mn += __shfl_xor_sync(0xffffffffu, mn, o);
      ps += __shfl_xor_sync(0xffffffffu, ps, o);
      qs += __shfl_xor_sync(0xffffffffu, qs, o);
    }
    __shared__ float part[2][3];
    if (lane == 0) { part[warp][0] = mn; part[warp][1] = ps; part[warp][2] = qs; }
    asm volatile("bar.sync 1, 64;" ::: "memory");
    if (tid == 0) {
      const float mins = part[0][0] + part[1][0], psum = part[0][1] + part[1][1], qsum = part[0][2] + part[1][2];
      A.alpha[row] = mins + fminf(fmaxf(1.f - psum, 0.f), fmaxf(1.f - qsum, 0.f));
    }
  }
}

// Gradient of the mean objective with respect to the reconstructed head logits (first step of the backward pass).
// Row (cycle c, position k): dL/dalpha = -(prod_{i<k} alpha_i) D_k / M with the chain sums cut at L = min(j, K)
// (Eq. 8 with the gate of Eq. 9), 0 for k >= L and for a dead chain (M = 0).  alpha is piecewise linear in q: slope
// g_e = 1[q_e < p_e] - 1[q_res < p_res] on the retained tokens, 0 elsewhere (ties: slope 0);
// dalpha/dlogit_v = q_v (g_v - G) / T with G = sum_e q_e g_e.  One CTA per row: one pass for the softmax statistics
// (running maximum and rescaled sum), the 64 retained entries, then one pass that writes the whole row.
constexpr int DG_THREADS = 512;
__global__ void __launch_bounds__(DG_THREADS) dca_grad_kernel(const DcaGradArgs A) {
  __shared__ float red_m[DG_THREADS / 32], red_z[DG_THREADS / 32];
  __shared__ float sh_lse, sh_G;
  __shared__ float part[2][3];
  __shared__ int sh_res;
  const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int c = row / A.K, kk = row % A.K;
  const __nv_bfloat16 *x = A.logits + static_cast<size_t>(row) * A.V;
  const uint4 *xv = reinterpret_cast<const uint4 *>(x);
  uint4 *ov = reinterpret_cast<uint4 *>(A.grad + static_cast<size_t>(row) * A.V);
  const int nvec = A.V >> 3;
  pdl_prologue();
  float coef = 0.f;
  {
    const int L = min(max(A.accepted[c], 1), A.K);
    if (kk < L) {
      float a[GM_MAX_K_];
      for (int i = 0; i < L; ++i) a[i] = A.alpha[static_cast<size_t>(c) * A.K + i];
      float M = 0.f, run = 1.f, pre = 1.f;
      for (int l = 0; l < L; ++l) { if (l == kk) pre = run; run *= a[l]; M += run; }
      float D = 0.f, t = 1.f;
      for (int l = kk; l < L; ++l) { if (l > kk) t *= a[l]; D += t; }
      if (M > 0.f) coef = -(pre * D / M) / static_cast<float>(A.n_total > 0 ? A.n_total : A.n);
    }
  }
  if (coef == 0.f) {
    for (int i = tid; i < nvec; i += DG_THREADS) ov[i] = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  float lse;
  if (A.lse) lse = A.lse[row];
  else lse = row_lse<DG_THREADS>(xv, nvec, A.inv_temp, red_m, red_z, &sh_lse);
  int idx = -1;
  float qe = 0.f, ge = 0.f;
  if (warp < 2) {                                          // the 64 retained entries: two warps
    idx = A.top_index[static_cast<size_t>(row) * 64 + tid];
    float p = 0.f;
    if (idx >= 0 && idx < A.V) {
      p = expf(bf16_to_float(A.top_logprob[static_cast<size_t>(row) * 64 + tid]));
      qe = expf(bf16_to_float(x[idx]) * A.inv_temp - lse);
    } else {
      idx = -1;
    }
    ge = (idx >= 0 && qe < p) ? 1.f : 0.f;
    float ps = p, qs = qe, gq = qe * ge;
    for (int o = 16; o; o >>= 1) {
      ps += __shfl_xor_sync(0xffffffffu, ps, o);
      qs += __shfl_xor_sync(0xffffffffu, qs, o);
      gq += __shfl_xor_sync(0xffffffffu, gq, o);
    }
    if (lane == 0) { part[warp][0] = ps; part[warp][1] = qs; part[warp][2] = gq; }
  }
  __syncthreads();
  if (tid == 0) {
    const float psum = part[0][0] + part[1][0], qsum = part[0][1] + part[1][1];
    const int res = fmaxf(1.f - qsum, 0.f) < fmaxf(1.f - psum, 0.f);
    sh_res = res;
    sh_G = part[0][2] + part[1][2] - (res ? qsum : 0.f);
  }
  __syncthreads();
  const float G = sh_G, scale = coef * A.inv_temp;
  const float base = -G * scale;                           // every token outside the retained set: q_v * base
  for (int i = tid; i < nvec; i += DG_THREADS) {
    const uint4 v = xv[i];
    const uint32_t wds[4] = {v.x, v.y, v.z, v.w};
    uint32_t o4[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const float q0 = __expf(bf16_lo(wds[t]) * A.inv_temp - lse), q1 = __expf(bf16_hi(wds[t]) * A.inv_temp - lse);
      o4[t] = pack_bf16(q0 * base, q1 * base);
    }
    ov[i] = make_uint4(o4[0], o4[1], o4[2], o4[3]);
  }
  __syncthreads();                                         // the retained entries are rewritten after the row pass
  if (warp < 2 && idx >= 0) {
    if (sh_res) ge -= 1.f;
    A.grad[static_cast<size_t>(row) * A.V + idx] = __float2bfloat16_rn(qe * (ge - G) * scale);
  }
}

// Per cycle: L = -log sum_{l=1..min(j,K)} prod_{i<=l} alpha_i (Eq. 9), in the log domain (Eq. 7); then the mean over
// cycles, added in a fixed order (one CTA).
constexpr int DL_THREADS = 1024;
__global__ void __launch_bounds__(DL_THREADS) dca_loss_kernel(const float *alpha, const int32_t *accepted, int n, int K,
                                                               float *loss, float *mean) {
  __shared__ double red[DL_THREADS];
  pdl_prologue();
  double acc = 0.0;
  for (int c = threadIdx.x; c < n; c += DL_THREADS) {
    const int L = min(max(accepted[c], 1), K);
    float s = 0.f, mx = -INFINITY, terms[GM_MAX_K_];
    for (int l = 0; l < L; ++l) {
      s += logf(alpha[static_cast<size_t>(c) * K + l]);    // log 0 = -inf: the chain is dead from here on
      terms[l] = s;
      mx = fmaxf(mx, s);
    }
    float v;
    if (mx == -INFINITY) {
      v = INFINITY;
    } else {
      float t = 0.f;
      for (int l = 0; l < L; ++l) t += expf(terms[l] - mx);
      v = -(mx + logf(t));
    }
    loss[c] = v;
    acc += static_cast<double>(v);
  }
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int o = DL_THREADS / 2; o; o >>= 1) {
    if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) *mean = static_cast<float>(red[0] / static_cast<double>(n));
}

__global__ void __launch_bounds__(128)
capture_chunk_kernel(const __nv_bfloat16 *src, const int32_t *row_n, const int32_t *row_base, int vr, int QT, int d,
                     __nv_bfloat16 *dst, int dst_stride) {
  const int m = blockIdx.x, v = m / QT, j = m % QT;
  pdl_prologue();
  if (j >= row_n[v] || row_base[v] + j >= dst_stride) return;
  const uint4 *s = reinterpret_cast<const uint4 *>(src + static_cast<size_t>(m) * d);
  uint4 *o = reinterpret_cast<uint4 *>(dst + (static_cast<size_t>(v / vr) * dst_stride + row_base[v] + j) * d);
  for (int i = threadIdx.x; i < d / 8; i += blockDim.x) o[i] = s[i];
}
__global__ void __launch_bounds__(128)
capture_cycle_kernel(const __nv_bfloat16 *src, const int32_t *accept_len, const int32_t *kv_len, const int32_t *finished,
                     int k, int d, __nv_bfloat16 *dst, int dst_stride) {
  const int b = blockIdx.x / (k + 1), l = blockIdx.x % (k + 1);
  pdl_prologue();
  if (finished && finished[b]) return;
  const int a = accept_len[b];
  const int pos = kv_len[b] - (a + 1) + l;
  if (l > a || pos < 0 || pos >= dst_stride) return;
  const uint4 *s = reinterpret_cast<const uint4 *>(src + static_cast<size_t>(blockIdx.x) * d);
  uint4 *o = reinterpret_cast<uint4 *>(dst + (static_cast<size_t>(b) * dst_stride + pos) * d);
  for (int i = threadIdx.x; i < d / 8; i += blockDim.x) o[i] = s[i];
}

// ---- backward through the head's final norm (Alg. 1, "update phi"; the norm of App. B.1) -----------------------------------
// y = x r w with r = (mean(x^2) + eps)^(-1/2):  dL/dx = r (w gy) - x r^3 mean(x w gy).  One CTA per row, fp32.
constexpr int NG_THREADS = 256;
__global__ void __launch_bounds__(NG_THREADS)
rmsnorm_grad_kernel(const float *gy, const float *x, const __nv_bfloat16 *w, float *gx, int d, float eps, const float *res,
                    float *wterm, int gy_ld) {
  __shared__ float red[2][NG_THREADS / 32];
  const size_t row = static_cast<size_t>(blockIdx.x) * d;
  gy += static_cast<size_t>(blockIdx.x) * gy_ld - row;        // gy rows may be wider than d (a column block of a larger matrix)
  const int tid = threadIdx.x, lane = tid & 31, wp = tid >> 5;
  pdl_prologue();
  float sq = 0.f, dot = 0.f;
  for (int i = tid; i < d; i += NG_THREADS) {
    const float xv = x[row + i];
    sq = fmaf(xv, xv, sq);
    dot = fmaf(xv, bf16_to_float(w[i]) * gy[row + i], dot);
  }
  sq = warp_sum(sq); dot = warp_sum(dot);
  if (lane == 0) { red[0][wp] = sq; red[1][wp] = dot; }
  __syncthreads();
  sq = 0.f; dot = 0.f;
#pragma unroll
  for (int i = 0; i < NG_THREADS / 32; ++i) { sq += red[0][i]; dot += red[1][i]; }   // same order in every thread
  const float inv_d = 1.0f / static_cast<float>(d);
  const float r = rsqrtf(sq * inv_d + eps);
  const float c = r * r * r * dot * inv_d;
  for (int i = tid; i < d; i += NG_THREADS) {
    const float g = gy[row + i], xv = x[row + i];
    if (gx) gx[row + i] = (res ? res[row + i] : 0.f) + (r * bf16_to_float(w[i]) * g - xv * c);     // res: the residual path's gradient
    if (wterm) wterm[row + i] = g * xv * r;                    // this row's term of dL/dw (summed over the rows afterwards)
  }
}

// out[j] (+)= sum over the rows of t[row][j] (fp32), in a fixed order whatever the launch: a CTA sums 32 columns of one
// chunk of rows - 32 row lanes striding the chunk, then the lanes in order - and, when the rows were split into several
// chunks, a second kernel adds the chunks' partial sums in chunk order.
constexpr int CS_COLS = 32, CS_LANES = 32, CS_MAX_CHUNKS = 64;
__global__ void __launch_bounds__(CS_COLS * CS_LANES)
colsum_kernel(const float *t, int rows, int d, int chunk_rows, float *out, int add) {
  __shared__ float red[CS_LANES][CS_COLS + 1];
  const int col = blockIdx.x * CS_COLS + threadIdx.x, ty = threadIdx.y;
  const int r0 = blockIdx.y * chunk_rows, r1 = min(rows, r0 + chunk_rows);
  pdl_prologue();
  float acc = 0.f;
  if (col < d)
    for (int r = r0 + ty; r < r1; r += CS_LANES) acc += t[static_cast<size_t>(r) * d + col];
  red[ty][threadIdx.x] = acc;
  __syncthreads();
  if (ty == 0 && col < d) {
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < CS_LANES; ++i) sum += red[i][threadIdx.x];
    float *dst = out + static_cast<size_t>(blockIdx.y) * d + col;       // gridDim.y > 1: out is the partial-sum scratch
    *dst = (add && gridDim.y == 1) ? *dst + sum : sum;
  }
}
__global__ void __launch_bounds__(256) colsum_finish_kernel(const float *part, int chunks, int d, float *out, int add) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  pdl_prologue();
  if (j >= d) return;
  float acc = 0.f;
  for (int c = 0; c < chunks; ++c) acc += part[static_cast<size_t>(c) * d + j];
  out[j] = add ? out[j] + acc : acc;
}

// ---- bookkeeping of the backward pass over a reconstruction (Alg. 1, "update phi"; Eq. 4) ---------------------------------------
// Rows of draft application k (from 1) of every chain: the (hidden, token) pair that entered, the gradient of the state
// it produced, and its position.  One CTA per chain.
__global__ void __launch_bounds__(128) step_rows_kernel(const StepRowsArgs A) {
  const int c = blockIdx.x;
  pdl_prologue();
  const int k = A.k;
  if (threadIdx.x == 0) {
    int tok = k == 1 ? A.first_tok[static_cast<size_t>(c) * A.first_tok_stride] : A.drafts[static_cast<size_t>(c) * A.K + k - 2];
    if (tok < 0 || tok >= A.vocab) { set_status(A.status, ST_BAD_TOKEN); tok = 0; }
    A.tok[c] = tok;
    A.base[c] = A.start_pos[c] + k - 3;
    A.count[c] = 1;
  }
  const size_t row = static_cast<size_t>(c) * A.d;
  for (int i = threadIdx.x; i < A.d; i += blockDim.x) {
    A.hidden[row + i] = k == 1 ? bf16_to_float(A.start_hidden[row + i]) : A.states[(static_cast<size_t>(c) * A.K + k - 2) * A.d + i];
    A.dg[row + i] = A.dstate[(static_cast<size_t>(c) * A.K + k - 1) * A.d + i];
  }
}
// dstate[c][k] += dhidden[c]: the recurrence's term of the previous state's gradient (Eq. 4)
__global__ void __launch_bounds__(128) add_state_grad_kernel(float *dstate, const float *dhidden, int K, int k, int d) {
  const int c = blockIdx.x;
  pdl_prologue();
  for (int i = threadIdx.x; i < d; i += blockDim.x) dstate[(static_cast<size_t>(c) * K + k) * d + i] += dhidden[static_cast<size_t>(c) * d + i];
}
// A chain's private boundary page started as a copy of its sequence's shared page: what the chain's rows left on the
// copied entries (positions before the chain's first) belongs to the originals.  One CTA per chain, both planes.
__global__ void __launch_bounds__(128) fold_boundary_kernel(const FoldArgs A) {
  const int c = blockIdx.x;
  pdl_prologue();
  const int seq = A.cycle_seq[c], len = A.start_pos[c];
  if (seq < 0 || seq >= A.n_seq || len < 2) return;
  const int pb = (len - 2) >> 4, slots = (len - 2) & 15;
  const int orig = A.head_page_table[static_cast<size_t>(seq) * A.max_pages_per_seq + pb], p0 = A.scratch_pages[2 * c];
  if (orig < 0 || orig >= A.num_pages || p0 < 0 || p0 >= A.num_pages || orig == p0) return;
  const int per_head = 16 * A.hd;
  for (int i = threadIdx.x; i < A.n_kv * slots * A.hd; i += blockDim.x) {
    const int h = i / (slots * A.hd), r = i % (slots * A.hd);
    const size_t o = (static_cast<size_t>(orig) * A.n_kv + h) * per_head + r, s = (static_cast<size_t>(p0) * A.n_kv + h) * per_head + r;
    if (A.dk_fix) {                                     // integer additions: the same sum in any order
      const long long a = A.dk_fix[s], b = A.dv_fix[s];
      if (a) atomicAdd(reinterpret_cast<unsigned long long *>(A.dk_fix + o), static_cast<unsigned long long>(a));
      if (b) atomicAdd(reinterpret_cast<unsigned long long *>(A.dv_fix + o), static_cast<unsigned long long>(b));
      continue;
    }
    const float a = A.dk_pool[s], b = A.dv_pool[s];
    if (a != 0.f) atomicAdd(A.dk_pool + o, a);
    if (b != 0.f) atomicAdd(A.dv_pool + o, b);
  }
}
__global__ void __launch_bounds__(256) fix_to_float_kernel(const long long *src, float *dst, size_t n) {
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  pdl_prologue();
  for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += stride) dst[i] = fix_get(src + i);
}
__global__ void __launch_bounds__(256) widen_bf16_kernel(const __nv_bfloat16 *src, float *dst, size_t n) {
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  pdl_prologue();
  for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += stride) dst[i] = bf16_to_float(src[i]);
}
// fp32 copy of bf16 rows; row m = v * QT + j is zero when j >= row_n[v]
__global__ void __launch_bounds__(128) rows_to_f32_kernel(const __nv_bfloat16 *src, const int32_t *row_n, int QT, int d, float *dst) {
  const int m = blockIdx.x, v = m / QT, j = m % QT;
  pdl_prologue();
  const bool live = j < row_n[v];
  for (int i = threadIdx.x; i < d; i += blockDim.x)
    dst[static_cast<size_t>(m) * d + i] = live ? bf16_to_float(src[static_cast<size_t>(m) * d + i]) : 0.f;
}

// fp32 -> bf16, n elements (n % 4 == 0)
__global__ void __launch_bounds__(256) cast_bf16_kernel(const float *src, __nv_bfloat16 *dst, size_t n4) {
  const size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  pdl_prologue();
  if (i >= n4) return;
  const float4 v = reinterpret_cast<const float4 *>(src)[i];
  reinterpret_cast<uint2 *>(dst)[i] = make_uint2(pack_bf16(v.x, v.y), pack_bf16(v.z, v.w));
}

// Backward of the SwiGLU activation h = silu(a) * b on interleaved rows (a_f at column 2f, b_f at 2f + 1):
//   dab[2f] = dh_f b_f sig (1 + a_f (1 - sig)),  dab[2f + 1] = dh_f silu(a_f),  h_f recomputed for the down projection's
//   weight gradient.  One thread per (row, f) pair.
__global__ void __launch_bounds__(256)
swiglu_grad_kernel(const __nv_bfloat16 *ab, const float *dh, __nv_bfloat16 *dab, __nv_bfloat16 *h, size_t n, int F) {
  const size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  pdl_prologue();
  if (i >= n) return;
  const uint32_t w = reinterpret_cast<const uint32_t *>(ab)[i];
  const float a = bf16_lo(w), b = bf16_hi(w), g = dh[i];
  const float sig = 1.0f / (1.0f + __expf(-a)), act = a * sig;
  reinterpret_cast<uint32_t *>(dab)[i] = pack_bf16(g * b * sig * (1.0f + a * (1.0f - sig)), g * act);
  h[i] = __float2bfloat16(act * b);
  }

// ---- between the QKV projection and the attention core, backward (App. B.1) -------------------------------------------------
// One CTA per token row, a warp per head.  Lane l holds elements l*EH .. l*EH + EH - 1 of the head's first half and their
// rotation partners in the second half (EH = hd / 64).
template <int EH>
__global__ void __launch_bounds__(256) qkv_grad_rows_kernel(const QkvGradArgs A) {
  constexpr int HD = 64 * EH, HALF = 32 * EH;
  const int m = blockIdx.x, b = m / A.QT, j = m % A.QT;
  const int lane = threadIdx.x & 31, wp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const int ncols = (A.n_q + 2 * A.n_kv) * HD;
  pdl_prologue();
  const int qn = A.qn[b], pos = A.qbase[b] + j;
  float *out = A.dqkv + static_cast<size_t>(m) * ncols;
  __nv_bfloat16 *outb = A.dqkv_bf + static_cast<size_t>(m) * ncols;
  int page = -1;
  if (j < qn) {
    page = A.page_table[static_cast<size_t>(b) * A.max_pages_per_seq + (pos >> 4)];
    if (page < 0 || page >= A.num_pages) { if (threadIdx.x == 0) set_status(A.status, ST_BAD_PAGE); page = -1; }
  }
  const size_t page_elems = static_cast<size_t>(A.n_kv) * 16 * HD;
  for (int h = wp; h < A.n_q + 2 * A.n_kv; h += nw) {
    const bool is_q = h < A.n_q, is_k = !is_q && h < A.n_q + A.n_kv;
    const int kvh = is_q ? 0 : (is_k ? h - A.n_q : h - A.n_q - A.n_kv);
    float *tn = is_q ? (A.tq ? A.tq + (static_cast<size_t>(m) * A.n_q + h) * HD : nullptr)
                     : (is_k && A.tk ? A.tk + (static_cast<size_t>(m) * A.n_kv + kvh) * HD : nullptr);
    float g1[EH], g2[EH];
    if (page < 0) {                                    // padding row (or a page outside the pool): no gradient
#pragma unroll
      for (int t = 0; t < EH; ++t) {
        const int i = lane * EH + t;
        out[h * HD + i] = 0.f; out[h * HD + HALF + i] = 0.f;
        outb[h * HD + i] = __float2bfloat16(0.f); outb[h * HD + HALF + i] = __float2bfloat16(0.f);
        if (tn) { tn[i] = 0.f; tn[HALF + i] = 0.f; }
      }
      continue;
    }
    const size_t so = is_q ? (static_cast<size_t>(m) * A.n_q + h) * HD
                           : static_cast<size_t>(page) * page_elems + (static_cast<size_t>(kvh) * 16 + (pos & 15)) * HD;
    if (A.dk_fix) {
      const long long *src = (is_q ? A.dq_fix : (is_k ? A.dk_fix : A.dv_fix)) + so;
#pragma unroll
      for (int t = 0; t < EH; ++t) { g1[t] = fix_get(src + lane * EH + t); g2[t] = fix_get(src + HALF + lane * EH + t); }
    } else {
      const float *src = (is_q ? A.dq : (is_k ? A.dk_pool : A.dv_pool)) + so;
#pragma unroll
      for (int t = 0; t < EH; ++t) { g1[t] = src[lane * EH + t]; g2[t] = src[HALF + lane * EH + t]; }
    }
    if (is_q || is_k) {
      // the rotation's transpose: turn back by the position's angle
      const float2 *cs = A.rope + static_cast<size_t>(pos) * HALF;
#pragma unroll
      for (int t = 0; t < EH; ++t) {
        const float2 c = cs[lane * EH + t];
        const float y1 = g1[t], y2 = g2[t];
        g1[t] = y1 * c.x + y2 * c.y;
        g2[t] = y2 * c.x - y1 * c.y;
      }
      const __nv_bfloat16 *wn = is_q ? A.qnorm : A.knorm;
      if (wn) {                                        // y = x0 r w over the head: dx0 = r (w g) - x0 r^3 mean(x0 w g)
        float x1[EH], x2[EH], w1[EH], w2[EH];
        float ss = 0.f, dot = 0.f;
#pragma unroll
        for (int t = 0; t < EH; ++t) {
          const int i = lane * EH + t;
          x1[t] = bf16_to_float(A.qkv[static_cast<size_t>(m) * ncols + h * HD + i]);
          x2[t] = bf16_to_float(A.qkv[static_cast<size_t>(m) * ncols + h * HD + HALF + i]);
          if (A.bias) { x1[t] += bf16_to_float(A.bias[h * HD + i]); x2[t] += bf16_to_float(A.bias[h * HD + HALF + i]); }
          w1[t] = bf16_to_float(wn[i]); w2[t] = bf16_to_float(wn[HALF + i]);
          ss += x1[t] * x1[t] + x2[t] * x2[t];
          dot += x1[t] * w1[t] * g1[t] + x2[t] * w2[t] * g2[t];
        }
        ss = warp_sum(ss); dot = warp_sum(dot);
        const float r = rsqrtf(ss / static_cast<float>(HD) + A.eps);
        const float c3 = r * r * r * dot / static_cast<float>(HD);
#pragma unroll
        for (int t = 0; t < EH; ++t) {
          const int i = lane * EH + t;
          if (tn) { tn[i] = g1[t] * x1[t] * r; tn[HALF + i] = g2[t] * x2[t] * r; }
          g1[t] = r * w1[t] * g1[t] - x1[t] * c3;
          g2[t] = r * w2[t] * g2[t] - x2[t] * c3;
        }
      }
    }
#pragma unroll
    for (int t = 0; t < EH; ++t) {
      const int i = lane * EH + t;
      out[h * HD + i] = g1[t]; out[h * HD + HALF + i] = g2[t];
      outb[h * HD + i] = __float2bfloat16(g1[t]); outb[h * HD + HALF + i] = __float2bfloat16(g2[t]);
    }
  }
}

// dst[c][r] = src[r][c] for a row-major bf16 matrix [rows, cols]; 64 x 64 tiles through shared memory.
__global__ void __launch_bounds__(256) transpose_bf16_kernel(const __nv_bfloat16 *src, int rows, int cols, __nv_bfloat16 *dst, int dst_ld) {
  __shared__ __nv_bfloat16 tile[64][66];
  const int r0 = blockIdx.y * 64, c0 = blockIdx.x * 64;
  const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;
  pdl_prologue();
  for (int i = ty; i < 64; i += 4)
    if (r0 + i < rows && c0 + tx < cols) tile[i][tx] = src[static_cast<size_t>(r0 + i) * cols + c0 + tx];
  __syncthreads();
  for (int i = ty; i < 64; i += 4)
    if (c0 + i < cols && r0 + tx < rows) dst[static_cast<size_t>(c0 + i) * dst_ld + r0 + tx] = tile[tx][i];
}

// ---- AdamW on the head's parameters (Alg. 1, "update phi"; App. B: optimizer and learning rate) ------------------------------
// Per element: m <- b1 m + (1 - b1) g,  v <- b2 v + (1 - b2) g^2,  p <- p (1 - lr wd) - lr (m c1) / (sqrt(v c2) + eps), with the
// bias corrections c1 = 1 / (1 - b1^t), c2 = 1 / (1 - b2^t) formed on the host in double.  fp32 master parameters and
// moments; the bf16 copy the forward pass reads is rewritten in the same pass.  Pure streaming: 16 bytes in, 14 out per element.
struct AdamwArgs {
  float *master, *m, *v;
  const float *grad;
  __nv_bfloat16 *param;                            // or null
  size_t n;
  float lr, b1, b2, eps, decay, c1, c2, gscale;
};
__device__ __forceinline__ float adamw_one(float p, float g, float &m, float &v, const AdamwArgs &A) {
  g *= A.gscale;
  m = fmaf(A.b1, m, (1.0f - A.b1) * g);
  v = fmaf(A.b2, v, (1.0f - A.b2) * g * g);
  return p * A.decay - A.lr * (m * A.c1) / (sqrtf(v * A.c2) + A.eps);
}
__global__ void __launch_bounds__(256) adamw_kernel(const AdamwArgs A) {
  const size_t n4 = A.n >> 2, stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  pdl_prologue();
  for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n4; i += stride) {
    float4 p = reinterpret_cast<float4 *>(A.master)[i], m = reinterpret_cast<float4 *>(A.m)[i], v = reinterpret_cast<float4 *>(A.v)[i];
    const float4 g = reinterpret_cast<const float4 *>(A.grad)[i];
    p.x = adamw_one(p.x, g.x, m.x, v.x, A); p.y = adamw_one(p.y, g.y, m.y, v.y, A);
    p.z = adamw_one(p.z, g.z, m.z, v.z, A); p.w = adamw_one(p.w, g.w, m.w, v.w, A);
    reinterpret_cast<float4 *>(A.master)[i] = p;
    reinterpret_cast<float4 *>(A.m)[i] = m;
    reinterpret_cast<float4 *>(A.v)[i] = v;
    if (A.param) reinterpret_cast<uint2 *>(A.param)[i] = make_uint2(pack_bf16(p.x, p.y), pack_bf16(p.z, p.w));
  }
  if (blockIdx.x == 0 && threadIdx.x < (A.n & 3)) {                        // the last one to three elements
    const size_t i = (n4 << 2) + threadIdx.x;
    float m = A.m[i], v = A.v[i];
    const float p = adamw_one(A.master[i], A.grad[i], m, v, A);
    A.master[i] = p; A.m[i] = m; A.v[i] = v;
    if (A.param) A.param[i] = __float2bfloat16(p);
  }
}

// The head's input rows for given (token, hidden) pairs (App. B.1): zin[row] = [RMSNorm(E[token]; we) ; RMSNorm(hidden; wh)]
// in bf16, and the embedding row itself in fp32 (the norm's backward needs it).  One CTA per row.
__global__ void __launch_bounds__(NG_THREADS)
head_input_rows_kernel(const __nv_bfloat16 *embed, const int32_t *tokens, const float *hidden, const __nv_bfloat16 *we,
                       const __nv_bfloat16 *wh, int d, int vocab, float eps, __nv_bfloat16 *zin, float *e_out, uint32_t *status) {
  __shared__ float red[2][NG_THREADS / 32];
  const int m = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wp = tid >> 5;
  pdl_prologue();
  int tok = tokens[m];
  if (tok < 0 || tok >= vocab) { if (tid == 0) set_status(status, ST_BAD_TOKEN); tok = 0; }
  const __nv_bfloat16 *er = embed + static_cast<size_t>(tok) * d;
  const float *hr = hidden + static_cast<size_t>(m) * d;
  float se = 0.f, sh = 0.f;
  for (int i = tid; i < d; i += NG_THREADS) {
    const float e = bf16_to_float(er[i]), h = hr[i];
    e_out[static_cast<size_t>(m) * d + i] = e;
    se = fmaf(e, e, se); sh = fmaf(h, h, sh);
  }
  se = warp_sum(se); sh = warp_sum(sh);
  if (lane == 0) { red[0][wp] = se; red[1][wp] = sh; }
  __syncthreads();
  se = 0.f; sh = 0.f;
#pragma unroll
  for (int i = 0; i < NG_THREADS / 32; ++i) { se += red[0][i]; sh += red[1][i]; }
  const float re = rsqrtf(se / static_cast<float>(d) + eps), rh = rsqrtf(sh / static_cast<float>(d) + eps);
  __nv_bfloat16 *out = zin + static_cast<size_t>(m) * 2 * d;
  for (int i = tid; i < d; i += NG_THREADS) {
    out[i] = __float2bfloat16(bf16_to_float(er[i]) * re * bf16_to_float(we[i]));
    out[d + i] = __float2bfloat16(hr[i] * rh * bf16_to_float(wh[i]));
  }
}

}  // namespace

cudaError_t launch_capture_chunk(const __nv_bfloat16 *src, const int32_t *row_n, const int32_t *row_base, int rows, int vr,
                                 int QT, int d, __nv_bfloat16 *dst, int dst_stride, cudaStream_t stream) {
  return launch_k(capture_chunk_kernel, dim3(rows * QT), dim3(128), 0, stream, 1, src, row_n, row_base, vr, QT, d, dst,
                  dst_stride);
}
cudaError_t launch_capture_cycle(const __nv_bfloat16 *src, const int32_t *accept_len, const int32_t *kv_len,
                                 const int32_t *finished, int batch, int k, int d, __nv_bfloat16 *dst, int dst_stride,
                                 cudaStream_t stream) {
  return launch_k(capture_cycle_kernel, dim3(batch * (k + 1)), dim3(128), 0, stream, 1, src, accept_len, kv_len, finished,
                  k, d, dst, dst_stride);
}

cudaError_t launch_chain_setup(const ChainSetupArgs &A, int chains, cudaStream_t stream) {
  return launch_k(chain_setup_kernel, dim3(chains), dim3(128), 0, stream, 1, A);
}
cudaError_t launch_gather_chunk_hidden(const __nv_bfloat16 *seq_hidden, int hid_stride, const int32_t *row_base, int rows,
                                       int vr, int QT, int d, const int32_t *row_n, __nv_bfloat16 *out, cudaStream_t stream) {
  return launch_k(gather_chunk_hidden_kernel, dim3(rows * QT), dim3(128), 0, stream, 1, seq_hidden, hid_stride, row_base, vr,
                  QT, d, row_n, out);
}
cudaError_t launch_overlap(const OverlapArgs &A, int rows, cudaStream_t stream) {
  return launch_k(overlap_kernel, dim3(rows), dim3(OV_THREADS), 0, stream, 1, A);
}
cudaError_t launch_dca_grad(const DcaGradArgs &A, cudaStream_t stream) {
  return launch_k(dca_grad_kernel, dim3(A.n * A.K), dim3(DG_THREADS), 0, stream, 1, A);
}
cudaError_t launch_dca_loss(const float *alpha, const int32_t *accepted, int n, int K, float *loss, float *mean,
                            cudaStream_t stream) {
  return launch_k(dca_loss_kernel, dim3(1), dim3(DL_THREADS), 0, stream, 1, alpha, accepted, n, K, loss, mean);
}
cudaError_t launch_rmsnorm_grad(const float *gy, const float *x, const __nv_bfloat16 *w, float *gx, int rows, int d, float eps,
                                cudaStream_t stream, const float *res, float *wterm, int gy_ld) {
  return launch_k(rmsnorm_grad_kernel, dim3(rows), dim3(NG_THREADS), 0, stream, 1, gy, x, w, gx, d, eps, res, wterm,
                  gy_ld > 0 ? gy_ld : d);
}
cudaError_t launch_transpose_bf16(const __nv_bfloat16 *src, int rows, int cols, __nv_bfloat16 *dst, cudaStream_t stream, int dst_ld) {
  transpose_bf16_kernel<<<dim3((cols + 63) / 64, (rows + 63) / 64), 256, 0, stream>>>(src, rows, cols, dst, dst_ld > 0 ? dst_ld : rows);
  return cudaGetLastError();
}
cudaError_t launch_head_input_rows(const __nv_bfloat16 *embed, const int32_t *tokens, const float *hidden, const __nv_bfloat16 *we,
                                   const __nv_bfloat16 *wh, int rows, int d, int vocab, float eps, __nv_bfloat16 *zin, float *e_out,
                                   uint32_t *status, cudaStream_t stream) {
  return launch_k(head_input_rows_kernel, dim3(rows), dim3(NG_THREADS), 0, stream, 1, embed, tokens, hidden, we, wh, d, vocab, eps, zin,
                  e_out, status);
}
size_t colsum_scratch_floats(int d) { return static_cast<size_t>(CS_MAX_CHUNKS) * d; }
cudaError_t launch_colsum(const float *t, int rows, int d, float *out, cudaStream_t stream, bool add, float *scratch) {
  // enough CTAs to fill the device when there are many rows; a single chunk needs no scratch
  const int col_blocks = (d + CS_COLS - 1) / CS_COLS;
  int chunks = 1;
  if (scratch) chunks = std::max(1, std::min(std::min(CS_MAX_CHUNKS, rows / 64), (4 * 148 + col_blocks - 1) / col_blocks));
  const int chunk_rows = (rows + chunks - 1) / chunks;
  chunks = (rows + chunk_rows - 1) / chunk_rows;
  const dim3 grid(col_blocks, chunks), block(CS_COLS, CS_LANES);
  if (chunks == 1) return launch_k(colsum_kernel, grid, block, 0, stream, 1, t, rows, d, chunk_rows, out, add ? 1 : 0);
  if (cudaError_t e = launch_k(colsum_kernel, grid, block, 0, stream, 1, t, rows, d, chunk_rows, scratch, 0); e != cudaSuccess) return e;
  return launch_k(colsum_finish_kernel, dim3((d + 255) / 256), dim3(256), 0, stream, 1, static_cast<const float *>(scratch), chunks, d, out,
                  add ? 1 : 0);
}
cudaError_t launch_step_rows(const StepRowsArgs &A, int chains, cudaStream_t stream) {
  return launch_k(step_rows_kernel, dim3(chains), dim3(128), 0, stream, 1, A);
}
cudaError_t launch_add_state_grad(float *dstate, const float *dhidden, int chains, int K, int k, int d, cudaStream_t stream) {
  return launch_k(add_state_grad_kernel, dim3(chains), dim3(128), 0, stream, 1, dstate, dhidden, K, k, d);
}
cudaError_t launch_fold_boundary(const FoldArgs &A, int chains, cudaStream_t stream) {
  return launch_k(fold_boundary_kernel, dim3(chains), dim3(128), 0, stream, 1, A);
}
cudaError_t launch_fix_to_float(const long long *src, float *dst, size_t n, cudaStream_t stream) {
  const size_t blocks = std::min<size_t>((n + 255) / 256, 148 * 8);
  return launch_k(fix_to_float_kernel, dim3(static_cast<unsigned>(std::max<size_t>(blocks, 1))), dim3(256), 0, stream, 1, src, dst, n);
}
cudaError_t launch_widen_bf16(const __nv_bfloat16 *src, float *dst, size_t n, cudaStream_t stream) {
  const size_t blocks = std::min<size_t>((n + 255) / 256, 148 * 8);
  return launch_k(widen_bf16_kernel, dim3(static_cast<unsigned>(std::max<size_t>(blocks, 1))), dim3(256), 0, stream, 1, src, dst, n);
}
cudaError_t launch_rows_to_f32(const __nv_bfloat16 *src, const int32_t *row_n, int rows, int QT, int d, float *dst, cudaStream_t stream) {
  return launch_k(rows_to_f32_kernel, dim3(rows), dim3(128), 0, stream, 1, src, row_n, QT, d, dst);
}
cudaError_t launch_cast_bf16(const float *src, __nv_bfloat16 *dst, size_t n, cudaStream_t stream) {
  cast_bf16_kernel<<<static_cast<unsigned>((n / 4 + 255) / 256), 256, 0, stream>>>(src, dst, n / 4);
  return cudaGetLastError();
}
cudaError_t launch_qkv_grad_rows(const QkvGradArgs &A, cudaStream_t stream) {
  if (A.hd == 128) return launch_k(qkv_grad_rows_kernel<2>, dim3(A.batch * A.QT), dim3(256), 0, stream, 1, A);
  if (A.hd == 64) return launch_k(qkv_grad_rows_kernel<1>, dim3(A.batch * A.QT), dim3(256), 0, stream, 1, A);
  return cudaErrorInvalidValue;
}
cudaError_t launch_swiglu_grad(const __nv_bfloat16 *ab, const float *dh, __nv_bfloat16 *dab, __nv_bfloat16 *h, int rows, int F,
                               cudaStream_t stream) {
  const size_t n = static_cast<size_t>(rows) * F;
  swiglu_grad_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, stream>>>(ab, dh, dab, h, n, F);
  return cudaGetLastError();
}
cudaError_t launch_adamw(float *master, __nv_bfloat16 *param, const float *grad, float *m, float *v, size_t n, float lr, float b1,
                         float b2, float eps, float decay, float c1, float c2, float gscale, int sm_count, cudaStream_t stream) {
  AdamwArgs A{master, m, v, grad, param, n, lr, b1, b2, eps, decay, c1, c2, gscale};
  const size_t want = ((n >> 2) + 255) / 256;
  const unsigned grid = static_cast<unsigned>(std::max<size_t>(1, std::min<size_t>(want, static_cast<size_t>(sm_count) * 8)));
  adamw_kernel<<<grid, 256, 0, stream>>>(A);
  return cudaGetLastError();
}

}  // namespace gm
