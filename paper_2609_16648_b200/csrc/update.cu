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

// alpha = sum_i min(p_i, q_i) + min(1 - sum p_i, 1 - sum q_i) over the record's retained entries; one CTA per row.
constexpr int OV_THREADS = 256;
__global__ void __launch_bounds__(OV_THREADS) overlap_kernel(const OverlapArgs A) {
  __shared__ float red[OV_THREADS / 32];
  __shared__ float sh_lse;
  const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const __nv_bfloat16 *x = A.logits + static_cast<size_t>(row) * A.V;
  const uint4 *xv = reinterpret_cast<const uint4 *>(x);
  const int nvec = A.V >> 3;
  pdl_prologue();
  float m = -INFINITY;
  for (int i = tid; i < nvec; i += OV_THREADS) {
    const uint4 v = xv[i];
    m = fmaxf(m, fmaxf(fmaxf(fmaxf(bf16_lo(v.x), bf16_hi(v.x)), fmaxf(bf16_lo(v.y), bf16_hi(v.y))),
                       fmaxf(fmaxf(bf16_lo(v.z), bf16_hi(v.z)), fmaxf(bf16_lo(v.w), bf16_hi(v.w)))));
  }
  for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if (lane == 0) red[warp] = m;
  __syncthreads();
  m = red[0];
  for (int w = 1; w < OV_THREADS / 32; ++w) m = fmaxf(m, red[w]);
  __syncthreads();
  float z = 0.f;
  for (int i = tid; i < nvec; i += OV_THREADS) {
    const uint4 v = xv[i];
    const uint32_t wds[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int t = 0; t < 4; ++t) z += __expf((bf16_lo(wds[t]) - m) * A.inv_temp) + __expf((bf16_hi(wds[t]) - m) * A.inv_temp);
  }
  for (int o = 16; o; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
  if (lane == 0) red[warp] = z;
  __syncthreads();
  if (tid == 0) {
    float t = 0.f;
    for (int w = 0; w < OV_THREADS / 32; ++w) t += red[w];
    sh_lse = m * A.inv_temp + logf(t);
  }
  __syncthreads();
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
cudaError_t launch_dca_loss(const float *alpha, const int32_t *accepted, int n, int K, float *loss, float *mean,
                            cudaStream_t stream) {
  return launch_k(dca_loss_kernel, dim3(1), dim3(DL_THREADS), 0, stream, 1, alpha, accepted, n, K, loss, mean);
}

}  // namespace gm
