// Memory-bound glue of the decoder: embedding gather, RMSNorm, rotary embedding + KV append,
// SwiGLU, residual/split-K reduction, and the per-phase plan.  One CTA per token row; rows are
// M = batch * QT with a fixed stride QT per sequence (rows j >= qn[b] are padding).
#include "common.cuh"
#include "kernels.h"

namespace gm {

constexpr int EW_THREADS = 256;
constexpr int EW_MAXC = 8;            // float4 chunks per thread: rows up to 8192 wide

__device__ __forceinline__ float block_sum(float v) {
  __shared__ float red[EW_THREADS / 32];
  __shared__ float total;
  v = warp_sum(v);
  __syncthreads();                    // protects `red`/`total` against a previous call
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x < 32) {
    float t = threadIdx.x < EW_THREADS / 32 ? red[threadIdx.x] : 0.f;
    t = warp_sum(t);
    if (threadIdx.x == 0) total = t;
  }
  __syncthreads();
  return total;
}

// y = v * rsqrt(mean(v^2) + eps) * w, written as bf16; v holds this thread's chunks of the row.
__device__ __forceinline__ void rmsnorm_store(const float4 (&v)[EW_MAXC], int d4, int d, float eps,
                                              const __nv_bfloat16 *w, __nv_bfloat16 *out) {
  float ss = 0.f;
  uint2 wv[EW_MAXC];                         // the weights are requested before the reduction: their latency hides behind it
#pragma unroll
  for (int c = 0; c < EW_MAXC; ++c) {
    const int i = threadIdx.x + c * EW_THREADS;
    wv[c] = make_uint2(0u, 0u);
    if (i < d4) {
      wv[c] = *reinterpret_cast<const uint2 *>(w + 4 * i);
      ss += v[c].x * v[c].x + v[c].y * v[c].y + v[c].z * v[c].z + v[c].w * v[c].w;
    }
  }
  const float inv = rsqrtf(block_sum(ss) / static_cast<float>(d) + eps);
#pragma unroll
  for (int c = 0; c < EW_MAXC; ++c) {
    const int i = threadIdx.x + c * EW_THREADS;
    if (i < d4) {
      uint2 o;
      o.x = pack_bf16(v[c].x * inv * bf16_lo(wv[c].x), v[c].y * inv * bf16_hi(wv[c].x));
      o.y = pack_bf16(v[c].z * inv * bf16_lo(wv[c].y), v[c].w * inv * bf16_hi(wv[c].y));
      *reinterpret_cast<uint2 *>(out + 4 * i) = o;
    }
  }
}

__device__ __forceinline__ float4 load_bf16x4(const __nv_bfloat16 *p) {
  const uint2 r = *reinterpret_cast<const uint2 *>(p);
  return make_float4(bf16_lo(r.x), bf16_hi(r.x), bf16_lo(r.y), bf16_hi(r.y));
}

// ---- plan -----------------------------------------------------------------------------------------------
__global__ void plan_kernel(const PlanArgs A) {
  __shared__ int pages[1024];
  const int B = A.batch;
  pdl_prologue();
  for (int b = threadIdx.x; b < B; b += blockDim.x) {
    const int len = A.kv_len[b];
    int qn, qbase;
    if (A.mode == PHASE_VERIFY) { qn = A.k_or_j + 1; qbase = len; }
    else if (A.mode == PHASE_DRAFT_FIRST) { qn = A.pending_n[b]; qbase = len - qn; }
    else if (A.mode == PHASE_CHUNK) { qn = A.row_n[b]; qbase = A.row_base ? A.row_base[b] : A.k_or_j; }
    else { qn = 1; qbase = len + A.k_or_j - 2; }
    bool ok = qn >= 1 && qbase >= 0 && qbase + qn <= A.max_pages_per_seq * 16;
    if (A.finished && A.finished[b]) { A.qn[b] = 0; A.qbase[b] = 0; pages[b] = 0; continue; }    // sits the phase out
    if (A.mode == PHASE_CHUNK) {
      if (qn == 0) { A.qn[b] = 0; A.qbase[b] = 0; pages[b] = 0; continue; }      // sits this pass out
      ok = ok && qn <= A.QT;
    }
    if (A.mode == PHASE_DRAFT_FIRST) ok = ok && qn <= A.k_or_j;     // k_or_j carries max_k + 1 here
    if (!ok) { set_status(A.status, ST_KV_CAPACITY); qn = 0; qbase = 0; }
    A.qn[b] = qn;
    A.qbase[b] = qbase;
    pages[b] = qn > 0 ? (qbase + qn + 15) >> 4 : 0;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int acc = 0;
    for (int b = 0; b < B; ++b) { A.page_start[b] = acc; acc += pages[b]; }
    A.page_start[B] = acc;
  }
}
cudaError_t launch_plan(const PlanArgs &A, cudaStream_t stream) {
  if (A.batch > 1024) return cudaErrorInvalidValue;
  return launch_k(plan_kernel, dim3(1), dim3(256), 0, stream, 1, A);
}

// ---- rollout bookkeeping ------------------------------------------------------------------------------------
__global__ void rollout_append_kernel(const RolloutArgs A, int begin) {
  __shared__ int running;
  pdl_prologue();
  if (threadIdx.x == 0) running = 0;
  __syncthreads();
  for (int b = threadIdx.x; b < A.batch; b += blockDim.x) {
    int fin = begin ? 0 : A.finished[b];
    int len = begin ? 0 : A.out_len[b];
    if (!fin) {
      const int n_new = begin ? 1 : A.accept_len[b] + 1;
      int32_t *row = A.out_tok + static_cast<size_t>(b) * A.out_stride;
      if (len >= A.max_new) fin = 2;
      for (int i = 0; i < n_new && !fin; ++i) {
        const int tok = begin ? A.pending_tok[b * A.pend_stride]
                              : (i < n_new - 1 ? A.draft_tok[b * A.k + i] : A.next_token[b]);
        row[len++] = tok;
        if (tok == A.eos_token) fin = 1;
        else if (len >= A.max_new) fin = 2;
      }
      A.out_len[b] = len;
      A.finished[b] = fin;
    }
    if (!fin) atomicAdd(&running, 1);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    *A.n_running = running;
    if (A.step_counter) *A.step_counter += 1;
  }
}
cudaError_t launch_rollout_append(const RolloutArgs &A, bool begin, cudaStream_t stream) {
  return launch_k(rollout_append_kernel, dim3(1), dim3(256), 0, stream, 1, A, begin ? 1 : 0);
}

__global__ void set_step_kernel(uint64_t *dst, uint64_t value) {
  pdl_prologue();
  if (threadIdx.x == 0) *dst = value;
}
cudaError_t launch_set_step(uint64_t *dst, uint64_t value, cudaStream_t stream) {
  return launch_k(set_step_kernel, dim3(1), dim3(32), 0, stream, 1, dst, value);
}

__global__ void page_reset_kernel(const PageAllocArgs A) {
  pdl_prologue();
  const int t = blockIdx.x * blockDim.x + threadIdx.x, n = gridDim.x * blockDim.x;
  for (int i = t; i < A.num_pages; i += n) A.free_list[i] = A.num_pages - 1 - i;      // page 0 is handed out first
  for (int i = t; i < A.batch * A.max_pages_per_seq; i += n) A.page_table[i] = -1;
  for (int i = t; i < A.batch; i += n) A.held[i] = 0;
  if (t == 0) *A.free_top = A.num_pages;
}
cudaError_t launch_page_reset(const PageAllocArgs &A, cudaStream_t stream) {
  return launch_k(page_reset_kernel, dim3(64), dim3(256), 0, stream, 1, A);
}
// Reserve / release for both pools in one launch (block p = pool p), one thread per row.  A block-wide exclusive prefix
// sum of the rows' page counts gives every row its slice of the free stack, which is exactly the slice the rows would
// get one after the other: the assignment does not depend on thread scheduling.
__device__ __forceinline__ int block_exclusive_scan_1024(int v, int *total) {
  __shared__ int warp_tot[32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
  for (int o = 1; o < 32; o <<= 1) {
    const int up = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += up;
  }
  __syncthreads();                                   // warp_tot may still be read from a previous call
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  int before = 0, all = 0;
  for (int w = 0; w < static_cast<int>(blockDim.x >> 5); ++w) {
    const int t = warp_tot[w];
    if (w < warp) before += t;
    all += t;
  }
  *total = all;
  return before + incl - v;
}
__global__ void __launch_bounds__(1024) page_reserve_kernel(const PageAllocArgs A0, const PageAllocArgs A1) {
  const PageAllocArgs &A = blockIdx.x == 0 ? A0 : A1;
  pdl_prologue();
  const int b = threadIdx.x;
  int have = 0, want = 0;
  if (b < A.batch && !(A.finished && A.finished[b])) {
    const int need = (A.length[b] + A.extra + 15) >> 4;
    have = A.held[b];
    if (need > A.max_pages_per_seq) set_status(A.status, ST_KV_CAPACITY);
    else want = max(need - have, 0);
  }
  int total = 0;
  const int off = block_exclusive_scan_1024(want, &total);
  const int top = *A.free_top;
  const int grant = min(want, max(top - off, 0));
  if (grant < want) set_status(A.status, ST_KV_CAPACITY);      // the stack ran out
  for (int i = 0; i < grant; ++i)
    A.page_table[static_cast<size_t>(b) * A.max_pages_per_seq + have + i] = A.free_list[top - 1 - (off + i)];
  if (b < A.batch && grant > 0) A.held[b] = have + grant;
  __syncthreads();                                   // every thread has read free_top
  if (threadIdx.x == 0) *A.free_top = top - min(total, top);
}
cudaError_t launch_page_reserve(const PageAllocArgs &A0, const PageAllocArgs &A1, cudaStream_t stream) {
  if (A0.batch > 1024 || A1.batch > 1024) return cudaErrorInvalidValue;
  return launch_k(page_reserve_kernel, dim3(2), dim3(1024), 0, stream, 1, A0, A1);
}
__global__ void __launch_bounds__(1024) page_release_kernel(const PageAllocArgs A0, const PageAllocArgs A1) {
  const PageAllocArgs &A = blockIdx.x == 0 ? A0 : A1;
  pdl_prologue();
  const int b = threadIdx.x;
  const int n = (b < A.batch && A.finished[b]) ? A.held[b] : 0;
  int total = 0;
  const int off = block_exclusive_scan_1024(n, &total);
  const int top = *A.free_top;
  int32_t *row = A.page_table + static_cast<size_t>(b < A.batch ? b : 0) * A.max_pages_per_seq;
  for (int k = 0; k < n; ++k) {                       // the row's pages go back last-reserved first
    const int i = n - 1 - k;
    if (top + off + k < A.num_pages) A.free_list[top + off + k] = row[i];
    row[i] = -1;
  }
  if (n > 0) A.held[b] = 0;
  __syncthreads();
  if (threadIdx.x == 0) *A.free_top = min(top + total, A.num_pages);
}
cudaError_t launch_page_release(const PageAllocArgs &A0, const PageAllocArgs &A1, cudaStream_t stream) {
  if (A0.batch > 1024 || A1.batch > 1024) return cudaErrorInvalidValue;
  return launch_k(page_release_kernel, dim3(2), dim3(1024), 0, stream, 1, A0, A1);
}

// ---- prompt prefill: chunk bookkeeping ----------------------------------------------------------------------
__global__ void chunk_setup_kernel(const ChunkSetupArgs A) {
  pdl_prologue();
  for (int v = blockIdx.x * blockDim.x + threadIdx.x; v < A.batch * A.vr; v += gridDim.x * blockDim.x) {
    const int b = v / A.vr, p0 = A.base + (v % A.vr) * A.QT;
    const int L = A.prompt_len[b];
    const bool bad = L < 1 || L > A.max_len || L > A.stride;
    if (bad && p0 == 0) set_status(A.status, ST_KV_CAPACITY);
    const int n = bad ? 0 : min(max(L - p0, 0), A.QT);
    const int hn = bad ? 0 : min(max(L - 1 - p0, 0), A.QT);
    A.row_n[v] = n;
    A.head_n[v] = hn;
    A.row_base[v] = p0;
    for (int j = 0; j < A.QT; ++j)
      A.pair_tok[v * A.pair_stride + j] = j < hn ? A.prompt_tok[static_cast<size_t>(b) * A.stride + p0 + j + 1] : 0;
  }
}
cudaError_t launch_chunk_setup(const ChunkSetupArgs &A, cudaStream_t stream) {
  return launch_k(chunk_setup_kernel, dim3((A.batch * A.vr + 127) / 128), dim3(128), 0, stream, 1, A);
}

__global__ void dup_table_rows_kernel(const int32_t *src, int vr, int cols, int32_t *dst) {
  pdl_prologue();
  const int v = blockIdx.x;
  for (int i = threadIdx.x; i < cols; i += blockDim.x) dst[static_cast<size_t>(v) * cols + i] = src[static_cast<size_t>(v / vr) * cols + i];
}
cudaError_t launch_dup_table_rows(const int32_t *src, int rows, int vr, int cols, int32_t *dst, cudaStream_t stream) {
  return launch_k(dup_table_rows_kernel, dim3(rows * vr), dim3(128), 0, stream, 1, src, vr, cols, dst);
}

__global__ void __launch_bounds__(EW_THREADS)
embed_chunk_kernel(const __nv_bfloat16 *embed, const __nv_bfloat16 *w, const int32_t *prompt_tok, int stride,
                   const int32_t *row_base, const int32_t *row_n, int vr, int QT, int d, int vocab, float eps, float *x,
                   __nv_bfloat16 *xn, uint32_t *status) {
  const int m = blockIdx.x, vrow = m / QT, j = m % QT;
  pdl_prologue();
  int tok = j < row_n[vrow] ? prompt_tok[static_cast<size_t>(vrow / vr) * stride + row_base[vrow] + j] : 0;
  if (tok < 0 || tok >= vocab) { if (threadIdx.x == 0) set_status(status, ST_BAD_TOKEN); tok = 0; }
  const int d4 = d >> 2;
  float4 v[EW_MAXC];
#pragma unroll
  for (int c = 0; c < EW_MAXC; ++c) {
    const int i = threadIdx.x + c * EW_THREADS;
    if (i < d4) {
      v[c] = load_bf16x4(embed + static_cast<size_t>(tok) * d + 4 * i);
      reinterpret_cast<float4 *>(x + static_cast<size_t>(m) * d)[i] = v[c];
    }
  }
  rmsnorm_store(v, d4, d, eps, w, xn + static_cast<size_t>(m) * d);
}
cudaError_t launch_embed_chunk(const __nv_bfloat16 *embed, const __nv_bfloat16 *w, const int32_t *prompt_tok, int stride,
                               const int32_t *row_base, const int32_t *row_n, int rows, int vr, int QT, int d, int vocab,
                               float eps, float *x, __nv_bfloat16 *xn, uint32_t *status, cudaStream_t stream) {
  return launch_k(embed_chunk_kernel, dim3(rows * QT), dim3(EW_THREADS), 0, stream, 1, embed, w, prompt_tok, stride,
                  row_base, row_n, vr, QT, d, vocab, eps, x, xn, status);
}

__global__ void __launch_bounds__(EW_THREADS)
prefill_last_kernel(const float *x, const __nv_bfloat16 *hidden, const int32_t *row_n, const int32_t *row_base,
                    const int32_t *prompt_len, int vr, int QT, int d, int pend_stride, float *xlast,
                    __nv_bfloat16 *pending_hidden) {
  const int v = blockIdx.x, b = v / vr;
  pdl_prologue();
  const int n = row_n[v];
  if (n < 1 || row_base[v] + n != prompt_len[b]) return;
  const size_t m = static_cast<size_t>(v) * QT + n - 1;
  for (int i = threadIdx.x; i < d; i += EW_THREADS) {
    xlast[static_cast<size_t>(b) * d + i] = x[m * d + i];
    pending_hidden[static_cast<size_t>(b) * pend_stride * d + i] = hidden[m * d + i];
  }
}
cudaError_t launch_prefill_last(const float *x, const __nv_bfloat16 *hidden, const int32_t *row_n,
                                const int32_t *row_base, const int32_t *prompt_len, int rows, int vr, int QT, int d,
                                int pend_stride, float *xlast, __nv_bfloat16 *pending_hidden, cudaStream_t stream) {
  return launch_k(prefill_last_kernel, dim3(rows), dim3(EW_THREADS), 0, stream, 1, x, hidden, row_n, row_base,
                  prompt_len, vr, QT, d, pend_stride, xlast, pending_hidden);
}

__global__ void prefill_finish_kernel(const int32_t *prompt_len, const int32_t *first_tok, int batch, int pend_stride,
                                      int32_t *kv_len, int32_t *pending_n, int32_t *pending_tok) {
  pdl_prologue();
  for (int b = blockIdx.x * blockDim.x + threadIdx.x; b < batch; b += gridDim.x * blockDim.x) {
    kv_len[b] = prompt_len[b];
    pending_n[b] = 1;
    pending_tok[b * pend_stride] = first_tok[b];
  }
}
cudaError_t launch_prefill_finish(const int32_t *prompt_len, const int32_t *first_tok, int batch, int pend_stride,
                                  int32_t *kv_len, int32_t *pending_n, int32_t *pending_tok, cudaStream_t stream) {
  return launch_k(prefill_finish_kernel, dim3((batch + 127) / 128), dim3(128), 0, stream, 1, prompt_len, first_tok, batch,
                  pend_stride, kv_len, pending_n, pending_tok);
}

// ---- embedding gather + first RMSNorm of the verify forward ------------------------------------------------
__global__ void __launch_bounds__(EW_THREADS)
embed_norm_kernel(const __nv_bfloat16 *embed, const __nv_bfloat16 *w, const int32_t *pending_tok,
                  const int32_t *pending_n, const int32_t *draft_tok, int K, int max_k, int d, int vocab, float eps,
                  float *x, __nv_bfloat16 *xn, uint32_t *status) {
  const int m = blockIdx.x, b = m / (K + 1), j = m % (K + 1);
  pdl_prologue();
  int tok;
  if (j == 0) {
    const int n = min(max(pending_n[b], 1), max_k + 1);
    tok = pending_tok[b * (max_k + 1) + n - 1];
  } else {
    tok = draft_tok[b * K + j - 1];
  }
  if (tok < 0 || tok >= vocab) { if (threadIdx.x == 0) set_status(status, ST_BAD_TOKEN); tok = 0; }
  const int d4 = d >> 2;
  float4 v[EW_MAXC];
#pragma unroll
  for (int c = 0; c < EW_MAXC; ++c) {
    const int i = threadIdx.x + c * EW_THREADS;
    if (i < d4) {
      v[c] = load_bf16x4(embed + static_cast<size_t>(tok) * d + 4 * i);
      reinterpret_cast<float4 *>(x + static_cast<size_t>(m) * d)[i] = v[c];
    }
  }
  rmsnorm_store(v, d4, d, eps, w, xn + static_cast<size_t>(m) * d);
}
cudaError_t launch_embed_norm(const __nv_bfloat16 *embed, const __nv_bfloat16 *w, const int32_t *pending_tok,
                              const int32_t *pending_n, const int32_t *draft_tok, int batch, int K, int max_k, int d,
                              int vocab, float eps, float *x, __nv_bfloat16 *xn, uint32_t *status,
                              cudaStream_t stream) {
  return launch_k(embed_norm_kernel, dim3(batch * (K + 1)), dim3(EW_THREADS), 0, stream, 1, embed, w, pending_tok,
                  pending_n, draft_tok, K, max_k, d, vocab, eps, x, xn, status);
}

// ---- draft-head input: [RMSNorm_e(embedding) ; RMSNorm_h(hidden)] ---------------------------------------------
__global__ void __launch_bounds__(EW_THREADS) head_input_kernel(const HeadInputArgs A) {
  const int m = blockIdx.x, b = m / A.QT, j = m % A.QT;
  const int d = A.d, d4 = d >> 2;
  __nv_bfloat16 *out = A.zin + static_cast<size_t>(m) * 2 * d;
  pdl_prologue();
  int tok = 0;
  bool valid = true;
  const __nv_bfloat16 *hid_bf = nullptr;
  const float *hid_f = nullptr;
  if (A.mode == PHASE_DRAFT_FIRST) {
    const int n = A.pending_n[b];
    valid = j < n && n <= A.max_k + 1;
    if (valid) {
      tok = A.pending_tok[b * (A.max_k + 1) + j];
      hid_bf = A.pending_hidden + (static_cast<size_t>(b) * (A.max_k + 1) + j) * d;
    }
  } else {
    tok = A.draft_tok[b * A.k + A.j - 2];
    hid_f = A.g_prev + static_cast<size_t>(b) * d;
  }
  if (!valid) {
    for (int i = threadIdx.x; i < 2 * d4; i += EW_THREADS) reinterpret_cast<uint2 *>(out)[i] = make_uint2(0u, 0u);
    return;
  }
  if (tok < 0 || tok >= A.vocab) { if (threadIdx.x == 0) set_status(A.status, ST_BAD_TOKEN); tok = 0; }
  float4 v[EW_MAXC];
#pragma unroll
  for (int c = 0; c < EW_MAXC; ++c) {
    const int i = threadIdx.x + c * EW_THREADS;
    if (i < d4) v[c] = load_bf16x4(A.embed + static_cast<size_t>(tok) * d + 4 * i);
  }
  rmsnorm_store(v, d4, d, A.eps, A.we, out);
#pragma unroll
  for (int c = 0; c < EW_MAXC; ++c) {
    const int i = threadIdx.x + c * EW_THREADS;
    if (i < d4) v[c] = hid_bf ? load_bf16x4(hid_bf + 4 * i) : reinterpret_cast<const float4 *>(hid_f)[i];
  }
  rmsnorm_store(v, d4, d, A.eps, A.wh, out + d);
}
cudaError_t launch_head_input(const HeadInputArgs &A, cudaStream_t stream) {
  return launch_k(head_input_kernel, dim3(A.batch * A.QT), dim3(EW_THREADS), 0, stream, 1, A);
}

// ---- RMSNorm of the fp32 residual stream ------------------------------------------------------------------------------
__global__ void __launch_bounds__(EW_THREADS)
rmsnorm_kernel(const float *x, const __nv_bfloat16 *w, __nv_bfloat16 *xn, __nv_bfloat16 *hidden_out, int d, float eps) {
  const int m = blockIdx.x, d4 = d >> 2;
  pdl_prologue();
  float4 v[EW_MAXC];
#pragma unroll
  for (int c = 0; c < EW_MAXC; ++c) {
    const int i = threadIdx.x + c * EW_THREADS;
    if (i < d4) {
      v[c] = reinterpret_cast<const float4 *>(x + static_cast<size_t>(m) * d)[i];
      if (hidden_out) {
        uint2 o;
        o.x = pack_bf16(v[c].x, v[c].y);
        o.y = pack_bf16(v[c].z, v[c].w);
        *reinterpret_cast<uint2 *>(hidden_out + static_cast<size_t>(m) * d + 4 * i) = o;
      }
    }
  }
  if (xn) rmsnorm_store(v, d4, d, eps, w, xn + static_cast<size_t>(m) * d);
}
cudaError_t launch_rmsnorm(const float *x, const __nv_bfloat16 *w, __nv_bfloat16 *xn, __nv_bfloat16 *hidden_out,
                           int M, int d, float eps, cudaStream_t stream) {
  return launch_k(rmsnorm_kernel, dim3(M), dim3(EW_THREADS), 0, stream, 1, x, w, xn, hidden_out, d, eps);
}

// ---- rotary embedding + KV append + Q rearrangement --------------------------------------------------------------------
// One CTA per token row; a work item is 8 consecutive head dimensions (one 16-byte load per half of the
// rotate-half pair, two 16-byte stores).
__device__ __forceinline__ void unpack8f(const uint4 &v, float (&x)[8]) {
  x[0] = bf16_lo(v.x); x[1] = bf16_hi(v.x); x[2] = bf16_lo(v.y); x[3] = bf16_hi(v.y);
  x[4] = bf16_lo(v.z); x[5] = bf16_hi(v.z); x[6] = bf16_lo(v.w); x[7] = bf16_hi(v.w);
}
__device__ __forceinline__ uint4 pack8f(const float (&x)[8]) {
  return make_uint4(pack_bf16(x[0], x[1]), pack_bf16(x[2], x[3]), pack_bf16(x[4], x[5]), pack_bf16(x[6], x[7]));
}
__global__ void __launch_bounds__(EW_THREADS) rope_append_kernel(const RopeAppendArgs A) {
  const int m = blockIdx.x, b = m / A.QT, j = m % A.QT;
  const int hd = A.hd, half = hd >> 1, group = A.n_q / A.n_kv;
  const int ncols = (A.n_q + 2 * A.n_kv) * hd;
  pdl_prologue();
  // Everything that does not depend on another load is requested at once: the query count, the first position and
  // this thread's first work item of the projection row (the kernel is a chain of latencies, not of bandwidth).
  const int qn = A.qn[b];
  const int qb = A.qbase[b];
  const int hv = half >> 3;                                       // 8-wide items per half head
  const __nv_bfloat16 *src = A.qkv + static_cast<size_t>(m) * ncols;
  const int n_rot = (A.n_q + A.n_kv) * hv, n_v = A.n_kv * (hd >> 3);
  uint4 first1 = make_uint4(0u, 0u, 0u, 0u), first2 = first1;
  if (static_cast<int>(threadIdx.x) < n_rot) {
    const int h = threadIdx.x / hv, e = (threadIdx.x % hv) * 8;
    first1 = *reinterpret_cast<const uint4 *>(src + h * hd + e);
    first2 = *reinterpret_cast<const uint4 *>(src + h * hd + e + half);
  } else if (static_cast<int>(threadIdx.x) < n_rot + n_v) {
    const int iv = threadIdx.x - n_rot, h = iv / (hd >> 3), e = (iv % (hd >> 3)) * 8;
    first1 = *reinterpret_cast<const uint4 *>(src + (A.n_q + A.n_kv) * hd + h * hd + e);
  }
  __nv_bfloat16 *qdst = A.qbuf + static_cast<size_t>(b) * A.n_kv * A.qrows * hd;
  if (j >= qn) {                           // padding row: zero its query rows, append nothing
    for (int i = threadIdx.x; i < A.n_q * (hd >> 3); i += EW_THREADS) {
      const int h = i / (hd >> 3), e = (i % (hd >> 3)) * 8;
      *reinterpret_cast<uint4 *>(qdst + (static_cast<size_t>(h / group) * A.qrows + j * group + h % group) * hd + e) =
          make_uint4(0u, 0u, 0u, 0u);
    }
    return;
  }
  const int pos = qb + j;
  const int page = A.page_table[static_cast<size_t>(b) * A.max_pages_per_seq + (pos >> 4)];
  const bool in_pool = page >= 0 && page < A.num_pages;
  if (!in_pool && threadIdx.x == 0) set_status(A.status, ST_BAD_PAGE);
  const bool page_ok = in_pool && A.pool != nullptr;              // no pool: queries only, nothing is appended
  const float2 *cs = A.rope + static_cast<size_t>(pos) * half;
  const size_t page_elems = static_cast<size_t>(A.n_kv) * 16 * hd;
  __nv_bfloat16 *kdst = A.pool + ((static_cast<size_t>(A.layer) * 2 + 0) * A.num_pages + (page_ok ? page : 0)) * page_elems;
  __nv_bfloat16 *vdst = A.pool + ((static_cast<size_t>(A.layer) * 2 + 1) * A.num_pages + (page_ok ? page : 0)) * page_elems;
  const int slot = pos & 15;
  // the hv lanes that share one head are consecutive and aligned (hv is a power of two <= 32)
  const unsigned lane = threadIdx.x & 31u;
  const unsigned head_lanes = hv >= 32 ? 0xffffffffu : ((1u << hv) - 1u) << (lane & ~static_cast<unsigned>(hv - 1));
  for (int i = threadIdx.x; i < n_rot + n_v; i += EW_THREADS) {
    if (i < n_rot) {
      const int h = i / hv, e = (i % hv) * 8;
      float x1[8], x2[8], y1[8], y2[8];
      const bool is_first = i == static_cast<int>(threadIdx.x);
      unpack8f(is_first ? first1 : *reinterpret_cast<const uint4 *>(src + h * hd + e), x1);
      unpack8f(is_first ? first2 : *reinterpret_cast<const uint4 *>(src + h * hd + e + half), x2);
      if (A.bias) {
        float b1[8], b2[8];
        unpack8f(*reinterpret_cast<const uint4 *>(A.bias + h * hd + e), b1);
        unpack8f(*reinterpret_cast<const uint4 *>(A.bias + h * hd + e + half), b2);
#pragma unroll
        for (int t = 0; t < 8; ++t) { x1[t] += b1[t]; x2[t] += b2[t]; }
      }
      const __nv_bfloat16 *nw = h < A.n_q ? A.qnorm : A.knorm;
      if (nw) {                                       // RMSNorm over the head dimension, before the rotation
        float ss = 0.f;
#pragma unroll
        for (int t = 0; t < 8; ++t) ss += x1[t] * x1[t] + x2[t] * x2[t];
        for (int off = hv >> 1; off >= 1; off >>= 1) ss += __shfl_xor_sync(head_lanes, ss, off);
        const float inv = rsqrtf(ss / static_cast<float>(hd) + A.eps);
        float w1[8], w2[8];
        unpack8f(*reinterpret_cast<const uint4 *>(nw + e), w1);
        unpack8f(*reinterpret_cast<const uint4 *>(nw + e + half), w2);
#pragma unroll
        for (int t = 0; t < 8; ++t) { x1[t] = x1[t] * inv * w1[t]; x2[t] = x2[t] * inv * w2[t]; }
      }
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        const float2 c = cs[e + t];
        y1[t] = x1[t] * c.x - x2[t] * c.y;
        y2[t] = x2[t] * c.x + x1[t] * c.y;
      }
      __nv_bfloat16 *dst;
      if (h < A.n_q) dst = qdst + (static_cast<size_t>(h / group) * A.qrows + j * group + h % group) * hd;
      else if (page_ok) dst = kdst + (static_cast<size_t>(h - A.n_q) * 16 + slot) * hd;
      else continue;
      *reinterpret_cast<uint4 *>(dst + e) = pack8f(y1);
      *reinterpret_cast<uint4 *>(dst + e + half) = pack8f(y2);
    } else if (page_ok) {
      const int iv = i - n_rot, h = iv / (hd >> 3), e = (iv % (hd >> 3)) * 8;
      uint4 val = i == static_cast<int>(threadIdx.x) ? first1
                                                     : *reinterpret_cast<const uint4 *>(src + (A.n_q + A.n_kv) * hd + h * hd + e);
      if (A.bias) {
        float x[8], bv[8];
        unpack8f(val, x);
        unpack8f(*reinterpret_cast<const uint4 *>(A.bias + (A.n_q + A.n_kv) * hd + h * hd + e), bv);
#pragma unroll
        for (int t = 0; t < 8; ++t) x[t] += bv[t];
        val = pack8f(x);
      }
      *reinterpret_cast<uint4 *>(vdst + (static_cast<size_t>(h) * 16 + slot) * hd + e) = val;
    }
  }
}
cudaError_t launch_rope_append(const RopeAppendArgs &A, cudaStream_t stream) {
  return launch_k(rope_append_kernel, dim3(A.batch * A.QT), dim3(EW_THREADS), 0, stream, 1, A);
}

// ---- head output row: last valid row of each sequence + the head's final norm ----------------------------------------------
__global__ void __launch_bounds__(EW_THREADS)
head_out_kernel(const float *x, const int32_t *qn, int QT, int d, const __nv_bfloat16 *w, float eps, float *g,
                __nv_bfloat16 *gn) {
  const int b = blockIdx.x, d4 = d >> 2;
  pdl_prologue();
  const int j = min(max(qn[b], 1), QT) - 1;
  const float4 *src = reinterpret_cast<const float4 *>(x + (static_cast<size_t>(b) * QT + j) * d);
  float4 v[EW_MAXC];
#pragma unroll
  for (int c = 0; c < EW_MAXC; ++c) {
    const int i = threadIdx.x + c * EW_THREADS;
    if (i < d4) {
      v[c] = src[i];
      reinterpret_cast<float4 *>(g + static_cast<size_t>(b) * d)[i] = v[c];
    }
  }
  rmsnorm_store(v, d4, d, eps, w, gn + static_cast<size_t>(b) * d);
}
cudaError_t launch_head_out(const float *x, const int32_t *qn, int batch, int QT, int d, const __nv_bfloat16 *w,
                            float eps, float *g, __nv_bfloat16 *gn, cudaStream_t stream) {
  return launch_k(head_out_kernel, dim3(batch), dim3(EW_THREADS), 0, stream, 1, x, qn, QT, d, w, eps, g, gn);
}

}  // namespace gm
