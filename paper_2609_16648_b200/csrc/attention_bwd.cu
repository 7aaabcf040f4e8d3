// Backward of the paged multi-query attention core (scores, softmax, weighted values) for the head update (Alg. 1,
// "update phi"): gradients with respect to the queries and to every cached key and value.
//
// For a query row with output gradient dO, keys k_j, values v_j, P = softmax(q k^T / sqrt(hd)) over its visible keys:
//     dP_j = dO . v_j,   D = sum_j P_j dP_j,   dS_j = P_j (dP_j - D),
//     dq = sum_j dS_j k_j / sqrt(hd),   dk_j += dS_j q / sqrt(hd),   dv_j += P_j dO.
// Two passes, no attention matrix in memory.  The first walks a row's keys once for the softmax statistics (running
// maximum and sum) and D (accumulated with the same rescaling).  The second has one CTA per (sequence, KV head) with one
// warp per query head of the group: a key and its value are read once, every query row that sees them adds its terms
// in registers, the group's warps are summed through shared memory, and one vector of atomic additions per key goes to
// the gradient planes - sequences whose page tables share pages (the chains of one sequence share its committed prefix)
// accumulate into the same entries.  Few query rows per sequence (k + 1 at most), so the walk is a stream over the
// cache, like the forward kernel; it uses plain loads and warp reductions, not the tensor cores.  Two forms of the two
// passes: keys split over warps and CTAs (few query rows per KV head: the usual case), and a CTA per (sequence, KV
// head) with a warp per query head for the rest.
#include "common.cuh"
#include "kernels.h"

namespace gm {
namespace {

constexpr int AB_MAX_ROWS = 8;                        // query rows per sequence (max_k + 1)
constexpr int AB_MAX_GROUP = 8;                       // query heads per KV head

__device__ __forceinline__ float ab_bf(const __nv_bfloat16 v) { return __bfloat162float(v); }

// one head vector of hd = 32 * E elements: lane l holds elements l*E .. l*E + E - 1
template <int E>
__device__ __forceinline__ void ab_load_bf16(const __nv_bfloat16 *p, int lane, float (&x)[E]) {
  if constexpr (E == 4) {
    const uint2 w = reinterpret_cast<const uint2 *>(p)[lane];
    x[0] = bf16_lo(w.x); x[1] = bf16_hi(w.x); x[2] = bf16_lo(w.y); x[3] = bf16_hi(w.y);
  } else if constexpr (E == 2) {
    const uint32_t w = reinterpret_cast<const uint32_t *>(p)[lane];
    x[0] = bf16_lo(w); x[1] = bf16_hi(w);
  } else {
#pragma unroll
    for (int e = 0; e < E; ++e) x[e] = ab_bf(p[lane * E + e]);
  }
}
template <int E>
__device__ __forceinline__ float ab_dot(const float (&a)[E], const float (&b)[E]) {
  float s = 0.f;
#pragma unroll
  for (int e = 0; e < E; ++e) s = fmaf(a[e], b[e], s);
  return warp_sum(s);
}

// ---- pass 1: (max, sum, D) of every (row, query head) -------------------------------------------------------------------
// grid (B * QT, n_kv), one warp per query head of the group
template <int E>
__global__ void __launch_bounds__(AB_MAX_GROUP * 32) attn_bwd_stats_kernel(const AttnBwdArgs A) {
  const int m = blockIdx.x, b = m / A.QT, j = m % A.QT, kvh = blockIdx.y;
  const int lane = threadIdx.x & 31, g = threadIdx.x >> 5, hd = 32 * E;
  pdl_prologue();
  if (g >= A.group || j >= A.qn[b]) return;
  const int h = kvh * A.group + g, pos = A.qbase[b] + j;
  float q[E], dO[E];
  ab_load_bf16<E>(A.q + ((static_cast<size_t>(b) * A.n_kv + kvh) * A.qrows + j * A.group + g) * hd, lane, q);
#pragma unroll
  for (int e = 0; e < E; ++e) dO[e] = A.dout[(static_cast<size_t>(m) * A.n_kv * A.group + h) * hd + lane * E + e];
  const size_t page_elems = static_cast<size_t>(A.n_kv) * 16 * hd;
  const __nv_bfloat16 *kplane = A.pool + (static_cast<size_t>(A.layer) * 2 + 0) * A.num_pages * page_elems;
  const __nv_bfloat16 *vplane = A.pool + (static_cast<size_t>(A.layer) * 2 + 1) * A.num_pages * page_elems;
  float mx = -INFINITY, l = 0.f, dacc = 0.f;
  for (int p = 0; p <= pos; ++p) {
    const int page = A.page_table[static_cast<size_t>(b) * A.max_pages_per_seq + (p >> 4)];
    if (page < 0 || page >= A.num_pages) { if (lane == 0) set_status(A.status, ST_BAD_PAGE); return; }
    const size_t off = static_cast<size_t>(page) * page_elems + (static_cast<size_t>(kvh) * 16 + (p & 15)) * hd;
    float k[E], v[E];
    ab_load_bf16<E>(kplane + off, lane, k);
    ab_load_bf16<E>(vplane + off, lane, v);
    const float s = ab_dot<E>(q, k) * A.scale, dp = ab_dot<E>(dO, v);
    if (s > mx) { const float r = __expf(mx - s); l *= r; dacc *= r; mx = s; }      // exp(-inf) = 0 on the first key
    const float e = __expf(s - mx);
    l += e;
    dacc = fmaf(e, dp, dacc);
  }
  if (lane == 0) {
    float *st = A.stats + (static_cast<size_t>(m) * A.n_kv * A.group + h) * 3;
    st[0] = mx; st[1] = 1.0f / l; st[2] = dacc / l;
  }
}

// ---- pass 2: gradients ---------------------------------------------------------------------------------------------------
// grid (B, n_kv), one warp per query head of the group; rows and their statistics staged in shared memory
template <int E>
__global__ void __launch_bounds__(AB_MAX_GROUP * 32) attn_bwd_grad_kernel(const AttnBwdArgs A) {
  constexpr int HD = 32 * E;
  extern __shared__ float ab_smem[];                  // q [QT][group][HD], dO [QT][group][HD], red [2][group][HD]
  __shared__ float sst[AB_MAX_ROWS][AB_MAX_GROUP][3];
  const int G = A.group;
  float *sq = ab_smem, *sdo = sq + static_cast<size_t>(A.QT) * G * HD, *red = sdo + static_cast<size_t>(A.QT) * G * HD;
  const int b = blockIdx.x, kvh = blockIdx.y;
  const int lane = threadIdx.x & 31, g = threadIdx.x >> 5;
  pdl_prologue();
  const int qn = min(A.qn[b], A.QT), qbase = A.qbase[b];
  if (qn <= 0) return;
  const bool mine = g < A.group;
  const int h = kvh * A.group + g;
  if (mine)
    for (int j = 0; j < qn; ++j) {
      const int m = b * A.QT + j;
      const __nv_bfloat16 *qp = A.q + ((static_cast<size_t>(b) * A.n_kv + kvh) * A.qrows + j * A.group + g) * HD;
#pragma unroll
      for (int e = 0; e < E; ++e) {
        sq[(j * G + g) * HD + lane * E + e] = ab_bf(qp[lane * E + e]);
        sdo[(j * G + g) * HD + lane * E + e] = A.dout[(static_cast<size_t>(m) * A.n_kv * A.group + h) * HD + lane * E + e];
      }
      if (lane < 3) sst[j][g][lane] = A.stats[(static_cast<size_t>(m) * A.n_kv * A.group + h) * 3 + lane];
    }
  __syncthreads();
  float dq[AB_MAX_ROWS][E];
#pragma unroll
  for (int j = 0; j < AB_MAX_ROWS; ++j)
#pragma unroll
    for (int e = 0; e < E; ++e) dq[j][e] = 0.f;
  const size_t page_elems = static_cast<size_t>(A.n_kv) * 16 * HD;
  const __nv_bfloat16 *kplane = A.pool + (static_cast<size_t>(A.layer) * 2 + 0) * A.num_pages * page_elems;
  const __nv_bfloat16 *vplane = A.pool + (static_cast<size_t>(A.layer) * 2 + 1) * A.num_pages * page_elems;
  const int last = qbase + qn - 1;
  for (int p = 0; p <= last; ++p) {
    const int page = A.page_table[static_cast<size_t>(b) * A.max_pages_per_seq + (p >> 4)];
    if (page < 0 || page >= A.num_pages) { if (threadIdx.x == 0) set_status(A.status, ST_BAD_PAGE); return; }   // uniform
    const size_t off = static_cast<size_t>(page) * page_elems + (static_cast<size_t>(kvh) * 16 + (p & 15)) * HD;
    float k[E], v[E], dk[E], dv[E];
    ab_load_bf16<E>(kplane + off, lane, k);
    ab_load_bf16<E>(vplane + off, lane, v);
#pragma unroll
    for (int e = 0; e < E; ++e) dk[e] = dv[e] = 0.f;
    if (mine) {
#pragma unroll
      for (int j = 0; j < AB_MAX_ROWS; ++j) {
        if (j < qn && p <= qbase + j) {               // warp-uniform
          float qv[E], dov[E];
#pragma unroll
          for (int e = 0; e < E; ++e) { qv[e] = sq[(j * G + g) * HD + lane * E + e]; dov[e] = sdo[(j * G + g) * HD + lane * E + e]; }
          const float s = ab_dot<E>(qv, k) * A.scale, dp = ab_dot<E>(dov, v);
          const float pr = __expf(s - sst[j][g][0]) * sst[j][g][1];
          const float ds = pr * (dp - sst[j][g][2]) * A.scale;
#pragma unroll
          for (int e = 0; e < E; ++e) {
            dq[j][e] = fmaf(ds, k[e], dq[j][e]);
            dk[e] = fmaf(ds, qv[e], dk[e]);
            dv[e] = fmaf(pr, dov[e], dv[e]);
          }
        }
      }
    }
    // the group's heads share this key and value: sum their terms, then one set of atomic additions
#pragma unroll
    for (int e = 0; e < E; ++e) { red[g * HD + lane * E + e] = dk[e]; red[(G + g) * HD + lane * E + e] = dv[e]; }
    __syncthreads();
    for (int i = threadIdx.x; i < 2 * HD; i += blockDim.x) {
      const int which = i / HD, c = i % HD;
      float acc = 0.f;
      for (int gg = 0; gg < G; ++gg) acc += red[(which * G + gg) * HD + c];
      if (A.dk_fix) fix_add((which ? A.dv_fix : A.dk_fix) + off + c, acc);
      else if (acc != 0.f) atomicAdd((which ? A.dv_pool : A.dk_pool) + off + c, acc);
    }
    __syncthreads();
  }
  if (mine) {
#pragma unroll
    for (int j = 0; j < AB_MAX_ROWS; ++j)
      if (j < qn) {
        const int m = b * A.QT + j;
#pragma unroll
        for (int e = 0; e < E; ++e) {
          const size_t o = (static_cast<size_t>(m) * A.n_kv * A.group + h) * HD + lane * E + e;
          if (A.dq_fix) fix_add(A.dq_fix + o, dq[j][e]);
          else A.dq[o] = dq[j][e];
        }
      }
  }
}

// ---- the same two passes with the keys split over warps and CTAs ----------------------------------------------------------
// While a (sequence, KV head) has at most NP (row, query head) pairs, a warp can keep every pair's running statistics -
// or its dq - in registers and take whole keys: CTA (b, kv head, segment of ATTN_BWD_SEG keys), warp w takes keys
// w, w + 8, ... of the segment, reads a key and its value once, and visits the pairs that see it.  No barrier per key,
// no cross-warp sum per key (a key's dk / dv terms all come from the warp that holds it); the statistics are merged
// across warps and segments afterwards, dq across warps through shared memory and across segments with atomic additions.
constexpr int AB_WARPS = 8;

template <int E, int NP>
__global__ void __launch_bounds__(AB_WARPS * 32) attn_bwd_stats_split_kernel(const AttnBwdArgs A) {
  constexpr int HD = 32 * E;
  __shared__ float sq[NP][HD], sdo[NP][HD];
  __shared__ float wpart[AB_WARPS][NP][3];
  const int b = blockIdx.x, kvh = blockIdx.y, seg = blockIdx.z, G = A.group;
  const int lane = threadIdx.x & 31, wp = threadIdx.x >> 5;
  pdl_prologue();
  const int qn = min(A.qn[b], A.QT), qbase = A.qbase[b], np = qn * G;
  const int last = qbase + qn - 1, p0 = seg * ATTN_BWD_SEG;
  if (qn <= 0 || p0 > last) return;
  for (int i = wp; i < np; i += AB_WARPS) {
    const int j = i / G, g = i % G, m = b * A.QT + j, h = kvh * G + g;
    const __nv_bfloat16 *qp = A.q + ((static_cast<size_t>(b) * A.n_kv + kvh) * A.qrows + i) * HD;
#pragma unroll
    for (int e = 0; e < E; ++e) {
      sq[i][lane * E + e] = ab_bf(qp[lane * E + e]);
      sdo[i][lane * E + e] = A.dout[(static_cast<size_t>(m) * A.n_kv * G + h) * HD + lane * E + e];
    }
  }
  __syncthreads();
  float mx[NP], l[NP], da[NP];
#pragma unroll
  for (int i = 0; i < NP; ++i) { mx[i] = -INFINITY; l[i] = 0.f; da[i] = 0.f; }
  const size_t page_elems = static_cast<size_t>(A.n_kv) * 16 * HD;
  const __nv_bfloat16 *kplane = A.pool + (static_cast<size_t>(A.layer) * 2 + 0) * A.num_pages * page_elems;
  const __nv_bfloat16 *vplane = A.pool + (static_cast<size_t>(A.layer) * 2 + 1) * A.num_pages * page_elems;
  const int p1 = min(p0 + ATTN_BWD_SEG - 1, last);
  for (int p = p0 + wp; p <= p1; p += AB_WARPS) {
    const int page = A.page_table[static_cast<size_t>(b) * A.max_pages_per_seq + (p >> 4)];
    if (page < 0 || page >= A.num_pages) { if (lane == 0) set_status(A.status, ST_BAD_PAGE); continue; }
    const size_t off = static_cast<size_t>(page) * page_elems + (static_cast<size_t>(kvh) * 16 + (p & 15)) * HD;
    float k[E], v[E];
    ab_load_bf16<E>(kplane + off, lane, k);
    ab_load_bf16<E>(vplane + off, lane, v);
#pragma unroll
    for (int i = 0; i < NP; ++i) {
      if (i < np && p <= qbase + i / G) {                 // warp-uniform
        float qv[E], dov[E];
#pragma unroll
        for (int e = 0; e < E; ++e) { qv[e] = sq[i][lane * E + e]; dov[e] = sdo[i][lane * E + e]; }
        const float s = ab_dot<E>(qv, k) * A.scale, dp = ab_dot<E>(dov, v);
        if (s > mx[i]) { const float r = __expf(mx[i] - s); l[i] *= r; da[i] *= r; mx[i] = s; }
        const float e = __expf(s - mx[i]);
        l[i] += e;
        da[i] = fmaf(e, dp, da[i]);
      }
    }
  }
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < NP; ++i) { wpart[wp][i][0] = mx[i]; wpart[wp][i][1] = l[i]; wpart[wp][i][2] = da[i]; }
  }
  __syncthreads();
  if (static_cast<int>(threadIdx.x) < np) {                // merge the warps, in warp order
    const int i = threadIdx.x;
    float M = -INFINITY;
    for (int w = 0; w < AB_WARPS; ++w) M = fmaxf(M, wpart[w][i][0]);
    float L = 0.f, D = 0.f;
    for (int w = 0; w < AB_WARPS; ++w) {
      const float r = wpart[w][i][1] > 0.f ? __expf(wpart[w][i][0] - M) : 0.f;
      L = fmaf(wpart[w][i][1], r, L); D = fmaf(wpart[w][i][2], r, D);
    }
    float *o = A.part + (((static_cast<size_t>(b) * A.n_kv + kvh) * A.nseg + seg) * NP + i) * 3;
    o[0] = M; o[1] = L; o[2] = D;
  }
}

template <int E, int NP>
__global__ void __launch_bounds__(AB_WARPS * 32) attn_bwd_grad_split_kernel(const AttnBwdArgs A) {
  constexpr int HD = 32 * E;
  __shared__ float sq[NP][HD], sdo[NP][HD], sdq[NP][HD];
  __shared__ float sst[NP][3];
  const int b = blockIdx.x, kvh = blockIdx.y, seg = blockIdx.z, G = A.group;
  const int lane = threadIdx.x & 31, wp = threadIdx.x >> 5;
  pdl_prologue();
  const int qn = min(A.qn[b], A.QT), qbase = A.qbase[b], np = qn * G;
  const int last = qbase + qn - 1, p0 = seg * ATTN_BWD_SEG;
  if (qn <= 0 || p0 > last) return;
  for (int i = wp; i < np; i += AB_WARPS) {
    const int j = i / G, g = i % G, m = b * A.QT + j, h = kvh * G + g;
    const __nv_bfloat16 *qp = A.q + ((static_cast<size_t>(b) * A.n_kv + kvh) * A.qrows + i) * HD;
#pragma unroll
    for (int e = 0; e < E; ++e) {
      sq[i][lane * E + e] = ab_bf(qp[lane * E + e]);
      sdo[i][lane * E + e] = A.dout[(static_cast<size_t>(m) * A.n_kv * G + h) * HD + lane * E + e];
      sdq[i][lane * E + e] = 0.f;
    }
  }
  if (static_cast<int>(threadIdx.x) < np) {                // this pair's statistics over all its segments, in segment order
    const int i = threadIdx.x, nseg = (qbase + i / G) / ATTN_BWD_SEG + 1;
    const float *src = A.part + ((static_cast<size_t>(b) * A.n_kv + kvh) * A.nseg * NP + i) * 3;
    float M = -INFINITY;
    for (int s = 0; s < nseg; ++s) M = fmaxf(M, src[static_cast<size_t>(s) * NP * 3]);
    float L = 0.f, D = 0.f;
    for (int s = 0; s < nseg; ++s) {
      const float *ps = src + static_cast<size_t>(s) * NP * 3;
      const float r = ps[1] > 0.f ? __expf(ps[0] - M) : 0.f;
      L = fmaf(ps[1], r, L); D = fmaf(ps[2], r, D);
    }
    sst[i][0] = M; sst[i][1] = 1.0f / L; sst[i][2] = D / L;
  }
  __syncthreads();
  float dq[NP][E];
#pragma unroll
  for (int i = 0; i < NP; ++i)
#pragma unroll
    for (int e = 0; e < E; ++e) dq[i][e] = 0.f;
  const size_t page_elems = static_cast<size_t>(A.n_kv) * 16 * HD;
  const __nv_bfloat16 *kplane = A.pool + (static_cast<size_t>(A.layer) * 2 + 0) * A.num_pages * page_elems;
  const __nv_bfloat16 *vplane = A.pool + (static_cast<size_t>(A.layer) * 2 + 1) * A.num_pages * page_elems;
  const int p1 = min(p0 + ATTN_BWD_SEG - 1, last);
  for (int p = p0 + wp; p <= p1; p += AB_WARPS) {
    const int page = A.page_table[static_cast<size_t>(b) * A.max_pages_per_seq + (p >> 4)];
    if (page < 0 || page >= A.num_pages) { if (lane == 0) set_status(A.status, ST_BAD_PAGE); continue; }
    const size_t off = static_cast<size_t>(page) * page_elems + (static_cast<size_t>(kvh) * 16 + (p & 15)) * HD;
    float k[E], v[E], dk[E], dv[E];
    ab_load_bf16<E>(kplane + off, lane, k);
    ab_load_bf16<E>(vplane + off, lane, v);
#pragma unroll
    for (int e = 0; e < E; ++e) dk[e] = dv[e] = 0.f;
#pragma unroll
    for (int i = 0; i < NP; ++i) {
      if (i < np && p <= qbase + i / G) {                 // warp-uniform
        float qv[E], dov[E];
#pragma unroll
        for (int e = 0; e < E; ++e) { qv[e] = sq[i][lane * E + e]; dov[e] = sdo[i][lane * E + e]; }
        const float s = ab_dot<E>(qv, k) * A.scale, dp = ab_dot<E>(dov, v);
        const float pr = __expf(s - sst[i][0]) * sst[i][1];
        const float ds = pr * (dp - sst[i][2]) * A.scale;
#pragma unroll
        for (int e = 0; e < E; ++e) {
          dq[i][e] = fmaf(ds, k[e], dq[i][e]);
          dk[e] = fmaf(ds, qv[e], dk[e]);
          dv[e] = fmaf(pr, dov[e], dv[e]);
        }
      }
    }
#pragma unroll
    for (int e = 0; e < E; ++e) {                          // every visible pair's term of this key, from this warp alone
      if (A.dk_fix) {
        fix_add(A.dk_fix + off + lane * E + e, dk[e]);
        fix_add(A.dv_fix + off + lane * E + e, dv[e]);
      } else {
        atomicAdd(A.dk_pool + off + lane * E + e, dk[e]);
        atomicAdd(A.dv_pool + off + lane * E + e, dv[e]);
      }
    }
  }
  for (int w = 0; w < AB_WARPS; ++w) {                 // the warps' partial dq, added in warp order
    if (wp == w) {
#pragma unroll
      for (int i = 0; i < NP; ++i)
        if (i < np) {
#pragma unroll
          for (int e = 0; e < E; ++e) sdq[i][lane * E + e] += dq[i][e];
        }
    }
    __syncthreads();
  }
  for (int t = threadIdx.x; t < np * HD; t += blockDim.x) {
    const int i = t / HD, c = t % HD, j = i / G, g = i % G, m = b * A.QT + j, h = kvh * G + g;
    const size_t o = (static_cast<size_t>(m) * A.n_kv * G + h) * HD + c;
    if (A.dq_fix) fix_add(A.dq_fix + o, sdq[i][c]);
    else atomicAdd(A.dq + o, sdq[i][c]);
  }
}

template <int E, int NP>
cudaError_t launch_split(const AttnBwdArgs &A, cudaStream_t stream) {
  const dim3 grid(A.batch, A.n_kv, A.nseg), blk(AB_WARPS * 32);
  if (cudaError_t e = launch_k(attn_bwd_stats_split_kernel<E, NP>, grid, blk, 0, stream, 1, A); e != cudaSuccess) return e;
  return launch_k(attn_bwd_grad_split_kernel<E, NP>, grid, blk, 0, stream, 1, A);
}

}  // namespace

cudaError_t launch_attention_backward(const AttnBwdArgs &A, cudaStream_t stream) {
  if (A.QT > AB_MAX_ROWS || A.group > AB_MAX_GROUP || (A.hd != 64 && A.hd != 128)) return cudaErrorInvalidValue;
  const int pairs = A.QT * A.group;
  if (A.part && A.nseg > 0 && pairs <= ATTN_BWD_MAX_PAIRS) {
    if (A.hd == 128) return pairs <= 4 ? launch_split<4, 4>(A, stream) : (pairs <= 8 ? launch_split<4, 8>(A, stream) : launch_split<4, 16>(A, stream));
    return pairs <= 4 ? launch_split<2, 4>(A, stream) : (pairs <= 8 ? launch_split<2, 8>(A, stream) : launch_split<2, 16>(A, stream));
  }
  const dim3 g1(A.batch * A.QT, A.n_kv), g2(A.batch, A.n_kv), blk(A.group * 32);
  const size_t dyn = (static_cast<size_t>(2) * A.QT + 2) * A.group * A.hd * sizeof(float);
  if (dyn > 48 * 1024) return cudaErrorInvalidValue;
  if (A.hd == 128) {
    if (cudaError_t e = launch_k(attn_bwd_stats_kernel<4>, g1, blk, 0, stream, 1, A); e != cudaSuccess) return e;
    return launch_k(attn_bwd_grad_kernel<4>, g2, blk, dyn, stream, 1, A);
  }
  if (cudaError_t e = launch_k(attn_bwd_stats_kernel<2>, g1, blk, 0, stream, 1, A); e != cudaSuccess) return e;
  return launch_k(attn_bwd_grad_kernel<2>, g2, blk, dyn, stream, 1, A);
}

}  // namespace gm
