// Fused vocab-wide softmax + speculative rejection sampling + residual resampling (Sec. 2.2, Eq. 1).
//
// One thread-block cluster of 8 CTAs owns one sequence; each CTA owns a contiguous eighth of the
// vocabulary.  Pass 1 streams all 2K+1 logit rows once (128-bit loads) and reduces a running
// (max, sum exp) per row: thread -> warp shuffle -> CTA -> cluster (distributed shared memory), in a
// fixed order, so every CTA ends with bit-identical row statistics.  The K accept tests then need
// only the gathered logits of the draft tokens.  Pass 2 re-reads just the two rows of position a+1
// (still L2-resident), turns max(0, p - q) into 64-bit integer weights trunc(r * 2^44), sums them
// (integer sums do not depend on the reduction order), and the CTA that holds the target quantile
// walks its slice to the token.  With K = 0 the same kernel is the plain draw of the draft phase.
//
// Built without fast-math: the accept test and the weights are IEEE fp32 operations (denormals kept),
// written with explicit round-to-nearest intrinsics so that no contraction can change them between
// the debug dump of p/q and their use.
#include <cooperative_groups.h>

#include "common.cuh"
#include "kernels.h"

namespace cg = cooperative_groups;

namespace gm {

constexpr int SAMP_WARPS = SAMP_THREADS / 32;
constexpr int SAMP_MAX_ROWS = 2 * GM_MAX_K_ + 1;

struct MZ { float m, z; };

__device__ __forceinline__ MZ mz_merge(MZ a, MZ b) {
  const float m = fmaxf(a.m, b.m);
  if (m == -INFINITY) return MZ{m, 0.f};
  return MZ{m, a.z * expf(a.m - m) + b.z * expf(b.m - m)};
}

// softmax probability of a scaled logit given the row statistics: exp(x - max) / Z, both IEEE.
__device__ __forceinline__ float prob_of(float x_scaled, float m, float Z) {
  return __fdiv_rn(expf(__fsub_rn(x_scaled, m)), Z);
}

__device__ __forceinline__ void unpack8(const uint4 &v, float inv_temp, float (&x)[8]) {
  x[0] = __fmul_rn(bf16_lo(v.x), inv_temp); x[1] = __fmul_rn(bf16_hi(v.x), inv_temp);
  x[2] = __fmul_rn(bf16_lo(v.y), inv_temp); x[3] = __fmul_rn(bf16_hi(v.y), inv_temp);
  x[4] = __fmul_rn(bf16_lo(v.z), inv_temp); x[5] = __fmul_rn(bf16_hi(v.z), inv_temp);
  x[6] = __fmul_rn(bf16_lo(v.w), inv_temp); x[7] = __fmul_rn(bf16_hi(v.w), inv_temp);
}

__device__ __forceinline__ void mz_update(MZ &s, const uint4 &v, float inv_temp) {
  float x[8];
  unpack8(v, inv_temp, x);
  float vm = fmaxf(fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3])), fmaxf(fmaxf(x[4], x[5]), fmaxf(x[6], x[7])));
  if (vm > s.m) { s.z *= expf(s.m - vm); s.m = vm; }
  float acc = 0.f;
#pragma unroll
  for (int j = 0; j < 8; ++j) acc += expf(x[j] - s.m);
  s.z += acc;
}

// integer weight of one residual entry
__device__ __forceinline__ unsigned long long weight_of(float p, float q, bool use_q) {
  const float r = use_q ? __fsub_rn(p, q) : p;
  return r > 0.f ? __float2ull_rz(__fmul_rn(r, 17592186044416.0f /* 2^44 */)) : 0ull;
}

__global__ void __cluster_dims__(SAMP_CLUSTER, 1, 1) __launch_bounds__(SAMP_THREADS)
sampler_kernel(const SamplerArgs A) {
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = static_cast<int>(cluster.block_rank());
  const int b = blockIdx.x / SAMP_CLUSTER;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int K = A.K, V = A.V, R = 2 * K + 1;

  extern __shared__ __align__(16) unsigned char dyn_smem[];
  unsigned long long *vecsum = reinterpret_cast<unsigned long long *>(dyn_smem);   // [vpc]

  __shared__ MZ warp_mz[SAMP_MAX_ROWS][SAMP_WARPS];
  __shared__ MZ local_mz[SAMP_MAX_ROWS];          // this CTA's slice statistics (read by peers)
  __shared__ MZ row_mz[SAMP_MAX_ROWS];            // whole-row statistics
  __shared__ unsigned long long warp_w[SAMP_WARPS];
  __shared__ unsigned long long local_w;          // this CTA's integer mass (read by peers)
  __shared__ unsigned long long scan_w[SAMP_WARPS];
  __shared__ int local_cand;                      // argmax fallback candidate (read by peers)
  __shared__ int sh_a, sh_tok;

  const int nvec_total = V >> 3;
  const int vpc = (nvec_total + SAMP_CLUSTER - 1) / SAMP_CLUSTER;
  const int v_lo = min(rank * vpc, nvec_total);
  const int n = min(v_lo + vpc, nvec_total) - v_lo;

  const __nv_bfloat16 *tgt = A.target_logits + static_cast<size_t>(b) * A.tgt_bstride;
  const __nv_bfloat16 *drf = A.draft_logits ? A.draft_logits + static_cast<size_t>(b) * A.drf_bstride : nullptr;
  auto row_ptr = [&](int r) -> const uint4 * {
    const __nv_bfloat16 *p = r <= K ? tgt + static_cast<size_t>(r) * V : drf + static_cast<size_t>(r - K - 1) * V;
    return reinterpret_cast<const uint4 *>(p) + v_lo;
  };

  // ---- pass 1: (max, sum exp) of every row over this CTA's slice ------------------------------------
  for (int r = 0; r < R; ++r) {
    const uint4 *row = row_ptr(r);
    MZ s{-INFINITY, 0.f};
    for (int i0 = tid; i0 < n; i0 += 4 * SAMP_THREADS) {
      uint4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * SAMP_THREADS;
        if (i < n) v[u] = __ldg(row + i);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (i0 + u * SAMP_THREADS < n) mz_update(s, v[u], A.inv_temp);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      MZ t{__shfl_xor_sync(0xffffffffu, s.m, o), __shfl_xor_sync(0xffffffffu, s.z, o)};
      // order the operands by lane so both partners compute the identical expression
      s = (lane & o) ? mz_merge(t, s) : mz_merge(s, t);
    }
    if (lane == 0) warp_mz[r][warp] = s;
  }
  __syncthreads();
  if (tid < R) {
    MZ s = warp_mz[tid][0];
    for (int w = 1; w < SAMP_WARPS; ++w) s = mz_merge(s, warp_mz[tid][w]);
    local_mz[tid] = s;
  }
  cluster.sync();
  if (tid < R) {
    MZ s = *cluster.map_shared_rank(&local_mz[tid], 0);
    for (int c = 1; c < SAMP_CLUSTER; ++c) s = mz_merge(s, *cluster.map_shared_rank(&local_mz[tid], c));
    row_mz[tid] = s;
  }
  __syncthreads();

  // ---- optional dump of the probabilities the decisions use ------------------------------------------
  if (A.dbg_p != nullptr || A.dbg_q != nullptr) {
    for (int r = 0; r < R; ++r) {
      float *dst = r <= K ? (A.dbg_p ? A.dbg_p + static_cast<size_t>(b) * A.tgt_bstride + static_cast<size_t>(r) * V : nullptr)
                          : (A.dbg_q ? A.dbg_q + static_cast<size_t>(b) * A.drf_bstride + static_cast<size_t>(r - K - 1) * V : nullptr);
      if (dst == nullptr) continue;
      const uint4 *row = row_ptr(r);
      const MZ st = row_mz[r];
      for (int i = tid; i < n; i += SAMP_THREADS) {
        float x[8];
        unpack8(__ldg(row + i), A.inv_temp, x);
#pragma unroll
        for (int j = 0; j < 8; ++j) dst[static_cast<size_t>(v_lo + i) * 8 + j] = prob_of(x[j], st.m, st.z);
      }
    }
  }

  // ---- accept tests (every CTA redundantly; identical inputs give identical results) ---------------
  if (tid == 0) {
    int a = 0;
    for (; a < K; ++a) {
      int d = A.draft_tok[static_cast<size_t>(b) * A.tok_in_stride + a];
      if (d < 0 || d >= V) { set_status(A.status, ST_BAD_TOKEN); break; }
      const float xp = __fmul_rn(__bfloat162float(tgt[static_cast<size_t>(a) * V + d]), A.inv_temp);
      const float xq = __fmul_rn(__bfloat162float(drf[static_cast<size_t>(a) * V + d]), A.inv_temp);
      const float p = prob_of(xp, row_mz[a].m, row_mz[a].z);
      const float q = prob_of(xq, row_mz[K + 1 + a].m, row_mz[K + 1 + a].z);
      const uint32_t u24 = A.u24 ? A.u24[static_cast<size_t>(b) * A.u_stride + a]
                                 : philox_u24(A.seed, A.step, b, A.slot_accept + a);
      const float uq = __fmul_rn(__fmul_rn(static_cast<float>(u24), 5.9604644775390625e-8f /* 2^-24 */), q);
      if (!(p >= q || uq < p)) break;
    }
    sh_a = a;
  }
  __syncthreads();
  const int a = sh_a;

  // ---- pass 2: integer weights of position a+1 and the draw -----------------------------------------
  const uint4 *prow = row_ptr(a);
  const uint4 *qrow = a < K ? row_ptr(K + 1 + a) : nullptr;
  const MZ ps = row_mz[a];
  const MZ qs = a < K ? row_mz[K + 1 + a] : MZ{0.f, 1.f};
  bool use_q = a < K;
  unsigned long long Wc[SAMP_CLUSTER];
  unsigned long long W = 0;
  for (int attempt = 0; attempt < 2; ++attempt) {
    unsigned long long tsum = 0;
    for (int i = tid; i < n; i += SAMP_THREADS) {
      float xp[8], xq[8];
      unpack8(__ldg(prow + i), A.inv_temp, xp);
      if (use_q) unpack8(__ldg(qrow + i), A.inv_temp, xq);
      unsigned long long s = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j)
        s += weight_of(prob_of(xp[j], ps.m, ps.z), use_q ? prob_of(xq[j], qs.m, qs.z) : 0.f, use_q);
      vecsum[i] = s;
      tsum += s;
    }
    tsum = warp_sum_u64(tsum);
    if (lane == 0) warp_w[warp] = tsum;
    __syncthreads();
    if (tid == 0) {
      unsigned long long s = 0;
      for (int w = 0; w < SAMP_WARPS; ++w) s += warp_w[w];
      local_w = s;
    }
    cluster.sync();
    W = 0;
#pragma unroll
    for (int c = 0; c < SAMP_CLUSTER; ++c) { Wc[c] = *cluster.map_shared_rank(&local_w, c); W += Wc[c]; }
    cluster.sync();                         // every CTA has read before anyone overwrites local_w
    if (W != 0 || !use_q) break;
    use_q = false;                          // residual mass underflowed: draw from p instead
    if (rank == 0 && tid == 0) set_status(A.status, ST_ZERO_RESID);
  }

  const uint32_t u_final = A.u24 ? A.u24[static_cast<size_t>(b) * A.u_stride + K]
                                 : philox_u24(A.seed, A.step, b, A.slot_final);
  int winner = -1;                          // CTA that owns the quantile
  unsigned long long t_local = 0;
  if (W != 0) {
    // t = floor(u24 * W / 2^24) without a 128-bit product: W = Wh 2^24 + Wl
    const unsigned long long t = static_cast<unsigned long long>(u_final) * (W >> 24) +
                                 ((static_cast<unsigned long long>(u_final) * (W & 0xFFFFFFull)) >> 24);
    unsigned long long pre = 0;
#pragma unroll
    for (int c = 0; c < SAMP_CLUSTER; ++c) {
      if (winner < 0 && t < pre + Wc[c]) { winner = c; t_local = t - pre; }
      pre += Wc[c];
    }
  }

  if (W == 0) {
    // no mass at all (cannot happen for a softmax of finite logits): lowest index of the row maximum
    if (tid == 0) local_cand = 0x7fffffff;
    __syncthreads();
    for (int i = tid; i < n; i += SAMP_THREADS) {
      float x[8];
      unpack8(__ldg(prow + i), A.inv_temp, x);
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (x[j] == ps.m) atomicMin(&local_cand, (v_lo + i) * 8 + j);
    }
    cluster.sync();
    if (rank == 0 && tid == 0) {
      int best = 0x7fffffff;
      for (int c = 0; c < SAMP_CLUSTER; ++c) best = min(best, *cluster.map_shared_rank(&local_cand, c));
      if (best == 0x7fffffff) best = 0;
      sh_tok = best;
      set_status(A.status, ST_ZERO_MASS);
    }
    winner = 0;
    __syncthreads();
  } else if (rank == winner) {
    // block-wide search of t_local in the inclusive prefix sums of vecsum[0..n)
    const int seg = (n + SAMP_THREADS - 1) / SAMP_THREADS;
    const int lo = min(tid * seg, n), hi = min(lo + seg, n);
    unsigned long long mine = 0;
    for (int i = lo; i < hi; ++i) mine += vecsum[i];
    unsigned long long incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += up;
    }
    if (lane == 31) scan_w[warp] = incl;
    __syncthreads();
    unsigned long long base = 0;
    for (int w = 0; w < warp; ++w) base += scan_w[w];
    const unsigned long long excl = base + incl - mine;
    if (mine != 0 && t_local >= excl && t_local < excl + mine) {
      unsigned long long rem = t_local - excl;
      int iv = lo;
      while (rem >= vecsum[iv]) { rem -= vecsum[iv]; ++iv; }     // stops inside [lo, hi): rem < mine
      float xp[8], xq[8];
      unpack8(__ldg(prow + iv), A.inv_temp, xp);
      if (use_q) unpack8(__ldg(qrow + iv), A.inv_temp, xq);
      int tok = (v_lo + iv) * 8 + 7;
      for (int j = 0; j < 8; ++j) {
        const unsigned long long w =
            weight_of(prob_of(xp[j], ps.m, ps.z), use_q ? prob_of(xq[j], qs.m, qs.z) : 0.f, use_q);
        if (rem < w) { tok = (v_lo + iv) * 8 + j; break; }
        rem -= w;
      }
      sh_tok = tok;
    }
    __syncthreads();
  }

  // ---- outputs and state commit (by the CTA that found the token) -----------------------------------
  if (rank == winner) {
    const int tok = sh_tok;
    if (tid == 0) {
      A.next_token[static_cast<size_t>(b) * A.tok_out_stride] = tok;
      if (A.accept_len) A.accept_len[b] = a;
    }
    if (A.commit) {
      const int kp1 = A.max_k + 1;
      if (tid == 0) {
        A.kv_len[b] += a + 1;
        A.pending_n[b] = a + 1;
      }
      if (tid <= a)
        A.pending_tok[static_cast<size_t>(b) * kp1 + tid] =
            tid < a ? A.draft_tok[static_cast<size_t>(b) * A.tok_in_stride + tid] : tok;
      // pending_hidden rows 0..a <- target_hidden rows 0..a   (d_model % 8 == 0)
      const int vec_per_row = A.d_model >> 3;
      const uint4 *src = reinterpret_cast<const uint4 *>(A.target_hidden + static_cast<size_t>(b) * (K + 1) * A.d_model);
      uint4 *dst = reinterpret_cast<uint4 *>(A.pending_hidden + static_cast<size_t>(b) * kp1 * A.d_model);
      for (int i = tid; i < (a + 1) * vec_per_row; i += SAMP_THREADS) dst[i] = src[i];
    }
  }
  cluster.sync();                            // keep shared memory alive until every peer has read it
}

cudaError_t launch_sampler(const SamplerArgs &A, int batch, cudaStream_t stream) {
  const int nvec_total = A.V >> 3;
  const int vpc = (nvec_total + SAMP_CLUSTER - 1) / SAMP_CLUSTER;
  const size_t dyn = static_cast<size_t>(vpc) * sizeof(unsigned long long);
  static size_t configured = 0;
  if (dyn > configured) {
    cudaError_t e = cudaFuncSetAttribute(sampler_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(dyn));
    if (e != cudaSuccess) return e;
    configured = dyn;
  }
  sampler_kernel<<<batch * SAMP_CLUSTER, SAMP_THREADS, dyn, stream>>>(A);
  return cudaGetLastError();
}

}  // namespace gm
