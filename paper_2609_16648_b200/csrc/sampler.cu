// Fused vocab-wide softmax + speculative rejection sampling + residual resampling (Sec. 2.2, Eq. 1).
//
// One thread-block cluster of 8 CTAs owns one sequence; each CTA owns a contiguous eighth of the
// vocabulary.  Positions are walked in order: one thread issues bulk asynchronous copies of the CTA's
// slices of the rows p_k and q_k into a two-stage shared-memory ring, the warps reduce a (max, sum exp)
// pair per row from shared memory with 128-bit reads - first the maximum (packed bf16), then the
// exponentials against it (one multiply-add, one ex2 and one add per logit); thread -> warp shuffle ->
// CTA -> cluster (distributed shared memory) merges run in a fixed order, so every CTA ends with
// bit-identical row statistics - and accept test k needs only the gathered logits of draft k.  The walk
// stops at the first rejection (or at the bonus position): rows of later positions are never read, and the
// two rows of position a+1 are still in the ring, so the resampling pass turns max(0, p - q) into 64-bit
// integer weights trunc(r * 2^44) straight from shared memory, sums them (integer sums do not depend on
// the reduction order), and the CTA that holds the target quantile walks its slice to the token.  With
// K = 0 the same kernel is the plain draw of the draft phase.
//
// Arithmetic.  Everything is fp32 in the base-2 domain with s = log2(e) / T: the row maximum m is taken on
// the raw bf16 logits (packed bf16x2 max, exact), c = -fl(m * s), and
//     p(x) = ex2(fma(x, s, c)) * (1 / Z),   Z = sum ex2(fma(x, s, c))
// with the hardware ex2.approx (2 ulp): per logit one unpack, one fused multiply-add, one ex2, one add.
// One device function computes p wherever it is needed (accept test, weights, debug dump), with explicit
// round-to-nearest intrinsics, so the dumped probabilities are exactly the ones the decisions used.  The
// accept test and the weights are IEEE operations on those values.
#include <cooperative_groups.h>

#include "sampler_common.cuh"

namespace cg = cooperative_groups;

namespace gm {

__global__ void __cluster_dims__(SAMP_CLUSTER, 1, 1) __launch_bounds__(SAMP_THREADS, 2)
sampler_kernel(const SamplerArgs A) {
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = static_cast<int>(cluster.block_rank());
  const int b = blockIdx.x / SAMP_CLUSTER;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int K = A.K, V = A.V, R = 2 * K + 1;
  const float s = A.inv_temp * 1.4426950408889634f;            // logits -> base-2 exponents
  pdl_prologue();
  if (A.finished && A.finished[b]) {               // the row sits out: the whole cluster leaves before any barrier
    if (rank == 0 && tid == 0) {
      if (A.accept_len) A.accept_len[b] = 0;
      A.next_token[static_cast<size_t>(b) * A.tok_out_stride] = A.accept_len ? -1 : 0;   // a plain draw leaves a valid id
    }
    return;
  }

  const int nvec_total = V >> 3;
  const int vpc = (nvec_total + SAMP_CLUSTER - 1) / SAMP_CLUSTER;
  const int v_lo = min(rank * vpc, nvec_total);
  const int n = min(v_lo + vpc, nvec_total) - v_lo;
  const uint32_t stage_b = (static_cast<uint32_t>(vpc) * 16u + 127u) & ~127u;

  extern __shared__ __align__(128) unsigned char dyn_smem[];
  const uint4 *stage[2] = {reinterpret_cast<const uint4 *>(dyn_smem), reinterpret_cast<const uint4 *>(dyn_smem + stage_b)};
  unsigned long long *vecsum = reinterpret_cast<unsigned long long *>(dyn_smem + 2 * stage_b);   // [vpc]
  __shared__ uint64_t full[2];

  __shared__ MZ warp_mz[SAMP_MAX_ROWS][SAMP_WARPS];
  __shared__ MZ local_mz[2][2];                   // this CTA's slice statistics (read by peers), double-buffered by call parity
  __shared__ MZ row_mz[SAMP_MAX_ROWS];            // whole-row statistics: .m holds c = -fl(max * s), .z holds 1 / Z
  __shared__ unsigned long long warp_w[SAMP_WARPS];
  __shared__ unsigned long long local_w;          // this CTA's integer mass (read by peers)
  __shared__ unsigned long long scan_w[SAMP_WARPS];
  __shared__ int local_cand;                      // argmax fallback candidate (read by peers)
  __shared__ int sh_a, sh_tok;

  const __nv_bfloat16 *tgt = A.target_logits + static_cast<size_t>(b) * A.tgt_bstride;
  const __nv_bfloat16 *drf = A.draft_logits ? A.draft_logits + static_cast<size_t>(b) * A.drf_bstride : nullptr;
  auto row_ptr = [&](int r) -> const uint4 * {
    const __nv_bfloat16 *p = r <= K ? tgt + static_cast<size_t>(r) * V : drf + static_cast<size_t>(r - K - 1) * V;
    return reinterpret_cast<const uint4 *>(p) + v_lo;
  };

  // ---- shared-memory ring: stage 0 holds the target row, stage 1 the draft row of the position in flight ----------
  if (tid == 0) {
    mbar_init(&full[0], 1);
    mbar_init(&full[1], 1);
    mbar_fence_init();
  }
  __syncthreads();
  uint32_t uses[2] = {0u, 0u};                    // completed phases of each stage's barrier (parity = uses & 1)
  auto issue = [&](int st_i, const uint4 *src) {  // thread 0 only
    if (n > 0) {
      mbar_expect_tx(&full[st_i], static_cast<uint32_t>(n) * 16u);
      bulk_load(const_cast<uint4 *>(stage[st_i]), src, static_cast<uint32_t>(n) * 16u, &full[st_i]);
    }
  };
  __shared__ int sh_alive;
  if (tid == 0) sh_alive = 1;
  bool alive = true;                              // false after a bounded wait expired: finish without touching the data
  // One thread polls the mbarrier (bounded); everybody else sleeps at the CTA barrier instead of spinning.
  auto wait_stage = [&](int st_i) {
    if (tid == 0 && n > 0 && sh_alive && !mbar_wait(&full[st_i], uses[st_i] & 1u)) {
      sh_alive = 0;
      set_status(A.status, ST_TIMEOUT);
    }
    ++uses[st_i];
    __syncthreads();
    alive = sh_alive != 0;
  };
  const uint32_t NEG_INF2 = 0xff80ff80u;          // two bf16 -inf
  // (max, sum 2^((x - max) s)) of the row slice in `buf`, per warp, into warp_mz[slot]
  auto slice_stats = [&](const uint4 *buf, int slot) {
    MZ st{-INFINITY, 0.f};
    if (alive && tid < n) {
      uint32_t m2 = NEG_INF2;
      for (int i = tid; i < n; i += SAMP_THREADS) {
        const uint4 v = buf[i];
        m2 = bmax2(bmax2(m2, bmax2(v.x, v.y)), bmax2(v.z, v.w));
      }
      const float mx = fmaxf(bf16_lo(m2), bf16_hi(m2));
      const float c = -mx * s;
      float acc = 0.f;
      if (mx != -INFINITY) {                      // a thread that saw only -inf (masked-out) logits contributes nothing
        for (int i = tid; i < n; i += SAMP_THREADS) {
          float x[8];
          unpack8(buf[i], x);
#pragma unroll
          for (int j = 0; j < 8; ++j) acc += ex2(fmaf(x[j], s, c));
        }
      }
      st = MZ{mx, acc};
    }
    const float wm = warp_max(st.m);              // butterfly: every lane ends with the same maximum
    float z = wm == -INFINITY ? 0.f : st.z * ex2((st.m - wm) * s);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);   // commutative pairs: same sum on every lane
    if (lane == 0) warp_mz[slot][warp] = MZ{wm, z};
  };
  // whole-row (c, 1 / Z) of slots 0..nslots-1 from the slice statistics: warps, then the 8 CTAs in rank order, so
  // that every CTA of the cluster holds bit-identical values in row_mz
  int stats_calls = 0;                            // same sequence in every CTA of the cluster
  auto finish_stats = [&](int nslots) {
    MZ *mine = local_mz[stats_calls & 1];         // a buffer is rewritten two calls later: the call in between has a
    ++stats_calls;                                // cluster barrier that every peer passes only after reading it
    __syncthreads();                              // also: every warp has finished reading the stages
    if (tid < nslots) {
      MZ st = warp_mz[tid][0];
      for (int w = 1; w < SAMP_WARPS; ++w) st = mz_merge(st, warp_mz[tid][w], s);
      mine[tid] = st;
    }
    cluster.sync();
    if (tid < nslots) {
      MZ st = *cluster.map_shared_rank(&mine[tid], 0);
      for (int c = 1; c < SAMP_CLUSTER; ++c) st = mz_merge(st, *cluster.map_shared_rank(&mine[tid], c), s);
      row_mz[tid] = MZ{-st.m * s, __frcp_rn(st.z)};
    }
    __syncthreads();
  };

  // ---- optional dump of the probabilities (debug): every row through the same statistics code ---------------------
  if (A.dbg_p != nullptr || A.dbg_q != nullptr) {
    for (int r = 0; r < R; ++r) {
      float *dst = r <= K ? (A.dbg_p ? A.dbg_p + static_cast<size_t>(b) * A.tgt_bstride + static_cast<size_t>(r) * V : nullptr)
                          : (A.dbg_q ? A.dbg_q + static_cast<size_t>(b) * A.drf_bstride + static_cast<size_t>(r - K - 1) * V : nullptr);
      if (tid == 0) { fence_proxy_async(); issue(0, row_ptr(r)); }
      wait_stage(0);
      slice_stats(stage[0], 0);
      finish_stats(1);
      const MZ st = row_mz[0];
      if (dst != nullptr && alive)
        for (int i = tid; i < n; i += SAMP_THREADS) {
          float x[8];
          unpack8(stage[0][i], x);
#pragma unroll
          for (int j = 0; j < 8; ++j) dst[static_cast<size_t>(v_lo + i) * 8 + j] = prob_of(x[j], s, st.m, st.z);
        }
      __syncthreads();
    }
  }

  // ---- positions in order: statistics of (p_k, q_k), accept test k; stop at the first rejection -----------------
  // The rows of the position where the walk stops are then still in the ring: the resampling pass reads them from
  // shared memory, and the rows of later positions are never loaded.
  int a = K;
  for (int k = 0; k <= K; ++k) {
    const bool bonus = k == K;
    if (tid == 0) {
      fence_proxy_async();                        // order the generic reads of the stages before the asynchronous overwrite
      issue(0, row_ptr(k));
      if (!bonus) issue(1, row_ptr(K + 1 + k));
    }
    wait_stage(0);
    if (!bonus) wait_stage(1);
    slice_stats(stage[0], 0);
    if (!bonus) slice_stats(stage[1], 1);
    finish_stats(bonus ? 1 : 2);
    if (bonus) break;
    if (tid == 0) {                               // every CTA redundantly, identical inputs
      bool ok = false;
      const int d = A.draft_tok[static_cast<size_t>(b) * A.tok_in_stride + k];
      if (d < 0 || d >= V) {
        set_status(A.status, ST_BAD_TOKEN);
      } else {
        const float xp = __bfloat162float(tgt[static_cast<size_t>(k) * V + d]);
        const float xq = __bfloat162float(drf[static_cast<size_t>(k) * V + d]);
        const float p = prob_of(xp, s, row_mz[0].m, row_mz[0].z);
        const float q = prob_of(xq, s, row_mz[1].m, row_mz[1].z);
        const uint32_t u24 = A.u24 ? A.u24[static_cast<size_t>(b) * A.u_stride + k]
                                   : philox_u24(A.seed, step_of(A), b, A.slot_accept + k);
        const float uq = __fmul_rn(__fmul_rn(static_cast<float>(u24), 5.9604644775390625e-8f /* 2^-24 */), q);
        ok = p >= q || uq < p;
      }
      sh_a = ok ? 1 : 0;
    }
    __syncthreads();
    if (!sh_a) { a = k; break; }
  }

  // ---- resampling at position a+1 from the rows in the ring: integer weights and the draw -------------------------
  const MZ ps = row_mz[0];
  const MZ qs = a < K ? row_mz[1] : MZ{0.f, 1.f};
  bool use_q = a < K;
  unsigned long long Wc[SAMP_CLUSTER];
  unsigned long long W = 0;
  for (int attempt = 0; attempt < 2; ++attempt) {
    unsigned long long tsum = 0;
    for (int i = tid; i < n && alive; i += SAMP_THREADS) {
      float xp[8], xq[8];
      unpack8(stage[0][i], xp);
      if (use_q) unpack8(stage[1][i], xq);
      unsigned long long sm = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j)
        sm += weight_of(prob_of(xp[j], s, ps.m, ps.z), use_q ? prob_of(xq[j], s, qs.m, qs.z) : 0.f, use_q);
      vecsum[i] = sm;
      tsum += sm;
    }
    tsum = warp_sum_u64(tsum);
    if (lane == 0) warp_w[warp] = tsum;
    __syncthreads();
    if (tid == 0) {
      unsigned long long sm = 0;
      for (int w = 0; w < SAMP_WARPS; ++w) sm += warp_w[w];
      local_w = sm;
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
                                 : philox_u24(A.seed, step_of(A), b, A.slot_final);
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
      unpack8(stage[0][i], x);
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (-x[j] * s == ps.m) atomicMin(&local_cand, (v_lo + i) * 8 + j);
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
      unpack8(stage[0][iv], xp);
      if (use_q) unpack8(stage[1][iv], xq);
      int tok = (v_lo + iv) * 8 + 7;
      for (int j = 0; j < 8; ++j) {
        const unsigned long long w =
            weight_of(prob_of(xp[j], s, ps.m, ps.z), use_q ? prob_of(xq[j], s, qs.m, qs.z) : 0.f, use_q);
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
  const size_t stage_b = (static_cast<size_t>(vpc) * 16 + 127) & ~size_t(127);
  const size_t dyn = 2 * stage_b + static_cast<size_t>(vpc) * sizeof(unsigned long long);
  if (dyn > 227 * 1024 - 4096) return cudaErrorInvalidValue;      // vocabulary too large for the shared-memory ring
  static SmemConfigured configured;
  if (cudaError_t e = ensure_dyn_smem(sampler_kernel, dyn, configured); e != cudaSuccess) return e;
  return launch_k(sampler_kernel, dim3(batch * SAMP_CLUSTER), dim3(SAMP_THREADS), dyn, stream, 1, A);
}

}  // namespace gm
