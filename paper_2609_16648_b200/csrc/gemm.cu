// Dense projections out[M, N] = x[M, K] * w[N, K]^T (bf16 operands, fp32 accumulation).
//
// gemm_tc_kernel (the product path).  The step's projections have few rows (M = batch * (K+1)
// <= a few hundred tokens) and many output features, so the operands are swapped onto the tensor
// core: a CTA takes 128 output features as the MMA's M extent (one TMEM lane per feature) and up
// to 256 tokens as its N extent, and streams its 128 x K weight slab exactly once.  Warp 0 (one
// elected thread) is the TMA producer filling a ring of 128-byte-swizzled stages (64 K-elements per
// stage: a 128 x 64 weight box and a T x 64 activation box); warp 1 owns the tensor memory
// allocation and one of its threads issues tcgen05.mma (four K=16 instructions per stage),
// releasing each stage with tcgen05.commit; warps 2-9 read the fp32 accumulator out of tensor
// memory with tcgen05.ld once the last commit lands (two warps per TMEM lane quadrant, alternating
// 16-column chunks), and all 16 warps run the reduction and the epilogue.
//
// Split-K without a trip through HBM.  Projections with few output tiles (N = d_model gives 20)
// are cut along K over blockIdx.z, and the CTAs of one output tile form a thread-block cluster.
// Every CTA parks its accumulator in its own shared memory (the pipeline stages are free by
// then), the cluster synchronises, and each CTA sums one slice of the tile's tokens over all
// peers through distributed shared memory in rank order (so the result does not depend on
// timing) and applies the epilogue: store bf16 / fp32, add into the fp32 residual stream, or
// SwiGLU on interleaved gate/up rows.  Every wait is bounded; on expiry the kernel records
// ST_TIMEOUT, still meets every barrier and frees its tensor memory.
//
// gemm_pair_kernel: the same projection on pairs of CTAs (tcgen05 cta_group::2) for full waves of one-slice tiles;
// gemm_pair_split_kernel: pairs with K slices (cluster 2 x slices) for split projections.  Both described at the kernels.
//
// gemm_simple_kernel: a plain warp-level mma.sync version with the same epilogues, kept as an
// independent on-device cross-check and for shapes the tcgen05 kernel does not take.
#include <cooperative_groups.h>

#include <cstdlib>
#include "common.cuh"
#include "kernels.h"

namespace cg = cooperative_groups;

namespace gm {

constexpr int GT_BN = 128;            // output features per MMA (its M extent); a CTA owns wt = 1 or 2 such sub-tiles
constexpr int GT_BK = 64;             // K elements per stage (one 128-byte swizzle row)
constexpr int GT_THREADS = 512;     // warp 0: TMA producer, warp 1: MMA issuer, warps 2-9: TMEM readers; all 16 warps reduce + store
constexpr int GT_SMEM_BUDGET = 200 * 1024;

static int gt_stages(int block_t, int wt) {
  int s = GT_SMEM_BUDGET / (wt * GT_BN * 128 + block_t * 128);
  return s > 8 ? 8 : s;
}
static size_t gt_smem(int block_t, int wt) {
  size_t pipe = static_cast<size_t>(gt_stages(block_t, wt)) * (wt * GT_BN * 128 + block_t * 128);
  const size_t park = static_cast<size_t>(block_t) * GT_BN * 4;      // one accumulator parked as fp32 [T][128]
  if (park > pipe) pipe = park;
  return pipe + 1024 + 256;
}

// Epilogue on four consecutive features n..n+3 of token row m.
__device__ __forceinline__ void epilogue4(const GemmArgs &A, int m, int n, float4 v) {
  if (A.epi == EPI_SWIGLU_BF16) {           // (gate, up, gate, up) -> two outputs
    if (n + 1 >= A.N) return;
    const float a0 = __fdividef(v.x, 1.f + __expf(-v.x)) * v.y;        // fast reciprocal: the result is rounded to bf16
    __nv_bfloat16 *out = reinterpret_cast<__nv_bfloat16 *>(A.out) + static_cast<size_t>(m) * A.ldo + (n >> 1);
    if (n + 3 < A.N) {
      const float a1 = __fdividef(v.z, 1.f + __expf(-v.z)) * v.w;
      *reinterpret_cast<uint32_t *>(out) = pack_bf16(a0, a1);
    } else {
      out[0] = __float2bfloat16(a0);
    }
    return;
  }
  const float e[4] = {v.x, v.y, v.z, v.w};
  if (A.epi == EPI_STORE_BF16) {
    __nv_bfloat16 *out = reinterpret_cast<__nv_bfloat16 *>(A.out) + static_cast<size_t>(m) * A.ldo + n;
    if (n + 3 < A.N && (A.ldo & 3) == 0) {
      uint2 o;
      o.x = pack_bf16(v.x, v.y);
      o.y = pack_bf16(v.z, v.w);
      *reinterpret_cast<uint2 *>(out) = o;
    } else {
      for (int i = 0; i < 4 && n + i < A.N; ++i) out[i] = __float2bfloat16(e[i]);
    }
    return;
  }
  float *out = reinterpret_cast<float *>(A.out) + static_cast<size_t>(m) * A.ldo + n;
  if (n + 3 < A.N && (A.ldo & 3) == 0) {
    float4 o = v;
    if (A.epi == EPI_ADD_F32) {
      const float4 r = *reinterpret_cast<const float4 *>(out);
      o.x += r.x; o.y += r.y; o.z += r.z; o.w += r.w;
    }
    *reinterpret_cast<float4 *>(out) = o;
  } else {
    for (int i = 0; i < 4 && n + i < A.N; ++i) out[i] = (A.epi == EPI_ADD_F32 ? out[i] : 0.f) + e[i];
  }
}

// EPI_QKV_ROPE: one warp holds the 128 features [n0, n0 + 128) of token row m (lane l: features 4l .. 4l + 3), i.e. one
// head of 128 or two heads of 64.  The value is rounded to bf16 first, exactly as the stand-alone projection stores it;
// then bias, the head's RMSNorm, the rotary embedding (the partner half of a head sits hd/8 lanes away), and the
// destination: the attention kernel's query layout, or the sequence's key / value page.
__device__ __forceinline__ void rope_epilogue(const GemmArgs &G, int m, int n0, int lane, float4 acc) {
  const RopeAppendArgs &A = G.rope;
  const int hd = A.hd, half = hd >> 1, lph = hd >> 2;              // lanes per head
  const int b = m / A.QT, j = m % A.QT;
  const int n = n0 + 4 * lane, h = n / hd, fh = n % hd;
  const int group = A.n_q / A.n_kv;
  const int qn = A.qn[b];
  float x[4] = {__bfloat162float(__float2bfloat16(acc.x)), __bfloat162float(__float2bfloat16(acc.y)),
                __bfloat162float(__float2bfloat16(acc.z)), __bfloat162float(__float2bfloat16(acc.w))};
  if (j >= qn) {                           // padding row: zero its query rows, append nothing
    if (h < A.n_q)
      *reinterpret_cast<uint2 *>(A.qbuf + ((static_cast<size_t>(b) * A.n_kv + h / group) * A.qrows + j * group + h % group) * hd + fh) =
          make_uint2(0u, 0u);
    return;
  }
  const int pos = A.qbase[b] + j;
  if (A.bias) {
    const uint2 bv = *reinterpret_cast<const uint2 *>(A.bias + n);
    x[0] += bf16_lo(bv.x); x[1] += bf16_hi(bv.x); x[2] += bf16_lo(bv.y); x[3] += bf16_hi(bv.y);
  }
  const bool is_v = h >= A.n_q + A.n_kv;
  {
    // RMSNorm over the head dimension, before the rotation (the reduction runs in every lane: a warp may hold two heads)
    float ss = x[0] * x[0] + x[1] * x[1] + x[2] * x[2] + x[3] * x[3];
    for (int off = lph >> 1; off >= 1; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
    const __nv_bfloat16 *nw = is_v ? nullptr : (h < A.n_q ? A.qnorm : A.knorm);
    if (nw) {
      const float inv = rsqrtf(ss / static_cast<float>(hd) + A.eps);
      const uint2 wv = *reinterpret_cast<const uint2 *>(nw + fh);
      x[0] = x[0] * inv * bf16_lo(wv.x); x[1] = x[1] * inv * bf16_hi(wv.x);
      x[2] = x[2] * inv * bf16_lo(wv.y); x[3] = x[3] * inv * bf16_hi(wv.y);
    }
  }
  // the other half of the head (every lane takes part in the exchange, value heads too)
  float xp[4];
#pragma unroll
  for (int t = 0; t < 4; ++t) xp[t] = __shfl_xor_sync(0xffffffffu, x[t], lph >> 1);
  float y[4] = {x[0], x[1], x[2], x[3]};
  if (!is_v) {
    const bool lower = fh < half;
    const float2 *cs = A.rope + static_cast<size_t>(pos) * half + (lower ? fh : fh - half);
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const float2 c = cs[t];
      y[t] = lower ? x[t] * c.x - xp[t] * c.y : x[t] * c.x + xp[t] * c.y;
    }
  }
  const uint2 o = make_uint2(pack_bf16(y[0], y[1]), pack_bf16(y[2], y[3]));
  if (h < A.n_q) {
    *reinterpret_cast<uint2 *>(A.qbuf + ((static_cast<size_t>(b) * A.n_kv + h / group) * A.qrows + j * group + h % group) * hd + fh) = o;
    return;
  }
  const int page = A.page_table[static_cast<size_t>(b) * A.max_pages_per_seq + (pos >> 4)];
  if (page < 0 || page >= A.num_pages) {
    if (lane == 0) set_status(A.status, ST_BAD_PAGE);
    return;
  }
  const int kvh = is_v ? h - A.n_q - A.n_kv : h - A.n_q;
  const size_t page_elems = static_cast<size_t>(A.n_kv) * 16 * hd;
  __nv_bfloat16 *dst = A.pool + ((static_cast<size_t>(A.layer) * 2 + (is_v ? 1 : 0)) * A.num_pages + page) * page_elems +
                       (static_cast<size_t>(kvh) * 16 + (pos & 15)) * hd + fh;
  *reinterpret_cast<uint2 *>(dst) = o;
}

template <int MINB>
__global__ void __launch_bounds__(GT_THREADS, MINB)
gemm_tc_kernel(const __grid_constant__ GemmArgs A, const int nstages) {
  extern __shared__ unsigned char gt_smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(gt_smem_raw) + 1023) & ~uintptr_t(1023));
  const int T = A.block_t, wt = A.wtiles;
  const int a_bytes = wt * GT_BN * 128, b_bytes = T * 128, stage_b = a_bytes + b_bytes;
  size_t pipe_b = static_cast<size_t>(nstages) * stage_b;
  if (static_cast<size_t>(T) * GT_BN * 4 > pipe_b) pipe_b = static_cast<size_t>(T) * GT_BN * 4;
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + pipe_b);
  uint64_t *empty = full + 8;
  uint64_t *acc_full = empty + 8;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);
  float *park = reinterpret_cast<float *>(smem);                // [T][128] fp32, reuses the pipeline stages

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // token blocks vary fastest in the grid, so that the CTAs that share a weight tile run together and it leaves HBM once
  const int n0 = A.n_base + blockIdx.y * GT_BN * wt, m0 = blockIdx.x * T, split = blockIdx.z, ns = A.nsplit;
  const int KB = A.K / GT_BK;
  const int kb_lo = static_cast<int>(static_cast<long long>(split) * KB / ns);
  const int kb_hi = static_cast<int>(static_cast<long long>(split + 1) * KB / ns);
  const uint32_t acc_cols = T <= 32 ? 32u : T <= 64 ? 64u : T <= 128 ? 128u : 256u;   // per accumulator
  const uint32_t ncols = acc_cols * wt;

  if (threadIdx.x == 0) {
    for (int s = 0; s < nstages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    mbar_fence_init();
  }
  if (warp == 1) {
    tc_alloc(tmem_slot, ncols);
    tc_relinquish();
  }
  if (warp == 0 && lane == 0) {
    tma_prefetch_desc(&A.w_map);
    tma_prefetch_desc(&A.x_map);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // The weights are never written by a kernel of the stream, so the first ring of weight boxes may be requested before
  // the previous kernel has finished (their bytes are counted on the stage barrier before its expect-tx arrives, which
  // the barrier allows: the phase cannot complete until that arrival).  The activations wait for the dependency.
  const int pre = A.early_weights ? min(nstages, kb_hi - kb_lo) : 0;
  if (warp == 0 && lane == 0)
    for (int it = 0; it < pre; ++it)
      for (int a = 0; a < wt; ++a)
        tma_load_2d(smem + static_cast<size_t>(it) * stage_b + a * GT_BN * 128, &A.w_map, (kb_lo + it) * GT_BK, n0 + a * GT_BN, &full[it]);
  pdl_prologue();                                  // everything above touches no data a kernel writes: it overlaps the previous kernel

  if (warp == 0) {
    if (lane == 0) {
      for (int kb = kb_lo, it = 0; kb < kb_hi; ++kb, ++it) {
        const int s = it % nstages;
        if (!mbar_wait(&empty[s], ((it / nstages) & 1) ^ 1)) { set_status(A.status, ST_TIMEOUT); break; }
        mbar_expect_tx(&full[s], stage_b);
        unsigned char *dst = smem + static_cast<size_t>(s) * stage_b;
        if (it >= pre)
          for (int a = 0; a < wt; ++a) tma_load_2d(dst + a * GT_BN * 128, &A.w_map, kb * GT_BK, n0 + a * GT_BN, &full[s]);
        tma_load_2d(dst + a_bytes, &A.x_map, kb * GT_BK, m0, &full[s]);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = tc_idesc_bf16(GT_BN, T);
      bool ok = true;
      for (int kb = kb_lo, it = 0; kb < kb_hi; ++kb, ++it) {
        const int s = it % nstages;
        if (!mbar_wait(&full[s], (it / nstages) & 1)) { set_status(A.status, ST_TIMEOUT); ok = false; break; }
        tc_fence_after();
        const uint32_t a_addr = smem_u32(smem + static_cast<size_t>(s) * stage_b);
        const uint64_t bdesc = tc_smem_desc_sw128(a_addr + a_bytes);
        for (int a = 0; a < wt; ++a) {
          const uint64_t adesc = tc_smem_desc_sw128(a_addr + a * GT_BN * 128);
#pragma unroll
          for (int k = 0; k < GT_BK / 16; ++k)    // +32 bytes (2 x 16-byte units) per K=16 step
            tc_mma_bf16(tmem + a * acc_cols, adesc + 2 * k, bdesc + 2 * k, idesc, (it > 0 || k > 0) ? 1u : 0u);
        }
        tc_commit(&empty[s]);                      // the stage is free once these MMAs have read it
      }
      if (ok) tc_commit(acc_full);                 // accumulators complete
    }
  }
  bool acc_ok = kb_hi > kb_lo;
  const bool reader = warp >= 2 && warp < 10;
  if (reader) {
    if (acc_ok && !mbar_wait(acc_full, 0)) { set_status(A.status, ST_TIMEOUT); acc_ok = false; }
    tc_fence_after();
  }
  cg::cluster_group cluster = cg::this_cluster();
  const int per = (T + ns - 1) / ns;               // this CTA reduces tokens [c_lo, c_hi) of every sub-tile
  const int c_lo = split * per, c_hi = min(T, c_lo + per);
  for (int a = 0; a < wt; ++a) {
    __syncthreads();                               // the pipeline stages (first pass) / the previous sub-tile are done with
    if (reader) {
      // TMEM -> registers -> parked fp32 tile in shared memory (lanes = consecutive features: no bank conflicts)
      const int quad = warp & 3;                   // the TMEM lane quadrant this warp may read
      const int r = quad * 32 + lane;
      for (int c0 = ((warp - 2) >> 2) * 16; c0 < T; c0 += 32) {
        uint32_t v[16];
        if (acc_ok) {
          tc_ld_32x16(tmem + (static_cast<uint32_t>(quad * 32) << 16) + a * acc_cols + c0, v);
          tc_wait_ld();
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = 0u;
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) park[(c0 + j) * GT_BN + r] = __uint_as_float(v[j]);
      }
    }
    __syncthreads();
    if (ns > 1) cluster.sync();
    // sum the cluster's K slices in rank order (all peer loads issued before the adds) and apply the epilogue
    for (int idx = threadIdx.x; idx < (c_hi - c_lo) * (GT_BN / 4); idx += GT_THREADS) {
      const int c = c_lo + idx / (GT_BN / 4), r4 = (idx % (GT_BN / 4)) * 4;
      const int m = m0 + c, n = n0 + a * GT_BN + r4;
      if (m >= A.M || n >= A.N) continue;
      float4 acc;
      if (ns == 1) {
        acc = *reinterpret_cast<const float4 *>(park + c * GT_BN + r4);
      } else {
        float4 v[8];
#pragma unroll
        for (int p = 0; p < 8; ++p)
          v[p] = p < ns ? *reinterpret_cast<const float4 *>(cluster.map_shared_rank(park, p) + c * GT_BN + r4)
                        : make_float4(0.f, 0.f, 0.f, 0.f);
        acc = v[0];
#pragma unroll
        for (int p = 1; p < 8; ++p) { acc.x += v[p].x; acc.y += v[p].y; acc.z += v[p].z; acc.w += v[p].w; }
      }
      if (A.epi == EPI_QKV_ROPE) rope_epilogue(A, m, n0 + a * GT_BN, lane, acc);
      else epilogue4(A, m, n, acc);
    }
    if (ns > 1) cluster.sync();                    // peers may still be reading this CTA's parked tile
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tc_dealloc(tmem, ncols);
}

// ---- CTA-pair variant --------------------------------------------------------------------------------------------------
// Projections with one K slice per tile are bound by filling shared memory from L2: every CTA re-reads the whole
// activation tile for its 128 features.  Here two CTAs on neighbouring feature tiles form a pair (a cluster of
// two): each stages its own 128 x 64 weight box and only HALF of the activation box per K block, and one
// tcgen05.mma of the pair (M = 256 features, N = T tokens) reads both halves, so a CTA moves 2/3 of the bytes per K
// block (at T = 256) and its ring holds more K blocks.  The accumulator rows of a CTA's own 128 features land in its
// own tensor memory, so the epilogue is the single-CTA one.
//   even CTA (leader): producer + the MMA issuer for the pair.  Its `full` barriers count the bytes of both CTAs.
//   odd CTA: producer only; its loads complete on the leader's barriers.  The leader's tcgen05.commit arrives on
//   the `empty` / accumulator barriers of both CTAs (relaying those arrivals through the leader's waiting threads
//   instead made every stage refill ~3 us longer and the main loop 0.93 us per K block instead of 0.50).
__global__ void __launch_bounds__(GT_THREADS, 1)
gemm_pair_kernel(const __grid_constant__ GemmArgs A, const int nstages) {
  extern __shared__ unsigned char gt_smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(gt_smem_raw) + 1023) & ~uintptr_t(1023));
  const int T = A.block_t, H = T / 2;
  const int a_bytes = GT_BN * 128, b_bytes = H * 128, stage_b = a_bytes + b_bytes;
  size_t pipe_b = static_cast<size_t>(nstages) * stage_b;
  if (static_cast<size_t>(T) * GT_BN * 4 > pipe_b) pipe_b = static_cast<size_t>(T) * GT_BN * 4;
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + pipe_b);
  uint64_t *empty = full + 8;
  uint64_t *acc_full = empty + 8;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);
  float *park = reinterpret_cast<float *>(smem);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();            // 0: leader, 1: peer
  const bool leader = rank == 0;
  const int n0 = A.n_base + blockIdx.x * GT_BN, m0 = blockIdx.y * T;     // the pair = two neighbouring feature tiles
  const int KB = A.K / GT_BK;
  const uint32_t ncols = T <= 32 ? 32u : T <= 64 ? 64u : T <= 128 ? 128u : 256u;

  if (threadIdx.x == 0) {
    for (int s = 0; s < nstages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    mbar_fence_init();
  }
  if (warp == 1) {
    tc2_alloc(tmem_slot, ncols);
    tc2_relinquish();
  }
  if (warp == 0 && lane == 0) {
    tma_prefetch_desc(&A.w_map);
    tma_prefetch_desc(&A.x_half_map);
  }
  tc_fence_before();
  cg::cluster_group cluster = cg::this_cluster();
  cluster.sync();                                  // both CTAs' barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_prologue();

  if (warp == 0) {
    if (lane == 0) {
      for (int kb = 0; kb < KB; ++kb) {
        const int s = kb % nstages;
        if (!mbar_wait(&empty[s], ((kb / nstages) & 1) ^ 1)) { set_status(A.status, ST_TIMEOUT); break; }
        if (leader) {
          mbar_expect_tx(&full[s], 2 * stage_b);
        }
        const uint32_t bar = cluster_addr(&full[s], 0);
        unsigned char *dst = smem + static_cast<size_t>(s) * stage_b;
        tma2_load_2d(dst, &A.w_map, kb * GT_BK, n0, bar);
        tma2_load_2d(dst + a_bytes, &A.x_half_map, kb * GT_BK, m0 + static_cast<int>(rank) * H, bar);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && leader) {
      const uint32_t idesc = tc_idesc_bf16(2 * GT_BN, T);
      bool ok = true;
      for (int kb = 0; kb < KB; ++kb) {
        const int s = kb % nstages;
        if (!mbar_wait(&full[s], (kb / nstages) & 1)) { set_status(A.status, ST_TIMEOUT); ok = false; break; }
        tc_fence_after();
        const uint32_t a_addr = smem_u32(smem + static_cast<size_t>(s) * stage_b);
        const uint64_t adesc = tc_smem_desc_sw128(a_addr), bdesc = tc_smem_desc_sw128(a_addr + a_bytes);
#pragma unroll
        for (int k = 0; k < GT_BK / 16; ++k)
          tc2_mma_bf16(tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb > 0 || k > 0) ? 1u : 0u);
        tc2_commit_mc(&empty[s], 3);                // the stage is free in both CTAs
      }
      if (ok) tc2_commit_mc(acc_full, 3);
    }
  }
  bool acc_ok = KB > 0;
  const bool reader = warp >= 2 && warp < 10;
  if (reader) {
    if (acc_ok && !mbar_wait(acc_full, 0)) { set_status(A.status, ST_TIMEOUT); acc_ok = false; }
    tc_fence_after();
  }
  __syncthreads();                                 // the pipeline stages are done with (both CTAs' MMAs have completed)
  if (reader) {
    const int quad = warp & 3;
    const int r = quad * 32 + lane;
    for (int c0 = ((warp - 2) >> 2) * 16; c0 < T; c0 += 32) {
      uint32_t v[16];
      if (acc_ok) {
        tc_ld_32x16(tmem + (static_cast<uint32_t>(quad * 32) << 16) + c0, v);
        tc_wait_ld();
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = 0u;
      }
#pragma unroll
      for (int j = 0; j < 16; ++j) park[(c0 + j) * GT_BN + r] = __uint_as_float(v[j]);
    }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < T * (GT_BN / 4); idx += GT_THREADS) {
    const int c = idx / (GT_BN / 4), r4 = (idx % (GT_BN / 4)) * 4;
    const int m = m0 + c, n = n0 + r4;
    if (m >= A.M || n >= A.N) continue;
    epilogue4(A, m, n, *reinterpret_cast<const float4 *>(park + c * GT_BN + r4));
  }
  tc_fence_before();
  cluster.sync();                                  // neither CTA frees tensor memory while the other still reads its own
  if (warp == 1) tc2_dealloc(tmem, ncols);
}

// ---- CTA pairs with K slices ---------------------------------------------------------------------------------------------
// The pair kernel for projections with few output tiles: cluster (2, 1, ns) = ns pairs on one 256-feature tile, pair z
// taking K slice z.  Inside a pair everything is as above (the leader is the even rank of the pair; barriers and commits
// address the pair's two CTAs by their cluster ranks); afterwards every CTA parks its 128-feature accumulator and sums
// one slice of the tile's tokens over the ns CTAs that hold the same features, in slice order, through distributed
// shared memory - the reduction of gemm_tc_kernel.
__global__ void __launch_bounds__(GT_THREADS, 1)
gemm_pair_split_kernel(const __grid_constant__ GemmArgs A, const int nstages) {
  extern __shared__ unsigned char gt_smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(gt_smem_raw) + 1023) & ~uintptr_t(1023));
  const int T = A.block_t, H = T / 2;
  const int a_bytes = GT_BN * 128, b_bytes = H * 128, stage_b = a_bytes + b_bytes;
  size_t pipe_b = static_cast<size_t>(nstages) * stage_b;
  if (static_cast<size_t>(T) * GT_BN * 4 > pipe_b) pipe_b = static_cast<size_t>(T) * GT_BN * 4;
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + pipe_b);
  uint64_t *empty = full + 8;
  uint64_t *acc_full = empty + 8;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);
  float *park = reinterpret_cast<float *>(smem);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();            // x + 2 z within the cluster
  const uint32_t half = rank & 1u, lead_rank = rank & ~1u;
  const bool leader = half == 0;
  const int ns = A.nsplit, split = blockIdx.z;
  const int n0 = A.n_base + blockIdx.x * GT_BN, m0 = blockIdx.y * T;
  const int KB = A.K / GT_BK;
  const int kb_lo = static_cast<int>(static_cast<long long>(split) * KB / ns);
  const int kb_hi = static_cast<int>(static_cast<long long>(split + 1) * KB / ns);
  const uint32_t ncols = T <= 32 ? 32u : T <= 64 ? 64u : T <= 128 ? 128u : 256u;
  const uint16_t pair_mask = static_cast<uint16_t>(3u << lead_rank);

  if (threadIdx.x == 0) {
    for (int s = 0; s < nstages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    mbar_fence_init();
  }
  if (warp == 1) {
    tc2_alloc(tmem_slot, ncols);
    tc2_relinquish();
  }
  if (warp == 0 && lane == 0) {
    tma_prefetch_desc(&A.w_map);
    tma_prefetch_desc(&A.x_half_map);
  }
  tc_fence_before();
  cg::cluster_group cluster = cg::this_cluster();
  cluster.sync();                                  // every CTA's barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_prologue();

  if (warp == 0) {
    if (lane == 0) {
      for (int kb = kb_lo, it = 0; kb < kb_hi; ++kb, ++it) {
        const int s = it % nstages;
        if (!mbar_wait(&empty[s], ((it / nstages) & 1) ^ 1)) { set_status(A.status, ST_TIMEOUT); break; }
        if (leader) mbar_expect_tx(&full[s], 2 * stage_b);
        const uint32_t bar = cluster_addr(&full[s], lead_rank);
        unsigned char *dst = smem + static_cast<size_t>(s) * stage_b;
        tma2_load_2d(dst, &A.w_map, kb * GT_BK, n0, bar);
        tma2_load_2d(dst + a_bytes, &A.x_half_map, kb * GT_BK, m0 + static_cast<int>(half) * H, bar);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && leader) {
      const uint32_t idesc = tc_idesc_bf16(2 * GT_BN, T);
      bool ok = true;
      for (int kb = kb_lo, it = 0; kb < kb_hi; ++kb, ++it) {
        const int s = it % nstages;
        if (!mbar_wait(&full[s], (it / nstages) & 1)) { set_status(A.status, ST_TIMEOUT); ok = false; break; }
        tc_fence_after();
        const uint32_t a_addr = smem_u32(smem + static_cast<size_t>(s) * stage_b);
        const uint64_t adesc = tc_smem_desc_sw128(a_addr), bdesc = tc_smem_desc_sw128(a_addr + a_bytes);
#pragma unroll
        for (int k = 0; k < GT_BK / 16; ++k)
          tc2_mma_bf16(tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (it > 0 || k > 0) ? 1u : 0u);
        tc2_commit_mc(&empty[s], pair_mask);        // the stage is free in both CTAs of the pair
      }
      if (ok) tc2_commit_mc(acc_full, pair_mask);
    }
  }
  bool acc_ok = kb_hi > kb_lo;
  const bool reader = warp >= 2 && warp < 10;
  if (reader) {
    if (acc_ok && !mbar_wait(acc_full, 0)) { set_status(A.status, ST_TIMEOUT); acc_ok = false; }
    tc_fence_after();
  }
  __syncthreads();                                 // the pipeline stages are done with (the pair's MMAs have completed)
  if (reader) {
    const int quad = warp & 3;
    const int r = quad * 32 + lane;
    for (int c0 = ((warp - 2) >> 2) * 16; c0 < T; c0 += 32) {
      uint32_t v[16];
      if (acc_ok) {
        tc_ld_32x16(tmem + (static_cast<uint32_t>(quad * 32) << 16) + c0, v);
        tc_wait_ld();
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = 0u;
      }
#pragma unroll
      for (int j = 0; j < 16; ++j) park[(c0 + j) * GT_BN + r] = __uint_as_float(v[j]);
    }
  }
  __syncthreads();
  cluster.sync();                                  // every slice's accumulator is parked
  const int per = (T + ns - 1) / ns;               // this CTA reduces tokens [c_lo, c_hi) of its 128 features
  const int c_lo = split * per, c_hi = min(T, c_lo + per);
  for (int idx = threadIdx.x; idx < (c_hi - c_lo) * (GT_BN / 4); idx += GT_THREADS) {
    const int c = c_lo + idx / (GT_BN / 4), r4 = (idx % (GT_BN / 4)) * 4;
    const int m = m0 + c, n = n0 + r4;
    if (m >= A.M || n >= A.N) continue;
    float4 v[8];
#pragma unroll
    for (int p = 0; p < 8; ++p)
      v[p] = p < ns ? *reinterpret_cast<const float4 *>(cluster.map_shared_rank(park, half + 2u * p) + c * GT_BN + r4)
                    : make_float4(0.f, 0.f, 0.f, 0.f);
    float4 acc = v[0];
#pragma unroll
    for (int p = 1; p < 8; ++p) { acc.x += v[p].x; acc.y += v[p].y; acc.z += v[p].z; acc.w += v[p].w; }
    epilogue4(A, m, n, acc);
  }
  tc_fence_before();
  cluster.sync();                                  // peers may still be reading this CTA's parked tile / tensor memory in use
  if (warp == 1) tc2_dealloc(tmem, ncols);
}

// The kernel may use the whole opt-in shared memory of an SM (227 KB); set once per device.
static cudaError_t gt_configure() {
  static SmemConfigured configured;
  return ensure_dyn_smem(gemm_tc_kernel<1>, 227 * 1024, configured);
}

cudaError_t gemm_tc_max_clusters(int block_t, int nsplit, int *out) {
  const size_t smem = gt_smem(block_t, 1);
  cudaError_t e = gt_configure();
  if (e != cudaSuccess) return e;
  if (nsplit > 8) {
    e = cudaFuncSetAttribute(gemm_tc_kernel<1>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(1, 1, nsplit);
  cfg.blockDim = dim3(GT_THREADS);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = nsplit;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaOccupancyMaxActiveClusters(out, gemm_tc_kernel<1>, &cfg);
}

static int pair_stages(int T) {
  int s = GT_SMEM_BUDGET / (GT_BN * 128 + (T / 2) * 128);
  return s > 8 ? 8 : s;
}
cudaError_t launch_gemm_pair(const GemmArgs &A, cudaStream_t stream) {
  const int T = A.block_t;
  if (T < 32 || T > 256 || (T & 31) || (A.K % GT_BK) || A.nsplit != 1 || A.wtiles != 1 || A.n_tiles < 2 ||
      (A.n_tiles & 1) || A.n_base < 0)
    return cudaErrorInvalidValue;
  static SmemConfigured configured;
  if (cudaError_t e = ensure_dyn_smem(gemm_pair_kernel, 227 * 1024, configured); e != cudaSuccess) return e;
  const int st = pair_stages(T);
  size_t pipe = static_cast<size_t>(st) * (GT_BN * 128 + (T / 2) * 128);
  const size_t park = static_cast<size_t>(T) * GT_BN * 4;
  if (park > pipe) pipe = park;
  const dim3 grid(A.n_tiles, (A.M + T - 1) / T, 1);
  return launch_kc(gemm_pair_kernel, grid, dim3(GT_THREADS), pipe + 1024 + 256, stream, dim3(2, 1, 1), A, st);
}

cudaError_t launch_gemm_pair_split(const GemmArgs &A, cudaStream_t stream) {
  const int T = A.block_t;
  if (T < 32 || T > 256 || (T & 31) || (A.K % GT_BK) || A.nsplit < 2 || A.nsplit > 8 || A.nsplit > A.K / GT_BK || A.wtiles != 1 ||
      A.n_tiles < 2 || (A.n_tiles & 1) || A.n_base < 0)
    return cudaErrorInvalidValue;
  static SmemConfigured configured;
  if (cudaError_t e = ensure_dyn_smem(gemm_pair_split_kernel, 227 * 1024, configured); e != cudaSuccess) return e;
  if (A.nsplit > 4)                                  // clusters of more than 8 CTAs are an opt-in
    if (cudaError_t e = cudaFuncSetAttribute(gemm_pair_split_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1); e != cudaSuccess) return e;
  const int st = pair_stages(T);
  size_t pipe = static_cast<size_t>(st) * (GT_BN * 128 + (T / 2) * 128);
  const size_t park = static_cast<size_t>(T) * GT_BN * 4;
  if (park > pipe) pipe = park;
  const dim3 grid(A.n_tiles, (A.M + T - 1) / T, A.nsplit);
  return launch_kc(gemm_pair_split_kernel, grid, dim3(GT_THREADS), pipe + 1024 + 256, stream, dim3(2, 1, A.nsplit), A, st);
}
cudaError_t gemm_pair_split_max_clusters(int block_t, int nsplit, int *out) {
  static SmemConfigured configured;
  if (cudaError_t e = ensure_dyn_smem(gemm_pair_split_kernel, 227 * 1024, configured); e != cudaSuccess) return e;
  if (nsplit > 4)
    if (cudaError_t e = cudaFuncSetAttribute(gemm_pair_split_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1); e != cudaSuccess) return e;
  const int st = pair_stages(block_t);
  size_t pipe = static_cast<size_t>(st) * (GT_BN * 128 + (block_t / 2) * 128);
  const size_t park = static_cast<size_t>(block_t) * GT_BN * 4;
  if (park > pipe) pipe = park;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2, 1, nsplit);
  cfg.blockDim = dim3(GT_THREADS);
  cfg.dynamicSmemBytes = pipe + 1024 + 256;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = nsplit;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaOccupancyMaxActiveClusters(out, gemm_pair_split_kernel, &cfg);
}

cudaError_t launch_gemm_tc(const GemmArgs &A, cudaStream_t stream) {
  const int T = A.block_t;
  if (T < 16 || T > 256 || (T & 15) || (A.K % GT_BK) || A.nsplit < 1 || A.nsplit > A.K / GT_BK || A.nsplit > 8 ||
      A.wtiles < 1 || A.wtiles > 2 || A.n_tiles < 1 || A.n_base < 0)
    return cudaErrorInvalidValue;
  const size_t smem = gt_smem(T, A.wtiles);
  cudaError_t ec = gt_configure();
  if (ec != cudaSuccess) return ec;
  const dim3 grid((A.M + T - 1) / T, A.n_tiles, A.nsplit);
  // Few tokens, many tiles per SM (the draft phase's LM head): two CTAs per SM with half the ring each, so that one
  // CTA's epilogue and its successor's first fill run under the other's main loop.
  static const bool no_two = std::getenv("GM_NO_GEMM_2CTA") != nullptr;
  if (!no_two && A.nsplit == 1 && T <= 64 && static_cast<long long>(grid.x) * grid.y >= 4LL * 148) {
    const int stage = A.wtiles * GT_BN * 128 + T * 128;
    int st = (100 * 1024) / stage;
    if (st >= 2) {
      if (st > 8) st = 8;
      size_t pipe = static_cast<size_t>(st) * stage;
      const size_t park = static_cast<size_t>(T) * GT_BN * 4;
      if (park > pipe) pipe = park;
      static SmemConfigured configured2;
      if (cudaError_t e = ensure_dyn_smem(gemm_tc_kernel<2>, 112 * 1024, configured2); e != cudaSuccess) return e;
      return launch_k(gemm_tc_kernel<2>, grid, dim3(GT_THREADS), pipe + 1024 + 256, stream, 1, A, st);
    }
  }
  return launch_k(gemm_tc_kernel<1>, grid, dim3(GT_THREADS), smem, stream, A.nsplit, A, gt_stages(T, A.wtiles));
}

// ---- plain mma.sync GEMM ----------------------------------------------------------------------------------------------
// CTA = 4 warps; warp w computes rows [m0 + 16 w, +16) x columns [n0, n0 + 64) with fragments loaded
// straight from global memory (both operands are K-major, so fragments are plain 32-bit loads).
__global__ void __launch_bounds__(128) gemm_simple_kernel(const GemmArgs A) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, t4 = lane & 3, r8 = lane >> 2;
  const int m0 = blockIdx.y * 64 + warp * 16, n0 = blockIdx.x * 64;
  pdl_prologue();
  float acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
  const int ra = m0 + r8, rb = m0 + r8 + 8;
  for (int k = 0; k < A.K; k += 16) {
    uint32_t a[4];
    const __nv_bfloat16 *pa = A.x + static_cast<size_t>(ra) * A.K + k + 2 * t4;
    const __nv_bfloat16 *pb = A.x + static_cast<size_t>(rb) * A.K + k + 2 * t4;
    a[0] = ra < A.M ? *reinterpret_cast<const uint32_t *>(pa) : 0u;
    a[1] = rb < A.M ? *reinterpret_cast<const uint32_t *>(pb) : 0u;
    a[2] = ra < A.M ? *reinterpret_cast<const uint32_t *>(pa + 8) : 0u;
    a[3] = rb < A.M ? *reinterpret_cast<const uint32_t *>(pb + 8) : 0u;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const int n = n0 + nt * 8 + r8;
      uint32_t b0 = 0u, b1 = 0u;
      if (n < A.N) {
        const __nv_bfloat16 *pw = A.w + static_cast<size_t>(n) * A.K + k + 2 * t4;
        b0 = *reinterpret_cast<const uint32_t *>(pw);
        b1 = *reinterpret_cast<const uint32_t *>(pw + 8);
      }
      mma_16816(acc[nt], a, b0, b1);
    }
  }
  // each thread holds column pairs (n, n+1) with n even: (gate, up) of one SwiGLU output
#pragma unroll
  for (int nt = 0; nt < 8; ++nt)
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int m = m0 + r8 + h * 8, n = n0 + nt * 8 + 2 * t4;
      if (m >= A.M) continue;
      const float v0 = acc[nt][h * 2], v1 = acc[nt][h * 2 + 1];
      if (A.epi == EPI_SWIGLU_BF16) {
        if (n + 1 < A.N)
          reinterpret_cast<__nv_bfloat16 *>(A.out)[static_cast<size_t>(m) * A.ldo + (n >> 1)] =
              __float2bfloat16(v0 / (1.f + __expf(-v0)) * v1);
        continue;
      }
      for (int e = 0; e < 2; ++e) {
        if (n + e >= A.N) continue;
        const float v = e ? v1 : v0;
        const size_t o = static_cast<size_t>(m) * A.ldo + n + e;
        if (A.epi == EPI_STORE_BF16) reinterpret_cast<__nv_bfloat16 *>(A.out)[o] = __float2bfloat16(v);
        else if (A.epi == EPI_ADD_F32) reinterpret_cast<float *>(A.out)[o] += v;
        else reinterpret_cast<float *>(A.out)[o] = v;
      }
    }
}

cudaError_t launch_gemm_simple(const GemmArgs &A, cudaStream_t stream) {
  if (A.K % 16) return cudaErrorInvalidValue;
  dim3 grid((A.N + 63) / 64, (A.M + 63) / 64, 1);
  return launch_k(gemm_simple_kernel, grid, dim3(128), 0, stream, 1, A);
}

}  // namespace gm
