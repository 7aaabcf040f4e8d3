// chain_kernel: a decoder layer's dense projections as ONE persistent launch.
//
// Between two attention calls a layer runs four dependent projections on the same few hundred token rows - output
// projection (+ residual), gate/up (+ SwiGLU), down (+ residual), and the next layer's QKV - with an RMSNorm in front
// of the second and the fourth.  As separate launches each pays its own set-up, first fill of the stage ring, split-K
// reduction and drain, which at these sizes is as long as the main loop itself.  Here the whole chain is one grid of
// CTA pairs (one pair per two SMs) that walks the projections ("phases") in order:
//
//   * every pair keeps one ring of shared-memory stages alive across phases.  Weights depend on nothing, so the
//     producer thread streams the next phase's weight boxes into free stages while the current phase is still
//     draining; only the activation boxes wait for the grid-wide barrier that ends the phase before.
//   * a phase's tiles (256 features x T tokens on tcgen05 cta_group::2: each CTA stages its own 128 x 64 weight box and
//     half of the activation box per K block) are dealt out by formula: whole tiles round-robin over the pairs, and
//     the tiles that do not fill a round are cut along K over ns consecutive pairs.  The K slices of a tile leave
//     their fp32 partial sums in an L2-resident scratch slot per CTA, meet at a barrier of their own, and each slice
//     owner reduces one slice of the tile's tokens over all partials in slice order - the result does not depend on timing.
//   * the RMSNorms are folded around the projections: W (x g / rms) = (W (x g)) / rms.  The phase that updates the
//     residual stream x also writes bf16(x g) for the next norm's weight g and the sum of squares of every 32
//     features of each token row (plain stores, no atomics); the consuming phase adds those partial sums in a fixed
//     order and scales its accumulator rows by rsqrt(mean + eps) in the epilogue.
//   * two accumulators alternate in tensor memory, so the MMA thread starts a pair's next tile while the epilogue
//     warps drain the previous one straight from tensor memory to global memory.
//
// Every wait (mbarrier, grid barrier, tile barrier) is bounded: on expiry the kernel records ST_TIMEOUT, raises a
// CTA-wide abort flag that makes every later wait return at once, still meets its CTA / cluster barriers, frees its
// tensor memory and returns.  The grid barrier needs all CTAs resident at once; the launcher sizes the grid from the
// occupancy query for clusters of two.
#include <cooperative_groups.h>

#include "common.cuh"
#include "kernels.h"

namespace cg = cooperative_groups;

namespace gm {

constexpr int CH_MAX_NPW = 2, CH_MAX_NPA = 2;      // producer warps: weights, activations
constexpr int CH_PROD_WARPS = CH_MAX_NPW + CH_MAX_NPA;
constexpr int CH_MMA_WARP = CH_PROD_WARPS;         // tensor-memory owner + MMA issuer
constexpr int CH_EPI_WARP0 = CH_MMA_WARP + 1;      // first of the 16 epilogue warps
constexpr int CH_EPI_WARPS = 16;
constexpr int CH_THREADS = (CH_EPI_WARP0 + CH_EPI_WARPS) * 32;
constexpr int CH_EPI_THREADS = CH_EPI_WARPS * 32;
constexpr int CH_MAX_PHASES = 4;
constexpr int CH_BK = 64;              // K elements per stage (one 128-byte swizzle row)
constexpr int CH_TOK = 128;            // token rows per CTA (a pair's tile has 256)
constexpr int CH_FEAT = 256;           // features per pair tile; each CTA stages half of them
constexpr int CH_W_BYTES = (CH_FEAT / 2) * 128;    // one CTA's weight box: 128 features x 64 K elements
constexpr int CH_STAGE_BYTES = CH_W_BYTES + CH_TOK * 128;   // + its activation box: 128 tokens x 64 K elements
constexpr int CH_STAGES = 6;
constexpr uint32_t CH_SPIN_LIMIT = 1u << 22;

// ---- global-memory barriers (sense reversing: {count, generation}) ------------------------------------------------------
__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_u32(uint32_t *p, uint32_t v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t atom_add_acq_rel(uint32_t *p, uint32_t v) {
  uint32_t r;
  asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(r) : "l"(p), "r"(v) : "memory");
  return r;
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
// One thread per participant.  Returns the generation the caller has to see change.
__device__ __forceinline__ uint32_t gbar_arrive(uint32_t *bar, uint32_t n) {
  const uint32_t g = ld_acquire_u32(bar + 1);
  __threadfence();
  if (atom_add_acq_rel(bar, 1u) == n - 1) {
    bar[0] = 0u;                                   // ordered before the release below
    st_release_u32(bar + 1, g + 1);
  }
  return g;
}

__device__ __forceinline__ bool mbar_test_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Arrival on an mbarrier of another CTA of the cluster (address in the cluster window).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar_addr) : "memory");
}
// Flags in shared memory that the leader CTA of a pair sets in both CTAs (release / acquire at cluster scope).
__device__ __forceinline__ void st_release_cluster_smem(uint32_t cluster_addr_, uint32_t v) {
  asm volatile("st.release.cluster.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr_), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire_cluster_smem(const volatile uint32_t *p) {
  uint32_t v;
  asm volatile("ld.acquire.cluster.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(const_cast<const uint32_t *>(p))) : "memory");
  return v;
}
// Bounded wait that gives up at once when the CTA has raised its abort flag.
__device__ __forceinline__ bool mbar_wait_abortable(uint64_t *bar, uint32_t parity, volatile int *abort_flag) {
  for (uint32_t i = 0; i < CH_SPIN_LIMIT; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 255u) == 255u && *abort_flag) return false;
  }
  return false;
}

// ---- the schedule: which tiles of a phase a pair works on ---------------------------------------------------------------
struct ChainItem {
  int unit;        // tile index: token block = unit % mblocks, feature pair-tile = unit / mblocks
  int split, ns;   // K slice and slices of this tile
  int base;        // first pair of the tile's slice group
  int kb_lo, kb_hi;
};
__device__ __forceinline__ bool chain_item(const ChainPhase &ph, int P, int pair, int idx, ChainItem &it) {
  if (idx < ph.full) {
    it.unit = pair + idx * P; it.split = 0; it.ns = 1; it.base = pair; it.kb_lo = 0; it.kb_hi = ph.K / CH_BK;
    return true;
  }
  if (idx == ph.full && ph.ns > 0 && pair < ph.rem * ph.ns) {
    const int KB = ph.K / CH_BK;
    it.unit = ph.full * P + pair / ph.ns; it.split = pair % ph.ns; it.ns = ph.ns; it.base = pair - it.split;
    it.kb_lo = static_cast<int>(static_cast<long long>(it.split) * KB / ph.ns);
    it.kb_hi = static_cast<int>(static_cast<long long>(it.split + 1) * KB / ph.ns);
    return true;
  }
  return false;
}
// Walks the K blocks of all items of all phases of one pair in order (producer and MMA thread use the same walk).
struct SlotIter {
  int ph, idx, kb;
  ChainItem it;
  bool valid;
  __device__ __forceinline__ void seek(const ChainArgs &A, int pair) {
    while (ph < A.n_phases) {
      if (chain_item(A.ph[ph], A.P, pair, idx, it)) {
        if (it.kb_lo < it.kb_hi) { kb = it.kb_lo; valid = true; return; }
        ++idx;
        continue;
      }
      ++ph; idx = 0;
    }
    valid = false;
  }
  __device__ __forceinline__ void start(const ChainArgs &A, int pair) { ph = 0; idx = 0; kb = 0; seek(A, pair); }
  __device__ __forceinline__ void next(const ChainArgs &A, int pair) {
    if (++kb >= it.kb_hi) { ++idx; seek(A, pair); }
  }
};

// Optional trace (ChainArgs::timeline): nanosecond stamps per CTA, 32 slots each.  Slot 0 entry, 1 set-up done,
// 2 previous kernel complete (producer), 31 exit; per phase p from slot 4 + 6 p: first activation box issued, first
// stage consumed by the MMA thread, last MMA issued, first accumulator complete, epilogue of the phase done, the
// barrier that ends the phase seen complete.
__device__ __forceinline__ void trace(const ChainArgs &A, int slot) {
  if (A.timeline) {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)::"memory");
    A.timeline[static_cast<size_t>(blockIdx.x) * 64 + slot] = t;
  }
}

__device__ __forceinline__ float silu_mul(float g, float u) { return __fdividef(g, 1.f + __expf(-g)) * u; }

__global__ void __launch_bounds__(CH_THREADS, 1)
chain_kernel(const __grid_constant__ ChainArgs A) {
  extern __shared__ unsigned char ch_smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(ch_smem_raw) + 1023) & ~uintptr_t(1023));
  constexpr int nstages = CH_STAGES, stage_b = CH_STAGE_BYTES;
  unsigned char *ctl = smem + static_cast<size_t>(nstages) * stage_b;
  uint64_t *full = reinterpret_cast<uint64_t *>(ctl);
  uint64_t *empty = full + CH_STAGES;
  uint64_t *acc_full = empty + CH_STAGES;            // [2]
  uint64_t *acc_empty = acc_full + 2;                // [2] (the leader's are the ones waited on)
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  float *rstd = reinterpret_cast<float *>(tmem_slot + 4);   // [128] 1 / rms of this CTA's token rows
  float *rtmp = rstd + CH_TOK;                               // [4][128] partial sums while rstd is built
  // pub[p] != 0: the grid barrier that ends phase p is complete.  Only one thread of each pair (the leader CTA's first
  // epilogue thread) polls the barrier word in global memory - more pollers slow every other access to that L2 slice -
  // and sets the flag in both CTAs; the producers and the other CTA's epilogue wait on their own shared memory.
  volatile uint32_t *pub = reinterpret_cast<volatile uint32_t *>(rtmp + 4 * CH_TOK);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();
  const bool leader = rank == 0;
  const int pair = blockIdx.x >> 1;
  constexpr uint32_t acc_cols = 256u, ncols = 512u;  // two accumulators of 128 token lanes x 256 feature columns
  const uint32_t n_ctas = static_cast<uint32_t>(A.P) * 2u;
  uint32_t *grid_bar = A.sync;
  if (threadIdx.x == 0) trace(A, 0);

  if (threadIdx.x == 0) {
    for (int s = 0; s < nstages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 2 * CH_EPI_WARPS); }
    *abort_flag = 0;
    for (int p = 0; p < CH_MAX_PHASES; ++p) pub[p] = 0u;
    mbar_fence_init();
  }
  if (warp == CH_MMA_WARP) {
    tc2_alloc(tmem_slot, ncols);
    tc2_relinquish();
  }
  if (warp == 0 && lane == 0)
    for (int p = 0; p < A.n_phases; ++p) { tma_prefetch_desc(&A.ph[p].w_map); tma_prefetch_desc(&A.ph[p].x_map); }
  tc_fence_before();
  cg::cluster_group cluster = cg::this_cluster();
  cluster.sync();                                    // both CTAs' barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (threadIdx.x == 0) trace(A, 1);

  if (warp < CH_PROD_WARPS) {
    // ================= producers: one thread issues a K block's weight box or its activation box =================
    // The K blocks are dealt out over npw weight producers and npa activation producers (one warp each).  Weights
    // depend on nothing: their producers run ahead as far as the ring allows, across phases and before the previous
    // kernel has finished.  Activation producers wait for the barrier that ends the phase before.
    const bool is_w = warp < CH_MAX_NPW;
    const int pi = is_w ? warp : warp - CH_MAX_NPW;              // index among the producers of its kind
    const int np = is_w ? A.npw : A.npa;
    if (lane == 0 && pi < np) {
      SlotIter it;
      it.start(A, pair);
      const uint32_t full0 = cluster_addr(&full[0], 0);
      int phase_ok = 0;                              // activations of phases below this one may be read
      int q = 0, last_q = -1;
      bool ok = true;
      for (; it.valid && ok; it.next(A, pair), ++q) {
        if (q % np != pi) continue;
        const int s = q % nstages;
        if (!is_w && it.ph >= phase_ok) {
          if (it.ph == 0) {                          // the first phase's input comes from the previous kernel
            asm volatile("griddepcontrol.wait;" ::: "memory");
            if (pi == 0) trace(A, 2);
          } else {
            bool seen = false;
            for (uint32_t i = 0; i < CH_SPIN_LIMIT && !seen; ++i) {
              seen = ld_acquire_cluster_smem(&pub[it.ph - 1]) != 0u;
              if (!seen) { if (*abort_flag) break; __nanosleep(100); }
            }
            if (!seen) { ok = false; break; }
            fence_proxy_async_all();                 // other CTAs' stores, seen through the barrier, before the TMA reads
          }
          phase_ok = it.ph + 1;
          if (pi == 0) trace(A, 4 + 6 * it.ph);
        }
        if (!mbar_wait_abortable(&empty[s], ((q / nstages) & 1) ^ 1, abort_flag)) { ok = false; break; }
        const ChainPhase &ph = A.ph[it.ph];
        unsigned char *dst = smem + static_cast<size_t>(s) * stage_b;
        if (is_w) {
          if (leader) mbar_expect_tx(&full[s], 2 * stage_b);
          const int n0 = (it.it.unit / A.mblocks) * CH_FEAT + static_cast<int>(rank) * (CH_FEAT / 2);
          tma2_load_2d(dst, &ph.w_map, it.kb * CH_BK, n0, full0 + s * 8);
        } else {
          const int m0 = (it.it.unit % A.mblocks) * (2 * CH_TOK) + static_cast<int>(rank) * CH_TOK;
          tma2_load_2d(dst + CH_W_BYTES, &ph.x_map, it.kb * CH_BK, m0, full0 + s * 8);
        }
        last_q = q;
      }
      if (!ok) { set_status(A.status, ST_TIMEOUT); *abort_flag = 1; }
      // the copies this thread issued have landed before the CTA may exit: their stages have been consumed
      if (last_q >= 0) {
        bool done = false;
        for (uint32_t i = 0; i < (1u << 16) && !done; ++i) done = mbar_try_wait(&empty[last_q % nstages], (last_q / nstages) & 1);
      }
    }
  } else if (warp == CH_MMA_WARP) {
    // ================= MMA issuer (leader CTA of the pair) =================
    // D[256 tokens x 256 features] += A[256 tokens x 64] * B[256 features x 64]^T: each CTA holds its 128 token rows of A
    // and of D, and stages 128 of the 256 feature rows of B.
    if (lane == 0 && leader) {
      const uint32_t idesc = tc_idesc_bf16(2 * CH_TOK, CH_FEAT);
      SlotIter mi;
      mi.start(A, pair);
      int q = 0, item_no = 0;
      bool ok = true;
      while (mi.valid && ok) {
        const int buf = item_no & 1;
        if (mi.kb == mi.it.kb_lo) {                  // a new tile: its accumulator must have been drained
          if (!mbar_wait_abortable(&acc_empty[buf], ((item_no >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
          tc_fence_after();
        }
        const int s = q % nstages;
        if (!mbar_wait_abortable(&full[s], (q / nstages) & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        if (mi.idx == 0 && mi.kb == mi.it.kb_lo) trace(A, 5 + 6 * mi.ph);
        const uint32_t w_addr = smem_u32(smem + static_cast<size_t>(s) * stage_b);
        const uint64_t bdesc = tc_smem_desc_sw128(w_addr), adesc = tc_smem_desc_sw128(w_addr + CH_W_BYTES);
        const uint32_t d_tmem = tmem + buf * acc_cols;
#pragma unroll
        for (int k = 0; k < CH_BK / 16; ++k)
          tc2_mma_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (mi.kb > mi.it.kb_lo || k > 0) ? 1u : 0u);
        tc2_commit_mc(&empty[s], 3);                 // the stage is free in both CTAs once these MMAs have read it
        if (mi.kb == mi.it.kb_hi - 1) {
          tc2_commit_mc(&acc_full[buf], 3);          // the tile's accumulator is complete in both CTAs
          ++item_no;
          trace(A, 6 + 6 * mi.ph);
        }
        mi.next(A, pair);
        ++q;
      }
      if (!ok) { set_status(A.status, ST_TIMEOUT); *abort_flag = 1; }
    }
  } else {
    // ================= epilogue warps (both CTAs: each drains its 128 token rows x 256 features) =================
    // Warp (quad, chunk): token lanes quad * 32 .. + 31 (the quadrant of tensor memory the warp may read), feature
    // columns chunk * 64 .. + 63.  A thread owns one token row and 64 consecutive features: vector stores, SwiGLU pairs
    // in neighbouring registers, the row's sum of squares without a shuffle.
    const int ew = warp - CH_EPI_WARP0, quad = warp & 3, chunk = ew >> 2;
    const int et = threadIdx.x - CH_EPI_WARP0 * 32;  // 0 .. 511
    asm volatile("griddepcontrol.wait;" ::: "memory");
    uint32_t g_prev = 0;                             // generation seen by thread et == 0 when it arrived at the last barrier
    const uint32_t acc_empty_leader0 = cluster_addr(&acc_empty[0], 0);
    float *part = A.partial + (static_cast<size_t>(pair) * 2 + rank) * (static_cast<size_t>(CH_TOK) * CH_FEAT);
    int item_no = 0;
    for (int p = 0; p < A.n_phases; ++p) {
      const ChainPhase &ph = A.ph[p];
      if (p > 0) {                                   // phase p - 1 is complete everywhere (its outputs, its sums of squares)
        if (et == 0) {
          bool ok = false;
          if (leader) {
            for (uint32_t i = 0; i < CH_SPIN_LIMIT && !ok; ++i) {
              ok = ld_acquire_u32(grid_bar + 1) != g_prev;
              if (!ok) { if (*abort_flag) break; __nanosleep(200); }
            }
            if (ok) {
              st_release_cluster_smem(cluster_addr(const_cast<uint32_t *>(&pub[p - 1]), 1), 1u);
              st_release_cluster_smem(cluster_addr(const_cast<uint32_t *>(&pub[p - 1]), 0), 1u);
            }
          } else {
            for (uint32_t i = 0; i < CH_SPIN_LIMIT && !ok; ++i) {
              ok = ld_acquire_cluster_smem(&pub[p - 1]) != 0u;
              if (!ok) { if (*abort_flag) break; __nanosleep(100); }
            }
          }
          if (!ok) { set_status(A.status, ST_TIMEOUT); *abort_flag = 1; }
          trace(A, 9 + 6 * (p - 1));
        }
        asm volatile("bar.sync 1, %0;" ::"n"(CH_EPI_THREADS) : "memory");
      }
      ChainItem it;
      for (int idx = 0; chain_item(ph, A.P, pair, idx, it); ++idx) {
        const int m0 = (it.unit % A.mblocks) * (2 * CH_TOK) + static_cast<int>(rank) * CH_TOK;   // this CTA's first token row
        const int n0 = (it.unit / A.mblocks) * CH_FEAT;
        const int buf = item_no & 1;
        // 1 / rms of this CTA's token rows, from the producing phase's sums of squares per 64 features: four partial
        // sums per row (groups g = part mod 4, ascending), added in a fixed order
        if (ph.sq_in) {
          const int t = et & (CH_TOK - 1), part4 = et >> 7;
          float sacc = 0.f;
          if (m0 + t < A.M)
            for (int g = part4; g < ph.sq_groups; g += 4) sacc += __ldcg(ph.sq_in + static_cast<size_t>(g) * A.m_pad + m0 + t);
          rtmp[part4 * CH_TOK + t] = sacc;
        }
        asm volatile("bar.sync 1, %0;" ::"n"(CH_EPI_THREADS) : "memory");
        if (et < CH_TOK)
          rstd[et] = ph.sq_in ? rsqrtf(((rtmp[et] + rtmp[CH_TOK + et]) + (rtmp[2 * CH_TOK + et] + rtmp[3 * CH_TOK + et])) * ph.inv_dim + A.eps)
                              : 1.f;
        asm volatile("bar.sync 1, %0;" ::"n"(CH_EPI_THREADS) : "memory");
        bool acc_ok = mbar_wait_abortable(&acc_full[buf], (item_no >> 1) & 1, abort_flag);
        if (!acc_ok) { set_status(A.status, ST_TIMEOUT); *abort_flag = 1; }
        tc_fence_after();
        if (et == 0 && idx == 0) trace(A, 7 + 6 * p);
        if (lane == 0 && idx == 0 && p == A.trace_phase) trace(A, 48 + ew);
        const int tl = quad * 32 + lane, m = m0 + tl;            // token lane, token row
        const bool row_live = m < A.M;
        const float rs = rstd[tl];
        float ssq = 0.f;                                         // sum of squares of this thread's 64 results
#pragma unroll 1
        for (int h = 0; h < 2; ++h) {
          const int cbase = chunk * 64 + h * 32, n = n0 + cbase; // 32 feature columns
          uint32_t v[32];
          if (acc_ok) {
            tc_ld_32x32(tmem + (static_cast<uint32_t>(quad * 32) << 16) + buf * acc_cols + cbase, v);
            tc_wait_ld();
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = 0u;
          }
          if (it.ns > 1) {                           // K slice: park the partial sums, [token][256 features]
            float4 *dst = reinterpret_cast<float4 *>(part + static_cast<size_t>(tl) * CH_FEAT + cbase);
#pragma unroll
            for (int j = 0; j < 8; ++j)
              dst[j] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]),
                                   __uint_as_float(v[4 * j + 3]));
            continue;
          }
          if (!row_live || n >= ph.N) continue;      // N is a multiple of 32 (launch_chain checks)
          if (ph.epi == EPI_SWIGLU_BF16) {           // columns (2 i, 2 i + 1) = (gate_i, up_i)
            uint32_t o[8];
#pragma unroll
            for (int j = 0; j < 8; ++j)
              o[j] = pack_bf16(silu_mul(__uint_as_float(v[4 * j]) * rs, __uint_as_float(v[4 * j + 1]) * rs),
                               silu_mul(__uint_as_float(v[4 * j + 2]) * rs, __uint_as_float(v[4 * j + 3]) * rs));
            uint4 *dst = reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(ph.out) + static_cast<size_t>(m) * ph.ldo + (n >> 1));
            dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
            dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
          } else if (ph.epi == EPI_STORE_BF16) {
            uint4 *dst = reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(ph.out) + static_cast<size_t>(m) * ph.ldo + n);
#pragma unroll
            for (int j = 0; j < 4; ++j)
              dst[j] = make_uint4(pack_bf16(__uint_as_float(v[8 * j]) * rs, __uint_as_float(v[8 * j + 1]) * rs),
                                  pack_bf16(__uint_as_float(v[8 * j + 2]) * rs, __uint_as_float(v[8 * j + 3]) * rs),
                                  pack_bf16(__uint_as_float(v[8 * j + 4]) * rs, __uint_as_float(v[8 * j + 5]) * rs),
                                  pack_bf16(__uint_as_float(v[8 * j + 6]) * rs, __uint_as_float(v[8 * j + 7]) * rs));
          } else {                                   // residual-stream update (EPI_ADD_F32) or plain fp32 store
            float4 *o4 = reinterpret_cast<float4 *>(reinterpret_cast<float *>(ph.out) + static_cast<size_t>(m) * ph.ldo + n);
            float x[32];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
              if (ph.epi == EPI_ADD_F32) r = o4[j];
              x[4 * j] = __uint_as_float(v[4 * j]) * rs + r.x; x[4 * j + 1] = __uint_as_float(v[4 * j + 1]) * rs + r.y;
              x[4 * j + 2] = __uint_as_float(v[4 * j + 2]) * rs + r.z; x[4 * j + 3] = __uint_as_float(v[4 * j + 3]) * rs + r.w;
              o4[j] = make_float4(x[4 * j], x[4 * j + 1], x[4 * j + 2], x[4 * j + 3]);
            }
#pragma unroll
            for (int j = 0; j < 32; ++j) ssq += x[j] * x[j];
            if (ph.xg) {
              const uint4 *gw = reinterpret_cast<const uint4 *>(ph.gamma + n);
              uint4 *dst = reinterpret_cast<uint4 *>(ph.xg + static_cast<size_t>(m) * ph.N + n);
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const uint4 g = gw[j];
                dst[j] = make_uint4(pack_bf16(x[8 * j] * bf16_lo(g.x), x[8 * j + 1] * bf16_hi(g.x)),
                                    pack_bf16(x[8 * j + 2] * bf16_lo(g.y), x[8 * j + 3] * bf16_hi(g.y)),
                                    pack_bf16(x[8 * j + 4] * bf16_lo(g.z), x[8 * j + 5] * bf16_hi(g.z)),
                                    pack_bf16(x[8 * j + 6] * bf16_lo(g.w), x[8 * j + 7] * bf16_hi(g.w)));
              }
            }
          }
        }
        if (it.ns == 1 && ph.sq_out && row_live && n0 + chunk * 64 < ph.N)
          ph.sq_out[static_cast<size_t>((n0 >> 6) + chunk) * A.m_pad + m] = ssq;
        // this accumulator may be overwritten by the pair's next tile
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(acc_empty_leader0 + buf * 8);
        ++item_no;
        if (it.ns > 1) {
          // all K slices of the tile have parked their partial sums
          asm volatile("bar.sync 1, %0;" ::"n"(CH_EPI_THREADS) : "memory");
          if (et == 0 && p == A.trace_phase) trace(A, 56);
          if (et == 0) {
            uint32_t *tb = A.sync + 4 + (static_cast<size_t>(it.base) * 2 + rank) * 2;
            const uint32_t g = gbar_arrive(tb, static_cast<uint32_t>(it.ns));
            bool ok = false;
            for (uint32_t i = 0; i < CH_SPIN_LIMIT && !ok; ++i) {
              ok = ld_acquire_u32(tb + 1) != g;
              if (!ok) { if (*abort_flag) break; __nanosleep(100); }
            }
            if (!ok) { set_status(A.status, ST_TIMEOUT); *abort_flag = 1; }
            if (p == A.trace_phase) trace(A, 57);
          }
          asm volatile("bar.sync 1, %0;" ::"n"(CH_EPI_THREADS) : "memory");
          // this CTA's K slice owner reduces one slice of its 128 token rows over all partials, in slice order
          const bool go = !*abort_flag;
          const int per = (CH_TOK + it.ns - 1) / it.ns;
          const int c_lo = it.split * per, c_hi = min(CH_TOK, c_lo + per);
          const float *pbase = A.partial + (static_cast<size_t>(it.base) * 2 + rank) * (static_cast<size_t>(CH_TOK) * CH_FEAT);
          const size_t pstride = 2 * static_cast<size_t>(CH_TOK) * CH_FEAT;   // next slice's slot of the same rank
          for (int i = et; go && i < (c_hi - c_lo) * (CH_FEAT / 4); i += CH_EPI_THREADS) {
            const int c = c_lo + i / (CH_FEAT / 4), r4 = (i % (CH_FEAT / 4)) * 4;
            const int mm = m0 + c, nn = n0 + r4;
            const bool live = mm < A.M && nn < ph.N;                         // N is a multiple of 32: four features are in or out together
            float4 xo = make_float4(0.f, 0.f, 0.f, 0.f);
            float *o = reinterpret_cast<float *>(ph.out) + static_cast<size_t>(mm) * ph.ldo + nn;
            if (live && ph.epi == EPI_ADD_F32) xo = *reinterpret_cast<const float4 *>(o);
            float4 pv[8];
#pragma unroll
            for (int q = 0; q < 8; ++q)
              pv[q] = q < it.ns ? __ldcg(reinterpret_cast<const float4 *>(pbase + q * pstride + static_cast<size_t>(c) * CH_FEAT + r4))
                                : make_float4(0.f, 0.f, 0.f, 0.f);
            float4 acc = pv[0];
#pragma unroll
            for (int q = 1; q < 8; ++q) { acc.x += pv[q].x; acc.y += pv[q].y; acc.z += pv[q].z; acc.w += pv[q].w; }
            const float rs2 = rstd[c];
            acc.x *= rs2; acc.y *= rs2; acc.z *= rs2; acc.w *= rs2;
            if (ph.epi == EPI_SWIGLU_BF16) {
              if (live)
                *reinterpret_cast<uint32_t *>(reinterpret_cast<__nv_bfloat16 *>(ph.out) + static_cast<size_t>(mm) * ph.ldo + (nn >> 1)) =
                    pack_bf16(silu_mul(acc.x, acc.y), silu_mul(acc.z, acc.w));
            } else if (ph.epi == EPI_STORE_BF16) {
              if (live) {
                uint2 ov;
                ov.x = pack_bf16(acc.x, acc.y);
                ov.y = pack_bf16(acc.z, acc.w);
                *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(ph.out) + static_cast<size_t>(mm) * ph.ldo + nn) = ov;
              }
            } else {
              acc.x += xo.x; acc.y += xo.y; acc.z += xo.z; acc.w += xo.w;
              if (live) {
                *reinterpret_cast<float4 *>(o) = acc;
                if (ph.xg) {
                  const uint2 gw = *reinterpret_cast<const uint2 *>(ph.gamma + nn);
                  uint2 ov;
                  ov.x = pack_bf16(acc.x * bf16_lo(gw.x), acc.y * bf16_hi(gw.x));
                  ov.y = pack_bf16(acc.z * bf16_lo(gw.y), acc.w * bf16_hi(gw.y));
                  *reinterpret_cast<uint2 *>(ph.xg + static_cast<size_t>(mm) * ph.N + nn) = ov;
                }
              } else {
                acc = make_float4(0.f, 0.f, 0.f, 0.f);
              }
              if (ph.sq_out) {                       // sixteen lanes cover 64 features
                float ss = acc.x * acc.x + acc.y * acc.y + acc.z * acc.z + acc.w * acc.w;
                ss += __shfl_xor_sync(0xffffffffu, ss, 1);
                ss += __shfl_xor_sync(0xffffffffu, ss, 2);
                ss += __shfl_xor_sync(0xffffffffu, ss, 4);
                ss += __shfl_xor_sync(0xffffffffu, ss, 8);
                if ((lane & 15) == 0 && live) ph.sq_out[static_cast<size_t>(nn >> 6) * A.m_pad + mm] = ss;
              }
            }
          }
          if (lane == 0 && p == A.trace_phase) trace(A, 32 + ew);
        }
      }
      if (p + 1 < A.n_phases) {                      // this CTA's part of the phase is in global memory
        asm volatile("bar.sync 1, %0;" ::"n"(CH_EPI_THREADS) : "memory");
        if (et == 0) {
          trace(A, 8 + 6 * p);
          fence_proxy_async_all();
          g_prev = gbar_arrive(grid_bar, n_ctas);
        }
      }
    }
    if (et == 0) trace(A, 30);
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) trace(A, 31);
  cluster.sync();                                    // neither CTA frees tensor memory or exits while the other may still use it
  if (warp == CH_MMA_WARP) tc2_dealloc(tmem, ncols);
}

// ---- host side --------------------------------------------------------------------------------------------------------------
static size_t chain_smem() { return static_cast<size_t>(CH_STAGES) * CH_STAGE_BYTES + 4096 + 1024; }
static cudaError_t chain_configure() {
  static bool done[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev] = true;
  return e;
}

cudaError_t chain_max_pairs(int *out) {
  cudaError_t e = chain_configure();
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2, 1, 1);
  cfg.blockDim = dim3(CH_THREADS);
  cfg.dynamicSmemBytes = chain_smem();
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaOccupancyMaxActiveClusters(out, chain_kernel, &cfg);
}

void chain_schedule(ChainPhase &ph, int mblocks, int P) {
  const int ptiles = (ph.N + CH_FEAT - 1) / CH_FEAT, KB = ph.K / CH_BK;
  const int U = ptiles * mblocks;
  if (U >= P) {
    ph.full = U / P;
    ph.rem = U % P;
    ph.ns = ph.rem ? P / ph.rem : 0;
  } else {
    ph.full = 0;
    ph.rem = U;
    ph.ns = P / U;
  }
  if (ph.ns > 8) ph.ns = 8;
  if (ph.ns > KB) ph.ns = KB;
}

cudaError_t launch_chain(const ChainArgs &A, cudaStream_t stream) {
  if (A.n_phases < 1 || A.n_phases > CH_MAX_PHASES || A.M < 1 || A.P < 1 || A.mblocks != (A.M + 2 * CH_TOK - 1) / (2 * CH_TOK) ||
      !A.partial || !A.sync || !A.status || A.npw < 1 || A.npw > CH_MAX_NPW || A.npa < 1 || A.npa > CH_MAX_NPA)
    return cudaErrorInvalidValue;
  for (int p = 0; p < A.n_phases; ++p)
    if ((A.ph[p].K % CH_BK) || (A.ph[p].N % 32) || A.ph[p].K < CH_BK || (A.ph[p].ldo % 8)) return cudaErrorInvalidValue;
  cudaError_t e = chain_configure();
  if (e != cudaSuccess) return e;
  return launch_kc(chain_kernel, dim3(2 * A.P), dim3(CH_THREADS), chain_smem(), stream, dim3(2, 1, 1), A);
}

}  // namespace gm
