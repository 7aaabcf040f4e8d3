// chain_kernel: a decoder layer's dense projections as ONE persistent launch.
//
// Between two attention calls a layer runs four dependent projections on the same few hundred token rows - output
// projection (+ residual), gate/up (+ SwiGLU), down (+ residual), and the next layer's QKV - with an RMSNorm in front
// of the second and the fourth.  As separate launches each pays its own set-up, first fill of the stage ring, split-K
// reduction and drain, which at these sizes is as long as the main loop itself.  Here the whole chain is one grid of
// CTA pairs (one pair per two SMs, all resident at once) that walks the projections ("phases") in order:
//
//   * a pair's tile is 256 token rows (128 per CTA, on the lanes of tensor memory) x W output features, W a multiple of
//     16 up to 288, computed by tcgen05.mma cta_group::2 (M = 256, N = W as one or two instructions per K step).  Per
//     K block of 64 a CTA stages its own 128 x 64 activation box and W / 2 weight rows.  The features of a phase are
//     dealt out in near-equal tiles, as many as there are pairs, so every phase is one wave: wide projections get
//     W = 256 / 272, narrow ones thin tiles (W = 32 ... 96) instead of a deep split along K - a thin tile re-reads the
//     activations from L2 more often, but leaves nothing to reduce across SMs.  Only a projection with a long K and few
//     features (down) is cut along K as well, over ns = 2 ... 8 consecutive pairs: the K slices leave fp32 partial sums
//     in an L2-resident scratch slot per CTA, meet at a counter of their own, and each slice owner reduces one slice of
//     the tile's token rows over all partials in slice order (the result does not depend on timing).
//   * every pair keeps one ring of shared-memory stages alive across phases.  Weights depend on nothing, so the weight
//     producers stream the next phase's boxes into free stages while the current phase is still draining; only the
//     activation boxes wait for the grid-wide barrier that ends the phase before.  One thread sustains only about four
//     (wait, copy) rounds per microsecond, so weights and activations have two producer threads each.
//   * the RMSNorms are folded around the projections: W (x g / rms) = (W (x g)) / rms.  The phase that updates the
//     residual stream x also writes bf16(x g) for the next norm's weight g and, per tile and token row, the sum of
//     squares of its results (plain stores, no atomics); the consuming phase adds those partial sums in a fixed order
//     and scales its accumulator rows by rsqrt(mean + eps) in the epilogue.
//   * the epilogue warps read the accumulator straight out of tensor memory: a thread owns one token row and 16
//     consecutive features at a time, so stores are whole 32-byte sectors, SwiGLU pairs sit in neighbouring registers
//     and a row's sum of squares needs no shuffle.
//
// Barriers in global memory are monotonic 64-bit counters (one atomic per arrival; the barrier is complete when the
// counter reaches the next multiple of the participant count).  Only one thread per pair polls the grid counter - more
// pollers slow every other access to that L2 slice - and hands the news to both CTAs through shared memory.
// Every wait (mbarrier, grid barrier, slice barrier) is bounded: on expiry the kernel records ST_TIMEOUT, raises a
// CTA-wide abort flag that makes every later wait return at once, still meets its CTA / cluster barriers, frees its
// tensor memory and returns.
#include <cooperative_groups.h>

#include "common.cuh"
#include "kernels.h"

namespace cg = cooperative_groups;

namespace gm {

constexpr int CH_MAX_NPW = 4, CH_MAX_NPA = 2;      // producer warps: weights, activations
constexpr int CH_PROD_WARPS = CH_MAX_NPW + CH_MAX_NPA;
constexpr int CH_MMA_WARP = CH_PROD_WARPS;         // tensor-memory owner + MMA issuer
constexpr int CH_EPI_WARP0 = CH_MMA_WARP + 1;      // first of the 16 epilogue warps
constexpr int CH_EPI_WARPS = 16;
constexpr int CH_EPI_THREADS = CH_EPI_WARPS * 32;
constexpr int CH_THREADS = (CH_EPI_WARP0 + CH_EPI_WARPS) * 32;
constexpr int CH_MAX_PHASES = 4;
constexpr int CH_BK = 64;              // K elements per stage (one 128-byte swizzle row)
constexpr int CH_TOK = 128;            // token rows per CTA (a pair's tile has 256)
constexpr int CH_WMAX = 288;           // widest tile (features); each CTA stages half of a tile's weight rows
constexpr int CH_A_BYTES = CH_TOK * 128;                    // activation box: 128 tokens x 64 K elements
constexpr int CH_STAGE_BYTES = CH_A_BYTES + (CH_WMAX / 2) * 128;   // + up to 144 weight rows
constexpr int CH_STAGES = 6;
constexpr uint32_t CH_SPIN_LIMIT = 1u << 22;

// ---- global-memory barriers: monotonic counters ---------------------------------------------------------------------------
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long *p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
// One thread per participant, after a CTA-level barrier that follows the CTA's stores.  Returns the count at which the
// barrier of n participants is complete.
__device__ __forceinline__ unsigned long long gbar_arrive(unsigned long long *cnt, unsigned long long n) {
  unsigned long long old;
  __threadfence();
  asm volatile("atom.acq_rel.gpu.global.add.u64 %0, [%1], 1;" : "=l"(old) : "l"(cnt) : "memory");
  return (old / n + 1) * n;
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

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
__device__ __forceinline__ bool mbar_wait_abortable(uint64_t *bar, uint32_t parity, volatile int *abort_flag) {
  for (uint32_t i = 0; i < CH_SPIN_LIMIT; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 255u) == 255u && *abort_flag) return false;
  }
  return false;
}

// The same for the many threads that wait out a whole main loop: polls a few times per microsecond and sleeps in
// between, so that the waiters take no issue slots from the producer and MMA warps.
__device__ __forceinline__ bool mbar_wait_sleeping(uint64_t *bar, uint32_t parity, volatile int *abort_flag) {
  for (uint32_t i = 0; i < CH_SPIN_LIMIT; ++i) {
    if (mbar_test_wait(bar, parity)) return true;
    if ((i & 15u) == 15u && *abort_flag) return false;
    __nanosleep(200);
  }
  return false;
}

// ---- the schedule: which tile of a phase a pair works on --------------------------------------------------------------------
// A phase has `tiles` feature tiles x mblocks token blocks = U units, each cut into ns K slices: U * ns items.  Pair p
// of the first P' = P - P % ns pairs takes items p, p + P', ...; item v = (unit v / ns, slice v % ns), so the slices of
// a unit sit on ns consecutive pairs starting at a multiple of ns.
struct ChainItem {
  int mb, tile;    // token block, feature tile
  int f0, W;       // first feature and width of the tile
  int split, ns;   // K slice and slices of this unit
  int base;        // first pair of the unit's slice group
  int kb_lo, kb_hi;
};
__device__ __forceinline__ bool chain_item(const ChainPhase &ph, int mblocks, int P, int pair, int idx, ChainItem &it) {
  const int Pp = P - P % ph.ns;
  if (pair >= Pp) return false;
  const int v = pair + idx * Pp;
  if (v >= ph.tiles * mblocks * ph.ns) return false;
  const int unit = v / ph.ns;
  it.split = v % ph.ns; it.ns = ph.ns; it.base = pair - it.split;
  it.mb = unit % mblocks; it.tile = unit / mblocks;              // token blocks vary fastest: neighbours share a weight tile
  const int g_lo = static_cast<int>(static_cast<long long>(it.tile) * ph.G / ph.tiles);
  const int g_hi = static_cast<int>(static_cast<long long>(it.tile + 1) * ph.G / ph.tiles);
  it.f0 = g_lo * 16; it.W = (g_hi - g_lo) * 16;
  const int KB = ph.K / CH_BK;
  it.kb_lo = static_cast<int>(static_cast<long long>(it.split) * KB / ph.ns);
  it.kb_hi = static_cast<int>(static_cast<long long>(it.split + 1) * KB / ph.ns);
  return true;
}
// Walks the K blocks of all items of all phases of one pair in order (producers and MMA thread use the same walk).
struct SlotIter {
  int ph, idx, kb;
  ChainItem it;
  bool valid;
  __device__ __forceinline__ void seek(const ChainArgs &A, int pair) {
    while (ph < A.n_phases) {
      if (chain_item(A.ph[ph], A.mblocks, A.P, pair, idx, it)) {
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
// Feature (relative to the tile's first) held by accumulator column `col` (a multiple of 4; runs of 8 columns stay
// contiguous).  One MMA (W <= 256): the even CTA's W / 2 weight rows are columns [0, W/2), the odd CTA's [W/2, W):
// identity.  Two MMAs (W > 256) of n1 and W - n1 columns: the first takes the first n1 / 2 weight rows of both CTAs'
// boxes, the second the rows behind.
__device__ __forceinline__ int chain_n1(int W) { return W <= 256 ? W : 16 * ((W + 31) / 32); }
__device__ __forceinline__ int chain_col_feature(int col, int W) {
  if (W <= 256) return col;
  const int hw = W >> 1, n1 = chain_n1(W), h1 = n1 >> 1;      // first MMA: n1 columns, h1 weight rows of each CTA
  if (col < n1) return (col / h1) * hw + col % h1;
  const int h2 = (W - n1) >> 1, c2 = col - n1;
  return (c2 / h2) * hw + h1 + c2 % h2;
}

// Optional trace (ChainArgs::timeline): nanosecond stamps per CTA, 64 slots each.  Slot 0 entry, 1 set-up done,
// 2 previous kernel complete (activation producer), 30 epilogue warps done, 31 exit; per phase p from slot 4 + 6 p:
// first activation box issued, first stage consumed by the MMA thread, last MMA issued, first accumulator complete,
// epilogue of the phase done, the barrier that ends the phase seen complete.  For phase trace_phase: 56 partial sums
// parked, 57 slice barrier passed, 32 + w reduction of epilogue warp w done, 48 + w its accumulator wait returned.
__device__ __forceinline__ void trace(const ChainArgs &A, int slot) {
  if (A.timeline) {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)::"memory");
    A.timeline[static_cast<size_t>(blockIdx.x) * 64 + slot] = t;
  }
}

__device__ __forceinline__ unsigned long long now_ns() {     // SM clock cycles (cheap to read), for interval sums
  unsigned long long t;
  asm volatile("mov.u64 %0, %%clock64;" : "=l"(t)::"memory");
  return t;
}
__device__ __forceinline__ void trace_value(const ChainArgs &A, int slot, unsigned long long v) {
  if (A.timeline) A.timeline[static_cast<size_t>(blockIdx.x) * 64 + slot] = v;
}

// 32-byte store: a whole L2 sector per thread and instruction
__device__ __forceinline__ void st_v8(float *p, const uint32_t *v) {
  asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(__uint_as_float(v[0])), "f"(__uint_as_float(v[1])),
               "f"(__uint_as_float(v[2])), "f"(__uint_as_float(v[3])), "f"(__uint_as_float(v[4])), "f"(__uint_as_float(v[5])),
               "f"(__uint_as_float(v[6])), "f"(__uint_as_float(v[7]))
               : "memory");
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
  uint64_t *acc_full = empty + CH_STAGES;
  uint64_t *acc_empty = acc_full + 1;                // the leader's is the one waited on
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 1);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  float *rstd = reinterpret_cast<float *>(tmem_slot + 4);   // [128] 1 / rms of this CTA's token rows
  float *rtmp = rstd + CH_TOK;                               // [4][128] partial sums (1 / rms input; sums of squares output)
  volatile uint32_t *pub = reinterpret_cast<volatile uint32_t *>(rtmp + 4 * CH_TOK);   // pub[p] != 0: the barrier that ends phase p is complete

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();
  const bool leader = rank == 0;
  const int pair = blockIdx.x >> 1;
  constexpr uint32_t ncols = 512u;                   // one accumulator: 128 token lanes x up to 288 feature columns
  const unsigned long long n_ctas = static_cast<unsigned long long>(A.P) * 2u;
  unsigned long long *grid_bar = A.sync;
  if (threadIdx.x == 0) trace(A, 0);

  if (threadIdx.x == 0) {
    for (int s = 0; s < nstages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    mbar_init(acc_empty, 2 * CH_EPI_WARPS);
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
      unsigned long long t_wait = 0, t_issue = 0;
      const bool timed = A.timeline != nullptr && A.trace_phase >= 100 && pi == 0;   // interval sums perturb the loop: on request only
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
              if (!seen) { if (*abort_flag) break; __nanosleep(50); }
            }
            if (!seen) { ok = false; break; }
            fence_proxy_async_all();                 // other CTAs' stores, seen through the barrier, before the TMA reads
          }
          phase_ok = it.ph + 1;
          if (pi == 0) trace(A, 4 + 6 * it.ph);
        }
        const unsigned long long ta = timed ? now_ns() : 0;
        if (!mbar_wait_abortable(&empty[s], ((q / nstages) & 1) ^ 1, abort_flag)) { ok = false; break; }
        const unsigned long long tb = timed ? now_ns() : 0;
        const ChainPhase &ph = A.ph[it.ph];
        unsigned char *dst = smem + static_cast<size_t>(s) * stage_b;
        if (is_w) {
          if (leader) mbar_expect_tx(&full[s], 2 * (CH_A_BYTES + ph.wbox * 128));
          tma2_load_2d(dst + CH_A_BYTES, &ph.w_map, it.kb * CH_BK, it.it.f0 + static_cast<int>(rank) * (it.it.W >> 1), full0 + s * 8);
        } else {
          tma2_load_2d(dst, &ph.x_map, it.kb * CH_BK, it.it.mb * (2 * CH_TOK) + static_cast<int>(rank) * CH_TOK, full0 + s * 8);
        }
        if (timed) { t_wait += tb - ta; t_issue += now_ns() - tb; }
        last_q = q;
      }
      if (timed) { trace_value(A, is_w ? 60 : 62, t_wait); trace_value(A, is_w ? 61 : 63, t_issue); }
      if (!ok) { set_status(A.status, ST_TIMEOUT); *abort_flag = 1; }
      // the copies this thread issued have landed before the CTA may exit: their stages have been consumed
      if (last_q >= 0) {
        bool done = false;
        for (uint32_t i = 0; i < (1u << 16) && !done; ++i) done = mbar_try_wait(&empty[last_q % nstages], (last_q / nstages) & 1);
      }
    }
  } else if (warp == CH_MMA_WARP) {
    // ================= MMA issuer (leader CTA of the pair) =================
    // D[256 tokens x W features] += A[256 tokens x 64] * B[W features x 64]^T: each CTA holds its 128 token rows of A
    // and of D and stages W / 2 of the feature rows of B.
    if (lane == 0 && leader) {
      int q = 0, item_no = 0;
      bool ok = true;
      unsigned long long t_wait = 0, t_issue = 0, pw[4] = {0, 0, 0, 0}, pi_[4] = {0, 0, 0, 0};
      const bool timed = A.timeline != nullptr && A.trace_phase >= 100;
      const uint32_t smem0 = smem_u32(smem);
      for (int p = 0; p < A.n_phases && ok; ++p) {
        ChainItem it;
        for (int idx = 0; ok && chain_item(A.ph[p], A.mblocks, A.P, pair, idx, it); ++idx) {
          // a new tile: the accumulator must have been drained
          if (!mbar_wait_abortable(acc_empty, (item_no & 1) ^ 1, abort_flag)) { ok = false; break; }
          tc_fence_after();
          // one MMA per K step for tiles up to 256 features; wider tiles as two of about half the width each (an
          // instruction of this shape takes at least ~85 cycles however narrow, and N / 2 cycles beyond N = 170)
          const int W = it.W, n1 = chain_n1(W), n2 = W - n1;
          const uint32_t idesc1 = tc_idesc_bf16(2 * CH_TOK, n1), idesc2 = n2 ? tc_idesc_bf16(2 * CH_TOK, n2) : 0u;
          const uint32_t b2_off = static_cast<uint32_t>(n1 >> 1) * 128u;
          for (int kb = it.kb_lo; kb < it.kb_hi; ++kb, ++q) {
            const int s = q % nstages;
            const unsigned long long ta = timed ? now_ns() : 0;
            if (!mbar_wait_abortable(&full[s], (q / nstages) & 1, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const unsigned long long tb = timed ? now_ns() : 0;
            if (idx == 0 && kb == it.kb_lo) trace(A, 5 + 6 * p);
            const uint32_t a_addr = smem0 + static_cast<uint32_t>(s) * stage_b;
            const uint64_t adesc = tc_smem_desc_sw128(a_addr), bdesc = tc_smem_desc_sw128(a_addr + CH_A_BYTES);
            const uint32_t acc = kb > it.kb_lo ? 1u : 0u;
            if (n2 == 0) {
              tc2_mma_bf16(tmem, adesc, bdesc, idesc1, acc);
#pragma unroll
              for (int k = 1; k < CH_BK / 16; ++k) tc2_mma_bf16(tmem, adesc + 2 * k, bdesc + 2 * k, idesc1, 1u);
            } else {
              // Two column ranges (the second from the weight rows behind the first n1 / 2 of both CTAs' boxes), issued
              // alternately: consecutive MMAs into the SAME accumulator wait for one another (about 85 cycles each,
              // measured), MMAs into different column ranges overlap.
              const uint64_t bdesc2 = tc_smem_desc_sw128(a_addr + CH_A_BYTES + b2_off);
#pragma unroll
              for (int k = 0; k < CH_BK / 16; ++k) {
                tc2_mma_bf16(tmem, adesc + 2 * k, bdesc + 2 * k, idesc1, k > 0 ? 1u : acc);
                tc2_mma_bf16(tmem + n1, adesc + 2 * k, bdesc2 + 2 * k, idesc2, k > 0 ? 1u : acc);
              }
            }
            tc2_commit_mc(&empty[s], 3);             // the stage is free in both CTAs once these MMAs have read it
            if (timed) {
              const unsigned long long tc = now_ns();
              t_wait += tb - ta; t_issue += tc - tb;
              pw[p] += tb - ta; pi_[p] += tc - tb;
            }
          }
          if (!ok) break;
          tc2_commit_mc(acc_full, 3);                // the tile's accumulator is complete in both CTAs
          ++item_no;
          trace(A, 6 + 6 * p);
        }
      }
      if (timed) {
        trace_value(A, 58, t_wait); trace_value(A, 59, t_issue);
        for (int p = 0; p < 4; ++p) { trace_value(A, 40 + 2 * p, pw[p]); trace_value(A, 41 + 2 * p, pi_[p]); }
      }
      if (!ok) { set_status(A.status, ST_TIMEOUT); *abort_flag = 1; }
    }
  } else {
    // ================= epilogue warps (both CTAs: each drains its 128 token rows x W features) =================
    // Warp (quad, chunk): token lanes quad * 32 .. + 31 (the quadrant of tensor memory the warp may read), 16-column
    // blocks chunk, chunk + 4, ...
    const int ew = warp - CH_EPI_WARP0, quad = warp & 3, chunk = ew >> 2;
    const int et = threadIdx.x - CH_EPI_WARP0 * 32;  // 0 .. 511
    asm volatile("griddepcontrol.wait;" ::: "memory");
    unsigned long long g_target = 0;                 // count at which the barrier thread et == 0 last arrived at is complete
    const uint32_t acc_empty_leader = cluster_addr(acc_empty, 0);
    float *part = A.partial + (static_cast<size_t>(pair) * 2 + rank) * (static_cast<size_t>(CH_TOK) * CH_WMAX);
    int item_no = 0;
    for (int p = 0; p < A.n_phases; ++p) {
      const ChainPhase &ph = A.ph[p];
      if (p > 0) {                                   // phase p - 1 is complete everywhere (its outputs, its sums of squares)
        if (et == 0) {
          bool ok = false;
          if (leader) {
            for (uint32_t i = 0; i < CH_SPIN_LIMIT && !ok; ++i) {
              ok = ld_acquire_u64(grid_bar) >= g_target;
              if (!ok) { if (*abort_flag) break; __nanosleep(100); }
            }
            if (ok) {
              st_release_cluster_smem(cluster_addr(const_cast<uint32_t *>(&pub[p - 1]), 1), 1u);
              st_release_cluster_smem(cluster_addr(const_cast<uint32_t *>(&pub[p - 1]), 0), 1u);
            }
          } else {
            for (uint32_t i = 0; i < CH_SPIN_LIMIT && !ok; ++i) {
              ok = ld_acquire_cluster_smem(&pub[p - 1]) != 0u;
              if (!ok) { if (*abort_flag) break; __nanosleep(50); }
            }
          }
          if (!ok) { set_status(A.status, ST_TIMEOUT); *abort_flag = 1; }
          trace(A, 9 + 6 * (p - 1));
        }
        asm volatile("bar.sync 1, %0;" ::"n"(CH_EPI_THREADS) : "memory");
      }
      ChainItem it;
      for (int idx = 0; chain_item(ph, A.mblocks, A.P, pair, idx, it); ++idx) {
        const int m0 = it.mb * (2 * CH_TOK) + static_cast<int>(rank) * CH_TOK;   // this CTA's first token row
        const int W = it.W, nblk = W >> 4;
        // 1 / rms of this CTA's token rows, from the producing phase's sums of squares per tile: four partial sums per
        // row (tiles g = part mod 4, ascending), added in a fixed order
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
        bool acc_ok = mbar_wait_sleeping(acc_full, item_no & 1, abort_flag);
        if (!acc_ok) { set_status(A.status, ST_TIMEOUT); *abort_flag = 1; }
        tc_fence_after();
        if (et == 0 && idx == 0) trace(A, 7 + 6 * p);
        if (lane == 0 && idx == 0 && p == A.trace_phase) trace(A, 48 + ew);
        const int tl = quad * 32 + lane, m = m0 + tl;            // token lane, token row
        const bool row_live = m < A.M;
        const float rs = rstd[tl];
        float ssq = 0.f;                                         // sum of squares of this thread's results
#pragma unroll 1
        for (int b = chunk; b < nblk; b += 4) {
          const int col = b << 4;                    // 16 accumulator columns
          uint32_t v[16];
          if (acc_ok) {
            tc_ld_32x16(tmem + (static_cast<uint32_t>(quad * 32) << 16) + col, v);
            tc_wait_ld();
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = 0u;
          }
          if (it.ns > 1) {                           // K slice: park the partial sums, [token][columns]
            float *dst = part + static_cast<size_t>(tl) * CH_WMAX + col;
            st_v8(dst, v);
            st_v8(dst + 8, v + 8);
            continue;
          }
          if (!row_live) continue;
          // two runs of 8 columns, each 8 consecutive features (the runs of a block need not be neighbours in a tile of two MMAs)
#pragma unroll
          for (int h8 = 0; h8 < 2; ++h8) {
            const int n = it.f0 + chain_col_feature(col + 8 * h8, W);
            const uint32_t *u = v + 8 * h8;
            if (ph.epi == EPI_SWIGLU_BF16) {         // columns (2 i, 2 i + 1) = (gate_i, up_i)
              uint2 o;
              o.x = pack_bf16(silu_mul(__uint_as_float(u[0]) * rs, __uint_as_float(u[1]) * rs),
                              silu_mul(__uint_as_float(u[2]) * rs, __uint_as_float(u[3]) * rs));
              o.y = pack_bf16(silu_mul(__uint_as_float(u[4]) * rs, __uint_as_float(u[5]) * rs),
                              silu_mul(__uint_as_float(u[6]) * rs, __uint_as_float(u[7]) * rs));
              *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(ph.out) + static_cast<size_t>(m) * ph.ldo + (n >> 1)) = o;
            } else if (ph.epi == EPI_STORE_BF16) {
              *reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(ph.out) + static_cast<size_t>(m) * ph.ldo + n) =
                  make_uint4(pack_bf16(__uint_as_float(u[0]) * rs, __uint_as_float(u[1]) * rs),
                             pack_bf16(__uint_as_float(u[2]) * rs, __uint_as_float(u[3]) * rs),
                             pack_bf16(__uint_as_float(u[4]) * rs, __uint_as_float(u[5]) * rs),
                             pack_bf16(__uint_as_float(u[6]) * rs, __uint_as_float(u[7]) * rs));
            } else {                                 // residual-stream update (EPI_ADD_F32) or plain fp32 store
              float4 *o4 = reinterpret_cast<float4 *>(reinterpret_cast<float *>(ph.out) + static_cast<size_t>(m) * ph.ldo + n);
              float x[8];
#pragma unroll
              for (int j = 0; j < 2; ++j) {
                float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
                if (ph.epi == EPI_ADD_F32) r = o4[j];
                x[4 * j] = __uint_as_float(u[4 * j]) * rs + r.x; x[4 * j + 1] = __uint_as_float(u[4 * j + 1]) * rs + r.y;
                x[4 * j + 2] = __uint_as_float(u[4 * j + 2]) * rs + r.z; x[4 * j + 3] = __uint_as_float(u[4 * j + 3]) * rs + r.w;
                o4[j] = make_float4(x[4 * j], x[4 * j + 1], x[4 * j + 2], x[4 * j + 3]);
              }
#pragma unroll
              for (int j = 0; j < 8; ++j) ssq += x[j] * x[j];
              if (ph.xg) {
                const uint4 g = *reinterpret_cast<const uint4 *>(ph.gamma + n);
                *reinterpret_cast<uint4 *>(ph.xg + static_cast<size_t>(m) * ph.N + n) =
                    make_uint4(pack_bf16(x[0] * bf16_lo(g.x), x[1] * bf16_hi(g.x)), pack_bf16(x[2] * bf16_lo(g.y), x[3] * bf16_hi(g.y)),
                               pack_bf16(x[4] * bf16_lo(g.z), x[5] * bf16_hi(g.z)), pack_bf16(x[6] * bf16_lo(g.w), x[7] * bf16_hi(g.w)));
              }
            }
          }
        }
        // the accumulator may be overwritten by the pair's next tile
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
        ++item_no;
        if (it.ns == 1) {
          if (ph.sq_out) {                           // the row's sum of squares over this tile: four column chunks, fixed order
            rtmp[chunk * CH_TOK + tl] = ssq;
            asm volatile("bar.sync 1, %0;" ::"n"(CH_EPI_THREADS) : "memory");
            if (et < CH_TOK && m0 + et < A.M)
              ph.sq_out[static_cast<size_t>(it.tile) * A.m_pad + m0 + et] =
                  (rtmp[et] + rtmp[CH_TOK + et]) + (rtmp[2 * CH_TOK + et] + rtmp[3 * CH_TOK + et]);
          }
        } else {
          // all K slices of the tile have parked their partial sums
          asm volatile("bar.sync 1, %0;" ::"n"(CH_EPI_THREADS) : "memory");
          if (et == 0 && p == A.trace_phase) trace(A, 56);
          if (et == 0) {
            // the slice groups differ from phase to phase, so their barrier is a {count, generation} pair that the last
            // arrival resets: 32-bit halves of one counter word
            uint32_t *tb = reinterpret_cast<uint32_t *>(A.sync + 1 + static_cast<size_t>(it.base) * 2 + rank);
            uint32_t g, old;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(g) : "l"(tb + 1) : "memory");
            __threadfence();
            asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(old) : "l"(tb) : "memory");
            bool ok = old == static_cast<uint32_t>(it.ns) - 1;
            if (ok) {
              tb[0] = 0u;                            // ordered before the release below
              asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(tb + 1), "r"(g + 1) : "memory");
            }
            for (uint32_t i = 0; i < CH_SPIN_LIMIT && !ok; ++i) {
              uint32_t g2;
              asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(g2) : "l"(tb + 1) : "memory");
              ok = g2 != g;
              if (!ok) { if (*abort_flag) break; __nanosleep(100); }
            }
            if (!ok) { set_status(A.status, ST_TIMEOUT); *abort_flag = 1; }
            if (p == A.trace_phase) trace(A, 57);
          }
          asm volatile("bar.sync 1, %0;" ::"n"(CH_EPI_THREADS) : "memory");
          // this CTA's K slice owner reduces one slice of its 128 token rows over all partials, in slice order: a warp
          // takes whole rows (float4 index = lane, lane + 32, lane + 64), so a row's sum of squares is one warp reduction
          const bool go = !*abort_flag;
          const int per = (CH_TOK + it.ns - 1) / it.ns;
          const int c_lo = it.split * per, c_hi = min(CH_TOK, c_lo + per);
          const float *pbase = A.partial + (static_cast<size_t>(it.base) * 2 + rank) * (static_cast<size_t>(CH_TOK) * CH_WMAX);
          const size_t pstride = 2 * static_cast<size_t>(CH_TOK) * CH_WMAX;   // next slice's slot of the same rank
          for (int c = c_lo + ew; go && c < c_hi; c += CH_EPI_WARPS) {
            const int mm = m0 + c;
            const bool live_row = mm < A.M;
            const float rs2 = rstd[c];
            float ss = 0.f;
#pragma unroll 1
            for (int f4 = lane; f4 < (W >> 2); f4 += 32) {
              const int col = f4 << 2, nn = it.f0 + chain_col_feature(col, W);
              float4 xo = make_float4(0.f, 0.f, 0.f, 0.f);
              float *o = reinterpret_cast<float *>(ph.out) + static_cast<size_t>(mm) * ph.ldo + nn;
              if (live_row && ph.epi == EPI_ADD_F32) xo = *reinterpret_cast<const float4 *>(o);
              float4 pv[8];
#pragma unroll
              for (int q = 0; q < 8; ++q)
                pv[q] = q < it.ns ? __ldcg(reinterpret_cast<const float4 *>(pbase + q * pstride + static_cast<size_t>(c) * CH_WMAX + col))
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
              float4 acc = pv[0];
#pragma unroll
              for (int q = 1; q < 8; ++q) { acc.x += pv[q].x; acc.y += pv[q].y; acc.z += pv[q].z; acc.w += pv[q].w; }
              acc.x *= rs2; acc.y *= rs2; acc.z *= rs2; acc.w *= rs2;
              if (!live_row) continue;
              if (ph.epi == EPI_SWIGLU_BF16) {
                *reinterpret_cast<uint32_t *>(reinterpret_cast<__nv_bfloat16 *>(ph.out) + static_cast<size_t>(mm) * ph.ldo + (nn >> 1)) =
                    pack_bf16(silu_mul(acc.x, acc.y), silu_mul(acc.z, acc.w));
              } else if (ph.epi == EPI_STORE_BF16) {
                uint2 ov;
                ov.x = pack_bf16(acc.x, acc.y);
                ov.y = pack_bf16(acc.z, acc.w);
                *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(ph.out) + static_cast<size_t>(mm) * ph.ldo + nn) = ov;
              } else {
                acc.x += xo.x; acc.y += xo.y; acc.z += xo.z; acc.w += xo.w;
                *reinterpret_cast<float4 *>(o) = acc;
                if (ph.xg) {
                  const uint2 gw = *reinterpret_cast<const uint2 *>(ph.gamma + nn);
                  uint2 ov;
                  ov.x = pack_bf16(acc.x * bf16_lo(gw.x), acc.y * bf16_hi(gw.x));
                  ov.y = pack_bf16(acc.z * bf16_lo(gw.y), acc.w * bf16_hi(gw.y));
                  *reinterpret_cast<uint2 *>(ph.xg + static_cast<size_t>(mm) * ph.N + nn) = ov;
                }
                ss += acc.x * acc.x + acc.y * acc.y + acc.z * acc.z + acc.w * acc.w;
              }
            }
            if (ph.sq_out) {
              ss = warp_sum(ss);
              if (lane == 0 && live_row) ph.sq_out[static_cast<size_t>(it.tile) * A.m_pad + mm] = ss;
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
          g_target = gbar_arrive(grid_bar, n_ctas);
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
  static SmemConfigured configured;
  return ensure_dyn_smem(chain_kernel, 227 * 1024, configured);
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

size_t chain_partial_floats(int pairs) { return static_cast<size_t>(pairs) * 2 * CH_TOK * CH_WMAX; }

// Tiling of one phase: `tiles` near-equal feature tiles (multiples of 16 features, at most 288) and ns K slices per
// tile, chosen from a cost estimate per pair - K blocks x the slower of the tensor time and the time to fill shared
// memory (activation box + weight rows), per wave, plus what the slices' partial sums cost - over ns = 1 ... 8.  A
// deterministic function of (N, K, mblocks, P): the arithmetic of a token row does not depend on the batch it is in.
void chain_schedule(ChainPhase &ph, int mblocks, int P, int force_ns) {
  const int G = ph.N / 16, KB = ph.K / CH_BK;        // groups of 16 features
  ph.G = G;
  const int min_tiles = (G + CH_WMAX / 16 - 1) / (CH_WMAX / 16);
  double best = 1e30;
  int best_ns = 1, best_tiles = min_tiles;
  for (int ns = 1; ns <= 8 && ns <= KB; ++ns) {
    if (force_ns > 0 && ns != force_ns && !(ns == 1 && force_ns > KB)) continue;
    int tiles = (P / ns) / mblocks;                  // one wave if the tiles may be that thin
    if (tiles > G) tiles = G;
    if (tiles < min_tiles) { if (ns > 1) continue; tiles = min_tiles; }   // several waves: no K slices
    const int Pp = P - P % ns;
    const int waves = (tiles * mblocks * ns + Pp - 1) / Pp;
    const int gw = (G + tiles - 1) / tiles;          // widest tile in groups of 16 features
    const int w = 16 * gw, n1 = w <= 256 ? w : 16 * ((w + 31) / 32), n2 = w - n1;
    // measured on B200: one MMA of this shape per K step of 16 takes max(85, N / 2) cycles at 1.965 GHz; a K block costs
    // about 0.1 us of barrier round trips on top; a CTA fills shared memory at roughly 140 KB per us
    const double cyc = (n1 / 2 > 85 ? n1 / 2 : 85) + (n2 ? (n2 / 2 > 85 ? n2 / 2 : 85) : 0);
    const double t_mma = 4.0 * cyc / 1965.0 + 0.1;
    const double t_fill = (CH_A_BYTES + w * 64.0) / 140e3;
    const double blocks = (KB + ns - 1) / ns;
    double t = waves * blocks * (t_mma > t_fill ? t_mma : t_fill);
    // epilogue: straight from tensor memory, or parked partial sums + slice barrier + reduction
    t += ns > 1 ? 5.0 + 2.0 * ns * 256.0 * mblocks * ph.N * 4.0 / 7e6 : 1.5 + 2.0 * w / 256.0;
    if (t < best) { best = t; best_ns = ns; best_tiles = tiles; }
  }
  ph.ns = best_ns;
  ph.tiles = best_tiles;
  ph.wbox = ((G + best_tiles - 1) / best_tiles) * 8;            // weight rows per CTA of the widest tile
}

cudaError_t launch_chain(const ChainArgs &A, cudaStream_t stream) {
  if (A.n_phases < 1 || A.n_phases > CH_MAX_PHASES || A.M < 1 || A.P < 1 || A.mblocks != (A.M + 2 * CH_TOK - 1) / (2 * CH_TOK) ||
      !A.partial || !A.sync || !A.status || A.npw < 1 || A.npw > CH_MAX_NPW || A.npa < 1 || A.npa > CH_MAX_NPA)
    return cudaErrorInvalidValue;
  for (int p = 0; p < A.n_phases; ++p) {
    const ChainPhase &ph = A.ph[p];
    if ((ph.K % CH_BK) || (ph.N % 16) || ph.K < CH_BK || (ph.ldo % 8) || ph.ns < 1 || ph.ns > 8 || ph.tiles < 1 ||
        ph.G != ph.N / 16 || ph.wbox < 8 || ph.wbox > CH_WMAX / 2 || (ph.G + ph.tiles - 1) / ph.tiles * 8 > ph.wbox ||
        (ph.ns > 1 && ph.tiles * A.mblocks * ph.ns > A.P) || (ph.sq_in && ph.sq_out))
      return cudaErrorInvalidValue;
  }
  cudaError_t e = chain_configure();
  if (e != cudaSuccess) return e;
  return launch_kc(chain_kernel, dim3(2 * A.P), dim3(CH_THREADS), chain_smem(), stream, dim3(2, 1, 1), A);
}

}  // namespace gm
