// Speculative rejection sampler, vocabulary-sliced variant (Sec. 2.2, Eq. 1).
//
// Same decisions and the same arithmetic as the other two mappings (sampler_common.cuh); what differs is who does the
// work.  A sequence's walk is serial (position k+1 is looked at only if draft k was accepted, the resampled position is
// known only at the first rejection) and its length varies, so one CTA or cluster per sequence leaves the SMs that drew
// short walks idle while the longest one finishes.  Here every CTA (one per SM) owns the same slice of the vocabulary in
// EVERY row of EVERY sequence, so all CTAs do identical work whatever the walks look like.  The walk of sequence b is
// a list of stages - STAT k (running max and sum of 2^x of the rows p_k, q_k), RES (sum of the 64-bit residual weights
// at the resampled position), SEARCH (token search in the one slice that holds the quantile) - and a stage is done when
// every CTA has delivered its slice: partials go to device memory, an arrival counter per (sequence, stage) is bumped
// with a fire-and-forget reduction.  The CTA that owns the sequence (b mod grid) watches that counter with a warp of
// its own, merges the slices in a fixed order, takes the accept decision and publishes the next stage word; all CTAs
// sweep the sequences round by round (round r = the r-th stage of every walk), so by the time a sweep comes back to a
// sequence its next stage has long been published.  Rows after the first rejection are never read.
//
// Inside a CTA: a producer warp walks the rounds, reads the stage words 32 sequences at a time and starts the bulk
// copies of each item's two row slices into a shared-memory ring; sixteen compute warps each take every sixteenth ring
// slot, reduce it on their own (no CTA-wide barrier anywhere) and deliver; the merger warp serves the owned sequences.
// Every wait (ring barriers, stage words, arrival counters) is a bounded poll that records a timeout and unwinds.
// Stage words carry the launch's epoch (a counter in the workspace that the last CTA to leave advances), so nothing
// has to be cleared between launches; arrival counters are reset by the merger that consumed them.
#include "sampler_common.cuh"

namespace gm {
namespace {

constexpr int SF_CWARPS = 16;                         // compute warps
constexpr int SF_PRODUCER = SF_CWARPS;                // warp index of the producer
constexpr int SF_MERGER = SF_CWARPS + 1;              // warp index of the merger
constexpr int SF_THREADS = (SF_CWARPS + 2) * 32;
constexpr int SF_EPL = 5;                             // deliveries of a stage a merger lane holds: up to 160 slices
constexpr int SF_UMAX = 8;                            // vectors (8 logits) per lane and row: slices of up to 256 vectors
constexpr int SF_RING_BYTES = 216 * 1024;
constexpr int SF_MAX_R = 64;                          // ring slots at most
constexpr int SF_MAX_OWN = 8;                         // sequences a CTA may own: batch <= 8 * grid
constexpr uint32_t SF_SPIN_LIMIT = 1u << 22;
enum { SF_NONE = 0, SF_STAT = 1, SF_RES = 2, SF_SEARCH = 3, SF_ARGMAX = 4, SF_QUIT = 7 };
enum { SF_EPOCH = 0, SF_EXIT = 32, SF_CTRL_WORDS = 64 };       // control words, 128 bytes apart

struct SFSeq {                                        // per-sequence walk state, written by the owner before it publishes a stage
  float c_p, iz_p, c_q, iz_q;                         // (c, 1 / Z) of the two rows of the resampled position
  unsigned long long t_local;                         // quantile inside the chosen slice
  unsigned int pad[2];
};
static_assert(sizeof(SFSeq) == 32, "SFSeq layout");

struct SFWs {
  uint32_t *ctrl;                                     // epoch, exit counter
  SFSeq *seq;                                         // [B]
  unsigned long long *stage;                          // [B][rounds]: epoch << 32 | owner_slice << 8 | k << 4 | type
  uint32_t *cnt;                                      // [B][rounds] arrivals
  unsigned long long *ent;                            // [B][4][NA] deliveries: tag << 32 | 32 payload bits (p max, p sum, q max, q sum;
                                                      // or the low and high half of a slice's residual weight)
  int G, vps, tail, NA, rounds, R, nmain, wide;                    // CTAs, vectors per slice, vectors after the last slice, deliveries per stage
};

__device__ __forceinline__ unsigned long long sf_word(uint32_t epoch, int type, int k, int slice) {
  return (static_cast<unsigned long long>(epoch) << 32) | (static_cast<unsigned long long>(slice) << 8) |
         (static_cast<unsigned long long>(k) << 4) | static_cast<unsigned long long>(type);
}
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long *p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_u64(unsigned long long *p, unsigned long long v) {
  asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
// Arrival hint: the counter only tells the owner when to look; what it then reads is validated word by word (every
// delivered 64-bit word carries the tag of its launch and round), so no fence has to order the stores before it.
__device__ __forceinline__ void red_relaxed_inc(uint32_t *p) {
  asm volatile("red.relaxed.gpu.global.add.u32 [%0], 1;" ::"l"(p) : "memory");
}
__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long *p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long *p, unsigned long long v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ uint32_t sf_tag(uint32_t epoch, int r) { return ((epoch << 4) | static_cast<uint32_t>(r)) + 1u; }
__device__ __forceinline__ uint4 ldg_nc(const uint4 *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ const uint4 *sf_row(const SamplerArgs &A, int b, int r) {      // r <= K: target row r; else draft row r-K-1
  const __nv_bfloat16 *p = r <= A.K ? A.target_logits + static_cast<size_t>(b) * A.tgt_bstride + static_cast<size_t>(r) * A.V
                                    : A.draft_logits + static_cast<size_t>(b) * A.drf_bstride + static_cast<size_t>(r - A.K - 1) * A.V;
  return reinterpret_cast<const uint4 *>(p);
}

// One reduction for every level (lanes of a warp, slices of a row): the maximum first, every partial sum rescaled to
// it once, then a butterfly of plain additions - symmetric, so every lane ends with the same bits, and the
// probability dump below reproduces the walk's statistics exactly.
__device__ __forceinline__ MZ sf_reduce(MZ st, float s) {
  const float wm = warp_max(st.m);
  float z = (wm == -INFINITY || st.m == -INFINITY) ? 0.f : __fmul_rn(st.z, ex2(__fmul_rn(__fsub_rn(st.m, wm), s)));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) z = __fadd_rn(z, __shfl_xor_sync(0xffffffffu, z, o));
  return MZ{wm, z};
}
__device__ __forceinline__ MZ sf_merge2(MZ a, MZ b, float s) {
  const float m = fmaxf(a.m, b.m);
  if (m == -INFINITY) return MZ{m, 0.f};
  const float za = a.m == -INFINITY ? 0.f : __fmul_rn(a.z, ex2(__fmul_rn(__fsub_rn(a.m, m), s)));
  const float zb = b.m == -INFINITY ? 0.f : __fmul_rn(b.z, ex2(__fmul_rn(__fsub_rn(b.m, m), s)));
  return MZ{m, __fadd_rn(za, zb)};
}
// a warp's statistics of n vectors at src (shared or global memory).  Per block of 128 vectors lane l holds vectors
// l, l + 32, l + 64, l + 96: packed maximum over all of them first, then one exponential per logit against that maximum.
constexpr int SF_UBLK = 4;
template <bool GLOBAL>
__device__ __forceinline__ void sf_load_block(const uint4 *src, int base, int n, int lane, uint4 (&v)[SF_UBLK], uint32_t fill) {
#pragma unroll
  for (int t = 0; t < SF_UBLK; ++t) {
    const int i = base + lane + t * 32;
    v[t] = i < n ? (GLOBAL ? ldg_nc(src + i) : src[i]) : make_uint4(fill, fill, fill, fill);
  }
}
__device__ __forceinline__ MZ sf_block_stats(const uint4 (&v)[SF_UBLK], float s) {
  uint32_t m2 = 0xff80ff80u;
#pragma unroll
  for (int t = 0; t < SF_UBLK; ++t) m2 = bmax2(bmax2(m2, bmax2(v[t].x, v[t].y)), bmax2(v[t].z, v[t].w));
  const float mx = fmaxf(bf16_lo(m2), bf16_hi(m2));
  MZ blk{mx, 0.f};
  if (mx != -INFINITY) {
    const float c = -mx * s;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int t = 0; t < SF_UBLK; ++t) {
      float x[8];
      unpack8(v[t], x);
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[j & 3] = __fadd_rn(acc[j & 3], ex2(fmaf(x[j], s, c)));
    }
    blk.z = __fadd_rn(__fadd_rn(acc[0], acc[1]), __fadd_rn(acc[2], acc[3]));
  }
  return blk;
}
template <bool GLOBAL>
__device__ __forceinline__ MZ sf_slice_stats(const uint4 *src, int n, int lane, float s) {
  MZ st{-INFINITY, 0.f};
  for (int base = 0; base < n; base += 32 * SF_UBLK) {
    uint4 v[SF_UBLK];
    sf_load_block<GLOBAL>(src, base, n, lane, v, 0xff80ff80u);
    const MZ blk = sf_block_stats(v, s);
    st = base == 0 ? blk : sf_merge2(st, blk, s);
  }
  return sf_reduce(st, s);
}
// NA slice partials of one row -> the row's (c, 1 / Z): lane l merges partials l, l + 32, ... in order, then the butterfly
template <typename F>
__device__ __forceinline__ MZ sf_merge_slices(F ld, int NA, int lane, float s) {
  MZ st{-INFINITY, 0.f};
  for (int i = lane; i < NA; i += 32) st = sf_merge2(st, ld(i), s);
  st = sf_reduce(st, s);
  return MZ{-st.m * s, __frcp_rn(st.z)};
}

constexpr int SF_MAX_B = 2048;
constexpr int SF_ROUNDS = GM_MAX_K_ + 4;              // stride of the per-sequence stage arrays (STAT x (K+1), RES, RES again, SEARCH)

struct SFShared {
  uint64_t full[SF_MAX_R], empty[SF_MAX_R];
  uint32_t desc[SF_MAX_R];                            // type | use_q << 3 | k << 4 | tail << 8 | round << 9 | b << 16
  volatile uint32_t use[SF_MAX_R];                    // 1 + the use count a slot is armed for (0: never)
  uint32_t done_mask[SF_MAX_B / 32];                  // producer: sequences whose walk has ended
  volatile int dead;
};

__device__ __forceinline__ uint32_t sf_desc(int type, int use_q, int k, int tail, int r, int b) {
  return static_cast<uint32_t>(type) | (static_cast<uint32_t>(use_q) << 3) | (static_cast<uint32_t>(k) << 4) |
         (static_cast<uint32_t>(tail) << 8) | (static_cast<uint32_t>(r) << 9) | (static_cast<uint32_t>(b) << 16);
}

// 64-bit integer weights of one vector of the resampled position
__device__ __forceinline__ unsigned long long sf_vec_weight(const uint4 &vp, const uint4 &vq, bool use_q, float s, const SFSeq &q,
                                                            unsigned long long (&w)[8]) {
  float xp[8], xq[8];
  unpack8(vp, xp);
  if (use_q) unpack8(vq, xq);
  unsigned long long sum = 0;
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    w[e] = weight_of(prob_of(xp[e], s, q.c_p, q.iz_p), use_q ? prob_of(xq[e], s, q.c_q, q.iz_q) : 0.f, use_q);
    sum += w[e];
  }
  return sum;
}
__device__ __forceinline__ SFSeq sf_load_seq(const SFSeq *p) {
  SFSeq q;
  q.c_p = __ldcg(&p->c_p); q.iz_p = __ldcg(&p->iz_p); q.c_q = __ldcg(&p->c_q); q.iz_q = __ldcg(&p->iz_q);
  q.t_local = __ldcg(&p->t_local);
  return q;
}

// outputs and state commit of sequence b by one warp
__device__ __forceinline__ void sf_finish(const SamplerArgs &A, int b, int a, int tok, int lane) {
  const int K = A.K;
  if (lane == 0) {
    A.next_token[static_cast<size_t>(b) * A.tok_out_stride] = tok;
    if (A.accept_len) A.accept_len[b] = a;
  }
  if (A.commit) {
    const int kp1 = A.max_k + 1;
    if (lane == 0) {
      A.kv_len[b] += a + 1;
      A.pending_n[b] = a + 1;
    }
    if (lane <= a)
      A.pending_tok[static_cast<size_t>(b) * kp1 + lane] =
          lane < a ? A.draft_tok[static_cast<size_t>(b) * A.tok_in_stride + lane] : tok;
    const int vec_per_row = A.d_model >> 3;
    const uint4 *src = reinterpret_cast<const uint4 *>(A.target_hidden + static_cast<size_t>(b) * (K + 1) * A.d_model);
    uint4 *dst = reinterpret_cast<uint4 *>(A.pending_hidden + static_cast<size_t>(b) * kp1 * A.d_model);
    for (int i = lane; i < (a + 1) * vec_per_row; i += 32) dst[i] = src[i];
  }
}

__global__ void __launch_bounds__(SF_THREADS, 1) sampler_flow_kernel(const SamplerArgs A, const SFWs W, const int B) {
  __shared__ SFShared sh;
  extern __shared__ __align__(128) unsigned char sf_smem[];
  uint4 *ring = reinterpret_cast<uint4 *>(sf_smem);   // [R][2][vps]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int c = blockIdx.x, G = W.G, vps = W.vps, NA = W.NA, R = W.R, rounds = W.rounds;
  const int K = A.K, V = A.V;
  const float s = A.inv_temp * 1.4426950408889634f;
  // `wide` neighbouring CTAs share a slice index and split the sequences among them (b mod wide): wider slices, fewer items
  const int wide = W.wide, Gs = G / wide, grp = c % wide, sidx = c / wide;
  const int nseq = B > grp ? (B - grp + wide - 1) / wide : 0;
  const int nblk = (nseq + 31) / 32;
  auto owner_of = [=](int b) { return wide == 1 ? b % G : ((b / wide) % Gs) * wide + (b % wide); };

  if (tid == 0) {
    for (int i = 0; i < R; ++i) { mbar_init(&sh.full[i], 1); mbar_init(&sh.empty[i], 1); }
    mbar_fence_init();
    sh.dead = 0;
  }
  for (int i = tid; i < SF_MAX_B / 32; i += SF_THREADS) sh.done_mask[i] = 0u;
  for (int i = tid; i < SF_MAX_R; i += SF_THREADS) sh.use[i] = 0u;
  __syncthreads();
  pdl_prologue();
  const uint32_t epoch = ld_acquire_u32(&W.ctrl[SF_EPOCH]);

  // bounded wait on a ring barrier; gives up at once when another warp has already recorded a timeout
  auto wait_bar = [&](uint64_t *bar, uint32_t parity) -> bool {
    for (uint32_t i = 0; i < SF_SPIN_LIMIT; ++i) {
      if (mbar_try_wait(bar, parity)) return true;
      if ((i & 63u) == 63u && sh.dead) return false;
    }
    if (!sh.dead) { sh.dead = 1; set_status(A.status, ST_TIMEOUT); }
    return false;
  };

  // ======================================================= producer =======================================================
  if (warp == SF_PRODUCER) {
    uint32_t n = 0;                                   // ring items posted so far (same value in every lane)
    bool alive = true;
    // every lane that holds an item takes the next free ring slots in lane order and starts its own copies
    auto post = [&](bool has_all, uint32_t desc, const uint4 *prow, const uint4 *qrow) {
      const int npass = R >= 32 ? 1 : 2;              // a small ring takes sixteen lanes at a time: never more items than slots
      for (int pass = 0; pass < npass; ++pass) {
        const bool has = has_all && (npass == 1 || (lane >> 4) == pass);
        const uint32_t m = __ballot_sync(0xffffffffu, has);
        if (has) {
          const uint32_t mine = n + __popc(m & ((1u << lane) - 1u));
          const int slot = mine % R;
          if (wait_bar(&sh.empty[slot], ((mine / R) & 1u) ^ 1u)) {
            sh.desc[slot] = desc;
            if (R < 2 * SF_CWARPS + 2) sh.use[slot] = mine / R + 1u;   // armed for this use (before the barrier operations below)
            if (prow != nullptr) {
              const uint32_t bytes = static_cast<uint32_t>(vps) * 16u;
              mbar_expect_tx(&sh.full[slot], qrow ? 2u * bytes : bytes);
              fence_proxy_async();
              bulk_load(ring + static_cast<size_t>(slot) * 2 * vps, prow + static_cast<size_t>(sidx) * vps, bytes, &sh.full[slot]);
              if (qrow) bulk_load(ring + (static_cast<size_t>(slot) * 2 + 1) * vps, qrow + static_cast<size_t>(sidx) * vps, bytes, &sh.full[slot]);
            } else {
              mbar_arrive(&sh.full[slot]);
            }
          }
        }
        n += __popc(m);
        __syncwarp();
      }
    };
    for (int r = 0; r < rounds && alive; ++r) {
      bool any = false;
      for (int blk = 0; blk < nblk && alive; ++blk) {
        const int b = grp + wide * (blk * 32 + lane);
        bool act = b < B && !((sh.done_mask[blk] >> lane) & 1u);
        int type = SF_NONE, k = 0, use_q = 0, slice = 0;
        if (r == 0) {
          if (act && A.finished && A.finished[b]) {   // the row sits out: its owner writes the outputs
            if (owner_of(b) == c) {
              if (A.accept_len) A.accept_len[b] = 0;
              A.next_token[static_cast<size_t>(b) * A.tok_out_stride] = A.accept_len ? -1 : 0;
            }
            act = false;
            atomicOr(&sh.done_mask[blk], 1u << lane);
          }
          type = SF_STAT;
        } else {
          const unsigned long long *wp = W.stage + static_cast<size_t>(b < B ? b : 0) * SF_ROUNDS + r;
          unsigned long long w = 0;
          bool ready = !act;
          for (uint32_t i = 0; i < SF_SPIN_LIMIT; ++i) {
            if (!ready) {
              w = ld_acquire_u64(wp);
              ready = static_cast<uint32_t>(w >> 32) == epoch && (w & 7u) != 0u;
            }
            if (__all_sync(0xffffffffu, ready)) break;
            if (sh.dead) break;
            __nanosleep(64);
          }
          if (!__all_sync(0xffffffffu, ready)) {
            if (lane == 0 && !sh.dead) { sh.dead = 1; set_status(A.status, ST_TIMEOUT); }
            alive = false;
            break;
          }
          type = static_cast<int>(w & 7u); use_q = static_cast<int>((w >> 3) & 1u); k = static_cast<int>((w >> 4) & 15u);
          slice = static_cast<int>((w >> 8) & 0xffffu);
        }
        any = any || __any_sync(0xffffffffu, act);
        const bool bulk = act && (type == SF_STAT || type == SF_RES);
        const int prow_r = k, qrow_r = K + 1 + k;     // STAT k and RES at position a = k read the rows (p_k, q_k)
        const bool has_q = type == SF_STAT ? k < K : use_q != 0;
        // the slice every CTA holds
        post(bulk && vps > 0, sf_desc(type, use_q, k, 0, r, b), bulk ? sf_row(A, b, prow_r) : nullptr,
             bulk && has_q ? sf_row(A, b, qrow_r) : nullptr);
        // what only one CTA does: the vectors after the last slice, the token search, the fallback
        const bool own = act && owner_of(b) == c;
        post(bulk && own && W.tail > 0, sf_desc(type, use_q, k, 1, r, b), nullptr, nullptr);
        const bool fin = act && (type == SF_SEARCH || type == SF_ARGMAX);
        post(fin && (type == SF_ARGMAX ? own : (slice == W.nmain ? own : slice == sidx)), sf_desc(type, use_q, k, slice == W.nmain ? 1 : 0, r, b),
             nullptr, nullptr);
        if (fin) atomicOr(&sh.done_mask[blk], 1u << lane);
        __syncwarp();
      }
      if (!any) break;                                // every walk has ended
    }
    // one quit marker per compute warp
    post(lane < SF_CWARPS && !sh.dead, static_cast<uint32_t>(SF_QUIT), nullptr, nullptr);
    if (lane == 0) {                                  // the last CTA to leave opens the next epoch
      const uint32_t old = atomicAdd(&W.ctrl[SF_EXIT], 1u);
      if (old == gridDim.x - 1) {
        W.ctrl[SF_EXIT] = 0u;
        __threadfence();
        atomicAdd(&W.ctrl[SF_EPOCH], 1u);
      }
    }
    return;
  }

  // ======================================================== merger ========================================================
  // Lane i watches the arrival counter of the i-th sequence this CTA owns; a completed stage is merged by the whole warp.
  if (warp == SF_MERGER) {
    const int my_b = grp + wide * (sidx + Gs * lane);         // the sequences with owner_of(b) == c
    bool active = lane < SF_MAX_OWN && my_b < B && !(A.finished && A.finished[my_b]);
    int r = 0, type = SF_STAT, k = 0, use_q = 0;      // the stage in flight of lane i's sequence
    // what the accept decision of that stage will need, requested when the stage starts
    float pd_xp = 0.f, pd_xq = 0.f;
    uint32_t pd_u24 = 0;
    int pd_ok = 0;
    auto prefetch_decision = [&]() {
      pd_ok = 0;
      if (active && type == SF_STAT && k < K) {
        const int d = A.draft_tok[static_cast<size_t>(my_b) * A.tok_in_stride + k];
        if (d >= 0 && d < V) {
          pd_ok = 1;
          pd_xp = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(sf_row(A, my_b, k))[d]);
          pd_xq = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(sf_row(A, my_b, K + 1 + k))[d]);
        }
        pd_u24 = A.u24 ? A.u24[static_cast<size_t>(my_b) * A.u_stride + k] : philox_u24(A.seed, step_of(A), my_b, A.slot_accept + k);
      }
    };
    prefetch_decision();
    uint32_t spins = 0;
    while (__any_sync(0xffffffffu, active)) {
      bool ready = false;
      if (active) ready = ld_acquire_u32(&W.cnt[static_cast<size_t>(my_b) * SF_ROUNDS + r]) == static_cast<uint32_t>(NA);
      uint32_t m = __ballot_sync(0xffffffffu, ready);
      if (m == 0u) {
        __nanosleep(100);
        if (++spins >= SF_SPIN_LIMIT || sh.dead) {
          if (lane == 0 && !sh.dead) { sh.dead = 1; set_status(A.status, ST_TIMEOUT); }
          break;
        }
        continue;
      }
      spins = 0;
      while (m != 0u) {
        const int src = __ffs(m) - 1;
        m &= m - 1u;
        const int b = __shfl_sync(0xffffffffu, my_b, src), rr = __shfl_sync(0xffffffffu, r, src);
        const int ty = __shfl_sync(0xffffffffu, type, src), kk = __shfl_sync(0xffffffffu, k, src);
        const int uq = __shfl_sync(0xffffffffu, use_q, src);
        int n_type = SF_NONE, n_k = kk, n_uq = 0, n_slice = 0;
        SFSeq *sq = &W.seq[b];
        // the delivered words: validated by their tag (the counter was only the hint to look)
        const unsigned long long *ent = W.ent + static_cast<size_t>(b) * 4 * NA;
        const uint32_t tag = sf_tag(epoch, rr);
        const bool bonus = ty == SF_STAT && kk == K;
        const int per = (NA + 31) / 32;               // RES: lane l holds slices l*per .. l*per + per - 1; STAT: l, l + 32, ...
        uint32_t val[2][SF_EPL];                     // two word kinds at a time: (max, sum) of a row, or (low, high) of a weight
        // all words of kinds k0, k0 + 1 into val; false if one of them never shows this stage's tag
        auto load2 = [&](int k0) -> bool {
          bool good = false;
          for (uint32_t tries = 0; tries < (1u << 16) && !good; ++tries) {
            unsigned long long w[2][SF_EPL];
#pragma unroll
            for (int kind = 0; kind < 2; ++kind) {    // all loads first ...
#pragma unroll
              for (int t = 0; t < SF_EPL; ++t) {
                const int i = ty == SF_STAT ? lane + 32 * t : lane * per + t;
                w[kind][t] = (i < NA && (ty == SF_STAT || t < per)) ? ld_relaxed_u64(&ent[static_cast<size_t>(k0 + kind) * NA + i])
                                                                     : (static_cast<unsigned long long>(tag) << 32);
              }
            }
            good = true;
#pragma unroll
            for (int kind = 0; kind < 2; ++kind) {    // ... then the checks
#pragma unroll
              for (int t = 0; t < SF_EPL; ++t) {
                good = good && static_cast<uint32_t>(w[kind][t] >> 32) == tag;
                val[kind][t] = static_cast<uint32_t>(w[kind][t]);
              }
            }
            good = __all_sync(0xffffffffu, good);
            if (!good) __nanosleep(200);
          }
          return good;
        };
        auto merged = [&]() -> MZ {
          MZ st{-INFINITY, 0.f};
#pragma unroll
          for (int t = 0; t < SF_EPL; ++t)
            if (lane + 32 * t < NA) st = sf_merge2(st, MZ{__uint_as_float(val[0][t]), __uint_as_float(val[1][t])}, s);
          st = sf_reduce(st, s);
          return MZ{-st.m * s, __frcp_rn(st.z)};
        };
        bool good = load2(0);
        MZ ps{0.f, 1.f}, qs{0.f, 1.f};
        if (good && ty == SF_STAT) {
          ps = merged();
          if (!bonus) {
            good = load2(2);
            if (good) qs = merged();
          }
        }
        if (!good) {                                  // a word never arrived: give up, the host reports the timeout
          if (lane == 0 && !sh.dead) { sh.dead = 1; set_status(A.status, ST_TIMEOUT); }
          active = false;
          break;
        }
        if (ty == SF_STAT) {
          int ok = 0;
          if (lane == src && !bonus) {
            if (!pd_ok) {
              set_status(A.status, ST_BAD_TOKEN);
            } else {
              const float p = prob_of(pd_xp, s, ps.m, ps.z);
              const float q = prob_of(pd_xq, s, qs.m, qs.z);
              const float uq24 = __fmul_rn(__fmul_rn(static_cast<float>(pd_u24), 5.9604644775390625e-8f /* 2^-24 */), q);
              ok = (p >= q || uq24 < p) ? 1 : 0;
            }
          }
          ok = __shfl_sync(0xffffffffu, ok, src);
          if (ok) {
            n_type = SF_STAT; n_k = kk + 1;
          } else {
            if (lane == 0) { sq->c_p = ps.m; sq->iz_p = ps.z; sq->c_q = qs.m; sq->iz_q = qs.z; }
            n_type = SF_RES; n_k = kk; n_uq = bonus ? 0 : 1;
          }
        } else {                                      // SF_RES: total weight, quantile, the slice that holds it
          unsigned long long mine = 0;
#pragma unroll
          for (int t = 0; t < SF_EPL; ++t) mine += (static_cast<unsigned long long>(val[1][t]) << 32) | val[0][t];
          unsigned long long incl = mine;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
          }
          const unsigned long long Wt = __shfl_sync(0xffffffffu, incl, 31);
          if (Wt == 0ull && uq) {                     // residual mass underflowed: draw from p instead
            if (lane == 0) set_status(A.status, ST_ZERO_RESID);
            n_type = SF_RES; n_uq = 0;
          } else if (Wt == 0ull) {                    // no mass at all (cannot happen for a softmax of finite logits)
            n_type = SF_ARGMAX;
          } else {
            const uint32_t u_final = A.u24 ? A.u24[static_cast<size_t>(b) * A.u_stride + K]
                                           : philox_u24(A.seed, step_of(A), b, A.slot_final);
            const unsigned long long t = static_cast<unsigned long long>(u_final) * (Wt >> 24) +
                                         ((static_cast<unsigned long long>(u_final) * (Wt & 0xFFFFFFull)) >> 24);
            const unsigned long long excl = incl - mine;
            int js = -1;
            unsigned long long t_rem = 0;
            if (mine != 0ull && t >= excl && t < excl + mine) {
              unsigned long long rem = t - excl;
              bool found = false;
#pragma unroll
              for (int t2 = 0; t2 < SF_EPL; ++t2) {
                const unsigned long long wl = (static_cast<unsigned long long>(val[1][t2]) << 32) | val[0][t2];
                if (!found && lane * per + t2 < NA && t2 < per) {
                  if (rem < wl) { found = true; js = lane * per + t2; }
                  else rem -= wl;
                }
              }
              if (!found) { js = min(NA, lane * per + per) - 1; }
              t_rem = rem;
            }
            const uint32_t who = __ballot_sync(0xffffffffu, js >= 0);
            n_slice = who ? __shfl_sync(0xffffffffu, js, __ffs(who) - 1) : 0;
            t_rem = who ? __shfl_sync(0xffffffffu, t_rem, __ffs(who) - 1) : 0ull;
            if (lane == 0) sq->t_local = t_rem;
            n_type = SF_SEARCH; n_uq = uq;
          }
        }
        __syncwarp();
        if (lane == 0) {
          W.cnt[static_cast<size_t>(b) * SF_ROUNDS + rr] = 0u;                   // clean for the next launch
          const unsigned long long word = sf_word(epoch, n_type, n_k, n_slice) | (static_cast<unsigned long long>(n_uq) << 3);
          unsigned long long *dst = &W.stage[static_cast<size_t>(b) * SF_ROUNDS + rr + 1];
          if (n_type == SF_STAT) st_relaxed_u64(dst, word);                      // nothing but the word itself to see
          else st_release_u64(dst, word);                                        // after the state this lane wrote above
        }
        if (lane == src) {
          r = rr + 1; type = n_type; k = n_k; use_q = n_uq;
          if (n_type == SF_SEARCH || n_type == SF_ARGMAX || r >= rounds) active = false;
          prefetch_decision();
        }
      }
    }
    return;
  }

  // ==================================================== compute warps ====================================================
  for (uint32_t n = warp;; n += SF_CWARPS) {
    const int slot = n % R;
    // A ring shorter than two rounds of warps lets a warp get here before the slot's PREVIOUS use has even landed, and a
    // parity wait cannot tell "not yet" from "already": wait until the producer has armed the slot for THIS use first.
    if (R < 2 * SF_CWARPS + 2) {
      const uint32_t want_use = n / R + 1u;
      bool ok = false;
      for (uint32_t i = 0; i < SF_SPIN_LIMIT; ++i) {
        if (sh.use[slot] == want_use) { ok = true; break; }
        if ((i & 63u) == 63u && sh.dead) break;
      }
      if (!ok) {
        if (!sh.dead) { sh.dead = 1; set_status(A.status, ST_TIMEOUT); }
        return;
      }
    }
    if (!wait_bar(&sh.full[slot], (n / R) & 1u)) return;
    const uint32_t desc = sh.desc[slot];
    const int type = desc & 7u, use_q = (desc >> 3) & 1u, k = (desc >> 4) & 15u, is_tail = (desc >> 8) & 1u, r = (desc >> 9) & 15u;
    const int b = desc >> 16;
    if (type == SF_QUIT) return;
    const int idx = is_tail ? W.nmain : sidx;                  // which delivery of the stage this is
    const int v_lo = is_tail ? W.nmain * vps : sidx * vps, nv = is_tail ? W.tail : vps;
    const uint4 *sp = ring + static_cast<size_t>(slot) * 2 * vps, *sq_ = sp + vps;
    bool released = false;                            // the ring slot has already been given back
    if (type == SF_STAT) {
      const bool bonus = k == K;
      MZ mp, mq{-INFINITY, 0.f};
      if (is_tail) {
        mp = sf_slice_stats<true>(sf_row(A, b, k) + v_lo, nv, lane, s);
        if (!bonus) mq = sf_slice_stats<true>(sf_row(A, b, K + 1 + k) + v_lo, nv, lane, s);
      } else if (nv <= 32 * SF_UBLK) {                // the usual case: take the slice into registers, give the slot back, then reduce
        uint4 vp[SF_UBLK], vq[SF_UBLK];
        sf_load_block<false>(sp, 0, nv, lane, vp, 0xff80ff80u);
        if (!bonus) sf_load_block<false>(sq_, 0, nv, lane, vq, 0xff80ff80u);
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.empty[slot]);
        released = true;
        mp = sf_reduce(sf_block_stats(vp, s), s);
        if (!bonus) mq = sf_reduce(sf_block_stats(vq, s), s);
      } else {
        mp = sf_slice_stats<false>(sp, nv, lane, s);
        if (!bonus) mq = sf_slice_stats<false>(sq_, nv, lane, s);
      }
      // every lane holds the same (mp, mq): lanes 0..3 store one tagged word each
      if (lane < (bonus ? 2 : 4)) {
        const float f = lane == 0 ? mp.m : lane == 1 ? mp.z : lane == 2 ? mq.m : mq.z;
        st_relaxed_u64(&W.ent[(static_cast<size_t>(b) * 4 + lane) * NA + idx],
                       (static_cast<unsigned long long>(sf_tag(epoch, r)) << 32) | __float_as_uint(f));
      }
      __syncwarp();
      if (lane == 0) red_relaxed_inc(&W.cnt[static_cast<size_t>(b) * SF_ROUNDS + r]);
    } else if (type == SF_RES) {
      const SFSeq q = sf_load_seq(&W.seq[b]);
      const uint4 *gp = sf_row(A, b, k) + v_lo, *gq = use_q ? sf_row(A, b, K + 1 + k) + v_lo : nullptr;
      unsigned long long tsum = 0;
      if (!is_tail && nv <= 32 * SF_UBLK) {
        uint4 vp[SF_UBLK], vq[SF_UBLK];
        sf_load_block<false>(sp, 0, nv, lane, vp, 0u);
        if (use_q) sf_load_block<false>(sq_, 0, nv, lane, vq, 0u);
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.empty[slot]);
        released = true;
#pragma unroll
        for (int t = 0; t < SF_UBLK; ++t) {
          if (lane + 32 * t < nv) {
            unsigned long long w[8];
            tsum += sf_vec_weight(vp[t], use_q ? vq[t] : make_uint4(0u, 0u, 0u, 0u), use_q != 0, s, q, w);
          }
        }
      } else {
        for (int i = lane; i < nv; i += 32) {
          unsigned long long w[8];
          const uint4 vp = is_tail ? ldg_nc(gp + i) : sp[i];
          const uint4 vq = use_q ? (is_tail ? ldg_nc(gq + i) : sq_[i]) : make_uint4(0u, 0u, 0u, 0u);
          tsum += sf_vec_weight(vp, vq, use_q != 0, s, q, w);
        }
      }
      tsum = warp_sum_u64(tsum);
      if (lane < 2)
        st_relaxed_u64(&W.ent[(static_cast<size_t>(b) * 4 + lane) * NA + idx],
                       (static_cast<unsigned long long>(sf_tag(epoch, r)) << 32) | static_cast<uint32_t>(lane == 0 ? tsum : tsum >> 32));
      __syncwarp();
      if (lane == 0) red_relaxed_inc(&W.cnt[static_cast<size_t>(b) * SF_ROUNDS + r]);
    } else if (type == SF_SEARCH) {
      // token search in this CTA's slice (or the tail): lane l owns `per` consecutive vectors
      const SFSeq q = sf_load_seq(&W.seq[b]);
      const uint4 *gp = sf_row(A, b, k) + v_lo, *gq = use_q ? sf_row(A, b, K + 1 + k) + v_lo : nullptr;
      const int per = (nv + 31) / 32, lo = min(nv, lane * per), hi = min(nv, lo + per);
      unsigned long long mine = 0;
      for (int i = lo; i < hi; ++i) {
        unsigned long long w[8];
        mine += sf_vec_weight(ldg_nc(gp + i), use_q ? ldg_nc(gq + i) : make_uint4(0u, 0u, 0u, 0u), use_q != 0, s, q, w);
      }
      unsigned long long incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
      }
      const unsigned long long excl = incl - mine;
      int tok = -1;
      if (mine != 0ull && q.t_local >= excl && q.t_local < excl + mine) {
        unsigned long long rem = q.t_local - excl;
        for (int i = lo; i < hi && tok < 0; ++i) {
          unsigned long long w[8];
          const unsigned long long vs = sf_vec_weight(ldg_nc(gp + i), use_q ? ldg_nc(gq + i) : make_uint4(0u, 0u, 0u, 0u), use_q != 0, s, q, w);
          if (rem >= vs && i < hi - 1) { rem -= vs; continue; }
          tok = (v_lo + i) * 8 + 7;
          bool found = false;
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            if (!found && rem < w[e]) { tok = (v_lo + i) * 8 + e; found = true; }
            if (!found) rem -= w[e];
          }
        }
      }
      const uint32_t who = __ballot_sync(0xffffffffu, tok >= 0);
      tok = who ? __shfl_sync(0xffffffffu, tok, __ffs(who) - 1) : 0;
      sf_finish(A, b, k, tok, lane);
    } else if (type == SF_ARGMAX) {                   // lowest index of the row maximum
      const float c_p = __ldcg(&W.seq[b].c_p);
      const uint4 *gp = sf_row(A, b, k);
      int best = 0x7fffffff;
      for (int i = lane; i < (V >> 3); i += 32) {
        float x[8];
        unpack8(ldg_nc(gp + i), x);
#pragma unroll
        for (int e = 7; e >= 0; --e)
          if (-x[e] * s == c_p) best = min(best, i * 8 + e);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) best = min(best, __shfl_xor_sync(0xffffffffu, best, o));
      if (best == 0x7fffffff) best = 0;
      if (lane == 0) set_status(A.status, ST_ZERO_MASS);
      sf_finish(A, b, k, best, lane);
    }
    __syncwarp();
    if (lane == 0 && !released) mbar_arrive(&sh.empty[slot]);
  }
}

// Probabilities of every row with exactly the statistics the walk computes (same slices, same merges): debug dump.
constexpr int SF_DUMP_THREADS = 256;
__global__ void __launch_bounds__(SF_DUMP_THREADS) sampler_flow_dump_kernel(const SamplerArgs A, const int G, const int vps,
                                                                            const int tail, MZ *scratch) {
  __shared__ MZ row_mz;
  const int K = A.K, V = A.V, R = 2 * K + 1, nmain = vps > 0 ? G : 0, NA = nmain + (tail > 0 ? 1 : 0);
  const int b = blockIdx.x / R, r = blockIdx.x % R;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float s = A.inv_temp * 1.4426950408889634f;
  const int nvec = V >> 3;
  float *dst = r <= K ? (A.dbg_p ? A.dbg_p + static_cast<size_t>(b) * A.tgt_bstride + static_cast<size_t>(r) * V : nullptr)
                      : (A.dbg_q ? A.dbg_q + static_cast<size_t>(b) * A.drf_bstride + static_cast<size_t>(r - K - 1) * V : nullptr);
  if (dst == nullptr || (A.finished && A.finished[b])) return;
  const uint4 *row = sf_row(A, b, r);
  MZ *part = scratch + static_cast<size_t>(blockIdx.x) * NA;
  for (int j = warp; j < NA; j += SF_DUMP_THREADS / 32) {
    const MZ st = j < nmain ? sf_slice_stats<true>(row + static_cast<size_t>(j) * vps, vps, lane, s)
                            : sf_slice_stats<true>(row + static_cast<size_t>(nmain) * vps, tail, lane, s);
    if (lane == 0) part[j] = st;
  }
  __threadfence_block();
  __syncthreads();
  if (warp == 0) {
    const MZ st = sf_merge_slices([&](int l) { return part[l]; }, NA, lane, s);
    if (lane == 0) row_mz = st;
  }
  __syncthreads();
  const MZ st = row_mz;
  for (int i = tid; i < nvec; i += SF_DUMP_THREADS) {
    float x[8];
    unpack8(ldg_nc(row + i), x);
#pragma unroll
    for (int e = 0; e < 8; ++e) dst[static_cast<size_t>(i) * 8 + e] = prob_of(x[e], s, st.m, st.z);
  }
}

struct SFGeom { int G, vps, tail, NA, R, nmain, wide; };
// batch = 0: the widest geometry (one slice per CTA), which sizes the workspace
SFGeom sf_geometry(int V, int sm_count, int batch) {
  SFGeom g;
  const int nvec = V >> 3;
  g.G = std::max(1, std::min(sm_count, nvec / 32));
  // Large batches: pairs of CTAs share a slice index and take every other sequence each - slices twice as wide, half the
  // items, copies and deliveries per stage (the per-item costs of the producer and of the compute warps are what binds).
  g.wide = (batch >= 160 && g.G % 2 == 0 && nvec / (32 * (g.G / 2)) <= SF_UMAX) ? 2 : 1;
  if (const char *ov = std::getenv("GM_SF_WIDE")) { const int v = std::atoi(ov); if ((v == 1 || v == 2 || v == 4) && g.G % v == 0) g.wide = v; }
  const int gs = g.G / g.wide;
  g.vps = 32 * (nvec / (32 * gs));
  g.tail = nvec - gs * g.vps;
  g.nmain = g.vps > 0 ? gs : 0;                       // slices that a CTA holds one of
  g.NA = g.nmain + (g.tail > 0 ? 1 : 0);
  g.R = g.vps > 0 ? std::min(SF_MAX_R, SF_RING_BYTES / (2 * g.vps * 16)) : SF_MAX_R;
  return g;
}
size_t sf_align(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

}  // namespace

bool sampler_flow_supported(int V, int batch, int K, int sm_count) {
  if ((V % 8) != 0 || V < 8 || batch < 1 || batch > SF_MAX_B || batch > 65535 || K > GM_MAX_K_) return false;
  const SFGeom g = sf_geometry(V, sm_count, batch);
  return g.vps <= 32 * SF_UMAX && g.NA <= 32 * SF_EPL && batch <= SF_MAX_OWN * g.G && g.R >= 16 && g.G <= 65535;
}

// Workspace: control words, per-sequence state, stage words, arrival counters, slice partials (zero-initialised once;
// the kernel leaves the counters clean and tags the stage words with its epoch).  Its layout depends only on the
// capacity it was sized for, so launches of any smaller batch and any depth share it.  The tail is scratch of the dump.
size_t sampler_flow_ws_bytes(int cap_batch, int V, int sm_count) {
  const SFGeom g = sf_geometry(V, sm_count, 0);
  const size_t B = static_cast<size_t>(cap_batch), NA = static_cast<size_t>(g.NA);
  return sf_align(SF_CTRL_WORDS * 4) + sf_align(B * sizeof(SFSeq)) + sf_align(B * SF_ROUNDS * 8) + sf_align(B * SF_ROUNDS * 4) +
         sf_align(B * 4 * NA * 8) + sf_align(B * (2 * GM_MAX_K_ + 1) * NA * sizeof(MZ));
}

cudaError_t launch_sampler_flow(const SamplerArgs &A, int batch, void *ws, int cap_batch, int sm_count, cudaStream_t stream) {
  const SFGeom g = sf_geometry(A.V, sm_count, batch);
  const size_t B = static_cast<size_t>(cap_batch), NA = static_cast<size_t>(sf_geometry(A.V, sm_count, 0).NA);   // the layout's capacity
  if (batch > cap_batch) return cudaErrorInvalidValue;
  SFWs W;
  W.G = g.G; W.vps = g.vps; W.tail = g.tail; W.NA = g.NA; W.R = g.R; W.rounds = A.K + 4; W.nmain = g.nmain; W.wide = g.wide;
  unsigned char *p = static_cast<unsigned char *>(ws);
  W.ctrl = reinterpret_cast<uint32_t *>(p); p += sf_align(SF_CTRL_WORDS * 4);
  W.seq = reinterpret_cast<SFSeq *>(p); p += sf_align(B * sizeof(SFSeq));
  W.stage = reinterpret_cast<unsigned long long *>(p); p += sf_align(B * SF_ROUNDS * 8);
  W.cnt = reinterpret_cast<uint32_t *>(p); p += sf_align(B * SF_ROUNDS * 4);
  W.ent = reinterpret_cast<unsigned long long *>(p); p += sf_align(B * 4 * NA * 8);
  MZ *dump_scratch = reinterpret_cast<MZ *>(p);
  if (A.dbg_p != nullptr || A.dbg_q != nullptr) {
    sampler_flow_dump_kernel<<<batch * (2 * A.K + 1), SF_DUMP_THREADS, 0, stream>>>(A, g.G / g.wide, g.vps, g.tail, dump_scratch);
    if (cudaError_t e = cudaGetLastError(); e != cudaSuccess) return e;
  }
  const size_t dyn = static_cast<size_t>(g.R) * 2 * std::max(g.vps, 1) * 16;
  static SmemConfigured configured;
  if (cudaError_t e = ensure_dyn_smem(sampler_flow_kernel, dyn, configured); e != cudaSuccess) return e;
  return launch_k(sampler_flow_kernel, dim3(g.G), dim3(SF_THREADS), dyn, stream, 1, A, W, batch);
}


}  // namespace gm
