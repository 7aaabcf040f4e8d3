// Speculative rejection sampler, CTA-per-sequence variant for large batches (Sec. 2.2, Eq. 1).
//
// Same decisions and the same arithmetic as sampler.cu (sampler_common.cuh), different mapping: with a
// few hundred sequences there is enough parallelism to give every sequence ONE CTA, which removes every
// cluster-wide barrier.  The CTA streams whole logit rows in 24 KB chunks through a four-stage
// shared-memory ring: a producer warp issues bulk asynchronous copies as stages are released, sixteen
// compute warps wait on the stage's mbarrier on their own, reduce their 96 vectors of the chunk and
// release it - no CTA-wide synchronisation inside a row.  Positions are walked in order and the walk stops
// at the first rejection; the two rows of position a+1 are then streamed again (they are L2-resident) for
// the 64-bit integer weights, with one total per chunk, and the single chunk that holds the quantile is
// streamed once more for the token search.  The producer follows small commands the controller thread
// leaves in shared memory between CTA barriers (which rows, which chunks, sequential or interleaved).
#include "sampler_common.cuh"

namespace gm {

constexpr int SS_CWARPS = 16;                         // compute warps
constexpr int SS_CTHREADS = SS_CWARPS * 32;
constexpr int SS_THREADS = SS_CTHREADS + 32;          // + the producer warp
constexpr int SS_CH = 1536;                           // vectors (8 logits each) per chunk: 24 KB
constexpr int SS_NST = 4;                             // ring stages
constexpr int SS_VPW = SS_CH / SS_CWARPS;             // 96 vectors of a chunk per warp, 3 per lane
constexpr int SS_MAXCH = 64;                          // chunks per row: vocabularies up to 786k

struct SSCmd {
  const uint4 *row_a, *row_b;                         // row_b may be null
  int c_lo, c_hi;                                     // chunk range
  int interleave;                                     // 0: all chunks of a, then all chunks of b; 1: (a, b) chunk by chunk
  int quit;
};

__device__ __forceinline__ void ss_bar_compute() { asm volatile("bar.sync 1, %0;" ::"n"(SS_CTHREADS) : "memory"); }

__global__ void __launch_bounds__(SS_THREADS, 2) sampler_stream_kernel(const SamplerArgs A) {
  const int b = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool is_producer = warp == SS_CWARPS;
  const int K = A.K, V = A.V, R = 2 * K + 1;
  const float s = A.inv_temp * 1.4426950408889634f;
  const int nvec = V >> 3;
  const int C = (nvec + SS_CH - 1) / SS_CH;

  extern __shared__ __align__(128) unsigned char ss_smem[];
  const uint4 *ring = reinterpret_cast<const uint4 *>(ss_smem);                                  // [NST][CH]
  unsigned long long *vecsum = reinterpret_cast<unsigned long long *>(ss_smem + SS_NST * SS_CH * 16);   // [CH]
  __shared__ uint64_t full[SS_NST], empty[SS_NST];
  __shared__ SSCmd cmd;
  __shared__ MZ warp_mz[2][SS_CWARPS];
  __shared__ MZ row_mz[2];                            // (c, 1 / Z) of the rows in flight
  __shared__ unsigned long long chunk_w[SS_MAXCH];
  __shared__ unsigned long long scan_w[SS_CWARPS];
  __shared__ volatile int sh_dead;
  __shared__ int sh_ok, sh_tok;

  pdl_prologue();
  if (A.finished && A.finished[b]) {                  // the row sits out
    if (tid == 0) {
      if (A.accept_len) A.accept_len[b] = 0;
      A.next_token[static_cast<size_t>(b) * A.tok_out_stride] = A.accept_len ? -1 : 0;   // a plain draw leaves a valid id
    }
    return;
  }
  if (tid == 0) {
    for (int i = 0; i < SS_NST; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], SS_CWARPS); }
    mbar_fence_init();
    sh_dead = 0;
  }
  __syncthreads();

  const __nv_bfloat16 *tgt = A.target_logits + static_cast<size_t>(b) * A.tgt_bstride;
  const __nv_bfloat16 *drf = A.draft_logits ? A.draft_logits + static_cast<size_t>(b) * A.drf_bstride : nullptr;
  auto row_ptr = [&](int r) -> const uint4 * {
    const __nv_bfloat16 *p = r <= K ? tgt + static_cast<size_t>(r) * V : drf + static_cast<size_t>(r - K - 1) * V;
    return reinterpret_cast<const uint4 *>(p);
  };
  auto chunk_nv = [&](int ch) { return min(SS_CH, nvec - ch * SS_CH); };
  // bounded wait that gives up at once when another warp has already recorded a timeout
  auto wait_bar = [&](uint64_t *bar, uint32_t parity) -> bool {
    for (uint32_t i = 0; i < (1u << 22); ++i) {
      if (mbar_try_wait(bar, parity)) return true;
      if ((i & 255u) == 255u && sh_dead) return false;
    }
    sh_dead = 1;
    set_status(A.status, ST_TIMEOUT);
    return false;
  };

  uint32_t g = 0;                                     // job counter: the same sequence on both sides of the ring

  // ---- producer warp: executes the commands -----------------------------------------------------------------------
  if (is_producer) {
    for (;;) {
      __syncthreads();                                // a command is ready
      const SSCmd c = cmd;
      if (c.quit) break;
      if (lane == 0) {
        const int nrows = c.row_b ? 2 : 1;
        const int per = c.c_hi - c.c_lo;
        for (int j = 0; j < nrows * per; ++j, ++g) {
          const int which = c.interleave ? j % nrows : j / per;
          const int ch = c.c_lo + (c.interleave ? j / nrows : j % per);
          const int st = g % SS_NST;
          if (!wait_bar(&empty[st], ((g / SS_NST) & 1u) ^ 1u)) continue;       // dead: issue nothing more
          const uint32_t bytes = static_cast<uint32_t>(chunk_nv(ch)) * 16u;
          mbar_expect_tx(&full[st], bytes);
          fence_proxy_async();
          bulk_load(const_cast<uint4 *>(ring + st * SS_CH), (which ? c.row_b : c.row_a) + static_cast<size_t>(ch) * SS_CH,
                    bytes, &full[st]);
        }
      }
      g = __shfl_sync(0xffffffffu, g, 0);
    }
    return;
  }

  // ---- compute warps ------------------------------------------------------------------------------------------------
  // acquire / release of one job's stage by a warp
  auto acquire = [&]() -> const uint4 * {
    const int st = g % SS_NST;
    bool ok = true;
    if (lane == 0) ok = wait_bar(&full[st], (g / SS_NST) & 1u);
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    return ok ? ring + st * SS_CH : nullptr;
  };
  auto release = [&]() {
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty[g % SS_NST]);
    ++g;
  };
  auto post = [&](const uint4 *ra, const uint4 *rb, int c_lo, int c_hi, int interleave, int quit) {   // controller + barrier
    if (tid == 0) cmd = SSCmd{ra, rb, c_lo, c_hi, interleave, quit};
    __syncthreads();
  };
  const int v0 = warp * SS_VPW + lane;                // this lane's vectors of a chunk: v0, v0 + 32, v0 + 64
  const uint32_t NEG_INF2 = 0xff80ff80u;

  // (c, 1 / Z) of one or two rows streamed one after the other; result in row_mz[0..nrows-1]
  auto stats_rows = [&](const uint4 *ra, const uint4 *rb) {
    post(ra, rb, 0, C, 0, 0);
    const int nrows = rb ? 2 : 1;
    for (int r = 0; r < nrows; ++r) {
      MZ st{-INFINITY, 0.f};
      for (int ch = 0; ch < C; ++ch) {
        const uint4 *buf = acquire();
        const int nv = chunk_nv(ch);
        if (buf != nullptr && v0 < nv) {
          uint4 v[3];
          uint32_t m2 = NEG_INF2;
#pragma unroll
          for (int t = 0; t < 3; ++t) {
            v[t] = v0 + 32 * t < nv ? buf[v0 + 32 * t] : make_uint4(NEG_INF2, NEG_INF2, NEG_INF2, NEG_INF2);
            m2 = bmax2(bmax2(m2, bmax2(v[t].x, v[t].y)), bmax2(v[t].z, v[t].w));
          }
          const float mx = fmaxf(bf16_lo(m2), bf16_hi(m2));
          if (mx > st.m) { st.z *= ex2((st.m - mx) * s); st.m = mx; }          // 0 * 2^-inf = 0 on the first chunk
          const float c = -st.m * s;
          float acc = 0.f;
          if (st.m != -INFINITY) {                                              // only -inf (masked-out) logits so far: nothing to add
#pragma unroll
            for (int t = 0; t < 3; ++t) {
              float x[8];
              unpack8(v[t], x);
#pragma unroll
              for (int j = 0; j < 8; ++j) acc += ex2(fmaf(x[j], s, c));         // padding lanes: 2^-inf = 0
            }
          }
          st.z += acc;
        }
        release();
      }
      const float wm = warp_max(st.m);
      float z = wm == -INFINITY ? 0.f : st.z * ex2((st.m - wm) * s);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
      if (lane == 0) warp_mz[r][warp] = MZ{wm, z};
    }
    ss_bar_compute();
    if (tid < nrows) {
      MZ st = warp_mz[tid][0];
      for (int w = 1; w < SS_CWARPS; ++w) st = mz_merge(st, warp_mz[tid][w], s);
      row_mz[tid] = MZ{-st.m * s, __frcp_rn(st.z)};
    }
    ss_bar_compute();
  };

  // ---- optional dump of the probabilities (debug): statistics, then the row once more --------------------------------
  if (A.dbg_p != nullptr || A.dbg_q != nullptr) {
    for (int r = 0; r < R; ++r) {
      float *dst = r <= K ? (A.dbg_p ? A.dbg_p + static_cast<size_t>(b) * A.tgt_bstride + static_cast<size_t>(r) * V : nullptr)
                          : (A.dbg_q ? A.dbg_q + static_cast<size_t>(b) * A.drf_bstride + static_cast<size_t>(r - K - 1) * V : nullptr);
      stats_rows(row_ptr(r), nullptr);
      const MZ st = row_mz[0];
      post(row_ptr(r), nullptr, 0, C, 0, 0);
      for (int ch = 0; ch < C; ++ch) {
        const uint4 *buf = acquire();
        const int nv = chunk_nv(ch);
        if (buf != nullptr && dst != nullptr)
          for (int t = 0; t < 3; ++t) {
            const int i = v0 + 32 * t;
            if (i < nv) {
              float x[8];
              unpack8(buf[i], x);
#pragma unroll
              for (int j = 0; j < 8; ++j) dst[(static_cast<size_t>(ch) * SS_CH + i) * 8 + j] = prob_of(x[j], s, st.m, st.z);
            }
          }
        release();
      }
      ss_bar_compute();
    }
  }

  // ---- positions in order, stop at the first rejection ------------------------------------------------------------------
  int a = K;
  for (int k = 0; k <= K; ++k) {
    const bool bonus = k == K;
    stats_rows(row_ptr(k), bonus ? nullptr : row_ptr(K + 1 + k));
    if (bonus) break;
    if (tid == 0) {
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
      sh_ok = ok ? 1 : 0;
    }
    ss_bar_compute();
    const int ok = sh_ok;
    ss_bar_compute();                                 // sh_ok is rewritten only after everybody has read it
    if (!ok) { a = k; break; }
  }

  // ---- resampling at position a+1: integer weights, one total per chunk -----------------------------------------------------
  const uint4 *prow = row_ptr(a);
  const uint4 *qrow = a < K ? row_ptr(K + 1 + a) : nullptr;
  const MZ ps = row_mz[0];
  const MZ qs = a < K ? row_mz[1] : MZ{0.f, 1.f};
  bool use_q = a < K;
  unsigned long long W = 0;
  for (int attempt = 0; attempt < 2; ++attempt) {
    for (int i = tid; i < SS_MAXCH; i += SS_CTHREADS) chunk_w[i] = 0ull;
    post(prow, use_q ? qrow : nullptr, 0, C, 1, 0);   // the barrier inside also publishes the zeroed totals
    for (int ch = 0; ch < C; ++ch) {
      const uint4 *bp = acquire();
      const int nv = chunk_nv(ch);
      uint4 vp[3];
#pragma unroll
      for (int t = 0; t < 3; ++t) vp[t] = (bp != nullptr && v0 + 32 * t < nv) ? bp[v0 + 32 * t] : make_uint4(0u, 0u, 0u, 0u);
      const bool have = bp != nullptr;
      release();
      const uint4 *bq = nullptr;
      if (use_q) bq = acquire();
      unsigned long long tsum = 0;
      if (have && (!use_q || bq != nullptr)) {
#pragma unroll
        for (int t = 0; t < 3; ++t) {
          if (v0 + 32 * t < nv) {
            float xp[8], xq[8];
            unpack8(vp[t], xp);
            if (use_q) unpack8(bq[v0 + 32 * t], xq);
#pragma unroll
            for (int j = 0; j < 8; ++j)
              tsum += weight_of(prob_of(xp[j], s, ps.m, ps.z), use_q ? prob_of(xq[j], s, qs.m, qs.z) : 0.f, use_q);
          }
        }
      }
      if (use_q) release();
      tsum = warp_sum_u64(tsum);
      if (lane == 0 && tsum != 0ull) atomicAdd(&chunk_w[ch], tsum);            // integer: order-free
    }
    ss_bar_compute();
    W = 0;
    for (int ch = 0; ch < C; ++ch) W += chunk_w[ch];
    ss_bar_compute();
    if (W != 0 || !use_q) break;
    use_q = false;                                    // residual mass underflowed: draw from p instead
    if (tid == 0) set_status(A.status, ST_ZERO_RESID);
  }

  const uint32_t u_final = A.u24 ? A.u24[static_cast<size_t>(b) * A.u_stride + K]
                                 : philox_u24(A.seed, step_of(A), b, A.slot_final);
  if (W != 0) {
    const unsigned long long t = static_cast<unsigned long long>(u_final) * (W >> 24) +
                                 ((static_cast<unsigned long long>(u_final) * (W & 0xFFFFFFull)) >> 24);
    int cstar = 0;
    unsigned long long pre = 0;
    for (; cstar < C - 1; ++cstar) {
      if (t < pre + chunk_w[cstar]) break;
      pre += chunk_w[cstar];
    }
    const unsigned long long t_local = t - pre;
    // stream the chunk that holds the quantile once more and search it
    post(prow, use_q ? qrow : nullptr, cstar, cstar + 1, 1, 0);
    const uint4 *bp = acquire();
    const uint32_t g_p = g;
    ++g;                                              // keep the stage: released together with the q stage below
    const uint4 *bq = use_q ? acquire() : nullptr;
    const int nv = chunk_nv(cstar);
    const bool have = bp != nullptr && (!use_q || bq != nullptr);
    auto vec_weights = [&](int i, unsigned long long (&w)[8]) {
      float xp[8], xq[8];
      unpack8(bp[i], xp);
      if (use_q) unpack8(bq[i], xq);
#pragma unroll
      for (int j = 0; j < 8; ++j) w[j] = weight_of(prob_of(xp[j], s, ps.m, ps.z), use_q ? prob_of(xq[j], s, qs.m, qs.z) : 0.f, use_q);
    };
    for (int t3 = 0; t3 < 3; ++t3) {
      const int i = v0 + 32 * t3;
      unsigned long long sm = 0;
      if (have && i < nv) {
        unsigned long long w[8];
        vec_weights(i, w);
#pragma unroll
        for (int j = 0; j < 8; ++j) sm += w[j];
      }
      vecsum[i] = sm;
    }
    ss_bar_compute();
    // block-wide search over vecsum[0..CH): thread owns 3 consecutive vectors
    const int lo = tid * 3;
    const unsigned long long mine = vecsum[lo] + vecsum[lo + 1] + vecsum[lo + 2];
    unsigned long long incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += up;
    }
    if (lane == 31) scan_w[warp] = incl;
    if (tid == 0) sh_tok = 0;
    ss_bar_compute();
    unsigned long long base = 0;
    for (int w2 = 0; w2 < warp; ++w2) base += scan_w[w2];
    const unsigned long long excl = base + incl - mine;
    if (have && mine != 0 && t_local >= excl && t_local < excl + mine) {
      unsigned long long rem = t_local - excl;
      int iv = lo;
      while (rem >= vecsum[iv]) { rem -= vecsum[iv]; ++iv; }
      unsigned long long w[8];
      vec_weights(iv, w);
      int tok = (cstar * SS_CH + iv) * 8 + 7;
      for (int j = 0; j < 8; ++j) {
        if (rem < w[j]) { tok = (cstar * SS_CH + iv) * 8 + j; break; }
        rem -= w[j];
      }
      sh_tok = tok;
    }
    ss_bar_compute();
    // release both stages
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty[g_p % SS_NST]);
    if (use_q) release();
  } else {
    // no mass at all (cannot happen for a softmax of finite logits): lowest index of the row maximum
    if (tid == 0) sh_tok = 0x7fffffff;
    post(prow, nullptr, 0, C, 0, 0);
    for (int ch = 0; ch < C; ++ch) {
      const uint4 *bp = acquire();
      const int nv = chunk_nv(ch);
      if (bp != nullptr)
        for (int t3 = 0; t3 < 3; ++t3) {
          const int i = v0 + 32 * t3;
          if (i < nv) {
            float x[8];
            unpack8(bp[i], x);
#pragma unroll
            for (int j = 0; j < 8; ++j)
              if (-x[j] * s == ps.m) atomicMin(&sh_tok, (ch * SS_CH + i) * 8 + j);
          }
        }
      release();
    }
    ss_bar_compute();
    if (tid == 0) {
      if (sh_tok == 0x7fffffff) sh_tok = 0;
      set_status(A.status, ST_ZERO_MASS);
    }
    ss_bar_compute();
  }
  post(nullptr, nullptr, 0, 0, 0, 1);                 // the producer leaves

  // ---- outputs and state commit ------------------------------------------------------------------------------------------
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
    const int vec_per_row = A.d_model >> 3;
    const uint4 *src = reinterpret_cast<const uint4 *>(A.target_hidden + static_cast<size_t>(b) * (K + 1) * A.d_model);
    uint4 *dst = reinterpret_cast<uint4 *>(A.pending_hidden + static_cast<size_t>(b) * kp1 * A.d_model);
    for (int i = tid; i < (a + 1) * vec_per_row; i += SS_CTHREADS) dst[i] = src[i];
  }
}

bool sampler_stream_supported(int V) { return ((V >> 3) + SS_CH - 1) / SS_CH <= SS_MAXCH; }

cudaError_t launch_sampler_stream(const SamplerArgs &A, int batch, cudaStream_t stream) {
  const size_t dyn = static_cast<size_t>(SS_NST) * SS_CH * 16 + static_cast<size_t>(SS_CH) * sizeof(unsigned long long);
  static SmemConfigured configured;
  if (cudaError_t e = ensure_dyn_smem(sampler_stream_kernel, dyn, configured); e != cudaSuccess) return e;
  return launch_k(sampler_stream_kernel, dim3(batch), dim3(SS_THREADS), dyn, stream, 1, A);
}

}  // namespace gm
