// The per-cycle record of a speculative rollout (App. D.2, what is recorded during the rollout): for each of the K verification
// positions the target's top-64 log-probabilities (bf16, full-vocabulary normalisation) with their token ids,
// plus the cycle's start hidden state, start position, drafts and accepted length.
//
// top-64 of a 150k-entry bf16 row: one CTA per row, the row streamed from global memory twice (it is L2-resident: the
// LM head has just written it, the sampler has just read it).  The selection works on the 16-bit order-preserving key
// of the bf16 logit.  Pass 1: (max, sum exp) with a running maximum, and every thread's own largest key; the 64th
// largest of the 512 thread maxima is a lower bound L of the row's 64th largest entry (they are 64 different entries).
// Pass 2 keeps aside every entry with key >= L - typically 70 to 100 of 150k, so the shared-memory atomics are rare -
// and the 64 places are the entries' ranks by (key descending, token id ascending) inside that list.  Rows with more
// than 1024 entries at or above L (long runs of equal values) take the general path instead: 256-bin histograms of the
// key (high byte, then low byte inside the boundary bin) fix the cut, a third pass collects the entries above it in
// any order and the ties at the cut in token order (block-wide scan, early exit), a bitonic sort orders the 64.
#include "common.cuh"
#include "kernels.h"

namespace gm {

constexpr int REC_THREADS = 512;
constexpr int REC_WARPS = REC_THREADS / 32;
constexpr int REC_TOP = 64;
constexpr int REC_UNROLL = 8;                         // row vectors a thread has in flight in the streaming passes
constexpr int REC_LIST = 1024;                        // entries kept aside in pass 2 (more than that: the general path)

__device__ __forceinline__ float rec_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// order-preserving 16-bit key of a bf16 value (larger value -> larger key; -0 is folded onto +0)
__device__ __forceinline__ uint32_t rec_key(uint32_t bits16) {
  if (bits16 == 0x8000u) bits16 = 0u;
  return (bits16 & 0x8000u) ? (~bits16 & 0xFFFFu) : (bits16 | 0x8000u);
}
__device__ __forceinline__ float rec_value(uint32_t key) {
  const uint32_t bits16 = (key & 0x8000u) ? (key & 0x7FFFu) : (~key & 0xFFFFu);
  return __uint_as_float(bits16 << 16);
}
__device__ __forceinline__ void rec_keys8(const uint4 &v, uint32_t (&k)[8]) {
  k[0] = rec_key(v.x & 0xFFFFu); k[1] = rec_key(v.x >> 16); k[2] = rec_key(v.y & 0xFFFFu); k[3] = rec_key(v.y >> 16);
  k[4] = rec_key(v.z & 0xFFFFu); k[5] = rec_key(v.z >> 16); k[6] = rec_key(v.w & 0xFFFFu); k[7] = rec_key(v.w >> 16);
}
__device__ __forceinline__ uint4 rec_ldg(const uint4 *p) {
  uint4 v;
  asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t rec_bmax2(uint32_t a, uint32_t b) {      // packed bf16x2 maximum
  __nv_bfloat162 r = __hmax2(*reinterpret_cast<__nv_bfloat162 *>(&a), *reinterpret_cast<__nv_bfloat162 *>(&b));
  return *reinterpret_cast<uint32_t *>(&r);
}

__device__ __forceinline__ uint32_t rec_ge2(uint32_t a, uint32_t b) {       // per half: 0xFFFF where a >= b
  return __hge2_mask(*reinterpret_cast<__nv_bfloat162 *>(&a), *reinterpret_cast<__nv_bfloat162 *>(&b));
}

struct RecMZ { float m, z; };

__global__ void __launch_bounds__(REC_THREADS, 2) record_topk_kernel(const RecordTopkArgs A) {
  const int b = blockIdx.x / A.K, k = blockIdx.x % A.K;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int V = A.V, nvec = V >> 3;
  const float s = A.inv_temp * 1.4426950408889634f;

  __shared__ uint32_t hist[REC_WARPS][256];
  __shared__ uint32_t hsum[256];
  __shared__ unsigned long long cand[REC_TOP];
  __shared__ RecMZ warp_mz[REC_WARPS];
  __shared__ int sh_cut, sh_above, sh_cnt, sh_nlist;
  __shared__ unsigned long long wlist[REC_LIST];          // pass 2: every entry at or above the lower bound
  __shared__ int warp_tot[REC_WARPS];
  __shared__ uint32_t tkeys[REC_THREADS];
  __shared__ uint32_t sh_low;

  pdl_prologue();
  const uint4 *row = reinterpret_cast<const uint4 *>(A.target_logits + static_cast<size_t>(b) * A.bstride + static_cast<size_t>(k) * V);
  if (tid < REC_TOP) cand[tid] = 0ull;
  if (tid == 0) { sh_cnt = 0; sh_nlist = 0; }

  // ---- pass 1: (max, sum 2^((x - max) s)) with a running maximum; the largest key ---------------------------------------
  RecMZ st{-INFINITY, 0.f};
  uint32_t tm2 = 0xff80ff80u;                          // packed maximum of this thread's entries
  for (int i0 = tid; i0 < nvec; i0 += REC_UNROLL * REC_THREADS) {
    uint4 v[REC_UNROLL];
    uint32_t m2 = 0xff80ff80u;
#pragma unroll
    for (int t = 0; t < REC_UNROLL; ++t) {
      const int i = i0 + t * REC_THREADS;
      v[t] = i < nvec ? rec_ldg(row + i) : make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
      m2 = rec_bmax2(rec_bmax2(m2, rec_bmax2(v[t].x, v[t].y)), rec_bmax2(v[t].z, v[t].w));
    }
    tm2 = rec_bmax2(tm2, m2);
    const float mx = fmaxf(bf16_lo(m2), bf16_hi(m2));
    if (mx > st.m) { st.z *= rec_ex2((st.m - mx) * s); st.m = mx; }           // 0 * 2^-inf = 0 on the first block
    if (st.m != -INFINITY) {
      const float c = -st.m * s;
      float acc = 0.f;
#pragma unroll
      for (int t = 0; t < REC_UNROLL; ++t)
        acc += rec_ex2(fmaf(bf16_lo(v[t].x), s, c)) + rec_ex2(fmaf(bf16_hi(v[t].x), s, c)) + rec_ex2(fmaf(bf16_lo(v[t].y), s, c)) +
               rec_ex2(fmaf(bf16_hi(v[t].y), s, c)) + rec_ex2(fmaf(bf16_lo(v[t].z), s, c)) + rec_ex2(fmaf(bf16_hi(v[t].z), s, c)) +
               rec_ex2(fmaf(bf16_lo(v[t].w), s, c)) + rec_ex2(fmaf(bf16_hi(v[t].w), s, c));
      st.z += acc;
    }
  }
  {
    const float wm = warp_max(st.m);
    float z = (wm == -INFINITY || st.m == -INFINITY) ? 0.f : st.z * rec_ex2((st.m - wm) * s);
    z = warp_sum(z);
    if (lane == 0) warp_mz[warp] = RecMZ{wm, z};
    // a thread without entries counts as the lowest key
    tkeys[tid] = tid < nvec ? rec_key(__float_as_uint(fmaxf(bf16_lo(tm2), bf16_hi(tm2))) >> 16) : 0u;
  }
  __syncthreads();
  RecMZ rowst{-INFINITY, 0.f};
  for (int w = 0; w < REC_WARPS; ++w) rowst.m = fmaxf(rowst.m, warp_mz[w].m);
  for (int w = 0; w < REC_WARPS; ++w)
    if (warp_mz[w].z > 0.f) rowst.z += warp_mz[w].z * rec_ex2((warp_mz[w].m - rowst.m) * s);   // same order in every thread
  const uint32_t kmax = rec_key(__float_as_uint(rowst.m) >> 16);

  // ---- lower bound of the 64th largest entry, the entries at or above it, their ranks ---------------------------------------
  const int want = min(REC_TOP, V);
  {
    const uint32_t mine = tkeys[tid];
    int rnk = 0;
    for (int j = 0; j < REC_THREADS; ++j) {
      const uint32_t o = tkeys[j];
      rnk += (o > mine) || (o == mine && j < tid);
    }
    if (rnk == REC_TOP - 1) sh_low = mine;
  }
  __syncthreads();
  const uint32_t low = max(sh_low, 0x007Fu);            // not below the key of -inf (threads without entries hold key 0)
  const uint32_t low_bits = __float_as_uint(rec_value(low)) >> 16, low2 = (low_bits << 16) | low_bits;
  for (int i0 = tid; i0 < nvec; i0 += REC_UNROLL * REC_THREADS) {
    uint4 v[REC_UNROLL];
#pragma unroll
    for (int t = 0; t < REC_UNROLL; ++t) {
      const int i = i0 + t * REC_THREADS;
      v[t] = i < nvec ? rec_ldg(row + i) : make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
    }
#pragma unroll
    for (int t = 0; t < REC_UNROLL; ++t) {
      // numeric packed comparison first (-0 equals +0 there as in the key): almost no vector holds an entry at or above the bound
      if (i0 + t * REC_THREADS < nvec && (rec_ge2(v[t].x, low2) | rec_ge2(v[t].y, low2) | rec_ge2(v[t].z, low2) | rec_ge2(v[t].w, low2)) != 0u) {
        uint32_t key[8];
        rec_keys8(v[t], key);
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (key[j] >= low) {
            const int pos = atomicAdd(&sh_nlist, 1);
            if (pos < REC_LIST)
              wlist[pos] = (static_cast<unsigned long long>(key[j]) << 32) |
                           (0xFFFFFFFFull - static_cast<unsigned long long>((i0 + t * REC_THREADS) * 8 + j));
          }
      }
    }
  }
  __syncthreads();
  const bool from_list = sh_nlist <= REC_LIST;
  if (from_list) {
    const int nl = sh_nlist;
    for (int i = tid; i < nl; i += REC_THREADS) {
      const unsigned long long e = wlist[i];
      int rnk = 0;
      for (int j = 0; j < nl; ++j) rnk += wlist[j] > e;        // larger composite: larger key, then lower token id
      if (rnk < REC_TOP) cand[rnk] = e;
    }
  } else {
    // ---- the general path.  The cut: 256-bin histograms of the key, high byte first, then the low byte inside the boundary bin
    if (tid == 0) sh_cnt = 0;
    uint32_t base = 0u;
    int shift = 8;
    for (int level = 0; level < 2; ++level) {
      for (int i = tid; i < REC_WARPS * 256; i += REC_THREADS) (&hist[0][0])[i] = 0u;
      __syncthreads();
      for (int i0 = tid; i0 < nvec; i0 += 4 * REC_THREADS) {
        uint4 v[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const int i = i0 + t * REC_THREADS;
          v[t] = i < nvec ? rec_ldg(row + i) : make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
        }
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          if (i0 + t * REC_THREADS < nvec) {
            uint32_t key[8];
            rec_keys8(v[t], key);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const uint32_t rel = (key[j] - base) >> shift;
              if (key[j] >= base && rel < 256u) atomicAdd(&hist[warp][rel], 1u);
            }
          }
        }
      }
      __syncthreads();
      if (tid < 256) {
        uint32_t t = 0;
        for (int w = 0; w < REC_WARPS; ++w) t += hist[w][tid];
        hsum[tid] = t;
      }
      __syncthreads();
      if (tid == 0) {
        // walk down from the largest bin until `need` entries are covered
        const int need = level == 1 ? want - sh_above : want;
        int above = 0, bin = 255;
        for (; bin > 0; --bin) {
          if (above + static_cast<int>(hsum[bin]) >= need) break;
          above += static_cast<int>(hsum[bin]);
        }
        sh_cut = level == 0 ? bin : bin + static_cast<int>(base);     // the boundary bin, then the cut key
        if (level == 1) sh_above += above; else sh_above = above;
      }
      __syncthreads();
      base = static_cast<uint32_t>(sh_cut) << 8; shift = 0;
      __syncthreads();                                // sh_* have been read before the next level rewrites them
    }
    const uint32_t cut = static_cast<uint32_t>(sh_cut);     // entries with key > cut are in; `take` of the ties at the cut
    const int above = sh_above, take = want - above;

    // ---- pass 3: entries above the cut in any order; ties at the cut in token order --------------------------------------
    int tie_base = 0;
    for (int i0 = 0; i0 < nvec; i0 += REC_THREADS) {
      const int i = i0 + tid;
      uint32_t key[8];
      int mine = 0;
      if (i < nvec) {
        rec_keys8(rec_ldg(row + i), key);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          mine += key[j] == cut;
          if (key[j] > cut) {
            const int pos = atomicAdd(&sh_cnt, 1);
            if (pos < REC_TOP)
              cand[pos] = (static_cast<unsigned long long>(key[j]) << 32) | (0xFFFFFFFFull - static_cast<unsigned long long>(i * 8 + j));
          }
        }
      }
      if (tie_base < take) {                                // uniform: tie_base is the same in every thread
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int up = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += up;
        }
        __syncthreads();                                    // warp_tot of the previous iteration has been read
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        int basep = tie_base, total = 0;
        for (int w = 0; w < REC_WARPS; ++w) { if (w < warp) basep += warp_tot[w]; total += warp_tot[w]; }
        int rnk = basep + incl - mine;
        if (i < nvec && mine > 0) {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (key[j] == cut) {
              if (rnk < take)
                cand[above + rnk] = (static_cast<unsigned long long>(cut) << 32) | (0xFFFFFFFFull - static_cast<unsigned long long>(i * 8 + j));
              ++rnk;
            }
        }
        tie_base += total;
      }
    }
    __syncthreads();
    // order the 64 candidates (key descending, then lower token id first)
    for (int size = 2; size <= REC_TOP; size <<= 1)
      for (int stride = size >> 1; stride > 0; stride >>= 1) {
        if (tid < REC_TOP) {
          const int partner = tid ^ stride;
          if (partner > tid) {
            const unsigned long long a2 = cand[tid], c2 = cand[partner];
            const bool desc = (tid & size) == 0;
            if (desc ? a2 < c2 : a2 > c2) { cand[tid] = c2; cand[partner] = a2; }
          }
        }
        __syncthreads();
      }
  }
  __syncthreads();

  // ---- the record ----------------------------------------------------------------------------------------------------------
  if (tid < REC_TOP) {
    const unsigned long long e = cand[tid];
    const size_t o = (static_cast<size_t>(b) * A.K + k) * REC_TOP + tid;
    if (e == 0ull) {
      A.top_index[o] = -1;
      A.top_logprob[o] = __float2bfloat16(-INFINITY);
    } else {
      const float x = rec_value(static_cast<uint32_t>(e >> 32));
      A.top_index[o] = static_cast<int32_t>(0xFFFFFFFFull - (e & 0xFFFFFFFFull));
      // ln p = ((x - max) s - log2 Z) ln 2
      A.top_logprob[o] = __float2bfloat16(((x - rowst.m) * s - log2f(rowst.z)) * 0.6931471805599453f);
    }
  }
}

cudaError_t launch_record_topk(const RecordTopkArgs &A, int batch, cudaStream_t stream) {
  return launch_k(record_topk_kernel, dim3(batch * A.K), dim3(REC_THREADS), 0, stream, 1, A);
}

// ---- the other items of the record -----------------------------------------------------------------------------------------
// begin: hidden state and position of the cycle's start (before the cycle advances the state)
__global__ void record_begin_kernel(const int32_t *kv_len, const int32_t *pending_n, const __nv_bfloat16 *pending_hidden,
                                    int max_k, int d, __nv_bfloat16 *start_hidden, int32_t *start_pos) {
  const int b = blockIdx.x;
  pdl_prologue();
  const int n = min(max(pending_n[b], 1), max_k + 1);
  const uint4 *src = reinterpret_cast<const uint4 *>(pending_hidden + (static_cast<size_t>(b) * (max_k + 1) + n - 1) * d);
  uint4 *dst = reinterpret_cast<uint4 *>(start_hidden + static_cast<size_t>(b) * d);
  for (int i = threadIdx.x; i < (d >> 3); i += blockDim.x) dst[i] = src[i];
  if (threadIdx.x == 0) start_pos[b] = kv_len[b] + 1;      // context length at which drafting starts
}
// end: drafts and the accepted length with the final token counted
__global__ void record_end_kernel(const int32_t *draft_tok, const int32_t *accept_len, int batch, int k, int32_t *drafts,
                                  int32_t *accepted) {
  pdl_prologue();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < batch * k) drafts[i] = draft_tok[i];
  if (i < batch) accepted[i] = accept_len[i] + 1;
}
cudaError_t launch_record_begin(const int32_t *kv_len, const int32_t *pending_n, const __nv_bfloat16 *pending_hidden,
                                int batch, int max_k, int d, __nv_bfloat16 *start_hidden, int32_t *start_pos,
                                cudaStream_t stream) {
  return launch_k(record_begin_kernel, dim3(batch), dim3(128), 0, stream, 1, kv_len, pending_n, pending_hidden, max_k, d,
                  start_hidden, start_pos);
}
cudaError_t launch_record_end(const int32_t *draft_tok, const int32_t *accept_len, int batch, int k, int32_t *drafts,
                              int32_t *accepted, cudaStream_t stream) {
  const int n = batch * k;
  return launch_k(record_end_kernel, dim3((n + 255) / 256), dim3(256), 0, stream, 1, draft_tok, accept_len, batch, k, drafts,
                  accepted);
}

}  // namespace gm
