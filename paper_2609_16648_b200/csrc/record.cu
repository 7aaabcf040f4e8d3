// The per-cycle record of a speculative rollout (App. D.2 "Recording in Rollout"): for each of the K verification
// positions the target's top-64 log-probabilities (bf16, full-vocabulary normalisation) with their token ids,
// plus the cycle's start hidden state, start position, drafts and accepted length.
//
// top-64 of a 150k-entry bf16 row.  One cluster of 8 CTAs per row, each CTA one eighth of the vocabulary, copied
// once into shared memory (bulk asynchronous copy).  Every global top-64 entry is in its CTA's local top-64, so a
// CTA selects its local 64 exactly with two 256-bin histogram passes over the 16-bit order-preserving key of the
// bf16 logit (high byte, then low byte inside the boundary bin), collects the entries above the cut in any order
// and the ties at the cut in token order (block-wide scan), and the cluster's first CTA merges the 8 x 64
// candidates with a bitonic sort on (key descending, token id ascending).  Log-probabilities use the row's
// (max, sum exp) reduced over the cluster in fixed order.
#include <cooperative_groups.h>

#include "common.cuh"
#include "kernels.h"

namespace cg = cooperative_groups;

namespace gm {

constexpr int REC_THREADS = 512;
constexpr int REC_WARPS = REC_THREADS / 32;
constexpr int REC_CLUSTER = 8;
constexpr int REC_TOP = 64;

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

struct RecMZ { float m, z; };

__global__ void __cluster_dims__(REC_CLUSTER, 1, 1) __launch_bounds__(REC_THREADS)
record_topk_kernel(const RecordTopkArgs A) {
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = static_cast<int>(cluster.block_rank());
  const int row_id = blockIdx.x / REC_CLUSTER, b = row_id / A.K, k = row_id % A.K;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int V = A.V;
  const float s = A.inv_temp * 1.4426950408889634f;

  const int nvec_total = V >> 3;
  const int vpc = (nvec_total + REC_CLUSTER - 1) / REC_CLUSTER;
  const int v_lo = min(rank * vpc, nvec_total);
  const int n = min(v_lo + vpc, nvec_total) - v_lo;

  extern __shared__ __align__(128) unsigned char rec_smem[];
  const uint4 *buf = reinterpret_cast<const uint4 *>(rec_smem);                           // [vpc] the row slice
  __shared__ uint32_t hist[REC_WARPS][256];
  __shared__ uint32_t hsum[256];
  __shared__ unsigned long long cand[REC_TOP];            // this CTA's candidates (read by the first CTA)
  __shared__ unsigned long long merge[REC_CLUSTER * REC_TOP];
  __shared__ RecMZ warp_mz[REC_WARPS];
  __shared__ RecMZ local_mz;                              // read by the first CTA
  __shared__ uint64_t full_bar;
  __shared__ int sh_cut, sh_above, sh_take, sh_cnt, sh_alive;
  __shared__ int warp_tot[REC_WARPS];

  pdl_prologue();
  if (tid == 0) {
    mbar_init(&full_bar, 1);
    mbar_fence_init();
    sh_alive = 1;
    sh_cnt = 0;
  }
  if (tid < REC_TOP) cand[tid] = 0ull;
  __syncthreads();
  const uint4 *src = reinterpret_cast<const uint4 *>(A.target_logits + static_cast<size_t>(b) * A.bstride +
                                                      static_cast<size_t>(k) * V) + v_lo;
  if (tid == 0 && n > 0) {
    mbar_expect_tx(&full_bar, static_cast<uint32_t>(n) * 16u);
    bulk_load(const_cast<uint4 *>(buf), src, static_cast<uint32_t>(n) * 16u, &full_bar);
    if (!mbar_wait(&full_bar, 0)) { sh_alive = 0; set_status(A.status, ST_TIMEOUT); }
  }
  __syncthreads();
  const bool alive = sh_alive != 0;
  const int n_use = alive ? n : 0;

  // ---- (max, sum 2^((x - max) s)) of the slice ----------------------------------------------------------------------
  {
    float mx = -INFINITY;
    for (int i = tid; i < n_use; i += REC_THREADS) {
      const uint4 v = buf[i];
      mx = fmaxf(mx, fmaxf(fmaxf(fmaxf(bf16_lo(v.x), bf16_hi(v.x)), fmaxf(bf16_lo(v.y), bf16_hi(v.y))),
                           fmaxf(fmaxf(bf16_lo(v.z), bf16_hi(v.z)), fmaxf(bf16_lo(v.w), bf16_hi(v.w)))));
    }
    mx = warp_max(mx);
    if (lane == 0) warp_mz[warp].m = mx;
    __syncthreads();
    float m = -INFINITY;
    for (int w = 0; w < REC_WARPS; ++w) m = fmaxf(m, warp_mz[w].m);
    const float c = -m * s;
    float z = 0.f;
    for (int i = tid; i < n_use; i += REC_THREADS) {
      const uint4 v = buf[i];
      z += rec_ex2(fmaf(bf16_lo(v.x), s, c)) + rec_ex2(fmaf(bf16_hi(v.x), s, c)) + rec_ex2(fmaf(bf16_lo(v.y), s, c)) +
           rec_ex2(fmaf(bf16_hi(v.y), s, c)) + rec_ex2(fmaf(bf16_lo(v.z), s, c)) + rec_ex2(fmaf(bf16_hi(v.z), s, c)) +
           rec_ex2(fmaf(bf16_lo(v.w), s, c)) + rec_ex2(fmaf(bf16_hi(v.w), s, c));
    }
    z = warp_sum(z);
    if (lane == 0) warp_mz[warp].z = z;
    __syncthreads();
    if (tid == 0) {
      float zt = 0.f;
      for (int w = 0; w < REC_WARPS; ++w) zt += warp_mz[w].z;
      local_mz = RecMZ{m, n_use > 0 ? zt : 0.f};
    }
  }

  // ---- local top-64: two histogram levels on the 16-bit key ---------------------------------------------------------
  const int want = min(REC_TOP, n_use * 8);
  int hi_bin = -1;                                           // level 1 boundary bin; level 2 runs inside it
  for (int level = 0; level < 2; ++level) {
    for (int i = tid; i < REC_WARPS * 256; i += REC_THREADS) (&hist[0][0])[i] = 0u;
    __syncthreads();
    for (int i = tid; i < n_use; i += REC_THREADS) {
      uint32_t key[8];
      rec_keys8(buf[i], key);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if (level == 0) atomicAdd(&hist[warp][key[j] >> 8], 1u);
        else if (static_cast<int>(key[j] >> 8) == hi_bin) atomicAdd(&hist[warp][key[j] & 0xFFu], 1u);
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
      int need = level == 0 ? want : want - sh_above;
      int above = 0, bin = 255;
      for (; bin > 0; --bin) {
        if (above + static_cast<int>(hsum[bin]) >= need) break;
        above += static_cast<int>(hsum[bin]);
      }
      if (level == 0) { sh_cut = bin; sh_above = above; }
      else { sh_cut = (hi_bin << 8) | bin; sh_above += above; sh_take = want - sh_above; }
    }
    __syncthreads();
    if (level == 0) hi_bin = sh_cut;
  }
  const uint32_t cut = static_cast<uint32_t>(sh_cut);       // entries with key > cut are in; `take` of the ties at the cut
  const int above = sh_above, take = sh_take;

  // entries above the cut, any order
  for (int i = tid; i < n_use; i += REC_THREADS) {
    uint32_t key[8];
    rec_keys8(buf[i], key);
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (key[j] > cut) {
        const int pos = atomicAdd(&sh_cnt, 1);
        if (pos < REC_TOP)
          cand[pos] = (static_cast<unsigned long long>(key[j]) << 32) |
                      (0xFFFFFFFFull - static_cast<unsigned long long>((v_lo + i) * 8 + j));
      }
  }
  // ties at the cut, in token order: block-wide exclusive scan of the per-vector tie counts
  int tie_base = 0;
  for (int i0 = 0; i0 < n_use && tie_base < take; i0 += REC_THREADS) {
    const int i = i0 + tid;
    uint32_t key[8];
    int mine = 0;
    if (i < n_use) {
      rec_keys8(buf[i], key);
#pragma unroll
      for (int j = 0; j < 8; ++j) mine += key[j] == cut;
    }
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int up = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += up;
    }
    __syncthreads();                                        // warp_tot of the previous iteration has been read
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    int base = tie_base;
    for (int w = 0; w < warp; ++w) base += warp_tot[w];
    int total = 0;
    for (int w = 0; w < REC_WARPS; ++w) total += warp_tot[w];
    int rnk = base + incl - mine;
    if (i < n_use && mine > 0) {
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (key[j] == cut) {
          if (rnk < take)
            cand[above + rnk] = (static_cast<unsigned long long>(cut) << 32) |
                                (0xFFFFFFFFull - static_cast<unsigned long long>((v_lo + i) * 8 + j));
          ++rnk;
        }
    }
    tie_base += total;
  }
  cluster.sync();

  // ---- merge in the first CTA -------------------------------------------------------------------------------------------
  if (rank == 0) {
    merge[tid] = *(cluster.map_shared_rank(&cand[0], tid / REC_TOP) + (tid % REC_TOP));     // 8 x 64 = 512 = REC_THREADS
    __shared__ RecMZ row;
    if (tid == 0) {
      float m = -INFINITY;
      RecMZ parts[REC_CLUSTER];
      for (int c2 = 0; c2 < REC_CLUSTER; ++c2) { parts[c2] = *cluster.map_shared_rank(&local_mz, c2); m = fmaxf(m, parts[c2].m); }
      float z = 0.f;
      for (int c2 = 0; c2 < REC_CLUSTER; ++c2)
        if (parts[c2].z > 0.f) z += parts[c2].z * rec_ex2((parts[c2].m - m) * s);
      row = RecMZ{m, z};
    }
    __syncthreads();
    // bitonic sort, descending, 512 composites (key, then lower token id first)
    for (int size = 2; size <= REC_CLUSTER * REC_TOP; size <<= 1)
      for (int stride = size >> 1; stride > 0; stride >>= 1) {
        const int partner = tid ^ stride;
        if (partner > tid) {
          const unsigned long long a = merge[tid], c2 = merge[partner];
          const bool desc = (tid & size) == 0;
          if (desc ? a < c2 : a > c2) { merge[tid] = c2; merge[partner] = a; }
        }
        __syncthreads();
      }
    if (tid < REC_TOP) {
      const unsigned long long e = merge[tid];
      const size_t o = (static_cast<size_t>(b) * A.K + k) * REC_TOP + tid;
      if (e == 0ull) {
        A.top_index[o] = -1;
        A.top_logprob[o] = __float2bfloat16(-INFINITY);
      } else {
        const float x = rec_value(static_cast<uint32_t>(e >> 32));
        A.top_index[o] = static_cast<int32_t>(0xFFFFFFFFull - (e & 0xFFFFFFFFull));
        // ln p = ((x - max) s - log2 Z) ln 2
        A.top_logprob[o] = __float2bfloat16(((x - row.m) * s - log2f(row.z)) * 0.6931471805599453f);
      }
    }
  }
  cluster.sync();                                           // the peers' shared memory stays alive until it has been read
}

cudaError_t launch_record_topk(const RecordTopkArgs &A, int batch, cudaStream_t stream) {
  const int vpc = ((A.V >> 3) + REC_CLUSTER - 1) / REC_CLUSTER;
  const size_t dyn = (static_cast<size_t>(vpc) * 16 + 127) & ~size_t(127);
  if (dyn > 160 * 1024) return cudaErrorInvalidValue;
  static SmemConfigured configured;
  if (cudaError_t e = ensure_dyn_smem(record_topk_kernel, dyn, configured); e != cudaSuccess) return e;
  return launch_k(record_topk_kernel, dim3(batch * A.K * REC_CLUSTER), dim3(REC_THREADS), dyn, stream, 1, A);
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
