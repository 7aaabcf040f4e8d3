// Nucleus (top-p) truncation of target logit rows.
//
// The paper's evaluation samples with top-p 0.7 (its rollouts with top-p 1).  The truncation is applied to the
// target's rows before the accept test: entries outside the nucleus are replaced by -inf, so that the sampler's own
// softmax over the filtered row is the renormalised truncated distribution.  The head's rows are not touched.
//
// The set is defined on integer weights, so that it does not depend on the order the masses are added in:
//   e[v] = 2^((x[v] - max) s)   (fp32, the sampler's formula),   w[v] = trunc(e[v] * 2^44),   W = sum w,
//   v is kept iff  (sum of w over entries with a larger logit) * 2^24 < tp24 * W,   tp24 = round(top_p * 2^24).
// A bf16 logit has 65536 possible values, so "larger logit" is a comparison of 16-bit keys, and the weight is a
// function of the key alone.  The kernel therefore counts, in shared memory, how often each key of a window of the
// NU_WIN keys just below the row maximum occurs (32-bit counters: plain native atomics, spread over a thousand
// populated keys), adds up W in registers in the same pass, and then finds the cut by an exclusive prefix sum of
// count x weight over the window.  If the whole window lies inside the nucleus (a very flat row) the window slides
// down and the count pass repeats; at most 65536 / NU_WIN times.  One CTA per row; normally three passes over the
// row (maximum, count, write), which stays in L2.
#include "sampler_common.cuh"

namespace gm {
namespace {

constexpr int NU_THREADS = 512;
constexpr int NU_WARPS = NU_THREADS / 32;
constexpr int NU_UNROLL = 4;
constexpr int NU_WIN = 8192;                           // keys per window: 64 binades of bf16
static_assert(NU_WIN % NU_THREADS == 0, "each thread owns a whole number of window keys");

// bf16 bit pattern -> 16-bit key that orders like the value (negative values reversed, positives above them)
__device__ __forceinline__ uint32_t order_key(uint32_t bits) {
  return (bits & 0x8000u) ? (~bits & 0xFFFFu) : (bits | 0x8000u);
}
// above * 2^24 < tp24 * W in 128-bit arithmetic
__device__ __forceinline__ bool below_cut(unsigned long long above, unsigned long long W, uint32_t tp24) {
  const unsigned long long lhs_hi = above >> 40, lhs_lo = above << 24;
  const unsigned long long rhs_hi = __umul64hi(W, static_cast<unsigned long long>(tp24)), rhs_lo = W * tp24;
  return lhs_hi < rhs_hi || (lhs_hi == rhs_hi && lhs_lo < rhs_lo);
}
__device__ __forceinline__ unsigned long long int_weight(float e) {
  return e > 0.f ? __float2ull_rz(__fmul_rn(e, 17592186044416.0f /* 2^44 */)) : 0ull;
}

__device__ __forceinline__ uint32_t key_bits(uint32_t key) {          // inverse of order_key
  return (key & 0x8000u) ? (key & 0x7FFFu) : (~key & 0xFFFFu);
}

__global__ void __launch_bounds__(NU_THREADS) nucleus_kernel(const NucleusArgs A) {
  __shared__ uint32_t cnt[NU_WIN];                     // occurrences of key (top - d), d = 0 .. NU_WIN-1
  __shared__ unsigned long long warp_sum[NU_WARPS];
  __shared__ float red[NU_WARPS];
  __shared__ unsigned long long s_total, s_above;
  __shared__ int s_cut;
  const int row = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nvec = A.V >> 3;
  const uint4 *src = reinterpret_cast<const uint4 *>(A.in + static_cast<size_t>(row) * A.V);
  uint4 *dst = reinterpret_cast<uint4 *>(A.out + static_cast<size_t>(row) * A.V);
  const float s = A.inv_temp * 1.4426950408889634f;
  pdl_prologue();

  // every pass walks the row NU_UNROLL vectors per thread at a time, all loads issued before the first use
  const uint4 pad = make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);       // -inf: weight 0, lowest key
  auto for_each_vec = [&](auto &&body) {
    for (int i0 = tid; i0 < nvec; i0 += NU_THREADS * NU_UNROLL) {
      uint4 v[NU_UNROLL];
#pragma unroll
      for (int u = 0; u < NU_UNROLL; ++u) {
        const int i = i0 + u * NU_THREADS;
        v[u] = i < nvec ? src[i] : pad;
      }
#pragma unroll
      for (int u = 0; u < NU_UNROLL; ++u) body(i0 + u * NU_THREADS, v[u]);
    }
  };
  auto block_sum = [&](unsigned long long v) -> unsigned long long {      // the same total in every thread
    for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    __syncthreads();
    if (lane == 0) warp_sum[warp] = v;
    __syncthreads();
    unsigned long long t = 0;
    for (int w = 0; w < NU_WARPS; ++w) t += warp_sum[w];
    return t;
  };

  // row maximum
  uint32_t m2 = 0xff80ff80u;
  for_each_vec([&](int, const uint4 &v) { m2 = bmax2(bmax2(m2, bmax2(v.x, v.y)), bmax2(v.z, v.w)); });
  float m = fmaxf(bf16_lo(m2), bf16_hi(m2));
  for (int off = 16; off >= 1; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
  if (lane == 0) red[warp] = m;
  __syncthreads();
  m = red[0];
  for (int w = 1; w < NU_WARPS; ++w) m = fmaxf(m, red[w]);
  const float c = -__fmul_rn(m, s);
  auto weight_of_bits = [&](uint32_t bits) { return int_weight(ex2(__fmaf_rn(__uint_as_float(bits << 16), s, c))); };

  uint32_t top = order_key(__float_as_uint(m) >> 16);  // largest key of the current window
  uint32_t cut_key = 0;
  for (int round = 0; round < 65536 / NU_WIN + 1; ++round) {
    for (int i = tid; i < NU_WIN; i += NU_THREADS) cnt[i] = 0u;
    if (tid == 0) s_cut = -1;
    __syncthreads();
    unsigned long long wsum = 0;
    for_each_vec([&](int, const uint4 &v) {
      const uint32_t wds[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        const uint32_t bits = (t & 1) ? (wds[t >> 1] >> 16) : (wds[t >> 1] & 0xFFFFu);
        const uint32_t d = top - order_key(bits);      // wraps to a large number for keys above the window
        if (d < static_cast<uint32_t>(NU_WIN)) atomicAdd(&cnt[d], 1u);
        if (round == 0) wsum += weight_of_bits(bits);
      }
    });
    if (round == 0) {
      const unsigned long long W = block_sum(wsum);
      if (tid == 0) { s_total = W; s_above = 0ull; }
    }
    __syncthreads();
    // exclusive prefix of count x weight over the window, keys from the top down; each thread owns NU_WIN / NU_THREADS keys
    constexpr int PER = NU_WIN / NU_THREADS;
    unsigned long long mass[PER], mine = 0;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      const uint32_t d = tid * PER + j;
      const uint32_t n = cnt[d];
      mass[j] = (n && d <= top) ? n * weight_of_bits(key_bits(top - d)) : 0ull;
      mine += mass[j];
    }
    unsigned long long incl = mine;                    // inclusive scan over the warp, then over the warps
    for (int off = 1; off < 32; off <<= 1) {
      const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, off);
      if (lane >= off) incl += up;
    }
    __syncthreads();
    if (lane == 31) warp_sum[warp] = incl;
    __syncthreads();
    unsigned long long above = s_above + incl - mine;
    for (int w = 0; w < warp; ++w) above += warp_sum[w];
    const unsigned long long W = s_total;
    int last = -1;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      if (mass[j] && below_cut(above, W, A.tp24)) last = tid * PER + j;
      above += mass[j];
    }
    if (last >= 0) atomicMax(&s_cut, last);
    __syncthreads();
    unsigned long long win = 0;
    for (int w = 0; w < NU_WARPS; ++w) win += warp_sum[w];
    const unsigned long long after = s_above + win;    // mass above everything below this window
    const int cut = s_cut;
    if (cut >= 0) cut_key = top - static_cast<uint32_t>(cut);
    // the next window can hold kept keys only if this one is entirely inside the nucleus and keys remain below it
    const bool go_on = below_cut(after, W, A.tp24) && after < W && top >= static_cast<uint32_t>(NU_WIN);
    __syncthreads();
    if (!go_on) break;
    if (tid == 0) s_above = after;
    top -= NU_WIN;
  }

  // pass 4: write the filtered row
  for_each_vec([&](int i, const uint4 &v) {
    if (i >= nvec) return;
    uint32_t wds[4] = {v.x, v.y, v.z, v.w};
    float e[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      const uint32_t bits = (t & 1) ? (wds[t >> 1] >> 16) : (wds[t >> 1] & 0xFFFFu);
      const bool keep = order_key(bits) >= cut_key;
      if (A.dbg_e) e[t] = ex2(__fmaf_rn(__uint_as_float(bits << 16), s, c));
      if (!keep) wds[t >> 1] = (t & 1) ? ((wds[t >> 1] & 0x0000FFFFu) | 0xFF800000u) : ((wds[t >> 1] & 0xFFFF0000u) | 0x0000FF80u);
    }
    dst[i] = make_uint4(wds[0], wds[1], wds[2], wds[3]);
    if (A.dbg_e) {
      float4 *d = reinterpret_cast<float4 *>(A.dbg_e + static_cast<size_t>(row) * A.V) + 2 * i;
      d[0] = make_float4(e[0], e[1], e[2], e[3]);
      d[1] = make_float4(e[4], e[5], e[6], e[7]);
    }
  });
}

}  // namespace

cudaError_t launch_nucleus(const NucleusArgs &A, cudaStream_t stream) {
  return launch_k(nucleus_kernel, dim3(A.rows), dim3(NU_THREADS), 0, stream, 1, A);
}

}  // namespace gm
