// Dense projections out[M, N] = x[M, K] * w[N, K]^T (bf16 operands, fp32 accumulation).
//
// gemm_tc_kernel (the product path).  The step's projections have few rows (M = batch * (K+1)
// <= a few hundred tokens) and many output features, so the operands are swapped onto the tensor
// core: a CTA takes 128 output features as the MMA's M extent (one TMEM lane per feature) and up
// to 256 tokens as its N extent, and streams its 128 x K weight slab exactly once.  Warp 0 (one
// elected thread) is the TMA producer filling a ring of 128-byte-swizzled stages (64 K-elements per
// stage: a 128 x 64 weight box and a T x 64 activation box); warp 1 owns the tensor memory
// allocation and one of its threads issues tcgen05.mma (four K=16 instructions per stage),
// releasing each stage with tcgen05.commit; warps 2-5 read the fp32 accumulator out of tensor
// memory with tcgen05.ld once the last commit lands and store it transposed (lanes = consecutive
// features, so stores coalesce).  Optional split-K over blockIdx.z writes fp32 partials that the
// consumer kernels sum in a fixed order.  Every wait is bounded; on expiry the kernel records
// ST_TIMEOUT, still meets the final barrier and frees its tensor memory.
//
// gemm_simple_kernel: a plain warp-level mma.sync version with the same interface, kept as an
// independent on-device cross-check and for shapes the tcgen05 kernel does not take.
#include "common.cuh"
#include "kernels.h"

namespace gm {

constexpr int GT_BN = 128;            // output features per CTA (MMA M)
constexpr int GT_BK = 64;             // K elements per stage (one 128-byte swizzle row)
constexpr int GT_THREADS = 192;
constexpr int GT_SMEM_BUDGET = 200 * 1024;

static int gt_stages(int block_t) {
  int s = GT_SMEM_BUDGET / (GT_BN * 128 + block_t * 128);
  return s > 8 ? 8 : s;
}
static size_t gt_smem(int block_t) {
  return static_cast<size_t>(gt_stages(block_t)) * (GT_BN * 128 + block_t * 128) + 1024 + 256;
}

__global__ void __launch_bounds__(GT_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ GemmArgs A, const int nstages) {
  extern __shared__ unsigned char gt_smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(gt_smem_raw) + 1023) & ~uintptr_t(1023));
  const int T = A.block_t;
  const int a_bytes = GT_BN * 128, b_bytes = T * 128, stage_b = a_bytes + b_bytes;
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + static_cast<size_t>(nstages) * stage_b);
  uint64_t *empty = full + 8;
  uint64_t *acc_full = empty + 8;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * GT_BN, m0 = blockIdx.y * T, split = blockIdx.z;
  const int KB = A.K / GT_BK;
  const int kb_lo = static_cast<int>(static_cast<long long>(split) * KB / A.nsplit);
  const int kb_hi = static_cast<int>(static_cast<long long>(split + 1) * KB / A.nsplit);
  const uint32_t ncols = T <= 32 ? 32u : T <= 64 ? 64u : T <= 128 ? 128u : 256u;

  if (threadIdx.x == 0) {
    for (int s = 0; s < nstages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    mbar_fence_init();
  }
  if (warp == 1) {
    tc_alloc(tmem_slot, ncols);
    tc_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      tma_prefetch_desc(&A.w_map);
      tma_prefetch_desc(&A.x_map);
      for (int kb = kb_lo, it = 0; kb < kb_hi; ++kb, ++it) {
        const int s = it % nstages;
        if (!mbar_wait(&empty[s], ((it / nstages) & 1) ^ 1)) { set_status(A.status, ST_TIMEOUT); break; }
        mbar_expect_tx(&full[s], stage_b);
        unsigned char *dst = smem + static_cast<size_t>(s) * stage_b;
        tma_load_2d(dst, &A.w_map, kb * GT_BK, n0, &full[s]);
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
        const uint64_t adesc = tc_smem_desc_sw128(a_addr), bdesc = tc_smem_desc_sw128(a_addr + a_bytes);
#pragma unroll
        for (int k = 0; k < GT_BK / 16; ++k)      // +32 bytes (2 x 16-byte units) per K=16 step
          tc_mma_bf16(tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (it > 0 || k > 0) ? 1u : 0u);
        tc_commit(&empty[s]);                      // the stage is free once these MMAs have read it
      }
      if (ok) tc_commit(acc_full);                 // accumulator complete
    }
  } else {
    // ---- epilogue: TMEM -> registers -> global, transposed --------------------------------------------------
    const int quad = warp & 3;                     // the TMEM lane quadrant this warp may read
    const int n = n0 + quad * 32 + lane;
    bool ok = kb_hi > kb_lo;
    if (ok && !mbar_wait(acc_full, 0)) { set_status(A.status, ST_TIMEOUT); ok = false; }
    tc_fence_after();
    if (ok) {
      for (int c0 = 0; c0 < T; c0 += 16) {
        uint32_t r[16];
        tc_ld_32x16(tmem + (static_cast<uint32_t>(quad * 32) << 16) + c0, r);
        tc_wait_ld();
        if (n < A.N) {
          if (A.out_fp32) {
            float *out = reinterpret_cast<float *>(A.out) + split * A.split_stride;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int m = m0 + c0 + j;
              if (m < A.M) out[static_cast<size_t>(m) * A.ldo + n] = __uint_as_float(r[j]);
            }
          } else {
            __nv_bfloat16 *out = reinterpret_cast<__nv_bfloat16 *>(A.out);
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int m = m0 + c0 + j;
              if (m < A.M) out[static_cast<size_t>(m) * A.ldo + n] = __float2bfloat16(__uint_as_float(r[j]));
            }
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tc_dealloc(tmem, ncols);
}

cudaError_t launch_gemm_tc(const GemmArgs &A, cudaStream_t stream) {
  const int T = A.block_t;
  if (T < 16 || T > 256 || (T & 15) || (A.K % GT_BK) || A.nsplit < 1 || A.nsplit > A.K / GT_BK) return cudaErrorInvalidValue;
  if (!A.out_fp32 && A.nsplit != 1) return cudaErrorInvalidValue;
  const size_t smem = gt_smem(T);
  static size_t configured = 0;
  if (smem > configured) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    configured = smem;
  }
  dim3 grid((A.N + GT_BN - 1) / GT_BN, (A.M + T - 1) / T, A.nsplit);
  gemm_tc_kernel<<<grid, GT_THREADS, smem, stream>>>(A, gt_stages(T));
  return cudaGetLastError();
}

// ---- plain mma.sync GEMM ----------------------------------------------------------------------------------------------
// CTA = 4 warps; warp w computes rows [m0 + 16 w, +16) x columns [n0, n0 + 64) with fragments loaded
// straight from global memory (both operands are K-major, so fragments are plain 32-bit loads).
__global__ void __launch_bounds__(128) gemm_simple_kernel(const GemmArgs A) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, t4 = lane & 3, r8 = lane >> 2;
  const int m0 = blockIdx.y * 64 + warp * 16, n0 = blockIdx.x * 64, split = blockIdx.z;
  const int k_lo = static_cast<int>(static_cast<long long>(split) * (A.K / 16) / A.nsplit) * 16;
  const int k_hi = static_cast<int>(static_cast<long long>(split + 1) * (A.K / 16) / A.nsplit) * 16;
  float acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
  const int ra = m0 + r8, rb = m0 + r8 + 8;
  for (int k = k_lo; k < k_hi; k += 16) {
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
#pragma unroll
  for (int nt = 0; nt < 8; ++nt)
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int m = m0 + r8 + h * 8, n = n0 + nt * 8 + 2 * t4 + e;
        if (m < A.M && n < A.N) {
          const float v = acc[nt][h * 2 + e];
          if (A.out_fp32) reinterpret_cast<float *>(A.out)[split * A.split_stride + static_cast<size_t>(m) * A.ldo + n] = v;
          else reinterpret_cast<__nv_bfloat16 *>(A.out)[static_cast<size_t>(m) * A.ldo + n] = __float2bfloat16(v);
        }
      }
}

cudaError_t launch_gemm_simple(const GemmArgs &A, cudaStream_t stream) {
  if ((A.K % 16) || A.nsplit < 1 || A.nsplit > A.K / 16) return cudaErrorInvalidValue;
  if (!A.out_fp32 && A.nsplit != 1) return cudaErrorInvalidValue;
  dim3 grid((A.N + 63) / 64, (A.M + 63) / 64, A.nsplit);
  gemm_simple_kernel<<<grid, 128, 0, stream>>>(A);
  return cudaGetLastError();
}

}  // namespace gm
