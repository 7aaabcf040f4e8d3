// Multi-query paged decode attention with grouped-query heads over ragged KV lengths.
//
// Work partition.  The pages every sequence attends are laid end to end (page_start is their
// prefix sum) and cut into gridDim.x equal contiguous ranges, one per CTA, so every SM streams the
// same number of bytes whatever the length mix.  A range may cover the tail of one sequence and
// the head of the next: each (CTA, sequence) piece is a "segment" that yields an un-normalised
// partial (max, sum, output); segment id = cta + sequence index, which is unique and consecutive
// within a sequence.  A second kernel merges the segments of each sequence (log-sum-exp).
//
// Inside a CTA.  Warp h of the first HPC warps owns KV head h; one extra warp is the producer.
// The producer walks the range page by page, looks the physical page up in the page table and
// issues TMA tensor copies (128-byte swizzle) of that page's keys and values for all HPC heads
// - 16 KB boxes, contiguous in the pool - into a ring of shared-memory stages guarded by
// full/empty mbarriers.  A compute warp holds its (K+1) x group <= 16*MT query rows as mma.sync
// A-fragments in registers, forms S = Q K^T for the page's 16 keys with m16n8k16 bf16 MMAs fed by
// ldmatrix, runs the online softmax in registers (quad shuffles for the row statistics) and
// accumulates O += P V with V fetched by ldmatrix.trans.  The 16-row M extent is why this is the
// warp-level MMA and not tcgen05 (whose minimum M is 64).
#include <cstdlib>

#include "common.cuh"
#include "kernels.h"

namespace gm {

constexpr int ATT_MAX_HPC = 8;        // KV heads (= compute warps) per CTA
constexpr int ATT_SMEM_BUDGET = 200 * 1024;

template <int HD> struct AttCfg {
  static constexpr int NSUB = HD / 64;                                   // 128-byte sub-tiles per row
  static __host__ __device__ constexpr int tile_bytes(int hpc) { return hpc * 16 * 128; }       // one sub-tile
  static __host__ __device__ constexpr int stage_bytes(int hpc) { return 2 * NSUB * tile_bytes(hpc); }
};

static int att_hpc(int n_kv) { return n_kv < ATT_MAX_HPC ? n_kv : ATT_MAX_HPC; }
// With two 16-row query tiles the Q fragments do not fit in registers next to the output accumulators:
// they are kept in shared memory (32 rows x head_dim per KV head) and fetched with ldmatrix per page.
static int att_q_bytes(int n_kv, int hd, int mt) { return mt >= 2 ? att_hpc(n_kv) * 32 * hd * 2 : 0; }
static int att_stages(int n_kv, int hd, int mt) {
  const int sb = 2 * (hd / 64) * att_hpc(n_kv) * 16 * 128;
  int s = (ATT_SMEM_BUDGET - att_q_bytes(n_kv, hd, mt)) / sb;
  return s > 8 ? 8 : (s < 2 ? 2 : s);
}
size_t attention_smem_bytes(int n_kv, int hd, int mt) {
  return static_cast<size_t>(att_stages(n_kv, hd, mt)) * 2 * (hd / 64) * att_hpc(n_kv) * 16 * 128 + 1024 + 1024 +
         att_q_bytes(n_kv, hd, mt);
}
int attention_max_ctas(int n_kv, int hd) {
  (void)n_kv; (void)hd;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  return sms;
}

// CTA that owns global page x when P pages are cut into G ranges [i*P/G, (i+1)*P/G).
__device__ __forceinline__ int cta_of_page(long long x, long long P, long long G) {
  return static_cast<int>(((x + 1) * G - 1) / P);
}

// RT > 1 (with MT = 1): RT warps per KV head, each owning one 16-row query tile (rows rt*16 ..) and consuming every page
// of its head - more warps to hide latency where two tiles in one warp are bound by instruction issue.  17 warps are
// allocated as 20 (granularity 4), which leaves 96 registers per thread: a few spills; 112 or 120 do not launch.
template <int HD, int MT, int RT = 1>
__global__ void __launch_bounds__((ATT_MAX_HPC * RT + 1) * 32, 1)
attention_kernel(const __grid_constant__ AttnArgs A, const int hpc, const int nstages) {
  using C = AttCfg<HD>;
  constexpr int NSUB = C::NSUB;
  constexpr int KSTEPS = HD / 16;
  constexpr int NT = HD / 8;                    // 8-wide output column tiles

  extern __shared__ unsigned char att_smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(att_smem_raw) + 1023) & ~uintptr_t(1023));
  const int tile_b = C::tile_bytes(hpc);
  const int stage_b = C::stage_bytes(hpc);
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + static_cast<size_t>(nstages) * stage_b);
  uint64_t *empty = full + 8;
  // Q staging area (two-tile variant only), 1024-byte aligned after the barriers
  unsigned char *qsm = smem + ((static_cast<size_t>(nstages) * stage_b + 128 + 1023) & ~size_t(1023));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int B = A.batch;
  // barrier set-up touches shared memory only: it runs before the wait for the previous kernel
  if (threadIdx.x == 0) {
    for (int s = 0; s < nstages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], hpc * RT); }
    mbar_fence_init();
  }
  __syncthreads();
  pdl_prologue();
  const long long P = A.page_start[B];
  // never more ranges than pages: every active CTA then owns at least one page, so the CTAs that hold
  // pieces of one sequence are consecutive and so are its segment ids
  const long long G = P < static_cast<long long>(gridDim.x) ? P : static_cast<long long>(gridDim.x);
  if (static_cast<long long>(blockIdx.x) >= G) return;
  const int lo = static_cast<int>(blockIdx.x * P / G), hi = static_cast<int>((blockIdx.x + 1) * P / G);
  const int hg = blockIdx.y;                    // head group (n_kv > 8)
  if (lo >= hi) return;

  // first sequence of the range: largest b with page_start[b] <= lo
  int b0 = 0;
  {
    int l = 0, r = B - 1;
    while (l < r) { const int mid = (l + r + 1) >> 1; if (A.page_start[mid] <= lo) l = mid; else r = mid - 1; }
    b0 = l;
  }

  if (warp == hpc * RT) {
    // ---- producer ------------------------------------------------------------------------------------------
    if (lane == 0) {
      tma_prefetch_desc(&A.kv_map);
      int b = b0;
      const long long rows_per_page = static_cast<long long>(A.n_kv) * 16;
      for (int p = lo, it = 0; p < hi; ++p, ++it) {
        while (p >= A.page_start[b + 1]) ++b;
        int page = A.page_table[static_cast<size_t>(b) * A.max_pages_per_seq + (p - A.page_start[b])];
        if (page < 0 || page >= A.num_pages) { set_status(A.status, ST_BAD_PAGE); page = 0; }
        const int s = it % nstages;
        if (!mbar_wait(&empty[s], ((it / nstages) & 1) ^ 1)) { set_status(A.status, ST_TIMEOUT); break; }
        mbar_expect_tx(&full[s], stage_b);
        unsigned char *dst = smem + static_cast<size_t>(s) * stage_b;
        const long long row_k = ((static_cast<long long>(A.layer) * 2 + 0) * A.num_pages + page) * rows_per_page + hg * hpc * 16;
        const long long row_v = ((static_cast<long long>(A.layer) * 2 + 1) * A.num_pages + page) * rows_per_page + hg * hpc * 16;
#pragma unroll
        for (int sub = 0; sub < NSUB; ++sub) {
          tma_load_2d(dst + sub * tile_b, &A.kv_map, sub * 64, static_cast<int>(row_k), &full[s]);
          tma_load_2d(dst + (NSUB + sub) * tile_b, &A.kv_map, sub * 64, static_cast<int>(row_v), &full[s]);
        }
      }
    }
    return;
  }
  if (warp > hpc * RT) return;

  // ---- compute warp: KV head = hg*hpc + warp -------------------------------------------------------------------
  const int hw = warp % hpc, rt = warp / hpc;     // head within the CTA, row tile
  const int head = hg * hpc + hw;
  const int row0 = rt * 16;
  const int t4 = lane & 3, r8 = lane >> 2;
  const float c = A.scale_log2e;
  const uint32_t smem_base = smem_u32(smem);
  // per-lane ldmatrix offsets inside one 128-byte-row sub-tile (row index inside the warp's 16 rows)
  const int mi = lane >> 3;
  const int k_tok = (mi >> 1) * 8 + (lane & 7), k_chunk = mi & 1;        // K: non-transposed
  const int v_tok = (mi & 1) * 8 + (lane & 7), v_chunk = mi >> 1;        // V: transposed
  const uint32_t k_row_off = (hw * 16 + k_tok) * 128, v_row_off = (hw * 16 + v_tok) * 128;
  const int k_sw = k_tok & 7, v_sw = v_tok & 7;

  int it = 0;
  bool dead = false;
  for (int b = b0; b < B && !dead; ++b) {
    const int ps = A.page_start[b], pe = A.page_start[b + 1];
    if (ps >= hi) break;
    const int seg_lo = max(lo, ps), seg_hi = min(hi, pe);
    if (seg_lo >= seg_hi) continue;
    const int qn = A.qn[b], qbase = A.qbase[b];

    // query fragments: in registers for one 16-row tile; staged in shared memory (128-byte rows, XOR swizzle)
    // for two tiles and fetched per page
    constexpr bool QSM = MT > 1 || RT > 1;        // Q staged in shared memory (register pressure)
    constexpr int QROWS = MT * 16;                // rows this warp stages
    constexpr int QREG = QSM ? 1 : KSTEPS;
    uint32_t qf[MT][QREG][4];
    const __nv_bfloat16 *qp = A.qbuf + (static_cast<size_t>(b) * A.n_kv + head) * A.qrows * HD;
    const uint32_t q_smem = smem_u32(qsm) + warp * (QROWS * HD * 2);
    if constexpr (!QSM) {
#pragma unroll
      for (int ks = 0; ks < KSTEPS; ++ks) {
        const __nv_bfloat16 *r0 = qp + (row0 + r8) * HD + ks * 16 + 2 * t4;
        qf[0][ks][0] = *reinterpret_cast<const uint32_t *>(r0);
        qf[0][ks][1] = *reinterpret_cast<const uint32_t *>(r0 + 8 * HD);
        qf[0][ks][2] = *reinterpret_cast<const uint32_t *>(r0 + 8);
        qf[0][ks][3] = *reinterpret_cast<const uint32_t *>(r0 + 8 * HD + 8);
      }
    } else {
      __syncwarp();                               // the previous segment's fragment reads are done
      constexpr int CPR = HD / 8;                 // 16-byte chunks per row
      for (int idx = lane; idx < QROWS * CPR; idx += 32) {
        const int row = idx / CPR, ch = idx % CPR;
        const uint4 v = *reinterpret_cast<const uint4 *>(qp + (row0 + row) * HD + ch * 8);
        unsigned char *dst = qsm + warp * (QROWS * HD * 2) + (ch >> 3) * (QROWS * 128) + row * 128 + (((ch & 7) ^ (row & 7)) << 4);
        *reinterpret_cast<uint4 *>(dst) = v;
      }
      __syncwarp();
    }
    const int q_row = (lane & 7) + ((lane >> 3) & 1) * 8, q_chunk = lane >> 4;   // ldmatrix lane address (A fragment)
    float o[MT][NT][4];
    float mrow[MT][2], lrow[MT][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      mrow[mt][0] = mrow[mt][1] = -INFINITY;
      lrow[mt][0] = lrow[mt][1] = 0.f;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) o[mt][nt][0] = o[mt][nt][1] = o[mt][nt][2] = o[mt][nt][3] = 0.f;
    }

    for (int p = seg_lo; p < seg_hi; ++p, ++it) {
      const int s = it % nstages;
      if (!mbar_wait(&full[s], (it / nstages) & 1)) { set_status(A.status, ST_TIMEOUT); dead = true; break; }
      const uint32_t kbase = smem_base + s * stage_b, vbase = kbase + NSUB * tile_b;

      float sc[MT][2][4];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int n = 0; n < 2; ++n) sc[mt][n][0] = sc[mt][n][1] = sc[mt][n][2] = sc[mt][n][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KSTEPS; ++ks) {
        uint32_t kf[4];
        const int chunk = (ks & 3) * 2 + k_chunk;
        ldmatrix_x4(kf, kbase + (ks >> 2) * tile_b + k_row_off + ((chunk ^ k_sw) << 4));
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          if constexpr (!QSM) {
            mma_16816(sc[mt][0], qf[mt][ks], kf[0], kf[1]);
            mma_16816(sc[mt][1], qf[mt][ks], kf[2], kf[3]);
          } else {
            const int row = mt * 16 + q_row;
            ldmatrix_x4(qf[mt][0], q_smem + (ks >> 2) * (QROWS * 128) + row * 128 + ((((ks & 3) * 2 + q_chunk) ^ (row & 7)) << 4));
            mma_16816(sc[mt][0], qf[mt][0], kf[0], kf[1]);
            mma_16816(sc[mt][1], qf[mt][0], kf[2], kf[3]);
          }
        }
      }

      // causal / length mask: key position kp is visible to row r iff kp <= qbase + r/group and r/group < qn
      const int kp0 = (p - ps) * 16;
      const bool need_mask = kp0 + 15 > qbase;
      uint32_t pa[MT][4];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        if (need_mask) {
#pragma unroll
          for (int hrow = 0; hrow < 2; ++hrow) {
            const int j = (row0 + mt * 16 + r8 + hrow * 8) / A.group;
            const int lim = j < qn ? qbase + j : -1;
#pragma unroll
            for (int n = 0; n < 2; ++n)
#pragma unroll
              for (int e = 0; e < 2; ++e)
                if (kp0 + n * 8 + 2 * t4 + e > lim) sc[mt][n][hrow * 2 + e] = -INFINITY;
          }
        }
        float alpha[2];
#pragma unroll
        for (int hrow = 0; hrow < 2; ++hrow) {
          float mx = fmaxf(fmaxf(sc[mt][0][hrow * 2], sc[mt][0][hrow * 2 + 1]),
                           fmaxf(sc[mt][1][hrow * 2], sc[mt][1][hrow * 2 + 1]));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
          const float m_new = fmaxf(mrow[mt][hrow], mx);
          const float m_use = m_new == -INFINITY ? 0.f : m_new;
          alpha[hrow] = exp2f((mrow[mt][hrow] - m_use) * c);       // exp2(-inf) = 0 on the first page
          mrow[mt][hrow] = m_new;
          const float mc = m_use * c;
          float rs = 0.f;
#pragma unroll
          for (int n = 0; n < 2; ++n)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const float pv = exp2f(fmaf(sc[mt][n][hrow * 2 + e], c, -mc));
              sc[mt][n][hrow * 2 + e] = pv;
              rs += pv;
            }
          lrow[mt][hrow] = lrow[mt][hrow] * alpha[hrow] + rs;
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          o[mt][nt][0] *= alpha[0]; o[mt][nt][1] *= alpha[0];
          o[mt][nt][2] *= alpha[1]; o[mt][nt][3] *= alpha[1];
        }
        pa[mt][0] = pack_bf16(sc[mt][0][0], sc[mt][0][1]);
        pa[mt][1] = pack_bf16(sc[mt][0][2], sc[mt][0][3]);
        pa[mt][2] = pack_bf16(sc[mt][1][0], sc[mt][1][1]);
        pa[mt][3] = pack_bf16(sc[mt][1][2], sc[mt][1][3]);
      }

      // O += P V
#pragma unroll
      for (int n2 = 0; n2 < NT / 2; ++n2) {
        uint32_t vf[4];
        const int chunk = (n2 & 3) * 2 + v_chunk;
        ldmatrix_x4_trans(vf, vbase + (n2 >> 2) * tile_b + v_row_off + ((chunk ^ v_sw) << 4));
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          mma_16816(o[mt][2 * n2], pa[mt], vf[0], vf[1]);
          mma_16816(o[mt][2 * n2 + 1], pa[mt], vf[2], vf[3]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);
    }
    if (dead) break;

    // ---- write this segment's partial ----------------------------------------------------------------------
    const size_t slot = static_cast<size_t>(blockIdx.x) + b;
    float *po = A.part_o + ((slot * A.n_kv + head) * A.qrows) * HD;
    float *pml = A.part_ml + ((slot * A.n_kv + head) * A.qrows) * 2;
    const int rows_valid = qn * A.group;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int hrow = 0; hrow < 2; ++hrow) {
        float l = lrow[mt][hrow];
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        const int row = row0 + mt * 16 + r8 + hrow * 8;
        if (row < rows_valid) {
          if (t4 == 0) {
            pml[row * 2 + 0] = mrow[mt][hrow] == -INFINITY ? -INFINITY : mrow[mt][hrow] * c;
            pml[row * 2 + 1] = l;
          }
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
            *reinterpret_cast<float2 *>(po + static_cast<size_t>(row) * HD + nt * 8 + 2 * t4) =
                make_float2(o[mt][nt][hrow * 2], o[mt][nt][hrow * 2 + 1]);
        }
      }
  }
}


// ---- transposed formulation for 17..24 query rows -----------------------------------------------------------------------
// With two 16-row M tiles (rows padded to 32) the kernel above is bound by the warp-level MMA rate, not by HBM.  Here the
// roles are swapped: the page's 16 keys are the M extent and the query rows the N extent (tiles of 8, so 24 rows are
// exactly three tiles):  S^T = K Q^T  with K as the A operand (same ldmatrix loads, registers permuted) and Q^T as B
// fragments held in registers;  O^T += V^T P^T  with V^T as the A operand (same ldmatrix.trans loads) and P^T obtained
// from the S^T accumulators by an 8x8 register transpose (movmatrix).  48 MMAs per page instead of 64.
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

template <int HD, int NR>
__global__ void __launch_bounds__((ATT_MAX_HPC + 1) * 32, 1)
attention_t_kernel(const __grid_constant__ AttnArgs A, const int hpc, const int nstages) {
  using C = AttCfg<HD>;
  constexpr int NSUB = C::NSUB;
  constexpr int KSTEPS = HD / 16;
  constexpr int MTILES = HD / 16;               // 16-wide tiles of the head dimension (M extent of O^T)

  extern __shared__ unsigned char att_smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(att_smem_raw) + 1023) & ~uintptr_t(1023));
  const int tile_b = C::tile_bytes(hpc);
  const int stage_b = C::stage_bytes(hpc);
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + static_cast<size_t>(nstages) * stage_b);
  uint64_t *empty = full + 8;
  unsigned char *qsm = smem + ((static_cast<size_t>(nstages) * stage_b + 128 + 1023) & ~size_t(1023));   // Q staging

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int B = A.batch;
  if (threadIdx.x == 0) {                       // shared memory only: before the wait for the previous kernel
    for (int s = 0; s < nstages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], hpc); }
    mbar_fence_init();
  }
  __syncthreads();
  pdl_prologue();
  const long long P = A.page_start[B];
  const long long G = P < static_cast<long long>(gridDim.x) ? P : static_cast<long long>(gridDim.x);
  if (static_cast<long long>(blockIdx.x) >= G) return;
  const int lo = static_cast<int>(blockIdx.x * P / G), hi = static_cast<int>((blockIdx.x + 1) * P / G);
  const int hg = blockIdx.y;
  if (lo >= hi) return;

  int b0 = 0;
  {
    int l = 0, r = B - 1;
    while (l < r) { const int mid = (l + r + 1) >> 1; if (A.page_start[mid] <= lo) l = mid; else r = mid - 1; }
    b0 = l;
  }

  if (warp == hpc) {
    // ---- producer: identical to the kernel above ---------------------------------------------------------------
    if (lane == 0) {
      tma_prefetch_desc(&A.kv_map);
      int b = b0;
      const long long rows_per_page = static_cast<long long>(A.n_kv) * 16;
      for (int p = lo, it = 0; p < hi; ++p, ++it) {
        while (p >= A.page_start[b + 1]) ++b;
        int page = A.page_table[static_cast<size_t>(b) * A.max_pages_per_seq + (p - A.page_start[b])];
        if (page < 0 || page >= A.num_pages) { set_status(A.status, ST_BAD_PAGE); page = 0; }
        const int s = it % nstages;
        if (!mbar_wait(&empty[s], ((it / nstages) & 1) ^ 1)) { set_status(A.status, ST_TIMEOUT); break; }
        mbar_expect_tx(&full[s], stage_b);
        unsigned char *dst = smem + static_cast<size_t>(s) * stage_b;
        const long long row_k = ((static_cast<long long>(A.layer) * 2 + 0) * A.num_pages + page) * rows_per_page + hg * hpc * 16;
        const long long row_v = ((static_cast<long long>(A.layer) * 2 + 1) * A.num_pages + page) * rows_per_page + hg * hpc * 16;
#pragma unroll
        for (int sub = 0; sub < NSUB; ++sub) {
          tma_load_2d(dst + sub * tile_b, &A.kv_map, sub * 64, static_cast<int>(row_k), &full[s]);
          tma_load_2d(dst + (NSUB + sub) * tile_b, &A.kv_map, sub * 64, static_cast<int>(row_v), &full[s]);
        }
      }
    }
    return;
  }
  if (warp > hpc) return;

  const int head = hg * hpc + warp;
  const int t4 = lane & 3, r8 = lane >> 2;
  const float c = A.scale_log2e;
  const uint32_t smem_base = smem_u32(smem);
  const int mi = lane >> 3;
  const int k_tok = (mi >> 1) * 8 + (lane & 7), k_chunk = mi & 1;
  const int v_tok = (mi & 1) * 8 + (lane & 7), v_chunk = mi >> 1;
  const uint32_t k_row_off = (warp * 16 + k_tok) * 128, v_row_off = (warp * 16 + v_tok) * 128;
  const int k_sw = k_tok & 7, v_sw = v_tok & 7;

  int it = 0;
  bool dead = false;
  for (int b = b0; b < B && !dead; ++b) {
    const int ps = A.page_start[b], pe = A.page_start[b + 1];
    if (ps >= hi) break;
    const int seg_lo = max(lo, ps), seg_hi = min(hi, pe);
    if (seg_lo >= seg_hi) continue;
    const int qn = A.qn[b], qbase = A.qbase[b];

    // Q rows staged in shared memory (128-byte rows, XOR swizzle), fetched per page as B fragments with ldmatrix: one
    // x4 load gives (k lo, k hi) of two consecutive K steps for the 8 rows of a tile.  (In registers they would be 48
    // more per thread, and this kernel's 9 warps are limited to 168.)
    const __nv_bfloat16 *qp = A.qbuf + (static_cast<size_t>(b) * A.n_kv + head) * A.qrows * HD;
    unsigned char *q_stage = qsm + warp * (NR * 8 * HD * 2);
    const uint32_t q_smem = smem_u32(q_stage);
    __syncwarp();                                 // the previous segment's fragment reads are done
    {
      constexpr int CPR = HD / 8;                 // 16-byte chunks per row
      for (int idx = lane; idx < NR * 8 * CPR; idx += 32) {
        const int row = idx / CPR, ch = idx % CPR;
        const uint4 v = *reinterpret_cast<const uint4 *>(qp + row * HD + ch * 8);
        *reinterpret_cast<uint4 *>(q_stage + (ch >> 3) * (NR * 8 * 128) + row * 128 + (((ch & 7) ^ (row & 7)) << 4)) = v;
      }
    }
    __syncwarp();
    const int qb_row = lane & 7, qb_chunk = lane >> 3;   // ldmatrix lane address: 8 rows x (4 chunks = 2 K steps)
    float ot[MTILES][NR][4];
    float mrow[NR][2], lrow[NR][2];
#pragma unroll
    for (int nr = 0; nr < NR; ++nr) {
      mrow[nr][0] = mrow[nr][1] = -INFINITY;
      lrow[nr][0] = lrow[nr][1] = 0.f;
#pragma unroll
      for (int mt = 0; mt < MTILES; ++mt) ot[mt][nr][0] = ot[mt][nr][1] = ot[mt][nr][2] = ot[mt][nr][3] = 0.f;
    }

    for (int p = seg_lo; p < seg_hi; ++p, ++it) {
      const int s = it % nstages;
      if (!mbar_wait(&full[s], (it / nstages) & 1)) { set_status(A.status, ST_TIMEOUT); dead = true; break; }
      const uint32_t kbase = smem_base + s * stage_b, vbase = kbase + NSUB * tile_b;

      // S^T[key][row]: accumulator e of tile nr = (key r8 + 8*(e>>1), row nr*8 + 2*t4 + (e&1))
      float st[NR][4];
#pragma unroll
      for (int nr = 0; nr < NR; ++nr) st[nr][0] = st[nr][1] = st[nr][2] = st[nr][3] = 0.f;
#pragma unroll
      for (int kp = 0; kp < KSTEPS / 2; ++kp) {
        uint32_t kf0[4], kf1[4];
        const int ks0 = 2 * kp, ks1 = 2 * kp + 1;
        ldmatrix_x4(kf0, kbase + (ks0 >> 2) * tile_b + k_row_off + (((((ks0 & 3) * 2 + k_chunk)) ^ k_sw) << 4));
        ldmatrix_x4(kf1, kbase + (ks1 >> 2) * tile_b + k_row_off + (((((ks1 & 3) * 2 + k_chunk)) ^ k_sw) << 4));
        // A operand = keys x k: (keys 0-7, k lo) (keys 8-15, k lo) (keys 0-7, k hi) (keys 8-15, k hi)
        const uint32_t a0[4] = {kf0[0], kf0[2], kf0[1], kf0[3]};
        const uint32_t a1[4] = {kf1[0], kf1[2], kf1[1], kf1[3]};
#pragma unroll
        for (int nr = 0; nr < NR; ++nr) {
          uint32_t qf[4];                               // (ks0: k lo, k hi) (ks1: k lo, k hi) of rows nr*8 .. nr*8+7
          const int row = nr * 8 + qb_row, ch = (ks0 & 3) * 2 + qb_chunk;
          ldmatrix_x4(qf, q_smem + (ks0 >> 2) * (NR * 8 * 128) + row * 128 + ((ch ^ (row & 7)) << 4));
          mma_16816(st[nr], a0, qf[0], qf[1]);
          mma_16816(st[nr], a1, qf[2], qf[3]);
        }
      }

      const int kp0 = (p - ps) * 16;
      const bool need_mask = kp0 + 15 > qbase;
      uint32_t pb[NR][2];
#pragma unroll
      for (int nr = 0; nr < NR; ++nr) {
        if (need_mask) {                                         // only the last pages of a sequence come here
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            // accumulator columns are query rows nr*8 + 2*t4 + e: the last key position the row may see
            const int j = (nr * 8 + 2 * t4 + e) / A.group;
            const int lim = j < qn ? qbase + j : -1;
            if (kp0 + r8 > lim) st[nr][e] = -INFINITY;
            if (kp0 + r8 + 8 > lim) st[nr][e + 2] = -INFINITY;
          }
        }
        float alpha[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          float mx = fmaxf(st[nr][e], st[nr][e + 2]);             // this thread's two keys of the row
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
          const float m_new = fmaxf(mrow[nr][e], mx);
          const float m_use = m_new == -INFINITY ? 0.f : m_new;
          alpha[e] = exp2f((mrow[nr][e] - m_use) * c);
          mrow[nr][e] = m_new;
          const float mc = m_use * c;
          const float p0 = exp2f(fmaf(st[nr][e], c, -mc)), p1 = exp2f(fmaf(st[nr][e + 2], c, -mc));
          st[nr][e] = p0; st[nr][e + 2] = p1;
          lrow[nr][e] = lrow[nr][e] * alpha[e] + p0 + p1;         // this thread's keys only; lanes are added at the end
        }
#pragma unroll
        for (int mt = 0; mt < MTILES; ++mt) {
          ot[mt][nr][0] *= alpha[0]; ot[mt][nr][1] *= alpha[1];
          ot[mt][nr][2] *= alpha[0]; ot[mt][nr][3] *= alpha[1];
        }
        // P^T as B fragments: transpose the two 8x8 blocks (keys 0-7 and keys 8-15) held as (key r8, rows 2*t4, 2*t4+1)
        pb[nr][0] = movmatrix_trans(pack_bf16(st[nr][0], st[nr][1]));
        pb[nr][1] = movmatrix_trans(pack_bf16(st[nr][2], st[nr][3]));
      }

      // O^T += V^T P^T
#pragma unroll
      for (int n2 = 0; n2 < MTILES; ++n2) {
        uint32_t vf[4];
        const int chunk = (n2 & 3) * 2 + v_chunk;
        ldmatrix_x4_trans(vf, vbase + (n2 >> 2) * tile_b + v_row_off + ((chunk ^ v_sw) << 4));
        const uint32_t af[4] = {vf[0], vf[2], vf[1], vf[3]};      // (hd 0-7,keys lo) (hd 8-15,keys lo) (hd 0-7,keys hi) (hd 8-15,keys hi)
#pragma unroll
        for (int nr = 0; nr < NR; ++nr) mma_16816(ot[n2][nr], af, pb[nr][0], pb[nr][1]);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);
    }
    if (dead) break;

    // ---- write this segment's partial: part_o[slot][head][row][hd], part_ml[slot][head][row][2] ----------------------
    const size_t slot = static_cast<size_t>(blockIdx.x) + b;
    float *po = A.part_o + ((slot * A.n_kv + head) * A.qrows) * HD;
    float *pml = A.part_ml + ((slot * A.n_kv + head) * A.qrows) * 2;
    const int rows_valid = qn * A.group;
#pragma unroll
    for (int nr = 0; nr < NR; ++nr)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        float l = lrow[nr][e];
        l += __shfl_xor_sync(0xffffffffu, l, 4);
        l += __shfl_xor_sync(0xffffffffu, l, 8);
        l += __shfl_xor_sync(0xffffffffu, l, 16);
        const int row = nr * 8 + 2 * t4 + e;
        if (row < rows_valid) {
          if (r8 == 0) {
            pml[row * 2 + 0] = mrow[nr][e] == -INFINITY ? -INFINITY : mrow[nr][e] * c;
            pml[row * 2 + 1] = l;
          }
#pragma unroll
          for (int mt = 0; mt < MTILES; ++mt) {
            po[static_cast<size_t>(row) * HD + mt * 16 + r8] = ot[mt][nr][e];
            po[static_cast<size_t>(row) * HD + mt * 16 + r8 + 8] = ot[mt][nr][e + 2];
          }
        }
      }
  }
}

template <int HD, int NR>
static cudaError_t launch_att_t(const AttnArgs &A, cudaStream_t stream) {
  // shared-memory layout of the two-tile variant: its 32-row Q staging area holds this kernel's 8*NR rows.  (A third
  // stage - first tile's fragments in registers, smaller staging area - was measured and is no faster: the kernel is
  // bound by instruction issue, not by the depth of the ring.)
  const int hpc = att_hpc(A.n_kv), nst = att_stages(A.n_kv, HD, 2);
  const size_t smem = attention_smem_bytes(A.n_kv, HD, 2);
  static SmemConfigured configured;
  if (cudaError_t e = ensure_dyn_smem(attention_t_kernel<HD, NR>, smem, configured); e != cudaSuccess) return e;
  dim3 grid(A.n_ctas, A.n_kv / hpc);
  return launch_k(attention_t_kernel<HD, NR>, grid, dim3((hpc + 1) * 32), smem, stream, 1, A, hpc, nst);
}

template <int HD, int MT, int RT = 1>
static cudaError_t launch_att(const AttnArgs &A, cudaStream_t stream) {
  // the variants that stage Q in shared memory share one layout: 32 rows x head_dim per KV head
  const int hpc = att_hpc(A.n_kv), nst = att_stages(A.n_kv, HD, MT * RT);
  const size_t smem = attention_smem_bytes(A.n_kv, HD, MT * RT);
  static SmemConfigured configured;
  if (cudaError_t e = ensure_dyn_smem(attention_kernel<HD, MT, RT>, smem, configured); e != cudaSuccess) return e;
  dim3 grid(A.n_ctas, A.n_kv / hpc);
  return launch_k(attention_kernel<HD, MT, RT>, grid, dim3((hpc * RT + 1) * 32), smem, stream, 1, A, hpc, nst);
}

cudaError_t launch_attention(const AttnArgs &A, cudaStream_t stream) {
  const int mt = A.qrows / 16;
  if (A.n_kv % att_hpc(A.n_kv) != 0) return cudaErrorInvalidValue;
  // 17..24 query rows: the transposed formulation (three 8-row tiles) instead of two padded 16-row tiles
  static const bool no_t = std::getenv("GM_NO_ATT_T") != nullptr;
  if (!no_t && A.hd == 128 && mt == 2 && A.rows_used > 16 && A.rows_used <= 24) return launch_att_t<128, 3>(A, stream);
  if (A.hd == 128 && mt == 1) return launch_att<128, 1>(A, stream);
  // 25..32 query rows: two warps per KV head, one 16-row tile each (GM_NO_ATT_RT2: one warp with two tiles)
  static const bool no_rt2 = std::getenv("GM_NO_ATT_RT2") != nullptr;
  if (!no_rt2 && A.hd == 128 && mt == 2) return launch_att<128, 1, 2>(A, stream);
  if (A.hd == 128 && mt == 2) return launch_att<128, 2>(A, stream);
  if (A.hd == 64 && mt == 1) return launch_att<64, 1>(A, stream);
  if (A.hd == 64 && mt == 2) return launch_att<64, 2>(A, stream);
  return cudaErrorInvalidValue;
}

// ---- merge the segments of each sequence ------------------------------------------------------------------------------
// One warp per (sequence, kv head, query row): lanes first fetch the segments' (max, sum) pairs in parallel,
// then each lane accumulates its 4 output dimensions over the segments with independent 16-byte loads.
__global__ void __launch_bounds__(128) attention_combine_kernel(const AttnCombineArgs A) {
  const int b = blockIdx.x / A.n_kv, head = blockIdx.x % A.n_kv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_prologue();
  const int qn = A.qn[b];
  const int row_first = blockIdx.y * 4 + warp;     // one query row per warp: the dependent loads of a row are paid once
  const long long P = A.page_start[A.batch];
  const long long G = P < static_cast<long long>(A.n_ctas) ? P : static_cast<long long>(A.n_ctas);   // as in the kernel above
  const int ps = A.page_start[b], pe = A.page_start[b + 1];
  if (qn <= 0 || pe <= ps) return;
  const int s_first = cta_of_page(ps, P, G) + b, s_last = cta_of_page(pe - 1, P, G) + b;
  const int nseg = s_last - s_first + 1;
  const int rows = qn * A.group, hd = A.hd;
  for (int row = row_first; row < rows; row += 4 * gridDim.y) {
    const size_t base0 = (static_cast<size_t>(s_first) * A.n_kv + head) * A.qrows + row;
    const size_t seg_stride = static_cast<size_t>(A.n_kv) * A.qrows;
    const int c4 = lane;
    // the partial outputs of the first segments are requested before the statistics are reduced: their latency
    // overlaps the two warp reductions (most sequences have at most four segments)
    constexpr int NPRE = 4;
    float4 pre[NPRE];
#pragma unroll
    for (int s = 0; s < NPRE; ++s)
      pre[s] = (s < nseg && c4 * 4 < hd) ? reinterpret_cast<const float4 *>(A.part_o + (base0 + s * seg_stride) * hd)[c4]
                                         : make_float4(0.f, 0.f, 0.f, 0.f);
    // lane s holds (max, sum) of segment s (and s + 32, ...)
    float2 ml = make_float2(-INFINITY, 0.f);
    if (lane < nseg) ml = *reinterpret_cast<const float2 *>(A.part_ml + (base0 + lane * seg_stride) * 2);
    float mt = ml.x;
    for (int s = lane + 32; s < nseg; s += 32) mt = fmaxf(mt, A.part_ml[(base0 + s * seg_stride) * 2]);
    mt = warp_max(mt);
    float l = ml.x != -INFINITY ? exp2f(ml.x - mt) * ml.y : 0.f;
    for (int s = lane + 32; s < nseg; s += 32) {
      const float ms = A.part_ml[(base0 + s * seg_stride) * 2];
      if (ms != -INFINITY) l += exp2f(ms - mt) * A.part_ml[(base0 + s * seg_stride) * 2 + 1];
    }
    l = warp_sum(l);
    const float inv = l > 0.f ? 1.f / l : 0.f;
    const float w_lane = ml.x == -INFINITY ? 0.f : exp2f(ml.x - mt);      // weight of segment `lane`
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int s = 0; s < NPRE; ++s) {
      const float w = __shfl_sync(0xffffffffu, w_lane, s);
      if (s < nseg && w != 0.f) { acc.x += w * pre[s].x; acc.y += w * pre[s].y; acc.z += w * pre[s].z; acc.w += w * pre[s].w; }
    }
    for (int s = NPRE; s < nseg; ++s) {
      float w;
      if (s < 32) {
        w = __shfl_sync(0xffffffffu, w_lane, s);
      } else {
        const float ms = A.part_ml[(base0 + s * seg_stride) * 2];
        w = ms == -INFINITY ? 0.f : exp2f(ms - mt);
      }
      if (c4 * 4 < hd && w != 0.f) {
        const float4 ov = reinterpret_cast<const float4 *>(A.part_o + (base0 + s * seg_stride) * hd)[c4];
        acc.x += w * ov.x; acc.y += w * ov.y; acc.z += w * ov.z; acc.w += w * ov.w;
      }
    }
    if (c4 * 4 < hd) {
      const int j = row / A.group, g = row % A.group;
      __nv_bfloat16 *dst = A.out + (static_cast<size_t>(b) * A.QT + j) * (A.n_kv * A.group * hd) +
                           (static_cast<size_t>(head) * A.group + g) * hd + c4 * 4;
      uint2 ov2;
      ov2.x = pack_bf16(acc.x * inv, acc.y * inv);
      ov2.y = pack_bf16(acc.z * inv, acc.w * inv);
      *reinterpret_cast<uint2 *>(dst) = ov2;
    }
  }
}
cudaError_t launch_attention_combine(const AttnCombineArgs &A, cudaStream_t stream) {
  return launch_k(attention_combine_kernel, dim3(A.batch * A.n_kv, (A.QT * A.group + 3) / 4), dim3(128), 0, stream, 1, A);
}

// ---- page prefix for a caller-given query layout (stand-alone attention calls) -------------------------------------------
// page_start[b] = pages attended by the sequences before b; a sequence whose queries do not fit its page-table row
// is reported and given no pages (its output rows are then left untouched).
__global__ void page_prefix_kernel(const int32_t *qn, const int32_t *qbase, int batch, int max_pages_per_seq,
                                   int q_stride, int32_t *page_start, uint32_t *status) {
  pdl_prologue();
  if (threadIdx.x != 0) return;
  int acc = 0;
  for (int b = 0; b < batch; ++b) {
    page_start[b] = acc;
    const int n = qn[b], base = qbase[b];
    const bool ok = n >= 1 && n <= q_stride && base >= 0 && base + n <= max_pages_per_seq * 16;
    if (!ok && n != 0) set_status(status, ST_KV_CAPACITY);
    acc += ok ? (base + n + 15) >> 4 : 0;
  }
  page_start[batch] = acc;
}
cudaError_t launch_page_prefix(const int32_t *qn, const int32_t *qbase, int batch, int max_pages_per_seq, int q_stride,
                               int32_t *page_start, uint32_t *status, cudaStream_t stream) {
  return launch_k(page_prefix_kernel, dim3(1), dim3(32), 0, stream, 1, qn, qbase, batch, max_pages_per_seq, q_stride,
                  page_start, status);
}

}  // namespace gm
