// gm_attention_noalloc: the paged attention kernel for callers that must not allocate.
//
// Who needs this.  Some hosts of this library may not call cudaMalloc at the moment they need
// attention: a latency-critical serving thread on which a device allocation (which can
// synchronise the whole device) is forbidden, a plug-in that is handed a stream but owns no
// memory pool, a process whose device memory has been fully handed out to another component's
// allocator.  gm_attention needs a gm_ctx, and gm_init allocates.  This entry point needs no
// context and allocates nothing: its scratch (the per-segment partial outputs, the page prefix and
// a status word) lives in one file-scope device array that every GPU loading the library holds
// until the process exits.
//
// The array's name is only a host-side stand-in in host code, never a device address; its address
// is obtained once per device with cudaGetSymbolAddress (with that device current) and then passed
// to the kernels like any other pointer.
#include <cmath>
#include <cstring>
#include <mutex>

#include <cudaTypedefs.h>

#include "../../include/gm.h"
#include "common.cuh"
#include "kernels.h"

namespace {

using namespace gm;

// Maximum scratch: 16 MiB per GPU.  Layout: [status word | page prefix (GM_NOALLOC_MAX_BATCH+1 ints)] in the
// first 4 KiB, then the (max, sum) pairs and the partial outputs of the attention segments.
constexpr size_t NA_BYTES = GM_NOALLOC_SCRATCH_BYTES;
constexpr size_t NA_HEADER = 4096;
static __device__ __align__(256) unsigned char g_noalloc_scratch[NA_BYTES];

constexpr int NA_MAX_DEVICES = 64;
std::mutex g_mu;
unsigned char *g_dev_ptr[NA_MAX_DEVICES] = {};      // device address of the array, per device ordinal
int g_sm_count[NA_MAX_DEVICES] = {};
PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;

// First call on a device: resolve the array's device address (and the SM count, and the driver's
// tensor-map encoder).  Nothing here allocates device memory.
int setup_device(int dev) {
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_dev_ptr[dev] != nullptr) return GM_OK;
  if (g_encode == nullptr) {
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn)
      return GM_ERR_CUDA;
    g_encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
  }
  int major = 0, sms = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return GM_ERR_CUDA;
  if (major != 10) return GM_ERR_NO_EXTENSION;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return GM_ERR_CUDA;
  unsigned char *ptr = nullptr;
  cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_noalloc_scratch);
  if (e != cudaSuccess || ptr == nullptr) return GM_ERR_CUDA;
  g_sm_count[dev] = sms;
  g_dev_ptr[dev] = ptr;
  return GM_OK;
}

}  // namespace

extern "C" int gm_attention_noalloc(int n_q_heads, int n_kv_heads, int head_dim, int max_pages_per_seq, const void *q,
                                    const void *kv_pool, int pool_layers, int num_pages, int layer,
                                    const int32_t *page_table, const int32_t *q_count, const int32_t *q_base,
                                    int batch, int q_stride, void *out, void *cuda_stream) {
  if (!q || !kv_pool || !page_table || !q_count || !q_base || !out) return GM_ERR_INVALID_ARG;
  if (n_q_heads < 1 || n_kv_heads < 1 || batch < 1 || q_stride < 1 || pool_layers < 1 || layer < 0 ||
      layer >= pool_layers || num_pages < 1 || max_pages_per_seq < 1)
    return GM_ERR_INVALID_ARG;
  if ((head_dim != 64 && head_dim != 128) || (n_q_heads % n_kv_heads) || (n_kv_heads > 8 && n_kv_heads % 8))
    return GM_ERR_UNSUPPORTED;
  const int group = n_q_heads / n_kv_heads;
  if (q_stride * group > 32) return GM_ERR_UNSUPPORTED;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return GM_ERR_CUDA;
  if (dev < 0 || dev >= NA_MAX_DEVICES) return GM_ERR_UNSUPPORTED;
  int rc = setup_device(dev);
  if (rc != GM_OK) return rc;

  // does the request fit the static scratch?
  const int qrows = (q_stride * group + 15) & ~15;
  const int n_ctas = g_sm_count[dev];
  const size_t slots = static_cast<size_t>(n_ctas) + batch;
  const size_t ml_bytes = ((slots * n_kv_heads * qrows * 2 * sizeof(float)) + 255) & ~size_t(255);
  const size_t o_bytes = slots * n_kv_heads * qrows * head_dim * sizeof(float);
  if (batch > GM_NOALLOC_MAX_BATCH || NA_HEADER + ml_bytes + o_bytes > NA_BYTES) return GM_ERR_SCRATCH_LIMIT;

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  unsigned char *base = g_dev_ptr[dev];
  uint32_t *status = reinterpret_cast<uint32_t *>(base);
  int32_t *page_start = reinterpret_cast<int32_t *>(base + 256);
  float *part_ml = reinterpret_cast<float *>(base + NA_HEADER);
  float *part_o = reinterpret_cast<float *>(base + NA_HEADER + ml_bytes);

  // The array keeps the previous call's contents.  Only the status word must start at zero: the page prefix
  // is rewritten in full, and the merge reads exactly the partial slots this call's attention kernel writes.
  if (cudaMemsetAsync(status, 0, sizeof(uint32_t), stream) != cudaSuccess) return GM_ERR_CUDA;

  // tensor map of the pool: rows of head_dim elements, box 64 x (heads per CTA * 16), 128-byte swizzle
  AttnArgs T;
  std::memset(&T, 0, sizeof(T));
  {
    const int hpc = n_kv_heads < 8 ? n_kv_heads : 8;
    const unsigned long long rows = static_cast<unsigned long long>(pool_layers) * 2 * num_pages * n_kv_heads * 16;
    cuuint64_t dims[2] = {static_cast<cuuint64_t>(head_dim), rows};
    cuuint64_t strides[1] = {static_cast<cuuint64_t>(head_dim) * 2};
    cuuint32_t box[2] = {64, static_cast<cuuint32_t>(hpc * 16)};
    cuuint32_t estr[2] = {1, 1};
    if (g_encode(&T.kv_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(kv_pool), dims, strides, box, estr,
                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return GM_ERR_CUDA;
  }
  if (launch_page_prefix(q_count, q_base, batch, max_pages_per_seq, q_stride, page_start, status, stream) != cudaSuccess)
    return GM_ERR_CUDA;
  T.qbuf = static_cast<const __nv_bfloat16 *>(q); T.qn = q_count; T.qbase = q_base; T.page_start = page_start;
  T.page_table = page_table; T.batch = batch; T.n_kv = n_kv_heads; T.group = group; T.hd = head_dim; T.qrows = qrows;
  T.layer = layer; T.num_pages = num_pages; T.max_pages_per_seq = max_pages_per_seq; T.n_ctas = n_ctas;
  T.scale_log2e = static_cast<float>(1.4426950408889634 / std::sqrt(static_cast<double>(head_dim)));
  T.part_o = part_o; T.part_ml = part_ml; T.status = status;
  if (launch_attention(T, stream) != cudaSuccess) return GM_ERR_CUDA;
  AttnCombineArgs Cb;
  Cb.part_o = part_o; Cb.part_ml = part_ml; Cb.qn = q_count; Cb.page_start = page_start; Cb.batch = batch;
  Cb.n_kv = n_kv_heads; Cb.group = group; Cb.hd = head_dim; Cb.qrows = qrows; Cb.QT = q_stride; Cb.n_ctas = n_ctas;
  Cb.out = static_cast<__nv_bfloat16 *>(out);
  if (launch_attention_combine(Cb, stream) != cudaSuccess) return GM_ERR_CUDA;
  return GM_OK;
}
