// Paged decode attention for callers that cannot hand the library any scratch memory.
//
// Some hosts of this library have no way to allocate device memory at the moment they need a decode
// step: a serving engine that gave its whole HBM budget to the weight and KV-block pools at start-up,
// a plugin that runs inside someone else's memory pool without an allocator handle, or the activation
// path right after a handover, where a cudaMalloc would synchronise the device and can fail outright
// because the pool already owns the memory.  For them the split-KV partial results live in a fixed
// array that is part of the loaded module instead of a caller-supplied buffer.
#include <mutex>

#include "common.cuh"

namespace {

// 4 MiB of split-KV partials (m, l, acc[head_dim] per query head and key split).  Every GPU that loads
// the library holds this array until the process exits.
constexpr long long kNoAllocScratchBytes = KV_NOALLOC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void *g_scratch_addr[kMaxDevices] = {};

// In host code the array's name only stands for the symbol; the address a kernel can use has to be
// asked for, once per device, while that device is current.
int scratch_for_current_device(void **out) {
  int device = 0;
  KV_CUDA(cudaGetDevice(&device));
  if (device < 0 || device >= kMaxDevices) return KV_ERR_ARG;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_addr[device] == nullptr) {
    void *p = nullptr;
    KV_CUDA(cudaGetSymbolAddress(&p, g_noalloc_scratch));
    if (p == nullptr) return KV_ERR_CUDA;
    g_scratch_addr[device] = p;
  }
  *out = g_scratch_addr[device];
  return KV_OK;
}

}  // namespace

extern "C" int32_t kv_op_paged_attention_noalloc(const float *q_dev, int32_t n_q_heads, const kv_cache_desc *cache,
                                                 int32_t layer, const int32_t *block_table_dev, int32_t n_ctx,
                                                 float *out_dev, void *stream) {
  using namespace kvr;
  if (q_dev == nullptr || block_table_dev == nullptr || out_dev == nullptr || n_ctx <= 0 || n_q_heads <= 0)
    return KV_ERR_ARG;
  if (((uintptr_t)q_dev & 7) || ((uintptr_t)out_dev & 3)) return KV_ERR_ARG;
  // the same descriptor checks as kv_op_paged_attention (alignment of the base and of every stride included:
  // the kernel reads pages with 16-byte copies)
  int rc = check_cache_desc(cache);
  if (rc != KV_OK) return rc;
  if (layer < 0 || layer >= cache->n_layers || n_q_heads % cache->n_kv_heads != 0 ||
      (cache->head_dim != 64 && cache->head_dim != 128))
    return KV_ERR_SHAPE;
  // the fixed array bounds the context length: reject what does not fit instead of spilling past it
  if (paged_attention_scratch_bytes(n_q_heads, cache->head_dim, n_ctx) > kNoAllocScratchBytes) return KV_ERR_WORKSPACE;
  void *scratch = nullptr;
  rc = scratch_for_current_device(&scratch);
  if (rc != KV_OK) return rc;
  // Every partial record the merge pass reads is written by the split pass of the same call, so nothing
  // left in the array by an earlier call is ever consumed and nothing needs clearing.
  return paged_attention(q_dev, n_q_heads, make_view(cache), layer, block_table_dev, n_ctx, scratch, out_dev,
                         (cudaStream_t)stream);
}
