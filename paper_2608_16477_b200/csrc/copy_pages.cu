// Pack (paged cache -> contiguous wire buffer) and unpack (wire buffer -> pages): byte-exact page copies.
//
// One launch moves every page of up to kMaxIds logical blocks: block ids travel in the kernel
// parameter block, so no device-side staging of the id list and no extra copy precede the kernel.
// A page (block_size * n_kv_heads * head_dim bf16) is contiguous on both sides; each CTA streams
// 16 KiB pieces of pages with 16-byte vector loads/stores, four independent loads in flight per
// thread.  HBM-bound: 2 * page bytes of traffic per page, nothing is re-read.
#include "common.cuh"

namespace kvr {

constexpr int kMaxIds = 960;          // keeps the parameter block under 4 KiB
constexpr int kCopyThreads = 256;
constexpr int kUnroll = 4;            // 16-byte vectors per thread per piece

struct PageCopyParams {
  CacheView cache;
  char *wire;
  int n_layers;
  int n_blocks;              // blocks in this launch
  int layout;                // KV_WIRE_BLOCK_MAJOR / KV_WIRE_LAYER_MAJOR
  int total_blocks;          // blocks in the whole wire buffer (layer-major stride)
  int first_block;           // index of this launch's first block inside the wire buffer
  int vec_per_page;          // page bytes / 16
  int pieces_per_page;       // ceil(vec_per_page / (kCopyThreads * kUnroll))
  int ids[kMaxIds];
};

template <bool TO_WIRE>
__global__ void __launch_bounds__(kCopyThreads) copy_pages_kernel(const __grid_constant__ PageCopyParams p) {
  const long long page_bytes = (long long)p.vec_per_page * 16;
  const long long n_pages = (long long)p.n_blocks * p.n_layers * 2;
  const long long n_items = n_pages * p.pieces_per_page;
  for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
    const long long pg = item / p.pieces_per_page;
    const int piece = (int)(item - pg * p.pieces_per_page);
    const int i = (int)(pg / (2 * p.n_layers));
    const int rem = (int)(pg - (long long)i * 2 * p.n_layers);
    const int layer = rem >> 1, kv = rem & 1;
    long long wire_page;
    if (p.layout == KV_WIRE_BLOCK_MAJOR)
      wire_page = ((long long)(p.first_block + i) * p.n_layers + layer) * 2 + kv;
    else
      wire_page = ((long long)layer * 2 + kv) * p.total_blocks + p.first_block + i;
    int4 *cpage = reinterpret_cast<int4 *>(p.cache.page(layer, kv, p.ids[i]));
    int4 *wpage = reinterpret_cast<int4 *>(p.wire + wire_page * page_bytes);
    const int4 *src = TO_WIRE ? cpage : wpage;
    int4 *dst = TO_WIRE ? wpage : cpage;
    const int v0 = piece * kCopyThreads * kUnroll + threadIdx.x;
    int4 r[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int v = v0 + u * kCopyThreads;
      if (v < p.vec_per_page) r[u] = __ldcs(src + v);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int v = v0 + u * kCopyThreads;
      if (v < p.vec_per_page) __stcs(dst + v, r[u]);
    }
  }
}

int copy_pages(CacheView cache, int n_layers, const int *ids_host, int n_blocks, char *wire, int wire_layout,
               int total_blocks_in_wire, int first_block_in_wire, bool to_wire, cudaStream_t st) {
  int device = 0, sms = 148;
  KV_CUDA(cudaGetDevice(&device));
  KV_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
  for (int done = 0; done < n_blocks; done += kMaxIds) {
    PageCopyParams p;
    p.cache = cache;
    p.wire = wire;
    p.n_layers = n_layers;
    p.n_blocks = (n_blocks - done < kMaxIds) ? n_blocks - done : kMaxIds;
    p.layout = wire_layout;
    p.total_blocks = total_blocks_in_wire;
    p.first_block = first_block_in_wire + done;
    p.vec_per_page = (int)(cache.page_bytes() / 16);
    p.pieces_per_page = (p.vec_per_page + kCopyThreads * kUnroll - 1) / (kCopyThreads * kUnroll);
    for (int i = 0; i < p.n_blocks; ++i) p.ids[i] = ids_host[done + i];
    const long long items = (long long)p.n_blocks * n_layers * 2 * p.pieces_per_page;
    const long long cap = (long long)sms * 8;   // 8 resident CTAs of 256 threads per SM
    const int grid = (int)(items < cap ? items : cap);
    if (to_wire)
      copy_pages_kernel<true><<<grid, kCopyThreads, 0, st>>>(p);
    else
      copy_pages_kernel<false><<<grid, kCopyThreads, 0, st>>>(p);
    KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  }
  return KV_OK;
}

// Counter-based fill: word w = mix(seed + w); the host-side generator computes the same function.
__global__ void fill_pattern_kernel(unsigned long long *dst, long long n_words, unsigned long long seed,
                                    long long word0) {
  for (long long w = blockIdx.x * (long long)blockDim.x + threadIdx.x; w < n_words;
       w += (long long)gridDim.x * blockDim.x) {
    unsigned long long z = ((unsigned long long)(word0 + w) + seed) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    dst[w] = z ^ (z >> 31);
  }
}

int fill_pattern(void *dst, long long bytes, unsigned long long seed, long long offset, cudaStream_t st) {
  const long long n_words = bytes / 8;
  if (n_words == 0) return KV_OK;
  long long blocks = (n_words + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  fill_pattern_kernel<<<(int)blocks, 256, 0, st>>>((unsigned long long *)dst, n_words, seed, offset / 8);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

}  // namespace kvr
