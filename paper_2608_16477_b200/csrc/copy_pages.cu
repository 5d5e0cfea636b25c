// Pack (paged cache -> contiguous wire buffer) and unpack (wire buffer -> pages): byte-exact page copies.
//
// One launch moves every page of up to kMaxIds logical blocks: block ids travel in the kernel
// parameter block, so no device-side staging of the id list and no extra copy precede the kernel.
// A page (block_size * n_kv_heads * head_dim bf16) is contiguous on both sides; it moves as 16 KiB
// bulk copies (cp.async.bulk) through a shared-memory ring.  HBM-bound: 2 * page bytes of traffic
// per page, nothing is re-read.
#include "common.cuh"

namespace kvr {

constexpr int kMaxIds = 960;          // keeps the parameter block under 4 KiB
#ifndef KV_COPY_PIECE
#define KV_COPY_PIECE 16384
#define KV_COPY_BUFS 8
#define KV_COPY_LAG 4
#define KV_COPY_CTAS 1
#endif
constexpr int kPieceBytes = KV_COPY_PIECE;   // bytes per bulk copy
constexpr int kBufs = KV_COPY_BUFS;          // shared-memory ring: 128 KiB per CTA, one CTA per SM (measured best: ~128 KiB in flight per SM)
constexpr int kLag = KV_COPY_LAG;            // stores left in flight before a slot is refilled (kBufs - kLag loads in flight)
constexpr int kCopyThreads = 32;
constexpr int kCtasPerSm = KV_COPY_CTAS;
constexpr long long kCopyWaitLimit = 2000000000ll;   // cycles (~1 s): far beyond any legitimate wait

struct PageCopyParams {
  CacheView cache;
  char *wire;
  int n_layers;
  int n_blocks;              // blocks in this launch
  int layout;                // KV_WIRE_BLOCK_MAJOR / KV_WIRE_LAYER_MAJOR
  int total_blocks;          // blocks in the whole wire buffer (layer-major stride)
  int first_block;           // index of this launch's first block inside the wire buffer
  int page_bytes;
  int pieces_per_page;       // ceil(page_bytes / kPieceBytes)
  int ids[kMaxIds];
};

// Set by a copy kernel whose bounded wait ran out (the kernel then stops copying and returns).
__device__ int g_copy_wait_expired = 0;

__device__ __forceinline__ uint32_t cp_smem(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ bool cp_wait(uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  for (uint32_t it = 0;; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (ok) return true;
    if ((it & 0xff) == 0xff && clock64() - t0 > kCopyWaitLimit) {
      g_copy_wait_expired = 1;
      return false;
    }
  }
}

// One thread per CTA drives a ring of bulk copies: global -> shared (completion on an mbarrier), then
// shared -> global (bulk group).  Neither the LSU nor registers touch the payload, so the achieved
// bandwidth does not depend on the SM clock.  A slot is refilled once the store that read it has
// finished reading (wait_group.read), which keeps kBufs - kLag loads and kLag stores in flight per CTA.
template <bool TO_WIRE>
__global__ void __launch_bounds__(kCopyThreads) copy_pages_kernel(const __grid_constant__ PageCopyParams p) {
  extern __shared__ __align__(128) unsigned char ring[];
  __shared__ __align__(8) unsigned long long full[kBufs];
  if (threadIdx.x != 0) return;
  const long long n_pages = (long long)p.n_blocks * p.n_layers * 2;
  const long long n_items = n_pages * p.pieces_per_page;
  // this CTA's items: blockIdx.x, blockIdx.x + gridDim.x, ...
  const long long mine = (n_items - blockIdx.x + gridDim.x - 1) / gridDim.x;
  if (mine <= 0) return;
  for (int b = 0; b < kBufs; ++b)
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(cp_smem(&full[b])));
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");

  auto locate = [&](long long k, const char *&src, char *&dst, uint32_t &bytes) {
    const long long item = blockIdx.x + k * gridDim.x;
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
    const long long off = (long long)piece * kPieceBytes;
    char *c = p.cache.page(layer, kv, p.ids[i]) + off;
    char *w = p.wire + wire_page * p.page_bytes + off;
    src = TO_WIRE ? c : w;
    dst = TO_WIRE ? w : c;
    const long long left = p.page_bytes - off;
    bytes = (uint32_t)(left < kPieceBytes ? left : kPieceBytes);
  };
  auto load = [&](long long k) {
    const int slot = (int)(k % kBufs);
    const char *src; char *dst; uint32_t bytes;
    locate(k, src, dst, bytes);
    const uint32_t bar = cp_smem(&full[slot]);
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(cp_smem(ring + slot * kPieceBytes)), "l"(src), "r"(bytes), "r"(bar) : "memory");
  };

  const long long prologue = mine < kBufs ? mine : kBufs;
  for (long long k = 0; k < prologue; ++k) load(k);
  for (long long k = 0; k < mine; ++k) {
    const int slot = (int)(k % kBufs);
    if (!cp_wait(cp_smem(&full[slot]), (uint32_t)((k / kBufs) & 1))) break;
    const char *src; char *dst; uint32_t bytes;
    locate(k, src, dst, bytes);
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(dst), "r"(cp_smem(ring + slot * kPieceBytes)), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    // refill the slot of item k - kLag once its store has read it: up to kLag younger stores stay pending, so
    // the issuing thread never waits on the store it has just issued
    if (k >= kLag && k - kLag + kBufs < mine) {
      asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(kLag) : "memory");
      load(k - kLag + kBufs);
    }
  }
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // all stores complete before the CTA exits
}

int copy_pages(CacheView cache, int n_layers, const int *ids_host, int n_blocks, char *wire, int wire_layout,
               int total_blocks_in_wire, int first_block_in_wire, bool to_wire, cudaStream_t st) {
  static bool attr_set[kMaxDevices] = {};
  const int device = current_device();
  if (device < 0) return KV_ERR_CUDA;
  if (!attr_set[device]) {
    KV_CUDA(cudaFuncSetAttribute(copy_pages_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kBufs * kPieceBytes));
    KV_CUDA(cudaFuncSetAttribute(copy_pages_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kBufs * kPieceBytes));
    attr_set[device] = true;
  }
  const int sms = sm_count(device);
  for (int done = 0; done < n_blocks; done += kMaxIds) {
    PageCopyParams p;
    p.cache = cache;
    p.wire = wire;
    p.n_layers = n_layers;
    p.n_blocks = (n_blocks - done < kMaxIds) ? n_blocks - done : kMaxIds;
    p.layout = wire_layout;
    p.total_blocks = total_blocks_in_wire;
    p.first_block = first_block_in_wire + done;
    p.page_bytes = (int)cache.page_bytes();
    p.pieces_per_page = (p.page_bytes + kPieceBytes - 1) / kPieceBytes;
    for (int i = 0; i < p.n_blocks; ++i) p.ids[i] = ids_host[done + i];
    const long long items = (long long)p.n_blocks * n_layers * 2 * p.pieces_per_page;
    const long long cap = (long long)sms * kCtasPerSm;
    const int grid = (int)(items < cap ? items : cap);
    if (to_wire)
      copy_pages_kernel<true><<<grid, kCopyThreads, kBufs * kPieceBytes, st>>>(p);
    else
      copy_pages_kernel<false><<<grid, kCopyThreads, kBufs * kPieceBytes, st>>>(p);
    KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  }
  return KV_OK;
}

int copy_wait_expired(cudaStream_t st) {
  int flag = 0;
  KV_CUDA(cudaStreamSynchronize(st));
  KV_CUDA(cudaMemcpyFromSymbol(&flag, g_copy_wait_expired, sizeof(int)));
  return flag ? KV_ERR_DEVICE : KV_OK;
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
