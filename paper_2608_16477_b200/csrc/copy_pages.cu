// Pack (paged cache -> contiguous wire buffers) and unpack (wire buffers -> pages): byte-exact page copies.
//
// One launch moves every page of every request of a call: the physical block ids and one small record per
// request (its wire buffer and its slice of the id list) travel in the kernel parameter block, so no
// device-side staging of the id list and no extra copy precede the kernel.  Two parameter-block sizes are
// compiled: up to 896 ids / 8 requests (under 4 KiB, the single-request calls of the migration path) and up
// to 7,680 ids / 64 requests (under the 32 KiB limit of the launch interface, the batched calls); longer
// lists are split over several launches.
// A page (block_size * n_kv_heads * head_dim bf16) is contiguous on both sides; it moves as 16 KiB
// bulk copies (cp.async.bulk) through a shared-memory ring.  HBM-bound: 2 * page bytes of traffic
// per page, nothing is re-read.
#include <vector>

#include "common.cuh"

namespace kvr {

constexpr int kPieceBytes = 16384;    // bytes per bulk copy
constexpr int kBufs = 8;              // shared-memory ring: 128 KiB per CTA, one CTA per SM (measured best: ~128 KiB in flight per SM)
constexpr int kLag = 4;               // stores left in flight before a slot is refilled (kBufs - kLag loads in flight)
constexpr int kCopyThreads = 32;
constexpr long long kCopyWaitLimit = 2000000000ll;   // cycles (~1 s): far beyond any legitimate wait

// One request (or one slice of a request) inside a launch: ids[first_id .. first_id + n_blocks) are its blocks, in
// the order they occupy wire positions wire_first .. wire_first + n_blocks - 1 of a wire buffer of wire_total blocks.
struct CopySegment {
  char *wire;
  int first_id, n_blocks, wire_first, wire_total;
};

template <int MAX_IDS, int MAX_SEGS>
struct PageCopyParams {
  CacheView cache;
  int n_layers;
  int n_blocks;              // blocks in this launch (all segments)
  int n_segs;
  int layout;                // KV_WIRE_BLOCK_MAJOR / KV_WIRE_LAYER_MAJOR
  int page_bytes;
  int pieces_per_page;       // ceil(page_bytes / kPieceBytes)
  CopySegment segs[MAX_SEGS];
  int ids[MAX_IDS];
};
typedef PageCopyParams<896, 8> SmallCopyParams;
typedef PageCopyParams<7680, 64> LargeCopyParams;
static_assert(sizeof(SmallCopyParams) <= 4096, "single-request parameter block must stay under 4 KiB");
static_assert(sizeof(LargeCopyParams) <= 32764, "parameter block exceeds the launch interface's limit");

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
template <bool TO_WIRE, typename Params>
__global__ void __launch_bounds__(kCopyThreads) copy_pages_kernel(const __grid_constant__ Params p) {
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

  // Items are visited in increasing order by the loads and, a few items behind, by the stores: each of the two
  // walks keeps its own cursor into the segment list instead of searching it.
  auto locate = [&](long long k, int &seg, const char *&src, char *&dst, uint32_t &bytes) {
    const long long item = blockIdx.x + k * gridDim.x;
    const long long pg = item / p.pieces_per_page;
    const int piece = (int)(item - pg * p.pieces_per_page);
    const int i = (int)(pg / (2 * p.n_layers));                      // block index inside the launch
    const int rem = (int)(pg - (long long)i * 2 * p.n_layers);
    const int layer = rem >> 1, kv = rem & 1;
    while (seg + 1 < p.n_segs && i >= p.segs[seg].first_id + p.segs[seg].n_blocks) ++seg;
    const CopySegment &sg = p.segs[seg];
    const int w = sg.wire_first + (i - sg.first_id);                 // block position inside the request's wire
    long long wire_page;
    if (p.layout == KV_WIRE_BLOCK_MAJOR)
      wire_page = ((long long)w * p.n_layers + layer) * 2 + kv;
    else
      wire_page = ((long long)layer * 2 + kv) * sg.wire_total + w;
    const long long off = (long long)piece * kPieceBytes;
    char *c = p.cache.page(layer, kv, p.ids[i]) + off;
    char *wp = sg.wire + wire_page * p.page_bytes + off;
    src = TO_WIRE ? c : wp;
    dst = TO_WIRE ? wp : c;
    const long long left = p.page_bytes - off;
    bytes = (uint32_t)(left < kPieceBytes ? left : kPieceBytes);
  };
  int load_seg = 0, store_seg = 0;
  auto load = [&](long long k) {
    const int slot = (int)(k % kBufs);
    const char *src; char *dst; uint32_t bytes;
    locate(k, load_seg, src, dst, bytes);
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
    locate(k, store_seg, src, dst, bytes);
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

namespace {

template <typename Params>
int launch_copy(const Params &p, bool to_wire, int sms, cudaStream_t st) {
  const long long items = (long long)p.n_blocks * p.n_layers * 2 * p.pieces_per_page;
  const int grid = (int)(items < sms ? items : sms);
  if (to_wire)
    copy_pages_kernel<true, Params><<<grid, kCopyThreads, kBufs * kPieceBytes, st>>>(p);
  else
    copy_pages_kernel<false, Params><<<grid, kCopyThreads, kBufs * kPieceBytes, st>>>(p);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

// Fills parameter blocks of one size from the request list, starting a new launch whenever the ids or the
// segment records of the current one are used up (a request may continue in the next launch).
template <typename Params, int MAX_IDS, int MAX_SEGS>
int copy_requests(const CacheView &cache, int n_layers, const CopyRequest *reqs, int n_req, int wire_layout, bool to_wire,
                  int sms, cudaStream_t st) {
  Params p;
  auto reset = [&]() {
    p.cache = cache;
    p.n_layers = n_layers;
    p.layout = wire_layout;
    p.page_bytes = (int)cache.page_bytes();
    p.pieces_per_page = (p.page_bytes + kPieceBytes - 1) / kPieceBytes;
    p.n_blocks = 0;
    p.n_segs = 0;
  };
  reset();
  for (int r = 0; r < n_req; ++r) {
    int done = 0;
    while (done < reqs[r].n_blocks) {
      if (p.n_blocks == MAX_IDS || p.n_segs == MAX_SEGS) {
        int rc = launch_copy(p, to_wire, sms, st);
        if (rc != KV_OK) return rc;
        reset();
      }
      const int take = reqs[r].n_blocks - done < MAX_IDS - p.n_blocks ? reqs[r].n_blocks - done : MAX_IDS - p.n_blocks;
      CopySegment &sg = p.segs[p.n_segs++];
      sg.wire = reqs[r].wire;
      sg.first_id = p.n_blocks;
      sg.n_blocks = take;
      sg.wire_first = done;
      sg.wire_total = reqs[r].n_blocks;
      for (int i = 0; i < take; ++i) p.ids[p.n_blocks + i] = reqs[r].ids_host[done + i];
      p.n_blocks += take;
      done += take;
    }
  }
  if (p.n_blocks > 0) return launch_copy(p, to_wire, sms, st);
  return KV_OK;
}

}  // namespace

int copy_pages(CacheView cache, int n_layers, const CopyRequest *reqs, int n_req, int wire_layout, bool to_wire,
               cudaStream_t st) {
  static bool attr_set[kMaxDevices] = {};
  const int device = current_device();
  if (device < 0) return KV_ERR_CUDA;
  if (!attr_set[device]) {
    KV_CUDA(cudaFuncSetAttribute(copy_pages_kernel<true, SmallCopyParams>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kBufs * kPieceBytes));
    KV_CUDA(cudaFuncSetAttribute(copy_pages_kernel<false, SmallCopyParams>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kBufs * kPieceBytes));
    KV_CUDA(cudaFuncSetAttribute(copy_pages_kernel<true, LargeCopyParams>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kBufs * kPieceBytes));
    KV_CUDA(cudaFuncSetAttribute(copy_pages_kernel<false, LargeCopyParams>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kBufs * kPieceBytes));
    attr_set[device] = true;
  }
  const int sms = sm_count(device);
  long long total = 0;
  int live = 0;
  for (int r = 0; r < n_req; ++r) {
    total += reqs[r].n_blocks;
    live += reqs[r].n_blocks > 0 ? 1 : 0;
  }
  if (total == 0) return KV_OK;
  if (total <= 896 && live <= 8)
    return copy_requests<SmallCopyParams, 896, 8>(cache, n_layers, reqs, n_req, wire_layout, to_wire, sms, st);
  return copy_requests<LargeCopyParams, 7680, 64>(cache, n_layers, reqs, n_req, wire_layout, to_wire, sms, st);
}

// Reads the flag a copy kernel raises when one of its bounded waits ran out, and clears it, so that one expired
// wait is reported once and later, healthy copies on the device are not blamed for it.
int copy_wait_expired(cudaStream_t st) {
  int flag = 0;
  KV_CUDA(cudaStreamSynchronize(st));
  KV_CUDA(cudaMemcpyFromSymbol(&flag, g_copy_wait_expired, sizeof(int)));
  if (flag != 0) {
    const int zero = 0;
    KV_CUDA(cudaMemcpyToSymbol(g_copy_wait_expired, &zero, sizeof(int)));
    return KV_ERR_DEVICE;
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
