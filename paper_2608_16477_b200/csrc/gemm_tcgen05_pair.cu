// CTA-pair variant of the projection GEMM: tcgen05.mma with cta_group::2.
//
// Two CTAs of a cluster (two SMs) compute one 256 x BN tile.  Each CTA loads only ITS 128 rows of A and ITS
// half of the W tile (BN/2 rows) by TMA into its own shared memory; the MMA warp of the leader CTA (converged,
// one elected lane per instruction) issues M=256 MMAs that read A and W from both CTAs' shared memory and accumulate rows 0-127 into the leader's TMEM
// and rows 128-255 into the peer's.  Per SM this halves the W bytes fetched from L2 and read from shared
// memory per flop (16 KiB + 16 KiB per stage instead of 16 + 32) and leaves room for a 6-stage ring.
// No load is shared between the CTAs: every TMA copy lands in the shared memory of the CTA that issued it;
// only its completion is counted on the leader's mbarrier.
//
//   warp 0 (both CTAs)  TMA producer for the CTA's own A rows and W rows; completion bytes go to the
//                       LEADER's full barrier (the leader expects both CTAs' bytes).
//   warp 1              TMEM allocation (cta_group::2, both CTAs); in the leader: MMA issue, stage release
//                       and accumulator hand-off committed to both CTAs' barriers.
//   warps 2-5 (both)    epilogue of the CTA's own 128 rows (same code as the one-CTA kernel); the peer's
//                       epilogue threads arrive on the leader's tmem_empty barrier remotely.
// Every mbarrier wait is bounded; the two CTAs synchronise as a cluster once after barrier set-up and once
// before TMEM is freed.
#include <cstring>

#include "gemm_epilogue.cuh"

namespace kvr {

namespace {

constexpr int BM = 128;              // rows per CTA (256 per pair)
constexpr int BK = 64;
constexpr int kABytes = BM * BK * 2;
constexpr int kTmemCols = 512;
constexpr int kTmemBufStride = 256;
constexpr int kThreads = 192;
constexpr int kMaxSmem = 232448;

enum WaitTag2 { TAG2_EMPTY = 21, TAG2_FULL = 22, TAG2_TMEM_EMPTY = 23, TAG2_TMEM_FULL = 24 };

template <int MODE, int BN>
struct PairCfg {
  static constexpr int kBBytes = (BN / 2) * BK * 2;             // this CTA's half of the W tile
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kEpiBytes = (MODE == GEMM_RESID_F32) ? kEpiStageBytes : 0;
  static constexpr int kStagesFit = (kMaxSmem - 1024 - 256 - kEpiBytes) / kStageBytes;
  static constexpr int kStages = kStagesFit > 8 ? 8 : kStagesFit;
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 + 256 + kEpiBytes;
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA tile load into this CTA's shared memory whose completion bytes are counted on `bar_cluster`, an
// mbarrier that may live in the pair's other CTA.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst_smem, const CUtensorMap *map, int x, int y,
                                                 uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst_smem), "l"((uint64_t)map), "r"(x), "r"(y), "r"(bar_cluster)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t holder_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder_smem), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// Whole-warp forms (every lane calls with the same operands, one elected lane issues).
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred pe, p;\n\t"
      "elect.sync _|pe, 0xffffffff;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "@pe tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// one arrival on the mbarrier at `bar_cluster` (own or peer CTA) once all MMAs issued so far are done
__device__ __forceinline__ void umma_commit_pair(uint32_t bar_cluster) {
  asm volatile(
      "{\n\t.reg .pred pe;\n\t"
      "elect.sync _|pe, 0xffffffff;\n\t"
      "@pe tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(bar_cluster) : "memory");
}

template <int MODE, int BN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap tma_a, const __grid_constant__ CUtensorMap tma_b, int m, int n,
                    int k, bf16 *__restrict__ out, float *__restrict__ resid, DeviceStatus *status,
                    const __grid_constant__ QkvRopeArgs qa) {
  constexpr int kStages = PairCfg<MODE, BN>::kStages;
  constexpr int kStageBytes = PairCfg<MODE, BN>::kStageBytes;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *smem_gen = smem_raw + (smem_base - tc::smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + kStages * kStageBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * kStages + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * kStages + 2 + b); };
  uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(smem_gen + kStages * kStageBytes + 8 * (2 * kStages + 4));
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0: leader (issues the MMAs), 1: peer
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  constexpr int kOutCols = (MODE == GEMM_SWIGLU) ? BN / 2 : BN;
  const int m_tiles = (m + 2 * BM - 1) / (2 * BM);  // 256-row tiles
  const int n_tiles = (n + kOutCols - 1) / kOutCols;
  const int total_tiles = m_tiles * n_tiles;
  const int k_blocks = (k + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      tc::mbar_init(full_bar(s), 1);     // used in the leader only: one expect_tx arrival, bytes of both CTAs
      tc::mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      tc::mbar_init(tfull_bar(b), 1);
      tc::mbar_init(tempty_bar(b), 256); // used in the leader only: epilogue threads of both CTAs
    }
    *abort_flag = 0;
    tc::fence_barrier_init();
  }
  if (warp == 1) tmem_alloc_pair(tc::smem_u32(tmem_holder), kTmemCols);
  tc::tc_fence_before();
  __syncthreads();
  cluster_sync_all();                    // both CTAs' barriers exist before anything remote touches them
  tc::tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (own A rows, own W rows)
    if (lane == 0) {
      tc::tma_prefetch_desc(&tma_a);
      tc::tma_prefetch_desc(&tma_b);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
        const int m0 = (tile % m_tiles) * 2 * BM + (int)rank * BM;
        const int n0 = (tile / m_tiles) * kOutCols;
        // W rows of this CTA: plain/residual/QKV tiles split their BN rows in two halves; a SwiGLU tile has
        // its gate rows in the leader and the matching up rows in the peer
        const int w_row = (MODE == GEMM_SWIGLU) ? (rank == 0 ? n0 : n + n0) : n0 + (int)rank * (BN / 2);
        for (int kb = 0; kb < k_blocks; ++kb) {
          ok = tc::mbar_wait(empty_bar(stage), phase ^ 1, abort_flag, status, TAG2_EMPTY);
          if (!ok) break;
          const uint32_t a_s = smem_base + stage * kStageBytes;
          const uint32_t b_s = a_s + kABytes;
          const uint32_t leader_full = map_to_cta(full_bar(stage), 0);
          if (rank == 0) tc::mbar_expect_tx(full_bar(stage), 2 * kStageBytes);
          tma_load_2d_pair(a_s, &tma_a, kb * BK, m0, leader_full);
          tma_load_2d_pair(b_s, &tma_b, kb * BK, w_row, leader_full);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (rank == 0) {
      auto wwait = [&](uint32_t b_, uint32_t parity, int tag) {
        return __all_sync(0xffffffffu, tc::mbar_wait(b_, parity, abort_flag, status, tag)) != 0;
      };
      constexpr uint32_t idesc = tc::umma_idesc_bf16(2 * BM, BN);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int local = 0;
      for (int tile = pair; tile < total_tiles && ok; tile += n_pairs, ++local) {
        const int buf = local & 1;
        const uint32_t acc_phase = (local >> 1) & 1;
        ok = wwait(tempty_bar(buf), acc_phase ^ 1, TAG2_TMEM_EMPTY);
        if (!ok) break;
        tc::tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * kTmemBufStride;
        for (int kb = 0; kb < k_blocks; ++kb) {
          ok = wwait(full_bar(stage), phase, TAG2_FULL);
          if (!ok) break;
          tc::tc_fence_after();
          const uint32_t a_s = smem_base + stage * kStageBytes;
          const uint64_t a_desc = tc::umma_desc_k128(a_s);
          const uint64_t b_desc = tc::umma_desc_k128(a_s + kABytes);
#pragma unroll
          for (int ks = 0; ks < BK / 16; ++ks)
            umma_bf16_pair(d_tmem, a_desc + 2 * ks, b_desc + 2 * ks, idesc, (kb | ks) != 0);
          // the stage is free in BOTH CTAs once these MMAs have read it
          umma_commit_pair(empty_bar(stage));
          umma_commit_pair(map_to_cta(empty_bar(stage), 1));
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (ok) {
          umma_commit_pair(tfull_bar(buf));
          umma_commit_pair(map_to_cta(tfull_bar(buf), 1));
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue of this CTA's 128 rows
    const int quarter = warp & 3;
    bool ok = true;
    int local = 0;
    for (int tile = pair; tile < total_tiles && ok; tile += n_pairs, ++local) {
      const int buf = local & 1;
      const uint32_t acc_phase = (local >> 1) & 1;
      const int m0 = (tile % m_tiles) * 2 * BM + (int)rank * BM;
      const int n0 = (tile / m_tiles) * kOutCols;
      ok = tc::mbar_wait(tfull_bar(buf), acc_phase, abort_flag, status, TAG2_TMEM_FULL);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc::tc_fence_after();
      const int row = m0 + quarter * 32 + lane;
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * kTmemBufStride;
      gemm_epilogue_slab<MODE, BN>(t_row, row, m0, n0, m, n, quarter, lane, warp, out, resid, qa,
                                   reinterpret_cast<float4 *>(smem_gen + kStages * kStageBytes + 256));
      tc::tc_fence_before();
      mbar_arrive_cluster(map_to_cta(tempty_bar(buf), 0));   // the leader's MMA thread waits for both CTAs
    }
  }

  // teardown: neither CTA may leave (or free TMEM) while the other still reads its shared memory or barriers
  tc::tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc::tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

template <int MODE, int BN>
int launch_pair(const CUtensorMap &ta, const CUtensorMap &tb, int m, int n, int k, bf16 *out, float *resid,
                DeviceStatus *status, const QkvRopeArgs &qa, int sms, cudaStream_t st) {
  static bool attr_set[kMaxDevices] = {};
  const int device = current_device();
  if (device < 0) return KV_ERR_CUDA;
  if (!attr_set[device]) {
    KV_CUDA(cudaFuncSetAttribute(gemm_tc_pair_kernel<MODE, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 PairCfg<MODE, BN>::kSmemBytes));
    attr_set[device] = true;
  }
  const int out_cols = (MODE == GEMM_SWIGLU) ? BN / 2 : BN;
  const int tiles = ((m + 2 * BM - 1) / (2 * BM)) * ((n + out_cols - 1) / out_cols);
  int pairs = sms / 2;
  if (tiles < pairs) pairs = tiles;
  gemm_tc_pair_kernel<MODE, BN><<<2 * pairs, kThreads, PairCfg<MODE, BN>::kSmemBytes, st>>>(ta, tb, m, n, k, out, resid,
                                                                                           status, qa);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

// Tile width minimising waves x width / efficiency over the SM pairs (same model as the one-CTA kernel).
int pick_bn_pair(int m, int n_out, int sms, int mode, int head_dim) {
  const int widths[5] = {256, 224, 192, 160, 128};
  const double eff[5] = {1.00, 0.99, 0.98, 0.92, 0.78};     // measured per-column cost relative to 256-wide tiles
  const long long m_tiles = (m + 2 * BM - 1) / (2 * BM);
  const int pairs = sms / 2;
  int best = 256;
  double best_cost = -1.0;
  for (int i = 0; i < 5; ++i) {
    const int bn = widths[i];
    if (mode == GEMM_QKV_ROPE && (bn % head_dim) != 0) continue;
    if (mode == GEMM_SWIGLU && (bn % 64) != 0) continue;
    const int out_cols = (mode == GEMM_SWIGLU) ? bn / 2 : bn;
    const long long tiles = m_tiles * ((n_out + out_cols - 1) / out_cols);
    const double cost = (double)((tiles + pairs - 1) / pairs) * bn / eff[i];
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost;
      best = bn;
    }
  }
  return best;
}

}  // namespace

int gemm_tc_pair_tile_width(int m, int n_out, int sms, int mode, int head_dim) {
  return pick_bn_pair(m, n_out, sms, mode, head_dim);
}

// CTA-pair GEMM, 256 x BN tiles.  Same contract as gemm_tc.
int gemm_tc_pair(const bf16 *a, int lda, const bf16 *w, int m, int n, int k, int mode, bf16 *out, float *resid,
                 int *status_dev, cudaStream_t st, const QkvRopeArgs *qkv_args) {
  if (m <= 0 || n <= 0 || k <= 0) return KV_OK;
  QkvRopeArgs qa;
  memset(&qa, 0, sizeof(qa));
  if (mode == GEMM_QKV_ROPE) {
    if (qkv_args == nullptr) return KV_ERR_ARG;
    qa = *qkv_args;
    if (qa.head_dim != 64 && qa.head_dim != 128) return KV_ERR_SHAPE;
    if (n != (qa.n_q_heads + 2 * qa.n_kv_heads) * qa.head_dim) return KV_ERR_SHAPE;
  }
  if ((k % 8) != 0 || (lda % 8) != 0 || (n % 8) != 0) return KV_ERR_SHAPE;
  if (((uintptr_t)a & 15) || ((uintptr_t)w & 15) || ((uintptr_t)out & 15) || ((uintptr_t)resid & 15)) return KV_ERR_ARG;
  const int sms = sm_count(current_device());
  const int bn = pick_bn_pair(m, n, sms, mode, mode == GEMM_QKV_ROPE ? qa.head_dim : 0);
  CUtensorMap ta, tb;
  int rc = tc::make_tmap_2d(&ta, a, m, k, lda, BM);
  if (rc != KV_OK) return rc;
  const long long w_rows = (mode == GEMM_SWIGLU) ? 2ll * n : n;
  rc = tc::make_tmap_2d(&tb, w, w_rows, k, k, bn / 2);
  if (rc != KV_OK) return rc;
  DeviceStatus *status = reinterpret_cast<DeviceStatus *>(status_dev);
#define KV_PAIR_CASE(MODE_, BN_) \
  if (mode == MODE_ && bn == BN_) return launch_pair<MODE_, BN_>(ta, tb, m, n, k, out, resid, status, qa, sms, st)
  KV_PAIR_CASE(GEMM_RESID_F32, 256);
  KV_PAIR_CASE(GEMM_RESID_F32, 224);
  KV_PAIR_CASE(GEMM_RESID_F32, 192);
  KV_PAIR_CASE(GEMM_RESID_F32, 160);
  KV_PAIR_CASE(GEMM_RESID_F32, 128);
  KV_PAIR_CASE(GEMM_STORE_BF16, 256);
  KV_PAIR_CASE(GEMM_STORE_BF16, 224);
  KV_PAIR_CASE(GEMM_STORE_BF16, 192);
  KV_PAIR_CASE(GEMM_STORE_BF16, 160);
  KV_PAIR_CASE(GEMM_STORE_BF16, 128);
  KV_PAIR_CASE(GEMM_SWIGLU, 256);
  KV_PAIR_CASE(GEMM_SWIGLU, 192);
  KV_PAIR_CASE(GEMM_SWIGLU, 128);
  KV_PAIR_CASE(GEMM_QKV_ROPE, 256);
  KV_PAIR_CASE(GEMM_QKV_ROPE, 192);
  KV_PAIR_CASE(GEMM_QKV_ROPE, 128);
#undef KV_PAIR_CASE
  return KV_ERR_ARG;
}

}  // namespace kvr
