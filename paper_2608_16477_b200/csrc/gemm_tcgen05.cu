// Dense projections on the 5th-generation tensor cores:  C[M,N] = A[M,K] * W[N,K]^T, bf16 in, fp32 accumulate.
//
// Persistent, warp-specialised kernel, one CTA per SM:
//   warp 0   TMA producer: 128x64 A tile and 256x64 W tile per stage into a 4-deep shared-memory ring
//            (128-byte swizzle, K-major on both operands, so neither matrix is ever transposed);
//   warp 1   allocates TMEM (512 columns = two 128x256 fp32 accumulators) and issues tcgen05.mma
//            (M=128, N=256, K=16; four per stage), committing each stage back to the producer and each
//            finished accumulator to the epilogue;
//   warps 2-5  epilogue: tcgen05.ld 32 columns at a time, fused epilogue, direct global stores.  The
//            second accumulator lets the epilogue of tile i overlap the main loop of tile i+1.
// Epilogues: bf16 store; fp32 residual add (x += A W^T); SwiGLU (W tile = 128 gate rows + the matching
// 128 up rows, output silu(gate) * up); QKV with RoPE applied to the fp32 accumulators (rotate-half pairs
// sit d/2 columns apart inside the same tile) and the rotated K and the V stored straight into the paged
// cache through the block table, so K/V are rounded to bf16 exactly once.
// Tiles are walked M-fastest so concurrently running CTAs share the same W tiles through L2.
// Every mbarrier wait is bounded; a wait that runs out records itself in the status block and the CTA
// drains and frees its TMEM instead of hanging.
#include <cstring>

#include "gemm_epilogue.cuh"

namespace kvr {

namespace {

constexpr int BM = 128;
constexpr int BK = 64;       // 128 bytes of bf16: one swizzle atom
constexpr int kABytes = BM * BK * 2;            // 16 KiB
constexpr int kTmemCols = 512;
constexpr int kTmemBufStride = 256;             // the two accumulators sit at columns 0 and 256
constexpr int kThreads = 192;
constexpr int kMaxSmem = 232448;                // 227 KiB per CTA

// Tile width BN (accumulator columns) is a template parameter: 256 by default, narrower tiles where they
// remove a mostly empty last wave (e.g. N = 5120 over 148 SMs: 23 tiles of 224 fill 4.97 waves, 20 of 256 need 5 of 4.3).
template <int MODE, int BN>
struct TileCfg {
  static constexpr int kBBytes = BN * BK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kEpiBytes = (MODE == GEMM_RESID_F32) ? kEpiStageBytes : 0;
  static constexpr int kStagesFit = (kMaxSmem - 1024 - 256 - kEpiBytes) / kStageBytes;
  static constexpr int kStages = kStagesFit > 6 ? 6 : kStagesFit;
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/ + kEpiBytes;
};

enum WaitTag { TAG_EMPTY = 1, TAG_FULL = 2, TAG_TMEM_EMPTY = 3, TAG_TMEM_FULL = 4 };

template <int MODE, int BN>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tma_a, const __grid_constant__ CUtensorMap tma_b, int m, int n,
               int k, bf16 *__restrict__ out, float *__restrict__ resid, DeviceStatus *status,
               const __grid_constant__ QkvRopeArgs qa) {
  constexpr int kStages = TileCfg<MODE, BN>::kStages;
  constexpr int kBBytes = TileCfg<MODE, BN>::kBBytes;
  constexpr int kStageBytes = TileCfg<MODE, BN>::kStageBytes;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *smem_gen = smem_raw + (smem_base - tc::smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + kStages * kStageBytes;
  // barrier layout (8 bytes each): full[kStages], empty[kStages], tmem_full[2], tmem_empty[2], then holder + abort
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * kStages + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * kStages + 2 + b); };
  uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(smem_gen + kStages * kStageBytes + 8 * (2 * kStages + 4));
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int kOutCols = (MODE == GEMM_SWIGLU) ? BN / 2 : BN;   // output columns per tile
  const int m_tiles = (m + BM - 1) / BM;
  const int n_tiles = (n + kOutCols - 1) / kOutCols;
  const int total_tiles = m_tiles * n_tiles;
  const int k_blocks = (k + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      tc::mbar_init(full_bar(s), 1);
      tc::mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      tc::mbar_init(tfull_bar(b), 1);
      tc::mbar_init(tempty_bar(b), 128);
    }
    *abort_flag = 0;
    tc::fence_barrier_init();
  }
  if (warp == 1) tc::tmem_alloc(tc::smem_u32(tmem_holder), kTmemCols);
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tc::tma_prefetch_desc(&tma_a);
      tc::tma_prefetch_desc(&tma_b);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile % m_tiles) * BM;
        const int n0 = (tile / m_tiles) * kOutCols;
        for (int kb = 0; kb < k_blocks; ++kb) {
          ok = tc::mbar_wait(empty_bar(stage), phase ^ 1, abort_flag, status, TAG_EMPTY);
          if (!ok) break;
          const uint32_t a_s = smem_base + stage * kStageBytes;
          const uint32_t b_s = a_s + kABytes;
          tc::mbar_expect_tx(full_bar(stage), kStageBytes);
          tc::tma_load_2d(a_s, &tma_a, kb * BK, m0, full_bar(stage));
          if (MODE == GEMM_SWIGLU) {
            tc::tma_load_2d(b_s, &tma_b, kb * BK, n0, full_bar(stage));                    // gate rows
            tc::tma_load_2d(b_s + kBBytes / 2, &tma_b, kb * BK, n + n0, full_bar(stage));  // up rows
          } else {
            tc::tma_load_2d(b_s, &tma_b, kb * BK, n0, full_bar(stage));
          }
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // The whole warp runs the loop and one elected lane issues each instruction: operands prepared per warp
    // reach tcgen05.mma far faster than from a single-lane branch.
    {
      auto wwait = [&](uint32_t b_, uint32_t parity, int tag) {
        return __all_sync(0xffffffffu, tc::mbar_wait(b_, parity, abort_flag, status, tag)) != 0;
      };
      constexpr uint32_t idesc = tc::umma_idesc_bf16(BM, BN);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int local = 0;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++local) {
        const int buf = local & 1;
        const uint32_t acc_phase = (local >> 1) & 1;
        ok = wwait(tempty_bar(buf), acc_phase ^ 1, TAG_TMEM_EMPTY);
        if (!ok) break;
        tc::tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * kTmemBufStride;
        for (int kb = 0; kb < k_blocks; ++kb) {
          ok = wwait(full_bar(stage), phase, TAG_FULL);
          if (!ok) break;
          tc::tc_fence_after();
          const uint32_t a_s = smem_base + stage * kStageBytes;
          const uint64_t a_desc = tc::umma_desc_k128(a_s);
          const uint64_t b_desc = tc::umma_desc_k128(a_s + kABytes);
#pragma unroll
          for (int ks = 0; ks < BK / 16; ++ks)   // +32 bytes (2 descriptor units) per K=16 slice
            tc::umma_bf16_warp(d_tmem, a_desc + 2 * ks, b_desc + 2 * ks, idesc, (kb | ks) != 0);
          tc::umma_commit_warp(empty_bar(stage));
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (ok) tc::umma_commit_warp(tfull_bar(buf));
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int quarter = warp & 3;   // TMEM lanes this warp may read: 32*quarter .. +31
    bool ok = true;
    int local = 0;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++local) {
      const int buf = local & 1;
      const uint32_t acc_phase = (local >> 1) & 1;
      const int m0 = (tile % m_tiles) * BM;
      const int n0 = (tile / m_tiles) * kOutCols;
      ok = tc::mbar_wait(tfull_bar(buf), acc_phase, abort_flag, status, TAG_TMEM_FULL);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc::tc_fence_after();
      const int row = m0 + quarter * 32 + lane;
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * kTmemBufStride;
      gemm_epilogue_slab<MODE, BN>(t_row, row, m0, n0, m, n, quarter, lane, warp, out, resid, qa,
                                   reinterpret_cast<float4 *>(smem_gen + kStages * kStageBytes + 256));
      tc::tc_fence_before();
      tc::mbar_arrive(tempty_bar(buf));
    }
  }

  // teardown: every role has left its loop (normally or through the abort flag)
  tc::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc::tc_fence_after();
    tc::tmem_dealloc(tmem_base, kTmemCols);
  }
}

template <int MODE, int BN>
int launch_gemm(const CUtensorMap &ta, const CUtensorMap &tb, int m, int n, int k, bf16 *out, float *resid,
                DeviceStatus *status, const QkvRopeArgs &qa, int sms, cudaStream_t st) {
  static bool attr_set[kMaxDevices] = {};
  const int device = current_device();
  if (device < 0) return KV_ERR_CUDA;
  if (!attr_set[device]) {
    KV_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<MODE, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 TileCfg<MODE, BN>::kSmemBytes));
    attr_set[device] = true;
  }
  const int out_cols = (MODE == GEMM_SWIGLU) ? BN / 2 : BN;
  const int tiles = ((m + BM - 1) / BM) * ((n + out_cols - 1) / out_cols);
  const int grid = tiles < sms ? tiles : sms;
  gemm_tc_kernel<MODE, BN><<<grid, kThreads, TileCfg<MODE, BN>::kSmemBytes, st>>>(ta, tb, m, n, k, out, resid, status, qa);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

// Tile width that minimises the modelled time (waves x tile width / relative efficiency of that width) for an
// M x N problem on `sms` SMs.  SwiGLU tiles hold a gate half and an up half, so a BN-wide tile yields BN / 2
// output columns; QKV tiles must hold whole heads.
int pick_bn(int m, int n_out, int sms, int mode, int head_dim) {
  const int widths[5] = {256, 224, 192, 160, 128};
  const double eff[5] = {1.00, 1.00, 0.99, 0.96, 0.85};     // measured: narrower tiles re-read A more often and
                                                             // amortise the per-stage barrier work over fewer flops
  const long long m_tiles = (m + BM - 1) / BM;
  int best = 256;
  double best_cost = -1.0;
  for (int i = 0; i < 5; ++i) {
    const int bn = widths[i];
    if (mode == GEMM_QKV_ROPE && (bn % head_dim) != 0) continue;        // tiles must hold whole heads
    if (mode == GEMM_SWIGLU && (bn % 64) != 0) continue;                // halves are multiples of 32 columns
    const int out_cols = (mode == GEMM_SWIGLU) ? bn / 2 : bn;
    const long long tiles = m_tiles * ((n_out + out_cols - 1) / out_cols);
    const double cost = (double)((tiles + sms - 1) / sms) * bn / eff[i];
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost;
      best = bn;
    }
  }
  return best;
}

}  // namespace

int gemm_tc_tile_width(int m, int n_out, int sms, int mode, int head_dim) { return pick_bn(m, n_out, sms, mode, head_dim); }

int gemm_tc(const bf16 *a, int lda, const bf16 *w, int m, int n, int k, int mode, bf16 *out, float *resid,
            int *status_dev, cudaStream_t st, const QkvRopeArgs *qkv_args) {
  if (m <= 0 || n <= 0 || k <= 0) return KV_OK;
  QkvRopeArgs qa;
  memset(&qa, 0, sizeof(qa));
  if (mode == GEMM_QKV_ROPE) {
    if (qkv_args == nullptr) return KV_ERR_ARG;
    qa = *qkv_args;
    if (qa.head_dim != 64 && qa.head_dim != 128 && qa.head_dim != 256) return KV_ERR_SHAPE;
    if (n != (qa.n_q_heads + 2 * qa.n_kv_heads) * qa.head_dim) return KV_ERR_SHAPE;
  }
  if ((k % 8) != 0 || (lda % 8) != 0 || (n % 8) != 0) return KV_ERR_SHAPE;
  if (((uintptr_t)a & 15) || ((uintptr_t)w & 15) || ((uintptr_t)out & 15) || ((uintptr_t)resid & 15)) return KV_ERR_ARG;
  const int sms = sm_count(current_device());
  const int bn = pick_bn(m, n, sms, mode, mode == GEMM_QKV_ROPE ? qa.head_dim : 0);
  CUtensorMap ta, tb;
  int rc = tc::make_tmap_2d(&ta, a, m, k, lda, BM);
  if (rc != KV_OK) return rc;
  const long long w_rows = (mode == GEMM_SWIGLU) ? 2ll * n : n;
  rc = tc::make_tmap_2d(&tb, w, w_rows, k, k, (mode == GEMM_SWIGLU) ? bn / 2 : bn);
  if (rc != KV_OK) return rc;
  DeviceStatus *status = reinterpret_cast<DeviceStatus *>(status_dev);
#define KV_GEMM_CASE(MODE_, BN_) \
  if (mode == MODE_ && bn == BN_) return launch_gemm<MODE_, BN_>(ta, tb, m, n, k, out, resid, status, qa, sms, st)
  KV_GEMM_CASE(GEMM_RESID_F32, 256);
  KV_GEMM_CASE(GEMM_RESID_F32, 224);
  KV_GEMM_CASE(GEMM_RESID_F32, 192);
  KV_GEMM_CASE(GEMM_RESID_F32, 160);
  KV_GEMM_CASE(GEMM_RESID_F32, 128);
  KV_GEMM_CASE(GEMM_STORE_BF16, 256);
  KV_GEMM_CASE(GEMM_STORE_BF16, 224);
  KV_GEMM_CASE(GEMM_STORE_BF16, 192);
  KV_GEMM_CASE(GEMM_STORE_BF16, 160);
  KV_GEMM_CASE(GEMM_STORE_BF16, 128);
  KV_GEMM_CASE(GEMM_SWIGLU, 256);
  KV_GEMM_CASE(GEMM_SWIGLU, 192);
  KV_GEMM_CASE(GEMM_SWIGLU, 128);
  KV_GEMM_CASE(GEMM_QKV_ROPE, 256);
  KV_GEMM_CASE(GEMM_QKV_ROPE, 192);
  KV_GEMM_CASE(GEMM_QKV_ROPE, 128);
#undef KV_GEMM_CASE
  return KV_ERR_ARG;
}

}  // namespace kvr
