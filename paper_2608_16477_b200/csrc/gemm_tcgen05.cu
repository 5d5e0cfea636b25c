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

#include "tc_common.cuh"

namespace kvr {

namespace {

constexpr int BM = 128;
constexpr int BK = 64;       // 128 bytes of bf16: one swizzle atom
constexpr int kABytes = BM * BK * 2;            // 16 KiB
constexpr int kTmemCols = 512;
constexpr int kTmemBufStride = 256;             // the two accumulators sit at columns 0 and 256
constexpr int kThreads = 192;
constexpr int kMaxSmem = 232448;                // 227 KiB per CTA
constexpr int kEpiStageBytes = 4 * 32 * 8 * 4;  // per epilogue warp: a 32-row x 8-column fp32 transpose buffer (1 KiB)

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

#ifdef KV_GEMM_TRACE
__device__ long long g_gemm_trace[64 * 8];
#define KV_TRACE(slot, idx) \
  do { if (blockIdx.x == 0 && (idx) < 64) g_gemm_trace[(idx) * 8 + (slot)] = clock64(); } while (0)
#else
#define KV_TRACE(slot, idx) do { } while (0)
#endif

enum WaitTag { TAG_EMPTY = 1, TAG_FULL = 2, TAG_TMEM_EMPTY = 3, TAG_TMEM_FULL = 4 };

__device__ __forceinline__ float silu_f(float a) { return a / (1.f + __expf(-a)); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&h);
}

__device__ __forceinline__ void store_chunk_bf16(bf16 *dst, const float (&v)[32]) {
  uint4 *d4 = reinterpret_cast<uint4 *>(dst);
#pragma unroll
  for (int q = 0; q < 4; ++q)
    d4[q] = make_uint4(pack_bf16(v[8 * q], v[8 * q + 1]), pack_bf16(v[8 * q + 2], v[8 * q + 3]),
                       pack_bf16(v[8 * q + 4], v[8 * q + 5]), pack_bf16(v[8 * q + 6], v[8 * q + 7]));
}

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
        KV_TRACE(0, (tile - (int)blockIdx.x) / (int)gridDim.x);
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
    if (lane == 0) {
      constexpr uint32_t idesc = tc::umma_idesc_bf16(BM, BN);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int local = 0;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++local) {
        const int buf = local & 1;
        const uint32_t acc_phase = (local >> 1) & 1;
        KV_TRACE(1, local);
        ok = tc::mbar_wait(tempty_bar(buf), acc_phase ^ 1, abort_flag, status, TAG_TMEM_EMPTY);
        if (!ok) break;
        KV_TRACE(2, local);
        tc::tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * kTmemBufStride;
        for (int kb = 0; kb < k_blocks; ++kb) {
          ok = tc::mbar_wait(full_bar(stage), phase, abort_flag, status, TAG_FULL);
          if (!ok) break;
          tc::tc_fence_after();
          const uint32_t a_s = smem_base + stage * kStageBytes;
          const uint64_t a_desc = tc::umma_desc_k128(a_s);
          const uint64_t b_desc = tc::umma_desc_k128(a_s + kABytes);
#pragma unroll
          for (int ks = 0; ks < BK / 16; ++ks)   // +32 bytes (2 descriptor units) per K=16 slice
            tc::umma_bf16(d_tmem, a_desc + 2 * ks, b_desc + 2 * ks, idesc, (kb | ks) != 0);
          tc::umma_commit(empty_bar(stage));
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (ok) tc::umma_commit(tfull_bar(buf));
        KV_TRACE(3, local);
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
      if (warp == 2 && lane == 0) KV_TRACE(4, local);
      ok = tc::mbar_wait(tfull_bar(buf), acc_phase, abort_flag, status, TAG_TMEM_FULL);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (warp == 2 && lane == 0) KV_TRACE(5, local);
      tc::tc_fence_after();
      const int row = m0 + quarter * 32 + lane;
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * kTmemBufStride;
      if (MODE == GEMM_QKV_ROPE) {
        // columns of this tile are whole heads (head_dim divides 256); a head's pair (j, j + d/2) lies in
        // chunks c and c + d/64.  The row is token `row` of the call, at absolute position pos0 + row.
        const int d = qa.head_dim, half = d >> 1, pair = d >> 6;
        const bool live = row < m;
        long long slot_off = 0;
        int block = 0;
        if (live) {
          const int pos = qa.row_pos != nullptr ? qa.row_pos[row] : qa.pos0 + row;
          block = qa.row_block != nullptr ? qa.row_block[row] : qa.block_table[pos / qa.cache.block_size];
          slot_off = (long long)(pos % qa.cache.block_size) * qa.cache.n_kv_heads * d;
        }
        const float2 *cs_row = qa.rope + (long long)row * half;
        bf16 *orow = out + (long long)row * n;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          const int col = n0 + c * 32;
          if (col >= n) break;                       // uniform across the warp
          const int head = col / d, j0 = col - head * d;
          if (head < qa.n_q_heads + qa.n_kv_heads) {
            if (j0 >= half) continue;                // second half of a pair: written with its partner
            uint32_t lo[32], hi[32];
            tc::tmem_ld32(t_row + c * 32, lo);
            tc::tmem_ld32(t_row + (c + pair) * 32, hi);
            tc::tmem_ld_wait();
            if (live) {
              float a[32], b[32];
#pragma unroll
              for (int i = 0; i < 32; ++i) {
                const float2 cs = cs_row[j0 + i];
                const float x = __uint_as_float(lo[i]), y = __uint_as_float(hi[i]);
                a[i] = x * cs.x - y * cs.y;
                b[i] = y * cs.x + x * cs.y;
              }
              store_chunk_bf16(orow + col, a);
              store_chunk_bf16(orow + col + half, b);
              if (head >= qa.n_q_heads) {
                bf16 *kp = reinterpret_cast<bf16 *>(qa.cache.page(qa.layer, 0, block)) + slot_off +
                           (head - qa.n_q_heads) * d + j0;
                store_chunk_bf16(kp, a);
                store_chunk_bf16(kp + half, b);
              }
            }
          } else {
            uint32_t r[32];
            tc::tmem_ld32(t_row + c * 32, r);
            tc::tmem_ld_wait();
            if (live) {
              float v[32];
#pragma unroll
              for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
              store_chunk_bf16(orow + col, v);
              bf16 *vp = reinterpret_cast<bf16 *>(qa.cache.page(qa.layer, 1, block)) + slot_off +
                         (head - qa.n_q_heads - qa.n_kv_heads) * d + j0;
              store_chunk_bf16(vp, v);
            }
          }
        }
      } else if (MODE == GEMM_SWIGLU) {
#pragma unroll 1
        for (int c = 0; c < (BN / 2) / 32; ++c) {
          uint32_t g[32], u[32];
          tc::tmem_ld32(t_row + c * 32, g);
          tc::tmem_ld32(t_row + BN / 2 + c * 32, u);
          tc::tmem_ld_wait();
          const int col = n0 + c * 32;
          if (row < m && col < n) {
            uint32_t packed[16];
#pragma unroll
            for (int j = 0; j < 16; ++j)
              packed[j] = pack_bf16(silu_f(__uint_as_float(g[2 * j])) * __uint_as_float(u[2 * j]),
                                    silu_f(__uint_as_float(g[2 * j + 1])) * __uint_as_float(u[2 * j + 1]));
            uint4 *dst = reinterpret_cast<uint4 *>(out + (long long)row * n + col);
#pragma unroll
            for (int v = 0; v < 4; ++v)
              if (col + v * 8 < n) dst[v] = make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]);
          }
        }
      } else if (MODE == GEMM_RESID_F32) {
        // x[row, col..] += acc.  A thread owns a row of the accumulator, but rows are 4 * n bytes apart in
        // memory and a thread-per-row update would touch half a 32-byte sector per row and instruction.
        // Each warp therefore transposes 32 rows x 8 columns at a time through a 1 KiB shared-memory buffer
        // and updates x with two lanes per row: every instruction then moves whole 32-byte sectors of 16 rows.
        float4 *stage = reinterpret_cast<float4 *>(smem_gen + kStages * kStageBytes + 256) + (warp - 2) * 64;
        const int sub_row = lane >> 1, c4 = lane & 1;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          const int col = n0 + c * 32;
          if (col >= n) break;
          uint32_t r[32];
          tc::tmem_ld32(t_row + c * 32, r);
          tc::tmem_ld_wait();
#pragma unroll
          for (int s8 = 0; s8 < 4; ++s8) {         // 8 columns per pass
            const int scol = col + s8 * 8 + c4 * 4;
            // stage[row][2 chunks], chunk index XORed with bit 2 of the row: conflict-free both ways
            stage[lane * 2 + (0 ^ ((lane >> 2) & 1))] =
                make_float4(__uint_as_float(r[8 * s8]), __uint_as_float(r[8 * s8 + 1]), __uint_as_float(r[8 * s8 + 2]),
                            __uint_as_float(r[8 * s8 + 3]));
            stage[lane * 2 + (1 ^ ((lane >> 2) & 1))] =
                make_float4(__uint_as_float(r[8 * s8 + 4]), __uint_as_float(r[8 * s8 + 5]),
                            __uint_as_float(r[8 * s8 + 6]), __uint_as_float(r[8 * s8 + 7]));
            __syncwarp();
#pragma unroll
            for (int it = 0; it < 2; ++it) {
              const int rr = it * 16 + sub_row;
              const int grow = m0 + quarter * 32 + rr;
              if (grow < m && scol < n) {
                const float4 a4 = stage[rr * 2 + (c4 ^ ((rr >> 2) & 1))];
                float4 *px = reinterpret_cast<float4 *>(resid + (long long)grow * n + scol);
                float4 x = __ldcs(px);
                x.x += a4.x; x.y += a4.y; x.z += a4.z; x.w += a4.w;
                *px = x;
              }
            }
            __syncwarp();
          }
        }
      } else {
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          uint32_t r[32];
          tc::tmem_ld32(t_row + c * 32, r);
          tc::tmem_ld_wait();
          const int col = n0 + c * 32;
          if (row < m && col < n) {
            uint4 *dst = reinterpret_cast<uint4 *>(out + (long long)row * n + col);
#pragma unroll
            for (int v = 0; v < 4; ++v)
              if (col + v * 8 < n)
                dst[v] = make_uint4(pack_bf16(__uint_as_float(r[8 * v]), __uint_as_float(r[8 * v + 1])),
                                    pack_bf16(__uint_as_float(r[8 * v + 2]), __uint_as_float(r[8 * v + 3])),
                                    pack_bf16(__uint_as_float(r[8 * v + 4]), __uint_as_float(r[8 * v + 5])),
                                    pack_bf16(__uint_as_float(r[8 * v + 6]), __uint_as_float(r[8 * v + 7])));
          }
        }
      }
      tc::tc_fence_before();
      tc::mbar_arrive(tempty_bar(buf));
      if (warp == 2 && lane == 0) KV_TRACE(6, local);
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
  const double eff[5] = {1.00, 0.97, 0.92, 0.85, 0.75};     // measured: narrower tiles re-read A more often and
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
  if (((uintptr_t)a & 15) || ((uintptr_t)w & 15)) return KV_ERR_ARG;
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
  KV_GEMM_CASE(GEMM_QKV_ROPE, 128);
#undef KV_GEMM_CASE
  return KV_ERR_ARG;
}

#ifdef KV_GEMM_TRACE
extern "C" int kv_debug_gemm_trace(long long *out_host) {
  return cudaMemcpyFromSymbol(out_host, g_gemm_trace, sizeof(long long) * 64 * 8) == cudaSuccess ? 0 : -13;
}
#endif

}  // namespace kvr
