// Causal GQA flash attention for prefill on the 5th-generation tensor cores (head_dim 64 or 128).
// The qkv buffer holds one row per context position: rows [0, pos0) carry the K/V of an already cached
// prefix (gathered from its pages), rows [pos0, pos0 + T) the chunk's post-RoPE Q, K and V.
//
// A work item is ONE 128-row query tile of TWO query heads that share a KV head (tiles "a" and "b"), so
// every K/V tile fetched by TMA feeds both.  A KV head with an odd number of query heads pairs its last
// query head with itself: both tiles then compute and store the same rows.
//
//   warp 0      TMA producer of Q (once per item) and of the K and V tiles (128 keys each).
//   warps 1, 2  S = Q K^T of tile a and of tile b (both operands K-major in shared memory); warp 1 also
//               allocates TMEM.  The whole warp runs the loop, one elected lane issues each tcgen05.mma.
//   warp 3      O += P V of both tiles (P read from TMEM, V as an MN-major shared-memory operand: no
//               transposes).
//   warps 4-7   softmax of tile a, warps 8-11 softmax of tile b: one thread per query row (= TMEM lane).
//               The row of S is read once into registers (setmaxnreg moves registers from warps 0-3 to the
//               softmax warps) and the S columns are handed back at once: the two tiles take turns on ONE
//               score buffer, and each has its own columns for the bf16 probabilities, so the scores of a
//               tile's NEXT key tile are computed while this one is exponentiated.
//               Statistics stay in fp32; the running maximum is only advanced (and O rescaled in TMEM) when
//               it grows by more than 8 in the log2 domain, which keeps exp2 arguments <= 8 and makes
//               rescaling rare.
// Per key tile a softmax warpgroup therefore waits only for things issued most of a step earlier (S of this
// tile, P V of the previous one); the tensor pipe and the exponentials overlap instead of alternating.
// TMEM columns: S [0,128)  P_a [128,192)  P_b [192,256)  O_a [256,256+D)  O_b [384,384+D).
// The kernel is persistent: one CTA per SM walks a list of work items (row tile, head pair), heaviest row tiles
// first (causal work grows with the row tile index); the pipeline keeps running across items.
// Every mbarrier wait is bounded; a wait that runs out is recorded in the status block and the CTA drains.
#include "tc_common.cuh"

namespace kvr {

namespace {

constexpr int kBM = 128;            // query rows per tile
constexpr int kBN = 128;            // keys per KV tile
constexpr int kAttnThreads = 384;   // 12 warps
constexpr uint32_t kTmemS = 0, kTmemP0 = 128, kTmemP1 = 192, kTmemO0 = 256, kTmemO1 = 384;
constexpr float kRescaleThreshold = 8.0f;
// setmaxnreg moves registers inside the pool the CTA was launched with (threads x registers per thread as
// compiled), and setmaxnreg.inc blocks, with no timeout, until the registers it asks for have been released.
// The launcher therefore checks 256 x (kRegsSoftmax - compiled) <= 128 x (compiled - kRegsOther) before the
// first launch and refuses to launch otherwise (compiled = 168 here: 256 x 48 = 128 x 96).
constexpr int kRegsOther = 72;      // registers per thread of warps 0-3 after the hand-back
constexpr int kRegsSoftmax = 216;   // registers per thread of the softmax warps

enum AttnTag { ATAG_Q = 11, ATAG_K_EMPTY = 12, ATAG_K = 13, ATAG_V = 14, ATAG_S = 15, ATAG_P = 16, ATAG_O = 17,
               ATAG_V_EMPTY = 18, ATAG_S_FREE = 19, ATAG_PV = 20, ATAG_QK_ISSUED = 21 };

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

// MN-major shared-memory operand (V: keys are the K dimension, head dims contiguous), 128-byte swizzle:
// 8-key groups are 1024 bytes apart (stride byte offset), 64-dim column blocks `lbo_bytes` apart.
__device__ __forceinline__ uint64_t umma_desc_mn128(uint32_t smem_addr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);
  d |= (uint64_t)(lbo_bytes >> 4) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&h);
}

// ---- packed fp32 pairs (two floats in one 64-bit register pair, one instruction for both) and 3-input max:
// they halve the instruction count of the softmax's scaling, row sums and running maximum.
__device__ __forceinline__ uint64_t pk2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpk2(uint64_t v, float &lo, float &hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t add2_rm(uint64_t a, uint64_t b) {      // rounds towards minus infinity
  uint64_t d;
  asm("add.rm.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 2^x for a pair on the FMA and integer pipes instead of the special-function unit: x = n + f with n = floor(x)
// (taken from the mantissa of x + 1.5 * 2^23 added with rounding towards minus infinity) and f in [0, 1),
// 2^f by a cubic (coefficients fitted for minimal relative error with p(0) = 1 and p(1) = 2: 1.0e-4, twenty times
// below the bf16 rounding the probabilities get anyway), then n is added into the exponent field.  Arguments are
// clamped at -126, so masked scores (minus infinity) come out as 2^-126 instead of 0: eight orders of magnitude
// below anything a bf16 sum or product can notice.
constexpr int kPolyPairs = 4;     // pairs per 16-pair chunk whose exponentials take this path (a quarter of all:
                                  // measured best among 0, 2, 4, 6, 8 and 16)
__device__ __forceinline__ void exp2_pair_fma(uint64_t x2, float &p0, float &p1) {
  float x0, x1;
  unpk2(x2, x0, x1);
  const uint64_t xc = pk2(fmaxf(x0, -126.f), fmaxf(x1, -126.f));
  const uint64_t magic = pk2(12582912.f, 12582912.f);
  const uint64_t t = add2_rm(xc, magic);
  const uint64_t f = sub2(xc, sub2(t, magic));
  uint64_t p = fma2(f, pk2(0.07826797f, 0.07826797f), pk2(0.22630768f, 0.22630768f));
  p = fma2(p, f, pk2(0.69542435f, 0.69542435f));
  p = fma2(p, f, pk2(1.f, 1.f));
  float q0, q1, t0, t1;
  unpk2(p, q0, q1);
  unpk2(t, t0, t1);
  p0 = __int_as_float(__float_as_int(q0) + (__float_as_int(t0) << 23));
  p1 = __int_as_float(__float_as_int(q1) + (__float_as_int(t1) << 23));
}

// Shared memory: two Q tiles, a ring of K tiles and a ring of V tiles.
template <int D>
struct AttnSmem {
  static constexpr int kKStages = 2;
  static constexpr int kVStages = 2;
  static constexpr int kTileBytes = kBM * D * 2;                 // one Q, K or V tile
  static constexpr int kQOff = 0;
  static constexpr int kKOff = 2 * kTileBytes;
  static constexpr int kVOff = kKOff + kKStages * kTileBytes;
  static constexpr int kStageOff = kVOff + kVStages * kTileBytes;  // 2 KiB per softmax warp: output transposition
  static constexpr int kBarOff = kStageOff + 8 * 2048;
  static constexpr int kBytes = kBarOff + 256 + 1024;            // barriers + alignment slack
};

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_prefill_tc_kernel(const __grid_constant__ CUtensorMap tma_qkv, int n_tokens, int pos0, int n_q_heads,
                            int n_kv_heads, float scale_log2, bf16 *__restrict__ out, DeviceStatus *status) {
  using L = AttnSmem<D>;
  constexpr int kAtoms = D / 64;                   // 64-column (128-byte) boxes per tile row
  constexpr int kBoxBytes = kBM * 128;             // one 128-row x 64-col box
  constexpr int kKS = L::kKStages, kVS = L::kVStages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *smem_gen = smem_raw + (smem_base - tc::smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + L::kBarOff;
  // barriers, two of each: Q full, K full, V full, K empty, V empty, S full, S free, P ready, P V done, Q K^T issued,
  // O free (read by the epilogue), and one Q empty
  enum { B_Q = 0, B_K = 1, B_V = 2, B_K_EMPTY = 3, B_V_EMPTY = 4, B_S = 5, B_S_FREE = 6, B_P = 7, B_PV = 8, B_QK_ISSUED = 9,
         B_O_FREE = 10, B_Q_EMPTY = 11, B_GROUPS = 12 };
  auto bar = [&](int group, int idx) { return bar_base + 8u * (group * 2 + idx); };
  uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(smem_gen + L::kBarOff + 8 * 2 * B_GROUPS);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int group = n_q_heads / n_kv_heads;
  const int pairs_per_group = (group + 1) / 2;
  const int pairs = n_kv_heads * pairs_per_group;
  const int m_tiles = (n_tokens + kBM - 1) / kBM;
  const int n_items = m_tiles * pairs;
  const int n_ctx = pos0 + n_tokens;
  // Work items (row tile, head pair), heaviest row tiles first.
  // Every role walks the same list and keeps running counters, so the pipeline never drains between items: the
  // loads and the first Q K^T of the next item run under the last step and the epilogue of this one.
  // The k-th item of this CTA: rounds of gridDim.x items, walked forwards in even rounds and backwards in odd ones,
  // so that the CTA with the heaviest item of one round gets the lightest of the next (the list is sorted).
  auto item_of = [&](int k) {
    const int base = k * (int)gridDim.x;
    return base + ((k & 1) ? (int)gridDim.x - 1 - (int)blockIdx.x : (int)blockIdx.x);
  };
  struct Item {
    int m0, n_kv, head_a, head_b, q_col0, q_col1, k_col, v_col;
  };
  auto get_item = [&](int it) {
    Item w;
    const int m_tile = m_tiles - 1 - it / pairs;
    const int pair = it % pairs;
    const int kv_head = pair / pairs_per_group;
    w.head_a = kv_head * group + 2 * (pair % pairs_per_group);
    w.head_b = min(w.head_a + 1, kv_head * group + group - 1);
    w.m0 = m_tile * kBM;                                    // first chunk row of this tile
    // causal: key tiles up to the one holding the last row's own position
    w.n_kv = min((n_ctx + kBN - 1) / kBN, (pos0 + w.m0 + kBM - 1) / kBN + 1);
    w.q_col0 = w.head_a * D;
    w.q_col1 = w.head_b * D;
    w.k_col = (n_q_heads + kv_head) * D;
    w.v_col = (n_q_heads + n_kv_heads + kv_head) * D;
    return w;
  };

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      tc::mbar_init(bar(B_Q, i), 1);
      tc::mbar_init(bar(B_K, i), 1);
      tc::mbar_init(bar(B_V, i), 1);
      tc::mbar_init(bar(B_K_EMPTY, i), 2);     // one arrival per Q K^T issuer
      tc::mbar_init(bar(B_V_EMPTY, i), 1);
      tc::mbar_init(bar(B_S, i), 1);
      tc::mbar_init(bar(B_S_FREE, i), 128);
      tc::mbar_init(bar(B_P, i), 128);
      tc::mbar_init(bar(B_PV, i), 1);
      tc::mbar_init(bar(B_QK_ISSUED, i), 1);
      tc::mbar_init(bar(B_O_FREE, i), 128);
    }
    tc::mbar_init(bar(B_Q_EMPTY, 0), 2);       // one arrival per Q K^T issuer, after its last MMA of an item
    *abort_flag = 0;
    tc::fence_barrier_init();
  }
  if (warp == 1) tc::tmem_alloc(tc::smem_u32(tmem_holder), 512);
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  // the softmax warpgroups hold a full row of S in registers; warps 0-3 give registers back (first statement
  // of every role so the register budget of each branch is known at compile time)
  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer: Q, then K and V tiles
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
    if (lane == 0) {
      tc::tma_prefetch_desc(&tma_qkv);
      int lk = 0, lv = 0;                       // K and V tiles loaded so far (ring positions)
      bool ok = true;
      for (int k = 0, it = item_of(0); it < n_items && ok; it = item_of(++k)) {
        const Item w = get_item(it);
        auto load_k = [&](int j) {
          const int st = lk % kKS;
          if (!tc::mbar_wait(bar(B_K_EMPTY, st), ((lk / kKS) & 1) ^ 1, abort_flag, status, ATAG_K_EMPTY)) return false;
          const uint32_t k_s = smem_base + L::kKOff + st * L::kTileBytes;
          tc::mbar_expect_tx(bar(B_K, st), L::kTileBytes);
          for (int a = 0; a < kAtoms; ++a)
            tc::tma_load_2d(k_s + a * kBoxBytes, &tma_qkv, w.k_col + a * 64, j * kBN, bar(B_K, st));
          ++lk;
          return true;
        };
        auto load_v = [&](int j) {
          const int st = lv % kVS;
          if (!tc::mbar_wait(bar(B_V_EMPTY, st), ((lv / kVS) & 1) ^ 1, abort_flag, status, ATAG_V_EMPTY)) return false;
          const uint32_t v_s = smem_base + L::kVOff + st * L::kTileBytes;
          tc::mbar_expect_tx(bar(B_V, st), L::kTileBytes);
          for (int a = 0; a < kAtoms; ++a)
            tc::tma_load_2d(v_s + a * kBoxBytes, &tma_qkv, w.v_col + a * 64, j * kBN, bar(B_V, st));
          ++lv;
          return true;
        };
        // the Q tiles may be replaced once the last Q K^T of the previous item has run
        ok = tc::mbar_wait(bar(B_Q_EMPTY, 0), (k & 1) ^ 1, abort_flag, status, ATAG_Q);
        if (!ok) break;
        for (int t = 0; t < 2; ++t) {
          tc::mbar_expect_tx(bar(B_Q, t), L::kTileBytes);
          for (int a = 0; a < kAtoms; ++a)
            tc::tma_load_2d(smem_base + L::kQOff + t * L::kTileBytes + a * kBoxBytes, &tma_qkv,
                            (t == 0 ? w.q_col0 : w.q_col1) + a * 64, pos0 + w.m0, bar(B_Q, t));
        }
        // in the order the tiles are consumed: K_0, then K_{j+1} before V_j
        ok = load_k(0);
        for (int j = 0; j < w.n_kv && ok; ++j) {
          if (j + 1 < w.n_kv) ok = load_k(j + 1);
          if (ok) ok = load_v(j);
        }
      }
    }
  } else if (warp == 1 || warp == 2) {
    // ---------------------------------------------------------------- MMA issuers: S = Q K^T, warp 1 for tile a,
    // warp 2 for tile b.  While a warp issues tcgen05.mma with shared-memory operands, the other warps of its
    // scheduler get fewer issue slots; one issuer per tile spreads that over two schedulers, and the P V issuer
    // sits on a third.
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
    {
      // every lane waits, and the outcome is made uniform so that the warp stays converged for elect.sync
      auto wwait = [&](uint32_t b_, uint32_t parity, volatile int *af, DeviceStatus *st_, int tag) {
        return __all_sync(0xffffffffu, tc::mbar_wait(b_, parity, af, st_, tag)) != 0;
      };
      constexpr uint32_t idesc_qk = tc::umma_idesc_bf16(kBM, kBN);
      const uint32_t s_tmem = tmem_base + kTmemS;
      const int t = warp - 1;
      const uint32_t q_s = smem_base + L::kQOff + t * L::kTileBytes;
      // The score buffer is used in the order a_0 b_0 a_1 b_1 ... (across items too): each use starts once the
      // previous user (the other tile) has taken its scores into registers (S free).
      int s = 0;                                // key-tile steps so far, over all items
      bool ok = true;
      for (int k = 0, it = item_of(0); it < n_items && ok; it = item_of(++k)) {
        const int n_kv = get_item(it).n_kv;
        ok = wwait(bar(B_Q, t), k & 1, abort_flag, status, ATAG_Q);
        for (int j = 0; j < n_kv && ok; ++j, ++s) {
          const int kst = s % kKS;
          ok = wwait(bar(B_K, kst), (s / kKS) & 1, abort_flag, status, ATAG_K);
          if (ok && s + t > 0) ok = wwait(bar(B_S_FREE, t ^ 1), (t == 0 ? s - 1 : s) & 1, abort_flag, status, ATAG_S_FREE);
          if (!ok) break;
          tc::tc_fence_after();
          const uint32_t k_s = smem_base + L::kKOff + kst * L::kTileBytes;
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            const uint32_t off = (ks / 4) * kBoxBytes + (ks % 4) * 32;
            tc::umma_bf16_warp(s_tmem, tc::umma_desc_k128(q_s + off), tc::umma_desc_k128(k_s + off), idesc_qk, ks != 0);
          }
          tc::umma_commit_warp(bar(B_S, t));
          tc::umma_commit_warp(bar(B_K_EMPTY, kst));      // second of the two arrivals frees the K stage
          if (j == n_kv - 1) tc::umma_commit_warp(bar(B_Q_EMPTY, 0));
          if (lane == 0) tc::mbar_arrive(bar(B_QK_ISSUED, t));   // tells the P V issuer that these MMAs are queued
          __syncwarp();
        }
      }
    }
  } else if (warp == 3) {
    // ---------------------------------------------------------------- MMA issuer: O += P V
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
    {
      auto wwait = [&](uint32_t b_, uint32_t parity, volatile int *af, DeviceStatus *st_, int tag) {
        return __all_sync(0xffffffffu, tc::mbar_wait(b_, parity, af, st_, tag)) != 0;
      };
      constexpr uint32_t idesc_pv = tc::umma_idesc_bf16(kBM, D) | (1u << 16);   // B (= V) is MN-major
      const uint32_t p_tmem[2] = {tmem_base + kTmemP0, tmem_base + kTmemP1};
      const uint32_t o_tmem[2] = {tmem_base + kTmemO0, tmem_base + kTmemO1};
      int s = 0;
      bool ok = true;
      for (int k = 0, it = item_of(0); it < n_items && ok; it = item_of(++k)) {
        const int n_kv = get_item(it).n_kv;
        for (int j = 0; j < n_kv && ok; ++j, ++s) {
          const int vst = s % kVS;
          ok = wwait(bar(B_V, vst), (s / kVS) & 1, abort_flag, status, ATAG_V);
          const uint32_t v_s = smem_base + L::kVOff + vst * L::kTileBytes;
          for (int t = 0; t < 2 && ok; ++t) {
            ok = wwait(bar(B_P, t), s & 1, abort_flag, status, ATAG_P);
            // The tile's softmax warps take their next scores into registers right after handing over P, and that
            // releases the score buffer for the OTHER tile's Q K^T (key tile j + 1 for tile b, j + 2 for tile a).
            // The tensor pipe runs MMAs in issue order and the score buffer is what both tiles wait for, so P V
            // is queued behind that Q K^T, not in front of it (inside an item; at its end P V must not wait).
            const int j_qk = j + 1 + t;
            if (ok && j_qk < n_kv) ok = wwait(bar(B_QK_ISSUED, t ^ 1), (s + 1 + t) & 1, abort_flag, status, ATAG_QK_ISSUED);
            // the first P V of an item overwrites O: the epilogue of the previous item must have read it
            if (ok && j == 0) ok = wwait(bar(B_O_FREE, t), (k & 1) ^ 1, abort_flag, status, ATAG_O);
            if (!ok) break;
            tc::tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < kBN / 16; ++ks)   // 16 keys per slice: 8 TMEM columns of P, 2048 bytes of V
              tc::umma_bf16_ts_warp(o_tmem[t], p_tmem[t] + ks * 8, umma_desc_mn128(v_s + ks * 2048, kBoxBytes), idesc_pv,
                                    (j | ks) != 0);
            tc::umma_commit_warp(bar(B_PV, t));
          }
          if (!ok) break;
          tc::umma_commit_warp(bar(B_V_EMPTY, vst));
        }
      }
    }
  } else {
    // ---------------------------------------------------------------- softmax warpgroups
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
    const int t = (warp - 4) >> 2;                 // 0: tile a, 1: tile b
    const int quarter = warp & 3;
    const int row_in_tile = quarter * 32 + lane;
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const uint32_t s_t = tmem_base + lane_base + kTmemS;
    const uint32_t p_t = tmem_base + lane_base + (t == 0 ? kTmemP0 : kTmemP1);
    const uint32_t o_t = tmem_base + lane_base + (t == 0 ? kTmemO0 : kTmemO1);
    int s = 0;                                     // key-tile steps so far, over all items
    bool ok = true;
    for (int k = 0, it = item_of(0); it < n_items && ok; it = item_of(++k)) {
      const Item w = get_item(it);
      const int m0 = w.m0, n_kv = w.n_kv;
      const int qi = pos0 + m0 + row_in_tile;      // absolute query position
      float m_ref = -INFINITY, l_sum = 0.f;
      for (int j = 0; j < n_kv; ++j, ++s) {
        ok = tc::mbar_wait(bar(B_S, t), s & 1, abort_flag, status, ATAG_S);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc::tc_fence_after();
        const bool diag = (j * kBN + kBN - 1 > pos0 + m0);   // tile reaches past the first row's position
        const int limit = qi - j * kBN;              // keys with column > limit are masked
        // the whole row of S (128 fp32) in registers: four loads in flight, one wait; then S may be overwritten
        uint32_t r0[32], r1[32], r2[32], r3[32];
        tc::tmem_ld32(s_t + 0, r0);
        tc::tmem_ld32(s_t + 32, r1);
        tc::tmem_ld32(s_t + 64, r2);
        tc::tmem_ld32(s_t + 96, r3);
        tc::tmem_ld_wait();
        tc::tc_fence_before();
        tc::mbar_arrive(bar(B_S_FREE, t));
        float mx = -INFINITY;
        if (diag) {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            if (i > limit) r0[i] = 0xff800000u;        // -inf
            if (32 + i > limit) r1[i] = 0xff800000u;
            if (64 + i > limit) r2[i] = 0xff800000u;
            if (96 + i > limit) r3[i] = 0xff800000u;
          }
        }
        {
          // four independent chains of 3-input maxima (16 dependent steps each instead of 64 in a row)
          float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            m0 = max3(m0, __uint_as_float(r0[i]), __uint_as_float(r0[i + 1]));
            m1 = max3(m1, __uint_as_float(r1[i]), __uint_as_float(r1[i + 1]));
            m2 = max3(m2, __uint_as_float(r2[i]), __uint_as_float(r2[i + 1]));
            m3 = max3(m3, __uint_as_float(r3[i]), __uint_as_float(r3[i + 1]));
          }
          mx = fmaxf(max3(m0, m1, m2), m3);
        }
        mx *= scale_log2;
        bool rescale = false;
        float factor = 1.f;
        if (j == 0) {
          m_ref = mx;
        } else if (mx > m_ref + kRescaleThreshold) {
          rescale = true;
          factor = exp2f(m_ref - mx);
          m_ref = mx;
          l_sum *= factor;
        }
        // probabilities as packed bf16 (two keys per 32-bit column); masked scores are -inf -> 0.  The whole row is
        // exponentiated before the wait for the P columns, so that the wait finds P V_{j-1} done.
        const uint64_t scale2 = pk2(scale_log2, scale_log2), neg_m2 = pk2(-m_ref, -m_ref);
        uint64_t sum2 = pk2(0.f, 0.f);
        auto exps = [&](const uint32_t (&r)[32], uint32_t (&pk)[16]) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const uint64_t x2 = fma2(pk2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1])), scale2, neg_m2);
            float p0, p1;
            if (i >= 16 - kPolyPairs) {
              exp2_pair_fma(x2, p0, p1);
            } else {
              float x0, x1;
              unpk2(x2, x0, x1);
              p0 = ex2_approx(x0);
              p1 = ex2_approx(x1);
            }
            sum2 = add2(sum2, pk2(p0, p1));
            pk[i] = pack2(p0, p1);
          }
        };
        auto store = [&](const uint32_t (&pk)[16], int c) { tmem_st16(p_t + c * 16, pk); };   // 32 keys
        uint32_t pk0[16], pk1[16], pk2[16], pk3[16];
        exps(r0, pk0);
        exps(r1, pk1);
        exps(r2, pk2);
        exps(r3, pk3);
        // P V of the previous key tile must be done before its P columns are overwritten or O is rescaled (for the
        // first key tile of an item the epilogue of the previous item has already waited for it)
        if (j > 0) {
          ok = tc::mbar_wait(bar(B_PV, t), (s - 1) & 1, abort_flag, status, ATAG_PV);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc::tc_fence_after();
        }
        if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll 1
          for (int c = 0; c < D / 32; ++c) {
            uint32_t r[32];
            tc::tmem_ld32(o_t + c * 32, r);
            tc::tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * factor);
            tmem_st32(o_t + c * 32, r);
          }
        }
        store(pk0, 0);
        store(pk1, 1);
        store(pk2, 2);
        store(pk3, 3);
        {
          float sum0, sum1;
          unpk2(sum2, sum0, sum1);
          l_sum += sum0 + sum1;
        }
        tc::tmem_st_wait();
        tc::tc_fence_before();
        tc::mbar_arrive(bar(B_P, t));
      }
      if (!ok) break;
      // ---- epilogue of the item: O / l -> bf16 rows.  O is taken into registers in one go and handed back, so
      // the next item's first P V does not wait for the stores.
      ok = tc::mbar_wait(bar(B_PV, t), (s - 1) & 1, abort_flag, status, ATAG_O);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc::tc_fence_after();
      uint32_t o_r[D / 32][32];
#pragma unroll
      for (int c = 0; c < D / 32; ++c) tc::tmem_ld32(o_t + c * 32, o_r[c]);
      tc::tmem_ld_wait();
      tc::tc_fence_before();
      tc::mbar_arrive(bar(B_O_FREE, t));
      const float inv = 1.f / l_sum;
      const int head = t == 0 ? w.head_a : w.head_b;
      // A thread owns a row, and rows are n_q_heads * D * 2 bytes apart in memory: stored directly, every
      // instruction would touch 32 different lines.  Each 32-column slab therefore goes through a 2 KiB
      // shared-memory buffer of the warp (16-byte pieces XOR-swizzled by the row), and is written out with four
      // lanes per row: every store instruction then covers 8 rows x 64 contiguous bytes.
      const uint32_t stage = smem_base + L::kStageOff + (uint32_t)((warp - 4) * 2048);
      const int rd_row = lane >> 2, rd_piece = lane & 3;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        __syncwarp();
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const uint32_t addr = stage + (uint32_t)lane * 64 + (uint32_t)((v ^ ((lane >> 1) & 3)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr),
                       "r"(pack2(__uint_as_float(o_r[c][8 * v]) * inv, __uint_as_float(o_r[c][8 * v + 1]) * inv)),
                       "r"(pack2(__uint_as_float(o_r[c][8 * v + 2]) * inv, __uint_as_float(o_r[c][8 * v + 3]) * inv)),
                       "r"(pack2(__uint_as_float(o_r[c][8 * v + 4]) * inv, __uint_as_float(o_r[c][8 * v + 5]) * inv)),
                       "r"(pack2(__uint_as_float(o_r[c][8 * v + 6]) * inv, __uint_as_float(o_r[c][8 * v + 7]) * inv))
                       : "memory");
        }
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int r = rd_row + 8 * i;                       // row inside this warp's 32
          const int out_row = m0 + quarter * 32 + r;          // row inside the chunk
          uint4 val;
          const uint32_t addr = stage + (uint32_t)r * 64 + (uint32_t)((rd_piece ^ ((r >> 1) & 3)) << 4);
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w) : "r"(addr));
          if (out_row < n_tokens)
            *reinterpret_cast<uint4 *>(out + (long long)out_row * n_q_heads * D + head * D + c * 32 + rd_piece * 8) = val;
        }
      }
    }
  }

  tc::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc::tc_fence_after();
    tc::tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

// Copies the cached prefix's K and V (positions [0, pos0)) of one layer from their pages into rows [0, pos0)
// of the qkv buffer, so the attention kernel's TMA map covers the whole context with one row pitch.
__global__ void __launch_bounds__(128) gather_prefix_kv_kernel(bf16 *__restrict__ qkv, int qkv_dim, int k_col,
                                                               int v_col, CacheView cache, int layer,
                                                               const int *__restrict__ block_table) {
  const int pos = blockIdx.x;
  const int block = block_table[pos / cache.block_size];
  const long long off = (long long)(pos % cache.block_size) * cache.n_kv_heads * cache.head_dim;
  const int vecs = cache.n_kv_heads * cache.head_dim / 8;
  const uint4 *ksrc = reinterpret_cast<const uint4 *>(reinterpret_cast<const bf16 *>(cache.page(layer, 0, block)) + off);
  const uint4 *vsrc = reinterpret_cast<const uint4 *>(reinterpret_cast<const bf16 *>(cache.page(layer, 1, block)) + off);
  uint4 *kdst = reinterpret_cast<uint4 *>(qkv + (long long)pos * qkv_dim + k_col);
  uint4 *vdst = reinterpret_cast<uint4 *>(qkv + (long long)pos * qkv_dim + v_col);
  for (int v = threadIdx.x; v < vecs; v += blockDim.x) {
    kdst[v] = ksrc[v];
    vdst[v] = vsrc[v];
  }
}

int gather_prefix_kv(bf16 *qkv_ctx, int pos0, int n_q_heads, int n_kv_heads, int head_dim, CacheView cache, int layer,
                     const int *block_table_dev, cudaStream_t st) {
  if (pos0 <= 0) return KV_OK;
  const int qkv_dim = (n_q_heads + 2 * n_kv_heads) * head_dim;
  gather_prefix_kv_kernel<<<pos0, 128, 0, st>>>(qkv_ctx, qkv_dim, n_q_heads * head_dim,
                                                (n_q_heads + n_kv_heads) * head_dim, cache, layer, block_table_dev);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

// head_dim 64 or 128.  qkv_ctx has pos0 + n_tokens rows (see the file header); out has n_tokens rows.
int attention_prefill_tc(const bf16 *qkv_ctx, int n_tokens, int pos0, int n_q_heads, int n_kv_heads, int head_dim,
                         bf16 *out, int *status_dev, cudaStream_t st) {
  if (n_tokens <= 0) return KV_OK;
  if ((head_dim != 64 && head_dim != 128) || n_kv_heads <= 0 || n_q_heads <= 0 || n_q_heads % n_kv_heads != 0)
    return KV_ERR_SHAPE;
  const int qkv_dim = (n_q_heads + 2 * n_kv_heads) * head_dim;
  CUtensorMap map;
  int rc = tc::make_tmap_2d(&map, qkv_ctx, pos0 + n_tokens, qkv_dim, qkv_dim, kBM);
  if (rc != KV_OK) return rc;
  static int regs_ok_dev[kMaxDevices] = {};   // 0: not checked, 1: ok, 2: unbalanced
  const int device = current_device();
  if (device < 0) return KV_ERR_CUDA;
  if (regs_ok_dev[device] == 0) {
    int regs_ok;
    KV_CUDA(cudaFuncSetAttribute(attention_prefill_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 AttnSmem<64>::kBytes));
    KV_CUDA(cudaFuncSetAttribute(attention_prefill_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 AttnSmem<128>::kBytes));
    // the register hand-over must balance inside the CTA's own pool, or setmaxnreg.inc would wait forever
    regs_ok = 1;
    cudaFuncAttributes fa;
    KV_CUDA(cudaFuncGetAttributes(&fa, attention_prefill_tc_kernel<64>));
    const int r64 = fa.numRegs;
    KV_CUDA(cudaFuncGetAttributes(&fa, attention_prefill_tc_kernel<128>));
    const int r128 = fa.numRegs;
    for (int compiled : {r64, r128}) {
      const int softmax_threads = kAttnThreads - 128;
      if (compiled < kRegsOther || softmax_threads * (kRegsSoftmax - compiled) > 128 * (compiled - kRegsOther)) regs_ok = 0;
    }
    regs_ok_dev[device] = regs_ok ? 1 : 2;
  }
  if (regs_ok_dev[device] != 1) return KV_ERR_SHAPE;
  const int m_tiles = (n_tokens + kBM - 1) / kBM;
  const int items = m_tiles * n_kv_heads * ((n_q_heads / n_kv_heads + 1) / 2);
  const int sms = sm_count(device);
  const int grid = items < sms ? items : sms;      // persistent: one CTA per SM walks the items
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)head_dim);
  DeviceStatus *status = reinterpret_cast<DeviceStatus *>(status_dev);
  if (head_dim == 64)
    attention_prefill_tc_kernel<64><<<grid, kAttnThreads, AttnSmem<64>::kBytes, st>>>(map, n_tokens, pos0, n_q_heads,
                                                                                     n_kv_heads, scale_log2, out, status);
  else
    attention_prefill_tc_kernel<128><<<grid, kAttnThreads, AttnSmem<128>::kBytes, st>>>(map, n_tokens, pos0, n_q_heads,
                                                                                       n_kv_heads, scale_log2, out, status);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

}  // namespace kvr
