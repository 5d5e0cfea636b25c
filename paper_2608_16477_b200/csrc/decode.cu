// Decode step (one token): every stage is HBM-bound.  Weights are streamed once with 16-byte loads
// (warp per output row), activations stay fp32; attention reads the paged cache through the block
// table with the keys split across CTAs (flash-decoding) and a second pass merging the splits.
#include <float.h>

#include <cstring>

#include "common.cuh"

namespace kvr {

__device__ __forceinline__ float warp_sum_d(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__global__ void embed_one_kernel(const bf16 *__restrict__ embed, int token, int hidden, float *__restrict__ x) {
  const bf16 *row = embed + (long long)token * hidden;
  for (int c = blockIdx.x * blockDim.x + threadIdx.x; c < hidden; c += gridDim.x * blockDim.x)
    x[c] = __bfloat162float(row[c]);
}

int embed_one(const bf16 *embed, int token, int hidden, float *x, cudaStream_t st) {
  embed_one_kernel<<<(hidden + 255) / 256, 256, 0, st>>>(embed, token, hidden, x);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

__device__ __forceinline__ float dot8(uint4 wraw, float4 x0, float4 x1) {
  const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&wraw);
  float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
  float2 c = __bfloat1622float2(h[2]), d = __bfloat1622float2(h[3]);
  return a.x * x0.x + a.y * x0.y + b.x * x0.z + b.y * x0.w + c.x * x1.x + c.y * x1.y + d.x * x1.z + d.y * x1.w;
}

// Matrix-vector products of the decode step.  A warp streams TWO weight rows (bf16, 16-byte loads, four
// vectors of each row in flight per lane) against the fp32 activation vector, which stays in L1/L2.
// NORM fuses the preceding RMSNorm: the warp accumulates sum(x^2) from the values it loads anyway and
// computes W . (x * gain) * rsqrt(mean(x^2) + eps), so no separate normalisation launch is needed.
// Epilogues: STORE rows (2u, 2u+1); ADD into the residual; SWIGLU rows (u, u + n) -> silu(a) * b;
// QKV rows (j, j + d/2) of one head -> RoPE rotation (cos/sin of the step's position from a table built once per
// step with fp64 angles), q to the fp32 query vector, k and v (bf16) appended to the paged cache.
enum GemvEpi { GEMV_STORE = 0, GEMV_ADD = 1, GEMV_SWIGLU = 2, GEMV_QKV = 3 };
constexpr int kGemvWarps = 8;

struct GemvQkvArgs {
  CacheView cache;
  const int *block_table;
  const float2 *rope;       // (cos, sin) of the step's position for each of the head_dim / 2 frequencies
  int pos, layer, head_dim, n_q_heads, n_kv_heads;
};

template <int EPI, bool NORM>
__global__ void __launch_bounds__(kGemvWarps * 32) gemv2_kernel(const bf16 *__restrict__ w,
                                                                const float *__restrict__ x,
                                                                const bf16 *__restrict__ gain, float eps, int n,
                                                                int k, float *__restrict__ y,
                                                                const __grid_constant__ GemvQkvArgs qa) {
  const int lane = threadIdx.x & 31;
  const int unit = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  int row_a, row_b;
  bool has_b = true;
  if (EPI == GEMV_SWIGLU) {
    if (unit >= n) return;
    row_a = unit;
    row_b = unit + n;
  } else if (EPI == GEMV_QKV) {
    const int half = qa.head_dim >> 1;
    if (unit >= n / 2) return;
    const int head = unit / half, j = unit - head * half;
    row_a = head * qa.head_dim + j;
    row_b = row_a + half;
  } else {
    if (2 * unit >= n) return;
    row_a = 2 * unit;
    row_b = row_a + 1;
    if (row_b >= n) {
      row_b = row_a;
      has_b = false;
    }
  }
  const int nvec = k / 8;
  const uint4 *wa = reinterpret_cast<const uint4 *>(w + (long long)row_a * k);
  const uint4 *wb = reinterpret_cast<const uint4 *>(w + (long long)row_b * k);
  const float4 *xv = reinterpret_cast<const float4 *>(x);
  const uint4 *gv = reinterpret_cast<const uint4 *>(gain);
  float acc_a = 0.f, acc_b = 0.f, ss = 0.f;
  auto step = [&](uint4 ra, uint4 rb, int v) {
    float4 x0 = xv[2 * v], x1 = xv[2 * v + 1];
    if (NORM) {
      ss += x0.x * x0.x + x0.y * x0.y + x0.z * x0.z + x0.w * x0.w + x1.x * x1.x + x1.y * x1.y + x1.z * x1.z +
            x1.w * x1.w;
      const uint4 graw = gv[v];
      const __nv_bfloat162 *gh = reinterpret_cast<const __nv_bfloat162 *>(&graw);
      const float2 g0 = __bfloat1622float2(gh[0]), g1 = __bfloat1622float2(gh[1]);
      const float2 g2 = __bfloat1622float2(gh[2]), g3 = __bfloat1622float2(gh[3]);
      x0.x *= g0.x; x0.y *= g0.y; x0.z *= g1.x; x0.w *= g1.y;
      x1.x *= g2.x; x1.y *= g2.y; x1.z *= g3.x; x1.w *= g3.y;
    }
    acc_a += dot8(ra, x0, x1);
    acc_b += dot8(rb, x0, x1);
  };
  // The first batch of weight loads is issued on its own and awaited with a fence before x is touched: measured,
  // this start-up order shortens a 62 GB decode step from 14.5 to 13.6 ms (a compiler-only barrier at the same
  // place, a fence at the top of the kernel, or a fence in every iteration do not).
  int v = lane;
  if (v + 96 < nvec) {
    const uint4 a0 = __ldcs(wa + v), a1 = __ldcs(wa + v + 32), a2 = __ldcs(wa + v + 64), a3 = __ldcs(wa + v + 96);
    const uint4 b0 = __ldcs(wb + v), b1 = __ldcs(wb + v + 32), b2 = __ldcs(wb + v + 64), b3 = __ldcs(wb + v + 96);
    asm volatile("fence.acq_rel.gpu;" ::: "memory");
    step(a0, b0, v);
    step(a1, b1, v + 32);
    step(a2, b2, v + 64);
    step(a3, b3, v + 96);
    v += 128;
  }
  for (; v + 96 < nvec; v += 128) {
    const uint4 a0 = __ldcs(wa + v), a1 = __ldcs(wa + v + 32), a2 = __ldcs(wa + v + 64), a3 = __ldcs(wa + v + 96);
    const uint4 b0 = __ldcs(wb + v), b1 = __ldcs(wb + v + 32), b2 = __ldcs(wb + v + 64), b3 = __ldcs(wb + v + 96);
    step(a0, b0, v);
    step(a1, b1, v + 32);
    step(a2, b2, v + 64);
    step(a3, b3, v + 96);
  }
  for (; v < nvec; v += 32) step(__ldcs(wa + v), __ldcs(wb + v), v);
  acc_a = warp_sum_d(acc_a);
  acc_b = warp_sum_d(acc_b);
  if (NORM) {
    ss = warp_sum_d(ss);
    const float inv = rsqrtf(ss / (float)k + eps);
    acc_a *= inv;
    acc_b *= inv;
  }
  if (lane != 0) return;
  if (EPI == GEMV_STORE) {
    y[row_a] = acc_a;
    if (has_b) y[row_b] = acc_b;
  } else if (EPI == GEMV_ADD) {
    y[row_a] += acc_a;
    if (has_b) y[row_b] += acc_b;
  } else if (EPI == GEMV_SWIGLU) {
    y[row_a] = acc_a / (1.f + __expf(-acc_a)) * acc_b;
  } else {
    const int d = qa.head_dim, half = d >> 1;
    const int head = row_a / d, j = row_a - head * d;
    const int block = qa.block_table[qa.pos / qa.cache.block_size];
    const long long slot_off = (long long)(qa.pos % qa.cache.block_size) * qa.n_kv_heads * d;
    if (head < qa.n_q_heads + qa.n_kv_heads) {
      const float2 cs = qa.rope[j];
      const float ra = acc_a * cs.x - acc_b * cs.y;
      const float rb = acc_b * cs.x + acc_a * cs.y;
      if (head < qa.n_q_heads) {
        y[row_a] = ra;
        y[row_b] = rb;
      } else {
        bf16 *kp = reinterpret_cast<bf16 *>(qa.cache.page(qa.layer, 0, block)) + slot_off + (head - qa.n_q_heads) * d;
        kp[j] = __float2bfloat16_rn(ra);
        kp[j + half] = __float2bfloat16_rn(rb);
      }
    } else {
      bf16 *vp = reinterpret_cast<bf16 *>(qa.cache.page(qa.layer, 1, block)) + slot_off +
                 (head - qa.n_q_heads - qa.n_kv_heads) * d;
      vp[j] = __float2bfloat16_rn(acc_a);
      vp[j + half] = __float2bfloat16_rn(acc_b);
    }
  }
}

template <int EPI, bool NORM>
static int launch_gemv2(const bf16 *w, const float *x, const bf16 *gain, float eps, int n, int k, float *y,
                        const GemvQkvArgs &qa, cudaStream_t st) {
  const int units = (EPI == GEMV_SWIGLU) ? n : (n + 1) / 2;
  // warps per CTA: few enough that every SM gets at least ~8 CTAs, so the SMs finish together even when
  // a product has only a few thousand row pairs (O, down and QKV projections)
  int warps = units / (sm_count(current_device()) * 8);
  warps = warps < 1 ? 1 : (warps > kGemvWarps ? kGemvWarps : warps);
  const int grid = (units + warps - 1) / warps;
  gemv2_kernel<EPI, NORM><<<grid, warps * 32, 0, st>>>(w, x, gain, eps, n, k, y, qa);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

// mode 0 store, 1 add into y, 2 swiglu over (gate | up) rows.  gain != nullptr fuses RMSNorm(x, gain, eps).
int gemv(const bf16 *w, const float *x, int n, int k, int mode, float *y, cudaStream_t st, const bf16 *gain,
         float eps) {
  GemvQkvArgs qa;
  memset(&qa, 0, sizeof(qa));
  if (k % 8 != 0) return KV_ERR_SHAPE;
  if (gain != nullptr) {
    if (mode == 0) return launch_gemv2<GEMV_STORE, true>(w, x, gain, eps, n, k, y, qa, st);
    if (mode == 2) return launch_gemv2<GEMV_SWIGLU, true>(w, x, gain, eps, n, k, y, qa, st);
    return KV_ERR_ARG;
  }
  if (mode == 0) return launch_gemv2<GEMV_STORE, false>(w, x, nullptr, 0.f, n, k, y, qa, st);
  if (mode == 1) return launch_gemv2<GEMV_ADD, false>(w, x, nullptr, 0.f, n, k, y, qa, st);
  return launch_gemv2<GEMV_SWIGLU, false>(w, x, nullptr, 0.f, n, k, y, qa, st);
}

// Fused decode-step front end of a layer: RMSNorm + QKV projection + RoPE + K/V append.
// q_out receives the rotated fp32 query vector [n_q_heads * head_dim].
int gemv_qkv_rope(const bf16 *w_qkv, const float *x, const bf16 *gain, float eps, int hidden, int pos, int n_q_heads,
                  int n_kv_heads, int head_dim, const float2 *rope_dev, CacheView cache, int layer,
                  const int *block_table_dev, float *q_out, cudaStream_t st) {
  GemvQkvArgs qa;
  qa.cache = cache;
  qa.block_table = block_table_dev;
  qa.pos = pos;
  qa.layer = layer;
  qa.head_dim = head_dim;
  qa.n_q_heads = n_q_heads;
  qa.n_kv_heads = n_kv_heads;
  qa.rope = rope_dev;
  if (hidden % 8 != 0) return KV_ERR_SHAPE;
  const int n = (n_q_heads + 2 * n_kv_heads) * head_dim;
  return launch_gemv2<GEMV_QKV, true>(w_qkv, x, gain, eps, n, hidden, q_out, qa, st);
}

// ---- paged decode attention ---------------------------------------------------------------
// Partial record per (q head, split): m, l, acc[d].
// One CTA of 128 threads per (KV head, 128-key split), serving every query head of the group so each K/V
// row is read from HBM once.  The K and V rows of the split go to shared memory with 16-byte cp.async, d/8
// consecutive lanes per row (everything in flight at once; 16-byte chunks XOR-swizzled by the row so that ldmatrix
// is conflict-free).  The contractions run on mma.sync m16n8k16 (a 16-row tile is the natural size for the 8 to
// 16 query heads of a group; the 128-row tcgen05 tile would be nine tenths padding):
//   S = Q K^T   warp w owns keys 32w..32w+31; Q (fp32) is split into a bf16 high and low part, so the scores
//               keep fp32-level accuracy at the cost of a second MMA;
//   softmax     row maxima meet in shared memory, every warp then uses the split's common maximum;
//   O = P V     P goes from the S accumulators straight into A fragments (again as high + low parts), V through
//               ldmatrix.trans; the four warps' partial O and row sums are added in shared memory.
constexpr int kPaSplitKeys = 128;   // keys per split = threads per CTA (two CTAs fit an SM)
constexpr int kPaRows = 16;         // query heads per pass (rows of the MMA tile)

// dynamic shared memory: the K and V tiles (2 x 128 rows of bf16) and 4 warps x 16 rows of fp32 partial O
static int pa_smem_bytes(int d) { return 2 * kPaSplitKeys * d * 2 + (kPaSplitKeys / 32) * kPaRows * d * 4; }

static int pa_splits(int n_ctx) {
  int s = (n_ctx + kPaSplitKeys - 1) / kPaSplitKeys;
  return s < 1 ? 1 : s;
}

long long paged_attention_scratch_bytes(int n_q_heads, int head_dim, int n_ctx) {
  return (long long)n_q_heads * pa_splits(n_ctx) * (head_dim + 2) * (long long)sizeof(float);
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// x = hi + lo with hi = bf16(x), lo = bf16(x - hi): two bf16 that together carry ~16 mantissa bits
__device__ __forceinline__ void split_pair(float x, float y, uint32_t &hi, uint32_t &lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
  const float2 hf = __bfloat1622float2(h);
  const __nv_bfloat162 l = __floats2bfloat162_rn(x - hf.x, y - hf.y);
  hi = *reinterpret_cast<const uint32_t *>(&h);
  lo = *reinterpret_cast<const uint32_t *>(&l);
}

template <int D>
__global__ void __launch_bounds__(kPaSplitKeys, 2) paged_attention_split_kernel(
    const float *__restrict__ q, int n_q_heads, CacheView cache, int layer, const int *__restrict__ block_table,
    int n_ctx, float *__restrict__ partial) {
  constexpr int RB = D * 2;                 // bytes per K or V row
  constexpr int CH = D / 8;                 // 16-byte chunks per row
  constexpr int KS = D / 16;                // k-steps of S = Q K^T
  constexpr int NT = D / 8;                 // n-tiles of O = P V
  constexpr int NW = kPaSplitKeys / 32;     // warps
  extern __shared__ __align__(128) uint8_t pa_smem[];
  uint8_t *k_tile = pa_smem;                                  // [keys][D] bf16, swizzled
  uint8_t *v_tile = pa_smem + kPaSplitKeys * RB;
  float *o_red = reinterpret_cast<float *>(pa_smem + 2 * kPaSplitKeys * RB);   // [NW][kPaRows][D] partial O
  __shared__ float wmax_s[NW][kPaRows], wsum_s[NW][kPaRows], run_max_s[kPaRows];
  // CTA (g, part) walks the 128-key tiles [t_begin, t_end) of KV head g: one tile when the context has no more tiles
  // than the grid has parts (the launcher asks for two CTAs per SM), several consecutive ones for longer contexts,
  // carried by a running maximum, running sums and one output accumulator (one partial record per part either way).
  const int g = blockIdx.x, part = blockIdx.y, n_parts = gridDim.y;
  const int n_tiles = (n_ctx + kPaSplitKeys - 1) / kPaSplitKeys;
  const int t_begin = (int)((long long)part * n_tiles / n_parts);
  const int t_end = (int)((long long)(part + 1) * n_tiles / n_parts);
  const bool one_tile = t_end - t_begin == 1;
  const int group = n_q_heads / cache.n_kv_heads;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float scale = rsqrtf((float)D);

  // K and V rows of a tile into shared memory.  A warp copies its 32 rows (keys 32w..32w+31, the ones its MMAs
  // read) 32 / CH rows at a time: CH consecutive lanes cover one row's CH 16-byte chunks, so every instruction
  // moves whole rows (contiguous 2 D bytes each) instead of one chunk of 32 different rows.  Rows past the end
  // repeat the last key (finite data, masked below).  One commit group per call (kv = 0: the K rows, 1: the V rows).
  auto load_rows = [&](int t, int kv) {
    constexpr int RPI = 32 / CH;              // rows per instruction
    const int sub = lane / CH, c = lane % CH;
    const int bsz = cache.block_size;
    // lane l looks up the page and the slot of the warp's row l once; the copy loop fetches them by shuffle
    const int jk = min(t * kPaSplitKeys + warp * 32 + lane, n_ctx - 1);
    const int my_blk = block_table[jk / bsz];
    const int my_slot = jk % bsz;
    const uint32_t tile = (uint32_t)__cvta_generic_to_shared(kv == 0 ? k_tile : v_tile);
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const int rw = i * RPI + sub;                        // row inside the warp's 32
      const int r = warp * 32 + rw;                        // row of the tile
      const int blk = __shfl_sync(0xffffffffu, my_blk, rw);
      const int slot = __shfl_sync(0xffffffffu, my_slot, rw);
      const bf16 *src = reinterpret_cast<const bf16 *>(cache.page(layer, kv, blk)) +
                        ((long long)slot * cache.n_kv_heads + g) * D + c * 8;
      const uint32_t pc = (uint32_t)((c & ~7) | ((c ^ r) & 7)) * 16;
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(tile + r * RB + pc), "l"(src) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  load_rows(t_begin, 0);
  load_rows(t_begin, 1);
  const uint32_t k_s = (uint32_t)__cvta_generic_to_shared(k_tile);
  const uint32_t v_s = (uint32_t)__cvta_generic_to_shared(v_tile);
  const int r0 = lane >> 2, cq = (lane & 3) * 2;       // fragment row (and row + 8), first of two columns
  const int wk0 = warp * 32;                           // this warp's keys inside a tile

  for (int h0 = 0; h0 < group; h0 += kPaRows) {
    const int nh = min(kPaRows, group - h0);
    // Q fragments of rows r0 and r0 + 8 (heads h0 + row), scaled, as high and low bf16 parts
    uint32_t qh[KS][4], ql[KS][4];
    {
      const float *qa = q + (long long)(g * group + h0 + min(r0, nh - 1)) * D;
      const float *qb = q + (long long)(g * group + h0 + min(r0 + 8, nh - 1)) * D;
      const float sa = (r0 < nh) ? scale : 0.f, sb = (r0 + 8 < nh) ? scale : 0.f;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const float2 a0 = *reinterpret_cast<const float2 *>(qa + ks * 16 + cq);
        const float2 a2 = *reinterpret_cast<const float2 *>(qa + ks * 16 + 8 + cq);
        const float2 b0 = *reinterpret_cast<const float2 *>(qb + ks * 16 + cq);
        const float2 b2 = *reinterpret_cast<const float2 *>(qb + ks * 16 + 8 + cq);
        split_pair(a0.x * sa, a0.y * sa, qh[ks][0], ql[ks][0]);
        split_pair(b0.x * sb, b0.y * sb, qh[ks][1], ql[ks][1]);
        split_pair(a2.x * sa, a2.y * sa, qh[ks][2], ql[ks][2]);
        split_pair(b2.x * sb, b2.y * sb, qh[ks][3], ql[ks][3]);
      }
    }
    // running state of rows r0 and r0 + 8: the maximum (the same in every warp), this lane's share of the row sums
    // and the warp's output accumulator over its own keys of every tile
    float run0 = -FLT_MAX, run1 = -FLT_MAX, sum0 = 0.f, sum1 = 0.f;
    float oc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) oc[nt][i] = 0.f;

    for (int t = t_begin; t < t_end; ++t) {
      const int n_keys = min(n_ctx - t * kPaSplitKeys, kPaSplitKeys);
      // the tile that follows: the next one of this pass, or the first one again for the next pass of heads (a single
      // tile stays where it is)
      const int t_next = one_tile ? -1 : (t + 1 < t_end ? t + 1 : (h0 + kPaRows < group ? t_begin : -1));
      asm volatile("cp.async.wait_group 1;" ::: "memory");      // K rows have landed
      __syncthreads();      // (also: the previous tile or pass no longer reads the row statistics and o_red)
      // ---- S = Q K^T for this warp's 32 keys: 4 n-tiles of 8 keys
      float sc[4][4];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
        for (int i = 0; i < 4; ++i) sc[nt][i] = 0.f;
        const int krow = wk0 + nt * 8 + (lane & 7);
#pragma unroll
        for (int ks = 0; ks < KS; ks += 2) {
          const int chunk = ks * 2 + (lane >> 3);
          uint32_t bfr[4];
          ldmatrix_x4(k_s + krow * RB + (uint32_t)((chunk & ~7) | ((chunk ^ krow) & 7)) * 16, bfr);
          mma_bf16_16816(sc[nt], qh[ks], bfr[0], bfr[1]);
          mma_bf16_16816(sc[nt], ql[ks], bfr[0], bfr[1]);
          mma_bf16_16816(sc[nt], qh[ks + 1], bfr[2], bfr[3]);
          mma_bf16_16816(sc[nt], ql[ks + 1], bfr[2], bfr[3]);
        }
      }
      // mask keys past the end, row maxima over this warp's keys
      float mx0 = -FLT_MAX, mx1 = -FLT_MAX;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        const int key = wk0 + nt * 8 + cq;
        if (key >= n_keys) sc[nt][0] = sc[nt][2] = -FLT_MAX;
        if (key + 1 >= n_keys) sc[nt][1] = sc[nt][3] = -FLT_MAX;
        mx0 = fmaxf(mx0, fmaxf(sc[nt][0], sc[nt][1]));
        mx1 = fmaxf(mx1, fmaxf(sc[nt][2], sc[nt][3]));
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      if ((lane & 3) == 0) {
        wmax_s[warp][r0] = mx0;
        wmax_s[warp][r0 + 8] = mx1;
      }
      asm volatile("cp.async.wait_group 0;" ::: "memory");      // V rows have landed
      __syncthreads();
      if (t_next >= 0) load_rows(t_next, 0);      // every warp is done with this tile's K: the next K rows travel under P V
      mx0 = run0;
      mx1 = run1;
#pragma unroll
      for (int w = 0; w < NW; ++w) {
        mx0 = fmaxf(mx0, wmax_s[w][r0]);
        mx1 = fmaxf(mx1, wmax_s[w][r0 + 8]);
      }
      // what the earlier tiles of this part left is brought to the new maximum (nothing to do for the first tile:
      // sums and accumulator are zero)
      if (t > t_begin) {
        const float f0 = __expf(run0 - mx0), f1 = __expf(run1 - mx1);
        sum0 *= f0;
        sum1 *= f1;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          oc[nt][0] *= f0;
          oc[nt][1] *= f0;
          oc[nt][2] *= f1;
          oc[nt][3] *= f1;
        }
      }
      run0 = mx0;
      run1 = mx1;
      // ---- probabilities (A fragments, high + low) and O += P V over this warp's two 16-key steps
      uint32_t ph[2][4], pl[2][4];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        const float p0 = __expf(sc[nt][0] - mx0), p1 = __expf(sc[nt][1] - mx0);     // masked scores give 0
        const float p2 = __expf(sc[nt][2] - mx1), p3 = __expf(sc[nt][3] - mx1);
        sum0 += p0 + p1;
        sum1 += p2 + p3;
        split_pair(p0, p1, ph[nt >> 1][(nt & 1) * 2], pl[nt >> 1][(nt & 1) * 2]);
        split_pair(p2, p3, ph[nt >> 1][(nt & 1) * 2 + 1], pl[nt >> 1][(nt & 1) * 2 + 1]);
      }
#pragma unroll
      for (int kk = 0; kk < 2; ++kk) {
        const int vrow = wk0 + kk * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
        for (int nt = 0; nt < NT; nt += 2) {
          const int chunk = nt + (lane >> 4);
          uint32_t bfr[4];
          ldmatrix_x4_trans(v_s + vrow * RB + (uint32_t)((chunk & ~7) | ((chunk ^ vrow) & 7)) * 16, bfr);
          mma_bf16_16816(oc[nt], ph[kk], bfr[0], bfr[1]);
          mma_bf16_16816(oc[nt], pl[kk], bfr[0], bfr[1]);
          mma_bf16_16816(oc[nt + 1], ph[kk], bfr[2], bfr[3]);
          mma_bf16_16816(oc[nt + 1], pl[kk], bfr[2], bfr[3]);
        }
      }
      if (t_next >= 0) {
        __syncthreads();      // every warp is done with this tile's V
        load_rows(t_next, 1);
      }
    }
    // ---- the four warps' shares of O and of the row sums meet in shared memory
    sum0 += __shfl_xor_sync(0xffffffffu, sum0, 1);
    sum0 += __shfl_xor_sync(0xffffffffu, sum0, 2);
    sum1 += __shfl_xor_sync(0xffffffffu, sum1, 1);
    sum1 += __shfl_xor_sync(0xffffffffu, sum1, 2);
    if ((lane & 3) == 0) {
      wsum_s[warp][r0] = sum0;
      wsum_s[warp][r0 + 8] = sum1;
      if (warp == 0) {
        run_max_s[r0] = run0;
        run_max_s[r0 + 8] = run1;
      }
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      float *oa = o_red + ((long long)(warp * kPaRows + r0) * D) + nt * 8 + cq;
      float *ob = o_red + ((long long)(warp * kPaRows + r0 + 8) * D) + nt * 8 + cq;
      *reinterpret_cast<float2 *>(oa) = make_float2(oc[nt][0], oc[nt][1]);
      *reinterpret_cast<float2 *>(ob) = make_float2(oc[nt][2], oc[nt][3]);
    }
    __syncthreads();
    for (int e = tid; e < nh * D; e += kPaSplitKeys) {
      const int h = e / D, c = e % D;
      float a = 0.f;
#pragma unroll
      for (int w = 0; w < NW; ++w) a += o_red[(long long)(w * kPaRows + h) * D + c];
      float *rec = partial + ((long long)(g * group + h0 + h) * n_parts + part) * (D + 2);
      rec[2 + c] = a;
      if (c == 0) {
        float l = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) l += wsum_s[w][h];
        rec[0] = run_max_s[h];
        rec[1] = l;
      }
    }
  }
}

// Combines the splits of one query head: weights exp(m_s - max m) are formed once per split, then each
// thread reduces one output dim over the splits (coalesced reads of the partial records).
constexpr int kPaMergeMaxSplits = 2048;
__global__ void __launch_bounds__(128) paged_attention_merge_kernel(const float *__restrict__ partial, int n_splits,
                                                                    int d, float *__restrict__ out) {
  __shared__ float w_s[kPaMergeMaxSplits];
  __shared__ float red[4];
  const int head = blockIdx.x, tid = threadIdx.x;
  const float *rec = partial + (long long)head * n_splits * (d + 2);
  float mx = -FLT_MAX;
  for (int s = tid; s < n_splits; s += 128) mx = fmaxf(mx, rec[(long long)s * (d + 2)]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if ((tid & 31) == 0) red[tid >> 5] = mx;
  __syncthreads();
  mx = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
  __syncthreads();
  float ll = 0.f;
  for (int s = tid; s < n_splits; s += 128) {
    const float wgt = __expf(rec[(long long)s * (d + 2)] - mx);
    w_s[s] = wgt;
    ll += rec[(long long)s * (d + 2) + 1] * wgt;
  }
  ll = warp_sum_d(ll);
  if ((tid & 31) == 0) red[tid >> 5] = ll;
  __syncthreads();
  ll = red[0] + red[1] + red[2] + red[3];
  const float inv = 1.f / ll;
  for (int c = tid; c < d; c += 128) {
    float a = 0.f;
    for (int s = 0; s < n_splits; ++s) a += rec[(long long)s * (d + 2) + 2 + c] * w_s[s];
    out[head * d + c] = a * inv;
  }
}

int paged_attention(const float *q, int n_q_heads, CacheView cache, int layer, const int *block_table_dev,
                    int n_ctx, void *scratch, float *out, cudaStream_t st) {
  const int device = current_device();
  if (device < 0) return KV_ERR_CUDA;
  // one part per 128-key tile up to two CTAs per SM; longer contexts give a part several consecutive tiles
  const int tiles = pa_splits(n_ctx);
  int parts = 2 * sm_count(device) / cache.n_kv_heads;
  parts = parts < 1 ? 1 : (parts > kPaMergeMaxSplits ? kPaMergeMaxSplits : parts);
  if (parts > tiles) parts = tiles;
  const dim3 grid(cache.n_kv_heads, parts);
  float *partial = (float *)scratch;
  static bool attr_set[kMaxDevices] = {};
  if (!attr_set[device]) {
    KV_CUDA(cudaFuncSetAttribute(paged_attention_split_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 pa_smem_bytes(64)));
    KV_CUDA(cudaFuncSetAttribute(paged_attention_split_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 pa_smem_bytes(128)));
    attr_set[device] = true;
  }
  if (cache.head_dim == 64)
    paged_attention_split_kernel<64><<<grid, kPaSplitKeys, pa_smem_bytes(64), st>>>(
        q, n_q_heads, cache, layer, block_table_dev, n_ctx, partial);
  else if (cache.head_dim == 128)
    paged_attention_split_kernel<128><<<grid, kPaSplitKeys, pa_smem_bytes(128), st>>>(
        q, n_q_heads, cache, layer, block_table_dev, n_ctx, partial);
  else
    return KV_ERR_SHAPE;
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  paged_attention_merge_kernel<<<n_q_heads, 128, 0, st>>>(partial, parts, cache.head_dim, out);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

}  // namespace kvr
