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
// QKV rows (j, j + d/2) of one head -> RoPE rotation, q to the fp32 query vector, k and v (bf16) appended
// to the paged cache.
enum GemvEpi { GEMV_STORE = 0, GEMV_ADD = 1, GEMV_SWIGLU = 2, GEMV_QKV = 3 };
constexpr int kGemvWarps = 8;

struct GemvQkvArgs {
  CacheView cache;
  const int *block_table;
  int pos, layer, head_dim, n_q_heads, n_kv_heads;
  float base;
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
  int v = lane;
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
      double sn, cs;
      sincos((double)qa.pos * pow((double)qa.base, -(double)j / (double)half), &sn, &cs);
      const float ra = acc_a * (float)cs - acc_b * (float)sn;
      const float rb = acc_b * (float)cs + acc_a * (float)sn;
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
                  int n_kv_heads, int head_dim, float base, CacheView cache, int layer, const int *block_table_dev,
                  float *q_out, cudaStream_t st) {
  GemvQkvArgs qa;
  qa.cache = cache;
  qa.block_table = block_table_dev;
  qa.pos = pos;
  qa.layer = layer;
  qa.head_dim = head_dim;
  qa.n_q_heads = n_q_heads;
  qa.n_kv_heads = n_kv_heads;
  qa.base = base;
  if (hidden % 8 != 0) return KV_ERR_SHAPE;
  const int n = (n_q_heads + 2 * n_kv_heads) * head_dim;
  return launch_gemv2<GEMV_QKV, true>(w_qkv, x, gain, eps, n, hidden, q_out, qa, st);
}

// ---- paged decode attention ---------------------------------------------------------------
// Partial record per (q head, split): m, l, acc[d].
// One CTA of 256 threads per (KV head, 256-key split), serving every query head of the group so each K/V
// row is read from HBM once:
//   phase 1  thread t loads the whole K row of key t (16-byte loads, all in flight at once) and scores it
//            against the group's queries held in shared memory;
//   phase 2  one warp per head: maximum, exponentials and their sum over the split's scores;
//   phase 3  warp w walks keys 32w..32w+31, each lane owning d/32 dims of V, accumulating p * v for all
//            heads; the eight warps' partial sums meet in shared memory.
constexpr int kPaSplitKeys = 256;   // keys per split = threads per CTA
constexpr int kPaHeadChunk = 8;     // query heads handled per pass over the keys

static int pa_splits(int n_ctx) {
  int s = (n_ctx + kPaSplitKeys - 1) / kPaSplitKeys;
  return s < 1 ? 1 : s;
}

long long paged_attention_scratch_bytes(int n_q_heads, int head_dim, int n_ctx) {
  return (long long)n_q_heads * pa_splits(n_ctx) * (head_dim + 2) * (long long)sizeof(float);
}

// DPL consecutive bf16 -> fp32 with one vector load (the address is DPL*2-byte aligned)
template <int DPL>
__device__ __forceinline__ void load_bf16(const bf16 *p, float (&out)[DPL]) {
  static_assert(DPL == 2 || DPL == 4 || DPL == 8, "dims per lane");
  if constexpr (DPL == 8) {
    const uint4 raw = *reinterpret_cast<const uint4 *>(p);
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&raw);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __bfloat1622float2(h[i]);
      out[2 * i] = f.x;
      out[2 * i + 1] = f.y;
    }
  } else if constexpr (DPL == 4) {
    const uint2 raw = *reinterpret_cast<const uint2 *>(p);
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&raw);
    const float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
    out[0] = a.x; out[1] = a.y; out[2] = b.x; out[3] = b.y;
  } else {
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(p));
    out[0] = a.x; out[1] = a.y;
  }
}

template <int D>
__global__ void __launch_bounds__(kPaSplitKeys) paged_attention_split_kernel(
    const float *__restrict__ q, int n_q_heads, CacheView cache, int layer, const int *__restrict__ block_table,
    int n_ctx, float *__restrict__ partial) {
  constexpr int DPL = D / 32;
  constexpr int HC = kPaHeadChunk;
  __shared__ __align__(16) float q_s[HC][D];
  __shared__ float p_s[HC][kPaSplitKeys];
  __shared__ __align__(16) float red_s[kPaSplitKeys / 32][HC][D];
  __shared__ float ml_s[HC][2];
  const int g = blockIdx.x, split = blockIdx.y, n_splits = gridDim.y;
  const int group = n_q_heads / cache.n_kv_heads;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float scale = rsqrtf((float)D);
  const int j0 = split * kPaSplitKeys;
  const int n_keys = min(n_ctx - j0, kPaSplitKeys);

  // this thread's key: K row into registers (phase 1 operand), V row address for later
  const int jk = j0 + min(tid, n_keys - 1);
  const long long row_off = ((long long)(jk % cache.block_size) * cache.n_kv_heads + g) * D;
  const int blk_k = block_table[jk / cache.block_size];
  uint4 kraw[D / 8];
  {
    const uint4 *kp = reinterpret_cast<const uint4 *>(reinterpret_cast<const bf16 *>(cache.page(layer, 0, blk_k)) + row_off);
#pragma unroll
    for (int v = 0; v < D / 8; ++v) kraw[v] = kp[v];
  }

  for (int h0 = 0; h0 < group; h0 += HC) {
    const int nh = min(HC, group - h0);
    __syncthreads();   // previous chunk fully consumed
    for (int e = tid; e < nh * D; e += kPaSplitKeys)
      q_s[e / D][e % D] = q[(long long)(g * group + h0 + e / D) * D + e % D] * scale;
    __syncthreads();
    // ---- phase 1: scores of this thread's key against nh heads
    {
      float sc[HC];
#pragma unroll
      for (int h = 0; h < HC; ++h) sc[h] = 0.f;
#pragma unroll
      for (int v = 0; v < D / 8; ++v) {
        const __nv_bfloat162 *hk = reinterpret_cast<const __nv_bfloat162 *>(&kraw[v]);
        const float2 k0 = __bfloat1622float2(hk[0]), k1 = __bfloat1622float2(hk[1]);
        const float2 k2 = __bfloat1622float2(hk[2]), k3 = __bfloat1622float2(hk[3]);
#pragma unroll
        for (int h = 0; h < HC; ++h) {
          if (h < nh) {
            const float4 qa = *reinterpret_cast<const float4 *>(&q_s[h][v * 8]);
            const float4 qb = *reinterpret_cast<const float4 *>(&q_s[h][v * 8 + 4]);
            sc[h] += k0.x * qa.x + k0.y * qa.y + k1.x * qa.z + k1.y * qa.w + k2.x * qb.x + k2.y * qb.y + k3.x * qb.z +
                     k3.y * qb.w;
          }
        }
      }
#pragma unroll
      for (int h = 0; h < HC; ++h)
        if (h < nh) p_s[h][tid] = (tid < n_keys) ? sc[h] : -FLT_MAX;
    }
    __syncthreads();
    // ---- phase 2: warp h turns the scores of head h into exponentials
    if (warp < nh) {
      float v[kPaSplitKeys / 32];
      float mx = -FLT_MAX;
#pragma unroll
      for (int i = 0; i < kPaSplitKeys / 32; ++i) {
        v[i] = p_s[warp][lane + 32 * i];
        mx = fmaxf(mx, v[i]);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      float sum = 0.f;
#pragma unroll
      for (int i = 0; i < kPaSplitKeys / 32; ++i) {
        const float e = (lane + 32 * i < n_keys) ? __expf(v[i] - mx) : 0.f;
        p_s[warp][lane + 32 * i] = e;
        sum += e;
      }
      sum = warp_sum_d(sum);
      if (lane == 0) {
        ml_s[warp][0] = mx;
        ml_s[warp][1] = sum;
      }
    }
    __syncthreads();
    // ---- phase 3: p * V, warp w over keys 32w .. 32w+31, lane owns DPL dims
    {
      float acc[HC][DPL];
#pragma unroll
      for (int h = 0; h < HC; ++h)
#pragma unroll
        for (int i = 0; i < DPL; ++i) acc[h][i] = 0.f;
      const int kb = warp * 32;
      constexpr int U = 8;
      for (int kk = 0; kk < 32 && kb + kk < n_keys; kk += U) {
        float vf[U][DPL];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int j = j0 + min(kb + kk + u, n_keys - 1);
          const int blk = block_table[j / cache.block_size];
          const bf16 *vp = reinterpret_cast<const bf16 *>(cache.page(layer, 1, blk)) +
                           ((long long)(j % cache.block_size) * cache.n_kv_heads + g) * D + lane * DPL;
          load_bf16<DPL>(vp, vf[u]);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          if (kb + kk + u < n_keys) {
#pragma unroll
            for (int h = 0; h < HC; ++h) {
              if (h < nh) {
                const float p = p_s[h][kb + kk + u];
#pragma unroll
                for (int i = 0; i < DPL; ++i) acc[h][i] += p * vf[u][i];
              }
            }
          }
        }
      }
#pragma unroll
      for (int h = 0; h < HC; ++h)
        if (h < nh) {
#pragma unroll
          for (int i = 0; i < DPL; ++i) red_s[warp][h][lane * DPL + i] = acc[h][i];
        }
    }
    __syncthreads();
    for (int e = tid; e < nh * D; e += kPaSplitKeys) {
      const int h = e / D, c = e % D;
      float a = 0.f;
#pragma unroll
      for (int w = 0; w < kPaSplitKeys / 32; ++w) a += red_s[w][h][c];
      float *rec = partial + ((long long)(g * group + h0 + h) * n_splits + split) * (D + 2);
      rec[2 + c] = a;
      if (c == 0) {
        rec[0] = ml_s[h][0];
        rec[1] = ml_s[h][1];
      }
    }
  }
}

// Combines the splits of one query head: weights exp(m_s - max m) are formed once per split, then each
// thread reduces one output dim over the splits (coalesced reads of the partial records).
constexpr int kPaMergeMaxSplits = 1024;
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
  const int splits = pa_splits(n_ctx);
  if (splits > kPaMergeMaxSplits) return KV_ERR_SHAPE;   // 262,144 context tokens
  const dim3 grid(cache.n_kv_heads, splits);
  float *partial = (float *)scratch;
  if (cache.head_dim == 64)
    paged_attention_split_kernel<64><<<grid, kPaSplitKeys, 0, st>>>(q, n_q_heads, cache, layer, block_table_dev, n_ctx, partial);
  else if (cache.head_dim == 128)
    paged_attention_split_kernel<128><<<grid, kPaSplitKeys, 0, st>>>(q, n_q_heads, cache, layer, block_table_dev, n_ctx, partial);
  else
    return KV_ERR_SHAPE;
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  paged_attention_merge_kernel<<<n_q_heads, 128, 0, st>>>(partial, splits, cache.head_dim, out);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

}  // namespace kvr
