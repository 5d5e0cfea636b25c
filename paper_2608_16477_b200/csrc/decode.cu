// Decode step (one token): every stage is HBM-bound.  Weights are streamed once with 16-byte loads
// (warp per output row), activations stay fp32; attention reads the paged cache through the block
// table with the keys split across CTAs (flash-decoding) and a second pass merging the splits.
#include <float.h>

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

__global__ void __launch_bounds__(1024) rmsnorm_vec_kernel(const float *__restrict__ x,
                                                           const bf16 *__restrict__ gain, int dim, float eps,
                                                           float *__restrict__ out) {
  __shared__ float red[32];
  float ss = 0.f;
  for (int c = threadIdx.x; c < dim; c += blockDim.x) ss += x[c] * x[c];
  ss = warp_sum_d(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float t = (threadIdx.x & 31) < (blockDim.x >> 5) ? red[threadIdx.x & 31] : 0.f;
  t = warp_sum_d(t);
  const float inv = rsqrtf(t / (float)dim + eps);
  for (int c = threadIdx.x; c < dim; c += blockDim.x) out[c] = x[c] * inv * __bfloat162float(gain[c]);
}

int rmsnorm_vec(const float *x, const bf16 *gain, int dim, float eps, float *out, cudaStream_t st) {
  rmsnorm_vec_kernel<<<1, 1024, 0, st>>>(x, gain, dim, eps, out);
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

// Warp per output row; W row-major [rows, k] bf16 streamed once, x fp32 (L1/L2 resident).
// MODE 0: y[n] = W[n].x   MODE 1: y[n] += W[n].x   MODE 2: y[n] = silu(W[n].x) * (W[n + N].x)
constexpr int kGemvWarps = 8;
template <int MODE>
__global__ void __launch_bounds__(kGemvWarps * 32) gemv_kernel(const bf16 *__restrict__ w,
                                                               const float *__restrict__ x, int n, int k,
                                                               float *__restrict__ y) {
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * kGemvWarps + (threadIdx.x >> 5);
  if (row >= n) return;
  const int nvec = k / 8;
  const uint4 *wr = reinterpret_cast<const uint4 *>(w + (long long)row * k);
  const uint4 *wr2 = reinterpret_cast<const uint4 *>(w + (long long)(row + n) * k);
  const float4 *xv = reinterpret_cast<const float4 *>(x);
  float acc = 0.f, acc2 = 0.f;
  int v = lane;
  for (; v + 96 < nvec; v += 128) {
    uint4 w0 = __ldcs(wr + v), w1 = __ldcs(wr + v + 32), w2 = __ldcs(wr + v + 64), w3 = __ldcs(wr + v + 96);
    uint4 u0, u1, u2, u3;
    if (MODE == 2) { u0 = __ldcs(wr2 + v); u1 = __ldcs(wr2 + v + 32); u2 = __ldcs(wr2 + v + 64); u3 = __ldcs(wr2 + v + 96); }
    float4 a0 = xv[2 * v], a1 = xv[2 * v + 1], b0 = xv[2 * (v + 32)], b1 = xv[2 * (v + 32) + 1];
    float4 c0 = xv[2 * (v + 64)], c1 = xv[2 * (v + 64) + 1], d0 = xv[2 * (v + 96)], d1 = xv[2 * (v + 96) + 1];
    acc += dot8(w0, a0, a1) + dot8(w1, b0, b1) + dot8(w2, c0, c1) + dot8(w3, d0, d1);
    if (MODE == 2) acc2 += dot8(u0, a0, a1) + dot8(u1, b0, b1) + dot8(u2, c0, c1) + dot8(u3, d0, d1);
  }
  for (; v < nvec; v += 32) {
    float4 a0 = xv[2 * v], a1 = xv[2 * v + 1];
    acc += dot8(__ldcs(wr + v), a0, a1);
    if (MODE == 2) acc2 += dot8(__ldcs(wr2 + v), a0, a1);
  }
  acc = warp_sum_d(acc);
  if (MODE == 2) acc2 = warp_sum_d(acc2);
  if (lane == 0) {
    if (MODE == 0) y[row] = acc;
    if (MODE == 1) y[row] += acc;
    if (MODE == 2) y[row] = acc / (1.f + __expf(-acc)) * acc2;
  }
}

int gemv(const bf16 *w, const float *x, int n, int k, int mode, float *y, cudaStream_t st) {
  const int grid = (n + kGemvWarps - 1) / kGemvWarps;
  if (mode == 0) gemv_kernel<0><<<grid, kGemvWarps * 32, 0, st>>>(w, x, n, k, y);
  else if (mode == 1) gemv_kernel<1><<<grid, kGemvWarps * 32, 0, st>>>(w, x, n, k, y);
  else gemv_kernel<2><<<grid, kGemvWarps * 32, 0, st>>>(w, x, n, k, y);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

// Rotate the Q and K heads of the fp32 qkv vector in place and append K/V (bf16) to the cache.
// The d/2 angles pos * base^(-2j/d) are formed once in fp64 (one thread per frequency) and shared.
__global__ void __launch_bounds__(256) rope_store_kv_one_kernel(float *__restrict__ qkv, int pos, int n_q_heads,
                                                                int n_kv_heads, int head_dim, float base,
                                                                CacheView cache, int layer,
                                                                const int *__restrict__ block_table) {
  __shared__ float2 cs[128];
  const int half = head_dim / 2;
  for (int j = threadIdx.x; j < half; j += blockDim.x) {
    double s, c;
    sincos((double)pos * pow((double)base, -(double)j / (double)half), &s, &c);
    cs[j] = make_float2((float)c, (float)s);
  }
  __syncthreads();
  const int block = block_table[pos / cache.block_size];
  const int slot = pos % cache.block_size;
  bf16 *kpage = reinterpret_cast<bf16 *>(cache.page(layer, 0, block)) + (long long)slot * n_kv_heads * head_dim;
  bf16 *vpage = reinterpret_cast<bf16 *>(cache.page(layer, 1, block)) + (long long)slot * n_kv_heads * head_dim;
  const int n_rot = (n_q_heads + n_kv_heads) * half;
  for (int idx = threadIdx.x; idx < n_rot; idx += blockDim.x) {
    const int head = idx / half, j = idx - head * half;
    const float2 c = cs[j];
    float *h = qkv + head * head_dim;
    const float a = h[j], b = h[j + half];
    const float ra = a * c.x - b * c.y, rb = b * c.x + a * c.y;
    h[j] = ra;
    h[j + half] = rb;
    if (head >= n_q_heads) {
      bf16 *kd = kpage + (head - n_q_heads) * head_dim;
      kd[j] = __float2bfloat16_rn(ra);
      kd[j + half] = __float2bfloat16_rn(rb);
    }
  }
  const float *v = qkv + (n_q_heads + n_kv_heads) * head_dim;
  for (int c = threadIdx.x; c < n_kv_heads * head_dim; c += blockDim.x) vpage[c] = __float2bfloat16_rn(v[c]);
}

int rope_store_kv_one(float *qkv, int pos, int n_q_heads, int n_kv_heads, int head_dim, float base,
                      CacheView cache, int layer, const int *block_table_dev, cudaStream_t st) {
  rope_store_kv_one_kernel<<<1, 256, 0, st>>>(qkv, pos, n_q_heads, n_kv_heads, head_dim, base, cache, layer,
                                              block_table_dev);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
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

__global__ void paged_attention_merge_kernel(const float *__restrict__ partial, int n_splits, int d,
                                             float *__restrict__ out) {
  const int head = blockIdx.x;
  const float *rec = partial + (long long)head * n_splits * (d + 2);
  float mm = -FLT_MAX;
  for (int s = 0; s < n_splits; ++s) mm = fmaxf(mm, rec[s * (d + 2)]);
  float ll = 0.f;
  for (int s = 0; s < n_splits; ++s) ll += rec[s * (d + 2) + 1] * __expf(rec[s * (d + 2)] - mm);
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    float a = 0.f;
    for (int s = 0; s < n_splits; ++s) a += rec[s * (d + 2) + 2 + c] * __expf(rec[s * (d + 2)] - mm);
    out[head * d + c] = a / ll;
  }
}

int paged_attention(const float *q, int n_q_heads, CacheView cache, int layer, const int *block_table_dev,
                    int n_ctx, void *scratch, float *out, cudaStream_t st) {
  const int splits = pa_splits(n_ctx);
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
