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

// Rotate the Q and K heads of the fp32 qkv vector in place (angles in fp64) and append K/V (bf16) to the cache.
__global__ void __launch_bounds__(256) rope_store_kv_one_kernel(float *__restrict__ qkv, int pos, int n_q_heads,
                                                                int n_kv_heads, int head_dim, float base,
                                                                CacheView cache, int layer,
                                                                const int *__restrict__ block_table) {
  const int half = head_dim / 2;
  const int block = block_table[pos / cache.block_size];
  const int slot = pos % cache.block_size;
  bf16 *kpage = reinterpret_cast<bf16 *>(cache.page(layer, 0, block)) + (long long)slot * n_kv_heads * head_dim;
  bf16 *vpage = reinterpret_cast<bf16 *>(cache.page(layer, 1, block)) + (long long)slot * n_kv_heads * head_dim;
  const int n_rot = (n_q_heads + n_kv_heads) * half;
  for (int idx = threadIdx.x; idx < n_rot; idx += blockDim.x) {
    const int head = idx / half, j = idx - head * half;
    double s, c;
    sincos((double)pos * pow((double)base, -(double)j / (double)half), &s, &c);
    float *h = qkv + head * head_dim;
    const float a = h[j], b = h[j + half];
    const float ra = a * (float)c - b * (float)s, rb = b * (float)c + a * (float)s;
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
constexpr int kPaWarps = 4;
constexpr int kPaSplitKeys = 256;   // keys per split (multiple of any block size in use)
constexpr int kPaMaxDimsPerLane = 8;  // head_dim <= 256

static int pa_splits(int n_ctx) {
  int s = (n_ctx + kPaSplitKeys - 1) / kPaSplitKeys;
  return s < 1 ? 1 : s;
}

long long paged_attention_scratch_bytes(int n_q_heads, int head_dim, int n_ctx) {
  return (long long)n_q_heads * pa_splits(n_ctx) * (head_dim + 2) * (long long)sizeof(float);
}

__global__ void __launch_bounds__(kPaWarps * 32) paged_attention_split_kernel(
    const float *__restrict__ q, int n_q_heads, CacheView cache, int layer, const int *__restrict__ block_table,
    int n_ctx, float *__restrict__ partial) {
  const int head = blockIdx.x, split = blockIdx.y, n_splits = gridDim.y;
  const int d = cache.head_dim;
  const int g = head / (n_q_heads / cache.n_kv_heads);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int dpl = d / 32;   // dims per lane, lane owns dims lane*dpl .. lane*dpl+dpl-1
  const float scale = rsqrtf((float)d);
  float qr[kPaMaxDimsPerLane], acc[kPaMaxDimsPerLane];
#pragma unroll
  for (int i = 0; i < kPaMaxDimsPerLane; ++i) {
    qr[i] = (i < dpl) ? q[head * d + lane * dpl + i] * scale : 0.f;
    acc[i] = 0.f;
  }
  float m = -FLT_MAX, l = 0.f;
  const int j0 = split * kPaSplitKeys;
  const int j1 = min(n_ctx, j0 + kPaSplitKeys);
  for (int j = j0 + warp; j < j1; j += kPaWarps) {
    const int block = block_table[j / cache.block_size];
    const long long off = ((long long)(j % cache.block_size) * cache.n_kv_heads + g) * d + lane * dpl;
    const bf16 *kp = reinterpret_cast<const bf16 *>(cache.page(layer, 0, block)) + off;
    const bf16 *vp = reinterpret_cast<const bf16 *>(cache.page(layer, 1, block)) + off;
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < kPaMaxDimsPerLane; ++i)
      if (i < dpl) s += qr[i] * __bfloat162float(kp[i]);
    s = warp_sum_d(s);
    const float mn = fmaxf(m, s);
    const float corr = __expf(m - mn), p = __expf(s - mn);
    l = l * corr + p;
#pragma unroll
    for (int i = 0; i < kPaMaxDimsPerLane; ++i)
      if (i < dpl) acc[i] = acc[i] * corr + p * __bfloat162float(vp[i]);
    m = mn;
  }
  // merge the warps of this CTA
  __shared__ float sm_m[kPaWarps], sm_l[kPaWarps];
  __shared__ float sm_acc[kPaWarps][256];
  if (lane == 0) { sm_m[warp] = m; sm_l[warp] = l; }
#pragma unroll
  for (int i = 0; i < kPaMaxDimsPerLane; ++i)
    if (i < dpl) sm_acc[warp][lane * dpl + i] = acc[i];
  __syncthreads();
  float *rec = partial + ((long long)head * n_splits + split) * (d + 2);
  float mm = -FLT_MAX;
  for (int w = 0; w < kPaWarps; ++w) mm = fmaxf(mm, sm_m[w]);
  if (threadIdx.x == 0) {
    float ll = 0.f;
    for (int w = 0; w < kPaWarps; ++w) ll += sm_l[w] * __expf(sm_m[w] - mm);
    rec[0] = mm;
    rec[1] = ll;
  }
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    float a = 0.f;
    for (int w = 0; w < kPaWarps; ++w) a += sm_acc[w][c] * __expf(sm_m[w] - mm);
    rec[2 + c] = a;
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
  paged_attention_split_kernel<<<dim3(n_q_heads, splits), kPaWarps * 32, 0, st>>>(
      q, n_q_heads, cache, layer, block_table_dev, n_ctx, (float *)scratch);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  paged_attention_merge_kernel<<<n_q_heads, 128, 0, st>>>((const float *)scratch, splits, cache.head_dim, out);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

}  // namespace kvr
