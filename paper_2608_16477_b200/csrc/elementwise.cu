// Bandwidth-bound steps of the prefill path: embedding gather, RMSNorm, RoPE table.
#include "common.cuh"

namespace kvr {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// block-wide sum for blockDim.x <= 1024 (multiple of 32); every thread gets the result
__device__ __forceinline__ float block_sum(float v, float *red) {
  v = warp_sum(v);
  const int w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  if ((threadIdx.x & 31) == 0) red[w] = v;
  __syncthreads();
  float t = (threadIdx.x & 31) < nw ? red[threadIdx.x & 31] : 0.f;
  t = warp_sum(t);
  __syncthreads();
  return t;
}

// x[t, :] = float(E[ids[t], :])
__global__ void embed_rows_kernel(const bf16 *__restrict__ embed, const int *__restrict__ ids, int hidden,
                                  float *__restrict__ x) {
  const int t = blockIdx.x;
  const uint4 *src = reinterpret_cast<const uint4 *>(embed + (long long)ids[t] * hidden);
  float4 *dst = reinterpret_cast<float4 *>(x + (long long)t * hidden);
  for (int v = threadIdx.x; v < hidden / 8; v += blockDim.x) {
    uint4 raw = src[v];
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&raw);
    float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
    float2 c = __bfloat1622float2(h[2]), d = __bfloat1622float2(h[3]);
    dst[2 * v] = make_float4(a.x, a.y, b.x, b.y);
    dst[2 * v + 1] = make_float4(c.x, c.y, d.x, d.y);
  }
}

int embed_rows(const bf16 *embed, const int *ids_dev, int n_tokens, int hidden, float *x, cudaStream_t st) {
  embed_rows_kernel<<<n_tokens, 128, 0, st>>>(embed, ids_dev, hidden, x);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

// out[r, :] = bf16( x[r, :] * rsqrt(mean(x[r, :]^2) + eps) * gain ), statistics in fp32.
// One CTA per row.  Rows of up to 256 * 4 * kRmsVecs floats are read from HBM exactly once and kept in
// registers between the reduction and the scaling; longer rows are read a second time (from L1/L2).
constexpr int kRmsVecs = 8;
__global__ void __launch_bounds__(256) rmsnorm_rows_kernel(const float *__restrict__ x,
                                                           const bf16 *__restrict__ gain, int dim, float eps,
                                                           bf16 *__restrict__ out) {
  __shared__ float red[32];
  const float4 *row = reinterpret_cast<const float4 *>(x + (long long)blockIdx.x * dim);
  const int nvec = dim / 4;
  const bool cached = nvec <= 256 * kRmsVecs;
  float4 keep[kRmsVecs];
  float ss = 0.f;
  if (cached) {
#pragma unroll
    for (int i = 0; i < kRmsVecs; ++i) {
      const int v = threadIdx.x + i * 256;
      keep[i] = (v < nvec) ? __ldcs(row + v) : make_float4(0.f, 0.f, 0.f, 0.f);
      ss += keep[i].x * keep[i].x + keep[i].y * keep[i].y + keep[i].z * keep[i].z + keep[i].w * keep[i].w;
    }
  } else {
    for (int v = threadIdx.x; v < nvec; v += blockDim.x) {
      float4 a = row[v];
      ss += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
    }
  }
  ss = block_sum(ss, red);
  const float inv = rsqrtf(ss / (float)dim + eps);
  uint2 *o = reinterpret_cast<uint2 *>(out + (long long)blockIdx.x * dim);
  const uint2 *g = reinterpret_cast<const uint2 *>(gain);
  auto emit = [&](int v, float4 a) {
    const uint2 graw = g[v];
    const float2 g0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&graw.x));
    const float2 g1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&graw.y));
    __nv_bfloat162 lo = __floats2bfloat162_rn(a.x * inv * g0.x, a.y * inv * g0.y);
    __nv_bfloat162 hi = __floats2bfloat162_rn(a.z * inv * g1.x, a.w * inv * g1.y);
    uint2 packed;
    packed.x = *reinterpret_cast<uint32_t *>(&lo);
    packed.y = *reinterpret_cast<uint32_t *>(&hi);
    o[v] = packed;
  };
  if (cached) {
#pragma unroll
    for (int i = 0; i < kRmsVecs; ++i) {
      const int v = threadIdx.x + i * 256;
      if (v < nvec) emit(v, keep[i]);
    }
  } else {
    for (int v = threadIdx.x; v < nvec; v += blockDim.x) emit(v, row[v]);
  }
}

int rmsnorm_rows(const float *x, const bf16 *gain, int rows, int dim, float eps, bf16 *out, cudaStream_t st) {
  if (rows <= 0) return KV_OK;
  rmsnorm_rows_kernel<<<rows, 256, 0, st>>>(x, gain, dim, eps, out);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

// table[j, t] = (cos, sin)(pos_t * base^(-2j/d)) (frequency-major), angle formed in fp64 so that positions in the
// tens of thousands keep full fp32 accuracy after the final rounding.
__global__ void rope_table_kernel(float2 *table, int pos0, int n_tokens, int half, float base,
                                  const int *__restrict__ row_pos) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_tokens * half) return;
  const int j = idx / n_tokens, t = idx - j * n_tokens;      // consecutive threads: consecutive tokens of one frequency
  const double theta = pow((double)base, -(double)j / (double)half);
  double s, c;
  const int pos = row_pos != nullptr ? row_pos[t] : pos0 + t;
  sincos((double)pos * theta, &s, &c);
  table[(long long)j * n_tokens + t] = make_float2((float)c, (float)s);
}

int rope_table(float2 *table, int pos0, int n_tokens, int head_dim, float base, cudaStream_t st, const int *row_pos) {
  const int n = n_tokens * (head_dim / 2);
  if (n <= 0) return KV_OK;
  rope_table_kernel<<<(n + 255) / 256, 256, 0, st>>>(table, pos0, n_tokens, head_dim / 2, base, row_pos);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

}  // namespace kvr
