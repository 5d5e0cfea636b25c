// Causal GQA attention over a prefill chunk: dispatch, and the general CUDA-core kernel.
//
// Query rows are the chunk's positions pos0 .. pos0+T-1; keys/values of the chunk come from the
// contiguous post-RoPE qkv buffer, earlier positions [0,pos0) from the paged cache through the block
// table.  Online softmax in fp32 (running max / sum), outputs bf16.
// head_dim 64/128 with an even number of query heads per KV head runs on the tensor-core kernel
// (attention_tcgen05.cu); the prefill path gathers a cached prefix into the qkv buffer for it.  The kernel
// below reads earlier positions straight from the pages and serves the remaining head layouts and the
// single-kernel entry point with pos0 > 0.
#include <float.h>

#include "common.cuh"

namespace kvr {

// Warp per (query row, head); lanes score 32 keys at a time, then each lane accumulates d/32 output dims.
constexpr int kApWarps = 4;
constexpr int kApMaxD = 256;

__global__ void __launch_bounds__(kApWarps * 32) attention_prefill_simt_kernel(
    const bf16 *__restrict__ qkv, int n_tokens, int pos0, int n_q_heads, int n_kv_heads, int head_dim,
    CacheView cache, int layer, const int *__restrict__ block_table, bf16 *__restrict__ out) {
  __shared__ float qs[kApWarps][kApMaxD];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int head = blockIdx.y;
  const int t = blockIdx.x * kApWarps + warp;
  if (t >= n_tokens) return;
  const int d = head_dim;
  const int g = head / (n_q_heads / n_kv_heads);
  const int qkv_dim = (n_q_heads + 2 * n_kv_heads) * d;
  const int koff = (n_q_heads + g) * d, voff = (n_q_heads + n_kv_heads + g) * d;
  const float scale = rsqrtf((float)d);
  const bf16 *qrow = qkv + (long long)t * qkv_dim + head * d;
  for (int c = lane; c < d; c += 32) qs[warp][c] = __bfloat162float(qrow[c]) * scale;
  __syncwarp();
  const int dpl = d / 32;
  float acc[kApMaxD / 32];
#pragma unroll
  for (int i = 0; i < kApMaxD / 32; ++i) acc[i] = 0.f;
  float m = -FLT_MAX, l = 0.f;
  const int last = pos0 + t;   // highest visible key position
  for (int j0 = 0; j0 <= last; j0 += 32) {
    const int j = j0 + lane;
    const bf16 *kp = nullptr, *vp = nullptr;
    if (j <= last) {
      if (j >= pos0) {
        kp = qkv + (long long)(j - pos0) * qkv_dim + koff;
        vp = qkv + (long long)(j - pos0) * qkv_dim + voff;
      } else {
        const int block = block_table[j / cache.block_size];
        const long long off = ((long long)(j % cache.block_size) * n_kv_heads + g) * d;
        kp = reinterpret_cast<const bf16 *>(cache.page(layer, 0, block)) + off;
        vp = reinterpret_cast<const bf16 *>(cache.page(layer, 1, block)) + off;
      }
    }
    float s = -FLT_MAX;
    if (kp) {
      s = 0.f;
      const uint4 *kv4 = reinterpret_cast<const uint4 *>(kp);
      for (int v = 0; v < d / 8; ++v) {
        uint4 raw = kv4[v];
        const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&raw);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float2 f = __bfloat1622float2(h[e]);
          s += qs[warp][v * 8 + 2 * e] * f.x + qs[warp][v * 8 + 2 * e + 1] * f.y;
        }
      }
    }
    float mx = s;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    const float mn = fmaxf(m, mx);
    const float corr = __expf(m - mn);
    const float p = kp ? __expf(s - mn) : 0.f;
    float ps = p;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
    l = l * corr + ps;
#pragma unroll
    for (int i = 0; i < kApMaxD / 32; ++i) acc[i] *= corr;
    m = mn;
    const int nk = min(32, last - j0 + 1);
    for (int jj = 0; jj < nk; ++jj) {
      const float pj = __shfl_sync(0xffffffffu, p, jj);
      const unsigned long long vaddr = __shfl_sync(0xffffffffu, (unsigned long long)vp, jj);
      const bf16 *vr = reinterpret_cast<const bf16 *>(vaddr);
#pragma unroll
      for (int i = 0; i < kApMaxD / 32; ++i)
        if (i < dpl) acc[i] += pj * __bfloat162float(vr[lane + 32 * i]);
    }
  }
  bf16 *orow = out + (long long)t * n_q_heads * d + head * d;
  const float inv = 1.f / l;
#pragma unroll
  for (int i = 0; i < kApMaxD / 32; ++i)
    if (i < dpl) orow[lane + 32 * i] = __float2bfloat16_rn(acc[i] * inv);
}


int attention_prefill(const bf16 *qkv, int n_tokens, int pos0, int n_q_heads, int n_kv_heads, int head_dim,
                      CacheView cache, int layer, const int *block_table_dev, bf16 *out, int *status_dev,
                      cudaStream_t st) {
  if (n_tokens <= 0) return KV_OK;
  if (pos0 == 0 && attention_tc_supported(n_q_heads, n_kv_heads, head_dim))
    return attention_prefill_tc(qkv, n_tokens, 0, n_q_heads, n_kv_heads, head_dim, out, status_dev, st);
  dim3 grid((n_tokens + kApWarps - 1) / kApWarps, n_q_heads);
  attention_prefill_simt_kernel<<<grid, kApWarps * 32, 0, st>>>(qkv, n_tokens, pos0, n_q_heads, n_kv_heads,
                                                               head_dim, cache, layer, block_table_dev, out);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

}  // namespace kvr
