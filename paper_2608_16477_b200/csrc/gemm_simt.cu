// Plain CUDA-core GEMM used only to cross-check the tensor-core kernel in unit tests
// (bf16 operands, fp32 accumulation, the same three epilogues).  Not on the product path.
#include "common.cuh"

namespace kvr {

constexpr int ST = 64;   // tile edge
constexpr int SK = 16;   // k slice

__device__ __forceinline__ float silu_f(float a) { return a / (1.f + __expf(-a)); }

// C tile 64x64 per CTA of 256 threads, 4x4 outputs per thread.
template <int MODE>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const bf16 *__restrict__ a, int lda,
                                                        const bf16 *__restrict__ w, int m, int n, int k,
                                                        bf16 *__restrict__ out, float *__restrict__ resid) {
  __shared__ float As[SK][ST + 1];
  __shared__ float Bs[(MODE == GEMM_SWIGLU) ? 2 : 1][SK][ST + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int m0 = blockIdx.y * ST, n0 = blockIdx.x * ST;
  float acc[4][4] = {}, acc2[4][4] = {};
  for (int k0 = 0; k0 < k; k0 += SK) {
    for (int e = threadIdx.x; e < ST * SK; e += 256) {
      const int r = e / SK, c = e % SK;
      const int gm = m0 + r, gn = n0 + r;
      As[c][r] = (gm < m && k0 + c < k) ? __bfloat162float(a[(long long)gm * lda + k0 + c]) : 0.f;
      Bs[0][c][r] = (gn < n && k0 + c < k) ? __bfloat162float(w[(long long)gn * k + k0 + c]) : 0.f;
      if (MODE == GEMM_SWIGLU)
        Bs[MODE == GEMM_SWIGLU ? 1 : 0][c][r] =
            (gn < n && k0 + c < k) ? __bfloat162float(w[(long long)(gn + n) * k + k0 + c]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int c = 0; c < SK; ++c) {
      float av[4], bv[4], bv2[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        av[i] = As[c][ty * 4 + i];
        bv[i] = Bs[0][c][tx * 4 + i];
        bv2[i] = (MODE == GEMM_SWIGLU) ? Bs[MODE == GEMM_SWIGLU ? 1 : 0][c][tx * 4 + i] : 0.f;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[i][j] += av[i] * bv[j];
          if (MODE == GEMM_SWIGLU) acc2[i][j] += av[i] * bv2[j];
        }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gm = m0 + ty * 4 + i, gn = n0 + tx * 4 + j;
      if (gm >= m || gn >= n) continue;
      const long long o = (long long)gm * n + gn;
      if (MODE == GEMM_STORE_BF16) out[o] = __float2bfloat16_rn(acc[i][j]);
      if (MODE == GEMM_RESID_F32) resid[o] += acc[i][j];
      if (MODE == GEMM_SWIGLU) out[o] = __float2bfloat16_rn(silu_f(acc[i][j]) * acc2[i][j]);
    }
}

int gemm_simt(const bf16 *a, int lda, const bf16 *w, int m, int n, int k, int mode, bf16 *out, float *resid,
              cudaStream_t st) {
  if (m <= 0 || n <= 0) return KV_OK;
  dim3 grid((n + ST - 1) / ST, (m + ST - 1) / ST);
  if (mode == GEMM_STORE_BF16)
    gemm_simt_kernel<GEMM_STORE_BF16><<<grid, 256, 0, st>>>(a, lda, w, m, n, k, out, resid);
  else if (mode == GEMM_RESID_F32)
    gemm_simt_kernel<GEMM_RESID_F32><<<grid, 256, 0, st>>>(a, lda, w, m, n, k, out, resid);
  else
    gemm_simt_kernel<GEMM_SWIGLU><<<grid, 256, 0, st>>>(a, lda, w, m, n, k, out, resid);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

}  // namespace kvr
