// Shared host/device helpers of the kvrebuild library (internal).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/kvrebuild.h"

namespace kvr {

typedef __nv_bfloat16 bf16;

// Geometry of a paged cache as the kernels see it (byte strides).
struct CacheView {
  char *base;
  long long layer_stride, kv_stride, block_stride;
  int block_size, n_kv_heads, head_dim;
  __host__ __device__ long long page_bytes() const { return (long long)block_size * n_kv_heads * head_dim * 2; }
  __device__ __forceinline__ char *page(int layer, int kv, int block) const {
    return base + layer * layer_stride + kv * kv_stride + block * block_stride;
  }
};

inline CacheView make_view(const kv_cache_desc *c) {
  CacheView v;
  v.base = (char *)c->base_dev;
  v.layer_stride = c->layer_stride;
  v.kv_stride = c->kv_stride;
  v.block_stride = c->block_stride;
  v.block_size = c->block_size;
  v.n_kv_heads = c->n_kv_heads;
  v.head_dim = c->head_dim;
  return v;
}

// Host-side validation of a cache descriptor, shared by every entry point that takes one.
inline int check_cache_desc(const kv_cache_desc *c) {
  if (c == nullptr || c->base_dev == nullptr) return KV_ERR_ARG;
  if (c->num_blocks <= 0 || c->block_size <= 0 || c->n_layers <= 0 || c->n_kv_heads <= 0 || c->head_dim <= 0)
    return KV_ERR_ARG;
  if (c->elem_bytes != 2) return KV_ERR_SHAPE;
  const long long page = (long long)c->block_size * c->n_kv_heads * c->head_dim * 2;
  if (page % 16 != 0) return KV_ERR_SHAPE;
  if (((uintptr_t)c->base_dev & 15) || (c->layer_stride & 15) || (c->kv_stride & 15) || (c->block_stride & 15))
    return KV_ERR_ARG;
  if (c->block_stride < page || c->kv_stride <= 0 || c->layer_stride <= 0) return KV_ERR_ARG;
  return KV_OK;
}

// Layout of the device status word block at the start of every prefill/decode workspace.
struct DeviceStatus {
  int error;      // 0, or the code of the first bounded wait that ran out
  int where;      // kernel-specific tag of that wait
  int detail[6];
};

void set_cuda_error(cudaError_t e, const char *what);

// Number of kernels launched by this library so far (host counter, bumped by every launcher).
extern std::atomic<long long> g_launches;
#define KV_COUNT_LAUNCH() (::kvr::g_launches.fetch_add(1, std::memory_order_relaxed))

// Kernel classes reported by the optional event profiler (kv_profile_*).
enum ProfKind {
  PROF_EMBED = 0, PROF_RMSNORM, PROF_GEMM_QKV, PROF_ROPE_STORE, PROF_ATTENTION, PROF_GEMM_O, PROF_GEMM_GATE_UP,
  PROF_GEMM_DOWN, PROF_LM_HEAD, PROF_PACK, PROF_UNPACK, PROF_DECODE_GEMV, PROF_DECODE_ATTENTION, PROF_DECODE_OTHER,
  PROF_KINDS
};
#define KV_CUDA(call)                                  \
  do {                                                 \
    cudaError_t e__ = (call);                          \
    if (e__ != cudaSuccess) {                          \
      ::kvr::set_cuda_error(e__, #call);               \
      return KV_ERR_CUDA;                              \
    }                                                  \
  } while (0)

// Per-device one-time set-up (opt-in shared-memory sizes, SM counts): function attributes belong to a device,
// so the "done" state is kept per device ordinal, not per process.
constexpr int kMaxDevices = 64;
inline int current_device() {
  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return -1;
  return device;
}
int sm_count(int device);   // multiprocessors of `device` (cached)

// ---- launchers implemented in the .cu files (all enqueue on `st` and return a status) ----
enum GemmMode { GEMM_STORE_BF16 = 0, GEMM_RESID_F32 = 1, GEMM_SWIGLU = 2, GEMM_QKV_ROPE = 3 };

// Extra arguments of the fused QKV epilogue: RoPE on the accumulators, K/V stored into the paged cache.
struct QkvRopeArgs {
  const float2 *rope;       // [head_dim/2, rope_rows] (cos, sin) of each row's position: the 32 rows of a warp read
                            // consecutive entries
  int rope_rows;            // rows of that table (tokens of the call)
  const int *block_table;   // device; single request: row r is position pos0 + r of this table
  const int *row_pos;       // batched requests (else nullptr): position of each row inside its request
  const int *row_block;     // batched requests: physical block that holds each row
  CacheView cache;
  int pos0, head_dim, n_q_heads, n_kv_heads, layer;
};

int gemm_tc(const bf16 *a, int lda, const bf16 *w, int m, int n, int k, int mode, bf16 *out,
            float *resid, int *status_dev, cudaStream_t st, const QkvRopeArgs *qkv_args = nullptr);
// CTA-pair (cta_group::2) variant with 256 x 256 tiles; same contract
int gemm_tc_pair(const bf16 *a, int lda, const bf16 *w, int m, int n, int k, int mode, bf16 *out, float *resid,
                 int *status_dev, cudaStream_t st, const QkvRopeArgs *qkv_args = nullptr);
// the tile width (columns of W per tile) the launchers above pick for an m x n_out problem on `sms` SMs
int gemm_tc_tile_width(int m, int n_out, int sms, int mode, int head_dim);
int gemm_tc_pair_tile_width(int m, int n_out, int sms, int mode, int head_dim);

int embed_rows(const bf16 *embed, const int *ids_dev, int n_tokens, int hidden, float *x, cudaStream_t st);
int rmsnorm_rows(const float *x, const bf16 *gain, int rows, int dim, float eps, bf16 *out, cudaStream_t st);
// positions pos0 + t, or row_pos[t] when row_pos is given (rows of several requests)
int rope_table(float2 *table, int pos0, int n_tokens, int head_dim, float base, cudaStream_t st,
               const int *row_pos = nullptr);
int attention_prefill_tc(const bf16 *qkv_ctx, int n_tokens, int pos0, int n_q_heads, int n_kv_heads, int head_dim,
                         bf16 *out, int *status_dev, cudaStream_t st);
int gather_prefix_kv(bf16 *qkv_ctx, int pos0, int n_q_heads, int n_kv_heads, int head_dim, CacheView cache, int layer,
                     const int *block_table_dev, cudaStream_t st);

// decode-step kernels (one token, fp32 activations)
int embed_one(const bf16 *embed, int token, int hidden, float *x, cudaStream_t st);
// y[n] (+)= sum_k W[n,k] x[k]; mode 0 store, 1 add into y, 2 swiglu over (gate | up) rows
// gain != nullptr fuses RMSNorm(x, gain, eps) into the product (modes 0 and 2)
int gemv(const bf16 *w, const float *x, int n, int k, int mode, float *y, cudaStream_t st,
         const bf16 *gain = nullptr, float eps = 0.f);
// RMSNorm + QKV projection + RoPE + K/V append of one decode token; q_out = rotated fp32 queries;
// rope_dev: (cos, sin) of position `pos` for the head_dim / 2 frequencies (rope_table with one token)
int gemv_qkv_rope(const bf16 *w_qkv, const float *x, const bf16 *gain, float eps, int hidden, int pos, int n_q_heads,
                  int n_kv_heads, int head_dim, const float2 *rope_dev, CacheView cache, int layer,
                  const int *block_table_dev, float *q_out, cudaStream_t st);
long long paged_attention_scratch_bytes(int n_q_heads, int head_dim, int n_ctx);
int paged_attention(const float *q, int n_q_heads, CacheView cache, int layer, const int *block_table_dev,
                    int n_ctx, void *scratch, float *out, cudaStream_t st);

// One request of a pack/unpack call: n_blocks physical ids (host array) and the request's wire buffer (device).
struct CopyRequest {
  const int *ids_host;
  int n_blocks;
  char *wire;
};
// Every page of every request in as few launches as the parameter block allows (one for up to 7,680 blocks
// of up to 64 requests).
int copy_pages(CacheView cache, int n_layers, const CopyRequest *reqs, int n_req, int wire_layout, bool to_wire,
               cudaStream_t st);
int copy_wait_expired(cudaStream_t st);   // KV_ERR_DEVICE if a pack/unpack kernel gave up a wait since the last check
int fill_pattern(void *dst, long long bytes, unsigned long long seed, long long offset, cudaStream_t st);

}  // namespace kvr
