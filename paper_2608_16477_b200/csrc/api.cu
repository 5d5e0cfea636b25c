// C ABI: argument validation on the host, workspace carving and the launch sequences of the four operations.
#include <algorithm>
#include <cstdlib>
#include <atomic>
#include <cstring>
#include <mutex>
#include <string>
#include <vector>

#include "tc_common.cuh"

namespace kvr {

static thread_local std::string g_cuda_error;

void set_cuda_error(cudaError_t e, const char *what) {
  g_cuda_error = std::string(cudaGetErrorName(e)) + ": " + cudaGetErrorString(e) + " in " + what;
  (void)cudaGetLastError();
}

std::atomic<long long> g_launches{0};

int sm_count(int device) {
  static int cached[kMaxDevices] = {};
  if (device < 0 || device >= kMaxDevices) return 148;
  if (cached[device] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || n <= 0) n = 148;
    cached[device] = n;
  }
  return cached[device];
}

// ---- page-locked staging of the host arrays of a call (token ids, block tables, per-row metadata) ----
// A call copies each host array into a page-locked slot owned by the library and enqueues the transfer from there:
// the caller's array may be reused as soon as the call returns whether it is pageable or page-locked, and the
// transfer never makes the host wait for earlier work of the stream.  A slot is reused after kStageSlots later
// uploads on the same device; an event recorded behind its transfer says when that is safe.  Slots grow to the
// largest array seen and live until the process ends.
class HostStage {
 public:
  int upload(void *dst_dev, const void *src_host, size_t bytes, cudaStream_t st) {
    if (bytes == 0) return KV_OK;
    const int device = current_device();
    if (device < 0) return KV_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu_);
    Slot &s = slots_[device][next_[device]];
    next_[device] = (next_[device] + 1) % kStageSlots;
    if (s.busy) {
      KV_CUDA(cudaEventSynchronize(s.done));
      s.busy = false;
    }
    if (s.cap < bytes) {
      if (s.mem != nullptr) KV_CUDA(cudaFreeHost(s.mem));
      s.mem = nullptr;
      s.cap = 0;
      const size_t cap = (bytes + 65535) & ~(size_t)65535;
      KV_CUDA(cudaHostAlloc(&s.mem, cap, cudaHostAllocPortable));
      s.cap = cap;
    }
    if (s.done == nullptr) KV_CUDA(cudaEventCreateWithFlags(&s.done, cudaEventDisableTiming));
    memcpy(s.mem, src_host, bytes);
    KV_CUDA(cudaMemcpyAsync(dst_dev, s.mem, bytes, cudaMemcpyHostToDevice, st));
    KV_CUDA(cudaEventRecord(s.done, st));
    s.busy = true;
    return KV_OK;
  }

 private:
  static constexpr int kStageSlots = 16;
  struct Slot {
    void *mem = nullptr;
    size_t cap = 0;
    cudaEvent_t done = nullptr;
    bool busy = false;
  };
  std::mutex mu_;
  Slot slots_[kMaxDevices][kStageSlots];
  int next_[kMaxDevices] = {};
};

static HostStage &host_stage() {
  static HostStage *stage = new HostStage();   // never destroyed: page-locked memory must not be freed at exit
  return *stage;
}

// ---- optional event profiler: CUDA events around each kernel class, on the caller's stream ----
struct ProfRecord {
  int kind;
  long long launches;
  cudaEvent_t start, stop;
};
static bool g_prof_on = false;
static std::vector<ProfRecord> g_prof_records;
static std::vector<cudaEvent_t> g_prof_pool;

static cudaEvent_t prof_event() {
  if (!g_prof_pool.empty()) {
    cudaEvent_t e = g_prof_pool.back();
    g_prof_pool.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

struct ProfScope {
  int kind;
  cudaStream_t st;
  cudaEvent_t start;
  long long launches0;
  ProfScope(int k, cudaStream_t s) : kind(k), st(s), start(nullptr), launches0(g_launches) {
    if (g_prof_on) {
      start = prof_event();
      cudaEventRecord(start, st);
    }
  }
  ~ProfScope() {
    if (start != nullptr) {
      cudaEvent_t stop = prof_event();
      cudaEventRecord(stop, st);
      g_prof_records.push_back({kind, g_launches - launches0, start, stop});
    }
  }
};

namespace tc {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

int make_tmap_nd(CUtensorMap *map, const void *base, int rank, const unsigned long long *dims,
                 const unsigned long long *strides_bytes, const unsigned int *box) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) {
    g_cuda_error = "cuTensorMapEncodeTiled entry point not available";
    return KV_ERR_CUDA;
  }
  cuuint64_t gdim[5], gstride[5];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < rank; ++i) {
    gdim[i] = dims[i];
    bx[i] = box[i];
    es[i] = 1;
    if (i > 0) gstride[i - 1] = strides_bytes[i - 1];
  }
  const CUtensorMapSwizzle sw = (box[0] * 2 == 128) ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE;
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void *>(base), gdim, gstride,
                  bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    g_cuda_error = "cuTensorMapEncodeTiled failed with CUresult " + std::to_string((int)r);
    return KV_ERR_CUDA;
  }
  return KV_OK;
}

int make_tmap_2d(CUtensorMap *map, const void *base, long long rows, long long cols, long long ld, int box_rows,
                 int box_cols) {
  const unsigned long long dims[2] = {(unsigned long long)cols, (unsigned long long)rows};
  const unsigned long long strides[1] = {(unsigned long long)ld * 2ull};
  const unsigned int box[2] = {(unsigned int)box_cols, (unsigned int)box_rows};
  return make_tmap_nd(map, base, 2, dims, strides, box);
}

}  // namespace tc
}  // namespace kvr

using namespace kvr;

// Self-test of the bounded-wait machinery every tensor-core kernel relies on: thread 0 waits, with the kernels' own
// wait routine and a short limit, on an mbarrier that nothing ever arrives on.  The wait must give up, record itself in
// the status block and raise the CTA's abort flag; the second warp, waiting on the same barrier, must leave through
// that flag without recording anything; the kernel then returns normally.  detail[3] = number of threads whose wait
// reported failure (64 when everything works).
constexpr int kTagSelfTest = 99;
__global__ void bounded_wait_selftest_kernel(DeviceStatus *status, long long limit_cycles) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  __shared__ int gave_up;
  if (threadIdx.x == 0) {
    tc::mbar_init(tc::smem_u32(&bar), 1);
    abort_flag = 0;
    gave_up = 0;
    tc::fence_barrier_init();
  }
  __syncthreads();
  // thread 0 carries the short limit; everybody else would wait for the full ~1 s and must be released by the flag
  const bool ok = tc::mbar_wait(tc::smem_u32(&bar), 0, &abort_flag, status, kTagSelfTest,
                                threadIdx.x == 0 ? limit_cycles : tc::kWaitLimitCycles);
  if (!ok) atomicAdd(&gave_up, 1);
  __syncthreads();
  if (threadIdx.x == 0) status->detail[3] = gave_up;
}

struct kv_model {
  kv_model_desc d;
  const bf16 *embed, *lm_head, *final_norm;
  std::vector<const bf16 *> attn_norm, w_qkv, w_o, ffn_norm, w_gate_up, w_down;
};

namespace {

inline long long align_up(long long v, long long a) { return (v + a - 1) / a * a; }

struct Carver {
  char *base;
  long long off;
  explicit Carver(void *b) : base((char *)b), off(0) {}
  template <typename T>
  T *take(long long count) {
    T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
    off = align_up(off + count * (long long)sizeof(T), 1024);
    return p;
  }
};

struct PrefillWs {
  DeviceStatus *status;
  int *ids, *table, *row_meta;
  float2 *rope;
  float *x, *xf;
  bf16 *h, *qkv, *attn, *mid;
  long long bytes;
};

// The layout depends on the model and on max_tokens only (the block table is sized for one block per token), so
// kv_workspace_bytes and kv_workspace_residual describe exactly what the operations carve.
PrefillWs carve_prefill(const kv_model_desc &d, void *base, int max_tokens, int /*block_size*/) {
  Carver c(base);
  PrefillWs w;
  const long long t = max_tokens;
  const long long qkv_dim = (long long)(d.n_q_heads + 2 * d.n_kv_heads) * d.head_dim;
  w.status = c.take<DeviceStatus>(1);
  w.ids = c.take<int>(t);
  w.table = c.take<int>(t + 1);
  w.row_meta = c.take<int>(2 * t);
  w.rope = c.take<float2>(t * (d.head_dim / 2));
  w.x = c.take<float>(t * d.hidden);
  w.xf = c.take<float>(d.hidden);
  w.h = c.take<bf16>(t * d.hidden);
  w.qkv = c.take<bf16>(t * qkv_dim);
  w.attn = c.take<bf16>(t * d.n_q_heads * d.head_dim);
  w.mid = c.take<bf16>(t * d.ffn);
  w.bytes = c.off;
  return w;
}

struct DecodeWs {
  DeviceStatus *status;
  int *table;
  float2 *rope;
  float *x, *h, *qkv, *o, *mid;
  void *scratch;
  long long bytes;
};

DecodeWs carve_decode(const kv_model_desc &d, void *base, int max_ctx, int /*block_size*/) {
  Carver c(base);
  DecodeWs w;
  const long long qkv_dim = (long long)(d.n_q_heads + 2 * d.n_kv_heads) * d.head_dim;
  w.status = c.take<DeviceStatus>(1);
  w.table = c.take<int>(max_ctx + 1);
  w.rope = c.take<float2>(d.head_dim / 2);
  w.x = c.take<float>(d.hidden);
  w.h = c.take<float>(d.hidden);
  w.qkv = c.take<float>(qkv_dim);
  w.o = c.take<float>((long long)d.n_q_heads * d.head_dim);
  w.mid = c.take<float>(d.ffn);
  w.scratch = c.take<char>(paged_attention_scratch_bytes(d.n_q_heads, d.head_dim, max_ctx));
  w.bytes = c.off;
  return w;
}

int check_cache(const kv_cache_desc *c) { return check_cache_desc(c); }

int check_cache_vs_model(const kv_cache_desc *c, const kv_model_desc &d) {
  int rc = check_cache(c);
  if (rc != KV_OK) return rc;
  if (c->n_layers != d.n_layers || c->n_kv_heads != d.n_kv_heads || c->head_dim != d.head_dim) return KV_ERR_SHAPE;
  return KV_OK;
}

int check_ids(const int32_t *ids, int n, int num_blocks, bool reject_duplicates) {
  for (int i = 0; i < n; ++i)
    if (ids[i] < 0 || ids[i] >= num_blocks) return KV_ERR_BLOCK_RANGE;
  if (reject_duplicates) {
    std::vector<int32_t> s(ids, ids + n);
    std::sort(s.begin(), s.end());
    if (std::adjacent_find(s.begin(), s.end()) != s.end()) return KV_ERR_BLOCK_ALIAS;
  }
  return KV_OK;
}

long long wire_bytes_needed(const kv_cache_desc *c, int n_blocks) {
  return (long long)n_blocks * c->n_layers * 2 * c->block_size * c->n_kv_heads * c->head_dim * 2;
}

// Up to 128 rows (one row tile) the one-CTA kernel runs; from there on the CTA-pair kernel was as fast or faster
// for every projection measured (512 to 16,384 rows).
inline bool gemm_uses_pair(int rows) { return rows > 128; }

int run_gemm(const kv_model *, const bf16 *a, int lda, const bf16 *w, int rows, int n, int k, int mode, bf16 *out,
             float *resid, DeviceStatus *status, cudaStream_t st, const QkvRopeArgs *qa = nullptr) {
  if (gemm_uses_pair(rows))
    return gemm_tc_pair(a, lda, w, rows, n, k, mode, out, resid, reinterpret_cast<int *>(status), st, qa);
  return gemm_tc(a, lda, w, rows, n, k, mode, out, resid, reinterpret_cast<int *>(status), st, qa);
}

}  // namespace

extern "C" {

int32_t kv_model_create(const kv_model_desc *desc, const kv_weights *w, kv_model **out) {
  if (desc == nullptr || w == nullptr || out == nullptr) return KV_ERR_ARG;
  const kv_model_desc &d = *desc;
  if (d.n_layers <= 0 || d.hidden <= 0 || d.n_q_heads <= 0 || d.n_kv_heads <= 0 || d.head_dim <= 0 || d.ffn <= 0 ||
      d.vocab <= 0)
    return KV_ERR_ARG;
  if (d.n_q_heads % d.n_kv_heads != 0 || (d.head_dim != 64 && d.head_dim != 128) || d.hidden % 8 != 0 ||
      d.ffn % 8 != 0)
    return KV_ERR_SHAPE;
  if (!w->embed_dev || !w->lm_head_dev || !w->final_norm_dev || !w->attn_norm_dev || !w->w_qkv_dev || !w->w_o_dev ||
      !w->ffn_norm_dev || !w->w_gate_up_dev || !w->w_down_dev)
    return KV_ERR_ARG;
  if (((uintptr_t)w->embed_dev & 15) || ((uintptr_t)w->lm_head_dev & 15) || ((uintptr_t)w->final_norm_dev & 15))
    return KV_ERR_ARG;
  kv_model *m = new kv_model();
  m->d = d;
  m->embed = (const bf16 *)w->embed_dev;
  m->lm_head = (const bf16 *)w->lm_head_dev;
  m->final_norm = (const bf16 *)w->final_norm_dev;
  for (int l = 0; l < d.n_layers; ++l) {
    const void *ptrs[6] = {w->attn_norm_dev[l], w->w_qkv_dev[l], w->w_o_dev[l],
                           w->ffn_norm_dev[l],  w->w_gate_up_dev[l], w->w_down_dev[l]};
    for (const void *p : ptrs)
      if (p == nullptr || ((uintptr_t)p & 15)) {
        delete m;
        return KV_ERR_ARG;
      }
    m->attn_norm.push_back((const bf16 *)ptrs[0]);
    m->w_qkv.push_back((const bf16 *)ptrs[1]);
    m->w_o.push_back((const bf16 *)ptrs[2]);
    m->ffn_norm.push_back((const bf16 *)ptrs[3]);
    m->w_gate_up.push_back((const bf16 *)ptrs[4]);
    m->w_down.push_back((const bf16 *)ptrs[5]);
  }
  *out = m;
  return KV_OK;
}

int32_t kv_model_destroy(kv_model *m) {
  delete m;
  return KV_OK;
}

int64_t kv_workspace_bytes(const kv_model *m, int32_t op, int32_t max_tokens) {
  if (m == nullptr || max_tokens <= 0) return KV_ERR_ARG;
  if (op == KV_OP_PREFILL) return carve_prefill(m->d, nullptr, max_tokens, 1).bytes;
  if (op == KV_OP_DECODE) return carve_decode(m->d, nullptr, max_tokens, 1).bytes;
  return KV_ERR_ARG;
}

int32_t kv_workspace_residual(const kv_model *m, int32_t op, int32_t max_tokens, int64_t *offset_out,
                              int64_t *bytes_out) {
  if (m == nullptr || max_tokens <= 0 || offset_out == nullptr || bytes_out == nullptr) return KV_ERR_ARG;
  // carve over a made-up base address (never dereferenced) to learn where the piece sits
  char *fake = reinterpret_cast<char *>((uintptr_t)1 << 40);
  if (op == KV_OP_PREFILL) {
    const PrefillWs w = carve_prefill(m->d, fake, max_tokens, 1);
    *offset_out = (int64_t)(reinterpret_cast<const char *>(w.x) - fake);
    *bytes_out = (int64_t)max_tokens * m->d.hidden * 4;
    return KV_OK;
  }
  if (op == KV_OP_DECODE) {
    const DecodeWs w = carve_decode(m->d, fake, max_tokens, 1);
    *offset_out = (int64_t)(reinterpret_cast<const char *>(w.x) - fake);
    *bytes_out = (int64_t)m->d.hidden * 4;
    return KV_OK;
  }
  return KV_ERR_ARG;
}

const char *kv_status_string(int32_t s) {
  switch (s) {
    case KV_OK: return "ok";
    case KV_ERR_ARG: return "invalid argument";
    case KV_ERR_SHAPE: return "shape mismatch or unsupported shape";
    case KV_ERR_BLOCK_RANGE: return "physical block id out of range";
    case KV_ERR_BLOCK_ALIAS: return "physical block id used twice";
    case KV_ERR_GAP: return "logical suffix block missing";
    case KV_ERR_OVERLAP: return "logical suffix block duplicated or outside the suffix";
    case KV_ERR_SPLIT_UNALIGNED: return "split position not block-aligned";
    case KV_ERR_TABLE_SHORT: return "block table does not cover the tokens";
    case KV_ERR_WIRE_SIZE: return "wire buffer too small";
    case KV_ERR_WORKSPACE: return "workspace too small or misaligned";
    case KV_ERR_STALE_EPOCH: return "stale migration epoch";
    case KV_ERR_TOKEN_RANGE: return "token id out of range";
    case KV_ERR_CUDA: return "CUDA call failed";
    case KV_ERR_DEVICE: return "device-side bounded wait ran out";
    default: return "unknown status";
  }
}

const char *kv_last_cuda_error(void) { return g_cuda_error.c_str(); }

int64_t kv_bytes_per_token(int32_t n_layers, int32_t n_kv_heads, int32_t head_dim, int32_t elem_bytes) {
  return 2ll * n_layers * n_kv_heads * head_dim * elem_bytes;
}

int32_t kv_check_device_status(const void *workspace_dev, void *stream) {
  if (workspace_dev == nullptr) return KV_ERR_ARG;
  DeviceStatus s;
  KV_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
  KV_CUDA(cudaMemcpy(&s, workspace_dev, sizeof(s), cudaMemcpyDeviceToHost));
  if (s.error != 0) {
    g_cuda_error = "device wait ran out: tag " + std::to_string(s.where) + " block " + std::to_string(s.detail[0]) +
                   " thread " + std::to_string(s.detail[1]);
    return KV_ERR_DEVICE;
  }
  return KV_OK;
}

#define KV_TRY(expr)            \
  do {                          \
    int rc__ = (expr);          \
    if (rc__ != KV_OK) return rc__; \
  } while (0)

namespace {

// One request inside a prefill launch sequence: rows [row0, row0 + n_tokens) of the activation buffers.
struct PrefillSegment {
  int row0, n_tokens;
  float *logits;   // nullable
};

// The layer loop shared by the single-request and the batched entry points.  All rows of all segments go
// through the projections together; attention runs per segment (requests do not attend to each other).
// Single request: pos0 may be > 0 (continued prefill) and rows map to the request's block table.  Batched:
// pos0 = 0 and every row carries its own position and physical block (row_pos / row_block on the device).
int prefill_layers(kv_model *m, const CacheView &cv, PrefillWs &w, int total_rows, int pos0,
                   const std::vector<PrefillSegment> &segs, const int *row_pos, const int *row_block, bool any_logits,
                   cudaStream_t st) {
  const kv_model_desc &d = m->d;
  const int t = total_rows;
  const int qkv_dim = (d.n_q_heads + 2 * d.n_kv_heads) * d.head_dim;
  const int q_dim = d.n_q_heads * d.head_dim;
  { ProfScope ps(PROF_ROPE_STORE, st); KV_TRY(rope_table(w.rope, pos0, t, d.head_dim, d.rope_base, st, row_pos)); }
  // the qkv buffer has one row per context position; the chunk's rows start at pos0
  bf16 *qkv_chunk = w.qkv + (long long)pos0 * qkv_dim;
  { ProfScope ps(PROF_EMBED, st); KV_TRY(embed_rows(m->embed, w.ids, t, d.hidden, w.x, st)); }
  for (int l = 0; l < d.n_layers; ++l) {
    { ProfScope ps(PROF_RMSNORM, st); KV_TRY(rmsnorm_rows(w.x, m->attn_norm[l], t, d.hidden, d.rms_eps, w.h, st)); }
    {
      ProfScope ps(PROF_GEMM_QKV, st);
      QkvRopeArgs qa;
      qa.rope = w.rope;
      qa.rope_rows = t;
      qa.block_table = w.table;
      qa.row_pos = row_pos;
      qa.row_block = row_block;
      qa.cache = cv;
      qa.pos0 = pos0;
      qa.head_dim = d.head_dim;
      qa.n_q_heads = d.n_q_heads;
      qa.n_kv_heads = d.n_kv_heads;
      qa.layer = l;
      KV_TRY(run_gemm(m, w.h, d.hidden, m->w_qkv[l], t, qkv_dim, d.hidden, GEMM_QKV_ROPE, qkv_chunk, nullptr, w.status, st, &qa));
    }
    if (l == d.n_layers - 1 && !any_logits) break;   // K/V of the last layer are complete
    {
      ProfScope ps(PROF_ATTENTION, st);
      for (const PrefillSegment &sg : segs) {
        bf16 *seg_qkv = w.qkv + (long long)sg.row0 * qkv_dim;     // rows of this request (its context starts here)
        bf16 *seg_out = w.attn + (long long)sg.row0 * q_dim;
        KV_TRY(gather_prefix_kv(seg_qkv, pos0, d.n_q_heads, d.n_kv_heads, d.head_dim, cv, l, w.table, st));
        KV_TRY(attention_prefill_tc(seg_qkv, sg.n_tokens, pos0, d.n_q_heads, d.n_kv_heads, d.head_dim, seg_out,
                                    reinterpret_cast<int *>(w.status), st));
      }
    }
    { ProfScope ps(PROF_GEMM_O, st); KV_TRY(run_gemm(m, w.attn, q_dim, m->w_o[l], t, d.hidden, q_dim, GEMM_RESID_F32, nullptr, w.x, w.status, st)); }
    { ProfScope ps(PROF_RMSNORM, st); KV_TRY(rmsnorm_rows(w.x, m->ffn_norm[l], t, d.hidden, d.rms_eps, w.h, st)); }
    { ProfScope ps(PROF_GEMM_GATE_UP, st); KV_TRY(run_gemm(m, w.h, d.hidden, m->w_gate_up[l], t, d.ffn, d.hidden, GEMM_SWIGLU, w.mid, nullptr, w.status, st)); }
    { ProfScope ps(PROF_GEMM_DOWN, st); KV_TRY(run_gemm(m, w.mid, d.ffn, m->w_down[l], t, d.hidden, d.ffn, GEMM_RESID_F32, nullptr, w.x, w.status, st)); }
  }
  for (const PrefillSegment &sg : segs) {
    if (sg.logits == nullptr) continue;
    ProfScope ps(PROF_LM_HEAD, st);
    KV_TRY(gemv(m->lm_head, w.x + (long long)(sg.row0 + sg.n_tokens - 1) * d.hidden, d.vocab, d.hidden, 0, sg.logits, st,
                m->final_norm, d.rms_eps));
  }
  return KV_OK;
}

}  // namespace

int32_t kv_prefill_prefix(kv_model *m, const kv_cache_desc *cache, const int32_t *token_ids_host, int32_t n_tokens,
                          int32_t pos0, const int32_t *block_table_host, int32_t n_blocks, void *workspace_dev,
                          int64_t workspace_bytes, float *logits_out_dev, void *stream) {
  if (m == nullptr || token_ids_host == nullptr || block_table_host == nullptr || n_tokens <= 0 || pos0 < 0 ||
      n_blocks <= 0)
    return KV_ERR_ARG;
  const kv_model_desc &d = m->d;
  int rc = check_cache_vs_model(cache, d);
  if (rc != KV_OK) return rc;
  const int bs = cache->block_size;
  if (pos0 % bs != 0) return KV_ERR_SPLIT_UNALIGNED;
  const long long n_ctx = (long long)pos0 + n_tokens;
  const long long need_blocks = (n_ctx + bs - 1) / bs;
  if (n_blocks < need_blocks) return KV_ERR_TABLE_SHORT;
  rc = check_ids(block_table_host, (int)need_blocks, cache->num_blocks, true);
  if (rc != KV_OK) return rc;
  for (int i = 0; i < n_tokens; ++i)
    if (token_ids_host[i] < 0 || token_ids_host[i] >= d.vocab) return KV_ERR_TOKEN_RANGE;
  if (workspace_dev == nullptr || ((uintptr_t)workspace_dev & 1023)) return KV_ERR_WORKSPACE;
  PrefillWs w = carve_prefill(d, workspace_dev, (int)n_ctx, bs);
  if (workspace_bytes < w.bytes) return KV_ERR_WORKSPACE;
  // buffers are sized by the context length n_ctx; only the first n_tokens rows are used
  cudaStream_t st = (cudaStream_t)stream;
  KV_CUDA(cudaMemsetAsync(w.status, 0, sizeof(DeviceStatus), st));
  KV_TRY(host_stage().upload(w.ids, token_ids_host, sizeof(int) * n_tokens, st));
  KV_TRY(host_stage().upload(w.table, block_table_host, sizeof(int) * need_blocks, st));
  std::vector<PrefillSegment> segs{{0, n_tokens, logits_out_dev}};
  return prefill_layers(m, make_view(cache), w, n_tokens, pos0, segs, nullptr, nullptr, logits_out_dev != nullptr, st);
}

int32_t kv_prefill_prefix_batched(kv_model *m, const kv_cache_desc *cache, int32_t n_req,
                                  const int32_t *token_offsets_host, const int32_t *token_ids_host,
                                  const int32_t *table_offsets_host, const int32_t *block_tables_host,
                                  void *workspace_dev, int64_t workspace_bytes, float *logits_out_dev, void *stream) {
  if (m == nullptr || n_req <= 0 || token_offsets_host == nullptr || token_ids_host == nullptr ||
      table_offsets_host == nullptr || block_tables_host == nullptr)
    return KV_ERR_ARG;
  const kv_model_desc &d = m->d;
  int rc = check_cache_vs_model(cache, d);
  if (rc != KV_OK) return rc;
  const int bs = cache->block_size;
  if (token_offsets_host[0] != 0 || table_offsets_host[0] != 0) return KV_ERR_ARG;
  const int total = token_offsets_host[n_req];
  const int total_blocks = table_offsets_host[n_req];
  if (total <= 0 || total_blocks <= 0) return KV_ERR_ARG;
  std::vector<int> row_meta(2 * (size_t)total);   // [0, total): position in request, [total, 2 total): physical block
  std::vector<PrefillSegment> segs;
  for (int r = 0; r < n_req; ++r) {
    const int n_tok = token_offsets_host[r + 1] - token_offsets_host[r];
    const int n_blk = table_offsets_host[r + 1] - table_offsets_host[r];
    if (n_tok <= 0 || n_blk < 0) return KV_ERR_ARG;
    if ((long long)n_blk * bs < n_tok) return KV_ERR_TABLE_SHORT;
    const int32_t *tab = block_tables_host + table_offsets_host[r];
    for (int i = 0; i < n_tok; ++i) {
      row_meta[token_offsets_host[r] + i] = i;
      row_meta[(size_t)total + token_offsets_host[r] + i] = tab[i / bs];
    }
    segs.push_back({token_offsets_host[r], n_tok, logits_out_dev ? logits_out_dev + (long long)r * d.vocab : nullptr});
  }
  // physical blocks: in range and distinct across ALL requests (two requests must never share a page)
  rc = check_ids(block_tables_host, total_blocks, cache->num_blocks, true);
  if (rc != KV_OK) return rc;
  for (int i = 0; i < total; ++i)
    if (token_ids_host[i] < 0 || token_ids_host[i] >= d.vocab) return KV_ERR_TOKEN_RANGE;
  if (workspace_dev == nullptr || ((uintptr_t)workspace_dev & 1023)) return KV_ERR_WORKSPACE;
  PrefillWs w = carve_prefill(d, workspace_dev, total, bs);
  if (workspace_bytes < w.bytes) return KV_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  KV_CUDA(cudaMemsetAsync(w.status, 0, sizeof(DeviceStatus), st));
  KV_TRY(host_stage().upload(w.ids, token_ids_host, sizeof(int) * total, st));
  KV_TRY(host_stage().upload(w.row_meta, row_meta.data(), sizeof(int) * 2 * total, st));
  return prefill_layers(m, make_view(cache), w, total, 0, segs, w.row_meta, w.row_meta + total, logits_out_dev != nullptr,
                        st);
}

int32_t kv_decode_step(kv_model *m, const kv_cache_desc *cache, int32_t token_id, int32_t pos,
                       const int32_t *block_table_host, int32_t n_blocks, void *workspace_dev,
                       int64_t workspace_bytes, float *logits_out_dev, void *stream) {
  if (m == nullptr || block_table_host == nullptr || pos < 0 || n_blocks <= 0 || logits_out_dev == nullptr)
    return KV_ERR_ARG;
  const kv_model_desc &d = m->d;
  int rc = check_cache_vs_model(cache, d);
  if (rc != KV_OK) return rc;
  const int bs = cache->block_size;
  const int n_ctx = pos + 1;
  const int need_blocks = (n_ctx + bs - 1) / bs;
  if (n_blocks < need_blocks) return KV_ERR_TABLE_SHORT;
  rc = check_ids(block_table_host, need_blocks, cache->num_blocks, true);
  if (rc != KV_OK) return rc;
  if (token_id < 0 || token_id >= d.vocab) return KV_ERR_TOKEN_RANGE;
  if (workspace_dev == nullptr || ((uintptr_t)workspace_dev & 1023)) return KV_ERR_WORKSPACE;
  DecodeWs w = carve_decode(d, workspace_dev, n_ctx, bs);
  if (workspace_bytes < w.bytes) return KV_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  const CacheView cv = make_view(cache);
  const int q_dim = d.n_q_heads * d.head_dim;

  KV_CUDA(cudaMemsetAsync(w.status, 0, sizeof(DeviceStatus), st));
  KV_TRY(host_stage().upload(w.table, block_table_host, sizeof(int) * need_blocks, st));
  {
    ProfScope ps(PROF_DECODE_OTHER, st);
    KV_TRY(rope_table(w.rope, pos, 1, d.head_dim, d.rope_base, st));
    KV_TRY(embed_one(m->embed, token_id, d.hidden, w.x, st));
  }
  for (int l = 0; l < d.n_layers; ++l) {
    { ProfScope ps(PROF_DECODE_GEMV, st); KV_TRY(gemv_qkv_rope(m->w_qkv[l], w.x, m->attn_norm[l], d.rms_eps, d.hidden, pos, d.n_q_heads, d.n_kv_heads, d.head_dim, w.rope, cv, l, w.table, w.qkv, st)); }
    { ProfScope ps(PROF_DECODE_ATTENTION, st); KV_TRY(paged_attention(w.qkv, d.n_q_heads, cv, l, w.table, n_ctx, w.scratch, w.o, st)); }
    { ProfScope ps(PROF_DECODE_GEMV, st); KV_TRY(gemv(m->w_o[l], w.o, d.hidden, q_dim, 1, w.x, st)); }
    { ProfScope ps(PROF_DECODE_GEMV, st); KV_TRY(gemv(m->w_gate_up[l], w.x, d.ffn, d.hidden, 2, w.mid, st, m->ffn_norm[l], d.rms_eps)); }
    { ProfScope ps(PROF_DECODE_GEMV, st); KV_TRY(gemv(m->w_down[l], w.mid, d.hidden, d.ffn, 1, w.x, st)); }
  }
  { ProfScope ps(PROF_LM_HEAD, st); KV_TRY(gemv(m->lm_head, w.x, d.vocab, d.hidden, 0, logits_out_dev, st, m->final_norm, d.rms_eps)); }
  return KV_OK;
}

int32_t kv_pack_blocks(const kv_cache_desc *src, const int32_t *block_ids_host, int32_t n_blocks, void *wire_dev,
                       int64_t wire_bytes, int32_t wire_layout, void *stream) {
  if (block_ids_host == nullptr || n_blocks < 0 || wire_dev == nullptr || ((uintptr_t)wire_dev & 15)) return KV_ERR_ARG;
  if (wire_layout != KV_WIRE_BLOCK_MAJOR && wire_layout != KV_WIRE_LAYER_MAJOR) return KV_ERR_ARG;
  int rc = check_cache(src);
  if (rc != KV_OK) return rc;
  rc = check_ids(block_ids_host, n_blocks, src->num_blocks, false);
  if (rc != KV_OK) return rc;
  if (wire_bytes < wire_bytes_needed(src, n_blocks)) return KV_ERR_WIRE_SIZE;
  if (n_blocks == 0) return KV_OK;
  ProfScope ps(PROF_PACK, (cudaStream_t)stream);
  const CopyRequest req{block_ids_host, n_blocks, (char *)wire_dev};
  return copy_pages(make_view(src), src->n_layers, &req, 1, wire_layout, true, (cudaStream_t)stream);
}

int32_t kv_unpack_assemble(const kv_cache_desc *dst, const void *wire_dev, int64_t wire_bytes, int32_t wire_layout,
                           const int32_t *logical, const int32_t *dst_ids, int32_t n_suffix,
                           const int32_t *prefix_table, int32_t n_prefix, int32_t n_tokens_total, uint32_t epoch,
                           uint32_t expected_epoch, int32_t *merged_out, void *stream) {
  if (epoch != expected_epoch) return KV_ERR_STALE_EPOCH;
  if (n_suffix < 0 || n_prefix < 0 || n_tokens_total < 0 || merged_out == nullptr) return KV_ERR_ARG;
  if ((n_suffix > 0 && (logical == nullptr || dst_ids == nullptr || wire_dev == nullptr)) ||
      (n_prefix > 0 && prefix_table == nullptr) || ((uintptr_t)wire_dev & 15))
    return KV_ERR_ARG;
  if (wire_layout != KV_WIRE_BLOCK_MAJOR && wire_layout != KV_WIRE_LAYER_MAJOR) return KV_ERR_ARG;
  int rc = check_cache(dst);
  if (rc != KV_OK) return rc;
  const int bs = dst->block_size;
  const long long total_blocks = ((long long)n_tokens_total + bs - 1) / bs;
  // physical ids: in range, pairwise distinct across prefix and suffix ("without ... conflicts")
  std::vector<int32_t> phys(prefix_table, prefix_table + n_prefix);
  phys.insert(phys.end(), dst_ids, dst_ids + n_suffix);
  rc = check_ids(phys.data(), (int)phys.size(), dst->num_blocks, true);
  if (rc != KV_OK) return rc;
  // logical blocks: exactly {n_prefix .. total_blocks-1}, each once ("without gaps")
  std::vector<char> seen((size_t)std::max<long long>(total_blocks, 1), 0);
  long long covered = 0;
  for (int i = 0; i < n_suffix; ++i) {
    const long long lb = logical[i];
    if (lb < n_prefix || lb >= total_blocks || seen[(size_t)lb]) return KV_ERR_OVERLAP;
    seen[(size_t)lb] = 1;
    ++covered;
  }
  if (covered != total_blocks - n_prefix) return KV_ERR_GAP;
  if (wire_bytes < wire_bytes_needed(dst, n_suffix)) return KV_ERR_WIRE_SIZE;
  if (n_suffix > 0) {
    ProfScope ps(PROF_UNPACK, (cudaStream_t)stream);
    const CopyRequest req{dst_ids, n_suffix, (char *)const_cast<void *>(wire_dev)};
    rc = copy_pages(make_view(dst), dst->n_layers, &req, 1, wire_layout, false, (cudaStream_t)stream);
    if (rc != KV_OK) return rc;
  }
  for (int i = 0; i < n_prefix; ++i) merged_out[i] = prefix_table[i];
  for (int i = 0; i < n_suffix; ++i) merged_out[logical[i]] = dst_ids[i];
  return KV_OK;
}

static int32_t batched(const kv_cache_desc *c, int32_t n_req, const int32_t *offs, const int32_t *ids,
                       void *const *wires, int32_t layout, bool to_wire, void *stream) {
  if (n_req < 0 || offs == nullptr || ids == nullptr || wires == nullptr) return KV_ERR_ARG;
  if (layout != KV_WIRE_BLOCK_MAJOR && layout != KV_WIRE_LAYER_MAJOR) return KV_ERR_ARG;
  int rc = check_cache(c);
  if (rc != KV_OK) return rc;
  if (n_req == 0) return KV_OK;
  if (offs[0] != 0) return KV_ERR_ARG;
  for (int r = 0; r < n_req; ++r) {
    if (offs[r + 1] < offs[r]) return KV_ERR_ARG;
    if (offs[r + 1] > offs[r] && (wires[r] == nullptr || ((uintptr_t)wires[r] & 15))) return KV_ERR_ARG;
  }
  // destinations must not alias across the whole batch; sources may repeat
  rc = check_ids(ids, offs[n_req], c->num_blocks, !to_wire);
  if (rc != KV_OK) return rc;
  std::vector<CopyRequest> reqs;
  for (int r = 0; r < n_req; ++r)
    if (offs[r + 1] > offs[r]) reqs.push_back({ids + offs[r], offs[r + 1] - offs[r], (char *)wires[r]});
  if (reqs.empty()) return KV_OK;
  ProfScope ps(to_wire ? PROF_PACK : PROF_UNPACK, (cudaStream_t)stream);
  return copy_pages(make_view(c), c->n_layers, reqs.data(), (int)reqs.size(), layout, to_wire, (cudaStream_t)stream);
}

int32_t kv_pack_blocks_batched(const kv_cache_desc *src, int32_t n_req, const int32_t *blk_offsets_host,
                               const int32_t *block_ids_host, void *const *wire_dev_ptrs_host, int32_t wire_layout,
                               void *stream) {
  return batched(src, n_req, blk_offsets_host, block_ids_host, wire_dev_ptrs_host, wire_layout, true, stream);
}

int32_t kv_unpack_blocks_batched(const kv_cache_desc *dst, int32_t n_req, const int32_t *blk_offsets_host,
                                 const int32_t *dst_block_ids_host, const void *const *wire_dev_ptrs_host,
                                 int32_t wire_layout, void *stream) {
  return batched(dst, n_req, blk_offsets_host, dst_block_ids_host, const_cast<void *const *>(wire_dev_ptrs_host),
                 wire_layout, false, stream);
}

int32_t kv_op_gemm(const void *a_dev, int32_t lda, const void *w_dev, int32_t m, int32_t n, int32_t k, int32_t mode,
                   void *out_dev, float *resid_dev, int32_t *status_dev, void *stream) {
  const bool pair = (mode & KV_GEMM_CTA_PAIR) != 0;
  mode &= ~KV_GEMM_CTA_PAIR;
  if (a_dev == nullptr || w_dev == nullptr || mode < 0 || mode > 2) return KV_ERR_ARG;
  if (m < 0 || n <= 0 || k <= 0 || lda < k) return KV_ERR_ARG;
  if ((mode == GEMM_RESID_F32 && resid_dev == nullptr) || (mode != GEMM_RESID_F32 && out_dev == nullptr)) return KV_ERR_ARG;
  // the epilogues store 16-byte vectors (bf16 output) and update the residual stream as float4
  if (((uintptr_t)out_dev & 15) || ((uintptr_t)resid_dev & 15) || ((uintptr_t)status_dev & 3)) return KV_ERR_ARG;
  if (pair)
    return gemm_tc_pair((const bf16 *)a_dev, lda, (const bf16 *)w_dev, m, n, k, mode, (bf16 *)out_dev, resid_dev,
                        status_dev, (cudaStream_t)stream);
  return gemm_tc((const bf16 *)a_dev, lda, (const bf16 *)w_dev, m, n, k, mode, (bf16 *)out_dev, resid_dev, status_dev,
                 (cudaStream_t)stream);
}

int32_t kv_gemm_plan(int32_t m, int32_t n, int32_t mode, int32_t head_dim, int32_t *cta_pair_out,
                     int32_t *tile_width_out) {
  if (m <= 0 || n <= 0 || mode < 0 || mode > GEMM_QKV_ROPE || cta_pair_out == nullptr || tile_width_out == nullptr)
    return KV_ERR_ARG;
  if (mode == GEMM_QKV_ROPE && head_dim != 64 && head_dim != 128) return KV_ERR_SHAPE;
  const int sms = sm_count(current_device());
  const int hd = mode == GEMM_QKV_ROPE ? head_dim : 0;
  *cta_pair_out = gemm_uses_pair(m) ? 1 : 0;
  *tile_width_out = gemm_uses_pair(m) ? gemm_tc_pair_tile_width(m, n, sms, mode, hd) : gemm_tc_tile_width(m, n, sms, mode, hd);
  return KV_OK;
}

int32_t kv_op_gemv(const void *w_dev, const float *x_dev, int32_t n, int32_t k, int32_t mode, const void *gain_dev,
                   float eps, float *y_dev, void *stream) {
  if (w_dev == nullptr || x_dev == nullptr || y_dev == nullptr || n <= 0 || k <= 0 || mode < 0 || mode > 2)
    return KV_ERR_ARG;
  if (((uintptr_t)w_dev & 15) || ((uintptr_t)x_dev & 15) || (gain_dev != nullptr && ((uintptr_t)gain_dev & 15)))
    return KV_ERR_ARG;
  if (gain_dev != nullptr && mode == 1) return KV_ERR_ARG;
  return gemv((const bf16 *)w_dev, x_dev, n, k, mode, y_dev, (cudaStream_t)stream, (const bf16 *)gain_dev, eps);
}

int32_t kv_op_rmsnorm(const float *x_dev, const void *gain_dev, int32_t rows, int32_t dim, float eps, void *out_dev,
                      void *stream) {
  if (x_dev == nullptr || gain_dev == nullptr || out_dev == nullptr || rows < 0 || dim <= 0 || dim % 4 != 0)
    return KV_ERR_ARG;
  // the kernel reads x as float4 and gain as 4 x bf16, and writes 4 x bf16 at a time
  if (((uintptr_t)x_dev & 15) || ((uintptr_t)gain_dev & 7) || ((uintptr_t)out_dev & 7)) return KV_ERR_ARG;
  return rmsnorm_rows(x_dev, (const bf16 *)gain_dev, rows, dim, eps, (bf16 *)out_dev, (cudaStream_t)stream);
}

int32_t kv_op_attention_prefill(void *qkv_ctx_dev, int32_t n_tokens, int32_t pos0, int32_t n_q_heads,
                                int32_t n_kv_heads, int32_t head_dim, const kv_cache_desc *cache, int32_t layer,
                                const int32_t *block_table_dev, void *out_dev, int32_t *status_dev, void *stream) {
  if (qkv_ctx_dev == nullptr || out_dev == nullptr || n_tokens < 0 || pos0 < 0 || n_q_heads <= 0 || n_kv_heads <= 0)
    return KV_ERR_ARG;
  if (((uintptr_t)qkv_ctx_dev & 15) || ((uintptr_t)out_dev & 15)) return KV_ERR_ARG;
  if ((head_dim != 64 && head_dim != 128) || n_q_heads % n_kv_heads != 0) return KV_ERR_SHAPE;
  if (pos0 > 0) {
    int rc = check_cache(cache);
    if (rc != KV_OK) return rc;
    if (block_table_dev == nullptr || layer < 0 || layer >= cache->n_layers) return KV_ERR_ARG;
    if (cache->n_kv_heads != n_kv_heads || cache->head_dim != head_dim) return KV_ERR_SHAPE;
    if (pos0 % cache->block_size != 0) return KV_ERR_SPLIT_UNALIGNED;
    KV_TRY(gather_prefix_kv((bf16 *)qkv_ctx_dev, pos0, n_q_heads, n_kv_heads, head_dim, make_view(cache), layer,
                            block_table_dev, (cudaStream_t)stream));
  }
  return attention_prefill_tc((const bf16 *)qkv_ctx_dev, n_tokens, pos0, n_q_heads, n_kv_heads, head_dim,
                              (bf16 *)out_dev, status_dev, (cudaStream_t)stream);
}

int64_t kv_paged_attention_scratch_bytes(int32_t n_q_heads, int32_t head_dim, int32_t n_ctx) {
  if (n_q_heads <= 0 || head_dim <= 0 || n_ctx <= 0) return KV_ERR_ARG;
  return paged_attention_scratch_bytes(n_q_heads, head_dim, n_ctx);
}

int32_t kv_op_paged_attention(const float *q_dev, int32_t n_q_heads, const kv_cache_desc *cache, int32_t layer,
                              const int32_t *block_table_dev, int32_t n_ctx, void *scratch_dev, int64_t scratch_bytes,
                              float *out_dev, void *stream) {
  if (q_dev == nullptr || block_table_dev == nullptr || scratch_dev == nullptr || out_dev == nullptr || n_ctx <= 0 ||
      n_q_heads <= 0)
    return KV_ERR_ARG;
  // the kernels read q as float2 and write fp32 partials and outputs
  if (((uintptr_t)q_dev & 7) || ((uintptr_t)out_dev & 3) || ((uintptr_t)scratch_dev & 15)) return KV_ERR_ARG;
  int rc = check_cache(cache);
  if (rc != KV_OK) return rc;
  if (layer < 0 || layer >= cache->n_layers || n_q_heads % cache->n_kv_heads != 0 ||
      (cache->head_dim != 64 && cache->head_dim != 128))
    return KV_ERR_SHAPE;
  if (scratch_bytes < paged_attention_scratch_bytes(n_q_heads, cache->head_dim, n_ctx)) return KV_ERR_WORKSPACE;
  return paged_attention(q_dev, n_q_heads, make_view(cache), layer, block_table_dev, n_ctx, scratch_dev, out_dev,
                         (cudaStream_t)stream);
}

int32_t kv_check_copy_status(void *stream) { return copy_wait_expired((cudaStream_t)stream); }

int32_t kv_selftest_bounded_wait(void *status_dev, int32_t limit_us, void *stream) {
  if (status_dev == nullptr || ((uintptr_t)status_dev & 15) || limit_us <= 0 || limit_us > 100000) return KV_ERR_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  KV_CUDA(cudaMemsetAsync(status_dev, 0, sizeof(DeviceStatus), st));
  bounded_wait_selftest_kernel<<<1, 64, 0, st>>>(reinterpret_cast<DeviceStatus *>(status_dev), (long long)limit_us * 2000ll);
  KV_COUNT_LAUNCH();
  KV_CUDA(cudaGetLastError());
  return KV_OK;
}

int32_t kv_profile_enable(int32_t on) {
  g_prof_on = on != 0;
  return KV_OK;
}

int64_t kv_launch_count(void) { return g_launches; }

int32_t kv_profile_read(float *ms_by_kind_host, int64_t *launches_by_kind_host, int32_t n_kinds) {
  if (ms_by_kind_host == nullptr || launches_by_kind_host == nullptr || n_kinds < PROF_KINDS) return KV_ERR_ARG;
  for (int i = 0; i < n_kinds; ++i) {
    ms_by_kind_host[i] = 0.f;
    launches_by_kind_host[i] = 0;
  }
  for (const ProfRecord &r : g_prof_records) {
    KV_CUDA(cudaEventSynchronize(r.stop));
    float ms = 0.f;
    KV_CUDA(cudaEventElapsedTime(&ms, r.start, r.stop));
    ms_by_kind_host[r.kind] += ms;
    launches_by_kind_host[r.kind] += r.launches;
    g_prof_pool.push_back(r.start);
    g_prof_pool.push_back(r.stop);
  }
  g_prof_records.clear();
  return KV_OK;
}

int32_t kv_fill_pattern(void *dst_dev, int64_t bytes, uint64_t seed, int64_t pattern_offset_bytes, void *stream) {
  if (dst_dev == nullptr || bytes < 0 || (bytes & 7) || (pattern_offset_bytes & 7) || ((uintptr_t)dst_dev & 7))
    return KV_ERR_ARG;
  return fill_pattern(dst_dev, bytes, seed, pattern_offset_bytes, (cudaStream_t)stream);
}

}  // extern "C"
