/* kvrebuild.h -- C ABI of the B200 (sm_100a) target-side KV-cache reconstruction library.
 *
 * The library implements the data-parallel hot path of proactive KV-cache migration:
 *   - the target reconstructs the KV cache of the stable prefix [0,k) by a local prefill from the
 *     exact prefix token ids and writes every layer's K/V into a paged block cache
 *     (Section 4.3, "Initialization and parallel preparation"; Section 5, "Parallel state preparation");
 *   - the source gathers the KV blocks of the evolving suffix from its paged cache into a
 *     contiguous wire buffer (Section 5: physical block ids -> per-layer KV tensors -> bytes);
 *   - the target scatters those blocks into freshly allocated pages, builds the merged block table
 *     and checks the state-consistency conditions (Section 4.3, "State consistency"; Section 5,
 *     "Final synchronization and activation");
 *   - decoding resumes at position n on the merged cache without repeating prefill over [0,n).
 *
 * Conventions
 *   - Every function returns an int32 status (KV_OK = 0, errors negative) unless stated otherwise.
 *     Nothing throws, aborts or prints.
 *   - Pointers named *_dev are DEVICE pointers, *_host are HOST pointers.  All device buffers
 *     (weights, caches, wire buffers, workspaces, logits) are owned by the caller; the library never
 *     allocates or frees device memory.  Host arrays (pageable or page-locked) may be reused as soon as a
 *     call returns: the library copies them into page-locked staging slots of its own (host memory, a few
 *     slots per device that grow to the largest array seen) and transfers from there.
 *   - Work is enqueued on the caller's stream (a cudaStream_t passed as void*); calls do not
 *     synchronise except where stated.  Argument errors are detected on the host before anything is
 *     enqueued, so on a negative status other than KV_ERR_CUDA / KV_ERR_DEVICE no device memory was
 *     touched.
 *   - bf16 everywhere for weights, activations fed to tensor cores and cache elements; fp32 for
 *     the residual stream, norm/softmax statistics, accumulators and logits.
 *
 * Model (shapes only; no QK-norm, no biases, untied LM head): pre-norm decoder with RMSNorm,
 * fused QKV projection (rows ordered Q | K | V, heads contiguous), rotate-half RoPE, causal
 * grouped-query attention (query head h reads KV head h / (Hq/Hkv)), output projection, RMSNorm,
 * SwiGLU FFN (rows of w_gate_up ordered gate | up), final RMSNorm and LM head.
 * All matrices are row-major [out, in]; y = x W^T.  head_dim must be 64 or 128, hidden and ffn multiples of 8.
 *
 * Paged cache: page(layer, kv, block) is block_size * n_kv_heads * head_dim contiguous bf16,
 * laid out [slot][kv_head][dim], at base + layer*layer_stride + kv*kv_stride + block*block_stride
 * (strides in bytes, multiples of 16).  Token position p lives in block block_table[p / block_size],
 * slot p % block_size (PagedAttention, block size 16 in the paper's prototype, Section 5).
 *
 * Wire buffer: headerless raw pages.  Layout KV_WIRE_BLOCK_MAJOR: [block i][layer][kv][page bytes], so
 * each completed block is one contiguous self-contained message ("newly completed suffix KV-cache
 * blocks are streamed ... with their logical token positions", Section 4.3).  KV_WIRE_LAYER_MAJOR:
 * [layer][kv][block i][page bytes].  Logical positions, request id and epoch travel as host metadata.
 */
#ifndef KVREBUILD_H_
#define KVREBUILD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---------------------------------------------------------------- status codes */
enum {
  KV_OK = 0,
  KV_ERR_ARG = -1,             /* null pointer, non-positive size, misaligned (<16 B) pointer or stride */
  KV_ERR_SHAPE = -2,           /* cache geometry does not match the model / unsupported shape */
  KV_ERR_BLOCK_RANGE = -3,     /* physical block id outside [0, num_blocks) */
  KV_ERR_BLOCK_ALIAS = -4,     /* duplicate physical id, or a suffix id equal to a prefix id */
  KV_ERR_GAP = -5,             /* some logical suffix block in [k/Bs, ceil(n/Bs)) is missing */
  KV_ERR_OVERLAP = -6,         /* a logical suffix block appears twice or lies outside [k/Bs, ceil(n/Bs)) */
  KV_ERR_SPLIT_UNALIGNED = -7, /* prefix length / start position is not a multiple of block_size */
  KV_ERR_TABLE_SHORT = -8,     /* block table does not cover the token positions */
  KV_ERR_WIRE_SIZE = -9,       /* wire buffer smaller than n_blocks * layers * 2 * page bytes */
  KV_ERR_WORKSPACE = -10,      /* workspace smaller than kv_workspace_bytes() or misaligned */
  KV_ERR_STALE_EPOCH = -11,    /* blocks of a cancelled preparation attempt (epoch != expected) */
  KV_ERR_TOKEN_RANGE = -12,    /* token id outside [0, vocab) */
  KV_ERR_CUDA = -13,           /* a CUDA runtime/driver call failed; see kv_last_cuda_error() */
  KV_ERR_DEVICE = -14          /* a kernel reported a bounded wait that ran out (read by kv_check_device_status) */
};

enum { KV_WIRE_BLOCK_MAJOR = 0, KV_WIRE_LAYER_MAJOR = 1 };
enum { KV_OP_PREFILL = 0, KV_OP_DECODE = 1 };

/* ---------------------------------------------------------------- descriptors */
typedef struct {
  int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab;
  float rope_base; /* 1e6 */
  float rms_eps;   /* 1e-6 */
} kv_model_desc;

/* Device pointers to bf16 weights, caller-owned, each 16-byte aligned.  The per-layer members are
 * HOST arrays of n_layers device pointers. */
typedef struct {
  const void *embed_dev;      /* [vocab, hidden] */
  const void *lm_head_dev;    /* [vocab, hidden] */
  const void *final_norm_dev; /* [hidden] */
  const void *const *attn_norm_dev; /* [hidden] */
  const void *const *w_qkv_dev;     /* [(Hq + 2 Hkv) * d, hidden] */
  const void *const *w_o_dev;       /* [hidden, Hq * d] */
  const void *const *ffn_norm_dev;  /* [hidden] */
  const void *const *w_gate_up_dev; /* [2 * ffn, hidden] */
  const void *const *w_down_dev;    /* [hidden, ffn] */
} kv_weights;

typedef struct {
  void *base_dev;
  int64_t layer_stride, kv_stride, block_stride; /* bytes */
  int32_t num_blocks, block_size, n_layers, n_kv_heads, head_dim, elem_bytes /* 2 */;
} kv_cache_desc;

typedef struct kv_model kv_model; /* opaque host handle */

/* ---------------------------------------------------------------- handle and queries */

/* Creates the host handle (copies the descriptor and the pointer arrays; touches no device memory). */
int32_t kv_model_create(const kv_model_desc *desc, const kv_weights *weights, kv_model **out);
int32_t kv_model_destroy(kv_model *m);

/* Bytes of caller-owned device workspace an operation needs for up to max_tokens tokens
 * (KV_OP_PREFILL: pos0 + n_tokens of the call; KV_OP_DECODE: context length pos + 1).  Negative status on error.
 * The workspace must be 1024-byte aligned. */
int64_t kv_workspace_bytes(const kv_model *m, int32_t op, int32_t max_tokens);

/* Where the residual stream (the hidden state x, fp32) sits inside a workspace of kv_workspace_bytes(m, op, max_tokens)
 * bytes: *offset_out bytes from its base, *bytes_out long (KV_OP_PREFILL: [max_tokens, hidden] rows of the call's
 * tokens; KV_OP_DECODE: [hidden]).  After a call it holds the output of the last layer that ran: for a K/V-only
 * prefill (logits_out_dev = NULL) that is the INPUT of the model's last layer, whose K/V depend on nothing else.  Lets a
 * caller read hidden states, and lets a test check any single layer of a deep model against the oracle on that
 * layer's true input. */
int32_t kv_workspace_residual(const kv_model *m, int32_t op, int32_t max_tokens, int64_t *offset_out,
                              int64_t *bytes_out);

const char *kv_status_string(int32_t status);
/* Text of the last CUDA error seen by this thread's calls ("" if none). */
const char *kv_last_cuda_error(void);

/* Eq. (1): s_KV = 2 * L * H_KV * d_h * b bytes per token. */
int64_t kv_bytes_per_token(int32_t n_layers, int32_t n_kv_heads, int32_t head_dim, int32_t elem_bytes);

/* Synchronises `stream` and reads the device status word kept in `workspace_dev` by the last
 * prefill/decode call on it: KV_OK, or KV_ERR_DEVICE if a kernel's bounded wait ran out. */
int32_t kv_check_device_status(const void *workspace_dev, void *stream);

/* Synchronises `stream` and reports whether any pack/unpack kernel on the current device gave up a bounded wait
 * since the last call of this function (KV_ERR_DEVICE; the copy it belonged to is then incomplete); the record is
 * cleared by the call.  KV_OK otherwise. */
int32_t kv_check_copy_status(void *stream);

/* Self-test of the kernels' bounded waits (no counterpart in the paper; failure detection of this library): launches
 * one small kernel whose threads wait, with the routine every tensor-core kernel uses, on a barrier that nothing
 * signals.  The wait gives up after about limit_us microseconds (1..100000), records itself in the status block at
 * status_dev (>= 32 bytes, 16-byte aligned; a prefill/decode workspace will do) and the kernel returns normally; a
 * following kv_check_device_status(status_dev, stream) must report KV_ERR_DEVICE.  The GPU context stays usable. */
int32_t kv_selftest_bounded_wait(void *status_dev, int32_t limit_us, void *stream);

/* ---------------------------------------------------------------- the four operations */

/* Target-side prefix reconstruction (Section 4.3 / Section 5: the target reconstructs the prefix KV
 * cache through local prefill from the exact prefix token ids).  Runs the decoder over
 * token_ids_host[0..n_tokens) at absolute positions pos0 .. pos0+n_tokens-1 and stores the post-RoPE
 * K and the V of every layer into `cache` through block_table_host (n_blocks entries covering
 * positions [0, pos0+n_tokens)).  pos0 must be a multiple of block_size; pos0 > 0 continues a prefill
 * whose first pos0 positions are already in the cache (chunked prefill, Section 4.5).
 * logits_out_dev: NULL => K/V only (the last layer stops once its K/V are stored); otherwise
 * fp32 [vocab] next-token logits of the last row. */
int32_t kv_prefill_prefix(kv_model *m, const kv_cache_desc *cache,
                          const int32_t *token_ids_host, int32_t n_tokens, int32_t pos0,
                          const int32_t *block_table_host, int32_t n_blocks,
                          void *workspace_dev, int64_t workspace_bytes,
                          float *logits_out_dev, void *stream);

/* Several prefix reconstructions in one call (concurrent migrations sharing the target GPU, Section 4.5:
 * handover-handover contention).  Request r owns tokens token_ids_host[token_offsets_host[r] ..
 * token_offsets_host[r+1]) and the block table block_tables_host[table_offsets_host[r] .. table_offsets_host[r+1]);
 * every request starts at position 0.  All rows go through the projections together (one GEMM per layer over
 * the sum of the prefix lengths), attention runs per request.  Physical blocks must be distinct across the whole
 * batch.  Results are identical to n_req separate kv_prefill_prefix calls.  workspace: kv_workspace_bytes(m,
 * KV_OP_PREFILL, total tokens).  logits_out_dev: NULL or fp32 [n_req, vocab]. */
int32_t kv_prefill_prefix_batched(kv_model *m, const kv_cache_desc *cache, int32_t n_req,
                                  const int32_t *token_offsets_host, const int32_t *token_ids_host,
                                  const int32_t *table_offsets_host, const int32_t *block_tables_host,
                                  void *workspace_dev, int64_t workspace_bytes, float *logits_out_dev, void *stream);

/* Source-side suffix block extraction (Section 5: physical block ids from the block manager ->
 * per-layer KV tensors -> bytes).  wire[i] <- all pages of block block_ids_host[i], i in logical
 * order.  Bytes are copied verbatim.  Duplicate ids are allowed. */
int32_t kv_pack_blocks(const kv_cache_desc *src, const int32_t *block_ids_host, int32_t n_blocks,
                       void *wire_dev, int64_t wire_bytes, int32_t wire_layout, void *stream);

/* Target-side assembly (Section 5: allocate a new physical block table and copy the buffered suffix
 * blocks into the corresponding GPU locations; Section 4.3: coverage of [0,n) without gaps or
 * conflicts, epoch check).  pages of suffix_dst_block_ids_host[i] <- wire[i];
 * merged_block_table_out_host[0..ceil(n/Bs)) = prefix table followed by the destination ids ordered
 * by logical block (suffix_logical_blocks_host[i] is the logical block index of wire block i).
 * The prefix covers whole blocks: k = n_prefix_blocks * block_size.  The last block may be partial
 * (n % Bs != 0); it travels as a full page.  On any error the destination cache is untouched. */
int32_t kv_unpack_assemble(const kv_cache_desc *dst, const void *wire_dev, int64_t wire_bytes,
                           int32_t wire_layout,
                           const int32_t *suffix_logical_blocks_host,
                           const int32_t *suffix_dst_block_ids_host, int32_t n_suffix_blocks,
                           const int32_t *prefix_block_table_host, int32_t n_prefix_blocks,
                           int32_t n_tokens_total, uint32_t epoch, uint32_t expected_epoch,
                           int32_t *merged_block_table_out_host, void *stream);

/* Resume decoding (Section 4.3: the target activates the request in the decoding stage, generating
 * the next token without repeating prefill).  Feeds token_id at absolute position pos, attends over
 * cached positions [0,pos) plus itself, appends its K/V at slot pos (block_table_host must cover
 * position pos) and writes fp32 [vocab] logits. */
int32_t kv_decode_step(kv_model *m, const kv_cache_desc *cache, int32_t token_id, int32_t pos,
                       const int32_t *block_table_host, int32_t n_blocks,
                       void *workspace_dev, int64_t workspace_bytes,
                       float *logits_out_dev, void *stream);

/* Batched forms over n_req requests (CSR offsets blk_offsets_host[0..n_req] into block_ids_host);
 * request r uses wire buffer wire_dev_ptrs_host[r].  Same semantics per request as above, without
 * the table assembly.  All requests share ONE kernel launch (up to 7,680 blocks and 64 requests per launch;
 * beyond that the list continues in further launches). */
int32_t kv_pack_blocks_batched(const kv_cache_desc *src, int32_t n_req, const int32_t *blk_offsets_host,
                               const int32_t *block_ids_host, void *const *wire_dev_ptrs_host,
                               int32_t wire_layout, void *stream);
int32_t kv_unpack_blocks_batched(const kv_cache_desc *dst, int32_t n_req, const int32_t *blk_offsets_host,
                                 const int32_t *dst_block_ids_host, const void *const *wire_dev_ptrs_host,
                                 int32_t wire_layout, void *stream);

/* ---------------------------------------------------------------- single-kernel entry points
 * The steps of the prefill/decode path, callable on their own (unit parity tests, profiling).  */

/* Dense projection on the tensor cores: A bf16 [M, K] (row stride lda elements), W bf16 [N_w, K].
 * mode 0: out_dev bf16 [M, N] = A W^T.
 * mode 1: resid_dev fp32 [M, N] += A W^T (residual stream update).
 * mode 2: W is [2N, K] (gate | up); out_dev bf16 [M, N] = silu(A Wg^T) * (A Wu^T)  (SwiGLU).
 * K, lda and N must be multiples of 8, lda >= K; out_dev and resid_dev 16-byte aligned.  M is arbitrary.
 * mode | KV_GEMM_CTA_PAIR selects the kernel in which two CTAs
 * (two SMs) share one 256 x 256 tile through tcgen05 cta_group::2; results are identical. */
#define KV_GEMM_CTA_PAIR 0x100
int32_t kv_op_gemm(const void *a_dev, int32_t lda, const void *w_dev, int32_t m, int32_t n, int32_t k,
                   int32_t mode, void *out_dev, float *resid_dev, int32_t *status_dev, void *stream);

/* Matrix-vector product of the decode step: W bf16 [rows, k] row-major, x fp32 [k], y fp32.
 * mode 0: y[n] = W[n] . x (n rows).  mode 1: y[n] += W[n] . x.  mode 2: W is [2n, k] (gate | up),
 * y[n] = silu(W[n] . x) * (W[n + n_rows] . x).  gain_dev != NULL (bf16 [k], modes 0 and 2) fuses the preceding
 * RMSNorm: x is replaced by x * gain * rsqrt(mean(x^2) + eps).  k must be a multiple of 8. */
int32_t kv_op_gemv(const void *w_dev, const float *x_dev, int32_t n, int32_t k, int32_t mode, const void *gain_dev,
                   float eps, float *y_dev, void *stream);

/* Which kernel and tile the projection launcher uses for an m-row problem with n output columns: *cta_pair_out = 1
 * when two CTAs share a 256-row tile (tcgen05 cta_group::2), 0 for the one-CTA kernel; *tile_width_out = columns of W
 * per tile (128..256; a SwiGLU tile holds tile_width/2 gate and tile_width/2 up rows).  mode 0..2 as in kv_op_gemm,
 * 3 = the fused QKV projection (head_dim required: tiles hold whole heads).  Read-only; depends on the current
 * device's SM count.  Lets a test or a report state which instantiation a given problem size runs. */
int32_t kv_gemm_plan(int32_t m, int32_t n, int32_t mode, int32_t head_dim, int32_t *cta_pair_out,
                     int32_t *tile_width_out);

/* RMSNorm of fp32 rows x [rows, dim] with bf16 gain -> bf16 out [rows, dim].  dim a multiple of 4; x_dev 16-byte,
 * gain_dev and out_dev 8-byte aligned. */
int32_t kv_op_rmsnorm(const float *x_dev, const void *gain_dev, int32_t rows, int32_t dim, float eps,
                      void *out_dev, void *stream);

/* Causal GQA flash attention of a prefill chunk (step 4 of a decoder layer inside kv_prefill_prefix; Section 4.5 for
 * pos0 > 0).  qkv_ctx_dev bf16 [pos0 + T, (Hq+2Hkv) d], one row per context position: rows [pos0, pos0+T) hold the
 * chunk's post-RoPE Q and K and its V.  With pos0 > 0 (a multiple of block_size) the call first copies the K and V of
 * positions [0,pos0) from the paged cache (through block_table_dev) into the K and V columns of rows [0,pos0); the Q
 * columns of those rows are not touched or read.  out_dev bf16 [T, Hq d].  head_dim 64 or 128. */
int32_t kv_op_attention_prefill(void *qkv_ctx_dev, int32_t n_tokens, int32_t pos0,
                                int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                const kv_cache_desc *cache, int32_t layer, const int32_t *block_table_dev,
                                void *out_dev, int32_t *status_dev, void *stream);

/* Paged decode attention of one query token: q_dev fp32 [Hq, d] (post-RoPE), keys/values of
 * positions [0, n_ctx) read from layer `layer` of the cache through block_table_dev;
 * out_dev fp32 [Hq, d].  scratch_dev: kv_paged_attention_scratch_bytes() bytes of device memory. */
int64_t kv_paged_attention_scratch_bytes(int32_t n_q_heads, int32_t head_dim, int32_t n_ctx);
int32_t kv_op_paged_attention(const float *q_dev, int32_t n_q_heads, const kv_cache_desc *cache,
                              int32_t layer, const int32_t *block_table_dev, int32_t n_ctx,
                              void *scratch_dev, int64_t scratch_bytes, float *out_dev, void *stream);

/* Paged decode attention without any caller-supplied scratch (the paper has no counterpart: this exists
 * for hosts of the library that cannot allocate device memory when they need a decode step, e.g. an engine
 * whose start-up pools already own all of HBM, code running inside a foreign memory pool, or the activation
 * path after a handover where a cudaMalloc would stall the device or fail).  Same inputs, outputs and
 * arithmetic as kv_op_paged_attention; the split-KV partials go to a fixed KV_NOALLOC_SCRATCH_BYTES array
 * inside the library, which every GPU that loads the library keeps until exit.
 *  - Limit: kv_paged_attention_scratch_bytes(n_q_heads, head_dim, n_ctx) must not exceed
 *    KV_NOALLOC_SCRATCH_BYTES, otherwise KV_ERR_WORKSPACE is returned and nothing is launched
 *    (64 query heads of dimension 128 fit up to 16,128 context tokens).
 *  - The call never allocates or frees memory.  Its first call on a device looks up the array's device
 *    address (once per device).
 *  - All calls on a device share the one array and it keeps whatever the last call left there.  A call
 *    writes every partial it later reads, so stale contents are harmless, but two calls whose kernels can
 *    overlap on the GPU (different streams) race on it: serialise them. */
#define KV_NOALLOC_SCRATCH_BYTES (4 * 1024 * 1024)
int32_t kv_op_paged_attention_noalloc(const float *q_dev, int32_t n_q_heads, const kv_cache_desc *cache,
                                      int32_t layer, const int32_t *block_table_dev, int32_t n_ctx,
                                      float *out_dev, void *stream);

/* ---------------------------------------------------------------- window selection (host scalar code)
 * The Scheduler Engine's cost model and online selection (Section 4.1, Eqs. 3-9; Section 4.2, Algorithm 1;
 * Section 4.4, Eq. 10).  Units: seconds, tokens, tokens/s, bytes, bytes/s.  No device work, no allocation. */
typedef struct {
  double k_curr;    /* K_curr: current context length (tokens) */
  double r_p;       /* effective prefill throughput at the target (tokens/s), > 0 */
  double r_d;       /* per-request decode throughput at the source (tokens/s) */
  double goodput;   /* B: effective inter-node goodput (bytes/s), > 0 */
  double s_kv;      /* Eq. (1): KV bytes per token */
  double t0;        /* T_0: assembly + activation + first decode step (s) */
  double t_load;    /* T_load: model load latency (0 when resident) */
  double alpha;     /* weight of T_SIT in Eq. (8), in [0, 1] */
  double t_remain;  /* predicted remaining time to handover (s) */
} kv_window_inputs;

typedef struct {
  double t_w, l_hist, t_hist, t_res, t_sit, t_early, cost;
} kv_window_eval;

/* Eqs. (3)-(9) for one candidate window T_w. */
int32_t kv_window_evaluate(const kv_window_inputs *in, double t_w, kv_window_eval *out);
/* Algorithm 1 after admission: candidates {0, dT, ..., T_limit}, T_limit = min(T_max, T_remain); *best receives the
 * arg-min (ties: the smallest window), *trigger is 1 iff T_remain <= T_w*. */
int32_t kv_window_select(const kv_window_inputs *in, double t_max, double d_t, kv_window_eval *best, int32_t *trigger);
/* Eq. (10): bound on discarded preparation, max{T_max + E_early - T_avail, 0}. */
double kv_window_waste_bound(double t_max, double e_early, double t_avail);
/* Telemetry smoothing (Section 4.2): beta * sample + (1 - beta) * old. */
double kv_ewma(double old_value, double sample, double beta);

/* Event profiler (off by default).  While enabled, every kernel class launched by the operations above is
 * bracketed by CUDA events on the caller's stream.  kv_profile_read waits for the recorded events, adds the
 * elapsed milliseconds and kernel-launch counts per class into the two host arrays (n_kinds >= 14) and clears
 * the record list.  Classes, in order: embed, rmsnorm, gemm_qkv, rope_store, attention, gemm_o, gemm_gate_up,
 * gemm_down, lm_head, pack, unpack, decode_gemv, decode_attention, decode_other.  Not thread-safe.
 * kv_launch_count returns the number of kernels this library has launched since it was loaded. */
int32_t kv_profile_enable(int32_t on);
int32_t kv_profile_read(float *ms_by_kind_host, int64_t *launches_by_kind_host, int32_t n_kinds);
int64_t kv_launch_count(void);

/* Fills `bytes` bytes (multiple of 8) at dst_dev with the counter-based test pattern: 64-bit word w
 * (byte offset 8w from pattern_offset_bytes) = splitmix64-style mix of (seed + w).  Used to give large
 * caches reproducible content without holding a host copy. */
int32_t kv_fill_pattern(void *dst_dev, int64_t bytes, uint64_t seed, int64_t pattern_offset_bytes,
                        void *stream);

#ifdef __cplusplus
}
#endif
#endif /* KVREBUILD_H_ */
