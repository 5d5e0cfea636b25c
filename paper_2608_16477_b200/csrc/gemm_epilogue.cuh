// Epilogues of the tensor-core GEMM, shared by the one-CTA and the CTA-pair kernels.  A thread owns one row
// of a 128-row accumulator slab in TMEM (lane = row) and walks its columns 32 at a time.
#pragma once
#include "tc_common.cuh"

namespace kvr {

constexpr int kEpiStageBytes = 4 * 32 * 8 * 4;  // per epilogue warp: a 32-row x 8-column fp32 transpose buffer (1 KiB)

__device__ __forceinline__ float silu_f(float a) { return a / (1.f + __expf(-a)); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&h);
}

__device__ __forceinline__ void store_chunk_bf16(bf16 *dst, const float (&v)[32]) {
  uint4 *d4 = reinterpret_cast<uint4 *>(dst);
#pragma unroll
  for (int q = 0; q < 4; ++q)
    d4[q] = make_uint4(pack_bf16(v[8 * q], v[8 * q + 1]), pack_bf16(v[8 * q + 2], v[8 * q + 3]),
                       pack_bf16(v[8 * q + 4], v[8 * q + 5]), pack_bf16(v[8 * q + 6], v[8 * q + 7]));
}

// t_row: TMEM address of this warp's lane quarter and accumulator buffer; row: global output row of this
// thread; m0/n0: first row / output column of the slab; stage_base: the four warps' transpose buffers
// (used by the residual epilogue only); warp: warp index in the CTA (epilogue warps are 2..5).
template <int MODE, int BN>
__device__ __forceinline__ void gemm_epilogue_slab(uint32_t t_row, int row, int m0, int n0, int m, int n, int quarter,
                                                   int lane, int warp, bf16 *__restrict__ out,
                                                   float *__restrict__ resid, const QkvRopeArgs &qa,
                                                   float4 *stage_base) {
  if (MODE == GEMM_QKV_ROPE) {
    // columns of this tile are whole heads (head_dim divides 256); a head's pair (j, j + d/2) lies in
    // chunks c and c + d/64.  The row is token `row` of the call, at absolute position pos0 + row.
    const int d = qa.head_dim, half = d >> 1, pair = d >> 6;
    const bool live = row < m;
    long long slot_off = 0;
    int block = 0;
    if (live) {
      const int pos = qa.row_pos != nullptr ? qa.row_pos[row] : qa.pos0 + row;
      block = qa.row_block != nullptr ? qa.row_block[row] : qa.block_table[pos / qa.cache.block_size];
      slot_off = (long long)(pos % qa.cache.block_size) * qa.cache.n_kv_heads * d;
    }
    const float2 *cs_row = qa.rope + (live ? row : 0);      // entry j of this row: cs_row[j * rope_rows]
    bf16 *orow = out + (long long)row * n;
#pragma unroll 1
    for (int c = 0; c < BN / 32; ++c) {
      const int col = n0 + c * 32;
      if (col >= n) break;                       // uniform across the warp
      const int head = col / d, j0 = col - head * d;
      if (head < qa.n_q_heads + qa.n_kv_heads) {
        if (j0 >= half) continue;                // second half of a pair: written with its partner
        uint32_t lo[32], hi[32];
        tc::tmem_ld32(t_row + c * 32, lo);
        tc::tmem_ld32(t_row + (c + pair) * 32, hi);
        tc::tmem_ld_wait();
        if (live) {
          float a[32], b[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float2 cs = cs_row[(long long)(j0 + i) * qa.rope_rows];
            const float x = __uint_as_float(lo[i]), y = __uint_as_float(hi[i]);
            a[i] = x * cs.x - y * cs.y;
            b[i] = y * cs.x + x * cs.y;
          }
          store_chunk_bf16(orow + col, a);
          store_chunk_bf16(orow + col + half, b);
          if (head >= qa.n_q_heads) {
            bf16 *kp = reinterpret_cast<bf16 *>(qa.cache.page(qa.layer, 0, block)) + slot_off +
                       (head - qa.n_q_heads) * d + j0;
            store_chunk_bf16(kp, a);
            store_chunk_bf16(kp + half, b);
          }
        }
      } else {
        uint32_t r[32];
        tc::tmem_ld32(t_row + c * 32, r);
        tc::tmem_ld_wait();
        if (live) {
          float v[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
          store_chunk_bf16(orow + col, v);
          bf16 *vp = reinterpret_cast<bf16 *>(qa.cache.page(qa.layer, 1, block)) + slot_off +
                     (head - qa.n_q_heads - qa.n_kv_heads) * d + j0;
          store_chunk_bf16(vp, v);
        }
      }
    }
  } else if (MODE == GEMM_SWIGLU) {
#pragma unroll 1
    for (int c = 0; c < (BN / 2) / 32; ++c) {
      uint32_t g[32], u[32];
      tc::tmem_ld32(t_row + c * 32, g);
      tc::tmem_ld32(t_row + BN / 2 + c * 32, u);
      tc::tmem_ld_wait();
      const int col = n0 + c * 32;
      if (row < m && col < n) {
        uint32_t packed[16];
#pragma unroll
        for (int j = 0; j < 16; ++j)
          packed[j] = pack_bf16(silu_f(__uint_as_float(g[2 * j])) * __uint_as_float(u[2 * j]),
                                silu_f(__uint_as_float(g[2 * j + 1])) * __uint_as_float(u[2 * j + 1]));
        uint4 *dst = reinterpret_cast<uint4 *>(out + (long long)row * n + col);
#pragma unroll
        for (int v = 0; v < 4; ++v)
          if (col + v * 8 < n) dst[v] = make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]);
      }
    }
  } else if (MODE == GEMM_RESID_F32) {
    // x[row, col..] += acc.  A thread owns a row of the accumulator, but rows are 4 * n bytes apart in
    // memory and a thread-per-row update would touch half a 32-byte sector per row and instruction.
    // Each warp therefore transposes 32 rows x 8 columns at a time through a 1 KiB shared-memory buffer
    // and updates x with two lanes per row: every instruction then moves whole 32-byte sectors of 16 rows.
    // The old values of x for a 32-column slab (eight float4 per thread) are fetched one slab ahead, so the
    // global-memory latency is paid once per tile instead of once per pass.
    float4 *stage = stage_base + (warp - 2) * 64;
    const int sub_row = lane >> 1, c4 = lane & 1;
    auto x_ptr = [&](int c, int s8, int it) {
      const int grow = m0 + quarter * 32 + it * 16 + sub_row;
      const int scol = n0 + c * 32 + s8 * 8 + c4 * 4;
      return (grow < m && scol < n) ? reinterpret_cast<float4 *>(resid + (long long)grow * n + scol) : nullptr;
    };
    auto fetch = [&](int c, float4 (&x)[8]) {
#pragma unroll
      for (int s8 = 0; s8 < 4; ++s8)
#pragma unroll
        for (int it = 0; it < 2; ++it) {
          const float4 *px = x_ptr(c, s8, it);
          x[s8 * 2 + it] = px != nullptr ? __ldcs(px) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    float4 x_cur[8], x_next[8];
    fetch(0, x_cur);
#pragma unroll 1
    for (int c = 0; c < BN / 32; ++c) {
      const int col = n0 + c * 32;
      if (col >= n) break;
      if (c + 1 < BN / 32) fetch(c + 1, x_next);
      uint32_t r[32];
      tc::tmem_ld32(t_row + c * 32, r);
      tc::tmem_ld_wait();
#pragma unroll
      for (int s8 = 0; s8 < 4; ++s8) {         // 8 columns per pass
        // stage[row][2 chunks], chunk index XORed with bit 2 of the row: conflict-free both ways
        stage[lane * 2 + (0 ^ ((lane >> 2) & 1))] =
            make_float4(__uint_as_float(r[8 * s8]), __uint_as_float(r[8 * s8 + 1]), __uint_as_float(r[8 * s8 + 2]),
                        __uint_as_float(r[8 * s8 + 3]));
        stage[lane * 2 + (1 ^ ((lane >> 2) & 1))] =
            make_float4(__uint_as_float(r[8 * s8 + 4]), __uint_as_float(r[8 * s8 + 5]),
                        __uint_as_float(r[8 * s8 + 6]), __uint_as_float(r[8 * s8 + 7]));
        __syncwarp();
#pragma unroll
        for (int it = 0; it < 2; ++it) {
          const int rr = it * 16 + sub_row;
          float4 *px = x_ptr(c, s8, it);
          if (px != nullptr) {
            const float4 a4 = stage[rr * 2 + (c4 ^ ((rr >> 2) & 1))];
            float4 x = x_cur[s8 * 2 + it];
            x.x += a4.x; x.y += a4.y; x.z += a4.z; x.w += a4.w;
            *px = x;
          }
        }
        __syncwarp();
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) x_cur[i] = x_next[i];
    }
  } else {
#pragma unroll 1
    for (int c = 0; c < BN / 32; ++c) {
      uint32_t r[32];
      tc::tmem_ld32(t_row + c * 32, r);
      tc::tmem_ld_wait();
      const int col = n0 + c * 32;
      if (row < m && col < n) {
        uint4 *dst = reinterpret_cast<uint4 *>(out + (long long)row * n + col);
#pragma unroll
        for (int v = 0; v < 4; ++v)
          if (col + v * 8 < n)
            dst[v] = make_uint4(pack_bf16(__uint_as_float(r[8 * v]), __uint_as_float(r[8 * v + 1])),
                                pack_bf16(__uint_as_float(r[8 * v + 2]), __uint_as_float(r[8 * v + 3])),
                                pack_bf16(__uint_as_float(r[8 * v + 4]), __uint_as_float(r[8 * v + 5])),
                                pack_bf16(__uint_as_float(r[8 * v + 6]), __uint_as_float(r[8 * v + 7])));
      }
    }
  }
}

}  // namespace kvr
