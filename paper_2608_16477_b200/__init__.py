"""B200-native target-side KV-cache reconstruction: thin Python binding of libkvrebuild.so.

Every step of the path runs in the library's CUDA kernels; this package only marshals arguments
(torch supplies device memory and streams).  There is no CPU fallback: `load()` raises if the
shared library is missing and cannot be built.
"""
from .binding import (KVError, load, lib_path, status_string, Model, PagedCache, kv_bytes_per_token,
                      kv_prefill_prefix, kv_prefill_prefix_batched, kv_pack_blocks, kv_unpack_assemble, kv_decode_step,
                      kv_pack_blocks_batched, kv_unpack_blocks_batched, kv_workspace_bytes, kv_workspace_residual,
                      kv_check_device_status, kv_check_copy_status, kv_selftest_bounded_wait, kv_window_evaluate, kv_window_select,
                      kv_window_waste_bound, kv_ewma, kv_op_gemm, kv_gemm_plan, kv_op_gemv, kv_op_rmsnorm,
                      kv_op_attention_prefill, kv_op_paged_attention, kv_op_paged_attention_noalloc, kv_paged_attention_scratch_bytes,
                      kv_fill_pattern, kv_profile_enable, kv_profile_read, kv_launch_count, PROFILE_KINDS, EXPORTS, KV_OP_PREFILL, KV_OP_DECODE, KV_WIRE_BLOCK_MAJOR,
                      KV_WIRE_LAYER_MAJOR, KV_GEMM_CTA_PAIR)

__all__ = [n for n in dir() if not n.startswith("_")]
