"""ctypes binding of the C ABI declared in include/kvrebuild.h (argument marshalling only)."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB = None

KV_OP_PREFILL, KV_OP_DECODE = 0, 1
KV_WIRE_BLOCK_MAJOR, KV_WIRE_LAYER_MAJOR = 0, 1

# every symbol include/kvrebuild.h declares
EXPORTS = [
    "kv_model_create", "kv_model_destroy", "kv_workspace_bytes", "kv_status_string", "kv_last_cuda_error",
    "kv_bytes_per_token", "kv_check_device_status", "kv_prefill_prefix", "kv_pack_blocks",
    "kv_unpack_assemble", "kv_decode_step", "kv_pack_blocks_batched", "kv_unpack_blocks_batched",
    "kv_op_gemm", "kv_gemm_plan", "kv_op_rmsnorm",
    "kv_op_attention_prefill", "kv_paged_attention_scratch_bytes", "kv_op_paged_attention", "kv_fill_pattern",
    "kv_profile_enable", "kv_profile_read", "kv_launch_count", "kv_op_paged_attention_noalloc", "kv_check_copy_status", "kv_op_gemv",
    "kv_window_evaluate", "kv_window_select", "kv_window_waste_bound", "kv_ewma", "kv_prefill_prefix_batched",
    "kv_selftest_bounded_wait", "kv_workspace_residual",
]

PROFILE_KINDS = ("embed", "rmsnorm", "gemm_qkv", "rope_store", "attention", "gemm_o", "gemm_gate_up", "gemm_down",
                 "lm_head", "pack", "unpack", "decode_gemv", "decode_attention", "decode_other")


class KVError(RuntimeError):
    def __init__(self, status: int, what: str = ""):
        self.status = status
        detail = ""
        if _LIB is not None:
            detail = _LIB.kv_status_string(status).decode()
            if status in (-13, -14):
                detail += " [" + _LIB.kv_last_cuda_error().decode() + "]"
        super().__init__(f"{what}: status {status} ({detail})")


class ModelDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "hidden", "n_q_heads", "n_kv_heads", "head_dim", "ffn", "vocab")] \
        + [("rope_base", C.c_float), ("rms_eps", C.c_float)]


class Weights(C.Structure):
    _fields_ = [("embed_dev", C.c_void_p), ("lm_head_dev", C.c_void_p), ("final_norm_dev", C.c_void_p)] + \
        [(n, C.POINTER(C.c_void_p)) for n in ("attn_norm_dev", "w_qkv_dev", "w_o_dev", "ffn_norm_dev",
                                              "w_gate_up_dev", "w_down_dev")]


class WindowInputs(C.Structure):
    _fields_ = [(n, C.c_double) for n in ("k_curr", "r_p", "r_d", "goodput", "s_kv", "t0", "t_load", "alpha", "t_remain")]


class WindowEval(C.Structure):
    _fields_ = [(n, C.c_double) for n in ("t_w", "l_hist", "t_hist", "t_res", "t_sit", "t_early", "cost")]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class CacheDesc(C.Structure):
    _fields_ = [("base_dev", C.c_void_p), ("layer_stride", C.c_int64), ("kv_stride", C.c_int64),
                ("block_stride", C.c_int64)] + \
        [(n, C.c_int32) for n in ("num_blocks", "block_size", "n_layers", "n_kv_heads", "head_dim", "elem_bytes")]


def lib_path() -> str:
    return os.path.join(_PKG, "libkvrebuild.so")


def load(build_if_missing: bool = True):
    """Loads libkvrebuild.so.  Raises if it is missing and cannot be built: there is no fallback path."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = lib_path()
    if not os.path.exists(path):
        if not build_if_missing:
            raise RuntimeError(f"{path} is missing: run __graft_entry__.build() (no CPU fallback exists)")
        from . import build as _build
        _build.build()
    lib = C.CDLL(path)
    i32, i64, vp = C.c_int32, C.c_int64, C.c_void_p
    pi32 = C.POINTER(C.c_int32)
    sig = {
        "kv_model_create": (i32, [C.POINTER(ModelDesc), C.POINTER(Weights), C.POINTER(vp)]),
        "kv_model_destroy": (i32, [vp]),
        "kv_workspace_bytes": (i64, [vp, i32, i32]),
        "kv_workspace_residual": (i32, [vp, i32, i32, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]),
        "kv_status_string": (C.c_char_p, [i32]),
        "kv_last_cuda_error": (C.c_char_p, []),
        "kv_bytes_per_token": (i64, [i32, i32, i32, i32]),
        "kv_check_device_status": (i32, [vp, vp]),
        "kv_prefill_prefix": (i32, [vp, C.POINTER(CacheDesc), pi32, i32, i32, pi32, i32, vp, i64, vp, vp]),
        "kv_prefill_prefix_batched": (i32, [vp, C.POINTER(CacheDesc), i32, pi32, pi32, pi32, pi32, vp, i64, vp, vp]),
        "kv_pack_blocks": (i32, [C.POINTER(CacheDesc), pi32, i32, vp, i64, i32, vp]),
        "kv_unpack_assemble": (i32, [C.POINTER(CacheDesc), vp, i64, i32, pi32, pi32, i32, pi32, i32, i32,
                                     C.c_uint32, C.c_uint32, pi32, vp]),
        "kv_decode_step": (i32, [vp, C.POINTER(CacheDesc), i32, i32, pi32, i32, vp, i64, vp, vp]),
        "kv_pack_blocks_batched": (i32, [C.POINTER(CacheDesc), i32, pi32, pi32, C.POINTER(vp), i32, vp]),
        "kv_unpack_blocks_batched": (i32, [C.POINTER(CacheDesc), i32, pi32, pi32, C.POINTER(vp), i32, vp]),
        "kv_op_gemm": (i32, [vp, i32, vp, i32, i32, i32, i32, vp, vp, vp, vp]),
        "kv_gemm_plan": (i32, [i32, i32, i32, i32, pi32, pi32]),
        "kv_op_rmsnorm": (i32, [vp, vp, i32, i32, C.c_float, vp, vp]),
        "kv_op_attention_prefill": (i32, [vp, i32, i32, i32, i32, i32, C.POINTER(CacheDesc), i32, vp, vp, vp, vp]),
        "kv_paged_attention_scratch_bytes": (i64, [i32, i32, i32]),
        "kv_op_paged_attention": (i32, [vp, i32, C.POINTER(CacheDesc), i32, vp, i32, vp, i64, vp, vp]),
        "kv_fill_pattern": (i32, [vp, i64, C.c_uint64, i64, vp]),
        "kv_op_paged_attention_noalloc": (i32, [vp, i32, C.POINTER(CacheDesc), i32, vp, i32, vp, vp]),
        "kv_check_copy_status": (i32, [vp]),
        "kv_selftest_bounded_wait": (i32, [vp, i32, vp]),
        "kv_window_evaluate": (i32, [C.POINTER(WindowInputs), C.c_double, C.POINTER(WindowEval)]),
        "kv_window_select": (i32, [C.POINTER(WindowInputs), C.c_double, C.c_double, C.POINTER(WindowEval),
                                   C.POINTER(C.c_int32)]),
        "kv_window_waste_bound": (C.c_double, [C.c_double, C.c_double, C.c_double]),
        "kv_ewma": (C.c_double, [C.c_double, C.c_double, C.c_double]),
        "kv_op_gemv": (i32, [vp, vp, i32, i32, i32, vp, C.c_float, vp, vp]),
        "kv_profile_enable": (i32, [i32]),
        "kv_profile_read": (i32, [C.POINTER(C.c_float), C.POINTER(C.c_int64), i32]),
        "kv_launch_count": (i64, []),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _LIB = lib
    return lib


def status_string(status: int) -> str:
    return load().kv_status_string(status).decode()


def _check(status: int, what: str) -> None:
    if status != 0:
        raise KVError(status, what)


def _i32(a):
    arr = np.ascontiguousarray(a, dtype=np.int32)
    return arr, arr.ctypes.data_as(C.POINTER(C.c_int32))


def _stream(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return getattr(stream, "cuda_stream", stream)


def _ptr(t) -> int:
    return 0 if t is None else (t.data_ptr() if hasattr(t, "data_ptr") else int(t))


class PagedCache:
    """A paged KV cache in device memory (torch tensor of bf16 bit patterns) plus its descriptor.

    layout "layer_major": [L][2][num_blocks][page]; "block_major": [num_blocks][L][2][page].
    """

    def __init__(self, shape, num_blocks: int, layout: str = "layer_major", device="cuda", fill=None):
        import torch
        self.n_layers, self.n_kv_heads, self.head_dim = shape.n_layers, shape.n_kv_heads, shape.head_dim
        self.block_size, self.num_blocks, self.layout = shape.block_size, num_blocks, layout
        page_elems = self.block_size * self.n_kv_heads * self.head_dim
        self.page_bytes = page_elems * 2
        if layout == "layer_major":
            dims = (self.n_layers, 2, num_blocks, page_elems)
            strides = (2 * num_blocks * self.page_bytes, num_blocks * self.page_bytes, self.page_bytes)
        elif layout == "block_major":
            dims = (num_blocks, self.n_layers, 2, page_elems)
            strides = (2 * self.page_bytes, self.page_bytes, 2 * self.n_layers * self.page_bytes)
        else:
            raise ValueError(layout)
        self.data = torch.empty(dims, dtype=torch.int16, device=device)
        if fill is not None:
            self.data.fill_(fill)
        self.desc = CacheDesc(self.data.data_ptr(), strides[0], strides[1], strides[2], num_blocks, self.block_size,
                              self.n_layers, self.n_kv_heads, self.head_dim, 2)

    def pages(self, block_ids):
        """int16 tensor [len(ids), L, 2, page_elems] of the given blocks (torch indexing; test helper)."""
        import torch
        idx = torch.as_tensor(np.asarray(block_ids, dtype=np.int64), device=self.data.device)
        if self.layout == "layer_major":
            return self.data[:, :, idx].permute(2, 0, 1, 3)
        return self.data[idx]

    def as_logical_numpy(self) -> np.ndarray:
        """uint16 array [L, 2, num_blocks, Bs, Hkv, d] on the host."""
        d = self.data if self.layout == "layer_major" else self.data.permute(1, 2, 0, 3)
        return d.contiguous().cpu().numpy().view(np.uint16).reshape(
            self.n_layers, 2, self.num_blocks, self.block_size, self.n_kv_heads, self.head_dim)


class Model:
    """Uploads bf16 weights to the device and creates the library handle."""

    def __init__(self, shape, head: dict | None = None, layers=None, device="cuda"):
        import torch
        self.shape = shape
        self._lib = load()
        self._keep = []
        self.device = device

        def up(arr):
            if isinstance(arr, torch.Tensor):
                t = arr.to(device=device, dtype=torch.bfloat16).contiguous()
            else:
                t = torch.from_numpy(np.ascontiguousarray(arr, dtype=np.float32)).to(device).to(torch.bfloat16)
            self._keep.append(t)
            return t.data_ptr()

        names = ("attn_norm", "w_qkv", "w_o", "ffn_norm", "w_gate_up", "w_down")
        arrays = {n: (C.c_void_p * shape.n_layers)() for n in names}
        for l in range(shape.n_layers):
            w = layers(l)
            for n in names:
                arrays[n][l] = up(w[n])
        self._arrays = arrays
        self._w = Weights(up(head["embed"]), up(head["lm_head"]), up(head["final_norm"]),
                          *[C.cast(arrays[n], C.POINTER(C.c_void_p)) for n in names])
        self._desc = ModelDesc(shape.n_layers, shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                               shape.ffn, shape.vocab, shape.rope_base, shape.rms_eps)
        handle = C.c_void_p()
        _check(self._lib.kv_model_create(C.byref(self._desc), C.byref(self._w), C.byref(handle)), "kv_model_create")
        self.handle = handle
        self._ws = {}

    def workspace(self, op: int, max_tokens: int):
        """A cached, caller-side (torch) workspace tensor large enough for `op` over max_tokens."""
        import torch
        need = kv_workspace_bytes(self, op, max_tokens)
        cur = self._ws.get(op)
        if cur is None or cur.numel() - ((-cur.data_ptr()) % 1024) < need:
            cur = torch.empty(need + 1024, dtype=torch.uint8, device=self.device)
            self._ws[op] = cur
        off = (-cur.data_ptr()) % 1024            # the library wants a 1 KiB-aligned base
        return cur[off:off + need]

    def __del__(self):
        try:
            if getattr(self, "handle", None):
                self._lib.kv_model_destroy(self.handle)
                self.handle = None
        except Exception:
            pass


def kv_bytes_per_token(n_layers, n_kv_heads, head_dim, elem_bytes=2) -> int:
    return load().kv_bytes_per_token(n_layers, n_kv_heads, head_dim, elem_bytes)


def kv_workspace_bytes(model: Model, op: int, max_tokens: int) -> int:
    r = load().kv_workspace_bytes(model.handle, op, max_tokens)
    if r < 0:
        raise KVError(int(r), "kv_workspace_bytes")
    return int(r)


def kv_workspace_residual(model: Model, op: int, max_tokens: int):
    """(offset, bytes) of the fp32 residual stream inside a workspace sized for (op, max_tokens)."""
    off, nbytes = C.c_int64(), C.c_int64()
    _check(load().kv_workspace_residual(model.handle, op, max_tokens, C.byref(off), C.byref(nbytes)), "kv_workspace_residual")
    return int(off.value), int(nbytes.value)


def kv_check_device_status(workspace, stream=None) -> None:
    _check(load().kv_check_device_status(_ptr(workspace), _stream(stream)), "kv_check_device_status")


def kv_prefill_prefix(model: Model, cache: PagedCache, token_ids, block_table, pos0: int = 0, logits_out=None,
                      workspace=None, stream=None):
    ids, pids = _i32(token_ids)
    tab, ptab = _i32(block_table)
    ws = workspace if workspace is not None else model.workspace(KV_OP_PREFILL, pos0 + len(ids))
    _check(load().kv_prefill_prefix(model.handle, C.byref(cache.desc), pids, len(ids), pos0, ptab, len(tab),
                                    _ptr(ws), ws.numel(), _ptr(logits_out), _stream(stream)), "kv_prefill_prefix")
    return ws


def kv_decode_step(model: Model, cache: PagedCache, token_id: int, pos: int, block_table, logits_out,
                   workspace=None, stream=None):
    tab, ptab = _i32(block_table)
    ws = workspace if workspace is not None else model.workspace(KV_OP_DECODE, pos + 1)
    _check(load().kv_decode_step(model.handle, C.byref(cache.desc), int(token_id), int(pos), ptab, len(tab),
                                 _ptr(ws), ws.numel(), _ptr(logits_out), _stream(stream)), "kv_decode_step")
    return ws


def kv_pack_blocks(cache: PagedCache, block_ids, wire, wire_layout: int = KV_WIRE_BLOCK_MAJOR, stream=None,
                   wire_bytes=None):
    ids, pids = _i32(block_ids)
    nbytes = wire.numel() * wire.element_size() if wire_bytes is None else wire_bytes
    _check(load().kv_pack_blocks(C.byref(cache.desc), pids, len(ids), _ptr(wire), nbytes, wire_layout,
                                 _stream(stream)), "kv_pack_blocks")


def kv_unpack_assemble(cache: PagedCache, wire, logical_blocks, dst_block_ids, prefix_block_table,
                       n_tokens_total: int, epoch: int = 0, expected_epoch: int = 0,
                       wire_layout: int = KV_WIRE_BLOCK_MAJOR, stream=None, wire_bytes=None) -> np.ndarray:
    lg, plg = _i32(logical_blocks)
    ds, pds = _i32(dst_block_ids)
    pf, ppf = _i32(prefix_block_table)
    bs = cache.block_size
    merged = np.full(max(-(-n_tokens_total // bs), len(pf) + len(ds), 1), -1, dtype=np.int32)
    nbytes = (wire.numel() * wire.element_size() if wire is not None else 0) if wire_bytes is None else wire_bytes
    _check(load().kv_unpack_assemble(C.byref(cache.desc), _ptr(wire), nbytes, wire_layout, plg, pds, len(ds), ppf,
                                     len(pf), n_tokens_total, epoch, expected_epoch,
                                     merged.ctypes.data_as(C.POINTER(C.c_int32)), _stream(stream)),
           "kv_unpack_assemble")
    return merged[: -(-n_tokens_total // bs)]


def _batched(fn_name, cache, blk_offsets, block_ids, wires, wire_layout, stream):
    offs, poffs = _i32(blk_offsets)
    ids, pids = _i32(block_ids)
    ptrs = (C.c_void_p * len(wires))(*[_ptr(w) for w in wires])
    _check(getattr(load(), fn_name)(C.byref(cache.desc), len(wires), poffs, pids, ptrs, wire_layout,
                                    _stream(stream)), fn_name)


def kv_pack_blocks_batched(cache, blk_offsets, block_ids, wires, wire_layout=KV_WIRE_BLOCK_MAJOR, stream=None):
    _batched("kv_pack_blocks_batched", cache, blk_offsets, block_ids, wires, wire_layout, stream)


def kv_unpack_blocks_batched(cache, blk_offsets, dst_block_ids, wires, wire_layout=KV_WIRE_BLOCK_MAJOR, stream=None):
    _batched("kv_unpack_blocks_batched", cache, blk_offsets, dst_block_ids, wires, wire_layout, stream)


KV_GEMM_CTA_PAIR = 0x100


def kv_op_gemm(a, w, mode: int, out=None, resid=None, status=None, stream=None, n=None):
    """mode 0 store / 1 residual add / 2 SwiGLU, optionally | KV_GEMM_CTA_PAIR for the two-SM kernel."""
    m, k = a.shape
    base_mode = mode & ~KV_GEMM_CTA_PAIR
    n = n if n is not None else (w.shape[0] // 2 if base_mode == 2 else w.shape[0])
    want = (m, n)
    for t in (out, resid):
        if t is not None and hasattr(t, "shape") and tuple(t.shape) != want:
            raise ValueError(f"output shape {tuple(t.shape)} does not match the product's {want}")
    _check(load().kv_op_gemm(_ptr(a), a.stride(0), _ptr(w), m, n, k, mode, _ptr(out), _ptr(resid), _ptr(status),
                             _stream(stream)), "kv_op_gemm")


def kv_gemm_plan(m: int, n: int, mode: int, head_dim: int = 0):
    """(cta_pair, tile_width) the projection launcher picks for an m x n problem (mode 3 = fused QKV)."""
    pair, bn = C.c_int32(), C.c_int32()
    _check(load().kv_gemm_plan(m, n, mode, head_dim, C.byref(pair), C.byref(bn)), "kv_gemm_plan")
    return bool(pair.value), int(bn.value)


def kv_op_rmsnorm(x, gain, eps: float, out, stream=None):
    _check(load().kv_op_rmsnorm(_ptr(x), _ptr(gain), x.shape[0], x.shape[1], eps, _ptr(out), _stream(stream)),
           "kv_op_rmsnorm")


def kv_op_attention_prefill(qkv_ctx, n_q_heads, n_kv_heads, head_dim, out, pos0=0, cache=None, layer=0,
                            block_table_dev=None, status=None, stream=None):
    """qkv_ctx has pos0 + T rows (the chunk's rows last); with pos0 > 0 the call fills the K/V columns of the first
    pos0 rows from the cache."""
    _check(load().kv_op_attention_prefill(_ptr(qkv_ctx), qkv_ctx.shape[0] - pos0, pos0, n_q_heads, n_kv_heads, head_dim,
                                          C.byref(cache.desc) if cache is not None else None, layer,
                                          _ptr(block_table_dev), _ptr(out), _ptr(status), _stream(stream)),
           "kv_op_attention_prefill")


def kv_paged_attention_scratch_bytes(n_q_heads, head_dim, n_ctx) -> int:
    return int(load().kv_paged_attention_scratch_bytes(n_q_heads, head_dim, n_ctx))


def kv_op_paged_attention(q, cache: PagedCache, layer, block_table_dev, n_ctx, scratch, out, stream=None):
    _check(load().kv_op_paged_attention(_ptr(q), q.shape[0], C.byref(cache.desc), layer, _ptr(block_table_dev), n_ctx,
                                        _ptr(scratch), scratch.numel() * scratch.element_size(), _ptr(out),
                                        _stream(stream)), "kv_op_paged_attention")


def kv_fill_pattern(dst, nbytes: int, seed: int, pattern_offset: int = 0, stream=None):
    _check(load().kv_fill_pattern(_ptr(dst), nbytes, seed, pattern_offset, _stream(stream)), "kv_fill_pattern")


def kv_profile_enable(on: bool) -> None:
    _check(load().kv_profile_enable(int(on)), "kv_profile_enable")


def kv_profile_read() -> dict:
    """{kind: (milliseconds, kernel launches)} accumulated since the last read."""
    n = len(PROFILE_KINDS)
    ms = (C.c_float * n)()
    cnt = (C.c_int64 * n)()
    _check(load().kv_profile_read(ms, cnt, n), "kv_profile_read")
    return {k: (float(ms[i]), int(cnt[i])) for i, k in enumerate(PROFILE_KINDS)}


def kv_launch_count() -> int:
    return int(load().kv_launch_count())


def kv_op_paged_attention_noalloc(q, cache: PagedCache, layer, block_table_dev, n_ctx, out, stream=None):
    """kv_op_paged_attention for callers that cannot provide scratch memory: the partial results live in a
    fixed array inside the library (limit KV_NOALLOC_SCRATCH_BYTES; larger contexts raise KVError)."""
    _check(load().kv_op_paged_attention_noalloc(_ptr(q), q.shape[0], C.byref(cache.desc), layer,
                                                _ptr(block_table_dev), n_ctx, _ptr(out), _stream(stream)),
           "kv_op_paged_attention_noalloc")


def kv_selftest_bounded_wait(status_buf, limit_us: int = 200, stream=None) -> None:
    """Launches the bounded-wait self-test into `status_buf`; kv_check_device_status(status_buf) then raises KVError(-14)."""
    _check(load().kv_selftest_bounded_wait(_ptr(status_buf), limit_us, _stream(stream)), "kv_selftest_bounded_wait")


def kv_check_copy_status(stream=None) -> None:
    _check(load().kv_check_copy_status(_stream(stream)), "kv_check_copy_status")


def kv_op_gemv(w, x, mode: int, y, gain=None, eps: float = 0.0, stream=None, n=None):
    rows, k = w.shape
    n = n if n is not None else (rows // 2 if mode == 2 else rows)
    _check(load().kv_op_gemv(_ptr(w), _ptr(x), n, k, mode, _ptr(gain), eps, _ptr(y), _stream(stream)), "kv_op_gemv")


def kv_window_evaluate(t_w: float, **inputs) -> dict:
    win, out = WindowInputs(**inputs), WindowEval()
    _check(load().kv_window_evaluate(C.byref(win), t_w, C.byref(out)), "kv_window_evaluate")
    return out.as_dict()


def kv_window_select(t_max: float, d_t: float, **inputs):
    """Returns (evaluation at T_w*, trigger)."""
    win, out, trig = WindowInputs(**inputs), WindowEval(), C.c_int32()
    _check(load().kv_window_select(C.byref(win), t_max, d_t, C.byref(out), C.byref(trig)), "kv_window_select")
    return out.as_dict(), bool(trig.value)


def kv_window_waste_bound(t_max: float, e_early: float, t_avail: float) -> float:
    return float(load().kv_window_waste_bound(t_max, e_early, t_avail))


def kv_ewma(old: float, sample: float, beta: float) -> float:
    return float(load().kv_ewma(old, sample, beta))


def kv_prefill_prefix_batched(model: Model, cache: PagedCache, token_id_lists, block_tables, logits_out=None,
                              workspace=None, stream=None):
    """Prefix reconstruction of several requests in one call (lists of per-request token ids / block tables)."""
    tok_off = np.concatenate([[0], np.cumsum([len(t) for t in token_id_lists])]).astype(np.int32)
    tab_off = np.concatenate([[0], np.cumsum([len(t) for t in block_tables])]).astype(np.int32)
    ids, pids = _i32(np.concatenate([np.asarray(t, dtype=np.int32) for t in token_id_lists]))
    tabs, ptabs = _i32(np.concatenate([np.asarray(t, dtype=np.int32) for t in block_tables]))
    toff, ptoff = _i32(tok_off)
    boff, pboff = _i32(tab_off)
    ws = workspace if workspace is not None else model.workspace(KV_OP_PREFILL, int(tok_off[-1]))
    _check(load().kv_prefill_prefix_batched(model.handle, C.byref(cache.desc), len(token_id_lists), ptoff, pids, pboff,
                                            ptabs, _ptr(ws), ws.numel(), _ptr(logits_out), _stream(stream)),
           "kv_prefill_prefix_batched")
    return ws
