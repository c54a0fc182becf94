"""ctypes binding of ``libtaq.so``: the same entry points as ``include/taq.h``, taking torch CUDA tensors.

Only argument marshalling happens here (pointers, sizes, the current CUDA stream); every step of the TAQ
cross-attention path runs in the library's kernels.  There is no CPU path: a missing library raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libtaq.so")

TAQ_OK = 0
TAQ_ERR_INVALID_ARG, TAQ_ERR_SHAPE, TAQ_ERR_ALIGNMENT, TAQ_ERR_BUFFER_TOO_SMALL = 1, 2, 3, 4
TAQ_ERR_UNSUPPORTED, TAQ_ERR_CUDA, TAQ_ERR_TIMEOUT = 5, 6, 7
TAQ_OUT_F16, TAQ_OUT_F32, TAQ_OUT_INT8_HEAD_ROWS = 0, 1, 2

EXPORTS = [
    "taq_status_string", "taq_last_error", "taq_version", "taq_packed_weight_bytes", "taq_pack_weights",
    "taq_unpack_weights", "taq_quantize_rows", "taq_kv_layout_of", "taq_kv_bytes", "taq_kv_project",
    "taq_quantized_linear", "taq_cross_attention", "taq_workspace_bytes", "taq_layer_forward",
    "taq_layer_forward_batched", "taq_kv_project_batched", "taq_poll_device_status",
    "taq_static_workspace_capacity", "taq_layer_forward_static", "taq_kv_finalize", "taq_query_attention",
    "taq_quantize_rows_f16", "taq_quantized_linear_i8", "taq_workspace_bytes_a8", "taq_layer_forward_a8",
    "taq_kv_project_a8_workspace_bytes", "taq_kv_project_a8", "taq_token_sensitivity_workspace_bytes",
    "taq_token_sensitivity", "taq_kv_set_prob_mask", "taq_hash_prompt", "taq_kv_cache_create", "taq_kv_cache_destroy",
    "taq_kv_cache_acquire", "taq_kv_cache_release", "taq_kv_cache_drop_checkpoint", "taq_kv_cache_get_stats",
    "taq_dispatch_counts", "taq_dispatch_reset", "taq_linear_plan", "taq_selftest_wait_expiry",
]


class TaqError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"taq status {status}: {message}")
        self.status = status


class WeightDesc(C.Structure):
    _fields_ = [("n_out", C.c_int32), ("k_in", C.c_int32), ("bits", C.c_int32), ("group", C.c_int32)]


class LayerDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("batch", "n_query", "channels", "heads", "n_ctx", "ctx_dim", "w_bits",
                                          "w_group", "q_bits", "kv_bits", "p_bits", "max_trigger", "p_log")]

    @property
    def d_head(self) -> int:
        return self.channels // self.heads


class KvCacheStats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("capacity", "used", "hits", "misses", "evictions")]


class KvLayout(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in ("block_bytes", "off_k_codes", "off_v_codes", "off_k_scales", "off_v_scales",
                                           "off_k_trigger", "off_v_trigger", "off_trig_slot", "off_operands",
                                           "operand_head_bytes")]


class Request(C.Structure):
    _fields_ = [("Wq", C.c_void_p), ("Wout", C.c_void_p), ("kv", C.c_void_p), ("trig_mask", C.c_void_p)]


_lib = None


def lib() -> C.CDLL:
    """Loads the shared library on first use.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2603_22943_b200.build` "
                               "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        vp, sz, i32, i64 = C.c_void_p, C.c_size_t, C.c_int32, C.c_int64
        L.taq_status_string.restype = C.c_char_p
        L.taq_status_string.argtypes = [C.c_int]
        L.taq_last_error.restype = C.c_char_p
        L.taq_last_error.argtypes = []
        L.taq_version.restype = C.c_int
        L.taq_packed_weight_bytes.restype = sz
        L.taq_packed_weight_bytes.argtypes = [C.POINTER(WeightDesc)]
        L.taq_pack_weights.argtypes = [C.POINTER(WeightDesc), vp, vp, vp, sz, vp]
        L.taq_unpack_weights.argtypes = [C.POINTER(WeightDesc), vp, vp, vp, vp]
        L.taq_quantize_rows.argtypes = [vp, i64, i32, i32, vp, vp, vp]
        L.taq_kv_layout_of.argtypes = [C.POINTER(LayerDesc), C.POINTER(KvLayout)]
        L.taq_kv_bytes.restype = sz
        L.taq_kv_bytes.argtypes = [C.POINTER(LayerDesc)]
        L.taq_kv_project.argtypes = [C.POINTER(LayerDesc), vp, vp, vp, vp, vp, sz, vp]
        L.taq_kv_finalize.argtypes = [C.POINTER(LayerDesc), vp, sz, vp]
        L.taq_quantized_linear.argtypes = [C.POINTER(WeightDesc), vp, i64, vp, vp, i32, i32, vp, vp]
        L.taq_cross_attention.argtypes = [C.POINTER(LayerDesc), vp, vp, vp, vp, vp, vp]
        L.taq_workspace_bytes.restype = sz
        L.taq_workspace_bytes.argtypes = [C.POINTER(LayerDesc), i32]
        L.taq_layer_forward.argtypes = [C.POINTER(LayerDesc), vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.taq_query_attention.argtypes = [C.POINTER(LayerDesc), vp, vp, vp, vp, vp, vp, sz, vp]
        L.taq_layer_forward_batched.argtypes = [C.POINTER(LayerDesc), vp, i32, vp, vp, vp, sz, vp]
        L.taq_kv_project_batched.argtypes = [C.POINTER(LayerDesc), vp, i32, vp, vp]
        L.taq_poll_device_status.argtypes = [vp, C.POINTER(i32)]
        L.taq_dispatch_counts.argtypes = [C.POINTER(i64), i32]
        L.taq_dispatch_reset.restype = None
        L.taq_dispatch_reset.argtypes = []
        L.taq_linear_plan.argtypes = [C.POINTER(WeightDesc), i64, i32, i32, i32, i32, C.POINTER(i32)]
        L.taq_selftest_wait_expiry.argtypes = [i64, vp]
        L.taq_static_workspace_capacity.restype = sz
        L.taq_static_workspace_capacity.argtypes = []
        L.taq_layer_forward_static.argtypes = [C.POINTER(LayerDesc), vp, vp, vp, vp, vp, vp, vp]
        L.taq_quantize_rows_f16.argtypes = [vp, i64, i32, vp, vp, vp]
        L.taq_quantized_linear_i8.argtypes = [C.POINTER(WeightDesc), vp, vp, i64, vp, vp, i32, i32, vp, vp]
        L.taq_workspace_bytes_a8.restype = sz
        L.taq_workspace_bytes_a8.argtypes = [C.POINTER(LayerDesc)]
        L.taq_layer_forward_a8.argtypes = [C.POINTER(LayerDesc), vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.taq_kv_project_a8_workspace_bytes.restype = sz
        L.taq_kv_project_a8_workspace_bytes.argtypes = [C.POINTER(LayerDesc)]
        L.taq_kv_project_a8.argtypes = [C.POINTER(LayerDesc), vp, vp, vp, vp, vp, sz, vp, sz, vp]
        L.taq_token_sensitivity_workspace_bytes.restype = sz
        L.taq_token_sensitivity_workspace_bytes.argtypes = [C.POINTER(LayerDesc)]
        L.taq_token_sensitivity.argtypes = [C.POINTER(LayerDesc), vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.taq_kv_set_prob_mask.argtypes = [C.POINTER(LayerDesc), vp, sz, vp, vp]
        u64 = C.c_uint64
        L.taq_hash_prompt.restype = u64
        L.taq_hash_prompt.argtypes = [C.POINTER(i32), i32]
        L.taq_kv_cache_create.restype = vp
        L.taq_kv_cache_create.argtypes = [vp, sz, sz]
        L.taq_kv_cache_destroy.restype = None
        L.taq_kv_cache_destroy.argtypes = [vp]
        L.taq_kv_cache_acquire.argtypes = [vp, u64, u64, C.POINTER(vp), C.POINTER(i32)]
        L.taq_kv_cache_release.argtypes = [vp, u64, u64]
        L.taq_kv_cache_drop_checkpoint.argtypes = [vp, u64]
        L.taq_kv_cache_get_stats.argtypes = [vp, C.POINTER(KvCacheStats)]
        for name in EXPORTS:
            f = getattr(L, name)
            if f.restype is C.c_int and name not in ("taq_version",):
                f.restype = C.c_int
        _lib = L
    return _lib


def _check(status: int) -> None:
    if status != TAQ_OK:
        raise TaqError(status, lib().taq_last_error().decode())


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise TypeError("device tensor expected")
    if not t.is_contiguous():
        raise TypeError("contiguous tensor expected")
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def weight_desc(n_out: int, k_in: int, bits: int, group: int) -> WeightDesc:
    return WeightDesc(n_out, k_in, bits, group)


def layer_desc(batch, n_query, channels, heads, n_ctx, ctx_dim, w_bits, w_group, q_bits=8, kv_bits=8, p_bits=8,
               max_trigger=8, p_log=0) -> LayerDesc:
    return LayerDesc(batch, n_query, channels, heads, n_ctx, ctx_dim, w_bits, w_group, q_bits, kv_bits, p_bits, max_trigger, p_log)


# ------------------------------------------------------------------------------------------------
# Entry points (same names as the C ABI)
# ------------------------------------------------------------------------------------------------

def taq_packed_weight_bytes(desc: WeightDesc) -> int:
    return lib().taq_packed_weight_bytes(C.byref(desc))


def taq_pack_weights(desc: WeightDesc, W: torch.Tensor, bias: Optional[torch.Tensor] = None,
                     packed: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """W fp32 [n_out,k_in] -> packed blob (uint8 tensor)."""
    nbytes = taq_packed_weight_bytes(desc)
    if packed is None:
        if nbytes == 0:
            _check(lib().taq_pack_weights(C.byref(desc), _ptr(W), _ptr(bias), None, 0, _stream(stream)))
        packed = torch.zeros(nbytes, dtype=torch.uint8, device=W.device)
    _check(lib().taq_pack_weights(C.byref(desc), _ptr(W), _ptr(bias), _ptr(packed), packed.numel(), _stream(stream)))
    return packed


def taq_unpack_weights(desc: WeightDesc, packed: torch.Tensor, stream=None):
    g = desc.k_in if desc.group == 0 else desc.group
    n_groups = (desc.k_in + g - 1) // g
    codes = torch.empty((desc.n_out, desc.k_in), dtype=torch.int8, device=packed.device)
    scales = torch.empty((desc.n_out, n_groups), dtype=torch.float32, device=packed.device)
    _check(lib().taq_unpack_weights(C.byref(desc), _ptr(packed), _ptr(codes), _ptr(scales), _stream(stream)))
    return codes, scales


def taq_quantize_rows(x: torch.Tensor, qmax: int = 127, stream=None):
    """x fp32 [rows, cols] -> (int8 codes, fp32 scales)."""
    rows, cols = x.shape
    codes = torch.empty((rows, cols), dtype=torch.int8, device=x.device)
    scales = torch.empty((rows,), dtype=torch.float32, device=x.device)
    _check(lib().taq_quantize_rows(_ptr(x), rows, cols, qmax, _ptr(codes), _ptr(scales), _stream(stream)))
    return codes, scales


def taq_kv_layout_of(desc: LayerDesc) -> KvLayout:
    out = KvLayout()
    _check(lib().taq_kv_layout_of(C.byref(desc), C.byref(out)))
    return out


def taq_kv_bytes(desc: LayerDesc) -> int:
    return lib().taq_kv_bytes(C.byref(desc))


def taq_kv_project(desc: LayerDesc, ctx: torch.Tensor, Wk_packed: torch.Tensor, Wv_packed: torch.Tensor,
                   trig_mask: torch.Tensor, kv: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    if kv is None:
        kv = torch.zeros(max(taq_kv_bytes(desc), 16), dtype=torch.uint8, device=ctx.device)
    _check(lib().taq_kv_project(C.byref(desc), _ptr(ctx), _ptr(Wk_packed), _ptr(Wv_packed), _ptr(trig_mask), _ptr(kv),
                                kv.numel(), _stream(stream)))
    return kv


def taq_kv_finalize(desc: LayerDesc, kv: torch.Tensor, stream=None) -> torch.Tensor:
    """Rebuilds the operand images of hand-assembled K~/V~ blocks."""
    _check(lib().taq_kv_finalize(C.byref(desc), _ptr(kv), kv.numel(), _stream(stream)))
    return kv


def taq_quantized_linear(desc: WeightDesc, x: torch.Tensor, W_packed: torch.Tensor, out_kind: int = TAQ_OUT_F16,
                         heads: int = 1, y: Optional[torch.Tensor] = None, scales: Optional[torch.Tensor] = None, stream=None):
    rows = x.numel() // desc.k_in
    if y is None:
        dt = {TAQ_OUT_F16: torch.float16, TAQ_OUT_F32: torch.float32, TAQ_OUT_INT8_HEAD_ROWS: torch.int8}[out_kind]
        y = torch.empty((rows, desc.n_out), dtype=dt, device=x.device)
    if out_kind == TAQ_OUT_INT8_HEAD_ROWS and scales is None:
        scales = torch.empty((rows, heads), dtype=torch.float32, device=x.device)
    _check(lib().taq_quantized_linear(C.byref(desc), _ptr(x), rows, _ptr(W_packed), _ptr(y), out_kind, heads, _ptr(scales), _stream(stream)))
    return (y, scales) if out_kind == TAQ_OUT_INT8_HEAD_ROWS else y


def taq_quantize_rows_f16(x: torch.Tensor, stream=None):
    """Q_a per token on fp16 data: returns (int8 codes of x's shape, fp32 scales without the last axis)."""
    cols = x.shape[-1]
    rows = x.numel() // cols
    codes = torch.empty(x.shape, dtype=torch.int8, device=x.device)
    scales = torch.empty(x.shape[:-1], dtype=torch.float32, device=x.device)
    _check(lib().taq_quantize_rows_f16(_ptr(x), rows, cols, _ptr(codes), _ptr(scales), _stream(stream)))
    return codes, scales


def taq_quantized_linear_i8(desc: WeightDesc, x_codes: torch.Tensor, x_scales: torch.Tensor, W_packed: torch.Tensor,
                            out_kind: int = TAQ_OUT_F16, heads: int = 1, y: Optional[torch.Tensor] = None,
                            scales: Optional[torch.Tensor] = None, stream=None):
    """The integer-activation projection: int8 codes and per-token scales in."""
    rows = x_codes.numel() // desc.k_in
    if y is None:
        dt = {TAQ_OUT_F16: torch.float16, TAQ_OUT_F32: torch.float32, TAQ_OUT_INT8_HEAD_ROWS: torch.int8}[out_kind]
        y = torch.empty((rows, desc.n_out), dtype=dt, device=x_codes.device)
    if out_kind == TAQ_OUT_INT8_HEAD_ROWS and scales is None:
        scales = torch.empty((rows, heads), dtype=torch.float32, device=x_codes.device)
    _check(lib().taq_quantized_linear_i8(C.byref(desc), _ptr(x_codes), _ptr(x_scales), rows, _ptr(W_packed), _ptr(y), out_kind, heads,
                                         _ptr(scales), _stream(stream)))
    return (y, scales) if out_kind == TAQ_OUT_INT8_HEAD_ROWS else y


def taq_workspace_bytes_a8(desc: LayerDesc) -> int:
    return lib().taq_workspace_bytes_a8(C.byref(desc))


def taq_layer_forward_a8(desc: LayerDesc, x: torch.Tensor, Wq_packed: torch.Tensor, Wout_packed: torch.Tensor, kv: torch.Tensor,
                         trig_mask: torch.Tensor, y: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                         stream=None) -> torch.Tensor:
    """The layer pass with int8 X and O (integer to_q and to_out)."""
    if y is None:
        y = torch.empty((desc.batch, desc.n_query, desc.channels), dtype=torch.float16, device=x.device)
    if workspace is None:
        workspace = torch.empty(max(taq_workspace_bytes_a8(desc), 128), dtype=torch.uint8, device=x.device)
    _check(lib().taq_layer_forward_a8(C.byref(desc), _ptr(x), _ptr(Wq_packed), _ptr(Wout_packed), _ptr(kv), _ptr(trig_mask), _ptr(y),
                                      _ptr(workspace), workspace.numel(), _stream(stream)))
    return y


def taq_kv_project_a8(desc: LayerDesc, ctx: torch.Tensor, Wk_packed: torch.Tensor, Wv_packed: torch.Tensor,
                      trig_mask: torch.Tensor, kv: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                      stream=None) -> torch.Tensor:
    """K/V projection with an int8 text context."""
    if kv is None:
        kv = torch.zeros(max(taq_kv_bytes(desc), 16), dtype=torch.uint8, device=ctx.device)
    if workspace is None:
        workspace = torch.empty(max(lib().taq_kv_project_a8_workspace_bytes(C.byref(desc)), 128), dtype=torch.uint8, device=ctx.device)
    _check(lib().taq_kv_project_a8(C.byref(desc), _ptr(ctx), _ptr(Wk_packed), _ptr(Wv_packed), _ptr(trig_mask), _ptr(kv), kv.numel(),
                                   _ptr(workspace), workspace.numel(), _stream(stream)))
    return kv


def taq_hash_prompt(token_ids) -> int:
    ids = (C.c_int32 * len(token_ids))(*[int(t) for t in token_ids])
    return int(lib().taq_hash_prompt(ids, len(token_ids)))


class KvCache:
    """Host-side K~/V~ cache over a device arena (address + size; the cache never touches the memory)."""

    def __init__(self, arena_ptr: int, arena_bytes: int, entry_bytes: int):
        self._h = lib().taq_kv_cache_create(arena_ptr, arena_bytes, entry_bytes)
        if not self._h:
            raise ValueError("taq_kv_cache_create refused its arguments (arena and entry size must be 128-byte aligned, at least one entry)")
        self.arena_ptr, self.entry_bytes = arena_ptr, entry_bytes

    def acquire(self, checkpoint: int, prompt: int):
        """Returns (entry address, hit)."""
        p, hit = C.c_void_p(), C.c_int32()
        st = lib().taq_kv_cache_acquire(self._h, checkpoint, prompt, C.byref(p), C.byref(hit))
        if st != TAQ_OK:
            raise TaqError(st, "every cache entry is pinned" if st == TAQ_ERR_BUFFER_TOO_SMALL else "kv cache acquire")
        return int(p.value), bool(hit.value)

    def release(self, checkpoint: int, prompt: int) -> None:
        st = lib().taq_kv_cache_release(self._h, checkpoint, prompt)
        if st != TAQ_OK:
            raise TaqError(st, "release of an entry that is not pinned")

    def drop_checkpoint(self, checkpoint: int) -> None:
        st = lib().taq_kv_cache_drop_checkpoint(self._h, checkpoint)
        if st != TAQ_OK:
            raise TaqError(st, "checkpoint still has pinned entries")

    def stats(self) -> dict:
        s = KvCacheStats()
        lib().taq_kv_cache_get_stats(self._h, C.byref(s))
        return {n: getattr(s, n) for n, _ in KvCacheStats._fields_}

    def close(self) -> None:
        if self._h:
            lib().taq_kv_cache_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()


def taq_kv_set_prob_mask(desc: LayerDesc, kv: torch.Tensor, mask_a: torch.Tensor, stream=None) -> torch.Tensor:
    """Eq. 3's M_A independent of Eq. 2's M_KV: the columns marked in mask_a stay fp16."""
    _check(lib().taq_kv_set_prob_mask(C.byref(desc), _ptr(kv), kv.numel(), _ptr(mask_a), _stream(stream)))
    return kv


def taq_token_sensitivity(desc: LayerDesc, x: torch.Tensor, ctx: torch.Tensor, Wq_packed: torch.Tensor, Wk_packed: torch.Tensor,
                          Wv_packed: torch.Tensor, Wout_packed: torch.Tensor, stream=None) -> torch.Tensor:
    """Eq. 1 at layer level: fp64 [n_ctx], Delta_i for b = desc.kv_bits."""
    delta = torch.zeros(desc.n_ctx, dtype=torch.float64, device=x.device)
    ws = torch.empty(max(lib().taq_token_sensitivity_workspace_bytes(C.byref(desc)), 128), dtype=torch.uint8, device=x.device)
    _check(lib().taq_token_sensitivity(C.byref(desc), _ptr(x), _ptr(ctx), _ptr(Wq_packed), _ptr(Wk_packed), _ptr(Wv_packed),
                                       _ptr(Wout_packed), _ptr(delta), _ptr(ws), ws.numel(), _stream(stream)))
    return delta


def taq_cross_attention(desc: LayerDesc, q: torch.Tensor, q_scales: Optional[torch.Tensor], kv: torch.Tensor,
                        trig_mask: torch.Tensor, o: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    if o is None:
        o = torch.empty((desc.batch, desc.n_query, desc.channels), dtype=torch.float16, device=kv.device)
    _check(lib().taq_cross_attention(C.byref(desc), _ptr(q), _ptr(q_scales), _ptr(kv), _ptr(trig_mask), _ptr(o), _stream(stream)))
    return o


def taq_workspace_bytes(desc: LayerDesc, n_requests: int = 1) -> int:
    return lib().taq_workspace_bytes(C.byref(desc), n_requests)


def taq_layer_forward(desc: LayerDesc, x: torch.Tensor, Wq_packed: torch.Tensor, Wout_packed: torch.Tensor, kv: torch.Tensor,
                      trig_mask: torch.Tensor, y: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                      stream=None) -> torch.Tensor:
    if y is None:
        y = torch.empty((desc.batch, desc.n_query, desc.channels), dtype=torch.float16, device=x.device)
    if workspace is None:
        workspace = torch.empty(max(taq_workspace_bytes(desc, 1), 128), dtype=torch.uint8, device=x.device)
    _check(lib().taq_layer_forward(C.byref(desc), _ptr(x), _ptr(Wq_packed), _ptr(Wout_packed), _ptr(kv), _ptr(trig_mask), _ptr(y),
                                   _ptr(workspace), workspace.numel(), _stream(stream)))
    return y


def taq_query_attention(desc: LayerDesc, x: torch.Tensor, Wq_packed: torch.Tensor, kv: torch.Tensor, trig_mask: torch.Tensor,
                        o: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """x -> O (to_q, Q_a, attention); one fused kernel for C = 320 / 8 heads / W4."""
    if o is None:
        o = torch.empty((desc.batch, desc.n_query, desc.channels), dtype=torch.float16, device=x.device)
    if workspace is None:
        workspace = torch.empty(max(taq_workspace_bytes(desc, 1), 128), dtype=torch.uint8, device=x.device)
    _check(lib().taq_query_attention(C.byref(desc), _ptr(x), _ptr(Wq_packed), _ptr(kv), _ptr(trig_mask), _ptr(o), _ptr(workspace),
                                     workspace.numel(), _stream(stream)))
    return o


def taq_static_workspace_capacity() -> int:
    return lib().taq_static_workspace_capacity()


def taq_layer_forward_static(desc: LayerDesc, x: torch.Tensor, Wq_packed: torch.Tensor, Wout_packed: torch.Tensor,
                             kv: torch.Tensor, trig_mask: torch.Tensor, y: torch.Tensor, stream=None) -> torch.Tensor:
    """The layer pass on the library's built-in scratch array.  ``y`` must be supplied: this wrapper, like the
    entry point under it, allocates nothing."""
    _check(lib().taq_layer_forward_static(C.byref(desc), _ptr(x), _ptr(Wq_packed), _ptr(Wout_packed), _ptr(kv), _ptr(trig_mask),
                                          _ptr(y), _stream(stream)))
    return y


def make_request_table(entries: Sequence[Sequence[torch.Tensor]], device) -> torch.Tensor:
    """Device array of taq_request from (Wq, Wout, kv, mask) tensor tuples (4 pointers per entry)."""
    flat = []
    for e in entries:
        flat.extend(int(t.data_ptr()) for t in e)
    return torch.tensor(flat, dtype=torch.int64).to(device)


def taq_layer_forward_batched(desc: LayerDesc, reqs: torch.Tensor, n_requests: int, x: torch.Tensor,
                              y: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    if y is None:
        y = torch.empty((n_requests, desc.n_query, desc.channels), dtype=torch.float16, device=x.device)
    if workspace is None:
        workspace = torch.empty(max(taq_workspace_bytes(desc, n_requests), 128), dtype=torch.uint8, device=x.device)
    _check(lib().taq_layer_forward_batched(C.byref(desc), _ptr(reqs), n_requests, _ptr(x), _ptr(y), _ptr(workspace),
                                           workspace.numel(), _stream(stream)))
    return y


def taq_kv_project_batched(desc: LayerDesc, reqs: torch.Tensor, n_requests: int, ctx: torch.Tensor, stream=None) -> None:
    _check(lib().taq_kv_project_batched(C.byref(desc), _ptr(reqs), n_requests, _ptr(ctx), _stream(stream)))


KERNEL_FAMILIES = ("linear_tensor", "linear_generic", "attention_tensor", "attention_generic", "query_attention_fused",
                   "layer_fused", "layer_fused_a8")


def taq_dispatch_counts() -> dict:
    """Launches per kernel family since the last taq_dispatch_reset()."""
    arr = (C.c_int64 * len(KERNEL_FAMILIES))()
    _check(lib().taq_dispatch_counts(arr, len(KERNEL_FAMILIES)))
    return {k: int(arr[i]) for i, k in enumerate(KERNEL_FAMILIES)}


def taq_dispatch_reset() -> None:
    lib().taq_dispatch_reset()


LINEAR_PLAN_FIELDS = ("bn", "nstage", "mode", "ring_bytes", "staging_bytes", "off_raw", "off_bias", "off_bars", "total", "limit")


def taq_linear_plan(desc: "WeightDesc", rows: int, out_kind: int, heads: int = 1, int8_activations: bool = False, batched: bool = False) -> dict:
    """Shared-memory plan of the tensor-core dequant-GEMM for a problem (host arithmetic; needs no GPU)."""
    arr = (C.c_int32 * 10)()
    _check(lib().taq_linear_plan(C.byref(desc), rows, out_kind, heads, int(int8_activations), int(batched), arr))
    return {k: int(arr[i]) for i, k in enumerate(LINEAR_PLAN_FIELDS)}


def taq_selftest_wait_expiry(limit_cycles: int, stream=None) -> None:
    """Launches one block that waits (bounded by limit_cycles) on a barrier nothing arrives on."""
    _check(lib().taq_selftest_wait_expiry(limit_cycles, _stream(stream)))


def taq_poll_device_status(stream=None) -> int:
    """Synchronises the stream; raises TaqError if a kernel recorded a device-side error."""
    blk = C.c_int32(-1)
    _check(lib().taq_poll_device_status(_stream(stream), C.byref(blk)))
    return TAQ_OK
