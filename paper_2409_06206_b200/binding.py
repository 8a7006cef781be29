"""ctypes binding of libgswa.so: argument marshalling only, every step runs in the CUDA library.

The functions mirror the C entry points of include/gswa.h one to one.  Tensors
are torch tensors used purely as device (or pinned host) memory; their
`data_ptr()` is what crosses the boundary.  There is no CPU fallback: if the
library cannot be loaded, importing-and-calling raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libgswa.so")

GSWA_F32, GSWA_BF16 = 0, 1
FLAG_ACCUMULATE, FLAG_GENERIC, FLAG_FUSED_FWD, FLAG_TCGEN05_ATTN, FLAG_COPY_LOADERS = 1, 2, 4, 8, 16

STATIC_SCRATCH_BYTES = 16 << 20

EXPORTS = ("gswa_workspace_query", "gswa_forward", "gswa_forward_static", "gswa_static_status", "gswa_backward",
           "gswa_astl_workspace_query", "gswa_astl_forward", "gswa_astl_backward",
           "gswa_index_maps", "gswa_debug_index_maps", "gswa_debug_expire_wait", "gswa_step_host", "gswa_scratch_status", "gswa_profile_enable", "gswa_profile_read", "gswa_launch_count", "gswa_status_string")


class GswaError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__("libgswa status %d: %s" % (status, text))
        self.status = status


class _Desc(C.Structure):
    _fields_ = [("B", C.c_int32), ("H", C.c_int32), ("W", C.c_int32), ("C", C.c_int32), ("num_heads", C.c_int32),
                ("window", C.c_int32), ("num_groups", C.c_int32), ("group_heads", C.POINTER(C.c_int32)),
                ("group_shift", C.POINTER(C.c_int32)), ("dtype", C.c_int32), ("qk_dim", C.c_int32),
                ("v_dim", C.c_int32), ("flags", C.c_uint32)]


ASTL_PARAMS = ("ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_proj", "b_proj", "bias_table", "ln2_g", "ln2_b", "w_fc1", "b_fc1",
               "w_fc2", "b_fc2")
ASTL_GRADS = ("dln1_g", "dln1_b", "dw_qkv", "db_qkv", "dw_proj", "db_proj", "dbias_table", "dln2_g", "dln2_b", "dw_fc1",
              "db_fc1", "dw_fc2", "db_fc2")


class _AstlParams(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ASTL_PARAMS]


class _AstlGrads(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ASTL_GRADS]


class Desc:
    """Owns a gswa_desc and the two host arrays it points to."""

    def __init__(self, B: int, H: int, W: int, C_: int, num_heads: int, window: int, group_heads: Sequence[int],
                 group_shift: Sequence[int], dtype: str = "bf16", flags: int = 0, qk_dim: int = 0, v_dim: int = 0):
        if len(group_heads) != len(group_shift):
            raise ValueError("group_heads and group_shift differ in length")
        G = len(group_heads)
        self._gh = (C.c_int32 * max(G, 1))(*group_heads)
        self._gs = (C.c_int32 * max(G, 1))(*group_shift)
        self.c = _Desc(B, H, W, C_, num_heads, window, G, C.cast(self._gh, C.POINTER(C.c_int32)),
                       C.cast(self._gs, C.POINTER(C.c_int32)), {"f32": GSWA_F32, "bf16": GSWA_BF16}[dtype], qk_dim,
                       v_dim, flags)
        self.dtype = dtype
        self.shape = (B, H, W, C_)
        self.num_heads, self.window = num_heads, window

    @classmethod
    def from_config(cls, cfg, layer: int = 0, batch: Optional[int] = None, flags: int = 0) -> "Desc":
        from .inputs import layer_groups
        gh, gs = layer_groups(cfg, layer)
        return cls(cfg.B if batch is None else batch, cfg.H, cfg.W, cfg.C, cfg.num_heads, cfg.window, gh, gs,
                   cfg.dtype, flags, getattr(cfg, "qk_dim", 0), getattr(cfg, "v_dim", 0))

    def with_flags(self, flags: int) -> "Desc":
        B, H, W, C_ = self.shape
        return Desc(B, H, W, C_, self.num_heads, self.window, list(self._gh)[:self.c.num_groups],
                    list(self._gs)[:self.c.num_groups], self.dtype, flags, self.c.qk_dim, self.c.v_dim)


_lib = None


def lib() -> C.CDLL:
    """Loads libgswa.so (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libgswa.so is missing: build it with `python -m paper_2409_06206_b200.build` "
                               "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, sz, dp = C.c_void_p, C.c_size_t, C.POINTER(_Desc)
        szp = C.POINTER(C.c_size_t)
        L.gswa_workspace_query.argtypes = [dp, szp, szp, szp, szp]
        L.gswa_forward.argtypes = [dp] + [vp] * 9 + [sz, vp]
        L.gswa_forward_static.argtypes = [dp] + [vp] * 8
        L.gswa_forward_static.restype = C.c_int
        L.gswa_backward.argtypes = [dp] + [vp] * 14 + [sz, vp]
        L.gswa_index_maps.argtypes = [dp, C.c_int32] + [vp] * 6
        L.gswa_step_host.argtypes = [dp] + [vp] * 15 + [sz, szp, vp]
        L.gswa_scratch_status.argtypes = [dp, vp, vp]
        L.gswa_scratch_status.restype = C.c_int
        L.gswa_static_status.argtypes = [vp]
        L.gswa_static_status.restype = C.c_int
        L.gswa_astl_workspace_query.argtypes = [dp, C.c_int32, szp, szp, szp, szp]
        L.gswa_astl_forward.argtypes = [dp, C.c_int32, vp, C.POINTER(_AstlParams), vp, vp, vp, sz, vp]
        L.gswa_astl_backward.argtypes = [dp, C.c_int32, vp, C.POINTER(_AstlParams), vp, vp, vp, C.POINTER(_AstlGrads), vp, sz, vp]
        for name in ("gswa_astl_workspace_query", "gswa_astl_forward", "gswa_astl_backward"):
            getattr(L, name).restype = C.c_int
        L.gswa_debug_index_maps.argtypes = [dp, C.c_int32] + [vp] * 5
        L.gswa_debug_index_maps.restype = C.c_int
        L.gswa_debug_expire_wait.argtypes = [dp, vp, vp]
        L.gswa_debug_expire_wait.restype = C.c_int
        L.gswa_profile_enable.argtypes = [C.c_int]
        L.gswa_profile_read.argtypes = [C.c_int32, C.c_char_p, C.POINTER(C.c_float), C.POINTER(C.c_int32)]
        L.gswa_profile_enable.restype = C.c_int
        L.gswa_profile_read.restype = C.c_int
        L.gswa_launch_count.argtypes = []
        L.gswa_launch_count.restype = C.c_uint64
        L.gswa_status_string.argtypes = [C.c_int]
        L.gswa_status_string.restype = C.c_char_p
        for name in ("gswa_workspace_query", "gswa_forward", "gswa_backward", "gswa_index_maps", "gswa_step_host"):
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def gswa_status_string(status: int) -> str:
    return lib().gswa_status_string(int(status)).decode()


def _check(status: int) -> None:
    if status != 0:
        raise GswaError(status, gswa_status_string(status))


def gswa_workspace_query(desc: Desc):
    """-> (saved_bytes, fwd_scratch_bytes, infer_scratch_bytes, bwd_scratch_bytes)"""
    out = [C.c_size_t(0) for _ in range(4)]
    _check(lib().gswa_workspace_query(C.byref(desc.c), *[C.byref(o) for o in out]))
    return tuple(int(o.value) for o in out)


def gswa_forward(desc: Desc, x, w_qkv, b_qkv, w_proj, b_proj, bias_table, y, saved, scratch, scratch_bytes=None,
                 stream=None) -> None:
    if scratch_bytes is None:
        scratch_bytes = 0 if scratch is None else scratch.numel() * scratch.element_size()
    _check(lib().gswa_forward(C.byref(desc.c), _ptr(x), _ptr(w_qkv), _ptr(b_qkv), _ptr(w_proj), _ptr(b_proj),
                              _ptr(bias_table), _ptr(y), _ptr(saved), _ptr(scratch), scratch_bytes, _stream(stream)))


def gswa_forward_static(desc: Desc, x, w_qkv, b_qkv, w_proj, b_proj, bias_table, y, stream=None) -> None:
    """Inference forward without any caller-provided scratch: for hosts that cannot allocate device memory.

    The library keeps the intermediates in a fixed array of STATIC_SCRATCH_BYTES inside its own device image;
    larger layers raise GswaError(-5).  Calls share that array, so calls that overlap on the GPU race."""
    _check(lib().gswa_forward_static(C.byref(desc.c), _ptr(x), _ptr(w_qkv), _ptr(b_qkv), _ptr(w_proj), _ptr(b_proj),
                                     _ptr(bias_table), _ptr(y), _stream(stream)))


def gswa_backward(desc: Desc, x, w_qkv, b_qkv, w_proj, bias_table, saved, dy, dx, dw_qkv, db_qkv, dw_proj, db_proj,
                  dbias_table, scratch, scratch_bytes=None, stream=None) -> None:
    if scratch_bytes is None:
        scratch_bytes = 0 if scratch is None else scratch.numel() * scratch.element_size()
    _check(lib().gswa_backward(C.byref(desc.c), _ptr(x), _ptr(w_qkv), _ptr(b_qkv), _ptr(w_proj), _ptr(bias_table),
                               _ptr(saved), _ptr(dy), _ptr(dx), _ptr(dw_qkv), _ptr(db_qkv), _ptr(dw_proj),
                               _ptr(db_proj), _ptr(dbias_table), _ptr(scratch), scratch_bytes, _stream(stream)))


def gswa_index_maps(desc: Desc, group: int, win, slot, region, token_of, rel_index, stream=None) -> None:
    _check(lib().gswa_index_maps(C.byref(desc.c), group, _ptr(win), _ptr(slot), _ptr(region), _ptr(token_of),
                                 _ptr(rel_index), _stream(stream)))


def gswa_astl_workspace_query(desc: Desc, mlp_hidden: int):
    """-> (saved_bytes, fwd_scratch_bytes, infer_scratch_bytes, bwd_scratch_bytes) of the whole layer"""
    out = [C.c_size_t(0) for _ in range(4)]
    _check(lib().gswa_astl_workspace_query(C.byref(desc.c), mlp_hidden, *[C.byref(o) for o in out]))
    return tuple(int(o.value) for o in out)


def _astl_struct(cls, names, tensors):
    return cls(*[_ptr(tensors.get(n)) for n in names])


def gswa_astl_forward(desc: Desc, mlp_hidden: int, x, params: dict, y, saved, scratch, stream=None) -> None:
    """params: name -> tensor for the names of ASTL_PARAMS (missing / None entries are passed as NULL)."""
    q = _astl_struct(_AstlParams, ASTL_PARAMS, params)
    _check(lib().gswa_astl_forward(C.byref(desc.c), mlp_hidden, _ptr(x), C.byref(q), _ptr(y), _ptr(saved), _ptr(scratch),
                                   scratch.numel() * scratch.element_size(), _stream(stream)))


def gswa_astl_backward(desc: Desc, mlp_hidden: int, x, params: dict, saved, dy, dx, grads: dict, scratch, stream=None) -> None:
    q = _astl_struct(_AstlParams, ASTL_PARAMS, params)
    g = _astl_struct(_AstlGrads, ASTL_GRADS, grads)
    _check(lib().gswa_astl_backward(C.byref(desc.c), mlp_hidden, _ptr(x), C.byref(q), _ptr(saved), _ptr(dy), _ptr(dx),
                                    C.byref(g), _ptr(scratch), scratch.numel() * scratch.element_size(), _stream(stream)))


def gswa_debug_index_maps(desc: Desc, group: int, win_id, slot, region, rel_index, stream=None) -> None:
    _check(lib().gswa_debug_index_maps(C.byref(desc.c), group, _ptr(win_id), _ptr(slot), _ptr(region), _ptr(rel_index),
                                       _stream(stream)))


def gswa_debug_expire_wait(desc: Desc, scratch, stream=None) -> None:
    """Test hook: makes a bounded device-side wait run out on purpose (sets the error word of `scratch`)."""
    _check(lib().gswa_debug_expire_wait(C.byref(desc.c), _ptr(scratch), _stream(stream)))


def gswa_static_status(stream=None) -> None:
    """Waits for the stream and raises GswaError(-7) if the last gswa_forward_static on this device gave up a wait."""
    _check(lib().gswa_static_status(_stream(stream)))


def gswa_step_host_arena_bytes(desc: Desc) -> int:
    need = C.c_size_t(0)
    lib().gswa_step_host(C.byref(desc.c), *([None] * 15), 0, C.byref(need), None)
    return int(need.value)


def gswa_step_host(desc: Desc, x, w_qkv, b_qkv, w_proj, b_proj, bias_table, dy, y, dx, dw_qkv, db_qkv, dw_proj,
                   db_proj, dbias_table, arena, stream=None) -> None:
    """All tensors except `arena` are HOST tensors (pinned for asynchronous copies)."""
    need = C.c_size_t(0)
    _check(lib().gswa_step_host(C.byref(desc.c), _ptr(x), _ptr(w_qkv), _ptr(b_qkv), _ptr(w_proj), _ptr(b_proj),
                                _ptr(bias_table), _ptr(dy), _ptr(y), _ptr(dx), _ptr(dw_qkv), _ptr(db_qkv),
                                _ptr(dw_proj), _ptr(db_proj), _ptr(dbias_table), _ptr(arena),
                                arena.numel() * arena.element_size(), C.byref(need), _stream(stream)))


def gswa_scratch_status(desc: Desc, scratch, stream=None) -> None:
    """Waits for the stream and raises GswaError(-7) if a kernel of the last call on `scratch` gave up a wait."""
    _check(lib().gswa_scratch_status(C.byref(desc.c), _ptr(scratch), _stream(stream)))


def gswa_profile_enable(on: bool) -> None:
    _check(lib().gswa_profile_enable(1 if on else 0))


def gswa_profile_read(max_records: int = 4096):
    """-> list of (kernel name, milliseconds), one entry per launch recorded since the last read."""
    names = C.create_string_buffer(max_records * 32)
    ms = (C.c_float * max_records)()
    n = C.c_int32(0)
    _check(lib().gswa_profile_read(max_records, names, ms, C.byref(n)))
    raw = names.raw
    return [(raw[i * 32:(i + 1) * 32].split(b"\0", 1)[0].decode(), float(ms[i])) for i in range(n.value)]


def gswa_launch_count() -> int:
    return int(lib().gswa_launch_count())
