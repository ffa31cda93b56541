"""Thin ctypes binding of libgd.so: argument marshalling only.

Every function has the name and the meaning of the C entry point in include/gd.h; tensors are
passed for device (or page-locked host) buffers and only their addresses cross the boundary.
PyTorch is used for device memory and streams; all arithmetic happens inside the library.  There
is no fallback: if the library cannot be loaded, the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

from . import build as _build

GD_OK = 0
GD_ERR_INVALID_ARG = -1
GD_ERR_TOO_LARGE = -2
GD_ERR_WORKSPACE = -3
GD_ERR_CUDA = -4
GD_ERR_DEVICE_TIMEOUT = -5
GD_ERR_INTERNAL = -6
GD_SCOPE_GLOBAL = 0
GD_SCOPE_PER_LAYER = 1
GD_VALUES_FP32 = 0
GD_VALUES_TWO_MEANS = 1
GD_VALUES_THRESHOLD = 2
GD_VALUES_COLUMN_MEANS = 3
GD_FLAG_NO_PREDICTION = 1
GD_FLAG_SAMPLED_THRESHOLD = 2
GD_FLAG_QUANT_ERROR_FEEDBACK = 4
GD_FLAG_NO_EARLY_ZERO = 8
GD_FLAG_PLAIN_RADIX = 16
GD_FLAG_PREDICT_ALWAYS = 32
GD_ERR_OVERFLOW = -7
GD_APPLY_ATOMIC = 1

EXPORTS = [
    "gd_status_string", "gd_kept_count", "gd_total_kept", "gd_workspace_bytes", "gd_apply_workspace_bytes",
    "gd_compress", "gd_decompress_apply", "gd_residual_reset", "gd_status", "gd_get_stats", "gd_step_host",
    "gd_profile_enable", "gd_profile_collect", "gd_launch_count", "gd_compress_static",
    "gd_selftest_bounded_wait", "gd_sampled_capacity", "gd_means_pairs",
]
GD_STATIC_WORKSPACE_BYTES = 16 << 20


class GdError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


class _CompressArgs(C.Structure):
    _fields_ = [
        ("grad", C.c_void_p), ("residual", C.c_void_p), ("n", C.c_uint64),
        ("layer_off", C.POINTER(C.c_uint64)), ("n_layers", C.c_uint32), ("n_shards", C.c_uint32),
        ("shard_off", C.POINTER(C.c_uint64)), ("drop_ppm", C.c_uint32), ("scope_mode", C.c_int32),
        ("value_mode", C.c_int32), ("flags", C.c_uint32),
        ("out_idx", C.c_void_p), ("out_val", C.c_void_p), ("out_shard_cnt_off", C.c_void_p),
        ("out_tau", C.c_void_p), ("out_means", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t), ("delta_base", C.c_void_p),
        ("layer_cols", C.POINTER(C.c_uint32)),
    ]


class _Push(C.Structure):
    _fields_ = [("idx", C.c_void_p), ("val", C.c_void_p), ("shard_cnt_off", C.c_void_p), ("means", C.c_void_p)]


class _ApplyArgs(C.Structure):
    _fields_ = [
        ("params", C.POINTER(C.c_void_p)), ("shard_off", C.POINTER(C.c_uint64)),
        ("n_shards", C.c_uint32), ("n_pushes", C.c_uint32), ("pushes", C.POINTER(_Push)),
        ("value_mode", C.c_int32), ("alpha", C.c_float),
        ("layer_off", C.POINTER(C.c_uint64)), ("n_layers", C.c_uint32), ("flags", C.c_uint32),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t), ("layer_cols", C.POINTER(C.c_uint32)),
    ]


class _Stats(C.Structure):
    _fields_ = [("status", C.c_int32), ("n_scopes", C.c_uint32), ("n_scopes_predicted", C.c_uint32),
                ("n_scopes_dense", C.c_uint32), ("n_candidates", C.c_uint64), ("n_kept", C.c_uint64)]


class _HostIo(C.Structure):
    _fields_ = [("grad_host", C.c_void_p), ("idx_host", C.c_void_p), ("val_host", C.c_void_p),
                ("shard_cnt_off_host", C.c_void_p), ("means_host", C.c_void_p)]


_lib = None


def library_path() -> str:
    return _build.LIB_PATH


def load_library():
    """Loads libgd.so (once).  Raises if it has not been built: there is no other code path."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_1704_05021_b200.build`")
    lib = C.CDLL(path)
    lib.gd_status_string.restype = C.c_char_p
    lib.gd_status_string.argtypes = [C.c_int]
    lib.gd_kept_count.argtypes = [C.c_uint64, C.c_uint32, C.POINTER(C.c_uint64)]
    lib.gd_total_kept.argtypes = [C.POINTER(C.c_uint64), C.c_uint32, C.c_int, C.c_uint32, C.POINTER(C.c_uint64)]
    lib.gd_workspace_bytes.argtypes = [C.POINTER(C.c_uint64), C.c_uint32, C.POINTER(C.c_uint32), C.c_uint32, C.c_int,
                                       C.c_uint32, C.POINTER(C.c_size_t)]
    lib.gd_means_pairs.argtypes = [C.c_uint32, C.POINTER(C.c_uint32), C.c_int, C.POINTER(C.c_uint64)]
    lib.gd_apply_workspace_bytes.argtypes = [C.c_uint32, C.c_uint32, C.POINTER(C.c_size_t)]
    lib.gd_compress.argtypes = [C.POINTER(_CompressArgs), C.c_void_p]
    lib.gd_decompress_apply.argtypes = [C.POINTER(_ApplyArgs), C.c_void_p]
    lib.gd_residual_reset.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p]
    lib.gd_status.argtypes = [C.c_void_p, C.c_void_p]
    lib.gd_get_stats.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(_Stats)]
    lib.gd_step_host.argtypes = [C.POINTER(_CompressArgs), C.POINTER(_ApplyArgs), C.POINTER(_HostIo), C.c_void_p]
    lib.gd_compress_static.argtypes = [C.POINTER(_CompressArgs), C.c_void_p, C.POINTER(C.c_void_p)]
    lib.gd_selftest_bounded_wait.argtypes = [C.c_void_p, C.c_size_t, C.c_uint32, C.c_void_p]
    lib.gd_sampled_capacity.argtypes = [C.POINTER(C.c_uint64), C.c_uint32, C.c_int, C.c_uint32, C.POINTER(C.c_uint64)]
    lib.gd_profile_enable.argtypes = [C.c_int]
    lib.gd_profile_collect.argtypes = [C.POINTER(C.c_float), C.POINTER(C.c_uint32), C.c_uint32, C.POINTER(C.c_uint32)]
    lib.gd_launch_count.argtypes = [C.POINTER(C.c_uint64)]
    for name in EXPORTS:
        if name != "gd_status_string":
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _u64_array(values: Sequence[int]):
    return (C.c_uint64 * len(values))(*[int(v) for v in values])


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream_handle(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(code: int, where: str):
    if code != GD_OK:
        raise GdError(code, where)


def status_string(code: int) -> str:
    return load_library().gd_status_string(int(code)).decode()


def gd_kept_count(n_scope: int, drop_ppm: int) -> int:
    out = C.c_uint64(0)
    _check(load_library().gd_kept_count(n_scope, drop_ppm, C.byref(out)), "gd_kept_count")
    return out.value


def gd_total_kept(layer_off: Sequence[int], scope_mode: int, drop_ppm: int) -> int:
    out = C.c_uint64(0)
    arr = _u64_array(layer_off)
    _check(load_library().gd_total_kept(arr, len(layer_off) - 1, scope_mode, drop_ppm, C.byref(out)), "gd_total_kept")
    return out.value


def _u32_array(values: Optional[Sequence[int]]):
    return None if values is None else (C.c_uint32 * len(values))(*[int(v) for v in values])


def gd_workspace_bytes(layer_off: Sequence[int], n_shards: int, scope_mode: int, drop_ppm: int,
                       layer_cols: Optional[Sequence[int]] = None) -> int:
    out = C.c_size_t(0)
    arr = _u64_array(layer_off)
    _check(load_library().gd_workspace_bytes(arr, len(layer_off) - 1, _u32_array(layer_cols), n_shards, scope_mode,
                                             drop_ppm, C.byref(out)), "gd_workspace_bytes")
    return out.value


def gd_means_pairs(n_layers: int, layer_cols: Optional[Sequence[int]], value_mode: int) -> int:
    out = C.c_uint64(0)
    _check(load_library().gd_means_pairs(n_layers, _u32_array(layer_cols), value_mode, C.byref(out)), "gd_means_pairs")
    return out.value


def gd_apply_workspace_bytes(n_shards: int, n_layers: int) -> int:
    out = C.c_size_t(0)
    _check(load_library().gd_apply_workspace_bytes(n_shards, n_layers, C.byref(out)), "gd_apply_workspace_bytes")
    return out.value


class CompressCall:
    """The marshalled argument block of one gd_compress call (kept so it can be re-issued cheaply)."""

    def __init__(self, grad, residual, layer_off, shard_off, drop_ppm, scope_mode, value_mode, out_idx, out_val,
                 out_shard_cnt_off, out_tau, out_means, workspace, flags=0, delta_base=None, layer_cols=None):
        self._keep = (grad, residual, out_idx, out_val, out_shard_cnt_off, out_tau, out_means, workspace, delta_base)
        self._layer_off = _u64_array(layer_off)
        self._shard_off = _u64_array(shard_off)
        a = _CompressArgs()
        a.grad, a.residual, a.n = _ptr(grad), _ptr(residual), int(layer_off[-1])
        a.layer_off, a.n_layers = self._layer_off, len(layer_off) - 1
        a.shard_off, a.n_shards = self._shard_off, len(shard_off) - 1
        a.drop_ppm, a.scope_mode, a.value_mode, a.flags = drop_ppm, scope_mode, value_mode, flags
        a.out_idx, a.out_val, a.out_shard_cnt_off = _ptr(out_idx), _ptr(out_val), _ptr(out_shard_cnt_off)
        a.out_tau, a.out_means = _ptr(out_tau), _ptr(out_means)
        a.workspace = _ptr(workspace)
        a.workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        a.delta_base = _ptr(delta_base)
        self._layer_cols = _u32_array(layer_cols)
        if self._layer_cols is not None:
            a.layer_cols = self._layer_cols
        self.args = a

    def set_grad(self, grad: torch.Tensor):
        self._keep = (grad,) + self._keep[1:]
        self.args.grad = grad.data_ptr()


class ApplyCall:
    """The marshalled argument block of one gd_decompress_apply call."""

    def __init__(self, params: Sequence[torch.Tensor], shard_off, pushes, value_mode, alpha, workspace,
                 layer_off=None, layer_cols=None, flags=0):
        self._keep = (list(params), pushes, workspace)
        n_shards = len(shard_off) - 1
        self._params = (C.c_void_p * n_shards)(*[p.data_ptr() if p.numel() else None for p in params])
        self._shard_off = _u64_array(shard_off)
        self._pushes = (_Push * max(len(pushes), 1))()
        for i, p in enumerate(pushes):
            self._pushes[i].idx = _ptr(p["idx"])
            self._pushes[i].val = _ptr(p.get("val"))
            self._pushes[i].shard_cnt_off = _ptr(p["shard_cnt_off"])
            self._pushes[i].means = _ptr(p.get("means"))
        self._layer_off = _u64_array(layer_off) if layer_off is not None else None
        a = _ApplyArgs()
        a.params, a.shard_off, a.n_shards = self._params, self._shard_off, n_shards
        a.n_pushes, a.pushes = len(pushes), self._pushes
        a.value_mode, a.alpha, a.flags = value_mode, float(alpha), int(flags)
        if self._layer_off is not None:
            a.layer_off, a.n_layers = self._layer_off, len(layer_off) - 1
        a.workspace = _ptr(workspace)
        a.workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        self._layer_cols = _u32_array(layer_cols)
        if self._layer_cols is not None:
            a.layer_cols = self._layer_cols
        self.args = a


def gd_compress(call: CompressCall, stream=None) -> None:
    _check(load_library().gd_compress(C.byref(call.args), _stream_handle(stream)), "gd_compress")


def gd_decompress_apply(call: ApplyCall, stream=None) -> None:
    _check(load_library().gd_decompress_apply(C.byref(call.args), _stream_handle(stream)), "gd_decompress_apply")


def gd_residual_reset(residual: torch.Tensor, stream=None) -> None:
    _check(load_library().gd_residual_reset(residual.data_ptr(), residual.numel(), _stream_handle(stream)),
           "gd_residual_reset")


def gd_status(workspace: torch.Tensor, stream=None) -> int:
    return load_library().gd_status(workspace.data_ptr(), _stream_handle(stream))


def gd_get_stats(workspace: torch.Tensor, stream=None) -> dict:
    st = _Stats()
    _check(load_library().gd_get_stats(workspace.data_ptr(), _stream_handle(stream), C.byref(st)), "gd_get_stats")
    return {name: getattr(st, name) for name, _ in _Stats._fields_}


def gd_step_host(call: CompressCall, apply: Optional[ApplyCall], grad_host: torch.Tensor,
                 idx_host: Optional[torch.Tensor] = None, val_host: Optional[torch.Tensor] = None,
                 shard_cnt_off_host: Optional[torch.Tensor] = None, means_host: Optional[torch.Tensor] = None,
                 stream=None) -> None:
    io = _HostIo(_ptr(grad_host), _ptr(idx_host), _ptr(val_host), _ptr(shard_cnt_off_host), _ptr(means_host))
    ap = C.byref(apply.args) if apply is not None else None
    _check(load_library().gd_step_host(C.byref(call.args), ap, C.byref(io), _stream_handle(stream)), "gd_step_host")


PROFILE_TAGS = ["setup", "sample_select", "add_emit", "dense_select", "dense_compact", "cand_select", "cand_compact",
                "finalize", "apply", "pack_sampled", "means", "feedback", "cand_select_compact", "setup_predict", "dense_hist", "dense_find", "dense_fused"]
# Kernels one gd_compress launches, in order, by the path the call takes (each is one launch and, with
# gd_profile_enable(2), one tagged event pair); gd_decompress_apply adds one "apply" per push.
STEP_KERNELS = {
    "predicted": ["setup_predict", "add_emit", "cand_select_compact"],
    "predicted_large_sample": ["setup", "sample_select", "add_emit", "cand_select_compact"],
    "predicted_many_scopes": ["setup", "sample_select", "add_emit", "cand_select", "cand_compact"],
    "dense": ["setup", "dense_hist", "dense_find", "dense_hist", "dense_find", "add_emit", "cand_select_compact"],
    "dense_short_vector": ["dense_fused"],
    "dense_many_scopes": ["setup", "add_emit", "dense_select", "dense_compact"],
    "sampled": ["setup", "sample_select", "add_emit", "pack_sampled"],
}


def gd_profile_enable(mode) -> None:
    """0 / False: off; 1 / True: time the fused pass of every gd_compress; 2: time every kernel."""
    _check(load_library().gd_profile_enable(int(mode)), "gd_profile_enable")


def gd_profile_collect(capacity: int = 4096, with_tags: bool = False):
    buf = (C.c_float * capacity)()
    tags = (C.c_uint32 * capacity)()
    cnt = C.c_uint32(0)
    _check(load_library().gd_profile_collect(buf, tags, capacity, C.byref(cnt)), "gd_profile_collect")
    if with_tags:
        return [(PROFILE_TAGS[tags[i]], buf[i]) for i in range(cnt.value)]
    return [buf[i] for i in range(cnt.value)]


def gd_launch_count() -> int:
    out = C.c_uint64(0)
    _check(load_library().gd_launch_count(C.byref(out)), "gd_launch_count")
    return out.value


def gd_compress_static(call: CompressCall, stream=None) -> int:
    """gd_compress on the library's built-in scratch area (for callers that cannot allocate a workspace).

    The workspace stored in `call` is ignored.  Returns the device address of the scratch area, which
    is what gd_status_at / gd_get_stats_at take.  Calls on one device must not overlap on the GPU.
    """
    out = C.c_void_p(0)
    _check(load_library().gd_compress_static(C.byref(call.args), _stream_handle(stream), C.byref(out)),
           "gd_compress_static")
    return out.value or 0


def gd_status_at(workspace_address: int, stream=None) -> int:
    """gd_status for a workspace known by its device address (e.g. the one gd_compress_static returns)."""
    return load_library().gd_status(C.c_void_p(workspace_address), _stream_handle(stream))


def gd_get_stats_at(workspace_address: int, stream=None) -> dict:
    """gd_get_stats for a workspace known by its device address (e.g. the one gd_compress_static returns)."""
    st = _Stats()
    _check(load_library().gd_get_stats(C.c_void_p(workspace_address), _stream_handle(stream), C.byref(st)), "gd_get_stats")
    return {name: getattr(st, name) for name, _ in _Stats._fields_}


def gd_selftest_bounded_wait(workspace: torch.Tensor, spin_limit: int = 2000, stream=None) -> None:
    _check(load_library().gd_selftest_bounded_wait(workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                                   spin_limit, _stream_handle(stream)), "gd_selftest_bounded_wait")


def gd_sampled_capacity(layer_off: Sequence[int], scope_mode: int, drop_ppm: int) -> int:
    out = C.c_uint64(0)
    arr = _u64_array(layer_off)
    _check(load_library().gd_sampled_capacity(arr, len(layer_off) - 1, scope_mode, drop_ppm, C.byref(out)),
           "gd_sampled_capacity")
    return out.value
