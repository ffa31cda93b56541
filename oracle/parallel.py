"""Loader for the all-cores restatement of the oracle (oracle/graddrop_oracle_par.cpp).

TEST INFRASTRUCTURE ONLY, like the rest of this package: imported by the tests and by the
benchmark's cpu-baseline leg.  Builds the shared object with g++ -fopenmp next to its source on
first use (or through build()), and wraps its two calls with numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
SOURCE = os.path.join(_HERE, "graddrop_oracle_par.cpp")
LIBRARY = os.path.join(_HERE, "libgraddrop_oracle_par.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(LIBRARY) or os.path.getmtime(LIBRARY) < os.path.getmtime(SOURCE):
        tmp = LIBRARY + f".{os.getpid()}.tmp"
        subprocess.run(["g++", "-O2", "-fopenmp", "-shared", "-fPIC", SOURCE, "-o", tmp], check=True)
        os.replace(tmp, LIBRARY)
    return LIBRARY


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u64p, u32p, f32p = (ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_uint32),
                            ctypes.POINTER(ctypes.c_float))
        lib.oracle_par_threads.restype = ctypes.c_int
        lib.oracle_par_compress.restype = ctypes.c_int
        lib.oracle_par_compress.argtypes = [f32p, f32p, f32p, ctypes.c_uint64, u64p, ctypes.c_uint32, u64p,
                                            ctypes.c_uint32, ctypes.c_uint32, ctypes.c_int, ctypes.c_int,
                                            u32p, f32p, u32p, u32p, f32p]
        lib.oracle_par_apply.restype = ctypes.c_int
        lib.oracle_par_apply.argtypes = [f32p, u32p, f32p, ctypes.c_uint64, ctypes.c_float, ctypes.c_int, f32p,
                                         u64p, ctypes.c_uint32]
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().oracle_par_threads())


def set_threads(count: int = 0) -> int:
    """Use `count` threads from now on (0: every core this process may run on); returns the count in use."""
    _load().oracle_par_set_threads(int(count))
    return threads()


def _ptr(a, ty):
    return a.ctypes.data_as(ctypes.POINTER(ty))


def compress(grad, residual, layer_off, shard_off, drop_ppm, scope_mode=0, value_mode=0):
    """Same contract as graddrop_oracle.compress for value modes 0 (fp32) and 1 (two means per layer)."""
    lib = _load()
    g = np.ascontiguousarray(grad, dtype=np.float32)
    r = np.ascontiguousarray(residual, dtype=np.float32)
    n = g.shape[0]
    lo = np.asarray([int(x) for x in layer_off], dtype=np.uint64)
    so = np.asarray([int(x) for x in shard_off], dtype=np.uint64)
    n_layers, n_shards = lo.shape[0] - 1, so.shape[0] - 1
    scopes = [(0, n)] if scope_mode == 0 else [(int(lo[i]), int(lo[i + 1])) for i in range(n_layers)]
    k_total = sum((b - a) - ((b - a) * int(drop_ppm)) // 1_000_000 for a, b in scopes)
    out = {
        "idx": np.empty(k_total, dtype=np.uint32),
        "val": np.empty(k_total, dtype=np.float32),
        "residual": np.empty(n, dtype=np.float32),
        "tau": np.empty(len(scopes), dtype=np.uint32),
        "shard_cnt_off": np.empty(n_shards + 1, dtype=np.uint32),
        "means": np.zeros((n_layers, 2), dtype=np.float32),
    }
    rc = lib.oracle_par_compress(_ptr(g, ctypes.c_float), _ptr(r, ctypes.c_float),
                                 _ptr(out["residual"], ctypes.c_float), n, _ptr(lo, ctypes.c_uint64), n_layers,
                                 _ptr(so, ctypes.c_uint64), n_shards, int(drop_ppm), int(scope_mode), int(value_mode),
                                 _ptr(out["idx"], ctypes.c_uint32), _ptr(out["val"], ctypes.c_float),
                                 _ptr(out["shard_cnt_off"], ctypes.c_uint32), _ptr(out["tau"], ctypes.c_uint32),
                                 _ptr(out["means"], ctypes.c_float))
    if rc != 0:
        raise ValueError("oracle_par_compress rejected its arguments")
    return out


def apply(params, push, alpha=1.0, value_mode=0, layer_off=(0,)):
    """p[idx] += alpha * value over the flat parameter vector, in place (fp32 fused multiply-add)."""
    lib = _load()
    assert params.dtype == np.float32 and params.flags["C_CONTIGUOUS"]
    lo = np.asarray([int(x) for x in layer_off], dtype=np.uint64)
    means = np.ascontiguousarray(push.get("means", np.zeros((1, 2), dtype=np.float32)), dtype=np.float32)
    lib.oracle_par_apply(_ptr(params, ctypes.c_float), _ptr(push["idx"], ctypes.c_uint32),
                         _ptr(push["val"], ctypes.c_float), push["idx"].shape[0], float(alpha), int(value_mode),
                         _ptr(means, ctypes.c_float), _ptr(lo, ctypes.c_uint64), max(lo.shape[0] - 1, 1))
    return params
