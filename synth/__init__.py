"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU oracle's callers.

The generator is a small C library (``synth.c``) built in-tree with gcc.  A value depends only on
``(seed, tensor_id, logical dense linear index)``; see the header of ``synth.c`` for the recipe.
This module contains no index-map arithmetic and imports neither the oracle nor the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "synth.c")
_LIB = os.path.join(_HERE, "libsynth.so")

UNIFORM = 0
NORMAL = 1


def build(force: bool = False) -> str:
    """Compile ``synth.c`` into ``libsynth.so`` next to it (no-op when up to date)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u64, dbl, cint, vp = ctypes.c_uint64, ctypes.c_double, ctypes.c_int, ctypes.c_void_p
        lib.synth_fill_linear.argtypes = [u64, u64, cint, dbl, cint, u64, u64, vp]
        lib.synth_fill_linear.restype = None
        lib.synth_fill_symmetric_row.argtypes = [u64, u64, cint, dbl, cint, u64, u64, vp]
        lib.synth_fill_symmetric_row.restype = None
        lib.synth_stream_upper_triangle.argtypes = [u64, u64, cint, dbl, cint, u64, vp]
        lib.synth_stream_upper_triangle.restype = u64
        lib.synth_stream_upper_half_cube.argtypes = [u64, u64, cint, dbl, u64, u64, u64, vp]
        lib.synth_stream_upper_half_cube.restype = u64
        lib.synth_stream_band_rows.argtypes = [u64, u64, cint, dbl, u64, u64, vp]
        lib.synth_stream_band_rows.restype = u64
        lib.synth_stream_tetrahedron.argtypes = [u64, u64, cint, dbl, cint, u64, vp]
        lib.synth_stream_tetrahedron.restype = u64
        lib.synth_stream_band_diagonals.argtypes = [u64, u64, cint, dbl, u64, u64, ctypes.c_uint32, vp]
        lib.synth_stream_band_diagonals.restype = u64
        _lib = lib
    return _lib


def _out(n: int, bf16: bool, out):
    """Return (array, pointer); bf16 values are carried as uint16 bit patterns."""
    dt = np.uint16 if bf16 else np.float32
    if out is None:
        out = np.empty(int(n), dtype=dt)
    else:
        assert out.dtype == dt and out.size >= n and out.flags["C_CONTIGUOUS"]
    return out, out.ctypes.data


def dense(seed, tensor_id, shape, dist=UNIFORM, scale=1.0, bf16=False, out=None):
    """Whole dense tensor of ``shape`` in row-major order."""
    n = int(np.prod(shape))
    arr, ptr = _out(n, bf16, out)
    _load().synth_fill_linear(seed, tensor_id, dist, scale, int(bf16), 0, n, ptr)
    return arr[:n].reshape(shape)


def linear_slice(seed, tensor_id, first, n, dist=UNIFORM, scale=1.0, bf16=False, out=None):
    """Values of dense linear indices ``[first, first + n)``."""
    arr, ptr = _out(n, bf16, out)
    _load().synth_fill_linear(seed, tensor_id, dist, scale, int(bf16), int(first), int(n), ptr)
    return arr[:n]


def symmetric_row(seed, tensor_id, N, i, dist=UNIFORM, scale=1.0, out=None):
    """Row ``i`` of the full symmetric matrix whose upper triangle is tensor ``tensor_id``."""
    arr, ptr = _out(N, False, out)
    _load().synth_fill_symmetric_row(seed, tensor_id, dist, scale, 0, int(N), int(i), ptr)
    return arr[:N]


def upper_triangle_stream(seed, tensor_id, N, dist=UNIFORM, scale=1.0, bf16=False, out=None):
    """Values of ``{(i, j): 0 <= i <= j < N}`` in (i, j) order; ``out`` may be a larger buffer."""
    n = _load().synth_stream_upper_triangle(seed, tensor_id, dist, scale, int(bf16), int(N), None)
    arr, ptr = _out(n, bf16, out)
    got = _load().synth_stream_upper_triangle(seed, tensor_id, dist, scale, int(bf16), int(N), ptr)
    assert got == n
    return arr[:n]


def upper_half_cube_stream(seed, tensor_id, M, N, Q, dist=UNIFORM, scale=1.0, out=None):
    """Values of ``{(i, j, l): 0 <= i < M, i <= j < N, 0 <= l < Q}`` in (i, j, l) order."""
    cnt = _load().synth_stream_upper_half_cube(seed, tensor_id, dist, scale, int(M), int(N), int(Q), None)
    arr, ptr = _out(cnt, False, out)
    got = _load().synth_stream_upper_half_cube(seed, tensor_id, dist, scale, int(M), int(N), int(Q), ptr)
    assert got == cnt
    return arr[:cnt]


def band_rows_stream(seed, tensor_id, N, w, dist=UNIFORM, scale=1.0, out=None):
    """Values of ``{(i, j): |i - j| <= w}`` row after row (j ascending), without padding."""
    cnt = _load().synth_stream_band_rows(seed, tensor_id, dist, scale, int(N), int(w), None)
    arr, ptr = _out(cnt, False, out)
    got = _load().synth_stream_band_rows(seed, tensor_id, dist, scale, int(N), int(w), ptr)
    assert got == cnt
    return arr[:cnt]


def tetrahedron_stream(seed, tensor_id, n, dist=UNIFORM, scale=1.0, out=None):
    """Values of ``{(i, j, k): 0 <= i <= j <= k < n}`` in (i, j, k) order."""
    n = int(n)
    cnt = _load().synth_stream_tetrahedron(seed, tensor_id, dist, scale, 0, n, None)
    arr, ptr = _out(cnt, False, out)
    got = _load().synth_stream_tetrahedron(seed, tensor_id, dist, scale, 0, n, ptr)
    assert got == cnt
    return arr[:cnt]


def band_diagonals_stream(seed, tensor_id, N, w, dist=UNIFORM, scale=1.0, pad_bits=0, out=None):
    """``2w+1`` diagonals of ``N`` slots each (diagonal ``d = j - i + w`` outer, row ``i`` inner)."""
    cnt = (2 * int(w) + 1) * int(N)
    arr, ptr = _out(cnt, False, out)
    got = _load().synth_stream_band_diagonals(seed, tensor_id, dist, scale, int(N), int(w),
                                              int(pad_bits), ptr)
    assert got == cnt
    return arr[:cnt].reshape(2 * int(w) + 1, int(N))
