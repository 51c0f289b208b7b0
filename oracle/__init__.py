"""CPU oracle (test infrastructure only): ctypes wrapper over ``oracle.c``.

Only the tests, the smoke check and the benchmark's CPU-baseline leg use this package.  It shares
no code with the CUDA library and does not import it.  What each function computes, and the
passages of the paper it follows, are stated in the header of ``oracle.c``.

A descriptor is any object with ``dims``, ``params``, ``rows``, ``is_eq`` and ``mirror`` attributes
(see ``synth.structures``).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Compile ``oracle.c`` into ``liboracle.so`` next to it (no-op when up to date)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


class _Desc(ctypes.Structure):
    _fields_ = [
        ("rank", ctypes.c_int32),
        ("nparams", ctypes.c_int32),
        ("nrows", ctypes.c_int32),
        ("dims", ctypes.c_void_p),
        ("rows", ctypes.c_void_p),
        ("is_eq", ctypes.c_void_p),
        ("params", ctypes.c_void_p),
    ]


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        P, vp, i64 = ctypes.POINTER(_Desc), ctypes.c_void_p, ctypes.c_int64
        lib.orc_count.argtypes = [P]
        lib.orc_count.restype = i64
        lib.orc_rank_table.argtypes = [P, vp]
        lib.orc_unrank_table.argtypes = [P, vp]
        lib.orc_rank_point.argtypes = [P, vp]
        lib.orc_rank_point.restype = i64
        lib.orc_pack.argtypes = [P, i64, vp, vp]
        lib.orc_unpack.argtypes = [P, vp, i64, vp, vp]
        lib.orc_band_pack.argtypes = [i64, i64, vp, vp]
        lib.orc_band_unpack.argtypes = [i64, i64, vp, vp]
        lib.orc_band_slot_table.argtypes = [i64, i64, vp]
        lib.orc_matvec.argtypes = [P, i64, vp, vp, vp, vp, vp]
        lib.orc_symv.argtypes = [i64, vp, vp, vp, vp]
        lib.orc_matmat.argtypes = [P, ctypes.c_int, i64, vp, vp, vp, i64, vp, vp]
        lib.orc_mttkrp.argtypes = [P, i64, vp, vp, vp, vp, i64, vp, vp]
        lib.orc_ttm.argtypes = [P, i64, vp, vp, vp, i64, vp, vp]
        lib.orc_moment2.argtypes = [P, ctypes.c_int, i64, vp, vp, i64, vp, vp]
        lib.orc_moment3.argtypes = [P, ctypes.c_int, i64, vp, vp, i64, vp, vp]
        lib.orc_hadamard.argtypes = [P, vp, vp, vp, vp]
        lib.orc_num_threads.restype = ctypes.c_int
        ci = ctypes.c_int
        lib.orc_clip_matvec_upper.argtypes = [i64, vp, vp, vp, ci]
        lib.orc_clip_symv.argtypes = [i64, vp, vp, vp, ci]
        lib.orc_clip_band_matmat.argtypes = [i64, i64, vp, vp, i64, vp, ci]
        lib.orc_clip_mttkrp_tetra.argtypes = [i64, vp, vp, vp, i64, vp, ci]
        lib.orc_clip_matmat_upper_bf16.argtypes = [i64, i64, vp, vp, vp, i64, vp, ci]
        for name in ("orc_clip_matvec_upper", "orc_clip_symv", "orc_clip_band_matmat", "orc_clip_mttkrp_tetra",
                     "orc_clip_matmat_upper_bf16"):
            getattr(lib, name).restype = None
        for name in ("orc_rank_table", "orc_unrank_table", "orc_pack", "orc_unpack", "orc_band_pack",
                     "orc_band_unpack", "orc_band_slot_table", "orc_matvec", "orc_symv",
                     "orc_matmat", "orc_mttkrp", "orc_ttm", "orc_moment2", "orc_moment3", "orc_hadamard"):
            getattr(lib, name).restype = None
        _lib = lib
    return _lib


class _Held:
    """A C descriptor plus the arrays its pointers refer to."""

    def __init__(self, desc):
        self.dims = np.ascontiguousarray(desc.dims, dtype=np.int64)
        self.params = np.ascontiguousarray(desc.params, dtype=np.int64)
        self.rows = np.ascontiguousarray(desc.rows, dtype=np.int64)
        self.is_eq = np.ascontiguousarray(desc.is_eq, dtype=np.uint8)
        rank, nparams = len(self.dims), len(self.params)
        assert self.rows.ndim == 2 and self.rows.shape[1] == rank + nparams + 1
        self.c = _Desc(rank, nparams, self.rows.shape[0], self.dims.ctypes.data,
                       self.rows.ctypes.data, self.is_eq.ctypes.data, self.params.ctypes.data)
        self.rank = rank

    @property
    def ref(self):
        return ctypes.byref(self.c)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def num_threads() -> int:
    return int(_load().orc_num_threads())


# ---- index maps -------------------------------------------------------------------------------

def count(desc) -> int:
    h = _Held(desc)
    return int(_load().orc_count(h.ref))


def rank_table(desc) -> np.ndarray:
    """int64 array of shape ``dims``: packed position of every point, -1 outside the set."""
    h = _Held(desc)
    table = np.empty(tuple(int(v) for v in h.dims), dtype=np.int64)
    _load().orc_rank_table(h.ref, table.ctypes.data)
    return table


def unrank_table(desc) -> np.ndarray:
    """int32 array ``[count, rank]``: the point stored at every packed position."""
    h = _Held(desc)
    n = int(_load().orc_count(h.ref))
    out = np.empty((n, h.rank), dtype=np.int32)
    _load().orc_unrank_table(h.ref, out.ctypes.data)
    return out


def rank_point(desc, point) -> int:
    h = _Held(desc)
    p = np.ascontiguousarray(point, dtype=np.int64)
    return int(_load().orc_rank_point(h.ref, p.ctypes.data))


# ---- compress / decompress --------------------------------------------------------------------

def pack(desc, dense: np.ndarray) -> np.ndarray:
    h = _Held(desc)
    dense = np.ascontiguousarray(dense)
    assert dense.shape == tuple(int(v) for v in h.dims)
    out = np.empty(int(_load().orc_count(h.ref)), dtype=dense.dtype)
    _load().orc_pack(h.ref, dense.dtype.itemsize, dense.ctypes.data, out.ctypes.data)
    return out


def unpack(desc, packed: np.ndarray) -> np.ndarray:
    h = _Held(desc)
    packed = np.ascontiguousarray(packed)
    out = np.empty(tuple(int(v) for v in h.dims), dtype=packed.dtype)
    mirror = None
    mptr = None
    if getattr(desc, "mirror", None) is not None:
        mirror = np.ascontiguousarray(desc.mirror, dtype=np.int32)
        mptr = mirror.ctypes.data
    _load().orc_unpack(h.ref, mptr, packed.dtype.itemsize, packed.ctypes.data, out.ctypes.data)
    return out


def band_pack(N: int, w: int, dense: np.ndarray) -> np.ndarray:
    dense = _f32(dense)
    out = np.empty((2 * w + 1, N), dtype=np.float32)
    _load().orc_band_pack(N, w, dense.ctypes.data, out.ctypes.data)
    return out


def band_unpack(N: int, w: int, packed: np.ndarray) -> np.ndarray:
    packed = _f32(packed)
    out = np.empty((N, N), dtype=np.float32)
    _load().orc_band_unpack(N, w, packed.ctypes.data, out.ctypes.data)
    return out


def band_slot_table(N: int, w: int) -> np.ndarray:
    out = np.empty((N, N), dtype=np.int64)
    _load().orc_band_slot_table(N, w, out.ctypes.data)
    return out


# ---- contractions (fp64 accumulation) ------------------------------------------------------------
# Each returns (sum, sum_of_absolute_products) as float64 arrays.

def _sel(sel, n):
    if sel is None:
        sel = np.arange(n, dtype=np.int64)
    return np.ascontiguousarray(sel, dtype=np.int64)


def matvec(desc, A_rows, x, sel=None):
    """``y[i] = sum_j [(i,j) in set] A[i][j] x[j]``; ``A_rows[s]`` is dense row ``sel[s]``."""
    h = _Held(desc)
    sel = _sel(sel, int(h.dims[0]))
    A_rows, x = _f32(A_rows), _f32(x)
    assert A_rows.shape == (len(sel), int(h.dims[1])) and x.shape == (int(h.dims[1]),)
    out, out_abs = np.empty(len(sel)), np.empty(len(sel))
    _load().orc_matvec(h.ref, len(sel), sel.ctypes.data, A_rows.ctypes.data, x.ctypes.data,
                       out.ctypes.data, out_abs.ctypes.data)
    return out, out_abs


def symv(U, x):
    """``y = Sfull x`` with ``Sfull[i][j] = U[min(i,j)][max(i,j)]``; U dense N x N."""
    U, x = _f32(U), _f32(x)
    N = U.shape[0]
    assert U.shape == (N, N) and x.shape == (N,)
    out, out_abs = np.empty(N), np.empty(N)
    _load().orc_symv(N, U.ctypes.data, x.ctypes.data, out.ctypes.data, out_abs.ctypes.data)
    return out, out_abs


def matmat(desc, A_rows, B, sel=None):
    """``C[i][c] = sum_j [(i,j) in set] A[i][j] B[j][c]``.  fp32 arrays, or uint16 arrays holding
    bf16 bit patterns (both operands then)."""
    h = _Held(desc)
    sel = _sel(sel, int(h.dims[0]))
    is_bf16 = A_rows.dtype == np.uint16
    if is_bf16:
        assert B.dtype == np.uint16
        A_rows, B = np.ascontiguousarray(A_rows), np.ascontiguousarray(B)
    else:
        A_rows, B = _f32(A_rows), _f32(B)
    N = int(h.dims[1])
    assert A_rows.shape == (len(sel), N) and B.shape[0] == N
    ncols = B.shape[1]
    out, out_abs = np.empty((len(sel), ncols)), np.empty((len(sel), ncols))
    _load().orc_matmat(h.ref, int(is_bf16), len(sel), sel.ctypes.data, A_rows.ctypes.data,
                       B.ctypes.data, ncols, out.ctypes.data, out_abs.ctypes.data)
    return out, out_abs


def mttkrp(desc, T_slabs, B, C, sel=None):
    """``M[i][r] = sum_{j,k} [(i,j,k) in set] T[i][j][k] B[j][r] C[k][r]``; ``T_slabs[s]`` is the
    dense slab ``sel[s]``."""
    h = _Held(desc)
    sel = _sel(sel, int(h.dims[0]))
    T_slabs, B, C = _f32(T_slabs), _f32(B), _f32(C)
    nj, nk = int(h.dims[1]), int(h.dims[2])
    assert T_slabs.shape == (len(sel), nj, nk)
    R = B.shape[1]
    assert B.shape == (nj, R) and C.shape == (nk, R)
    out, out_abs = np.empty((len(sel), R)), np.empty((len(sel), R))
    _load().orc_mttkrp(h.ref, len(sel), sel.ctypes.data, T_slabs.ctypes.data, B.ctypes.data,
                       C.ctypes.data, R, out.ctypes.data, out_abs.ctypes.data)
    return out, out_abs


def ttm(desc, B_slabs, C, sel=None):
    """``A[i][j][k] = sum_l [(i,j,l) in set] B[i][j][l] C[k][l]``; ``B_slabs[s]`` is the dense
    ``N x Q`` slab ``sel[s]`` of B, C is ``K x Q``.  Returns ``[len(sel), N, K]`` arrays."""
    h = _Held(desc)
    sel = _sel(sel, int(h.dims[0]))
    B_slabs, C = _f32(B_slabs), _f32(C)
    N, Q = int(h.dims[1]), int(h.dims[2])
    assert B_slabs.shape == (len(sel), N, Q) and C.shape[1] == Q
    K = C.shape[0]
    out, out_abs = np.empty((len(sel), N, K)), np.empty((len(sel), N, K))
    _load().orc_ttm(h.ref, len(sel), sel.ctypes.data, B_slabs.ctypes.data, C.ctypes.data, K,
                    out.ctypes.data, out_abs.ctypes.data)
    return out, out_abs


def moment2(desc, B, sel=None):
    """``A2[i1][i2] = sum_x [(i1,i2) in set] B[x][i1] B[x][i2]`` for the rows ``i1`` in ``sel``; B is
    ``M x n`` (fp32, or uint16 holding bf16 bit patterns).  Returns ``[len(sel), n]`` arrays (dense
    rows, zero outside the set)."""
    h = _Held(desc)
    sel = _sel(sel, int(h.dims[0]))
    is_bf16 = B.dtype == np.uint16
    B = np.ascontiguousarray(B) if is_bf16 else _f32(B)
    n = int(h.dims[1])
    assert B.ndim == 2 and B.shape[1] == n and int(h.dims[0]) == n
    out, out_abs = np.empty((len(sel), n)), np.empty((len(sel), n))
    _load().orc_moment2(h.ref, int(is_bf16), len(sel), sel.ctypes.data, B.ctypes.data, B.shape[0],
                        out.ctypes.data, out_abs.ctypes.data)
    return out, out_abs


def moment3(desc, B, sel=None):
    """``A3[i1][i2][i3] = sum_x [(i1,i2,i3) in set] B[x][i1] B[x][i2] B[x][i3]`` for the slabs ``i1`` in
    ``sel``; B is ``M x n`` (fp32, or uint16 holding bf16 bit patterns).  Returns ``[len(sel), n, n]``
    arrays (dense slabs, zero outside the set)."""
    h = _Held(desc)
    sel = _sel(sel, int(h.dims[0]))
    is_bf16 = B.dtype == np.uint16
    B = np.ascontiguousarray(B) if is_bf16 else _f32(B)
    n = int(h.dims[1])
    assert B.ndim == 2 and B.shape[1] == n and int(h.dims[0]) == n and int(h.dims[2]) == n
    out, out_abs = np.empty((len(sel), n, n)), np.empty((len(sel), n, n))
    _load().orc_moment3(h.ref, int(is_bf16), len(sel), sel.ctypes.data, B.ctypes.data, B.shape[0],
                        out.ctypes.data, out_abs.ctypes.data)
    return out, out_abs


def hadamard(desc, B, C):
    """``A[idx] = [idx in set] B[idx] C[idx]`` over the whole box (dense fp32 arrays in, dense fp64
    arrays out, zero outside the set)."""
    h = _Held(desc)
    B, C = _f32(B), _f32(C)
    shape = tuple(int(v) for v in h.dims)
    assert B.shape == shape and C.shape == shape
    out, out_abs = np.empty(shape), np.empty(shape)
    _load().orc_hadamard(h.ref, B.ctypes.data, C.ctypes.data, out.ctypes.data, out_abs.ctypes.data)
    return out, out_abs


# ---- timed variants: loops clipped to the domain, packed operand (the CPU baseline) --------------
# Same products as the masked forms; see the header of ``oracle.c``.  ``threads`` = OpenMP threads.

def _threads(threads):
    return int(threads) if threads else num_threads()


def clip_matvec_upper(N, packed, x, threads=None):
    packed, x = _f32(packed), _f32(x)
    assert packed.size >= N * (N + 1) // 2 and x.shape == (N,)
    y = np.empty(N)
    _load().orc_clip_matvec_upper(N, packed.ctypes.data, x.ctypes.data, y.ctypes.data, _threads(threads))
    return y


def clip_symv(N, packed, x, threads=None):
    packed, x = _f32(packed), _f32(x)
    assert packed.size >= N * (N + 1) // 2 and x.shape == (N,)
    y = np.empty(N)
    _load().orc_clip_symv(N, packed.ctypes.data, x.ctypes.data, y.ctypes.data, _threads(threads))
    return y


def clip_band_matmat(N, w, diags, B, threads=None):
    diags, B = _f32(diags), _f32(B)
    assert diags.size == (2 * w + 1) * N and B.shape[0] == N
    out = np.empty((N, B.shape[1]))
    _load().orc_clip_band_matmat(N, w, diags.ctypes.data, B.ctypes.data, B.shape[1], out.ctypes.data,
                                 _threads(threads))
    return out


def clip_mttkrp_tetra(n, packed, B, C, threads=None):
    packed, B, C = _f32(packed), _f32(B), _f32(C)
    R = B.shape[1]
    assert packed.size >= n * (n + 1) * (n + 2) // 6 and B.shape == (n, R) and C.shape == (n, R)
    out = np.empty((n, R))
    _load().orc_clip_mttkrp_tetra(n, packed.ctypes.data, B.ctypes.data, C.ctypes.data, R, out.ctypes.data,
                                  _threads(threads))
    return out


def clip_matmat_upper_bf16(N, packed, B, sel=None, threads=None):
    sel = _sel(sel, N)
    packed, B = np.ascontiguousarray(packed), np.ascontiguousarray(B)
    assert packed.dtype == np.uint16 and B.dtype == np.uint16 and B.shape[0] == N
    out = np.empty((len(sel), B.shape[1]))
    _load().orc_clip_matmat_upper_bf16(N, len(sel), sel.ctypes.data, packed.ctypes.data, B.ctypes.data,
                                       B.shape[1], out.ctypes.data, _threads(threads))
    return out
