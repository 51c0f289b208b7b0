"""Thin ctypes binding over ``libdastac.so``: argument marshalling only.

Function names follow ``include/dastac.h``.  torch tensors supply device memory (or pinned host
memory) and the current CUDA stream; every step of the computation runs in the library's kernels.
There is no fallback: if the shared library is missing or fails to load, importing this module
raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdastac.so")

F32, BF16 = 0, 1
MEM_DEVICE, MEM_HOST = 0, 1
(KIND_EMPTY, KIND_DENSE, KIND_UPPER, KIND_LOWER, KIND_BAND_DIAGONALS, KIND_TETRAHEDRON, KIND_BAND_EXACT,
 KIND_UPPER_SHIFTED, KIND_BAND_OFFSETS, KIND_PLANE, KIND_GENERIC) = range(11)
LAYOUT_LEXICOGRAPHIC, LAYOUT_PADDED_DIAGONALS = 0, 1

EXPORTS = [
    "dastac_structure_create", "dastac_structure_destroy", "dastac_structure_count",
    "dastac_structure_kind", "dastac_rank", "dastac_unrank", "dastac_rank_batch",
    "dastac_unrank_batch", "dastac_pack", "dastac_unpack", "dastac_contract_workspace",
    "dastac_contract", "dastac_status_string", "dastac_launch_count", "dastac_trimm_bf16_noalloc",
    "dastac_device_error", "dastac_selftest_wait_expiry", "dastac_piecewise_fuse",
    "dastac_rule_create", "dastac_rule_destroy", "dastac_rule_size", "dastac_rule_summand", "dastac_rule_pack",
    "dastac_rule_contract_workspace", "dastac_rule_contract", "dastac_mttkrp_split_tf32",
    "dastac_bandmm_split_tf32", "dastac_ttm_split_tf32",
]
NOALLOC_MAX_N = 2048


class DastacError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class _StructureDesc(ctypes.Structure):
    _fields_ = [("rank", ctypes.c_int32), ("nparams", ctypes.c_int32), ("nrows", ctypes.c_int32),
                ("dims", ctypes.c_void_p), ("rows", ctypes.c_void_p), ("is_eq", ctypes.c_void_p),
                ("params", ctypes.c_void_p), ("mirror", ctypes.c_void_p), ("layout", ctypes.c_int32)]


class _Operand(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("dtype", ctypes.c_int32), ("space", ctypes.c_int32),
                ("structure", ctypes.c_void_p), ("rank", ctypes.c_int32), ("batch", ctypes.c_int32),
                ("batch_stride", ctypes.c_int64), ("dims", ctypes.c_int64 * 4),
                ("strides", ctypes.c_int64 * 4)]


if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2407_13726_b200.build` "
        "(there is no non-CUDA fallback)")
_lib = ctypes.CDLL(LIB_PATH)

_vp, _i64, _i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32
_lib.dastac_structure_create.argtypes = [ctypes.POINTER(_StructureDesc), ctypes.POINTER(_vp)]
_lib.dastac_structure_destroy.argtypes = [_vp]
_lib.dastac_structure_destroy.restype = None
_lib.dastac_structure_count.argtypes = [_vp, ctypes.POINTER(_i64), ctypes.POINTER(_i64)]
_lib.dastac_structure_kind.argtypes = [_vp, ctypes.POINTER(_i32), ctypes.POINTER(_i32)]
_lib.dastac_rank.argtypes = [_vp, ctypes.POINTER(_i32), ctypes.POINTER(_i64)]
_lib.dastac_unrank.argtypes = [_vp, _i64, ctypes.POINTER(_i32)]
_lib.dastac_rank_batch.argtypes = [_vp, _vp, _i64, _vp, _vp]
_lib.dastac_unrank_batch.argtypes = [_vp, _vp, _i64, _vp, _vp]
_lib.dastac_pack.argtypes = [_vp, _i32, _vp, ctypes.POINTER(_i64), _vp, _vp]
_lib.dastac_unpack.argtypes = [_vp, _i32, _vp, _vp, ctypes.POINTER(_i64), _vp]
_lib.dastac_contract_workspace.argtypes = [ctypes.c_char_p, ctypes.POINTER(_Operand), _i32,
                                           ctypes.POINTER(_Operand), ctypes.POINTER(ctypes.c_size_t)]
_lib.dastac_contract.argtypes = [ctypes.c_char_p, ctypes.POINTER(_Operand), _i32,
                                 ctypes.POINTER(_Operand), _i32, _vp, ctypes.c_size_t, _vp, _vp]
_lib.dastac_status_string.argtypes = [ctypes.c_int]
_lib.dastac_status_string.restype = ctypes.c_char_p
_lib.dastac_trimm_bf16_noalloc.argtypes = [_vp, _vp, _vp, _i64, _i64, _vp, _i64, _i32, _vp, _vp]
_lib.dastac_launch_count.argtypes = []
_lib.dastac_launch_count.restype = _i64
_lib.dastac_device_error.argtypes = [ctypes.POINTER(_i32), _i32, _vp]
_lib.dastac_selftest_wait_expiry.argtypes = [_i64, _vp]
_lib.dastac_piecewise_fuse.argtypes = [_vp, _i32, _vp]
_lib.dastac_mttkrp_split_tf32.argtypes = [_vp, _vp, _vp, _i64, _vp, _i64, _vp, _i64, _i64, _i32, _vp, _vp]
_lib.dastac_bandmm_split_tf32.argtypes = [_vp, _vp, _vp, _i64, _vp, _i64, _i64, _i32, _vp, _vp]
_lib.dastac_ttm_split_tf32.argtypes = [_vp, _vp, _vp, _i64, _i64, _vp, _i32, _vp, _vp]
_lib.dastac_rule_create.argtypes = [_vp, _i32, ctypes.POINTER(_vp)]
_lib.dastac_rule_destroy.argtypes = [_vp]
_lib.dastac_rule_destroy.restype = None
_lib.dastac_rule_size.argtypes = [_vp, ctypes.POINTER(_i32), ctypes.POINTER(_i32)]
_lib.dastac_rule_summand.argtypes = [_vp, _i32, ctypes.POINTER(_vp), ctypes.POINTER(_i32)]
_lib.dastac_rule_pack.argtypes = [_vp, _i32, _vp, _vp, _vp, _vp]
_lib.dastac_rule_contract_workspace.argtypes = [_vp, _vp, _i32, _vp, _i32, _vp, ctypes.POINTER(ctypes.c_size_t)]
_lib.dastac_rule_contract.argtypes = [_vp, _vp, _i32, _vp, _vp, _vp, _i32, _vp, _i32, _vp, ctypes.c_size_t, _vp, _vp]


def status_string(status: int) -> str:
    return _lib.dastac_status_string(int(status)).decode()


def launch_count() -> int:
    return int(_lib.dastac_launch_count())


def device_error(clear: bool = True):
    """``(status, word)`` of the current device's error word after everything enqueued on the current
    stream (synchronises it): status 0, or 9 (TIMEOUT) with the recorded code."""
    word = _i32(0)
    st = _lib.dastac_device_error(ctypes.byref(word), int(bool(clear)), _stream())
    return int(st), int(word.value)


def selftest_wait_expiry(budget_cycles: int) -> None:
    _check(_lib.dastac_selftest_wait_expiry(int(budget_cycles), _stream()), "dastac_selftest_wait_expiry")


def _check(status: int, where: str):
    if status != 0:
        raise DastacError(status, where)


def _stream() -> Optional[int]:
    return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else None


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _marshal_desc(desc):
    """The C descriptor of ``desc`` plus the arrays its pointers refer to (keep them alive)."""
    import numpy as np

    dims = np.ascontiguousarray(desc.dims, dtype=np.int64)
    params = np.ascontiguousarray(desc.params, dtype=np.int64)
    rows = np.ascontiguousarray(desc.rows, dtype=np.int64)
    is_eq = np.ascontiguousarray(desc.is_eq, dtype=np.uint8)
    mirror = getattr(desc, "mirror", None)
    mirror_arr = None if mirror is None else np.ascontiguousarray(mirror, dtype=np.int32)
    layout = LAYOUT_PADDED_DIAGONALS if getattr(desc, "padded_diagonals", False) else LAYOUT_LEXICOGRAPHIC
    nrows = rows.shape[0] if rows.ndim == 2 else 0
    c = _StructureDesc(len(dims), len(params), nrows, dims.ctypes.data,
                       rows.ctypes.data if nrows else None, is_eq.ctypes.data if nrows else None,
                       params.ctypes.data if len(params) else None,
                       None if mirror_arr is None else mirror_arr.ctypes.data, layout)
    return c, (dims, params, rows, is_eq, mirror_arr)


class _Poly(ctypes.Structure):
    _fields_ = [("nvars", ctypes.c_int32), ("nterms", ctypes.c_int32), ("exps", ctypes.c_void_p),
                ("num", ctypes.c_void_p), ("den", ctypes.c_int64)]


class _Piece(ctypes.Structure):
    _fields_ = [("domain", _StructureDesc), ("poly", _Poly)]


def piecewise_fuse(pieces):
    """Algorithm 2 on ``[(descriptor, terms, den), ...]`` where ``terms`` is a list of
    ``(numerator, exponents)``: returns ``owner`` (see ``dastac_piecewise_fuse``)."""
    import numpy as np

    n = len(pieces)
    arr = (_Piece * max(n, 1))()
    keep = []
    for k, (desc, terms, den) in enumerate(pieces):
        c, held = _marshal_desc(desc)
        nv = len(desc.dims)
        exps = np.ascontiguousarray([list(e) for _, e in terms], dtype=np.int32).reshape(len(terms), nv)
        num = np.ascontiguousarray([v for v, _ in terms], dtype=np.int64)
        keep.append((held, exps, num))
        arr[k].domain = c
        arr[k].poly = _Poly(nv, len(terms), exps.ctypes.data if len(terms) else None,
                            num.ctypes.data if len(terms) else None, int(den))
    owner = (ctypes.c_int32 * max(n, 1))()
    _check(_lib.dastac_piecewise_fuse(arr, n, owner), "dastac_piecewise_fuse")
    return [int(owner[k]) for k in range(n)]


class Structure:
    """Owns a ``dastac_structure`` created from a descriptor (any object with ``dims``,
    ``params``, ``rows``, ``is_eq``, ``mirror`` and ``padded_diagonals`` attributes)."""

    def __init__(self, desc):
        c, keep = _marshal_desc(desc)
        dims = keep[0]
        handle = _vp()
        _check(_lib.dastac_structure_create(ctypes.byref(c), ctypes.byref(handle)),
               "dastac_structure_create")
        self._h = handle
        self.rank = len(dims)
        self.dims = [int(v) for v in dims]
        slots, nnz = _i64(), _i64()
        _check(_lib.dastac_structure_count(self._h, ctypes.byref(slots), ctypes.byref(nnz)),
               "dastac_structure_count")
        self.slots, self.nnz = int(slots.value), int(nnz.value)
        kind, sym = _i32(), _i32()
        _check(_lib.dastac_structure_kind(self._h, ctypes.byref(kind), ctypes.byref(sym)),
               "dastac_structure_kind")
        self.kind, self.symmetric = int(kind.value), bool(sym.value)

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h and _lib is not None:  # module globals are already cleared at interpreter shutdown
            _lib.dastac_structure_destroy(h)

    def capacity(self, dtype: torch.dtype) -> int:
        """Elements a packed buffer must hold: ``slots`` rounded up to 16 bytes."""
        per16 = 16 // torch.empty((), dtype=dtype).element_size()
        return (self.slots + per16 - 1) // per16 * per16

    def empty_packed(self, dtype=torch.float32, device="cuda", batch: int = 1) -> torch.Tensor:
        cap = self.capacity(dtype)
        shape = (cap,) if batch == 1 else (batch, cap)
        return torch.zeros(shape, dtype=dtype, device=device)


def structure_create(desc) -> Structure:
    return Structure(desc)


def structure_count(s: Structure):
    return s.slots, s.nnz


def rank(s: Structure, idx: Sequence[int]) -> int:
    arr = (_i32 * s.rank)(*[int(v) for v in idx])
    off = _i64()
    _check(_lib.dastac_rank(s._h, arr, ctypes.byref(off)), "dastac_rank")
    return int(off.value)


def unrank(s: Structure, off: int):
    arr = (_i32 * 3)()
    _check(_lib.dastac_unrank(s._h, int(off), arr), "dastac_unrank")
    return tuple(int(arr[k]) for k in range(s.rank))


def rank_batch(s: Structure, idx: torch.Tensor) -> torch.Tensor:
    assert idx.is_cuda and idx.dtype == torch.int32 and idx.is_contiguous() and idx.shape[-1] == s.rank
    n = idx.numel() // s.rank
    off = torch.empty(n, dtype=torch.int64, device=idx.device)
    _check(_lib.dastac_rank_batch(s._h, idx.data_ptr(), n, off.data_ptr(), _stream()),
           "dastac_rank_batch")
    return off


def unrank_batch(s: Structure, off: torch.Tensor) -> torch.Tensor:
    assert off.is_cuda and off.dtype == torch.int64 and off.is_contiguous()
    idx = torch.empty((off.numel(), s.rank), dtype=torch.int32, device=off.device)
    _check(_lib.dastac_unrank_batch(s._h, off.data_ptr(), off.numel(), idx.data_ptr(), _stream()),
           "dastac_unrank_batch")
    return idx


def pack(s: Structure, dense: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    assert dense.is_cuda and list(dense.shape) == s.dims
    if out is None:
        out = s.empty_packed(dense.dtype, dense.device)
    assert out.is_cuda and out.dtype == dense.dtype and out.numel() >= s.capacity(dense.dtype)
    strides = (_i64 * s.rank)(*dense.stride())
    _check(_lib.dastac_pack(s._h, _dtype_code(dense), dense.data_ptr(), strides, out.data_ptr(),
                            _stream()), "dastac_pack")
    return out


def unpack(s: Structure, packed: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    assert packed.is_cuda and packed.numel() >= s.capacity(packed.dtype)
    if out is None:
        out = torch.empty(s.dims, dtype=packed.dtype, device=packed.device)
    assert out.is_cuda and list(out.shape) == s.dims and out.dtype == packed.dtype
    strides = (_i64 * s.rank)(*out.stride())
    _check(_lib.dastac_unpack(s._h, _dtype_code(packed), packed.data_ptr(), out.data_ptr(), strides,
                              _stream()), "dastac_unpack")
    return out


def _operand(t: torch.Tensor, structure: Optional[Structure], batch: int) -> _Operand:
    op = _Operand()
    op.data = t.data_ptr()
    op.dtype = _dtype_code(t)
    op.space = MEM_DEVICE if t.is_cuda else MEM_HOST
    op.structure = structure._h if structure is not None else None
    op.batch = batch
    if structure is not None:
        op.rank = structure.rank
        for k, v in enumerate(structure.dims):
            op.dims[k] = v
        op.batch_stride = t.stride(0) if batch > 1 else 0
    else:
        shape, strides = list(t.shape), list(t.stride())
        if batch > 1:
            op.batch_stride = strides[0]
            shape, strides = shape[1:], strides[1:]
        op.rank = len(shape)
        for k in range(len(shape)):
            op.dims[k] = shape[k]
            op.strides[k] = strides[k]
    return op


def _operands(s, packed, dense_inputs, out, batch, out_structure=None):
    ins = (_Operand * (1 + len(dense_inputs)))()
    ins[0] = _operand(packed, s, batch)
    for k, t in enumerate(dense_inputs):
        ins[1 + k] = _operand(t, None, batch)
    o = _operand(out, out_structure, batch)
    return ins, o


def contract_workspace(expr: str, s: Structure, packed: torch.Tensor,
                       dense_inputs: Sequence[torch.Tensor], out: torch.Tensor, batch: int = 1,
                       out_structure: Optional[Structure] = None) -> int:
    ins, o = _operands(s, packed, dense_inputs, out, batch, out_structure)
    nbytes = ctypes.c_size_t()
    _check(_lib.dastac_contract_workspace(expr.encode(), ins, len(ins), ctypes.byref(o),
                                          ctypes.byref(nbytes)), "dastac_contract_workspace")
    return int(nbytes.value)


def contract(expr: str, s: Structure, packed: torch.Tensor, dense_inputs: Sequence[torch.Tensor],
             out: torch.Tensor, accumulate: bool = False, workspace: Optional[torch.Tensor] = None,
             err_word: Optional[torch.Tensor] = None, batch: int = 1,
             out_structure: Optional[Structure] = None) -> torch.Tensor:
    """Evaluate ``expr`` with ``packed`` (structure ``s``) as first operand.  Tensors may live on
    the device or in (pinned) host memory; host tensors are staged through ``workspace``.
    ``out_structure`` marks ``out`` as a packed buffer of that structure (rules with packed output).
    For the rule without a packed input (``"xi,xj->ij"``) pass ``s=None`` and the dense tensor itself
    as ``packed`` and again as the only entry of ``dense_inputs``."""
    ins, o = _operands(s, packed, dense_inputs, out, batch, out_structure)
    ws_ptr, ws_bytes = None, 0
    if workspace is not None:
        ws_ptr, ws_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
    _check(_lib.dastac_contract(expr.encode(), ins, len(ins), ctypes.byref(o), int(accumulate),
                                ws_ptr, ws_bytes,
                                None if err_word is None else err_word.data_ptr(), _stream()),
           "dastac_contract")
    return out


class _SummandView:
    """Counts and kind of a summand's structure (the structure itself belongs to the rule)."""

    def __init__(self, handle, dims):
        self._h = handle
        self.rank, self.dims = len(dims), list(dims)
        slots, nnz, kind, sym = _i64(), _i64(), _i32(), _i32()
        _check(_lib.dastac_structure_count(handle, ctypes.byref(slots), ctypes.byref(nnz)), "dastac_structure_count")
        _check(_lib.dastac_structure_kind(handle, ctypes.byref(kind), ctypes.byref(sym)), "dastac_structure_kind")
        self.slots, self.nnz, self.kind = int(slots.value), int(nnz.value), int(kind.value)

    capacity = Structure.capacity
    empty_packed = Structure.empty_packed


class Rule:
    """Owns a ``dastac_rule``: a structured operand given as a list of summand descriptors."""

    def __init__(self, descs):
        arr = (_StructureDesc * len(descs))()
        keep = []
        for k, d in enumerate(descs):
            arr[k], held = _marshal_desc(d)
            keep.append(held)
        handle = _vp()
        _check(_lib.dastac_rule_create(arr, len(descs), ctypes.byref(handle)), "dastac_rule_create")
        self._h = handle
        ns, nb = _i32(), _i32()
        _check(_lib.dastac_rule_size(handle, ctypes.byref(ns), ctypes.byref(nb)), "dastac_rule_size")
        self.n_summands, self.n_buffers = int(ns.value), int(nb.value)
        self.summands, self.buffer = [], []
        for k in range(self.n_summands):
            sh, b = _vp(), _i32()
            _check(_lib.dastac_rule_summand(handle, k, ctypes.byref(sh), ctypes.byref(b)), "dastac_rule_summand")
            self.summands.append(_SummandView(sh, descs[k].dims))
            self.buffer.append(int(b.value))

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h and _lib is not None:
            _lib.dastac_rule_destroy(h)

    def empty_buffers(self, dtype=torch.float32, device="cuda"):
        """One packed buffer per distinct region, sized for the first summand that uses it."""
        bufs = [None] * self.n_buffers
        for s, b in zip(self.summands, self.buffer):
            if bufs[b] is None:
                bufs[b] = s.empty_packed(dtype, device)
        return bufs

    def pack(self, dense: torch.Tensor, buffers=None):
        buffers = buffers if buffers is not None else self.empty_buffers(dense.dtype, dense.device)
        ptrs = (_vp * self.n_buffers)(*[t.data_ptr() for t in buffers])
        strides = (_i64 * dense.dim())(*dense.stride())
        _check(_lib.dastac_rule_pack(self._h, _dtype_code(dense), dense.data_ptr(), strides, ptrs, _stream()),
               "dastac_rule_pack")
        return buffers

    def _rest(self, dense_inputs, out, batch):
        rest = (_Operand * len(dense_inputs))()
        for k, t in enumerate(dense_inputs):
            rest[k] = _operand(t, None, batch)
        return rest, _operand(out, None, batch)

    def contract_workspace(self, expr, buffers, dense_inputs, out, batch: int = 1) -> int:
        rest, o = self._rest(dense_inputs, out, batch)
        nbytes = ctypes.c_size_t()
        _check(_lib.dastac_rule_contract_workspace(expr.encode(), self._h, _dtype_code(buffers[0]), rest, len(dense_inputs),
                                                   ctypes.byref(o), ctypes.byref(nbytes)), "dastac_rule_contract_workspace")
        return int(nbytes.value)

    def contract(self, expr, buffers, dense_inputs, out, accumulate=False, workspace=None, err_word=None, batch: int = 1):
        """``out = sum over the summands of contract(expr, summand, dense_inputs...)`` in one call."""
        rest, o = self._rest(dense_inputs, out, batch)
        ptrs = (_vp * self.n_buffers)(*[t.data_ptr() for t in buffers])
        ws_ptr, ws_bytes = None, 0
        if workspace is not None:
            ws_ptr, ws_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
        _check(_lib.dastac_rule_contract(expr.encode(), self._h, _dtype_code(buffers[0]), ptrs, None, rest, len(dense_inputs),
                                         ctypes.byref(o), int(accumulate), ws_ptr, ws_bytes,
                                         None if err_word is None else err_word.data_ptr(), _stream()),
               "dastac_rule_contract")
        return out


def mttkrp_split_tf32(s: Structure, packed: torch.Tensor, B: torch.Tensor, C: torch.Tensor, out: torch.Tensor,
                      accumulate: bool = False, err_word: Optional[torch.Tensor] = None) -> torch.Tensor:
    """The tetrahedral MTTKRP through the split-precision tensor-core entry point (see ``dastac.h``)."""
    assert packed.is_cuda and B.is_cuda and C.is_cuda and out.is_cuda
    assert packed.dtype == B.dtype == C.dtype == out.dtype == torch.float32
    assert B.dim() == 2 and C.dim() == 2 and out.dim() == 2 and B.shape[1] == C.shape[1] == out.shape[1]
    assert (B.shape[1] <= 1 or (B.stride(1) == 1 and C.stride(1) == 1 and out.stride(1) == 1))
    _check(_lib.dastac_mttkrp_split_tf32(s._h, packed.data_ptr(), B.data_ptr(), B.stride(0), C.data_ptr(), C.stride(0),
                                         out.data_ptr(), out.stride(0), B.shape[1], int(accumulate),
                                         None if err_word is None else err_word.data_ptr(), _stream()),
           "dastac_mttkrp_split_tf32")
    return out


def bandmm_split_tf32(s: Structure, packed: torch.Tensor, B: torch.Tensor, out: torch.Tensor,
                      accumulate: bool = False, err_word: Optional[torch.Tensor] = None) -> torch.Tensor:
    """``out = A B`` (or ``+=``) for a packed band through the split-precision tensor-core entry point
    (see ``dastac.h``)."""
    assert packed.is_cuda and B.is_cuda and out.is_cuda and B.dim() == 2 and out.dim() == 2
    assert packed.dtype == B.dtype == out.dtype == torch.float32
    assert (B.shape[1] <= 1 or (B.stride(1) == 1 and out.stride(1) == 1)) and out.shape == (s.dims[0], B.shape[1])
    _check(_lib.dastac_bandmm_split_tf32(s._h, packed.data_ptr(), B.data_ptr(), B.stride(0), out.data_ptr(),
                                         out.stride(0), B.shape[1], int(accumulate),
                                         None if err_word is None else err_word.data_ptr(), _stream()),
           "dastac_bandmm_split_tf32")
    return out


def ttm_split_tf32(s: Structure, packed: torch.Tensor, C: torch.Tensor, out: torch.Tensor,
                   accumulate: bool = False, err_word: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Tensor times matrix, packed in and packed out (``out`` holds ``count / Q * K`` values), through the
    split-precision tensor-core entry point (see ``dastac.h``)."""
    assert packed.is_cuda and C.is_cuda and out.is_cuda and C.dim() == 2
    assert packed.dtype == C.dtype == out.dtype == torch.float32
    assert C.shape[0] <= 1 or C.stride(1) == 1 or C.shape[1] <= 1
    _check(_lib.dastac_ttm_split_tf32(s._h, packed.data_ptr(), C.data_ptr(), C.stride(0), C.shape[0], out.data_ptr(),
                                      int(accumulate), None if err_word is None else err_word.data_ptr(), _stream()),
           "dastac_ttm_split_tf32")
    return out


def trimm_bf16_noalloc(s: Structure, packed: torch.Tensor, B: torch.Tensor, out: torch.Tensor,
                       accumulate: bool = False, err_word: Optional[torch.Tensor] = None) -> torch.Tensor:
    """``out = A B`` (or ``+=``) for a packed bf16 upper triangle of at most ``NOALLOC_MAX_N`` rows,
    through the entry point that takes no workspace and allocates nothing (see ``dastac.h``)."""
    assert packed.is_cuda and B.is_cuda and out.is_cuda and B.dim() == 2 and out.dim() == 2
    assert packed.dtype == torch.bfloat16 and B.dtype == torch.bfloat16 and out.dtype == torch.float32
    assert B.stride(1) == 1 and out.stride(1) == 1 and out.shape == (s.dims[0], B.shape[1])
    _check(_lib.dastac_trimm_bf16_noalloc(s._h, packed.data_ptr(), B.data_ptr(), B.stride(0), B.shape[1],
                                          out.data_ptr(), out.stride(0), int(accumulate),
                                          None if err_word is None else err_word.data_ptr(), _stream()),
           "dastac_trimm_bf16_noalloc")
    return out
