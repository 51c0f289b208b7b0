"""Structure descriptors of the synthetic workloads, as plain data.

A descriptor is the conjunction of affine comparisons that defines a unique set: each row holds
coefficients over ``(indices..., params..., 1)`` and means ``row . (idx, params, 1) >= 0`` (or
``== 0``).  These are inputs, written down once and handed unchanged to whichever implementation is
under test; nothing here evaluates them.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np


@dataclass
class Descriptor:
    dims: List[int]                      # extent of every index
    params: List[int]                    # concrete values of the size symbols
    rows: np.ndarray                     # int64 [nrows, rank + nparams + 1]
    is_eq: np.ndarray                    # uint8 [nrows]
    mirror: Optional[List[int]] = None   # redundancy map as an index permutation
    padded_diagonals: bool = False       # band stored as 2w+1 diagonals of N slots
    name: str = ""
    meta: dict = field(default_factory=dict)

    @property
    def rank(self) -> int:
        return len(self.dims)


def _rows(rank: int, nparams: int, items: Sequence[Sequence[int]]):
    width = rank + nparams + 1
    arr = np.zeros((len(items), width), dtype=np.int64)
    for r, it in enumerate(items):
        assert len(it) == width
        arr[r] = it
    return arr


def _box_rows(rank: int, nparams: int, size_param_of: Sequence[int]):
    """0 <= idx_k  and  idx_k <= param - 1 for every index."""
    items = []
    for k in range(rank):
        lo = [0] * (rank + nparams + 1)
        lo[k] = 1
        items.append(lo)
        hi = [0] * (rank + nparams + 1)
        hi[k] = -1
        hi[rank + size_param_of[k]] = 1
        hi[-1] = -1
        items.append(hi)
    return items


def dense_box(dims: Sequence[int]) -> Descriptor:
    rank = len(dims)
    items = _box_rows(rank, rank, list(range(rank)))
    return Descriptor(list(dims), list(dims), _rows(rank, rank, items),
                      np.zeros(len(items), np.uint8), name="dense")


def upper_triangle(N: int, symmetric: bool = False) -> Descriptor:
    """{(i, j) : 0 <= i < N, 0 <= j < N, i <= j}; ``symmetric`` adds the swap (j, i) -> (i, j)."""
    items = _box_rows(2, 1, [0, 0]) + [[-1, 1, 0, 0]]
    return Descriptor([N, N], [N], _rows(2, 1, items), np.zeros(len(items), np.uint8),
                      mirror=[1, 0] if symmetric else None,
                      name="symmetric_upper" if symmetric else "upper_triangle")


def lower_triangle(N: int) -> Descriptor:
    """{(i, j) : 0 <= i < N, 0 <= j < N, j <= i}."""
    items = _box_rows(2, 1, [0, 0]) + [[1, -1, 0, 0]]
    return Descriptor([N, N], [N], _rows(2, 1, items), np.zeros(len(items), np.uint8),
                      name="lower_triangle")


def band(N: int, w: int, padded_diagonals: bool = True) -> Descriptor:
    """{(i, j) : |i - j| <= w} inside the N x N box; params = (N, w)."""
    items = _box_rows(2, 2, [0, 0]) + [[-1, 1, 0, 1, 0], [1, -1, 0, 1, 0]]
    return Descriptor([N, N], [N, w], _rows(2, 2, items), np.zeros(len(items), np.uint8),
                      padded_diagonals=padded_diagonals, name="band", meta={"w": w})


def band_exact(N: int, w: int) -> Descriptor:
    """The same set {(i, j) : |i - j| <= w}, packed row after row without padding."""
    d = band(N, w, padded_diagonals=False)
    d.name = "band_exact"
    return d


def tetrahedron(n: int) -> Descriptor:
    """{(i, j, k) : 0 <= i <= j <= k < n}."""
    items = _box_rows(3, 1, [0, 0, 0]) + [[-1, 1, 0, 0, 0], [0, -1, 1, 0, 0]]
    return Descriptor([n, n, n], [n], _rows(3, 1, items), np.zeros(len(items), np.uint8),
                      name="tetrahedron")


def upper_half_cube(M: int, N: int, Q: int) -> Descriptor:
    """{(i, j, l) : 0 <= i < M, i <= j < N, 0 <= l < Q}; params = (M, N, Q)."""
    items = _box_rows(3, 3, [0, 1, 2]) + [[-1, 1, 0, 0, 0, 0, 0]]
    return Descriptor([M, N, Q], [M, N, Q], _rows(3, 3, items), np.zeros(len(items), np.uint8),
                      name="upper_half_cube")


def diagonal(N: int) -> Descriptor:
    """{(i, j) : 0 <= i < N, i = j}."""
    items = _box_rows(2, 1, [0, 0]) + [[1, -1, 0, 0]]
    eq = np.zeros(len(items), np.uint8)
    eq[-1] = 1
    return Descriptor([N, N], [N], _rows(2, 1, items), eq, name="diagonal")


def sub_triangle(N: int, k: int) -> Descriptor:
    """{(i, j) : 0 <= i < N, 0 <= j < N, j - i >= N - k}: the triangle of size k in the top right
    corner of the N x N box; params = (N, k)."""
    items = _box_rows(2, 2, [0, 0]) + [[-1, 1, -1, 1, 0]]
    return Descriptor([N, N], [N, k], _rows(2, 2, items), np.zeros(len(items), np.uint8),
                      name="sub_triangle", meta={"k": k})


def offset_band(N: int, lo: int, hi: int) -> Descriptor:
    """{(i, j) : lo <= j - i <= hi} inside the N x N box (a single diagonal at distance s when
    lo = hi = s); params = (N,)."""
    items = _box_rows(2, 1, [0, 0]) + [[-1, 1, 0, -lo], [1, -1, 0, hi]]
    return Descriptor([N, N], [N], _rows(2, 1, items), np.zeros(len(items), np.uint8),
                      name="offset_band", meta={"lo": lo, "hi": hi})


def fixed_index(dims: Sequence[int], axis: int, value: int) -> Descriptor:
    """{idx : idx[axis] = value} inside the box ``dims`` (the "Fixed i" / "Fixed j" structures)."""
    rank = len(dims)
    items = _box_rows(rank, rank, list(range(rank)))
    row = [0] * (2 * rank + 1)
    row[axis] = 1
    row[-1] = -value
    items.append(row)
    eq = np.zeros(len(items), np.uint8)
    eq[-1] = 1
    return Descriptor(list(dims), list(dims), _rows(rank, rank, items), eq, name="fixed_index",
                      meta={"axis": axis, "value": value})


def equal_indices(dims: Sequence[int], a: int, b: int) -> Descriptor:
    """{idx : idx[a] = idx[b]} inside the box ``dims`` (a diagonal plane such as i = j)."""
    rank = len(dims)
    items = _box_rows(rank, rank, list(range(rank)))
    row = [0] * (2 * rank + 1)
    row[a], row[b] = 1, -1
    items.append(row)
    eq = np.zeros(len(items), np.uint8)
    eq[-1] = 1
    return Descriptor(list(dims), list(dims), _rows(rank, rank, items), eq, name="equal_indices",
                      meta={"a": a, "b": b})


def affine_set(dims: Sequence[int], comparisons: Sequence[Sequence[int]], name: str = "affine_set") -> Descriptor:
    """Any conjunction of affine comparisons inside the box ``dims``: every item of ``comparisons``
    is ``(a_0, ..., a_{rank-1}, c)`` and states ``sum a_k idx_k + c >= 0``.  params = dims."""
    rank = len(dims)
    items = _box_rows(rank, rank, list(range(rank)))
    for cmp_ in comparisons:
        assert len(cmp_) == rank + 1
        items.append(list(cmp_[:rank]) + [0] * rank + [cmp_[rank]])
    return Descriptor(list(dims), list(dims), _rows(rank, rank, items), np.zeros(len(items), np.uint8), name=name)


def anti_triangle(N: int) -> Descriptor:
    """{(i, j) : i + j <= N - 1}: the triangle above the anti-diagonal."""
    return affine_set([N, N], [[-1, -1, N - 1]], name="anti_triangle")
