"""Host-side checks of the C-ABI library that need no GPU: exported symbols, descriptor analysis,
host rank/unrank against the oracle's enumeration, and argument errors (none of which launch)."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from synth import structures as st

import paper_2407_13726_b200 as dastac
from paper_2407_13726_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "dastac.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(dastac_[a-z0-9_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert dastac.status_string(0) == "ok" and "unsupported" in dastac.status_string(2)


CASES = [st.upper_triangle(1), st.upper_triangle(2), st.upper_triangle(37), st.upper_triangle(12, True),
         st.lower_triangle(1), st.lower_triangle(23), st.tetrahedron(1), st.tetrahedron(2),
         st.tetrahedron(15), st.upper_half_cube(4, 6, 3), st.upper_half_cube(6, 4, 2),
         st.upper_half_cube(5, 5, 1), st.dense_box([3, 4]), st.dense_box([2, 3, 4]), st.dense_box([7]),
         st.band_exact(1, 0), st.band_exact(7, 0), st.band_exact(7, 3), st.band_exact(8, 3), st.band_exact(23, 4),
         st.band_exact(40, 11), st.sub_triangle(7, 3), st.sub_triangle(6, 1), st.sub_triangle(9, 8),
         st.sub_triangle(40, 17), st.sub_triangle(5, 5), st.offset_band(9, 3, 3), st.offset_band(9, -4, -4),
         st.offset_band(12, -2, 5), st.offset_band(12, -9, 1), st.offset_band(7, -6, -1), st.offset_band(10, -8, 8),
         st.offset_band(11, 2, 6), st.offset_band(6, -5, 4), st.offset_band(1, 0, 0), st.offset_band(8, -7, -7),
         st.band_exact(6, 3), st.band_exact(9, 7), st.fixed_index([5, 7, 3], 0, 2), st.fixed_index([5, 7, 3], 1, 6),
         st.fixed_index([5, 7, 3], 2, 0), st.equal_indices([6, 6, 4], 0, 1), st.equal_indices([4, 6, 3], 0, 1),
         st.equal_indices([7, 5, 2], 0, 1), st.equal_indices([5, 4, 4], 1, 2), st.equal_indices([5, 3, 5], 0, 2),
         st.fixed_index([6, 9], 0, 3), st.fixed_index([6, 9], 1, 8), st.equal_indices([4, 7], 0, 1)]


@pytest.mark.parametrize("desc", CASES, ids=lambda d: f"{d.name}{d.dims}")
def test_host_rank_unrank_match_enumeration(desc):
    s = dastac.Structure(desc)
    table = oracle.rank_table(desc)
    points = oracle.unrank_table(desc)
    assert s.nnz == oracle.count(desc) == s.slots
    for idx in np.ndindex(*desc.dims):
        if table[idx] >= 0:
            assert dastac.rank(s, idx) == table[idx]
        else:
            with pytest.raises(dastac.DastacError):
                dastac.rank(s, idx)
    for p, pt in enumerate(points):
        assert dastac.unrank(s, p) == tuple(int(v) for v in pt)
    for bad in (-1, s.slots):
        with pytest.raises(dastac.DastacError):
            dastac.unrank(s, bad)


@pytest.mark.parametrize("N,w", [(1, 0), (6, 0), (9, 2), (20, 3), (12, 10)])
def test_band_padded_diagonals_host(N, w):
    desc = st.band(N, w)
    s = dastac.Structure(desc)
    assert s.kind == binding.KIND_BAND_DIAGONALS
    slots = oracle.band_slot_table(N, w)
    assert s.slots == (2 * w + 1) * N and s.nnz == (slots >= 0).sum()
    seen = set()
    for i in range(N):
        for j in range(N):
            if slots[i, j] >= 0:
                assert dastac.rank(s, (i, j)) == slots[i, j]
                assert dastac.unrank(s, int(slots[i, j])) == (i, j)
                seen.add(int(slots[i, j]))
    for p in range(s.slots):
        if p not in seen:
            assert dastac.unrank(s, p)[1] == -1   # padding slot


def test_recognition_is_independent_of_how_rows_are_written():
    N = 9
    base = st.upper_triangle(N)
    # the same set with redundant, scaled and re-ordered rows:  2j - 2i >= 0,  j <= N-1 twice, i <= j + 0
    rows = np.array([[0, -1, 1, -1], [-2, 2, 0, 0], [1, 0, 0, 0], [0, 1, 0, 0], [0, -1, 1, -1],
                     [-1, 0, 1, -1], [-1, 1, 0, 3]], dtype=np.int64)
    d2 = st.Descriptor([N, N], [N], rows, np.zeros(len(rows), np.uint8))
    s1, s2 = dastac.Structure(base), dastac.Structure(d2)
    assert (s1.kind, s1.nnz) == (s2.kind, s2.nnz) == (binding.KIND_UPPER, N * (N + 1) // 2)
    # strict inequality written as i - j + 1 <= 0 is a different set: strictly upper = the sub-triangle with shift 1
    strict = st.Descriptor([N, N], [N], np.array([[-1, 1, 0, -1]], dtype=np.int64), np.zeros(1, np.uint8))
    ss = dastac.Structure(strict)
    assert (ss.kind, ss.nnz) == (dastac.KIND_UPPER_SHIFTED, N * (N - 1) // 2) and oracle.count(strict) == ss.nnz
    # a lower bound on i alone (i >= 2) is none of the recognised classes: it gets a fitted map
    rows_from_2 = st.Descriptor([N, N], [N], np.array([[1, 0, 0, -2]], dtype=np.int64), np.zeros(1, np.uint8))
    g = dastac.Structure(rows_from_2)
    assert (g.kind, g.nnz) == (dastac.KIND_GENERIC, (N - 2) * N) and oracle.count(rows_from_2) == g.nnz
    # ... unless the innermost index carries a coefficient other than -1, 0, 1 (i <= 2j: a quasi-polynomial count)
    with pytest.raises(dastac.DastacError) as e:
        dastac.Structure(st.Descriptor([N, N], [N], np.array([[-1, 2, 0, 0]], dtype=np.int64), np.zeros(1, np.uint8)))
    assert e.value.status == 2
    # an equality row (diagonal) closes to the band of half width 0, packed exactly: N points, rank(i, i) = i
    diag = dastac.Structure(st.diagonal(5))
    assert (diag.kind, diag.nnz) == (dastac.KIND_BAND_EXACT, 5) and dastac.rank(diag, (3, 3)) == 3
    assert oracle.count(st.diagonal(5)) == 5
    # a row coupling three indices is not a difference bound: fitted map as well
    three = st.Descriptor([4, 4, 4], [4], np.array([[1, 1, -1, 0, 0]], dtype=np.int64), np.zeros(1, np.uint8))
    g3 = dastac.Structure(three)
    assert (g3.kind, g3.nnz) == (dastac.KIND_GENERIC, oracle.count(three))
    # the padded-diagonal layout and a redundancy map are for recognised classes only
    odd = st.anti_triangle(6)
    odd.padded_diagonals = True
    with pytest.raises(dastac.DastacError) as e:
        dastac.Structure(odd)
    assert e.value.status == 2
    odd = st.anti_triangle(6)
    odd.mirror = [1, 0]
    with pytest.raises(dastac.DastacError) as e:
        dastac.Structure(odd)
    assert e.value.status == 2
    # contradictory rows give the empty set
    empty = st.Descriptor([5, 5], [5], np.array([[1, -1, 0, -1], [-1, 1, 0, -1]], dtype=np.int64),
                          np.zeros(2, np.uint8))
    assert dastac.Structure(empty).nnz == 0
    assert oracle.count(empty) == 0
    # zero extent
    assert dastac.Structure(st.upper_triangle(0)).nnz == 0
    # band without the padded layout: the exact row-after-row pack; wider than half the matrix: the general
    # offset band (same layout rule); in the padded layout a band as wide as the matrix is refused
    assert dastac.Structure(st.band(8, 2, padded_diagonals=False)).kind == dastac.KIND_BAND_EXACT
    assert dastac.Structure(st.band(8, 4, padded_diagonals=False)).kind == dastac.KIND_BAND_OFFSETS
    with pytest.raises(dastac.DastacError):
        dastac.Structure(st.band(8, 7))
    # symmetric swap only on a square upper triangle
    bad = st.lower_triangle(5)
    bad.mirror = [1, 0]
    with pytest.raises(dastac.DastacError):
        dastac.Structure(bad)
    bad = st.upper_triangle(5)
    bad.mirror = [0, 0]
    with pytest.raises(dastac.DastacError) as e:
        dastac.Structure(bad)
    assert e.value.status == 1


def test_config_cardinalities_and_overflow():
    assert dastac.Structure(st.upper_triangle(1024)).nnz == 524800
    assert dastac.Structure(st.upper_triangle(65536, True)).nnz == 2147516416
    assert dastac.Structure(st.upper_triangle(8192)).nnz == 33558528
    assert dastac.Structure(st.tetrahedron(512)).nnz == 22500864
    b = dastac.Structure(st.band(32768, 32))
    assert b.slots == 65 * 32768 and b.nnz == 65 * 32768 - 32 * 33
    with pytest.raises(dastac.DastacError) as e:
        dastac.Structure(st.upper_triangle(2 ** 30 + 1))
    assert e.value.status == 6
    with pytest.raises(dastac.DastacError) as e:
        dastac.Structure(st.tetrahedron(2 ** 20 + 1))
    assert e.value.status == 6
    # products of three accepted extents that leave 63 bits: the dense box and the half cube
    for desc in (st.dense_box([2 ** 22, 2 ** 22, 2 ** 22]), st.upper_half_cube(2 ** 30, 2 ** 30, 2 ** 30)):
        with pytest.raises(dastac.DastacError) as e:
            dastac.Structure(desc)
        assert e.value.status == 6
    # the largest products that still fit are accepted, with the exact count
    assert dastac.Structure(st.dense_box([2 ** 20, 2 ** 20, 2 ** 20])).nnz == 2 ** 60


def test_large_offsets_round_trip_on_host():
    """rank(unrank(p)) == p around 2^31 and at row starts of the 65536 triangle; tetra at n=512."""
    N = 65536
    s = dastac.Structure(st.upper_triangle(N, True))
    rng = np.random.default_rng(0)
    probes = [0, 1, s.nnz - 1, s.nnz - 2, 2 ** 31 - 1, 2 ** 31, 2 ** 31 + 1]
    probes += [int(v) for v in rng.integers(0, s.nnz, 2000)]
    start = 0
    for i in range(0, N, 997):          # row starts by running sum, +-1
        start = sum(N - r for r in range(i)) if i < 3000 else None
        if start is not None:
            probes += [start, max(start - 1, 0), start + 1]
    for p in probes:
        i, j = dastac.unrank(s, p)
        assert 0 <= i <= j < N
        assert dastac.rank(s, (i, j)) == p
    t = dastac.Structure(st.tetrahedron(512))
    for p in [0, 1, t.nnz - 1] + [int(v) for v in rng.integers(0, t.nnz, 2000)]:
        i, j, k = dastac.unrank(t, p)
        assert 0 <= i <= j <= k < 512 and dastac.rank(t, (i, j, k)) == p
    # the largest supported triangle
    big = dastac.Structure(st.upper_triangle(2 ** 30))
    for p in [0, big.nnz - 1, big.nnz // 2, big.nnz // 3]:
        assert dastac.rank(big, dastac.unrank(big, p)) == p


def test_argument_errors_do_not_launch():
    before = dastac.launch_count()
    lib = ctypes.CDLL(binding.LIB_PATH)
    lib.dastac_contract.restype = ctypes.c_int
    assert lib.dastac_contract(b"ij,j->i", None, 2, None, 0, None, 0, None, None) == 1
    nbytes = ctypes.c_size_t()
    assert lib.dastac_contract_workspace(b"ij,j->i", None, 2, None, ctypes.byref(nbytes)) == 1
    assert lib.dastac_structure_create(None, None) == 1
    assert lib.dastac_pack(None, 0, None, None, None, None) == 1
    assert lib.dastac_rank_batch(None, None, ctypes.c_int64(4), None, None) == 1
    # operand-level validation: unknown expression, wrong structure, wrong shapes
    s = dastac.Structure(st.upper_triangle(8))
    ins = (binding._Operand * 2)()
    ins[0].structure = s._h
    ins[0].rank = 2
    ins[1].rank = 1
    ins[1].dims[0] = 8
    ins[1].strides[0] = 1
    out = binding._Operand()
    out.rank = 1
    out.dims[0] = 8
    out.strides[0] = 1
    args = (ins, 2, ctypes.byref(out), ctypes.byref(nbytes))
    assert lib.dastac_contract_workspace(b"ij,jk->ik", *args) == 3
    assert lib.dastac_contract_workspace(b"ij,j->i", *args) == 0 and nbytes.value == 0
    out.dims[0] = 7
    assert lib.dastac_contract_workspace(b"ij,j->i", *args) == 4
    out.dims[0] = 8
    ins[0].dtype = 1
    assert lib.dastac_contract_workspace(b"ij,j->i", *args) == 3
    ins[0].dtype = 0
    # host operands are staged: the workspace covers them
    ins[0].space = 1
    ins[1].space = 1
    out.space = 1
    assert lib.dastac_contract_workspace(b"ij,j->i", *args) == 0
    assert nbytes.value == 256 + 256 + 256
    # null data with a non-empty operand is rejected before any copy or launch
    assert lib.dastac_contract(b"ij,j->i", ins, 2, ctypes.byref(out), 0, None, 0, None, None) == 7
    t = dastac.Structure(st.tetrahedron(4))
    ins[0].structure = t._h
    assert lib.dastac_contract_workspace(b"ij,j->i", *args) == 3
    assert dastac.launch_count() == before


def test_sub_triangle_kind_and_limits():
    """j - i >= N - k: the size-k triangle in the top right corner (Section 6.4, density experiment)."""
    s = dastac.Structure(st.sub_triangle(16, 5))
    assert s.kind == dastac.KIND_UPPER_SHIFTED and s.nnz == s.slots == 15
    assert dastac.rank(s, (0, 11)) == 0 and dastac.rank(s, (4, 15)) == 14 and dastac.unrank(s, 5) == (1, 12)
    assert dastac.Structure(st.sub_triangle(16, 16)).kind == dastac.KIND_UPPER       # k = N: the whole upper triangle
    assert dastac.Structure(st.sub_triangle(16, 0)).nnz == 0                          # k = 0: empty
    big = dastac.Structure(st.sub_triangle(2 ** 16, 2 ** 14))
    assert big.nnz == 2 ** 14 * (2 ** 14 + 1) // 2
    for p in (0, 1, 12345678, big.nnz - 1):
        assert dastac.rank(big, dastac.unrank(big, p)) == p
    sym = st.sub_triangle(8, 3)
    sym.mirror = [1, 0]
    with pytest.raises(dastac.DastacError):
        dastac.Structure(sym)


def test_offset_band_kinds_and_large_sizes():
    """lo <= j - i <= hi: a single off-diagonal is a per-summand buffer of the strided band (Section 6.4)."""
    N, sdist = 2 ** 16, 2 ** 12
    up = dastac.Structure(st.offset_band(N, sdist, sdist))
    dn = dastac.Structure(st.offset_band(N, -sdist, -sdist))
    assert up.kind == dn.kind == dastac.KIND_BAND_OFFSETS and up.nnz == dn.nnz == N - sdist
    assert dastac.rank(up, (5, 5 + sdist)) == 5 and dastac.rank(dn, (sdist + 7, 7)) == 7
    assert dastac.unrank(dn, 0) == (sdist, 0) and dastac.unrank(up, N - sdist - 1) == (N - sdist - 1, N - 1)
    # classes with faster kernels keep their kind: the symmetric band, the diagonal, the sub-triangle, the triangles
    assert dastac.Structure(st.offset_band(64, -3, 3)).kind == dastac.KIND_BAND_EXACT
    assert dastac.Structure(st.offset_band(64, 0, 0)).kind == dastac.KIND_BAND_EXACT
    assert dastac.Structure(st.offset_band(64, 5, 63)).kind == dastac.KIND_UPPER_SHIFTED
    assert dastac.Structure(st.offset_band(64, 0, 63)).kind == dastac.KIND_UPPER
    assert dastac.Structure(st.offset_band(64, -63, 0)).kind == dastac.KIND_LOWER
    assert dastac.Structure(st.offset_band(64, -63, 63)).kind == dastac.KIND_DENSE
    assert dastac.Structure(st.offset_band(64, 70, 80)).nnz == 0
    strictly_lower = dastac.Structure(st.offset_band(64, -63, -1))
    assert strictly_lower.kind == dastac.KIND_BAND_OFFSETS and strictly_lower.nnz == 64 * 63 // 2
    big = dastac.Structure(st.offset_band(2 ** 20, -1000, 37))
    assert big.nnz == oracle_count_offset_band(2 ** 20, -1000, 37)
    for p in (0, 1, 500_500, 123_456_789, big.nnz - 1):
        assert dastac.rank(big, dastac.unrank(big, p)) == p


def oracle_count_offset_band(N, lo, hi):
    """Points of lo <= j - i <= hi in the N x N box, one diagonal at a time (diagonal d has N - |d| points)."""
    return sum(N - abs(d) for d in range(lo, hi + 1) if abs(d) < N)


def test_plane_structures_kind_and_refusals():
    """One index fixed or equal to an earlier one (Table 1: fixed i, fixed j, diagonal plane)."""
    s = dastac.Structure(st.equal_indices([100, 100, 8], 0, 1))
    assert s.kind == dastac.KIND_PLANE and s.nnz == s.slots == 800 and dastac.rank(s, (7, 7, 3)) == 59
    f = dastac.Structure(st.fixed_index([100, 50, 8], 1, 49))
    assert f.kind == dastac.KIND_PLANE and f.nnz == 800 and dastac.unrank(f, 17) == (2, 49, 1)
    assert dastac.Structure(st.fixed_index([100, 50, 8], 1, 50)).nnz == 0        # outside the box: empty
    assert dastac.Structure(st.equal_indices([9, 9], 0, 1)).kind == dastac.KIND_BAND_EXACT   # square matrix: the w = 0 band
    # two determined indices (a line) and an equality combined with an order are not planes: they get fitted maps
    two = st.fixed_index([5, 6, 7], 0, 1)
    two.rows = np.vstack([two.rows, [0, 1, 0, 0, 0, 0, -2]])
    two.is_eq = np.append(two.is_eq, 1).astype(np.uint8)
    line = dastac.Structure(two)
    assert (line.kind, line.nnz) == (dastac.KIND_GENERIC, 7) and dastac.unrank(line, 4) == (1, 2, 4)
    mixed = st.equal_indices([6, 6, 6], 0, 1)
    mixed.rows = np.vstack([mixed.rows, [0, -1, 1, 0, 0, 0, 0]])                  # j <= k as well
    mixed.is_eq = np.append(mixed.is_eq, 0).astype(np.uint8)
    wedge = dastac.Structure(mixed)
    assert (wedge.kind, wedge.nnz) == (dastac.KIND_GENERIC, oracle.count(mixed))


def test_exact_band_limits_and_kind():
    s = dastac.Structure(st.band_exact(9, 2))
    assert s.kind == dastac.KIND_BAND_EXACT and s.nnz == s.slots == 5 * 9 - 2 * 3
    wide = dastac.Structure(st.band_exact(6, 3))        # 2w + 1 > N: rows clipped on both sides -> the general offset band
    assert wide.kind == dastac.KIND_BAND_OFFSETS and wide.nnz == 7 * 6 - 3 * 4
    big = dastac.Structure(st.band_exact(2 ** 20, 1000))
    assert dastac.unrank(big, big.nnz - 1) == (2 ** 20 - 1, 2 ** 20 - 1)
    for p in (0, 1, 500_500, 123_456_789, big.nnz - 2):
        assert dastac.rank(big, dastac.unrank(big, p)) == p


def test_moment2_plan_is_validated_on_the_host():
    """"xi,xj->ij": dense bf16 input given twice, packed f32 upper triangle out; no launch, no GPU."""
    before = dastac.launch_count()
    lib = ctypes.CDLL(binding.LIB_PATH)
    n, M = 24, 100
    s = dastac.Structure(st.upper_triangle(n, symmetric=True))
    ins = (binding._Operand * 2)()
    for k in range(2):
        ins[k].data = 4096          # never dereferenced: planning only
        ins[k].dtype = binding.BF16
        ins[k].rank = 2
        ins[k].dims[0], ins[k].dims[1] = M, n
        ins[k].strides[0], ins[k].strides[1] = n, 1
    out = binding._Operand()
    out.structure = s._h
    out.rank = 2
    nbytes = ctypes.c_size_t(123)
    args = (ins, 2, ctypes.byref(out), ctypes.byref(nbytes))
    ws = lib.dastac_contract_workspace
    assert ws(b"xi,xj->ij", *args) == 0 and nbytes.value == 0        # row pitch 48 bytes: read in place
    ins[0].strides[0] = ins[1].strides[0] = n + 1                      # 50 bytes: a re-pitched copy of B
    assert ws(b"xi,xj->ij", *args) == 0 and nbytes.value == -(-M * n * 2 // 256) * 256
    ins[0].strides[0] = ins[1].strides[0] = n
    ins[0].space = ins[1].space = 1                                    # host input: staged once, not twice
    out.space = 1
    assert ws(b"xi,xj->ij", *args) == 0
    assert nbytes.value == -(-M * n * 2 // 256) * 256 + -(-s.capacity(__import__("torch").float32) * 4 // 256) * 256
    ins[0].space = ins[1].space = out.space = 0
    ins[1].data = 8192                                                 # two different tensors
    assert ws(b"xi,xj->ij", *args) == 3
    ins[1].data = 4096
    ins[1].strides[0] = n + 8
    assert ws(b"xi,xj->ij", *args) == 3
    ins[1].strides[0] = n
    ins[0].dtype = ins[1].dtype = binding.F32
    assert ws(b"xi,xj->ij", *args) == 3
    ins[0].dtype = ins[1].dtype = binding.BF16
    out.structure = None                                               # dense output
    assert ws(b"xi,xj->ij", *args) == 3
    bigger, lower = dastac.Structure(st.upper_triangle(n + 1)), dastac.Structure(st.lower_triangle(n))
    out.structure = bigger._h                                          # wrong extent
    assert ws(b"xi,xj->ij", *args) == 4
    out.structure = lower._h                                           # not the unique part i <= j
    assert ws(b"xi,xj->ij", *args) == 3
    assert ws(b"xi,xj->ij", ins, 1, ctypes.byref(out), ctypes.byref(nbytes)) == 1
    assert dastac.launch_count() == before


def test_moment3_plan_is_validated_on_the_host():
    """"xi,xj,xk->ijk": the same dense bf16 tensor three times, packed f32 tetrahedron out; planning only."""
    before = dastac.launch_count()
    lib = ctypes.CDLL(binding.LIB_PATH)
    n, M = 24, 100
    tet = dastac.Structure(st.tetrahedron(n))
    ins = (binding._Operand * 3)()
    for k in range(3):
        ins[k].data = 4096
        ins[k].dtype = binding.BF16
        ins[k].rank = 2
        ins[k].dims[0], ins[k].dims[1] = M, n
        ins[k].strides[0], ins[k].strides[1] = n, 1
    out = binding._Operand()
    out.structure = tet._h
    out.rank = 3
    nbytes = ctypes.c_size_t(123)
    ws = lib.dastac_contract_workspace
    args = (ins, 3, ctypes.byref(out), ctypes.byref(nbytes))
    bt = -(-n * (-(-M // 8) * 8) * 2 // 256) * 256                          # transposed copy of B, rows padded to 16 bytes
    assert ws(b"xi,xj,xk->ijk", *args) == 0 and nbytes.value == bt
    ins[0].strides[0] = ins[1].strides[0] = ins[2].strides[0] = n + 3     # 54-byte pitch: re-pitched copy as well
    assert ws(b"xi,xj,xk->ijk", *args) == 0 and nbytes.value == -(-(bt + M * n * 2) // 256) * 256
    ins[0].strides[0] = ins[1].strides[0] = ins[2].strides[0] = n
    ins[2].data = 8192                                                     # third factor is another tensor
    assert ws(b"xi,xj,xk->ijk", *args) == 3
    ins[2].data = 4096
    tri2 = dastac.Structure(st.upper_triangle(n, symmetric=True))
    out.structure = tri2._h                                                # degree-2 output structure
    assert ws(b"xi,xj,xk->ijk", *args) == 3
    other = dastac.Structure(st.tetrahedron(n + 1))
    out.structure = other._h
    assert ws(b"xi,xj,xk->ijk", *args) == 4
    assert ws(b"xi,xj,xk->ijk", ins, 2, ctypes.byref(out), ctypes.byref(nbytes)) == 1
    assert dastac.launch_count() == before


def test_hadamard_plan_is_validated_on_the_host():
    """"ijk,ijk->ijk": packed structured operand, dense operand of the same box, packed result of the same structure."""
    before = dastac.launch_count()
    lib = ctypes.CDLL(binding.LIB_PATH)
    d = st.upper_half_cube(6, 8, 4)
    s, same, other = dastac.Structure(d), dastac.Structure(d), dastac.Structure(st.upper_half_cube(6, 8, 5))
    ins = (binding._Operand * 2)()
    ins[0].structure = s._h
    ins[0].rank = 3
    ins[1].rank = 3
    for k, (n, stv) in enumerate(zip((6, 8, 4), (32, 4, 1))):
        ins[1].dims[k], ins[1].strides[k] = n, stv
    out = binding._Operand()
    out.structure = same._h
    out.rank = 3
    nbytes = ctypes.c_size_t(1)
    ws = lib.dastac_contract_workspace
    args = (ins, 2, ctypes.byref(out), ctypes.byref(nbytes))
    assert ws(b"ijk,ijk->ijk", *args) == 0 and nbytes.value == 0
    assert ws(b"ij,ij->ij", *args) == 3                 # rank of the expression and of the structure differ
    out.structure = other._h
    assert ws(b"ijk,ijk->ijk", *args) == 4              # the result must have the structure of the packed operand
    out.structure = None
    assert ws(b"ijk,ijk->ijk", *args) == 3              # dense result: not this rule
    out.structure = same._h
    ins[1].dims[2] = 5
    assert ws(b"ijk,ijk->ijk", *args) == 4
    ins[1].dims[2] = 4
    ins[1].dtype = binding.BF16
    assert ws(b"ijk,ijk->ijk", *args) == 3
    ins[1].dtype = binding.F32
    ins[1].space = 1                                    # host dense operand: staged through the workspace
    assert ws(b"ijk,ijk->ijk", *args) == 0 and nbytes.value == 768
    assert dastac.launch_count() == before


def _check_against_enumeration(desc):
    """Host maps of a recognised structure against the oracle's enumeration (count, rank, unrank)."""
    try:
        s = dastac.Structure(desc)
    except dastac.DastacError as e:
        assert e.status == 2          # valid descriptor, not a recognised class: nothing to compare
        return None
    table = oracle.rank_table(desc)
    assert s.nnz == oracle.count(desc)
    if s.kind == binding.KIND_BAND_DIAGONALS:
        return s.kind
    assert s.slots == s.nnz
    for p, pt in enumerate(oracle.unrank_table(desc)):
        pt = tuple(int(v) for v in pt)
        assert dastac.unrank(s, p) == pt and dastac.rank(s, pt) == p and table[pt] == p
    return s.kind


def test_random_two_index_difference_bounds():
    """Random pairs of bounds lo <= j - i <= hi in square boxes: whichever class the closure picks (dense, upper,
    lower, exact band, sub-triangle, offset band, empty), its maps equal the enumeration."""
    hypothesis = pytest.importorskip("hypothesis")
    from hypothesis import given, settings, strategies as hs

    seen = set()

    @settings(max_examples=150, deadline=None, derandomize=True)
    @given(hs.integers(1, 14), hs.integers(-16, 16), hs.integers(-16, 16))
    def run(N, a, b):
        lo, hi = min(a, b), max(a, b)
        seen.add(_check_against_enumeration(st.offset_band(N, lo, hi)))

    run()
    assert {binding.KIND_EMPTY, binding.KIND_DENSE, binding.KIND_UPPER, binding.KIND_LOWER, binding.KIND_BAND_EXACT,
            binding.KIND_UPPER_SHIFTED, binding.KIND_BAND_OFFSETS} <= seen


def test_random_planes_and_boxes():
    """Random rank-3 boxes with one index fixed or two indices equal."""
    hypothesis = pytest.importorskip("hypothesis")
    from hypothesis import given, settings, strategies as hs

    @settings(max_examples=80, deadline=None, derandomize=True)
    @given(hs.tuples(hs.integers(1, 6), hs.integers(1, 6), hs.integers(1, 6)), hs.integers(0, 2), hs.integers(0, 6),
           hs.booleans(), hs.integers(0, 2))
    def run(dims, axis, value, equal, other):
        if equal:
            a, b = sorted((axis, other))
            if a == b:
                return
            desc = st.equal_indices(list(dims), a, b)
        else:
            desc = st.fixed_index(list(dims), axis, value)
        _check_against_enumeration(desc)

    run()


# ---- descriptors outside the recognised classes: fitted maps ----------------------------------------

GENERIC_CASES = [
    st.anti_triangle(1), st.anti_triangle(2), st.anti_triangle(23),
    st.affine_set([17, 40], [[-2, 1, 0]], name="2i<=j"),
    st.affine_set([14, 40], [[3, -1, 2]], name="j<=3i+2"),
    st.affine_set([30, 30], [[-1, -1, 40], [1, 1, -12], [3, -1, 9]], name="polygon"),
    st.affine_set([25, 25], [[1, 0, -4], [-1, 0, 19], [-1, 1, 3]], name="rows4to19_band"),
    st.affine_set([12, 12, 12], [[-1, 1, 0, 0], [1, -1, 1, 0]], name="i<=j<=i+k"),
    st.affine_set([9, 11, 13], [[-1, -1, -1, 15]], name="i+j+k<=15"),
    st.affine_set([14, 14, 14], [[-1, 1, 0, 0], [0, -1, 1, 0], [1, 0, -1, 4]], name="i<=j<=k<=i+4"),
    st.affine_set([10, 12, 9], [[1, 1, -1, 0], [-1, 0, 1, 3], [0, -1, 0, 8]], name="k<=i+j,k>=i-3,j<=8"),
    st.affine_set([8, 8, 8], [[2, -1, 0, 0], [0, 1, -1, 2], [-3, 0, 1, 6]], name="j<=2i,k<=j+2,k>=3i-6"),
    st.affine_set([6, 6, 6], [[1, -1, 0, -10]], name="empty_by_rows_3d"),
]


@pytest.mark.parametrize("desc", GENERIC_CASES, ids=lambda d: f"{d.name}{d.dims}")
def test_fitted_maps_match_enumeration(desc):
    """Sets that are none of the recognised classes: the map fitted to the library's own slab counts
    equals the oracle's enumeration at every point, in both directions."""
    s = dastac.Structure(desc)
    table = oracle.rank_table(desc)
    points = oracle.unrank_table(desc)
    assert s.nnz == oracle.count(desc) == s.slots
    if s.nnz:
        assert s.kind == dastac.KIND_GENERIC
    for idx in np.ndindex(*desc.dims):
        if table[idx] >= 0:
            assert dastac.rank(s, idx) == table[idx]
        else:
            with pytest.raises(dastac.DastacError):
                dastac.rank(s, idx)
    for p, pt in enumerate(points):
        assert dastac.unrank(s, p) == tuple(int(v) for v in pt)


def test_fitted_maps_on_random_affine_sets():
    rng = np.random.default_rng(11)
    made = 0
    for trial in range(60):
        rank = int(rng.integers(2, 4))
        dims = [int(v) for v in rng.integers(3, 11, rank)]
        cmps = []
        for _ in range(int(rng.integers(1, 4))):
            a = [int(v) for v in rng.integers(-2, 3, rank)]
            a[-1] = int(rng.integers(-1, 2))
            if rank == 3:
                a[1] = int(rng.integers(-1, 2))
            cmps.append(a + [int(rng.integers(-4, 12))])
        desc = st.affine_set(dims, cmps, name=f"random{trial}")
        try:
            s = dastac.Structure(desc)
        except dastac.DastacError as e:
            assert e.status == 2
            continue
        made += 1
        points = oracle.unrank_table(desc)
        assert s.nnz == len(points)
        for p, pt in enumerate(points):
            assert dastac.rank(s, [int(v) for v in pt]) == p
            assert dastac.unrank(s, p) == tuple(int(v) for v in pt)
    assert made >= 40


def test_piecewise_fusion_on_the_printed_triangle_example():
    """Section 4, "Piecewise Polynomial Simplification": counting the lower triangle gives the piece
    j > 0 with i/2 + i^2/2 + j and the piece j = 0 with i/2 + i^2/2; the second agrees with the first on
    its own domain and is fused away.  The polynomials are the golden file's entries."""
    golden = {}
    for line in open(os.path.join(ROOT, "tests", "golden", "printed_polynomials.txt")):
        if line.strip() and not line.startswith("#"):
            name, _, _, _, expr = [f.strip() for f in line.split("|")]
            golden[name] = expr
    assert golden["lower_triangle"] == "H * i + H * i**2 + j" and golden["lower_triangle_piece_j0"] == "H * i + H * i**2"
    P = [(1, (1, 0)), (1, (2, 0)), (2, (0, 1))]     # (i + i^2 + 2 j) / 2
    Pj0 = [(1, (1, 0)), (1, (2, 0))]                # (i + i^2) / 2
    N = 37
    base = st.lower_triangle(N)

    def piece(extra_row, is_eq):
        rows = np.vstack([base.rows, np.array([extra_row], dtype=np.int64)])
        return st.Descriptor([N, N], [N], rows, np.append(base.is_eq, np.uint8(is_eq)))

    D, Dj0 = piece([0, 1, 0, -1], 0), piece([0, 1, 0, 0], 1)      # j >= 1 ; j == 0
    assert dastac.piecewise_fuse([(D, P, 2), (Dj0, Pj0, 2)]) == [0, 0]
    assert dastac.piecewise_fuse([(Dj0, Pj0, 2), (D, P, 2)]) == [1, 1]   # whichever comes first, P survives
    # the fused polynomial is the oracle's position on the whole triangle
    table = oracle.rank_table(base)
    for i in range(N):
        for j in range(i + 1):
            assert (i + i * i + 2 * j) // 2 == table[i, j]
    # a piece that does not agree stays: i/2 + i^2/2 + 1 on j = 0
    assert dastac.piecewise_fuse([(D, P, 2), (Dj0, Pj0 + [(2, (0, 0))], 2)]) == [0, 1]
    # equality between two variables: on the diagonal j = i the polynomial j^2 equals i*j
    diag = piece([1, -1, 0, 0], 1)
    assert dastac.piecewise_fuse([(D, [(1, (1, 1))], 1), (diag, [(1, (0, 2))], 1)]) == [0, 0]
    # no symbolic argument, decided on the integer points: i (i - 1) (i - 2) vanishes on 0 <= i <= 2
    small = st.Descriptor([3], [3], np.zeros((0, 3), np.int64), np.zeros(0, np.uint8))
    cubic = [(1, (3,)), (-3, (2,)), (2, (1,))]
    assert dastac.piecewise_fuse([(small, cubic, 1), (small, [], 1)]) == [0, 0]
    big = st.Descriptor([4], [4], np.zeros((0, 3), np.int64), np.zeros(0, np.uint8))
    assert dastac.piecewise_fuse([(big, cubic, 1), (big, [], 1)]) == [0, 1]


def test_rule_summands_share_buffers_of_equal_regions():
    N, s = 50, 7
    rule = dastac.Rule([st.offset_band(N, 0, 0), st.offset_band(N, s, s), st.offset_band(N, -s, -s), st.offset_band(N, s, s)])
    assert (rule.n_summands, rule.n_buffers, rule.buffer) == (4, 3, [0, 1, 2, 1])
    assert [v.nnz for v in rule.summands] == [N, N - s, N - s, N - s]
    # summands must live in the same box
    with pytest.raises(dastac.DastacError) as e:
        dastac.Rule([st.offset_band(N, 0, 0), st.offset_band(N + 1, 1, 1)])
    assert e.value.status == 4
    with pytest.raises(dastac.DastacError):
        dastac.Rule([])
