"""Pins for the CPU oracle: every function is checked against something other than itself.

The oracle computes packed positions with a counter during enumeration and contractions with
masked dense loops.  Here those results are compared with what the paper prints and the
mathematics fixes: printed ranking polynomials, closed-form cardinalities, the combinatorial number
system, textbook special cases and numpy/torch fp64 library routines the special cases reduce to.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
import synth
from synth import structures as st

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _printed():
    out = {}
    with open(os.path.join(GOLDEN, "printed_polynomials.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, cite, idx, syms, expr = [s.strip() for s in line.split("|")]
            out[name] = (idx.split(), syms.split(), expr)
    return out


def _eval_printed(name, idx, syms):
    names_i, names_s, expr = _printed()[name]
    env = {"H": Fraction(1, 2)}
    env.update({k: Fraction(int(v)) for k, v in zip(names_i, idx)})
    env.update({k: Fraction(int(v)) for k, v in zip(names_s, syms)})
    val = eval(expr, {"__builtins__": {}}, env)  # noqa: S307 - fixture text, rational arithmetic only
    assert val.denominator == 1
    return int(val)


# ---- index maps -------------------------------------------------------------------------------

@pytest.mark.parametrize("N", [1, 2, 3, 4, 7, 16, 33, 40])
def test_upper_triangle_positions(N):
    d = st.upper_triangle(N)
    table = oracle.rank_table(d)
    cnt = oracle.count(d)
    assert cnt == N * (N + 1) // 2                       # closed-form cardinality
    inside = table >= 0
    assert inside.sum() == cnt
    assert np.array_equal(inside, np.triu(np.ones((N, N), bool)))
    vals = table[inside]                                  # row-major = lexicographic order
    assert np.array_equal(vals, np.arange(cnt))           # bijection onto [0,count), monotone
    # The printed upper-half-cube polynomial with a trailing extent Q = 1 and l = 0 is this map.
    for i in range(N):
        for j in range(i, N):
            assert table[i, j] == _eval_printed("upper_half_cube", (i, j, 0), (N, N, 1))
            assert oracle.rank_point(d, (i, j)) == table[i, j] if N <= 7 else True
    assert oracle.rank_point(d, (N - 1, 0)) == (-1 if N > 1 else 0)


@pytest.mark.parametrize("N", [1, 2, 5, 12, 31])
def test_lower_triangle_printed_polynomial(N):
    d = st.lower_triangle(N)
    table = oracle.rank_table(d)
    assert oracle.count(d) == N * (N + 1) // 2
    for i in range(N):
        for j in range(i + 1):
            assert table[i, j] == _eval_printed("lower_triangle", (i, j), (N,))
        # the boundary piece the fusion step removes agrees with the fused polynomial on j = 0
        assert table[i, 0] == _eval_printed("lower_triangle_piece_j0", (i, 0), (N,))
    assert (table[np.triu_indices(N, 1)] == -1).all()


@pytest.mark.parametrize("M,N,Q", [(3, 3, 1), (4, 6, 3), (6, 4, 2), (5, 5, 4), (1, 7, 2)])
def test_upper_half_cube_printed_polynomial(M, N, Q):
    d = st.upper_half_cube(M, N, Q)
    table = oracle.rank_table(d)
    cnt = 0
    for i in range(M):
        for j in range(N):
            for l in range(Q):
                if i <= j:
                    assert table[i, j, l] == _eval_printed("upper_half_cube", (i, j, l), (M, N, Q))
                    # integer evaluation with every term doubled and one final halving, the way
                    # the generated loop nest of the running example evaluates it
                    doubled = -i * Q + 2 * i * N * Q - i * i * Q + 2 * j * Q + 2 * l
                    assert doubled % 2 == 0 and doubled // 2 == table[i, j, l]
                    cnt += 1
                else:
                    assert table[i, j, l] == -1
    assert oracle.count(d) == cnt


@pytest.mark.parametrize("n", [1, 2, 3, 5, 9, 17, 24])
def test_tetrahedron_positions(n):
    d = st.tetrahedron(n)
    table = oracle.rank_table(d)
    cnt = oracle.count(d)
    assert cnt == n * (n + 1) * (n + 2) // 6
    inside = table >= 0
    assert np.array_equal(table[inside], np.arange(cnt))
    # Reversed position is the degree-3 combinatorial number system of (a, b, c) = n-1-(i, j, k).
    for i in range(n):
        for j in range(n):
            for k in range(n):
                if i <= j <= k:
                    a, b, c = n - 1 - i, n - 1 - j, n - 1 - k
                    q = math.comb(a + 2, 3) + math.comb(b + 1, 2) + math.comb(c, 1)
                    assert table[i, j, k] == cnt - 1 - q
                else:
                    assert table[i, j, k] == -1


@pytest.mark.parametrize("N,w", [(1, 0), (5, 0), (6, 1), (9, 2), (8, 7), (20, 3), (4, 6)])
def test_band_slots(N, w):
    slots = oracle.band_slot_table(N, w)
    i, j = np.indices((N, N))
    inside = np.abs(i - j) <= w
    assert np.array_equal(slots >= 0, inside)
    assert np.array_equal(slots[inside], ((j - i + w) * N + i)[inside])    # affine, diagonal-major
    assert len(np.unique(slots[inside])) == inside.sum()
    w_eff = min(w, N - 1) if N > 0 else 0
    nnz = (2 * w_eff + 1) * N - w_eff * (w_eff + 1)
    assert inside.sum() == nnz
    assert oracle.count(st.band(N, w)) == nnz
    if w <= N - 1:
        assert nnz == (2 * w + 1) * N - w * (w + 1)


@pytest.mark.parametrize("desc", [st.upper_triangle(13), st.lower_triangle(9), st.tetrahedron(8),
                                  st.upper_half_cube(4, 6, 3), st.band(11, 2), st.diagonal(7),
                                  st.dense_box([3, 4])])
def test_unrank_is_inverse(desc):
    table = oracle.rank_table(desc)
    points = oracle.unrank_table(desc)
    assert points.shape == (oracle.count(desc), desc.rank)
    for p, pt in enumerate(points):
        assert table[tuple(pt)] == p
    # lexicographic and strictly increasing
    as_tuples = [tuple(int(v) for v in pt) for pt in points]
    assert as_tuples == sorted(as_tuples) and len(set(as_tuples)) == len(as_tuples)


def test_diagonal_and_dense_counts():
    assert oracle.count(st.diagonal(17)) == 17
    assert oracle.count(st.dense_box([3, 4, 5])) == 60
    assert np.array_equal(oracle.rank_table(st.dense_box([3, 4])), np.arange(12).reshape(3, 4))


# ---- compress / decompress ---------------------------------------------------------------------

def _special_bits(shape, seed):
    """fp32 payloads including NaNs with payload bits, infinities and signed zeros."""
    rng = np.random.default_rng(seed)
    bits = rng.integers(0, 2**32, size=shape, dtype=np.uint64).astype(np.uint32)
    flat = bits.reshape(-1)
    flat[::7] = 0x80000000      # -0.0
    flat[3::11] = 0x7FC12345    # quiet NaN with payload
    flat[5::13] = 0xFF800000    # -inf
    return bits


@pytest.mark.parametrize("desc", [st.upper_triangle(9), st.lower_triangle(6), st.tetrahedron(6),
                                  st.upper_half_cube(3, 5, 2), st.diagonal(5)])
def test_pack_unpack_bit_exact(desc):
    bits = _special_bits(tuple(desc.dims), 1)
    table = oracle.rank_table(desc)
    packed = oracle.pack(desc, bits)
    assert packed.shape == (oracle.count(desc),)
    assert np.array_equal(packed, bits[table >= 0])              # lexicographic gather of the set
    back = oracle.unpack(desc, packed)
    assert np.array_equal(back, np.where(table >= 0, bits, 0))   # unpack(pack) = mask * dense
    assert np.array_equal(oracle.pack(desc, back), packed)       # pack(unpack) = id
    # 16-bit elements move the same way
    b16 = (bits & 0xFFFF).astype(np.uint16)
    assert np.array_equal(oracle.unpack(desc, oracle.pack(desc, b16)), np.where(table >= 0, b16, 0))


def test_symmetric_unpack_fills_mirror():
    N = 8
    desc = st.upper_triangle(N, symmetric=True)
    bits = _special_bits((N, N), 2)
    packed = oracle.pack(desc, bits)
    full = oracle.unpack(desc, packed)
    up = np.triu(np.ones((N, N), bool))
    assert np.array_equal(full[up], bits[up])
    assert np.array_equal(full, np.where(up, bits, bits.T))


def test_band_pack_unpack():
    N, w = 9, 2
    dense = _special_bits((N, N), 3).view(np.float32)
    packed = oracle.band_pack(N, w, dense)
    slots = oracle.band_slot_table(N, w)
    flat = packed.reshape(-1).view(np.uint32)
    assert np.array_equal(flat[slots[slots >= 0]], dense.view(np.uint32)[slots >= 0])
    pad = np.ones(flat.shape, bool)
    pad[slots[slots >= 0]] = False
    assert (flat[pad] == 0).all()                                # pads are +0.0f
    assert pad.sum() == w * (w + 1)
    back = oracle.band_unpack(N, w, packed)
    assert np.array_equal(back.view(np.uint32), np.where(slots >= 0, dense.view(np.uint32), 0))
    # unpack ignores the pad contents
    poisoned = flat.copy()
    poisoned[pad] = 0x7FC00000
    again = oracle.band_unpack(N, w, poisoned.view(np.float32).reshape(2 * w + 1, N))
    assert np.array_equal(again.view(np.uint32), back.view(np.uint32))


# ---- the generator's structured streams agree with the oracle's compress -------------------------

def test_streams_match_oracle_pack():
    N = 37
    dense = synth.dense(5, 1, (N, N))
    assert np.array_equal(oracle.pack(st.upper_triangle(N), dense), synth.upper_triangle_stream(5, 1, N))
    n = 11
    T = synth.dense(6, 2, (n, n, n))
    assert np.array_equal(oracle.pack(st.tetrahedron(n), T), synth.tetrahedron_stream(6, 2, n))
    N, w = 23, 3
    A = synth.dense(7, 3, (N, N))
    assert np.array_equal(oracle.band_pack(N, w, A), synth.band_diagonals_stream(7, 3, N, w))
    assert np.array_equal(oracle.pack(st.band_exact(N, w), A), synth.band_rows_stream(7, 3, N, w))
    for M, N, Q in ((6, 9, 5), (9, 6, 3)):
        H = synth.dense(10, 5, (M, N, Q))
        assert np.array_equal(oracle.pack(st.upper_half_cube(M, N, Q), H), synth.upper_half_cube_stream(10, 5, M, N, Q))
    N = 19
    U = synth.dense(8, 4, (N, N), dist=synth.NORMAL)
    full = oracle.unpack(st.upper_triangle(N, symmetric=True),
                         oracle.pack(st.upper_triangle(N), U))
    for i in (0, 7, 18):
        assert np.array_equal(full[i], synth.symmetric_row(8, 4, N, i, dist=synth.NORMAL))
    # bf16 stream = round-to-nearest-even of the fp32 stream (torch's conversion is RNE)
    s32 = synth.upper_triangle_stream(9, 0, 21, dist=synth.NORMAL, scale=0.1)
    s16 = synth.upper_triangle_stream(9, 0, 21, dist=synth.NORMAL, scale=0.1, bf16=True)
    ref = torch.from_numpy(s32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(s16, ref)


def test_generator_distributions():
    u = synth.dense(0, 0, (200000,))
    assert u.min() >= -1.0 and u.max() < 1.0 and abs(u.mean()) < 0.01 and abs(u.std() - 3 ** -0.5) < 0.01
    z = synth.dense(2, 0, (200000,), dist=synth.NORMAL)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1.0) < 0.01 and np.isfinite(z).all()
    assert not np.array_equal(synth.dense(0, 0, (64,)), synth.dense(0, 1, (64,)))
    assert np.array_equal(synth.dense(3, 1, (10, 10)).reshape(-1)[40:70], synth.linear_slice(3, 1, 40, 30))


# ---- contractions -------------------------------------------------------------------------------

def test_matvec_closed_forms_and_library():
    N = 45
    d = st.upper_triangle(N)
    ones = np.ones((N, N), np.float32)
    y, ya = oracle.matvec(d, ones, np.ones(N, np.float32))
    assert np.array_equal(y, N - np.arange(N)) and np.array_equal(ya, y)     # row lengths
    A = synth.dense(0, 0, (N, N))
    x = synth.dense(0, 1, (N,))
    y, ya = oracle.matvec(d, A, x)
    ref = torch.triu(torch.from_numpy(A).double()) @ torch.from_numpy(x).double()
    np.testing.assert_allclose(y, ref.numpy(), rtol=0, atol=1e-13)
    refa = torch.triu(torch.from_numpy(A).double()).abs() @ torch.from_numpy(x).double().abs()
    np.testing.assert_allclose(ya, refa.numpy(), rtol=1e-13)
    for k in (0, 17, N - 1):                                                  # x = e_k -> column k
        e = np.zeros(N, np.float32)
        e[k] = 1
        yk, _ = oracle.matvec(d, A, e)
        assert np.array_equal(yk, np.triu(A)[:, k].astype(np.float64))
    # identity inside the structure returns x
    yi, _ = oracle.matvec(d, np.eye(N, dtype=np.float32), x)
    assert np.array_equal(yi, x.astype(np.float64))
    # a row subset is the same rows
    sel = np.array([3, 0, 44])
    ys, _ = oracle.matvec(d, A[sel], x, sel=sel)
    assert np.array_equal(ys, y[sel])
    # lower triangle: a transposed operand would fail this one
    yl, _ = oracle.matvec(st.lower_triangle(N), A, x)
    np.testing.assert_allclose(yl, np.tril(A).astype(np.float64) @ x.astype(np.float64), atol=1e-13)


def test_symv_against_triangular_identity():
    N = 53
    U = synth.dense(2, 0, (N, N), dist=synth.NORMAL)
    x = synth.dense(2, 1, (N,), dist=synth.NORMAL)
    y, ya = oracle.symv(U, x)
    Ud, xd = np.triu(U).astype(np.float64), x.astype(np.float64)
    ref = Ud @ xd + Ud.T @ xd - np.diag(Ud) * xd        # y = U x + U^T x - diag(U) x
    np.testing.assert_allclose(y, ref, atol=1e-12)
    S = torch.from_numpy(Ud + Ud.T - np.diag(np.diag(Ud)))
    np.testing.assert_allclose(y, (S @ torch.from_numpy(xd)).numpy(), atol=1e-12)
    np.testing.assert_allclose(ya, (S.abs() @ torch.from_numpy(np.abs(xd))).numpy(), rtol=1e-13)
    # content below the diagonal of U is never read
    U2 = U.copy()
    U2[np.tril_indices(N, -1)] = np.nan
    y2, _ = oracle.symv(U2, x)
    assert np.array_equal(y, y2)
    # rows of the full matrix, taken with the dense-box structure, give the same numbers
    full = oracle.unpack(st.upper_triangle(N, symmetric=True), oracle.pack(st.upper_triangle(N), U))
    sel = np.array([0, 20, 52])
    ys, _ = oracle.matvec(st.dense_box([N, N]), full[sel], x, sel=sel)
    np.testing.assert_allclose(ys, y[sel], atol=1e-13)


def test_band_matmat():
    N, w, C = 40, 3, 5
    d = st.band(N, w)
    A = synth.dense(1, 0, (N, N))
    B = synth.dense(1, 1, (N, C))
    out, outa = oracle.matmat(d, A, B)
    i, j = np.indices((N, N))
    Am = np.where(np.abs(i - j) <= w, A, 0).astype(np.float64)
    np.testing.assert_allclose(out, Am @ B.astype(np.float64), atol=1e-13)
    np.testing.assert_allclose(outa, np.abs(Am) @ np.abs(B.astype(np.float64)), rtol=1e-13)
    ones, _ = oracle.matmat(d, np.ones((N, N), np.float32), np.ones((N, C), np.float32))
    assert np.array_equal(ones[:, 0], (np.abs(i - j) <= w).sum(1))            # row nnz
    sel = np.array([0, 39, 12])
    sub, _ = oracle.matmat(d, A[sel], B, sel=sel)
    assert np.array_equal(sub, out[sel])
    # linearity in B
    B2 = synth.dense(1, 2, (N, C))
    o2, _ = oracle.matmat(d, A, B2)
    o3, _ = oracle.matmat(d, A, (B.astype(np.float64) + B2).astype(np.float32))
    np.testing.assert_allclose(o3, Am @ (B.astype(np.float64) + B2).astype(np.float32), atol=1e-12)
    np.testing.assert_allclose(out + o2, Am @ (B.astype(np.float64) + B2.astype(np.float64)), atol=1e-12)


def test_triangular_matmat_bf16():
    N, C = 33, 7
    d = st.upper_triangle(N)
    A = synth.dense(4, 0, (N, N), dist=synth.NORMAL, scale=N ** -0.5, bf16=True)
    B = synth.dense(4, 1, (N, C), dist=synth.NORMAL, scale=N ** -0.5, bf16=True)
    out, outa = oracle.matmat(d, A, B)
    At = torch.from_numpy(A.view(np.int16)).view(torch.bfloat16).double()
    Bt = torch.from_numpy(B.view(np.int16)).view(torch.bfloat16).double()
    ref = torch.triu(At) @ Bt
    np.testing.assert_allclose(out, ref.numpy(), atol=1e-14)
    np.testing.assert_allclose(outa, (torch.triu(At).abs() @ Bt.abs()).numpy(), rtol=1e-13)
    one = np.full((N, N), 0x3F80, np.uint16)       # bf16 1.0
    o, _ = oracle.matmat(d, one, np.full((N, C), 0x3F80, np.uint16))
    assert np.array_equal(o[:, 0], N - np.arange(N))


def test_mttkrp():
    n, R = 12, 4
    d = st.tetrahedron(n)
    T = synth.dense(3, 0, (n, n, n))
    B = synth.dense(3, 1, (n, R))
    C = synth.dense(3, 2, (n, R))
    out, outa = oracle.mttkrp(d, T, B, C)
    i, j, k = np.indices((n, n, n))
    Tm = np.where((i <= j) & (j <= k), T, 0).astype(np.float64)
    ref = np.einsum("ijk,jr,kr->ir", Tm, B.astype(np.float64), C.astype(np.float64))
    np.testing.assert_allclose(out, ref, atol=1e-13)
    refa = np.einsum("ijk,jr,kr->ir", np.abs(Tm), np.abs(B).astype(np.float64), np.abs(C).astype(np.float64))
    np.testing.assert_allclose(outa, refa, rtol=1e-13)
    ones, _ = oracle.mttkrp(d, np.ones((n, n, n), np.float32), np.ones((n, R), np.float32),
                            np.ones((n, R), np.float32))
    m = n - np.arange(n)
    assert np.array_equal(ones[:, 0], m * (m + 1) // 2)       # Tri(n - i)
    # B and C are not interchangeable: j indexes B, k indexes C
    swapped = np.einsum("ijk,kr,jr->ir", Tm, B.astype(np.float64), C.astype(np.float64))
    assert np.abs(swapped - out).max() > 1e-3
    sel = np.array([11, 2])
    sub, _ = oracle.mttkrp(d, T[sel], B, C, sel=sel)
    assert np.array_equal(sub, out[sel])


def test_ttm_upper_half_cube():
    """Tensor-times-matrix of the paper's running example: A(i,j,k) = B(i,j,l) C(k,l), B nonzero for i <= j."""
    M, N, Q, K = 5, 7, 4, 6
    d = st.upper_half_cube(M, N, Q)
    B = synth.dense(5, 0, (M, N, Q))
    C = synth.dense(5, 1, (K, Q))
    out, outa = oracle.ttm(d, B, C)
    i, j, _ = np.indices((M, N, Q))
    Bm = np.where(i <= j, B, 0).astype(np.float64)
    ref = np.einsum("ijl,kl->ijk", Bm, C.astype(np.float64))
    np.testing.assert_allclose(out, ref, atol=1e-13)
    np.testing.assert_allclose(outa, np.einsum("ijl,kl->ijk", np.abs(Bm), np.abs(C).astype(np.float64)), rtol=1e-13)
    # closed forms: all ones -> Q on the set, 0 elsewhere; C = identity returns the masked B itself
    ones, _ = oracle.ttm(d, np.ones((M, N, Q), np.float32), np.ones((K, Q), np.float32))
    ii, jj = np.indices((M, N))
    assert np.array_equal(ones[:, :, 0], np.where(ii <= jj, Q, 0))
    same, _ = oracle.ttm(d, B, np.eye(Q, dtype=np.float32))
    assert np.array_equal(same, Bm)
    # C is indexed (k, l): the transposed operand gives something else
    Csq = synth.dense(5, 2, (Q, Q))
    a1, _ = oracle.ttm(d, B, Csq)
    a2, _ = oracle.ttm(d, B, np.ascontiguousarray(Csq.T))
    assert np.abs(a1 - a2).max() > 1e-3
    sel = np.array([4, 1])
    sub, _ = oracle.ttm(d, B[sel], C, sel=sel)
    assert np.array_equal(sub, out[sel])
    # the packed result follows the output's own layout: same (i, j) set, trailing extent K
    dA = st.upper_half_cube(M, N, K)
    packedA = oracle.pack(dA, out)
    assert packedA.shape == (oracle.count(dA),) and oracle.count(dA) == oracle.count(d) // Q * K


def test_moment2_packed_symmetric_output():
    """Degree-2 moments of polynomial regression: A2(i1,i2) = sum_x B(x,i1) B(x,i2), kept on i1 <= i2."""
    M, n = 37, 9
    d = st.upper_triangle(n, symmetric=True)
    B = synth.dense(6, 0, (M, n))
    out, outa = oracle.moment2(d, B)
    B64 = B.astype(np.float64)
    gram = B64.T @ B64                                   # library routine, all n x n entries
    np.testing.assert_allclose(out, np.triu(gram), atol=1e-12)
    np.testing.assert_allclose(outa, np.triu(np.abs(B64).T @ np.abs(B64)), rtol=1e-13)
    assert (out[np.tril_indices(n, -1)] == 0).all()      # outside the unique set nothing is computed
    # closed forms: a single sample gives the outer product; all ones gives M on the set;
    # the diagonal holds the squared column norms; orthonormal columns give the identity
    one, _ = oracle.moment2(d, B[:1])
    assert np.array_equal(one, np.triu(np.outer(B64[0], B64[0])))
    ones, _ = oracle.moment2(d, np.ones((M, n), np.float32))
    assert np.array_equal(ones, np.triu(np.full((n, n), float(M))))
    np.testing.assert_allclose(np.diag(out), (B64 ** 2).sum(0), rtol=1e-13)
    q, _ = np.linalg.qr(np.random.default_rng(0).standard_normal((M, n)))
    eye, _ = oracle.moment2(d, q.astype(np.float32))
    np.testing.assert_allclose(eye, np.eye(n), atol=1e-6)
    # the sum runs over the first index of B (samples): a square B and its transpose differ
    Bs = synth.dense(6, 1, (n, n))
    a1, _ = oracle.moment2(d, Bs)
    a2, _ = oracle.moment2(d, np.ascontiguousarray(Bs.T))
    assert np.abs(a1 - a2).max() > 1e-3
    # selected rows, and bf16 bit patterns widened exactly
    sel = np.array([7, 0, 3])
    sub, _ = oracle.moment2(d, B, sel=sel)
    assert np.array_equal(sub, out[sel])
    bits = synth.dense(6, 2, (M, n), bf16=True)
    wide = (bits.astype(np.uint32) << 16).view(np.float32)
    o16, _ = oracle.moment2(d, bits)
    o32, _ = oracle.moment2(d, wide)
    assert np.array_equal(o16, o32)
    # the stored result is the packed upper triangle: position of (i1, i2) = number of kept entries before it
    packed = oracle.pack(d, out)
    assert packed.shape == (n * (n + 1) // 2,)
    assert packed[oracle.rank_point(d, (2, 5))] == out[2, 5] and packed[n] == out[1, 1]


def test_moment3_packed_tetrahedral_output():
    """Degree-3 moments: A3(i1,i2,i3) = sum_x B(x,i1) B(x,i2) B(x,i3), kept on i1 <= i2 <= i3."""
    M, n = 23, 7
    d = st.tetrahedron(n)
    B = synth.dense(9, 0, (M, n))
    out, outa = oracle.moment3(d, B)
    B64 = B.astype(np.float64)
    full = np.einsum("xi,xj,xk->ijk", B64, B64, B64)          # library routine, all n^3 entries
    i, j, k = np.indices((n, n, n))
    keep = (i <= j) & (j <= k)
    np.testing.assert_allclose(out, np.where(keep, full, 0), atol=1e-12)
    np.testing.assert_allclose(outa, np.where(keep, np.einsum("xi,xj,xk->ijk", *(np.abs(B64),) * 3), 0), rtol=1e-13)
    assert (out[~keep] == 0).all()
    # closed forms: one sample gives the triple outer product; all ones give M on the set;
    # the body diagonal holds the sums of cubes; a constant third factor reduces it to the degree-2 moments
    one, _ = oracle.moment3(d, B[:1])
    assert np.array_equal(one, np.where(keep, np.einsum("i,j,k->ijk", B64[0], B64[0], B64[0]), 0))
    ones, _ = oracle.moment3(d, np.ones((M, n), np.float32))
    assert np.array_equal(ones, np.where(keep, float(M), 0.0))
    np.testing.assert_allclose(out[np.arange(n), np.arange(n), np.arange(n)], (B64 ** 3).sum(0), rtol=1e-13)
    Bc = B.copy()
    Bc[:, n - 1] = 1.0                                           # last feature = the constant 1
    o3, _ = oracle.moment3(d, Bc)
    o2, _ = oracle.moment2(st.upper_triangle(n, symmetric=True), Bc)
    np.testing.assert_allclose(o3[:, :, n - 1], o2, atol=1e-12)
    # the sum runs over the first index of B
    Bs = synth.dense(9, 1, (n, n))
    a1, _ = oracle.moment3(d, Bs)
    a2, _ = oracle.moment3(d, np.ascontiguousarray(Bs.T))
    assert np.abs(a1 - a2).max() > 1e-3
    # selected slabs; bf16 bit patterns widened exactly; packed order of the result
    sel = np.array([5, 0, 2])
    sub, _ = oracle.moment3(d, B, sel=sel)
    assert np.array_equal(sub, out[sel])
    bits = synth.dense(9, 2, (M, n), bf16=True)
    wide = (bits.astype(np.uint32) << 16).view(np.float32)
    assert np.array_equal(oracle.moment3(d, bits)[0], oracle.moment3(d, wide)[0])
    packed = oracle.pack(d, out)
    assert packed.shape == (n * (n + 1) * (n + 2) // 6,)
    assert packed[oracle.rank_point(d, (1, 3, 4))] == out[1, 3, 4] and packed[0] == out[0, 0, 0]


def test_hadamard_structured_times_dense():
    """Tensor Hadamard product A(i,j,k) = B(i,j,k) C(i,j,k) with a structured B (Table 1, THP)."""
    for desc in (st.upper_half_cube(5, 7, 3), st.tetrahedron(6), st.upper_triangle(9), st.band_exact(8, 2), st.dense_box([4])):
        shape = tuple(desc.dims)
        B = synth.dense(10, 0, shape)
        C = synth.dense(10, 1, shape)
        out, outa = oracle.hadamard(desc, B, C)
        mask = oracle.rank_table(desc) >= 0
        ref = np.where(mask, B.astype(np.float64) * C.astype(np.float64), 0.0)   # plain definition in numpy
        assert np.array_equal(out, ref) and np.array_equal(outa, np.abs(ref))
        # closed forms: C = 1 returns the masked B; both all ones give the indicator of the set
        same, _ = oracle.hadamard(desc, B, np.ones(shape, np.float32))
        assert np.array_equal(same, np.where(mask, B, 0).astype(np.float64))
        ones, _ = oracle.hadamard(desc, np.ones(shape, np.float32), np.ones(shape, np.float32))
        assert ones.sum() == oracle.count(desc)
        # the packed result is the element-wise product of the two packed operands
        assert np.array_equal(oracle.pack(desc, out), oracle.pack(desc, B).astype(np.float64) * oracle.pack(desc, C))


@pytest.mark.parametrize("threads", [1, 3])
def test_clipped_timed_variants_equal_the_masked_forms(threads):
    """The loops that are timed as the CPU baseline visit only the stored elements of the packed
    operand; they must give the masked definition's sums (same products, fp64; only the order of
    the additions may differ)."""
    tol = dict(rtol=1e-12, atol=1e-12)
    for N in (1, 2, 37, 130):
        d = st.upper_triangle(N)
        A = synth.dense(0, 0, (N, N), dist=synth.NORMAL)
        x = synth.dense(0, 1, (N,), dist=synth.NORMAL)
        pk = oracle.pack(d, A)
        np.testing.assert_allclose(oracle.clip_matvec_upper(N, pk, x, threads), oracle.matvec(d, A, x)[0], **tol)
        np.testing.assert_allclose(oracle.clip_symv(N, pk, x, threads), oracle.symv(A, x)[0], **tol)
    for N, w, C in ((1, 0, 3), (9, 2, 5), (70, 8, 33), (40, 19, 4)):
        A = synth.dense(1, 0, (N, N))
        B = synth.dense(1, 1, (N, C))
        got = oracle.clip_band_matmat(N, w, oracle.band_pack(N, w, A), B, threads)
        np.testing.assert_allclose(got, oracle.matmat(st.band(N, w), A, B)[0], **tol)
    for n, R in ((1, 1), (5, 3), (33, 8)):
        d = st.tetrahedron(n)
        T = synth.dense(3, 0, (n, n, n))
        B = synth.dense(3, 1, (n, R))
        C = synth.dense(3, 2, (n, R))
        got = oracle.clip_mttkrp_tetra(n, oracle.pack(d, T), B, C, threads)
        np.testing.assert_allclose(got, oracle.mttkrp(d, T, B, C)[0], **tol)
    for N, C in ((1, 1), (50, 7)):
        d = st.upper_triangle(N)
        A = synth.dense(4, 0, (N, N), dist=synth.NORMAL, bf16=True)
        B = synth.dense(4, 1, (N, C), dist=synth.NORMAL, bf16=True)
        sel = np.arange(0, N, 3, dtype=np.int64)
        got = oracle.clip_matmat_upper_bf16(N, oracle.pack(d, A), B, sel=sel, threads=threads)
        np.testing.assert_allclose(got, oracle.matmat(d, A[sel], B, sel=sel)[0], **tol)
