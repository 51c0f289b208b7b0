"""GPU parity: every entry point of the C-ABI library against the CPU oracle, element by element,
on seeded inputs at sizes spanning several tiles and ragged tails."""
import numpy as np
import pytest
import torch

import oracle
import synth
from synth import structures as st

from _util import TOL_BF16, TOL_F32, dev, packed_dev, rel_err

pytestmark = pytest.mark.gpu

dastac = pytest.importorskip("paper_2407_13726_b200") if torch.cuda.is_available() else None


# ---- index maps: bit exact ------------------------------------------------------------------------

INDEX_CASES = [st.upper_triangle(1), st.upper_triangle(2), st.upper_triangle(97), st.upper_triangle(128, True),
               st.lower_triangle(61), st.tetrahedron(1), st.tetrahedron(2), st.tetrahedron(48),
               st.upper_half_cube(9, 14, 5), st.upper_half_cube(14, 9, 3), st.dense_box([5, 6, 7]),
               st.band(50, 4), st.band(7, 0), st.upper_triangle(1000), st.band_exact(50, 4), st.band_exact(9, 4),
               st.band_exact(300, 32), st.sub_triangle(60, 13), st.sub_triangle(9, 1), st.sub_triangle(300, 299),
               st.offset_band(50, 7, 7), st.offset_band(50, -20, 3), st.offset_band(33, -30, 28), st.offset_band(200, -199, -1),
               st.fixed_index([9, 11, 5], 0, 4), st.fixed_index([9, 11, 5], 1, 10), st.fixed_index([9, 11, 5], 2, 2),
               st.equal_indices([12, 12, 6], 0, 1), st.equal_indices([7, 9, 9], 1, 2), st.equal_indices([8, 5, 11], 0, 2),
               st.fixed_index([13, 40], 0, 5), st.fixed_index([13, 40], 1, 39), st.equal_indices([10, 31], 0, 1)]


@pytest.mark.parametrize("desc", INDEX_CASES, ids=lambda d: f"{d.name}{d.dims}")
def test_rank_unrank_batch_exhaustive(desc):
    s = dastac.Structure(desc)
    if desc.name == "band":
        table = oracle.band_slot_table(desc.dims[0], desc.meta["w"])
    else:
        table = oracle.rank_table(desc)
    grid = np.stack(np.meshgrid(*[np.arange(d) for d in desc.dims], indexing="ij"), -1)
    idx = torch.from_numpy(grid.reshape(-1, desc.rank).astype(np.int32)).cuda()
    off = dastac.rank_batch(s, idx).cpu().numpy().reshape(table.shape)
    assert np.array_equal(off, table)
    # out-of-box points rank to -1
    bad = torch.tensor([[-1] * desc.rank, list(desc.dims)], dtype=torch.int32).cuda()
    assert (dastac.rank_batch(s, bad).cpu().numpy() == -1).all()
    # unrank of every slot
    got = dastac.unrank_batch(s, torch.arange(s.slots, dtype=torch.int64).cuda()).cpu().numpy()
    if desc.name == "band":
        exp = np.full((s.slots, 2), -1, np.int32)
        ii, jj = np.nonzero(table >= 0)
        exp[table[ii, jj], 0] = ii
        exp[table[ii, jj], 1] = jj
        pad = exp[:, 0] < 0
        exp[pad, 0] = (np.arange(s.slots) % desc.dims[0])[pad]
        assert np.array_equal(got, exp)
    else:
        assert np.array_equal(got, oracle.unrank_table(desc))
    oob = dastac.unrank_batch(s, torch.tensor([-1, s.slots], dtype=torch.int64).cuda()).cpu().numpy()
    assert (oob == -1).all()


@pytest.mark.parametrize("desc", [st.upper_triangle(65536, True), st.upper_triangle(8192),
                                  st.upper_triangle(1024), st.tetrahedron(512), st.upper_triangle(2 ** 30)],
                         ids=lambda d: f"{d.name}{d.dims[0]}")
def test_index_maps_at_config_sizes(desc):
    """Properties that fix the map at any size: it starts at 0, ends at count-1, moves by one
    between lexicographic neighbours, and unrank inverts it; checked around 2^31 as well."""
    s = dastac.Structure(desc)
    rng = np.random.default_rng(7)
    N = desc.dims[0]
    probes = np.concatenate([np.array([0, 1, s.nnz - 2, s.nnz - 1, 2 ** 31 - 1, 2 ** 31, 2 ** 31 + 1]) % s.nnz,
                             rng.integers(0, s.nnz, 1_000_000)]).astype(np.int64)
    p = torch.from_numpy(probes).cuda()
    idx = dastac.unrank_batch(s, p)
    back = dastac.rank_batch(s, idx)
    assert torch.equal(back, p)
    idn = idx.cpu().numpy().astype(np.int64)
    if desc.rank == 2:
        assert ((0 <= idn[:, 0]) & (idn[:, 0] <= idn[:, 1]) & (idn[:, 1] < N)).all()
    else:
        assert ((0 <= idn[:, 0]) & (idn[:, 0] <= idn[:, 1]) & (idn[:, 1] <= idn[:, 2]) & (idn[:, 2] < N)).all()
    # lexicographic successor has the next position
    nxt = idn.copy()
    last = desc.rank - 1
    nxt[:, last] += 1
    for k in range(last, 0, -1):
        wrap = nxt[:, k] >= N
        nxt[wrap, k - 1] += 1
        for kk in range(k, desc.rank):
            nxt[wrap, kk] = nxt[wrap, k - 1]
    ok = nxt[:, 0] < N
    succ = dastac.rank_batch(s, torch.from_numpy(nxt[ok].astype(np.int32)).cuda()).cpu().numpy()
    assert np.array_equal(succ, probes[ok] + 1)
    ends = torch.tensor([[0] * desc.rank, [N - 1] * desc.rank], dtype=torch.int32).cuda()
    assert dastac.rank_batch(s, ends).cpu().tolist() == [0, s.nnz - 1]
    # host and device maps agree
    host = [dastac.unrank(s, int(q)) for q in probes[:300]]
    assert np.array_equal(np.array(host), idn[:300])


# ---- compress / decompress: bit exact -----------------------------------------------------------

def _bits(shape, seed, sixteen=False):
    rng = np.random.default_rng(seed)
    bits = rng.integers(0, 2 ** 32, size=shape, dtype=np.uint64).astype(np.uint32)
    flat = bits.reshape(-1)
    flat[::7] = 0x80000000
    flat[3::11] = 0x7FC12345
    flat[5::13] = 0xFF800000
    return (bits >> 16).astype(np.uint16) if sixteen else bits


PACK_CASES = [st.upper_triangle(1), st.upper_triangle(3), st.upper_triangle(33), st.upper_triangle(129),
              st.upper_triangle(1000), st.upper_triangle(130, True), st.lower_triangle(77),
              st.tetrahedron(2), st.tetrahedron(37), st.upper_half_cube(11, 17, 3),
              st.upper_half_cube(17, 11, 6), st.dense_box([6, 10]), st.band_exact(11, 5), st.band_exact(130, 7),
              st.band_exact(1000, 32), st.sub_triangle(11, 4), st.sub_triangle(130, 77), st.sub_triangle(1000, 333),
              st.offset_band(40, 9, 9), st.offset_band(130, -50, 7), st.offset_band(1000, -3, 40), st.offset_band(90, -85, 80),
              st.dense_box([7]), st.dense_box([5000]), st.dense_box([3, 4, 5]), st.dense_box([2, 3, 2100]), st.tetrahedron(130),
              st.lower_triangle(2100), st.upper_triangle(4100), st.upper_half_cube(40, 64, 32), st.upper_half_cube(20, 33, 8),
              st.upper_half_cube(33, 20, 4), st.upper_half_cube(9, 9, 1), st.fixed_index([9, 11, 8], 0, 4),
              st.fixed_index([9, 11, 8], 1, 3), st.fixed_index([9, 11, 5], 2, 2), st.equal_indices([40, 40, 32], 0, 1),
              st.equal_indices([7, 9, 9], 1, 2), st.equal_indices([8, 5, 11], 0, 2), st.fixed_index([13, 2100], 0, 5),
              st.fixed_index([13, 40], 1, 39)]


@pytest.mark.parametrize("sixteen", [False, True], ids=["f32", "bf16"])
@pytest.mark.parametrize("desc", PACK_CASES, ids=lambda d: f"{d.name}{d.dims}")
def test_pack_unpack_bit_exact(desc, sixteen):
    s = dastac.Structure(desc)
    bits = _bits(tuple(desc.dims), 11, sixteen)
    tdt = torch.bfloat16 if sixteen else torch.float32
    idt = torch.int16 if sixteen else torch.int32
    d_dense = torch.from_numpy(bits.view(np.int16 if sixteen else np.int32)).cuda().view(tdt)
    packed = dastac.pack(s, d_dense)
    got = packed.view(idt).cpu().numpy().view(bits.dtype)
    exp = oracle.pack(desc, bits)
    assert np.array_equal(got[: s.nnz], exp)
    assert (got[s.nnz:] == 0).all()
    out = torch.full(desc.dims, float("nan"), dtype=tdt, device="cuda")
    dastac.unpack(s, packed, out)
    back = out.view(idt).cpu().numpy().view(bits.dtype)
    assert np.array_equal(back, oracle.unpack(desc, exp))
    # non-contiguous dense tensors (a padded leading dimension, then a transposed view)
    big = torch.zeros([d + 3 for d in desc.dims], dtype=tdt, device="cuda")
    view = big[tuple(slice(1, 1 + d) for d in desc.dims)]
    view.copy_(d_dense)
    assert torch.equal(dastac.pack(s, view).view(idt), packed.view(idt))
    out2 = torch.full_like(big, float("nan"))
    v2 = out2[tuple(slice(1, 1 + d) for d in desc.dims)]
    dastac.unpack(s, packed, v2)
    assert np.array_equal(v2.contiguous().view(idt).cpu().numpy().view(bits.dtype), back)
    if desc.rank == 2 and desc.dims[0] == desc.dims[1]:
        tr = d_dense.t().contiguous().t()     # same values, column-major strides
        assert torch.equal(dastac.pack(s, tr).view(idt), packed.view(idt))


@pytest.mark.parametrize("N,w", [(1, 0), (9, 2), (130, 5), (1000, 32), (64, 62)])
def test_band_pack_unpack(N, w):
    desc = st.band(N, w)
    s = dastac.Structure(desc)
    dense = _bits((N, N), 5).view(np.float32)
    packed = dastac.pack(s, torch.from_numpy(dense.view(np.int32)).cuda().view(torch.float32))
    exp = oracle.band_pack(N, w, dense)
    assert np.array_equal(packed.view(torch.int32).cpu().numpy()[: s.slots], exp.reshape(-1).view(np.int32))
    # padding content must not matter to unpack
    slots = oracle.band_slot_table(N, w)
    poisoned = packed.clone()
    pad = np.ones(s.slots, bool)
    pad[slots[slots >= 0]] = False
    poisoned[: s.slots][torch.from_numpy(pad).cuda()] = float("nan")
    out = dastac.unpack(s, poisoned)
    assert np.array_equal(out.view(torch.int32).cpu().numpy(), oracle.band_unpack(N, w, exp).view(np.int32))


# ---- contractions -----------------------------------------------------------------------------

@pytest.mark.parametrize("N", [1, 2, 3, 31, 32, 33, 127, 128, 129, 1000, 1024, 2500, 8191, 8192, 9001])
def test_trmv(N):
    desc = st.upper_triangle(N)
    s = dastac.Structure(desc)
    A = synth.dense(0, 0, (N, N))
    x = synth.dense(0, 1, (N,))
    ref, ref_abs = oracle.matvec(desc, A, x)
    packed = packed_dev(s, synth.upper_triangle_stream(0, 0, N))
    y = torch.full((N,), float("nan"), device="cuda")
    dastac.contract("ij,j->i", s, packed, [dev(x)], y)
    assert rel_err(y.cpu().numpy(), ref, ref_abs) <= TOL_F32
    # accumulate: y += A x
    y0 = synth.dense(0, 2, (N,))
    y2 = dev(y0)
    dastac.contract("ij,j->i", s, packed, [dev(x)], y2, accumulate=True)
    assert rel_err(y2.cpu().numpy(), ref + y0, ref_abs + np.abs(y0)) <= TOL_F32


@pytest.mark.parametrize("N,k", [(2, 1), (9, 4), (64, 64), (100, 33), (1000, 128), (1024, 1000), (4096, 512), (3000, 2500)])
def test_trmv_sub_triangle(N, k):
    """y = A x for the sub-triangular structure j - i >= N - k (Section 6.4): rows k .. N-1 of y are zero."""
    desc = st.sub_triangle(N, k)
    s = dastac.Structure(desc)
    A = synth.dense(0, 0, (N, N))
    x = synth.dense(0, 1, (N,))
    ref, ref_abs = oracle.matvec(desc, A, x)
    packed = packed_dev(s, oracle.pack(desc, A))
    y = torch.full((N,), float("nan"), device="cuda")
    dastac.contract("ij,j->i", s, packed, [dev(x)], y)
    assert rel_err(y.cpu().numpy(), ref, ref_abs) <= TOL_F32
    y0 = synth.dense(0, 2, (N,))
    y2 = dev(y0)
    dastac.contract("ij,j->i", s, packed, [dev(x)], y2, accumulate=True)
    assert rel_err(y2.cpu().numpy(), ref + y0, ref_abs + np.abs(y0)) <= TOL_F32
    assert np.array_equal(y2.cpu().numpy()[k:], y0[k:])          # rows without stored elements are left alone
    # the library's own pack gives the same stream; batched instances with strided operands
    assert np.array_equal(dastac.pack(s, dev(A)).cpu().numpy()[: s.nnz], oracle.pack(desc, A))
    batch = 3
    cap = s.capacity(torch.float32)
    pk = torch.full((batch, cap + 4), float("nan"), device="cuda")[:, :cap]
    xs = torch.empty((batch, N + 2), device="cuda")[:, :N]
    ys = torch.full((batch, N + 1), float("nan"), device="cuda")[:, :N]
    refs = []
    for b in range(batch):
        Ab, xb = synth.dense(30 + b, 0, (N, N)), synth.dense(30 + b, 1, (N,))
        pk[b, : s.nnz] = dev(oracle.pack(desc, Ab))
        xs[b] = dev(xb)
        refs.append(oracle.matvec(desc, Ab, xb))
    dastac.contract("ij,j->i", s, pk, [xs], ys, batch=batch)
    for b in range(batch):
        assert rel_err(ys[b].cpu().numpy(), refs[b][0], refs[b][1]) <= TOL_F32


def _trapezoid(M, N):
    """{(i, j) : 0 <= i < M, i <= j < N} with M < N."""
    rows = np.array([[1, 0, 0, 0, 0], [-1, 0, 1, 0, -1], [0, 1, 0, 0, 0], [0, -1, 0, 1, -1], [-1, 1, 0, 0, 0]], dtype=np.int64)
    return st.Descriptor([M, N], [M, N], rows, np.zeros(len(rows), np.uint8), name="trapezoid")


ROWSPAN_CASES = [st.dense_box([1, 1]), st.dense_box([7, 13]), st.dense_box([1, 50]), _trapezoid(20, 70), st.dense_box([300, 70]), st.dense_box([64, 1000]),
                 st.lower_triangle(1), st.lower_triangle(33), st.lower_triangle(600), st.band_exact(9, 4),
                 st.band_exact(500, 32), st.band_exact(2000, 1), st.offset_band(100, 17, 17), st.offset_band(100, -99, -99),
                 st.offset_band(1000, -30, 200), st.offset_band(700, -699, -1), st.offset_band(257, -200, 190),
                 st.offset_band(4096, 1024, 1024)]


@pytest.mark.parametrize("desc", ROWSPAN_CASES, ids=lambda d: f"{d.name}{d.dims}{sorted(d.meta.items()) if d.meta else ''}")
def test_matvec_row_contiguous_classes(desc):
    """y = A x for the classes whose rows are stored contiguously: dense, lower, exact and offset bands."""
    s = dastac.Structure(desc)
    M, N = desc.dims
    A = synth.dense(0, 0, (M, N))
    x = synth.dense(0, 1, (N,))
    ref, ref_abs = oracle.matvec(desc, A, x)
    packed = packed_dev(s, oracle.pack(desc, A))
    y = torch.full((M,), float("nan"), device="cuda")
    dastac.contract("ij,j->i", s, packed, [dev(x)], y)
    assert rel_err(y.cpu().numpy(), ref, ref_abs) <= TOL_F32
    y0 = synth.dense(0, 2, (M,))
    y2 = dev(y0)
    dastac.contract("ij,j->i", s, packed, [dev(x)], y2, accumulate=True)
    assert rel_err(y2.cpu().numpy(), ref + y0, ref_abs + np.abs(y0)) <= TOL_F32
    batch = 3
    cap = s.capacity(torch.float32)
    pk = torch.full((batch, cap + 4), float("nan"), device="cuda")[:, :cap]
    xs = torch.empty((batch, N + 2), device="cuda")[:, :N]
    ys = torch.full((batch, M + 1), float("nan"), device="cuda")[:, :M]
    refs = []
    for b in range(batch):
        Ab, xb = synth.dense(40 + b, 0, (M, N)), synth.dense(40 + b, 1, (N,))
        pk[b, : s.nnz] = dev(oracle.pack(desc, Ab))
        xs[b] = dev(xb)
        refs.append(oracle.matvec(desc, Ab, xb))
    dastac.contract("ij,j->i", s, pk, [xs], ys, batch=batch)
    for b in range(batch):
        assert rel_err(ys[b].cpu().numpy(), refs[b][0], refs[b][1]) <= TOL_F32


@pytest.mark.parametrize("N,sdist", [(64, 1), (1000, 37), (4096, 512), (5000, 4999)])
def test_strided_band_one_buffer_per_summand(N, sdist):
    """The strided band of Section 6.4, B_U = (j = i) + (j - i = s) + (i - j = s): three summands, each with
    its own packed buffer, evaluated one after the other into the same y."""
    A = synth.dense(7, 0, (N, N))
    x = synth.dense(7, 1, (N,))
    y = torch.full((N,), float("nan"), device="cuda")
    ref = np.zeros(N)
    ref_abs = np.zeros(N)
    total = 0
    for k, (lo, hi) in enumerate([(0, 0), (sdist, sdist), (-sdist, -sdist)]):
        desc = st.offset_band(N, lo, hi)
        s = dastac.Structure(desc)
        total += s.nnz
        packed = dastac.pack(s, dev(A))
        assert np.array_equal(packed.cpu().numpy()[: s.nnz], oracle.pack(desc, A))
        dastac.contract("ij,j->i", s, packed, [dev(x)], y, accumulate=k > 0)
        r, ra = oracle.matvec(desc, A, x)
        ref += r
        ref_abs += ra
    assert total == N + 2 * (N - sdist)
    assert rel_err(y.cpu().numpy(), ref, ref_abs) <= TOL_F32
    # the same numbers from the dense definition of the three diagonals
    i = np.arange(N)
    dense_ref = A[i, i].astype(np.float64) * x
    dense_ref[: N - sdist] += A[i[: N - sdist], i[: N - sdist] + sdist].astype(np.float64) * x[sdist:]
    dense_ref[sdist:] += A[i[sdist:], i[sdist:] - sdist].astype(np.float64) * x[: N - sdist]
    np.testing.assert_allclose(ref, dense_ref, rtol=1e-12, atol=1e-12)


def test_leslie_matrix_first_row_plus_subdiagonal():
    """A Leslie matrix (Table 1, SpMV_L): a dense first row and the sub-diagonal, as two summands."""
    N = 3000
    A = synth.dense(8, 0, (N, N))
    x = synth.dense(8, 1, (N,))
    y = torch.zeros(N, device="cuda")
    first = st.dense_box([1, N])
    s1 = dastac.Structure(first)
    dastac.contract("ij,j->i", s1, packed_dev(s1, A[0]), [dev(x)], y[:1])
    sub = st.offset_band(N, -1, -1)
    s2 = dastac.Structure(sub)
    dastac.contract("ij,j->i", s2, packed_dev(s2, oracle.pack(sub, A)), [dev(x)], y, accumulate=True)
    r1, a1 = oracle.matvec(first, A[:1], x)
    r2, a2 = oracle.matvec(sub, A, x)
    ref, ref_abs = r2.copy(), a2.copy()
    ref[0] += r1[0]
    ref_abs[0] += a1[0]
    assert rel_err(y.cpu().numpy(), ref, ref_abs) <= TOL_F32


def test_trmv_closed_forms():
    N = 515
    s = dastac.Structure(st.upper_triangle(N))
    ones = packed_dev(s, np.ones(s.nnz, np.float32))
    y = torch.empty(N, device="cuda")
    dastac.contract("ij,j->i", s, ones, [torch.ones(N, device="cuda")], y)
    assert np.array_equal(y.cpu().numpy(), (N - np.arange(N)).astype(np.float32))


def test_trmv_batched():
    N, batch = 257, 5
    desc = st.upper_triangle(N)
    s = dastac.Structure(desc)
    cap = s.capacity(torch.float32)
    packed = torch.full((batch, cap + 4), float("nan"), device="cuda")[:, :cap]   # strided instances
    xs = torch.empty((batch, N), device="cuda")
    refs = []
    for b in range(batch):
        A = synth.dense(20 + b, 0, (N, N))
        x = synth.dense(20 + b, 1, (N,))
        packed[b, : s.nnz] = dev(synth.upper_triangle_stream(20 + b, 0, N))
        xs[b] = dev(x)
        refs.append(oracle.matvec(desc, A, x))
    y = torch.full((batch, N), float("nan"), device="cuda")
    dastac.contract("ij,j->i", s, packed, [xs], y, batch=batch)
    for b in range(batch):
        assert rel_err(y[b].cpu().numpy(), refs[b][0], refs[b][1]) <= TOL_F32


@pytest.mark.parametrize("N", [1, 2, 63, 64, 65, 1023, 1025, 2100, 3000])
def test_symv(N):
    desc = st.upper_triangle(N, symmetric=True)
    s = dastac.Structure(desc)
    U = synth.dense(2, 0, (N, N), dist=synth.NORMAL)
    x = synth.dense(2, 1, (N,), dist=synth.NORMAL)
    ref, ref_abs = oracle.symv(U, x)
    packed = packed_dev(s, synth.upper_triangle_stream(2, 0, N, dist=synth.NORMAL))
    ws = _workspace("ij,j->i", s, packed, [dev(x)], torch.empty(N, device="cuda"))
    y = torch.full((N,), float("nan"), device="cuda")
    dastac.contract("ij,j->i", s, packed, [dev(x)], y, workspace=ws)
    assert rel_err(y.cpu().numpy(), ref, ref_abs) <= TOL_F32
    y0 = synth.dense(2, 2, (N,))
    y2 = dev(y0)
    dastac.contract("ij,j->i", s, packed, [dev(x)], y2, accumulate=True, workspace=ws)
    assert rel_err(y2.cpu().numpy(), ref + y0, ref_abs + np.abs(y0)) <= TOL_F32
    # repeated runs stay within tolerance of each other (atomics may reorder sums)
    y3 = torch.empty(N, device="cuda")
    dastac.contract("ij,j->i", s, packed, [dev(x)], y3, workspace=ws)
    assert rel_err(y3.cpu().numpy(), y.cpu().numpy().astype(np.float64), ref_abs) <= TOL_F32


def _workspace(expr, s, packed, ins, out, batch=1):
    n = dastac.contract_workspace(expr, s, packed, ins, out, batch=batch)
    return torch.empty(max(n, 1), dtype=torch.uint8, device="cuda") if n else None


@pytest.mark.parametrize("N,w,C", [(1, 0, 1), (5, 0, 3), (40, 3, 5), (300, 32, 256), (1000, 7, 130),
                                   (2048, 32, 64), (97, 40, 33)])
def test_band_matmat(N, w, C):
    desc = st.band(N, w)
    s = dastac.Structure(desc)
    A = synth.dense(1, 0, (N, N))
    B = synth.dense(1, 1, (N, C))
    ref, ref_abs = oracle.matmat(desc, A, B)
    # padding slots are poisoned: the contraction must not depend on them
    packed = packed_dev(s, synth.band_diagonals_stream(1, 0, N, w, pad_bits=0x7FC00000))
    out = torch.full((N, C), float("nan"), device="cuda")
    dastac.contract("ij,jc->ic", s, packed, [dev(B)], out)
    assert rel_err(out.cpu().numpy(), ref, ref_abs) <= TOL_F32
    C0 = synth.dense(1, 2, (N, C))
    out2 = dev(C0)
    dastac.contract("ij,jc->ic", s, packed, [dev(B)], out2, accumulate=True)
    assert rel_err(out2.cpu().numpy(), ref + C0, ref_abs + np.abs(C0)) <= TOL_F32
    # padded leading dimensions
    Bp = torch.zeros((N, C + 3), device="cuda")[:, :C]
    Bp.copy_(dev(B))
    outp = torch.full((N, C + 5), float("nan"), device="cuda")[:, :C]
    dastac.contract("ij,jc->ic", s, packed, [Bp], outp)
    assert rel_err(outp.cpu().numpy(), ref, ref_abs) <= TOL_F32


@pytest.mark.parametrize("n,R", [(1, 1), (2, 5), (7, 32), (8, 3), (9, 32), (33, 32), (63, 16), (64, 32), (65, 8),
                                 (70, 40), (130, 32), (96, 7), (200, 32), (257, 33), (300, 64)])
def test_mttkrp(n, R):
    desc = st.tetrahedron(n)
    s = dastac.Structure(desc)
    T = synth.dense(3, 0, (n, n, n))
    B = synth.dense(3, 1, (n, R))
    C = synth.dense(3, 2, (n, R))
    ref, ref_abs = oracle.mttkrp(desc, T, B, C)
    packed = packed_dev(s, synth.tetrahedron_stream(3, 0, n))
    out = torch.full((n, R), float("nan"), device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = _workspace("ijk,jr,kr->ir", s, packed, [dev(B), dev(C)], out)
    dastac.contract("ijk,jr,kr->ir", s, packed, [dev(B), dev(C)], out, workspace=ws, err_word=err)
    assert int(err.item()) == 0
    assert rel_err(out.cpu().numpy(), ref, ref_abs) <= TOL_F32
    M0 = synth.dense(3, 3, (n, R))
    out2 = dev(M0)
    dastac.contract("ijk,jr,kr->ir", s, packed, [dev(B), dev(C)], out2, accumulate=True, workspace=ws, err_word=err)
    assert int(err.item()) == 0
    assert rel_err(out2.cpu().numpy(), ref + M0, ref_abs + np.abs(M0)) <= TOL_F32
    # factor matrices and result with padded leading dimensions (rows not 16-byte aligned)
    Bp = torch.zeros((n, R + 3), device="cuda")[:, :R]
    Bp.copy_(dev(B))
    Cp = torch.zeros((n, R + 1), device="cuda")[:, :R]
    Cp.copy_(dev(C))
    outp = torch.full((n, R + 5), float("nan"), device="cuda")[:, :R]
    dastac.contract("ijk,jr,kr->ir", s, packed, [Bp, Cp], outp, workspace=ws, err_word=err)
    assert int(err.item()) == 0
    assert rel_err(outp.cpu().numpy(), ref, ref_abs) <= TOL_F32


@pytest.mark.parametrize("N,C", [(1, 1), (17, 9), (128, 256), (129, 64), (300, 200), (1000, 264), (512, 512)])
def test_triangular_matmat_bf16(N, C):
    desc = st.upper_triangle(N)
    s = dastac.Structure(desc)
    scale = N ** -0.5
    A = synth.dense(4, 0, (N, N), dist=synth.NORMAL, scale=scale, bf16=True)
    B = synth.dense(4, 1, (N, C), dist=synth.NORMAL, scale=scale, bf16=True)
    ref, ref_abs = oracle.matmat(desc, A, B)
    packed = packed_dev(s, synth.upper_triangle_stream(4, 0, N, dist=synth.NORMAL, scale=scale, bf16=True),
                        dtype=torch.bfloat16)
    out = torch.full((N, C), float("nan"), device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = _workspace("ij,jc->ic", s, packed, [dev(B, "bf16")], out)
    dastac.contract("ij,jc->ic", s, packed, [dev(B, "bf16")], out, workspace=ws, err_word=err)
    assert int(err.item()) == 0
    assert rel_err(out.cpu().numpy(), ref, ref_abs) <= TOL_BF16
    C0 = synth.dense(4, 2, (N, C))
    out2 = dev(C0)
    dastac.contract("ij,jc->ic", s, packed, [dev(B, "bf16")], out2, accumulate=True, workspace=ws, err_word=err)
    assert int(err.item()) == 0
    assert rel_err(out2.cpu().numpy(), ref + C0, ref_abs + np.abs(C0)) <= TOL_BF16


def test_host_operands_are_staged():
    """Host (pinned) buffers through the same call: copies in, kernel, copy out."""
    N = 700
    desc = st.upper_triangle(N)
    s = dastac.Structure(desc)
    A = synth.dense(0, 0, (N, N))
    x = synth.dense(0, 1, (N,))
    ref, ref_abs = oracle.matvec(desc, A, x)
    hp = torch.zeros(s.capacity(torch.float32)).pin_memory()
    hp[: s.nnz] = torch.from_numpy(synth.upper_triangle_stream(0, 0, N))
    hx = torch.from_numpy(x).pin_memory()
    hy = torch.full((N,), float("nan")).pin_memory()
    n = dastac.contract_workspace("ij,j->i", s, hp, [hx], hy)
    assert n >= hp.numel() * 4 + 2 * N * 4
    ws = torch.empty(n, dtype=torch.uint8, device="cuda")
    dastac.contract("ij,j->i", s, hp, [hx], hy, workspace=ws)
    torch.cuda.synchronize()
    assert rel_err(hy.numpy(), ref, ref_abs) <= TOL_F32
    with pytest.raises(dastac.DastacError) as e:
        dastac.contract("ij,j->i", s, hp, [hx], hy, workspace=ws[: n // 2])
    assert e.value.status == 7


def test_empty_and_degenerate_inputs():
    s0 = dastac.Structure(st.upper_triangle(0))
    y = torch.empty(0, device="cuda")
    dastac.contract("ij,j->i", s0, torch.empty(0, device="cuda"), [torch.empty(0, device="cuda")], y)
    dastac.pack(s0, torch.empty((0, 0), device="cuda"))
    assert dastac.rank_batch(s0, torch.empty((0, 2), dtype=torch.int32, device="cuda")).numel() == 0
    # zero right-hand-side columns
    s = dastac.Structure(st.band(16, 2))
    out = torch.empty((16, 0), device="cuda")
    dastac.contract("ij,jc->ic", s, s.empty_packed(), [torch.empty((16, 0), device="cuda")], out)
    torch.cuda.synchronize()


@pytest.mark.parametrize("M,N,Q,K", [(1, 1, 1, 1), (5, 7, 4, 6), (7, 5, 3, 5), (33, 40, 32, 32), (64, 64, 20, 12),
                                     (130, 130, 32, 64), (97, 97, 37, 33), (300, 300, 8, 40)])
def test_ttm_upper_half_cube_packed_in_packed_out(M, N, Q, K):
    """The paper's running example A(i,j,k) = B(i,j,l) C(k,l), i <= j: packed operand, packed result."""
    dB, dA = st.upper_half_cube(M, N, Q), st.upper_half_cube(M, N, K)
    sB, sA = dastac.Structure(dB), dastac.Structure(dA)
    B = synth.dense(5, 0, (M, N, Q))
    C = synth.dense(5, 1, (K, Q))
    ref, ref_abs = oracle.ttm(dB, B, C)
    exp, exp_abs = oracle.pack(dA, ref), oracle.pack(dA, ref_abs)
    assert sA.nnz == exp.size
    packedB = packed_dev(sB, synth.upper_half_cube_stream(5, 0, M, N, Q))
    out = sA.empty_packed()
    out.fill_(float("nan"))
    dastac.contract("ijl,kl->ijk", sB, packedB, [dev(C)], out, out_structure=sA)
    assert rel_err(out.cpu().numpy()[: sA.nnz], exp, exp_abs) <= TOL_F32
    A0 = synth.dense(5, 2, (sA.nnz,))
    out2 = sA.empty_packed()
    out2[: sA.nnz] = dev(A0)
    dastac.contract("ijl,kl->ijk", sB, packedB, [dev(C)], out2, accumulate=True, out_structure=sA)
    assert rel_err(out2.cpu().numpy()[: sA.nnz], exp + A0, exp_abs + np.abs(A0)) <= TOL_F32
    # a padded leading dimension of C
    Cp = torch.zeros((K, Q + 3), device="cuda")[:, :Q]
    Cp.copy_(dev(C))
    out3 = sA.empty_packed()
    dastac.contract("ijl,kl->ijk", sB, packedB, [Cp], out3, out_structure=sA)
    assert rel_err(out3.cpu().numpy()[: sA.nnz], exp, exp_abs) <= TOL_F32
    # the unpacked result is the dense rule on the set and zero off it
    dense = dastac.unpack(sA, out).cpu().numpy()
    ii, jj = np.indices((M, N))
    assert (dense[ii > jj] == 0).all()
    # shape errors are reported before anything runs
    if K > 1:
        with pytest.raises(dastac.DastacError) as e:
            dastac.contract("ijl,kl->ijk", sB, packedB, [dev(C[:-1])], out, out_structure=sA)
        assert e.value.status == 4


@pytest.mark.parametrize("N", [2047, 2048, 2049, 4097])
def test_matvec_kernels_around_tile_edges(N):
    """Sizes that straddle the kernels' own limits: 2048 is the last N of the quad TRMV kernel and one
    column tile of the SYMV kernel, 4097 leaves a one-column last tile."""
    U = synth.dense(12, 0, (N, N), dist=synth.NORMAL)
    x = synth.dense(12, 1, (N,), dist=synth.NORMAL)
    stream = synth.upper_triangle_stream(12, 0, N, dist=synth.NORMAL)
    d = st.upper_triangle(N)
    s = dastac.Structure(d)
    ref, ref_abs = oracle.matvec(d, U, x)
    y = torch.full((N,), float("nan"), device="cuda")
    dastac.contract("ij,j->i", s, packed_dev(s, stream), [dev(x)], y)
    assert rel_err(y.cpu().numpy(), ref, ref_abs) <= TOL_F32
    ss = dastac.Structure(st.upper_triangle(N, symmetric=True))
    ref, ref_abs = oracle.symv(U, x)
    y = torch.full((N,), float("nan"), device="cuda")
    dastac.contract("ij,j->i", ss, packed_dev(ss, stream), [dev(x)], y)
    assert rel_err(y.cpu().numpy(), ref, ref_abs) <= TOL_F32


def test_matvec_does_not_read_values_beyond_the_rows():
    """Non-finite values in a neighbouring row or in the padding behind the last row must not leak
    into a result through the masked first / last quads."""
    N = 203
    d = st.upper_triangle(N)
    s = dastac.Structure(d)
    A = synth.dense(13, 0, (N, N))
    A[5, 5:] = np.inf          # row 5 is all infinite: only y[5] may be non-finite
    x = np.abs(synth.dense(13, 1, (N,))) + 0.5
    packed = packed_dev(s, oracle.pack(d, A))      # tail of the buffer is NaN
    y = torch.empty(N, device="cuda")
    dastac.contract("ij,j->i", s, packed, [dev(x)], y)
    got = y.cpu().numpy()
    assert np.isinf(got[5]) and np.isfinite(np.delete(got, 5)).all()
    A[5, 5:] = 0
    ref, ref_abs = oracle.matvec(d, A, x)
    keep = np.arange(N) != 5
    assert rel_err(got[keep], ref[keep], ref_abs[keep]) <= TOL_F32


@pytest.mark.parametrize("desc", [st.tetrahedron(150), st.lower_triangle(1000), st.dense_box([3000]),
                                  st.dense_box([40, 50, 60]), st.upper_triangle(2050)],
                         ids=lambda d: f"{d.name}{d.dims}")
def test_pack_unpack_larger_f32(desc):
    s = dastac.Structure(desc)
    bits = _bits(tuple(desc.dims), 17)
    dense = torch.from_numpy(bits.view(np.int32)).cuda().view(torch.float32)
    packed = dastac.pack(s, dense)
    exp = oracle.pack(desc, bits)
    assert np.array_equal(packed.view(torch.int32).cpu().numpy().view(np.uint32)[: s.nnz], exp)
    out = torch.full(desc.dims, float("nan"), device="cuda")
    dastac.unpack(s, packed, out)
    assert np.array_equal(out.view(torch.int32).cpu().numpy().view(np.uint32), oracle.unpack(desc, exp))


@pytest.mark.parametrize("N,w,C", [(2, 0, 1), (7, 0, 3), (9, 4, 5), (300, 32, 256), (1000, 7, 130), (2048, 32, 64),
                                   (200, 40, 33), (513, 90, 64), (190, 94, 12)])
def test_band_matmat_exact_layout(N, w, C):
    """The band packed row after row without padding (three-piece ranking polynomial)."""
    desc = st.band_exact(N, w)
    s = dastac.Structure(desc)
    A = synth.dense(1, 0, (N, N))
    B = synth.dense(1, 1, (N, C))
    ref, ref_abs = oracle.matmat(desc, A, B)
    packed = packed_dev(s, oracle.pack(desc, A))
    out = torch.full((N, C), float("nan"), device="cuda")
    dastac.contract("ij,jc->ic", s, packed, [dev(B)], out)
    assert rel_err(out.cpu().numpy(), ref, ref_abs) <= TOL_F32
    C0 = synth.dense(1, 2, (N, C))
    out2 = dev(C0)
    dastac.contract("ij,jc->ic", s, packed, [dev(B)], out2, accumulate=True)
    assert rel_err(out2.cpu().numpy(), ref + C0, ref_abs + np.abs(C0)) <= TOL_F32
    # the library's own pack produces the same stream
    assert np.array_equal(dastac.pack(s, dev(A)).cpu().numpy()[: s.nnz], oracle.pack(desc, A))


@pytest.mark.parametrize("M,n", [(1, 1), (5, 8), (64, 128), (100, 200), (257, 300), (700, 520), (130, 1030),
                                 (2000, 256), (63, 77)])
@pytest.mark.parametrize("symmetric", [False, True], ids=["plain", "swap"])
def test_moment2_packed_symmetric_output(M, n, symmetric):
    """Degree-2 moments A2(i1,i2) = sum_x B(x,i1) B(x,i2) on i1 <= i2, packed (Table 1, polynomial regression)."""
    desc = st.upper_triangle(n, symmetric=symmetric)
    sA = dastac.Structure(desc)
    B = synth.dense(6, 0, (M, n), dist=synth.NORMAL, bf16=True)
    ref, ref_abs = oracle.moment2(desc, B)
    exp, exp_abs = oracle.pack(desc, ref), oracle.pack(desc, ref_abs)
    Bd = dev(B, "bf16")
    out = sA.empty_packed()
    out.fill_(float("nan"))
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    nws = dastac.contract_workspace("xi,xj->ij", None, Bd, [Bd], out, out_structure=sA)
    assert (nws == 0) == (n % 8 == 0)          # a row pitch that is not a multiple of 16 bytes needs a re-pitched copy
    ws = torch.empty(max(nws, 1), dtype=torch.uint8, device="cuda")
    dastac.contract("xi,xj->ij", None, Bd, [Bd], out, out_structure=sA, workspace=ws, err_word=err)
    assert int(err.item()) == 0
    got = out.cpu().numpy()
    assert rel_err(got[: sA.nnz], exp, exp_abs) <= TOL_BF16
    assert rel_err(got[: sA.nnz], exp, exp_abs) <= 1e-5     # exact products, fp32 sums: far inside the bf16 bar
    assert np.isnan(got[sA.nnz:]).all()                      # nothing is written beyond the set's count
    A0 = synth.dense(6, 1, (sA.nnz,))
    out2 = sA.empty_packed()
    out2[: sA.nnz] = dev(A0)
    dastac.contract("xi,xj->ij", None, Bd, [Bd], out2, accumulate=True, out_structure=sA, workspace=ws, err_word=err)
    assert int(err.item()) == 0
    assert rel_err(out2.cpu().numpy()[: sA.nnz], exp + A0, exp_abs + np.abs(A0)) <= 1e-5
    # a padded row pitch (multiple of 8 elements: read in place)
    Bp = torch.zeros((M, n + 8 - n % 8 + 8), dtype=torch.bfloat16, device="cuda")[:, :n]
    Bp.copy_(Bd)
    out3 = sA.empty_packed()
    dastac.contract("xi,xj->ij", None, Bp, [Bp], out3, out_structure=sA, err_word=err)
    assert rel_err(out3.cpu().numpy()[: sA.nnz], exp, exp_abs) <= 1e-5
    if symmetric:
        full = dastac.unpack(sA, out3).cpu().numpy()
        assert np.array_equal(full, full.T)
    # two different tensors, a dense output, fp32 inputs: refused before anything runs
    other = Bd.clone()
    with pytest.raises(dastac.DastacError) as e:
        dastac.contract("xi,xj->ij", None, Bd, [other], out3, out_structure=sA)
    assert e.value.status == 3
    with pytest.raises(dastac.DastacError):
        dastac.contract("xi,xj->ij", None, Bd, [Bd], torch.zeros((n, n), device="cuda"))
    Bf = Bd.float()
    with pytest.raises(dastac.DastacError):
        dastac.contract("xi,xj->ij", None, Bf, [Bf], out3, out_structure=sA)
    if n > 1:
        with pytest.raises(dastac.DastacError) as e:
            dastac.contract("xi,xj->ij", None, Bd, [Bd], out3, out_structure=dastac.Structure(st.upper_triangle(n - 1)))
        assert e.value.status == 4


def test_moment2_empty_sum_and_host_operands():
    n = 40
    desc = st.upper_triangle(n, symmetric=True)
    sA = dastac.Structure(desc)
    out = sA.empty_packed()
    out.fill_(float("nan"))
    B0 = torch.zeros((0, n), dtype=torch.bfloat16, device="cuda")
    dastac.contract("xi,xj->ij", None, B0, [B0], out, out_structure=sA)
    assert (out[: sA.nnz] == 0).all()
    # pinned host operands in and out, staged once through the workspace
    M = 300
    B = synth.dense(6, 3, (M, n), dist=synth.NORMAL, bf16=True)
    ref, ref_abs = oracle.moment2(desc, B)
    hB = torch.from_numpy(B).view(torch.int16).view(torch.bfloat16).pin_memory()
    hout = torch.full((sA.capacity(torch.float32),), float("nan")).pin_memory()
    nws = dastac.contract_workspace("xi,xj->ij", None, hB, [hB], hout, out_structure=sA)
    assert nws >= M * n * 2 + sA.nnz * 4
    ws = torch.empty(nws, dtype=torch.uint8, device="cuda")
    dastac.contract("xi,xj->ij", None, hB, [hB], hout, out_structure=sA, workspace=ws)
    torch.cuda.synchronize()
    assert rel_err(hout.numpy()[: sA.nnz], oracle.pack(desc, ref), oracle.pack(desc, ref_abs)) <= 1e-5


@pytest.mark.parametrize("M,n", [(1, 1), (5, 8), (64, 100), (100, 260), (300, 130), (40, 300), (1000, 77)])
def test_moment3_packed_tetrahedral_output(M, n):
    """Degree-3 moments A3(i1,i2,i3) = sum_x B(x,i1) B(x,i2) B(x,i3) on i1 <= i2 <= i3, packed tetrahedron."""
    desc = st.tetrahedron(n)
    sA = dastac.Structure(desc)
    B = synth.dense(9, 0, (M, n), dist=synth.NORMAL, bf16=True)
    ref, ref_abs = oracle.moment3(desc, B)
    exp, exp_abs = oracle.pack(desc, ref), oracle.pack(desc, ref_abs)
    Bd = dev(B, "bf16")
    out = sA.empty_packed()
    out.fill_(float("nan"))
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    nws = dastac.contract_workspace("xi,xj,xk->ijk", None, Bd, [Bd, Bd], out, out_structure=sA)
    assert nws >= n * M * 2                     # the transposed copy of B
    ws = torch.empty(nws, dtype=torch.uint8, device="cuda")
    dastac.contract("xi,xj,xk->ijk", None, Bd, [Bd, Bd], out, out_structure=sA, workspace=ws, err_word=err)
    assert int(err.item()) == 0
    got = out.cpu().numpy()
    # the pairwise product is rounded to bf16 (2^-9 relative) before the third factor: 4e-3 covers it
    assert rel_err(got[: sA.nnz], exp, exp_abs) <= 4e-3 <= TOL_BF16
    assert np.isnan(got[sA.nnz:]).all()
    A0 = synth.dense(9, 1, (sA.nnz,))
    out2 = sA.empty_packed()
    out2[: sA.nnz] = dev(A0)
    dastac.contract("xi,xj,xk->ijk", None, Bd, [Bd, Bd], out2, accumulate=True, out_structure=sA, workspace=ws, err_word=err)
    assert rel_err(out2.cpu().numpy()[: sA.nnz], exp + A0, exp_abs + np.abs(A0)) <= 4e-3
    # refused before anything runs: different tensors, wrong output structure, missing workspace
    with pytest.raises(dastac.DastacError) as e:
        dastac.contract("xi,xj,xk->ijk", None, Bd, [Bd, Bd.clone()], out, out_structure=sA, workspace=ws)
    assert e.value.status == 3
    with pytest.raises(dastac.DastacError):
        dastac.contract("xi,xj,xk->ijk", None, Bd, [Bd, Bd], out, out_structure=dastac.Structure(st.upper_triangle(n)), workspace=ws)
    with pytest.raises(dastac.DastacError) as e:
        dastac.contract("xi,xj,xk->ijk", None, Bd, [Bd, Bd], out, out_structure=sA)
    assert e.value.status == 7


HADAMARD_CASES = [st.upper_half_cube(5, 7, 3), st.upper_half_cube(40, 64, 32), st.tetrahedron(37), st.upper_triangle(130),
                  st.upper_triangle(1000), st.lower_triangle(77), st.band_exact(300, 7), st.band(50, 4), st.dense_box([9]),
                  st.dense_box([6, 10, 33]), st.sub_triangle(90, 31), st.offset_band(64, -5, 20), st.upper_triangle(64, True),
                  st.equal_indices([50, 50, 16], 0, 1), st.fixed_index([20, 30, 12], 0, 7), st.fixed_index([20, 30, 12], 1, 29),
                  st.fixed_index([20, 30, 12], 2, 11), st.equal_indices([9, 14, 14], 1, 2)]


@pytest.mark.parametrize("desc", HADAMARD_CASES, ids=lambda d: f"{d.name}{d.dims}")
def test_hadamard_structured_times_dense(desc):
    """A(idx) = B(idx) C(idx) on the set: packed structured B, dense C, packed result (Table 1, THP)."""
    s = dastac.Structure(desc)
    shape = tuple(desc.dims)
    expr = {1: "i,i->i", 2: "ij,ij->ij", 3: "ijk,ijk->ijk"}[len(shape)]
    B = synth.dense(10, 0, shape)
    C = synth.dense(10, 1, shape)
    ref, ref_abs = oracle.hadamard(desc, B, C)
    if desc.name == "band":
        N, w = desc.dims[0], desc.meta["w"]
        packedB = packed_dev(s, oracle.band_pack(N, w, B), poison_tail=False)
        exp, exp_abs = oracle.band_pack(N, w, ref).reshape(-1), oracle.band_pack(N, w, ref_abs).reshape(-1)
        live = oracle.band_pack(N, w, np.ones(shape, np.float32)).reshape(-1) != 0   # padding slots are don't-care
    else:
        packedB = packed_dev(s, oracle.pack(desc, B))
        exp, exp_abs = oracle.pack(desc, ref), oracle.pack(desc, ref_abs)
        live = np.ones(exp.shape, bool)
    n = exp.size
    out = s.empty_packed()
    out.fill_(float("nan"))
    dastac.contract(expr, s, packedB, [dev(C)], out, out_structure=s)
    got = out.cpu().numpy()[:n]
    # one fp32 multiply per element: exactly the rounded product
    assert np.array_equal(got[live], (exp.astype(np.float32))[live])
    assert rel_err(got[live], exp[live], exp_abs[live]) <= TOL_F32
    # accumulate, and a dense factor with padded strides (generic gather)
    A0 = synth.dense(10, 2, (n,))
    out2 = s.empty_packed()
    out2[:n] = dev(A0)
    L = (shape[-1] + 3) // 4 * 4 + 8                       # padded pitches; the view's first element stays 16-byte aligned
    big = torch.zeros([d + 2 for d in shape[:-1]] + [L], device="cuda")
    view = big[tuple(slice(1, 1 + d) for d in shape[:-1]) + (slice(4, 4 + shape[-1]),)]
    assert view.data_ptr() % 16 == 0 and not view.is_contiguous() or len(shape) == 1
    view.copy_(dev(C))
    dastac.contract(expr, s, packedB, [view], out2, accumulate=True, out_structure=s)
    strided = torch.zeros(shape[:-1] + (2 * shape[-1],), device="cuda")[..., ::2]   # inner stride 2: the generic gather
    strided.copy_(dev(C))
    out4 = s.empty_packed()
    dastac.contract(expr, s, packedB, [strided], out4, out_structure=s)
    assert np.array_equal(out4.cpu().numpy()[:n][live], exp.astype(np.float32)[live])
    assert rel_err(out2.cpu().numpy()[:n][live], (exp + A0)[live], (exp_abs + np.abs(A0))[live]) <= TOL_F32
    # a second structure object made from the same descriptor is the same structure; another one is not
    out3 = s.empty_packed()
    dastac.contract(expr, s, packedB, [dev(C)], out3, out_structure=dastac.Structure(desc))
    assert torch.equal(out3[:n][torch.from_numpy(live).cuda()], out[:n][torch.from_numpy(live).cuda()])
    with pytest.raises(dastac.DastacError):
        dastac.contract(expr, s, packedB, [dev(C)], out3, out_structure=dastac.Structure(st.dense_box(list(shape))) if desc.name != "dense" else None)
    with pytest.raises(dastac.DastacError):
        dastac.contract(expr, s, packedB, [dev(C)[..., :-1] if shape[-1] > 1 else torch.zeros([d + 1 for d in shape], device="cuda")], out3, out_structure=s)


@pytest.mark.parametrize("which", ["diagonal_plane", "fixed_j", "fixed_i"])
def test_ttm_over_plane_structures(which):
    """TTM_DP / TTM_J of Table 1: A(i,j,k) = B(i,j,l) C(k,l) with B on a plane; packed in, packed out."""
    N, Q, K = 33, 32, 24
    mk = {"diagonal_plane": lambda L: st.equal_indices([N, N, L], 0, 1), "fixed_j": lambda L: st.fixed_index([N, N, L], 1, 5),
          "fixed_i": lambda L: st.fixed_index([N, N, L], 0, 17)}[which]
    dB, dA = mk(Q), mk(K)
    sB, sA = dastac.Structure(dB), dastac.Structure(dA)
    assert sB.kind == sA.kind == dastac.KIND_PLANE and sA.nnz == sB.nnz // Q * K
    B = synth.dense(11, 0, (N, N, Q))
    C = synth.dense(11, 1, (K, Q))
    ref, ref_abs = oracle.ttm(dB, B, C)
    exp, exp_abs = oracle.pack(dA, ref), oracle.pack(dA, ref_abs)
    packedB = dastac.pack(sB, dev(B))
    assert np.array_equal(packedB.cpu().numpy()[: sB.nnz], oracle.pack(dB, B))
    out = sA.empty_packed()
    out.fill_(float("nan"))
    dastac.contract("ijl,kl->ijk", sB, packedB, [dev(C)], out, out_structure=sA)
    assert rel_err(out.cpu().numpy()[: sA.nnz], exp, exp_abs) <= TOL_F32
    dense = dastac.unpack(sA, out).cpu().numpy()
    assert np.array_equal(dense != 0, (oracle.rank_table(dA) >= 0) & (dense != 0))     # nothing off the plane
    # a plane on one side and a different plane on the other: refused
    with pytest.raises(dastac.DastacError):
        dastac.contract("ijl,kl->ijk", sB, packedB, [dev(C)], out, out_structure=dastac.Structure(st.fixed_index([N, N, K], 1, 6)))


def test_matvec_single_stored_row():
    """A matrix whose only stored row is i = c (the dense first row of a Leslie matrix inside the N x N box)."""
    N, c = 700, 0
    desc = st.fixed_index([N, N], 0, c)
    s = dastac.Structure(desc)
    A = synth.dense(12, 0, (N, N))
    x = synth.dense(12, 1, (N,))
    ref, ref_abs = oracle.matvec(desc, A, x)
    y = torch.full((N,), float("nan"), device="cuda")
    dastac.contract("ij,j->i", s, packed_dev(s, oracle.pack(desc, A)), [dev(x)], y)
    assert rel_err(y.cpu().numpy(), ref, ref_abs) <= TOL_F32 and (y[1:] == 0).all()


MTTKRP_FIBRE_CASES = [(st.upper_half_cube(9, 14, 20), 5), (st.upper_half_cube(30, 30, 33), 32), (st.dense_box([6, 7, 40]), 40),
                      (st.fixed_index([10, 12, 33], 1, 5), 16), (st.fixed_index([10, 12, 33], 0, 9), 32),
                      (st.equal_indices([12, 12, 40], 0, 1), 7), (st.dense_box([1, 1, 1]), 1)]


@pytest.mark.parametrize("desc,R", MTTKRP_FIBRE_CASES, ids=lambda v: f"{v.name}{v.dims}" if hasattr(v, "name") else str(v))
def test_mttkrp_other_structures(desc, R):
    """M(i,r) = sum_{j,k} T(i,j,k) B(j,r) C(k,r) over the other rank-3 structures with contiguous fibres
    (half cube, dense box, planes with a free trailing index: the MTTKRP structures of Table 1)."""
    s = dastac.Structure(desc)
    ni, nj, nk = desc.dims
    T = synth.dense(13, 0, (ni, nj, nk))
    B = synth.dense(13, 1, (nj, R))
    C = synth.dense(13, 2, (nk, R))
    ref, ref_abs = oracle.mttkrp(desc, T, B, C)
    packed = dastac.pack(s, dev(T))
    out = torch.full((ni, R), float("nan"), device="cuda")
    dastac.contract("ijk,jr,kr->ir", s, packed, [dev(B), dev(C)], out)
    assert rel_err(out.cpu().numpy(), ref, ref_abs) <= TOL_F32
    M0 = synth.dense(13, 3, (ni, R))
    out2 = dev(M0)
    dastac.contract("ijk,jr,kr->ir", s, packed, [dev(B), dev(C)], out2, accumulate=True)
    assert rel_err(out2.cpu().numpy(), ref + M0, ref_abs + np.abs(M0)) <= TOL_F32
    # a plane whose determined index is the trailing one has no contiguous fibres: refused
    with pytest.raises(dastac.DastacError):
        bad = dastac.Structure(st.fixed_index([ni + 1, nj + 1, nk + 1], 2, 0))
        dastac.contract("ijk,jr,kr->ir", bad, bad.empty_packed(), [torch.zeros((nj + 1, R), device="cuda"), torch.zeros((nk + 1, R), device="cuda")],
                        torch.zeros((ni + 1, R), device="cuda"))


@pytest.mark.parametrize("desc,C", [(st.dense_box([7, 13]), 5), (st.lower_triangle(100), 33), (st.offset_band(200, -30, 5), 64),
                                    (st.offset_band(64, 9, 9), 70), (_trapezoid(20, 70), 32), (st.fixed_index([30, 40], 0, 3), 17),
                                    (st.band_exact(90, 60), 40), (st.offset_band(300, -299, -1), 8)],
                         ids=lambda v: f"{v.name}{v.dims}" if hasattr(v, "name") else str(v))
def test_matmat_row_contiguous_classes(desc, C):
    """C = A B for the row-contiguous classes that the tiled band kernel does not take."""
    s = dastac.Structure(desc)
    M, N = desc.dims
    A = synth.dense(14, 0, (M, N))
    B = synth.dense(14, 1, (N, C))
    ref, ref_abs = oracle.matmat(desc, A, B)
    packed = packed_dev(s, oracle.pack(desc, A))
    out = torch.full((M, C), float("nan"), device="cuda")
    dastac.contract("ij,jc->ic", s, packed, [dev(B)], out)
    assert rel_err(out.cpu().numpy(), ref, ref_abs) <= TOL_F32
    C0 = synth.dense(14, 2, (M, C))
    out2 = torch.zeros((M, C + 3), device="cuda")[:, :C]          # padded row pitch of the result
    out2.copy_(dev(C0))
    dastac.contract("ij,jc->ic", s, packed, [dev(B)], out2, accumulate=True)
    assert rel_err(out2.cpu().numpy(), ref + C0, ref_abs + np.abs(C0)) <= TOL_F32


def _random_descriptors(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        kind = rng.integers(0, 6)
        if kind == 0:
            N = int(rng.integers(1, 700))
            a, b = sorted(int(v) for v in rng.integers(-N - 3, N + 4, 2))
            out.append(st.offset_band(N, a, b))
        elif kind == 1:
            out.append(st.upper_half_cube(int(rng.integers(1, 40)), int(rng.integers(1, 40)), int(rng.integers(1, 70))))
        elif kind == 2:
            out.append(st.tetrahedron(int(rng.integers(1, 60))))
        elif kind == 3:
            dims = [int(v) for v in rng.integers(1, 30, 3)]
            axis = int(rng.integers(0, 3))
            out.append(st.fixed_index(dims, axis, int(rng.integers(0, dims[axis]))))
        elif kind == 4:
            dims = [int(v) for v in rng.integers(1, 30, 3)]
            a, b = sorted(int(v) for v in rng.choice(3, 2, replace=False))
            out.append(st.equal_indices(dims, a, b))
        else:
            out.append(st.dense_box([int(v) for v in rng.integers(1, 50, int(rng.integers(1, 4)))]))
    return out


@pytest.mark.parametrize("sixteen", [False, True], ids=["f32", "bf16"])
def test_pack_unpack_random_structures(sixteen):
    """Forty random descriptors of the recognised families: pack and unpack bit for bit against the oracle."""
    tdt = torch.bfloat16 if sixteen else torch.float32
    idt = torch.int16 if sixteen else torch.int32
    for k, desc in enumerate(_random_descriptors(40, 123)):
        try:
            s = dastac.Structure(desc)
        except dastac.DastacError as e:
            assert e.status == 2
            continue
        bits = _bits(tuple(desc.dims), 50 + k, sixteen)
        d_dense = torch.from_numpy(bits.view(np.int16 if sixteen else np.int32)).cuda().view(tdt)
        packed = dastac.pack(s, d_dense)
        exp = oracle.pack(desc, bits)
        got = packed.view(idt).cpu().numpy().view(bits.dtype)
        assert np.array_equal(got[: s.nnz], exp), (desc.name, desc.dims, desc.meta)
        out = torch.full(desc.dims, float("nan"), dtype=tdt, device="cuda")
        dastac.unpack(s, packed, out)
        back = out.view(idt).cpu().numpy().view(bits.dtype)
        assert np.array_equal(back, oracle.unpack(desc, exp)), (desc.name, desc.dims, desc.meta)


def test_contractions_random_structures():
    """Random descriptors: matrix-vector, matrix x dense and Hadamard product wherever the structure's class has them."""
    done = {"mv": 0, "mm": 0, "had": 0}
    for k, desc in enumerate(_random_descriptors(60, 321)):
        try:
            s = dastac.Structure(desc)
        except dastac.DastacError:
            continue
        shape = tuple(desc.dims)
        if s.nnz == 0 or desc.name == "dense" and len(shape) == 1:
            continue
        A = synth.dense(60 + k, 0, shape)
        packed = packed_dev(s, oracle.pack(desc, A))
        # Hadamard product: every class and rank
        Cf = synth.dense(60 + k, 1, shape)
        ref, _ = oracle.hadamard(desc, A, Cf)
        out = s.empty_packed()
        dastac.contract({1: "i,i->i", 2: "ij,ij->ij", 3: "ijk,ijk->ijk"}[len(shape)], s, packed, [dev(Cf)], out, out_structure=s)
        assert np.array_equal(out.cpu().numpy()[: s.nnz], oracle.pack(desc, ref).astype(np.float32)), (desc.name, shape, desc.meta)
        done["had"] += 1
        if len(shape) != 2:
            continue
        M, N = shape
        x = synth.dense(60 + k, 2, (N,))
        r, ra = oracle.matvec(desc, A, x)
        y = torch.full((M,), float("nan"), device="cuda")
        try:
            dastac.contract("ij,j->i", s, packed, [dev(x)], y)
        except dastac.DastacError as e:
            assert e.status == 3
        else:
            assert rel_err(y.cpu().numpy(), r, ra) <= TOL_F32, (desc.name, shape, desc.meta)
            done["mv"] += 1
        B = synth.dense(60 + k, 3, (N, 19))
        r, ra = oracle.matmat(desc, A, B)
        Cm = torch.full((M, 19), float("nan"), device="cuda")
        try:
            dastac.contract("ij,jc->ic", s, packed, [dev(B)], Cm)
        except dastac.DastacError as e:
            assert e.status == 3
        else:
            assert rel_err(Cm.cpu().numpy(), r, ra) <= TOL_F32, (desc.name, shape, desc.meta)
            done["mm"] += 1
    assert done["mv"] >= 5 and done["mm"] >= 5 and done["had"] >= 30


@pytest.mark.parametrize("desc", [st.upper_triangle(1024), st.tetrahedron(512), st.upper_triangle(8192)],
                         ids=["triangle1024", "tetrahedron512", "triangle8192"])
def test_index_maps_exhaustive_against_the_oracle_at_kernel_sizes(desc):
    """Every point of the sets the kernels run on (all but the 2^31-point triangle): the device maps
    against the oracle's enumeration, bit for bit, in both directions."""
    s = dastac.Structure(desc)
    table = oracle.unrank_table(desc)                       # [count, rank]: the point at every position
    assert table.shape[0] == s.nnz
    idx = torch.from_numpy(table).cuda()
    positions = torch.arange(s.nnz, dtype=torch.int64, device="cuda")
    assert torch.equal(dastac.rank_batch(s, idx), positions)
    assert torch.equal(dastac.unrank_batch(s, positions), idx)
    if desc.rank == 2 and desc.dims[0] <= 1024:             # the whole box: points outside rank to -1
        full = oracle.rank_table(desc)
        N = desc.dims[0]
        ij = np.stack(np.meshgrid(np.arange(N), np.arange(N), indexing="ij"), -1).reshape(-1, 2).astype(np.int32)
        got = dastac.rank_batch(s, torch.from_numpy(ij).cuda()).cpu().numpy()
        assert np.array_equal(got, full.reshape(-1))


def test_expired_wait_is_reported_and_the_device_stays_usable():
    """The expiry path of the bounded waits, run on purpose: one warp waits about a millisecond on a
    barrier nothing arrives on, records its code and returns.  The host sees DASTAC_ERR_TIMEOUT with
    that code, the word clears, and the next kernels (a pack/unpack round trip through the bulk-copy
    kernels, which wait on barriers of the same kind) run as usual."""
    st0, _ = dastac.device_error(clear=True)          # whatever earlier tests left: cleared
    st1, word1 = dastac.device_error(clear=True)
    assert (st1, word1) == (0, 0)
    dastac.selftest_wait_expiry(2_000_000)
    st2, word2 = dastac.device_error(clear=False)
    assert st2 == 9 and word2 == 0x5354
    assert "wait" in dastac.status_string(st2)
    st3, word3 = dastac.device_error(clear=True)       # still set until cleared
    assert (st3, word3) == (9, 0x5354)
    assert dastac.device_error(clear=True) == (0, 0)
    N = 1500
    d = st.upper_triangle(N)
    s = dastac.Structure(d)
    A = synth.dense(7, 0, (N, N))
    pk = dastac.pack(s, dev(A))
    assert np.array_equal(pk.cpu().numpy()[: s.nnz], oracle.pack(d, A))
    assert np.array_equal(dastac.unpack(s, pk).cpu().numpy(), oracle.unpack(d, oracle.pack(d, A)))
    assert dastac.device_error(clear=True) == (0, 0)


FITTED = [
    st.anti_triangle(301),
    st.affine_set([150, 400], [[-2, 1, 0]], name="2i<=j"),
    st.affine_set([97, 97], [[-1, -1, 130], [1, 1, -40], [3, -1, 30]], name="polygon"),
    st.affine_set([40, 41, 45], [[-1, 1, 0, 0], [1, -1, 1, 0]], name="i<=j<=i+k"),
    st.affine_set([33, 47, 29], [[-1, -1, -1, 60]], name="i+j+k<=60"),
    st.affine_set([50, 50, 50], [[-1, 1, 0, 0], [0, -1, 1, 0], [1, 0, -1, 9]], name="i<=j<=k<=i+9"),
]


@pytest.mark.parametrize("desc", FITTED, ids=lambda d: f"{d.name}{d.dims}")
def test_fitted_maps_and_copies_on_the_device(desc):
    """Descriptors outside the recognised classes: device rank/unrank against the oracle's enumeration at
    every point of the box, pack and unpack bit for bit (fp32 with NaN payloads and -0, and bf16)."""
    s = dastac.Structure(desc)
    assert s.kind == dastac.KIND_GENERIC
    table = oracle.rank_table(desc)
    points = oracle.unrank_table(desc)
    assert s.nnz == len(points)
    box = np.stack(np.meshgrid(*[np.arange(n) for n in desc.dims], indexing="ij"), -1).reshape(-1, desc.rank).astype(np.int32)
    assert np.array_equal(dastac.rank_batch(s, torch.from_numpy(box).cuda()).cpu().numpy(), table.reshape(-1))
    pos = torch.arange(s.nnz, dtype=torch.int64, device="cuda")
    assert np.array_equal(dastac.unrank_batch(s, pos).cpu().numpy(), points)
    A = synth.dense(12, 0, tuple(desc.dims))
    bits = A.view(np.uint32).reshape(-1)
    bits[::7] = 0x7FC00123            # NaN with a payload
    bits[3::11] = 0x80000000          # -0.0
    pk = dastac.pack(s, dev(A))
    assert np.array_equal(pk.cpu().numpy().view(np.uint32)[: s.nnz], oracle.pack(desc, A).view(np.uint32))
    back = dastac.unpack(s, pk, torch.full(tuple(desc.dims), float("nan"), device="cuda"))
    assert np.array_equal(back.cpu().numpy().view(np.uint32), oracle.unpack(desc, oracle.pack(desc, A)).view(np.uint32))
    # bf16, and a dense tensor with padded strides
    H = synth.dense(12, 1, tuple(desc.dims), dist=synth.NORMAL, bf16=True)
    wide = torch.zeros(tuple(desc.dims[:-1]) + (desc.dims[-1] + 3,), dtype=torch.bfloat16, device="cuda")[..., : desc.dims[-1]]
    wide.copy_(dev(H, "bf16"))
    pkh = dastac.pack(s, wide)
    assert np.array_equal(pkh.view(torch.int16).cpu().numpy().view(np.uint16)[: s.nnz], oracle.pack(desc, H))
    backh = dastac.unpack(s, pkh)
    assert np.array_equal(backh.view(torch.int16).cpu().numpy().view(np.uint16), oracle.unpack(desc, oracle.pack(desc, H)))
    # a fitted map has no contraction kernels
    with pytest.raises(dastac.DastacError) as e:
        dastac.contract("ij,j->i" if desc.rank == 2 else "ijk,jr,kr->ir", s, pk,
                        [torch.zeros(desc.dims[1], device="cuda")] if desc.rank == 2 else
                        [torch.zeros((desc.dims[1], 4), device="cuda"), torch.zeros((desc.dims[2], 4), device="cuda")],
                        torch.zeros(desc.dims[0], device="cuda") if desc.rank == 2 else torch.zeros((desc.dims[0], 4), device="cuda"))
    assert e.value.status == 3


def _rule_reference(descs, A, x):
    """Sum over the summands of the masked definition (the regions of these rules are disjoint)."""
    ref, ref_abs = np.zeros(A.shape[0]), np.zeros(A.shape[0])
    for d in descs:
        r, ra = oracle.matvec(d, A, x)
        ref, ref_abs = ref + r, ref_abs + ra
    return ref, ref_abs


@pytest.mark.parametrize("name", ["strided_band", "leslie"])
def test_rule_with_several_summands_in_one_call(name):
    """A structured operand that is a sum of summands, each with its own compressed buffer (Section 4):
    the strided band j = i, j - i = +-s of Section 6.4 and the Leslie matrix of Table 1 (first row and
    sub-diagonal), packed and multiplied with a vector through one call each."""
    N = 1000
    if name == "strided_band":
        descs = [st.offset_band(N, 0, 0), st.offset_band(N, 37, 37), st.offset_band(N, -37, -37)]
    else:
        descs = [st.fixed_index([N, N], 0, 0), st.offset_band(N, -1, -1)]
    rule = dastac.Rule(descs)
    assert rule.n_buffers == len(descs)
    A = synth.dense(13, 0, (N, N))
    x = synth.dense(13, 1, (N,))
    bufs = rule.pack(dev(A))
    for d, b, v in zip(descs, bufs, rule.summands):
        assert np.array_equal(b.cpu().numpy()[: v.nnz], oracle.pack(d, A))
    ref, ref_abs = _rule_reference(descs, A, x)
    # the rule's value is the masked dense product as well
    mask = np.zeros((N, N), bool)
    for d in descs:
        mask |= oracle.rank_table(d) >= 0
    assert np.allclose((np.where(mask, A, 0).astype(np.float64) @ x.astype(np.float64)), ref, rtol=1e-12, atol=1e-12)
    y = torch.full((N,), float("nan"), device="cuda")
    n = rule.contract_workspace("ij,j->i", bufs, [dev(x)], y)
    ws = torch.empty(n, dtype=torch.uint8, device="cuda") if n else None
    rule.contract("ij,j->i", bufs, [dev(x)], y, workspace=ws)
    assert rel_err(y.cpu().numpy(), ref, ref_abs) <= TOL_F32
    y0 = synth.dense(13, 2, (N,))
    y2 = dev(y0)
    rule.contract("ij,j->i", bufs, [dev(x)], y2, accumulate=True, workspace=ws)
    assert rel_err(y2.cpu().numpy(), ref + y0, ref_abs + np.abs(y0)) <= TOL_F32
    # matrix times dense matrix through the same rule object
    B = synth.dense(13, 3, (N, 24))
    C = torch.full((N, 24), float("nan"), device="cuda")
    n = rule.contract_workspace("ij,jc->ic", bufs, [dev(B)], C)
    ws = torch.empty(n, dtype=torch.uint8, device="cuda") if n else None
    rule.contract("ij,jc->ic", bufs, [dev(B)], C, workspace=ws)
    refC, refC_abs = np.zeros((N, 24)), np.zeros((N, 24))
    for d in descs:
        r, ra = oracle.matmat(d, A, B)
        refC, refC_abs = refC + r, refC_abs + ra
    assert rel_err(C.cpu().numpy(), refC, refC_abs) <= TOL_F32


@pytest.mark.parametrize("n,R", [(1, 1), (2, 5), (7, 32), (31, 32), (32, 16), (33, 32), (64, 32), (65, 8), (127, 32),
                                 (128, 32), (129, 32), (130, 7), (200, 32), (257, 24), (300, 32)])
def test_mttkrp_split_precision_tensor_core_form(n, R):
    """The opt-in TF32 hi/lo form of the tetrahedral MTTKRP against the oracle, at the fp32 kernels' bound."""
    desc = st.tetrahedron(n)
    s = dastac.Structure(desc)
    T = synth.dense(3, 0, (n, n, n))
    B = synth.dense(3, 1, (n, R))
    C = synth.dense(3, 2, (n, R))
    ref, ref_abs = oracle.mttkrp(desc, T, B, C)
    packed = packed_dev(s, synth.tetrahedron_stream(3, 0, n))
    out = torch.full((n, R), float("nan"), device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    dastac.mttkrp_split_tf32(s, packed, dev(B), dev(C), out, err_word=err)
    assert int(err.item()) == 0
    assert rel_err(out.cpu().numpy(), ref, ref_abs) <= TOL_F32
    M0 = synth.dense(3, 3, (n, R))
    out2 = dev(M0)
    dastac.mttkrp_split_tf32(s, packed, dev(B), dev(C), out2, accumulate=True, err_word=err)
    assert int(err.item()) == 0
    assert rel_err(out2.cpu().numpy(), ref + M0, ref_abs + np.abs(M0)) <= TOL_F32
    # padded leading dimensions
    Bp = torch.zeros((n, R + 3), device="cuda")[:, :R]
    Bp.copy_(dev(B))
    Cp = torch.zeros((n, R + 1), device="cuda")[:, :R]
    Cp.copy_(dev(C))
    outp = torch.full((n, R + 5), float("nan"), device="cuda")[:, :R]
    dastac.mttkrp_split_tf32(s, packed, Bp, Cp, outp, err_word=err)
    assert int(err.item()) == 0
    assert rel_err(outp.cpu().numpy(), ref, ref_abs) <= TOL_F32


@pytest.mark.parametrize("exact", [False, True], ids=["diagonals", "exact"])
@pytest.mark.parametrize("N,w,C", [(2, 0, 1), (7, 0, 3), (40, 3, 5), (128, 32, 256), (129, 16, 257), (300, 32, 256),
                                   (1000, 7, 130), (2048, 32, 64), (200, 40, 33), (513, 90, 64), (190, 94, 12),
                                   (700, 200, 300)])
def test_band_matmat_split_precision_tensor_core_form(N, w, C, exact):
    """The opt-in TF32 hi/lo form of band x dense against the oracle, at the fp32 kernels' bound."""
    desc = st.band_exact(N, w) if exact else st.band(N, w)
    s = dastac.Structure(desc)
    A = synth.dense(1, 0, (N, N))
    B = synth.dense(1, 1, (N, C))
    ref, ref_abs = oracle.matmat(desc, A, B)
    # padding slots of the diagonal layout are poisoned: the product must not depend on them
    packed = packed_dev(s, oracle.pack(desc, A) if exact else synth.band_diagonals_stream(1, 0, N, w, pad_bits=0x7FC00000))
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.full((N, C), float("nan"), device="cuda")
    dastac.bandmm_split_tf32(s, packed, dev(B), out, err_word=err)
    assert int(err.item()) == 0
    assert rel_err(out.cpu().numpy(), ref, ref_abs) <= TOL_F32
    C0 = synth.dense(1, 2, (N, C))
    out2 = dev(C0)
    dastac.bandmm_split_tf32(s, packed, dev(B), out2, accumulate=True, err_word=err)
    assert int(err.item()) == 0
    assert rel_err(out2.cpu().numpy(), ref + C0, ref_abs + np.abs(C0)) <= TOL_F32
    # padded leading dimensions (rows of B and C not 16-byte aligned)
    Bp = torch.zeros((N, C + 3), device="cuda")[:, :C]
    Bp.copy_(dev(B))
    outp = torch.full((N, C + 5), float("nan"), device="cuda")[:, :C]
    dastac.bandmm_split_tf32(s, packed, Bp, outp, err_word=err)
    assert int(err.item()) == 0
    assert rel_err(outp.cpu().numpy(), ref, ref_abs) <= TOL_F32
    # the fp32 kernel and this form agree far inside the bound
    plain = torch.empty((N, C), device="cuda")
    dastac.contract("ij,jc->ic", s, packed, [dev(B)], plain)
    assert rel_err(out.cpu().numpy(), plain.cpu().numpy().astype(np.float64), ref_abs) <= TOL_F32


def test_band_matmat_split_precision_refusals():
    tri = dastac.Structure(st.upper_triangle(16))
    z = torch.zeros((16, 4), device="cuda")
    with pytest.raises(dastac.DastacError) as e:
        dastac.bandmm_split_tf32(tri, tri.empty_packed(), z, torch.zeros((16, 4), device="cuda"))
    assert e.value.status == 3


@pytest.mark.parametrize("M,N,Q,K", [(1, 1, 4, 1), (5, 7, 4, 6), (7, 5, 8, 5), (33, 40, 32, 32), (64, 64, 20, 12),
                                     (130, 130, 32, 64), (97, 97, 36, 33), (300, 300, 8, 40), (40, 50, 100, 32),
                                     (20, 30, 256, 7)])
def test_ttm_split_precision_tensor_core_form(M, N, Q, K):
    """The opt-in TF32 hi/lo form of the running example, packed in and out, at the fp32 kernels' bound."""
    dB, dA = st.upper_half_cube(M, N, Q), st.upper_half_cube(M, N, K)
    sB, sA = dastac.Structure(dB), dastac.Structure(dA)
    B = synth.dense(5, 0, (M, N, Q))
    C = synth.dense(5, 1, (K, Q))
    ref, ref_abs = oracle.ttm(dB, B, C)
    exp, exp_abs = oracle.pack(dA, ref), oracle.pack(dA, ref_abs)
    packedB = packed_dev(sB, synth.upper_half_cube_stream(5, 0, M, N, Q))
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = sA.empty_packed()
    out.fill_(float("nan"))
    dastac.ttm_split_tf32(sB, packedB, dev(C), out, err_word=err)
    assert int(err.item()) == 0
    assert rel_err(out.cpu().numpy()[: sA.nnz], exp, exp_abs) <= TOL_F32
    A0 = synth.dense(5, 2, (sA.nnz,))
    out2 = sA.empty_packed()
    out2[: sA.nnz] = dev(A0)
    dastac.ttm_split_tf32(sB, packedB, dev(C), out2, accumulate=True, err_word=err)
    assert int(err.item()) == 0
    assert rel_err(out2.cpu().numpy()[: sA.nnz], exp + A0, exp_abs + np.abs(A0)) <= TOL_F32
    # a padded leading dimension of C
    Cp = torch.zeros((K, Q + 3), device="cuda")[:, :Q]
    Cp.copy_(dev(C))
    out3 = sA.empty_packed()
    dastac.ttm_split_tf32(sB, packedB, Cp, out3, err_word=err)
    assert int(err.item()) == 0
    assert rel_err(out3.cpu().numpy()[: sA.nnz], exp, exp_abs) <= TOL_F32


def test_ttm_split_precision_refusals():
    tri = dastac.Structure(st.upper_triangle(16))
    with pytest.raises(dastac.DastacError) as e:
        dastac.ttm_split_tf32(tri, tri.empty_packed(), torch.zeros((4, 16), device="cuda"), torch.zeros(64, device="cuda"))
    assert e.value.status == 3
    odd = dastac.Structure(st.upper_half_cube(8, 8, 3))   # a packed row of 12 bytes is no tensor-map row
    with pytest.raises(dastac.DastacError) as e:
        dastac.ttm_split_tf32(odd, odd.empty_packed(), torch.zeros((4, 3), device="cuda"), torch.zeros(36 * 4, device="cuda"))
    assert e.value.status == 5


def test_mttkrp_split_precision_refusals():
    big = dastac.Structure(st.tetrahedron(513))
    z = torch.zeros((513, 4), device="cuda")
    with pytest.raises(dastac.DastacError) as e:
        dastac.mttkrp_split_tf32(big, big.empty_packed(), z, z, torch.zeros((513, 4), device="cuda"))
    assert e.value.status == 3
    tri = dastac.Structure(st.upper_triangle(16))
    with pytest.raises(dastac.DastacError) as e:
        dastac.mttkrp_split_tf32(tri, tri.empty_packed(), z[:16], z[:16], torch.zeros((16, 4), device="cuda"))
    assert e.value.status == 3
