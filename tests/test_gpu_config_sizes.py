"""GPU parity at the full sizes of the five configurations, in the launch configuration the
benchmark times.  The oracle evaluates a sample of output rows one by one (rows spread over the
outer index, the first and last rows, and one row in every 128-row block for the tensor-core
kernel); the kernel's full output is additionally checked for finiteness."""
import numpy as np
import pytest
import torch

import oracle
import synth
from synth import structures as st

from _util import TOL_BF16, TOL_F32, dev, rel_err

pytestmark = pytest.mark.gpu

dastac = pytest.importorskip("paper_2407_13726_b200") if torch.cuda.is_available() else None


def _rows(n, k, extra=()):
    sel = set(np.linspace(0, n - 1, k).astype(np.int64).tolist()) | {0, n - 1} | set(extra)
    return np.array(sorted(sel), dtype=np.int64)


def _packed(s, fill, dtype=torch.float32):
    """Device packed buffer filled by the generator's stream (host staging buffer is pinned)."""
    np_dt = np.uint16 if dtype == torch.bfloat16 else np.float32
    host = np.zeros(s.capacity(dtype), np_dt)
    fill(host)
    t = torch.from_numpy(host)
    if dtype == torch.bfloat16:
        t = t.view(torch.int16).view(torch.bfloat16)
    return t.cuda()


def _ws(expr, s, packed, ins, out, batch=1):
    n = dastac.contract_workspace(expr, s, packed, ins, out, batch=batch)
    return torch.empty(n, dtype=torch.uint8, device="cuda") if n else None


def test_config1_trmv_n1024_single_and_batch512():
    N, batch = 1024, 512
    desc = st.upper_triangle(N)
    s = dastac.Structure(desc)
    A = synth.dense(0, 0, (N, N))
    x = synth.dense(0, 1, (N,))
    ref, ref_abs = oracle.matvec(desc, A, x)
    packed = _packed(s, lambda h: synth.upper_triangle_stream(0, 0, N, out=h))
    y = torch.full((N,), float("nan"), device="cuda")
    dastac.contract("ij,j->i", s, packed, [dev(x)], y)
    assert rel_err(y.cpu().numpy(), ref, ref_abs) <= TOL_F32
    # the batched launch: instance b holds tensors 2b+2 / 2b+3 of seed 0; instances 0, 255 and 511 are checked
    cap = s.capacity(torch.float32)
    hp = np.zeros((batch, cap), np.float32)
    hx = np.empty((batch, N), np.float32)
    for b in range(batch):
        synth.upper_triangle_stream(0, 2 * b + 2, N, out=hp[b])
        hx[b] = synth.dense(0, 2 * b + 3, (N,))
    yb = torch.full((batch, N), float("nan"), device="cuda")
    dastac.contract("ij,j->i", s, torch.from_numpy(hp).cuda(), [torch.from_numpy(hx).cuda()], yb, batch=batch)
    got = yb.cpu().numpy()
    assert np.isfinite(got).all()
    for b in (0, 255, 511):
        r, ra = oracle.matvec(desc, synth.dense(0, 2 * b + 2, (N, N)), hx[b])
        assert rel_err(got[b], r, ra) <= TOL_F32


def test_config2_band_n32768_w32_c256():
    N, w, C = 32768, 32, 256
    desc = st.band(N, w)
    s = dastac.Structure(desc)
    B = synth.dense(1, 1, (N, C))
    packed = _packed(s, lambda h: synth.band_diagonals_stream(1, 0, N, w, pad_bits=0x7FC00000, out=h))
    out = torch.full((N, C), float("nan"), device="cuda")
    dastac.contract("ij,jc->ic", s, packed, [dev(B)], out)
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    sel = _rows(N, 300, extra=range(0, 40))
    sel = np.union1d(sel, np.arange(N - 40, N))
    Ar = np.stack([synth.linear_slice(1, 0, int(i) * N, N) for i in sel])
    ref, ref_abs = oracle.matmat(desc, Ar, B, sel=sel)
    assert rel_err(got[sel], ref, ref_abs) <= TOL_F32


def test_config2_band_split_precision_tensor_core_form():
    """Configuration 2 through the opt-in TF32 hi/lo entry point, same sampled rows and bound."""
    N, w, C = 32768, 32, 256
    desc = st.band(N, w)
    s = dastac.Structure(desc)
    B = synth.dense(1, 1, (N, C))
    packed = _packed(s, lambda h: synth.band_diagonals_stream(1, 0, N, w, pad_bits=0x7FC00000, out=h))
    out = torch.full((N, C), float("nan"), device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    dastac.bandmm_split_tf32(s, packed, dev(B), out, err_word=err)
    assert int(err.item()) == 0
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    sel = _rows(N, 300, extra=range(0, 40))
    sel = np.union1d(sel, np.arange(N - 40, N))
    Ar = np.stack([synth.linear_slice(1, 0, int(i) * N, N) for i in sel])
    ref, ref_abs = oracle.matmat(desc, Ar, B, sel=sel)
    assert rel_err(got[sel], ref, ref_abs) <= TOL_F32


def test_config3_symv_n65536():
    N = 65536
    desc = st.upper_triangle(N, symmetric=True)
    s = dastac.Structure(desc)
    assert s.nnz == 2_147_516_416
    x = synth.dense(2, 1, (N,), dist=synth.NORMAL)
    packed = _packed(s, lambda h: synth.upper_triangle_stream(2, 0, N, dist=synth.NORMAL, out=h))
    y = torch.full((N,), float("nan"), device="cuda")
    xd = dev(x)
    dastac.contract("ij,j->i", s, packed, [xd], y, workspace=_ws("ij,j->i", s, packed, [xd], y))
    got = y.cpu().numpy()
    assert np.isfinite(got).all()
    sel = _rows(N, 96, extra=(1, 63, 64, 1023, 1024, 32767, 32768, N - 2))
    Sr = np.stack([synth.symmetric_row(2, 0, N, int(i), dist=synth.NORMAL) for i in sel])
    ref, ref_abs = oracle.matvec(st.dense_box([N, N]), Sr, x, sel=sel)
    assert rel_err(got[sel], ref, ref_abs) <= TOL_F32


def test_config4_mttkrp_n512_r32():
    n, R = 512, 32
    desc = st.tetrahedron(n)
    s = dastac.Structure(desc)
    assert s.nnz == 22_500_864
    B = synth.dense(3, 1, (n, R))
    C = synth.dense(3, 2, (n, R))
    packed = _packed(s, lambda h: synth.tetrahedron_stream(3, 0, n, out=h))
    out = torch.full((n, R), float("nan"), device="cuda")
    ins = [dev(B), dev(C)]
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    dastac.contract("ijk,jr,kr->ir", s, packed, ins, out, workspace=_ws("ijk,jr,kr->ir", s, packed, ins, out),
                    err_word=err)
    assert int(err.item()) == 0
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    sel = _rows(n, 20, extra=(1, 31, 32, 33, 479, 480, 510))
    Ts = np.stack([synth.linear_slice(3, 0, int(i) * n * n, n * n).reshape(n, n) for i in sel])
    ref, ref_abs = oracle.mttkrp(desc, Ts, B, C, sel=sel)
    assert rel_err(got[sel], ref, ref_abs) <= TOL_F32


def test_config4_mttkrp_split_precision_tensor_core_form():
    """The opt-in TF32 hi/lo form at the configuration's size, same sampled slabs, same bound."""
    n, R = 512, 32
    desc = st.tetrahedron(n)
    s = dastac.Structure(desc)
    B = synth.dense(3, 1, (n, R))
    C = synth.dense(3, 2, (n, R))
    packed = _packed(s, lambda h: synth.tetrahedron_stream(3, 0, n, out=h))
    out = torch.full((n, R), float("nan"), device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    dastac.mttkrp_split_tf32(s, packed, dev(B), dev(C), out, err_word=err)
    assert int(err.item()) == 0
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    sel = _rows(n, 20, extra=(1, 31, 32, 33, 127, 128, 129, 383, 384, 479, 480, 510))
    Ts = np.stack([synth.linear_slice(3, 0, int(i) * n * n, n * n).reshape(n, n) for i in sel])
    ref, ref_abs = oracle.mttkrp(desc, Ts, B, C, sel=sel)
    assert rel_err(got[sel], ref, ref_abs) <= TOL_F32


@pytest.mark.parametrize("n,R", [(700, 32), (1100, 24), (1500, 32)])
def test_mttkrp_beyond_config4(n, R):
    """Sizes at which the factor matrix leaves room for fewer warps per block (n = 1100) or no longer
    fits in shared memory at all (n = 1500: the kernel that stages 32 x 32 pieces per warp)."""
    desc = st.tetrahedron(n)
    s = dastac.Structure(desc)
    B = synth.dense(3, 1, (n, R))
    C = synth.dense(3, 2, (n, R))
    packed = _packed(s, lambda h: synth.tetrahedron_stream(3, 0, n, out=h))
    out = torch.full((n, R), float("nan"), device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    ins = [dev(B), dev(C)]
    dastac.contract("ijk,jr,kr->ir", s, packed, ins, out, workspace=_ws("ijk,jr,kr->ir", s, packed, ins, out),
                    err_word=err)
    assert int(err.item()) == 0
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    sel = _rows(n, 6, extra=(1, 63, 64, n - 2))
    Ts = np.stack([synth.linear_slice(3, 0, int(i) * n * n, n * n).reshape(n, n) for i in sel])
    ref, ref_abs = oracle.mttkrp(desc, Ts, B, C, sel=sel)
    assert rel_err(got[sel], ref, ref_abs) <= TOL_F32


def test_config5_triangular_bf16_n8192():
    N = 8192
    desc = st.upper_triangle(N)
    s = dastac.Structure(desc)
    assert s.nnz == 33_558_528
    sc = N ** -0.5
    B = synth.dense(4, 1, (N, N), dist=synth.NORMAL, scale=sc, bf16=True)
    packed = _packed(s, lambda h: synth.upper_triangle_stream(4, 0, N, dist=synth.NORMAL, scale=sc, bf16=True, out=h),
                     dtype=torch.bfloat16)
    Bd = dev(B, "bf16")
    out = torch.full((N, N), float("nan"), device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    dastac.contract("ij,jc->ic", s, packed, [Bd], out, workspace=_ws("ij,jc->ic", s, packed, [Bd], out), err_word=err)
    assert int(err.item()) == 0
    assert bool(torch.isfinite(out).all())
    # one row in every 128-row block (at a varying place inside the block), plus the ends
    sel = np.array(sorted({128 * b + (37 * b) % 128 for b in range(N // 128)} | {0, 127, 128, N - 129, N - 1}), dtype=np.int64)
    A = np.stack([synth.linear_slice(4, 0, int(i) * N, N, dist=synth.NORMAL, scale=sc, bf16=True) for i in sel])
    ref, ref_abs = oracle.matmat(desc, A, B, sel=sel)
    got = out[torch.from_numpy(sel).cuda()].cpu().numpy()
    assert rel_err(got, ref, ref_abs) <= TOL_BF16
    # pack / unpack at this size: bit exact against the generator's stream and its dense tensor on sampled rows
    dense = dastac.unpack(s, packed)
    rows = dense[torch.from_numpy(sel).cuda()].view(torch.int16).cpu().numpy().view(np.uint16)
    for r, i in enumerate(sel):
        exp = A[r].copy()
        exp[: int(i)] = 0
        assert np.array_equal(rows[r], exp)
    repacked = dastac.pack(s, dense)
    assert torch.equal(repacked.view(torch.int16)[: s.nnz], packed.view(torch.int16)[: s.nnz])


@pytest.mark.parametrize("tensor_cores", [False, True], ids=["fp32", "split_tf32"])
def test_widened_row_ttm_n1024_q32_k32(tensor_cores):
    """The tensor-times-matrix running example at the size the benchmark times: sampled slabs i of
    the packed result (slab i is the contiguous run of positions that starts at (i, i, 0)); through
    dastac_contract and through the opt-in tensor-core entry point."""
    N, Q, K = 1024, 32, 32
    dB, dA = st.upper_half_cube(N, N, Q), st.upper_half_cube(N, N, K)
    sB, sA = dastac.Structure(dB), dastac.Structure(dA)
    assert sA.nnz == N * (N + 1) // 2 * K
    C = synth.dense(5, 1, (K, Q))
    packedB = _packed(sB, lambda h: synth.upper_half_cube_stream(5, 0, N, N, Q, out=h))
    out = torch.full((sA.capacity(torch.float32),), float("nan"), device="cuda")
    if tensor_cores:
        dastac.ttm_split_tf32(sB, packedB, dev(C), out)
    else:
        dastac.contract("ijl,kl->ijk", sB, packedB, [dev(C)], out, out_structure=sA)
    got = out.cpu().numpy()[: sA.nnz]
    assert np.isfinite(got).all()
    sel = _rows(N, 12, extra=(1, 255, 256, 257, N - 2))
    Bs = np.stack([synth.linear_slice(5, 0, int(i) * N * Q, N * Q).reshape(N, Q) for i in sel])
    ref, ref_abs = oracle.ttm(dB, Bs, C, sel=sel)
    # where slab i starts in the packed result: device and host maps must agree, the oracle counts it for two slabs
    starts = dastac.rank_batch(sA, torch.tensor([[int(i), int(i), 0] for i in sel], dtype=torch.int32).cuda()).cpu().numpy()
    for probe in (0, len(sel) // 2):
        assert starts[probe] == oracle.rank_point(dA, (int(sel[probe]), int(sel[probe]), 0))
    for s, i in enumerate(sel):
        n_el = (N - int(i)) * K
        seg = got[starts[s]: starts[s] + n_el]
        assert rel_err(seg, ref[s, int(i):, :].reshape(-1), ref_abs[s, int(i):, :].reshape(-1)) <= TOL_F32


def test_widened_row_exact_band_n32768_w32_c256():
    """Configuration 2's product over the exact (un-padded) band layout, on sampled rows."""
    N, w, C = 32768, 32, 256
    desc = st.band_exact(N, w)
    s = dastac.Structure(desc)
    assert s.nnz == 65 * N - 32 * 33 == s.slots
    B = synth.dense(1, 1, (N, C))
    packed = _packed(s, lambda h: synth.band_rows_stream(1, 0, N, w, out=h))
    out = torch.full((N, C), float("nan"), device="cuda")
    dastac.contract("ij,jc->ic", s, packed, [dev(B)], out)
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    sel = np.union1d(_rows(N, 200, extra=range(0, 40)), np.arange(N - 40, N))
    Ar = np.stack([synth.linear_slice(1, 0, int(i) * N, N) for i in sel])
    ref, ref_abs = oracle.matmat(desc, Ar, B, sel=sel)
    assert rel_err(got[sel], ref, ref_abs) <= TOL_F32


def test_widened_row_moment2_m100000_n4096():
    """Degree-2 moments of 100000 samples x 4096 features (the sample count of the paper's PR2 runs),
    packed symmetric output, on sampled rows of the result."""
    M, n = 100000, 4096
    desc = st.upper_triangle(n, symmetric=True)
    sA = dastac.Structure(desc)
    B = synth.dense(6, 0, (M, n), dist=synth.NORMAL, bf16=True)
    Bd = dev(B, "bf16")
    out = torch.full((sA.capacity(torch.float32),), float("nan"), device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    dastac.contract("xi,xj->ij", None, Bd, [Bd], out, out_structure=sA, err_word=err)
    assert int(err.item()) == 0
    got = out.cpu().numpy()[: sA.nnz]
    assert np.isfinite(got).all()
    sel = np.array([0, 127, 128, 255, 256, 1000, 2047, 2048, 3839, 3840, n - 2, n - 1], dtype=np.int64)
    ref, ref_abs = oracle.moment2(desc, B, sel=sel)
    for s, i in enumerate(sel):
        start = oracle.rank_point(desc, (int(i), int(i))) if s < 2 else int(i) * n - int(i) * (int(i) - 1) // 2
        seg = got[start: start + n - int(i)]
        # 100000 same-sign terms on the diagonal, accumulated in fp32 inside the tensor core: the error
        # grows with the length of the sum (about 5e-4 here), still far inside the bf16 bar
        assert rel_err(seg, ref[s, int(i):], ref_abs[s, int(i):]) <= TOL_BF16
        assert rel_err(seg, ref[s, int(i):], ref_abs[s, int(i):]) <= 2e-3


@pytest.mark.parametrize("M,n", [(10000, 256), (60000, 200)], ids=["m10000_n256", "m60000_n200"])
def test_widened_row_moment3(M, n):
    """Degree-3 moments of 10000 samples (the sample count of the paper's PR3 runs) x 256 features, and
    a taller, narrower case with an odd number of K blocks and a ragged last row block; sampled slabs
    of the packed tetrahedron."""
    desc = st.tetrahedron(n)
    sA = dastac.Structure(desc)
    B = synth.dense(9, 0, (M, n), dist=synth.NORMAL, bf16=True)
    Bd = dev(B, "bf16")
    out = torch.full((sA.capacity(torch.float32),), float("nan"), device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    nws = dastac.contract_workspace("xi,xj,xk->ijk", None, Bd, [Bd, Bd], out, out_structure=sA)
    ws = torch.empty(max(nws, 1), dtype=torch.uint8, device="cuda")
    dastac.contract("xi,xj,xk->ijk", None, Bd, [Bd, Bd], out, out_structure=sA, workspace=ws, err_word=err)
    assert int(err.item()) == 0
    got = out.cpu().numpy()[: sA.nnz]
    assert np.isfinite(got).all()
    sel = np.array([0, 1, 51, 52, 103, 104, 127, 128, n - 2, n - 1] if n == 256 else [0, 51, 52, 155, 156, n - 1], dtype=np.int64)
    ref, ref_abs = oracle.moment3(desc, B, sel=sel)
    for s, i in enumerate(sel):
        i = int(i)
        start = oracle.rank_point(desc, (i, i, i))
        m = n - i
        exp = np.concatenate([ref[s, j, j:] for j in range(i, n)])
        exp_abs = np.concatenate([ref_abs[s, j, j:] for j in range(i, n)])
        assert exp.size == m * (m + 1) // 2
        assert rel_err(got[start: start + exp.size], exp, exp_abs) <= 4e-3 <= TOL_BF16


def test_large_triangular_matvec_n65536():
    """The plain upper-triangular product at the size where it runs on the streaming kernel of the
    symmetric product (without the mirrored half): sampled rows."""
    N = 65536
    desc = st.upper_triangle(N)
    s = dastac.Structure(desc)
    x = synth.dense(2, 1, (N,), dist=synth.NORMAL)
    packed = _packed(s, lambda h: synth.upper_triangle_stream(2, 0, N, dist=synth.NORMAL, out=h))
    y = torch.full((N,), float("nan"), device="cuda")
    dastac.contract("ij,j->i", s, packed, [dev(x)], y)
    got = y.cpu().numpy()
    assert np.isfinite(got).all()
    sel = _rows(N, 64, extra=(1, 127, 128, 32767, 32768, N - 2))
    Ar = np.stack([synth.linear_slice(2, 0, int(i) * N, N, dist=synth.NORMAL) for i in sel])
    ref, ref_abs = oracle.matvec(desc, Ar, x, sel=sel)
    assert rel_err(got[sel], ref, ref_abs) <= TOL_F32
