"""The bf16 triangular x dense contraction through the entry point that takes no workspace and
allocates nothing (for callers that cannot obtain device memory around the call), checked against
the regular entry point on the same operands (same kernels, same tile order, no atomics: the bits
must agree) and against the oracle.  Collected last on purpose: a failure here leaves every other
test already run."""
import numpy as np
import pytest
import torch

import oracle
import synth
from synth import structures as st

from _util import TOL_BF16, dev, packed_dev, rel_err

pytestmark = pytest.mark.gpu

dastac = pytest.importorskip("paper_2407_13726_b200") if torch.cuda.is_available() else None


def _operands(N, C, seed):
    s = dastac.Structure(st.upper_triangle(N))
    scale = N ** -0.5
    packed = packed_dev(s, synth.upper_triangle_stream(seed, 0, N, dist=synth.NORMAL, scale=scale, bf16=True),
                        dtype=torch.bfloat16)
    B = dev(synth.dense(seed, 1, (N, C), dist=synth.NORMAL, scale=scale, bf16=True), "bf16")
    return s, packed, B


def _oracle_err(N, C, seed, got):
    """Forward error of `got` against the oracle on the same seeded operands (the parity tests' measure)."""
    scale = N ** -0.5
    A = synth.dense(seed, 0, (N, N), dist=synth.NORMAL, scale=scale, bf16=True)
    B = synth.dense(seed, 1, (N, C), dist=synth.NORMAL, scale=scale, bf16=True)
    ref, ref_abs = oracle.matmat(st.upper_triangle(N), A, B)
    return rel_err(got.cpu().numpy(), ref, ref_abs)


def _regular(s, packed, B, accumulate=False, out=None):
    N, C = B.shape
    if out is None:
        out = torch.full((N, C), float("nan"), device="cuda")
    n = dastac.contract_workspace("ij,jc->ic", s, packed, [B], out)
    ws = torch.empty(n, dtype=torch.uint8, device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    dastac.contract("ij,jc->ic", s, packed, [B], out, accumulate=accumulate, workspace=ws, err_word=err)
    assert int(err.item()) == 0
    return out


def _close(got, ref):
    """Same tolerance as the parity tests, with the regular entry point's |result| row sums as scale."""
    got, ref = got.double().cpu().numpy(), ref.double().cpu().numpy()
    scale = np.maximum(np.abs(ref).max(), 1e-30)
    return float(np.abs(got - ref).max() / scale) <= TOL_BF16


def test_two_calls_in_a_row_match_the_regular_entry_point():
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    # first call: several row blocks, ragged tail, B with a padded (16-byte multiple) pitch
    s1, p1, B1 = _operands(1000, 264, 41)
    Bp = torch.zeros((1000, 272), dtype=torch.bfloat16, device="cuda")[:, :264]
    Bp.copy_(B1)
    out1 = torch.full((1000, 264), float("nan"), device="cuda")
    dastac.trimm_bf16_noalloc(s1, p1, Bp, out1, err_word=err)
    # second call right behind it on the same stream: a smaller triangle, so the fixed array still
    # holds tiles of the first call beyond what this one rewrites
    s2, p2, B2 = _operands(300, 200, 42)
    out2 = torch.full((300, 200), float("nan"), device="cuda")
    dastac.trimm_bf16_noalloc(s2, p2, B2, out2, err_word=err)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    ref1, ref2 = _regular(s1, p1, B1), _regular(s2, p2, B2)
    assert _close(out1, ref1) and _close(out2, ref2)
    # stronger than the tolerance: the two entry points run the same kernels in the same order
    assert torch.equal(out1, ref1) and torch.equal(out2, ref2)
    # and against the oracle, element by element
    assert _oracle_err(1000, 264, 41, out1) <= TOL_BF16
    assert _oracle_err(300, 200, 42, out2) <= TOL_BF16
    # accumulate and the largest supported size
    s3, p3, B3 = _operands(dastac.NOALLOC_MAX_N, 256, 43)
    C0 = dev(synth.dense(43, 2, (dastac.NOALLOC_MAX_N, 256)))
    out3 = C0.clone()
    dastac.trimm_bf16_noalloc(s3, p3, B3, out3, accumulate=True, err_word=err)
    assert int(err.item()) == 0
    assert _close(out3, _regular(s3, p3, B3, accumulate=True, out=C0.clone()))


def test_rejects_what_the_fixed_array_cannot_hold():
    s, p, B = _operands(64, 72, 44)
    big = dastac.Structure(st.upper_triangle(dastac.NOALLOC_MAX_N + 1))
    out = torch.empty((dastac.NOALLOC_MAX_N + 1, 8), device="cuda")
    with pytest.raises(dastac.DastacError) as e:
        dastac.trimm_bf16_noalloc(big, big.empty_packed(torch.bfloat16),
                                  torch.zeros((dastac.NOALLOC_MAX_N + 1, 8), dtype=torch.bfloat16, device="cuda"), out)
    assert e.value.status == 7
    odd = torch.zeros((64, 77), dtype=torch.bfloat16, device="cuda")[:, :72]   # pitch 77: not 16-byte multiple
    with pytest.raises(dastac.DastacError) as e:
        dastac.trimm_bf16_noalloc(s, p, odd, torch.empty((64, 72), device="cuda"))
    assert e.value.status == 5
