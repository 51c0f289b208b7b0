"""Shared helpers of the GPU parity tests (no arithmetic of the method lives here)."""
import numpy as np
import torch

# Tolerances of the forward error |out - ref| / sum|products| per output element: fp32 kernels
# accumulate at most a few tens of thousands of fp32 products per output (unit roundoff 6e-8, sums
# re-associated in trees), the bf16 contraction multiplies exactly representable products and
# accumulates them in fp32, so both sit far below the stated bars.
TOL_F32 = 1e-5
TOL_BF16 = 2e-2


def rel_err(out, ref, ref_abs):
    """max_i |out_i - ref_i| / sum|terms|_i  (elements whose term sum is 0 must match exactly)."""
    out = np.asarray(out, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.asarray(ref_abs, dtype=np.float64)
    diff = np.abs(out - ref)
    zero = den == 0
    assert (diff[zero] == 0).all(), "element with no contributing term is not exactly zero"
    if zero.all():
        return 0.0
    return float((diff[~zero] / den[~zero]).max())


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype == "bf16":
        t = t.view(torch.int16).view(torch.bfloat16)
    return t.cuda()


def packed_dev(s, stream_values, dtype=torch.float32, poison_tail=True):
    """Device packed buffer of the structure's capacity holding `stream_values` (numpy)."""
    buf = s.empty_packed(dtype)
    src = torch.from_numpy(np.ascontiguousarray(stream_values).reshape(-1))
    if dtype == torch.bfloat16:
        src = src.view(torch.int16).view(torch.bfloat16)
    if poison_tail:
        buf.fill_(float("nan"))
    buf[: src.numel()] = src.cuda()
    return buf
