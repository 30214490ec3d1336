"""Helpers shared by the GPU parity tests (host <-> device marshalling, comparisons)."""
import numpy as np


def to_dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def to_host(t):
    return t.detach().cpu().numpy()


def rel_err(got, want):
    """max|got - want| / max|want| (the tolerance definition used for every fp32 output), and max-abs."""
    got = np.asarray(got, np.float64); want = np.asarray(want, np.float64)
    if got.size == 0:
        return 0.0, 0.0
    mabs = float(np.abs(got - want).max())
    den = float(np.abs(want).max())
    return (mabs / den if den > 0 else mabs), mabs


def set_qparams(qp, scale, zero_point):
    """Fill a device qbp_qparams record by hand (scale, stored zero-point)."""
    import torch
    qp.view(torch.float32)[0, 0] = float(scale)
    qp[0, 1] = int(zero_point)
    return qp


def random_codes(shape, seed, lo=-128, hi=127, dtype=np.int8):
    return np.random.Generator(np.random.PCG64(seed)).integers(lo, hi + 1, size=shape).astype(dtype)


FP32_TOL = 1e-5       # relative, per tensor (per channel for Range BN): max|a-b| / max|b|
