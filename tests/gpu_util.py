"""Helpers of the GPU parity tests: move oracle-packed arrays to the device, compare with the
normalised tolerance (|gpu - oracle| <= tol * sum|terms| per element; exact zero where the sum is 0)."""
import numpy as np
import torch

import paper_2102_05187_b200 as comet

FP64_TOL = 1e-12


def dev(a, dtype=None):
    t = torch.as_tensor(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def upload_packed(pk):
    """oracle.Packed -> comet.SpTensor over device copies of the same arrays (caller-built descriptor)."""
    pos = [dev(p, torch.int32) if p.size else None for p in pk.pos]
    crd = [dev(c, torch.int32) if c.size else None for c in pk.crd]
    return comet.SpTensor.from_arrays(pk.dims, pk.mode_order, pk.attr, pos, crd, dev(pk.val, torch.float64))


def assert_close(got, want, norm, tol=FP64_TOL, what=""):
    got = got.detach().cpu().numpy() if isinstance(got, torch.Tensor) else np.asarray(got)
    want = np.asarray(want)
    norm = np.asarray(norm)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    err = np.abs(got - want)
    bad = err > tol * norm
    if bad.any():
        idx = np.unravel_index(np.argmax(err - tol * norm), err.shape)
        raise AssertionError(f"{what}: {int(bad.sum())} elements off; worst at {idx}: got {got[idx]!r} want "
                             f"{want[idx]!r} norm {norm[idx]!r}")
    rel = np.max(err / np.where(norm > 0, norm, 1.0)) if err.size else 0.0
    return float(rel)


def assert_equal_arrays(got, want, what=""):
    got = got.detach().cpu().numpy() if isinstance(got, torch.Tensor) else np.asarray(got)
    want = np.asarray(want)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    if got.dtype.kind == "f":
        same = np.array_equal(got.view(np.int64), want.astype(np.float64).view(np.int64))
    else:
        same = np.array_equal(got, want)
    assert same, f"{what}: arrays differ"
