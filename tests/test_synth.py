"""The synthetic generators: determinism, distinct in-range cells, the stated shape of each workload."""
import numpy as np
import pytest
import torch

import synth
from synth import rng


def _keys(case):
    key = torch.zeros(case.nnz, dtype=torch.int64)
    for m, d in enumerate(case.dims):
        key = key * d + case.coords[m].long()
    return key


@pytest.mark.parametrize("config", [1, 2, 3, 4, 5])
def test_cases_are_distinct_in_range_and_reproducible(config):
    a = synth.make(config, scale=1 / 256)
    b = synth.make(config, scale=1 / 256)
    assert a.nnz > 0 and torch.unique(_keys(a)).numel() == a.nnz
    for m, d in enumerate(a.dims):
        assert a.coords[m].dtype == torch.int32 and int(a.coords[m].min()) >= 0 and int(a.coords[m].max()) < d
        assert torch.equal(a.coords[m], b.coords[m])
    assert torch.equal(a.val, b.val) and float(a.val.abs().max()) < 1.0
    for k in a.dense:
        assert torch.equal(a.dense[k], b.dense[k])
    c = synth.make(config, scale=1 / 256, seed=7)
    assert not torch.equal(a.val[:16], c.val[:16])


def test_uniform_stream_statistics():
    u = rng.uniform(1, 2, 200_000)
    assert 0.0 <= float(u.min()) and float(u.max()) < 1.0
    assert abs(float(u.mean()) - 0.5) < 5e-3 and abs(float(u.var()) - 1 / 12) < 2e-3
    assert torch.equal(u[1000:1010], rng.uniform(1, 2, 10, offset=1000))       # counter-addressable
    p = rng.permutation(3, 4, 1000)
    assert torch.equal(torch.sort(p).values, torch.arange(1000))


def test_spmm_row_lengths_follow_clipped_zipf():
    case = synth.make(2, scale=1 / 16)
    lengths = torch.bincount(case.coords[0].long(), minlength=case.dims[0]).numpy()
    assert lengths.min() >= 1 and lengths.max() <= 10_000
    assert abs((lengths == 1).mean() - 1 / 1.8822296) < 0.01                   # P(1) = 1 / zeta(1.8)
    assert abs((lengths == 2).mean() - 2 ** -1.8 / 1.8822296) < 0.01


def test_ttm_fibers_are_geometric_mean_8():
    case = synth.make(4, scale=1 / 64)
    key = case.coords[0].long() * case.dims[1] + case.coords[1].long()
    _, counts = torch.unique(key, return_counts=True)
    assert abs(float(counts.double().mean()) - 8.0) < 0.3
    assert abs(float((counts == 1).double().mean()) - 1 / 8) < 0.01


def test_ttv_slice_sizes_are_power_law():
    case = synth.make(3, scale=1 / 64)
    sizes = np.sort(torch.bincount(case.coords[0].long()).numpy())[::-1]
    assert abs(sizes[0] / case.nnz - 1 / 1.6449) < 0.01                        # top slice = 1/zeta(2) of nnz
    assert abs(sizes[1] / sizes[0] - 0.25) < 0.01
