"""Pins for the teacher top-K oracle: library routines, brute force, and the mass identity."""
import math

import numpy as np
import torch

from oracle.teacher_oracle import teacher_topk_oracle


def test_matches_torch_topk_and_logsumexp():
    rng = np.random.default_rng(1)
    h = rng.standard_normal((23, 12)); W = rng.standard_normal((157, 12))
    for tau in (1.0, 2.0):
        o = teacher_topk_oracle(h, W, 9, tau=tau)
        z = torch.tensor(h) @ torch.tensor(W).T
        v, i = torch.topk(z, 9, dim=1)
        np.testing.assert_allclose(o["val"], v.numpy(), rtol=1e-13)
        assert np.array_equal(o["idx"], i.numpy().astype(np.int32))      # no ties in random data
        np.testing.assert_allclose(o["lse"], torch.logsumexp(z / tau, 1).numpy(), rtol=1e-13)


def test_brute_force_selection_with_ties():
    h = np.array([[1.0, 0.0], [0.0, 1.0]])
    W = np.array([[2.0, 1.0], [2.0, 3.0], [0.5, 3.0], [2.0, -1.0], [-4.0, 3.0]])   # ties in both rows
    o = teacher_topk_oracle(h, W, 3)
    for t in range(2):
        z = [sum(h[t][j] * W[v][j] for j in range(2)) for v in range(5)]
        chosen = []
        for _ in range(3):                       # repeatedly take the largest, smallest index first on ties
            best = max((v for v in range(5) if v not in chosen), key=lambda v: (z[v], -v))
            chosen.append(best)
        assert list(o["idx"][t]) == chosen
        assert list(o["val"][t]) == [z[v] for v in chosen]
        assert abs(o["lse"][t] - math.log(sum(math.exp(x) for x in z))) < 1e-14
    assert list(o["idx"][0]) == [0, 1, 3] and list(o["idx"][1]) == [1, 2, 4]


def test_retained_mass_identity():
    rng = np.random.default_rng(2)
    h = rng.standard_normal((10, 8)); W = rng.standard_normal((64, 8))
    o = teacher_topk_oracle(h, W, 64)            # K = V: the record holds the whole distribution
    np.testing.assert_allclose(np.exp(o["val"] - o["lse"][:, None]).sum(1), 1.0, rtol=1e-13)
    o8 = teacher_topk_oracle(h, W, 8)
    mass = np.exp(o8["val"] - o8["lse"][:, None]).sum(1)
    assert np.all(mass < 1.0) and np.all(mass > 0.0)
    assert np.all(np.diff(o8["val"], axis=1) <= 0)
