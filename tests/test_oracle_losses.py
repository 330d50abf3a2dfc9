"""Pins for the oracle's drafter objectives (Sec. 3.2) against library routines and closed forms."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import losses

RNG = np.random.default_rng(11)


def test_terms_against_torch_functional():
    p, r = RNG.standard_normal((3, 17, 24)), RNG.standard_normal((3, 17, 24))
    e1, e2 = RNG.standard_normal((3, 4, 8, 8)), RNG.standard_normal((3, 4, 8, 8))
    tp, tr = torch.from_numpy(p), torch.from_numpy(r)
    assert np.isclose(losses.noise_mse(e1, e2), F.mse_loss(torch.from_numpy(e1), torch.from_numpy(e2)).item(), rtol=1e-13)
    assert np.isclose(losses.feature_cosine(p, r, 0.0), (1 - F.cosine_similarity(tp, tr, dim=-1, eps=0.0)).mean().item(), rtol=1e-12)
    for beta in (0.1, 1.0, 2.5):
        assert np.isclose(losses.smooth_l1(p, r, beta), F.smooth_l1_loss(tp, tr, beta=beta).item(), rtol=1e-13)


def test_closed_forms():
    p = RNG.standard_normal((5, 8))
    assert losses.feature_cosine(p, 3.0 * p, 0.0) < 1e-15                      # parallel features
    assert np.isclose(losses.feature_cosine(p, -p, 0.0), 2.0)                  # opposite
    a, b = np.array([[1.0, 0.0]]), np.array([[0.0, 2.0]])
    assert np.isclose(losses.feature_cosine(a, b, 0.0), 1.0)                   # orthogonal
    assert np.isclose(losses.feature_cosine(a, 2 * a, 2.0), 1 - 2.0 / (2.0 + 2.0))     # the constant sits beside the product of norms
    # Smooth-L1: quadratic inside, linear outside, continuous at beta
    z = np.zeros((1, 1))
    assert np.isclose(losses.smooth_l1(z + 0.5, z, 2.0), 0.5 * 0.25 / 2.0) and np.isclose(losses.smooth_l1(z + 3.0, z, 2.0), 3.0 - 1.0)
    assert np.isclose(losses.smooth_l1(z + 2.0, z, 2.0), 1.0)
    assert losses.noise_mse(p, p) == 0.0 and np.isclose(losses.noise_mse(p + 2.0, p), 4.0)


def test_total_is_the_weighted_sum():
    p, r = RNG.standard_normal((2, 6, 10)), RNG.standard_normal((2, 6, 10))
    e1, e2 = RNG.standard_normal((2, 12)), RNG.standard_normal((2, 12))
    ln, lf, ls, tot = losses.free_loss(e1, e2, p, r, 0.5, 0.01, beta=0.7)
    assert np.isclose(tot, ln + 0.5 * lf + 0.01 * ls) and ln > 0 and 0 < lf < 2 and ls > 0
    # the noise term and the feature terms do not mix
    assert losses.free_loss(e1, e1, p, p, 0.5, 0.01, eps_cos=0.0)[3] < 1e-12
