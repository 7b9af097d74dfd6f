"""Pins for the oracle's LREC objective (Section 3.2, Eq. 1-2 of the paper): CPU only."""
import math

import numpy as np

from oracle import qlora_oracle as orc
from helpers import rel_err


def test_loss_against_plain_loops_and_closed_forms():
    rng = np.random.default_rng(3)
    T, V = 3, 16
    z, t = rng.standard_normal((T, V)) * 2, rng.standard_normal((T, V)) * 2
    labels = np.array([5, -1, 15])
    lkl, lce = 0.7, 1.3
    loss, _ = orc.lrec_loss(z, t, labels, lkl, lce)
    for tok in range(T):                                   # written straight from Eq. 1
        pz = [math.exp(v) for v in z[tok]]; sz = sum(pz); p = [v / sz for v in pz]
        qt = [math.exp(v) for v in t[tok]]; st = sum(qt); q = [v / st for v in qt]
        kl = sum(pi * math.log(pi / qi) for pi, qi in zip(p, q))
        ce = -math.log(p[labels[tok]]) if labels[tok] >= 0 else 0.0
        assert abs(loss[tok] - (lkl * kl + lce * ce)) < 1e-12
    # identical distributions: KL = 0; shifting logits by a constant per token changes nothing
    l0, g0 = orc.lrec_loss(z, z + 3.0, None, 1.0, 0.0)
    assert np.allclose(l0, 0, atol=1e-12) and np.allclose(g0, 0, atol=1e-12)
    l1, g1 = orc.lrec_loss(z + 7.0, t - 2.0, labels, lkl, lce)
    assert np.allclose(l1, loss, atol=1e-10)
    # uniform student over V, one-hot-ish label: CE = log V
    lu, _ = orc.lrec_loss(np.zeros((1, V)), np.zeros((1, V)), np.array([3]), 0.0, 1.0)
    assert abs(lu[0] - math.log(V)) < 1e-12
    # KL is non-negative and the gradient of each token sums to zero (softmax gauge)
    assert (orc.lrec_loss(z, t, None, 1.0, 0.0)[0] >= 0).all()
    assert np.allclose(orc.lrec_loss(z, t, labels, lkl, lce)[1].sum(axis=1), 0, atol=1e-12)


def test_loss_gradient_by_central_differences():
    rng = np.random.default_rng(4)
    T, V = 2, 12
    z, t = rng.standard_normal((T, V)), rng.standard_normal((T, V))
    labels = np.array([0, 7])
    lkl, lce = 0.9, 0.4
    _, grad = orc.lrec_loss(z, t, labels, lkl, lce)
    num = np.zeros_like(z)
    eps = 1e-5
    for idx in np.ndindex(*z.shape):
        up, dn = z.copy(), z.copy()
        up[idx] += eps
        dn[idx] -= eps
        num[idx] = (orc.lrec_loss(up, t, labels, lkl, lce)[0].sum() - orc.lrec_loss(dn, t, labels, lkl, lce)[0].sum()) / (2 * eps)
    assert rel_err(grad, num) < 1e-7
    # a label outside the vocabulary drops the cross-entropy term only
    la, ga = orc.lrec_loss(z, t, np.array([-1, 99]), lkl, lce)
    lb, gb = orc.lrec_loss(z, t, None, lkl, 0.0)
    assert np.array_equal(la, lb) and np.array_equal(ga, gb)
