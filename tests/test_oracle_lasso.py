"""Pins for the oracle's group-lasso + SGD step and zero-group detection."""
import os

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _fixture(name):
    out = {}
    for line in open(os.path.join(GOLD, name)):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        out[k] = [float(t) for t in v]
    return out


def test_hand_example_eq2():
    fx = _fixture("lasso_hand_example.txt")
    w = np.array(fx["W"], np.float32).reshape(2, 1, 1, 2)
    z = np.zeros_like(w)
    # lr = -1, mu = 0, g = 0, lambda = 1  =>  v' = dR/dW and w' = w + dR/dW
    w_new, v_new, s_out, s_in, reg = oracle.lasso_sgd(w, z, z, lam=1.0, lr=-1.0, mu=0.0)
    assert reg == fx["R"][0]
    np.testing.assert_allclose(v_new.ravel(), fx["dR"], rtol=0, atol=1e-15)
    np.testing.assert_allclose(s_out, [25.0, 0.0]) and np.testing.assert_allclose(s_in, [9.0, 16.0])
    np.testing.assert_allclose((w_new - w).ravel(), fx["dR"], rtol=0, atol=1e-15)
    assert oracle.lasso_penalty([w], [True], [True]) == fx["R"][0]


def test_sgd_two_steps():
    fx = _fixture("sgd_two_steps.txt")
    w0, g, v0, mu, lr = fx["in"]
    w = np.full((1, 1, 1, 1), w0, np.float32)
    gg = np.full((1, 1, 1, 1), g, np.float32)
    v = np.full((1, 1, 1, 1), v0, np.float32)
    w1, v1, *_ = oracle.lasso_sgd(w, gg, v, lam=0.0, lr=lr, mu=mu)
    assert abs(v1.item() - fx["step1"][0]) < 1e-7 and abs(w1.item() - fx["step1"][1]) < 1e-7
    w2, v2, *_ = oracle.lasso_sgd(w1.astype(np.float32), gg, v1.astype(np.float32), lam=0.0, lr=lr, mu=mu)
    assert abs(v2.item() - fx["step2"][0]) < 1e-6 and abs(w2.item() - fx["step2"][1]) < 1e-6


@pytest.mark.parametrize("reg_in,reg_out", [(True, True), (False, True), (True, False)])
def test_lasso_gradient_by_finite_differences(reg_in, reg_out):
    rng = np.random.default_rng(3)
    w = rng.standard_normal((3, 2, 2, 4)).astype(np.float32)
    z = np.zeros_like(w)
    lam = 0.37
    _, grad, *_ = oracle.lasso_sgd(w, z, z, lam=lam, lr=0.0, mu=0.0, reg_in=reg_in, reg_out=reg_out)
    R = lambda ww: lam * oracle.lasso_penalty([ww], [reg_in], [reg_out])
    h = 1e-5
    for idx in np.ndindex(w.shape):
        wp, wm = w.astype(np.float64), w.astype(np.float64)
        wp[idx] += h
        wm[idx] -= h
        fd = (R(wp) - R(wm)) / (2 * h)
        assert abs(fd - grad[idx]) < 1e-8, (idx, fd, grad[idx])


def test_weight_decay_and_momentum_terms():
    rng = np.random.default_rng(4)
    w, g, v = (rng.standard_normal((2, 1, 1, 3)).astype(np.float32) for _ in range(3))
    w_new, v_new, *_ = oracle.lasso_sgd(w, g, v, lam=0.0, lr=0.25, mu=0.5, wd=0.125)
    exp_v = 0.5 * v.astype(np.float64) + g + 0.125 * w.astype(np.float64)
    np.testing.assert_allclose(v_new, exp_v, rtol=0, atol=1e-15)
    np.testing.assert_allclose(w_new, w - 0.25 * exp_v, rtol=0, atol=1e-15)


def test_zero_group_stays_zero_through_step():
    rng = np.random.default_rng(5)
    w = rng.standard_normal((4, 3, 3, 5)).astype(np.float32)
    g = rng.standard_normal(w.shape).astype(np.float32)
    v = rng.standard_normal(w.shape).astype(np.float32)
    for t in (w, g, v):
        t[1] = 0
        t[:, :, :, 3] = 0
    w_new, v_new, *_ = oracle.lasso_sgd(w, g, v, lam=1e-2, lr=0.1, mu=0.9)
    assert np.all(w_new[1] == 0) and np.all(v_new[1] == 0) and np.all(w_new[..., 3] == 0) and np.all(v_new[..., 3] == 0)


def test_set_coeff_roundtrip():
    lam = oracle.set_coeff(loss1=2.3, reg_sum=812.5, ratio=0.25)
    assert abs(lam * 812.5 / (2.3 + lam * 812.5) - 0.25) < 1e-15


def test_cross_entropy_closed_forms():
    """Pins of the classification loss used by Eq. 3: uniform logits give ln(classes); a one-hot limit gives 0; the loss
    does not move when a constant is added to a row; two classes reduce to the logistic loss log(1 + exp(-d))."""
    rng = np.random.default_rng(5)
    n, k = 7, 11
    lab = rng.integers(0, k, n)
    assert abs(oracle.cross_entropy(np.zeros((n, k)), lab) - np.log(k)) < 1e-15
    z = np.full((n, k), -800.0)
    z[np.arange(n), lab] = 0.0
    assert oracle.cross_entropy(z, lab) == 0.0
    z = rng.standard_normal((n, k)) * 4
    shift = rng.standard_normal((n, 1)) * 100
    assert abs(oracle.cross_entropy(z, lab) - oracle.cross_entropy(z + shift, lab)) < 1e-12
    d = rng.standard_normal(n) * 3                       # two classes: margin d of the true class
    z2 = np.stack([d, np.zeros(n)], axis=1)
    assert abs(oracle.cross_entropy(z2, np.zeros(n, int)) - np.mean(np.log1p(np.exp(-d)))) < 1e-14
    # brute force on a tiny case: exponentials written out
    z3 = np.array([[1.0, 2.0, 0.5], [0.0, -1.0, 3.0]])
    e = np.exp(z3)
    ref = -(np.log(e[0, 1] / e[0].sum()) + np.log(e[1, 0] / e[1].sum())) / 2
    assert abs(oracle.cross_entropy(z3, [1, 0]) - ref) < 1e-14


def test_set_coeff_reaches_the_requested_share_on_a_model():
    """Eq. 3 end to end on a small random model: with lambda from set_coeff the lasso term is `ratio` of the total loss."""
    rng = np.random.default_rng(9)
    ws = [rng.standard_normal((6, 3, 3, 4)), rng.standard_normal((5, 1, 1, 6))]
    R = oracle.lasso_penalty(ws, reg_in=[False, True], reg_out=[True, True])
    z = rng.standard_normal((8, 10))
    loss = oracle.cross_entropy(z, rng.integers(0, 10, 8))
    for ratio in (0.2, 0.25):
        lam = oracle.set_coeff(loss, R, ratio)
        assert abs(lam * R / (loss + lam * R) - ratio) < 1e-14 and lam > 0


def test_detection_boundaries():
    thr = np.float32(1e-4)
    w = np.ones((6, 1, 2, 5), np.float32)
    w[0] = thr                                   # max exactly at the threshold: kept (strict <)
    w[1] = np.nextafter(thr, np.float32(0))      # just below: zero
    w[2] = 0.0
    w[2, 0, 1, 3] = np.nan                       # NaN member: kept
    w[3] = 0.0                                   # all-zero: zero
    w[4] = -0.99e-4                              # sign does not matter
    w[5, 0, 0, :] = 0.0
    w[5, 0, 1, 2] = -1e-3                        # one big member keeps the group
    w[:, :, :, 4] = 0.5e-4                       # an input-channel group below threshold everywhere
    zo, zi = oracle.find_zero_groups(w, float(thr))
    assert zo.tolist() == [0, 1, 0, 1, 1, 0]
    assert zi.tolist() == [0, 0, 0, 0, 1]


def test_detection_brute_force_and_degenerate_shapes():
    rng = np.random.default_rng(6)
    for (K, R, C) in [(1, 1, 1), (1, 3, 4), (5, 1, 1), (7, 3, 6)]:
        w = rng.standard_normal((K, R, R, C)).astype(np.float32)
        w[rng.random(w.shape) < 0.6] = 0.5e-4
        if K > 2:
            w[1] = 1e-5
        zo, zi = oracle.find_zero_groups(w, 1e-4)
        a = np.abs(w)
        assert zo.tolist() == [int(a[k].max() < np.float32(1e-4)) for k in range(K)]
        assert zi.tolist() == [int(a[..., c].max() < np.float32(1e-4)) for c in range(C)]
