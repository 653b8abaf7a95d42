"""Pins of the oracle's batch normalisation + ReLU + residual (Sec. 2.1), independent of its own formulas."""
import numpy as np

import oracle


def _rand(shape, seed, scale=1.0, shift=0.0):
    return np.random.default_rng(seed).standard_normal(shape) * scale + shift


def test_forward_statistics_and_invariances():
    x = _rand((3, 4, 5, 6), 1, scale=2.5, shift=1.5)
    g, b = np.ones(6), np.zeros(6)
    y, mean, invstd, var = oracle.bn_relu_fwd(x, g, b, eps=1e-5, relu=False)
    flat = x.reshape(-1, 6)
    assert np.allclose(mean, flat.mean(axis=0), rtol=0, atol=1e-13)
    assert np.allclose(var, np.var(flat, axis=0), rtol=1e-13)           # library routine, biased variance
    assert np.allclose(invstd, 1 / np.sqrt(np.var(flat, axis=0) + 1e-5), rtol=1e-13)
    yf = y.reshape(-1, 6)
    assert np.abs(yf.mean(axis=0)).max() < 1e-13                           # normalised: zero mean ...
    assert np.allclose(yf.var(axis=0), var / (var + 1e-5), rtol=1e-12)     # ... and variance var/(var + eps)
    # a positive affine change of the input leaves the output unchanged up to eps
    y2, *_ = oracle.bn_relu_fwd(3.0 * x + 7.0, g, b, eps=0.0, relu=False)
    y1, *_ = oracle.bn_relu_fwd(x, g, b, eps=0.0, relu=False)
    assert np.allclose(y1, y2, atol=1e-12)
    # constant channel: xhat = 0, output = beta
    xc = np.full((2, 3, 3, 2), 4.25)
    yc, m, _, v = oracle.bn_relu_fwd(xc, np.array([2.0, -3.0]), np.array([0.5, -0.5]), relu=False)
    assert np.all(v == 0) and np.all(m == 4.25) and np.allclose(yc[..., 0], 0.5) and np.allclose(yc[..., 1], -0.5)


def test_scale_shift_residual_and_relu():
    x = _rand((2, 3, 3, 4), 2)
    g, b = _rand(4, 3), _rand(4, 4)
    r = _rand(x.shape, 5)
    y0, mean, invstd, _ = oracle.bn_relu_fwd(x, np.ones(4), np.zeros(4), relu=False)
    y1, *_ = oracle.bn_relu_fwd(x, g, b, residual=r, relu=False)
    assert np.allclose(y1, y0 * g + b + r, atol=1e-13)
    y2, *_ = oracle.bn_relu_fwd(x, g, b, residual=r, relu=True)
    assert np.array_equal(y2, np.maximum(y1, 0))


def test_running_statistics():
    mean, var = np.array([1.0, -2.0]), np.array([4.0, 0.25])
    rm, rv = oracle.bn_running_stats(np.zeros(2), np.ones(2), mean, var, M=10, momentum=0.1)
    assert np.allclose(rm, 0.1 * mean) and np.allclose(rv, 0.9 + 0.1 * var * 10 / 9)


def test_backward_against_finite_differences():
    """dx, dresidual, dgamma, dbeta of the analytic backward equal central differences of L = sum(y * G) through the
    oracle's forward (values kept away from the ReLU kink)."""
    rng = np.random.default_rng(7)
    x = rng.standard_normal((2, 3, 2, 3)) * 1.5
    g = rng.uniform(0.5, 1.5, 3)
    b = rng.uniform(0.2, 0.6, 3)
    r = rng.standard_normal(x.shape)
    G = rng.standard_normal(x.shape)
    eps = 1e-3

    def loss(x_, g_, b_, r_):
        y_, *_ = oracle.bn_relu_fwd(x_, g_, b_, eps=eps, residual=r_, relu=True)
        return float((y_ * G).sum())

    y, mean, invstd, _ = oracle.bn_relu_fwd(x, g, b, eps=eps, residual=r, relu=True)
    z = (x - mean) * invstd * g + b + r
    assert np.abs(z).min() > 1e-3                       # no element sits on the kink
    dx, dres, dgamma, dbeta = oracle.bn_relu_bwd(x, y, G, g, mean, invstd, relu=True)
    h = 1e-6
    for idx in np.ndindex(*x.shape):
        xp, xm = x.copy(), x.copy()
        xp[idx] += h
        xm[idx] -= h
        assert abs((loss(xp, g, b, r) - loss(xm, g, b, r)) / (2 * h) - dx[idx]) < 1e-6
        rp, rm_ = r.copy(), r.copy()
        rp[idx] += h
        rm_[idx] -= h
        assert abs((loss(x, g, b, rp) - loss(x, g, b, rm_)) / (2 * h) - dres[idx]) < 1e-6
    for c in range(3):
        gp, gm = g.copy(), g.copy()
        gp[c] += h
        gm[c] -= h
        assert abs((loss(x, gp, b, r) - loss(x, gm, b, r)) / (2 * h) - dgamma[c]) < 1e-6
        bp, bm = b.copy(), b.copy()
        bp[c] += h
        bm[c] -= h
        assert abs((loss(x, g, bp, r) - loss(x, g, bm, r)) / (2 * h) - dbeta[c]) < 1e-6


def test_backward_invariants():
    """The input gradient of a normalisation layer sums to zero per channel and (with eps = 0) is orthogonal to xhat."""
    x = _rand((4, 5, 5, 7), 11, scale=3.0, shift=-1.0)
    g, b = _rand(7, 12), _rand(7, 13)
    dy = _rand(x.shape, 14)
    y, mean, invstd, _ = oracle.bn_relu_fwd(x, g, b, eps=0.0, relu=True)
    dx, dres, dgamma, dbeta = oracle.bn_relu_bwd(x, y, dy, g, mean, invstd, relu=True)
    xhat = (x - mean) * invstd
    assert np.abs(dx.reshape(-1, 7).sum(axis=0)).max() < 1e-11
    assert np.abs((dx * xhat).reshape(-1, 7).sum(axis=0)).max() < 1e-10
    assert np.array_equal(dres, dy * (y > 0))
    assert np.allclose(dbeta, dres.reshape(-1, 7).sum(axis=0))
