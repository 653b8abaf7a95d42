"""Pins for the oracle's convolutions: each check is something the mathematics fixes,
evaluated independently of the loops under test."""
import numpy as np
import pytest

import oracle
from paper_1901_09290_b200 import workloads as W


def _bf(a):
    return oracle.round_bf16(a)


def _rand(shape, seed):
    return np.asarray(oracle.round_bf16(np.random.default_rng(seed).standard_normal(shape).astype(np.float32)),
                      np.float32)


def test_bf16_rounding_rne():
    # 1 + 2^-8 is exactly half-way between bf16 neighbours 1 and 1+2^-7: ties go to even (1.0)
    assert oracle.round_bf16(np.float32(1.0 + 2.0 ** -8))[()] == 1.0
    # 1 + 3*2^-8 is half-way between 1+2^-7 (odd mantissa) and 1+2^-6 (even): rounds up
    assert oracle.round_bf16(np.float32(1.0 + 3 * 2.0 ** -8))[()] == 1.0 + 2.0 ** -6
    assert oracle.round_bf16(np.float32(1.0 + 2.0 ** -8 + 2.0 ** -12))[()] == 1.0 + 2.0 ** -7
    assert np.isnan(oracle.round_bf16(np.float32(np.nan))[()])
    x = _rand((1000,), 1)
    assert np.array_equal(oracle.round_bf16(x), x.astype(np.float64))      # idempotent


def test_fwd_1x1_is_a_gemm():
    N, H, Wd, C, K = 3, 5, 7, 11, 6
    x, w = _rand((N, H, Wd, C), 2), _rand((K, 1, 1, C), 3)
    y = oracle.conv_fwd(x, w, 1, 0)
    ref = x.astype(np.float64).reshape(-1, C) @ w.astype(np.float64).reshape(K, C).T
    np.testing.assert_allclose(y.reshape(-1, K), ref, rtol=0, atol=1e-12)


def test_fwd_rounds_inputs_to_bf16():
    x = np.full((1, 1, 1, 1), 1.0 + 2.0 ** -8 + 2.0 ** -12, np.float32)
    w = np.full((1, 1, 1, 1), 3.0, np.float32)
    assert oracle.conv_fwd(x, w)[0, 0, 0, 0] == 3.0 * (1.0 + 2.0 ** -7)


def test_fwd_centre_delta_is_identity():
    C = 4
    x = _rand((2, 6, 5, C), 4)
    w = np.zeros((C, 3, 3, C), np.float32)
    for c in range(C):
        w[c, 1, 1, c] = 1.0
    assert np.array_equal(oracle.conv_fwd(x, w, 1, 1), x.astype(np.float64))


def test_fwd_off_centre_delta_shifts():
    # w[k=0, r=0, s=2, c=0] = 1  =>  y[p,q] = x[p-1, q+1] (cross-correlation, not flipped)
    x = _rand((1, 5, 6, 1), 5)
    w = np.zeros((1, 3, 3, 1), np.float32)
    w[0, 0, 2, 0] = 1.0
    y = oracle.conv_fwd(x, w, 1, 1)
    for p in range(5):
        for q in range(6):
            exp = x[0, p - 1, q + 1, 0] if (p - 1 >= 0 and q + 1 < 6) else 0.0
            assert y[0, p, q, 0] == exp


def test_fwd_all_ones_counts_taps():
    C = 5
    y = oracle.conv_fwd(np.ones((1, 6, 7, C), np.float32), np.ones((2, 3, 3, C), np.float32), 1, 1)
    assert y[0, 2, 3, 0] == 9 * C and y[0, 0, 3, 1] == 6 * C and y[0, 0, 0, 0] == 4 * C and y[0, 5, 6, 1] == 4 * C


@pytest.mark.parametrize("R,stride,pad,H,Wd", [(1, 1, 0, 5, 7), (3, 1, 1, 6, 5), (3, 2, 1, 8, 7), (1, 2, 0, 8, 6),
                                               (7, 2, 3, 15, 14), (3, 2, 1, 7, 9)])
def test_output_size_and_stride(R, stride, pad, H, Wd):
    x, w = _rand((2, H, Wd, 3), 6), _rand((4, R, R, 3), 7)
    y = oracle.conv_fwd(x, w, stride, pad)
    P, Q = (H + 2 * pad - R) // stride + 1, (Wd + 2 * pad - R) // stride + 1
    assert y.shape == (2, P, Q, 4)
    # strided output = stride-1 output subsampled
    y1 = oracle.conv_fwd(x, w, 1, pad)
    assert np.array_equal(y, y1[:, ::stride, ::stride, :][:, :P, :Q, :])


def test_fwd_linearity():
    x1, x2, w = _rand((2, 5, 5, 3), 8), _rand((2, 5, 5, 3), 9), _rand((4, 3, 3, 3), 10)
    # power-of-two scaling keeps bf16 representability, sum of two bf16 values may not: compare in w instead
    np.testing.assert_allclose(oracle.conv_fwd(2 * x1, w, 1, 1), 2 * oracle.conv_fwd(x1, w, 1, 1), rtol=0, atol=0)
    w2 = _rand((4, 3, 3, 3), 11)
    wa = np.concatenate([w, w2], 0)
    y = oracle.conv_fwd(x1, wa, 1, 1)
    assert np.array_equal(y[..., :4], oracle.conv_fwd(x1, w, 1, 1)) and np.array_equal(y[..., 4:], oracle.conv_fwd(x1, w2, 1, 1))


@pytest.mark.parametrize("R,stride,pad,H,Wd", [(1, 1, 0, 5, 6), (3, 1, 1, 6, 5), (3, 2, 1, 8, 7), (1, 2, 0, 8, 6),
                                               (7, 2, 3, 13, 12), (3, 2, 1, 7, 9), (3, 1, 0, 5, 5)])
def test_adjoint_identities(R, stride, pad, H, Wd):
    N, C, K = 2, 5, 3
    x, w = _rand((N, H, Wd, C), 12), _rand((K, R, R, C), 13)
    y = oracle.conv_fwd(x, w, stride, pad)
    dy = _rand(y.shape, 14)
    a = float((y * dy).sum())
    dx = oracle.conv_dgrad(dy, w, H, Wd, stride, pad)
    dw = oracle.conv_wgrad(x, dy, R, R, stride, pad)
    assert dx.shape == x.shape and dw.shape == w.shape
    assert abs(a - float((dx * x).sum())) <= 1e-12 * max(1.0, abs(a))
    assert abs(a - float((dw * w).sum())) <= 1e-12 * max(1.0, abs(a))


def test_gradients_by_finite_differences():
    # L(x, w) = <fwd(x, w), dy> is bilinear, so a central difference with a bf16-exact step is exact up to rounding.
    N, H, Wd, C, K, R, stride, pad = 1, 5, 4, 2, 3, 3, 2, 1
    x, w = _rand((N, H, Wd, C), 15), _rand((K, R, R, C), 16)
    dy = _rand(oracle.conv_fwd(x, w, stride, pad).shape, 17)
    dx = oracle.conv_dgrad(dy, w, H, Wd, stride, pad)
    dw = oracle.conv_wgrad(x, dy, R, R, stride, pad)
    L = lambda xx, ww: float((oracle.conv_fwd(xx, ww, stride, pad) * dy).sum())
    # a step of 2^k much larger than the value's ulp keeps x+h, x-h bf16-representable
    for idx in np.ndindex(x.shape):
        xp, xm = x.copy(), x.copy()
        xp[idx], xm[idx] = 64.0, -64.0           # replace the entry: L is affine in it
        fd = (L(xp, w) - L(xm, w)) / 128.0
        assert abs(fd - dx[idx]) < 1e-9
    for idx in list(np.ndindex(w.shape))[::2]:
        wp, wm = w.copy(), w.copy()
        wp[idx], wm[idx] = 64.0, -64.0
        fd = (L(x, wp) - L(x, wm)) / 128.0
        assert abs(fd - dw[idx]) < 1e-9


def test_dgrad_untouched_pixels_are_zero():
    # 1x1 stride 2: odd rows/columns of dx are reached by no tap
    dy, w = _rand((1, 3, 3, 2), 18), _rand((2, 1, 1, 3), 19)
    dx = oracle.conv_dgrad(dy, w, 6, 6, 2, 0)
    assert np.all(dx[:, 1::2] == 0) and np.all(dx[:, :, 1::2] == 0) and np.any(dx[:, ::2, ::2] != 0)


def test_sampled_versions_match_full():
    N, H, Wd, C, K, R, stride, pad = 2, 7, 6, 5, 4, 3, 2, 1
    x, w = _rand((N, H, Wd, C), 20), _rand((K, R, R, C), 21)
    y = oracle.conv_fwd(x, w, stride, pad)
    dy = _rand(y.shape, 22)
    dx = oracle.conv_dgrad(dy, w, H, Wd, stride, pad)
    dw = oracle.conv_wgrad(x, dy, R, R, stride, pad)
    for full, samp in ((y, oracle.conv_fwd_samples(x, w, np.arange(y.size), stride, pad)),
                       (dx, oracle.conv_dgrad_samples(dy, w, np.arange(dx.size), H, Wd, stride, pad)),
                       (dw, oracle.conv_wgrad_samples(x, dy, np.arange(dw.size), R, R, stride, pad))):
        np.testing.assert_allclose(samp, full.ravel(), rtol=0, atol=1e-12)


def test_zero_channels_give_zero_weight_gradient():
    # Eq. 4: a zero input channel / a zero upstream-gradient channel gives exactly-zero dw columns / rows
    x, dy = _rand((2, 5, 5, 4), 23), _rand((2, 5, 5, 3), 24)
    x[..., 1] = 0
    dy[..., 2] = 0
    dw = oracle.conv_wgrad(x, dy, 3, 3, 1, 1)
    assert np.all(dw[:, :, :, 1] == 0) and np.all(dw[2] == 0) and np.any(dw[0, :, :, 0] != 0)


def test_flops_closed_form_fixture():
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "flops_closed_form.txt")
    n = 0
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        name, N, H, C, K, R, stride, pad, flops = line.split()
        assert oracle.conv_flops(int(N), int(H), int(H), int(C), int(K), int(R), int(R), int(stride), int(pad)) == int(flops), name
        n += 1
    assert n == 8
    # MAC count equals the number of non-padding multiply-adds the loops execute only when nothing is clipped (pad 0)
    net = W.with_sizes(W.bottleneck_stage3(), [371, 93, 77])
    assert sum(oracle.conv_flops(64, l.H, l.H, l.C, l.K, l.R, l.R, l.stride, l.pad) for l in net.layers) == 12796786688
    assert sum(l.K * l.C * l.R * l.R for l in net.layers) == 127519
