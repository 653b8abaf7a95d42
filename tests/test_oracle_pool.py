"""Pins of the pooling oracle: a hand example, the tie rule, conservation of the gradient, and an independent library
routine (torch's max_pool2d and its autograd) on inputs without ties."""
import numpy as np
import torch

import oracle


def test_hand_example_4x4():
    x = np.array([[1, 5, 2, 0],
                  [3, 4, 9, 1],
                  [7, 0, 2, 2],
                  [1, 8, 3, 6]], np.float64).reshape(1, 4, 4, 1)
    y, sel = oracle.maxpool_fwd(x, 3, 2, 1)
    # windows (rows x cols): p=0 covers rows 0..1, p=1 rows 1..3; q likewise
    assert y[0, :, :, 0].tolist() == [[5, 9], [8, 9]]
    assert sel[0, :, :, 0].tolist() == [[1, 6], [13, 6]]
    dy = np.array([[10, 20], [30, 40]], np.float64).reshape(1, 2, 2, 1)
    dx = oracle.maxpool_bwd(dy, sel, 4, 4)[0, :, :, 0]
    want = np.zeros((4, 4)); want[0, 1] = 10; want[1, 2] = 60; want[3, 1] = 30
    assert np.array_equal(dx, want)


def test_first_of_equal_maxima_is_selected_and_padding_never():
    x = np.zeros((1, 4, 4, 2))
    x[..., 1] = -3.0                                   # all-negative channel: padding (outside the image) must not win
    y, sel = oracle.maxpool_fwd(x, 3, 2, 1)
    assert np.all(y[..., 0] == 0) and np.all(y[..., 1] == -3.0)
    # window (0,0) covers rows 0..1, cols 0..1 of the image: the first position in scan order is (0,0)
    assert sel[0, 0, 0, 0] == 0 and sel[0, 0, 1, 0] == 1 and sel[0, 1, 0, 0] == 4 and sel[0, 1, 1, 0] == 5
    dy = np.ones((1, 2, 2, 2))
    dx = oracle.maxpool_bwd(dy, sel, 4, 4)
    assert dx.sum() == dy.sum() and dx[0, 0, 0, 0] == 1 and dx[0, 3, 3, 0] == 0


def test_against_torch_on_inputs_without_ties():
    g = torch.Generator().manual_seed(3)
    for (N, H, W, C, R, s, pad) in [(2, 9, 7, 3, 3, 2, 1), (1, 8, 8, 2, 2, 2, 0), (2, 6, 6, 1, 3, 1, 1)]:
        x = torch.randn(N, C, H, W, generator=g, dtype=torch.float64, requires_grad=True)
        yt = torch.nn.functional.max_pool2d(x, R, s, pad)
        dy = torch.randn(yt.shape, generator=g, dtype=torch.float64)
        yt.backward(dy)
        y, sel = oracle.maxpool_fwd(x.detach().permute(0, 2, 3, 1).numpy(), R, s, pad)
        assert np.array_equal(y, yt.detach().permute(0, 2, 3, 1).numpy())
        dx = oracle.maxpool_bwd(dy.permute(0, 2, 3, 1).numpy(), sel, H, W)
        assert np.allclose(dx, x.grad.permute(0, 2, 3, 1).numpy(), rtol=0, atol=1e-15)
        assert abs(dx.sum() - float(dy.sum())) < 1e-9
