"""Max pooling through the C ABI against the oracle: forward bit for bit (a maximum of stored values), backward to one bf16
rounding of a sum of at most four gradients; ties (ReLU zeros) take the first position in scan order on both sides."""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_09290_b200 import binding as B
from paper_1901_09290_b200 import workloads as W
from tests import helpers as Hh

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("with_index", [False, True], ids=["recompute", "index"])
@pytest.mark.parametrize("shape", [(2, 8, 8, 5, 3, 2, 1), (3, 9, 9, 11, 3, 2, 1), (64, 112, 112, 55, 3, 2, 1), (2, 6, 6, 16, 2, 2, 0), (1, 5, 5, 3, 3, 1, 1)])
def test_maxpool_forward_and_backward(shape, with_index):
    N, H, _, C, R, stride, pad = shape
    if N * H * H * C > 2e7:
        N = 4                                                 # the stem's shape at a batch the oracle finishes quickly
    c = Hh.ctx()
    ld = W.pad16(C)
    x = W.bf16_round(W.gen_act(N, H, H, C, 77 + C))           # post-ReLU: many exact zeros, i.e. ties
    P = (H + 2 * pad - R) // stride + 1
    dy = W.bf16_round(W.gen_dy(N, P, P, C, 78 + C) * 64)
    d = B.make_pool_desc(N, H, H, C, ld, R, stride, pad)
    xd, dyd = Hh.to_dev_padded(x, ld), Hh.to_dev_padded(dy, ld)
    y = Hh.out_buffer((N, P, P), C, ld, False)
    dx = Hh.out_buffer((N, H, H), C, ld, False)
    index = torch.full((N, P, P, ld), 77, dtype=torch.uint8, device="cuda") if with_index else None
    B.pt_maxpool_fwd(c, d, xd, y, index=index)
    # with the selections stored, the backward pass does not need x
    B.pt_maxpool_bwd(c, d, None if with_index else xd, dyd, dx, index=index)
    torch.cuda.synchronize()
    c.poll()
    y_ref, sel = oracle.maxpool_fwd(x.numpy(), R, stride, pad)
    if with_index:
        # a stored selection is a position of the window that lies inside the image and holds the maximum
        ix = index.cpu().numpy()
        assert np.all(ix[..., C:] == 255) and np.all(ix[..., :C] < R * R)
        xn = x.numpy()
        n_, p_, q_, c_ = np.meshgrid(np.arange(N), np.arange(P), np.arange(P), np.arange(C), indexing="ij")
        hh = p_ * stride - pad + ix[..., :C] // R
        ww = q_ * stride - pad + ix[..., :C] % R
        assert np.all((hh >= 0) & (hh < H) & (ww >= 0) & (ww < H))
        assert np.array_equal(xn[n_, hh, ww, c_].astype(np.float64), y_ref)
    assert np.array_equal(y[..., :C].float().cpu().numpy().astype(np.float64), y_ref)
    assert torch.all(y[..., C:] == 0) and torch.all(dx[..., C:] == 0)
    dx_ref = oracle.maxpool_bwd(dy.numpy(), sel, H, H)
    want = W.bf16_round(torch.from_numpy(dx_ref).float()).numpy()
    assert np.array_equal(dx[..., :C].float().cpu().numpy(), want)
    for bad in (dict(ld=ld + 1), dict(pad=R), dict(C=0)):
        kw = dict(N=N, H=H, W=H, C=C, ld=ld, R=R, stride=stride, pad=pad)
        kw.update(bad)
        with pytest.raises(B.PtError):
            B.pt_maxpool_fwd(c, B.make_pool_desc(**kw), xd, y)
