"""Parity of the batch-normalisation + residual + ReLU kernels (through the C ABI) with the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_09290_b200 import binding as B
from paper_1901_09290_b200 import workloads as W
from tests import helpers as Hh

pytestmark = pytest.mark.gpu

# (N, H, W, C): ragged channel counts, one vector, many vectors, a single pixel row, more than one block per channel
SHAPES = [(2, 5, 7, 1), (3, 8, 8, 11), (4, 14, 14, 93), (2, 28, 28, 143), (1, 1, 1, 8), (8, 7, 7, 260), (64, 14, 14, 48)]


def _dev(t, ld):
    return Hh.to_dev_padded(t, ld)            # pad lanes hold NaN: they must never reach an output


def _bf(t):
    return W.bf16_round(t)


@pytest.mark.parametrize("relu", [True, False])
@pytest.mark.parametrize("with_res", [True, False])
@pytest.mark.parametrize("shape", SHAPES)
def test_bn_relu_forward_and_backward(shape, with_res, relu):
    N, H, Wd, C = shape
    c = Hh.ctx()
    ld = W.pad8(C)
    seed = W.BASE_SEED + 500 + C
    x = _bf(W.gen_act(N, H, Wd, C, seed) * 1.7 + 0.3)
    res = _bf(W.gen_act(N, H, Wd, C, seed + 1) - 0.4) if with_res else None
    dy = W.gen_dy(N, H, Wd, C, seed + 2) * 64.0
    g = torch.rand(C, generator=torch.Generator().manual_seed(seed + 3)) + 0.5
    b = torch.rand(C, generator=torch.Generator().manual_seed(seed + 4)) - 0.5
    rm0 = torch.rand(C, generator=torch.Generator().manual_seed(seed + 5))
    rv0 = torch.rand(C, generator=torch.Generator().manual_seed(seed + 6)) + 0.5
    eps, mom = 1e-5, 0.1
    d = B.make_bn_desc(N, H, Wd, C, ld, eps, mom, relu)
    ws = torch.empty(max(16, B.pt_bn_workspace_bytes(c, d)), dtype=torch.uint8, device="cuda")
    xd, rd, dyd = _dev(x, ld), (_dev(res, ld) if with_res else None), _dev(dy, ld)
    gd, bd, rm, rv = g.cuda(), b.cuda(), rm0.clone().cuda(), rv0.clone().cuda()
    sm, si = torch.empty(C, device="cuda"), torch.empty(C, device="cuda")
    y = Hh.out_buffer((N, H, Wd), C, ld, False)
    B.pt_bn_relu_fwd(c, d, xd, rd, gd, bd, rm, rv, sm, si, y, ws)
    torch.cuda.synchronize()
    y_ref, mean, invstd, var = oracle.bn_relu_fwd(x.numpy(), g.numpy().astype(np.float64), b.numpy().astype(np.float64), eps,
                                                  res.numpy() if with_res else None, relu)
    M = N * H * Wd
    # statistics: fp32 partial sums about a pivot, fp64 combination
    assert np.allclose(sm.cpu().numpy(), mean, rtol=1e-5, atol=1e-5)
    assert np.allclose(si.cpu().numpy(), invstd, rtol=2e-5)
    rm_ref, rv_ref = oracle.bn_running_stats(rm0.numpy(), rv0.numpy(), mean, var, M, mom)
    assert np.allclose(rm.cpu().numpy(), rm_ref, rtol=1e-5, atol=1e-6)
    assert np.allclose(rv.cpu().numpy(), rv_ref, rtol=1e-4, atol=1e-6)
    Hh.check_conv(y, C, y_ref, what="bn fwd")

    # backward: the mask input is the ORACLE's y rounded to bf16, given to both sides
    y_in = _bf(torch.from_numpy(y_ref).float())
    dx = Hh.out_buffer((N, H, Wd), C, ld, False)
    dres = Hh.out_buffer((N, H, Wd), C, ld, False) if with_res else None
    dg, db = torch.empty(C, device="cuda"), torch.empty(C, device="cuda")
    sm2, si2 = torch.from_numpy(mean).float().cuda(), torch.from_numpy(invstd).float().cuda()
    B.pt_bn_relu_bwd(c, d, xd, _dev(y_in, ld), dyd, gd, sm2, si2, dx, dres, dg, db, ws)
    torch.cuda.synchronize()
    c.poll()
    dx_ref, dres_ref, dg_ref, db_ref = oracle.bn_relu_bwd(x.numpy(), y_in.numpy(), dy.numpy(), g.numpy().astype(np.float64),
                                                          sm2.cpu().numpy().astype(np.float64), si2.cpu().numpy().astype(np.float64), relu)
    scale_g = np.sqrt(M) * np.abs(dy.numpy()).max()             # size of a sum of M terms of that magnitude
    assert np.abs(dg.cpu().numpy() - dg_ref).max() <= 1e-4 * scale_g * max(1.0, np.abs(invstd).max() * np.abs(x.numpy()).max())
    assert np.abs(db.cpu().numpy() - db_ref).max() <= 1e-4 * scale_g
    Hh.check_conv(dx, C, dx_ref, what="bn dx")
    if with_res:
        got = dres.float().cpu().numpy()[..., :C]
        assert np.array_equal(got, dres_ref.astype(np.float32)), "dresidual is dy under the ReLU mask, bit for bit"


def test_bn_is_run_to_run_identical_and_validates():
    c = Hh.ctx()
    N, H, C = 8, 28, 77
    ld = W.pad8(C)
    x = _bf(W.gen_act(N, H, H, C, W.BASE_SEED + 900))
    d = B.make_bn_desc(N, H, H, C, ld)
    ws = torch.empty(max(16, B.pt_bn_workspace_bytes(c, d)), dtype=torch.uint8, device="cuda")
    xd = _dev(x, ld)
    g, b = torch.ones(C, device="cuda"), torch.zeros(C, device="cuda")
    outs = []
    for _ in range(2):
        sm, si = torch.empty(C, device="cuda"), torch.empty(C, device="cuda")
        y = Hh.out_buffer((N, H, H), C, ld, False)
        B.pt_bn_relu_fwd(c, d, xd, None, g, b, None, None, sm, si, y, ws)
        outs.append((sm.cpu(), si.cpu(), y.cpu()))
    assert all(torch.equal(a, bb) for a, bb in zip(outs[0], outs[1]))
    bad = B.make_bn_desc(N, H, H, C, ld=C)          # pitch not a multiple of 8
    with pytest.raises(B.PtError):
        B.pt_bn_relu_fwd(c, bad, xd, None, g, b, None, None, sm, si, y, ws)
    with pytest.raises(B.PtError):
        B.pt_bn_relu_fwd(c, d, xd, None, g, b, sm, None, sm, si, y, ws)      # only one of the two moving statistics
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    if B.pt_bn_workspace_bytes(c, d) > 16:
        with pytest.raises(B.PtError):
            B.pt_bn_relu_fwd(c, d, xd, None, g, b, None, None, sm, si, y, small)
