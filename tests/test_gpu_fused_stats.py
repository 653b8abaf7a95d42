"""Convolution forward with the batch-normalisation statistics taken in its epilogue, then the normalisation from those
statistics -- against the oracle's composition conv -> (bf16 storage) -> batch norm + residual + ReLU, and against the
three-launch pt_bn_relu_fwd on the same stored tensor. Shapes are chosen to reach every forward kernel variant: the
pixel-linear kernel (1x1, strided, small maps; one and several channel tiles; one and several tiles per CTA), the halo
kernel (stride-1 3x3, with raster positions that are not output pixels) and the few-channel stem."""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_09290_b200 import binding as B
from paper_1901_09290_b200 import workloads as W
from tests import helpers as Hh

pytestmark = pytest.mark.gpu

# (N, H, C, K, R, stride)
SHAPES = [
    (8, 16, 16, 32, 1, 1),        # 1x1, one tile per CTA
    (64, 28, 77, 371, 1, 1),      # 1x1, two channel tiles, several tiles per CTA (resident weights do not apply)
    (64, 56, 59, 143, 1, 1),      # 1x1, many tiles per CTA, resident weights, two issuers
    (32, 28, 93, 77, 3, 1),       # halo kernel, garbage raster columns
    (16, 14, 213, 242, 3, 1),     # halo kernel, streamed weights
    (8, 7, 130, 90, 3, 1),        # 3x3 on a small map: the pixel-linear kernel through im2col boxes
    (16, 28, 112, 111, 3, 2),     # stride 2
    (8, 56, 143, 300, 1, 2),      # strided 1x1 (projection shortcut), two channel tiles
    (4, 64, 3, 55, 7, 2),         # the stem
]


@pytest.mark.parametrize("shape", SHAPES)
def test_conv_epilogue_statistics_feed_the_batch_norm(shape):
    N, H, C, K, R, stride = shape
    c = Hh.ctx()
    pad = R // 2
    seed = W.BASE_SEED + 7000 + K
    x = (W.gen_image if C <= 4 else W.gen_act)(N, H, H, C, seed)
    w = W.bf16_round(W.gen_weight(K, R, R, C, seed + 1))
    ldx, ldy = (8 if C <= 4 else W.pad16(C)), W.pad16(K)
    d = B.make_conv_desc(N, H, H, C, K, R, R, stride, pad, ldx, ldy, W.pad8(C), 0, 2)
    P = (H + 2 * pad - R) // stride + 1
    xd, wd = Hh.to_dev_padded(x, ldx), Hh.to_dev_padded(w, W.pad8(C))
    y = Hh.out_buffer((N, P, P), K, ldy, False)
    stats = torch.full((B.pt_conv_fwd_stats_bytes(c, d) // 4,), float("nan"), dtype=torch.float32, device="cuda")
    n_parts = B.pt_conv_fwd_stats(c, d, xd, wd, y, stats, Hh.conv_ws(d, B.PT_CONV_FWD))
    torch.cuda.synchronize()
    c.poll()
    assert n_parts >= 1
    # the convolution itself is the ordinary forward pass, bit for bit
    y2 = Hh.out_buffer((N, P, P), K, ldy, False)
    B.pt_conv_fwd(c, d, xd, wd, y2, Hh.conv_ws(d, B.PT_CONV_FWD))
    torch.cuda.synchronize()
    assert torch.equal(y[..., :K], y2[..., :K])
    y_ref = oracle.conv_fwd(x.numpy(), w.numpy(), stride, pad)
    Hh.check_conv(y, K, y_ref, what="conv fwd with statistics")
    # the rows of partial sums add up to the sums of the STORED bf16 values
    st = stats[: n_parts * 2 * ldy].view(n_parts, 2, ldy).cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(st))
    ys = y[..., :K].float().cpu().numpy().astype(np.float64).reshape(-1, K)
    s0, s1 = ys.sum(axis=0), (ys ** 2).sum(axis=0)
    assert np.allclose(st[:, 0, :K].sum(axis=0), s0, rtol=1e-5, atol=1e-5 * np.abs(ys).sum(axis=0).max())
    assert np.allclose(st[:, 1, :K].sum(axis=0), s1, rtol=1e-5)
    assert np.all(st[:, :, K:] == 0)
    # batch norm + residual + ReLU from those statistics
    g = torch.rand(K, generator=torch.Generator().manual_seed(seed + 3)) + 0.5
    b = torch.rand(K, generator=torch.Generator().manual_seed(seed + 4)) - 0.5
    res = W.bf16_round(W.gen_act(N, P, P, K, seed + 5) - 0.4)
    bd_ = B.make_bn_desc(N, P, P, K, ldy, 1e-5, 0.1, True)
    rd = Hh.to_dev_padded(res, ldy)
    gd, bd = g.cuda(), b.cuda()
    sm, si = torch.empty(K, device="cuda"), torch.empty(K, device="cuda")
    rm, rv = torch.zeros(K, device="cuda"), torch.ones(K, device="cuda")
    out = Hh.out_buffer((N, P, P), K, ldy, False)
    B.pt_bn_relu_fwd_stats(c, bd_, y, rd, gd, bd, rm, rv, sm, si, out, stats, n_parts)
    # the three-launch form on the same stored tensor
    sm3, si3 = torch.empty(K, device="cuda"), torch.empty(K, device="cuda")
    out3 = Hh.out_buffer((N, P, P), K, ldy, False)
    ws = torch.empty(max(16, B.pt_bn_workspace_bytes(c, bd_)), dtype=torch.uint8, device="cuda")
    B.pt_bn_relu_fwd(c, bd_, y, rd, gd, bd, None, None, sm3, si3, out3, ws)
    torch.cuda.synchronize()
    c.poll()
    # oracle: batch norm of the stored (bf16) convolution output
    y_st = y[..., :K].float().cpu().numpy()
    o_ref, mean, invstd, var = oracle.bn_relu_fwd(y_st, g.numpy().astype(np.float64), b.numpy().astype(np.float64), 1e-5, res.numpy(), True)
    scale = np.sqrt(var).max()
    assert np.allclose(sm.cpu().numpy(), mean, rtol=1e-5, atol=1e-5 * max(scale, 1e-3))
    assert np.allclose(si.cpu().numpy(), invstd, rtol=5e-5)
    assert np.allclose(sm.cpu().numpy(), sm3.cpu().numpy(), rtol=1e-5, atol=1e-5 * max(scale, 1e-3))
    Hh.check_conv(out, K, o_ref, what="bn from the convolution's statistics")
    M = N * P * P
    rm_ref, rv_ref = oracle.bn_running_stats(np.zeros(K), np.ones(K), mean, var, M, 0.1)
    assert np.allclose(rm.cpu().numpy(), rm_ref, rtol=1e-5, atol=1e-6) and np.allclose(rv.cpu().numpy(), rv_ref, rtol=1e-4, atol=1e-6)


def test_statistics_are_run_to_run_identical_and_refuse_what_they_cannot_serve():
    c = Hh.ctx()
    N, H, C, K = 16, 28, 93, 77
    x, w = W.gen_act(N, H, H, C, 5), W.bf16_round(W.gen_weight(K, 3, 3, C, 6))
    d = B.make_conv_desc(N, H, H, C, K, 3, 3, 1, 1, W.pad16(C), W.pad16(K), W.pad8(C), 0, 0)
    xd, wd = Hh.to_dev_padded(x, W.pad16(C)), Hh.to_dev_padded(w, W.pad8(C))
    y = Hh.out_buffer((N, H, H), K, W.pad16(K), False)
    runs = []
    for _ in range(2):
        stats = torch.zeros(B.pt_conv_fwd_stats_bytes(c, d) // 4, dtype=torch.float32, device="cuda")
        n = B.pt_conv_fwd_stats(c, d, xd, wd, y, stats, Hh.conv_ws(d, B.PT_CONV_FWD))
        torch.cuda.synchronize()
        runs.append((n, stats.clone()))
    assert runs[0][0] == runs[1][0] and torch.equal(runs[0][1], runs[1][1])
    small = torch.zeros(64, dtype=torch.float32, device="cuda")
    with pytest.raises(B.PtError) as e:
        B.pt_conv_fwd_stats(c, d, xd, wd, y, small, Hh.conv_ws(d, B.PT_CONV_FWD))
    assert e.value.status == 3                                   # PT_ERR_WORKSPACE
    d32 = B.make_conv_desc(N, H, H, C, K, 3, 3, 1, 1, W.pad16(C), W.pad16(K), W.pad8(C), 1, 0)
    with pytest.raises(B.PtError) as e:
        B.pt_conv_fwd_stats(c, d32, xd, wd, y, runs[0][1], Hh.conv_ws(d32, B.PT_CONV_FWD))
    assert e.value.status == 2                                   # fp32 outputs: PT_ERR_UNSUPPORTED
    torch.cuda.synchronize()
    c.poll()


def test_every_layer_of_the_bench_workload_at_full_size():
    """All 53 layers of the pruned ResNet-50 at batch 64 (the launch shapes of the chained bench step): the forward with the
    statistics epilogue stores bit for bit what the plain forward stores (which the network tests hold against the oracle at
    this size), and its rows of partial sums add up to the sums of those stored values."""
    c = Hh.ctx()
    net = W.resnet50()
    seed = W.BASE_SEED + 4
    counts = W.staged_keep_to_flops(net, seed, 0.60)
    netp = W.with_sizes(net, counts)
    N = 64
    g = torch.Generator(device="cuda").manual_seed(seed)
    for li, l in enumerate(netp.layers):
        ldx, ldy = (8 if l.C <= 4 else W.pad16(l.C)), W.pad16(l.K)
        d = B.make_conv_desc(N, l.H, l.H, l.C, l.K, l.R, l.R, l.stride, l.pad, ldx, ldy, W.pad8(l.C), 0, 2)
        x = torch.randn((N, l.H, l.H, ldx), generator=g, device="cuda")
        if li:
            x.clamp_(min=0)
        x = x.to(torch.bfloat16)
        w = (torch.randn((l.K, l.R, l.R, W.pad8(l.C)), generator=g, device="cuda") * (2.0 / (l.C * l.R * l.R)) ** 0.5).to(torch.bfloat16)
        y = torch.full((N, l.P, l.P, ldy), 7680.0, dtype=torch.bfloat16, device="cuda")
        y2 = torch.full_like(y, 7680.0)
        stats = torch.full((B.pt_conv_fwd_stats_bytes(c, d) // 4,), float("nan"), dtype=torch.float32, device="cuda")
        ws = Hh.conv_ws(d, B.PT_CONV_FWD)
        n_parts = B.pt_conv_fwd_stats(c, d, x, w, y, stats, ws)
        B.pt_conv_fwd(c, d, x, w, y2, ws)
        torch.cuda.synchronize()
        c.poll()
        assert torch.equal(y[..., :l.K], y2[..., :l.K]), l.name
        st = stats[: n_parts * 2 * ldy].view(n_parts, 2, ldy).double().sum(dim=0).cpu().numpy()
        ys = y[..., :l.K].reshape(-1, l.K).float().cpu().numpy().astype(np.float64)
        s0, s1 = ys.sum(axis=0), (ys ** 2).sum(axis=0)
        assert np.allclose(st[0, :l.K], s0, rtol=2e-5, atol=2e-5 * np.abs(ys).sum(axis=0).max()), l.name
        assert np.allclose(st[1, :l.K], s1, rtol=2e-5), l.name
        assert np.all(st[:, l.K:] == 0), l.name
        del x, w, y, y2, stats
