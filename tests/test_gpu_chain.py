"""A chained residual block through the C ABI -- conv, batch norm, ReLU, shortcut, residual add, and the whole backward pass
down to the weight gradients -- against the same composition of the oracle's functions. Every tensor the CUDA path stores
in bf16 is rounded to bf16 at the same place on the oracle side (a storage conversion, not arithmetic)."""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_09290_b200 import binding as B
from paper_1901_09290_b200 import workloads as W
from tests import helpers as Hh

pytestmark = pytest.mark.gpu


def _r(a):
    return oracle.round_bf16(np.asarray(a, np.float32)).astype(np.float64)


def _dev(a, ld):
    return Hh.to_dev_padded(torch.from_numpy(np.asarray(a, np.float32)), ld)


def _rel(got, ref):
    return np.linalg.norm((got - ref).ravel()) / max(np.linalg.norm(ref.ravel()), 1e-300)


class _Conv:
    def __init__(self, N, H, C, K, R, seed):
        self.N, self.H, self.C, self.K, self.R, self.pad = N, H, C, K, R, R // 2
        self.w = W.bf16_round(W.gen_weight(K, R, R, C, seed)).numpy()
        self.d = B.make_conv_desc(N, H, H, C, K, R, R, 1, self.pad, W.pad8(C), W.pad8(K), W.pad8(C))
        self.wd = _dev(self.w, W.pad8(C))

    def ws(self, which):
        return Hh.conv_ws(self.d, which)


class _Bn:
    def __init__(self, N, H, C, relu, seed):
        g = torch.Generator().manual_seed(seed)
        self.gamma = (torch.rand(C, generator=g) + 0.5).numpy().astype(np.float64)
        self.beta = (torch.rand(C, generator=g) - 0.5).numpy().astype(np.float64)
        self.C, self.relu = C, relu
        self.d = B.make_bn_desc(N, H, H, C, W.pad8(C), 1e-5, 0.1, relu)
        self.gd, self.bd = torch.from_numpy(self.gamma).float().cuda(), torch.from_numpy(self.beta).float().cuda()
        self.sm, self.si = torch.empty(C, device="cuda"), torch.empty(C, device="cuda")
        self.dg, self.db = torch.empty(C, device="cuda"), torch.empty(C, device="cuda")
        self.ws = torch.empty(max(16, B.pt_bn_workspace_bytes(Hh.ctx(), self.d)), dtype=torch.uint8, device="cuda")


def test_chained_bottleneck_block_forward_and_backward():
    c = Hh.ctx()
    N, H = 4, 12
    C0, C1, C2, C3 = 27, 19, 13, 44                       # ragged counts, as after pruning
    seed = W.BASE_SEED + 4100
    x0 = _r(W.gen_act(N, H, H, C0, seed).numpy())
    G = _r(W.gen_dy(N, H, H, C3, seed + 1).numpy() * 64)
    c1, c2, c3, ds = _Conv(N, H, C0, C1, 1, seed + 2), _Conv(N, H, C1, C2, 3, seed + 3), _Conv(N, H, C2, C3, 1, seed + 4), _Conv(N, H, C0, C3, 1, seed + 5)
    b1, b2, b3, bs = _Bn(N, H, C1, True, seed + 6), _Bn(N, H, C2, True, seed + 7), _Bn(N, H, C3, True, seed + 8), _Bn(N, H, C3, False, seed + 9)

    # ---------------- oracle: the block written out, bf16 storage rounding where the CUDA path stores bf16
    def o_conv(cv, x):
        return _r(oracle.conv_fwd(x.astype(np.float32), cv.w, 1, cv.pad))

    def o_bn(bn, y, res=None):
        a, mean, invstd, _ = oracle.bn_relu_fwd(y, bn.gamma, bn.beta, 1e-5, res, bn.relu)
        return _r(a), mean.astype(np.float32).astype(np.float64), invstd.astype(np.float32).astype(np.float64)

    y1 = o_conv(c1, x0); a1, m1, i1 = o_bn(b1, y1)
    y2 = o_conv(c2, a1); a2, m2, i2 = o_bn(b2, y2)
    y3 = o_conv(c3, a2)
    ys = o_conv(ds, x0); r, ms, is_ = o_bn(bs, ys)
    out, m3, i3 = o_bn(b3, y3, r)

    def o_bn_bwd(bn, y, a, da, mean, invstd):
        dx, dres, dg, db = oracle.bn_relu_bwd(y, a, da, bn.gamma, mean, invstd, bn.relu)
        return _r(dx), _r(dres), dg, db

    dy3, dr, dg3, db3 = o_bn_bwd(b3, y3, out, G, m3, i3)
    dys, _, dgs, dbs = o_bn_bwd(bs, ys, r, dr, ms, is_)
    dw3 = oracle.conv_wgrad(a2.astype(np.float32), dy3.astype(np.float32), 1, 1, 1, 0)
    dws = oracle.conv_wgrad(x0.astype(np.float32), dys.astype(np.float32), 1, 1, 1, 0)
    da2 = _r(oracle.conv_dgrad(dy3.astype(np.float32), c3.w, H, H, 1, 0))
    dy2, _, dg2, db2 = o_bn_bwd(b2, y2, a2, da2, m2, i2)
    dw2 = oracle.conv_wgrad(a1.astype(np.float32), dy2.astype(np.float32), 3, 3, 1, 1)
    da1 = _r(oracle.conv_dgrad(dy2.astype(np.float32), c2.w, H, H, 1, 1))
    dy1, _, dg1, db1 = o_bn_bwd(b1, y1, a1, da1, m1, i1)
    dw1 = oracle.conv_wgrad(x0.astype(np.float32), dy1.astype(np.float32), 1, 1, 1, 0)

    # ---------------- the same block through the C ABI
    def buf(C):
        return torch.zeros((N, H, H, W.pad8(C)), dtype=torch.bfloat16, device="cuda")

    def g_conv(cv, x):
        y = buf(cv.K)
        B.pt_conv_fwd(c, cv.d, x, cv.wd, y, cv.ws(B.PT_CONV_FWD))
        return y

    def g_bn(bn, y, res=None):
        a = buf(bn.C)
        B.pt_bn_relu_fwd(c, bn.d, y, res, bn.gd, bn.bd, None, None, bn.sm, bn.si, a, bn.ws)
        return a

    x0d = _dev(x0, W.pad8(C0))
    gy1 = g_conv(c1, x0d); ga1 = g_bn(b1, gy1)
    gy2 = g_conv(c2, ga1); ga2 = g_bn(b2, gy2)
    gy3 = g_conv(c3, ga2)
    gys = g_conv(ds, x0d); gr = g_bn(bs, gys)
    gout = g_bn(b3, gy3, gr)

    def g_bn_bwd(bn, y, a, da, want_res):
        dx, dres = buf(bn.C), (buf(bn.C) if want_res else None)
        B.pt_bn_relu_bwd(c, bn.d, y, a, da, bn.gd, bn.sm, bn.si, dx, dres, bn.dg, bn.db, bn.ws)
        return dx, dres

    def g_wgrad(cv, x, dy):
        dw = torch.empty((cv.K, cv.R, cv.R, cv.C), dtype=torch.float32, device="cuda")
        B.pt_conv_wgrad(c, cv.d, x, dy, dw, cv.ws(B.PT_CONV_WGRAD))
        return dw

    def g_dgrad(cv, dy):
        dx = buf(cv.C)
        B.pt_conv_dgrad(c, cv.d, dy, cv.wd, dx, cv.ws(B.PT_CONV_DGRAD))
        return dx

    Gd = _dev(G, W.pad8(C3))
    gdy3, gdr = g_bn_bwd(b3, gy3, gout, Gd, True)
    gdys, _ = g_bn_bwd(bs, gys, gr, gdr, False)
    gdw3, gdws = g_wgrad(c3, ga2, gdy3), g_wgrad(ds, x0d, gdys)
    gda2 = g_dgrad(c3, gdy3)
    gdy2, _ = g_bn_bwd(b2, gy2, ga2, gda2, False)
    gdw2 = g_wgrad(c2, ga1, gdy2)
    gda1 = g_dgrad(c2, gdy2)
    gdy1, _ = g_bn_bwd(b1, gy1, ga1, gda1, False)
    gdw1 = g_wgrad(c1, x0d, gdy1)
    torch.cuda.synchronize()
    c.poll()

    # ---------------- compare. Rounding differences compound along the chain and may flip a ReLU decision at isolated
    # near-zero elements, so the bound is on relative Frobenius errors: tight at the front, looser at the far end.
    f = lambda t, C: t.float().cpu().numpy()[..., :C].astype(np.float64)
    assert _rel(f(gout, C3), out) < 5e-3
    assert _rel(f(gdy3, C3), dy3) < 1e-2 and _rel(f(gdr, C3), dr) < 1e-2
    for got, ref, nm in ((gdw3, dw3, "c3"), (gdws, dws, "ds"), (gdw2, dw2, "c2"), (gdw1, dw1, "c1")):
        assert _rel(got.cpu().numpy().astype(np.float64), ref) < 2e-2, nm
    for bn, dg, db, nm in ((b3, dg3, db3, "bn3"), (bs, dgs, dbs, "bn_ds"), (b2, dg2, db2, "bn2"), (b1, dg1, db1, "bn1")):
        assert _rel(bn.dg.cpu().numpy().astype(np.float64), dg) < 2e-2, nm
        assert _rel(bn.db.cpu().numpy().astype(np.float64), db) < 2e-2, nm


# ------------------------------------------------------------------------------------------ a whole chained stage
def _oracle_chain(cs, model, x0, g_last):
    """The composition ChainedStep runs, written with the oracle's functions; bf16 storage rounding where the CUDA path
    stores bf16 (convolution outputs, activations, activation gradients). Returns the block output and the gradients.

    The forward pass is the oracle's own chain from the image (compared at the stage's output). The backward pass is then
    evaluated on the forward state the CUDA path stored (its convolution outputs, activations, batch statistics and pooled
    map, copied back): a ReLU or pooling decision is a comparison of stored values, and two forward chains that differ by
    rounding take it differently at a few near-zero elements, each of which changes the gradient by a whole term. Fed the
    same stored bits, both sides take every decision alike and what remains is the arithmetic of the backward chain."""
    L = cs.net.layers
    gam = {i: cs.gamma[i].cpu().numpy().astype(np.float64) for i in cs.used}
    bet = {i: cs.beta[i].cpu().numpy().astype(np.float64) for i in cs.used}
    w = {i: W.bf16_round(model.w[i]).numpy() for i in cs.used}
    ds_set = {b[1] for b in cs.blocks if b[1] is not None}
    y, a, st = {}, {}, {}

    def conv_bn(i, x, res=None):
        l = L[i]
        y[i] = _r(oracle.conv_fwd(x.astype(np.float32), w[i], l.stride, l.pad))
        out, mean, invstd, _ = oracle.bn_relu_fwd(y[i], gam[i], bet[i], 1e-5, res, i not in ds_set)
        a[i] = _r(out)
        st[i] = (mean.astype(np.float32).astype(np.float64), invstd.astype(np.float32).astype(np.float64))
        return a[i]

    cur = conv_bn(0, x0)
    sel = None
    if cs.pool:
        pooled, sel = oracle.maxpool_fwd(cur, 3, 2, 1)
        cur = _r(pooled)
    block_in = []
    for main, ds, _ in cs.blocks:
        block_in.append(cur)
        res = conv_bn(ds, cur) if ds is not None else cur
        t = cur
        for i in main[:-1]:
            t = conv_bn(i, t)
        cur = conv_bn(main[-1], t, res)
    out = cur
    dw, dgm, dbt = {}, {}, {}
    # the stored forward state of the CUDA path
    g64 = lambda t, C: t.float().cpu().numpy()[..., :C].astype(np.float64)
    for i in cs.used:
        y[i], a[i] = g64(cs.y[i], L[i].K), g64(cs.a[i], L[i].K)
        st[i] = (cs.sm[i].cpu().numpy().astype(np.float64), cs.si[i].cpu().numpy().astype(np.float64))
    if cs.pool:
        _, sel = oracle.maxpool_fwd(a[0], 3, 2, 1)
    block_in = [g64(t, L[b[0][0]].C) for t, b in zip(cs.block_in, cs.blocks)]

    def bn_bwd(i, d_out):
        dx, dres, dg, db = oracle.bn_relu_bwd(y[i], a[i], d_out, gam[i], st[i][0], st[i][1], i not in ds_set)
        dgm[i], dbt[i] = dg, db
        return _r(dx), _r(dres)

    d_cur = g_last
    for bi in range(len(cs.blocks) - 1, -1, -1):
        main, ds, _ = cs.blocks[bi]
        x_in = block_in[bi]
        dyl, dres = bn_bwd(main[-1], d_cur)
        d_t = None
        for k in range(len(main) - 1, -1, -1):
            i, l = main[k], L[main[k]]
            x_i = x_in if k == 0 else a[main[k - 1]]
            if k < len(main) - 1:
                dyl, _ = bn_bwd(i, d_t)
            dw[i] = oracle.conv_wgrad(x_i.astype(np.float32), dyl.astype(np.float32), l.R, l.R, l.stride, l.pad)
            d_t = _r(oracle.conv_dgrad(dyl.astype(np.float32), w[i], l.H, l.H, l.stride, l.pad))
        if ds is not None:
            l = L[ds]
            dys, _ = bn_bwd(ds, dres)
            dw[ds] = oracle.conv_wgrad(x_in.astype(np.float32), dys.astype(np.float32), l.R, l.R, l.stride, l.pad)
            sc = _r(oracle.conv_dgrad(dys.astype(np.float32), w[ds], l.H, l.H, l.stride, l.pad))
        else:
            sc = dres
        d_cur = _r(d_t + sc)
    if cs.pool:
        d_cur = _r(oracle.maxpool_bwd(d_cur, sel, L[0].P, L[0].P))
    dy0, _ = bn_bwd(0, d_cur)
    l0 = L[0]
    dw[0] = oracle.conv_wgrad(x0.astype(np.float32), dy0.astype(np.float32), l0.R, l0.R, l0.stride, l0.pad)
    return out, dw, dgm, dbt


@pytest.mark.parametrize("fused,streams", [(True, 0), (False, 0), (True, 2)], ids=["fused", "stand-alone", "fused-side-streams"])
def test_chained_stage_stem_pool_and_three_blocks(fused, streams):
    """Stem, max pooling and the whole first stage of a pruned ResNet-50 (a projection-shortcut block and two identity blocks),
    forward and backward, through the chained step -- with the normalisation statistics taken in the convolution epilogues
    and with the stand-alone normalisation, on one stream and with the weight gradients and the projection shortcut on side
    streams -- against the oracle's composition."""
    from paper_1901_09290_b200 import harness
    c = Hh.ctx()
    N = 4
    dense = W.resnet50(64)                                   # 64x64 images: stem 32x32, pooled 16x16
    seed = W.BASE_SEED + 4200
    net = W.with_sizes(dense, W.random_keep(dense, seed, 0.3, 0.6))
    model = W.gen_model(net, seed)
    l0 = net.layers[0]
    x0 = _r(W.gen_image(N, l0.H, l0.H, l0.C, seed + 1).numpy())
    cs = harness.ChainedStep(c, net, N, seed, fused_stats=fused, algo=2, max_blocks=3, model=model,
                             x0=torch.from_numpy(x0.astype(np.float32)), wgrad_streams=streams)
    lo = net.layers[cs.out_index]
    g_last = _r(W.gen_dy(N, lo.P, lo.P, lo.K, seed + 2).numpy() * 64)
    cs.g_last.zero_()
    cs.g_last[..., :lo.K] = torch.from_numpy(g_last.astype(np.float32)).to(torch.bfloat16).cuda()
    out_d = cs.forward()
    cs.backward()
    torch.cuda.synchronize()
    c.poll()
    c.set_wgrad_cta_limit(0)                                 # the context is shared with the other tests
    out, dw, dgm, dbt = _oracle_chain(cs, model, x0, g_last)
    f = lambda t, C: t.float().cpu().numpy()[..., :C].astype(np.float64)
    assert _rel(f(out_d, lo.K), out) < 1e-2
    # the backward chain on identical forward state: rounding of the stored gradients compounds along the eleven layers
    order = [i for b in reversed(cs.blocks) for i in ([b[1]] if b[1] is not None else []) + list(reversed(b[0]))] + [0]
    for rank, i in enumerate(order):
        tol = 5e-3 + 1e-3 * rank
        nm = net.layers[i].name
        assert _rel(cs.dm.g[i].cpu().numpy().astype(np.float64), dw[i]) < tol, (nm, _rel(cs.dm.g[i].cpu().numpy().astype(np.float64), dw[i]))
        assert _rel(cs.dg[i].cpu().numpy().astype(np.float64), dgm[i]) < tol, nm
        # the stem's dbeta sums 4096 signed terms that nearly cancel: its error is measured against a small number
        assert _rel(cs.db[i].cpu().numpy().astype(np.float64), dbt[i]) < (tol if i else 8e-2), nm
    # the lasso step still closes the iteration
    cs.update()
    torch.cuda.synchronize()
    c.poll()


def test_chained_step_at_bench_size_is_the_same_on_side_streams():
    """The whole pruned ResNet-50 at batch 64 as the bench chains it: with the weight gradients and the projection shortcuts on
    side streams every result must be what it is on one stream (a missing dependency between the streams would show as a
    difference): activations, data gradients, gamma/beta gradients bit for bit (the same launches); weight gradients to
    rounding (their CTA limit, hence the split of their sums, differs between the two modes) and bit for bit between two runs
    of the same mode."""
    from paper_1901_09290_b200 import harness
    c = Hh.ctx()
    net = W.resnet50()
    seed = W.BASE_SEED + 4
    netp = W.with_sizes(net, W.staged_keep_to_flops(net, seed, 0.60))
    model = W.gen_model(netp, seed + 5)
    runs = []
    for streams in (0, 2, 2):
        cs = harness.ChainedStep(c, netp, 64, seed + 5, fused_stats=True, algo=2, model=model, wgrad_streams=streams)
        out = cs.forward()
        cs.backward()
        torch.cuda.synchronize()
        c.poll()
        runs.append(dict(out=out.clone(), dw=[cs.dm.g[i].clone() for i in cs.used], dg=[cs.dg[i].clone() for i in cs.used],
                         db=[cs.db[i].clone() for i in cs.used], dy0=cs.dy[0].clone()))
        del cs
        torch.cuda.empty_cache()
    c.set_wgrad_cta_limit(0)
    one, a, b = runs
    for r in (a, b):
        assert torch.equal(r["out"], one["out"]) and torch.equal(r["dy0"], one["dy0"])
        for x, y in zip(r["dg"] + r["db"], one["dg"] + one["db"]):
            assert torch.equal(x, y)
        for x, y in zip(r["dw"], one["dw"]):
            scale = float(y.abs().max()) + 1e-30
            assert float((x - y).abs().max()) <= 2e-4 * scale           # fp32 sums over up to 800 K pixels, split differently
    for x, y in zip(a["dw"], b["dw"]):
        assert torch.equal(x, y)
