"""Parity of the group-lasso SGD step and zero-group detection with the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_09290_b200 import binding as B
from paper_1901_09290_b200 import workloads as W
from tests import helpers as Hh

pytestmark = pytest.mark.gpu


from paper_1901_09290_b200.harness import DeviceModel


def DevModel(model):
    return DeviceModel(Hh.ctx(), model)


def _check_step(model: W.Model, lam, lr, mu, wd):
    dm = DevModel(model)
    B.pt_group_lasso_sgd_step(Hh.ctx(), dm.arr, lam, lr, mu, wd, dm.reg, dm.ws)
    torch.cuda.synchronize()
    Hh.ctx().poll()
    reg_ref = 0.0
    for li, l in enumerate(model.net.layers):
        reg_in = model.net.space_stage[l.in_space] != 0
        w_new, v_new, s_out, s_in, reg = oracle.lasso_sgd(model.w[li].numpy(), model.g[li].numpy(), model.v[li].numpy(),
                                                          lam, lr, mu, wd, reg_in=reg_in, reg_out=True)
        reg_ref += reg
        Hh.check_update(dm.w[li], w_new, f"{l.name} w")
        Hh.check_update(dm.v[li], v_new, f"{l.name} v")
        np.testing.assert_allclose(dm.sq_out[li].cpu().numpy(), s_out, rtol=2e-5, atol=1e-30)
        np.testing.assert_allclose(dm.sq_in[li].cpu().numpy(), s_in, rtol=2e-5, atol=1e-30)
        # the shadow is the round-to-nearest-even bf16 of the GPU's own new fp32 weights, bit for bit
        assert torch.equal(dm.wb[li][..., :l.C], dm.w[li].to(torch.bfloat16)), l.name
        assert torch.all(torch.isnan(dm.wb[li][..., l.C:].float())), "shadow pad lanes were written"
        # zero groups stay exactly zero
        zo = (model.w[li].abs().amax(dim=(1, 2, 3)) == 0) & (model.g[li].abs().amax(dim=(1, 2, 3)) == 0) & \
             (model.v[li].abs().amax(dim=(1, 2, 3)) == 0)
        if zo.any():
            assert torch.all(dm.w[li][zo.cuda()] == 0) and torch.all(dm.v[li][zo.cuda()] == 0)
    assert abs(dm.reg.item() - reg_ref) <= 1e-5 * reg_ref
    return dm


def test_step_single_layer_config1():
    net = W.single_layer(16, 32, 3, 16)
    kept = W.choose_kept(net, [13, 27], W.BASE_SEED + 1)
    model = W.gen_model(net, W.BASE_SEED + 1, kept=kept)
    _check_step(model, 1e-4, 0.1, 0.9, 0.0)


@pytest.mark.parametrize("shape", [(1, 1, 1), (5, 3, 3), (33, 1, 70), (7, 3, 300), (64, 7, 3), (300, 1, 2500), (9, 3, 93)])
def test_step_odd_shapes(shape):
    K, R, C = shape
    net = W.single_layer(C, K, R, 8)
    model = W.gen_model(net, W.BASE_SEED + 50 + K)
    _check_step(model, 3e-3, 0.05, 0.9, 1e-4)


def test_step_resnet32_with_zero_groups_and_decoys():
    net = W.resnet32()
    kept = W.choose_kept(net, W.random_keep(net, W.BASE_SEED + 2), W.BASE_SEED + 2)
    model = W.gen_model(net, W.BASE_SEED + 2, kept=kept, decoys=2)
    _check_step(model, 1e-4, 0.1, 0.9, 0.0)


def test_step_is_run_to_run_identical_and_table_cache_reuploads():
    net = W.resnet32()
    model = W.gen_model(net, W.BASE_SEED + 3)
    a = _check_step(model, 1e-4, 0.1, 0.9, 0.0)
    b = _check_step(model, 1e-4, 0.1, 0.9, 0.0)          # new buffers: the cached table must be refreshed
    for x, y in zip(a.w, b.w):
        assert torch.equal(x, y)


def test_step_in_two_calls_equals_the_single_call():
    """pt_group_lasso_norms (on another stream, before the gradients exist) + pt_group_lasso_sgd_apply == pt_group_lasso_sgd_step."""
    net = W.resnet32()
    kept = W.choose_kept(net, W.random_keep(net, W.BASE_SEED + 6), W.BASE_SEED + 6)
    model = W.gen_model(net, W.BASE_SEED + 6, kept=kept, decoys=1)
    one = _check_step(model, 2e-4, 0.1, 0.9, 1e-4)          # single call, checked against the oracle
    dm = DevModel(model)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    B.pt_group_lasso_norms(Hh.ctx(), dm.arr, dm.reg, dm.ws, side)
    torch.cuda.current_stream().wait_stream(side)
    B.pt_group_lasso_sgd_apply(Hh.ctx(), dm.arr, 2e-4, 0.1, 0.9, 1e-4, dm.ws)
    torch.cuda.synchronize()
    Hh.ctx().poll()
    for li in range(len(model.net.layers)):
        assert torch.equal(dm.w[li], one.w[li]) and torch.equal(dm.v[li], one.v[li]) and torch.equal(dm.wb[li].view(torch.int16), one.wb[li].view(torch.int16))
        assert torch.equal(dm.sq_out[li], one.sq_out[li]) and torch.equal(dm.sq_in[li], one.sq_in[li])
    assert dm.reg.item() == one.reg.item()


def test_apply_by_layer_ranges_equals_the_single_call():
    """pt_group_lasso_sgd_apply_layers over ranges that cover every layer once == pt_group_lasso_sgd_apply, bit for bit."""
    net = W.resnet32()
    model = W.gen_model(net, W.BASE_SEED + 7, kept=W.choose_kept(net, W.random_keep(net, W.BASE_SEED + 7), W.BASE_SEED + 7))
    one = DevModel(model)
    B.pt_group_lasso_norms(Hh.ctx(), one.arr, one.reg, one.ws)
    B.pt_group_lasso_sgd_apply(Hh.ctx(), one.arr, 2e-4, 0.1, 0.9, 1e-4, one.ws)
    dm = DevModel(model)
    B.pt_group_lasso_norms(Hh.ctx(), dm.arr, dm.reg, dm.ws)
    n = len(net.layers)
    for first, count in [(20, n - 20), (0, 1), (7, 13), (1, 6), (5, 0)]:      # any order; an empty range is a no-op
        B.pt_group_lasso_sgd_apply_layers(Hh.ctx(), dm.arr, first, count, 2e-4, 0.1, 0.9, 1e-4, dm.ws)
    torch.cuda.synchronize()
    Hh.ctx().poll()
    for li in range(n):
        assert torch.equal(dm.w[li], one.w[li]) and torch.equal(dm.v[li], one.v[li]), net.layers[li].name
        assert torch.equal(dm.wb[li].view(torch.int16), one.wb[li].view(torch.int16))
    for bad in [(-1, 2), (n, 1), (3, n)]:
        with pytest.raises(B.PtError):
            B.pt_group_lasso_sgd_apply_layers(Hh.ctx(), dm.arr, bad[0], bad[1], 2e-4, 0.1, 0.9, 1e-4, dm.ws)


def test_step_resnet50_all_layers():
    net = W.resnet50()
    model = W.gen_model(net, W.BASE_SEED + 4)
    _check_step(model, 1e-4, 0.1, 0.9, 0.0)


def _check_detection(model: W.Model, thr=1e-4, zero_in_place=False):
    dm = DevModel(model)
    B.pt_find_zero_groups(Hh.ctx(), dm.arr, thr, zero_in_place, dm.ws)
    torch.cuda.synchronize()
    Hh.ctx().poll()
    for li, l in enumerate(model.net.layers):
        zo, zi = oracle.find_zero_groups(model.w[li].numpy(), thr)
        assert dm.z_out[li].cpu().numpy().tolist() == zo.tolist(), l.name
        assert dm.z_in[li].cpu().numpy().tolist() == zi.tolist(), l.name
        if zero_in_place:
            w = model.w[li].clone()
            w[torch.from_numpy(zo).bool()] = 0
            w[:, :, :, torch.from_numpy(zi).bool()] = 0
            assert torch.equal(dm.w[li].cpu().view(torch.int32), w.view(torch.int32))
            assert torch.all(dm.v[li].cpu()[torch.from_numpy(zo).bool()] == 0)
            assert torch.all(dm.wb[li][..., :l.C].float().cpu()[:, :, :, torch.from_numpy(zi).bool()] == 0)
    return dm


def test_detection_boundaries():
    thr = np.float32(1e-4)
    net = W.single_layer(5, 6, 2, 8)
    model = W.gen_model(net, 1)
    w = model.w[0]
    w[:] = 1.0
    w[0] = float(thr)
    w[1] = float(np.nextafter(thr, np.float32(0)))
    w[2] = 0.0
    w[2, 0, 1, 3] = float("nan")
    w[3] = 0.0
    w[4] = -0.99e-4
    w[5, 0, 0, :] = 0.0
    w[5, 0, 1, 2] = -1e-3
    w[:, :, :, 4] = 0.5e-4
    dm = _check_detection(model, float(thr))
    assert dm.z_out[0].cpu().tolist() == [0, 1, 0, 1, 1, 0] and dm.z_in[0].cpu().tolist() == [0, 0, 0, 0, 1]


@pytest.mark.parametrize("zero_in_place", [False, True])
def test_detection_resnet32(zero_in_place):
    net = W.resnet32()
    kept = W.choose_kept(net, W.random_keep(net, W.BASE_SEED + 2), W.BASE_SEED + 2)
    model = W.gen_model(net, W.BASE_SEED + 2, kept=kept, decoys=2)
    # near-threshold groups: scale some rows to just below / above 1e-4
    model.w[3][1] *= 1e-6
    model.w[5][:, :, :, 2] *= 1e-7
    _check_detection(model, 1e-4, zero_in_place)


def test_detection_config1_counts():
    net = W.single_layer(16, 32, 3, 16)
    kept = W.choose_kept(net, [13, 27], W.BASE_SEED + 1)
    dm = _check_detection(W.gen_model(net, W.BASE_SEED + 1, kept=kept))
    assert int(dm.z_out[0].sum()) == 5 and int(dm.z_in[0].sum()) == 3


@pytest.mark.parametrize("n,classes,ld", [(1, 1, 1), (3, 10, 10), (64, 1000, 1000), (128, 100, 104), (37, 33, 40)])
def test_cross_entropy_and_set_coeff(n, classes, ld):
    """Eq. 3: cross-entropy of the first forward pass and lambda from the penalty ratio, against the fp64 oracle."""
    c = Hh.ctx()
    logits, labels = W.gen_logits(n, classes, W.BASE_SEED + 77 + n)
    zd = torch.full((n, ld), float("nan"), dtype=torch.float32, device="cuda")      # pad lanes must never be read
    zd[:, :classes] = logits
    ld_ = labels.cuda()
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    ws = torch.empty(max(16, B.pt_cross_entropy_workspace_bytes(n)), dtype=torch.uint8, device="cuda")
    B.pt_cross_entropy(c, zd, ld_, n, classes, ld, loss, ws)
    B.pt_cross_entropy(c, zd, ld_, n, classes, ld, loss, ws)                        # run-to-run identical
    ref = oracle.cross_entropy(logits.numpy(), labels.numpy())
    got = float(loss.cpu()[0])
    assert abs(got - ref) <= 1e-5 * max(1.0, abs(ref)), (got, ref)
    a = loss.clone()
    B.pt_cross_entropy(c, zd, ld_, n, classes, ld, loss, ws)
    assert torch.equal(a, loss)
    reg = torch.tensor([812.5], dtype=torch.float64, device="cuda")
    lam = torch.zeros(1, dtype=torch.float32, device="cuda")
    for ratio in (0.2, 0.25):
        B.pt_set_coeff(c, loss, reg, ratio, lam)
        want = oracle.set_coeff(got, 812.5, float(np.float32(ratio)))
        assert abs(float(lam.cpu()[0]) - want) <= 2e-7 * abs(want) + 1e-30
    B.pt_set_coeff(c, loss, torch.zeros(1, dtype=torch.float64, device="cuda"), 0.25, lam)
    assert float(lam.cpu()[0]) == 0.0
    for bad in (0.0, 1.0, -0.1, float("nan")):
        with pytest.raises(B.PtError):
            B.pt_set_coeff(c, loss, reg, bad, lam)
    with pytest.raises(B.PtError):
        B.pt_cross_entropy(c, zd, ld_, n, classes, classes - 1, loss, ws)
    torch.cuda.synchronize()
    c.poll()


def test_carried_steps_follow_the_oracle_chain_and_feed_the_detection():
    """Two steps in the carried form (22 bytes per parameter: the norms of W_{i+1} are taken while step i writes it) against
    two oracle steps; the sums the second step uses are those the first one left. Then the masks from the carried maxima
    must be the oracle's brute-force masks of the GPU's own weights, and equal to the reading detection's, bit for bit."""
    ctx = Hh.ctx()
    net = W.resnet32()
    kept = W.choose_kept(net, W.random_keep(net, W.BASE_SEED + 21), W.BASE_SEED + 21)
    model = W.gen_model(net, W.BASE_SEED + 21, kept=kept, decoys=2)
    lam, lr, mu, wd = 2e-3, 0.1, 0.9, 1e-4
    dm = DevModel(model)
    reg_next = torch.zeros(1, dtype=torch.float64, device="cuda")
    B.pt_group_lasso_norms(ctx, dm.arr, dm.reg, dm.ws)
    B.pt_group_lasso_sgd_step_carried(ctx, dm.arr, lam, lr, mu, wd, reg_next, dm.ws)
    torch.cuda.synchronize()
    ctx.poll()
    ref_w, ref_v = [], []
    reg0 = reg1 = 0.0
    for li, l in enumerate(net.layers):
        reg_in = net.space_stage[l.in_space] != 0
        w1, v1, s_out, s_in, reg = oracle.lasso_sgd(model.w[li].numpy(), model.g[li].numpy(), model.v[li].numpy(), lam, lr, mu, wd,
                                                     reg_in=reg_in, reg_out=True)
        reg0 += reg
        Hh.check_update(dm.w[li], w1, f"{l.name} w step 1")
        Hh.check_update(dm.v[li], v1, f"{l.name} v step 1")
        # sums of squares of the NEW weights, as the carried form leaves them
        w1f = w1.astype(np.float32).astype(np.float64)
        np.testing.assert_allclose(dm.sq_out[li].cpu().numpy(), (w1f ** 2).sum(axis=(1, 2, 3)), rtol=3e-5, atol=1e-30)
        np.testing.assert_allclose(dm.sq_in[li].cpu().numpy(), (w1f ** 2).sum(axis=(0, 1, 2)), rtol=3e-5, atol=1e-30)
        w2, v2, _, _, r1 = oracle.lasso_sgd(w1.astype(np.float32), model.g[li].numpy(), v1.astype(np.float32), lam, lr, mu, wd,
                                            reg_in=reg_in, reg_out=True)
        reg1 += r1
        ref_w.append(w2)
        ref_v.append(v2)
    assert abs(dm.reg.item() - reg0) <= 1e-5 * reg0
    assert abs(reg_next.item() - reg1) <= 2e-5 * reg1          # Eq. 2's sum of the new weights
    B.pt_group_lasso_sgd_step_carried(ctx, dm.arr, lam, lr, mu, wd, reg_next, dm.ws, with_maxima=True)
    torch.cuda.synchronize()
    ctx.poll()
    for li, l in enumerate(net.layers):
        # the second step starts from the first step's fp32 results, which differ from the oracle's fp64 ones by rounding
        g = dm.w[li].cpu().numpy().astype(np.float64)
        assert np.linalg.norm(g - ref_w[li]) <= 2e-5 * np.linalg.norm(ref_w[li]), l.name
        assert torch.equal(dm.wb[li][..., :l.C], dm.w[li].to(torch.bfloat16)), l.name
        # zero groups stay exactly zero
        zo = (model.w[li].abs().amax(dim=(1, 2, 3)) == 0) & (model.g[li].abs().amax(dim=(1, 2, 3)) == 0) & \
             (model.v[li].abs().amax(dim=(1, 2, 3)) == 0)
        if zo.any():
            assert torch.all(dm.w[li][zo.cuda()] == 0)
    # detection from the maxima the step left behind
    B.pt_find_zero_groups_carried(ctx, dm.arr, 1e-4, False, dm.ws)
    torch.cuda.synchronize()
    carried = [(dm.z_out[li].clone(), dm.z_in[li].clone()) for li in range(len(net.layers))]
    n_zero = 0
    for li, l in enumerate(net.layers):
        zo, zi = oracle.find_zero_groups(dm.w[li].cpu().numpy(), 1e-4)
        assert carried[li][0].cpu().numpy().tolist() == zo.tolist(), l.name
        assert carried[li][1].cpu().numpy().tolist() == zi.tolist(), l.name
        n_zero += int(zo.sum()) + int(zi.sum())
    assert n_zero > 0
    B.pt_find_zero_groups(ctx, dm.arr, 1e-4, False, dm.ws)
    torch.cuda.synchronize()
    ctx.poll()
    for li in range(len(net.layers)):
        assert torch.equal(dm.z_out[li], carried[li][0]) and torch.equal(dm.z_in[li], carried[li][1])


@pytest.mark.parametrize("shape", [(1, 1, 1), (64, 7, 3), (7, 3, 300), (33, 1, 143), (300, 1, 2500)])
def test_carried_step_odd_shapes(shape):
    K, R, C = shape
    ctx = Hh.ctx()
    net = W.single_layer(C, K, R, 8)
    model = W.gen_model(net, W.BASE_SEED + 80 + K)
    dm = DevModel(model)
    B.pt_group_lasso_norms(ctx, dm.arr, dm.reg, dm.ws)
    B.pt_group_lasso_sgd_step_carried(ctx, dm.arr, 3e-3, 0.05, 0.9, 1e-4, None, dm.ws, with_maxima=True)
    torch.cuda.synchronize()
    ctx.poll()
    reg_in = net.space_stage[net.layers[0].in_space] != 0
    w1, v1, *_ = oracle.lasso_sgd(model.w[0].numpy(), model.g[0].numpy(), model.v[0].numpy(), 3e-3, 0.05, 0.9, 1e-4, reg_in=reg_in, reg_out=True)
    Hh.check_update(dm.w[0], w1, "w")
    Hh.check_update(dm.v[0], v1, "v")
    wf = dm.w[0].cpu().numpy().astype(np.float64)
    np.testing.assert_allclose(dm.sq_out[0].cpu().numpy(), (wf ** 2).sum(axis=(1, 2, 3)), rtol=3e-5, atol=1e-30)
    np.testing.assert_allclose(dm.sq_in[0].cpu().numpy(), (wf ** 2).sum(axis=(0, 1, 2)), rtol=3e-5, atol=1e-30)
    B.pt_find_zero_groups_carried(ctx, dm.arr, 1e-4, False, dm.ws)
    torch.cuda.synchronize()
    zo, zi = oracle.find_zero_groups(dm.w[0].cpu().numpy(), 1e-4)
    assert dm.z_out[0].cpu().numpy().tolist() == zo.tolist() and dm.z_in[0].cpu().numpy().tolist() == zi.tolist()


def test_conv_right_behind_the_update_reads_the_new_weights():
    """Stream order: the update writes the bf16 shadow, and a convolution launched right behind it on the same stream must
    read the new values, although its weight producers do not wait for the kernel before them (the update therefore does
    not release its dependents early). The last layer of the table is updated by the last blocks of the sweep."""
    net = W.resnet50(image=32)
    counts = W.uniform_keep(net, 0.3)
    model = W.gen_model(W.with_sizes(net, counts), W.BASE_SEED + 77)
    dm = DevModel(model)
    li = len(model.net.layers) - 1
    l = model.net.layers[li]
    N, H = 2, 7
    d = B.make_conv_desc(N, H, H, l.C, l.K, l.R, l.R, 1, l.pad, W.pad16(l.C), W.pad16(l.K), W.pad8(l.C), 0, 2)
    x = W.gen_act(N, H, H, l.C, W.BASE_SEED + 78)
    xd = Hh.to_dev_padded(x, d.ldx)
    ws = Hh.conv_ws(d, 0)
    for it in range(6):
        y = Hh.out_buffer((N, H, H), l.K, d.ldy, False)
        B.pt_group_lasso_sgd_step(Hh.ctx(), dm.arr, 1e-4, 0.5, 0.9, 0.0, dm.reg, dm.ws)     # lr 0.5: every step moves the weights visibly
        B.pt_conv_fwd(Hh.ctx(), d, xd, dm.wb[li], y, ws)
        torch.cuda.synchronize()
        Hh.ctx().poll()
        w_now = dm.wb[li][..., :l.C].float().cpu().numpy()
        ref = oracle.conv_fwd(x.numpy(), w_now, 1, l.pad)
        Hh.check_conv(y, l.K, ref, what=f"iteration {it}")
