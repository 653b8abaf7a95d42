"""Bit-exact parity of keep maps and the compaction gather with the oracle; the config-1 chain."""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_09290_b200 import binding as B
from paper_1901_09290_b200 import workloads as W
from tests import helpers as Hh
from tests.test_gpu_lasso import DevModel

pytestmark = pytest.mark.gpu


def reconfigure(dm: DevModel):
    """detect -> plan -> allocate the smaller model -> gather. Returns (new DevModel, new2old per space)."""
    net = dm.net
    c = Hh.ctx()
    B.pt_find_zero_groups(c, dm.arr, 1e-4, False, dm.ws)
    g_old = dm.graph()
    new2old = torch.full((sum(net.space_sizes),), -7, dtype=torch.int32, device="cuda")
    sizes = B.pt_reconfigure_plan(c, g_old, new2old)
    new_net = W.with_sizes(net, sizes)
    empty = W.Model(new_net,
                    [torch.full((l.K, l.R, l.R, l.C), 5555.0) for l in new_net.layers],
                    [torch.full((l.K, l.R, l.R, l.C), 5555.0) for l in new_net.layers],
                    [torch.zeros((l.K, l.R, l.R, l.C)) for l in new_net.layers],
                    [[torch.full((l.K,), 5555.0) for _ in range(4)] for l in new_net.layers])
    dn = DevModel(empty)
    B.pt_reconfigure(c, g_old, new2old, dn.graph())
    torch.cuda.synchronize()
    c.poll()
    maps, off = [], 0
    n2o = new2old.cpu().numpy()
    for s, size in enumerate(net.space_sizes):
        seg = n2o[off:off + size]
        assert np.all(seg[sizes[s]:] == -1)
        maps.append(seg[:sizes[s]].copy())
        off += size
    return dn, maps, sizes


def check_against_oracle(model: W.Model, dm: DevModel, dn: DevModel, maps, sizes, w_src=None):
    net = model.net
    ws = w_src if w_src is not None else [w.numpy() for w in model.w]
    zz = [oracle.find_zero_groups(w) for w in ws]
    graph = oracle.Graph(list(net.space_sizes), list(net.space_fixed), [(l.in_space, l.out_space) for l in net.layers])
    keep = oracle.keep_sets(graph, [z[0] for z in zz], [z[1] for z in zz])
    for s in range(len(net.space_sizes)):
        assert maps[s].tolist() == keep[s].tolist(), net.space_names[s]
        assert sizes[s] == len(keep[s])
    for li, l in enumerate(net.layers):
        mk, mc = keep[l.out_space], keep[l.in_space]
        if len(mk) == 0 or len(mc) == 0:
            continue
        ref_w = oracle.gather_weight(ws[li], mk, mc)
        assert np.array_equal(dn.w[li].cpu().numpy().view(np.uint32), ref_w.view(np.uint32)), l.name
        ref_v = oracle.gather_weight(dm.v[li].cpu().numpy(), mk, mc)
        assert np.array_equal(dn.v[li].cpu().numpy().view(np.uint32), ref_v.view(np.uint32)), l.name
        # shadow: gathered from the old shadow, bit for bit
        old_sh = dm.wb[li][..., :l.C].float().cpu().numpy()
        ref_sh = oracle.gather_weight(old_sh, mk, mc)
        assert np.array_equal(dn.wb[li][..., :len(mc)].float().cpu().numpy(), ref_sh), l.name
        for b in range(4):
            assert np.array_equal(dn.bn[li][b].cpu().numpy(), oracle.gather_vector(model.bn[li][b].numpy(), mk))
    return keep


def test_config1_chain_step_detect_compact():
    """Config 1: conv training step -> lasso step with g = wgrad -> detection -> compaction gives C' = 13, K' = 27."""
    N, H, C, K, R = 8, 16, 16, 32, 3
    seed = W.BASE_SEED + 1
    net = W.single_layer(C, K, R, H)
    kept = W.choose_kept(net, [13, 27], seed)
    model = W.gen_model(net, seed, kept=kept, with_grad=False)
    cz = np.setdiff1d(np.arange(C), kept[0])
    kz = np.setdiff1d(np.arange(K), kept[1])
    x = W.gen_act(N, H, H, C, seed + 7)
    dy = W.gen_dy(N, H, H, K, seed + 8)
    x[..., cz] = 0
    dy[..., kz] = 0
    dm = DevModel(model)
    c = Hh.ctx()
    d = B.make_conv_desc(N, H, H, C, K, R, R, 1, 1)
    xd, dyd = Hh.to_dev_padded(x, W.pad8(C)), Hh.to_dev_padded(dy, W.pad8(K))
    B.pt_conv_wgrad(c, d, xd, dyd, dm.g[0], Hh.conv_ws(d, B.PT_CONV_WGRAD))
    B.pt_group_lasso_sgd_step(c, dm.arr, 1e-4, 0.1, 0.9, 0.0, dm.reg, dm.ws)
    torch.cuda.synchronize()
    # oracle chain on the same inputs
    dw = oracle.conv_wgrad(x.numpy(), dy.numpy(), R, R, 1, 1)
    w_new, v_new, *_ = oracle.lasso_sgd(model.w[0].numpy(), dw.astype(np.float32), model.v[0].numpy(), 1e-4, 0.1, 0.9)
    zo, zi = oracle.find_zero_groups(w_new.astype(np.float32))
    assert int(zo.sum()) == 5 and int(zi.sum()) == 3
    # stage-wise bit-exact comparison: the oracle's detection/compaction is fed the GPU's own post-step weights
    w_gpu = dm.w[0].cpu().numpy().copy()
    dn, maps, sizes = reconfigure(dm)
    assert sizes == [13, 27]
    assert maps[0].tolist() == kept[0].tolist() and maps[1].tolist() == kept[1].tolist()
    check_against_oracle(model, dm, dn, maps, sizes, w_src=[w_gpu])
    # end to end the chain agrees with the all-oracle chain as well
    assert maps[1].tolist() == np.nonzero(zo == 0)[0].tolist() and maps[0].tolist() == np.nonzero(zi == 0)[0].tolist()
    Hh.check_update(dn.w[0], oracle.gather_weight(w_new.astype(np.float32), maps[1], maps[0]).astype(np.float64), "w'")
    # dense variant: no zero groups in x/dy/w -> nothing is pruned
    model2 = W.gen_model(net, seed + 1)
    dn2, maps2, sizes2 = reconfigure(DevModel(model2))
    assert sizes2 == [C, K]


def test_resnet32_union_with_decoys():
    net = W.resnet32()
    kept = W.choose_kept(net, W.random_keep(net, W.BASE_SEED + 2), W.BASE_SEED + 2)
    model = W.gen_model(net, W.BASE_SEED + 2, kept=kept, decoys=2)
    dm = DevModel(model)
    dn, maps, sizes = reconfigure(dm)
    keep = check_against_oracle(model, dm, dn, maps, sizes)
    for s in range(len(kept)):
        assert keep[s].tolist() == kept[s].tolist()


def test_vgg16_plain_stack_reconfiguration():
    """No shared node anywhere: every space has one writer and one reader, and a channel goes only if both agree."""
    net = W.vgg(16)
    kept = W.choose_kept(net, W.random_keep(net, W.BASE_SEED + 8), W.BASE_SEED + 8)
    model = W.gen_model(net, W.BASE_SEED + 8, kept=kept, decoys=2)
    dm = DevModel(model)
    dn, maps, sizes = reconfigure(dm)
    keep = check_against_oracle(model, dm, dn, maps, sizes)
    for s in range(len(kept)):
        assert keep[s].tolist() == kept[s].tolist()


def test_bottleneck_config3_counts():
    net = W.bottleneck_stage3()
    kept = W.choose_kept(net, [371, 93, 77], W.BASE_SEED + 3)
    model = W.gen_model(net, W.BASE_SEED + 3, kept=kept, decoys=2)
    dm = DevModel(model)
    dn, maps, sizes = reconfigure(dm)
    assert sizes == [371, 93, 77]
    check_against_oracle(model, dm, dn, maps, sizes)


def test_resnet50_full_reconfiguration():
    net = W.resnet50()
    counts = W.staged_keep_to_flops(net, W.BASE_SEED + 4)
    kept = W.choose_kept(net, counts, W.BASE_SEED + 4)
    model = W.gen_model(net, W.BASE_SEED + 4, kept=kept, decoys=2)
    dm = DevModel(model)
    dn, maps, sizes = reconfigure(dm)
    assert sizes == counts
    check_against_oracle(model, dm, dn, maps, sizes)


def test_empty_keep_set_and_second_reconfiguration():
    # a space whose every member is zero is reported with size 0; the layers around it are skipped
    net = W.bottleneck_stage3(8)
    kept = [np.arange(512, dtype=np.int32), np.arange(0, dtype=np.int32), np.arange(100, dtype=np.int32)]
    model = W.gen_model(net, 5, kept=kept)
    dm = DevModel(model)
    dn, maps, sizes = reconfigure(dm)
    assert sizes == [512, 0, 100]
    # composing two reconfigurations equals one with the composed map
    net2 = W.resnet32()
    keptA = W.choose_kept(net2, W.random_keep(net2, 11, 0.6, 0.9), 11)
    m = W.gen_model(net2, 12, kept=keptA)
    dmA = DevModel(m)
    dnA, mapsA, sizesA = reconfigure(dmA)
    for li, l in enumerate(dnA.net.layers):       # kill one more channel of every non-fixed space in the small model
        pass
    s_kill = 3
    for li, l in enumerate(dnA.net.layers):
        if l.out_space == s_kill:
            dnA.w[li][0] = 0
        if l.in_space == s_kill:
            dnA.w[li][:, :, :, 0] = 0
    dnB, mapsB, sizesB = reconfigure(dnA)
    assert sizesB[s_kill] == sizesA[s_kill] - 1
    for li, l in enumerate(net2.layers):
        mk = mapsA[l.out_space][mapsB[l.out_space]]
        mc = mapsA[l.in_space][mapsB[l.in_space]]
        ref = oracle.gather_weight(m.w[li].numpy(), mk, mc)
        assert np.array_equal(dnB.w[li].cpu().numpy(), ref)


def test_repeated_reconfiguration_reads_current_contents_and_rebuilds_for_new_arguments():
    """A repeated call with the same arguments launches from the cached gather table: the table holds addresses and shapes
    only, so the second call must carry over whatever the source buffers hold by then; a call with other destinations must
    not reuse it."""
    net = W.resnet32()
    kept = W.choose_kept(net, W.random_keep(net, W.BASE_SEED + 12), W.BASE_SEED + 12)
    model = W.gen_model(net, W.BASE_SEED + 12, kept=kept, decoys=1)
    dm = DevModel(model)
    dn, maps, sizes = reconfigure(dm)
    check_against_oracle(model, dm, dn, maps, sizes)
    c = Hh.ctx()
    # same masks and maps; the kept entries of the source get new values (zero groups stay zero, so the plan stands)
    new2old = torch.full((sum(net.space_sizes),), -1, dtype=torch.int32, device="cuda")
    off = 0
    for s, size in enumerate(net.space_sizes):
        new2old[off:off + sizes[s]] = torch.from_numpy(maps[s]).cuda()
        off += size
    g_old, g_new = dm.graph(), dn.graph()
    B.pt_reconfigure(c, g_old, new2old, g_new)          # builds the table for these arguments
    for w in dm.w:
        w.mul_(3.0)
    for v in dm.v:
        v.add_(0.25)
    B.pt_reconfigure(c, g_old, new2old, g_new)          # same arguments: cached table, current contents
    torch.cuda.synchronize()
    c.poll()
    for li, l in enumerate(net.layers):
        mk, mc = maps[l.out_space], maps[l.in_space]
        ref_w = oracle.gather_weight(dm.w[li].cpu().numpy(), mk, mc)
        ref_v = oracle.gather_weight(dm.v[li].cpu().numpy(), mk, mc)
        assert np.array_equal(dn.w[li].cpu().numpy().view(np.uint32), ref_w.view(np.uint32)), l.name
        assert np.array_equal(dn.v[li].cpu().numpy().view(np.uint32), ref_v.view(np.uint32)), l.name
    # other destinations: a fresh model of the same shapes must be filled, and the first one left as it is
    snap = [w.clone() for w in dn.w]
    for w in dm.w:
        w.mul_(0.5)
    new_net = W.with_sizes(net, sizes)
    empty = W.Model(new_net, [torch.full((l.K, l.R, l.R, l.C), 7.0) for l in new_net.layers],
                    [torch.full((l.K, l.R, l.R, l.C), 7.0) for l in new_net.layers],
                    [torch.zeros((l.K, l.R, l.R, l.C)) for l in new_net.layers],
                    [[torch.full((l.K,), 7.0) for _ in range(4)] for l in new_net.layers])
    d2 = DevModel(empty)
    B.pt_reconfigure(c, g_old, new2old, d2.graph())
    torch.cuda.synchronize()
    c.poll()
    for li, l in enumerate(net.layers):
        mk, mc = maps[l.out_space], maps[l.in_space]
        ref_w = oracle.gather_weight(dm.w[li].cpu().numpy(), mk, mc)
        assert np.array_equal(d2.w[li].cpu().numpy().view(np.uint32), ref_w.view(np.uint32)), l.name
        assert torch.equal(dn.w[li], snap[li]), l.name


def test_new_graph_larger_than_the_plan_is_reported_and_reads_nothing_out_of_range():
    """A destination model with one channel more than pt_reconfigure_plan counted makes the gather meet the -1 padding of
    the keep map: the entry is skipped (guard values stay in place) and the next poll reports PT_ERR_INVALID_ARG."""
    net = W.bottleneck_stage3(8)
    kept = W.choose_kept(net, [300, 90, 70], W.BASE_SEED + 13)
    model = W.gen_model(net, W.BASE_SEED + 13, kept=kept)
    dm = DevModel(model)
    c = Hh.ctx()
    B.pt_find_zero_groups(c, dm.arr, 1e-4, False, dm.ws)
    new2old = torch.full((sum(net.space_sizes),), -7, dtype=torch.int32, device="cuda")
    sizes = B.pt_reconfigure_plan(c, dm.graph(), new2old)
    assert sizes == [300, 90, 70]
    bad = [sizes[0], sizes[1] + 1, sizes[2]]                      # one channel too many in the first internal space
    bad_net = W.with_sizes(net, bad)
    guard = 5555.0
    empty = W.Model(bad_net, [torch.full((l.K, l.R, l.R, l.C), guard) for l in bad_net.layers],
                    [torch.full((l.K, l.R, l.R, l.C), guard) for l in bad_net.layers],
                    [torch.zeros((l.K, l.R, l.R, l.C)) for l in bad_net.layers],
                    [[torch.full((l.K,), guard) for _ in range(4)] for l in bad_net.layers])
    dn = DevModel(empty)
    B.pt_reconfigure(c, dm.graph(), new2old, dn.graph())
    torch.cuda.synchronize()
    with pytest.raises(B.PtError) as e:
        c.poll()
    assert e.value.status == 1                                     # PT_ERR_INVALID_ARG
    c.poll()
    # layer 0 writes space 1: its extra output channel (index 90) kept the guard in w, v and the BN vectors; the valid part
    # is the ordinary gather
    l0 = bad_net.layers[0]
    assert l0.K == 91
    assert torch.all(dn.w[0][90] == guard) and torch.all(dn.v[0][90] == guard)
    for b in range(4):
        assert float(dn.bn[0][b][90]) == guard
    ref = oracle.gather_weight(model.w[0].numpy(), kept[1], kept[0])
    assert np.array_equal(dn.w[0][:90].cpu().numpy(), ref)
    # layer 1 reads space 1: its extra input channel kept the guard
    assert torch.all(dn.w[1][:, :, :, 90] == guard)
