"""Parity of the channel-gating kernels (Sec. 4.2) with the oracle: index work and data movement are bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_09290_b200 import binding as B
from paper_1901_09290_b200 import workloads as W
from tests import helpers as Hh

pytestmark = pytest.mark.gpu


def _dev_act(a: np.ndarray, ld: int, fill=float("nan")):
    """[npix][C] fp32 values (bf16-representable) -> device bf16 [npix][ld] with poisoned pad lanes."""
    t = torch.full((a.shape[0], ld), fill, dtype=torch.bfloat16)
    t[:, :a.shape[1]] = torch.from_numpy(a).to(torch.bfloat16)
    return t.cuda()


@pytest.mark.parametrize("n", [1, 5, 64, 1000, 1024, 1025, 2048, 3001])
def test_dense_channel_list(n):
    g = np.random.default_rng(n)
    for frac in (0.0, 0.3, 1.0):
        z = (g.random(n) < frac).astype(np.uint8)
        idx = torch.full((n,), 77, dtype=torch.int32, device="cuda")
        cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.pt_dense_channel_list(Hh.ctx(), torch.from_numpy(z).cuda(), n, idx, cnt)
        torch.cuda.synchronize()
        want = oracle.dense_channel_list(z)
        assert int(cnt.item()) == len(want)
        got = idx.cpu().numpy()
        assert got[:len(want)].tolist() == want.tolist() and np.all(got[len(want):] == -1)


# (npix, node channels, selected channels)
CASES = [(1, 8, 1), (37, 11, 5), (64 * 14 * 14, 154, 93), (1000, 2048, 700), (513, 260, 260), (4099, 24, 17)]


@pytest.mark.parametrize("case", CASES)
def test_gather_and_scatter_add(case):
    npix, c_node, n_sel = case
    g = np.random.default_rng(W.BASE_SEED + npix)
    idx = g.permutation(c_node)[:n_sel].astype(np.int32)            # any order
    ld_n, ld_s = W.pad8(c_node), W.pad8(n_sel)
    node = W.bf16_round(torch.randn((npix, c_node), generator=torch.Generator().manual_seed(npix))).numpy()
    branch = W.bf16_round(torch.randn((npix, n_sel), generator=torch.Generator().manual_seed(npix + 1))).numpy()
    d_node, d_branch, d_idx = _dev_act(node, ld_n), _dev_act(branch, ld_s), torch.from_numpy(idx).cuda()
    c = Hh.ctx()
    # gather: pad lanes of the source are never read, pad lanes of the result are zeros
    out = torch.full((npix, ld_s), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.pt_channel_gather(c, d_node, ld_n, c_node, d_idx, n_sel, out, ld_s, npix)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy()
    assert np.array_equal(got[:, :n_sel], oracle.channel_gather(node, idx))
    assert np.all(got[:, n_sel:] == 0)
    # scatter-add with and without ReLU, out of place and in place, and with no node input
    for relu in (False, True):
        res = torch.full((npix, ld_n), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.pt_channel_scatter_add(c, d_branch, ld_s, d_idx, n_sel, d_node, res, ld_n, c_node, npix, relu)
        torch.cuda.synchronize()
        got = res.float().cpu().numpy()
        assert np.array_equal(got[:, :c_node], oracle.channel_scatter_add(branch, idx, node, relu=relu))
        assert np.all(got[:, c_node:] == 0)
    inplace = d_node.clone()
    B.pt_channel_scatter_add(c, d_branch, ld_s, d_idx, n_sel, inplace, inplace, ld_n, c_node, npix, False)
    res0 = torch.empty((npix, ld_n), dtype=torch.bfloat16, device="cuda")
    B.pt_channel_scatter_add(c, d_branch, ld_s, d_idx, n_sel, None, res0, ld_n, c_node, npix, False)
    torch.cuda.synchronize()
    assert np.array_equal(inplace.float().cpu().numpy()[:, :c_node], oracle.channel_scatter_add(branch, idx, node))
    assert np.array_equal(res0.float().cpu().numpy()[:, :c_node], oracle.channel_scatter_add(branch, idx, None, c_node=c_node))
    c.poll()


def test_gated_branch_equals_the_sparse_layer_on_the_gpu():
    """Gather -> convolution on the dense channels -> scatter-add reproduces the un-reconfigured layer whose sparsified
    groups are zero, up to the convolution's own tolerance."""
    N, H, C, K = 4, 14, 93, 77
    seed = W.BASE_SEED + 61
    g = np.random.default_rng(seed)
    zin, zout = (g.random(C) < 0.4).astype(np.uint8), (g.random(K) < 0.4).astype(np.uint8)
    x = W.gen_act(N, H, H, C, seed)
    w = W.bf16_round(W.gen_weight(K, 3, 3, C, seed + 1))
    w[:, :, :, torch.from_numpy(zin).bool()] = 0
    w[torch.from_numpy(zout).bool()] = 0
    ii, oi = oracle.dense_channel_list(zin), oracle.dense_channel_list(zout)
    c = Hh.ctx()
    npix = N * H * H
    d_x = _dev_act(x.reshape(npix, C).numpy(), W.pad8(C))
    xs = torch.empty((npix, W.pad8(len(ii))), dtype=torch.bfloat16, device="cuda")
    B.pt_channel_gather(c, d_x, W.pad8(C), C, torch.from_numpy(ii).cuda(), len(ii), xs, W.pad8(len(ii)), npix)
    torch.cuda.synchronize()
    xs_host = xs[:, :len(ii)].float().cpu().reshape(N, H, H, len(ii))
    w_dense = w[torch.from_numpy(oi).long()][:, :, :, torch.from_numpy(ii).long()].contiguous()
    dy = W.gen_dy(N, H, H, len(oi), seed + 2)
    y = Hh.run_conv_all(N, H, H, len(ii), len(oi), 3, 1, 1, xs_host, w_dense, dy, algo=2)[0]
    ld_y = y.shape[-1]
    node = torch.zeros((npix, W.pad8(K)), dtype=torch.bfloat16, device="cuda")
    B.pt_channel_scatter_add(c, y.reshape(npix, ld_y), ld_y, torch.from_numpy(oi).cuda(), len(oi), None, node, W.pad8(K), K, npix, False)
    torch.cuda.synchronize()
    want = oracle.conv_fwd(x.numpy(), w.numpy(), 1, 1)
    Hh.check_conv(node.reshape(N, H, H, W.pad8(K)), K, want, what="gated branch")
    assert torch.all(node[:, torch.from_numpy(np.flatnonzero(zout)).long().cuda()] == 0)
    c.poll()


def test_bad_arguments_and_indices():
    c = Hh.ctx()
    a = torch.zeros((16, 16), dtype=torch.bfloat16, device="cuda")
    b = torch.zeros((16, 8), dtype=torch.bfloat16, device="cuda")
    idx = torch.tensor([0, 3, 5], dtype=torch.int32, device="cuda")
    with pytest.raises(B.PtError):
        B.pt_channel_gather(c, a, 12, 12, idx, 3, b, 8, 16)           # pitch not a multiple of 8
    with pytest.raises(B.PtError):
        B.pt_channel_gather(c, a, 16, 16, idx, 3, b, 0, 16)           # pitch below the selection
    with pytest.raises(B.PtError):
        B.pt_channel_scatter_add(c, b, 8, idx, 3, None, a, 16, 2, 16, 0)   # more selected channels than the node has
    # an index outside the tensor is skipped (nothing is read or written there) and reported at the next poll
    bad = torch.tensor([0, 99, 5], dtype=torch.int32, device="cuda")
    B.pt_channel_gather(c, a, 16, 16, bad, 3, b, 8, 16)
    torch.cuda.synchronize()
    with pytest.raises(B.PtError):
        c.poll()
    c.poll()                                                          # the status word was cleared
