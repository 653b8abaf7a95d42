"""Parity on whole networks and at the bench's full sizes.

* config 2: every layer of the pruned ResNet-32 stack at batch 128, full tensors.
* config 4 at batch 2: every layer of the pruned ResNet-50, full tensors (identical channel shapes to the bench).
* config 4 / 5 at the bench's batch sizes, through the same harness buffers and launch path (CUDA-graph replay):
  4096 seeded sampled outputs per tensor, each computed alone by the oracle, plus all of dw for the smallest layers.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_09290_b200 import binding as B
from paper_1901_09290_b200 import harness
from paper_1901_09290_b200 import workloads as W
from tests import helpers as Hh

pytestmark = pytest.mark.gpu


def _layer_inputs(l, N, seed, first):
    x = (W.gen_image if first else W.gen_act)(N, l.H, l.H, l.C, seed)
    w = W.bf16_round(W.gen_weight(l.K, l.R, l.R, l.C, seed + 1))
    dy = W.gen_dy(N, l.P, l.P, l.K, seed + 2)
    return x, w, dy


def _full_layer_check(l, N, seed, first):
    x, w, dy = _layer_inputs(l, N, seed, first)
    # algo = 2: the tcgen05 kernels or an error -- a shape they decline must fail here, not pass on the CUDA-core kernels
    y, dx, dw, _ = Hh.run_conv_all(N, l.H, l.H, l.C, l.K, l.R, l.stride, l.pad, x, w, dy, algo=2)
    Hh.check_conv(y, l.K, oracle.conv_fwd(x.numpy(), w.numpy(), l.stride, l.pad), what=l.name + " fwd")
    Hh.check_conv(dx, l.C, oracle.conv_dgrad(dy.numpy(), w.numpy(), l.H, l.H, l.stride, l.pad), what=l.name + " dgrad")
    Hh.check_conv(dw, l.C, oracle.conv_wgrad(x.numpy(), dy.numpy(), l.R, l.R, l.stride, l.pad), what=l.name + " wgrad")


def test_config2_resnet32_every_layer_batch128():
    net = W.resnet32()
    counts = W.random_keep(net, W.BASE_SEED + 2)
    pruned = W.with_sizes(net, counts)
    for li, l in enumerate(pruned.layers):
        _full_layer_check(l, 128, W.layer_seed(2, li), li == 0)


def test_vgg13_plain_stack_every_layer_batch32():
    """The paper's second model family (Tab. 1: VGG on CIFAR): a plain 3x3 stack without short-cuts, pruned."""
    net = W.vgg(13)
    counts = W.random_keep(net, W.BASE_SEED + 8)
    pruned = W.with_sizes(net, counts)
    for li, l in enumerate(pruned.layers):
        _full_layer_check(l, 32, W.layer_seed(8, li), li == 0)


def test_vgg11_training_step_on_a_network_without_shortcuts():
    """The multi-stream, graph-replayed step on a plain stack: every weight gradient equals the single call on the same
    buffers, and the last layer's outputs agree with the oracle on the weights the step started from."""
    ctx = Hh.ctx()
    net = W.vgg(11)
    seed = W.BASE_SEED + 8
    counts = W.uniform_keep(net, 0.6)
    kept = W.choose_kept(net, counts, seed)
    ts = harness.TrainStep(ctx, net, counts, kept, 16, seed, algo=2, host_inputs=False, device_rng=True)
    ts.step()
    torch.cuda.synchronize()
    ts.build_graph(two_streams=True)
    li = len(net.layers) - 1
    l = ts.net.layers[li]
    ts.step()
    torch.cuda.synchronize()
    ctx.poll()
    # every step re-gathers the pruned model from the dense one before it trains: those are the weights the convs saw
    w_before = oracle.gather_weight(ts.md.wb[li][..., :net.layers[li].C].float().cpu().numpy(), kept[l.out_space], kept[l.in_space])
    x = ts.x[li][..., :l.C].float().cpu().numpy()
    dy = ts.dy[li][..., :l.K].float().cpu().numpy()
    Hh.check_conv(ts.y[li], l.K, oracle.conv_fwd(x, w_before, l.stride, l.pad), what="vgg fwd")
    Hh.check_conv(ts.dx[li], l.C, oracle.conv_dgrad(dy, w_before, l.H, l.H, l.stride, l.pad), what="vgg dgrad")
    for i in range(len(net.layers)):
        g_step = ts.mp.g[i].clone()
        ts.conv_wgrad(i)
        torch.cuda.synchronize()
        assert torch.equal(g_step, ts.mp.g[i]), net.layers[i].name
    Hh.check_conv(ts.mp.g[li], l.C, oracle.conv_wgrad(x, dy, l.R, l.R, l.stride, l.pad), what="vgg wgrad")


def test_config4_resnet50_every_layer_batch2():
    net = W.resnet50()
    counts = W.staged_keep_to_flops(net, W.BASE_SEED + 4)
    pruned = W.with_sizes(net, counts)
    for li, l in enumerate(pruned.layers):
        _full_layer_check(l, 2, W.layer_seed(4, li), li == 0)


def _bf16_ulp(a: np.ndarray) -> np.ndarray:
    return np.where(a != 0, np.exp2(np.floor(np.log2(np.maximum(np.abs(a), 1e-300))) - 7.0), 0.0)


def _f32_sampled_pass(ts, li, wsrc, x, dy, idx_y, idx_dx, y_bf16, dx_bf16, N):
    """The same layer once more with fp32 outputs (out_f32 = 1): the sampled elements are held to the PLAIN bound
    |err| <= 1e-2 * rms with no allowance for an output rounding, and the bf16 outputs of the step must be the
    nearest-even bf16 of these fp32 values (the kernels that serve a stride-2 data gradient differ between the two
    output types and may sum in another order: one bf16 ulp is allowed on at most 1 % of the samples there)."""
    ctx = Hh.ctx()
    l = ts.net.layers[li]
    d0 = ts.desc[li]
    d = B.make_conv_desc(N, l.H, l.H, l.C, l.K, l.R, l.R, l.stride, l.pad, d0.ldx, d0.ldy, d0.ldw, 1, 2)
    ws = [Hh.conv_ws(d, which) for which in (0, 1)]
    yf = torch.empty((N, l.P, l.P, d0.ldy), dtype=torch.float32, device="cuda")
    B.pt_conv_fwd(ctx, d, ts.x[li], ts.mp.wb[li], yf, ws[0])
    torch.cuda.synchronize()
    got = yf[..., :l.K].cpu().numpy().ravel()[idx_y]
    del yf
    ref = oracle.conv_fwd_samples(x, wsrc, idx_y, l.stride, l.pad)
    rms = float(np.sqrt(np.mean(ref ** 2))) if np.any(ref) else 1.0
    Hh.check_samples(got, ref, rms, False, f"{l.name} fwd fp32 N={N}")
    rn = torch.from_numpy(got.astype(np.float32)).to(torch.bfloat16).float().numpy()
    assert np.array_equal(rn, y_bf16), f"{l.name} fwd: bf16 output is not the nearest-even bf16 of the fp32 output"
    if li == 0:
        return
    dxf = torch.empty((N, l.H, l.H, d0.ldx), dtype=torch.float32, device="cuda")
    B.pt_conv_dgrad(ctx, d, ts.dy[li], ts.mp.wb[li], dxf, ws[1])
    torch.cuda.synchronize()
    got = dxf[..., :l.C].cpu().numpy().ravel()[idx_dx]
    del dxf
    ref = oracle.conv_dgrad_samples(dy, wsrc, idx_dx, l.H, l.H, l.stride, l.pad)
    rms = float(np.sqrt(np.mean(ref ** 2)))
    Hh.check_samples(got, ref, rms, False, f"{l.name} dgrad fp32 N={N}")
    rn = torch.from_numpy(got.astype(np.float32)).to(torch.bfloat16).float().numpy()
    diff = np.abs(rn.astype(np.float64) - dx_bf16)
    if l.stride == 1:
        assert np.array_equal(rn, dx_bf16), f"{l.name} dgrad: bf16 output is not the nearest-even bf16 of the fp32 output"
    else:
        assert np.all(diff <= _bf16_ulp(rn.astype(np.float64))) and np.mean(diff > 0) <= 0.01, f"{l.name} dgrad: bf16 vs fp32 outputs"


def _sampled_step_check(keep, N, layer_ids, n_samples=4096, full_dw_below=40000, f32_pass=False):
    """Runs the harness's graph-replayed training step at the bench's sizes on CPU-generated inputs and compares sampled
    outputs of the chosen layers with the oracle. algo = 2 throughout: a layer the tcgen05 kernels decline is an error."""
    ctx = Hh.ctx()
    net = W.resnet50()
    seed = W.BASE_SEED + 4
    counts = W.staged_keep_to_flops(net, seed, 0.60) if keep is None else W.uniform_keep(net, keep)
    kept = W.choose_kept(net, counts, seed)
    ts = harness.TrainStep(ctx, net, counts, kept, N, seed, algo=2, host_inputs=False, device_rng=True)
    ts.step()                       # eager: reconfiguration + training step (sets tables and attributes up)
    torch.cuda.synchronize()
    ts.build_graph(two_streams=True)
    ts.step()                       # the launch configuration the bench times
    torch.cuda.synchronize()
    ctx.poll()
    rng = np.random.default_rng(seed)
    if f32_pass:
        ts.reconfigure()            # the update has rewritten the pruned shadow: gather the weights the convs ran on again
        torch.cuda.synchronize()
    for li in layer_ids:
        l = ts.net.layers[li]
        # the buffers the step used, copied back: the oracle sees exactly the bits the kernels saw
        x = ts.x[li][..., :l.C].float().cpu().numpy()
        dy = ts.dy[li][..., :l.K].float().cpu().numpy()
        # the step's lasso update has already rewritten mp.wb: the convs ran on the weights gathered from the dense model
        wsrc = oracle.gather_weight(ts.md.wb[li][..., :ts.dense_net.layers[li].C].float().cpu().numpy(),
                                    kept[ts.net.layers[li].out_space], kept[ts.net.layers[li].in_space])
        y = ts.y[li][..., :l.K].float().cpu().numpy()
        idx = rng.integers(0, y.size, n_samples)
        idx_y, y_s = idx, y.ravel()[idx]
        ref = oracle.conv_fwd_samples(x, wsrc, idx, l.stride, l.pad)
        rms = float(np.sqrt(np.mean(ref ** 2))) if np.any(ref) else 1.0
        Hh.check_samples(y_s, ref, rms, True, f"{l.name} fwd N={N}")
        idx_dx, dx_s = None, None
        if li > 0:
            dx = ts.dx[li][..., :l.C].float().cpu().numpy()
            idx = rng.integers(0, dx.size, n_samples)
            idx_dx, dx_s = idx, dx.ravel()[idx]
            ref = oracle.conv_dgrad_samples(dy, wsrc, idx, l.H, l.H, l.stride, l.pad)
            rms = float(np.sqrt(np.mean(ref ** 2)))
            Hh.check_samples(dx_s, ref, rms, True, f"{l.name} dgrad N={N}")
        if f32_pass:
            _f32_sampled_pass(ts, li, wsrc, x, dy, idx_y, idx_dx, y_s, dx_s, N)
        dw = ts.mp.g[li].cpu().numpy()
        if dw.size <= full_dw_below:
            idx = np.arange(dw.size)
        else:
            idx = rng.integers(0, dw.size, 512)
        ref = oracle.conv_wgrad_samples(x, dy, idx, l.R, l.R, l.stride, l.pad)
        rms = float(np.sqrt(np.mean(ref ** 2)))
        Hh.check_samples(dw.ravel()[idx], ref, rms, False, f"{l.name} wgrad N={N}")
    return ts


def test_config4_full_size_sampled_batch64():
    # every one of the 53 layers in the launch configuration the bench times (several tiles per CTA, per-launch CTA limits),
    # plus an fp32-output pass of every layer held to the plain per-element bound
    _sampled_step_check(None, 64, list(range(53)), f32_pass=True)


@pytest.mark.parametrize("keep,N", [(0.3, 256), (0.4, 256), (0.6, 128), (0.8, 64), (1.0, 64)])
def test_config5_sweep_points_sampled(keep, N):
    _sampled_step_check(keep, N, [0, 2, 12, 26, 45], n_samples=2048)


def test_end_to_end_step_delivers_each_host_batch_one_step_later():
    """The end-to-end step copies the NEXT batch from pinned host memory while the current one trains: the stem must see
    batch k during call k + 1 (the first call brings its own), bit for bit, and the step's results must follow it."""
    ctx = Hh.ctx()
    net = W.vgg(11)
    seed = W.BASE_SEED + 9
    counts = W.uniform_keep(net, 0.6)
    kept = W.choose_kept(net, counts, seed)
    ts = harness.TrainStep(ctx, net, counts, kept, 16, seed, algo=2, host_inputs=True, device_rng=True)
    ts.step()
    torch.cuda.synchronize()
    ts.build_graph(two_streams=True)
    g = torch.Generator().manual_seed(seed)
    batches = [torch.randn(ts.h_image.shape, generator=g).to(ts.h_image.dtype) for _ in range(3)]
    l0 = ts.net.layers[0]
    ts.h_image.copy_(batches[0])
    ts.step_e2e()                                   # trains on batch 0 (its own copy), stages batch 0 again
    torch.cuda.synchronize()
    assert torch.equal(ts.x[0].cpu(), batches[0])
    ts.h_image.copy_(batches[1])                    # too late for the copy already made: call 2 still sees batch 0
    ts.step_e2e()
    torch.cuda.synchronize()
    assert torch.equal(ts.x[0].cpu(), batches[0])
    ts.h_image.copy_(batches[2])
    ts.step_e2e()                                   # sees batch 1, staged during call 2
    torch.cuda.synchronize()
    ctx.poll()
    assert torch.equal(ts.x[0].cpu(), batches[1])
    w0 = oracle.gather_weight(ts.md.wb[0][..., :net.layers[0].C].float().cpu().numpy(), kept[l0.out_space], kept[l0.in_space])
    x0 = batches[1][..., :l0.C].float().numpy()
    Hh.check_conv(ts.y[0], l0.K, oracle.conv_fwd(x0, w0, l0.stride, l0.pad), what="e2e stem fwd")
    assert float(ts.h_reg[0]) == float(ts.mp.reg.cpu()[0]) and float(ts.h_reg[0]) > 0
