"""Parity of the CUDA convolutions (through the C ABI) with the fp64 oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_09290_b200 import binding as B
from paper_1901_09290_b200 import workloads as W
from tests import helpers as Hh

pytestmark = pytest.mark.gpu

ALGOS = [0, 1]

# (N, H, W, C, K, R, stride)  -- odd and tiny channel counts, ragged pixel tails, stride 2, 7x7
SMALL = [
    (2, 5, 7, 1, 1, 1, 1), (2, 5, 7, 3, 7, 3, 1), (1, 1, 1, 8, 11, 1, 1), (3, 16, 16, 11, 27, 3, 1),
    (2, 16, 16, 16, 16, 1, 1), (2, 9, 9, 27, 8, 3, 2), (2, 8, 8, 7, 93, 1, 2), (1, 23, 23, 3, 16, 7, 2),
    (2, 14, 14, 93, 77, 3, 1), (1, 12, 10, 130, 70, 1, 1), (1, 7, 7, 260, 300, 3, 1),
    # few-channel stride-2 stems (space-to-depth path): 7x7, 5x5, 3x3; C = 1, 3, 4; non-square image
    (2, 32, 32, 3, 16, 7, 2), (1, 16, 20, 3, 55, 7, 2), (2, 12, 12, 1, 9, 5, 2), (2, 16, 16, 4, 24, 3, 2),
]


def _case(N, H, Wd, C, K, R, stride, seed):
    pad = R // 2
    x = W.gen_act(N, H, Wd, C, seed)
    w = W.bf16_round(W.gen_weight(K, R, R, C, seed + 1))
    P, Q = (H + 2 * pad - R) // stride + 1, (Wd + 2 * pad - R) // stride + 1
    dy = W.gen_dy(N, P, Q, K, seed + 2)
    return x, w, dy, pad


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("shape", SMALL)
def test_small_and_odd_shapes(shape, algo):
    N, H, Wd, C, K, R, stride = shape
    x, w, dy, pad = _case(*shape, seed=W.BASE_SEED + 11)
    y32, dx32, dw, _ = Hh.run_conv_all(N, H, Wd, C, K, R, stride, pad, x, w, dy, algo=algo, out_f32=1)
    y16, dx16, dw2, _ = Hh.run_conv_all(N, H, Wd, C, K, R, stride, pad, x, w, dy, algo=algo, out_f32=0)
    yr = oracle.conv_fwd(x.numpy(), w.numpy(), stride, pad)
    dxr = oracle.conv_dgrad(dy.numpy(), w.numpy(), H, Wd, stride, pad)
    Hh.check_conv(y32, K, yr, what="fwd f32")
    Hh.check_conv(dx32, C, dxr, what="dgrad f32")
    Hh.check_conv(dw, C, oracle.conv_wgrad(x.numpy(), dy.numpy(), R, R, stride, pad), what="wgrad")
    Hh.check_conv(y16, K, yr, what="fwd bf16")
    Hh.check_conv(dx16, C, dxr, what="dgrad bf16")
    # the bf16 output is the fp32 result rounded to nearest even, nothing else
    assert torch.equal(y16[..., :K], y32[..., :K].to(torch.bfloat16))
    assert torch.equal(dx16[..., :C], dx32[..., :C].to(torch.bfloat16))
    assert torch.equal(dw, dw2)


@pytest.mark.parametrize("algo", ALGOS)
def test_config1_single_layer_with_zero_groups(algo):
    """Batch 8, 16->32 channels, 16x16, 3x3: zero input channels / zero upstream-gradient channels give
    exactly-zero weight-gradient columns / rows (Eq. 4)."""
    N, H, C, K, R = 8, 16, 16, 32, 3
    seed = W.BASE_SEED + 1
    g = np.random.default_rng(seed)
    kz, cz = np.sort(g.permutation(K)[:5]), np.sort(g.permutation(C)[:3])
    x, w, dy, pad = _case(N, H, H, C, K, R, 1, seed)
    x[..., cz] = 0
    dy[..., kz] = 0
    w[kz] = 0
    w[:, :, :, cz] = 0
    y, dx, dw, _ = Hh.run_conv_all(N, H, H, C, K, R, 1, pad, x, w, dy, algo=algo)
    Hh.check_conv(y, K, oracle.conv_fwd(x.numpy(), w.numpy(), 1, pad), what="fwd")
    Hh.check_conv(dx, C, oracle.conv_dgrad(dy.numpy(), w.numpy(), H, H, 1, pad), what="dgrad")
    Hh.check_conv(dw, C, oracle.conv_wgrad(x.numpy(), dy.numpy(), R, R, 1, pad), what="wgrad")
    dwc = dw.cpu()
    assert torch.all(dwc[kz] == 0) and torch.all(dwc[:, :, :, cz] == 0)
    assert torch.all(y.float().cpu()[..., kz] == 0) and torch.all(dx.float().cpu()[..., cz] == 0)


@pytest.mark.parametrize("algo", ALGOS)
def test_config3_pruned_bottleneck(algo):
    """ResNet-50 stage-3 bottleneck at batch 64, 28x28, pruned to 371 -> 93 -> 77 -> 371: full-tensor parity."""
    net = W.with_sizes(W.bottleneck_stage3(), [371, 93, 77])
    for li, l in enumerate(net.layers):
        seed = W.layer_seed(3, li)
        x, w, dy, pad = _case(64, l.H, l.H, l.C, l.K, l.R, l.stride, seed)
        y, dx, dw, _ = Hh.run_conv_all(64, l.H, l.H, l.C, l.K, l.R, l.stride, pad, x, w, dy, algo=algo)
        Hh.check_conv(y, l.K, oracle.conv_fwd(x.numpy(), w.numpy(), l.stride, pad), what=l.name + " fwd")
        Hh.check_conv(dx, l.C, oracle.conv_dgrad(dy.numpy(), w.numpy(), l.H, l.H, l.stride, pad), what=l.name + " dgrad")
        Hh.check_conv(dw, l.C, oracle.conv_wgrad(x.numpy(), dy.numpy(), l.R, l.R, l.stride, pad), what=l.name + " wgrad")


# (N, H, W, C, K, R, stride): stride-2 weight gradients with few input channels (the generic kernel and the stem path):
# odd and even tap groups, K above and below 64, 5x5 and 7x7 stems
STRIDED_SMALL_C = [
    (2, 16, 16, 20, 36, 3, 2), (2, 18, 18, 64, 128, 3, 2), (3, 16, 16, 7, 70, 5, 2), (2, 32, 32, 3, 16, 7, 2), (2, 12, 12, 1, 9, 5, 2),
    (4, 20, 20, 33, 100, 2, 2),
]


@pytest.mark.parametrize("shape", STRIDED_SMALL_C)
def test_strided_weight_gradient_with_few_input_channels(shape):
    N, H, Wd, C, K, R, stride = shape
    x, w, dy, pad = _case(N, H, Wd, C, K, R, stride, seed=W.BASE_SEED + 53)
    dw = Hh.run_conv_all(N, H, Wd, C, K, R, stride, pad, x, w, dy, algo=2)[2]
    Hh.check_conv(dw, C, oracle.conv_wgrad(x.numpy(), dy.numpy(), R, R, stride, pad), what="wgrad")
    assert torch.equal(dw, Hh.run_conv_all(N, H, Wd, C, K, R, stride, pad, x, w, dy, algo=2)[2])


# (N, H, W, C, K, R, pad): stride-1 filters with several taps and at most 64 input channels -- the weight gradient that
# stages row blocks and pairs taps: two dy boxes (K > 64), several tap groups with an odd last one (K = 200), 25 taps,
# a wide image, an even filter, padding 0 and padding larger than (R - 1) / 2
ROW_BLOCK = [
    (3, 12, 12, 20, 100, 3, 1), (2, 10, 14, 64, 200, 3, 1), (2, 9, 9, 6, 10, 5, 2), (1, 8, 120, 9, 12, 3, 1),
    (2, 11, 11, 13, 21, 3, 0), (2, 7, 7, 5, 9, 3, 2), (2, 6, 6, 33, 40, 2, 0), (64, 20, 20, 38, 38, 3, 1),
    # 1x1 filters on large maps take the same kernel (single tap, K > 128 in one tile)
    (3, 30, 30, 59, 143, 1, 0), (2, 28, 28, 7, 19, 1, 0), (2, 40, 33, 64, 250, 1, 0),
    # more than 64 input channels (the generic kernel): ragged channel tiles, 25 taps, a 28x28 map
    (2, 14, 14, 93, 77, 3, 1), (2, 15, 16, 130, 40, 3, 1), (3, 14, 20, 213, 242, 3, 1), (2, 16, 16, 128, 100, 5, 2), (8, 28, 28, 113, 111, 3, 1),
]


@pytest.mark.parametrize("shape", ROW_BLOCK)
def test_row_block_weight_gradient(shape):
    N, H, Wd, C, K, R, pad = shape
    seed = W.BASE_SEED + 41
    x = W.gen_act(N, H, Wd, C, seed)
    w = W.bf16_round(W.gen_weight(K, R, R, C, seed + 1))
    P, Q = H + 2 * pad - R + 1, Wd + 2 * pad - R + 1
    dy = W.gen_dy(N, P, Q, K, seed + 2)
    y, dx, dw, _ = Hh.run_conv_all(N, H, Wd, C, K, R, 1, pad, x, w, dy, algo=2)
    Hh.check_conv(dw, C, oracle.conv_wgrad(x.numpy(), dy.numpy(), R, R, 1, pad), what="wgrad")
    Hh.check_conv(y, K, oracle.conv_fwd(x.numpy(), w.numpy(), 1, pad), what="fwd")
    Hh.check_conv(dx, C, oracle.conv_dgrad(dy.numpy(), w.numpy(), H, Wd, 1, pad), what="dgrad")
    again = Hh.run_conv_all(N, H, Wd, C, K, R, 1, pad, x, w, dy, algo=2)[2]
    assert torch.equal(dw, again)


@pytest.mark.parametrize("shape", [(2, 16, 16, 20, 36, 3, 1), (2, 14, 14, 37, 70, 3, 1), (2, 8, 8, 7, 33, 1, 1), (2, 16, 16, 41, 20, 3, 2)])
def test_pad_lanes_up_to_a_multiple_of_16_are_zero(shape):
    """With channel pitches that are multiples of 16 (as the training harness uses) the bf16 outputs are stored in whole
    32-byte sectors: the pad lanes receive zeros, never stale accumulator columns."""
    N, H, Wd, C, K, R, stride = shape
    pad = R // 2
    x, w, dy, _ = _case(N, H, Wd, C, K, R, stride, seed=W.BASE_SEED + 23)
    ldx, ldy, ldw = W.pad16(C), W.pad16(K), W.pad8(C)
    d = B.make_conv_desc(N, H, Wd, C, K, R, R, stride, pad, ldx, ldy, ldw, 0, 2)
    P, Q = (H + 2 * pad - R) // stride + 1, (Wd + 2 * pad - R) // stride + 1
    xd, wd, dyd = Hh.to_dev_padded(x, ldx), Hh.to_dev_padded(w, ldw), Hh.to_dev_padded(dy, ldy)
    y = Hh.out_buffer((N, P, Q), K, ldy, 0)
    dx = Hh.out_buffer((N, H, Wd), C, ldx, 0)
    B.pt_conv_fwd(Hh.ctx(), d, xd, wd, y, Hh.conv_ws(d, B.PT_CONV_FWD))
    B.pt_conv_dgrad(Hh.ctx(), d, dyd, wd, dx, Hh.conv_ws(d, B.PT_CONV_DGRAD))
    torch.cuda.synchronize()
    Hh.ctx().poll()
    Hh.check_conv(y, K, oracle.conv_fwd(x.numpy(), w.numpy(), stride, pad), what="fwd")
    Hh.check_conv(dx, C, oracle.conv_dgrad(dy.numpy(), w.numpy(), H, Wd, stride, pad), what="dgrad")
    assert torch.all(y[..., K:] == 0) and torch.all(dx[..., C:] == 0)


def test_wgrad_is_run_to_run_identical():
    N, H, C, K, R = 4, 14, 27, 19, 3
    x, w, dy, pad = _case(N, H, H, C, K, R, 1, W.BASE_SEED + 5)
    a = Hh.run_conv_all(N, H, H, C, K, R, 1, pad, x, w, dy)[2].cpu()
    b = Hh.run_conv_all(N, H, H, C, K, R, 1, pad, x, w, dy)[2].cpu()
    assert torch.equal(a, b)


@pytest.mark.parametrize("limit", [1, 7, 37])
def test_wgrad_with_a_cta_limit(limit):
    """The weight gradient may be held to fewer CTAs (to run beside other kernels): same result class, bounded by the limit."""
    c = Hh.ctx()
    try:
        B.pt_set_wgrad_cta_limit(c, limit)
        for (N, H, C, K, R) in [(4, 14, 93, 77, 3), (8, 28, 130, 70, 1), (3, 16, 11, 27, 3)]:
            x, w, dy, pad = _case(N, H, H, C, K, R, 1, W.BASE_SEED + 31 + limit)
            dw = Hh.run_conv_all(N, H, H, C, K, R, 1, pad, x, w, dy, algo=2)[2]
            Hh.check_conv(dw, C, oracle.conv_wgrad(x.numpy(), dy.numpy(), R, R, 1, pad), what=f"wgrad limit {limit}")
        with pytest.raises(B.PtError):
            B.pt_set_wgrad_cta_limit(c, -1)
    finally:
        B.pt_set_wgrad_cta_limit(c, 0)


def test_wgrad_cta_query_follows_the_limit():
    """pt_conv_wgrad_ctas reports tiles x splits at the current limit: never above a limit it can meet, whole multiples of
    the tile count, and an unsplit launch (more tiles than the limit) is reported as not waiting."""
    c = Hh.ctx()
    try:
        for (N, H, C, K, R, stride) in [(64, 14, 213, 242, 3, 1), (64, 56, 46, 59, 3, 1), (64, 28, 418, 113, 1, 1), (64, 7, 434, 495, 3, 1),
                                        (64, 224, 3, 55, 7, 2)]:
            d = B.make_conv_desc(N, H, H, C, K, R, R, stride, R // 2, 8 if C <= 4 else W.pad16(C), W.pad16(K))
            B.pt_set_wgrad_cta_limit(c, 1)
            tiles, waits = B.pt_conv_wgrad_ctas(c, d)
            assert tiles >= 1 and not waits
            prev = 0
            for lim in (8, 24, 49, 74, 148):
                B.pt_set_wgrad_cta_limit(c, lim)
                n, waits = B.pt_conv_wgrad_ctas(c, d)
                assert n % tiles == 0 and n >= prev
                assert (n <= lim and waits == (n > tiles)) or (n == tiles and not waits)
                prev = n
        assert B.pt_conv_wgrad_ctas(c, B.make_conv_desc(2, 8, 8, 16, 16, 3, 3, 1, 1, algo=1)) == (0, False)
    finally:
        B.pt_set_wgrad_cta_limit(c, 0)


def test_invalid_arguments_are_rejected_before_launch():
    c = Hh.ctx()
    buf = torch.zeros(4096, dtype=torch.bfloat16, device="cuda")
    good = B.make_conv_desc(1, 4, 4, 8, 8, 3, 3, 1, 1)
    for field, val in (("ldx", 9), ("ldy", 4), ("ldw", 12), ("C", 0), ("stride", 0), ("algo", 7)):
        d = B.make_conv_desc(1, 4, 4, 8, 8, 3, 3, 1, 1)
        setattr(d, field, val)
        with pytest.raises(B.PtError) as e:
            B.pt_conv_fwd(c, d, buf, buf, buf)
        assert e.value.status == 1
    with pytest.raises(B.PtError):
        B.pt_conv_fwd(c, good, None, buf, buf)
    d = B.make_conv_desc(2, 8, 8, 8, 8, 3, 3, 1, 1, algo=1)
    with pytest.raises(B.PtError) as e:       # the SIMT wgrad needs a workspace
        B.pt_conv_wgrad(c, d, buf, buf, torch.zeros(8 * 9 * 8, device="cuda"), None)
    assert e.value.status == 3
    c.poll()


@pytest.mark.parametrize("stride", [1, 2])
def test_tcgen05_path_takes_all_three_passes_when_forced(stride):
    """algo = 2 forces the tcgen05 kernels: the calls must not fall back silently."""
    N, H, C, K, R = 3, 12, 40, 24, 3
    x, w, dy, pad = _case(N, H, H, C, K, R, stride, W.BASE_SEED + 9)
    y, dx, dw, d = Hh.run_conv_all(N, H, H, C, K, R, stride, pad, x, w, dy, algo=2, out_f32=1)
    Hh.check_conv(y, K, oracle.conv_fwd(x.numpy(), w.numpy(), stride, pad), what="fwd tcgen05")
    Hh.check_conv(dx, C, oracle.conv_dgrad(dy.numpy(), w.numpy(), H, H, stride, pad), what="dgrad tcgen05")
    Hh.check_conv(dw, C, oracle.conv_wgrad(x.numpy(), dy.numpy(), R, R, stride, pad), what="wgrad tcgen05")
    # a 9x9 filter has more taps than the tcgen05 path's tap table: forcing it must fail loudly, auto must fall back
    d9 = B.make_conv_desc(1, 12, 12, 8, 8, 9, 9, 1, 4, algo=2)
    buf = torch.zeros(1 << 16, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.PtError) as e:
        B.pt_conv_fwd(Hh.ctx(), d9, buf, buf, buf)
    assert e.value.status == 2
