"""The bounded device-side waits, made to run out without any fault.

Every wait of the convolution kernels (on an mbarrier, or of a split weight gradient on its sibling CTAs) has a time
limit; when it runs out the CTA records the time-out, drains its copies, frees its tensor memory and exits, and
pt_poll_device_status returns PT_ERR_TIMEOUT. The tests shorten the limit to a few milliseconds, make ONE tiny launch
leave out one arrival through the library's test hook (no trap, no bad address, no unbounded loop), and check the
status, the time it took, and that the next ordinary launches on the same context -- which need the SMs' whole tensor
memory and, for the weight gradient, the same arrival counters -- still match the oracle.
"""
import time

import numpy as np
import pytest
import torch

import oracle
from paper_1901_09290_b200 import binding as B
from paper_1901_09290_b200 import workloads as W
from tests import helpers as Hh

pytestmark = pytest.mark.gpu

LIMIT_MS = 20


def _inputs(N, H, C, K, R, seed):
    x = W.gen_act(N, H, H, C, seed)
    w = W.bf16_round(W.gen_weight(K, R, R, C, seed + 1))
    dy = W.gen_dy(N, H, H, K, seed + 2)
    return x, w, dy


def _expect_timeout(ctx, launch):
    B.pt_test_set_wait_limit(ctx, LIMIT_MS)
    try:
        t0 = time.perf_counter()
        launch()
        with pytest.raises(B.PtError) as e:
            ctx.poll()
        dt = time.perf_counter() - t0
        assert e.value.status == 5, e.value                     # PT_ERR_TIMEOUT
        assert dt < 2.0, f"the wait took {dt:.2f} s to give up at a {LIMIT_MS} ms limit"
    finally:
        B.pt_test_skip_next_arrive(ctx, 0)
        B.pt_test_set_wait_limit(ctx, 0)
    ctx.poll()                                                  # the status word was cleared by the failing poll


def test_split_weight_gradient_wait_runs_out_and_the_context_recovers():
    ctx = Hh.ctx()
    N, H, C, K, R = 8, 16, 16, 32, 3                            # config-1 size
    x, w, dy = _inputs(N, H, C, K, R, W.BASE_SEED + 61)
    d = B.make_conv_desc(N, H, H, C, K, R, R, 1, 1, algo=2)
    ctas, waits = B.pt_conv_wgrad_ctas(ctx, d)
    assert waits and ctas > 1, "the shape must split its reduction over CTAs for this test"
    xd, dyd = Hh.to_dev_padded(x, d.ldx), Hh.to_dev_padded(dy, d.ldy)
    dw = torch.zeros((K, R, R, C), dtype=torch.float32, device="cuda")
    ws = Hh.conv_ws(d, B.PT_CONV_WGRAD)

    def launch():
        B.pt_test_skip_next_arrive(ctx, 1)
        B.pt_conv_wgrad(ctx, d, xd, dyd, dw, ws)

    _expect_timeout(ctx, launch)
    # the same split launch again (same counters after the reset), several times, and a launch that takes all 512 TMEM
    # columns on every SM: a CTA that had kept its tensor memory would make these wait for ever (they are bounded too)
    ref = oracle.conv_wgrad(x.numpy(), dy.numpy(), R, R, 1, 1)
    for _ in range(3):
        dw.fill_(7680.0)
        B.pt_conv_wgrad(ctx, d, xd, dyd, dw, ws)
        torch.cuda.synchronize()
        ctx.poll()
        Hh.check_conv(dw, C, ref, what="wgrad after a time-out")
    xb, wb, dyb = _inputs(4, 28, 256, 256, 1, W.BASE_SEED + 62)
    y, dx, dwb, _ = Hh.run_conv_all(4, 28, 28, 256, 256, 1, 1, 0, xb, wb, dyb, algo=2)
    Hh.check_conv(y, 256, oracle.conv_fwd(xb.numpy(), wb.numpy(), 1, 0), what="fwd after a time-out")
    Hh.check_conv(dwb, 256, oracle.conv_wgrad(xb.numpy(), dyb.numpy(), 1, 1, 1, 0), what="wide wgrad after a time-out")


def test_pipeline_barrier_wait_runs_out_and_the_context_recovers():
    ctx = Hh.ctx()
    N, H, C, K, R = 8, 16, 16, 32, 1                            # a 1x1 layer: the pixel-linear kernel
    x, w, dy = _inputs(N, H, C, K, R, W.BASE_SEED + 63)
    d = B.make_conv_desc(N, H, H, C, K, R, R, 1, 0, algo=2)
    xd, wd = Hh.to_dev_padded(x, d.ldx), Hh.to_dev_padded(w, d.ldw)
    y = torch.zeros((N, H, H, d.ldy), dtype=torch.bfloat16, device="cuda")

    def launch():
        B.pt_test_skip_next_arrive(ctx, 2)
        B.pt_conv_fwd(ctx, d, xd, wd, y, None)

    _expect_timeout(ctx, launch)
    ref = oracle.conv_fwd(x.numpy(), w.numpy(), 1, 0)
    for _ in range(3):
        yo = Hh.out_buffer((N, H, H), K, d.ldy, False)
        B.pt_conv_fwd(ctx, d, xd, wd, yo, None)
        torch.cuda.synchronize()
        ctx.poll()
        Hh.check_conv(yo, K, ref, what="fwd after a time-out")
