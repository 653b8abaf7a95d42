"""Times single conv passes of one layer of the pruned ResNet-50 workload (CUDA events, rotating buffers).

    python -m paper_1901_09290_b200.layerbench --layer s1b1.c3 --passes fwd,dgrad,wgrad --iters 20
    python -m paper_1901_09290_b200.layerbench --shape 64,56,36,143,1,1 --passes fwd      # N,H,C,K,R,stride
    python -m paper_1901_09290_b200.layerbench --bn 64,56,143                              # batch norm + ReLU + residual: N,H,C
    python -m paper_1901_09290_b200.layerbench --model --iters 5      # lasso step, detection, compaction of the whole model alone

It is also the small case ncu captures are taken on.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as B
from . import workloads as W


def model_main(args):
    """The HBM-bound model passes alone, in the order a step runs them, each timed with CUDA events after an L2 flush."""
    from .harness import TrainStep
    net = W.resnet50()
    seed = W.BASE_SEED + 4
    counts = W.staged_keep_to_flops(net, seed, 0.60)
    ctx = B.Context(0)
    ts = TrainStep(ctx, net, counts, W.choose_kept(net, counts, seed), 1, seed)
    md = ts.md
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    ops = [("detect", lambda: B.pt_find_zero_groups(ctx, md.arr, 1e-4, False, md.ws)),
           ("plan_incl_host_sync", lambda: B.pt_reconfigure_plan(ctx, md.graph(), ts.new2old)),
           ("gather", lambda: ts.gather()),
           ("lasso", lambda: ts.lasso()),
           ("lasso_norms", lambda: ts.lasso_norms()),
           ("lasso_carried", lambda: ts.lasso_carried())]
    tot = {k: 0.0 for k, _ in ops}
    for it in range(args.iters + 1):                    # the first round is the warm-up
        for k, fn in ops:
            flush.fill_(it)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record()
            torch.cuda.synchronize()
            if it:
                tot[k] += a.elapsed_time(b) * 1e3 / args.iters
    ctx.poll()
    print(json.dumps({"model": "resnet50 keep drawn to 0.60", "dense_params": md.n_params(), "kept_params": ts.mp.n_params(),
                      "us": {k: round(v, 1) for k, v in tot.items()},
                      "note": "eager launches with events around each call (host launch cost included)"}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layer", default=None)
    ap.add_argument("--shape", default=None, help="N,H,C,K,R,stride")
    ap.add_argument("--passes", default="fwd,dgrad,wgrad")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--sets", type=int, default=4, help="rotating buffer sets (footprint larger than L2)")
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--algo", type=int, default=0)
    ap.add_argument("--wgrad-ctas", type=int, default=0, help="CTA limit of the weight-gradient kernels (0 = one per SM)")
    ap.add_argument("--no-graph", action="store_true", help="time eager launches (includes host launch cost)")
    ap.add_argument("--bn", default=None, help="N,H,C: time pt_bn_relu_fwd / pt_bn_relu_bwd instead of a convolution")
    ap.add_argument("--gate", default=None, help="N,H,C,S: time pt_channel_gather / pt_channel_scatter_add of S of a node's C channels")
    ap.add_argument("--stats", action="store_true",
                    help="the forward pass through pt_conv_fwd_stats (batch-norm statistics taken in the epilogue)")
    ap.add_argument("--model", action="store_true",
                    help="time detection, plan, gather, the lasso step and its carried form over the bench's ResNet-50 model "
                         "alone (batch 1 activations: ~0.7 GB on the device, the model itself larger than L2)")
    args = ap.parse_args()
    if args.model:
        return model_main(args)
    if args.gate:
        return gate_main(args)
    if args.bn:
        return bn_main(args)
    if args.shape:
        N, H, C, K, R, stride = [int(t) for t in args.shape.split(",")]
        name = args.shape
    else:
        net = W.resnet50()
        counts = W.staged_keep_to_flops(net, W.BASE_SEED + 4, 0.60)
        l = [l for l in W.with_sizes(net, counts).layers if l.name == args.layer][0]
        N, H, C, K, R, stride = args.batch, l.H, l.C, l.K, l.R, l.stride
        name = l.name
    pad = R // 2
    P = (H + 2 * pad - R) // stride + 1
    ctx = B.Context(0)
    if args.wgrad_ctas:
        ctx.set_wgrad_cta_limit(args.wgrad_ctas)
    d = B.make_conv_desc(N, H, H, C, K, R, R, stride, pad, 8 if C <= 4 else W.pad16(C), W.pad16(K), algo=args.algo)
    g = torch.Generator(device="cuda").manual_seed(1)
    sets = []
    for _ in range(args.sets):
        x = torch.randn((N, H, H, d.ldx), generator=g, device="cuda").clamp_(min=0).to(torch.bfloat16)
        dy = (torch.randn((N, P, P, d.ldy), generator=g, device="cuda") * 2 ** -6).to(torch.bfloat16)
        w = (torch.randn((K, R, R, d.ldw), generator=g, device="cuda") * (2.0 / (C * R * R)) ** 0.5).to(torch.bfloat16)
        sets.append((x, dy, w, torch.empty_like(dy), torch.empty_like(x), torch.empty((K, R, R, C), device="cuda")))
    ws = torch.empty(max(16, max(B.pt_conv_workspace_bytes(ctx, d, i) for i in range(3))), dtype=torch.uint8, device="cuda")
    stats = None
    if args.stats:
        d.algo = 2                               # the statistics epilogue exists in the tcgen05 kernels only
        stats = torch.empty(B.pt_conv_fwd_stats_bytes(ctx, d) // 4, dtype=torch.float32, device="cuda")
    flops = 2 * N * P * P * K * C * R * R
    act = N * H * H * C * 2 + N * P * P * K * 2
    out = {"layer": name, "N": N, "H": H, "C": C, "K": K, "R": R, "stride": stride}
    for ps in args.passes.split(","):
        def run(i):
            x, dy, w, y, dx, dw = sets[i % len(sets)]
            if ps == "fwd" and stats is not None:
                B.pt_conv_fwd_stats(ctx, d, x, w, y, stats, ws)
            elif ps == "fwd":
                B.pt_conv_fwd(ctx, d, x, w, y, ws)
            elif ps == "dgrad":
                B.pt_conv_dgrad(ctx, d, dy, w, dx, ws)
            else:
                B.pt_conv_wgrad(ctx, d, x, dy, dw, ws)
        for i in range(3):
            run(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if args.no_graph:
            e0.record()
            for i in range(args.iters):
                run(i)
            e1.record()
        else:
            # the launches are captured once and replayed, so the device time is not hidden behind host launch cost
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for i in range(args.iters):
                    run(i)
            g.replay()
            torch.cuda.synchronize()
            e0.record()
            g.replay()
            e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / args.iters
        by = act + K * C * R * R * (4 if ps == "wgrad" else 2)
        out[ps] = {"us": round(us, 2), "tflops": round(flops / us / 1e6, 1), "gbs": round(by / us / 1e3, 1)}
    ctx.poll()
    print(json.dumps(out))


def bn_main(args):
    """Batch norm + residual + ReLU on one activation tensor: device time and algorithmic GB/s (every tensor counted once:
    forward x, residual, y = 6 B per element; backward x, y, dy, dx, dresidual = 10 B per element)."""
    N, H, C = [int(t) for t in args.bn.split(",")]
    ld = W.pad16(C)
    ctx = B.Context(0)
    d = B.make_bn_desc(N, H, H, C, ld)
    g = torch.Generator(device="cuda").manual_seed(1)
    mk = lambda: torch.randn((N, H, H, ld), generator=g, device="cuda").to(torch.bfloat16)
    sets = [tuple(mk() for _ in range(7)) for _ in range(args.sets)]
    gamma, beta = torch.ones(C, device="cuda"), torch.zeros(C, device="cuda")
    rm, rv = torch.zeros(C, device="cuda"), torch.ones(C, device="cuda")
    sm, si, dg, db = (torch.empty(C, device="cuda") for _ in range(4))
    ws = torch.empty(max(16, B.pt_bn_workspace_bytes(ctx, d)), dtype=torch.uint8, device="cuda")
    elems = N * H * H * C
    out = {"bn": args.bn, "ld": ld}
    for ps in ("fwd", "bwd"):
        def run(i):
            x, r, y, dy, dx, dr, _ = sets[i % len(sets)]
            if ps == "fwd":
                B.pt_bn_relu_fwd(ctx, d, x, r, gamma, beta, rm, rv, sm, si, y, ws)
            else:
                B.pt_bn_relu_bwd(ctx, d, x, y, dy, gamma, sm, si, dx, dr, dg, db, ws)
        for i in range(3):
            run(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr):
            for i in range(args.iters):
                run(i)
        gr.replay()
        torch.cuda.synchronize()
        e0.record()
        gr.replay()
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / args.iters
        by = elems * (6 if ps == "fwd" else 10)
        out[ps] = {"us": round(us, 2), "gbs": round(by / us / 1e3, 1)}
    ctx.poll()
    print(json.dumps(out))


def gate_main(args):
    """Channel gating on one node tensor: device time and GB/s of the bytes that must move (gather: the selected channels
    in and out, 4 B per selected element; scatter-add: node in, branch in, node out)."""
    N, H, C, S = [int(t) for t in args.gate.split(",")]
    ld_n, ld_s = W.pad8(C), W.pad8(S)
    npix = N * H * H
    ctx = B.Context(0)
    g = torch.Generator(device="cuda").manual_seed(1)
    idx = torch.sort(torch.randperm(C, generator=g, device="cuda")[:S])[0].to(torch.int32)
    mk = lambda ld: torch.randn((npix, ld), generator=g, device="cuda").to(torch.bfloat16)
    sets = [(mk(ld_n), mk(ld_s), mk(ld_n)) for _ in range(args.sets)]
    out = {"gate": args.gate}
    for ps in ("gather", "scatter_add"):
        def run(i):
            node, br, res = sets[i % len(sets)]
            if ps == "gather":
                B.pt_channel_gather(ctx, node, ld_n, C, idx, S, br, ld_s, npix)
            else:
                B.pt_channel_scatter_add(ctx, br, ld_s, idx, S, node, res, ld_n, C, npix, 1)
        for i in range(3):
            run(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr):
            for i in range(args.iters):
                run(i)
        gr.replay()
        torch.cuda.synchronize()
        e0.record()
        gr.replay()
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / args.iters
        by = npix * (4 * S if ps == "gather" else 4 * C + 2 * S)
        out[ps] = {"us": round(us, 2), "gbs": round(by / us / 1e3, 1)}
    ctx.poll()
    print(json.dumps(out))


if __name__ == "__main__":
    main()
