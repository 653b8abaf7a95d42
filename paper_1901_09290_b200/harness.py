"""Device-side staging around the C ABI: argument marshalling for whole models and whole steps.

Nothing here computes anything of the method: it allocates torch CUDA tensors as device memory,
fills the ABI structs and issues the ``pt_*`` calls in the order of Algorithm 1.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from . import binding as B
from . import workloads as W


class DeviceModel:
    """Device copies of a workloads.Model (fp32 w, v, g, BN vectors), the bf16 shadow and the per-layer
    scratch the ABI wants (group sums of squares, zero masks), plus the pt_layer array."""

    def __init__(self, ctx: B.Context, model: W.Model, shadow_fill: float = float("nan")):
        self.ctx = ctx
        self.net = model.net
        self.w = [t.clone().cuda() for t in model.w]
        self.v = [t.clone().cuda() for t in model.v]
        # the weight gradients of all layers are views of one flat buffer: a data-parallel run reduces them in one collective
        al = lambda n: (n + 63) // 64 * 64                  # every view starts on a 256-byte boundary
        self.g_flat = torch.zeros(sum(al(t.numel()) for t in model.g), dtype=torch.float32, device="cuda")
        self.g, off = [], 0
        for t in model.g:
            v = self.g_flat[off:off + t.numel()].view(t.shape)
            v.copy_(t)
            self.g.append(v)
            off += al(t.numel())
        self.bn = [[b.clone().cuda() for b in bb] for bb in model.bn]
        self.wb, self.sq_out, self.sq_in, self.z_out, self.z_in, self.layers = [], [], [], [], [], []
        for li, l in enumerate(self.net.layers):
            ldw = W.pad8(l.C)
            wb = torch.full((l.K, l.R, l.R, ldw), shadow_fill, dtype=torch.bfloat16, device="cuda")
            wb[..., :l.C] = self.w[li].to(torch.bfloat16)       # data conversion of the initial weights
            self.wb.append(wb)
            self.sq_out.append(torch.full((l.K,), -1.0, device="cuda"))
            self.sq_in.append(torch.full((l.C,), -1.0, device="cuda"))
            self.z_out.append(torch.full((l.K,), 9, dtype=torch.uint8, device="cuda"))
            self.z_in.append(torch.full((l.C,), 9, dtype=torch.uint8, device="cuda"))
            reg_in = self.net.space_stage[l.in_space] != 0     # only the image's channels are exempt (stage 0)
            self.layers.append(B.make_layer(self.w[li], self.g[li], self.v[li], wb, l.K, l.C, l.R * l.R, ldw,
                                            reg_in, True, self.sq_out[li], self.sq_in[li], self.z_out[li], self.z_in[li]))
        self.arr = B.layer_array(self.layers)
        n = B.pt_group_lasso_workspace_bytes(ctx, self.arr)
        self.ws = torch.empty(max(n, 256), dtype=torch.uint8, device="cuda")
        self.reg = torch.zeros(1, dtype=torch.float64, device="cuda")
        self._graph = None
        self._subgraphs = {}

    def reg_in(self, li: int) -> bool:
        return bool(self.layers[li].reg_in)

    def graph(self) -> B.GraphHandle:
        if self._graph is None:
            links = [(l.in_space, l.out_space) for l in self.net.layers]
            self._graph = B.GraphHandle(self.net.space_sizes, self.net.space_fixed, self.layers, links, self.bn)
        return self._graph

    def subgraph(self, first: int, count: int) -> B.GraphHandle:
        """The same channel spaces with layers [first, first + count) only (for a compaction done in parts)."""
        key = (first, count)
        if key not in self._subgraphs:
            ls = self.net.layers[first:first + count]
            links = [(l.in_space, l.out_space) for l in ls]
            self._subgraphs[key] = B.GraphHandle(self.net.space_sizes, self.net.space_fixed, self.layers[first:first + count], links,
                                                 self.bn[first:first + count])
        return self._subgraphs[key]

    def n_params(self) -> int:
        return sum(l.K * l.C * l.R * l.R for l in self.net.layers)


def empty_model(net: W.Net, fill: float = 0.0) -> W.Model:
    mk = lambda l: torch.full((l.K, l.R, l.R, l.C), fill)
    return W.Model(net, [mk(l) for l in net.layers], [mk(l) for l in net.layers],
                   [torch.zeros((l.K, l.R, l.R, l.C)) for l in net.layers],
                   [[torch.full((l.K,), fill) for _ in range(4)] for l in net.layers])


def conv_macs(net: W.Net, counts) -> int:
    """Forward multiply-accumulates per image with the given (C, K) per layer."""
    return sum(l.P * l.P * k * c * l.R * l.R for l, (c, k) in zip(net.layers, counts))


def allreduce_mean(flat: torch.Tensor, world: int):
    """The one exchange of a data-parallel step (Sec. 2.2, data parallelism: the partial weight gradients of all GPUs are
    reduced, then used to update the weights): the mean of the ranks' gradient buffers, in place, in one collective over
    the flat buffer whose size shrinks as the model is pruned. NCCL averages inside the collective; gloo (CPU tests) sums
    and the division follows."""
    import torch.distributed as dist
    if world <= 1:
        return
    if flat.is_cuda:
        dist.all_reduce(flat, op=dist.ReduceOp.AVG)
    else:
        dist.all_reduce(flat, op=dist.ReduceOp.SUM)
        flat.div_(world)


class TrainStep:
    """The hot path on one GPU for one network: reconfiguration of a dense-shaped model with embedded zero
    groups into the pruned model, then the pruned model's conv training step (every layer's forward, then data and
    weight gradients in reverse order, each on its own activation buffers) and the group-lasso SGD step.

    The layers are not chained through BN/ReLU/pooling (those are not on the path): every layer has its own
    seeded input x_l and upstream gradient dy_l, as in a training step's memory footprint.
    """

    def __init__(self, ctx: B.Context, dense_net: W.Net, counts: Sequence[int], kept, N: int, seed: int,
                 algo: int = 0, host_inputs: bool = False, decoys: int = 2, device_rng: bool = True,
                 wgrad_ctas: int = 49, wgrad_streams: int = 3, world: int = 1):
        self.ctx, self.N, self.algo = ctx, N, algo
        self.world = world          # > 1: data parallel, the weight gradients are averaged over the ranks before the update
        # weight gradients of different layers are independent: each launch is held to `wgrad_ctas` CTAs and the launches
        # go round-robin to `wgrad_streams` streams, each with a workspace of its own. The CTAs of a split weight gradient
        # wait for one another, one per SM, so streams x limit stays within the SM count (3 x 49 <= 148): every launch
        # that can be in flight then fits on the device together, whatever order the hardware picks its CTAs in.
        # `wgrad_ctas` is the nominal share; _wgrad_limits() refines it per launch under the same constraint.
        self.wgrad_ctas, self.wgrad_streams = wgrad_ctas, max(1, wgrad_streams)
        self.gather_split = 4       # layers whose weights are gathered before the forward pass starts (the rest beside it)
        ctx.set_wgrad_cta_limit(wgrad_ctas)
        self.dense_net = dense_net
        self.net = W.with_sizes(dense_net, counts)
        self.counts = list(counts)
        model_d = W.gen_model(dense_net, seed, kept=kept, decoys=decoys)
        self.md = DeviceModel(ctx, model_d)
        self.mp = DeviceModel(ctx, empty_model(self.net))
        self.new2old = torch.full((sum(dense_net.space_sizes),), -1, dtype=torch.int32, device="cuda")
        self.x, self.dy, self.y, self.dx, self.desc = [], [], [], [], []
        gen = torch.Generator(device="cuda").manual_seed(seed + 99) if device_rng else None
        ws_bytes = 16
        for li, l in enumerate(self.net.layers):
            ldx, ldy = (8 if l.C <= 4 else W.pad16(l.C)), W.pad16(l.K)
            P = l.P
            d = B.make_conv_desc(N, l.H, l.H, l.C, l.K, l.R, l.R, l.stride, l.pad, ldx, ldy, W.pad8(l.C), 0, algo)
            self.desc.append(d)
            if device_rng:
                if li == 0:
                    x = torch.randn((N, l.H, l.H, ldx), generator=gen, device="cuda", dtype=torch.float32)
                else:
                    x = torch.randn((N, l.H, l.H, ldx), generator=gen, device="cuda", dtype=torch.float32).clamp_(min=0)
                dy = torch.randn((N, P, P, ldy), generator=gen, device="cuda", dtype=torch.float32) * (2.0 ** -6)
                self.x.append(x.to(torch.bfloat16))
                self.dy.append(dy.to(torch.bfloat16))
                del x, dy
            else:
                sx, sd = W.layer_seed(4, li, 1), W.layer_seed(4, li, 2)
                xh = W.gen_image(N, l.H, l.H, l.C, sx) if li == 0 else W.gen_act(N, l.H, l.H, l.C, sx)
                dh = W.gen_dy(N, P, P, l.K, sd)
                xd = torch.zeros((N, l.H, l.H, ldx), dtype=torch.bfloat16, device="cuda")
                xd[..., :l.C] = xh.to(torch.bfloat16)
                dd = torch.zeros((N, P, P, ldy), dtype=torch.bfloat16, device="cuda")
                dd[..., :l.K] = dh.to(torch.bfloat16)
                self.x.append(xd)
                self.dy.append(dd)
            self.y.append(torch.empty((N, P, P, ldy), dtype=torch.bfloat16, device="cuda"))
            self.dx.append(torch.empty((N, l.H, l.H, ldx), dtype=torch.bfloat16, device="cuda") if li > 0 else None)
            for which in range(3):
                ws_bytes = max(ws_bytes, B.pt_conv_workspace_bytes(ctx, d, which))
        # Per-launch CTA limits: whole multiples of each layer's tiles (no idle share of a budget), larger for the layers
        # with more work, every three consecutive launches within the SM count (see _wgrad_limits)
        self.wgrad_limit = self._wgrad_limits() if (wgrad_streams == 3 and wgrad_ctas * 3 <= 148 and len(self.net.layers) >= 4) else {}
        for li, lim in self.wgrad_limit.items():
            ctx.set_wgrad_cta_limit(lim)
            ws_bytes = max(ws_bytes, B.pt_conv_workspace_bytes(ctx, self.desc[li], 2))
        ctx.set_wgrad_cta_limit(wgrad_ctas)
        self.ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
        self.ws_w = [torch.empty(ws_bytes, dtype=torch.uint8, device="cuda") for _ in range(self.wgrad_streams)]
        # e2e: the image batch arrives from pinned host memory every step
        l0 = self.net.layers[0]
        self.h_image = None
        if host_inputs:
            self.h_image = self.x[0].cpu().pin_memory()
        self.h_reg = torch.zeros(1, dtype=torch.float64).pin_memory()

    def _wgrad_work(self, li: int) -> float:
        """Rough device time (us on one SM) of a layer's weight gradient: the larger of its MMA count at 55+ cycles each
        and its tensor bytes at the ~35 GB/s one SM pulls; only ratios between layers are used."""
        l = self.net.layers[li]
        px = self.N * l.P * l.P
        taps = l.R * l.R
        if l.stride == 2 and l.C <= 4:                       # space-to-depth stem: (R+1)/2 vertical taps of 64 lanes, two per MMA
            mmas = px / 16 * (((l.R + 1) // 2 + 1) // 2)
            cyc = 55
        elif l.stride == 1 and l.C <= 64:                    # row-block kernel: two taps per MMA, N = K
            mmas = px / 16 * ((taps + 1) // 2)
            cyc = max(55, W.pad16(l.K) // 2 + 8)
        else:
            bn = min(256, W.pad16(l.C))
            mmas = px / 16 * taps * -(-l.K // 128) * -(-l.C // bn)
            cyc = max(55, bn // 2 + 8)
        t_mma = mmas * cyc / 1.9e3
        t_mem = (self.N * l.H * l.H * W.pad16(l.C) + px * W.pad16(l.K)) * 2 / 35e3
        return max(t_mma, t_mem)

    def _wgrad_limits(self) -> Dict[int, int]:
        """CTA limit of every weight-gradient launch. The launches go round-robin to three streams in reverse layer order,
        so any three consecutive ones can be in flight together and their CTAs (which wait for one another) must fit on
        the device at once. Within that constraint the limits minimise the sum over launches of work / CTAs (dynamic
        programme over the CTA counts each layer can actually use, as the library reports them), which gives the layers
        with more work the larger shares and wastes no part of a share on a tile count that does not divide it. The
        last three launches have nothing after them and end up sharing all SMs."""
        sm = torch.cuda.get_device_properties(0).multi_processor_count
        order = list(range(len(self.net.layers) - 1, -1, -1))
        cands = []
        for li in order:
            seen = {}
            for lim in range(16, min(sm, 128) + 1):
                self.ctx.set_wgrad_cta_limit(lim)
                ctas, waits = B.pt_conv_wgrad_ctas(self.ctx, self.desc[li])
                if ctas <= 0:
                    break
                # an unsplit launch waits for nobody and may run in waves: it only counts as a fair share in the sums
                room = ctas if waits else min(ctas, sm // 3)
                if (ctas, room) not in seen and room <= sm:
                    seen[(ctas, room)] = lim
            cands.append([(room, lim, ctas) for (ctas, room), lim in sorted(seen.items())] or [(self.wgrad_ctas, self.wgrad_ctas, self.wgrad_ctas)])
        self.ctx.set_wgrad_cta_limit(self.wgrad_ctas)
        work = [self._wgrad_work(li) for li in order]
        INF = float("inf")
        # best[(a, b)] = (cost, choices) over the first i launches with the last two using cands[i-2][a], cands[i-1][b]
        best = {(-1, -1): (0.0, [])}
        for i, cs in enumerate(cands):
            nxt = {}
            for (a, b), (cost, path) in best.items():
                ca = cands[i - 2][a][0] if a >= 0 else 0
                cb = cands[i - 1][b][0] if b >= 0 else 0
                for k, (room, _, ctas) in enumerate(cs):
                    if ca + cb + room > sm:
                        continue
                    c2 = cost + work[i] / min(ctas, sm)
                    key = (b, k)
                    if c2 < nxt.get(key, (INF,))[0]:
                        nxt[key] = (c2, path + [k])
            if not nxt:                                    # cannot happen with the smallest candidates; keep the default
                return {}
            best = nxt
        path = min(best.values(), key=lambda v: v[0])[1]
        lim = {li: cands[i][k][1] for i, (li, k) in enumerate(zip(order, path))}
        # the last three launches end the backward pass: what counts for them is that they finish together, i.e. shares in
        # proportion to their work rather than to its square root
        tail, wt = order[-3:], work[-3:]
        share = [max(16, int(sm * w / sum(wt))) for w in wt]
        while sum(share) > sm:
            share[share.index(max(share))] -= 1
        prev = [cands[i][path[i]][0] for i in (len(order) - 5, len(order) - 4)]
        if prev[0] + prev[1] + share[0] <= sm and prev[1] + share[0] + share[1] <= sm:
            lim.update({li: v for li, v in zip(tail, share)})
        return lim

    # ---- sizes used for reporting
    def conv_flops(self) -> Dict[str, int]:
        f = {"fwd": 0, "dgrad": 0, "wgrad": 0}
        for li, l in enumerate(self.net.layers):
            fl = 2 * self.N * l.P * l.P * l.K * l.C * l.R * l.R
            f["fwd"] += fl
            f["wgrad"] += fl
            if li > 0:
                f["dgrad"] += fl
        return f

    def layer_bytes(self, li: int, which: int) -> int:
        """Algorithmic bytes of one conv pass: each tensor touched once (bf16 activations and weights, fp32 dw)."""
        l = self.net.layers[li]
        a = self.N * l.H * l.H * l.C * 2 + self.N * l.P * l.P * l.K * 2
        return a + l.K * l.C * l.R * l.R * (4 if which == 2 else 2)

    def lasso_bytes(self, model: DeviceModel) -> int:
        return 26 * model.n_params()

    def reconf_bytes(self) -> int:
        """Detection reads the old weights once (4 B/param); the gather reads w, v (8 B) and writes w, v, shadow
        (10 B) per kept parameter."""
        return 4 * self.md.n_params() + 18 * self.mp.n_params()

    # ---- the path
    def reconfigure_plan(self, stream=None):
        """Detection and keep-set scan: everything up to (and including) the host synchronisation that returns the new sizes."""
        c = self.ctx
        B.pt_find_zero_groups(c, self.md.arr, 1e-4, False, self.md.ws, stream)
        sizes = B.pt_reconfigure_plan(c, self.md.graph(), self.new2old, stream)
        if sizes != self.counts:
            raise RuntimeError(f"reconfiguration plan returned {sizes}, expected {self.counts}")

    def gather(self, first: int = 0, count: Optional[int] = None, stream=None):
        """The compaction gather of layers [first, first + count) into the pruned model."""
        n = len(self.net.layers)
        count = n - first if count is None else count
        if first == 0 and count == n:
            B.pt_reconfigure(self.ctx, self.md.graph(), self.new2old, self.mp.graph(), stream)
        else:
            B.pt_reconfigure(self.ctx, self.md.subgraph(first, count), self.new2old, self.mp.subgraph(first, count), stream)

    def reconfigure(self, stream=None):
        self.reconfigure_plan(stream)
        self.gather(stream=stream)

    def conv_fwd(self, li, stream=None):
        B.pt_conv_fwd(self.ctx, self.desc[li], self.x[li], self.mp.wb[li], self.y[li], self.ws, stream)

    def conv_dgrad(self, li, stream=None):
        B.pt_conv_dgrad(self.ctx, self.desc[li], self.dy[li], self.mp.wb[li], self.dx[li], self.ws, stream)

    def conv_wgrad(self, li, stream=None, ws_index: int = 0):
        lim = self.wgrad_limit.get(li)
        if lim is not None:
            self.ctx.set_wgrad_cta_limit(lim)
        B.pt_conv_wgrad(self.ctx, self.desc[li], self.x[li], self.dy[li], self.mp.g[li], self.ws_w[ws_index], stream)
        if lim is not None:
            self.ctx.set_wgrad_cta_limit(self.wgrad_ctas)

    def lasso(self, stream=None, lam=1e-4, lr=0.1, mu=0.9):
        B.pt_group_lasso_sgd_step(self.ctx, self.mp.arr, lam, lr, mu, 0.0, self.mp.reg, self.mp.ws, stream)

    def lasso_carried(self, stream=None, lam=1e-4, lr=0.1, mu=0.9, with_maxima=False):
        """The step in its carried form: needs lasso_norms() (or a previous carried step) on the current weights."""
        B.pt_group_lasso_sgd_step_carried(self.ctx, self.mp.arr, lam, lr, mu, 0.0, self.mp.reg, self.mp.ws, stream, with_maxima)

    def lasso_norms(self, stream=None):
        B.pt_group_lasso_norms(self.ctx, self.mp.arr, self.mp.reg, self.mp.ws, stream)

    def lasso_apply(self, stream=None, lam=1e-4, lr=0.1, mu=0.9):
        B.pt_group_lasso_sgd_apply(self.ctx, self.mp.arr, lam, lr, mu, 0.0, self.mp.ws, stream)

    def train(self, stream=None):
        n = len(self.net.layers)
        for li in range(n):
            self.conv_fwd(li, stream)
        for li in range(n - 1, -1, -1):
            if li > 0:
                self.conv_dgrad(li, stream)
            self.conv_wgrad(li, stream)
        if self.world > 1:
            allreduce_mean(self.mp.g_flat, self.world)
        self.lasso(stream)

    def _branches(self):
        """(first layer of the block, index of the projection shortcut) for every block that has one: the shortcut reads
        the block's input and is only needed at the block's output, so it is independent of the block's other layers."""
        out = []
        names = [l.name for l in self.net.layers]
        for d, nm in enumerate(names):
            if nm.endswith(".ds"):
                pre = nm[:-3]
                first = min(i for i, x in enumerate(names) if x.startswith(pre + "."))
                out.append((first, d))
        return out

    def train_two_streams(self, fwd: bool = True, dgrad: bool = True, wgrad: bool = True, lasso: bool = True, gather: bool = False):
        """The same launches on several streams, following the network's own data dependencies: the weight gradient of a
        layer needs only x_l and dy_l, so it starts when dy_l exists and runs beside the data gradients below it (round-robin
        over the weight-gradient streams, each with its own workspace); a block's projection shortcut is independent of
        the block's other convolutions in both directions. The flags select passes (used to time one pass as scheduled)."""
        main = torch.cuda.current_stream()
        aux, ws = self._aux, self._wstreams
        n = len(self.net.layers)
        br = self._branches()
        fork_at = {f: d for f, d in br}          # before layer f: start shortcut d on the aux stream
        ds_set = {d for _, d in br}
        forked = set()                           # streams that joined this launch sequence and must be joined back
        gather_join = None
        if gather:
            # The gather needs no host: the first layers' weights are gathered on the main stream, the rest on a side stream
            # beside the first forward layers (large maps, latency bound, SMs to spare), joined back before their first use.
            k = min(self.gather_split, n)
            self.gather(0, k, main)
            if k < n:
                gstream = ws[0]
                gstream.wait_stream(main)
                forked.add(gstream)
                self.gather(k, n - k, gstream)
                gather_join = (k, gstream)
        if lasso and fwd:
            # the group norms need the weights only (GroupLassoReg(W_i) of Algorithm 1): they run beside the forward pass
            nstream = ws[-1]
            nstream.wait_stream(main)
            if gather_join is not None:
                nstream.wait_stream(gather_join[1])      # the norms read every layer's gathered weights
            forked.add(nstream)
            self.lasso_norms(nstream)
        for li in range(n if fwd else 0):
            if gather_join is not None and li == gather_join[0]:
                main.wait_stream(gather_join[1])
                aux.wait_stream(gather_join[1])
                gather_join = None
            if li in fork_at:
                aux.wait_stream(main)
                forked.add(aux)
                self.conv_fwd(fork_at[li], aux)
            if li in ds_set:
                main.wait_stream(aux)            # the block's output needs both branches
                continue
            self.conv_fwd(li, main)
        first_of = {d: f for f, d in br}
        join_after = None
        wi = 0
        for li in range(n - 1, -1, -1):
            # dy_l exists once the data gradients above layer l are done: the weight gradient of layer l starts there, next
            # to the layer's own data gradient
            wk = wi % len(ws)
            side = ws[wk]
            wi += 1
            if wgrad:
                side.wait_stream(main)
                forked.add(side)
                self.conv_wgrad(li, side, wk)
            if not dgrad:
                continue
            if li in ds_set:
                aux.wait_stream(main)            # both branches start from the gradient of the block's output
                forked.add(aux)
                if li > 0:
                    self.conv_dgrad(li, aux)
                join_after = first_of[li]
                continue
            if li > 0:
                self.conv_dgrad(li, main)
            if join_after == li:
                main.wait_stream(aux)            # the gradient of the block's input sums both branches
                join_after = None
        if gather_join is not None:
            main.wait_stream(gather_join[1])
        for w in forked:
            main.wait_stream(w)
        if lasso:
            if fwd:
                self.lasso_apply(main)
            else:
                self.lasso(main)

    def capture_pass(self, kind: str):
        """A CUDA graph of one pass kind ("fwd", "dgrad", "wgrad") with the stream assignment it has inside the step."""
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self.train_two_streams(fwd=kind == "fwd", dgrad=kind == "dgrad", wgrad=kind == "wgrad", lasso=False)
        return g

    def build_graph(self, two_streams: bool = True, gather_in_graph: bool = True):
        """Captures the training part of the step (every launch after the reconfiguration's host sync) into a CUDA graph.
        Call after at least one eager step, so that every table and kernel attribute is already set up."""
        self._side = torch.cuda.Stream()
        self._wstreams = [self._side] + [torch.cuda.Stream() for _ in range(self.wgrad_streams - 1)]
        self._aux = torch.cuda.Stream()
        self._graph_two = two_streams
        l0 = self.ctx.launch_count()
        self.graph = torch.cuda.CUDAGraph()
        self._graph_has_update = self.world <= 1
        self._graph_has_gather = bool(two_streams and gather_in_graph)
        if self._graph_has_gather:
            # the part gathers once eagerly: their device tables are then cached and the capture records kernels only
            n = len(self.net.layers)
            k = min(self.gather_split, n)
            self.gather(0, k)
            if k < n:
                self.gather(k, n - k)
            torch.cuda.synchronize()
            l0 = self.ctx.launch_count()
        with torch.cuda.graph(self.graph):
            if self.world > 1:
                # data parallel: the graph ends with the weight gradients; the collective and the update follow it eagerly
                self.train_two_streams(lasso=False, gather=self._graph_has_gather)
            elif two_streams:
                self.train_two_streams(gather=self._graph_has_gather)
            else:
                self.train()
        self.graph_launches = self.ctx.launch_count() - l0
        return self.graph

    def step(self, stream=None, before_train=None):
        if getattr(self, "graph", None) is not None and getattr(self, "_graph_has_gather", False):
            self.reconfigure_plan(stream)                 # the gather is part of the graph (in two parts, beside the first layers)
        else:
            self.reconfigure(stream)
        if before_train is not None:
            torch.cuda.current_stream().wait_event(before_train)     # e.g. the image batch has reached the stem's input
        if getattr(self, "graph", None) is not None:
            self.graph.replay()
            if not self._graph_has_update:
                allreduce_mean(self.mp.g_flat, self.world)       # the one exchange of a data-parallel step
                self.lasso(stream)
        else:
            self.train(stream)

    def step_e2e(self, stream=None):
        """The same step with the image batch copied from pinned host memory and the regulariser value read back.

        The stem's input is double buffered: while a step reads one buffer, the next batch is copied from pinned host memory
        into the other on a copy stream (one copy per step; the first call brings its own batch), and the next call trains
        on that buffer -- with a CUDA graph of its own, captured on first use, because a graph holds the address of the
        buffer its kernels read. Nothing is moved on the device. The copy of the next batch is enqueued AFTER this step's
        launches: enqueued before them it delayed the step by ~55 us whatever its size. The host batch must stay untouched
        until that copy has run (the next call, or a synchronize)."""
        main = torch.cuda.current_stream()
        if getattr(self, "_copy_stream", None) is None:
            self._copy_stream = torch.cuda.Stream()
            self._xbuf = [self.x[0], torch.empty_like(self.x[0])]
            self._xgraph = [getattr(self, "graph", None), None]
            self._ev_in = [torch.cuda.Event(), torch.cuda.Event()]
            self._cur = 0
            self._copy_stream.wait_stream(main)
            with torch.cuda.stream(self._copy_stream):
                self._xbuf[0].copy_(self.h_image, non_blocking=True)
                self._ev_in[0].record(self._copy_stream)
        cs = self._copy_stream
        cur, nxt = self._cur, 1 - self._cur
        self.x[0] = self._xbuf[cur]
        if getattr(self, "graph", None) is not None:
            if self._xgraph[cur] is None:
                self.build_graph(self._graph_two, self._graph_has_gather)        # the launches that read this buffer
                self._xgraph[cur] = self.graph
            self.graph = self._xgraph[cur]
        cs.wait_stream(main)                             # the previous step, the last reader of the other buffer, is done
        self.step(stream, before_train=self._ev_in[cur])
        with torch.cuda.stream(cs):
            self._xbuf[nxt].copy_(self.h_image, non_blocking=True)     # the next step's batch
            self._ev_in[nxt].record(cs)
        self._cur = nxt
        self.h_reg.copy_(self.mp.reg, non_blocking=True)

    def e2e_bytes(self):
        return self.h_image.numel() * self.h_image.element_size(), 8 + 4 * len(self.counts)


class ChainedStep:
    """A ResNet conv stack chained from the image to the last feature map through the C ABI: every convolution is followed
    by batch normalisation (training statistics) and ReLU, blocks end with the residual add, the stem is followed by the
    3x3 / stride-2 max pooling where the shape table halves there, and the backward pass runs the whole chain in reverse
    down to every weight gradient; the group-lasso SGD step closes the iteration. With `fused_stats` the convolutions take
    the normalisation statistics in their epilogues (pt_conv_fwd_stats + pt_bn_relu_fwd_stats: one pass over each
    convolution output instead of two). The classifier is not part of the library: the gradient with respect to the last
    feature map is a seeded input. Marshalling only: every tensor operation is an ABI call.

    Block structure is read from the layer names: "stem", then "<block>.c1", "<block>.c2", ... and an optional "<block>.ds"
    (projection shortcut) per block, in order."""

    def __init__(self, ctx: B.Context, net: W.Net, N: int, seed: int, fused_stats: bool = True, algo: int = 0,
                 max_blocks: Optional[int] = None, model: Optional[W.Model] = None, x0: Optional[torch.Tensor] = None,
                 g_last: Optional[torch.Tensor] = None, wgrad_streams: int = 0):
        self.ctx, self.net, self.N, self.fused = ctx, net, N, fused_stats
        # wgrad_streams > 0: a layer's weight gradient needs only its input and dy, so it goes to a side stream (round robin,
        # a workspace each) and runs beside the rest of the backward chain; the launches are held to SMs / streams CTAs so
        # that the split ones, whose CTAs wait for one another, always fit on the device together
        self.wgrad_streams = wgrad_streams
        self.wgrad_limit = 0 if wgrad_streams <= 0 else max(1, 148 // wgrad_streams)
        ctx.set_wgrad_cta_limit(self.wgrad_limit)       # sizes the workspaces (0: one stream, every weight gradient may take all SMs)
        names = [l.name for l in net.layers]
        self.blocks = []                                   # (main conv indices, shortcut index or None)
        for i, nm in enumerate(names):
            if nm == "stem" or nm.endswith(".ds"):
                continue
            pre = nm.rsplit(".", 1)[0]
            if not self.blocks or self.blocks[-1][2] != pre:
                ds = names.index(pre + ".ds") if pre + ".ds" in names else None
                self.blocks.append(([], ds, pre))
            self.blocks[-1][0].append(i)
        if max_blocks is not None:
            self.blocks = self.blocks[:max_blocks]
        self.used = [0] + [i for b in self.blocks for i in b[0]] + [b[1] for b in self.blocks if b[1] is not None]
        self.model = model if model is not None else W.gen_model(net, seed)
        self.dm = DeviceModel(ctx, self.model)
        L = net.layers
        self.ld = {i: W.pad16(L[i].K) for i in self.used}          # pitch of a layer's outputs
        l0 = L[0]
        self.ld_img = 8 if l0.C <= 4 else W.pad16(l0.C)
        dev = "cuda"
        bf = lambda n, h, ld: torch.zeros((n, h, h, ld), dtype=torch.bfloat16, device=dev)
        if x0 is None:
            x0 = W.gen_image(N, l0.H, l0.H, l0.C, seed + 11)
        self.x0 = torch.zeros((N, l0.H, l0.H, self.ld_img), dtype=torch.bfloat16, device=dev)
        self.x0[..., :l0.C] = x0.to(torch.bfloat16).cuda()
        first_h = L[self.blocks[0][0][0]].H if self.blocks else l0.P
        self.pool = l0.P != first_h
        if self.pool:
            self.pool_desc = B.make_pool_desc(N, l0.P, l0.P, l0.K, self.ld[0], 3, 2, 1)
            assert (l0.P + 2 - 3) // 2 + 1 == first_h
        self.desc, self.bn_desc, self.y, self.a, self.dy, self.gamma, self.beta, self.sm, self.si, self.dg, self.db = ({} for _ in range(11))
        ws_conv, ws_bn, st_bytes = 16, 16, 16
        gen = torch.Generator().manual_seed(seed + 12)
        for i in self.used:
            l = L[i]
            ldx = self.ld_img if i == 0 else W.pad16(l.C)
            self.desc[i] = B.make_conv_desc(N, l.H, l.H, l.C, l.K, l.R, l.R, l.stride, l.pad, ldx, self.ld[i], W.pad8(l.C), 0, algo)
            self.bn_desc[i] = None
            self.y[i] = bf(N, l.P, self.ld[i])             # convolution output
            self.a[i] = bf(N, l.P, self.ld[i])             # after normalisation (+ residual) (+ ReLU)
            self.dy[i] = bf(N, l.P, self.ld[i])            # gradient with respect to the convolution output
            self.gamma[i] = (torch.rand(l.K, generator=gen) + 0.5).cuda()
            self.beta[i] = (torch.rand(l.K, generator=gen) - 0.5).cuda()
            self.sm[i], self.si[i] = torch.empty(l.K, device=dev), torch.empty(l.K, device=dev)
            self.dg[i], self.db[i] = torch.empty(l.K, device=dev), torch.empty(l.K, device=dev)
            for which in range(3):
                ws_conv = max(ws_conv, B.pt_conv_workspace_bytes(ctx, self.desc[i], which))
            st_bytes = max(st_bytes, B.pt_conv_fwd_stats_bytes(ctx, self.desc[i]))
        ds_set = {b[1] for b in self.blocks if b[1] is not None}
        last_of = {b[0][-1] for b in self.blocks}
        for i in self.used:
            l = L[i]
            relu = i not in ds_set                         # the projection shortcut is normalised but not rectified
            self.bn_desc[i] = B.make_bn_desc(N, l.P, l.P, l.K, self.ld[i], 1e-5, 0.1, relu)
            ws_bn = max(ws_bn, B.pt_bn_workspace_bytes(ctx, self.bn_desc[i]))
        self.last_of = last_of
        self.ws = torch.empty(ws_conv, dtype=torch.uint8, device=dev)
        self.ws_side = [torch.empty(ws_conv, dtype=torch.uint8, device=dev) for _ in range(max(0, wgrad_streams))]
        self._side = [torch.cuda.Stream() for _ in range(max(0, wgrad_streams))]
        self._wi = 0
        # in the same mode a block's projection shortcut (convolution + batch norm) runs on a stream of its own beside the block's
        # main branch, in both directions, with workspaces of its own
        self._aux = torch.cuda.Stream() if wgrad_streams > 0 else None
        self.ws_aux = torch.empty(ws_conv, dtype=torch.uint8, device=dev) if self._aux else None
        self.ws_bn_aux = torch.empty(ws_bn, dtype=torch.uint8, device=dev) if self._aux else None
        self.stats_aux = torch.empty(st_bytes // 4, dtype=torch.float32, device=dev) if self._aux else None
        self.ws_bn = torch.empty(ws_bn, dtype=torch.uint8, device=dev)
        self.stats = torch.empty(st_bytes // 4, dtype=torch.float32, device=dev)
        if self.pool:
            self.pooled = bf(N, first_h, self.ld[0])
            self.pool_index = torch.empty((N, first_h, first_h, self.ld[0]), dtype=torch.uint8, device="cuda")   # selections of the forward pass
            self.d_pooled = bf(N, first_h, self.ld[0])
        # gradients with respect to activations: one buffer per distinct activation a convolution reads
        # gradient with respect to a convolution's INPUT (its data gradient), and with respect to the stem's activation
        self.da = {i: bf(N, L[i].H, W.pad16(L[i].C)) for i in self.used if i != 0}
        self.d_a0 = bf(N, l0.P, self.ld[0])
        self.da_tmp = {}
        self.dres = {}
        for main, ds, _ in self.blocks:
            lo = L[main[-1]]
            self.dres[main[-1]] = bf(N, lo.P, self.ld[main[-1]])             # gradient handed to the residual branch
        out_i = self.blocks[-1][0][-1] if self.blocks else 0
        lo = L[out_i]
        if g_last is None:
            g_last = W.gen_dy(N, lo.P, lo.P, lo.K, seed + 13) * 64.0
        self.g_last = torch.zeros((N, lo.P, lo.P, self.ld[out_i]), dtype=torch.bfloat16, device=dev)
        self.g_last[..., :lo.K] = g_last.to(torch.bfloat16).cuda()
        self.out_index = out_i
        self._idx = {}

    # ---- helpers
    def _arange(self, n):
        if n not in self._idx:
            self._idx[n] = torch.arange(n, dtype=torch.int32, device="cuda")
        return self._idx[n]

    def _add(self, a, b, out, C, ld, npix, stream=None):
        """out = a + b (bf16, one rounding) through the scatter-add with the identity selection."""
        B.pt_channel_scatter_add(self.ctx, b, ld, self._arange(C), C, a, out, ld, C, npix, False, stream)

    def _conv_bn(self, i, x, residual=None, stream=None, aux=False):
        c = self.ctx
        ws, ws_bn, stats = (self.ws_aux, self.ws_bn_aux, self.stats_aux) if aux else (self.ws, self.ws_bn, self.stats)
        if self.fused:
            n_parts = B.pt_conv_fwd_stats(c, self.desc[i], x, self.dm.wb[i], self.y[i], stats, ws, stream)
            B.pt_bn_relu_fwd_stats(c, self.bn_desc[i], self.y[i], residual, self.gamma[i], self.beta[i], None, None, self.sm[i], self.si[i],
                                   self.a[i], stats, n_parts, stream)
        else:
            B.pt_conv_fwd(c, self.desc[i], x, self.dm.wb[i], self.y[i], ws, stream)
            B.pt_bn_relu_fwd(c, self.bn_desc[i], self.y[i], residual, self.gamma[i], self.beta[i], None, None, self.sm[i], self.si[i],
                             self.a[i], ws_bn, stream)
        return self.a[i]

    # ---- the chain
    def forward(self, stream=None):
        cur = self._conv_bn(0, self.x0, None, stream)
        if self.pool:
            B.pt_maxpool_fwd(self.ctx, self.pool_desc, cur, self.pooled, stream, index=self.pool_index)
            cur = self.pooled
        self.block_in = []
        for main, ds, _ in self.blocks:
            self.block_in.append(cur)
            side = self._aux if ds is not None else None
            ms = stream if stream is not None else torch.cuda.current_stream()
            if side is not None:
                side.wait_stream(ms)
                res = self._conv_bn(ds, cur, None, side, aux=True)
            else:
                res = self._conv_bn(ds, cur, None, stream) if ds is not None else cur
            t = cur
            for i in main[:-1]:
                t = self._conv_bn(i, t, None, stream)
            if side is not None:
                ms.wait_stream(side)                      # the block's last batch norm adds the shortcut
            cur = self._conv_bn(main[-1], t, res, stream)
        return cur

    def _bn_bwd(self, i, d_out, dres, stream=None, aux=False):
        B.pt_bn_relu_bwd(self.ctx, self.bn_desc[i], self.y[i], self.a[i], d_out, self.gamma[i], self.sm[i], self.si[i], self.dy[i], dres,
                         self.dg[i], self.db[i], self.ws_bn_aux if aux else self.ws_bn, stream)

    def _wgrad(self, i, x_i, stream):
        """The weight gradient of layer i: on the caller's stream, or on the next side stream once that stream has dy_i."""
        if not self._side:
            B.pt_conv_wgrad(self.ctx, self.desc[i], x_i, self.dy[i], self.dm.g[i], self.ws, stream)
            return
        main = stream if stream is not None else torch.cuda.current_stream()
        k = self._wi % len(self._side)
        self._wi += 1
        side = self._side[k]
        side.wait_stream(main)
        B.pt_conv_wgrad(self.ctx, self.desc[i], x_i, self.dy[i], self.dm.g[i], self.ws_side[k], side)

    def backward(self, stream=None):
        c, L = self.ctx, self.net.layers
        self._wi = 0
        d_cur = self.g_last                                   # gradient w.r.t. the current block's output
        for bi in range(len(self.blocks) - 1, -1, -1):
            main, ds, _ = self.blocks[bi]
            x_in = self.block_in[bi]
            last = main[-1]
            self._bn_bwd(last, d_cur, self.dres[last], stream)
            ms = stream if stream is not None else torch.cuda.current_stream()
            side = self._aux if ds is not None else None
            if side is not None:
                # the shortcut's backward (batch norm, weight and data gradient) beside the main branch's
                side.wait_stream(ms)
                self._bn_bwd(ds, self.dres[last], None, side, aux=True)
                self._wgrad(ds, x_in, side)
                B.pt_conv_dgrad(c, self.desc[ds], self.dy[ds], self.dm.wb[ds], self.da[ds], self.ws_aux, side)
            d_t = None
            for k in range(len(main) - 1, -1, -1):
                i = main[k]
                x_i = x_in if k == 0 else self.a[main[k - 1]]
                if k < len(main) - 1:
                    self._bn_bwd(i, d_t, None, stream)
                self._wgrad(i, x_i, stream)
                d_t = self.da[i]
                B.pt_conv_dgrad(c, self.desc[i], self.dy[i], self.dm.wb[i], d_t, self.ws, stream)
            # d_t: gradient w.r.t. the block input through the main branch; the shortcut adds its own
            li = L[main[0]]
            npix, Cin, ld_in = self.N * li.H * li.H, li.C, W.pad16(li.C)
            if side is not None:
                ms.wait_stream(side)
                sc = self.da[ds]
            elif ds is not None:
                self._bn_bwd(ds, self.dres[last], None, stream)
                self._wgrad(ds, x_in, stream)
                B.pt_conv_dgrad(c, self.desc[ds], self.dy[ds], self.dm.wb[ds], self.da[ds], self.ws, stream)
                sc = self.da[ds]
            else:
                sc = self.dres[last]
            key = ("sum", bi)
            if key not in self.da_tmp:
                self.da_tmp[key] = torch.zeros_like(d_t)
            self._add(d_t, sc, self.da_tmp[key], Cin, ld_in, npix, stream)
            d_cur = self.da_tmp[key]
        if self.pool:
            B.pt_maxpool_bwd(c, self.pool_desc, self.a[0], d_cur, self.d_a0, stream, index=self.pool_index)
            d_cur = self.d_a0
        self._bn_bwd(0, d_cur, None, stream)
        self._wgrad(0, self.x0, stream)
        main = stream if stream is not None else torch.cuda.current_stream()
        for side in self._side:
            main.wait_stream(side)                        # the update needs every weight gradient

    def update(self, stream=None, lam=1e-4, lr=0.1, mu=0.9):
        B.pt_group_lasso_sgd_step(self.ctx, self.dm.arr, lam, lr, mu, 0.0, self.dm.reg, self.dm.ws, stream)

    def step(self, stream=None):
        self.ctx.set_wgrad_cta_limit(self.wgrad_limit)
        self.forward(stream)
        self.backward(stream)
        self.update(stream)

    def conv_flops(self) -> int:
        f = 0
        for i in self.used:
            l = self.net.layers[i]
            fl = 2 * self.N * l.P * l.P * l.K * l.C * l.R * l.R
            f += (2 if i == 0 else 3) * fl
        return f
