"""Seeded synthetic workloads: network shape tables and input generators.

This module holds NONE of the method's arithmetic (no convolution, no norms, no
update rule, no detection, no keep-set logic). It only describes layer shapes
and draws seeded random tensors, so both the CUDA path's tests/bench and the
CPU oracle's tests can be fed identical bits.

The tensors stand in for the paper's CIFAR-10/100 and ImageNet runs (Sec. 5,
evaluation methodology): same image sizes, batch sizes and ResNet layer shapes,
irregular post-pruning channel counts, but no dataset item and no trained
weight.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

BASE_SEED = 190109290


@dataclass
class LayerSpec:
    name: str
    C: int
    K: int
    R: int
    stride: int
    pad: int
    H: int            # input height = width
    in_space: int
    out_space: int

    @property
    def P(self) -> int:
        return (self.H + 2 * self.pad - self.R) // self.stride + 1


@dataclass
class Net:
    name: str
    layers: List[LayerSpec]
    space_names: List[str]
    space_sizes: List[int]
    space_fixed: List[bool]
    space_stage: List[int] = field(default_factory=list)

    def space_index(self, nm: str) -> int:
        return self.space_names.index(nm)


class _Builder:
    def __init__(self, name):
        self.net = Net(name, [], [], [], [], [])

    def space(self, nm, size, fixed=False, stage=1):
        n = self.net
        if nm not in n.space_names:
            n.space_names.append(nm)
            n.space_sizes.append(size)
            n.space_fixed.append(fixed)
            n.space_stage.append(stage)
        return n.space_names.index(nm)

    def conv(self, name, C, K, R, stride, H, isp, osp):
        self.net.layers.append(LayerSpec(name, C, K, R, stride, R // 2, H, isp, osp))


def resnet50(image: int = 224) -> Net:
    """torchvision-style ResNet-50 conv stack: 53 convs, 38 channel spaces, 23 454 912 conv parameters.
    Stride 2 sits on the 3x3 of the first block of stages 2-4; 1x1 stride-2 projection shortcuts."""
    b = _Builder("resnet50")
    img = b.space("img", 3, fixed=True, stage=0)
    n0 = b.space("n0", 64, stage=1)
    b.conv("stem", 3, 64, 7, 2, image, img, n0)
    H = image // 4                      # stem stride 2 then 3x3/2 max-pool (pooling itself is not on the path)
    inC, node = 64, n0
    for si, (mid, nb) in enumerate([(64, 3), (128, 4), (256, 6), (512, 3)]):
        out = mid * 4
        nn = b.space(f"n{si + 1}", out, fixed=(si == 3), stage=si + 1)
        for bi in range(nb):
            s = 2 if (bi == 0 and si > 0) else 1
            i1 = b.space(f"s{si + 1}b{bi}.i1", mid, stage=si + 1)
            i2 = b.space(f"s{si + 1}b{bi}.i2", mid, stage=si + 1)
            b.conv(f"s{si + 1}b{bi}.c1", inC, mid, 1, 1, H, node, i1)
            b.conv(f"s{si + 1}b{bi}.c2", mid, mid, 3, s, H, i1, i2)
            Ho = H // s
            b.conv(f"s{si + 1}b{bi}.c3", mid, out, 1, 1, Ho, i2, nn)
            if bi == 0:
                b.conv(f"s{si + 1}b{bi}.ds", inC, out, 1, s, H, node, nn)
            H, inC, node = Ho, out, nn
    return b.net


def resnet32(image: int = 32) -> Net:
    """CIFAR ResNet-32 conv stack with 1x1 stride-2 projection shortcuts: 33 convs, 19 spaces, 463 792 parameters."""
    b = _Builder("resnet32")
    img = b.space("img", 3, fixed=True, stage=0)
    node = b.space("n1", 16, stage=1)
    b.conv("stem", 3, 16, 3, 1, image, img, node)
    H, inC = image, 16
    for si, w in enumerate([16, 32, 64]):
        nn = node if si == 0 else b.space(f"n{si + 1}", w, fixed=(si == 2), stage=si + 1)
        for bi in range(5):
            s = 2 if (bi == 0 and si > 0) else 1
            i1 = b.space(f"s{si + 1}b{bi}.i1", w, stage=si + 1)
            b.conv(f"s{si + 1}b{bi}.c1", inC, w, 3, s, H, node, i1)
            Ho = H // s
            b.conv(f"s{si + 1}b{bi}.c2", w, w, 3, 1, Ho, i1, nn)
            if s == 2:
                b.conv(f"s{si + 1}b{bi}.ds", inC, w, 1, 2, H, node, nn)
            H, inC, node = Ho, w, nn
    return b.net


def bottleneck_stage3(H: int = 28) -> Net:
    """One ResNet-50 stage-3 identity bottleneck: 1x1 512->128, 3x3 128->128, 1x1 128->512 at 28x28."""
    b = _Builder("bottleneck")
    node = b.space("node", 512, stage=2)
    i1 = b.space("i1", 128, stage=2)
    i2 = b.space("i2", 128, stage=2)
    b.conv("c1", 512, 128, 1, 1, H, node, i1)
    b.conv("c2", 128, 128, 3, 1, H, i1, i2)
    b.conv("c3", 128, 512, 1, 1, H, i2, node)
    return b.net


def vgg(depth: int = 16, image: int = 32) -> Net:
    """Plain VGG-style stack (Tab. 1 trains VGG-11 and VGG-13 on CIFAR): 3x3 stride-1 convolutions in five groups of
    64..512 channels, a 2x2 pooling (not on the path) halving the map after each group, no short-cuts, so every channel
    space has one writer and one reader. Batch normalisation after every convolution, hence no conv bias."""
    cfg = {11: (1, 1, 2, 2, 2), 13: (2, 2, 2, 2, 2), 16: (2, 2, 3, 3, 3)}[depth]
    b = _Builder(f"vgg{depth}")
    prev = b.space("img", 3, fixed=True, stage=0)
    H, inC, n = image, 3, 0
    n_total = sum(cfg)
    for gi, (reps, width) in enumerate(zip(cfg, (64, 128, 256, 512, 512))):
        for _ in range(reps):
            n += 1
            sp = b.space(f"a{n}", width, fixed=(n == n_total), stage=gi + 1)
            b.conv(f"conv{n}", inC, width, 3, 1, H, prev, sp)
            prev, inC = sp, width
        H = max(1, H // 2)
    return b.net


def single_layer(C=16, K=32, R=3, H=16, stride=1) -> Net:
    """One conv as a 2-space graph: the layer is the only reader of its input space and the
    only writer of its output space."""
    b = _Builder("single")
    i = b.space("in", C, stage=1)
    o = b.space("out", K, stage=1)
    b.conv("conv", C, K, R, stride, H, i, o)
    return b.net


# --------------------------------------------------------------------------- kept-channel draws
def with_sizes(net: Net, sizes: Sequence[int]) -> Net:
    """The same graph with every layer's C/K replaced by the given per-space sizes."""
    layers = [LayerSpec(l.name, int(sizes[l.in_space]), int(sizes[l.out_space]), l.R, l.stride, l.pad, l.H,
                        l.in_space, l.out_space) for l in net.layers]
    return Net(net.name + "-pruned", layers, list(net.space_names), [int(s) for s in sizes],
               list(net.space_fixed), list(net.space_stage))


def fwd_macs(net: Net) -> int:
    """Multiply-accumulate count of one forward pass per image (shape bookkeeping for the keep-ratio draw)."""
    return sum(l.P * l.P * l.K * l.C * l.R * l.R for l in net.layers)


def uniform_keep(net: Net, r: float) -> List[int]:
    return [s if f else max(1, int(round(r * s))) for s, f in zip(net.space_sizes, net.space_fixed)]


def random_keep(net: Net, seed: int, lo=0.4, hi=0.9) -> List[int]:
    """Per-space keep ratio ~ U(lo, hi), kept = max(1, round(r*size)); fixed spaces keep everything."""
    g = np.random.default_rng(seed)
    out = []
    for s, f in zip(net.space_sizes, net.space_fixed):
        r = g.uniform(lo, hi)
        out.append(s if f else max(1, int(round(r * s))))
    return out


def staged_keep_to_flops(net: Net, seed: int, target: float = 0.60, lows=(0.35, 0.35, 0.40, 0.50, 0.60)) -> List[int]:
    """Per-space ratio ~ U(lo(stage), 1), then one global scale (ratios clipped to 1) found by bisection
    so that the pruned forward MACs are `target` of dense. Early stages get the smaller ratios."""
    g = np.random.default_rng(seed)
    base = np.array([1.0 if f else g.uniform(lows[min(st, len(lows) - 1)], 1.0)
                     for f, st in zip(net.space_fixed, net.space_stage)])
    dense = fwd_macs(net)

    def sizes(scale):
        return [s if f else max(1, int(round(min(1.0, b * scale) * s)))
                for s, f, b in zip(net.space_sizes, net.space_fixed, base)]

    a, b_ = 0.2, 2.0
    for _ in range(60):
        m = 0.5 * (a + b_)
        if fwd_macs(with_sizes(net, sizes(m))) / dense < target:
            a = m
        else:
            b_ = m
    return sizes(0.5 * (a + b_))


def choose_kept(net: Net, kept_counts: Sequence[int], seed: int) -> List[np.ndarray]:
    """Which channel indices of each space survive: a seeded random subset of the given size, ascending."""
    g = np.random.default_rng(seed)
    out = []
    for s, k in zip(net.space_sizes, kept_counts):
        out.append(np.sort(g.permutation(s)[:k]).astype(np.int32))
    return out


def per_layer_zero_masks(net: Net, kept_counts: Sequence[int], seed: int, extra: float = 0.1):
    """(zero_out[layer], zero_in[layer]) uint8 masks with sparsity that differs between the convolutions sharing a space,
    as learned sparsity does (Sec. 4.2: each later residual path adds new information to the shared node). Every space
    gets a common core of kept_counts[s] dense channels; in a space with several members each member additionally keeps
    each remaining channel with probability `extra`, independently. Private spaces (one writer, one reader) share the core
    exactly."""
    g = np.random.default_rng(seed)
    cores = choose_kept(net, kept_counts, seed + 1)
    zo = [np.ones(l.K, np.uint8) for l in net.layers]
    zi = [np.ones(l.C, np.uint8) for l in net.layers]
    for s, size in enumerate(net.space_sizes):
        members = [(li, "out") for li, l in enumerate(net.layers) if l.out_space == s] + \
                  [(li, "in") for li, l in enumerate(net.layers) if l.in_space == s]
        shared = sum(1 for _, sd in members if sd == "out") > 1 or sum(1 for _, sd in members if sd == "in") > 1
        for li, side in members:
            m = zo[li] if side == "out" else zi[li]
            m[cores[s]] = 0
            if net.space_fixed[s]:
                m[:] = 0
            elif shared and extra > 0:
                m[g.random(size) < extra] = 0
    return zo, zi


# --------------------------------------------------------------------------- tensors
def _gen(seed: int) -> torch.Generator:
    return torch.Generator(device="cpu").manual_seed(int(seed))


def bf16_round(t: torch.Tensor) -> torch.Tensor:
    """Data conversion only: the value a bf16 tensor holding `t` would contain, as fp32."""
    return t.to(torch.bfloat16).to(torch.float32)


def gen_weight(K, R, S, C, seed, fan_in: Optional[int] = None) -> torch.Tensor:
    """fp32 master weights ~ N(0, sqrt(2/fan_in)), layout [K][R][S][C]."""
    fan = fan_in if fan_in is not None else C * R * S
    return torch.randn((K, R, S, C), generator=_gen(seed), dtype=torch.float32) * float(np.sqrt(2.0 / fan))


def gen_image(N, H, W, C, seed) -> torch.Tensor:
    """Network input ~ N(0,1), bf16-representable fp32, [N][H][W][C]."""
    return bf16_round(torch.randn((N, H, W, C), generator=_gen(seed), dtype=torch.float32))


def gen_act(N, H, W, C, seed) -> torch.Tensor:
    """Input of a deeper layer: max(N(0,1), 0) (post-BN-ReLU statistics), bf16-representable fp32."""
    return bf16_round(torch.randn((N, H, W, C), generator=_gen(seed), dtype=torch.float32).clamp_(min=0))


def gen_dy(N, P, Q, K, seed) -> torch.Tensor:
    """Upstream gradient ~ N(0,1) * 2^-6, bf16-representable fp32."""
    return bf16_round(torch.randn((N, P, Q, K), generator=_gen(seed), dtype=torch.float32) * (2.0 ** -6))


def gen_logits(n, classes, seed, scale=3.0):
    """Classifier outputs of a freshly initialised network ~ N(0, scale) and uniform integer labels."""
    g = _gen(seed)
    logits = torch.randn((n, classes), generator=g, dtype=torch.float32) * scale
    labels = torch.randint(0, classes, (n,), generator=g, dtype=torch.int32)
    return logits, labels


def gen_small(shape, seed, std=1e-3) -> torch.Tensor:
    """Gradients / momenta for stand-alone update runs ~ N(0, std)."""
    return torch.randn(tuple(shape), generator=_gen(seed), dtype=torch.float32) * std


@dataclass
class Model:
    """Host-side fp32 state of every conv of a Net: weights, momentum, gradient, BN vectors."""
    net: Net
    w: List[torch.Tensor]
    v: List[torch.Tensor]
    g: List[torch.Tensor]
    bn: List[List[torch.Tensor]]       # gamma, beta, running mean, running var per layer (K each)


def gen_model(net: Net, seed: int, kept: Optional[List[np.ndarray]] = None, decoys: int = 0,
              with_grad: bool = True) -> Model:
    """Dense-shaped model. If `kept` is given, channels outside kept[space] are set exactly to zero in
    w, v and g of EVERY member of the space (rows of writers, columns of readers). `decoys` channels per
    space (drawn from the kept ones, only where the space has >= 2 members) are zeroed in all members but
    one, so a correct union rule must keep them."""
    ws, vs, gs, bns = [], [], [], []
    for li, l in enumerate(net.layers):
        sd = seed + 1000 * (li + 1)
        w = gen_weight(l.K, l.R, l.R, l.C, sd)
        v = gen_small(w.shape, sd + 1)
        g = gen_small(w.shape, sd + 2) if with_grad else torch.zeros_like(w)
        gam = 0.5 + torch.rand(l.K, generator=_gen(sd + 3))
        bet = 0.1 * torch.randn(l.K, generator=_gen(sd + 4))
        mean = 0.1 * torch.randn(l.K, generator=_gen(sd + 5))
        var = 0.5 + torch.rand(l.K, generator=_gen(sd + 6))
        ws.append(w); vs.append(v); gs.append(g); bns.append([gam, bet, mean, var])
    if kept is not None:
        rng = np.random.default_rng(seed + 77)
        for s, size in enumerate(net.space_sizes):
            dead = np.setdiff1d(np.arange(size), kept[s])
            members = [(li, "out") for li, l in enumerate(net.layers) if l.out_space == s] + \
                      [(li, "in") for li, l in enumerate(net.layers) if l.in_space == s]
            for li, side in members:
                for t in (ws[li], vs[li], gs[li]):
                    if side == "out":
                        t[torch.from_numpy(dead).long()] = 0.0
                    else:
                        t[:, :, :, torch.from_numpy(dead).long()] = 0.0
            if decoys and len(members) >= 2 and len(kept[s]) > decoys + 1 and not net.space_fixed[s]:
                dec = rng.choice(kept[s], size=decoys, replace=False)
                for j in dec:
                    alive = rng.integers(len(members))
                    for mi, (li, side) in enumerate(members):
                        if mi == alive:
                            continue
                        for t in (ws[li], vs[li], gs[li]):
                            if side == "out":
                                t[int(j)] = 0.0
                            else:
                                t[:, :, :, int(j)] = 0.0
    return Model(net, ws, vs, gs, bns)


def layer_seed(cfg_index: int, layer_index: int, what: int = 0) -> int:
    return BASE_SEED + cfg_index + 1000 * layer_index + 100000 * what


def pad8(c: int) -> int:
    """Smallest legal channel pitch: the next multiple of 8 elements (16 bytes of bf16)."""
    return (int(c) + 7) // 8 * 8


def pad16(c: int) -> int:
    """Preferred activation pitch: the next multiple of 16 elements, so every pixel row starts on a 32-byte sector
    (rows on odd 16-byte boundaries cost the TMA unit about 1.5x the time per row)."""
    return (int(c) + 15) // 16 * 16
