"""PruneTrain hot-path ORACLE -- test infrastructure, not product code.

A plain fp64 CPU statement of what the CUDA library computes, written from the
paper. Only ``tests/``, ``__graft_entry__.smoke()`` and ``bench.py``'s
``cpu_baseline`` / ``--impl reference`` legs may import this package; the
product package never does, and this package never imports the product's CUDA
path. The heavy loops live in ``pt_oracle.c`` (plain C, OpenMP over one outer
loop); the graph-level rules (keep sets, compaction, the toy network used for
the "compacted == masked" invariant, FLOP counts) are small numpy/Python loops
here.

Layouts: activations [N][H][W][C], weights [K][R][S][C], dense, numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pt_oracle.c")
_LIB = os.path.join(_HERE, "libpt_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile pt_oracle.c into libpt_oracle.so next to it (gcc -O2 -fopenmp, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _L():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.pto_num_threads.restype = ctypes.c_int
        _lib.pto_out_dim.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_L().pto_num_threads())


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def out_dim(H: int, R: int, stride: int, pad: int) -> int:
    t = H + 2 * pad - R
    return 0 if t < 0 else t // stride + 1


def round_bf16(a) -> np.ndarray:
    """bf16 round-to-nearest-even of fp32 values, widened to fp64."""
    a = _f32(a)
    out = np.empty(a.shape, dtype=np.float64)
    _L().pto_round_bf16(_p(a), _p(out), ctypes.c_size_t(a.size))
    return out


def _conv_args(N, H, W, C, K, R, S, stride, pad):
    return [ctypes.c_int(int(v)) for v in (N, H, W, C, K, R, S, stride, pad)]


def conv_fwd(x, w, stride: int = 1, pad: int = 0) -> np.ndarray:
    """y[n,p,q,k] = sum_{r,s,c} x[n,p*stride-pad+r,q*stride-pad+s,c] w[k,r,s,c]  (Sec. 2.1)."""
    x, w = _f32(x), _f32(w)
    N, H, W, C = x.shape
    K, R, S, C2 = w.shape
    assert C == C2
    P, Q = out_dim(H, R, stride, pad), out_dim(W, S, stride, pad)
    y = np.empty((N, P, Q, K), dtype=np.float64)
    rc = _L().pto_conv_fwd(_p(x), _p(w), _p(y), *_conv_args(N, H, W, C, K, R, S, stride, pad))
    assert rc == 0, rc
    return y


def conv_dgrad(dy, w, H: int, W: int, stride: int = 1, pad: int = 0) -> np.ndarray:
    """dx = adjoint of conv_fwd in x applied to dy (back-propagation through the layer)."""
    dy, w = _f32(dy), _f32(w)
    K, R, S, C = w.shape
    N, P, Q, K2 = dy.shape
    assert K == K2 and P == out_dim(H, R, stride, pad) and Q == out_dim(W, S, stride, pad)
    dx = np.empty((N, H, W, C), dtype=np.float64)
    rc = _L().pto_conv_dgrad(_p(dy), _p(w), _p(dx), *_conv_args(N, H, W, C, K, R, S, stride, pad))
    assert rc == 0, rc
    return dx


def conv_wgrad(x, dy, R: int, S: int, stride: int = 1, pad: int = 0) -> np.ndarray:
    """dw[k,r,s,c] = sum_{n,p,q} dy[n,p,q,k] x[n,p*stride-pad+r,q*stride-pad+s,c]  (Eq. 4)."""
    x, dy = _f32(x), _f32(dy)
    N, H, W, C = x.shape
    N2, P, Q, K = dy.shape
    assert N == N2 and P == out_dim(H, R, stride, pad) and Q == out_dim(W, S, stride, pad)
    dw = np.empty((K, R, S, C), dtype=np.float64)
    rc = _L().pto_conv_wgrad(_p(x), _p(dy), _p(dw), *_conv_args(N, H, W, C, K, R, S, stride, pad))
    assert rc == 0, rc
    return dw


def _samples(fn, a, b, idx, dims):
    a, b = _f32(a), _f32(b)
    idx = np.ascontiguousarray(np.asarray(idx, dtype=np.int64))
    out = np.empty(idx.shape, dtype=np.float64)
    rc = fn(_p(a), _p(b), _p(idx), ctypes.c_int64(idx.size), _p(out), *_conv_args(*dims))
    assert rc == 0, rc
    return out


def conv_fwd_samples(x, w, idx, stride=1, pad=0) -> np.ndarray:
    """Selected elements (flat indices into y[N][P][Q][K]) of conv_fwd, each summed alone."""
    N, H, W, C = np.shape(x)
    K, R, S, _ = np.shape(w)
    return _samples(_L().pto_conv_fwd_samples, x, w, idx, (N, H, W, C, K, R, S, stride, pad))


def conv_dgrad_samples(dy, w, idx, H, W, stride=1, pad=0) -> np.ndarray:
    """Selected elements (flat indices into dx[N][H][W][C]) of conv_dgrad."""
    N = np.shape(dy)[0]
    K, R, S, C = np.shape(w)
    return _samples(_L().pto_conv_dgrad_samples, dy, w, idx, (N, H, W, C, K, R, S, stride, pad))


def conv_wgrad_samples(x, dy, idx, R, S, stride=1, pad=0) -> np.ndarray:
    """Selected elements (flat indices into dw[K][R][S][C]) of conv_wgrad."""
    N, H, W, C = np.shape(x)
    K = np.shape(dy)[3]
    return _samples(_L().pto_conv_wgrad_samples, x, dy, idx, (N, H, W, C, K, R, S, stride, pad))


# --------------------------------------------------------------------------- lasso + SGD
def lasso_sgd(w, g, v, lam: float, lr: float, mu: float, wd: float = 0.0,
              reg_in: bool = True, reg_out: bool = True):
    """One group-lasso + momentum-SGD update of a conv weight w[K][R][S][C]  (Eq. 1-2, Algorithm 1).

    Returns (w_new, v_new, sumsq_out[K], sumsq_in[C], reg_sum) in fp64; reg_sum is Eq. 2
    without lambda, from the pre-update weights.
    """
    w, g, v = _f32(w), _f32(g), _f32(v)
    K, R, S, C = w.shape
    w_new = np.empty(w.shape, np.float64)
    v_new = np.empty(w.shape, np.float64)
    s_out = np.empty(K, np.float64)
    s_in = np.empty(C, np.float64)
    reg = ctypes.c_double(0.0)
    _L().pto_lasso_sgd(_p(w), _p(g), _p(v), ctypes.c_int(K), ctypes.c_int(C), ctypes.c_int(R * S),
                       ctypes.c_int(int(reg_in)), ctypes.c_int(int(reg_out)),
                       ctypes.c_double(lam), ctypes.c_double(lr), ctypes.c_double(mu), ctypes.c_double(wd),
                       _p(w_new), _p(v_new), _p(s_out), _p(s_in), ctypes.byref(reg))
    return w_new, v_new, s_out, s_in, reg.value


def lasso_penalty(ws: Sequence[np.ndarray], reg_in: Sequence[bool], reg_out: Sequence[bool]) -> float:
    """Eq. 2 without lambda: sum over layers of the input- and output-channel group L2 norms."""
    tot = 0.0
    for w, ri, ro in zip(ws, reg_in, reg_out):
        w = np.asarray(w, np.float64)
        if ro:
            tot += float(np.sqrt((w * w).sum(axis=(1, 2, 3))).sum())
        if ri:
            tot += float(np.sqrt((w * w).sum(axis=(0, 1, 2))).sum())
    return tot


def set_coeff(loss1: float, reg_sum: float, ratio: float) -> float:
    """Eq. 3 solved for lambda: ratio = lam*R / (loss1 + lam*R)."""
    return ratio * loss1 / ((1.0 - ratio) * reg_sum)


def cross_entropy(logits, labels) -> float:
    """The classification loss l(y, f(x, W)) of Eq. 1 / Eq. 3 for a softmax classifier: the batch mean of
    -log(softmax(logits)[label]), in fp64 (the paper names the cross-entropy loss after the first forward pass)."""
    z = np.asarray(logits, np.float64)
    lab = np.asarray(labels, np.int64)
    tot = 0.0
    for i in range(z.shape[0]):
        m = z[i].max()
        tot += m + np.log(np.exp(z[i] - m).sum()) - z[i, lab[i]]
    return tot / z.shape[0]


# --------------------------------------------------------------------------- detection
def find_zero_groups(w, thr: float = 1e-4) -> Tuple[np.ndarray, np.ndarray]:
    """(zero_out[K], zero_in[C]) uint8: group is zero iff every |w| < thr in fp32 (Sec. 4.1, Fig. 4)."""
    w = _f32(w)
    K, R, S, C = w.shape
    zo = np.empty(K, np.uint8)
    zi = np.empty(C, np.uint8)
    _L().pto_find_zero_groups(_p(w), ctypes.c_int(K), ctypes.c_int(C), ctypes.c_int(R * S),
                              ctypes.c_float(thr), _p(zo), _p(zi))
    return zo, zi


# --------------------------------------------------------------------------- keep sets + gather
@dataclass
class Graph:
    """Channel spaces and the conv layers that write / read them.

    A *channel space* is one set of channel indices shared by every conv that produces
    it (its output channels) or consumes it (its input channels): the paper's "node" for
    a residual stage, or the private tensor between two adjacent layers (Sec. 4.2).
    ``layers[i] = (in_space, out_space)``; ``fixed[s]`` marks spaces never pruned (image).
    """
    sizes: List[int]
    fixed: List[bool]
    layers: List[Tuple[int, int]]


def keep_sets(graph: Graph, zero_out: Sequence[np.ndarray], zero_in: Sequence[np.ndarray]) -> List[np.ndarray]:
    """Surviving channel indices of every space, ascending (Sec. 4.2, intersection rule / channel union).

    Channel j of a space is removed iff it is sparsified in ALL neighbouring convs: zero as an
    output channel of every writer and zero as an input channel of every reader. Otherwise
    (dense in at least one member: the union of dense channels) it is kept.
    """
    out = []
    for s, size in enumerate(graph.sizes):
        kept = []
        for j in range(size):
            keep = bool(graph.fixed[s])
            for li, (isp, osp) in enumerate(graph.layers):
                if osp == s and not zero_out[li][j]:
                    keep = True
                if isp == s and not zero_in[li][j]:
                    keep = True
            if keep:
                kept.append(j)
        out.append(np.asarray(kept, dtype=np.int32))
    return out


def gather_weight(w_old, mapK, mapC) -> np.ndarray:
    """new[k',r,s,c'] = old[mapK[k'],r,s,mapC[c']], bit for bit (fp32)."""
    w_old = _f32(w_old)
    K, R, S, C = w_old.shape
    mapK = np.ascontiguousarray(mapK, np.int32)
    mapC = np.ascontiguousarray(mapC, np.int32)
    out = np.empty((len(mapK), R, S, len(mapC)), np.float32)
    _L().pto_gather_f32(_p(w_old), ctypes.c_int(C), ctypes.c_int(R * S), _p(mapK), ctypes.c_int(len(mapK)),
                        _p(mapC), ctypes.c_int(len(mapC)), _p(out))
    return out


def gather_vector(vec, mapK) -> np.ndarray:
    vec = np.asarray(vec)
    out = np.empty(len(mapK), vec.dtype)
    for i, j in enumerate(mapK):
        out[i] = vec[j]
    return out


# --------------------------------------------------------------------------- FLOPs
def conv_flops(N, H, W, C, K, R, S, stride, pad) -> int:
    """Useful FLOPs of one conv pass (1 MAC = 2 FLOP) at the given (kept) channel counts."""
    P, Q = out_dim(H, R, stride, pad), out_dim(W, S, stride, pad)
    return 2 * N * P * Q * K * C * R * S


# --------------------------------------------------------------------------- dynamic mini-batch adjustment (Sec. 4.3)
def training_memory_bytes(shapes, batch: int) -> int:
    """Memory one training iteration needs (Sec. 4.3: the "memory context volume of a training iteration"), as the sum
    over the convolutions (H, W, C, K, R, S, stride, pad) of: the parameters' fp32 weight, gradient and momentum and their
    bf16 shadow; and, per sample, the layer's input and output in bf16 together with the gradients of both. Channel
    pitches are the channel counts rounded up to 8, as the tensors are stored."""
    pad8 = lambda c: -(-c // 8) * 8
    tot = 0
    for (H, W, C, K, R, S, stride, pad) in shapes:
        P, Q = out_dim(H, R, stride, pad), out_dim(W, S, stride, pad)
        tot += K * R * S * C * (4 + 4 + 4) + K * R * S * pad8(C) * 2
        tot += batch * 2 * 2 * (H * W * pad8(C) + P * Q * pad8(K))
    return tot


def update_mini_batch(shapes, capacity_bytes: int, cur_batch: int, cur_lr: float, granularity: int = 32):
    """Algorithm 1, UpdateMiniBatch(system_memory, Net): the largest mini-batch cur_batch + g*granularity (g >= 0) whose
    iteration still fits the device memory, found by stepping; the learning rate grows by the same ratio (Sec. 4.3)."""
    nb = cur_batch
    if training_memory_bytes(shapes, cur_batch) <= capacity_bytes:
        while training_memory_bytes(shapes, nb + granularity) <= capacity_bytes:
            nb += granularity
    return nb, cur_lr * nb / cur_batch


# --------------------------------------------------------------------------- feature normalisation (Sec. 2.1)
def bn_relu_fwd(x, gamma, beta, eps: float = 1e-5, residual=None, relu: bool = True):
    """Training-mode batch normalisation of x [N][H][W][C] followed by the residual add and the ReLU of a ResNet block.

    Sec. 2.1: the normalisation layer computes each channel's mean and variance over the mini-batch and the feature map
    and normalises with them; gamma and beta are the per-channel scale and shift that the compaction carries along
    (Sec. 4.2). Per channel c, over the M = N*H*W positions:
        mean = sum(x)/M,  var = sum((x - mean)^2)/M,  xhat = (x - mean)/sqrt(var + eps),
        z = gamma*xhat + beta (+ residual),  y = max(z, 0) if relu else z.
    Returns y, mean, invstd = 1/sqrt(var + eps), var (biased), all fp64."""
    x = np.asarray(x, np.float64)
    N, H, W, C = x.shape
    M = N * H * W
    y = np.empty_like(x)
    mean = np.empty(C)
    var = np.empty(C)
    for c in range(C):
        xc = x[..., c]
        mean[c] = xc.sum() / M
        var[c] = ((xc - mean[c]) ** 2).sum() / M
        z = gamma[c] * (xc - mean[c]) / np.sqrt(var[c] + eps) + beta[c]
        if residual is not None:
            z = z + np.asarray(residual, np.float64)[..., c]
        y[..., c] = np.maximum(z, 0.0) if relu else z
    return y, mean, 1.0 / np.sqrt(var + eps), var


def bn_running_stats(running_mean, running_var, mean, var, M: int, momentum: float = 0.1):
    """The moving statistics a normalisation layer keeps for inference (the vectors the compaction gathers, Sec. 4.2):
    r <- (1 - momentum)*r + momentum*batch statistic, with the unbiased variance var*M/(M-1) (M > 1)."""
    rm = (1.0 - momentum) * np.asarray(running_mean, np.float64) + momentum * mean
    rv = (1.0 - momentum) * np.asarray(running_var, np.float64) + momentum * var * (M / (M - 1.0) if M > 1 else 1.0)
    return rm, rv


def bn_relu_bwd(x, y, dy, gamma, mean, invstd, relu: bool = True):
    """Back-propagation through y = relu(gamma*xhat + beta + residual) with the batch statistics of the forward pass.

    dz = dy where the ReLU passed (y > 0), else 0; the residual branch receives dz unchanged;
        dbeta = sum(dz),  dgamma = sum(dz*xhat),
        dx = gamma*invstd/M * (M*dz - dbeta - xhat*dgamma)      (mean and variance depend on every position)
    Returns dx, dresidual, dgamma, dbeta (fp64)."""
    x = np.asarray(x, np.float64)
    dy = np.asarray(dy, np.float64)
    N, H, W, C = x.shape
    M = N * H * W
    dz = dy * (np.asarray(y, np.float64) > 0) if relu else dy.copy()
    dx = np.empty_like(x)
    dgamma = np.empty(C)
    dbeta = np.empty(C)
    for c in range(C):
        xhat = (x[..., c] - mean[c]) * invstd[c]
        dbeta[c] = dz[..., c].sum()
        dgamma[c] = (dz[..., c] * xhat).sum()
        dx[..., c] = gamma[c] * invstd[c] / M * (M * dz[..., c] - dbeta[c] - xhat * dgamma[c])
    return dx, dz, dgamma, dbeta


# --------------------------------------------------------------------------- pooling (Sec. 2.1)
def maxpool_fwd(x, R: int = 3, stride: int = 2, pad: int = 1):
    """Max pooling of x [N][H][W][C] (Sec. 2.1 lists pooling among the layers of a CNN; ResNet pools once, after its first
    convolution). y[n,p,q,c] = the maximum over the R x R window at (p*stride - pad, q*stride - pad); positions outside
    the image are never selected; of equal maxima the first in scan order (window rows, then columns) is the selected one.
    Returns y (fp64) and sel, the selected position h*W + w of every output element."""
    x = np.asarray(x, np.float64)
    N, H, W, C = x.shape
    P, Q = out_dim(H, R, stride, pad), out_dim(W, R, stride, pad)
    y = np.full((N, P, Q, C), -np.inf)
    sel = np.full((N, P, Q, C), -1, np.int64)
    for p in range(P):
        for q in range(Q):
            for r in range(R):
                h = p * stride - pad + r
                if h < 0 or h >= H:
                    continue
                for s in range(R):
                    w = q * stride - pad + s
                    if w < 0 or w >= W:
                        continue
                    v = x[:, h, w, :]
                    better = (v > y[:, p, q, :]) | (sel[:, p, q, :] < 0)      # strictly greater: the first maximum stays
                    y[:, p, q, :] = np.where(better, v, y[:, p, q, :])
                    sel[:, p, q, :] = np.where(better, h * W + w, sel[:, p, q, :])
    return y, sel


def maxpool_bwd(dy, sel, H: int, W: int) -> np.ndarray:
    """Back-propagation through the pooling: every output position hands its gradient to the input position it selected,
    dx[n,h,w,c] = sum of dy[n,p,q,c] over the (p,q) with sel[n,p,q,c] == h*W + w."""
    dy = np.asarray(dy, np.float64)
    N, P, Q, C = dy.shape
    dx = np.zeros((N, H * W, C))
    for n in range(N):
        for c in range(C):
            np.add.at(dx[n, :, c], sel[n, :, :, c].ravel(), dy[n, :, :, c].ravel())
    return dx.reshape(N, H, W, C)


# --------------------------------------------------------------------------- channel gating (Sec. 4.2)
def dense_channel_list(zero_flags) -> np.ndarray:
    """Ascending positions of the groups that are NOT sparsified: the "dense channel indices" a gating layer gathers
    and scatters (Sec. 4.2)."""
    out = []
    for i, z in enumerate(np.asarray(zero_flags)):
        if not z:
            out.append(i)
    return np.asarray(out, dtype=np.int32)


def channel_gather(x, idx) -> np.ndarray:
    """Gate at the entry of a residual branch (Sec. 4.2): the branch's first convolution sees only the listed channels
    of the node tensor x [N][H][W][C]: out[..., j] = x[..., idx[j]]."""
    x = np.asarray(x)
    out = np.empty(x.shape[:-1] + (len(idx),), x.dtype)
    for j, c in enumerate(idx):
        out[..., j] = x[..., int(c)]
    return out


def channel_scatter_add(branch, idx, node=None, c_node: Optional[int] = None, relu: bool = False) -> np.ndarray:
    """Gate at the merge point (Sec. 4.2): channel j of the branch output goes back to position idx[j] of the node, where
    it is added to what the node holds (the short-cut); every other channel of the node passes through unchanged.
    The paper fixes no precision; the tensors are bf16 and the sum decides a rounding, so, as in the CUDA path, the
    sum is formed in fp32 and rounded once to bf16 (returned as the fp32 value of that bf16)."""
    branch = np.asarray(branch, np.float32)
    if node is None:
        node = np.zeros(branch.shape[:-1] + (int(c_node),), np.float32)
    out = np.array(node, dtype=np.float32, copy=True)
    for j, c in enumerate(idx):
        out[..., int(c)] = out[..., int(c)] + branch[..., j]
    if relu:
        out = np.maximum(out, np.float32(0))
    return round_bf16(out)


def gating_channel_counts(graph: Graph, zero_out: Sequence[np.ndarray], zero_in: Sequence[np.ndarray],
                          keep: Sequence[np.ndarray]) -> List[Tuple[int, int]]:
    """(input channels, output channels) every convolution works on under channel gating (Sec. 4.2).

    A space shared by several branches (more than one writer or more than one reader: the node of a residual stage)
    keeps the union of dense channels, `keep`, but every convolution reading it is gated down to ITS OWN dense input
    channels and every convolution writing it to ITS OWN dense output channels. A private space between two adjacent
    layers has no gate: both sides use the kept channels."""
    writers = [0] * len(graph.sizes)
    readers = [0] * len(graph.sizes)
    for isp, osp in graph.layers:
        readers[isp] += 1
        writers[osp] += 1
    shared = [(writers[s] > 1 or readers[s] > 1) and not graph.fixed[s] for s in range(len(graph.sizes))]
    out = []
    for li, (isp, osp) in enumerate(graph.layers):
        c = sum(1 for j in keep[isp] if not zero_in[li][j]) if shared[isp] else len(keep[isp])
        k = sum(1 for j in keep[osp] if not zero_out[li][j]) if shared[osp] else len(keep[osp])
        out.append((c, k))
    return out


# --------------------------------------------------------------------------- toy network (invariant only)
def bn_affine(y, gamma, beta, mean, var, eps=1e-5):
    """Inference-form batch norm with given running statistics, per output channel."""
    return (y - mean) / np.sqrt(var + eps) * gamma + beta


def toy_stage_forward(x, blocks, shortcut=None):
    """fp64 forward of a small residual stage used to check "compacted == masked".

    x: [N][H][W][C0].  shortcut: optional dict(w, bn) 1x1 projection from the input node.
    blocks: list of dict(w1, bn1, w2, bn2): node -> conv3x3 -> BN -> ReLU -> conv3x3 -> BN -> (+node) -> ReLU.
    Activations are NOT rounded to bf16 between layers beyond what conv_fwd does to its inputs;
    callers pass bf16-representable data when bit-identity matters.
    """
    node = np.asarray(x, np.float64)
    if shortcut is not None:
        node = bn_affine(conv_fwd_f64(node, shortcut["w"], 1, 0), *shortcut["bn"])
    for b in blocks:
        t = np.maximum(bn_affine(conv_fwd_f64(node, b["w1"], 1, 1), *b["bn1"]), 0.0)
        t = bn_affine(conv_fwd_f64(t, b["w2"], 1, 1), *b["bn2"])
        node = np.maximum(t + node, 0.0)
    return node


def conv_fwd_f64(x, w, stride=1, pad=0) -> np.ndarray:
    """The same 7-loop definition in pure fp64 numpy (no bf16 rounding), for the toy network.
    Loops over taps and accumulates channel by channel in ascending order."""
    x = np.asarray(x, np.float64)
    w = np.asarray(w, np.float64)
    N, H, W, C = x.shape
    K, R, S, _ = w.shape
    P, Q = out_dim(H, R, stride, pad), out_dim(W, S, stride, pad)
    y = np.zeros((N, P, Q, K), np.float64)
    for r in range(R):
        for s in range(S):
            for p in range(P):
                h = p * stride - pad + r
                if h < 0 or h >= H:
                    continue
                for q in range(Q):
                    ww = q * stride - pad + s
                    if ww < 0 or ww >= W:
                        continue
                    for c in range(C):
                        y[:, p, q, :] += x[:, h, ww, c][:, None] * w[None, :, r, s, c]
    return y
