"""Pins of the oracle's channel-gating functions (Sec. 4.2) and the CPU-side bookkeeping that goes with them."""
import os

import numpy as np

import oracle
from paper_1901_09290_b200 import harness as Hn
from paper_1901_09290_b200 import workloads as W

HERE = os.path.dirname(os.path.abspath(__file__))


def _ints(shape, seed, lo=-3, hi=4):
    return np.random.default_rng(seed).integers(lo, hi, size=shape).astype(np.float32)


def test_dense_list_against_flatnonzero():
    g = np.random.default_rng(5)
    for n in (0, 1, 7, 64, 1500):
        z = (g.random(n) < 0.4).astype(np.uint8)
        assert oracle.dense_channel_list(z).tolist() == np.flatnonzero(z == 0).tolist()


def test_scatter_is_the_transpose_of_gather():
    """<gather(x), b> == <x, scatter(b)> for all x, b: the two gates are adjoint (each is the other's gradient)."""
    g = np.random.default_rng(6)
    idx = np.sort(g.permutation(11)[:5]).astype(np.int32)
    x = _ints((2, 3, 3, 11), 1)
    b = _ints((2, 3, 3, 5), 2)
    lhs = float((oracle.channel_gather(x, idx).astype(np.float64) * b).sum())
    rhs = float((x.astype(np.float64) * oracle.channel_scatter_add(b, idx, None, c_node=11)).sum())
    assert lhs == rhs
    # and gathering what was scattered gives the branch back; the other channels stay zero
    s = oracle.channel_scatter_add(b, idx, None, c_node=11)
    assert np.array_equal(oracle.channel_gather(s, idx), b)
    assert np.all(np.delete(s, idx, axis=-1) == 0)


def test_gated_convolution_equals_the_sparse_layer():
    """A branch that gathers its dense input channels and scatters its dense output channels computes exactly what the
    un-reconfigured layer with zeroed groups computes (the pinned convolution oracle on both sides)."""
    C, K = 9, 7
    x = _ints((2, 6, 6, C), 3)
    w = _ints((K, 3, 3, C), 4, -2, 3)
    node = _ints((2, 6, 6, K), 5)
    zin = np.array([0, 1, 0, 0, 1, 1, 0, 0, 1], np.uint8)
    zout = np.array([0, 0, 1, 0, 1, 0, 0], np.uint8)
    w_sparse = w.copy()
    w_sparse[:, :, :, zin == 1] = 0
    w_sparse[zout == 1] = 0
    want = node + oracle.conv_fwd(x, w_sparse, 1, 1)
    ii, oi = oracle.dense_channel_list(zin), oracle.dense_channel_list(zout)
    w_dense = w[oi][:, :, :, ii]
    got = oracle.channel_scatter_add(oracle.conv_fwd(oracle.channel_gather(x, ii), w_dense, 1, 1), oi, node)
    assert np.array_equal(got, want)              # small integers: every value is exact in bf16
    assert np.array_equal(oracle.channel_scatter_add(oracle.conv_fwd(oracle.channel_gather(x, ii), w_dense, 1, 1), oi, node, relu=True),
                          np.maximum(want, 0))


def test_scatter_add_rounds_the_fp32_sum_once_to_bf16():
    node = np.array([[1.0, 256.0, -3.0]], np.float32)
    br = np.array([[2.0 ** -8, 1.0]], np.float32)           # 1 + 2^-8 is a bf16 tie -> even (1.0); 257 -> 256 (tie to even)
    out = oracle.channel_scatter_add(br, np.array([0, 1], np.int32), node)
    assert out.tolist() == [[1.0, 256.0, -3.0]]
    out = oracle.channel_scatter_add(np.array([[3 * 2.0 ** -8, 3.0]], np.float32), np.array([0, 1], np.int32), node)
    assert out.tolist() == [[1.0 + 2.0 ** -6, 260.0, -3.0]]  # 1 + 3/256 -> tie between 1+2/256 and 1+4/256 -> even mantissa; 259 -> 260


def _hand():
    rows = [l.split() for l in open(os.path.join(HERE, "golden", "gating_hand_example.txt")) if l.strip() and not l.startswith("#")]
    return {r[0]: tuple(int(v) for v in r[1:]) for r in rows}


def _hand_graph():
    # spaces: 0 = node (4), 1 = A private (2), 2 = B private (2)
    graph = oracle.Graph([4, 2, 2], [False, False, False], [(0, 1), (1, 0), (0, 2), (2, 0)])
    z2 = np.zeros(2, np.uint8)
    zero_in = [np.array([0, 1, 0, 0], np.uint8), z2, np.array([0, 1, 1, 0], np.uint8), z2]
    zero_out = [z2, np.array([1, 1, 0, 0], np.uint8), z2, np.array([0, 1, 0, 1], np.uint8)]
    return graph, zero_out, zero_in


def test_hand_example_counts():
    graph, zo, zi = _hand_graph()
    keep = oracle.keep_sets(graph, zo, zi)
    assert [k.tolist() for k in keep] == [[0, 2, 3], [0, 1], [0, 1]]
    gate = oracle.gating_channel_counts(graph, zo, zi, keep)
    hand = _hand()
    for name, got in zip(["A.c1", "A.c3", "B.c1", "B.c3"], gate):
        assert got == hand[name][2:], name
    union = [(len(keep[i]), len(keep[o])) for i, o in graph.layers]
    for name, got in zip(["A.c1", "A.c3", "B.c1", "B.c3"], union):
        assert got == hand[name][:2], name


def _graph_of(net):
    return oracle.Graph(list(net.space_sizes), list(net.space_fixed), [(l.in_space, l.out_space) for l in net.layers])


def test_union_and_gating_channel_counts_order_the_flops():
    for net in (W.resnet32(), W.resnet50(), W.vgg(11)):
        dense = Hn.conv_macs(net, [(l.C, l.K) for l in net.layers])
        for extra in (0.0, 0.05):
            zo, zi = W.per_layer_zero_masks(net, W.uniform_keep(net, 0.6), W.BASE_SEED + 9, extra)
            graph = _graph_of(net)
            keep = oracle.keep_sets(graph, zo, zi)
            union = [(len(keep[l.in_space]), len(keep[l.out_space])) for l in net.layers]
            gate = oracle.gating_channel_counts(graph, zo, zi, keep)
            mu, mg = Hn.conv_macs(net, union), Hn.conv_macs(net, gate)
            assert mg <= mu <= dense
            if extra == 0.0 or net.name.startswith("vgg"):
                assert mg == mu          # identical masks in a space, or no shared space at all: nothing left to gate
            else:
                assert mg < mu


def test_vgg_tables():
    for depth, n in ((11, 8), (13, 10), (16, 13)):
        net = W.vgg(depth)
        assert len(net.layers) == n and net.layers[0].C == 3 and net.layers[-1].K == 512
        # a plain stack: every space has exactly one writer and one reader (the image and the last map aside)
        for s in range(len(net.space_sizes)):
            assert sum(1 for l in net.layers if l.out_space == s) <= 1 and sum(1 for l in net.layers if l.in_space == s) <= 1
