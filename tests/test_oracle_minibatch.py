"""Dynamic mini-batch adjustment (Sec. 4.3): pins of the oracle, and the library's host arithmetic against it."""
import os

import numpy as np
import pytest

import oracle
from paper_1901_09290_b200 import workloads as W

HERE = os.path.dirname(os.path.abspath(__file__))
ONE = [(4, 4, 3, 5, 3, 3, 1, 1)]


def _shapes(net):
    return [(l.H, l.H, l.C, l.K, l.R, l.R, l.stride, l.pad) for l in net.layers]


def test_hand_example_from_the_golden_file():
    rows = [l.split() for l in open(os.path.join(HERE, "golden", "mini_batch_hand_example.txt")) if l.strip() and not l.startswith("#")]
    for b, byts in rows[:3]:
        assert oracle.training_memory_bytes(ONE, int(b)) == int(byts)
    cap, cur, g, lr, nb, nlr = rows[3]
    got = oracle.update_mini_batch(ONE, int(cap), int(cur), float(lr), int(g))
    assert got[0] == int(nb) and abs(got[1] - float(nlr)) < 1e-12


def test_properties_on_resnet50():
    net = W.resnet50()
    shapes = _shapes(net)
    cap = oracle.training_memory_bytes(shapes, 64)                    # the dense model at 64 per GPU just fits (Sec. 5.3)
    assert oracle.update_mini_batch(shapes, cap, 64, 0.1, 32) == (64, 0.1)
    assert oracle.update_mini_batch(shapes, cap - 1, 64, 0.1, 32)[0] == 64        # never shrinks
    prev = 64
    for keep in (0.9, 0.8, 0.7, 0.6, 0.5, 0.4, 0.3):
        sp = _shapes(W.with_sizes(net, W.uniform_keep(net, keep)))
        nb, lr = oracle.update_mini_batch(sp, cap, 64, 0.1, 32)
        assert nb >= prev and (nb - 64) % 32 == 0
        assert oracle.training_memory_bytes(sp, nb) <= cap < oracle.training_memory_bytes(sp, nb + 32)   # the largest that fits
        assert abs(lr - 0.1 * nb / 64) < 1e-15                                       # same ratio as the mini-batch
        prev = nb
    assert prev >= 128                                                 # pruning this far frees room for at least 2x the batch
    # the closed form of the stepping rule
    f = oracle.training_memory_bytes(sp, 0)
    a = oracle.training_memory_bytes(sp, 1) - f
    assert prev == 64 + 32 * ((cap - f - 64 * a) // (32 * a))


def test_library_host_arithmetic_matches_the_oracle():
    from paper_1901_09290_b200 import binding as B
    try:
        B.lib()
    except RuntimeError:
        pytest.skip("library not built")
    net = W.resnet50()
    rng = np.random.default_rng(3)
    for keep in (1.0, 0.6, 0.3):
        sp = _shapes(W.with_sizes(net, W.uniform_keep(net, keep)))
        for batch in (1, 64, 96):
            assert B.pt_training_memory_bytes(sp, batch) == oracle.training_memory_bytes(sp, batch)
        for _ in range(5):
            cap = int(rng.integers(1 << 28, 1 << 36))
            cur = int(rng.integers(1, 200))
            g = int(rng.integers(1, 64))
            nb, lr = B.pt_update_mini_batch(sp, cap, cur, 0.1, g)
            onb, olr = oracle.update_mini_batch(sp, cap, cur, float(np.float32(0.1)), g)
            assert nb == onb and abs(lr - olr) <= 1e-6 * olr
    assert B.pt_training_memory_bytes(ONE, 2) == 4388
    with pytest.raises(B.PtError):
        B.pt_update_mini_batch(ONE, 10000, 0, 0.1, 32)
    with pytest.raises(B.PtError):
        B.pt_update_mini_batch([(4, 4, 3, 5, 3, 3, 0, 1)], 10000, 2, 0.1, 32)
