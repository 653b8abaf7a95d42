"""The allocation-free detection entry point against the oracle and the regular entry point.

Some users of the library cannot allocate device memory at the point where they need the zero masks (their framework
owns the device heap, or an allocation's synchronisation or a possible out-of-memory error is not acceptable there), so
they cannot provide the workspace pt_find_zero_groups wants. pt_find_zero_groups_noalloc keeps its scratch in a static device array that every call shares and that is never
cleared between calls. This file runs last on purpose and calls it twice in a row, with a second tensor whose zero
groups differ from the first one's, so that stale scratch from the first call (or from any earlier test) would show.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_09290_b200 import binding as B
from paper_1901_09290_b200 import workloads as W
from tests import helpers as Hh

pytestmark = pytest.mark.gpu


def _reference_masks(w, K, C, RS, thr):
    """The existing entry point, with a caller-provided workspace."""
    ctx = Hh.ctx()
    zo = torch.full((K,), 9, dtype=torch.uint8, device="cuda")
    zi = torch.full((C,), 9, dtype=torch.uint8, device="cuda")
    sq_o, sq_i = torch.empty(K, device="cuda"), torch.empty(C, device="cuda")
    layer = B.make_layer(w, None, w, None, K, C, RS, 0, True, True, sq_o, sq_i, zo, zi)
    arr = B.layer_array([layer])
    ws = torch.empty(max(256, B.pt_group_lasso_workspace_bytes(ctx, arr)), dtype=torch.uint8, device="cuda")
    B.pt_find_zero_groups(ctx, arr, thr, False, ws)
    torch.cuda.synchronize()
    return zo, zi


def _tensor(K, R, C, seed, dead_k, dead_c):
    w = W.gen_weight(K, R, R, C, seed)
    w[dead_k] = 0.0
    w[:, :, :, dead_c] = 0.5e-4          # below the threshold but not zero
    return w.cuda()


def test_noalloc_detection_matches_the_workspace_version_twice_in_a_row():
    thr = 1e-4
    cases = [(70, 3, 93, 1, [0, 5, 69], [2, 92]),        # first call
             (40, 3, 93, 2, [1, 39], [0, 50, 91]),       # second call: fewer rows, other dead groups, same scratch slots
             (300, 1, 2500, 3, [7, 299], [0, 1, 2499])]  # and a wider one
    for K, R, C, seed, dead_k, dead_c in cases:
        w = _tensor(K, R, C, seed, dead_k, dead_c)
        zo = torch.full((K,), 7, dtype=torch.uint8, device="cuda")
        zi = torch.full((C,), 7, dtype=torch.uint8, device="cuda")
        B.pt_find_zero_groups_noalloc(w, K, C, R * R, thr, zo, zi)
        torch.cuda.synchronize()
        # the checker is the oracle's brute-force search on the same bits; the regular entry point must agree too
        orc_o, orc_i = oracle.find_zero_groups(w.cpu().numpy(), thr)
        assert np.array_equal(zo.cpu().numpy(), orc_o) and np.array_equal(zi.cpu().numpy(), orc_i)
        ref_o, ref_i = _reference_masks(w, K, C, R * R, thr)
        assert torch.equal(zo, ref_o) and torch.equal(zi, ref_i)
        assert sorted(torch.nonzero(zo).flatten().tolist()) == sorted(dead_k)
        assert sorted(torch.nonzero(zi).flatten().tolist()) == sorted(dead_c)


def test_noalloc_detection_boundary_values():
    """What the header promises beyond the plain case: a NaN keeps its groups, the comparison is a strict '<' on the fp32
    values (an element exactly equal to the threshold keeps its groups), and threshold 0 marks nothing."""
    K, R, C = 24, 3, 40
    thr = np.float32(1e-4)
    w = torch.zeros((K, R, R, C), dtype=torch.float32)
    w[3] = 0.5e-4                                   # a dead row ...
    w[3, 1, 1, 7] = float(thr)                      # ... but for one element exactly at the threshold: kept, and so is column 7
    w[5] = 0.25e-4
    w[5, 0, 2, 11] = float("nan")                   # a NaN keeps row 5 and column 11
    w[9, :, :, :] = 1.0                             # a live row keeps every column
    w[9, :, :, 20] = 0.0                            # column 20 stays below the threshold in every row
    w[3, :, :, 20] = 0.0
    w[5, :, :, 20] = 0.0
    wd = w.cuda()
    for t in (float(thr), 0.0):
        zo = torch.full((K,), 7, dtype=torch.uint8, device="cuda")
        zi = torch.full((C,), 7, dtype=torch.uint8, device="cuda")
        B.pt_find_zero_groups_noalloc(wd, K, C, R * R, t, zo, zi)
        torch.cuda.synchronize()
        orc_o, orc_i = oracle.find_zero_groups(w.numpy(), t)
        assert np.array_equal(zo.cpu().numpy(), orc_o) and np.array_equal(zi.cpu().numpy(), orc_i)
        ref_o, ref_i = _reference_masks(wd, K, C, R * R, t)
        assert torch.equal(zo, ref_o) and torch.equal(zi, ref_i)
        if t > 0:
            assert zo[3] == 0 and zo[5] == 0 and zo[9] == 0 and zo[0] == 1
            assert zi[20] == 1 and zi[7] == 0 and zi[11] == 0
        else:
            assert int(zo.sum()) == 0 and int(zi.sum()) == 0


def test_noalloc_rejects_sizes_beyond_the_static_scratch():
    w = torch.zeros(16, device="cuda")
    z = torch.zeros(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.PtError) as e:
        B.pt_find_zero_groups_noalloc(w, 40000, 30000, 1, 1e-4, z, z)
    assert e.value.status == 2
    with pytest.raises(B.PtError) as e:
        B.pt_find_zero_groups_noalloc(None, 4, 4, 1, 1e-4, z, z)
    assert e.value.status == 1
