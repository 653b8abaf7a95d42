"""The allocation-free detection entry point against the regular one.

Some users of the library cannot allocate device memory at the point where they need the zero masks (their framework
owns the device heap, or an allocation's synchronisation or a possible out-of-memory error is not acceptable there), so
they cannot provide the workspace pt_find_zero_groups wants. pt_find_zero_groups_noalloc keeps its scratch in a static device array that every call shares and that is never
cleared between calls. This file runs last on purpose and calls it twice in a row, with a second tensor whose zero
groups differ from the first one's, so that stale scratch from the first call (or from any earlier test) would show.
"""
import pytest
import torch

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
        ref_o, ref_i = _reference_masks(w, K, C, R * R, thr)
        assert torch.equal(zo, ref_o) and torch.equal(zi, ref_i)
        assert sorted(torch.nonzero(zo).flatten().tolist()) == sorted(dead_k)
        assert sorted(torch.nonzero(zi).flatten().tolist()) == sorted(dead_c)


def test_noalloc_rejects_sizes_beyond_the_static_scratch():
    w = torch.zeros(16, device="cuda")
    z = torch.zeros(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.PtError) as e:
        B.pt_find_zero_groups_noalloc(w, 40000, 30000, 1, 1e-4, z, z)
    assert e.value.status == 2
    with pytest.raises(B.PtError) as e:
        B.pt_find_zero_groups_noalloc(None, 4, 4, 1, 1e-4, z, z)
    assert e.value.status == 1
