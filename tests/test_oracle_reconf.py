"""Pins for the oracle's keep sets (intersection rule / channel union), gather and the
"compacted model computes the same function" invariant (Sec. 4.2)."""
import itertools

import numpy as np

import oracle
from paper_1901_09290_b200 import workloads as W


def test_adjacent_layers_prune_only_the_intersection():
    # space 1 has one writer (layer 0) and one reader (layer 1)
    g = oracle.Graph(sizes=[3, 4, 2], fixed=[True, False, True], layers=[(0, 1), (1, 2)])
    zo = [np.array([1, 1, 0, 0], np.uint8), np.zeros(2, np.uint8)]
    zi = [np.zeros(3, np.uint8), np.array([1, 0, 1, 0], np.uint8)]
    keep = oracle.keep_sets(g, zo, zi)
    assert keep[1].tolist() == [1, 2, 3]          # only channel 0 is sparse on both sides
    assert keep[0].tolist() == [0, 1, 2] and keep[2].tolist() == [0, 1]


def test_single_member_spaces():
    # a layer that is the only reader of its input space and the only writer of its output space
    g = oracle.Graph(sizes=[4, 3], fixed=[False, False], layers=[(0, 1)])
    keep = oracle.keep_sets(g, [np.array([0, 1, 0], np.uint8)], [np.array([1, 0, 0, 1], np.uint8)])
    assert keep[0].tolist() == [1, 2] and keep[1].tolist() == [0, 2]


def _stage_graph():
    # node A (space 0, fixed) -> shortcut conv (layer 0) -> node B (space 1)
    # block 1: A -> c1 (layer 1) -> space 2 -> c2 (layer 2) -> B ; block 2: B -> c3 (layer 3) -> space 3 -> c4 (layer 4) -> B
    return oracle.Graph(sizes=[2, 3, 2, 2], fixed=[True, False, False, False],
                        layers=[(0, 1), (0, 2), (2, 1), (1, 3), (3, 1)])


def test_union_rule_exhaustive_on_a_small_stage():
    g = _stage_graph()
    # members of node B (space 1): writers 0, 2, 4 ; reader 3  -> 4 members x 3 channels = 12 bits
    members = [("o", 0), ("o", 2), ("o", 4), ("i", 3)]
    for bits in itertools.product([0, 1], repeat=12):
        zo = [np.zeros(g.sizes[o], np.uint8) for (_, o) in g.layers]
        zi = [np.zeros(g.sizes[i], np.uint8) for (i, _) in g.layers]
        for m, (side, li) in enumerate(members):
            for j in range(3):
                (zo if side == "o" else zi)[li][j] = bits[m * 3 + j]
        keep = oracle.keep_sets(g, zo, zi)
        # independent statement: removed iff the bit is set for all four members
        exp = [j for j in range(3) if not all(bits[m * 3 + j] for m in range(4))]
        assert keep[1].tolist() == exp
        assert keep[0].tolist() == [0, 1] and keep[2].tolist() == [0, 1] and keep[3].tolist() == [0, 1]


def test_empty_keep_set_is_reported_not_clamped():
    g = oracle.Graph(sizes=[2, 2, 2], fixed=[True, False, True], layers=[(0, 1), (1, 2)])
    keep = oracle.keep_sets(g, [np.ones(2, np.uint8), np.zeros(2, np.uint8)], [np.zeros(2, np.uint8), np.ones(2, np.uint8)])
    assert keep[1].size == 0


def test_gather_identity_and_composition():
    rng = np.random.default_rng(1)
    w = rng.standard_normal((6, 3, 3, 5)).astype(np.float32)
    w[2] = 0.0                                  # a zeroed group that survives stays exactly zero
    mk, mc = np.array([0, 2, 5], np.int32), np.array([1, 3, 4], np.int32)
    g1 = oracle.gather_weight(w, mk, mc)
    assert g1.shape == (3, 3, 3, 3)
    for a, k in enumerate(mk):
        for b, c in enumerate(mc):
            assert np.array_equal(g1[a, :, :, b].view(np.uint32), w[k, :, :, c].view(np.uint32))
    assert np.all(g1[1] == 0)
    mk2, mc2 = np.array([0, 2], np.int32), np.array([2], np.int32)
    g2 = oracle.gather_weight(g1, mk2, mc2)
    assert np.array_equal(g2, oracle.gather_weight(w, mk[mk2], mc[mc2]))
    assert oracle.gather_vector(np.arange(6.0), mk).tolist() == [0.0, 2.0, 5.0]


def test_compacted_stage_equals_masked_stage():
    """Remove only channels that are zero in every member: the smaller dense model computes the same
    function as the unpruned model with those weights zero, for any BN parameters (beta != 0 included)."""
    rng = np.random.default_rng(2)
    bf = lambda a: np.asarray(oracle.round_bf16(a.astype(np.float32)), np.float64)
    C0, CB, CI = 3, 6, 5
    x = bf(rng.standard_normal((2, 5, 5, C0)))
    bn = lambda K: [0.5 + rng.random(K), 0.3 * rng.standard_normal(K), 0.1 * rng.standard_normal(K), 0.5 + rng.random(K)]
    sc = {"w": bf(rng.standard_normal((CB, 1, 1, C0))), "bn": bn(CB)}
    blocks = [{"w1": bf(rng.standard_normal((CI, 3, 3, CB))), "bn1": bn(CI),
               "w2": bf(rng.standard_normal((CB, 3, 3, CI))), "bn2": bn(CB)} for _ in range(2)]
    deadB, deadI0 = [1, 4], [0, 3]               # node-B channels / block-0 internal channels to remove
    decoyB = 2                                   # zero in every member but one: must be kept
    sc["w"][deadB + [decoyB]] = 0
    for bi, b in enumerate(blocks):
        b["w1"][:, :, :, deadB + [decoyB]] = 0
        b["w2"][deadB] = 0
        if bi == 0:
            b["w2"][decoyB] = 0                  # block 1's w2 keeps channel decoyB alive
    blocks[0]["w1"][deadI0] = 0
    blocks[0]["w2"][:, :, :, deadI0] = 0

    graph = oracle.Graph(sizes=[C0, CB, CI, CI], fixed=[True, False, False, False],
                         layers=[(0, 1), (1, 2), (2, 1), (1, 3), (3, 1)])
    ws = [sc["w"], blocks[0]["w1"], blocks[0]["w2"], blocks[1]["w1"], blocks[1]["w2"]]
    zz = [oracle.find_zero_groups(w) for w in ws]
    keep = oracle.keep_sets(graph, [z[0] for z in zz], [z[1] for z in zz])
    assert keep[1].tolist() == [0, 2, 3, 5] and keep[2].tolist() == [1, 2, 4] and keep[3].tolist() == list(range(CI))

    full = oracle.toy_stage_forward(x, blocks, sc)
    gw = lambda w, li: oracle.gather_weight(w, keep[graph.layers[li][1]], keep[graph.layers[li][0]]).astype(np.float64)
    gb = lambda bnp, s: [oracle.gather_vector(v, keep[s]) for v in bnp]
    sc_c = {"w": gw(sc["w"], 0), "bn": gb(sc["bn"], 1)}
    blocks_c = [{"w1": gw(blocks[0]["w1"], 1), "bn1": gb(blocks[0]["bn1"], 2),
                 "w2": gw(blocks[0]["w2"], 2), "bn2": gb(blocks[0]["bn2"], 1)},
                {"w1": gw(blocks[1]["w1"], 3), "bn1": gb(blocks[1]["bn1"], 3),
                 "w2": gw(blocks[1]["w2"], 4), "bn2": gb(blocks[1]["bn2"], 1)}]
    comp = oracle.toy_stage_forward(x, blocks_c, sc_c)
    # kept channels are visited in the same ascending order and removed ones only ever added exact zeros
    assert np.array_equal(comp, full[..., keep[1]])
    # a removed node channel may carry a non-zero constant (BN beta) in the unpruned model, but nobody reads it
    assert np.any(full[..., deadB] != 0)


def test_toy_conv_matches_c_conv():
    rng = np.random.default_rng(3)
    x = np.asarray(oracle.round_bf16(rng.standard_normal((2, 5, 4, 3)).astype(np.float32)))
    w = np.asarray(oracle.round_bf16(rng.standard_normal((4, 3, 3, 3)).astype(np.float32)))
    np.testing.assert_allclose(oracle.conv_fwd_f64(x, w, 2, 1), oracle.conv_fwd(x, w, 2, 1), rtol=0, atol=1e-12)


def test_workload_generator_embeds_zero_groups_and_decoys():
    net = W.resnet32()
    counts = W.random_keep(net, W.BASE_SEED + 2)
    kept = W.choose_kept(net, counts, W.BASE_SEED + 2)
    model = W.gen_model(net, W.BASE_SEED + 2, kept=kept, decoys=2)
    ws = [w.numpy() for w in model.w]
    zz = [oracle.find_zero_groups(w) for w in ws]
    graph = oracle.Graph(list(net.space_sizes), list(net.space_fixed), [(l.in_space, l.out_space) for l in net.layers])
    keep = oracle.keep_sets(graph, [z[0] for z in zz], [z[1] for z in zz])
    for s in range(len(net.space_sizes)):
        assert keep[s].tolist() == kept[s].tolist(), net.space_names[s]
    # decoys exist: some kept channel is flagged zero by at least one member of its space
    n_decoy = 0
    for li, l in enumerate(net.layers):
        n_decoy += int(zz[li][0][kept[l.out_space]].sum()) + int(zz[li][1][kept[l.in_space]].sum())
    assert n_decoy > 0
