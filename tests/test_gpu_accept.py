"""GPU parity: s4c_tree_accept against the float64 oracle -- accepted length, path and next token bit-exact
on the same uniforms; sequences the oracle marks as near ties (|p/q - u| < 1e-6) are counted separately."""
import numpy as np
import pytest

from paper_2506_14158_b200 import workloads as W

from parity import accept_both, assert_accept_equal

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4"])
@pytest.mark.parametrize("mode", ["topk", "sampled"])
def test_named_configs(name, mode):
    cfg = W.CONFIGS[name]
    parent = W.make_trees(cfg)
    for tau in cfg.temperatures:
        if tau == 0.0 and mode == "sampled":
            continue
        x = W.make_accept_inputs(cfg, parent, tau, token_mode=mode)
        got, ref = accept_both(x, parent, tau, max_depth=cfg.max_depth)
        assert (ref["status"] == 0).all()
        excused = assert_accept_equal(got, ref, tau > 0)
        assert excused == 0, f"{excused} near-tie sequences differ"
        if tau > 0:
            np.testing.assert_array_equal(got["near_tie"], ref["near_tie"])


def _synthetic(B, T, V, seed, sigma=2.0, noise=1.0, tau=1.0, mode="sampled", max_tree_depth=6):
    from dataclasses import replace

    cfg = replace(W.CONFIGS["c2"], name="t", config_id=50 + seed, B=B, T=T, V=V, tree="random", logit_sigma=sigma,
                  max_tree_depth=max_tree_depth)
    parent = W.make_trees(cfg)
    x = W.make_accept_inputs(cfg, parent, tau, token_mode=mode)
    return cfg, parent, x


@pytest.mark.parametrize("V", [1, 3, 4, 8, 36, 257, 4096, 4099, 33333, 33336])
def test_odd_vocabulary_sizes(V):
    T = min(9, max(2, V))
    cfg, parent, x = _synthetic(8, T, V, seed=V % 97, tau=0.9)
    if V < 4:  # not enough distinct tokens for siblings: reuse tokens, still well defined
        x["tokens"] %= V
    for tau in (0.0, 0.9):
        got, ref = accept_both(x, parent, tau, max_depth=cfg.max_tree_depth)
        assert assert_accept_equal(got, ref, tau > 0) == 0


def test_many_sequences_walk_every_branch_kind():
    # 256 independent trees: accepted-at-first-sibling, accepted-at-later-sibling (extra residual passes),
    # all-rejected forks and full-depth leaves all occur; every one must match bit for bit.
    cfg, parent, x = _synthetic(256, 24, 2000, seed=7, tau=1.0)
    got, ref = accept_both(x, parent, 1.0, max_depth=cfg.max_tree_depth)
    assert assert_accept_equal(got, ref, True) == 0
    a = ref["accept_len"]
    assert a.min() == 0 and a.max() >= 3
    later = sum(1 for b in range(256) for j in range(1, a[b] + 1)
                if ref["path"][b, j] != W.children_of(parent[b], ref["path"][b, j - 1])[0])
    assert later > 10  # the multi-round (second sibling and beyond) code ran


def test_star_tree_with_many_siblings():
    from dataclasses import replace

    cfg = replace(W.CONFIGS["c2"], name="star", config_id=61, B=16, T=40, V=500)
    parent = np.tile(W.star_tree(40), (16, 1))
    x = W.make_accept_inputs(cfg, parent, 1.0, token_mode="sampled")
    x["uniforms"][:, 1:] = np.maximum(x["uniforms"][:, 1:], 0.97)  # force long rejection chains
    for b in range(4):  # ... and some forks where all 39 siblings fail: the target gives their tokens ~zero mass
        x["logits"][b, 0, x["tokens"][b, 1:]] = -60.0
    got, ref = accept_both(x, parent, 1.0, max_depth=1)
    assert assert_accept_equal(got, ref, True) == 0
    assert (ref["accept_len"][:4] == 0).all() and (ref["path"][4:, 1] >= 10).sum() >= 2


def test_accept_all_and_reject_all():
    cfg = W.CONFIGS["c1"]
    parent = W.make_trees(cfg)
    x = W.make_accept_inputs(cfg, parent, 1.0, token_mode="topk", draft_equals_target=True)  # q = p: ratio 1 > u
    got, ref = accept_both(x, parent, 1.0, max_depth=cfg.max_depth)
    assert ref["accept_len"][0] == cfg.max_depth
    assert_accept_equal(got, ref, True)
    x = W.make_accept_inputs(cfg, parent, 1.0, token_mode="topk")
    x["uniforms"][:, 1:] = np.float32(1.0) - np.float32(2.0 ** -24)
    x["draft_probs"][:] = 0
    x["draft_probs"][:, :, 0] = 1.0  # drafter is certain of token 0 ...
    x["tokens"][:, 1:] = 0
    x["logits"][:, :, 0] = -30.0     # ... which the target finds very unlikely
    got, ref = accept_both(x, parent, 1.0, max_depth=cfg.max_depth)
    assert ref["accept_len"][0] == 0
    assert_accept_equal(got, ref, True)


def test_padded_trees_and_flagged_sequences():
    cfg, parent, x = _synthetic(4, 12, 300, seed=11)
    n_nodes = np.array([12, 7, 1, 12], dtype=np.int32)
    x["tokens"][3, 5] = 300  # outside the vocabulary
    for tau in (0.0, 1.0):
        got, ref = accept_both(x, parent, tau, n_nodes=n_nodes, max_depth=cfg.max_tree_depth)
        assert ref["status"][3] == 2 and ref["accept_len"][3] == -1
        assert_accept_equal(got, ref, tau > 0)
    parent2 = parent.copy()
    parent2[0, 4] = 9
    got, ref = accept_both(x, parent2, 1.0, n_nodes=n_nodes, max_depth=1)  # too shallow a path buffer for some trees
    assert ref["status"][0] == 1 and ref["status"][1] == 8 and ref["status"][2] == 0
    assert_accept_equal(got, ref, True)


def test_greedy_ties_take_the_lowest_index():
    cfg, parent, x = _synthetic(4, 10, 9000, seed=13)
    x["logits"][:] = np.round(x["logits"])  # many exact ties in every row
    got, ref = accept_both(x, parent, 0.0, max_depth=cfg.max_tree_depth)
    assert assert_accept_equal(got, ref, False) == 0


@pytest.mark.parametrize("B,T,tau", [(16, 128, 1.0), (16, 64, 0.0), (4, 32, 0.7)])
def test_sweep_sized_batches_match_bit_for_bit(B, T, tau):
    # the acceptance problem of the full-depth sweep at its largest batch: V = 32000, trees of depth <= 8; 65 M logits take
    # the segment kernels, the smaller ones the row-in-registers clusters
    cfg, parent, x = _synthetic(B, T, 32000, seed=B + T, sigma=3.0, tau=max(tau, 0.5), mode="topk", max_tree_depth=8)
    got, ref = accept_both(x, parent, tau, max_depth=cfg.max_tree_depth)
    assert assert_accept_equal(got, ref, tau > 0) == 0


@pytest.mark.parametrize("V,B,T", [(300, 6, 12),          # row-in-registers clusters
                                   (4099, 6, 12),         # odd vocabulary: segment kernels, scalar loads
                                   (32000, 24, 16)])      # 12 M logits: segment kernels, vector loads
@pytest.mark.parametrize("tau", [0.0, 1.0])
def test_nonfinite_logits_flag_the_sequence_and_nothing_else(V, B, T, tau):
    # NaN, +Inf and -Inf planted in rows the walk visits and in rows it never reaches; both sides must flag the same
    # sequences (S4C_SEQ_NONFINITE = 64), skip them, and agree bit for bit on every other sequence of the batch
    cfg, parent, x = _synthetic(B, T, V, seed=31 + V % 7, tau=max(tau, 0.5), mode="topk")
    lg = x["logits"]
    lg[0, 0, V // 3] = np.nan                 # the root's row: always walked
    lg[1, T - 1, V - 1] = np.inf              # last node, last entry (a leaf, hardly ever reached)
    lg[2, 1, :] = -np.inf                     # a row without any mass
    lg[3, 2, 5 % V] = -np.inf                 # single masked tokens: legal, probability zero
    lg[3, 0, x["tokens"][3, 1]] = -np.inf     # ... one of them a drafted token at the root
    n_nodes = np.full(B, T, dtype=np.int32)
    n_nodes[4] = T - 3
    lg[4, T - 1, 0] = np.nan                  # a padding row: not part of the tree
    got, ref = accept_both(x, parent, tau, n_nodes=n_nodes, max_depth=cfg.max_tree_depth)
    assert ref["status"][:5].tolist() == [64, 64, 64, 0, 0] and (ref["status"][5:] == 0).all()
    assert (got["accept_len"][:3] == -1).all() and (got["next_token"][:3] == -1).all()
    assert assert_accept_equal(got, ref, tau > 0) == 0


@pytest.mark.parametrize("tau", [1e-6, 3e-9, 50.0])
@pytest.mark.parametrize("V,B,T", [(2000, 8, 10), (32000, 24, 16)])
def test_extreme_temperatures(tau, V, B, T):
    # a tiny temperature turns the softmax into (nearly) a one-hot row; below the float spacing of the logits the rows are
    # summed as counts of their maxima.  A large one flattens it.  Decisions stay bit-exact.
    cfg, parent, x = _synthetic(B, T, V, seed=3, tau=1.0, mode="topk")
    x["logits"][0] = np.round(x["logits"][0])  # exact ties at the maximum in some rows
    x["logits"][1] += 1000.0                   # large logits: coarser float spacing
    got, ref = accept_both(x, parent, tau, max_depth=cfg.max_tree_depth)
    assert (ref["status"] == 0).all()
    assert assert_accept_equal(got, ref, True) == 0
