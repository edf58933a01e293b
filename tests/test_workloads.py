"""Host-side checks of the seeded input generators (shapes and tree structure named by the configs)."""
import numpy as np

from paper_2506_14158_b200 import workloads as W


def _check_tree(parent, T):
    assert parent.shape == (T,) and parent[0] == -1
    assert all(0 <= parent[i] < i for i in range(1, T))
    assert all(parent[i] <= parent[i + 1] for i in range(1, T - 1))  # breadth-first: siblings contiguous


def test_branching_trees_match_the_named_configs():
    p1 = W.tree_from_branching((3, 2, 1), 15)
    _check_tree(p1, 15)
    assert W.tree_depths(p1).max() == 3 and len(W.children_of(p1, 0)) == 3
    p2 = W.tree_from_branching((4, 3, 2, 2, 1), 26)
    _check_tree(p2, 26)
    d2 = W.tree_depths(p2)
    assert d2.max() == 5 and len(W.children_of(p2, 0)) == 4
    assert max(len(W.children_of(p2, n)) for n in range(26) if d2[n] == 1) == 3


def test_random_trees_are_seeded_and_bounded():
    for name in ("c3", "c4"):
        cfg = W.CONFIGS[name]
        a, b = W.make_trees(cfg), W.make_trees(cfg)
        np.testing.assert_array_equal(a, b)
        for s in range(cfg.B):
            _check_tree(a[s], cfg.T)
            assert W.tree_depths(a[s]).max() <= cfg.max_tree_depth
            counts = np.bincount(a[s][1:], minlength=cfg.T)
            assert counts.max() <= 4
    c4 = W.make_trees(W.CONFIGS["c4"])
    assert not np.array_equal(c4[0], c4[1])  # independent trees per sequence


def test_accept_inputs_shapes_and_token_modes():
    cfg = W.CONFIGS["c1"]
    parent = W.make_trees(cfg)
    for mode in ("topk", "sampled"):
        x = W.make_accept_inputs(cfg, parent, 1.0, token_mode=mode)
        assert x["logits"].shape == (1, 15, 1000) and x["logits"].dtype == np.float32
        np.testing.assert_allclose(x["draft_probs"].sum(-1), 1.0, atol=1e-5)
        assert (x["uniforms"] >= 0).all() and (x["uniforms"] < 1).all()
        for n in range(cfg.T):
            kids = W.children_of(parent[0], n)
            toks = x["tokens"][0, kids]
            assert len(set(toks.tolist())) == len(kids)  # siblings carry distinct tokens
            if mode == "topk" and kids:
                order = np.argsort(-x["draft_probs"][0, n].astype(np.float64), kind="stable")
                assert list(toks) == list(order[: len(kids)])
    y = W.make_accept_inputs(cfg, parent, 1.0)
    np.testing.assert_array_equal(x["logits"], y["logits"])


def test_attention_inputs_layout():
    cfg = W.CONFIGS["c1"]
    q, k, v = W.make_attention_inputs(cfg)
    assert q.shape == (1, 4, 15, 64) and k.shape == (1, 4, cfg.C, 64) and cfg.C >= cfg.L + cfg.T
    assert (k[:, :, cfg.L + cfg.T:] == 0).all() and k[:, :, : cfg.L + cfg.T].abs().sum() > 0
    q2, _, _ = W.make_attention_inputs(cfg, layer=1)
    assert not np.array_equal(q.numpy(), q2.numpy())
