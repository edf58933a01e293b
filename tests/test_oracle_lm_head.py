"""Pins for the oracle's LM head + greedy choice (Eq. 6; Section 3.2) and for the greedy walk on known choices.

Nothing here re-calls the oracle's own matrix product: expected values come from integer arithmetic in plain Python
loops, from closed forms (one-hot states, duplicated vocabulary rows, permutations, scalings) and, for the walk, from the
separately pinned C oracle of greedy verification on full logits."""
import numpy as np
import pytest

import oracle
from paper_2506_14158_b200 import workloads as W


def test_small_integer_case_by_plain_loops():
    rng = np.random.default_rng(5)
    R, V, H = 4, 9, 6
    hid = rng.integers(-4, 5, (R, H))
    wgt = rng.integers(-4, 5, (V, H))
    want = [[sum(int(hid[r, h]) * int(wgt[v, h]) for h in range(H)) for v in range(V)] for r in range(R)]
    got = oracle.lm_head_greedy(hid.astype(np.float32), wgt.astype(np.float32))
    assert got["logits"].tolist() == [[float(x) for x in row] for row in want]   # exact: small integers
    for r in range(R):
        best = max(want[r])
        assert got["token"][r] == want[r].index(best)                             # first maximum
        assert got["max_logit"][r] == best


def test_one_hot_state_reads_a_column_of_the_head():
    rng = np.random.default_rng(6)
    V, H = 50, 12
    wgt = rng.standard_normal((V, H)).astype(np.float32)
    got = oracle.lm_head_greedy(np.eye(H, dtype=np.float32) * 2.5, wgt)
    np.testing.assert_array_equal(got["token"], np.argmax(wgt, axis=0))
    np.testing.assert_allclose(got["max_logit"], 2.5 * wgt.max(axis=0).astype(np.float64), rtol=0, atol=0)


def test_equal_rows_of_the_head_tie_to_the_lowest_token_and_permutations_move_the_choice():
    rng = np.random.default_rng(7)
    R, V, H = 16, 40, 8
    hid = rng.standard_normal((R, H)).astype(np.float32)
    wgt = rng.standard_normal((V, H)).astype(np.float32)
    base = oracle.lm_head_greedy(hid, wgt)["token"]
    dup = np.concatenate([wgt, wgt], axis=0)                       # every token twice: the first copy wins
    np.testing.assert_array_equal(oracle.lm_head_greedy(hid, dup)["token"], base)
    rev = np.concatenate([wgt[::-1], wgt], axis=0)                 # reversed copy first: its index wins
    np.testing.assert_array_equal(oracle.lm_head_greedy(hid, rev)["token"], V - 1 - base)
    perm = rng.permutation(V)
    np.testing.assert_array_equal(perm[oracle.lm_head_greedy(hid, wgt[perm])["token"]], base)


def test_scaling_the_state_keeps_or_reverses_the_choice():
    rng = np.random.default_rng(8)
    hid = rng.standard_normal((10, 16)).astype(np.float32)
    wgt = rng.standard_normal((30, 16)).astype(np.float32)
    ref = oracle.lm_head_greedy(hid, wgt)
    np.testing.assert_array_equal(oracle.lm_head_greedy(4.0 * hid, wgt)["token"], ref["token"])   # exact scaling by 4
    np.testing.assert_array_equal(oracle.lm_head_greedy(-hid, wgt)["token"], np.argmin(ref["logits"], axis=1))


def _planted(seed, B=40, T=14, V=30):
    rng = np.random.default_rng(seed)
    parent = np.stack([W.random_tree(T, 5, rng, 1, 3) for _ in range(B)])
    logits = rng.standard_normal((B, T, V)).astype(np.float32)
    tokens = rng.integers(0, V, (B, T)).astype(np.int32)
    for b in range(B):                      # plant matches (sometimes on two siblings) so that long paths occur
        for n in range(T):
            kids = W.children_of(parent[b], n)
            if kids and rng.random() < 0.7:
                tokens[b, kids[rng.integers(len(kids))]] = int(np.argmax(logits[b, n]))
                if len(kids) > 1 and rng.random() < 0.3:
                    tokens[b, kids[-1]] = int(np.argmax(logits[b, n]))
    return parent, logits, tokens


@pytest.mark.parametrize("seed", [1, 2])
def test_walk_on_known_choices_is_greedy_verification_on_the_logits(seed):
    parent, logits, tokens = _planted(seed)
    want = oracle.accept_greedy(logits, tokens, parent, max_depth=5)
    got = oracle.accept_greedy_tokens(np.argmax(logits, axis=2).astype(np.int32), tokens, parent, max_depth=5)
    assert want["accept_len"].max() >= 3
    for key in ("accept_len", "path", "next_token", "status"):
        np.testing.assert_array_equal(got[key], want[key], err_msg=key)


def test_walk_flags_and_padding_follow_greedy_verification():
    parent, logits, tokens = _planted(3, B=6)
    n_nodes = np.array([14, 9, 1, 14, 14, 14], dtype=np.int32)
    parent[3, 4] = 7                                               # a parent that comes later: malformed
    want = oracle.accept_greedy(logits, tokens, parent, n_nodes, max_depth=2)  # depth limit 2: deeper trees are flagged
    got = oracle.accept_greedy_tokens(np.argmax(logits, axis=2).astype(np.int32), tokens, parent, n_nodes, max_depth=2)
    assert want["status"][3] == oracle.SEQ_BAD_PARENT and (want["status"] & oracle.SEQ_DEPTH).any()
    for key in ("accept_len", "path", "next_token", "status"):
        np.testing.assert_array_equal(got[key], want[key], err_msg=key)


def test_head_then_walk_equals_greedy_verification_on_materialised_logits():
    # integer-valued states and head: the logits are exact in float32, so the two routes must agree exactly
    rng = np.random.default_rng(11)
    B, T, V, H = 12, 10, 25, 7
    parent = np.stack([W.random_tree(T, 4, rng, 1, 3) for _ in range(B)])
    hid = rng.integers(-3, 4, (B * T, H)).astype(np.float32)
    wgt = rng.integers(-3, 4, (V, H)).astype(np.float32)
    head = oracle.lm_head_greedy(hid, wgt)
    tokens = rng.integers(0, V, (B, T)).astype(np.int32)
    choice = head["token"].reshape(B, T)
    for b in range(B):
        for n in range(T):
            kids = W.children_of(parent[b], n)
            if kids:
                tokens[b, kids[0]] = choice[b, n]
    a = oracle.accept_greedy(head["logits"].reshape(B, T, V).astype(np.float32), tokens, parent)
    c = oracle.accept_greedy_tokens(choice, tokens, parent)
    for key in ("accept_len", "path", "next_token", "status"):
        np.testing.assert_array_equal(a[key], c[key], err_msg=key)


# ----------------------------------------------------------------------------- top-k of the head, tree from ranked choices
def test_topk_by_plain_loops_with_ties():
    rng = np.random.default_rng(21)
    R, V, H, k = 5, 11, 4, 4
    hid = rng.integers(-2, 3, (R, H))
    wgt = rng.integers(-2, 3, (V, H))          # few distinct integer logits: many ties
    got = oracle.lm_head_topk(hid.astype(np.float32), wgt.astype(np.float32), k)
    for r in range(R):
        logit = [sum(int(hid[r, h]) * int(wgt[v, h]) for h in range(H)) for v in range(V)]
        left = list(range(V))
        for j in range(k):                      # selection by hand: greatest logit, the lowest token among equals
            best = left[0]
            for v in left:
                if logit[v] > logit[best]:
                    best = v
            left.remove(best)
            assert got["token"][r, j] == best and got["logit"][r, j] == logit[best]


def test_topk_first_column_is_the_greedy_choice_and_rows_are_ranked():
    rng = np.random.default_rng(22)
    hid = rng.standard_normal((20, 16)).astype(np.float32)
    wgt = rng.standard_normal((70, 16)).astype(np.float32)
    top = oracle.lm_head_topk(hid, wgt, 6)
    np.testing.assert_array_equal(top["token"][:, 0], oracle.lm_head_greedy(hid, wgt)["token"])
    assert (np.diff(top["logit"], axis=1) <= 0).all()
    for r in range(20):
        assert len(set(top["token"][r])) == 6
        rest = np.delete(top["logits"][r], top["token"][r])
        assert rest.max() <= top["logit"][r, -1]            # nothing left out beats the last one kept
    wide = oracle.lm_head_topk(hid[:2], wgt[:3], 5)         # k beyond the vocabulary: padded
    assert (wide["token"][:, 3:] == -1).all() and sorted(wide["token"][0, :3]) == [0, 1, 2]


@pytest.mark.parametrize("branching,T", [((4, 3, 2, 2, 1), 26), ((3, 2, 1), 15), ((2, 2, 2), 9), ((4, 3, 2, 2, 1), 7), ((5,), 3),
                                         ((2, 3), 11), ((3,), 1)])
def test_tree_from_ranked_choices_is_the_tree_from_distributions(branching, T):
    # the separately pinned construction from draft distributions, fed with distributions whose ranking the choices are
    rng = np.random.default_rng(len(branching) * 100 + T)
    B, V = 3, 40
    q = rng.random((B, T, V)).astype(np.float32)
    q[0, :, 5] = q[0, :, 9]                                   # ties: the lower token ranks first on both routes
    root = rng.integers(0, V, B).astype(np.int32)
    cl = np.array([7, 0, 100], dtype=np.int32)
    want = oracle.build_tree(q, branching, root, cl)
    topk = np.argsort(-q, axis=2, kind="stable")[:, :, : max(branching)].astype(np.int32)
    got = oracle.build_tree_from_topk(topk, branching, root, T, cl)
    for key in ("tokens", "parent", "position", "n_nodes"):
        np.testing.assert_array_equal(got[key], want[key], err_msg=key)
