"""Pins for the oracle's acceptance step (Section 2 speculative sampling; Eq. 11, Eq. 12; greedy per Section 4.1.2).

What fixes the expected values here is never a retyped copy of the oracle's loops:
* greedy: token-by-token greedy decoding of a deterministic synthetic "model" (numpy argmax);
* stochastic: the guarantee stated in Sections 1-2 and 6 -- the emitted token follows the target
  distribution -- checked (a) exactly, by *measuring* the oracle's accept thresholds and resampling
  CDF with bisection over the uniforms and summing over every possible draft proposal, and (b) by a
  seeded Monte-Carlo chi-square test; plus closed-form special cases.
"""
import itertools
import zlib

import numpy as np
import pytest
from scipy import stats
from scipy.special import softmax

import oracle
from paper_2506_14158_b200 import workloads as W

ONE_MINUS = np.float32(1.0) - np.float32(2.0 ** -24)


# ------------------------------------------------------------------ greedy
def _model_logits(prefix, V):
    """Deterministic synthetic target model: logits are a seeded function of the whole token prefix."""
    seed = zlib.crc32(np.asarray(prefix, dtype=np.int64).tobytes())
    return np.random.default_rng(seed).standard_normal(V).astype(np.float32)


def _greedy_decode(prefix, n_new, V):
    seq = list(prefix)
    for _ in range(n_new):
        seq.append(int(np.argmax(_model_logits(seq, V))))
    return seq


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_greedy_verify_reproduces_token_by_token_greedy_decoding(seed):
    rng = np.random.default_rng(seed)
    V, T, n_target = 50, 12, 40
    prefix = [int(t) for t in rng.integers(0, V, 3)]
    want = _greedy_decode(prefix, n_target, V)
    seq = list(prefix)
    rounds = 0
    while len(seq) < len(want):
        parent = W.random_tree(T, 4, rng, 1, 3)
        tokens = np.zeros(T, dtype=np.int32)
        tokens[0] = seq[-1]  # root = last committed token
        node_prefix = {0: list(seq)}
        logits = np.zeros((1, T, V), dtype=np.float32)
        for i in range(T):
            if i > 0:
                node_prefix[i] = node_prefix[parent[i]] + [int(tokens[i])]
            logits[0, i] = _model_logits(node_prefix[i], V)
            kids = W.children_of(parent, i)
            if kids:
                right = int(np.argmax(logits[0, i]))
                cand = [int(t) for t in rng.permutation(V) if t != right][: len(kids)]
                if rng.random() < 0.7:  # a drafter that is right most of the time, at a random sibling rank
                    cand[int(rng.integers(len(kids)))] = right
                tokens[kids] = cand
        r = oracle.accept_greedy(logits, tokens[None], parent[None], max_depth=4)
        a = int(r["accept_len"][0])
        path = r["path"][0]
        assert path[0] == 0 and (path[a + 1:] == -1).all()
        seq += [int(tokens[path[j]]) for j in range(1, a + 1)] + [int(r["next_token"][0])]
        rounds += 1
    assert seq[: len(want)] == want
    assert rounds < n_target  # some drafts were accepted, so fewer rounds than tokens


def test_greedy_planted_trees():
    V = 20
    parent = np.array([-1, 0, 0, 1, 1, 2, 2, 3], dtype=np.int32)  # depths 0,1,1,2,2,2,2,3
    T = len(parent)
    logits = np.zeros((1, T, V), dtype=np.float32)
    g = [3, 7, 11, 2, 5, 9, 13, 17]
    for i, t in enumerate(g):
        logits[0, i, t] = 1.0
    # all-match along 0 -> 1 -> 3 -> 7
    tok = np.array([0, 3, 4, 7, 8, 1, 1, 2], dtype=np.int32)
    r = oracle.accept_greedy(logits, tok[None], parent[None], max_depth=3)
    assert r["accept_len"][0] == 3 and list(r["path"][0]) == [0, 1, 3, 7] and r["next_token"][0] == 17
    # none match: a = 0, bonus token is the argmax at the root
    tok = np.array([0, 4, 5, 7, 8, 1, 1, 2], dtype=np.int32)
    r = oracle.accept_greedy(logits, tok[None], parent[None], max_depth=3)
    assert r["accept_len"][0] == 0 and list(r["path"][0]) == [0, -1, -1, -1] and r["next_token"][0] == 3
    # match only on the second sibling at depth 1, then its second child
    tok = np.array([0, 4, 3, 7, 8, 1, 11, 2], dtype=np.int32)
    r = oracle.accept_greedy(logits, tok[None], parent[None], max_depth=3)
    assert r["accept_len"][0] == 2 and list(r["path"][0]) == [0, 2, 6, -1] and r["next_token"][0] == 13
    # a child whose token matches but whose parent was rejected does not count
    tok = np.array([0, 4, 5, 7, 8, 11, 1, 2], dtype=np.int32)
    r = oracle.accept_greedy(logits, tok[None], parent[None], max_depth=3)
    assert r["accept_len"][0] == 0
    # argmax ties go to the lowest index
    logits[0, 0, 1] = 1.0
    r = oracle.accept_greedy(logits, tok[None], parent[None], max_depth=3)
    assert r["next_token"][0] == 1


def test_greedy_status_flags():
    V = 5
    logits = np.zeros((2, 3, V), dtype=np.float32)
    parent = np.array([[-1, 0, 1], [-1, 0, 0]], dtype=np.int32)
    tokens = np.array([[0, 1, 7], [0, 1, 2]], dtype=np.int32)  # 7 >= V
    r = oracle.accept_greedy(logits, tokens, parent, max_depth=1)
    assert r["status"][0] == (oracle.SEQ_TOKEN_RANGE | oracle.SEQ_DEPTH) and r["accept_len"][0] == -1
    assert r["status"][1] == 0


# ------------------------------------------------------------------ stochastic
def _walk(logits, q, tokens, parent, u, tau=1.0):
    r = oracle.accept_stochastic(logits[None], q[None], tokens[None], parent[None], tau, u[None],
                                 max_depth=len(parent) - 1)
    assert r["status"][0] == 0
    return int(r["accept_len"][0]), [int(x) for x in r["path"][0]], int(r["next_token"][0])


def _bisect_threshold(pred):
    """Largest float32 u in [0,1) with pred(u) true, assuming pred is true below a threshold; returns that threshold."""
    lo, hi = 0.0, 1.0  # pred(lo) assumed true unless the threshold is 0
    if not pred(np.float32(0.0)):
        return 0.0
    if pred(ONE_MINUS):
        return 1.0
    for _ in range(40):
        mid = 0.5 * (lo + hi)
        if pred(np.float32(mid)):
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


def _measure_node(logits, q, tokens, parent, node, u_base, tau=1.0):
    """Measure, by bisection over the uniforms, the oracle's behaviour at `node` (reached with uniforms u_base).

    Returns (accept probabilities a_j of the children in order, each conditional on the earlier ones
    having been rejected; resampling distribution over the vocabulary once all are rejected).
    """
    V = logits.shape[-1]
    kids = W.children_of(parent, node)
    depth_node = int(W.tree_depths(parent)[node])
    u = u_base.copy()
    acc = []
    for c in kids:
        def accepted(x, c=c):
            uu = u.copy()
            uu[c] = x
            a, path, _ = _walk(logits, q, tokens, parent, uu, tau)
            return a > depth_node and path[depth_node + 1] == c
        acc.append(_bisect_threshold(accepted))
        u[c] = ONE_MINUS  # reject it (ratios of exactly >= 1 are handled by the caller's choice of inputs)
    if any(a_j >= 1.0 for a_j in acc):  # some child is always accepted: the fork is never reached
        return acc, np.zeros(V)
    # all children rejected: CDF of the final token as a function of u[0]
    cdf = np.zeros(V + 1)
    for v in range(V):
        def at_most(x, v=v):
            uu = u.copy()
            uu[0] = x
            a, _, tok = _walk(logits, q, tokens, parent, uu, tau)
            assert a == depth_node
            return tok <= v
        cdf[v + 1] = _bisect_threshold(at_most)
    return acc, np.diff(cdf)


def _probs_f32(rng, V):
    q = softmax(rng.standard_normal(V) * 1.5).astype(np.float32)
    return q


@pytest.mark.parametrize("k,tau", [(1, 1.0), (2, 1.0), (3, 1.0), (2, 0.6)])
def test_first_emitted_token_follows_target_exactly_by_enumeration(k, tau):
    """Sum over every ordered proposal of k distinct children (drawn from q without replacement) of
    P(proposal) * P(oracle emits x | proposal), the latter measured from the oracle: must equal p(x)."""
    rng = np.random.default_rng(7 + k)
    V = 5
    parent = np.array([-1] + [0] * k, dtype=np.int32)
    T = k + 1
    logits = np.zeros((T, V), dtype=np.float32)
    logits[0] = rng.standard_normal(V).astype(np.float32) * 1.5
    q = np.zeros((T, V), dtype=np.float32)
    q[0] = _probs_f32(rng, V)
    q[1:] = 1.0 / V
    p = softmax(logits[0].astype(np.float64) / tau)
    q0 = q[0].astype(np.float64)
    q0 = q0 / q0.sum()
    marginal = np.zeros(V)
    for sel in itertools.permutations(range(V), k):
        w, rest = 1.0, 1.0
        for x in sel:  # sequential draws without replacement
            w *= q0[x] / rest
            rest -= q0[x]
        tokens = np.array([0] + list(sel), dtype=np.int32)
        u = np.full(T, 0.5, dtype=np.float32)
        acc, resample = _measure_node(logits, q, tokens, parent, 0, u, tau)
        alive = 1.0
        for a_j, x in zip(acc, sel):
            marginal[x] += w * alive * a_j
            alive *= 1.0 - a_j
        marginal += w * alive * resample
    np.testing.assert_allclose(marginal, p, rtol=0, atol=2e-6)


def test_second_token_follows_target_row_of_the_accepted_child():
    # depth 2: once child c is accepted the walk must use row c of both the logits and the draft probabilities.
    rng = np.random.default_rng(21)
    V = 4
    parent = np.array([-1, 0, 0, 2, 2], dtype=np.int32)
    T = 5
    logits = (rng.standard_normal((T, V)) * 1.5).astype(np.float32)
    q = np.stack([_probs_f32(rng, V) for _ in range(T)])
    p2 = softmax(logits[2].astype(np.float64))
    q2 = q[2].astype(np.float64) / q[2].astype(np.float64).sum()
    marginal = np.zeros(V)
    for sel in itertools.permutations(range(V), 2):
        w = q2[sel[0]] * q2[sel[1]] / (1.0 - q2[sel[0]])
        tokens = np.array([0, 1, 2, sel[0], sel[1]], dtype=np.int32)
        u = np.full(T, 0.5, dtype=np.float32)
        u[1] = ONE_MINUS  # first sibling rejected ...
        u[2] = 0.0        # ... second accepted (needs a positive ratio only)
        # make sure token 2 has positive residual mass at the root so that u=0 accepts it
        logits_ = logits.copy()
        logits_[0] = np.array([0.0, -3.0, 3.0, 0.0], dtype=np.float32)
        q_ = q.copy()
        q_[0] = np.array([0.3, 0.5, 0.1, 0.1], dtype=np.float32)
        acc, resample = _measure_node(logits_, q_, tokens, parent, 2, u)
        alive = 1.0
        for a_j, x in zip(acc, sel):
            marginal[x] += w * alive * a_j
            alive *= 1.0 - a_j
        marginal += w * alive * resample
    np.testing.assert_allclose(marginal, p2, rtol=0, atol=2e-6)


def test_single_candidate_closed_form_dyadic():
    # p = (1/2,1/4,1/8,1/8), q uniform: accept probabilities min(1,p/q) = 1,1,1/2,1/2 and the
    # residual max(p-q,0) is all on token 0 (Section 2's rule for one candidate).
    p = np.array([0.5, 0.25, 0.125, 0.125])
    logits = np.log(p).astype(np.float32)[None].repeat(2, 0)
    q = np.full((2, 4), 0.25, dtype=np.float32)
    parent = np.array([-1, 0], dtype=np.int32)
    want_acc = [1.0, 1.0, 0.5, 0.5]
    for x in range(4):
        tokens = np.array([0, x], dtype=np.int32)
        acc, resample = _measure_node(logits, q, tokens, parent, 0, np.full(2, 0.5, dtype=np.float32))
        assert abs(acc[0] - want_acc[x]) < 1e-6
        if want_acc[x] < 1.0:
            np.testing.assert_allclose(resample, [1, 0, 0, 0], atol=1e-6)
    # at a leaf (no children) the token comes from the unmodified target distribution
    acc, resample = _measure_node(logits[:1], q[:1], np.array([0], dtype=np.int32), np.array([-1], dtype=np.int32),
                                  0, np.full(1, 0.5, dtype=np.float32))
    assert acc == []
    np.testing.assert_allclose(resample, p, atol=1e-6)


def test_temperature_is_applied_to_target_logits():
    logits = np.array([[2.0, 0.0, -1.0]], dtype=np.float32)
    q = np.full((1, 3), 1 / 3, dtype=np.float32)
    for tau in (0.5, 1.0, 2.0):
        _, resample = _measure_node(logits, q, np.array([0], dtype=np.int32), np.array([-1], dtype=np.int32), 0,
                                    np.full(1, 0.5, dtype=np.float32), tau)
        np.testing.assert_allclose(resample, softmax(logits[0].astype(np.float64) / tau), atol=1e-6)


def test_monte_carlo_chi_square_preserves_target_distribution():
    rng = np.random.default_rng(2024)
    N, V, k = 200_000, 8, 3
    T = k + 1
    parent = np.tile(np.array([-1, 0, 0, 0], dtype=np.int32), (N, 1))
    row_logits = (rng.standard_normal(V) * 1.5).astype(np.float32)
    row_q = _probs_f32(rng, V)
    logits = np.tile(row_logits, (N, T, 1))
    q = np.tile(row_q, (N, T, 1))
    q64 = row_q.astype(np.float64) / row_q.astype(np.float64).sum()
    tokens = np.zeros((N, T), dtype=np.int32)
    # children drawn from q sequentially without replacement (Gumbel top-k is that process)
    gumbel = -np.log(-np.log(rng.random((N, V))))
    tokens[:, 1:] = np.argsort(-(np.log(q64) + gumbel), axis=1)[:, :k]
    u = rng.random((N, T), dtype=np.float32)
    r = oracle.accept_stochastic(logits, q, tokens, parent, 1.0, u, max_depth=1)
    a = r["accept_len"]
    first = np.where(a >= 1, tokens[np.arange(N), np.maximum(r["path"][:, 1], 0)], r["next_token"])
    counts = np.bincount(first, minlength=V)
    p = softmax(row_logits.astype(np.float64))
    chi = stats.chisquare(counts, p * N)
    assert chi.pvalue > 1e-3, (chi, counts / N, p)
    # sanity: the test has power -- the draft distribution itself is rejected
    assert stats.chisquare(counts, q64 * N).pvalue < 1e-6


def test_special_cases_and_near_tie_flag():
    V = 6
    rng = np.random.default_rng(5)
    logits = (rng.standard_normal((3, V)) * 2).astype(np.float32)
    p_rows = softmax(logits.astype(np.float64), axis=-1)
    parent = np.array([-1, 0, 1], dtype=np.int32)
    # q == p (as float32): ratio ~ 1 > u for every u in [0,1): the chain is accepted to the leaf
    q = p_rows.astype(np.float32)
    tokens = np.array([0, 2, 4], dtype=np.int32)
    for u_val in (0.0, 0.5, 0.999):
        a, path, _ = _walk(logits, q, tokens, parent, np.full(3, u_val, dtype=np.float32))
        assert a == 2 and path == [0, 1, 2]
    # one-hot draft on x: accept probability is p(x)
    q1 = np.zeros((3, V), dtype=np.float32)
    q1[:, 2] = 1.0
    acc, _ = _measure_node(logits, q1, np.array([0, 2, 4], dtype=np.int32), parent, 0, np.full(3, 0.5, dtype=np.float32))
    assert abs(acc[0] - p_rows[0, 2]) < 1e-6
    # one-hot target: whatever happens, the emitted first token is that token
    hot = np.full((3, V), -1e4, dtype=np.float32)
    hot[:, 3] = 0.0
    qq = np.full((3, V), 1.0 / V, dtype=np.float32)
    for x in range(V):
        for u_val in (0.0, 0.3, 0.99):
            a, path, nxt = _walk(hot, qq, np.array([0, x, 3], dtype=np.int32), parent, np.full(3, u_val, dtype=np.float32))
            first = x if a >= 1 else nxt
            assert first == 3
    # u -> 1 rejects every child whose ratio < 1; u = 0 accepts every child with positive ratio
    qbig = np.full((3, V), 0.0, dtype=np.float32)
    qbig[:, 2] = 0.9
    qbig[:, 0] = 0.1
    lg = np.zeros((3, V), dtype=np.float32)  # uniform target: p(2) = 1/6 < 0.9
    a, _, _ = _walk(lg, qbig, np.array([0, 2, 2], dtype=np.int32), parent, np.full(3, ONE_MINUS, dtype=np.float32))
    assert a == 0
    a, _, _ = _walk(lg, qbig, np.array([0, 2, 2], dtype=np.int32), parent, np.zeros(3, dtype=np.float32))
    assert a == 2
    # near-tie flag: ratio = (1/6)/0.9 ; u set to that value (as float32) is flagged, u far away is not
    ratio = np.float32((1 / 6) / np.float64(np.float32(0.9)))
    u = np.array([0.5, ratio, 0.5], dtype=np.float32)
    r = oracle.accept_stochastic(lg[None], qbig[None], np.array([[0, 2, 2]], dtype=np.int32), parent[None], 1.0, u[None],
                                 max_depth=2)
    assert r["near_tie"][0, 1] == 1
    u[1] = 0.9
    r = oracle.accept_stochastic(lg[None], qbig[None], np.array([[0, 2, 2]], dtype=np.int32), parent[None], 1.0, u[None],
                                 max_depth=2)
    assert r["near_tie"].sum() == 0


def test_zero_draft_probability_and_duplicate_siblings():
    V = 4
    parent = np.array([-1, 0, 0], dtype=np.int32)
    lg = np.zeros((3, V), dtype=np.float32)
    q = np.zeros((3, V), dtype=np.float32)
    q[:, 0] = 1.0
    # child token 1 has q = 0 but p > 0: ratio = +inf, accepted for any u
    a, path, _ = _walk(lg, q, np.array([0, 1, 2], dtype=np.int32), parent, np.full(3, ONE_MINUS, dtype=np.float32))
    assert a == 1 and path[1] == 1
    # duplicate siblings (same token twice): second test of the token uses q = 0 after zeroing.
    q2 = np.zeros((3, V), dtype=np.float32)
    q2[:, 0] = 0.5
    q2[:, 1] = 0.5
    lg2 = np.log(np.array([0.1, 0.3, 0.3, 0.3])).astype(np.float32)[None].repeat(3, 0)
    # token 0: ratio 0.2 -> rejected at u=.9; residual = norm(0,0,.3,.3); token 0 again: p=0,q=0 -> ratio 0 -> rejected
    a, _, nxt = _walk(lg2, q2, np.array([0, 0, 0], dtype=np.int32), parent, np.array([0.1, 0.9, 0.0], dtype=np.float32))
    assert a == 0 and nxt == 2


# ------------------------------------------------------------------ non-finite logits (input validation of the boundary)
def _nonfinite_batch(seed=5, B=6, T=9, V=40):
    rng = np.random.default_rng(seed)
    parent = np.stack([W.random_tree(T, 4, rng, 1, 3) for _ in range(B)])
    logits = (rng.standard_normal((B, T, V)) * 2).astype(np.float32)
    dq = softmax(logits.astype(np.float64) + rng.standard_normal((B, T, V)), axis=-1).astype(np.float32)
    tokens = rng.integers(0, V, (B, T)).astype(np.int32)
    for b in range(B):
        for n in range(T):
            kids = W.children_of(parent[b], n)
            tokens[b, kids] = np.argsort(-dq[b, n], kind="stable")[: len(kids)]
    u = np.minimum(rng.random((B, T), dtype=np.float32), ONE_MINUS)
    return parent, logits, dq, tokens, u


@pytest.mark.parametrize("tau", [0.0, 1.0])
def test_nonfinite_logits_are_flagged_and_the_rest_of_the_batch_is_untouched(tau):
    parent, logits, dq, tokens, u = _nonfinite_batch()
    B, T, V = logits.shape
    run = lambda lg, nn=None: (oracle.accept_stochastic(lg, dq, tokens, parent, tau, u, nn) if tau > 0
                               else oracle.accept_greedy(lg, tokens, parent, nn))
    clean = run(logits)
    assert (clean["status"] == 0).all()
    bad = logits.copy()
    bad[0, 0, 3] = np.nan           # the root's row: always walked
    bad[1, T - 1, 7] = np.inf       # a leaf row that the walk may never reach: flagged all the same
    bad[2, 2, :] = -np.inf          # a row with no mass at all
    bad[3, 4, 5] = -np.inf          # a single masked token: legal
    nn = np.full(B, T, dtype=np.int32)
    nn[4] = T - 2
    bad[4, T - 1, 0] = np.nan       # a padding row (i >= n_nodes): not part of the tree, not looked at
    r = run(bad, nn)
    assert r["status"].tolist() == [64, 64, 64, 0, 0, 0]
    for b in (0, 1, 2):
        assert r["accept_len"][b] == -1 and r["next_token"][b] == -1 and (r["path"][b] == -1).all()
    # -Inf is probability zero: exactly the result of a logit so low that its exponential underflows to zero
    low = logits.copy()
    low[3, 4, 5] = -1e4
    want = run(low, nn)
    for key in ("accept_len", "path", "next_token"):
        np.testing.assert_array_equal(r[key][3:], want[key][3:])
    np.testing.assert_array_equal(r["accept_len"][5], clean["accept_len"][5])
    np.testing.assert_array_equal(r["next_token"][5], clean["next_token"][5])


def test_a_masked_token_is_never_emitted_and_never_accepted():
    # one candidate whose target logit is -Inf: p(x) = 0, so it is rejected for every u, and the resampled token is never x
    V, x = 8, 3
    logits = np.zeros((1, 2, V), dtype=np.float32)
    logits[0, 0, x] = -np.inf
    dq = np.full((1, 2, V), 1.0 / V, dtype=np.float32)
    parent = np.array([[-1, 0]], dtype=np.int32)
    tokens = np.array([[0, x]], dtype=np.int32)
    for u1 in (0.0, 0.5, float(ONE_MINUS)):
        for u0 in np.linspace(0, float(ONE_MINUS), 17):
            r = oracle.accept_stochastic(logits, dq, tokens, parent, 1.0, np.array([[u0, u1]], dtype=np.float32))
            assert r["status"][0] == 0 and r["accept_len"][0] == 0 and r["next_token"][0] != x
