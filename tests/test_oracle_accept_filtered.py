"""Pins for the oracle's filtered speculative sampling (top-k, then nucleus, applied to the target distribution before the
accept / resample steps of Section 2 and Eq. 11-12).

Expected values never come from the oracle's own filter: the kept set and its probabilities are computed here with a
library sort (numpy), the unfiltered and the greedy special cases are the oracle's other, separately pinned functions, and
the emitted distribution is checked by Monte-Carlo against the numpy-filtered target."""
import numpy as np
import pytest
from scipy import stats
from scipy.special import softmax

import oracle
from paper_2506_14158_b200 import workloads as W

ONE_MINUS = np.float32(1.0) - np.float32(2.0 ** -24)


def _filtered(logits, tau, top_k, top_p):
    """Temperature, then top-k, then nucleus, as a chain of warpers: library sort, ties to the lower index."""
    x = logits.astype(np.float64)
    p = softmax(x / tau)
    order = np.argsort(-logits, kind="stable")[: min(top_k, len(x))]
    pk = p[order] / p[order].sum()
    if top_p < 1.0:
        m = int(np.searchsorted(np.cumsum(pk), top_p, side="left")) + 1
        order, pk = order[:m], pk[:m] / pk[:m].sum()
    out = np.zeros_like(p)
    out[order] = pk
    return out


def _batch(seed, B=48, T=10, V=60, sigma=2.0):
    rng = np.random.default_rng(seed)
    parent = np.stack([W.random_tree(T, 4, rng, 1, 3) for _ in range(B)])
    logits = (rng.standard_normal((B, T, V)) * sigma).astype(np.float32)
    dq = softmax(logits.astype(np.float64) + rng.standard_normal((B, T, V)), axis=-1).astype(np.float32)
    tokens = rng.integers(0, V, (B, T)).astype(np.int32)
    for b in range(B):
        for n in range(T):
            kids = W.children_of(parent[b], n)
            tokens[b, kids] = np.argsort(-dq[b, n], kind="stable")[: len(kids)]
    u = np.minimum(rng.random((B, T), dtype=np.float32), ONE_MINUS)
    return parent, logits, dq, tokens, u


@pytest.mark.parametrize("tau,top_k,top_p", [(1.0, 5, 1.0), (0.7, 8, 0.9), (1.5, 50, 0.5), (1.0, 3, 0.95), (1.0, 12, 0.2)])
def test_the_resampling_distribution_at_a_leaf_is_the_filtered_target(tau, top_k, top_p):
    # a tree of the root alone: the emitted token is an inverse-CDF draw from the (filtered) target with uniforms[0].  A dense
    # grid of uniforms measures that CDF; it must be the CDF of the numpy-filtered distribution.
    rng = np.random.default_rng(int(tau * 10) + top_k)
    V, N = 12, 8192
    row = (rng.standard_normal(V) * 2).astype(np.float32)
    logits = np.tile(row, (N, 1, 1))
    dq = np.full((N, 1, V), 1.0 / V, dtype=np.float32)
    u = ((np.arange(N, dtype=np.float64) + 0.5) / N).astype(np.float32).reshape(N, 1)
    r = oracle.accept_filtered(logits, dq, np.zeros((N, 1), dtype=np.int32), np.full((N, 1), -1, dtype=np.int32), tau, top_k,
                               top_p, u)
    assert (r["status"] == 0).all() and (r["accept_len"] == 0).all()
    want = _filtered(row, tau, top_k, top_p)
    got = np.bincount(r["next_token"], minlength=V) / N
    np.testing.assert_allclose(got, want, atol=1.5 / N)
    assert set(np.nonzero(got)[0]) == set(np.nonzero(want)[0])  # exactly the kept tokens are ever emitted


def test_no_filter_left_is_the_unfiltered_walk():
    parent, logits, dq, tokens, u = _batch(1)
    V = logits.shape[2]
    for tau in (0.6, 1.0):
        a = oracle.accept_stochastic(logits, dq, tokens, parent, tau, u)
        b = oracle.accept_filtered(logits, dq, tokens, parent, tau, V, 1.0, u)
        for key in ("accept_len", "path", "next_token", "status"):
            np.testing.assert_array_equal(a[key], b[key], err_msg=key)


def test_top_1_is_greedy_verification_whatever_the_uniforms():
    # the filtered target is one-hot on the argmax: a child is accepted iff it carries the argmax, the emitted token is the argmax
    parent, logits, dq, tokens, u = _batch(2)
    for b in range(0, len(parent), 3):  # plant some matches so that paths of several tokens occur
        for n in range(parent.shape[1]):
            kids = W.children_of(parent[b], n)
            if kids:
                tokens[b, kids[len(kids) // 2]] = int(np.argmax(logits[b, n]))
    g = oracle.accept_greedy(logits, tokens, parent)
    f = oracle.accept_filtered(logits, dq, tokens, parent, 0.9, 1, 1.0, u)
    assert g["accept_len"].max() >= 2
    for key in ("accept_len", "path", "next_token", "status"):
        np.testing.assert_array_equal(f[key], g[key], err_msg=key)


def test_a_token_outside_the_kept_set_is_never_accepted():
    parent, logits, dq, tokens, u = _batch(3, B=64)
    u[:, 1:] = 0.0  # the most lenient draws: anything with positive filtered probability passes
    r = oracle.accept_filtered(logits, dq, tokens, parent, 1.0, 4, 1.0, u)
    for b in range(len(parent)):
        for j in range(1, r["accept_len"][b] + 1):
            node, par = r["path"][b, j], r["path"][b, j - 1]
            top4 = np.argsort(-logits[b, par], kind="stable")[:4]
            assert tokens[b, node] in top4
        last = r["path"][b, r["accept_len"][b]]
        assert r["next_token"][b] in np.argsort(-logits[b, last], kind="stable")[:4]


def test_monte_carlo_emitted_token_follows_the_filtered_target():
    rng = np.random.default_rng(77)
    N, V, k, top_k, top_p, tau = 200_000, 10, 3, 6, 0.9, 2.0
    T = k + 1
    parent = np.tile(np.array([-1, 0, 0, 0], dtype=np.int32), (N, 1))
    row_logits = (rng.standard_normal(V) * 1.5).astype(np.float32)
    row_q = softmax(rng.standard_normal(V)).astype(np.float32)
    logits, q = np.tile(row_logits, (N, T, 1)), np.tile(row_q, (N, T, 1))
    q64 = row_q.astype(np.float64) / row_q.astype(np.float64).sum()
    tokens = np.zeros((N, T), dtype=np.int32)
    gumbel = -np.log(-np.log(rng.random((N, V))))  # children drawn from q without replacement
    tokens[:, 1:] = np.argsort(-(np.log(q64) + gumbel), axis=1)[:, :k]
    u = rng.random((N, T), dtype=np.float32)
    r = oracle.accept_filtered(logits, q, tokens, parent, tau, top_k, top_p, u, max_depth=1)
    first = np.where(r["accept_len"] >= 1, tokens[np.arange(N), np.maximum(r["path"][:, 1], 0)], r["next_token"])
    counts = np.bincount(first, minlength=V)
    want = _filtered(row_logits, tau, top_k, top_p)
    keep = want > 0
    assert counts[~keep].sum() == 0
    assert stats.chisquare(counts[keep], want[keep] * N).pvalue > 1e-3
    assert keep.sum() >= 3
    # the test has power: the draft distribution restricted to the kept tokens is rejected
    assert stats.chisquare(counts[keep], q64[keep] / q64[keep].sum() * N).pvalue < 1e-6


def test_bad_filter_arguments():
    parent, logits, dq, tokens, u = _batch(4, B=2)
    for top_k, top_p in ((0, 1.0), (-3, 1.0), (5, 0.0), (5, 1.5)):
        with pytest.raises(ValueError):
            oracle.accept_filtered(logits, dq, tokens, parent, 1.0, top_k, top_p, u)
