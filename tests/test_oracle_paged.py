"""Pins for the paged-cache layout helper of the oracle: a paged cache is the contiguous cache its block table spells
out.  Checked against plain indexing written out slot by slot, against the identity layout, and by the invariance of the
attention result under a permutation of the pool."""
import numpy as np

import oracle
from paper_2506_14158_b200 import workloads as W


def test_gather_matches_slot_by_slot_indexing():
    rng = np.random.default_rng(0)
    n_pages, Hkv, ps, d, B, nb = 11, 2, 4, 3, 3, 3
    pages = rng.standard_normal((n_pages, Hkv, ps, d))
    bt = np.stack([rng.permutation(n_pages)[:nb] for _ in range(B)]).astype(np.int32)
    c = oracle.pages_to_contiguous(pages, bt)
    assert c.shape == (B, Hkv, nb * ps, d)
    for b in range(B):
        for h in range(Hkv):
            for s in range(nb * ps):
                np.testing.assert_array_equal(c[b, h, s], pages[bt[b, s // ps], h, s % ps])


def test_identity_table_is_a_reshape_and_scatter_inverts_gather():
    rng = np.random.default_rng(1)
    B, Hkv, ps, nb, d = 2, 3, 8, 4, 5
    cont = rng.standard_normal((B, Hkv, nb * ps, d))
    pages = np.zeros((B * nb, Hkv, ps, d))
    bt = np.arange(B * nb, dtype=np.int32).reshape(B, nb)
    oracle.scatter_to_pages(pages, bt, cont, [nb] * B)
    np.testing.assert_array_equal(oracle.pages_to_contiguous(pages, bt), cont)
    np.testing.assert_array_equal(pages.reshape(B, nb, Hkv, ps, d).transpose(0, 2, 1, 3, 4).reshape(B, Hkv, nb * ps, d), cont)


def test_attention_does_not_depend_on_where_the_pages_lie():
    rng = np.random.default_rng(2)
    B, Hq, Hkv, T, d, ps, nb = 2, 4, 2, 9, 16, 8, 6
    L = np.array([20, 31], dtype=np.int32)
    q = rng.standard_normal((B, Hq, T, d))
    k, v = rng.standard_normal((B, Hkv, nb * ps, d)), rng.standard_normal((B, Hkv, nb * ps, d))
    parent = np.stack([W.random_tree(T, 4, rng) for _ in range(B)])
    want, _ = oracle.tree_attention(q, k, v, L, parent)
    n_pages = 40
    perm = rng.permutation(n_pages)[: B * nb].reshape(B, nb).astype(np.int32)
    kp, vp = rng.standard_normal((n_pages, Hkv, ps, d)), rng.standard_normal((n_pages, Hkv, ps, d))
    oracle.scatter_to_pages(kp, perm, k, [nb] * B), oracle.scatter_to_pages(vp, perm, v, [nb] * B)
    got, _ = oracle.tree_attention(q, oracle.pages_to_contiguous(kp, perm), oracle.pages_to_contiguous(vp, perm), L, parent)
    np.testing.assert_array_equal(got, want)
