"""Pins for the oracle's compaction (Section 3.2, last paragraph: accepted tokens' K/V and features are kept).

The definition is a gather, so the expected result is numpy fancy indexing on a copy of the cache.
"""
import numpy as np

import oracle
from paper_2506_14158_b200 import workloads as W


def _caches(rng, n_layers, B, Hkv, C, d, dtype):
    mk = lambda: rng.integers(0, 60000, size=(B, Hkv, C, d)).astype(dtype)
    return [mk() for _ in range(n_layers)], [mk() for _ in range(n_layers)]


def _random_path(rng, parent, max_depth):
    depth = W.tree_depths(parent)
    e = int(rng.integers(len(parent)))
    path = np.full(max_depth + 1, -1, dtype=np.int32)
    t = e
    while t >= 0:
        path[depth[t]] = t
        t = parent[t]
    return path, int(depth[e])


def test_compaction_is_a_gather_of_the_accepted_path():
    rng = np.random.default_rng(0)
    n_layers, B, Hkv, T, d, hid, max_depth = 3, 4, 2, 12, 8, 20, 5
    Ls = np.array([0, 5, 17, 9], dtype=np.int32)
    C = int(Ls.max()) + T + 2
    for dtype in (np.uint16, np.float32):
        kc, vc = _caches(rng, n_layers, B, Hkv, C, d, dtype)
        k0, v0 = [c.copy() for c in kc], [c.copy() for c in vc]
        feat = rng.integers(0, 60000, size=(B, T, hid)).astype(dtype)
        feat_out = np.full((B, max_depth + 1, hid), 77, dtype=dtype)
        paths, alens = [], []
        for b in range(B):
            p, a = _random_path(rng, W.random_tree(T, max_depth, rng), max_depth)
            paths.append(p)
            alens.append(a)
        paths, alens = np.stack(paths), np.array(alens, dtype=np.int32)
        alens[1] = -1  # a sequence that failed validation upstream is skipped
        cl = Ls.copy()
        st = oracle.kv_compact(kc, vc, cl, paths, alens, T, feat, feat_out)
        assert (st == 0).all()
        for b in range(B):
            a, L = alens[b], Ls[b]
            if a < 0:
                assert cl[b] == L
                for l in range(n_layers):
                    np.testing.assert_array_equal(kc[l][b], k0[l][b])
                assert (feat_out[b] == 77).all()
                continue
            assert cl[b] == L + a + 1
            src = L + paths[b, : a + 1]
            for l in range(n_layers):
                for new, old in ((kc[l], k0[l]), (vc[l], v0[l])):
                    np.testing.assert_array_equal(new[b, :, L:L + a + 1], old[b][:, src])  # gathered rows
                    np.testing.assert_array_equal(new[b, :, :L], old[b, :, :L])            # prefix untouched
                    np.testing.assert_array_equal(new[b, :, L + T:], old[b, :, L + T:])    # beyond the tree untouched
            np.testing.assert_array_equal(feat_out[b, : a + 1], feat[b, paths[b, : a + 1]])
            assert (feat_out[b, a + 1:] == 77).all()


def test_identity_path_is_a_no_op_and_bad_paths_are_flagged():
    rng = np.random.default_rng(1)
    B, Hkv, T, d = 2, 1, 6, 4
    C = 3 + T
    kc, vc = _caches(rng, 1, B, Hkv, C, d, np.uint16)
    k0 = kc[0].copy()
    path = np.array([[0, 1, 2, 3, -1, -1], [0, 3, 2, -1, -1, -1]], dtype=np.int32)  # second: not increasing
    cl = np.array([3, 3], dtype=np.int32)
    st = oracle.kv_compact(kc, vc, cl, path, np.array([3, 2], dtype=np.int32), T)
    assert st[0] == 0 and st[1] & oracle.SEQ_BAD_PATH
    np.testing.assert_array_equal(kc[0], k0)
    assert list(cl) == [7, 3]
    cl = np.array([4, 3], dtype=np.int32)  # L + T > C
    st = oracle.kv_compact(kc, vc, cl, path, np.array([3, -1], dtype=np.int32), T)
    assert st[0] & oracle.SEQ_CAPACITY and list(cl) == [4, 3]
