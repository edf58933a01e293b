"""Pins for the oracle's q/k/v projection + rotary embedding + cache write (the verify layer's input side).

Expected values come from plain Python loops on integer-valued inputs, from what a rotation must do (identity at position
0, norms kept, scores that depend on the position difference only, composition of rotations) and from where the tree puts
a node (position = committed length + depth, slot = committed length + node index)."""
import math

import numpy as np
import pytest

import oracle
from paper_2506_14158_b200 import workloads as W


def test_rotation_by_plain_loops_and_at_position_zero():
    rng = np.random.default_rng(1)
    d, theta = 8, 100.0
    x = rng.standard_normal((5, d))
    pos = np.array([0, 1, 2, 7, 1000])
    got = oracle.rope_rotate(x, pos, theta)
    for r in range(5):
        for i in range(d // 2):
            a = pos[r] * theta ** (-2.0 * i / d)
            assert got[r, i] == pytest.approx(x[r, i] * math.cos(a) - x[r, i + d // 2] * math.sin(a), abs=1e-12)
            assert got[r, i + d // 2] == pytest.approx(x[r, i + d // 2] * math.cos(a) + x[r, i] * math.sin(a), abs=1e-12)
    np.testing.assert_array_equal(got[0], x[0])                     # position 0: nothing moves


def test_rotation_keeps_norms_composes_and_makes_scores_relative():
    rng = np.random.default_rng(2)
    d = 64
    qv, kv = rng.standard_normal(d), rng.standard_normal(d)
    np.testing.assert_allclose(np.linalg.norm(oracle.rope_rotate(qv, 37)), np.linalg.norm(qv), rtol=1e-13)
    np.testing.assert_allclose(oracle.rope_rotate(oracle.rope_rotate(qv, 5), 9), oracle.rope_rotate(qv, 14), atol=1e-12)
    s = [float(oracle.rope_rotate(qv, m) @ oracle.rope_rotate(kv, n)) for m, n in ((9, 4), (105, 100), (5, 0))]
    np.testing.assert_allclose(s, s[0], rtol=0, atol=1e-11)          # only m - n matters
    assert abs(float(oracle.rope_rotate(qv, 9) @ oracle.rope_rotate(kv, 5)) - s[0]) > 1e-3   # and it does matter


def _case(seed, B=3, T=7, H=6, Hq=4, Hkv=2, d=4, C=20, integer=True):
    rng = np.random.default_rng(seed)
    parent = np.stack([W.random_tree(T, 4, rng, 1, 3) for _ in range(B)])
    draw = (lambda s: rng.integers(-3, 4, s).astype(np.float64)) if integer else (lambda s: rng.standard_normal(s))
    x, w = draw((B, T, H)), draw(((Hq + 2 * Hkv) * d, H))
    cache_len = rng.integers(0, C - T + 1, B).astype(np.int32)
    return parent, x, w, cache_len


def test_projection_by_plain_loops_positions_and_slots():
    B, T, H, Hq, Hkv, d, C = 3, 7, 6, 4, 2, 4, 20
    parent, x, w, cache_len = _case(3)
    kc, vc = np.full((B, Hkv, C, d), 7.5), np.full((B, Hkv, C, d), -7.5)
    r = oracle.qkv_rope(x, w, cache_len, parent, Hq, Hkv, d, kc, vc, theta=50.0)
    assert (r["status"] == 0).all()
    for b in range(B):
        L = int(cache_len[b])
        depth = [0] * T
        for i in range(1, T):
            depth[i] = depth[parent[b, i]] + 1
        for t in range(T):
            proj = [sum(int(x[b, t, h]) * int(w[o, h]) for h in range(H)) for o in range((Hq + 2 * Hkv) * d)]  # exact integers
            for hq in range(Hq):
                want = oracle.rope_rotate(np.array(proj[hq * d:(hq + 1) * d], dtype=np.float64), L + depth[t], 50.0)
                np.testing.assert_allclose(r["q"][b, hq, t], want, atol=1e-12)
            for hk in range(Hkv):
                kw = oracle.rope_rotate(np.array(proj[(Hq + hk) * d:(Hq + hk + 1) * d], dtype=np.float64), L + depth[t], 50.0)
                np.testing.assert_allclose(kc[b, hk, L + t], kw, atol=1e-12)                 # slot: node index; position: depth
                np.testing.assert_array_equal(vc[b, hk, L + t], proj[(Hq + Hkv + hk) * d:(Hq + Hkv + hk + 1) * d])  # v is not rotated
        untouched = np.ones(C, dtype=bool)
        untouched[L:L + T] = False
        assert (kc[b][:, untouched] == 7.5).all() and (vc[b][:, untouched] == -7.5).all()


def test_chain_and_star_trees_place_positions_as_the_depth_says():
    B, T, H, Hq, Hkv, d, C = 2, 5, 8, 2, 1, 8, 16
    rng = np.random.default_rng(4)
    x = np.tile(rng.standard_normal((1, 1, H)), (B, T, 1))           # every node carries the same state
    w = rng.standard_normal(((Hq + 2 * Hkv) * d, H))
    parent = np.array([[-1, 0, 1, 2, 3], [-1, 0, 0, 0, 0]], dtype=np.int32)   # a chain and a star
    kc, vc = np.zeros((B, Hkv, C, d)), np.zeros((B, Hkv, C, d))
    r = oracle.qkv_rope(x, w, np.array([3, 3], dtype=np.int32), parent, Hq, Hkv, d, kc, vc)
    base = (x[0, 0] @ w.T)[Hq * d:(Hq + 1) * d]                       # the unrotated key of any node
    for t in range(T):
        np.testing.assert_allclose(kc[0, 0, 3 + t], oracle.rope_rotate(base, 3 + t), atol=1e-12)          # chain: position 3 + t
        np.testing.assert_allclose(kc[1, 0, 3 + t], oracle.rope_rotate(base, 3 + min(t, 1)), atol=1e-12)  # star: leaves share position 4
    np.testing.assert_allclose(r["q"][1, :, 1], r["q"][1, :, 4], atol=0)


def test_padding_and_flags():
    B, T, H, Hq, Hkv, d, C = 4, 7, 6, 4, 2, 4, 20
    parent, x, w, cache_len = _case(5, B=B, integer=False)
    cache_len[:] = [2, 14, 5, 0]                                      # sequence 1: 14 + 7 > 20
    parent[2, 3] = 5                                                  # sequence 2: malformed
    n_nodes = np.array([4, 7, 7, 7], dtype=np.int32)
    kc, vc = np.full((B, Hkv, C, d), 1.5), np.full((B, Hkv, C, d), 2.5)
    r = oracle.qkv_rope(x, w, cache_len, parent, Hq, Hkv, d, kc, vc, n_nodes)
    assert r["status"].tolist() == [0, oracle.SEQ_CAPACITY, oracle.SEQ_BAD_PARENT, 0]
    assert (kc[1] == 1.5).all() and (kc[2] == 1.5).all() and (r["q"][1] == 0).all() and (r["q"][2] == 0).all()
    assert (kc[0][:, 2 + 4:] == 1.5).all() and (r["q"][0][:, 4:] == 0).all() and (kc[0][:, 2:6] != 1.5).any()
    full = oracle.qkv_rope(x[3:], w, cache_len[3:], parent[3:], Hq, Hkv, d, np.zeros((1, Hkv, C, d)), np.zeros((1, Hkv, C, d)))
    np.testing.assert_array_equal(full["q"][0], r["q"][3])            # sequences are independent


def test_position_base_moves_the_rotation_and_nothing_else():
    # a root position that is not the cache length: values are rotated for position_base + depth (checked against plain
    # math.cos / math.sin on one element and against rope_rotate of the unrotated projection), slots stay cache_len + node,
    # v is untouched by the base, the cache length itself as base changes nothing, a negative base flags the sequence
    rng = np.random.default_rng(31)
    B, T, H, Hq, Hkv, d, C = 3, 6, 16, 2, 1, 8, 20
    x = rng.standard_normal((B, T, H))
    w = rng.standard_normal(((Hq + 2 * Hkv) * d, H))
    parent = np.array([[-1, 0, 0, 1, 1, 3]] * B, dtype=np.int32)
    depth = np.array([0, 1, 1, 2, 2, 3])
    cache_len = np.array([4, 0, 9], dtype=np.int32)
    base = np.array([11, 0, 100], dtype=np.int32)
    k0, v0 = rng.standard_normal((B, Hkv, C, d)), rng.standard_normal((B, Hkv, C, d))
    ka, va, kb, vb = k0.copy(), v0.copy(), k0.copy(), v0.copy()
    plain = oracle.qkv_rope(x, w, cache_len, parent, Hq, Hkv, d, ka, va)
    moved = oracle.qkv_rope(x, w, cache_len, parent, Hq, Hkv, d, kb, vb, position_base=base)
    assert (moved["status"] == 0).all()
    np.testing.assert_array_equal(va, vb)                                        # v does not know positions
    np.testing.assert_array_equal(moved["q"][1], plain["q"][1])                  # base == cache length (0): the same
    same = oracle.qkv_rope(x, w, cache_len, parent, Hq, Hkv, d, k0.copy(), v0.copy(), position_base=cache_len)
    np.testing.assert_array_equal(same["q"], plain["q"])
    theta = 10000.0
    for b in (0, 2):
        proj = x[b] @ w.T
        qh = proj[:, : Hq * d].reshape(T, Hq, d)
        kh = proj[:, Hq * d: (Hq + Hkv) * d].reshape(T, Hkv, d)
        pos = (base[b] + depth)[:, None]
        np.testing.assert_allclose(moved["q"][b], oracle.rope_rotate(qh, pos, theta).transpose(1, 0, 2), atol=1e-12)
        L = cache_len[b]
        np.testing.assert_allclose(kb[b, :, L:L + T], oracle.rope_rotate(kh, pos, theta).transpose(1, 0, 2), atol=1e-12)   # slots: L + node
        np.testing.assert_array_equal(kb[b, :, :L], k0[b, :, :L])
        np.testing.assert_array_equal(kb[b, :, L + T:], k0[b, :, L + T:])
        t, h, i = 5, 1, 2                                                        # one element by hand: node 5, depth 3
        a = (base[b] + 3) * theta ** (-2.0 * i / d)
        want = qh[t, h, i] * math.cos(a) - qh[t, h, i + d // 2] * math.sin(a)
        assert moved["q"][b, h, t, i] == pytest.approx(want, abs=1e-12)
        assert not np.allclose(moved["q"][b], plain["q"][b])                     # and it does differ from the default
    bad = oracle.qkv_rope(x, w, cache_len, parent, Hq, Hkv, d, k0.copy(), v0.copy(), position_base=np.array([3, -1, 3]))
    assert bad["status"].tolist() == [0, oracle.SEQ_CAPACITY, 0] and (bad["q"][1] == 0).all()
