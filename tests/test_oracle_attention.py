"""Pins for the oracle's tree-masked attention (Section 3.2 / Figure 3 tree mask).

The paper prints no numeric example, so the oracle is pinned to what the mathematics fixes, each
time against a *library* attention routine (torch's scaled_dot_product_attention in float64 on the
CPU) or a closed form -- never against a retyped copy of its own loops.
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from paper_2506_14158_b200 import workloads as W


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def _sdpa_causal_last_rows(q_rows, k_seq, v_seq, scale):
    """Ordinary causal attention of a linear sequence: q_rows are the last len(q_rows) positions."""
    n_q, n_k = q_rows.shape[0], k_seq.shape[0]
    mask = torch.ones(n_q, n_k, dtype=torch.bool).tril(diagonal=n_k - n_q)
    out = F.scaled_dot_product_attention(
        torch.from_numpy(q_rows)[None], torch.from_numpy(k_seq)[None], torch.from_numpy(v_seq)[None],
        attn_mask=mask[None], scale=scale)
    return out[0].numpy()


def _inputs(B, Hq, Hkv, T, d, L, C, seed):
    q = _rand((B, Hq, T, d), seed)
    k = _rand((B, Hkv, C, d), seed + 1)
    v = _rand((B, Hkv, C, d), seed + 2)
    return q, k, v


def test_chain_tree_is_causal_attention():
    # A chain (each draft token follows the previous one) is plain causal decoding of T more tokens.
    B, H, T, d, L = 2, 3, 9, 16, 21
    C = L + T + 3
    q, k, v = _inputs(B, H, H, T, d, L, C, 10)
    parent = np.tile(W.chain_tree(T), (B, 1))
    out, st = oracle.tree_attention(q, k, v, [L] * B, parent)
    assert (st == 0).all()
    scale = 1.0 / np.sqrt(d)
    for b in range(B):
        for h in range(H):
            ref = _sdpa_causal_last_rows(q[b, h], k[b, h, :L + T], v[b, h, :L + T], scale)
            np.testing.assert_allclose(out[b, h], ref, rtol=0, atol=1e-12)


def test_star_tree_rows_are_independent_prefix_conditioned_heads():
    # Depth-1 star: every leaf sees prefix + root + itself only (Medusa-style independent heads).
    H, T, d, L = 2, 6, 8, 13
    C = L + T
    q, k, v = _inputs(1, H, H, T, d, L, C, 20)
    out, _ = oracle.tree_attention(q, k, v, [L], W.star_tree(T)[None])
    scale = 1.0 / np.sqrt(d)
    for h in range(H):
        for i in range(1, T):
            idx = list(range(L)) + [L, L + i]
            ref = _sdpa_causal_last_rows(q[0, h, i:i + 1], k[0, h, idx], v[0, h, idx], scale)
            np.testing.assert_allclose(out[0, h, i], ref[0], rtol=0, atol=1e-12)
    # changing another leaf's K/V must not move this leaf's output
    k2, v2 = k.copy(), v.copy()
    k2[0, :, L + 2] += 5.0
    v2[0, :, L + 2] -= 3.0
    out2, _ = oracle.tree_attention(q, k2, v2, [L], W.star_tree(T)[None])
    keep = [i for i in range(T) if i != 2]
    np.testing.assert_array_equal(out[0, :, keep], out2[0, :, keep])
    assert np.abs(out[0, :, 2] - out2[0, :, 2]).max() > 1e-3


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_path_equivalence_random_trees(seed):
    # For any tree and node i: output == last row of causal attention over prefix ++ path(root..i).
    rng = np.random.default_rng(100 + seed)
    B, Hq, Hkv, T, d, L = 2, 4, 2, 14, 8, 11 + seed
    C = L + T + 1
    q, k, v = _inputs(B, Hq, Hkv, T, d, L, C, 30 + seed)
    parent = np.stack([W.random_tree(T, 5, rng) for _ in range(B)])
    scale = 0.37
    out, st = oracle.tree_attention(q, k, v, [L] * B, parent, scale=scale)
    assert (st == 0).all()
    G = Hq // Hkv
    for b in range(B):
        for i in range(T):
            path, t = [], i
            while t >= 0:
                path.append(t)
                t = parent[b, t]
            idx = list(range(L)) + [L + t for t in reversed(path)]
            for h in range(Hq):
                ref = _sdpa_causal_last_rows(q[b, h, i:i + 1], k[b, h // G, idx], v[b, h // G, idx], scale)
                np.testing.assert_allclose(out[b, h, i], ref[0], rtol=0, atol=1e-12)


def test_sibling_relabelling_leaves_outputs_unchanged():
    # Swapping two sibling subtrees (with their Q/K/V rows) permutes the outputs and nothing else.
    H, d, L = 2, 8, 5
    parent = np.array([-1, 0, 0, 1, 2, 2], dtype=np.int32)
    perm = np.array([0, 2, 1, 4, 5, 3])  # new index -> old index; children of old 1 <-> old 2
    parent2 = np.array([-1, 0, 0, 1, 1, 2], dtype=np.int32)
    T = 6
    C = L + T
    q, k, v = _inputs(1, H, H, T, d, L, C, 40)
    out, _ = oracle.tree_attention(q, k, v, [L], parent[None])
    q2 = q[:, :, perm]
    k2, v2 = k.copy(), v.copy()
    k2[:, :, L:L + T] = k[:, :, L + perm]
    v2[:, :, L:L + T] = v[:, :, L + perm]
    out2, st = oracle.tree_attention(q2, k2, v2, [L], parent2[None])
    assert (st == 0).all()
    np.testing.assert_allclose(out2, out[:, :, perm], rtol=0, atol=1e-13)


def test_constant_v_gives_that_constant():
    # Softmax weights sum to one: with V rows all equal to c the output is c whatever the scores.
    T, d, L = 7, 4, 9
    q, k, v = _inputs(1, 2, 2, T, d, L, L + T, 50)
    c = np.array([1.5, -2.0, 0.25, 3.0])
    v[...] = c
    out, _ = oracle.tree_attention(q, k, v, [L], W.tree_from_branching((2, 2), T)[None])
    np.testing.assert_allclose(out, np.broadcast_to(c, out.shape), rtol=0, atol=1e-13)


def test_single_node_is_decode_attention_and_empty_prefix():
    d = 8
    q, k, v = _inputs(1, 1, 1, 1, d, 6, 7, 60)
    out, _ = oracle.tree_attention(q, k, v, [6], np.array([[-1]]))
    ref = _sdpa_causal_last_rows(q[0, 0], k[0, 0, :7], v[0, 0, :7], 1 / np.sqrt(d))
    np.testing.assert_allclose(out[0, 0], ref, atol=1e-13)
    # L = 0: the root sees only itself -> its output is its own V row
    q, k, v = _inputs(1, 1, 1, 3, d, 0, 3, 61)
    out, _ = oracle.tree_attention(q, k, v, [0], W.chain_tree(3)[None])
    np.testing.assert_allclose(out[0, 0, 0], v[0, 0, 0], atol=1e-14)


def test_gqa_equals_mha_with_repeated_kv_heads():
    B, Hq, Hkv, T, d, L = 1, 6, 2, 5, 8, 7
    q, k, v = _inputs(B, Hq, Hkv, T, d, L, L + T, 70)
    parent = W.tree_from_branching((2, 1), T)[None]
    out, _ = oracle.tree_attention(q, k, v, [L], parent)
    k_rep = np.repeat(k, Hq // Hkv, axis=1)
    v_rep = np.repeat(v, Hq // Hkv, axis=1)
    out_rep, _ = oracle.tree_attention(q, k_rep, v_rep, [L], parent)
    np.testing.assert_array_equal(out, out_rep)


def test_padding_nodes_and_per_sequence_lengths():
    # n_nodes < T: padding rows are zero, real rows unaffected by the padding slots' contents.
    B, H, T, d = 2, 2, 6, 8
    Ls = [4, 9]
    C = 9 + T
    q, k, v = _inputs(B, H, H, T, d, 0, C, 80)
    parent = np.tile(W.tree_from_branching((2, 2), T), (B, 1))
    n_nodes = np.array([4, 6], dtype=np.int32)
    out, st = oracle.tree_attention(q, k, v, Ls, parent, n_nodes=n_nodes)
    assert (st == 0).all()
    assert (out[0, :, 4:] == 0).all()
    sub, _ = oracle.tree_attention(q[:1, :, :4], k[:1], v[:1], Ls[:1], parent[:1, :4])
    np.testing.assert_array_equal(out[0, :, :4], sub[0])


def test_malformed_tree_and_capacity_are_flagged():
    q, k, v = _inputs(2, 1, 1, 3, 4, 2, 5, 90)
    parent = np.array([[-1, 0, 1], [-1, 2, 0]], dtype=np.int32)  # second: parent[1] = 2 >= 1
    out, st = oracle.tree_attention(q, k, v, [2, 2], parent)
    assert st[0] == 0 and st[1] & oracle.SEQ_BAD_PARENT
    assert np.isnan(out[1]).all()  # untouched
    out, st = oracle.tree_attention(q, k, v, [3, 2], np.tile(W.chain_tree(3), (2, 1)))
    assert st[0] & oracle.SEQ_CAPACITY and st[1] == 0
