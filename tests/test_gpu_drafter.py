"""GPU: one head of the multi-head drafter (Eq. 3-6) composed from the entry points (`paper_2506_14158_b200/drafter.py`),
stage by stage against the oracle's stage run on what the previous GPU stage produced, and once as a CUDA graph."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_14158_b200 import workloads as W

from parity import dev

pytestmark = pytest.mark.gpu


def _f64(t):
    return t.double().cpu().numpy()


def _close(got, want, k_dim, xnorm=4.0, extra=0.0):
    slack = 8.0 * np.sqrt(k_dim) * 2.0 ** -24 * xnorm * 8.0 + 2e-3 + extra
    assert (np.abs(got - want) <= 2.0 ** -8 * np.abs(want) + slack).all(), float(np.abs(got - want).max())


def _check_head_stages(head, w, tokens, feats, cache_len, parent, k_cache, v_cache, k0, v0, r, position_base=None, min_clear=0.7):
    """Every stage of one head's pass against the oracle's stage on what the previous GPU stage produced."""
    B, T, Hq, Hkv, d, k = head.B, head.T, head.Hq, head.Hkv, head.d, head.k
    H = Hq * d
    inter = w.down.shape[1]
    e = oracle.embed_gather(_f64(w.embedding), tokens.reshape(-1))
    np.testing.assert_array_equal(_f64(head.e), e)                                                    # Eq. 6
    _close(_f64(head.h), oracle.linear(_f64(head.e), _f64(w.fc), x2=_f64(feats), bias=_f64(w.fc_bias)), 2 * H)   # Eq. 3
    _close(_f64(head.a), oracle.rmsnorm(_f64(head.h), _f64(w.norm1), head.eps), 1)
    kc, vc = k0.copy(), v0.copy()
    qk = oracle.qkv_rope(_f64(head.a).reshape(B, T, H), _f64(w.qkv), cache_len, parent, Hq, Hkv, d, kc, vc, position_base=position_base)
    _close(_f64(head.q), qk["q"], H)
    _close(_f64(k_cache), kc, H)
    _close(_f64(v_cache), vc, H)
    att, st = oracle.tree_attention(_f64(head.q), _f64(k_cache), _f64(v_cache), cache_len, parent)
    assert (st == 0).all()
    np.testing.assert_allclose(_f64(head.o_in), att.transpose(0, 2, 1, 3).reshape(B * T, H), atol=2e-2)   # rows [B*T, Hq*d]
    _close(_f64(head.h2), oracle.linear(_f64(head.o_in), _f64(w.o), residual=_f64(head.h)), H)
    _close(_f64(head.m), oracle.rmsnorm(_f64(head.h2), _f64(w.norm2), head.eps), 1)
    _close(_f64(head.act), oracle.linear(_f64(head.m), _f64(w.gate_up), gate=True), H, extra=2e-2)
    _close(_f64(head.f_out), oracle.linear(_f64(head.act), _f64(w.down), residual=_f64(head.h2)), inter)   # Eq. 4
    top = oracle.lm_head_topk(_f64(head.f_out), _f64(w.lm_head), k)                                   # Eq. 5
    srt = -np.sort(-top["logits"], axis=1)[:, : k + 1]
    clear = (-np.diff(srt, axis=1) > 2e-3).all(axis=1)
    got_tok = r["token"].cpu().numpy()
    np.testing.assert_array_equal(got_tok[clear], top["token"][clear])
    # everywhere (near ties included): the token chosen at rank j is, by the oracle's logits, as good as the oracle's j-th
    chosen = np.take_along_axis(top["logits"], got_tok.astype(np.int64), axis=1)
    assert (np.abs(chosen - top["logit"]) <= 4e-3).all()
    assert clear.mean() >= min_clear


def test_drafter_head_stage_by_stage_and_as_a_graph():
    from paper_2506_14158_b200 import drafter

    torch.manual_seed(0)
    B, T, V, Hq, Hkv, d, inter, L, C, k = 2, 12, 3000, 4, 2, 64, 384, 40, 64, 4
    H = Hq * d
    w = drafter.random_weights(V, H, Hq, Hkv, d, inter, "cuda", seed=3)
    head = drafter.DrafterHead(w, B, T, Hq, Hkv, d, C, k)
    rng = np.random.default_rng(4)
    parent = np.stack([W.random_tree(T, 4, rng, 1, 3) for _ in range(B)])
    tokens = rng.integers(0, V, (B, T)).astype(np.int32)
    feats = torch.randn(B * T, H, device="cuda").to(torch.bfloat16)
    cache_len = np.full(B, L, dtype=np.int32)
    k_cache = torch.randn(B, Hkv, C, d, device="cuda").to(torch.bfloat16)
    v_cache = torch.randn(B, Hkv, C, d, device="cuda").to(torch.bfloat16)
    k0, v0 = _f64(k_cache), _f64(v_cache)
    args = (dev(tokens), feats, dev(cache_len), dev(parent.astype(np.int32)), k_cache, v_cache)
    r = head.forward(*args, max_cache_len=L)
    torch.cuda.synchronize()
    assert int(head.status_qkv.abs().sum().item()) == 0 and int(head.status_attn.abs().sum().item()) == 0
    assert int(head.status_head.item()) == 0

    _check_head_stages(head, w, tokens, feats, cache_len, parent, k_cache, v_cache, k0, v0, r)

    # the same pass as one CUDA graph gives the same choices and features
    first = (r["token"].clone(), r["features"].clone())
    k_cache.copy_(torch.from_numpy(k0).to(torch.bfloat16))
    v_cache.copy_(torch.from_numpy(v0).to(torch.bfloat16))
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        head.forward(*args, max_cache_len=L)
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        head.forward(*args, max_cache_len=L)
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(head.token, first[0]) and torch.equal(head.f_out, first[1])


def test_three_heads_fill_the_tree_level_by_level():
    # a drafting round (Section 3.1.1 + 3.2): head j runs over the nodes of depth j as independent rows; every head's pass is
    # checked stage by stage against the oracle, the hand-over of tokens and features between the levels is exact, and the
    # tree equals the oracle's tree from the same ranked choices
    from paper_2506_14158_b200 import drafter, s4c

    torch.manual_seed(5)
    B, T, V, Hq, Hkv, d, inter, C, k = 2, 21, 3000, 4, 2, 64, 384, 40, 3
    branching = [2, 3, 1, 1]
    H = Hq * d
    ws_ = [drafter.random_weights(V, H, Hq, Hkv, d, inter, "cuda", seed=30 + j) for j in range(3)]
    for w in ws_[1:]:
        w.embedding, w.lm_head = ws_[0].embedding, ws_[0].lm_head   # the target's, shared by the heads (Section 3.1.1)
    mh = drafter.MultiHeadDrafter(ws_, B, T, branching, Hq, Hkv, d, C, k)
    assert mh.levels == [(1, 3), (3, 9), (9, 15), (15, 21)] and mh.n_passes == 3
    rng = np.random.default_rng(6)
    root = rng.integers(0, V, B).astype(np.int32)
    f0 = torch.randn(B, H, device="cuda").to(torch.bfloat16)
    cand = np.stack([rng.choice(V, k, replace=False) for _ in range(B)]).astype(np.int32)
    root_pos = np.array([33, 7], dtype=np.int32)
    caches, c0 = [], []
    for j in range(3):
        nj = mh.levels[j][1] - mh.levels[j][0]
        kc = torch.randn(B * nj, Hkv, C, d, device="cuda").to(torch.bfloat16)
        vc = torch.randn(B * nj, Hkv, C, d, device="cuda").to(torch.bfloat16)
        cl = rng.integers(0, C - 1, B * nj).astype(np.int32)
        caches.append((kc, vc, dev(cl)))
        c0.append((_f64(kc), _f64(vc), cl))
    out = mh.draft(dev(root), f0, dev(cand), dev(root_pos), caches)
    torch.cuda.synchronize()
    tokens, parent = out["tokens"].cpu().numpy(), out["parent"].cpu().numpy()
    topk_all = mh.topk_all.cpu().numpy()
    # the tree: the oracle's tree from the same ranked choices (choices of leaves are never read)
    ref = oracle.build_tree_from_topk(topk_all, branching, root, T, cache_len=root_pos)
    for key in ("tokens", "parent", "position", "n_nodes"):
        np.testing.assert_array_equal(out[key].cpu().numpy(), ref[key], err_msg=key)
    np.testing.assert_array_equal(topk_all[:, 0], cand)
    depth = np.zeros(T, dtype=np.int64)
    for i in range(1, T):
        depth[i] = depth[parent[0, i]] + 1
    feats_prev, n_prev, s_prev = _f64(f0), 1, 0
    for j in range(3):
        s, e = mh.levels[j]
        nj = e - s
        head = mh.heads[j]
        assert int(head.status_qkv.abs().sum().item()) == 0 and int(head.status_attn.abs().sum().item()) == 0
        tok_rows = tokens[:, s:e].reshape(-1, 1)
        np.testing.assert_array_equal(mh.tok_rows[j].cpu().numpy(), tok_rows)
        # a row's feature is its parent's output feature (depth 1: the target's f_0, shared)
        want_f = np.stack([feats_prev[b * n_prev + (parent[b, i] - s_prev if j else 0)] for b in range(B) for i in range(s, e)])
        np.testing.assert_array_equal(_f64(mh.feat_in[j]), want_f)
        pos = np.stack([root_pos[b] + depth[i] for b in range(B) for i in range(s, e)]).astype(np.int32)
        np.testing.assert_array_equal(mh.pos_rows[j].cpu().numpy(), pos)
        kc, vc, _ = caches[j]
        r = dict(token=head.token, features=head.f_out)
        _check_head_stages(head, ws_[j], tok_rows, mh.feat_in[j], c0[j][2], np.full((B * nj, 1), -1, dtype=np.int32), kc, vc,
                           c0[j][0], c0[j][1], r, position_base=pos, min_clear=0.0)
        np.testing.assert_array_equal(topk_all[:, s:e], head.token.cpu().numpy().reshape(B, nj, k))
        feats_prev, n_prev, s_prev = _f64(head.f_out), nj, s
