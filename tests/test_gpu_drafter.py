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

    e = oracle.embed_gather(_f64(w.embedding), tokens.reshape(-1))
    np.testing.assert_array_equal(_f64(head.e), e)                                                    # Eq. 6
    _close(_f64(head.h), oracle.linear(_f64(head.e), _f64(w.fc), x2=_f64(feats), bias=_f64(w.fc_bias)), 2 * H)   # Eq. 3
    _close(_f64(head.a), oracle.rmsnorm(_f64(head.h), _f64(w.norm1), head.eps), 1)
    kc, vc = k0.copy(), v0.copy()
    qk = oracle.qkv_rope(_f64(head.a).reshape(B, T, H), _f64(w.qkv), cache_len, parent, Hq, Hkv, d, kc, vc)
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
    assert clear.mean() > 0.8
    np.testing.assert_array_equal(r["token"].cpu().numpy()[clear], top["token"][clear])

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
