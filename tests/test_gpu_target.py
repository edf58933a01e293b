"""GPU: the target's greedy verify pass over the tree (`paper_2506_14158_b200/target.py`: embedding, n decoder layers, LM head
with the greedy choice, walk, compaction of every layer's cache) composed from the entry points -- each stage against the
oracle's stage run on what the previous GPU stage produced, the decision against the oracle's walk, and once as a CUDA graph."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_14158_b200 import workloads as W

from parity import dev

pytestmark = pytest.mark.gpu


def _f64(t):
    return t.double().cpu().numpy()


def _close(got, want, k_dim, extra=0.0):
    slack = 8.0 * np.sqrt(k_dim) * 2.0 ** -24 * 32.0 + 2e-3 + extra
    assert (np.abs(got - want) <= 2.0 ** -8 * np.abs(want) + slack).all(), float(np.abs(got - want).max())


def _setup(n_layers, B, T, V, Hq, Hkv, d, inter, L, C, max_depth, keep, seed):
    from paper_2506_14158_b200 import target

    H = Hq * d
    torch.manual_seed(seed)
    w = target.random_weights(n_layers, V, H, Hq, Hkv, d, inter, "cuda", seed=seed)
    kcs = [torch.randn(B, Hkv, C, d, device="cuda").to(torch.bfloat16) for _ in range(n_layers)]
    vcs = [torch.randn(B, Hkv, C, d, device="cuda").to(torch.bfloat16) for _ in range(n_layers)]
    tv = target.TargetVerify(w, B, T, Hq, Hkv, d, C, kcs, vcs, max_depth, keep=keep)
    rng = np.random.default_rng(seed)
    parent = np.stack([W.random_tree(T, 4, rng, 1, 3) for _ in range(B)]).astype(np.int32)
    tokens = rng.integers(0, V, (B, T)).astype(np.int32)
    cache_len = np.asarray([L - 3 * b for b in range(B)], dtype=np.int32)
    return w, kcs, vcs, tv, parent, tokens, cache_len


def test_verify_pass_stage_by_stage():
    n_layers, B, T, V, Hq, Hkv, d, inter, L, C, md = 2, 2, 12, 3000, 4, 2, 64, 384, 40, 64, 5
    H = Hq * d
    w, kcs, vcs, tv, parent, tokens, cache_len = _setup(n_layers, B, T, V, Hq, Hkv, d, inter, L, C, md, True, 11)
    k0, v0 = [_f64(k) for k in kcs], [_f64(v) for v in vcs]
    cl = dev(cache_len.copy())
    r = tv.forward(dev(tokens), cl, dev(parent), max_cache_len=L, compact=False)
    torch.cuda.synchronize()
    assert int(tv.status_qkv.abs().sum().item()) == 0 and int(tv.status_attn.abs().sum().item()) == 0
    assert int(tv.status_head.item()) == 0 and int(tv.status_accept.abs().sum().item()) == 0

    np.testing.assert_array_equal(_f64(tv.x[0]), oracle.embed_gather(_f64(w.embedding), tokens.reshape(-1)))
    _close(_f64(tv.a[0]), oracle.rmsnorm(_f64(tv.x[0]), _f64(w.layers[0].norm1), tv.eps), 1)
    for l, lw in enumerate(w.layers):
        kc, vc = k0[l].copy(), v0[l].copy()
        qk = oracle.qkv_rope(_f64(tv.a[l]).reshape(B, T, H), _f64(lw.qkv), cache_len, parent, Hq, Hkv, d, kc, vc)
        _close(_f64(tv.q[l]), qk["q"], H)
        _close(_f64(kcs[l]), kc, H)
        _close(_f64(vcs[l]), vc, H)
        att, st = oracle.tree_attention(_f64(tv.q[l]), _f64(kcs[l]), _f64(vcs[l]), cache_len, parent)
        assert (st == 0).all()
        np.testing.assert_allclose(_f64(tv.o_in[l]), att.transpose(0, 2, 1, 3).reshape(B * T, H), atol=2e-2)   # rows [B*T, Hq*d]
        _close(_f64(tv.h[l]), oracle.linear(_f64(tv.o_in[l]), _f64(lw.o), residual=_f64(tv.x[l])), H)
        _close(_f64(tv.m[l]), oracle.rmsnorm(_f64(tv.h[l]), _f64(lw.norm2), tv.eps), 1)
        _close(_f64(tv.act[l]), oracle.linear(_f64(tv.m[l]), _f64(lw.gate_up), gate=True), H, extra=2e-2)
        _close(_f64(tv.x[l + 1]), oracle.linear(_f64(tv.act[l]), _f64(lw.down), residual=_f64(tv.h[l])), inter)
        nxt = w.layers[l + 1].norm1 if l + 1 < n_layers else w.final_norm
        _close(_f64(tv.a[l + 1]), oracle.rmsnorm(_f64(tv.x[l + 1]), _f64(nxt), tv.eps), 1)
    # the target's choice per node (where the oracle's runner-up is clearly behind) and the walk on the choices
    top = oracle.lm_head_greedy(_f64(tv.a[n_layers]), _f64(w.lm_head))
    lg = _f64(tv.a[n_layers]) @ _f64(w.lm_head).T
    srt = -np.sort(-lg, axis=1)
    clear = (srt[:, 0] - srt[:, 1]) > 2e-3
    assert clear.mean() > 0.8
    got_tok = tv.target_token.cpu().numpy()
    np.testing.assert_array_equal(got_tok[clear], top["token"][clear])
    walk = oracle.accept_greedy_tokens(got_tok.reshape(B, T), tokens, parent, max_depth=md)
    np.testing.assert_array_equal(r["accept_len"].cpu().numpy(), walk["accept_len"])
    np.testing.assert_array_equal(r["next_token"].cpu().numpy(), walk["next_token"])
    a = walk["accept_len"]
    for b in range(B):
        np.testing.assert_array_equal(r["path"].cpu().numpy()[b, : a[b] + 1], walk["path"][b, : a[b] + 1])


def test_verify_step_compacts_every_layer_and_replays_as_a_graph():
    # tokens planted so that a path is accepted: the tree's tokens along one root-to-leaf path are the target's own choices
    n_layers, B, T, V, Hq, Hkv, d, inter, L, C, md = 3, 2, 10, 2000, 4, 4, 64, 256, 33, 48, 4
    w, kcs, vcs, tv, parent, tokens, cache_len = _setup(n_layers, B, T, V, Hq, Hkv, d, inter, L, C, md, False, 12)
    k0, v0 = [k.clone() for k in kcs], [v.clone() for v in vcs]
    # pass 1 (no compaction) tells the target's choice per node; give every child of an accepted node that token in turn
    tok = dev(tokens.copy())
    par = dev(parent)
    for _ in range(md):
        cl = dev(cache_len.copy())
        tv.forward(tok, cl, par, max_cache_len=L, compact=False)
        choice = tv.target_token.view(B, T).cpu().numpy()
        t_np = tok.cpu().numpy()
        for b in range(B):
            for i in range(1, T):
                if (parent[b][1:] == parent[b, i]).argmax() + 1 == i:  # the first child of its parent
                    t_np[b, i] = choice[b, parent[b, i]]
        tok = dev(t_np)
        for l in range(n_layers):
            kcs[l].copy_(k0[l]), vcs[l].copy_(v0[l])
    cl = dev(cache_len.copy())
    r = tv.forward(tok, cl, par, max_cache_len=L)
    torch.cuda.synchronize()
    a = r["accept_len"].cpu().numpy()
    assert (a >= 1).all(), a
    path = r["path"].cpu().numpy()
    np.testing.assert_array_equal(cl.cpu().numpy(), cache_len + a + 1)
    assert int(tv.status_compact.abs().sum().item()) == 0
    # every layer's cache: the accepted nodes' rows now sit at the committed slots L_b .. L_b + a; the prefix is untouched
    first = [k.clone() for k in kcs]
    for l in range(n_layers):
        kcs[l].copy_(k0[l]), vcs[l].copy_(v0[l])
    cl2 = dev(cache_len.copy())
    tv.forward(tok, cl2, par, max_cache_len=L, compact=False)  # the same pass, tree slots written, nothing moved
    torch.cuda.synchronize()
    for l in range(n_layers):
        for b in range(B):
            Lb = int(cache_len[b])
            for j in range(a[b] + 1):
                assert torch.equal(first[l][b, :, Lb + j], kcs[l][b, :, Lb + path[b, j]])
            assert torch.equal(first[l][b, :, :Lb], k0[l][b, :, :Lb])
    feats = tv.x[tv.last].view(B, T, -1)
    for b in range(B):
        for j in range(a[b] + 1):
            assert torch.equal(r["features"][b, j], feats[b, path[b, j]])

    # the whole step as one CUDA graph: the same decision
    want = (r["accept_len"].clone(), r["next_token"].clone(), r["path"].clone())
    for l in range(n_layers):
        kcs[l].copy_(k0[l]), vcs[l].copy_(v0[l])
    cl3 = dev(cache_len.copy())
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        tv.forward(tok, cl3, par, max_cache_len=L)
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        tv.forward(tok, cl3, par, max_cache_len=L)
    for l in range(n_layers):
        kcs[l].copy_(k0[l]), vcs[l].copy_(v0[l])
    cl3.copy_(dev(cache_len.copy()))
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(tv.accept_len, want[0]) and torch.equal(tv.next_token, want[1])
    for b in range(B):
        assert torch.equal(tv.path[b, : a[b] + 1], want[2][b, : a[b] + 1])
    np.testing.assert_array_equal(cl3.cpu().numpy(), cache_len + a + 1)


def test_verify_pass_by_speculative_sampling():
    # temperature > 0: the pass writes float32 logits and s4c_tree_accept walks them; the oracle's walk on the GPU's logits
    # must take the same decisions bit for bit, and the logits must be the oracle's LM head within the accumulation bound
    n_layers, B, T, V, Hq, Hkv, d, inter, L, C, md = 2, 3, 10, 2000, 4, 2, 64, 256, 30, 48, 4
    H = Hq * d
    from paper_2506_14158_b200 import target

    torch.manual_seed(21)
    w = target.random_weights(n_layers, V, H, Hq, Hkv, d, inter, "cuda", seed=21)
    kcs = [torch.randn(B, Hkv, C, d, device="cuda").to(torch.bfloat16) for _ in range(n_layers)]
    vcs = [torch.randn(B, Hkv, C, d, device="cuda").to(torch.bfloat16) for _ in range(n_layers)]
    tv = target.TargetVerify(w, B, T, Hq, Hkv, d, C, kcs, vcs, md, stochastic=True)
    rng = np.random.default_rng(22)
    parent = np.stack([W.random_tree(T, md, rng, 1, 3) for _ in range(B)]).astype(np.int32)
    tokens = rng.integers(0, V, (B, T)).astype(np.int32)
    dl = rng.standard_normal((B, T, V)) * 2.0
    dp = np.exp(dl - dl.max(axis=2, keepdims=True))
    draft_probs = (dp / dp.sum(axis=2, keepdims=True)).astype(np.float32)
    for b in range(B):  # children carry the drafter's most probable tokens of their parent's row, best first (Section 3.2)
        for n in range(T):
            kids = [i for i in range(1, T) if parent[b, i] == n]
            order = np.argsort(-draft_probs[b, n], kind="stable")
            for j, c in enumerate(kids):
                tokens[b, c] = order[j]
    uniforms = rng.random((B, T)).astype(np.float32)
    cache_len = np.asarray([L, L - 7, 3], dtype=np.int32)
    cl = dev(cache_len.copy())
    tau = 0.7
    r = tv.forward(dev(tokens), cl, dev(parent), max_cache_len=L, temperature=tau, draft_probs=dev(draft_probs), uniforms=dev(uniforms))
    torch.cuda.synchronize()
    assert int(tv.status_head.item()) == 0 and int(tv.status_accept.abs().sum().item()) == 0
    logits = tv.logits.cpu().numpy()
    want = oracle.lm_head_greedy(_f64(tv.a[tv.last]), _f64(w.lm_head))["logits"].reshape(B, T, V)
    assert np.abs(logits - want).max() <= 4.0 * np.sqrt(H) * 2.0 ** -24 * 64.0
    ref = oracle.accept_stochastic(logits, draft_probs, tokens, parent, float(np.float32(tau)), uniforms, None, md)
    a = ref["accept_len"]
    np.testing.assert_array_equal(r["accept_len"].cpu().numpy(), a)
    np.testing.assert_array_equal(r["next_token"].cpu().numpy(), ref["next_token"])
    for b in range(B):
        np.testing.assert_array_equal(r["path"].cpu().numpy()[b, : a[b] + 1], ref["path"][b, : a[b] + 1])
    np.testing.assert_array_equal(cl.cpu().numpy(), cache_len + a + 1)   # compacted and advanced like the greedy route
