"""GPU: one greedy drafting-and-verification round composed from the library's entry points, with no vocabulary-sized
array of logits or probabilities anywhere:

    drafter states --s4c_lm_head_topk--> ranked choices --s4c_tree_build_topk--> tree
    tree tokens' states --s4c_qkv_rope--> q, cache tree slots --s4c_tree_attention--> attention output
    (output taken as the final hidden state) --s4c_lm_head_greedy--> target choices --s4c_tree_accept_tokens--> path
    --s4c_kv_compact--> committed cache

Every stage is compared with the oracle's stage run on the values the previous GPU stage produced (so rounding does not
pile up across stages), integer stages bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_14158_b200 import workloads as W

from parity import dev

pytestmark = pytest.mark.gpu


def _bf16(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16)


def test_greedy_round_without_vocabulary_sized_arrays():
    from paper_2506_14158_b200 import s4c

    rng = np.random.default_rng(5)
    B, T, V, Hq, Hkv, d, L, C = 3, 26, 6000, 8, 2, 128, 70, 128
    H = Hq * d
    branching = (4, 3, 2, 2, 1)
    k = max(branching)
    w_draft, w_head = _bf16(rng.standard_normal((V, H)) * 0.05), _bf16(rng.standard_normal((V, H)) * 0.05)
    w_qkv = _bf16(rng.standard_normal(((Hq + 2 * Hkv) * d, H)) / np.sqrt(H))
    f_draft = _bf16(rng.standard_normal((B * T, H)))                  # the drafter's state at every tree position
    x_tree = _bf16(rng.standard_normal((B, T, H)))                    # the target layer's input at every tree token
    root = rng.integers(0, V, B).astype(np.int32)
    cache_len = np.full(B, L, dtype=np.int32)
    k_cache = _bf16(rng.standard_normal((B, Hkv, C, d)))
    v_cache = _bf16(rng.standard_normal((B, Hkv, C, d)))

    # ---- drafting: ranked choices, tree
    top = s4c.lm_head_topk(f_draft.cuda(), w_draft.cuda(), k)
    tree = s4c.tree_build_topk(top["token"].view(B, T, k), branching, dev(root), dev(cache_len))
    torch.cuda.synchronize()
    top_ref = oracle.lm_head_topk(f_draft.float().numpy(), w_draft.float().numpy(), k)
    srt = -np.sort(-top_ref["logits"], axis=1)[:, : k + 1]
    clear = (-np.diff(srt, axis=1) > 1e-3).all(axis=1)               # rows whose first k + 1 logits are clearly apart
    np.testing.assert_array_equal(top["token"].cpu().numpy()[clear], top_ref["token"][clear])
    assert clear.mean() > 0.9
    tree_ref = oracle.build_tree_from_topk(top["token"].cpu().numpy().reshape(B, T, k), branching, root, T, cache_len)
    for key in ("tokens", "parent", "position", "n_nodes"):
        np.testing.assert_array_equal(tree[key].cpu().numpy(), tree_ref[key], err_msg=key)
    parent = tree_ref["parent"]

    # ---- verification: q/k/v + rotary embedding into the cache, tree attention
    q_dev = torch.zeros((B, Hq, T, d), dtype=torch.bfloat16, device="cuda")
    k_dev, v_dev = k_cache.cuda(), v_cache.cuda()
    r = s4c.qkv_rope(x_tree.cuda(), w_qkv.cuda(), dev(cache_len), tree["parent"], q_dev, k_dev, v_dev)
    att = s4c.tree_attention(q_dev, k_dev, v_dev, dev(cache_len), tree["parent"], None, max_cache_len=L)
    torch.cuda.synchronize()
    assert int(r["status"].abs().sum().item()) == 0
    kc, vc = k_cache.double().numpy().copy(), v_cache.double().numpy().copy()
    qk_ref = oracle.qkv_rope(x_tree.double().numpy(), w_qkv.double().numpy(), cache_len, parent, Hq, Hkv, d, kc, vc)
    for got_t, want in ((q_dev, qk_ref["q"]), (k_dev, kc), (v_dev, vc)):
        assert (np.abs(got_t.double().cpu().numpy() - want) <= 2.0 ** -8 * np.abs(want) + 1e-3).all()
    att_ref, st = oracle.tree_attention(q_dev.double().cpu().numpy(), k_dev.double().cpu().numpy(), v_dev.double().cpu().numpy(),
                                        cache_len, parent)
    assert (st == 0).all()
    np.testing.assert_allclose(att.double().cpu().numpy(), att_ref, atol=2e-2)

    # ---- the target's choices and the walk (the attention output stands in for the final hidden state)
    hidden = att.permute(0, 2, 1, 3).reshape(B * T, H).contiguous()
    head = s4c.lm_head_greedy(hidden, w_head.cuda())
    walk = s4c.tree_accept_tokens(head["token"].view(B, T), tree["tokens"], tree["parent"], V, max_depth=len(branching))
    torch.cuda.synchronize()
    head_ref = oracle.lm_head_greedy(hidden.float().cpu().numpy(), w_head.float().numpy())
    s2 = np.sort(head_ref["logits"], axis=1)
    clear = s2[:, -1] - s2[:, -2] > 1e-3
    np.testing.assert_array_equal(head["token"].cpu().numpy()[clear], head_ref["token"][clear])
    choice = head["token"].cpu().numpy().reshape(B, T)
    walk_ref = oracle.accept_greedy_tokens(choice, tree_ref["tokens"], parent, None, len(branching), V=V)
    for key in ("accept_len", "path", "next_token", "status"):
        np.testing.assert_array_equal(walk[key].cpu().numpy(), walk_ref[key], err_msg=key)

    # ---- commit: the accepted path's K/V move to the front of the tree slots
    kb, vb = k_dev.double().cpu().numpy(), v_dev.double().cpu().numpy()
    ptrs_k, ptrs_v = s4c.cache_pointer_array([k_dev]), s4c.cache_pointer_array([v_dev])
    cl_dev = dev(cache_len.copy())
    s4c.kv_compact(ptrs_k, ptrs_v, 1, tuple(k_dev.shape), k_dev.dtype, cl_dev, walk["path"], walk["accept_len"], T)
    torch.cuda.synchronize()
    cl_ref = cache_len.copy()
    oracle.kv_compact([kb], [vb], cl_ref, walk_ref["path"], walk_ref["accept_len"], T)
    np.testing.assert_array_equal(cl_dev.cpu().numpy(), cl_ref)
    for b in range(B):
        np.testing.assert_array_equal(k_dev[b, :, : cl_ref[b]].double().cpu().numpy(), kb[b][:, : cl_ref[b]])
        np.testing.assert_array_equal(v_dev[b, :, : cl_ref[b]].double().cpu().numpy(), vb[b][:, : cl_ref[b]])
