"""GPU parity: s4c_lm_head_greedy and s4c_tree_accept_tokens (through the C ABI) against the oracle.

The kernel accumulates bf16 products in float32 in the tensor cores' order, the oracle in float64, so the greedy choice
can differ where two logits of a row are closer than that arithmetic resolves.  What is compared: the chosen token is
the oracle's, or its oracle logit lies within the bound of the row's maximum (then several answers are correct); the
reported maximum equals the oracle logit of the chosen token within the bound.  Bound: float32 accumulation of H products,
|error| <= H * 2^-24 * sum_h |hidden_h * weight_h| is crude; the tests use 4 * sqrt(H) * 2^-24 * ||hidden|| * ||weight_v||_max,
which the random inputs stay far inside.  The walk on choices is integer work: bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_14158_b200 import workloads as W

from parity import Guarded, dev

pytestmark = pytest.mark.gpu


def _bf16(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16)


def _run(hid, wgt):
    from paper_2506_14158_b200 import s4c

    R, H = hid.shape
    V = wgt.shape[0]
    g = dict(token=Guarded((R,), torch.int32, fill=-9), max_logit=Guarded((R,), torch.float32, fill=-9.0),
             status=Guarded((1,), torch.int32, fill=-9),
             workspace=Guarded((max(256, s4c.lm_head_greedy_workspace_bytes(R, V, H)),), torch.uint8, fill=0xCD))
    s4c.lm_head_greedy(hid.cuda(), wgt.cuda(), token=g["token"].t, max_logit=g["max_logit"].t, status=g["status"].t,
                       workspace=g["workspace"].t)
    torch.cuda.synchronize()
    for name, buf in g.items():
        buf.check("s4c_lm_head_greedy " + name)
    assert int(g["status"].t.item()) == 0
    return g["token"].t.cpu().numpy(), g["max_logit"].t.cpu().numpy()


def _check(hid, wgt, tok, mx, sample=None):
    """hid, wgt: bf16 torch tensors (the values both sides see).  sample: token ids to compare against (None = all)."""
    h = hid.float().numpy().astype(np.float64)
    R, H = h.shape
    rows = lambda idx: wgt[torch.from_numpy(np.asarray(idx, dtype=np.int64))].float().numpy().astype(np.float64)
    wmax = float(wgt.float().norm(dim=1).max())
    bound = 4.0 * np.sqrt(H) * 2.0 ** -24 * np.linalg.norm(h, axis=1) * wmax + 1e-30
    chosen = np.einsum("rh,rh->r", h, rows(tok))                # the oracle's logit of the token the kernel chose
    np.testing.assert_array_less(np.abs(mx - chosen), bound)
    cols = np.arange(wgt.shape[0]) if sample is None else sample
    ref = oracle.lm_head_greedy(h, rows(cols))
    assert (chosen >= ref["max_logit"] - bound).all()            # nothing (sampled) beats the choice by more than the bound
    if sample is None:
        same = tok == ref["token"]
        assert same.mean() > 0.95
        # where the oracle's runner-up is further away than the bound the choice is unique and must match
        srt = np.sort(ref["logits"], axis=1)
        unique = srt[:, -1] - srt[:, -2] > 2 * bound if srt.shape[1] > 1 else np.ones(len(srt), dtype=bool)
        np.testing.assert_array_equal(tok[unique], ref["token"][unique])


@pytest.mark.parametrize("R,V,H", [(1, 128, 64), (26, 1000, 128), (128, 4099, 256), (129, 640, 192), (200, 3001, 512),
                                   (256, 32000, 448), (300, 777, 64), (515, 2048, 128), (3, 1, 64), (5, 33, 64), (2, 40001, 8192),
                                   (64, 9999, 1024), (97, 257, 320)])
def test_shapes_against_the_oracle(R, V, H):
    rng = np.random.default_rng(R * 7 + V)
    hid, wgt = _bf16(rng.standard_normal((R, H))), _bf16(rng.standard_normal((V, H)) * 0.5)
    tok, mx = _run(hid, wgt)
    _check(hid, wgt, tok, mx)


def test_planted_winners_at_tile_and_vocabulary_edges():
    # the maximum sits at chosen places: first and last token, both sides of a 128-token tile boundary, the ragged tail
    rng = np.random.default_rng(3)
    R, V, H = 140, 128 * 5 + 37, 128
    places = [0, V - 1, 127, 128, 255, 256, 128 * 5, 128 * 5 + 36]
    want = np.array([places[r % len(places)] for r in range(R)])
    # one-hot states: row r looks only at hidden unit r % H; the head's column r % H peaks at a chosen token
    hid = torch.zeros(R, H)
    for r in range(R):
        hid[r, r % H] = 3.0
    wgt = torch.from_numpy(rng.standard_normal((V, H)).astype(np.float32) * 0.05)
    used = {}
    for r in range(R):
        used.setdefault(r % H, want[r])
    for col, v in used.items():
        wgt[v, col] = 4.0
    hid, wgt = hid.to(torch.bfloat16), wgt.to(torch.bfloat16)
    tok, mx = _run(hid, wgt)
    np.testing.assert_array_equal(tok, [used[r % H] for r in range(R)])
    np.testing.assert_allclose(mx, 12.0, rtol=1e-6)


def test_equal_logits_go_to_the_lower_token_across_tiles_and_ctas():
    rng = np.random.default_rng(4)
    R, V, H = 64, 128 * 300, 64          # 300 tiles: more tiles than CTAs, so ties cross CTAs as well as tiles
    hid = _bf16(rng.integers(-2, 3, (R, H)))
    base = rng.integers(-2, 3, (50, H)).astype(np.float32)
    wgt = _bf16(base[rng.integers(0, 50, V)])      # 50 distinct rows repeated all over the vocabulary: exact integer logits
    tok, mx = _run(hid, wgt)
    ref = oracle.lm_head_greedy(hid.float().numpy(), wgt.float().numpy())
    np.testing.assert_array_equal(tok, ref["token"])          # integer arithmetic: exact on both sides, first maximum
    np.testing.assert_array_equal(mx, ref["max_logit"])


def test_full_size_head_on_sampled_tokens():
    # the 8B-shaped head (256 rows, V = 128256, H = 4096) in the launch the benchmark times; the oracle checks the chosen
    # token's logit and 3000 sampled tokens per row (plus the neighbours of the choice)
    g = torch.Generator().manual_seed(9)
    R, V, H = 256, 128256, 4096
    hid = torch.randn(R, H, generator=g).to(torch.bfloat16)
    wgt = (torch.randn(V, H, generator=g) * 0.02).to(torch.bfloat16)
    tok, mx = _run(hid, wgt)
    assert (tok >= 0).all() and (tok < V).all()
    rng = np.random.default_rng(10)
    sample = np.unique(np.concatenate([rng.integers(0, V, 3000), tok, np.clip(tok + 1, 0, V - 1), np.clip(tok - 1, 0, V - 1),
                                       [0, V - 1, 128255, 127, 128]]))
    _check(hid, wgt, tok, mx, sample=sample)


def _planted(seed, B=40, T=14, V=30):
    rng = np.random.default_rng(seed)
    parent = np.stack([W.random_tree(T, 5, rng, 1, 3) for _ in range(B)])
    target = rng.integers(0, V, (B, T)).astype(np.int32)
    tokens = rng.integers(0, V, (B, T)).astype(np.int32)
    for b in range(B):
        for n in range(T):
            kids = W.children_of(parent[b], n)
            if kids and rng.random() < 0.7:
                tokens[b, kids[rng.integers(len(kids))]] = target[b, n]
                if len(kids) > 1 and rng.random() < 0.3:
                    tokens[b, kids[-1]] = target[b, n]
    return parent, target, tokens


def test_walk_on_choices_bit_exact_with_flags_and_padding():
    from paper_2506_14158_b200 import s4c

    parent, target, tokens = _planted(21, B=48, T=20, V=40)
    n_nodes = np.full(48, 20, dtype=np.int32)
    n_nodes[1], n_nodes[2] = 9, 1
    parent[3, 4] = 7          # malformed
    tokens[5, 6] = 40         # outside the vocabulary
    for md in (19, 2):
        ref = oracle.accept_greedy_tokens(target, tokens, parent, n_nodes, md, V=40)
        B = 48
        g = dict(accept_len=Guarded((B,), torch.int32, fill=-9), path=Guarded((B, md + 1), torch.int32, fill=-9),
                 next_token=Guarded((B,), torch.int32, fill=-9), status=Guarded((B,), torch.int32, fill=-9))
        s4c.tree_accept_tokens(dev(target), dev(tokens), dev(parent.astype(np.int32)), 40, dev(n_nodes), md,
                               accept_len=g["accept_len"].t, path=g["path"].t, next_token=g["next_token"].t, status=g["status"].t)
        torch.cuda.synchronize()
        for name, buf in g.items():
            buf.check("s4c_tree_accept_tokens " + name)
            np.testing.assert_array_equal(buf.t.cpu().numpy(), ref[name], err_msg=name)
    assert ref["status"][3] == oracle.SEQ_BAD_PARENT and ref["status"][5] & oracle.SEQ_TOKEN_RANGE
    assert (ref["status"] & oracle.SEQ_DEPTH).any()


def test_head_then_walk_equals_greedy_acceptance_on_materialised_logits():
    # the fused route (hidden states -> choices -> walk) against the library's own logits route on the same model
    from paper_2506_14158_b200 import s4c

    rng = np.random.default_rng(35)   # (a seed whose rows have no two logits closer than 0.03)
    B, T, V, H = 6, 26, 2000, 256
    parent = np.stack([W.random_tree(T, 5, rng, 1, 4) for _ in range(B)])
    hid, wgt = _bf16(rng.standard_normal((B * T, H))), _bf16(rng.standard_normal((V, H)) * 0.3)
    ref = oracle.lm_head_greedy(hid.float().numpy(), wgt.float().numpy())
    choice = ref["token"].reshape(B, T)
    tokens = rng.integers(0, V, (B, T)).astype(np.int32)
    for b in range(B):
        for n in range(T):
            kids = W.children_of(parent[b], n)
            if kids and rng.random() < 0.8:
                tokens[b, kids[0]] = choice[b, n]
    head = s4c.lm_head_greedy(hid.cuda(), wgt.cuda())
    got = s4c.tree_accept_tokens(head["token"].view(B, T), dev(tokens), dev(parent.astype(np.int32)), V, max_depth=5)
    torch.cuda.synchronize()
    want = oracle.accept_greedy(ref["logits"].reshape(B, T, V).astype(np.float32), tokens, parent, max_depth=5)
    srt = np.sort(ref["logits"], axis=1)
    assert (srt[:, -1] - srt[:, -2] > 1e-3).all()     # no row of this seed has a near tie: the choices are unique
    for key in ("accept_len", "path", "next_token", "status"):
        np.testing.assert_array_equal(got[key].cpu().numpy(), want[key], err_msg=key)
    assert want["accept_len"].max() >= 2


# ----------------------------------------------------------------------------- the k best per row; the tree from them
def _run_topk(hid, wgt, k):
    from paper_2506_14158_b200 import s4c

    R, H = hid.shape
    V = wgt.shape[0]
    g = dict(token=Guarded((R, k), torch.int32, fill=-9), logit=Guarded((R, k), torch.float32, fill=-9.0),
             status=Guarded((1,), torch.int32, fill=-9),
             workspace=Guarded((max(256, s4c.lm_head_topk_workspace_bytes(R, V, H, k)),), torch.uint8, fill=0xCD))
    s4c.lm_head_topk(hid.cuda(), wgt.cuda(), k, token=g["token"].t, logit=g["logit"].t, status=g["status"].t,
                     workspace=g["workspace"].t)
    torch.cuda.synchronize()
    for name, buf in g.items():
        buf.check("s4c_lm_head_topk " + name)
    assert int(g["status"].t.item()) == 0
    return g["token"].t.cpu().numpy(), g["logit"].t.cpu().numpy()


@pytest.mark.parametrize("R,V,H,k", [(26, 1000, 128, 4), (130, 4099, 256, 8), (7, 333, 64, 3), (256, 32000, 192, 2),
                                     (300, 777, 64, 5), (3, 6, 64, 8)])
def test_topk_against_the_oracle(R, V, H, k):
    rng = np.random.default_rng(R + V + k)
    hid, wgt = _bf16(rng.standard_normal((R, H))), _bf16(rng.standard_normal((V, H)) * 0.5)
    tok, lg = _run_topk(hid, wgt, k)
    ref = oracle.lm_head_topk(hid.float().numpy(), wgt.float().numpy(), k)
    h, w = hid.float().numpy().astype(np.float64), wgt.float().numpy().astype(np.float64)
    bound = 4.0 * np.sqrt(H) * 2.0 ** -24 * np.linalg.norm(h, axis=1) * np.linalg.norm(w, axis=1).max() + 1e-30
    kk = min(k, V)
    assert (tok[:, kk:] == -1).all() and np.isneginf(lg[:, kk:]).all()
    srt = -np.sort(-ref["logits"], axis=1)[:, : kk + 1]
    for r in range(R):
        assert len(set(tok[r, :kk])) == kk                                        # distinct tokens
        mine = ref["logits"][r, tok[r, :kk]]                                      # their oracle logits
        assert (np.abs(lg[r, :kk] - mine) <= bound[r]).all()                      # reported logits are theirs
        assert (np.abs(mine - ref["logit"][r, :kk]) <= bound[r]).all()            # rank j holds a token as good as the oracle's
        gaps = -np.diff(srt[r])                                                   # where neighbours are clearly apart ...
        clear = np.ones(kk, dtype=bool)
        clear[: len(gaps)] &= gaps[:kk] > 2 * bound[r]
        clear[1:] &= gaps[: kk - 1] > 2 * bound[r]
        np.testing.assert_array_equal(tok[r, :kk][clear], ref["token"][r, :kk][clear])   # ... the token is unique: equal


def test_topk_ties_follow_the_token_order_across_tiles_and_ctas():
    rng = np.random.default_rng(41)
    R, V, H, k = 40, 128 * 200, 64, 8
    hid = _bf16(rng.integers(-2, 3, (R, H)))
    base = rng.integers(-2, 3, (30, H)).astype(np.float32)
    wgt = _bf16(base[rng.integers(0, 30, V)])          # 30 distinct rows all over the vocabulary: exact integer logits, many ties
    tok, lg = _run_topk(hid, wgt, k)
    ref = oracle.lm_head_topk(hid.float().numpy(), wgt.float().numpy(), k)
    np.testing.assert_array_equal(tok, ref["token"])
    np.testing.assert_array_equal(lg, ref["logit"])


def test_drafting_round_without_a_vocabulary_sized_array():
    # drafter states -> ranked choices -> tree, against the oracle's head and its tree from ranked choices; then the
    # tree from ranked choices equals the library's own tree from the distributions those choices rank
    from paper_2506_14158_b200 import s4c

    rng = np.random.default_rng(46)   # (a seed without a near tie among the first k + 1 logits of any row)
    cfg = W.CONFIGS["c2"]
    B, T, V, H = 3, cfg.T, 5000, 256
    hid, wgt = _bf16(rng.standard_normal((B * T, H))), _bf16(rng.standard_normal((V, H)) * 0.3)
    k = max(cfg.branching)
    top = s4c.lm_head_topk(hid.cuda(), wgt.cuda(), k)
    root = rng.integers(0, V, B).astype(np.int32)
    cl = np.array([5, 0, 77], dtype=np.int32)
    tree = s4c.tree_build_topk(top["token"].view(B, T, k), cfg.branching, dev(root), dev(cl))
    torch.cuda.synchronize()
    ref_top = oracle.lm_head_topk(hid.float().numpy(), wgt.float().numpy(), k)
    srt = -np.sort(-ref_top["logits"], axis=1)[:, : k + 1]
    assert (-np.diff(srt, axis=1) > 1e-3).all()      # this seed has no near tie among the first k + 1: the choices are unique
    want = oracle.build_tree_from_topk(ref_top["token"].reshape(B, T, k), cfg.branching, root, T, cl)
    for key in ("tokens", "parent", "position", "n_nodes"):
        np.testing.assert_array_equal(tree[key].cpu().numpy(), want[key], err_msg=key)
    probs = torch.softmax(torch.from_numpy(ref_top["logits"]).float(), dim=1).view(B, T, V).contiguous()
    lib = s4c.tree_build(probs.cuda(), cfg.branching, dev(root), dev(cl))
    torch.cuda.synchronize()
    for key in ("tokens", "parent", "position", "n_nodes"):
        np.testing.assert_array_equal(tree[key].cpu().numpy(), lib[key].cpu().numpy(), err_msg=key)


@pytest.mark.parametrize("R,V,H", [(26, 32000, 512), (256, 5000, 256), (7, 8, 64), (130, 1000, 1024), (26, 32008, 128)])
def test_logits_written_out_for_stochastic_verification(R, V, H):
    # s4c_lm_head_logits: the float32 sums themselves, [R, V], against the oracle's float64 logits within the accumulation bound
    from paper_2506_14158_b200 import s4c
    from parity import Guarded

    rng = np.random.default_rng(R + V)
    hid = torch.from_numpy(rng.standard_normal((R, H)).astype(np.float32)).to(torch.bfloat16)
    wgt = torch.from_numpy((rng.standard_normal((V, H)) / np.sqrt(H)).astype(np.float32)).to(torch.bfloat16)
    out = Guarded((R, V), torch.float32, fill=-3.0)
    st = torch.full((1,), -9, dtype=torch.int32, device="cuda")
    s4c.lm_head_logits(hid.cuda(), wgt.cuda(), out.t, st)
    torch.cuda.synchronize()
    out.check("s4c_lm_head_logits logits")
    assert int(st.item()) == 0
    want = oracle.lm_head_greedy(hid.double().numpy(), wgt.double().numpy())["logits"]
    slack = 4.0 * np.sqrt(H) * 2.0 ** -24 * np.linalg.norm(hid.double().numpy(), axis=1, keepdims=True) * np.linalg.norm(wgt.double().numpy(), axis=1).max()
    assert (np.abs(out.t.double().cpu().numpy() - want) <= slack + 1e-7).all()
