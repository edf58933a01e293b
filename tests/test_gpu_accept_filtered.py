"""GPU parity: s4c_tree_accept_filtered (through the C ABI) against the oracle's filtered speculative sampling -- accepted
length, path and next token bit-exact on the same uniforms; near ties (|p/q - u| < 1e-6) are counted separately."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_14158_b200 import workloads as W

from parity import Guarded, assert_accept_equal, dev

pytestmark = pytest.mark.gpu


def _both(x, parent, tau, top_k, top_p, n_nodes=None, max_depth=None):
    from paper_2506_14158_b200 import s4c

    par = np.ascontiguousarray(parent, dtype=np.int32)
    nn = None if n_nodes is None else np.asarray(n_nodes, dtype=np.int32)
    B, T, V = x["logits"].shape
    max_depth = T - 1 if max_depth is None else max_depth
    i32 = torch.int32
    g = dict(accept_len=Guarded((B,), i32, fill=-9), path=Guarded((B, max_depth + 1), i32, fill=-9),
             next_token=Guarded((B,), i32, fill=-9), near_tie=Guarded((B, T), torch.uint8, fill=7), status=Guarded((B,), i32, fill=-9),
             workspace=Guarded((max(256, s4c.tree_accept_filtered_workspace_bytes(B, T, V, top_k)),), torch.uint8, fill=0xCD))
    r = s4c.tree_accept_filtered(dev(x["logits"]), dev(x["draft_probs"]), dev(x["tokens"]), dev(par), tau, top_k, top_p,
                                 dev(x["uniforms"]), None if nn is None else dev(nn), max_depth=max_depth,
                                 accept_len=g["accept_len"].t, path=g["path"].t, next_token=g["next_token"].t,
                                 near_tie=g["near_tie"].t, status=g["status"].t, workspace=g["workspace"].t)
    torch.cuda.synchronize()
    for name, buf in g.items():
        buf.check("s4c_tree_accept_filtered " + name)
    ref = oracle.accept_filtered(x["logits"], x["draft_probs"], x["tokens"], par, float(np.float32(tau)), top_k,
                                 float(np.float32(top_p)), x["uniforms"], nn, max_depth)
    return {k: v.cpu().numpy() for k, v in r.items()}, ref


def _synthetic(B, T, V, seed, sigma=2.0, tau=1.0, mode="topk", max_tree_depth=6):
    from dataclasses import replace

    cfg = replace(W.CONFIGS["c2"], name="t", config_id=70 + seed, B=B, T=T, V=V, tree="random", logit_sigma=sigma,
                  max_tree_depth=max_tree_depth)
    parent = W.make_trees(cfg)
    return cfg, parent, W.make_accept_inputs(cfg, parent, tau, token_mode=mode)


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4"])
@pytest.mark.parametrize("top_k,top_p", [(50, 0.9), (8, 1.0), (64, 0.5)])
def test_named_configs(name, top_k, top_p):
    cfg = W.CONFIGS[name]
    parent = W.make_trees(cfg)
    tau = [t for t in cfg.temperatures if t > 0][0]
    x = W.make_accept_inputs(cfg, parent, tau, token_mode="topk")
    got, ref = _both(x, parent, tau, top_k, top_p, max_depth=cfg.max_depth)
    assert (ref["status"] == 0).all()
    assert assert_accept_equal(got, ref, True) == 0


@pytest.mark.parametrize("V", [1, 3, 4, 36, 257, 4096, 4099, 33333, 33336])
@pytest.mark.parametrize("top_k,top_p", [(1, 1.0), (5, 0.8), (64, 0.97)])
def test_vocabulary_sizes(V, top_k, top_p):
    T = min(9, max(2, V))
    cfg, parent, x = _synthetic(8, T, V, seed=V % 91, tau=0.9, mode="sampled" if V >= 9 else "topk")
    if V < 4:
        x["tokens"] %= V
    got, ref = _both(x, parent, 0.9, top_k, top_p, max_depth=cfg.max_tree_depth)
    assert assert_accept_equal(got, ref, True) == 0


def test_many_sequences_walk_every_branch_kind():
    cfg, parent, x = _synthetic(256, 24, 2000, seed=7, tau=1.0, mode="sampled")
    got, ref = _both(x, parent, 1.0, 20, 0.9, max_depth=cfg.max_tree_depth)
    assert assert_accept_equal(got, ref, True) == 0
    a = ref["accept_len"]
    assert a.min() == 0 and a.max() >= 2
    later = sum(1 for b in range(256) for j in range(1, a[b] + 1)
                if ref["path"][b, j] != W.children_of(parent[b], ref["path"][b, j - 1])[0])
    assert later > 5  # acceptances at later siblings (after residual updates) occur


def test_top_1_equals_greedy_verification():
    cfg, parent, x = _synthetic(32, 20, 5000, seed=3, tau=1.0, mode="topk")
    got, _ = _both(x, parent, 0.8, 1, 1.0, max_depth=cfg.max_tree_depth)
    greedy = oracle.accept_greedy(x["logits"], x["tokens"], parent, None, cfg.max_tree_depth)
    for key in ("accept_len", "path", "next_token"):
        np.testing.assert_array_equal(got[key], greedy[key], err_msg=key)


def test_ties_duplicates_padding_and_flags():
    cfg, parent, x = _synthetic(6, 12, 300, seed=11, tau=1.0, mode="topk")
    x["logits"][0] = np.round(x["logits"][0])        # equal logits: rank by token
    x["tokens"][1, 2] = x["tokens"][1, 1]             # duplicate siblings
    x["tokens"][3, 5] = 300                           # outside the vocabulary
    x["logits"][4, 0, 7] = np.nan                     # unusable row
    x["logits"][5, 3, 2] = -np.inf                    # a masked token: legal
    n_nodes = np.array([12, 12, 7, 12, 12, 12], dtype=np.int32)
    x["uniforms"][1, 1:3] = 0.999
    got, ref = _both(x, parent, 1.0, 10, 0.95, n_nodes=n_nodes, max_depth=cfg.max_tree_depth)
    assert ref["status"].tolist() == [0, 0, 0, 2, 64, 0]
    assert assert_accept_equal(got, ref, True) == 0


def test_sweep_sized_batch():
    cfg, parent, x = _synthetic(16, 128, 32000, seed=5, sigma=3.0, tau=1.0, mode="topk", max_tree_depth=8)
    got, ref = _both(x, parent, 1.0, 50, 0.9, max_depth=cfg.max_tree_depth)
    assert assert_accept_equal(got, ref, True) == 0
