"""GPU parity: s4c_tree_build (through the C ABI) against the oracle's construction of the continuous verification
tree (Section 3.2, Figure 3) -- tokens, parent links, position ids and node counts bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_14158_b200 import workloads as W

from parity import Guarded, dev

pytestmark = pytest.mark.gpu


def _both(q, branching, root, L):
    from paper_2506_14158_b200 import s4c

    B, T, V = q.shape
    g = dict(tokens=Guarded((B, T), torch.int32, fill=-9), parent=Guarded((B, T), torch.int32, fill=-9),
             position=Guarded((B, T), torch.int32, fill=-9), n_nodes=Guarded((B,), torch.int32, fill=-9),
             workspace=Guarded((max(256, s4c.tree_build_workspace_bytes(B, T, V, max([1] + list(branching)))),), torch.uint8, fill=0))
    r = s4c.tree_build(dev(q), branching, dev(root), None if L is None else dev(L), tokens=g["tokens"].t, parent=g["parent"].t,
                       position=g["position"].t, n_nodes=g["n_nodes"].t, workspace=g["workspace"].t)
    torch.cuda.synchronize()
    for name, buf in g.items():
        buf.check("s4c_tree_build " + name)
    ref = oracle.build_tree(q, branching, root, L)
    for key in ("tokens", "parent", "position", "n_nodes"):
        np.testing.assert_array_equal(r[key].cpu().numpy(), ref[key], err_msg=key)
    return ref


def _probs(rng, B, T, V, sigma=3.0):
    x = rng.standard_normal((B, T, V)) * sigma
    e = np.exp(x - x.max(-1, keepdims=True))
    return (e / e.sum(-1, keepdims=True)).astype(np.float32)


@pytest.mark.parametrize("name,branching", [("c1", (3, 2, 1)), ("c2", (4, 3, 2, 2, 1))])
def test_named_configs_reproduce_the_benchmark_trees_and_tokens(name, branching):
    cfg = W.CONFIGS[name]
    parent = W.make_trees(cfg)
    x = W.make_accept_inputs(cfg, parent, 1.0, token_mode="topk")
    L = np.full(cfg.B, cfg.L, dtype=np.int32)
    ref = _both(x["draft_probs"], branching, x["tokens"][:, 0].copy(), L)
    # the device-built tree is the tree the benchmark's host generator lays out, with the same draft tokens
    np.testing.assert_array_equal(ref["parent"], parent)
    np.testing.assert_array_equal(ref["tokens"], x["tokens"])


@pytest.mark.parametrize("V", [1, 5, 64, 4096, 4099, 32000, 128256])
@pytest.mark.parametrize("branching,T", [((4, 3, 2, 2, 1), 26), ((2, 2, 2, 2, 2, 2), 64), ((16,), 17), ((1, 1, 1), 4), ((3, 3), 128)])
def test_vocabulary_sizes_and_shapes(V, branching, T):
    if max(branching) > V:
        branching = tuple(min(b, V) for b in branching)
    rng = np.random.default_rng(V + T)
    B = 3 if V < 100000 else 2
    q = _probs(rng, B, T, V)
    _both(q, branching, rng.integers(0, V, B).astype(np.int32), np.array([0, 4096, 31][:B], dtype=np.int32))


def test_ties_go_to_the_lower_token_across_segments():
    rng = np.random.default_rng(1)
    B, T, V = 2, 16, 20000
    q = np.round(_probs(rng, B, T, V, sigma=1.0) * 2000) / 2000  # many equal values, also across the 4096-entry segments
    q[0, 0, :] = 0.25                                             # a flat row: the lowest tokens win
    ref = _both(q.astype(np.float32), (4, 3), np.array([1, 2], dtype=np.int32), None)
    assert ref["tokens"][0, 1:5].tolist() == [0, 1, 2, 3]


def test_built_tree_feeds_the_verify_step_without_the_host():
    # drafter distributions -> s4c_tree_build -> s4c_tree_accept, all on one stream; the result equals the oracle's
    # acceptance on the oracle's tree
    from paper_2506_14158_b200 import s4c

    cfg = W.CONFIGS["c2"]
    parent = W.make_trees(cfg)
    x = W.make_accept_inputs(cfg, parent, 1.0, token_mode="topk")
    t = s4c.tree_build(dev(x["draft_probs"]), cfg.branching, dev(x["tokens"][:, 0].copy()))
    r = s4c.tree_accept(dev(x["logits"]), dev(x["draft_probs"]), t["tokens"], t["parent"], 1.0, dev(x["uniforms"]),
                        n_nodes=t["n_nodes"], max_depth=cfg.max_depth)
    torch.cuda.synchronize()
    tree = oracle.build_tree(x["draft_probs"], cfg.branching, x["tokens"][:, 0])
    ref = oracle.accept_stochastic(x["logits"], x["draft_probs"], tree["tokens"], tree["parent"], 1.0, x["uniforms"],
                                   tree["n_nodes"], cfg.max_depth)
    for key in ("accept_len", "path", "next_token", "status"):
        np.testing.assert_array_equal(r[key].cpu().numpy(), ref[key], err_msg=key)


def test_verify_step_with_the_tree_built_on_the_device():
    # the whole step of verify.py from drafter distributions: tree build, attention, acceptance, compaction in one CUDA
    # graph; decisions equal those of the same step fed with the host-generated tree
    from dataclasses import replace

    from paper_2506_14158_b200.verify import VerifyStep

    cfg = replace(W.CONFIGS["c2"], n_layers=2)
    parent = W.make_trees(cfg)
    x = W.make_accept_inputs(cfg, parent, 1.0, token_mode="topk")
    results = []
    for on_device in (False, True):
        qs, ks, vs = zip(*[[t.cuda() for t in W.make_attention_inputs(cfg, l)] for l in range(cfg.n_layers)])
        par = dev(parent) if not on_device else torch.zeros_like(dev(parent))
        tok = dev(x["tokens"]) if not on_device else torch.zeros_like(dev(x["tokens"]))
        step = VerifyStep(list(qs), list(ks), list(vs), torch.full((cfg.B,), cfg.L, dtype=torch.int32, device="cuda"), par, tok,
                          dev(x["logits"]), dev(x["draft_probs"]), dev(x["uniforms"]), 1.0, cfg.max_depth,
                          feat_in=W.make_features(cfg).cuda(), max_cache_len=cfg.L,
                          branching=cfg.branching if on_device else None,
                          root_token=dev(x["tokens"][:, 0].copy()) if on_device else None)
        g = step.capture("step")
        g.replay()
        torch.cuda.synchronize()
        results.append([t.cpu().numpy().copy() for t in (step.accept_len, step.path, step.next_token, step.cache_len,
                                                         step.attn_out[1].float(), step.feat_out.float(), step.parent, step.tokens)])
    for a, b in zip(*results):
        np.testing.assert_array_equal(a, b)
