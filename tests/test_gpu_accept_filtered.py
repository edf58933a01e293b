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


def test_verify_step_with_a_filter_in_one_graph():
    # the whole step (attention, filtered acceptance, compaction) replayed as one CUDA graph: the decision is the
    # oracle's filtered one and the committed lengths follow it
    from dataclasses import replace

    from paper_2506_14158_b200.verify import VerifyStep

    cfg = replace(W.CONFIGS["c2"], n_layers=2)
    parent = W.make_trees(cfg)
    x = W.make_accept_inputs(cfg, parent, 1.0, token_mode="topk")
    qs, ks, vs = zip(*[[t.cuda() for t in W.make_attention_inputs(cfg, l)] for l in range(cfg.n_layers)])
    step = VerifyStep(list(qs), list(ks), list(vs), torch.full((cfg.B,), cfg.L, dtype=torch.int32, device="cuda"),
                      dev(parent), dev(x["tokens"]), dev(x["logits"]), dev(x["draft_probs"]), dev(x["uniforms"]), 1.0,
                      cfg.max_depth, feat_in=W.make_features(cfg).cuda(), max_cache_len=cfg.L)
    step.set_filter(20, 0.9)
    g = step.capture("step")
    g.replay()
    torch.cuda.synchronize()
    ref = oracle.accept_filtered(x["logits"], x["draft_probs"], x["tokens"], np.ascontiguousarray(parent, dtype=np.int32), 1.0,
                                 20, float(np.float32(0.9)), x["uniforms"], None, cfg.max_depth)
    for key in ("accept_len", "path", "next_token"):
        np.testing.assert_array_equal(getattr(step, key).cpu().numpy(), ref[key], err_msg=key)
    np.testing.assert_array_equal(step.cache_len.cpu().numpy(), cfg.L + ref["accept_len"] + 1)
    plain = oracle.accept_stochastic(x["logits"], x["draft_probs"], x["tokens"], np.ascontiguousarray(parent, dtype=np.int32),
                                     1.0, x["uniforms"], None, cfg.max_depth)
    step.set_filter(None)
    step.run()
    torch.cuda.synchronize()
    np.testing.assert_array_equal(step.accept_len.cpu().numpy(), plain["accept_len"])


@pytest.mark.parametrize("V", [140000, 270001])
def test_rows_wider_than_one_merge_round(V):
    # more than 32 vocabulary segments per row: the row's best are folded over several rounds of list merges
    cfg, parent, x = _synthetic(2, 5, V, seed=V % 89, sigma=2.5, tau=1.0, mode="topk")
    x["logits"][0, 1, V - 3:] = 40.0    # winners in the last (ragged) segment, equal: ranked by token
    x["logits"][1, 0, ::4096] += 30.0   # one winner in every segment
    got, ref = _both(x, parent, 1.0, 64, 0.99, max_depth=cfg.max_tree_depth)
    assert assert_accept_equal(got, ref, True) == 0


@pytest.mark.parametrize("top_k,top_p", [(1, 1.0), (7, 1.0), (64, 0.9)])
def test_segments_the_threshold_selection_cannot_serve(top_k, top_p):
    # heavy ties and masked vocabularies: more than 256 entries at the threshold, or fewer than k finite thread maxima --
    # those segments take the exact sort-and-merge path
    cfg, parent, x = _synthetic(8, 6, 9000, seed=17, tau=1.0, mode="topk")
    lg = x["logits"]
    lg[0] = 1.25                                           # every logit equal: the k lowest tokens win
    lg[1] = np.where(lg[1] > 0, 2.0, -1.0)                 # two values
    lg[2] = np.round(lg[2] / 4.0)                          # a handful of values
    keep = lg[3, :, 4090:4100].copy()
    lg[3] = -np.inf                                        # nearly everything masked: ten finite logits across a
    lg[3, :, 4090:4100] = keep                             # segment boundary
    lg[4, :, :5000] = -np.inf                              # the first segment masked entirely, ties at -inf
    lg[5] = np.minimum(lg[5], 0.5)                         # a plateau at the top
    lg[6, :, 1:] = lg[6, :, :1]                            # every row constant, another value per row
    got, ref = _both(x, parent, 1.0, top_k, top_p, max_depth=cfg.max_tree_depth)
    assert (ref["status"] == 0).all()
    assert assert_accept_equal(got, ref, True) == 0
