"""GPU parity: s4c_kv_compact against the oracle gather -- bit-exact on raw bits."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_14158_b200 import workloads as W

from parity import accept_both, assert_compact_equal, compact_both

pytestmark = pytest.mark.gpu


def _paths_from_accept(cfg, tau):
    parent = W.make_trees(cfg)
    x = W.make_accept_inputs(cfg, parent, tau, token_mode="topk")
    _, ref = accept_both(x, parent, tau, max_depth=cfg.max_depth)
    return ref["path"], ref["accept_len"]


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4"])
def test_named_configs(name):
    cfg = W.CONFIGS[name]
    path, alen = _paths_from_accept(cfg, cfg.temperatures[-1])
    n_layers = 3
    ks, vs = [], []
    for l in range(n_layers):
        _, k, v = W.make_attention_inputs(cfg, layer=l)
        ks.append(k)
        vs.append(v)
    feat = W.make_features(cfg)
    old = np.full(cfg.B, cfg.L, dtype=np.int32)
    got, ref = compact_both(ks, vs, old, path, alen, cfg.T, feat)
    assert (ref[4] == 0).all() and (ref[2] == old + alen + 1).all()
    assert_compact_equal(got, ref, old, cfg.T)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_random_paths_ragged_lengths_and_skips(dtype):
    rng = np.random.default_rng(3)
    B, Hkv, T, d, max_depth, n_layers, hid = 6, 3, 128, 64, 20, 2, 48
    Ls = np.array([0, 1, 77, 200, 31, 5], dtype=np.int32)
    C = int(Ls.max()) + T
    g = torch.Generator().manual_seed(5)
    mk = lambda: torch.randn((B, Hkv, C, d), generator=g).to(dtype)
    ks, vs = [mk() for _ in range(n_layers)], [mk() for _ in range(n_layers)]
    feat = torch.randn((B, T, hid), generator=g).to(dtype)
    path = np.full((B, max_depth + 1), -1, dtype=np.int32)
    alen = np.zeros(B, dtype=np.int32)
    for b in range(B):
        a = int(rng.integers(0, max_depth + 1))
        path[b, : a + 1] = np.concatenate([[0], np.sort(rng.choice(np.arange(1, T), size=a, replace=False))])
        alen[b] = a
    alen[2] = -1                      # upstream-flagged sequence: skipped
    alen[4] = max(alen[4], 2)
    path[4, :3] = [0, 9, 4]           # not increasing: flagged, nothing written
    got, ref = compact_both(ks, vs, Ls, path, alen, T, feat)
    assert_compact_equal(got, ref, Ls, T)
    assert ref[4][4] & oracle.SEQ_BAD_PATH


def test_full_depth_path_and_no_layers():
    B, Hkv, T, d = 1, 2, 128, 128
    L = 3
    C = L + T
    g = torch.Generator().manual_seed(6)
    k = torch.randn((B, Hkv, C, d), generator=g).to(torch.bfloat16)
    v = torch.randn((B, Hkv, C, d), generator=g).to(torch.bfloat16)
    path = np.arange(0, 128, dtype=np.int32)[None]  # the chain: identity, nothing moves
    got, ref = compact_both([k], [v], [L], path, [127], T)
    assert_compact_equal(got, ref, [L], T)
    path = np.full((1, 128), -1, dtype=np.int32)
    path[0, :64] = np.arange(0, 128, 2)             # every second node
    got, ref = compact_both([k], [v], [L], path, [63], T)
    assert_compact_equal(got, ref, [L], T)
    # capacity violation is flagged, nothing written
    got, ref = compact_both([k], [v], [L + 1], path, [63], T)
    assert got[4][0] == oracle.SEQ_CAPACITY
    assert_compact_equal(got, ref, [L + 1], T)
