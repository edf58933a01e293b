"""GPU parity: s4c_qkv_rope (through the C ABI) against the oracle -- q in the attention layout, k / v in the caches' tree
slots, everything else untouched.

Tolerance: the kernel accumulates bf16 products in float32 and rounds the rotated result to bf16 once; the oracle works
in float64 on the same bf16 inputs.  |got - want| <= 2^-8 |want| (half a bf16 ulp, rounded up) + 8 sqrt(H) 2^-24 ||x|| ||w||
(float32 accumulation, rotation included)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_14158_b200 import workloads as W

from parity import Guarded, dev

pytestmark = pytest.mark.gpu


def _bf16(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16)


def _run(x, w, cache_len, parent, Hq, Hkv, d, C, n_nodes=None, theta=10000.0, seed=0, position_base=None):
    from paper_2506_14158_b200 import s4c

    B, T, H = x.shape
    g = torch.Generator().manual_seed(seed)
    k0 = torch.randn(B, Hkv, C, d, generator=g).to(torch.bfloat16)   # what the caches hold before the call
    v0 = torch.randn(B, Hkv, C, d, generator=g).to(torch.bfloat16)
    bufs = dict(q=Guarded((B, Hq, T, d), torch.bfloat16, fill=-3.0), k=Guarded((B, Hkv, C, d), torch.bfloat16, src=k0.cuda()),
                v=Guarded((B, Hkv, C, d), torch.bfloat16, src=v0.cuda()), status=Guarded((B,), torch.int32, fill=-9),
                ws=Guarded((max(256, s4c.qkv_rope_workspace_bytes(B, T, d)),), torch.uint8, fill=0xCD))
    s4c.qkv_rope(x.cuda(), w.cuda(), dev(cache_len), dev(parent.astype(np.int32)), bufs["q"].t, bufs["k"].t, bufs["v"].t,
                 None if n_nodes is None else dev(n_nodes), theta, status=bufs["status"].t, workspace=bufs["ws"].t,
                 position_base=None if position_base is None else dev(np.asarray(position_base, dtype=np.int32)))
    torch.cuda.synchronize()
    for name, buf in bufs.items():
        buf.check("s4c_qkv_rope " + name)
    kc, vc = k0.double().numpy().copy(), v0.double().numpy().copy()
    ref = oracle.qkv_rope(x.double().numpy(), w.double().numpy(), cache_len, parent, Hq, Hkv, d, kc, vc, n_nodes, theta,
                          position_base=position_base)
    got = dict(q=bufs["q"].t.double().cpu().numpy(), k=bufs["k"].t.double().cpu().numpy(), v=bufs["v"].t.double().cpu().numpy(),
               status=bufs["status"].t.cpu().numpy())
    return got, dict(q=ref["q"], k=kc, v=vc, status=ref["status"]), (k0.double().numpy(), v0.double().numpy())


def _compare(got, ref, x, w, cache_len, n_nodes, T):
    np.testing.assert_array_equal(got["status"], ref["status"])
    B = x.shape[0]
    H = x.shape[2]
    slack = 8.0 * np.sqrt(H) * 2.0 ** -24 * float(x.float().norm(dim=2).max()) * float(w.float().norm(dim=1).max())
    for b in range(B):
        n = T if n_nodes is None else int(n_nodes[b])
        if ref["status"][b]:
            assert (got["q"][b] == -3.0).all()                                    # nothing of a flagged sequence is written
            np.testing.assert_array_equal(got["k"][b], ref["k"][b])
            np.testing.assert_array_equal(got["v"][b], ref["v"][b])
            continue
        L = int(cache_len[b])
        for name, g_, r_ in (("q", got["q"][b][:, :n], ref["q"][b][:, :n]), ("k", got["k"][b][:, L:L + n], ref["k"][b][:, L:L + n]),
                             ("v", got["v"][b][:, L:L + n], ref["v"][b][:, L:L + n])):
            err = np.abs(g_ - r_)
            assert (err <= 2.0 ** -8 * np.abs(r_) + slack).all(), (name, b, float(err.max()))
        assert (got["q"][b][:, n:] == -3.0).all()                                 # rows of padding nodes: not written
        mask = np.ones(got["k"].shape[2], dtype=bool)
        mask[L:L + n] = False
        np.testing.assert_array_equal(got["k"][b][:, mask], ref["k"][b][:, mask])  # every other slot as it was
        np.testing.assert_array_equal(got["v"][b][:, mask], ref["v"][b][:, mask])


@pytest.mark.parametrize("B,T,H,Hq,Hkv,d,C", [(1, 1, 64, 1, 1, 64, 8), (2, 15, 128, 4, 4, 64, 160), (1, 26, 512, 8, 8, 128, 300),
                                              (4, 64, 256, 8, 2, 128, 200), (3, 50, 192, 6, 3, 128, 512), (5, 128, 128, 2, 1, 128, 1024),
                                              (2, 128, 64, 3, 1, 64, 256), (1, 33, 8192, 2, 2, 128, 64), (7, 19, 320, 5, 5, 64, 40)])
def test_shapes_against_the_oracle(B, T, H, Hq, Hkv, d, C):
    rng = np.random.default_rng(B * 100 + T)
    parent = np.stack([W.random_tree(T, 6, rng, 1, 4) for _ in range(B)]) if T > 1 else np.full((B, 1), -1, dtype=np.int32)
    x, w = _bf16(rng.standard_normal((B, T, H))), _bf16(rng.standard_normal(((Hq + 2 * Hkv) * d, H)) / np.sqrt(H))
    cache_len = rng.integers(0, C - T + 1, B).astype(np.int32)
    got, ref, _ = _run(x, w, cache_len, parent, Hq, Hkv, d, C)
    assert (ref["status"] == 0).all()
    _compare(got, ref, x, w, cache_len, None, T)


def test_long_contexts_rotate_accurately():
    # positions near 32768: the angles are large; cos / sin come from a float64 table
    rng = np.random.default_rng(7)
    B, T, H, Hq, Hkv, d, C = 2, 26, 256, 4, 2, 128, 32768
    parent = np.stack([W.random_tree(T, 5, rng, 1, 4) for _ in range(B)])
    x, w = _bf16(rng.standard_normal((B, T, H))), _bf16(rng.standard_normal(((Hq + 2 * Hkv) * d, H)) / np.sqrt(H))
    cache_len = np.array([32768 - T, 20011], dtype=np.int32)
    got, ref, _ = _run(x, w, cache_len, parent, Hq, Hkv, d, C)
    _compare(got, ref, x, w, cache_len, None, T)


def test_padding_flags_and_untouched_sequences():
    rng = np.random.default_rng(8)
    B, T, H, Hq, Hkv, d, C = 5, 20, 128, 4, 2, 128, 64
    parent = np.stack([W.random_tree(T, 5, rng, 1, 4) for _ in range(B)])
    x, w = _bf16(rng.standard_normal((B, T, H))), _bf16(rng.standard_normal(((Hq + 2 * Hkv) * d, H)) / np.sqrt(H))
    cache_len = np.array([3, 50, 10, 44, 0], dtype=np.int32)          # sequence 1: 50 + 20 > 64; sequence 3: 44 + 20 = 64 fits
    parent[2, 4] = 9                                                  # sequence 2: malformed
    n_nodes = np.array([20, 20, 20, 7, 1], dtype=np.int32)
    got, ref, _ = _run(x, w, cache_len, parent, Hq, Hkv, d, C, n_nodes)
    assert ref["status"].tolist() == [0, oracle.SEQ_CAPACITY, oracle.SEQ_BAD_PARENT, 0, 0]
    _compare(got, ref, x, w, cache_len, n_nodes, T)


@pytest.mark.parametrize("B,T,H,Hq,Hkv,d,C", [(5, 20, 128, 4, 2, 128, 64), (1, 26, 512, 8, 8, 64, 200), (3, 64, 256, 8, 2, 128, 300)])
def test_another_layer_on_the_same_tree_reuses_the_tables(B, T, H, Hq, Hkv, d, C):
    # layer 1 with the table kernel, layer 2 (other states, other weights, other caches) on what it left in the workspace:
    # the same bits as a full call for layer 2, flagged sequences skipped, the status array kept
    from paper_2506_14158_b200 import s4c

    rng = np.random.default_rng(B + T)
    parent = np.stack([W.random_tree(T, 5, rng, 1, 4) for _ in range(B)]).astype(np.int32)
    cache_len = rng.integers(0, C - T + 1, B).astype(np.int32)
    n_nodes = rng.integers(1, T + 1, B).astype(np.int32)
    if B >= 5:
        cache_len[1] = C - T + 5   # does not fit
        parent[2, 4] = 9           # malformed
    mk = lambda *shape, s=1.0: _bf16(rng.standard_normal(shape) * s).cuda()
    xs, ws_ = [mk(B, T, H), mk(B, T, H)], [mk((Hq + 2 * Hkv) * d, H, s=H ** -0.5), mk((Hq + 2 * Hkv) * d, H, s=H ** -0.5)]
    k0, v0 = mk(B, Hkv, C, d), mk(B, Hkv, C, d)
    wsp = torch.empty(s4c.qkv_rope_workspace_bytes(B, T, d), dtype=torch.uint8, device="cuda")
    # the full call for layer 2's inputs: what the reuse must reproduce
    q_full, k_full, v_full = torch.full((B, Hq, T, d), -3.0, dtype=torch.bfloat16, device="cuda"), k0.clone(), v0.clone()
    st_full = s4c.qkv_rope(xs[1], ws_[1], dev(cache_len), dev(parent), q_full, k_full, v_full, dev(n_nodes), workspace=wsp)["status"].clone()
    wsp.fill_(0xCD)
    q1, k1, v1 = torch.empty_like(q_full), k0.clone(), v0.clone()
    st = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    s4c.qkv_rope(xs[0], ws_[0], dev(cache_len), dev(parent), q1, k1, v1, dev(n_nodes), status=st, workspace=wsp)
    q2 = Guarded((B, Hq, T, d), torch.bfloat16, fill=-3.0)
    k2, v2 = Guarded((B, Hkv, C, d), torch.bfloat16, src=k0), Guarded((B, Hkv, C, d), torch.bfloat16, src=v0)
    s4c.qkv_rope_same_tree(xs[1], ws_[1], q2.t, k2.t, v2.t, wsp, status=st)
    torch.cuda.synchronize()
    for name, buf in (("q", q2), ("k", k2), ("v", v2)):
        buf.check("s4c_qkv_rope_same_tree " + name)
    assert torch.equal(st, st_full)
    assert torch.equal(q2.t, q_full) and torch.equal(k2.t, k_full) and torch.equal(v2.t, v_full)
    if B >= 5:
        assert st.tolist()[1] == oracle.SEQ_CAPACITY and st.tolist()[2] == oracle.SEQ_BAD_PARENT
        assert (q2.t[1] == -3.0).all() and torch.equal(k2.t[2], k0[2])


def test_root_position_apart_from_the_cache_length():
    # s4c_qkv_rope_at: positions count from position_base, slots from cache_len; a negative base flags its sequence
    rng = np.random.default_rng(19)
    B, T, H, Hq, Hkv, d, C = 4, 12, 256, 4, 2, 64, 40
    parent = np.stack([W.random_tree(T, 5, rng, 1, 3) for _ in range(B)])
    x, w = _bf16(rng.standard_normal((B, T, H))), _bf16(rng.standard_normal(((Hq + 2 * Hkv) * d, H)) / np.sqrt(H))
    cache_len = np.array([5, 0, 28, 17], dtype=np.int32)
    base = np.array([900, 3, -2, 17], dtype=np.int32)
    got, ref, _ = _run(x, w, cache_len, parent, Hq, Hkv, d, C, position_base=base)
    assert ref["status"].tolist() == [0, 0, oracle.SEQ_CAPACITY, 0]
    _compare(got, ref, x, w, cache_len, None, T)
    plain, _, _ = _run(x, w, cache_len, parent, Hq, Hkv, d, C)
    np.testing.assert_array_equal(got["q"][3], plain["q"][3])          # base == cache length: the plain call
    assert not np.array_equal(got["q"][0], plain["q"][0])


def test_full_size_layer_then_attention_reads_what_was_written():
    # the 8B-shaped layer (256 rows, H = 4096, 32/8 heads x 128) in the launch the benchmark times, and the hand-over:
    # s4c_tree_attention on the q and caches this call wrote equals the oracle's attention on the oracle's q / k / v
    from paper_2506_14158_b200 import s4c

    cfg = W.CONFIGS["c4"]
    rng = np.random.default_rng(9)
    B, T, H, Hq, Hkv, d = cfg.B, cfg.T, cfg.hid, cfg.Hq, cfg.Hkv, cfg.d
    L, C = 300, 512
    parent = W.make_trees(cfg)
    x = _bf16(rng.standard_normal((B, T, H)))
    w = _bf16(rng.standard_normal(((Hq + 2 * Hkv) * d, H)) / np.sqrt(H))
    cache_len = np.full(B, L, dtype=np.int32)
    got, ref, (k0, v0) = _run(x, w, cache_len, parent, Hq, Hkv, d, C)
    _compare(got, ref, x, w, cache_len, None, T)
    # hand-over on one sequence (the oracle's attention is slow): same caches, same q
    b = 1
    q_t = torch.from_numpy(got["q"][b:b + 1]).to(torch.bfloat16).cuda()
    k_t = torch.from_numpy(got["k"][b:b + 1]).to(torch.bfloat16).cuda()
    v_t = torch.from_numpy(got["v"][b:b + 1]).to(torch.bfloat16).cuda()
    out = s4c.tree_attention(q_t, k_t, v_t, dev(cache_len[b:b + 1]), dev(parent[b:b + 1].astype(np.int32)), None)
    torch.cuda.synchronize()
    want, st = oracle.tree_attention(got["q"][b:b + 1], got["k"][b:b + 1], got["v"][b:b + 1], cache_len[b:b + 1], parent[b:b + 1])
    assert int(st[0]) == 0
    np.testing.assert_allclose(out.double().cpu().numpy(), want, atol=2e-2)
