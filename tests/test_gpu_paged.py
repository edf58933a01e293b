"""GPU parity on paged caches: s4c_tree_attention_paged and s4c_kv_compact_paged (through the C ABI) against the oracle run on
the contiguous cache that the block table spells out."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_14158_b200 import workloads as W

from parity import ATTN_TOL, Guarded, dev

pytestmark = pytest.mark.gpu


def _paged_case(B, Hq, Hkv, T, Ls, page_size, seed, d=128, n_nodes=None, extra_pages=7, hint=True):
    from paper_2506_14158_b200 import s4c

    rng = np.random.default_rng(seed)
    nb = max((L + T + page_size - 1) // page_size for L in Ls) + 1           # blocks per sequence (one spare, never listed)
    n_pages = B * nb + extra_pages
    g = torch.Generator().manual_seed(seed)
    q = torch.randn((B, Hq, T, d), generator=g).bfloat16()
    kp = torch.randn((n_pages, Hkv, page_size, d), generator=g).bfloat16()
    vp = torch.randn((n_pages, Hkv, page_size, d), generator=g).bfloat16()
    bt = rng.permutation(n_pages)[: B * nb].reshape(B, nb).astype(np.int32)  # pages scattered over the pool
    parent = np.stack([W.random_tree(T, 8, rng) for _ in range(B)])
    cl = np.asarray(Ls, dtype=np.int32)
    for b in range(B):                                                        # blocks beyond the sequence are not listed
        used = (Ls[b] + T + page_size - 1) // page_size
        bt[b, used:] = -1
    nn = None if n_nodes is None else np.asarray(n_nodes, dtype=np.int32)
    out = Guarded(q.shape, torch.bfloat16, fill=float("nan"))
    st = Guarded((B,), torch.int32, fill=-1)
    kg, vg = Guarded(kp.shape, torch.bfloat16, src=kp), Guarded(vp.shape, torch.bfloat16, src=vp)
    s4c.tree_attention_paged(dev(q), kg.t, vg.t, dev(bt), dev(cl), dev(parent), None if nn is None else dev(nn), out=out.t,
                             status=st.t, max_cache_len=max(Ls) if hint else 0)
    torch.cuda.synchronize()
    for x in (out, st, kg, vg):
        x.check("s4c_tree_attention_paged")
    kc = oracle.pages_to_contiguous(W.to_f64(kp), bt)
    vc = oracle.pages_to_contiguous(W.to_f64(vp), bt)
    ref, rst = oracle.tree_attention(W.to_f64(q), kc, vc, cl, parent, nn)
    np.testing.assert_array_equal(st.t.cpu().numpy(), rst)
    got = out.t.double().cpu().numpy()
    assert np.isfinite(got).all() and np.abs(got - ref).max() <= ATTN_TOL["bf16"]
    return bt, kp, vp, parent


@pytest.mark.parametrize("page_size", [64, 128, 256])
@pytest.mark.parametrize("shape", ["7B layer", "8B layer", "ragged batch", "long, many splits", "two waves of half-SM CTAs"])
def test_paged_attention_matches_the_contiguous_definition(shape, page_size):
    if shape == "7B layer":
        _paged_case(1, 32, 32, 26, [1024], page_size, seed=1)
    elif shape == "8B layer":
        _paged_case(2, 32, 8, 64, [4096, 1000], page_size, seed=2)
    elif shape == "ragged batch":
        _paged_case(3, 8, 2, 37, [0, 333, 130], page_size, seed=3, n_nodes=[37, 5, 20])
    elif shape == "long, many splits":
        _paged_case(1, 8, 8, 16, [9000], page_size, seed=4, hint=False)
    else:
        _paged_case(10, 32, 32, 20, [300, 17, 0, 640, 129, 300, 64, 511, 1, 77], page_size, seed=5)


def test_a_page_outside_the_pool_flags_the_sequence_and_touches_nothing_else():
    from paper_2506_14158_b200 import s4c

    B, Hq, Hkv, T, d, ps = 2, 4, 4, 10, 128, 64
    g = torch.Generator().manual_seed(9)
    q = torch.randn((B, Hq, T, d), generator=g).bfloat16()
    kp = torch.randn((12, Hkv, ps, d), generator=g).bfloat16()
    bt = np.array([[0, 1, 2], [3, 99, 5]], dtype=np.int32)  # sequence 1 lists a page the pool does not have
    cl = np.array([100, 100], dtype=np.int32)
    parent = np.tile(W.chain_tree(T), (B, 1))
    st = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    out = s4c.tree_attention_paged(dev(q), dev(kp), dev(kp), dev(bt), dev(cl), dev(parent), status=st)
    torch.cuda.synchronize()
    assert st.cpu().tolist() == [0, s4c.SEQ_BAD_PAGE]
    kc = oracle.pages_to_contiguous(W.to_f64(kp), bt[:1])
    ref, _ = oracle.tree_attention(W.to_f64(q[:1]), kc, kc, cl[:1], parent[:1])
    assert np.abs(out[:1].double().cpu().numpy() - ref).max() <= ATTN_TOL["bf16"]


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("page_size", [64, 128])
def test_paged_compaction_is_bit_exact(dtype, page_size):
    from paper_2506_14158_b200 import s4c

    dt = {"f32": torch.float32, "bf16": torch.bfloat16}[dtype]
    bits = torch.int32 if dt == torch.float32 else torch.int16
    rng = np.random.default_rng(page_size)
    B, Hkv, T, d, n_layers, hid, max_depth = 4, 3, 40, 64, 3, 128, 8
    Ls = [0, 100, 63, 200]
    nb = max((L + T + page_size - 1) // page_size for L in Ls)
    n_pages = B * nb + 5
    bt = rng.permutation(n_pages)[: B * nb].reshape(B, nb).astype(np.int32)
    g = torch.Generator().manual_seed(3)
    kps = [torch.randn((n_pages, Hkv, page_size, d), generator=g).to(dt) for _ in range(n_layers)]
    vps = [torch.randn((n_pages, Hkv, page_size, d), generator=g).to(dt) for _ in range(n_layers)]
    feat = torch.randn((B, T, hid), generator=g).to(dt)
    path = np.full((B, max_depth + 1), -1, dtype=np.int32)
    accept = np.array([3, 0, -1, 8], dtype=np.int32)  # one sequence skipped
    for b in range(B):
        if accept[b] >= 0:
            path[b, : accept[b] + 1] = np.concatenate([[0], np.sort(rng.choice(np.arange(1, T), accept[b], replace=False))])
    kg, vg = [Guarded(c.shape, dt, src=c) for c in kps], [Guarded(c.shape, dt, src=c) for c in vps]
    cl = Guarded((B,), torch.int32, src=torch.tensor(Ls, dtype=torch.int32))
    fo = Guarded((B, max_depth + 1, hid), dt, fill=3.0)
    st = s4c.kv_compact_paged(s4c.cache_pointer_array([x.t for x in kg]), s4c.cache_pointer_array([x.t for x in vg]), n_layers,
                              tuple(kps[0].shape), dt, dev(bt), cl.t, dev(path), dev(accept), T, dev(feat), fo.t)
    torch.cuda.synchronize()
    for x in kg + vg + [cl, fo]:
        x.check("s4c_kv_compact_paged")
    # oracle: compact the contiguous caches the table spells out, then compare slot by slot through the table
    as_bits = lambda t: t.view(bits).numpy()
    kc = [oracle.pages_to_contiguous(as_bits(c), bt) for c in kps]
    vc = [oracle.pages_to_contiguous(as_bits(c), bt) for c in vps]
    rl = np.asarray(Ls, dtype=np.int32).copy()
    rfo = as_bits(torch.full((B, max_depth + 1, hid), 3.0, dtype=dt)).copy()
    rst = oracle.kv_compact(kc, vc, rl, path, accept, T, as_bits(feat).copy(), rfo)
    np.testing.assert_array_equal(st.cpu().numpy(), rst)
    np.testing.assert_array_equal(cl.t.cpu().numpy(), rl)
    np.testing.assert_array_equal(as_bits(fo.t.cpu()), rfo)
    for l in range(n_layers):
        for got_pool, ref in ((kg[l].t, kc[l]), (vg[l].t, vc[l])):
            got = oracle.pages_to_contiguous(as_bits(got_pool.cpu()), bt)
            for b in range(B):
                new = max(int(rl[b]), Ls[b])
                np.testing.assert_array_equal(got[b, :, :new], ref[b, :, :new])
    # pages that no sequence lists are untouched
    listed = set(bt.reshape(-1).tolist())
    for p in range(n_pages):
        if p not in listed:
            assert torch.equal(kg[0].t[p].cpu().view(bits), kps[0][p].view(bits))
