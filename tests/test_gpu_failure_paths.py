"""The failure path of the bf16 attention kernel, exercised without any GPU fault: s4c_selftest_attention_timeout runs
the real launch with one cache tile per CTA never requested and a wait limit of a millisecond or two.  The waits for that
tile run out, every role leaves its loop, and the kernel must return normally with S4C_SEQ_TIMEOUT, the output untouched,
and the stream fit for the next launch."""
import numpy as np
import pytest
import torch

from paper_2506_14158_b200 import workloads as W

from parity import ATTN_TOL, Guarded, dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,B,Hq,Hkv,T,L,tile", [
    ("7B layer: clusters of 4, pushed partials, 4 row copies", 1, 32, 32, 26, 1024, 1),
    ("8B layer: two row tiles per CTA, parked partials", 4, 32, 8, 64, 4096, 3),
    ("full row tile, two softmax groups taking turns", 1, 16, 16, 100, 6000, 2),
    ("half-SM CTAs, no merge", 8, 32, 32, 100, 300, 2),
    ("one split, two row copies", 4, 32, 32, 50, 700, 0),
])
def test_a_wait_that_runs_out_ends_the_launch_cleanly(name, B, Hq, Hkv, T, L, tile):
    from paper_2506_14158_b200 import s4c
    import oracle

    d = 128
    C = (L + T + 127) // 128 * 128
    g = torch.Generator(device="cuda").manual_seed(len(name))
    q = torch.randn((B, Hq, T, d), generator=g, device="cuda").bfloat16()
    k = torch.randn((B, Hkv, C, d), generator=g, device="cuda").bfloat16()
    v = torch.randn((B, Hkv, C, d), generator=g, device="cuda").bfloat16()
    rng = np.random.default_rng(5)
    parent_np = np.stack([W.random_tree(T, 8, rng) for _ in range(B)])
    parent, cl = dev(parent_np), torch.full((B,), L, dtype=torch.int32, device="cuda")
    out = Guarded(q.shape, torch.bfloat16, fill=float("nan"))
    status = Guarded((B,), torch.int32, fill=0)
    s4c.selftest_attention_timeout(q, k, v, cl, parent, out.t, status.t, withhold_tile=tile, limit_us=1500, max_cache_len=L)
    torch.cuda.synchronize()  # returns: nothing hung, no error is pending
    out.check("out"), status.check("status")
    assert (status.t.cpu().numpy() == s4c.SEQ_TIMEOUT).all(), status.t.tolist()
    assert bool(torch.isnan(out.t.float()).all()), "a launch that gave up must not store results"
    # the same stream, the same buffers, right away: an ordinary launch, checked against the oracle on one KV head
    st2 = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    s4c.tree_attention(q, k, v, cl, parent, out=out.t, status=st2, max_cache_len=L)
    torch.cuda.synchronize()
    assert (st2.cpu().numpy() == 0).all()
    G, b, hk = Hq // Hkv, B - 1, Hkv - 1
    ref, _ = oracle.tree_attention(W.to_f64(q[b:b + 1, hk * G:(hk + 1) * G].cpu()), W.to_f64(k[b:b + 1, hk:hk + 1].cpu()),
                                   W.to_f64(v[b:b + 1, hk:hk + 1].cpu()), np.array([L], dtype=np.int32), parent_np[b:b + 1])
    got = out.t[b:b + 1, hk * G:(hk + 1) * G].double().cpu().numpy()
    assert np.abs(got - ref).max() <= ATTN_TOL["bf16"]
