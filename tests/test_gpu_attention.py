"""GPU parity: s4c_tree_attention (through the C ABI) against the float64 oracle, element by element."""
import numpy as np
import pytest
import torch

from paper_2506_14158_b200 import workloads as W

from parity import ATTN_TOL, assert_attention_close, attention_both

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4"])
def test_named_configs(name):
    cfg = W.CONFIGS[name]
    q, k, v = W.make_attention_inputs(cfg)
    parent = W.make_trees(cfg)
    got, ref, gst, rst = attention_both(q, k, v, [cfg.L] * cfg.B, parent)
    assert (rst == 0).all()
    assert_attention_close(got, ref, gst, rst, ATTN_TOL[cfg.dtype])


def _case(B, Hq, Hkv, T, d, Ls, dtype, seed, tree="random", n_nodes=None, scale=0.0, C=None):
    rng = np.random.default_rng(seed)
    dt = {"f32": torch.float32, "bf16": torch.bfloat16}[dtype]
    C = C or (max(Ls) + T + 5)
    g = torch.Generator().manual_seed(seed)
    q = torch.randn((B, Hq, T, d), generator=g).to(dt)
    k = torch.randn((B, Hkv, C, d), generator=g).to(dt)
    v = torch.randn((B, Hkv, C, d), generator=g).to(dt)
    if tree == "chain":
        parent = np.tile(W.chain_tree(T), (B, 1))
    elif tree == "star":
        parent = np.tile(W.star_tree(T), (B, 1))
    else:
        parent = np.stack([W.random_tree(T, 8, rng) for _ in range(B)])
    got, ref, gst, rst = attention_both(q, k, v, Ls, parent, n_nodes, scale)
    assert_attention_close(got, ref, gst, rst, ATTN_TOL[dtype])
    return got, ref


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d", [64, 128])
def test_ragged_lengths_gqa_and_padding(dtype, d):
    # cache lengths that are not multiples of any tile, several tiles long, one empty prefix; padded trees
    _case(B=3, Hq=8, Hkv=2, T=37, d=d, Ls=[0, 333, 130], dtype=dtype, seed=1, n_nodes=[37, 5, 20])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("tree", ["chain", "star"])
def test_chain_and_star_trees(dtype, tree):
    _case(B=1, Hq=4, Hkv=4, T=33, d=128, Ls=[257], dtype=dtype, seed=2, tree=tree, scale=0.11)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_extreme_tree_sizes(dtype):
    _case(B=2, Hq=2, Hkv=1, T=1, d=128, Ls=[64, 1], dtype=dtype, seed=3)            # plain decode
    _case(B=1, Hq=2, Hkv=2, T=128, d=128, Ls=[700], dtype=dtype, seed=4)            # the maximum tree
    _case(B=1, Hq=4, Hkv=1, T=128, d=64, Ls=[0], dtype=dtype, seed=5, tree="chain")  # no prefix at all


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("Hq,Hkv,T", [(4, 4, 26), (8, 2, 64)])
def test_slots_past_the_sequence_end_may_hold_anything(dtype, Hq, Hkv, T):
    # K/V slots at and beyond L + n are not part of the sequence: NaN or Inf there must not reach the output
    # (their scores are masked by selection, their V rows never enter the product)
    from paper_2506_14158_b200 import s4c
    from parity import dev

    B, d, Ls, C = 2, 128, [1000, 70], 1152
    dt = {"f32": torch.float32, "bf16": torch.bfloat16}[dtype]
    rng = np.random.default_rng(11)
    g = torch.Generator().manual_seed(11)
    q = torch.randn((B, Hq, T, d), generator=g).to(dt)
    k = torch.randn((B, Hkv, C, d), generator=g).to(dt)
    v = torch.randn((B, Hkv, C, d), generator=g).to(dt)
    parent = np.stack([W.random_tree(T, 8, rng) for _ in range(B)])
    clean, ref, gst, rst = attention_both(q, k, v, Ls, parent)
    assert_attention_close(clean, ref, gst, rst, ATTN_TOL[dtype])
    kp, vp = k.clone(), v.clone()
    for b in range(B):
        kp[b, :, Ls[b] + T:] = float("nan")
        vp[b, :, Ls[b] + T:: 2] = float("nan")
        vp[b, :, Ls[b] + T + 1:: 2] = float("inf")
    status = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    out = torch.full(q.shape, float("nan"), dtype=q.dtype, device="cuda")
    s4c.tree_attention(dev(q), dev(kp), dev(vp), dev(np.asarray(Ls, dtype=np.int32)), dev(parent.astype(np.int32)), None,
                       out=out, status=status)
    torch.cuda.synchronize()
    assert (status.cpu().numpy() == 0).all()
    np.testing.assert_array_equal(out.double().cpu().numpy(), clean)


@pytest.mark.parametrize("B,Hq,Hkv,T,L", [(1, 32, 8, 64, 1000),   # 256 rows of a KV head over two CTAs, two softmax groups each
                                           (2, 16, 4, 40, 700),    # 160 rows: a full row tile and a partial one
                                           (1, 16, 2, 128, 300),   # 1024 rows: eight row tiles, one per CTA
                                           (1, 24, 24, 32, 3000)])  # 24 heads: clusters of 5, not 6
def test_small_grids_take_one_row_tile_per_cta(B, Hq, Hkv, T, L):
    _case(B=B, Hq=Hq, Hkv=Hkv, T=T, d=128, Ls=[L] * B, dtype="bf16", seed=21 + T)


def test_long_context_many_splits():
    _case(B=1, Hq=8, Hkv=8, T=16, d=128, Ls=[9000], dtype="bf16", seed=6)


def test_flagged_sequences_are_skipped_not_trapped():
    from parity import attention_both

    g = torch.Generator().manual_seed(9)
    B, H, T, d, C = 3, 2, 6, 128, 64
    q = torch.randn((B, H, T, d), generator=g).to(torch.bfloat16)
    k = torch.randn((B, H, C, d), generator=g).to(torch.bfloat16)
    v = torch.randn((B, H, C, d), generator=g).to(torch.bfloat16)
    parent = np.tile(W.chain_tree(T), (B, 1))
    parent[1, 3] = 4  # parent[i] >= i
    got, ref, gst, rst = attention_both(q, k, v, [10, 10, 60], parent)  # third: 60 + 6 > 64
    assert gst[0] == 0 and gst[1] == 1 and gst[2] == 4
    assert_attention_close(got, ref, gst, rst, ATTN_TOL["bf16"])


def test_results_do_not_depend_on_scheduling():
    cfg = W.CONFIGS["c2"]
    q, k, v = W.make_attention_inputs(cfg)
    parent = W.make_trees(cfg)
    a, _, _, _ = attention_both(q, k, v, [cfg.L], parent)
    b, _, _, _ = attention_both(q, k, v, [cfg.L], parent)
    np.testing.assert_array_equal(a, b)


@pytest.mark.parametrize("d", [64, 128])
def test_full_row_tile_with_two_softmax_groups_taking_turns(d):
    # 65..128 rows and a long cache: two softmax groups alternate over the tiles, merged inside the cluster ...
    _case(B=1, Hq=16, Hkv=16, T=100, d=d, Ls=[6000], dtype="bf16", seed=11)
    # ... an odd number of tiles per split, GQA rows (2 heads x 50 nodes), padded trees ...
    _case(B=2, Hq=16, Hkv=8, T=50, d=d, Ls=[5000, 4321], dtype="bf16", seed=12, n_nodes=[50, 33])
    # ... and a grid of few heads, which stays with the 8 splits of a cluster
    _case(B=1, Hq=4, Hkv=4, T=100, d=d, Ls=[20000], dtype="bf16", seed=13)


@pytest.mark.parametrize("d", [64, 128])
def test_two_row_tiles_of_few_heads_on_a_long_cache_merge_through_the_workspace(d):
    # 256 query rows per KV head, 2 KV heads, 386 tiles: 64 splits, partial results in the caller's workspace, second kernel
    _case(B=1, Hq=8, Hkv=2, T=64, d=d, Ls=[24600], dtype="bf16", seed=14)


@pytest.mark.parametrize("T", [20, 50, 100])
def test_grids_of_several_waves_share_an_sm_between_two_ctas(T):
    # 320 CTAs on 148 SMs: the launch takes the half-SM configuration (with 4, 2 and no row copies)
    _case(B=10, Hq=32, Hkv=32, T=T, d=128, Ls=[300, 17, 0, 640, 129, 300, 64, 511, 1, 77], dtype="bf16", seed=21 + T)


def _sampled_heads_case(B, Hq, Hkv, T, L, seed, kv_heads, seqs, C=None, max_cache_len=0, Ls=None):
    """The launch runs at full size (the grid, splits and kernel variant the benchmark times); the oracle checks the
    sampled (sequence, KV head) pairs, all their query heads and all their tree nodes, element by element.
    ``C``: cache capacity (default: as tight as L + T allows); ``max_cache_len``: the host's hint; ``Ls``: per-sequence
    lengths (default: L everywhere)."""
    from paper_2506_14158_b200 import s4c
    import oracle

    d, G = 128, Hq // Hkv
    C = C or (L + T + 127) // 128 * 128
    g = torch.Generator(device="cuda").manual_seed(seed)
    q = torch.randn((B, Hq, T, d), generator=g, device="cuda").bfloat16()
    k = torch.randn((B, Hkv, C, d), generator=g, device="cuda").bfloat16()
    v = torch.randn((B, Hkv, C, d), generator=g, device="cuda").bfloat16()
    rng = np.random.default_rng(seed)
    parent = np.stack([W.random_tree(T, 8, rng) for _ in range(B)])
    cl = np.full(B, L, dtype=np.int32) if Ls is None else np.asarray(Ls, dtype=np.int32)
    status = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    out = s4c.tree_attention(q, k, v, torch.from_numpy(cl).cuda(), torch.from_numpy(parent).cuda(), status=status,
                             max_cache_len=max_cache_len)
    torch.cuda.synchronize()
    assert (status.cpu().numpy() == 0).all()
    assert torch.isfinite(out.float()).all()
    worst = 0.0
    for b in seqs:
        for hk in kv_heads:
            qs = q[b:b + 1, hk * G:(hk + 1) * G].cpu()
            ks, vs = k[b:b + 1, hk:hk + 1].cpu(), v[b:b + 1, hk:hk + 1].cpu()
            ref, st = oracle.tree_attention(W.to_f64(qs), W.to_f64(ks), W.to_f64(vs), cl[b:b + 1], parent[b:b + 1])
            got = out[b:b + 1, hk * G:(hk + 1) * G].double().cpu().numpy()
            worst = max(worst, float(np.abs(got - ref).max()))
    assert worst <= ATTN_TOL["bf16"], f"max-abs error {worst:.3e}"


@pytest.mark.parametrize("name,B,Hq,Hkv,T,L,kv_heads,seqs", [
    ("sweep B1 T64 L32768: 4 splits in a cluster, 2 row copies", 1, 32, 32, 64, 32768, [0, 13, 31], [0]),
    ("sweep B1 T128 L32768: two softmax groups taking turns", 1, 32, 32, 128, 32768, [5, 31], [0]),
    ("sweep B16 T32 L4096: half-SM CTAs, 512 CTAs", 16, 32, 32, 32, 4096, [0, 17], [0, 9, 15]),
    ("sweep B4 T16 L8192: one split, 4 row copies", 4, 32, 32, 16, 8192, [3, 30], [1, 3]),
    ("8B shape at L16384: GQA, two row tiles per CTA", 4, 32, 8, 64, 16384, [0, 7], [0, 3]),
])
def test_full_size_launch_configurations_on_sampled_heads(name, B, Hq, Hkv, T, L, kv_heads, seqs):
    _sampled_heads_case(B, Hq, Hkv, T, L, seed=len(name), kv_heads=kv_heads, seqs=seqs)


# A serving cache is laid out for its longest context (C = 32768 here) while the sequences are far shorter.  The launch is
# shaped for the capacity when the host says nothing (hint 0) and for the live length when it passes its bound; a bound
# below the true length (hint 64 for a sequence of 4096) must still give the right answer.  Splits that receive no tile
# (L = 0 leaves a single tile for a cluster of 8) take part in the merge with zero weight.
@pytest.mark.parametrize("shape", ["7B", "8B"])
@pytest.mark.parametrize("L", [0, 1000, 4096])
@pytest.mark.parametrize("hint", ["none", "exact", "too small"])
def test_capacity_far_beyond_the_live_length(shape, L, hint):
    B, Hq, Hkv, T = (1, 32, 32, 26) if shape == "7B" else (4, 32, 8, 64)
    mcl = {"none": 0, "exact": max(L, 1), "too small": 64}[hint]
    _sampled_heads_case(B, Hq, Hkv, T, L, seed=100 + L % 97 + len(shape), kv_heads=[0, Hkv - 1], seqs=[0, B - 1], C=32768,
                        max_cache_len=mcl)


def test_capacity_far_beyond_ragged_live_lengths():
    # one batch, lengths from empty to 4096, capacity 32768, the bound the host would know (the longest sequence)
    _sampled_heads_case(4, 32, 8, 64, 4096, seed=77, kv_heads=[1, 6], seqs=[0, 1, 2, 3], C=32768, max_cache_len=4096,
                        Ls=[0, 4096, 37, 1500])


def test_the_hint_never_changes_the_result_class():
    # same inputs, three launch shapes (capacity, exact bound, a bound far too small): every one within tolerance of the
    # oracle, and the two runs with the same hint bit-identical
    cfg = W.CONFIGS["c2"]
    q, k, v = W.make_attention_inputs(cfg)
    big = torch.zeros((cfg.B, cfg.Hkv, 8192, cfg.d), dtype=k.dtype)
    kb, vb = big.clone(), big.clone()
    kb[:, :, :cfg.C], vb[:, :, :cfg.C] = k, v
    parent = W.make_trees(cfg)
    outs = []
    for mcl in (0, cfg.L, 16, cfg.L):
        got, ref, gst, rst = attention_both(q, kb, vb, [cfg.L], parent, max_cache_len=mcl)
        assert_attention_close(got, ref, gst, rst, ATTN_TOL["bf16"])
        outs.append(got)
    np.testing.assert_array_equal(outs[1], outs[3])


@pytest.mark.parametrize("B,Hq,Hkv,T,d,Ls", [
    (1, 32, 32, 26, 128, [1024]),            # the 7B shape: four row copies, pushed partials
    (4, 32, 8, 64, 128, [4096, 100, 0, 2000]),  # the 8B shape: two row tiles per CTA (GQA rows packed g * T + t)
    (2, 16, 8, 50, 64, [5000, 4321]),        # two softmax groups taking turns, GQA, d = 64
    (1, 8, 2, 64, 128, [24600]),             # merged through the workspace by the second kernel
    (10, 32, 32, 20, 128, [300, 17, 0, 640, 129, 300, 64, 511, 1, 77]),  # half-SM CTAs
    (1, 16, 2, 128, 128, [300]),             # eight row tiles, one per CTA
    (3, 4, 4, 7, 64, [5, 0, 33]),            # a single split, stored directly
])
def test_rows_layout_holds_the_same_values(B, Hq, Hkv, T, d, Ls):
    # s4c_tree_attention_rows writes out[b, t, h, :]: every element equals the [B,Hq,T,d] call's, bit for bit, padding and
    # flagged sequences included (neither call touches those rows)
    from paper_2506_14158_b200 import s4c
    from parity import Guarded, dev

    rng = np.random.default_rng(B * 100 + T)
    C = max(Ls) + T + 5
    g = torch.Generator().manual_seed(B + T)
    q = torch.randn((B, Hq, T, d), generator=g).to(torch.bfloat16).cuda()
    k = torch.randn((B, Hkv, C, d), generator=g).to(torch.bfloat16).cuda()
    v = torch.randn((B, Hkv, C, d), generator=g).to(torch.bfloat16).cuda()
    parent = np.stack([W.random_tree(T, 8, rng) for _ in range(B)]).astype(np.int32)
    n_nodes = rng.integers(max(1, T // 2), T + 1, B).astype(np.int32)
    if B >= 3:
        parent[1, min(3, T - 1)] = T - 1 if T > 4 else parent[1, min(3, T - 1)]   # sequence 1: malformed (a parent not before its child)
    cl = dev(np.asarray(Ls, dtype=np.int32))
    std = Guarded((B, Hq, T, d), torch.bfloat16, fill=-3.0)
    rows = Guarded((B, T, Hq, d), torch.bfloat16, fill=-3.0)
    st0, st1 = torch.empty(B, dtype=torch.int32, device="cuda"), torch.empty(B, dtype=torch.int32, device="cuda")
    s4c.tree_attention(q, k, v, cl, dev(parent), dev(n_nodes), out=std.t, status=st0, max_cache_len=max(Ls))
    s4c.tree_attention(q, k, v, cl, dev(parent), dev(n_nodes), out=rows.t, status=st1, max_cache_len=max(Ls), rows=True)
    torch.cuda.synchronize()
    std.check("s4c_tree_attention out"), rows.check("s4c_tree_attention_rows out")
    assert torch.equal(st0, st1)
    assert torch.equal(rows.t, std.t.permute(0, 2, 1, 3).contiguous())
    assert (std.t != -3.0).any()
