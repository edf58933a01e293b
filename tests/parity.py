"""Helpers that run one seeded workload through the CUDA library (via the C ABI binding) and through the
float64 oracle, and compare them.  Used by the -m gpu tests and by the smoke check."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2506_14158_b200 import workloads as W

ATTN_TOL = {"f32": 1e-4, "bf16": 2e-2}  # max-abs bound on attention outputs (inputs ~ N(0,1))


def dev(x, device="cuda"):
    if isinstance(x, np.ndarray):
        x = torch.from_numpy(np.ascontiguousarray(x))
    return x.to(device).contiguous()


def attention_both(q, k, v, cache_len, parent, n_nodes=None, scale=0.0):
    """q,k,v CPU torch tensors in storage dtype; returns (gpu_out f64 numpy, oracle_out, gpu_status, oracle_status)."""
    from paper_2506_14158_b200 import s4c

    B = q.shape[0]
    cl = np.asarray(cache_len, dtype=np.int32)
    par = np.ascontiguousarray(parent, dtype=np.int32)
    nn = None if n_nodes is None else np.asarray(n_nodes, dtype=np.int32)
    status = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    out = torch.full(q.shape, float("nan"), dtype=q.dtype, device="cuda")
    s4c.tree_attention(dev(q), dev(k), dev(v), dev(cl), dev(par), None if nn is None else dev(nn), out=out,
                       scale=scale, status=status)
    torch.cuda.synchronize()
    ref, ref_status = oracle.tree_attention(W.to_f64(q), W.to_f64(k), W.to_f64(v), cl, par, nn, scale=float(np.float32(scale)))
    return out.double().cpu().numpy(), ref, status.cpu().numpy(), ref_status


def assert_attention_close(got, ref, gst, rst, tol):
    np.testing.assert_array_equal(gst, rst)
    ok = rst == 0
    if ok.any():
        err = np.abs(got[ok] - ref[ok])
        assert np.isfinite(got[ok]).all()
        assert err.max() <= tol, f"max-abs error {err.max():.3e} > {tol}"
    if (~ok).any():
        assert np.isnan(got[~ok]).all()  # rows of flagged sequences are left untouched


def accept_both(x, parent, temperature, n_nodes=None, max_depth=None):
    """x: dict from workloads.make_accept_inputs (numpy).  Returns (gpu dict of numpy, oracle dict)."""
    from paper_2506_14158_b200 import s4c

    par = np.ascontiguousarray(parent, dtype=np.int32)
    nn = None if n_nodes is None else np.asarray(n_nodes, dtype=np.int32)
    tau = float(np.float32(temperature))
    B, T, V = x["logits"].shape
    if max_depth is None:
        max_depth = T - 1
    if tau > 0:
        r = s4c.tree_accept(dev(x["logits"]), dev(x["draft_probs"]), dev(x["tokens"]), dev(par), tau,
                            dev(x["uniforms"]), None if nn is None else dev(nn), max_depth=max_depth)
        ref = oracle.accept_stochastic(x["logits"], x["draft_probs"], x["tokens"], par, tau, x["uniforms"], nn, max_depth)
    else:
        r = s4c.tree_accept(dev(x["logits"]), None, dev(x["tokens"]), dev(par), 0.0, None,
                            None if nn is None else dev(nn), max_depth=max_depth)
        ref = oracle.accept_greedy(x["logits"], x["tokens"], par, nn, max_depth)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in r.items()}, ref


def assert_accept_equal(got, ref, stochastic):
    """Bit-exact on every integer output.  A sequence may differ only if the oracle flagged a near tie
    (|p/q - u| < 1e-6) on it; such sequences are counted and returned, never silently dropped."""
    np.testing.assert_array_equal(got["status"], ref["status"])
    excused = 0
    for b in range(len(ref["accept_len"])):
        same = (got["accept_len"][b] == ref["accept_len"][b] and (got["path"][b] == ref["path"][b]).all()
                and got["next_token"][b] == ref["next_token"][b])
        if same:
            continue
        tie = stochastic and (ref["near_tie"][b].any() or got["near_tie"][b].any())
        assert tie, (f"sequence {b}: gpu a={got['accept_len'][b]} path={got['path'][b]} next={got['next_token'][b]} "
                     f"oracle a={ref['accept_len'][b]} path={ref['path'][b]} next={ref['next_token'][b]}")
        excused += 1
    if stochastic:
        agree = got["near_tie"] == ref["near_tie"]
        assert agree.all() or excused > 0 or ref["near_tie"].any()
    return excused


def compact_both(k_layers, v_layers, cache_len, path, accept_len, T, feat=None):
    """k_layers/v_layers: lists of CPU torch caches.  Returns (gpu (k,v,len,feat_out,status), oracle (...)) as numpy (raw bits)."""
    from paper_2506_14158_b200 import s4c

    n_layers = len(k_layers)
    B, Hkv, C, d = k_layers[0].shape
    dtype = k_layers[0].dtype
    path = np.ascontiguousarray(path, dtype=np.int32)
    accept_len = np.asarray(accept_len, dtype=np.int32)
    max_depth = path.shape[1] - 1
    bits = torch.int32 if dtype == torch.float32 else torch.int16
    kd, vd = [dev(c) for c in k_layers], [dev(c) for c in v_layers]
    cl_d = dev(np.asarray(cache_len, dtype=np.int32))
    fo_d = None
    if feat is not None:
        fo_d = torch.full((B, max_depth + 1, feat.shape[2]), 3.0, dtype=dtype, device="cuda")
    st = s4c.kv_compact(s4c.cache_pointer_array(kd), s4c.cache_pointer_array(vd), n_layers, (B, Hkv, C, d), dtype, cl_d,
                        dev(path), dev(accept_len), T, None if feat is None else dev(feat), fo_d)
    torch.cuda.synchronize()
    as_bits = lambda t: t.cpu().view(bits).numpy()
    got = ([as_bits(c) for c in kd], [as_bits(c) for c in vd], cl_d.cpu().numpy(), None if fo_d is None else as_bits(fo_d),
           st.cpu().numpy())
    kn, vn = [as_bits(c.clone()).copy() for c in k_layers], [as_bits(c.clone()).copy() for c in v_layers]
    cl = np.asarray(cache_len, dtype=np.int32).copy()
    fo = None
    fi = None
    if feat is not None:
        fi = as_bits(feat.clone()).copy()
        fo = as_bits(torch.full((B, max_depth + 1, feat.shape[2]), 3.0, dtype=dtype)).copy()
    ost = oracle.kv_compact(kn, vn, cl, path, accept_len, T, fi, fo)
    return got, (kn, vn, cl, fo, ost)


def assert_compact_equal(got, ref, old_len, T):
    gk, gv, glen, gfeat, gst = got
    rk, rv, rlen, rfeat, rst = ref
    np.testing.assert_array_equal(gst, rst)
    np.testing.assert_array_equal(glen, rlen)
    B = len(rlen)
    for l in range(len(rk)):
        for g, r in ((gk[l], rk[l]), (gv[l], rv[l])):
            for b in range(B):
                L, new = int(old_len[b]), int(rlen[b])
                np.testing.assert_array_equal(g[b, :, :max(new, L)], r[b, :, :max(new, L)])  # prefix + compacted rows
                np.testing.assert_array_equal(g[b, :, L + T:], r[b, :, L + T:])              # beyond the tree slots
    if rfeat is not None:
        np.testing.assert_array_equal(gfeat, rfeat)
