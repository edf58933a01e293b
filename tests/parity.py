"""Helpers that run one seeded workload through the CUDA library (via the C ABI binding) and through the
float64 oracle, and compare them.  Used by the -m gpu tests and by the smoke check."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2506_14158_b200 import workloads as W

ATTN_TOL = {"f32": 1e-4, "bf16": 2e-2}  # max-abs bound on attention outputs (inputs ~ N(0,1))


class Guarded:
    """A device tensor with a pattern-filled guard region on either side (in place of a memory checker): the library
    must write inside the tensor only.  ``check()`` asserts that both guards still hold the pattern."""
    PAD, BYTE = 4096, 0xA5

    def __init__(self, shape, dtype, fill=None, src=None, device="cuda"):
        shape = tuple(int(x) for x in shape)
        self.nbytes = int(np.prod(shape, dtype=np.int64)) * torch.empty((), dtype=dtype).element_size()
        body = (self.nbytes + 255) // 256 * 256
        self.raw = torch.full((self.PAD + body + self.PAD,), self.BYTE, dtype=torch.uint8, device=device)
        self.t = self.raw[self.PAD:self.PAD + self.nbytes].view(dtype).view(shape)
        if src is not None:
            self.t.copy_(src)
        elif fill is not None:
            self.t.fill_(fill)

    def check(self, what="buffer"):
        lo, hi = self.raw[:self.PAD], self.raw[self.PAD + self.nbytes:]
        assert bool((lo == self.BYTE).all()), f"{what}: bytes before the tensor were overwritten"
        assert bool((hi == self.BYTE).all()), f"{what}: bytes after the tensor were overwritten"


def dev(x, device="cuda"):
    if isinstance(x, np.ndarray):
        x = torch.from_numpy(np.ascontiguousarray(x))
    return x.to(device).contiguous()


def attention_both(q, k, v, cache_len, parent, n_nodes=None, scale=0.0, max_cache_len=0):
    """q,k,v CPU torch tensors in storage dtype; returns (gpu_out f64 numpy, oracle_out, gpu_status, oracle_status).
    The output, the status words, the workspace and the caches sit between guard regions that are checked afterwards."""
    from paper_2506_14158_b200 import s4c

    B, Hq, T, d = q.shape
    _, Hkv, C, _ = k.shape
    cl = np.asarray(cache_len, dtype=np.int32)
    par = np.ascontiguousarray(parent, dtype=np.int32)
    nn = None if n_nodes is None else np.asarray(n_nodes, dtype=np.int32)
    status = Guarded((B,), torch.int32, fill=-1)
    out = Guarded(q.shape, q.dtype, fill=float("nan"))
    kd, vd = Guarded(k.shape, k.dtype, src=k), Guarded(v.shape, v.dtype, src=v)
    ws = Guarded((max(256, s4c.tree_attention_workspace_bytes(B, T, Hq, Hkv, d, C, q.dtype)),), torch.uint8, fill=0)
    s4c.tree_attention(dev(q), kd.t, vd.t, dev(cl), dev(par), None if nn is None else dev(nn), out=out.t,
                       scale=scale, status=status.t, workspace=ws.t, max_cache_len=max_cache_len)
    torch.cuda.synchronize()
    for g, what in ((status, "status"), (out, "out"), (kd, "k_cache"), (vd, "v_cache"), (ws, "workspace")):
        g.check("s4c_tree_attention " + what)
    assert torch.equal(kd.t.cpu().view(torch.int16 if k.dtype == torch.bfloat16 else torch.int32),
                       k.view(torch.int16 if k.dtype == torch.bfloat16 else torch.int32)), "k_cache was modified"
    ref, ref_status = oracle.tree_attention(W.to_f64(q), W.to_f64(k), W.to_f64(v), cl, par, nn, scale=float(np.float32(scale)))
    return out.t.double().cpu().numpy(), ref, status.t.cpu().numpy(), ref_status


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
    i32 = torch.int32
    g = dict(accept_len=Guarded((B,), i32, fill=-9), path=Guarded((B, max_depth + 1), i32, fill=-9),
             next_token=Guarded((B,), i32, fill=-9), near_tie=Guarded((B, T), torch.uint8, fill=7),
             status=Guarded((B,), i32, fill=-9),
             workspace=Guarded((max(256, s4c.tree_accept_workspace_bytes(B, T, V)),), torch.uint8, fill=0))
    kw = dict(max_depth=max_depth, accept_len=g["accept_len"].t, path=g["path"].t, next_token=g["next_token"].t,
              near_tie=g["near_tie"].t, status=g["status"].t, workspace=g["workspace"].t)
    if tau > 0:
        r = s4c.tree_accept(dev(x["logits"]), dev(x["draft_probs"]), dev(x["tokens"]), dev(par), tau,
                            dev(x["uniforms"]), None if nn is None else dev(nn), **kw)
        ref = oracle.accept_stochastic(x["logits"], x["draft_probs"], x["tokens"], par, tau, x["uniforms"], nn, max_depth)
    else:
        r = s4c.tree_accept(dev(x["logits"]), None, dev(x["tokens"]), dev(par), 0.0, None,
                            None if nn is None else dev(nn), **kw)
        ref = oracle.accept_greedy(x["logits"], x["tokens"], par, nn, max_depth)
    torch.cuda.synchronize()
    for name, buf in g.items():
        buf.check("s4c_tree_accept " + name)
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
        continue
    if stochastic:  # the near-tie report itself must agree on every sequence that was not excused above
        for b in range(len(ref["accept_len"])):
            same = (got["accept_len"][b] == ref["accept_len"][b] and (got["path"][b] == ref["path"][b]).all()
                    and got["next_token"][b] == ref["next_token"][b])
            if same:
                np.testing.assert_array_equal(got["near_tie"][b], ref["near_tie"][b], err_msg=f"near_tie of sequence {b}")
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
    # every buffer the call may write sits between guard regions (checked below)
    kg, vg = [Guarded(c.shape, dtype, src=c) for c in k_layers], [Guarded(c.shape, dtype, src=c) for c in v_layers]
    kd, vd = [g.t for g in kg], [g.t for g in vg]
    cl_g = Guarded((B,), torch.int32, src=torch.from_numpy(np.asarray(cache_len, dtype=np.int32)))
    cl_d = cl_g.t
    st_g = Guarded((B,), torch.int32, fill=-9)
    fo_d, fo_g = None, None
    if feat is not None:
        fo_g = Guarded((B, max_depth + 1, feat.shape[2]), dtype, fill=3.0)
        fo_d = fo_g.t
    st = s4c.kv_compact(s4c.cache_pointer_array(kd), s4c.cache_pointer_array(vd), n_layers, (B, Hkv, C, d), dtype, cl_d,
                        dev(path), dev(accept_len), T, None if feat is None else dev(feat), fo_d, status=st_g.t)
    torch.cuda.synchronize()
    for g in kg + vg + [cl_g, st_g] + ([fo_g] if fo_g is not None else []):
        g.check("s4c_kv_compact")
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
