"""Host-side checks of the C ABI: the library loads, exports everything include/s4c.h declares, sizes its
workspaces on the host and rejects bad arguments before touching CUDA.  No kernel is launched here."""
import ctypes
import os
import re

import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "s4c.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(s4c_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(s4c_lib):
    lib = ctypes.CDLL(s4c_lib)
    names = _declared_functions()
    assert "s4c_tree_attention" in names and "s4c_tree_accept" in names and "s4c_kv_compact" in names
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in include/s4c.h but not exported"
    from paper_2506_14158_b200 import s4c

    assert sorted(s4c.EXPORTS) == names
    assert s4c.version() >= 100


def test_sequence_flags_agree_between_header_binding_and_oracle(s4c_lib):
    from paper_2506_14158_b200 import s4c

    text = open(os.path.join(ROOT, "include", "s4c.h")).read()
    flags = {k: int(v) for k, v in re.findall(r"#define\s+S4C_(SEQ_[A-Z_]+)\s+(\d+)", text)}
    assert flags == {"SEQ_OK": 0, "SEQ_BAD_PARENT": 1, "SEQ_TOKEN_RANGE": 2, "SEQ_CAPACITY": 4, "SEQ_DEPTH": 8,
                     "SEQ_BAD_PATH": 16, "SEQ_TIMEOUT": 32, "SEQ_NONFINITE": 64, "SEQ_BAD_PAGE": 128}
    for k, v in flags.items():
        assert getattr(s4c, k) == v
        if k not in ("SEQ_TIMEOUT", "SEQ_BAD_PAGE"):  # the CPU oracle has no waits and no page tables
            assert getattr(oracle, k) == v


def test_workspace_queries_are_host_functions(s4c_lib):
    from paper_2506_14158_b200 import s4c

    assert s4c.tree_accept_workspace_bytes(1, 26, 32000) > 0
    assert s4c.tree_accept_workspace_bytes(4, 64, 128256) % 256 == 0
    assert s4c.tree_accept_workspace_bytes(0, 1, 1) == 0
    import torch

    # splits merge inside a thread-block cluster: no scratch, also for grids of few heads; only two row tiles per CTA
    # (256 query rows per KV head) on a very long cache of very few KV heads go wider than a cluster
    assert s4c.tree_attention_workspace_bytes(1, 26, 32, 32, 128, 1152, torch.bfloat16) == 0
    assert s4c.tree_attention_workspace_bytes(1, 16, 8, 8, 128, 9088, torch.bfloat16) == 0
    w = s4c.tree_attention_workspace_bytes(1, 64, 8, 2, 128, 24704, torch.bfloat16)
    assert w > 0 and w % 256 == 0
    assert s4c.tree_attention_workspace_bytes(1, 200, 32, 32, 128, 1152, torch.bfloat16) == 0  # T > 128: invalid


def test_bad_arguments_are_rejected_on_the_host(s4c_lib):
    lib = ctypes.CDLL(s4c_lib)
    vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.s4c_tree_attention.argtypes = [vp, vp, vp, vp, vp, vp, vp, i, i, i, i, i, i, i, i, f, vp, vp, sz, vp]
    lib.s4c_tree_accept.argtypes = [vp, vp, vp, vp, vp, f, vp, i, i, i, i, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.s4c_kv_compact.argtypes = [vp, vp, i, vp, vp, vp, i, vp, vp, i, i, i, i, i, i, i, vp, vp]
    lib.s4c_status_string.restype = ctypes.c_char_p
    P = 4096  # a fake, 16-byte aligned "pointer": rejected calls never dereference or launch
    att = lambda **kw: lib.s4c_tree_attention(*[kw.get(k, d) for k, d in [
        ("q", P), ("k", P), ("v", P), ("cl", P), ("par", P), ("nn", None), ("out", P), ("B", 1), ("T", 8), ("Hq", 4),
        ("Hkv", 2), ("d", 128), ("C", 256), ("hint", 0), ("dt", 1), ("scale", 0.0), ("st", None), ("ws", None), ("wsb", 0), ("s", None)]])
    assert att(q=None) == 1                      # S4C_ERR_NULL
    assert att(T=129) == 2 and att(T=0) == 2     # S4C_ERR_SHAPE
    assert att(Hq=4, Hkv=3) == 2 and att(d=96) == 2
    assert att(dt=5) == 3                        # S4C_ERR_DTYPE
    assert att(k=P + 2) == 4                     # S4C_ERR_ALIGN
    assert att(scale=-1.0) == 2 and att(hint=-1) == 2
    assert att(B=0) == 0
    assert att(T=64, Hq=8, Hkv=2, C=24704, ws=None) == 5   # this grid splits wider than a cluster and needs a workspace
    lib.s4c_tree_attention_rows.argtypes = lib.s4c_tree_attention.argtypes
    attr = lambda **kw: lib.s4c_tree_attention_rows(*[kw.get(k, d) for k, d in [
        ("q", P), ("k", P), ("v", P), ("cl", P), ("par", P), ("nn", None), ("out", P), ("B", 1), ("T", 8), ("Hq", 4),
        ("Hkv", 2), ("d", 128), ("C", 256), ("hint", 0), ("dt", 1), ("scale", 0.0), ("st", None), ("ws", None), ("wsb", 0), ("s", None)]])
    assert attr(out=None) == 1 and attr(T=129) == 2 and attr(k=P + 2) == 4 and attr(B=0) == 0
    assert attr(dt=0) == 6                       # S4C_ERR_UNSUPPORTED: the row layout is written by the bf16 kernel only
    acc = lambda **kw: lib.s4c_tree_accept(*[kw.get(k, d) for k, d in [
        ("lg", P), ("dp", P), ("tok", P), ("par", P), ("nn", None), ("tau", 1.0), ("u", P), ("B", 1), ("T", 8),
        ("V", 100), ("md", 7), ("al", P), ("path", P), ("nt", P), ("tie", None), ("st", None), ("ws", None), ("wsb", 0),
        ("s", None)]])
    assert acc(tau=-0.5) == 2 and acc(tau=float("nan")) == 2
    assert acc(dp=None) == 1 and acc(u=None) == 1 and acc(lg=None) == 1
    assert acc(T=500) == 2 and acc(V=0) == 2 and acc(md=128) == 2
    assert acc() == 5                            # no workspace
    assert acc(B=0) == 0
    cmp_ = lambda **kw: lib.s4c_kv_compact(*[kw.get(k, d) for k, d in [
        ("k", P), ("v", P), ("nl", 1), ("cl", P), ("path", P), ("al", P), ("md", 7), ("fi", None), ("fo", None), ("B", 1),
        ("T", 8), ("Hkv", 2), ("d", 128), ("C", 256), ("hid", 0), ("dt", 1), ("st", None), ("s", None)]])
    assert cmp_(cl=None) == 1 and cmp_(k=None) == 1
    assert cmp_(d=100) == 2                      # rows must be whole 16-byte words
    assert cmp_(fi=P) == 1                       # feat_in without feat_out
    assert cmp_(dt=9) == 3
    assert cmp_(B=0) == 0
    lib.s4c_tree_build.argtypes = [vp, vp, i, vp, vp, i, i, i, vp, vp, vp, vp, vp, sz, vp]
    lib.s4c_tree_build_workspace_bytes.restype = sz
    lib.s4c_tree_build_workspace_bytes.argtypes = [i, i, i, i]
    br = (ctypes.c_int32 * 3)(4, 3, 2)
    tb = lambda **kw: lib.s4c_tree_build(*[kw.get(k, d) for k, d in [
        ("q", P), ("br", ctypes.cast(br, vp)), ("D", 3), ("root", P), ("cl", None), ("B", 1), ("T", 26), ("V", 32000),
        ("tok", P), ("par", P), ("pos", P), ("nn", P), ("ws", None), ("wsb", 0), ("s", None)]])
    assert tb(q=None) == 1 and tb(nn=None) == 1 and tb(br=None) == 1
    assert tb(T=129) == 2 and tb(V=0) == 2 and tb(V=3) == 2     # V = 3: fewer tokens than the 4 children of the root
    assert tb(q=P + 4) == 4
    assert tb() == 5                                            # no workspace
    assert tb(B=0) == 0
    bad = (ctypes.c_int32 * 2)(17, 1)
    assert tb(br=ctypes.cast(bad, vp), D=2) == 2                # more than 16 children
    assert lib.s4c_tree_build_workspace_bytes(1, 26, 32000, 4) % 256 == 0 and lib.s4c_tree_build_workspace_bytes(1, 26, 32000, 4) > 0
    assert lib.s4c_tree_build_workspace_bytes(1, 26, 32000, 17) == 0
    lib.s4c_tree_accept_filtered.argtypes = [vp, vp, vp, vp, vp, f, i, f, vp, i, i, i, i, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.s4c_tree_accept_filtered_workspace_bytes.restype = sz
    lib.s4c_tree_accept_filtered_workspace_bytes.argtypes = [i, i, i, i]
    fl = lambda **kw: lib.s4c_tree_accept_filtered(*[kw.get(k, d) for k, d in [
        ("lg", P), ("dp", P), ("tok", P), ("par", P), ("nn", None), ("tau", 1.0), ("k", 50), ("p", 0.9), ("u", P), ("B", 1),
        ("T", 8), ("V", 100), ("md", 7), ("al", P), ("path", P), ("nt", P), ("tie", None), ("st", None), ("ws", None),
        ("wsb", 0), ("s", None)]])
    assert fl(lg=None) == 1 and fl(dp=None) == 1 and fl(u=None) == 1 and fl(nt=None) == 1
    assert fl(tau=0.0) == 2 and fl(tau=float("inf")) == 2 and fl(tau=float("nan")) == 2   # greedy goes through s4c_tree_accept
    assert fl(k=0) == 2 and fl(k=65) == 2 and fl(p=0.0) == 2 and fl(p=1.5) == 2 and fl(p=float("nan")) == 2
    assert fl(T=129) == 2 and fl(V=0) == 2 and fl(md=128) == 2
    assert fl(lg=P + 4) == 4
    assert fl() == 5                                            # no workspace
    assert fl(B=0) == 0
    wsb = lib.s4c_tree_accept_filtered_workspace_bytes
    assert wsb(1, 8, 32000, 50) % 256 == 0 and wsb(1, 8, 32000, 50) > 0
    assert wsb(1, 8, 32000, 65) == 0 and wsb(1, 8, 32000, 0) == 0
    assert wsb(1, 8, 10, 50) == wsb(1, 8, 10, 10)               # top_k is capped by the vocabulary
    lib.s4c_lm_head_greedy.argtypes = [vp, vp, i, i, i, vp, vp, vp, vp, sz, vp]
    lib.s4c_lm_head_greedy_workspace_bytes.restype = sz
    lib.s4c_lm_head_greedy_workspace_bytes.argtypes = [i, i, i]
    lm = lambda **kw: lib.s4c_lm_head_greedy(*[kw.get(k, d) for k, d in [
        ("h", P), ("w", P), ("R", 26), ("V", 32000), ("H", 4096), ("tok", P), ("mx", None), ("st", None), ("ws", None),
        ("wsb", 0), ("s", None)]])
    assert lm(h=None) == 1 and lm(w=None) == 1 and lm(tok=None) == 1
    assert lm(H=100) == 2 and lm(H=32) == 2 and lm(V=0) == 2 and lm(R=-1) == 2   # the hidden size comes in 64-element slices
    assert lm(w=P + 8) == 4
    assert lm() == 5                                            # no workspace
    assert lm(R=0) == 0
    assert lib.s4c_lm_head_greedy_workspace_bytes(26, 32000, 4096) % 256 == 0
    assert lib.s4c_lm_head_greedy_workspace_bytes(26, 32000, 4096) > 0 and lib.s4c_lm_head_greedy_workspace_bytes(0, 32000, 4096) == 0
    lib.s4c_tree_accept_tokens.argtypes = [vp, vp, vp, vp, i, i, i, i, vp, vp, vp, vp, vp]
    tw = lambda **kw: lib.s4c_tree_accept_tokens(*[kw.get(k, d) for k, d in [
        ("tgt", P), ("tok", P), ("par", P), ("nn", None), ("B", 1), ("T", 8), ("V", 100), ("md", 7), ("al", P), ("path", P),
        ("nt", P), ("st", None), ("s", None)]])
    assert tw(tgt=None) == 1 and tw(par=None) == 1 and tw(nt=None) == 1
    assert tw(T=129) == 2 and tw(V=0) == 2 and tw(md=128) == 2 and tw(B=-1) == 2
    assert tw(B=0) == 0
    lib.s4c_qkv_rope.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i, i, i, i, i, i, i, f, vp, vp, sz, vp]
    lib.s4c_qkv_rope_workspace_bytes.restype = sz
    lib.s4c_qkv_rope_workspace_bytes.argtypes = [i, i, i]
    qk = lambda **kw: lib.s4c_qkv_rope(*[kw.get(k, d) for k, d in [
        ("x", P), ("w", P), ("cl", P), ("par", P), ("nn", None), ("q", P), ("k", P), ("v", P), ("B", 1), ("T", 26), ("H", 4096),
        ("Hq", 32), ("Hkv", 8), ("d", 128), ("C", 2048), ("theta", 10000.0), ("st", None), ("ws", None), ("wsb", 0), ("s", None)]])
    assert qk(x=None) == 1 and qk(w=None) == 1 and qk(cl=None) == 1 and qk(k=None) == 1
    assert qk(d=96) == 2 and qk(H=100) == 2 and qk(Hkv=5) == 2 and qk(T=129) == 2 and qk(C=10) == 2
    assert qk(theta=1.0) == 2 and qk(theta=float("nan")) == 2
    assert qk(q=P + 2) == 4
    assert qk() == 5                                            # no workspace
    assert qk(B=0) == 0
    assert lib.s4c_qkv_rope_workspace_bytes(4, 64, 128) % 256 == 0 and lib.s4c_qkv_rope_workspace_bytes(4, 64, 128) > 0
    assert lib.s4c_qkv_rope_workspace_bytes(4, 64, 96) == 0
    lib.s4c_qkv_rope_at.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, i, i, i, i, i, i, i, f, vp, vp, sz, vp]
    qa = lambda **kw: lib.s4c_qkv_rope_at(*[kw.get(k, d) for k, d in [
        ("x", P), ("w", P), ("cl", P), ("pb", P), ("par", P), ("nn", None), ("q", P), ("k", P), ("v", P), ("B", 1), ("T", 26), ("H", 4096),
        ("Hq", 32), ("Hkv", 8), ("d", 128), ("C", 2048), ("theta", 10000.0), ("st", None), ("ws", None), ("wsb", 0), ("s", None)]])
    assert qa(pb=None) == 1 and qa(cl=None) == 1 and qa(d=96) == 2 and qa(q=P + 2) == 4 and qa() == 5 and qa(B=0) == 0
    lib.s4c_qkv_rope_same_tree.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, i, vp, vp, sz, vp]
    qs = lambda **kw: lib.s4c_qkv_rope_same_tree(*[kw.get(k, d) for k, d in [
        ("x", P), ("w", P), ("q", P), ("k", P), ("v", P), ("B", 1), ("T", 26), ("H", 4096), ("Hq", 32), ("Hkv", 8), ("d", 128),
        ("C", 2048), ("st", None), ("ws", None), ("wsb", 0), ("s", None)]])
    assert qs(x=None) == 1 and qs(v=None) == 1 and qs(d=96) == 2 and qs(Hkv=5) == 2 and qs(k=P + 2) == 4 and qs() == 5 and qs(B=0) == 0
    lib.s4c_lm_head_topk.argtypes = [vp, vp, i, i, i, i, vp, vp, vp, vp, sz, vp]
    lib.s4c_lm_head_topk_workspace_bytes.restype = sz
    lib.s4c_lm_head_topk_workspace_bytes.argtypes = [i, i, i, i]
    tk = lambda **kw: lib.s4c_lm_head_topk(*[kw.get(k, d) for k, d in [
        ("h", P), ("w", P), ("R", 26), ("V", 32000), ("H", 4096), ("k", 4), ("tok", P), ("lg", None), ("st", None), ("ws", None),
        ("wsb", 0), ("s", None)]])
    assert tk(h=None) == 1 and tk(tok=None) == 1 and tk(k=0) == 2 and tk(H=96) == 2
    assert tk(k=9) == 6                                         # S4C_ERR_UNSUPPORTED: at most 8 ranked choices
    assert tk() == 5 and tk(R=0) == 0
    assert lib.s4c_lm_head_topk_workspace_bytes(26, 32000, 4096, 8) > lib.s4c_lm_head_topk_workspace_bytes(26, 32000, 4096, 1) > 0
    assert lib.s4c_lm_head_topk_workspace_bytes(26, 32000, 4096, 9) == 0
    lib.s4c_tree_build_topk.argtypes = [vp, i, vp, i, vp, vp, i, i, vp, vp, vp, vp, vp]
    tbk = lambda **kw: lib.s4c_tree_build_topk(*[kw.get(k, d) for k, d in [
        ("topk", P), ("k", 4), ("br", ctypes.cast(br, vp)), ("D", 3), ("root", P), ("cl", None), ("B", 1), ("T", 26), ("tok", P),
        ("par", P), ("pos", P), ("nn", P), ("s", None)]])
    assert tbk(topk=None) == 1 and tbk(nn=None) == 1 and tbk(br=None) == 1
    assert tbk(T=129) == 2 and tbk(k=0) == 2 and tbk(k=3) == 2  # k = 3: fewer ranked choices than the 4 children of the root
    assert tbk(B=0) == 0
    lib.s4c_linear_workspace_bytes.restype = ctypes.c_size_t
    lib.s4c_linear_workspace_bytes.argtypes = [i, i, i, i, i]
    # 26 x 4096 outputs are 32 tiles: the K range is shared out and the partial sums need room; a wide output needs none
    assert lib.s4c_linear_workspace_bytes(26, 4096, 0, 4096, 0) >= 2 * 26 * 4096 * 4
    assert lib.s4c_linear_workspace_bytes(26, 4096, 0, 32768, 0) == 0 and lib.s4c_linear_workspace_bytes(26, 64, 0, 4096, 0) == 0
    lib.s4c_linear.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, i, vp, vp, ctypes.c_size_t, vp]
    ln = lambda **kw: lib.s4c_linear(*[kw.get(k, d) for k, d in [
        ("x1", P), ("x2", None), ("w", P), ("b", None), ("res", None), ("out", P), ("R", 26), ("K1", 4096), ("K2", 0), ("N", 4096),
        ("gate", 0), ("st", None), ("ws", P), ("wsb", 1 << 30), ("s", None)]])
    assert ln(x1=None) == 1 and ln(w=None) == 1 and ln(out=None) == 1 and ln(K2=4096) == 1      # a second width without a second input
    assert ln(K1=100) == 2 and ln(K2=32, x2=P) == 2 and ln(N=12) == 2 and ln(N=0) == 2 and ln(R=-1) == 2
    assert ln(w=P + 4) == 4 and ln(res=P + 2) == 4
    assert ln(ws=None) == 5 and ln(wsb=1024) == 5 and ln(ws=P + 16) == 5  # the shared-out K range needs its workspace
    assert ln(R=0) == 0
    lib.s4c_linear_rmsnorm.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, vp, f, vp, vp, vp, ctypes.c_size_t, vp]
    lnr = lambda **kw: lib.s4c_linear_rmsnorm(*[kw.get(k, d) for k, d in [
        ("x1", P), ("x2", None), ("w", P), ("b", None), ("res", None), ("out", P), ("R", 26), ("K1", 4096), ("K2", 0), ("N", 4096),
        ("g", P), ("eps", 1e-5), ("no", P), ("st", None), ("ws", P), ("wsb", 1 << 30), ("s", None)]])
    assert lnr(g=None) == 1 and lnr(no=None) == 1 and lnr(x1=None) == 1
    assert lnr(eps=-1.0) == 2 and lnr(N=12) == 2 and lnr(g=P + 2) == 4 and lnr(no=P + 8) == 4 and lnr(ws=None) == 5 and lnr(R=0) == 0
    lib.s4c_lm_head_logits.argtypes = [vp, vp, i, i, i, vp, vp, vp, ctypes.c_size_t, vp]
    lib.s4c_lm_head_logits_workspace_bytes.restype = ctypes.c_size_t
    lib.s4c_lm_head_logits_workspace_bytes.argtypes = [i, i, i]
    lg = lambda **kw: lib.s4c_lm_head_logits(*[kw.get(k, d) for k, d in [
        ("h", P), ("w", P), ("R", 26), ("V", 32000), ("H", 4096), ("out", P), ("st", None), ("ws", P), ("wsb", 1 << 30), ("s", None)]])
    assert lg(h=None) == 1 and lg(out=None) == 1 and lg(V=32001) == 2 and lg(H=100) == 2 and lg(out=P + 4) == 4 and lg(R=0) == 0
    assert lib.s4c_lm_head_logits_workspace_bytes(26, 32000, 4096) == lib.s4c_linear_workspace_bytes(26, 4096, 0, 32000, 0)
    lib.s4c_rmsnorm.argtypes = [vp, vp, f, i, i, vp, vp]
    rn = lambda **kw: lib.s4c_rmsnorm(*[kw.get(k, d) for k, d in [("x", P), ("g", P), ("eps", 1e-6), ("R", 4), ("H", 4096), ("out", P), ("s", None)]])
    assert rn(x=None) == 1 and rn(H=12) == 2 and rn(eps=-1.0) == 2 and rn(g=P + 2) == 4 and rn(R=0) == 0
    lib.s4c_embed_gather.argtypes = [vp, vp, i, i, i, vp, vp]
    eg = lambda **kw: lib.s4c_embed_gather(*[kw.get(k, d) for k, d in [("tab", P), ("tok", P), ("R", 4), ("V", 100), ("H", 64), ("out", P), ("s", None)]])
    assert eg(tok=None) == 1 and eg(V=0) == 2 and eg(H=4) == 2 and eg(out=P + 8) == 4 and eg(R=0) == 0
    assert b"workspace" in lib.s4c_status_string(5)
