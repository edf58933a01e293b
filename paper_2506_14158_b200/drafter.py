"""One head of the multi-head drafter (Section 3.1.1, Eq. 3-6), composed from the library's entry points.

    e = Embedding(t)                                   s4c_embed_gather           (Eq. 6)
    h = Linear(concat[e, f])                           s4c_linear_rmsnorm, two inputs (Eq. 3)
    f' = Decoder_layer(h)                                                         (Eq. 4; one LLaMA-family layer)
         a  = rmsnorm(h)                               (the same call)
         q, K/V tree slots = rope(a Wqkv^T)            s4c_qkv_rope
         o  = tree attention(q, cache)                 s4c_tree_attention_rows (written as rows [B*T, Hq*d])
         h2 = h + o Wo^T,  m = rmsnorm(h2)             s4c_linear_rmsnorm, residual
         f' = h2 + (silu(m Wg^T) * m Wu^T) Wd^T        s4c_linear (gated), s4c_linear (residual)
    ranked choices = top-k(LM_head(f'))                s4c_lm_head_topk           (Eq. 5; k = 1 is the Argmax)

Only buffers, views and the order of the calls live here; every step runs in the library's kernels.  Weights are whatever the caller passes: this repository has no trained drafter, the
benchmark and the tests use seeded random weights of the paper's models' shapes.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import torch

from . import s4c


@dataclass
class DrafterWeights:
    embedding: torch.Tensor   # [V, H]       the target's embedding table
    fc: torch.Tensor          # [H, 2H]      Eq. 3 (columns 0..H-1 meet e, H..2H-1 meet f)
    fc_bias: Optional[torch.Tensor]  # [H] or None
    norm1: torch.Tensor       # [H]
    qkv: torch.Tensor         # [(Hq + 2 Hkv) d, H]
    o: torch.Tensor           # [H, Hq d]
    norm2: torch.Tensor       # [H]
    gate_up: torch.Tensor     # [2 I, H]     the gate projection's rows, then the up projection's
    down: torch.Tensor        # [H, I]
    lm_head: torch.Tensor     # [V, H]       the target's LM head


def random_weights(V: int, H: int, Hq: int, Hkv: int, d: int, inter: int, device, seed: int = 0) -> DrafterWeights:
    """Seeded random weights of the given shapes (bf16; projections ~ N(0, 1/fan_in), norms near one)."""
    g = torch.Generator(device=device).manual_seed(seed)
    rn = lambda *shape, s=1.0: (torch.randn(*shape, generator=g, device=device, dtype=torch.float32) * s).to(torch.bfloat16)
    return DrafterWeights(
        embedding=rn(V, H), fc=rn(H, 2 * H, s=(2 * H) ** -0.5), fc_bias=rn(H, s=0.02), norm1=(1.0 + 0.05 * rn(H).float()).to(torch.bfloat16),
        qkv=rn((Hq + 2 * Hkv) * d, H, s=H ** -0.5), o=rn(H, Hq * d, s=(Hq * d) ** -0.5),
        norm2=(1.0 + 0.05 * rn(H).float()).to(torch.bfloat16), gate_up=rn(2 * inter, H, s=H ** -0.5), down=rn(H, inter, s=inter ** -0.5),
        lm_head=rn(V, H, s=H ** -0.5))


class DrafterHead:
    """Buffers for one head's pass over the T positions of B sequences; ``forward`` runs the chain above and can be
    captured in a CUDA graph (all buffers are allocated here, once)."""

    def __init__(self, w: DrafterWeights, B: int, T: int, Hq: int, Hkv: int, d: int, C: int, k: int, eps: float = 1e-5,
                 rope_theta: float = 10000.0):
        self.w, self.B, self.T, self.Hq, self.Hkv, self.d, self.C, self.k = w, B, T, Hq, Hkv, d, C, k
        self.eps, self.rope_theta = eps, rope_theta
        dev = w.fc.device
        H = w.fc.shape[0]
        inter = w.down.shape[1]
        R = B * T
        bf = dict(dtype=torch.bfloat16, device=dev)
        self.e, self.h, self.a = torch.empty(R, H, **bf), torch.empty(R, H, **bf), torch.empty(R, H, **bf)
        self.q = torch.empty(B, Hq, T, d, **bf)
        self.o_in = torch.empty(R, Hq * d, **bf)  # the attention output as rows [B*T, Hq*d] = [B,T,Hq,d]
        self.h2, self.m = torch.empty(R, H, **bf), torch.empty(R, H, **bf)
        self.act = torch.empty(R, inter, **bf)
        self.f_out = torch.empty(R, H, **bf)
        self.token = torch.empty(R, k, dtype=torch.int32, device=dev)
        self.logit = torch.empty(R, k, dtype=torch.float32, device=dev)
        i32 = dict(dtype=torch.int32, device=dev)
        self.status_qkv, self.status_attn = torch.empty(B, **i32), torch.empty(B, **i32)
        self.status_head = torch.zeros(1, **i32)
        V = w.lm_head.shape[0]
        self.ws_qkv = torch.empty(max(1, s4c.qkv_rope_workspace_bytes(B, T, d)), dtype=torch.uint8, device=dev)
        self.ws_attn = torch.empty(max(1, s4c.tree_attention_workspace_bytes(B, T, Hq, Hkv, d, C, torch.bfloat16)), dtype=torch.uint8,
                                   device=dev)
        self.ws_head = torch.empty(max(1, s4c.lm_head_topk_workspace_bytes(R, V, H, k)), dtype=torch.uint8, device=dev)
        ws_lin = max(s4c.linear_workspace_bytes(R, H, H, H), s4c.linear_workspace_bytes(R, Hq * d, 0, H),
                     s4c.linear_workspace_bytes(R, H, 0, inter, True), s4c.linear_workspace_bytes(R, inter, 0, H))
        self.ws_lin = torch.empty(max(1, ws_lin), dtype=torch.uint8, device=dev)  # the four products run one after another

    def forward(self, tokens: torch.Tensor, features: torch.Tensor, cache_len: torch.Tensor, parent: torch.Tensor,
                k_cache: torch.Tensor, v_cache: torch.Tensor, n_nodes: Optional[torch.Tensor] = None, max_cache_len: int = 0,
                position_base: Optional[torch.Tensor] = None):
        """tokens [B,T] int32 (t_i), features [B*T, H] bf16 (f_i), the head's own K/V cache [B,Hkv,C,d] (tree slots are written),
        the tree (``parent``: positions a token may look at; a chain for plain autoregressive drafting).
        ``position_base`` [B] int32: the roots' positions in the text when the head's own cache is shorter than the text
        (s4c_qkv_rope_at); None: the cache lengths.
        Returns dict(token [B*T,k], logit [B*T,k], features [B*T,H])."""
        w = self.w
        s4c.embed_gather(w.embedding, tokens.reshape(-1), out=self.e)
        s4c.linear_rmsnorm(self.e, w.fc, w.norm1, self.eps, x2=features, bias=w.fc_bias, out=self.h, norm_out=self.a,
                           workspace=self.ws_lin)
        s4c.qkv_rope(self.a.view(self.B, self.T, -1), w.qkv, cache_len, parent, self.q, k_cache, v_cache, n_nodes, self.rope_theta,
                     status=self.status_qkv, workspace=self.ws_qkv, position_base=position_base)
        s4c.tree_attention(self.q, k_cache, v_cache, cache_len, parent, n_nodes, out=self.o_in.view(self.B, self.T, self.Hq, self.d),
                           status=self.status_attn, workspace=self.ws_attn, max_cache_len=max_cache_len, rows=True)
        s4c.linear_rmsnorm(self.o_in, w.o, w.norm2, self.eps, residual=self.h, out=self.h2, norm_out=self.m, workspace=self.ws_lin)
        s4c.linear(self.m, w.gate_up, gate=True, out=self.act, workspace=self.ws_lin)
        s4c.linear(self.act, w.down, residual=self.h2, out=self.f_out, workspace=self.ws_lin)
        s4c.lm_head_topk(self.f_out, w.lm_head, self.k, token=self.token, logit=self.logit, status=self.status_head,
                         workspace=self.ws_head)
        return dict(token=self.token, logit=self.logit, features=self.f_out)


class MultiHeadDrafter:
    """One drafting round of the multi-head drafter (Section 3.1.1, Figure 2) that fills the continuous verification tree
    (Section 3.2, Figure 3) level by level.

    The tree's shape is fixed by (branching, T).  Head j (weights of its own, K/V cache of its own) runs once over the nodes of
    depth j, all of them in one pass and independent of each other -- a row per node, every row a sequence of its own for
    the attention call (T = 1), so a head's cache holds one copy of the prefix per row of its level.  A row's input is
    (Embedding(the node's token), the output feature of the node's parent); for depth 1 that parent is the root and its
    feature is the target's f_0, shared by all of the root's candidates.  The head's ranked choices give the node's children
    their tokens (child r = the r-th choice): `s4c_tree_build_topk` is called after every head on the choices known so far.
    A row's rotary position is root_position + depth (`position_base` of `s4c_qkv_rope_at`); its cache slot counts the
    head's own entries.

    Only buffers, the static row maps and the order of the calls live here; the per-row work is `DrafterHead`'s chain of
    library calls, the feature hand-over between levels is `s4c_embed_gather` with the previous level's features as its table.
    """

    def __init__(self, heads, B: int, T: int, branching, Hq: int, Hkv: int, d: int, C: int, k: int, eps: float = 1e-5,
                 rope_theta: float = 10000.0):
        assert k >= max(branching)
        self.B, self.T, self.k, self.branching = B, T, k, [int(x) for x in branching]
        dev = heads[0].fc.device
        i32 = dict(dtype=torch.int32, device=dev)
        self.H = heads[0].fc.shape[0]
        # the shape, from the library's own tree builder (any choices give the same parents)
        self.topk_all = torch.zeros(B, T, k, **i32)
        self.tree = s4c.tree_build_topk(self.topk_all, self.branching, torch.zeros(B, **i32))
        torch.cuda.synchronize()
        parent = self.tree["parent"][0].cpu().tolist()
        n = int(self.tree["n_nodes"][0].item())
        depth = [0] * n
        for i in range(1, n):
            depth[i] = depth[parent[i]] + 1
        self.levels = []  # (first node, one past the last) of depth 1, 2, ...: breadth-first numbering keeps a depth together
        for j in range(1, max(depth) + 1 if n > 1 else 1):
            nodes = [i for i in range(n) if depth[i] == j]
            assert nodes == list(range(nodes[0], nodes[-1] + 1))
            self.levels.append((nodes[0], nodes[-1] + 1))
        self.n_passes = min(len(heads), len(self.levels))  # leaves below the last head's level get tokens, no pass
        self.heads, self.parent_rows, self.minus_one, self.feat_in = [], [], [], []
        for j in range(self.n_passes):
            s, e = self.levels[j]
            nj = e - s
            self.heads.append(DrafterHead(heads[j], B * nj, 1, Hq, Hkv, d, C, k, eps, rope_theta))
            if j == 0:
                rows = [b for b in range(B) for _ in range(nj)]  # the root's feature f_0[b], reused by all its candidates
            else:
                ps, pe = self.levels[j - 1]
                rows = [b * (pe - ps) + parent[i] - ps for b in range(B) for i in range(s, e)]
            self.parent_rows.append(torch.tensor(rows, **i32))
            self.minus_one.append(torch.full((B * nj, 1), -1, **i32))
            self.feat_in.append(torch.empty(B * nj, self.H, dtype=torch.bfloat16, device=dev))
        self.tok_rows = [torch.empty(B * (e - s), 1, **i32) for s, e in self.levels[: self.n_passes]]
        self.pos_rows = [torch.empty(B * (e - s), **i32) for s, e in self.levels[: self.n_passes]]

    def draft(self, root_token: torch.Tensor, f0: torch.Tensor, target_topk: torch.Tensor, root_position: torch.Tensor, caches):
        """root_token [B] int32 (the last committed token), f0 [B,H] bf16 (the target's feature that produced the candidates),
        target_topk [B,k] int32 (the target's ranked candidates for the next token), root_position [B] int32, caches: per head
        (k_cache, v_cache, cache_len) with one sequence per row of the head's level ([B * n_j, Hkv, C, d], [B * n_j] int32).
        Returns dict(tokens, parent, position, n_nodes) of the tree and the heads' features per level."""
        B, k = self.B, self.k
        self.topk_all[:, 0, :].copy_(target_topk)
        tree = s4c.tree_build_topk(self.topk_all, self.branching, root_token, root_position, **self.tree)
        feats_prev = f0
        features = []
        for j in range(self.n_passes):
            s, e = self.levels[j]
            nj = e - s
            self.tok_rows[j].view(B, nj).copy_(tree["tokens"][:, s:e])
            self.pos_rows[j].view(B, nj).copy_(tree["position"][:, s:e])  # root_position + depth
            s4c.embed_gather(feats_prev, self.parent_rows[j], out=self.feat_in[j])
            kc, vc, cl = caches[j]
            out = self.heads[j].forward(self.tok_rows[j], self.feat_in[j], cl, self.minus_one[j], kc, vc, position_base=self.pos_rows[j])
            self.topk_all[:, s:e, :].copy_(out["token"].view(B, nj, k))
            feats_prev = out["features"]
            features.append(feats_prev)
            tree = s4c.tree_build_topk(self.topk_all, self.branching, root_token, root_position, **self.tree)
        return dict(tokens=tree["tokens"], parent=tree["parent"], position=tree["position"], n_nodes=tree["n_nodes"], features=features)
