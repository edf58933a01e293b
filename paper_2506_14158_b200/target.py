"""The target model's verify pass over the tree (Section 3.2: all candidates verified in one forward pass; Section 4.1:
greedy verification), composed from the library's entry points for a LLaMA-family target (the paper's Vicuna / LLaMA
chat models):

    x0 = Embedding(tree tokens)                                  s4c_embed_gather
    a0 = rmsnorm(x0)                                             s4c_rmsnorm
    per layer l:
        q, K/V tree slots = rope(a_l Wqkv^T)                     s4c_qkv_rope / s4c_qkv_rope_same_tree (position = committed length + depth; the rotary table once per pass)
        o  = tree attention(q, cache_l)                          s4c_tree_attention_rows (tree mask from parent[]; written as rows [B*T, Hq*d])
        h  = x_l + o Wo^T,          m = rmsnorm(h)               s4c_linear_rmsnorm
        g  = silu(m Wg^T) * (m Wu^T)                             s4c_linear, gated
        x_{l+1} = h + g Wd^T,       a_{l+1} = rmsnorm(x_{l+1})   s4c_linear_rmsnorm    (the next layer's norm, or the final norm)
    greedy (Section 4.1):
    target token per node = Argmax(LM_head(a_n))                 s4c_lm_head_greedy    (no [B,T,V] logits in memory)
    longest accepted path, next token                            s4c_tree_accept_tokens
    speculative sampling (Eq. 11-12, temperature > 0):
    logits = LM_head(a_n) as float32 [B,T,V]                     s4c_lm_head_logits
    accept / reject / residual resampling along the tree         s4c_tree_accept
    accepted K/V rows of every layer -> committed slots, features of the path gathered, lengths advanced     s4c_kv_compact

Only buffers and the order of the calls live here; every step runs in the library's kernels.  The
"features" handed to the next drafting round are the last layer's output x_n (before the final norm).  Weights are the
caller's: this repository has no trained model; tests and the benchmark use seeded random weights of the paper's
models' shapes.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import torch

from . import s4c


@dataclass
class LayerWeights:
    norm1: torch.Tensor    # [H]
    qkv: torch.Tensor      # [(Hq + 2 Hkv) d, H]
    o: torch.Tensor        # [H, Hq d]
    norm2: torch.Tensor    # [H]
    gate_up: torch.Tensor  # [2 I, H]  the gate projection's rows, then the up projection's
    down: torch.Tensor     # [H, I]


@dataclass
class TargetWeights:
    embedding: torch.Tensor  # [V, H]
    layers: List[LayerWeights]
    final_norm: torch.Tensor  # [H]
    lm_head: torch.Tensor     # [V, H]


def random_weights(n_layers: int, V: int, H: int, Hq: int, Hkv: int, d: int, inter: int, device, seed: int = 0) -> TargetWeights:
    """Seeded random weights of the given shapes (bf16; projections ~ N(0, 1/fan_in), norms near one)."""
    g = torch.Generator(device=device).manual_seed(seed)
    rn = lambda *shape, s=1.0: (torch.randn(*shape, generator=g, device=device, dtype=torch.float32) * s).to(torch.bfloat16)
    nrm = lambda: (1.0 + 0.05 * torch.randn(H, generator=g, device=device, dtype=torch.float32)).to(torch.bfloat16)
    layers = [LayerWeights(norm1=nrm(), qkv=rn((Hq + 2 * Hkv) * d, H, s=H ** -0.5), o=rn(H, Hq * d, s=(Hq * d) ** -0.5), norm2=nrm(),
                           gate_up=rn(2 * inter, H, s=H ** -0.5), down=rn(H, inter, s=inter ** -0.5)) for _ in range(n_layers)]
    return TargetWeights(embedding=rn(V, H), layers=layers, final_norm=nrm(), lm_head=rn(V, H, s=H ** -0.5))


class TargetVerify:
    """Buffers for one greedy verify step of B sequences with T-node trees; ``forward`` runs the chain above and can be
    captured in a CUDA graph (all buffers are allocated here, once; the caches are the caller's and are written in place).
    ``keep`` keeps every layer's intermediate rows (for tests); otherwise two sets of row buffers alternate."""

    def __init__(self, w: TargetWeights, B: int, T: int, Hq: int, Hkv: int, d: int, C: int, k_caches, v_caches, max_depth: int,
                 eps: float = 1e-5, rope_theta: float = 10000.0, keep: bool = False, stochastic: bool = False):
        self.w, self.B, self.T, self.Hq, self.Hkv, self.d, self.C = w, B, T, Hq, Hkv, d, C
        self.eps, self.rope_theta, self.max_depth = eps, rope_theta, max_depth
        self.k_caches, self.v_caches = list(k_caches), list(v_caches)
        n = len(w.layers)
        assert len(self.k_caches) == n and len(self.v_caches) == n
        dev = w.lm_head.device
        V, H = w.lm_head.shape
        inter = w.layers[0].down.shape[1]
        R = B * T
        self.V, self.H, self.R = V, H, R
        bf = dict(dtype=torch.bfloat16, device=dev)
        i32 = dict(dtype=torch.int32, device=dev)
        sets = n if keep else 2
        rows = lambda width: [torch.empty(R, width, **bf) for _ in range(sets)]
        self.x = [torch.empty(R, H, **bf) for _ in range(sets + 1)]  # x[l]: the input of layer l (x[0]: the embeddings)
        self.a = [torch.empty(R, H, **bf) for _ in range(sets + 1)]  # its normalisation
        self.q = [torch.empty(B, Hq, T, d, **bf) for _ in range(sets)]
        self.o_in, self.h, self.m, self.act = rows(Hq * d), rows(H), rows(H), rows(inter)
        self.sets = sets
        self.status_qkv = torch.zeros(1, B, **i32)  # written by the first layer's call, timeouts of the others OR-ed in
        self.status_attn = torch.zeros(n, B, **i32)
        self.status_head = torch.zeros(1, **i32)
        self.target_token = torch.empty(R, **i32)
        self.max_logit = torch.empty(R, dtype=torch.float32, device=dev)
        self.accept_len, self.next_token, self.status_accept = torch.empty(B, **i32), torch.empty(B, **i32), torch.empty(B, **i32)
        self.path = torch.empty(B, max_depth + 1, **i32)
        self.feat_out = torch.empty(B, max_depth + 1, H, **bf)
        self.status_compact = torch.empty(B, **i32)
        self.k_ptrs, self.v_ptrs = s4c.cache_pointer_array(self.k_caches), s4c.cache_pointer_array(self.v_caches)
        u8 = lambda nbytes: torch.empty(max(1, nbytes), dtype=torch.uint8, device=dev)
        self.ws_qkv = u8(s4c.qkv_rope_workspace_bytes(B, T, d))
        self.ws_attn = u8(s4c.tree_attention_workspace_bytes(B, T, Hq, Hkv, d, C, torch.bfloat16))
        self.ws_head = u8(s4c.lm_head_greedy_workspace_bytes(R, V, H))
        self.stochastic = stochastic
        if stochastic:  # the logits exist in memory only on this route
            self.logits = torch.empty(B, T, V, dtype=torch.float32, device=dev)
            self.near_tie = torch.empty(B, T, dtype=torch.uint8, device=dev)
            self.ws_logits = u8(s4c.lm_head_logits_workspace_bytes(R, V, H))
            self.ws_accept = u8(s4c.tree_accept_workspace_bytes(B, T, V))
        self.ws_lin = u8(max(s4c.linear_workspace_bytes(R, Hq * d, 0, H), s4c.linear_workspace_bytes(R, H, 0, inter, True),
                             s4c.linear_workspace_bytes(R, inter, 0, H)))  # the products run one after another

    def forward(self, tokens: torch.Tensor, cache_len: torch.Tensor, parent: torch.Tensor, n_nodes: Optional[torch.Tensor] = None,
                max_cache_len: int = 0, compact: bool = True, temperature: float = 0.0, draft_probs: Optional[torch.Tensor] = None,
                uniforms: Optional[torch.Tensor] = None):
        """tokens, parent [B,T] int32 (the tree), cache_len [B] int32 (advanced in place when ``compact``).
        temperature > 0 (a pass built with ``stochastic=True``): speculative sampling against draft_probs [B,T,V] float32 (row n: the
        drafter's distribution after node n) with the caller's uniforms (as s4c_tree_accept takes them).
        Returns dict(accept_len, path, next_token, target_token [B,T] (greedy route), features [B,max_depth+1,H], status)."""
        w, B, T = self.w, self.B, self.T
        n = len(w.layers)
        s4c.embed_gather(w.embedding, tokens.reshape(-1), out=self.x[0])
        s4c.rmsnorm(self.x[0], w.layers[0].norm1, self.eps, out=self.a[0])
        for l, lw in enumerate(w.layers):
            i, i_in, i_out = l % self.sets, l % (self.sets + 1), (l + 1) % (self.sets + 1)
            if l == 0:  # tree checks, cache positions and the rotary table: once per pass, the other layers reuse them
                s4c.qkv_rope(self.a[i_in].view(B, T, -1), lw.qkv, cache_len, parent, self.q[i], self.k_caches[l], self.v_caches[l], n_nodes,
                             self.rope_theta, status=self.status_qkv[0], workspace=self.ws_qkv)
            else:
                s4c.qkv_rope_same_tree(self.a[i_in].view(B, T, -1), lw.qkv, self.q[i], self.k_caches[l], self.v_caches[l], self.ws_qkv,
                                       status=self.status_qkv[0])
            s4c.tree_attention(self.q[i], self.k_caches[l], self.v_caches[l], cache_len, parent, n_nodes,
                               out=self.o_in[i].view(B, T, self.Hq, self.d), status=self.status_attn[l], workspace=self.ws_attn,
                               max_cache_len=max_cache_len, rows=True)
            s4c.linear_rmsnorm(self.o_in[i], lw.o, lw.norm2, self.eps, residual=self.x[i_in], out=self.h[i], norm_out=self.m[i],
                               workspace=self.ws_lin)
            s4c.linear(self.m[i], lw.gate_up, gate=True, out=self.act[i], workspace=self.ws_lin)
            next_norm = w.layers[l + 1].norm1 if l + 1 < n else w.final_norm
            s4c.linear_rmsnorm(self.act[i], lw.down, next_norm, self.eps, residual=self.h[i], out=self.x[i_out], norm_out=self.a[i_out],
                               workspace=self.ws_lin)
        last = n % (self.sets + 1)
        self.last = last
        if temperature > 0.0:
            if not self.stochastic:
                raise ValueError("build the pass with stochastic=True to verify by speculative sampling")
            s4c.lm_head_logits(self.a[last], w.lm_head, self.logits.view(self.R, self.V), self.status_head, self.ws_logits)
            s4c.tree_accept(self.logits, draft_probs, tokens, parent, temperature, uniforms, n_nodes, self.max_depth, self.accept_len,
                            self.path, self.next_token, self.near_tie, self.status_accept, self.ws_accept)
        else:
            s4c.lm_head_greedy(self.a[last], w.lm_head, self.target_token, self.max_logit, self.status_head, self.ws_head)
            s4c.tree_accept_tokens(self.target_token.view(B, T), tokens, parent, self.V, n_nodes, self.max_depth, self.accept_len,
                                   self.path, self.next_token, self.status_accept)
        if compact:
            s4c.kv_compact(self.k_ptrs, self.v_ptrs, n, (B, self.Hkv, self.C, self.d), torch.bfloat16, cache_len, self.path,
                           self.accept_len, T, feat_in=self.x[last].view(B, T, -1), feat_out=self.feat_out,
                           status=self.status_compact)
        return dict(accept_len=self.accept_len, path=self.path, next_token=self.next_token, target_token=self.target_token.view(B, T),
                    features=self.feat_out, status=self.status_accept)
