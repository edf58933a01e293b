"""Seeded synthetic inputs for the S4C verify step (trees, Q/K/V, logits, draft probabilities, uniforms).

This module only *prepares inputs*.  It holds none of the verify step's arithmetic (no attention,
no acceptance, no compaction) and imports neither the CUDA binding nor the CPU oracle, so both
sides can be fed identical bytes.  Everything is generated on the CPU from fixed seeds and
rounded to its storage dtype before anyone reads it.

The shapes stand in for the paper's workloads (Vicuna / LLaMA-2 7B and 13B layers, a Llama-3-8B
GQA layer, Section 4.1); the datasets and weights themselves are not used.  Trees follow the
construction of Section 3.2: the top-1 chain is laid down first ("vertically"), then siblings
are added depth by depth ("horizontally"), and nodes are renumbered breadth-first so that
``parent[i] < i`` and siblings are contiguous in rank order.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Optional, Sequence, Tuple

import numpy as np
import torch

BASE_SEED = 14158
_STREAMS = {"tree": 0, "tokens": 1, "logits": 2, "noise": 3, "uniforms": 4, "q": 5, "kv": 6, "feat": 7, "lm_head": 8, "qkv": 9}


def stream_seed(config_id: int, stream: str, extra: int = 0) -> int:
    """One independent seed per (config, input stream, layer/sequence index)."""
    return BASE_SEED * 1000 + 100 * config_id + _STREAMS[stream] + 1_000_003 * extra


# --------------------------------------------------------------------------- trees
def _bfs_renumber(parent: Sequence[int]) -> np.ndarray:
    n = len(parent)
    children = [[] for _ in range(n)]
    for i in range(1, n):
        children[parent[i]].append(i)
    order, head = [0], 0
    while head < len(order):
        order.extend(children[order[head]])
        head += 1
    new_id = {old: new for new, old in enumerate(order)}
    out = np.full(n, -1, dtype=np.int32)
    for old in range(1, n):
        out[new_id[old]] = new_id[parent[old]]
    return out


def tree_from_branching(branching: Sequence[int], T: int) -> np.ndarray:
    """Vertical-first tree: top-1 chain of depth len(branching), then siblings depth by depth, cut at T nodes."""
    D = len(branching)
    parent, depth, nchild = [-1], [0], [0]

    def add(p):
        parent.append(p)
        depth.append(depth[p] + 1)
        nchild.append(0)
        nchild[p] += 1

    tip = 0
    for _ in range(D):
        if len(parent) >= T:
            break
        add(tip)
        tip = len(parent) - 1
    for lvl in range(1, D + 1):
        for node in range(len(parent)):
            if depth[node] != lvl - 1:
                continue
            while nchild[node] < branching[lvl - 1] and len(parent) < T:
                add(node)
        # nodes appended during this level have depth lvl and are visited at the next level
    return _bfs_renumber(parent[:T])


def random_tree(T: int, max_depth: int, rng: np.random.Generator, kmin: int = 1, kmax: int = 4) -> np.ndarray:
    """Breadth-first growth: each popped node shallower than max_depth draws a child count in kmin..kmax."""
    parent, depth = [-1], [0]
    head = 0
    while len(parent) < T:
        if head >= len(parent):  # every frontier node was at max depth: restart from the root
            head = 0
        node = head
        head += 1
        if depth[node] >= max_depth:
            continue
        k = int(rng.integers(kmin, kmax + 1))
        for _ in range(k):
            if len(parent) >= T:
                break
            parent.append(node)
            depth.append(depth[node] + 1)
    return _bfs_renumber(parent)


def chain_tree(T: int) -> np.ndarray:
    return np.arange(-1, T - 1, dtype=np.int32)


def star_tree(T: int) -> np.ndarray:
    p = np.zeros(T, dtype=np.int32)
    p[0] = -1
    return p


def tree_depths(parent: np.ndarray) -> np.ndarray:
    d = np.zeros(len(parent), dtype=np.int32)
    for i in range(1, len(parent)):
        d[i] = d[parent[i]] + 1
    return d


def children_of(parent: np.ndarray, node: int) -> list:
    return [i for i in range(1, len(parent)) if parent[i] == node]


# --------------------------------------------------------------------------- configs
@dataclass(frozen=True)
class VerifyConfig:
    name: str
    config_id: int
    B: int
    Hq: int
    Hkv: int
    d: int
    dtype: str  # storage dtype of Q/K/V/features: "f32" or "bf16"
    L: int  # committed cache length per sequence
    T: int  # tree nodes including the root
    tree: str  # "branching" or "random"
    branching: Tuple[int, ...] = ()
    max_tree_depth: int = 8
    V: int = 32000
    logit_sigma: float = 3.0
    draft: str = "noisy"  # "noisy": q = softmax((logits + N(0,1))/tau); "independent": own logits
    n_layers: int = 1
    hid: int = 4096
    temperatures: Tuple[float, ...] = (0.0, 1.0)
    capacity: int = 0  # cache capacity in slots; 0: as tight as the step allows (see C)

    @property
    def C(self) -> int:
        """Cache capacity in slots: `capacity` if set (a serving cache laid out for its longest context), else L + T
        rounded up to a multiple of 128."""
        tight = (self.L + self.T + 127) // 128 * 128
        if self.capacity:
            assert self.capacity >= self.L + self.T, "capacity below L + T"
            return self.capacity
        return tight

    @property
    def max_depth(self) -> int:
        return len(self.branching) if self.tree == "branching" else self.max_tree_depth


CONFIGS = {
    "c1": VerifyConfig("c1", 1, B=1, Hq=4, Hkv=4, d=64, dtype="f32", L=128, T=15, tree="branching",
                       branching=(3, 2, 1), V=1000, logit_sigma=2.0, draft="independent", hid=256),
    "c2": VerifyConfig("c2", 2, B=1, Hq=32, Hkv=32, d=128, dtype="bf16", L=1024, T=26, tree="branching",
                       branching=(4, 3, 2, 2, 1), V=32000, hid=4096),
    "c3": VerifyConfig("c3", 3, B=1, Hq=40, Hkv=40, d=128, dtype="bf16", L=2048, T=60, tree="random",
                       max_tree_depth=6, V=32000, hid=5120, temperatures=(0.7,)),
    "c4": VerifyConfig("c4", 4, B=4, Hq=32, Hkv=8, d=128, dtype="bf16", L=4096, T=64, tree="random",
                       max_tree_depth=8, V=128256, hid=4096),
}
CONFIGS["c2x32"] = replace(CONFIGS["c2"], name="c2x32", config_id=5, n_layers=32)
CONFIGS["c4x32"] = replace(CONFIGS["c4"], name="c4x32", config_id=6, n_layers=32)


def sweep_config(L: int, T: int, B: int, n_layers: int = 32) -> VerifyConfig:
    """A point of the full-depth sweep: the 7B layer shape stacked n_layers times, random trees of T nodes."""
    return replace(CONFIGS["c2"], name=f"c5_L{L}_T{T}_B{B}", config_id=7, L=L, T=T, B=B, n_layers=n_layers,
                   tree="random", max_tree_depth=8, branching=())


# --------------------------------------------------------------------------- tensors
def _torch_dtype(name: str):
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def _randn(shape, seed: int, dtype, device="cpu") -> torch.Tensor:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return torch.randn(shape, generator=g, dtype=torch.float32).to(dtype)


def make_trees(cfg: VerifyConfig) -> np.ndarray:
    """parent[B,T] int32."""
    out = np.zeros((cfg.B, cfg.T), dtype=np.int32)
    for b in range(cfg.B):
        if cfg.tree == "branching":
            out[b] = tree_from_branching(cfg.branching, cfg.T)
        else:
            rng = np.random.default_rng(stream_seed(cfg.config_id, "tree", b))
            out[b] = random_tree(cfg.T, cfg.max_tree_depth, rng)
    return out


def make_attention_inputs(cfg: VerifyConfig, layer: int = 0):
    """(q [B,Hq,T,d], k_cache, v_cache [B,Hkv,C,d]) as CPU torch tensors in the storage dtype.

    Slots 0..L-1 hold the committed prefix, slots L..L+T-1 the tree tokens' own K/V, the rest zeros.
    """
    dt = _torch_dtype(cfg.dtype)
    q = _randn((cfg.B, cfg.Hq, cfg.T, cfg.d), stream_seed(cfg.config_id, "q", layer), dt)
    k = torch.zeros((cfg.B, cfg.Hkv, cfg.C, cfg.d), dtype=dt)
    v = torch.zeros((cfg.B, cfg.Hkv, cfg.C, cfg.d), dtype=dt)
    n = cfg.L + cfg.T
    k[:, :, :n] = _randn((cfg.B, cfg.Hkv, n, cfg.d), stream_seed(cfg.config_id, "kv", 2 * layer), dt)
    v[:, :, :n] = _randn((cfg.B, cfg.Hkv, n, cfg.d), stream_seed(cfg.config_id, "kv", 2 * layer + 1), dt)
    return q, k, v


def make_features(cfg: VerifyConfig) -> torch.Tensor:
    """feat_in [B,T,hid] in the storage dtype (the hidden state before the LM head, one row per node)."""
    return _randn((cfg.B, cfg.T, cfg.hid), stream_seed(cfg.config_id, "feat"), _torch_dtype(cfg.dtype))


def make_lm_head(cfg: VerifyConfig, device="cpu") -> torch.Tensor:
    """The LM head's weight [V, hid] in bfloat16, entries ~ N(0, 1/hid) (random: no trained weights exist here), drawn
    on ``device`` (the 8B-shaped head has 525 M entries) from this input's own seed."""
    g = torch.Generator(device=device)
    g.manual_seed(stream_seed(cfg.config_id, "lm_head"))
    w = torch.randn((cfg.V, cfg.hid), generator=g, dtype=torch.float32, device=device)
    return (w * (1.0 / float(cfg.hid) ** 0.5)).to(torch.bfloat16)


def make_qkv_weight(cfg: VerifyConfig, device="cpu") -> torch.Tensor:
    """A decoder layer's stacked projection weight [(Hq + 2 Hkv) d, hid] in bfloat16 (q heads, then k, then v), entries
    ~ N(0, 1/hid), random like the LM head's."""
    g = torch.Generator(device=device)
    g.manual_seed(stream_seed(cfg.config_id, "qkv"))
    w = torch.randn(((cfg.Hq + 2 * cfg.Hkv) * cfg.d, cfg.hid), generator=g, dtype=torch.float32, device=device)
    return (w * (1.0 / float(cfg.hid) ** 0.5)).to(torch.bfloat16)


def _softmax64(x: np.ndarray) -> np.ndarray:
    x = x.astype(np.float64)
    x = x - x.max(axis=-1, keepdims=True)
    e = np.exp(x)
    return e / e.sum(axis=-1, keepdims=True)


def make_accept_inputs(cfg: VerifyConfig, parent: np.ndarray, temperature: float, token_mode: str = "topk",
                       draft_equals_target: bool = False):
    """Target logits, draft probabilities, draft tokens and uniforms for one verify step.

    Returns dict(logits f32 [B,T,V], draft_probs f32 [B,T,V], tokens i32 [B,T], uniforms f32 [B,T]).
    ``token_mode``: "topk"  -- child j of node n carries the j-th most probable draft token of row n
                                (the construction of Section 3.2);
                    "sampled" -- children are drawn from row n without replacement.
    The draft distribution is given at the acceptance temperature (tau = 1 is used when the step is greedy).
    """
    B, T, V = cfg.B, cfg.T, cfg.V
    tau = temperature if temperature > 0 else 1.0
    rng_l = np.random.default_rng(stream_seed(cfg.config_id, "logits"))
    logits = (rng_l.standard_normal((B, T, V), dtype=np.float32) * np.float32(cfg.logit_sigma)).astype(np.float32)
    rng_n = np.random.default_rng(stream_seed(cfg.config_id, "noise"))
    draft_probs = np.empty((B, T, V), dtype=np.float32)
    for b in range(B):
        for n in range(T):
            if draft_equals_target:
                dl = logits[b, n].astype(np.float64)
            elif cfg.draft == "independent":
                dl = rng_n.standard_normal(V) * cfg.logit_sigma
            else:
                dl = logits[b, n].astype(np.float64) + rng_n.standard_normal(V)
            draft_probs[b, n] = _softmax64(dl / tau).astype(np.float32)
    rng_t = np.random.default_rng(stream_seed(cfg.config_id, "tokens"))
    tokens = np.zeros((B, T), dtype=np.int32)
    tokens[:, 0] = rng_t.integers(0, V, size=B)
    for b in range(B):
        for n in range(T):
            kids = children_of(parent[b], n)
            if not kids:
                continue
            row = draft_probs[b, n].astype(np.float64)
            if token_mode == "topk":
                top = np.argsort(-row, kind="stable")[: len(kids)]
            elif token_mode == "sampled":
                top = rng_t.choice(V, size=len(kids), replace=False, p=row / row.sum())
            else:
                raise ValueError(token_mode)
            tokens[b, kids] = top.astype(np.int32)
    rng_u = np.random.default_rng(stream_seed(cfg.config_id, "uniforms"))
    uniforms = rng_u.random((B, T), dtype=np.float32)
    uniforms = np.minimum(uniforms, np.float32(1.0) - np.float32(2.0 ** -24)).astype(np.float32)
    return dict(logits=logits, draft_probs=draft_probs, tokens=tokens, uniforms=uniforms)


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a stored tensor (f32 or bf16) to a float64 numpy array."""
    return t.detach().to("cpu").to(torch.float64).numpy()
