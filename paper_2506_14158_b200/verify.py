"""One whole S4C verify step on device buffers: [s4c_tree_build,] n_layers x s4c_tree_attention, s4c_tree_accept,
s4c_kv_compact.

:class:`VerifyStep` owns nothing but references to the caller's tensors plus the small output / scratch tensors
it allocates once.  ``run()`` enqueues the step on the current stream through the C ABI; ``capture()`` records
the same launches into a CUDA graph so that a replay costs one host call (the step is 34 tiny launches at the
7B shape -- launch-bound from Python otherwise).  ``run_host()`` is the end-to-end form: the step's per-step
inputs arrive in pinned host memory, are copied in, the step runs, and the decision is copied back.
All arithmetic happens inside libs4c's kernels.
"""
from __future__ import annotations

from typing import List, Optional

import torch

from . import s4c


class VerifyStep:
    def __init__(self, q: List[torch.Tensor], k_caches: List[torch.Tensor], v_caches: List[torch.Tensor],
                 cache_len: torch.Tensor, parent: torch.Tensor, tokens: torch.Tensor, target_logits: torch.Tensor,
                 draft_probs: Optional[torch.Tensor], uniforms: Optional[torch.Tensor], temperature: float,
                 max_depth: int, n_nodes: Optional[torch.Tensor] = None, feat_in: Optional[torch.Tensor] = None,
                 stacked: Optional[tuple] = None, max_cache_len: int = 0, branching: Optional[tuple] = None,
                 root_token: Optional[torch.Tensor] = None, block_table: Optional[torch.Tensor] = None):
        """``block_table`` [B,max_blocks] int32: the caches are paged -- every ``k_caches[l]`` / ``v_caches[l]`` is a pool
        [n_pages,Hkv,page_size,d] and the step calls s4c_tree_attention_paged / s4c_kv_compact_paged.
        ``branching`` (+ ``root_token`` [B] int32): the step then starts with s4c_tree_build, which writes the tree
        (``tokens``, ``parent``, ``n_nodes``, position ids) from ``draft_probs`` on the device -- no host tree in the loop;
        ``parent`` and ``tokens`` are then only buffers of the right shape.
        ``max_cache_len``: what the host knows about the committed lengths (an upper bound, 0 = nothing); it is handed
        to every s4c_tree_attention call, which shapes its launch for it instead of for the capacity.
        ``stacked`` = (q_all [n_layers,B,Hq,T,d], k_all, v_all [n_layers,B,Hkv,C,d]) when the per-layer tensors are
        views of three big ones: the host-buffer path then moves a step's inputs with three copies instead of three
        per layer."""
        self.n_layers = len(q)
        assert len(k_caches) == self.n_layers and len(v_caches) == self.n_layers
        self.q, self.k_caches, self.v_caches = q, k_caches, v_caches
        self.cache_len0 = cache_len
        self.parent, self.tokens, self.n_nodes = parent, tokens, n_nodes
        self.logits, self.draft_probs, self.uniforms = target_logits, draft_probs, uniforms
        self.temperature, self.max_depth = float(temperature), int(max_depth)
        self.max_cache_len = int(max_cache_len)
        self.branching, self.root_token = None, None
        self.filter = None
        self.feat_in = feat_in
        dev = cache_len.device
        B, T, V = target_logits.shape
        self.B, self.T, self.V = B, T, V
        self.cache_shape = tuple(k_caches[0].shape)
        self.block_table = block_table
        self.dtype = k_caches[0].dtype
        i32 = dict(dtype=torch.int32, device=dev)
        self.cache_len = cache_len.clone()            # working copy: the step advances it in place
        self.attn_out = [torch.empty_like(t) for t in q]
        self.accept_len = torch.empty(B, **i32)
        self.path = torch.empty(B, self.max_depth + 1, **i32)
        self.next_token = torch.empty(B, **i32)
        self.near_tie = torch.empty(B, T, dtype=torch.uint8, device=dev)
        self.status_attn = torch.empty(B, **i32)
        self.status_accept = torch.empty(B, **i32)
        self.status_compact = torch.empty(B, **i32)
        self.feat_out = None if feat_in is None else torch.zeros(B, self.max_depth + 1, feat_in.shape[2],
                                                                 dtype=feat_in.dtype, device=dev)
        _, Hq, _, d = q[0].shape
        _, Hkv, C, _ = self.cache_shape
        if block_table is not None:  # a sequence can hold max_blocks pages
            C = block_table.shape[1] * self.cache_shape[2]
        self.ws_attn = torch.empty(max(1, s4c.tree_attention_workspace_bytes(B, T, Hq, Hkv, d, C, self.dtype)),
                                   dtype=torch.uint8, device=dev)
        self.ws_accept = torch.empty(max(1, s4c.tree_accept_workspace_bytes(B, T, V)), dtype=torch.uint8, device=dev)
        self.k_ptrs = s4c.cache_pointer_array(k_caches)
        self.v_ptrs = s4c.cache_pointer_array(v_caches)
        self.stacked = stacked
        if branching is not None:
            self.enable_tree_build(branching, root_token)
        self.graph: Optional[torch.cuda.CUDAGraph] = None
        self._host = None

    # ------------------------------------------------------------------ the stages
    def enable_tree_build(self, branching, root_token: torch.Tensor):
        """From now on ``run()`` starts with s4c_tree_build (see the constructor)."""
        assert self.draft_probs is not None and root_token is not None, "building the tree needs draft_probs and root_token"
        self.branching = tuple(int(x) for x in branching)
        self.root_token = root_token
        i32 = dict(dtype=torch.int32, device=self.cache_len.device)
        if self.n_nodes is None:
            self.n_nodes = torch.full((self.B,), self.T, **i32)
        self.position = torch.empty(self.B, self.T, **i32)
        self.ws_tree = torch.empty(max(1, s4c.tree_build_workspace_bytes(self.B, self.T, self.V, max((1,) + self.branching))),
                                   dtype=torch.uint8, device=self.cache_len.device)

    def build_tree(self):
        s4c.tree_build(self.draft_probs, self.branching, self.root_token, self.cache_len, tokens=self.tokens,
                       parent=self.parent, position=self.position, n_nodes=self.n_nodes, workspace=self.ws_tree)

    def attention(self, l0: int = 0, l1: Optional[int] = None):
        for l in range(l0, self.n_layers if l1 is None else l1):
            if self.block_table is not None:
                s4c.tree_attention_paged(self.q[l], self.k_caches[l], self.v_caches[l], self.block_table, self.cache_len,
                                         self.parent, self.n_nodes, out=self.attn_out[l], status=self.status_attn,
                                         workspace=self.ws_attn, max_cache_len=self.max_cache_len)
                continue
            s4c.tree_attention(self.q[l], self.k_caches[l], self.v_caches[l], self.cache_len, self.parent, self.n_nodes,
                               out=self.attn_out[l], status=self.status_attn, workspace=self.ws_attn,
                               max_cache_len=self.max_cache_len)

    def set_filter(self, top_k: Optional[int], top_p: float = 1.0):
        """From now on ``accept()`` verifies against the top-k / nucleus filtered target distribution
        (s4c_tree_accept_filtered); ``top_k=None`` goes back to the unfiltered one."""
        assert top_k is None or self.temperature > 0, "the filter belongs to stochastic acceptance"
        self.filter = None if top_k is None else (int(top_k), float(top_p))
        if self.filter is not None:
            need = s4c.tree_accept_filtered_workspace_bytes(self.B, self.T, self.V, int(top_k))
            self.ws_filter = torch.empty(max(1, need), dtype=torch.uint8, device=self.cache_len.device)

    def accept(self):
        if self.filter is not None:
            s4c.tree_accept_filtered(self.logits, self.draft_probs, self.tokens, self.parent, self.temperature,
                                     self.filter[0], self.filter[1], self.uniforms, self.n_nodes, self.max_depth,
                                     self.accept_len, self.path, self.next_token, self.near_tie, self.status_accept,
                                     self.ws_filter)
            return
        s4c.tree_accept(self.logits, self.draft_probs, self.tokens, self.parent, self.temperature, self.uniforms,
                        self.n_nodes, self.max_depth, self.accept_len, self.path, self.next_token, self.near_tie,
                        self.status_accept, self.ws_accept)

    def compact(self):
        if self.block_table is not None:
            s4c.kv_compact_paged(self.k_ptrs, self.v_ptrs, self.n_layers, self.cache_shape, self.dtype, self.block_table,
                                 self.cache_len, self.path, self.accept_len, self.T, self.feat_in, self.feat_out,
                                 self.status_compact)
            return
        s4c.kv_compact(self.k_ptrs, self.v_ptrs, self.n_layers, self.cache_shape, self.dtype, self.cache_len, self.path,
                       self.accept_len, self.T, self.feat_in, self.feat_out, self.status_compact)

    def reset_lengths(self):
        """Rewind the working cache length to the committed length (so that a benchmark can repeat the step)."""
        self.cache_len.copy_(self.cache_len0)

    def run(self):
        self.reset_lengths()
        if self.branching is not None:
            self.build_tree()
        self.attention()
        self.accept()
        self.compact()

    # kernels launched by one run(): used by the benchmark to report its launch count
    def launches_per_step(self, attn_launches_per_layer: int) -> int:
        # acceptance: per-node statistics (one launch, cluster or segment kernel) and the walk; filtered: segment
        # selection, row selection and the walk
        accept = 3 if self.filter is not None else 2
        compact = 2 if self.n_layers > 0 else 1
        tree = 2 if self.branching is not None else 0
        return self.n_layers * attn_launches_per_layer + accept + compact + tree

    # ------------------------------------------------------------------ CUDA graph
    def capture(self, what: str = "step") -> torch.cuda.CUDAGraph:
        if what.startswith("layers:"):  # "layers:l0:l1": the attention launches of layers l0..l1-1 (the first rewinds the lengths)
            l0, l1 = (int(x) for x in what.split(":")[1:])
            fn = lambda: ((self.reset_lengths() if l0 == 0 else None), self.attention(l0, l1))
        else:
            fn = {"step": self.run, "attention": self.attention, "accept": self.accept, "tree": self.build_tree,
                  "compact": lambda: (self.reset_lengths(), self.compact()),
                  "head": lambda: (self.reset_lengths(), self.attention()),
                  "tail": lambda: (self.accept(), self.compact())}[what]
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            fn()  # warm-up outside capture (first-launch module loading must not happen while capturing)
        torch.cuda.current_stream().wait_stream(s)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        if what == "step":
            self.graph = g
        return g

    # ------------------------------------------------------------------ end to end from host memory
    def bind_host_inputs(self):
        """Allocate pinned host mirrors of the per-step inputs and outputs; returns (inputs dict, outputs dict).

        Per-step inputs: queries and the tree tokens' K/V rows of every layer, the tree, the draft tokens,
        target logits, draft probabilities, uniforms and features.  The committed cache prefix is state that
        lives on the device across steps and is not copied.
        """
        pin = lambda t: torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t)
        L = int(self.cache_len0.max().item())
        assert int(self.cache_len0.min().item()) == L, "run_host expects one committed length for the batch"
        T = self.T
        if self.stacked is not None:  # one pinned buffer per kind for all layers
            q_all, k_all, v_all = self.stacked
            layers = dict(q=[pin(q_all)], k_tree=[pin(k_all[:, :, :, L:L + T])], v_tree=[pin(v_all[:, :, :, L:L + T])])
        else:
            layers = dict(q=[pin(t) for t in self.q], k_tree=[pin(c[:, :, L:L + T]) for c in self.k_caches],
                          v_tree=[pin(c[:, :, L:L + T]) for c in self.v_caches])
        inp = dict(**layers,
                   parent=pin(self.parent), tokens=pin(self.tokens), logits=pin(self.logits))
        if self.draft_probs is not None:
            inp["draft_probs"] = pin(self.draft_probs)
            inp["uniforms"] = pin(self.uniforms)
        if self.feat_in is not None:
            inp["feat_in"] = pin(self.feat_in)
        out = dict(accept_len=pin(self.accept_len), path=pin(self.path), next_token=pin(self.next_token),
                   cache_len=pin(self.cache_len), status=pin(self.status_accept))
        self._host = (inp, out, L)
        nbytes = lambda x: sum(t.numel() * t.element_size() for t in (x if isinstance(x, list) else [x]))
        if self.graph is not None:  # the step as several graphs, so that later inputs can arrive while earlier layers run
            self._side_stream = torch.cuda.Stream()
            self.graph_head, self.graph_tail = self.capture("head"), self.capture("tail")
            self.graph_host = None
            if self.stacked is not None and self.n_layers >= 8:
                # two groups of layers: measured best on the 7B shape (0.78 ms unsplit, 0.69 with two groups, 0.76 with
                # four, 0.92 with eight -- every extra copy costs more than the overlap it buys)
                self.graph_host = self._capture_host_step(n_chunks=2)
        self.h2d_bytes = sum(nbytes(v) for v in inp.values())
        self.d2h_bytes = sum(nbytes(v) for v in out.values())
        return inp, out

    def _host_step_pipelined(self, n_chunks: int):
        """The host-buffer step with copies and layers overlapped: a second stream brings the inputs in layer-group
        order (then what only acceptance and compaction read); the first stream runs a group's attention launches as
        soon as that group's event has fired, then acceptance and compaction, then copies the decision back."""
        inp, out, L = self._host
        T = self.T
        q_all, k_all, v_all = self.stacked
        bounds = [self.n_layers * c // n_chunks for c in range(n_chunks + 1)]
        main, side = torch.cuda.current_stream(), torch.cuda.Stream()
        side.wait_stream(main)
        events = []
        with torch.cuda.stream(side):
            self.parent.copy_(inp["parent"], non_blocking=True)
            for l0, l1 in zip(bounds[:-1], bounds[1:]):
                q_all[l0:l1].copy_(inp["q"][0][l0:l1], non_blocking=True)
                k_all[l0:l1, :, :, L:L + T].copy_(inp["k_tree"][0][l0:l1], non_blocking=True)
                v_all[l0:l1, :, :, L:L + T].copy_(inp["v_tree"][0][l0:l1], non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(side)
                events.append(ev)
            self.tokens.copy_(inp["tokens"], non_blocking=True)
            self.logits.copy_(inp["logits"], non_blocking=True)
            if self.draft_probs is not None:
                self.draft_probs.copy_(inp["draft_probs"], non_blocking=True)
                self.uniforms.copy_(inp["uniforms"], non_blocking=True)
            if self.feat_in is not None:
                self.feat_in.copy_(inp["feat_in"], non_blocking=True)
        self.reset_lengths()
        for (l0, l1), ev in zip(zip(bounds[:-1], bounds[1:]), events):
            main.wait_event(ev)
            self.attention(l0, l1)
        main.wait_stream(side)  # the acceptance inputs are in; the second stream joins here
        self.accept()
        self.compact()
        out["accept_len"].copy_(self.accept_len, non_blocking=True)
        out["path"].copy_(self.path, non_blocking=True)
        out["next_token"].copy_(self.next_token, non_blocking=True)
        out["cache_len"].copy_(self.cache_len, non_blocking=True)
        out["status"].copy_(self.status_accept, non_blocking=True)

    def _capture_host_step(self, n_chunks: int) -> torch.cuda.CUDAGraph:
        """The pipelined host-buffer step as one CUDA graph (host-to-device and device-to-host copies are nodes of it:
        the pinned buffers keep their addresses, the caller rewrites their contents between replays)."""
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            self._host_step_pipelined(n_chunks)  # warm-up outside capture
        torch.cuda.current_stream().wait_stream(s)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self._host_step_pipelined(n_chunks)
        return g

    def run_host(self):
        """Copy the per-step inputs in (async, pinned), run the step, copy the decision back, and wait for it."""
        inp, out, L = self._host
        T = self.T
        if getattr(self, "graph_host", None) is not None:
            self.graph_host.replay()
            torch.cuda.current_stream().synchronize()
            return out
        if self.stacked is not None:
            q_all, k_all, v_all = self.stacked
            q_all.copy_(inp["q"][0], non_blocking=True)
            k_all[:, :, :, L:L + T].copy_(inp["k_tree"][0], non_blocking=True)
            v_all[:, :, :, L:L + T].copy_(inp["v_tree"][0], non_blocking=True)
        else:
            for l in range(self.n_layers):
                self.q[l].copy_(inp["q"][l], non_blocking=True)
                self.k_caches[l][:, :, L:L + T].copy_(inp["k_tree"][l], non_blocking=True)
                self.v_caches[l][:, :, L:L + T].copy_(inp["v_tree"][l], non_blocking=True)
        self.parent.copy_(inp["parent"], non_blocking=True)
        split = self.graph is not None and getattr(self, "graph_head", None) is not None
        main = torch.cuda.current_stream()
        # what only acceptance and compaction read (logits, draft probabilities, ...) travels on a second stream while
        # the attention layers run; the tail of the step waits for it
        side = self._side_stream if split else main
        if split:
            side.wait_stream(main)
        with torch.cuda.stream(side):
            self.tokens.copy_(inp["tokens"], non_blocking=True)
            self.logits.copy_(inp["logits"], non_blocking=True)
            if self.draft_probs is not None:
                self.draft_probs.copy_(inp["draft_probs"], non_blocking=True)
                self.uniforms.copy_(inp["uniforms"], non_blocking=True)
            if self.feat_in is not None:
                self.feat_in.copy_(inp["feat_in"], non_blocking=True)
        if split:
            self.graph_head.replay()
            main.wait_stream(side)
            self.graph_tail.replay()
        elif self.graph is not None:
            self.graph.replay()
        else:
            self.run()
        out["accept_len"].copy_(self.accept_len, non_blocking=True)
        out["path"].copy_(self.path, non_blocking=True)
        out["next_token"].copy_(self.next_token, non_blocking=True)
        out["cache_len"].copy_(self.cache_len, non_blocking=True)
        out["status"].copy_(self.status_accept, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        return out
