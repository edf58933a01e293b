"""s4c_tree_accept_noalloc: the acceptance step for callers that are not allowed to allocate device memory.

A serving loop that has given all device memory to its own pool, or a plug-in living inside another framework's
allocator, cannot hand the library a workspace obtained from cudaMalloc.  The no-allocation entry point uses a
scratch array compiled into the library instead.  This test calls it through the C ABI twice in a row (the second
call finds the first call's leftovers in the shared array) and requires exactly the results of s4c_tree_accept.
It lives in the last-collected file so that a run stopping at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2506_14158_b200 import workloads as W

from parity import dev

pytestmark = pytest.mark.gpu


def _both(cfg, tau, mode):
    from paper_2506_14158_b200 import s4c

    parent = W.make_trees(cfg)
    x = W.make_accept_inputs(cfg, parent, tau, token_mode=mode)
    args = (dev(x["logits"]), dev(x["draft_probs"]) if tau > 0 else None, dev(x["tokens"]), dev(parent), tau,
            dev(x["uniforms"]) if tau > 0 else None)
    ref = s4c.tree_accept(*args, max_depth=cfg.max_depth)
    got = s4c.tree_accept_noalloc(*args, max_depth=cfg.max_depth)
    torch.cuda.synchronize()
    return got, ref


def test_noalloc_entry_matches_the_workspace_entry_on_consecutive_calls():
    from paper_2506_14158_b200 import s4c

    calls = [(W.CONFIGS["c2"], 1.0, "sampled"), (W.CONFIGS["c1"], 1.0, "topk"), (W.CONFIGS["c2"], 0.0, "topk")]
    for cfg, tau, mode in calls:  # back to back: each call reuses the array the previous one dirtied
        assert s4c.tree_accept_workspace_bytes(cfg.B, cfg.T, cfg.V) <= s4c.NOALLOC_SCRATCH_BYTES
        got, ref = _both(cfg, tau, mode)
        for key in ("accept_len", "path", "next_token", "near_tie", "status"):
            assert torch.equal(got[key], ref[key]), key  # integer outputs: exact, the tolerance the other tests use
        assert int(ref["status"].abs().sum()) == 0 and int(ref["accept_len"].min()) >= 0


def test_noalloc_entry_leaves_device_memory_as_it_found_it():
    # the property the entry point exists for: with the outputs preallocated, a call changes neither what the process has
    # allocated nor what the device has free.  One problem on the cluster-statistics path, one on the segment path.
    from dataclasses import replace

    from paper_2506_14158_b200 import s4c

    seg = replace(W.CONFIGS["c2"], name="noalloc_seg", config_id=81, B=4, T=128, V=32000, tree="random", max_tree_depth=8)
    for cfg in (W.CONFIGS["c2"], seg):
        assert s4c.tree_accept_workspace_bytes(cfg.B, cfg.T, cfg.V) <= s4c.NOALLOC_SCRATCH_BYTES
        parent = W.make_trees(cfg)
        x = W.make_accept_inputs(cfg, parent, 1.0, token_mode="topk")
        args = (dev(x["logits"]), dev(x["draft_probs"]), dev(x["tokens"]), dev(parent), 1.0, dev(x["uniforms"]))
        md = cfg.max_depth
        ref = s4c.tree_accept(*args, max_depth=md)
        i32 = dict(dtype=torch.int32, device="cuda")
        out = dict(accept_len=torch.empty(cfg.B, **i32), path=torch.empty(cfg.B, md + 1, **i32),
                   next_token=torch.empty(cfg.B, **i32), near_tie=torch.empty(cfg.B, cfg.T, dtype=torch.uint8, device="cuda"),
                   status=torch.empty(cfg.B, **i32))
        s4c.tree_accept_noalloc(*args, max_depth=md, out=out)  # warm-up: module loading, the symbol lookup
        torch.cuda.synchronize()
        held, free = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
        for _ in range(3):
            s4c.tree_accept_noalloc(*args, max_depth=md, out=out)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == held and torch.cuda.mem_get_info()[0] == free
        for key in ("accept_len", "path", "next_token", "near_tie", "status"):
            assert torch.equal(out[key], ref[key]), key


def test_noalloc_entry_refuses_problems_beyond_its_built_in_scratch():
    from paper_2506_14158_b200 import s4c

    B, T, V = 64, 128, 32000  # 64*128*8 segments: far more scratch than the built-in 1 MiB
    assert s4c.tree_accept_workspace_bytes(B, T, V) > s4c.NOALLOC_SCRATCH_BYTES
    tokens = torch.zeros(B, T, dtype=torch.int32, device="cuda")
    with pytest.raises(s4c.S4CError) as err:
        s4c.tree_accept_noalloc(_FakeLogits(B, T, V), None, tokens, tokens, 0.0)
    assert err.value.code == 5  # S4C_ERR_WORKSPACE


class _FakeLogits:
    """Stands in for a [B,T,V] float32 CUDA tensor without allocating it (the refused call never reads it)."""

    def __init__(self, B, T, V):
        self.shape = (B, T, V)
        self._t = torch.zeros(4, device="cuda")
        self.device = self._t.device
        self.dtype = torch.float32
        self.is_cuda = True

    def is_contiguous(self):
        return True

    def data_ptr(self):
        return self._t.data_ptr()
