#!/usr/bin/env python
"""Benchmark of the S4C verify step on B200: verified tree-nodes/s per verify step and achieved HBM GB/s.

A step is one pass of the whole hot path over one batch of seeded synthetic input: n_layers tree-attention
launches, one acceptance, one compaction of every layer's cache (all through the C ABI, replayed as one CUDA
graph).  The default workload "c2x32" is the LLaMA-2-7B-shaped verify step at full depth: the config-2 layer
(32 heads x 128, bf16 cache of 1024 tokens, 26-node tree, vocab 32000) stacked 32 times with an independent
cache per layer, temperature 1.0.  Its 0.56 GB of KV per step is larger than L2, so no flush is needed.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2x32|c2|c3|c4|c4x32|c1|sweep --L --T --B]
                    [--capacity C] [--no-hint] [--no-also] [--no-verify-pass]
    python bench.py --impl reference     # the float64 CPU oracle on a bounded sample of the same workload
    python bench.py --workload launch-floor   # empty kernels with the launch shape of an attention launch
    python bench.py --workload sweep-all [--capacity C]   # every point of the full-depth sweep

The default line also carries, under "also", the 8B-shaped step (c4x32: batch 4, GQA 32/8, 4096-token caches, 64-node
trees, vocabulary 128256, 32 layers) with its own timing, roofline (HBM and tensor) and clock sample.
--capacity lays the caches out for C slots (a serving cache sized for its longest context) instead of L + T; the
host's bound on the live length (max_cache_len = L) is then what shapes the attention launches, unless --no-hint.

Prints one JSON line (rank 0).  With N > 1 (torchrun) every rank verifies its own independent batch: weak scaling,
no data-path collective; the only communication is the barrier and the max of the timings.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "verified tree-nodes/s per verify step"
UNIT = "nodes/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2x32")
    ap.add_argument("--L", type=int, default=4096)
    ap.add_argument("--T", type=int, default=64)
    ap.add_argument("--B", type=int, default=1)
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--temperature", type=float, default=1.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--capacity", type=int, default=0, help="cache capacity in slots (0: L + T rounded up to 128)")
    ap.add_argument("--no-hint", action="store_true", help="do not pass max_cache_len: launches are shaped for the capacity")
    ap.add_argument("--no-also", action="store_true", help="leave the 8B-shaped record out of the default line")
    ap.add_argument("--no-verify-pass", action="store_true", help="leave out the leg that runs the target's whole verify pass (all layers' weights: ~14 GB)")
    ap.add_argument("--min-seconds", type=float, default=0.5, help="keep timing K-step blocks until this much is timed")
    ap.add_argument("--paged", type=int, default=0, help="page size in slots (64, 128, ...): the caches become pools of pages "
                    "scattered at random, addressed through a block table (no host-buffer leg)")
    return ap.parse_args()


def get_config(args):
    from paper_2506_14158_b200 import workloads as W

    from dataclasses import replace

    cfg = W.sweep_config(args.L, args.T, args.B, args.layers) if args.workload == "sweep" else W.CONFIGS[args.workload]
    return replace(cfg, capacity=args.capacity) if args.capacity else cfg


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops_sustained"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1400.0, source="fallback")


# ----------------------------------------------------------------------------- DRAM traffic seen by ncu
# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of the dominant kernel, from the ncu capture summarised
# under profiles/ (the file named here).  It only describes the kernel it was taken on: the value is reported while
# the kernel source still has the recorded hash, otherwise null.
NCU_TRAFFIC = {
    "c2x32": dict(bytes=18115328, sha256="abfb0a4a2295214996ebd8db21767a047ee1b1afaf618733a225e19874f2dabe",
                  profile="profiles/tree_attention_tc_c2x32_ncu_full.md"),
    "c4x32": dict(bytes=71720448, sha256="abfb0a4a2295214996ebd8db21767a047ee1b1afaf618733a225e19874f2dabe",
                  profile="profiles/tree_attention_tc_c4x32_ncu_full.md"),
}


def ncu_traffic(workload):
    import hashlib

    rec = NCU_TRAFFIC.get(workload)
    if not rec or rec["bytes"] is None:
        return None
    src = os.path.join(ROOT, "paper_2506_14158_b200", "csrc", "tree_attention_tc.cu")
    try:
        sha = hashlib.sha256(open(src, "rb").read()).hexdigest()
    except OSError:
        return None
    return rec["bytes"] if sha == rec["sha256"] else None


# ----------------------------------------------------------------------------- algorithmic bytes
def algorithmic_bytes(cfg, temperature, accept_lens):
    """Bytes the method must move per step: K/V of the visible slots and Q/O once per layer; every logits row
    (and draft-probability row when sampling, see below) once; the accepted rows of every layer and the features."""
    s = 2 if cfg.dtype == "bf16" else 4
    attn_layer = 2 * cfg.B * cfg.Hkv * (cfg.L + cfg.T) * cfg.d * s + 2 * cfg.B * cfg.Hq * cfg.T * cfg.d * s
    rows = sum(int(a) + 1 for a in accept_lens)
    accept = cfg.B * cfg.T * cfg.V * (8 if temperature > 0 else 4)
    if temperature > 0 and (cfg.B * cfg.T * cfg.V > (8 << 20) or cfg.V % 4 or cfg.V > 131072):
        # large problems: the residual masses are computed on the walked rows only, so the draft probabilities of the
        # other rows are never needed: every logits row once, logits and draft probabilities of the walked rows once more
        accept = cfg.B * cfg.T * cfg.V * 4 + rows * cfg.V * 8
    compact = cfg.n_layers * 2 * 2 * cfg.Hkv * rows * cfg.d * s + 2 * rows * cfg.hid * s
    # the same step counted as "every logits row and every draft-probability row once" (B*T*V*8 when sampling), whether or
    # not the kernels need the draft probabilities of rows the walk never visits
    accept_all_rows = cfg.B * cfg.T * cfg.V * (8 if temperature > 0 else 4)
    return dict(attention_per_layer=attn_layer, attention=attn_layer * cfg.n_layers, accept=accept, compact=compact,
                total=attn_layer * cfg.n_layers + accept + compact, accept_all_rows=accept_all_rows,
                total_all_rows=attn_layer * cfg.n_layers + accept_all_rows + compact)


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc = [], None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = [r for r in self.rows if t0 - 0.05 <= r[0] <= t1 + 0.15] or self.rows
        for _, line in rows:
            f = [x.strip() for x in line.split(",")]
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=mx, reasons=sorted(reasons),
                    samples=len(sm))


# ----------------------------------------------------------------------------- oracle timing (CPU)
def oracle_sample(cfg, temperature, layers_sample=None, threads=None, budget_s=10.0):
    """Times the float64 oracle, as it stands, on a bounded sample of the workload: one untimed attention layer, then
    `layers_sample` timed ones (default: as many as fit about `budget_s` seconds, at least one) -- their MEAN is the
    layer time --, the whole acceptance, and the compaction of one layer; attention and compaction are scaled to
    n_layers.  `threads`: OpenMP threads (default: all the oracle would use).  Returns (seconds per step, description,
    acceptance result)."""
    import numpy as np

    import oracle
    from paper_2506_14158_b200 import workloads as W

    all_threads = oracle.max_threads()
    if threads:
        oracle.set_threads(threads)
    try:
        parent = W.make_trees(cfg)
        x = W.make_accept_inputs(cfg, parent, temperature, token_mode="topk")
        cl = np.full(cfg.B, cfg.L, dtype=np.int32)
        q, k, v = W.make_attention_inputs(cfg, 0)
        q64, k64, v64 = W.to_f64(q), W.to_f64(k), W.to_f64(v)
        t = time.perf_counter()
        oracle.tree_attention(q64, k64, v64, cl, parent)  # untimed in the figure: first touch of the arrays, thread start-up
        t_first = time.perf_counter() - t
        n_s = layers_sample or max(1, min(cfg.n_layers, int(budget_s / max(t_first, 1e-3))))
        t = time.perf_counter()
        for _ in range(n_s):
            oracle.tree_attention(q64, k64, v64, cl, parent)
        t_layer = (time.perf_counter() - t) / n_s
        t = time.perf_counter()
        tau = float(np.float32(temperature))
        if tau > 0:
            r = oracle.accept_stochastic(x["logits"], x["draft_probs"], x["tokens"], parent, tau, x["uniforms"],
                                         max_depth=cfg.max_depth)
        else:
            r = oracle.accept_greedy(x["logits"], x["tokens"], parent, max_depth=cfg.max_depth)
        t_accept = time.perf_counter() - t
        bits = k.view(torch_int_dtype(k)).numpy().copy()
        kc, vc = [bits.copy()], [bits.copy()]
        t = time.perf_counter()
        oracle.kv_compact(kc, vc, cl.copy(), r["path"], r["accept_len"], cfg.T)
        t_compact = time.perf_counter() - t
        used = threads or all_threads
    finally:
        if threads:
            oracle.set_threads(all_threads)
    total = t_layer * cfg.n_layers + t_accept + t_compact * cfg.n_layers
    desc = (f"float64 C oracle, {used} OpenMP thread(s): mean of {n_s} attention layer(s) of {cfg.n_layers} after one "
            f"untimed ({t_layer * 1e3:.1f} ms each), whole acceptance ({t_accept * 1e3:.1f} ms), compaction of 1 layer "
            f"({t_compact * 1e3:.2f} ms); attention and compaction scaled to {cfg.n_layers} layers")
    return total, desc, r


def torch_int_dtype(t):
    import torch

    return torch.int32 if t.dtype == torch.float32 else torch.int16


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle

    cfg = get_config(args)
    times = []
    steps = max(1, min(args.steps, 3))
    # every step is the same bounded sample that the CUDA arm's cpu_baseline quotes (about 3 s of attention layers, the
    # whole acceptance, one layer's compaction), so the two figures describe the same thing
    for _ in range(min(args.warmup, 1)):
        oracle_sample(cfg, args.temperature, layers_sample=1)
    desc = ""
    for _ in range(steps):
        t, desc, _ = oracle_sample(cfg, args.temperature, budget_s=3.0)
        times.append(t)
    tstep = statistics.median(times)
    value = cfg.B * cfg.T / tstep
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=steps,
                warmup=min(args.warmup, 1), ms_per_step=tstep * 1e3, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f64", data="synthetic (seeded)", config=config_record(cfg, args, 1),
                cpu_baseline=dict(value=value, unit=UNIT, cores=oracle.max_threads(), kind="oracle", sample=desc),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line), flush=True)


def config_record(cfg, args, world):
    """The `config` object of a line: identical keys in both arms, so that they can be compared field by field."""
    return dict(workload=cfg.name, B=cfg.B, T=cfg.T, L=cfg.L, C=cfg.C, Hq=cfg.Hq, Hkv=cfg.Hkv, d=cfg.d, V=cfg.V,
                n_layers=cfg.n_layers, temperature=args.temperature)


# ----------------------------------------------------------------------------- the CUDA arm
def build_step(cfg, temperature, device, seed_shift=0, hint=True, paged=0):
    import numpy as np
    import torch

    from paper_2506_14158_b200 import workloads as W
    from paper_2506_14158_b200.verify import VerifyStep

    from paper_2506_14158_b200 import replicas

    cfg_gen = replicas.rank_config(cfg, seed_shift)  # every replica verifies its own seeded batch
    parent = W.make_trees(cfg_gen)
    x = W.make_accept_inputs(cfg_gen, parent, temperature, token_mode="topk")
    kv_bytes = 2 * cfg.n_layers * cfg.B * cfg.Hkv * cfg.C * cfg.d * (2 if cfg.dtype == "bf16" else 4)
    on_device = kv_bytes > (1 << 30)
    dt = {"f32": torch.float32, "bf16": torch.bfloat16}[cfg.dtype]
    # every layer's tensors are views of three big ones (still an independent cache per layer): the host-buffer leg
    # then needs three copies per step, not three per layer
    q_all = torch.empty((cfg.n_layers, cfg.B, cfg.Hq, cfg.T, cfg.d), dtype=dt, device=device)
    k_all = torch.empty((cfg.n_layers, cfg.B, cfg.Hkv, cfg.C, cfg.d), dtype=dt, device=device)
    v_all = torch.empty((cfg.n_layers, cfg.B, cfg.Hkv, cfg.C, cfg.d), dtype=dt, device=device)
    qs, ks, vs = list(q_all.unbind(0)), list(k_all.unbind(0)), list(v_all.unbind(0))
    for l in range(cfg.n_layers):
        if on_device:  # very large sweeps: draw the caches on the device (values are N(0,1) either way)
            g = torch.Generator(device=device).manual_seed(W.stream_seed(cfg_gen.config_id, "kv", l))
            q = torch.randn((cfg.B, cfg.Hq, cfg.T, cfg.d), generator=g, device=device).to(dt)
            k = torch.randn((cfg.B, cfg.Hkv, cfg.C, cfg.d), generator=g, device=device).to(dt)
            v = torch.randn((cfg.B, cfg.Hkv, cfg.C, cfg.d), generator=g, device=device).to(dt)
        else:
            q, k, v = (t.to(device) for t in W.make_attention_inputs(cfg_gen, l))
        qs[l].copy_(q), ks[l].copy_(k), vs[l].copy_(v)
        del q, k, v
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device)
    block_table = None
    if paged:
        # the same caches as pools of pages: page i of (sequence b, layer l) lies wherever a seeded permutation put it
        ps = paged
        nb = (cfg.C + ps - 1) // ps
        n_pages = cfg.B * nb + 3
        perm = np.random.default_rng(W.stream_seed(cfg_gen.config_id, "tree", 99)).permutation(n_pages)[: cfg.B * nb]
        bt = torch.from_numpy(perm.reshape(cfg.B, nb).astype(np.int32)).to(device)
        pools_k = torch.zeros((cfg.n_layers, n_pages, cfg.Hkv, ps, cfg.d), dtype=dt, device=device)
        pools_v = torch.zeros_like(pools_k)
        pad = nb * ps - cfg.C
        for src, dst in ((k_all, pools_k), (v_all, pools_v)):
            blk = torch.nn.functional.pad(src, (0, 0, 0, pad)) if pad else src                     # [n_layers,B,Hkv,nb*ps,d]
            blk = blk.view(cfg.n_layers, cfg.B, cfg.Hkv, nb, ps, cfg.d).permute(0, 1, 3, 2, 4, 5)  # [n_layers,B,nb,Hkv,ps,d]
            dst[:, bt.long().reshape(-1)] = blk.reshape(cfg.n_layers, cfg.B * nb, cfg.Hkv, ps, cfg.d)
            del blk
        ks, vs = list(pools_k.unbind(0)), list(pools_v.unbind(0))
        del k_all, v_all
        k_all = v_all = None
        block_table = bt
    stoch = temperature > 0
    step = VerifyStep(qs, ks, vs, torch.full((cfg.B,), cfg.L, dtype=torch.int32, device=device), to(parent),
                      to(x["tokens"]), to(x["logits"]), to(x["draft_probs"]) if stoch else None,
                      to(x["uniforms"]) if stoch else None, temperature, cfg.max_depth,
                      feat_in=W.make_features(cfg_gen).to(device), stacked=None if paged else (q_all, k_all, v_all),
                      max_cache_len=cfg.L if hint else 0,  # what a host that tracks its sequences' lengths knows
                      block_table=block_table)
    return step


def replace_id(cfg, i):
    """The same configuration with another input-stream id (another layer's random weights)."""
    from dataclasses import replace

    return replace(cfg, config_id=cfg.config_id * 37 + 11 + i)


def time_graph(graph, iters, torch):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        graph.replay()
    e1.record()
    e1.synchronize()
    return e0.elapsed_time(e1) / iters  # ms per replay


def time_blocks(graph, iters, torch, min_seconds, max_blocks=200):
    """Blocks of `iters` replays, each between its own pair of CUDA events, until `min_seconds` have been timed
    (at least one block).  Returns the list of ms-per-replay figures, one per block."""
    out, total = [], 0.0
    while not out or (total < min_seconds * 1e3 and len(out) < max_blocks):
        ms = time_graph(graph, iters, torch)
        out.append(ms)
        total += ms * iters
    return out


def measure(cfg, args, device, rank, world, with_e2e):
    """Times one workload on this rank: the whole-step graph (K-step blocks), then the attention launches, acceptance
    and compaction alone.  Returns a dict of raw figures (milliseconds, max over ranks where a rank count matters)."""
    import torch

    from paper_2506_14158_b200 import replicas

    K, Wm = args.steps, max(3, args.warmup)
    step = build_step(cfg, args.temperature, device, seed_shift=rank, hint=not args.no_hint, paged=args.paged)
    with_e2e = with_e2e and not args.paged
    g_step = step.capture("step")
    g_attn = step.capture("attention")
    g_acc = step.capture("accept")
    g_cmp = step.capture("compact")

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize()

    for _ in range(Wm):
        g_step.replay()
    barrier()
    sampler = ClockSampler(device.index) if rank == 0 else None
    t0 = time.time()
    blocks = time_blocks(g_step, K, torch, args.min_seconds)  # the first block is the K steps of the contract
    barrier()
    t1 = time.time()
    clocks = sampler.stop(t0, t1) if sampler else None
    # dominant-kernel leg: the n_layers attention launches alone, same buffers, same stream, CUDA events
    step.reset_lengths()  # the step's compaction advanced the lengths: attention is timed on the committed ones
    for _ in range(3):
        g_attn.replay()
    torch.cuda.synchronize()
    attn_blocks = time_blocks(g_attn, K, torch, args.min_seconds / 2)
    ms_acc = time_graph(g_acc, K, torch)  # L2-resident when the logits fit L2: informational only
    ms_cmp = time_graph(g_cmp, K, torch)
    # the tree itself, built on the device from the draft probabilities (not part of the timed step: the step takes the
    # tree as input, as the three verify calls do); only for workloads whose tree comes from branching factors
    ms_tree = None
    if cfg.tree == "branching" and args.temperature > 0:
        step.enable_tree_build(cfg.branching, step.tokens[:, 0].contiguous())
        g_tree = step.capture("tree")
        ms_tree = time_graph(g_tree, K, torch)
    # the same acceptance against a top-k / nucleus filtered target (not part of the timed step either)
    ms_filt = None
    if args.temperature > 0:
        step.set_filter(FILTER_TOP_K, FILTER_TOP_P)
        ms_filt = time_graph(step.capture("accept"), K, torch)
        step.set_filter(None)
        g_acc.replay()  # the step's own decision is back in the output buffers
    # the LM head fused with the greedy choice, then the greedy walk on the choices: the route on which the [B,T,V] logits
    # never exist (timed alone; the step above takes the logits as input).  Weights larger than L2 on both shapes.
    lm = None
    if cfg.dtype == "bf16" and not args.paged:
        from paper_2506_14158_b200 import s4c
        from paper_2506_14158_b200 import workloads as Wl

        hid = step.feat_in.reshape(cfg.B * cfg.T, cfg.hid).contiguous()
        wgt = Wl.make_lm_head(cfg, device)
        choice = torch.empty(cfg.B * cfg.T, dtype=torch.int32, device=device)
        mx = torch.empty(cfg.B * cfg.T, dtype=torch.float32, device=device)
        st = torch.zeros(1, dtype=torch.int32, device=device)
        ws = torch.empty(s4c.lm_head_greedy_workspace_bytes(cfg.B * cfg.T, cfg.V, cfg.hid), dtype=torch.uint8, device=device)
        outs = [torch.empty_like(step.accept_len), torch.empty_like(step.path), torch.empty_like(step.next_token),
                torch.empty_like(step.status_accept)]

        def head_and_walk():
            s4c.lm_head_greedy(hid, wgt, choice, mx, st, ws)
            s4c.tree_accept_tokens(choice.view(cfg.B, cfg.T), step.tokens, step.parent, cfg.V, step.n_nodes, cfg.max_depth, *outs)

        sg = torch.cuda.Stream()
        sg.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(sg):
            head_and_walk()
        torch.cuda.current_stream().wait_stream(sg)
        torch.cuda.synchronize()
        g_lm = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_lm):
            head_and_walk()
        for _ in range(3):
            g_lm.replay()
        ms_lm = time_graph(g_lm, K, torch)
        assert int(st.item()) == 0, "s4c_lm_head_greedy gave up a wait"
        lm = dict(ms=ms_lm, rows=cfg.B * cfg.T, V=cfg.V, H=cfg.hid)
        del wgt, ws
    # the layer's input side: q/k/v projections + rotary embedding written into the attention layout and the cache's tree
    # slots (timed alone, on buffers of its own: the step above takes q and the tree K/V as input)
    qk = None
    if cfg.dtype == "bf16" and not args.paged and cfg.d in (64, 128):
        from paper_2506_14158_b200 import s4c
        from paper_2506_14158_b200 import workloads as Wl

        n_w = 4  # a few layers' weights in turn, so that the weights of a call do not sit in L2 from the call before
        ws_qk = [Wl.make_qkv_weight(replace_id(cfg, i), device) for i in range(n_w)]
        x_in = step.feat_in.contiguous()
        q_buf = torch.empty_like(step.q[0])
        kc = torch.zeros((cfg.B, cfg.Hkv, cfg.C, cfg.d), dtype=torch.bfloat16, device=device)
        vc = torch.zeros_like(kc)
        st_qk = torch.empty(cfg.B, dtype=torch.int32, device=device)
        wsp = torch.empty(s4c.qkv_rope_workspace_bytes(cfg.B, cfg.T, cfg.d), dtype=torch.uint8, device=device)

        def qkv_layers():
            for w_l in ws_qk:
                s4c.qkv_rope(x_in, w_l, step.cache_len0, step.parent, q_buf, kc, vc, step.n_nodes, 10000.0, st_qk, wsp)

        sg = torch.cuda.Stream()
        sg.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(sg):
            qkv_layers()
        torch.cuda.current_stream().wait_stream(sg)
        torch.cuda.synchronize()
        g_qk = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_qk):
            qkv_layers()
        for _ in range(3):
            g_qk.replay()
        ms_qk = time_graph(g_qk, K, torch) / n_w
        assert int(st_qk.abs().sum().item()) == 0, "s4c_qkv_rope flagged a sequence"
        qk = dict(ms=ms_qk, rows=cfg.B * cfg.T, N=(cfg.Hq + 2 * cfg.Hkv) * cfg.d, H=cfg.hid)
        del ws_qk, kc, vc
    # one head of the drafter (Eq. 3-6) composed from the library's calls: embedding, Linear(concat[e, f]), one decoder layer,
    # LM-head top-k -- random weights of the target's shapes, a cache of its own (timed alone)
    dr = None
    if cfg.dtype == "bf16" and not args.paged and cfg.d in (64, 128) and cfg.hid == cfg.Hq * cfg.d:
        from paper_2506_14158_b200 import drafter

        inter = {32000: 11008, 128256: 14336}.get(cfg.V, (cfg.hid * 8 // 3 + 255) // 256 * 256)  # the paper's models' MLP widths
        kk = max(cfg.branching) if cfg.tree == "branching" else 4
        wts = drafter.random_weights(cfg.V, cfg.hid, cfg.Hq, cfg.Hkv, cfg.d, inter, device, seed=cfg.config_id)
        head = drafter.DrafterHead(wts, cfg.B, cfg.T, cfg.Hq, cfg.Hkv, cfg.d, cfg.C, kk)
        kc = torch.zeros((cfg.B, cfg.Hkv, cfg.C, cfg.d), dtype=torch.bfloat16, device=device)
        vc = torch.zeros_like(kc)
        feats = step.feat_in.reshape(cfg.B * cfg.T, cfg.hid).contiguous()
        run_head = lambda: head.forward(step.tokens, feats, step.cache_len0, step.parent, kc, vc, step.n_nodes, max_cache_len=cfg.L)
        sg = torch.cuda.Stream()
        sg.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(sg):
            run_head()
        torch.cuda.current_stream().wait_stream(sg)
        torch.cuda.synchronize()
        g_dr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_dr):
            run_head()
        for _ in range(3):
            g_dr.replay()
        ms_dr = time_graph(g_dr, K, torch)
        assert int(head.status_head.item()) == 0 and int(head.status_qkv.abs().sum().item()) == 0
        wbytes = sum(t.numel() * 2 for t in (wts.fc, wts.qkv, wts.o, wts.gate_up, wts.down, wts.lm_head))
        dr = dict(ms=ms_dr, rows=cfg.B * cfg.T, weight_bytes=wbytes, inter=inter, k=kk,
                  flops=2.0 * cfg.B * cfg.T * (wbytes / 2))
        del head, kc, vc
        # a whole drafting round: three heads (weights of their own; the target's embedding and LM head shared) fill a 21-node tree
        # level by level (Section 3.1.1 + 3.2) -- rows 2, 6, 6 per sequence
        if cfg.name in ("c2x32", "c4x32", "c2", "c4"):
            br3, T3, k3 = [2, 3, 1, 1], 21, 3
            w3 = [wts] + [drafter.random_weights(8, cfg.hid, cfg.Hq, cfg.Hkv, cfg.d, inter, device, seed=cfg.config_id + 100 + j) for j in (1, 2)]
            for w_ in w3[1:]:
                w_.embedding, w_.lm_head = wts.embedding, wts.lm_head
            mh = drafter.MultiHeadDrafter(w3, cfg.B, T3, br3, cfg.Hq, cfg.Hkv, cfg.d, cfg.C, k3)
            caches3 = []
            for j in range(mh.n_passes):
                nj = mh.levels[j][1] - mh.levels[j][0]
                kc3 = torch.zeros((cfg.B * nj, cfg.Hkv, cfg.C, cfg.d), dtype=torch.bfloat16, device=device)
                caches3.append((kc3, torch.zeros_like(kc3), step.cache_len0.repeat_interleave(nj).contiguous()))
            root3, f03 = step.tokens[:, 0].contiguous(), step.feat_in[:, 0].contiguous()
            cand3 = torch.arange(k3, dtype=torch.int32, device=device).repeat(cfg.B, 1).contiguous()
            run_round = lambda: mh.draft(root3, f03, cand3, step.cache_len0, caches3)
            sg = torch.cuda.Stream()
            sg.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(sg):
                run_round()
            torch.cuda.current_stream().wait_stream(sg)
            torch.cuda.synchronize()
            g_mh = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_mh):
                run_round()
            for _ in range(3):
                g_mh.replay()
            dr["round_ms"] = time_graph(g_mh, K, torch)
            dr["round_weight_bytes"] = 3 * (wbytes - wts.lm_head.numel() * 2) + 3 * wts.lm_head.numel() * 2  # each head streams the LM head again
            dr["round_rows"] = [cfg.B * (e - s) for s, e in mh.levels[: mh.n_passes]]
            del mh, caches3, w3
        del wts
    # the whole greedy verify pass of the target (Section 3.2) composed from the library's calls: embedding of the tree tokens,
    # every decoder layer (q/k/v + rotary, tree attention, output projection, gated MLP), LM head with the greedy choice, walk,
    # compaction of every layer's cache -- random weights of the target's shapes, caches of its own (timed alone)
    vp = None
    if (cfg.dtype == "bf16" and not args.paged and not args.capacity and cfg.name in ("c2x32", "c4x32") and cfg.n_layers > 1
            and not args.no_verify_pass):  # (the two named model shapes; sweeps and capacity studies time attention only)
        from paper_2506_14158_b200 import target

        inter = {32000: 11008, 128256: 14336}.get(cfg.V, (cfg.hid * 8 // 3 + 255) // 256 * 256)
        tw = target.random_weights(cfg.n_layers, cfg.V, cfg.hid, cfg.Hq, cfg.Hkv, cfg.d, inter, device, seed=cfg.config_id)
        kcs = [torch.zeros((cfg.B, cfg.Hkv, cfg.C, cfg.d), dtype=torch.bfloat16, device=device) for _ in range(cfg.n_layers)]
        vcs = [torch.zeros_like(kcs[0]) for _ in range(cfg.n_layers)]
        tv = target.TargetVerify(tw, cfg.B, cfg.T, cfg.Hq, cfg.Hkv, cfg.d, cfg.C, kcs, vcs, cfg.max_depth)
        cl_run = step.cache_len0.clone()

        def run_pass():
            cl_run.copy_(step.cache_len0)  # the step commits its accepted tokens; every replay starts from the same lengths
            tv.forward(step.tokens, cl_run, step.parent, step.n_nodes, max_cache_len=cfg.L)

        sg = torch.cuda.Stream()
        sg.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(sg):
            run_pass()
        torch.cuda.current_stream().wait_stream(sg)
        torch.cuda.synchronize()
        g_vp = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_vp):
            run_pass()
        for _ in range(3):
            g_vp.replay()
        ms_vp = time_graph(g_vp, max(3, K // 4), torch)
        assert int(tv.status_head.item()) == 0 and int(tv.status_qkv.abs().sum().item()) == 0
        assert int(tv.status_attn.abs().sum().item()) == 0 and int(tv.status_compact.abs().sum().item()) == 0
        lw0 = tw.layers[0]
        wbytes = cfg.n_layers * sum(t.numel() * 2 for t in (lw0.qkv, lw0.o, lw0.gate_up, lw0.down)) + tw.lm_head.numel() * 2
        kv_bytes = cfg.n_layers * 2 * cfg.B * cfg.Hkv * (cfg.L + cfg.T) * cfg.d * 2
        vp = dict(ms=ms_vp, rows=cfg.B * cfg.T, n_layers=cfg.n_layers, weight_bytes=wbytes, kv_bytes=kv_bytes, inter=inter,
                  flops=2.0 * cfg.B * cfg.T * (wbytes / 2), calls=2 + 5 * cfg.n_layers + 3,
                  accept_len=tv.accept_len.cpu().tolist())
        del tw, tv, kcs, vcs
    ms_e2e = 0.0
    if with_e2e:
        # end to end: per-step inputs from pinned host memory, decision back to the host, every step
        step.bind_host_inputs()
        for _ in range(3):
            step.run_host()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        Ke = max(5, min(K, 50))
        e0.record()
        for _ in range(Ke):
            step.run_host()
        e1.record()
        e1.synchronize()
        ms_e2e = e0.elapsed_time(e1) / Ke
    accept_lens = step.accept_len.cpu().tolist()
    ms_first, ms_med, ms_best, ms_attn, ms_attn_best, ms_e2e = replicas.max_over_ranks(
        [blocks[0], statistics.median(blocks), min(blocks), statistics.median(attn_blocks), min(attn_blocks), ms_e2e],
        device=device)
    rec = dict(step=step, ms=ms_first, ms_median=ms_med, ms_best=ms_best, n_blocks=len(blocks), ms_attn=ms_attn,
               ms_attn_best=ms_attn_best, ms_acc=ms_acc, ms_cmp=ms_cmp, ms_tree=ms_tree, ms_filt=ms_filt, lm=lm, qk=qk, dr=dr, vp=vp, ms_e2e=ms_e2e, accept_lens=accept_lens,
               clocks=clocks, K=K, Wm=Wm)
    return rec


FILTER_TOP_K, FILTER_TOP_P = 50, 0.9  # the filter the extra acceptance timing uses
TARGET_FRAC = 0.70  # of HBM peak, for the whole step on the 7B- and 8B-shaped configurations


def roofline_records(cfg, args, rec, pk):
    """`step_hbm`, `roofline` and `breakdown_ms` of one measured workload."""
    ab = algorithmic_bytes(cfg, args.temperature, rec["accept_lens"])
    ms = rec["ms_median"]
    attn_launch_ms = rec["ms_attn"] / cfg.n_layers
    achieved = ab["attention_per_layer"] / (attn_launch_ms * 1e-3) / 1e9
    flops_layer = 4.0 * cfg.B * cfg.Hq * cfg.T * (cfg.L + cfg.T) * cfg.d
    tflops = flops_layer / (attn_launch_ms * 1e-3) / 1e12
    step_gbs = ab["total"] / (ms * 1e-3) / 1e9
    step_hbm = dict(algorithmic_bytes=ab["total"], achieved_gbs=step_gbs, frac_of_measured_peak=step_gbs / pk["hbm_gbs"],
                    frac_of_nominal_8tbs=step_gbs / 8000.0, target_frac=TARGET_FRAC,
                    accept_bytes_counted=ab["accept"], accept_bytes_all_rows=ab["accept_all_rows"],
                    frac_of_measured_peak_all_rows=ab["total_all_rows"] / (ms * 1e-3) / 1e9 / pk["hbm_gbs"])
    # intensity of the contraction: G*T flop per byte of K/V; above the ridge of this GPU the tensor pipe is the roof
    intensity = (cfg.Hq // cfg.Hkv) * cfg.T
    ridge = pk["bf16_tflops"] * 1e3 / pk["hbm_gbs"]
    hbm = dict(achieved=achieved, peak=pk["hbm_gbs"], unit="GB/s", frac=achieved / pk["hbm_gbs"],
               peak_source=pk["source"] + " copy bandwidth")
    tensor = dict(achieved=tflops, peak=pk["bf16_tflops"], unit="TFLOP/s", frac=tflops / pk["bf16_tflops"],
                  peak_source=pk["source"] + " sustained bf16 GEMM")
    bound = "tensor" if intensity >= ridge else "hbm"
    roofline = dict(kernel="tree_attention (one layer)", bound=bound, **(tensor if bound == "tensor" else hbm),
                    target_frac=TARGET_FRAC, traffic=ncu_traffic(cfg.name),
                    algorithmic_bytes_per_launch=ab["attention_per_layer"], flops_per_launch=flops_layer,
                    us_per_launch=attn_launch_ms * 1e3, us_per_launch_best=rec["ms_attn_best"] / cfg.n_layers * 1e3,
                    flop_per_kv_byte=intensity, ridge_flop_per_byte=ridge, hbm=hbm, tensor=tensor)
    breakdown = dict(attention_all_layers=rec["ms_attn"], accept=rec["ms_acc"], compact=rec["ms_cmp"])
    if rec.get("ms_tree") is not None:
        breakdown["tree_build_not_in_step"] = rec["ms_tree"]
    if rec.get("ms_filt") is not None:
        breakdown[f"accept_filtered_top{FILTER_TOP_K}_p{FILTER_TOP_P}_not_in_step"] = rec["ms_filt"]
    if rec.get("lm") is not None:
        lm = rec["lm"]
        breakdown["lm_head_greedy_and_walk_not_in_step"] = lm["ms"]
        flops = 2.0 * lm["rows"] * lm["V"] * lm["H"]
        byts = 2.0 * lm["V"] * lm["H"] + 2.0 * lm["rows"] * lm["H"]  # the weights and the hidden states once (bf16)
        t = lm["ms"] * 1e-3
        tensor_bound = flops / byts >= ridge
        roofline["lm_head"] = dict(
            kernel="lm_head_greedy_kernel (+ merge and the greedy walk on the choices)", rows=lm["rows"], V=lm["V"], H=lm["H"],
            us=lm["ms"] * 1e3, bound="tensor" if tensor_bound else "hbm",
            tflops=flops / t * 1e-12, frac_of_tensor_peak=flops / t * 1e-12 / pk["bf16_tflops"],
            gbs=byts / t * 1e-9, frac_of_hbm_peak=byts / t * 1e-9 / pk["hbm_gbs"], flop_per_byte=flops / byts)
    if rec.get("qk") is not None:
        qk = rec["qk"]
        breakdown["qkv_rope_one_layer_not_in_step"] = qk["ms"]
        flops = 2.0 * qk["rows"] * qk["N"] * qk["H"]
        byts = 2.0 * qk["N"] * qk["H"] + 2.0 * qk["rows"] * qk["H"] + 2.0 * qk["rows"] * qk["N"]  # weights, states, outputs (bf16)
        t = qk["ms"] * 1e-3
        roofline["qkv_rope"] = dict(
            kernel="qkv_rope_kernel (+ the tree / rotary-table kernel in front)", rows=qk["rows"], N=qk["N"], H=qk["H"],
            us=qk["ms"] * 1e3, bound="tensor" if flops / byts >= ridge else "hbm", tflops=flops / t * 1e-12,
            frac_of_tensor_peak=flops / t * 1e-12 / pk["bf16_tflops"], gbs=byts / t * 1e-9,
            frac_of_hbm_peak=byts / t * 1e-9 / pk["hbm_gbs"], flop_per_byte=flops / byts)
    if rec.get("dr") is not None:
        dr = rec["dr"]
        breakdown["drafter_head_not_in_step"] = dr["ms"]
        t = dr["ms"] * 1e-3
        roofline["drafter_head"] = dict(
            kernel="one drafter head, Eq. 3-6: embed, Linear(concat[e,f]), decoder layer, LM-head top-k (8 calls)", rows=dr["rows"],
            mlp_width=dr["inter"], top_k=dr["k"], us=dr["ms"] * 1e3, weight_bytes=dr["weight_bytes"],
            bound="tensor" if dr["flops"] / dr["weight_bytes"] >= ridge else "hbm", gbs=dr["weight_bytes"] / t * 1e-9,
            frac_of_hbm_peak=dr["weight_bytes"] / t * 1e-9 / pk["hbm_gbs"], tflops=dr["flops"] / t * 1e-12,
            frac_of_tensor_peak=dr["flops"] / t * 1e-12 / pk["bf16_tflops"])
        if "round_ms" in dr:
            breakdown["drafter_round_3_heads_not_in_step"] = dr["round_ms"]
            roofline["drafter_head"]["round_of_three_heads"] = dict(
                what="three heads fill a 21-node tree level by level (rows per head below), tree rebuilt from the ranked choices after each",
                rows_per_head=dr["round_rows"], us=dr["round_ms"] * 1e3, weight_bytes=dr["round_weight_bytes"],
                gbs=dr["round_weight_bytes"] / (dr["round_ms"] * 1e-3) * 1e-9,
                frac_of_hbm_peak=dr["round_weight_bytes"] / (dr["round_ms"] * 1e-3) * 1e-9 / pk["hbm_gbs"])
    if rec.get("vp") is not None:
        vp = rec["vp"]
        breakdown["full_verify_pass_not_in_step"] = vp["ms"]
        t = vp["ms"] * 1e-3
        byts = vp["weight_bytes"] + vp["kv_bytes"]
        roofline["verify_pass"] = dict(
            kernel="the target's whole greedy verify pass: embed, %d decoder layers (q/k/v + rotary, tree attention, projections, gated "
                   "MLP), LM head + greedy choice, walk, compaction (%d calls)" % (vp["n_layers"], vp["calls"]),
            rows=vp["rows"], n_layers=vp["n_layers"], mlp_width=vp["inter"], ms=vp["ms"], weight_bytes=vp["weight_bytes"],
            kv_bytes=vp["kv_bytes"], bound="tensor" if vp["flops"] / byts >= ridge else "hbm", gbs=byts / t * 1e-9,
            frac_of_hbm_peak=byts / t * 1e-9 / pk["hbm_gbs"], tflops=vp["flops"] / t * 1e-12,
            frac_of_tensor_peak=vp["flops"] / t * 1e-12 / pk["bf16_tflops"], nodes_per_s=vp["rows"] / t, accept_len=vp["accept_len"])
    return ab, step_hbm, roofline, breakdown


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2506_14158_b200 import replicas
    from paper_2506_14158_b200 import workloads as W

    rank, world, local = replicas.env_rank_world()
    if world != args.gpus:
        if world == 1 and args.gpus > 1:
            raise SystemExit("launch with torchrun for --gpus > 1")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    import __graft_entry__ as entry

    if rank == 0:
        entry.build()
    if world > 1:
        dist.barrier()
    cfg = get_config(args)
    rec = measure(cfg, args, device, rank, world, with_e2e=True)
    step, K, Wm = rec["step"], rec["K"], rec["Wm"]
    h2d, d2h = getattr(step, "h2d_bytes", 0), getattr(step, "d2h_bytes", 0)
    launches = K * rec["n_blocks"] * step.launches_per_step(attn_kernels_per_layer(cfg))
    rec["step"] = None
    del step
    also = None
    if cfg.name == "c2x32" and not args.no_also and not args.capacity and not args.paged:
        # the 8B-shaped step, measured the same way in the same run (no host-buffer leg: 365 MB per step over PCIe)
        import gc

        gc.collect()
        torch.cuda.empty_cache()
        cfg2 = W.CONFIGS["c4x32"]
        rec2 = measure(cfg2, args, device, rank, world, with_e2e=False)
        launches += K * rec2["n_blocks"] * rec2["step"].launches_per_step(attn_kernels_per_layer(cfg2))
        rec2["step"] = None
        also = (cfg2, rec2)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    pk = peaks()
    ab, step_hbm, roofline, breakdown = roofline_records(cfg, args, rec, pk)
    nodes = cfg.B * cfg.T * world
    ms = rec["ms"]
    accept_lens = rec["accept_lens"]
    config = config_record(cfg, args, world)
    config.update(parallelism=f"replicas x{world} (no collective)",
                  l2="inputs larger than L2 (independent KV cache per layer)" if ab["attention"] > (126 << 20)
                  else "working set fits L2: launch-latency case, not a bandwidth claim",
                  launch="whole step replayed as one CUDA graph",
                  max_cache_len_hint=0 if args.no_hint else cfg.L,
                  cache_layout=f"paged, {args.paged} slots per page, pages scattered" if args.paged else "contiguous")
    line = dict(
        metric=METRIC, value=replicas.aggregate_nodes_per_second(cfg.B * cfg.T, world, ms), unit=UNIT, n_gpus=world,
        steps=K, warmup=Wm, ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None,
        dtype="bf16" if cfg.dtype == "bf16" else "f32", data="synthetic (seeded)", config=config,
        timing=dict(blocks=rec["n_blocks"], steps_per_block=K, ms_per_step_first_block=ms,
                    ms_per_step_median=rec["ms_median"], ms_per_step_best=rec["ms_best"],
                    note="value and ms_per_step are the first block (exactly K steps); step_hbm and roofline use the medians"),
        step_hbm=step_hbm, roofline=roofline, breakdown_ms=breakdown,
        e2e=(dict(value=nodes / (rec["ms_e2e"] * 1e-3), unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                  ms_per_step=rec["ms_e2e"]) if rec["ms_e2e"] > 0 else None),
        gpu_launches=launches,
        accepted_per_step=dict(accept_len=accept_lens, mean_accepted_plus_bonus=sum(a + 1 for a in accept_lens) / len(accept_lens)),
        clocks=rec["clocks"],
        paper_context="S4C reports 2.26x-2.60x end-to-end speedup (A100 / 4x RTX 4090, FP16, batch 1); no verify-step number",
    )
    if also is not None:
        cfg2, rec2 = also
        ab2, step_hbm2, roofline2, breakdown2 = roofline_records(cfg2, args, rec2, pk)
        line["also"] = dict(workload=cfg2.name, config=config_record(cfg2, args, world),
                            value=replicas.aggregate_nodes_per_second(cfg2.B * cfg2.T, world, rec2["ms"]), unit=UNIT,
                            ms_per_step=rec2["ms"], ms_per_step_median=rec2["ms_median"], ms_per_step_best=rec2["ms_best"],
                            blocks=rec2["n_blocks"], step_hbm=step_hbm2, roofline=roofline2, breakdown_ms=breakdown2,
                            accept_len=rec2["accept_lens"], clocks=rec2["clocks"])
    if not args.no_cpu_baseline and world == 1:
        import oracle

        t_cpu, desc, ref = oracle_sample(cfg, args.temperature)
        t_one, desc_one, _ = oracle_sample(cfg, args.temperature, layers_sample=2, threads=1)
        line["cpu_baseline"] = dict(value=cfg.B * cfg.T / t_cpu, unit=UNIT, cores=oracle.max_threads(), kind="oracle",
                                    sample=desc + " -- this all-thread figure is the one quoted as `value`",
                                    single_thread=dict(value=cfg.B * cfg.T / t_one, unit=UNIT, cores=1, sample=desc_one))
        line["parity_in_bench"] = dict(accept_len_matches_oracle=[int(a) for a in ref["accept_len"]] == accept_lens)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_sweep_all(args):
    """Config 5, every point: the 7B layer shape x 32 layers with an independent cache per layer, context 512..32768,
    trees of 16..128 nodes, batch 1/4/16.  One JSON line per point (nodes/s, HBM GB/s of the step and of the attention
    launches); points whose 32 caches do not fit the device are recorded as such, never aliased."""
    import gc
    from dataclasses import replace

    import torch

    import __graft_entry__ as entry
    from paper_2506_14158_b200 import workloads as W

    entry.build()
    torch.cuda.set_device(0)
    device = torch.device("cuda", 0)
    pk = peaks()
    free_b, total_b = torch.cuda.mem_get_info()
    for B in (1, 4, 16):
        for T in (16, 32, 64, 128):
            for L in (512, 1024, 2048, 4096, 8192, 16384, 32768):
                cfg = W.sweep_config(L, T, B, args.layers)
                if args.capacity:
                    if args.capacity < L + T:
                        continue
                    cfg = replace(cfg, capacity=args.capacity)
                kv = 2 * cfg.n_layers * cfg.B * cfg.Hkv * cfg.C * cfg.d * 2
                point = dict(workload=cfg.name, B=B, T=T, L=L, C=cfg.C, hint=0 if args.no_hint else L,
                             n_layers=cfg.n_layers, kv_gb=round(kv / 1e9, 2))
                if kv > 0.8 * total_b:
                    point["result"] = "exceeds device memory"
                    print(json.dumps(point), flush=True)
                    continue
                step = build_step(cfg, args.temperature, device, hint=not args.no_hint)
                g_step, g_attn = step.capture("step"), step.capture("attention")
                iters = 20 if kv < (8 << 30) else 5
                for _ in range(3):
                    g_step.replay()
                torch.cuda.synchronize()
                ms = time_graph(g_step, iters, torch)
                step.reset_lengths()  # attention alone is timed on the committed lengths
                torch.cuda.synchronize()
                ms_attn = time_graph(g_attn, iters, torch)
                ab = algorithmic_bytes(cfg, args.temperature, step.accept_len.cpu().tolist())
                point.update(ms_per_step=round(ms, 4), nodes_per_s=round(B * T / (ms * 1e-3), 1),
                             step_gbs=round(ab["total"] / (ms * 1e-3) / 1e9, 1),
                             attn_us_per_layer=round(ms_attn / cfg.n_layers * 1e3, 2),
                             attn_gbs=round(ab["attention"] / (ms_attn * 1e-3) / 1e9, 1),
                             attn_frac_of_measured_peak=round(ab["attention"] / (ms_attn * 1e-3) / 1e9 / pk["hbm_gbs"], 3))
                print(json.dumps(point), flush=True)
                del step, g_step, g_attn
                gc.collect()
                torch.cuda.empty_cache()


def run_launch_floor(args):
    """The floor under one per-layer launch: CUDA graphs of `--layers` EMPTY kernels (s4c_launch_floor) with the launch
    shape of an attention launch -- block size, dynamic shared memory, cluster size, tensor-memory allocation, cluster
    barriers, programmatic dependent launch -- timed like the attention graph.  One JSON line per shape."""
    import torch

    import __graft_entry__ as entry

    entry.build()
    from paper_2506_14158_b200 import s4c

    torch.cuda.set_device(0)
    word = torch.full((1,), 1024, dtype=torch.int32, device="cuda")
    n = args.layers
    shapes = [  # (name, ctas, cluster, threads, smem, tmem columns, cluster barriers, dependent launch)
        ("bare: 128 CTAs x 224 threads, 1 KB", 128, 1, 224, 1024, 0, 0, False),
        ("+ programmatic dependent launch", 128, 1, 224, 1024, 0, 0, True),
        ("+ 200 KB shared memory", 128, 1, 224, 200 * 1024, 0, 0, True),
        ("+ 256 tensor-memory columns", 128, 1, 224, 200 * 1024, 256, 0, True),
        ("+ clusters of 4", 128, 4, 224, 200 * 1024, 256, 0, True),
        ("+ 1 cluster barrier (7B shape, pushed partials)", 128, 4, 224, 200 * 1024, 256, 1, True),
        ("+ 2 cluster barriers (parked partials)", 128, 4, 224, 200 * 1024, 256, 2, True),
        ("same without dependent launch", 128, 4, 224, 200 * 1024, 256, 1, False),
        ("148 CTAs, no cluster, dependent launch", 148, 1, 224, 200 * 1024, 256, 0, True),
        ("8B shape: 128 CTAs x 384 threads, clusters of 4, 512 columns, 2 barriers", 128, 4, 384, 220 * 1024, 512, 2, True),
        ("half-SM CTAs: 296 x 224 threads, 100 KB, 256 columns", 296, 1, 224, 100 * 1024, 256, 0, True),
    ]
    for name, ctas, cluster, threads, smem, tmem, syncs, pdl in shapes:
        fn = lambda: [s4c.launch_floor(ctas, cluster, threads, smem, tmem, syncs, pdl, word) for _ in range(n)]
        st = torch.cuda.Stream()
        st.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(st):
            fn()
        torch.cuda.current_stream().wait_stream(st)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        for _ in range(5):
            g.replay()
        torch.cuda.synchronize()
        blocks = time_blocks(g, args.steps, torch, 0.2)
        print(json.dumps(dict(workload="launch-floor", shape=name, ctas=ctas, cluster=cluster, threads=threads,
                              smem_bytes=smem, tmem_cols=tmem, cluster_barriers=syncs, dependent_launch=pdl,
                              launches_per_graph=n, us_per_launch_median=round(statistics.median(blocks) / n * 1e3, 3),
                              us_per_launch_best=round(min(blocks) / n * 1e3, 3))), flush=True)


def attn_kernels_per_layer(cfg):
    from paper_2506_14158_b200 import s4c
    import torch

    dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    return 2 if s4c.tree_attention_workspace_bytes(cfg.B, cfg.T, cfg.Hq, cfg.Hkv, cfg.d, cfg.C, dt) > 0 else 1


if __name__ == "__main__":
    a = parse_args()
    if a.workload == "sweep-all":
        run_sweep_all(a)
    elif a.workload == "launch-floor":
        run_launch_floor(a)
    elif a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
