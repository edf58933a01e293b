#!/usr/bin/env python
"""Benchmark of the S4C verify step on B200: verified tree-nodes/s per verify step and achieved HBM GB/s.

A step is one pass of the whole hot path over one batch of seeded synthetic input: n_layers tree-attention
launches, one acceptance, one compaction of every layer's cache (all through the C ABI, replayed as one CUDA
graph).  The default workload "c2x32" is the LLaMA-2-7B-shaped verify step at full depth: the config-2 layer
(32 heads x 128, bf16 cache of 1024 tokens, 26-node tree, vocab 32000) stacked 32 times with an independent
cache per layer, temperature 1.0.  Its 0.56 GB of KV per step is larger than L2, so no flush is needed.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2x32|c2|c3|c4|c4x32|c1|sweep --L --T --B]
    python bench.py --impl reference     # the float64 CPU oracle on a bounded sample of the same workload

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
    return ap.parse_args()


def get_config(args):
    from paper_2506_14158_b200 import workloads as W

    if args.workload == "sweep":
        return W.sweep_config(args.L, args.T, args.B, args.layers)
    return W.CONFIGS[args.workload]


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
    "c2x32": dict(bytes=18109696, sha256="b5c2563c704ac15f79435ccd87416aa470346baca80d7813807bbcc84aae89f9",
                  profile="profiles/tree_attention_tc_c2x32_ncu_full.md"),
    "c4x32": dict(bytes=71402496, sha256="b5c2563c704ac15f79435ccd87416aa470346baca80d7813807bbcc84aae89f9",
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
    return dict(attention_per_layer=attn_layer, attention=attn_layer * cfg.n_layers, accept=accept, compact=compact,
                total=attn_layer * cfg.n_layers + accept + compact)


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
def oracle_sample(cfg, temperature, layers_sample=None):
    """Times the float64 oracle, as it stands, on a bounded sample of the workload: `layers_sample` attention
    layers (default: as many as fit ~10 s, at least one), the whole acceptance, and the compaction of those
    layers; the attention and compaction times are scaled to n_layers.  Returns (seconds per step, description)."""
    import numpy as np

    import oracle
    from paper_2506_14158_b200 import workloads as W

    parent = W.make_trees(cfg)
    x = W.make_accept_inputs(cfg, parent, temperature, token_mode="topk")
    cl = np.full(cfg.B, cfg.L, dtype=np.int32)
    q, k, v = W.make_attention_inputs(cfg, 0)
    q64, k64, v64 = W.to_f64(q), W.to_f64(k), W.to_f64(v)
    t = time.perf_counter()
    oracle.tree_attention(q64, k64, v64, cl, parent)
    t_layer = time.perf_counter() - t
    n_s = layers_sample or max(1, min(cfg.n_layers, int(10.0 / max(t_layer, 1e-3))))
    for _ in range(n_s - 1):
        t = time.perf_counter()
        oracle.tree_attention(q64, k64, v64, cl, parent)
        t_layer = min(t_layer, time.perf_counter() - t) if n_s > 4 else (t_layer + time.perf_counter() - t)
    if n_s <= 4:
        t_layer /= n_s
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
    total = t_layer * cfg.n_layers + t_accept + t_compact * cfg.n_layers
    desc = (f"float64 C oracle, {oracle.max_threads()} OpenMP threads: {n_s} attention layer(s) of {cfg.n_layers} timed "
            f"({t_layer * 1e3:.1f} ms each), whole acceptance ({t_accept * 1e3:.1f} ms), compaction of 1 layer "
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
    for _ in range(min(args.warmup, 1)):
        oracle_sample(cfg, args.temperature, layers_sample=1)
    desc = ""
    for _ in range(steps):
        t, desc, _ = oracle_sample(cfg, args.temperature, layers_sample=1)
        times.append(t)
    tstep = statistics.median(times)
    value = cfg.B * cfg.T / tstep
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=steps,
                warmup=min(args.warmup, 1), ms_per_step=tstep * 1e3, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f64", data="synthetic (seeded)",
                config=dict(workload=cfg.name, B=cfg.B, T=cfg.T, L=cfg.L, Hq=cfg.Hq, Hkv=cfg.Hkv, d=cfg.d, V=cfg.V,
                            n_layers=cfg.n_layers, temperature=args.temperature),
                cpu_baseline=dict(value=value, unit=UNIT, cores=oracle.max_threads(), kind="oracle", sample=desc),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- the CUDA arm
def build_step(cfg, temperature, device, seed_shift=0):
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
    stoch = temperature > 0
    step = VerifyStep(qs, ks, vs, torch.full((cfg.B,), cfg.L, dtype=torch.int32, device=device), to(parent),
                      to(x["tokens"]), to(x["logits"]), to(x["draft_probs"]) if stoch else None,
                      to(x["uniforms"]) if stoch else None, temperature, cfg.max_depth,
                      feat_in=W.make_features(cfg_gen).to(device), stacked=(q_all, k_all, v_all))
    return step


def time_graph(graph, iters, torch):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        graph.replay()
    e1.record()
    e1.synchronize()
    return e0.elapsed_time(e1) / iters  # ms per replay


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2506_14158_b200 import replicas

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
    K, Wm = args.steps, max(3, args.warmup)
    step = build_step(cfg, args.temperature, device, seed_shift=rank)
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
    sampler = ClockSampler(local) if rank == 0 else None
    t0 = time.time()
    ms = time_graph(g_step, K, torch)
    barrier()
    t1 = time.time()
    clocks = sampler.stop(t0, t1) if sampler else None
    # dominant-kernel leg: the n_layers attention launches alone, same buffers, same stream, CUDA events
    step.reset_lengths()  # the step's compaction advanced the lengths: attention is timed on the committed ones
    for _ in range(3):
        g_attn.replay()
    torch.cuda.synchronize()
    ms_attn = time_graph(g_attn, K, torch)
    ms_acc = time_graph(g_acc, K, torch)  # L2-resident when the logits fit L2: informational only
    ms_cmp = time_graph(g_cmp, K, torch)
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

    ms, ms_attn, ms_e2e = replicas.max_over_ranks([ms, ms_attn, ms_e2e], device=device)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    pk = peaks()
    ab = algorithmic_bytes(cfg, args.temperature, accept_lens)
    nodes = cfg.B * cfg.T * world
    attn_launch_ms = ms_attn / cfg.n_layers
    achieved = ab["attention_per_layer"] / (attn_launch_ms * 1e-3) / 1e9
    flops_layer = 4.0 * cfg.B * cfg.Hq * cfg.T * (cfg.L + cfg.T) * cfg.d
    attn_kernels = attn_kernels_per_layer(cfg)
    line = dict(
        metric=METRIC, value=replicas.aggregate_nodes_per_second(cfg.B * cfg.T, world, ms), unit=UNIT, n_gpus=world, steps=K, warmup=Wm, ms_per_step=ms,
        higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16" if cfg.dtype == "bf16" else "f32",
        data="synthetic (seeded)",
        config=dict(workload=cfg.name, B=cfg.B, T=cfg.T, L=cfg.L, Hq=cfg.Hq, Hkv=cfg.Hkv, d=cfg.d, V=cfg.V,
                    n_layers=cfg.n_layers, temperature=args.temperature, parallelism=f"replicas x{world} (no collective)",
                    l2="inputs larger than L2 (independent KV cache per layer)" if ab["attention"] > (126 << 20)
                    else "working set fits L2: launch-latency case, not a bandwidth claim",
                    launch="whole step replayed as one CUDA graph"),
        step_hbm=dict(algorithmic_bytes=ab["total"], achieved_gbs=ab["total"] / (ms * 1e-3) / 1e9,
                      frac_of_measured_peak=ab["total"] / (ms * 1e-3) / 1e9 / pk["hbm_gbs"],
                      frac_of_nominal_8tbs=ab["total"] / (ms * 1e-3) / 1e9 / 8000.0),
        roofline=dict(kernel="tree_attention (one layer)", bound="hbm", achieved=achieved, peak=pk["hbm_gbs"],
                      unit="GB/s", frac=achieved / pk["hbm_gbs"], peak_source=pk["source"] + " copy bandwidth",
                      traffic=ncu_traffic(cfg.name), algorithmic_bytes_per_launch=ab["attention_per_layer"],
                      us_per_launch=attn_launch_ms * 1e3, tensor_tflops=flops_layer / (attn_launch_ms * 1e-3) / 1e12),
        breakdown_ms=dict(attention_all_layers=ms_attn, accept=ms_acc, compact=ms_cmp),
        e2e=dict(value=nodes / (ms_e2e * 1e-3), unit=UNIT, h2d_bytes_per_step=step.h2d_bytes,
                 d2h_bytes_per_step=step.d2h_bytes, ms_per_step=ms_e2e),
        gpu_launches=K * step.launches_per_step(attn_kernels),
        accepted_per_step=dict(accept_len=accept_lens, mean_accepted_plus_bonus=sum(a + 1 for a in accept_lens) / len(accept_lens)),
        clocks=clocks,
        paper_context="S4C reports 2.26x-2.60x end-to-end speedup (A100 / 4x RTX 4090, FP16, batch 1); no verify-step number",
    )
    if not args.no_cpu_baseline and world == 1:
        t_cpu, desc, ref = oracle_sample(cfg, args.temperature)
        import oracle

        line["cpu_baseline"] = dict(value=cfg.B * cfg.T / t_cpu, unit=UNIT, cores=oracle.max_threads(), kind="oracle",
                                    sample=desc)
        line["parity_in_bench"] = dict(accept_len_matches_oracle=[int(a) for a in ref["accept_len"]] == accept_lens)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_sweep_all(args):
    """Config 5, every point: the 7B layer shape x 32 layers with an independent cache per layer, context 512..32768,
    trees of 16..128 nodes, batch 1/4/16.  One JSON line per point (nodes/s, HBM GB/s of the step and of the attention
    launches); points whose 32 caches do not fit the device are recorded as such, never aliased."""
    import gc

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
                kv = 2 * cfg.n_layers * cfg.B * cfg.Hkv * cfg.C * cfg.d * 2
                point = dict(workload=cfg.name, B=B, T=T, L=L, n_layers=cfg.n_layers, kv_gb=round(kv / 1e9, 2))
                if kv > 0.8 * total_b:
                    point["result"] = "exceeds device memory"
                    print(json.dumps(point), flush=True)
                    continue
                step = build_step(cfg, args.temperature, device)
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


def attn_kernels_per_layer(cfg):
    from paper_2506_14158_b200 import s4c
    import torch

    dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    return 2 if s4c.tree_attention_workspace_bytes(cfg.B, cfg.T, cfg.Hq, cfg.Hkv, cfg.d, cfg.C, dt) > 0 else 1


if __name__ == "__main__":
    a = parse_args()
    if a.workload == "sweep-all":
        run_sweep_all(a)
    elif a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
