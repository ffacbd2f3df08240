#!/usr/bin/env python
"""Benchmark of the token-tree verify step (ancestor mask -> tree attention -> Algorithm 2 walk).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--temperature T]
    python bench.py --impl reference ...      # the fp64 CPU oracle on the host cores, same metric

One "step" is one pass of the whole hot path over one synthetic request.  The K timed steps are
captured in one CUDA graph and replayed between two CUDA events; inputs rotate over enough
independent copies that every step reads memory that is not in L2.  One JSON line is printed by
rank 0.  With N > 1 (torchrun) every rank verifies its own requests (weak scaling, no data-path
collective) and the time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2402_12374_b200 import workloads as W

METRIC = "us_per_tree_verify_step"
UNIT = "us/step"
L2_BYTES = 126 * 1024 * 1024

# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the attention kernel, from
# the ncu captures summarised under profiles/; None where no capture exists for that workload.
NCU_TRAFFIC_BYTES = {
    "tiny": 2560000,          # profiles/tree_attention_umma_traffic.md
    "llama2-7b": 18418432,    # profiles/tree_attention_umma_llama2-7b.md
    "llama2-13b": 45945856,   # profiles/tree_attention_umma_traffic.md
    "vicuna-33b": 65200128,   # profiles/tree_attention_umma_traffic.md
    "llama3-70b": 32801792,   # profiles/tree_attention_umma_llama3-70b.md
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"], source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.002):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:  # NVML missing: report nulls rather than fail the run
            self.nv = None
        self.period = period_s

    def _loop(self):
        nv = self.nv
        names = {
            "hw_slowdown": nv.nvmlClocksEventReasonHwSlowdown if hasattr(nv, "nvmlClocksEventReasonHwSlowdown") else 0x8,
            "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4, "hw_power_brake": 0x80,
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def max_over_ranks(value: float, device=None) -> float:
    """Maximum of a per-rank number over all ranks of the default process group (1 rank: itself)."""
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_us_per_step(ms_total_max: float, steps: int, world: int) -> float:
    """Every rank verifies its own request per step (weak scaling): the job completes `world` steps in
    the time of one, so the whole-job figure is the max-over-ranks step time divided by `world`."""
    return 1e3 * ms_total_max / steps / world


def rank_seed_base(rank: int) -> int:
    return 1000 * rank


def n_sets(bytes_per_set: int, lo: int = 2, hi: int = 48) -> int:
    return max(lo, min(hi, math.ceil(3 * L2_BYTES / max(1, bytes_per_set))))


def build_requests(cfg, T, rank, n_attn, n_verify, tree="random", parent=None):
    """Host-side inputs for this rank: n_attn attention sets and n_verify logit sets (seeds differ by rank).
    tree = "dp": the tree comes from the library's own construction (seq_tree_build, a host call) on the
    acceptance vector the paper prints, within the config's size, depth and fan-out bounds."""
    base = rank_seed_base(rank)
    if parent is not None:
        pass
    elif tree == "dp":
        from paper_2402_12374_b200 import binding as B

        parent, _ = B.seq_tree_build(W.PAPER_ACCEPTANCE_VECTOR, cfg.n_tree, cfg.max_depth, cfg.max_fanout or 31)
        assert len(parent) == cfg.n_tree
    else:
        parent = W.make_tree(cfg, base)
    attn = [W.make_attention_inputs(cfg, base + s, parent=parent) for s in range(n_attn)]
    ver = [W.make_verify_inputs(cfg, T, base + s, parent=parent) for s in range(n_verify)]
    return parent, attn, ver


def oracle_step_sample(cfg, parent, ai, vi, T, budget_flops=1.5e9):
    """Times the oracle on one step, attention restricted to a leading block of nodes (closed under
    'parent') when the whole tree would take too long; returns (seconds scaled to a full step, note)."""
    from oracle import oracle as O

    n = len(parent)
    L = cfg.prefix_len
    per_node = 4.0 * cfg.head_dim * cfg.num_q_heads * (L + 8)
    m = int(max(1, min(n, budget_flops // per_node)))
    t0 = time.perf_counter()
    O.tree_attention(ai.q[:m], ai.k_cache[:, : L + m], ai.v_cache[:, : L + m], parent[:m], L)
    t_attn = (time.perf_counter() - t0) * (n / m)
    t0 = time.perf_counter()
    O.mask_from_parents(parent)
    O.tree_verify(vi.parent, vi.tokens, vi.target_logits, vi.draft_logits, T, vi.uniforms)
    t_ver = time.perf_counter() - t0
    note = (f"1 step: mask + Algorithm 2 walk in full, attention on the first {m} of {n} nodes "
            f"(time scaled by {n}/{m}), fp64, gcc -O2 -fopenmp")
    return t_attn + t_ver, note


def run_reference(args, cfg, T):
    """--impl reference: the oracle, as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle as O

    parent = None
    if args.tree == "dp":  # this arm runs none of the library: the oracle's own statement of the dynamic program
        from oracle import tree_dp

        parent, _ = tree_dp.build_tree(W.PAPER_ACCEPTANCE_VECTOR, cfg.n_tree, cfg.max_depth, cfg.max_fanout or 31)
    parent, attn, ver = build_requests(cfg, T, 0, 1, 1, parent=parent)
    for _ in range(min(args.warmup, 2)):
        oracle_step_sample(cfg, parent, attn[0], ver[0], T)
    steps = min(args.steps, 20)
    times, note = [], ""
    for _ in range(steps):
        t, note = oracle_step_sample(cfg, parent, attn[0], ver[0], T)
        times.append(t)
    us = 1e6 * sum(times) / len(times)
    cores = O.num_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": us, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": min(args.warmup, 2), "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "temperature": T},
        "cpu_baseline": {"value": us, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": note},
        "e2e": {"value": us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def draft_sample_leg(cfg, parent, ver_h, T, dev, stream, peaks) -> dict:
    """Not part of the timed step: the draft side's draw of every internal node's children (exponential sort),
    timed on its own in a CUDA graph over rotating logit sets.  One row per internal node, k = the tree's
    largest fan-out, uniforms of the same shape as the logits (seeded on the device)."""
    from paper_2402_12374_b200 import binding as B

    kids = W.children_lists(parent)
    internal = [v for v in range(len(parent)) if kids[v]]
    k = min(64, max(len(kids[v]) for v in internal))
    rows = torch.tensor(internal, dtype=torch.long, device=dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(20240212)
    logit_sets = [vi.draft_logits.to(dev)[rows].contiguous() for vi in ver_h[:4]]
    unif_sets = [torch.rand(ls.shape, device=dev, generator=gen).clamp_(1e-7, 1 - 1e-7) for ls in logit_sets]
    out = torch.empty((len(internal), k), dtype=torch.int32, device=dev)
    ws = torch.empty(len(internal) * ((cfg.vocab + 4095) // 4096) * k * 8 + 256, dtype=torch.uint8, device=dev)
    reps = 40
    with torch.cuda.stream(stream):
        for i in range(3):
            B.seq_tree_draft_sample(logit_sets[i % len(logit_sets)], T, unif_sets[i % len(logit_sets)], k, tokens_out=out,
                                    workspace=ws, stream=stream)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(reps):
                B.seq_tree_draft_sample(logit_sets[i % len(logit_sets)], T, unif_sets[i % len(logit_sets)], k, tokens_out=out,
                                        workspace=ws, stream=stream)
        g.replay()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        g.replay()
        e1.record(stream)
        stream.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / reps
    nbytes = 2 * len(internal) * cfg.vocab * 4
    gbs = nbytes / (us * 1e-6) / 1e9
    return {"us_per_call": us, "rows": len(internal), "k": k, "vocab": cfg.vocab, "gpu_launches_per_call": 2,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "algorithmic_bytes": nbytes, "traffic": None},
            "note": "logits + uniforms of every internal node read once; outside the timed step"}


def kv_commit_leg(cfg, parent, dev, stream, peaks) -> dict:
    """Not part of the timed step: the commit of an accepted path into the whole model's key/value cache (every
    layer's planes), timed per call with event nodes inside one CUDA graph, a write of a buffer larger than L2
    before every call.  The path: the root and, level by level, the last child that has children of its own (else
    the last child), five nodes at most."""
    from paper_2402_12374_b200 import binding as B

    layers = W.NUM_LAYERS[cfg.name]
    kids = W.children_lists(parent)
    path = [0]
    while kids[path[-1]] and len(path) < 5:
        inner = [c for c in kids[path[-1]] if kids[c]]
        path.append(inner[-1] if inner else kids[path[-1]][-1])
    n, L = len(parent), cfg.prefix_len
    planes = layers * cfg.num_kv_heads
    dt = W.TORCH_DTYPES[cfg.dtype]
    k = torch.zeros((planes, L + n, cfg.head_dim), dtype=dt, device=dev)
    v = torch.zeros((planes, L + n, cfg.head_dim), dtype=dt, device=dev)
    k[:, L:].normal_()
    v[:, L:].normal_()
    path_d = torch.zeros(n, dtype=torch.int32, device=dev)
    path_d[: len(path)] = torch.tensor(path, dtype=torch.int32)
    plen = torch.tensor([len(path)], dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    flush = torch.empty(160 << 20, dtype=torch.uint8, device=dev)
    reps = 20
    evs = [[torch.cuda.Event(enable_timing=True, external=True) for _ in range(2)] for _ in range(reps)]
    with torch.cuda.stream(stream):
        for _ in range(3):
            B.seq_tree_kv_commit(k, v, L, n, path_d, plen, dev_status=status, stream=stream)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(reps):
                flush.fill_(i)
                evs[i][0].record(stream)
                B.seq_tree_kv_commit(k, v, L, n, path_d, plen, dev_status=status, stream=stream)
                evs[i][1].record(stream)
        g.replay()
        stream.synchronize()
        g.replay()
        stream.synchronize()
        # and back to back, the rows still in L2 from the call before (the device clock ticks coarsely: means, not medians)
        gw = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gw, stream=stream):
            for i in range(2 * reps):
                B.seq_tree_kv_commit(k, v, L, n, path_d, plen, dev_status=status, stream=stream)
        gw.replay()
        stream.synchronize()
        w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        w0.record(stream)
        gw.replay()
        w1.record(stream)
        stream.synchronize()
    if int(status.item()) != 0:
        raise RuntimeError(f"kv_commit dev_status = {int(status.item())}")
    us = float(np.mean([a.elapsed_time(b) * 1e3 for a, b in evs]))
    us_warm = w0.elapsed_time(w1) * 1e3 / (2 * reps)
    moved = sum(int(p != i) for i, p in enumerate(path))
    nbytes = 2 * 2 * planes * moved * cfg.head_dim * k.element_size()
    gbs = nbytes / (us * 1e-6) / 1e9
    return {"us_per_call": us, "us_per_call_l2_warm": us_warm, "layers": layers, "planes": planes, "path_len": len(path), "rows_moved": moved,
            "gpu_launches_per_call": 1, "l2": "flushed before every call",
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "algorithmic_bytes": nbytes, "traffic": None},
            "note": "moved rows of every plane read and written once; latency-bound at this size; outside the timed step"}


def tree_search_leg(cfg, T, dev, stream) -> dict:
    """Not part of the timed step: t(n) of this library's verify step (attention + verification; NOT a whole model
    forward, which a caller measures for itself) on trees from seq_tree_build of growing size, and the
    Speedup(n, d) = G(n, d) / (t(n) + d c) search of Section 4.1 on it for two draft costs c.  Inputs are drawn on
    the device; each size is timed as a CUDA graph of calls rotating over sets larger than L2."""
    from paper_2402_12374_b200 import binding as B

    Bmax = cfg.max_fanout or 31
    N, Dmax = cfg.n_tree, cfg.max_depth
    sizes = sorted({n for n in (1, 4, 16, 32, 64, 128, 256, 512, 768, 1024) if n < N} | {N})
    dt = W.TORCH_DTYPES[cfg.dtype]
    gen = torch.Generator(device=dev)
    gen.manual_seed(7)
    V = cfg.vocab
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    times = {}
    for n in sizes:
        parent, _ = B.seq_tree_build(W.PAPER_ACCEPTANCE_VECTOR, n, Dmax, Bmax)
        n = len(parent)
        kv_bytes = 2 * cfg.num_kv_heads * (cfg.prefix_len + n) * cfg.head_dim * 2
        sets = max(2, min(16, math.ceil(2 * L2_BYTES / kv_bytes)))
        parent_d = torch.from_numpy(parent).to(dev)
        kids = W.children_lists(parent)
        calls = []
        for s in range(sets):
            q = torch.randn((n, cfg.num_q_heads, cfg.head_dim), device=dev, generator=gen).to(dt)
            k = torch.randn((cfg.num_kv_heads, cfg.prefix_len + n, cfg.head_dim), device=dev, generator=gen).to(dt)
            v_ = torch.randn((cfg.num_kv_heads, cfg.prefix_len + n, cfg.head_dim), device=dev, generator=gen).to(dt)
            tl = 3.0 * torch.randn((n, V), device=dev, generator=gen)
            dl = tl + torch.randn((n, V), device=dev, generator=gen)
            u = torch.rand(n + 1, device=dev, generator=gen)
            # children = the first draws without replacement from the draft's distribution (Gumbel top-k), as in the
            # host-side recipe of the timed step
            tokens = torch.zeros(n, dtype=torch.int32, device=dev)
            for node, ch in enumerate(kids):
                if ch:
                    gum = -torch.log(-torch.log(torch.rand(V, device=dev, generator=gen).clamp_(1e-9, 1 - 1e-7)))
                    tokens[ch] = torch.topk(dl[node] / T + gum, len(ch)).indices.to(torch.int32)
            calls.append((B.AttentionCall(q, k, v_, None, cfg.prefix_len, parent=parent_d, dev_status=status),
                          B.VerifyCall(parent_d, tokens, tl, dl, T, u, dev_status=status)))
        reps = 4 * sets
        with torch.cuda.stream(stream):
            for a, vcall in calls[:2]:
                a.run(stream)
                vcall.run(stream)
            stream.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for i in range(reps):
                    calls[i % sets][0].run(stream)
                    calls[i % sets][1].run(stream)
            g.replay()
            stream.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            g.replay()
            e1.record(stream)
            stream.synchronize()
        times[n] = e0.elapsed_time(e1) * 1e3 / reps
        del calls
    if int(status.item()) != 0:
        raise RuntimeError(f"tree_search dev_status = {int(status.item())}")
    ns = sorted(times)
    t_of_n = np.interp(np.arange(N + 1), ns, [times[n] / times[1] for n in ns])
    t_of_n[0] = 1.0
    _, _, table = B.seq_tree_build(W.PAPER_ACCEPTANCE_VECTOR, N, Dmax, Bmax, want_table=True)
    chosen = {}
    for c in (0.02, 0.2):
        n_s, d_s, s = B.seq_tree_speedup_search(table, t_of_n, c)
        chosen[f"c={c}"] = {"n": n_s, "d": d_s, "speedup": s, "G": float(table[n_s, d_s])}
    return {"us_per_step_by_tree_size": {str(n): times[n] for n in ns}, "t_of_n": {str(n): times[n] / times[1] for n in ns},
            "bounds": {"max_size": N, "max_depth": Dmax, "max_branch": Bmax}, "speedup_search": chosen,
            "note": "t(n) of attention + verification only, sizes in between interpolated; acceptance vector: the one the "
                    "paper prints; outside the timed step"}


def top_p_leg(cfg, ver_h, T, dev, stream, peaks, top_p=0.9) -> dict:
    """Not part of the timed step: the nucleus filter over the target rows of every tree node, timed on its own in a
    CUDA graph over rotating logit sets (out of place)."""
    from paper_2402_12374_b200 import binding as B

    sets = [vi.target_logits.to(dev) for vi in ver_h[:4]]
    out = torch.empty_like(sets[0])
    kept = torch.empty(sets[0].shape[0], dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    reps = 24
    with torch.cuda.stream(stream):
        for i in range(3):
            B.seq_tree_top_p_filter(sets[i % len(sets)], T, top_p, out=out, kept_out=kept, dev_status=status, stream=stream)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(reps):
                B.seq_tree_top_p_filter(sets[i % len(sets)], T, top_p, out=out, kept_out=kept, dev_status=status, stream=stream)
        g.replay()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        g.replay()
        e1.record(stream)
        stream.synchronize()
    if int(status.item()) != 0:
        raise RuntimeError(f"top_p dev_status = {int(status.item())}")
    us = e0.elapsed_time(e1) * 1e3 / reps
    rows, V = sets[0].shape
    nbytes = 2 * rows * V * 4
    gbs = nbytes / (us * 1e-6) / 1e9
    return {"us_per_call": us, "rows": rows, "vocab": V, "top_p": top_p, "mean_kept": float(kept.float().mean().item()),
            "gpu_launches_per_call": 1,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "algorithmic_bytes": nbytes, "traffic": None},
            "note": "every row read once and written once (the four re-reads of the select come from L2); outside the timed step"}


def verify_batch_leg(cfg, parent, ver_h, T, dev, stream) -> dict:
    """Not part of the timed step: R requests verified by one launch (one cluster per request; 18 clusters fit the
    GPU at a time), against R launches of the single-request call; both as CUDA graphs, logits beyond L2."""
    from paper_2402_12374_b200 import binding as B

    per_req = 2 * cfg.n_tree * cfg.vocab * 4
    R = 18 if per_req < (100 << 20) else 4
    pick = [ver_h[i % len(ver_h)] for i in range(R)]
    stack = lambda f: torch.stack([f(v).to(dev) for v in pick])
    par = torch.from_numpy(parent).to(dev).unsqueeze(0).repeat(R, 1).contiguous()
    tok, tl, dl, un = stack(lambda v: v.tokens), stack(lambda v: v.target_logits), stack(lambda v: v.draft_logits), stack(lambda v: v.uniforms)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    singles = [B.VerifyCall(par[r], tok[r], tl[r], dl[r], T, un[r], dev_status=status) for r in range(R)]
    reps = 10

    def timed(fn):
        with torch.cuda.stream(stream):
            fn()
            stream.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for _ in range(reps):
                    fn()
            g.replay()
            stream.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            g.replay()
            e1.record(stream)
            stream.synchronize()
        return e0.elapsed_time(e1) * 1e3 / reps

    outs = {}

    def batched():
        outs["b"] = B.seq_tree_verify_batch(par, tok, tl, dl, T, un, dev_status=status, stream=stream)

    def one_by_one():
        for c in singles:
            c.run(stream)

    us_b, us_s = timed(batched), timed(one_by_one)
    torch.cuda.synchronize()
    same = sum(int(outs["b"][2][r].item()) == int(singles[r].bonus_token.item()) for r in range(R))
    if int(status.item()) != 0 or same < R - 2:  # (a draw inside the rounding band may differ between cluster sizes)
        raise RuntimeError(f"verify_batch: dev_status {int(status.item())}, {same} of {R} bonus tokens equal to single launches")
    return {"requests": R, "us_per_launch": us_b, "us_per_request": us_b / R, "us_per_request_single_launches": us_s / R,
            "gpu_launches_per_call": 1, "bonus_tokens_equal_to_single_launches": f"{same}/{R}",
            "note": "one cluster of 8 CTAs per request (a single request runs on a cluster of 16); outside the timed step"}


def attention_batch_leg(cfg, parent, attn_h, dev, stream, peaks) -> dict:
    """Not part of the timed step: R requests that share the tree and the prefix length in ONE attention launch, as R
    times the heads (q [n, R, Hq, d], caches concatenated along the kv-head axis); sets rotate beyond L2."""
    from paper_2402_12374_b200 import binding as B

    R = 4 if cfg.n_tree <= 256 else 2
    n, Hq = cfg.n_tree, cfg.num_q_heads
    per = W.attention_algorithmic_bytes(cfg)
    sets = max(2, min(len(attn_h) // R, math.ceil(2 * L2_BYTES / (R * per))))
    parent_d = torch.from_numpy(parent).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    calls = []
    for s in range(sets):
        grp = [attn_h[(s * R + r) % len(attn_h)] for r in range(R)]
        q = torch.stack([a.q for a in grp], dim=1).reshape(n, R * Hq, cfg.head_dim).contiguous().to(dev)
        k = torch.cat([a.k_cache for a in grp], dim=0).contiguous().to(dev)
        v = torch.cat([a.v_cache for a in grp], dim=0).contiguous().to(dev)
        calls.append(B.AttentionCall(q, k, v, None, cfg.prefix_len, parent=parent_d, dev_status=status))
    reps = 8 * sets
    with torch.cuda.stream(stream):
        for c in calls[:2]:
            c.run(stream)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(reps):
                calls[i % sets].run(stream)
        g.replay()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        g.replay()
        e1.record(stream)
        stream.synchronize()
    if int(status.item()) != 0:
        raise RuntimeError(f"attention_batch dev_status = {int(status.item())}")
    us = e0.elapsed_time(e1) * 1e3 / reps
    nbytes = R * per
    flops = R * W.attention_algorithmic_flops(cfg, parent)
    hbm_t, ten_t = nbytes / (peaks["hbm_gbs"] * 1e9), flops / (peaks["bf16_tflops"] * 1e12)
    if hbm_t >= ten_t:
        ach = nbytes / (us * 1e-6) / 1e9
        roof = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"]}
    else:
        ach = flops / (us * 1e-6) / 1e12
        roof = {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops"]}
    return {"requests": R, "us_per_launch": us, "us_per_request": us / R, "sets": sets, "roofline": roof,
            "note": "one launch for R requests with a common tree and prefix length; outside the timed step"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2-7b", choices=sorted(W.CONFIGS))
    ap.add_argument("--temperature", type=float, default=0.6)
    ap.add_argument("--kernel", type=int, default=0, help="0 auto, 1 CUDA-core, 2 tensor-core attention")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tree", default="random", choices=["random", "dp"],
                    help="random: seeded random tree within the config's bounds; dp: Sequoia's dynamic program on the paper's acceptance vector")
    ap.add_argument("--tree-search", action="store_true",
                    help="also time the step on trees of growing size and run the Speedup(n, d) search on that t(n)")
    ap.add_argument("--separate-mask", action="store_true",
                    help="build the ancestor mask with a launch of its own instead of inside the attention kernel")
    args = ap.parse_args()
    cfg = W.CONFIGS[args.workload]
    T = args.temperature
    if args.impl == "reference":
        run_reference(args, cfg, T)
        return

    from paper_2402_12374_b200 import binding as B

    B.load()  # fails loudly if the CUDA library is missing: there is no fallback
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)
    K, Wm = args.steps, max(3, args.warmup)

    attn_bytes = W.attention_algorithmic_bytes(cfg)
    n = cfg.n_tree
    logits_bytes_touched = 4 * 2 * cfg.vocab * 4  # a walk reads a few rows of each matrix
    na = n_sets(attn_bytes)
    nv = min(n_sets(logits_bytes_touched), 8 if cfg.vocab * n * 8 < (1 << 28) else 3)
    parent, attn_h, ver_h = build_requests(cfg, T, rank, na, nv, args.tree)

    status = torch.zeros(1, dtype=torch.int32, device=dev)
    parent_d = torch.from_numpy(parent).to(dev)
    mask = torch.empty((n, (n + 31) // 32), dtype=torch.int32, device=dev)
    depth = torch.empty(n, dtype=torch.int32, device=dev)
    attn_calls, ver_calls = [], []
    workspace = None
    # The ancestor mask: derived from the parent array inside the attention kernel (tensor-core kernel), or by a
    # launch of its own before it (--separate-mask, and always for the CUDA-core kernel).
    fused_mask = (not args.separate_mask and args.kernel != B.KERNEL_CUDA_CORE and cfg.dtype in ("fp16", "bf16")
                  and 128 % (cfg.num_q_heads // cfg.num_kv_heads) == 0)
    for ai in attn_h:
        call = B.AttentionCall(ai.q.to(dev), ai.k_cache.to(dev), ai.v_cache.to(dev), None if fused_mask else mask,
                               cfg.prefix_len, parent=parent_d, workspace=workspace, dev_status=status, kernel=args.kernel)
        workspace = call.workspace
        attn_calls.append(call)
    for vi in ver_h:
        ver_calls.append(B.VerifyCall(parent_d, vi.tokens.to(dev), vi.target_logits.to(dev), vi.draft_logits.to(dev),
                                      T, vi.uniforms.to(dev), dev_status=status))
    combine = args.kernel == B.KERNEL_CUDA_CORE and attn_calls[0].workspace_bytes_needed > 0  # split-KV partials merged by a second kernel
    launches_per_step = (0 if fused_mask else 1) + (2 if combine else 1) + 1

    stream = torch.cuda.Stream(device=dev)

    def step(i, s, ev=None):
        if not fused_mask:
            B.seq_tree_mask_from_parents(parent_d, mask_bits=mask, depth=depth, dev_status=status, stream=s)
        if ev:
            ev[0].record(s)
        attn_calls[i % na].run(s)
        if ev:
            ev[1].record(s)
        ver_calls[i % nv].run(s)
        if ev:
            ev[2].record(s)

    with torch.cuda.stream(stream):
        for i in range(Wm):
            step(i, stream)
        stream.synchronize()
        # graph A: the K timed steps, nothing else
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for i in range(K):
                step(Wm + i, stream)
        # graph B: the same K steps with event nodes around the kernels (per-kernel durations)
        Kb = min(K, 200)
        evs = [[torch.cuda.Event(enable_timing=True, external=True) for _ in range(3)] for _ in range(Kb)]
        graph_b = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph_b, stream=stream):
            for i in range(Kb):
                step(Wm + i, stream, evs[i])
        graph.replay()  # untimed replay: uploads the graph
        graph_b.replay()
        stream.synchronize()

        def barrier():
            torch.cuda.synchronize()
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize()

        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        with ClockSampler(local_rank) as clocks:
            e0.record(stream)
            graph.replay()
            e1.record(stream)
            stream.synchronize()
            # keep sampling over a few more replays so that short regions still see clocks under load
            t_end = time.time() + 0.25
            while time.time() < t_end:
                graph.replay()
                stream.synchronize()
        barrier()
        ms_total = e0.elapsed_time(e1)
        graph_b.replay()
        stream.synchronize()
        t_attn = [evs[i][0].elapsed_time(evs[i][1]) * 1e3 for i in range(Kb)]
        t_ver = [evs[i][1].elapsed_time(evs[i][2]) * 1e3 for i in range(Kb)]

        # each kernel's average launch duration: Kb launches of that kernel alone, back to back in one graph, between
        # two events (the event nodes of graph B add a few microseconds to every call they bracket)
        def alone(run_one):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for i in range(Kb):
                    run_one(Wm + i)
            g.replay()
            stream.synchronize()
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record(stream)
            g.replay()
            a1.record(stream)
            stream.synchronize()
            return a0.elapsed_time(a1) * 1e3 / Kb

        attn_alone_us = alone(lambda i: attn_calls[i % na].run(stream))
        ver_alone_us = alone(lambda i: ver_calls[i % nv].run(stream))

    if int(status.item()) != 0:
        raise RuntimeError(f"dev_status = {int(status.item())} after the timed region")
    ms_total = max_over_ranks(ms_total, dev)
    ms_per_step = ms_total / K
    value_us = whole_job_us_per_step(ms_total, K, world)

    # end to end from pinned host buffers through the public API, copies inside the timed region
    host = B.HostStep(attn_h[0].q, attn_h[0].k_cache, attn_h[0].v_cache, torch.from_numpy(parent), cfg.prefix_len,
                      ver_h[0].tokens, ver_h[0].target_logits, ver_h[0].draft_logits, T, ver_h[0].uniforms, device=dev,
                      fused_mask=fused_mask, kernel=args.kernel)
    Ke = min(K, 20)
    with torch.cuda.stream(stream):
        for _ in range(3):
            host.run(stream)
            stream.synchronize()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(Ke):
            host.run(stream)
            stream.synchronize()
        e2e_us = 1e6 * (time.perf_counter() - t0) / Ke
    e2e_us = max_over_ranks(e2e_us, dev) / world

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    attn_ev_us, ver_ev_us = statistics.mean(t_attn), statistics.mean(t_ver)
    attn_us, ver_us = attn_alone_us, ver_alone_us
    flops = W.attention_algorithmic_flops(cfg, parent)
    hbm_time = attn_bytes / (peaks["hbm_gbs"] * 1e9)
    tensor_time = flops / (peaks["bf16_tflops"] * 1e12)
    if hbm_time >= tensor_time:
        achieved = attn_bytes / (attn_us * 1e-6) / 1e9
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / peaks["hbm_gbs"]}
    else:
        achieved = flops / (attn_us * 1e-6) / 1e12
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                    "frac": achieved / peaks["bf16_tflops"]}
    roofline.update({
        "traffic": NCU_TRAFFIC_BYTES.get(cfg.name), "kernel": "seq_tree_attention", "us_per_launch": attn_us,
        "algorithmic_bytes": attn_bytes, "algorithmic_flops": flops, "peak_source": f"of {peaks['source']}",
        "us_per_launch_between_event_nodes": attn_ev_us,
        "timing": f"{Kb} launches of the kernel alone, back to back in one CUDA graph over the rotating inputs, between two "
                  f"CUDA events; between event nodes inside the replayed steps the same call reads {attn_ev_us:.1f} us",
    })
    # verification: HBM-bound in principle (the target row of every visited node, the draft row of every
    # visited node that has children), latency-bound in practice (one cluster of 8 CTAs walks the path)
    has_child = np.zeros(n, dtype=bool)
    has_child[parent[1:][parent[1:] >= 0]] = True
    vbytes = []
    for vc in ver_calls:
        plen = int(vc.path_len.item())
        nodes = vc.path[:plen].cpu().numpy()
        vbytes.append(sum(4 * cfg.vocab * (2 if has_child[v] else 1) for v in nodes))
    ver_bytes = float(np.mean(vbytes))
    ver_gbs = ver_bytes / (ver_us * 1e-6) / 1e9
    roofline_verify = {"bound": "hbm", "achieved": ver_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                       "frac": ver_gbs / peaks["hbm_gbs"], "traffic": None, "kernel": "seq_tree_verify",
                       "us_per_launch": ver_us, "algorithmic_bytes": ver_bytes,
                       "note": "logit rows of the visited nodes only; a dependent walk on one cluster, latency-bound"}

    line = {
        "metric": METRIC, "value": value_us, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": cfg.name, "temperature": T, "n_tree": n, "prefix_len": cfg.prefix_len,
                   "heads": f"{cfg.num_q_heads}/{cfg.num_kv_heads}", "vocab": cfg.vocab, "requests_per_gpu": 1,
                   "l2": f"inputs rotate over {na} attention sets ({na * attn_bytes >> 20} MiB) and {nv} logit sets, "
                         f"larger than the 126 MiB L2", "launch": "CUDA graph of the K steps",
                   "mask": "from the parent array inside the attention kernel" if fused_mask else "separate launch",
                   "tree": "seeded random within the config's depth and fan-out bounds" if args.tree == "random"
                           else "seq_tree_build on the paper's printed acceptance vector"},
        "clocks": clocks.summary(),
        "e2e": {"value": e2e_us, "unit": UNIT, "h2d_bytes_per_step": host.h2d_bytes, "d2h_bytes_per_step": host.d2h_bytes,
                "steps": Ke},
        "gpu_launches": K * launches_per_step,
        "roofline": roofline,
        "roofline_verify": roofline_verify,
        "breakdown_us": {"attention": attn_us, "verify": ver_us, "attention_between_event_nodes": attn_ev_us,
                         "verify_between_event_nodes": ver_ev_us,
                         "largest_share": "seq_tree_verify" if ver_us > attn_us else "seq_tree_attention"},
    }
    line["next_rows"] = {"kv_commit": kv_commit_leg(cfg, parent, dev, stream, peaks)}
    if T > 0 and args.tree_search:
        line["next_rows"]["tree_search"] = tree_search_leg(cfg, T, dev, stream)
    line["next_rows"]["attention_batch"] = attention_batch_leg(cfg, parent, attn_h, dev, stream, peaks)
    line["next_rows"]["verify_batch"] = verify_batch_leg(cfg, parent, ver_h, T, dev, stream)
    if T > 0:
        line["next_rows"]["top_p_filter"] = top_p_leg(cfg, ver_h, T, dev, stream, peaks)
        line["next_rows"]["draft_sample"] = draft_sample_leg(cfg, parent, ver_h, T, dev, stream, peaks)
    if not args.no_cpu_baseline:
        from oracle import oracle as O

        t, note = oracle_step_sample(cfg, parent, attn_h[0], ver_h[0], T)
        line["cpu_baseline"] = {"value": 1e6 * t, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle", "sample": note}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
