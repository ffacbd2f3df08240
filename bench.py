#!/usr/bin/env python
"""Benchmark of the token-tree verify step (ancestor mask -> tree attention -> Algorithm 2 walk).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload all|NAME] [--temperature T]
    python bench.py --impl reference ...      # the fp64 CPU oracle on the host cores, same metric

One "step" is one pass of the whole hot path over one synthetic request.  By default all five
workloads are measured in one run: the headline (`value`, `config`, `roofline`, `e2e`,
`cpu_baseline`) is the largest single-GPU one, llama3-70b, and `per_workload` carries the same
figures for each of the five.  The K steps of a workload are captured in one CUDA graph; the graph
is replayed 25 times, each replay between its own pair of CUDA events (median, minimum and maximum
are printed; the median is the value); inputs rotate over enough independent copies that every
step reads memory that is not in L2.  One JSON line is printed by rank 0.  With N > 1 (torchrun)
every rank verifies its own requests (weak scaling, no data-path collective) and every time is the
maximum over ranks.

    python bench.py --ncu-traffic-csv FILE    # no GPU work: turn an ncu --csv log of DRAM byte
                                              # counters into profiles/tree_attention_umma_traffic.json
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

HEADLINE = "llama3-70b"                     # the largest configuration that fits one GPU
ALL_WORKLOADS = ["tiny", "llama2-7b", "llama2-13b", "vicuna-33b", "llama3-70b"]
SPEC_HBM_GBS, SPEC_BF16_TFLOPS = 8000.0, 2250.0   # nominal figures, printed beside the measured ones
REPLAYS = 25                                 # timed replays of a workload's graph
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "tree_attention_umma_traffic.json")


def ncu_traffic_bytes(workload: str):
    """DRAM bytes per launch of the attention kernel (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu
    capture recorded in profiles/ (written by `bench.py --ncu-traffic-csv`); None without a capture."""
    try:
        return json.load(open(TRAFFIC_FILE))["bytes_per_launch"].get(workload)
    except (OSError, ValueError, KeyError):
        return None


def write_traffic_file(csv_path: str, workload: str, command: str) -> None:
    """Parses an `ncu --csv` log that holds dram__bytes_read.sum and dram__bytes_write.sum per captured launch
    and records the attention kernel's mean bytes per launch for `workload`."""
    import csv

    per_launch = {}
    with open(csv_path, newline="") as f:
        rows = [r for r in csv.reader(f) if len(r) > 5]
    header = next(r for r in rows if "Metric Name" in r)
    col = {name: header.index(name) for name in ("ID", "Kernel Name", "Metric Name", "Metric Unit", "Metric Value")}
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    for r in rows:
        if r is header or len(r) <= max(col.values()) or "tree_attention_umma" not in r[col["Kernel Name"]]:
            continue
        if r[col["Metric Name"]] in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
            val = float(r[col["Metric Value"]].replace(",", "")) * scale.get(r[col["Metric Unit"]], 1.0)
            per_launch[r[col["ID"]]] = per_launch.get(r[col["ID"]], 0.0) + val
    if not per_launch:
        raise SystemExit(f"{csv_path}: no dram byte counters of the attention kernel found")
    data = {"bytes_per_launch": {}, "source": {}}
    if os.path.exists(TRAFFIC_FILE):
        data = json.load(open(TRAFFIC_FILE))
    data["bytes_per_launch"][workload] = int(round(sum(per_launch.values()) / len(per_launch)))
    data["source"][workload] = {"launches": len(per_launch), "command": command}
    json.dump(data, open(TRAFFIC_FILE, "w"), indent=1, sort_keys=True)
    print(f"{TRAFFIC_FILE}: {workload} -> {data['bytes_per_launch'][workload]} B per launch over {len(per_launch)} launches")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        # the burst figure for a kernel timed alone in bursts of a few ms, the sustained one for a long loop of it
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


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


def oracle_step_sample(cfg, parent, ai, vi, T, budget_flops=3e10):
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


def config_dict(cfg, T, tree):
    """The workload's description, the same in both arms."""
    return {"workload": cfg.name, "temperature": T, "n_tree": cfg.n_tree, "prefix_len": cfg.prefix_len,
            "heads": f"{cfg.num_q_heads}/{cfg.num_kv_heads}", "vocab": cfg.vocab, "requests_per_gpu": 1,
            "tree": "seeded random within the config's depth and fan-out bounds" if tree == "random"
                    else "seq_tree_build on the paper's printed acceptance vector"}


def run_reference(args, cfg, T):
    """--impl reference: the oracle, as it stands, on the host cores; every step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle as O

    parent = None
    if args.tree == "dp":  # this arm runs none of the library: the oracle's own statement of the dynamic program
        from oracle import tree_dp

        parent, _ = tree_dp.build_tree(W.PAPER_ACCEPTANCE_VECTOR, cfg.n_tree, cfg.max_depth, cfg.max_fanout or 31)
    parent, attn, ver = build_requests(cfg, T, 0, 1, 1, parent=parent)
    for _ in range(args.warmup):
        oracle_step_sample(cfg, parent, attn[0], ver[0], T)
    times, note = [], ""
    for _ in range(args.steps):
        t, note = oracle_step_sample(cfg, parent, attn[0], ver[0], T)
        times.append(t)
    us = 1e6 * sum(times) / len(times)
    cores = O.num_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": us, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(cfg, T, args.tree),
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
            "note": "one cluster per request: of 16 CTAs (rows in registers) while the batch fits the GPU side by side, else of 8; outside the timed step"}


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


def device_verify_sets(cfg, parent, T, count, dev, seed):
    """Further logit sets of a workload, drawn on the device with the host recipe's distributions (target N(0, sigma^2),
    draft = target + noise, children's tokens by a Gumbel top-k draw from the draft at T, uniforms in [0, 1)): the
    first set of every workload comes from the host (it is the one the oracle is timed on); these only serve to
    rotate the verification's inputs through more memory than the L2 holds."""
    n, V = len(parent), cfg.vocab
    gen = torch.Generator(device=dev)
    gen.manual_seed(W.BASE_SEED + 7919 * cfg.config_id + seed)
    kids = W.children_lists(parent)
    sets = []
    for _ in range(count):
        tl = cfg.target_sigma * torch.randn((n, V), device=dev, generator=gen)
        dl = tl + cfg.draft_noise_sigma * torch.randn((n, V), device=dev, generator=gen)
        tokens = torch.zeros(n, dtype=torch.int32, device=dev)
        for node, ch in enumerate(kids):
            if ch:
                key = dl[node] / T if T > 0 else dl[node].clone()
                if T > 0:
                    key = key - torch.log(-torch.log(torch.rand(V, device=dev, generator=gen).clamp_(1e-9, 1 - 1e-7)))
                tokens[ch] = torch.topk(key, len(ch)).indices.to(torch.int32)
        u = torch.rand(n + 1, device=dev, generator=gen)
        sets.append((tokens, tl, dl, u))
    return sets


def timed_replays(graph, stream, replays, world, dev):
    """`replays` replays of one CUDA graph, each between its own pair of events after a barrier; per replay the
    maximum over ranks.  Returns the list of milliseconds."""
    import torch.distributed as dist

    out = []
    for _ in range(replays):
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        graph.replay()
        e1.record(stream)
        stream.synchronize()
        out.append(e0.elapsed_time(e1))
    if world > 1:
        t = torch.tensor(out, dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        out = t.tolist()
    return out


def spread(ms_list, per):
    us = sorted(1e3 * m / per for m in ms_list)
    return {"median": statistics.median(us), "min": us[0], "max": us[-1], "replays": len(us)}


def verify_bf16_leg(cfg, parent, ver_sets, T, dev, stream) -> dict:
    """Not part of the timed step: the verification with both logit matrices in bfloat16 (half the bytes per visited
    node), L2-cold like the fp32 figure (a 160 MiB write before each launch, the same graph without launches
    subtracted)."""
    from paper_2402_12374_b200 import binding as B

    status = torch.zeros(1, dtype=torch.int32, device=dev)
    parent_d = torch.from_numpy(parent).to(dev)
    calls = [B.VerifyCall(parent_d, tok, tl.to(torch.bfloat16), dl.to(torch.bfloat16), T, u, dev_status=status)
             for tok, tl, dl, u in ver_sets[:2]]
    flush = torch.empty(160 << 20, dtype=torch.uint8, device=dev)
    Kc = 12

    def graph_of(body):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(Kc):
                body(i)
        g.replay()
        stream.synchronize()
        return g

    with torch.cuda.stream(stream):
        calls[0].run(stream)
        stream.synchronize()
        g_cold = graph_of(lambda i: (flush.fill_(i & 127), calls[i % len(calls)].run(stream)))
        g_flush = graph_of(lambda i: flush.fill_(i & 127))
        ms = [statistics.median(timed_replays(g, stream, 7, 1, dev)) for g in (g_cold, g_flush)]
    if int(status.item()) != 0:
        raise RuntimeError(f"verify_bf16 dev_status = {int(status.item())}")
    return {"us_per_launch": (ms[0] - ms[1]) * 1e3 / Kc, "l2": "cold (160 MiB written before every launch)",
            "note": "SEQ_VERIFY_LOGITS_BF16: the same walk on bfloat16 logits; outside the timed step"}


def verify_greedy_leg(cfg, parent, ver_sets, dev, stream) -> dict:
    """Not part of the timed step: the verification at T = 0 (greedy decoding, the setting of the paper's first result
    tables), L2-cold like the sampling figure.  The walk is as long as the synthetic draft happens to agree with the
    target's arg-max; its length is reported beside the time."""
    from paper_2402_12374_b200 import binding as B

    status = torch.zeros(1, dtype=torch.int32, device=dev)
    parent_d = torch.from_numpy(parent).to(dev)
    calls = [B.VerifyCall(parent_d, tok, tl, dl, 0.0, u, dev_status=status) for tok, tl, dl, u in ver_sets[:2]]
    flush = torch.empty(160 << 20, dtype=torch.uint8, device=dev)
    Kc = 12

    def graph_of(body):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(Kc):
                body(i)
        g.replay()
        stream.synchronize()
        return g

    with torch.cuda.stream(stream):
        for c in calls:
            c.run(stream)
        stream.synchronize()
        visited = sum(int(c.path_len.item()) for c in calls) / len(calls)
        g_cold = graph_of(lambda i: (flush.fill_(i & 127), calls[i % len(calls)].run(stream)))
        g_flush = graph_of(lambda i: flush.fill_(i & 127))
        ms = [statistics.median(timed_replays(g, stream, 7, 1, dev)) for g in (g_cold, g_flush)]
    if int(status.item()) != 0:
        raise RuntimeError(f"verify_greedy dev_status = {int(status.item())}")
    return {"us_per_launch": (ms[0] - ms[1]) * 1e3 / Kc, "visited_nodes_mean": visited,
            "l2": "cold (160 MiB written before every launch)",
            "note": "T = 0: arg-max matching, one exchange per visited node; outside the timed step"}


def robustness_leg(dev, stream, vocab=2048, requests=1500) -> dict:
    """Not part of the timed step (--robustness): a synthetic analogue of the paper's rejection-rate figure (Section
    3.2.2: average rejection rate against the number of speculated child tokens at T = 0.2, 0.6, 1.0, for the three
    verification algorithms), on the library's three verifiers through seq_tree_verify_batch.  One node with k
    children per request, target logits N(0, 3^2), draft = target + N(0, 1): Sequoia (children drawn without
    replacement, Algorithm 2), SpecInfer (children drawn with replacement, Algorithm 2 without the draft update),
    top-k (children = the draft's top k, verification by sampling from the target).  Rejection = no child accepted."""
    from paper_2402_12374_b200 import binding as B

    gen = torch.Generator(device=dev)
    gen.manual_seed(W.BASE_SEED)
    ks = [1, 2, 4, 8, 16, 32]
    out = {"vocab": vocab, "requests_per_point": requests, "k": ks, "rejection_rate": {}}
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):  # inputs and launches on one stream
        for T in (0.2, 0.6, 1.0):
            rates = {"sequoia": [], "specinfer": [], "top_k": []}
            for k in ks:
                n = k + 1
                tl = 3.0 * torch.randn((requests, 1, vocab), device=dev, generator=gen)
                dl = tl + torch.randn((requests, 1, vocab), device=dev, generator=gen)
                TL, DL = tl.expand(requests, n, vocab).contiguous(), dl.expand(requests, n, vocab).contiguous()
                par = torch.zeros((requests, n), dtype=torch.int32, device=dev)
                par[:, 0] = -1
                u = torch.rand((requests, n + 1), device=dev, generator=gen)
                gum = -torch.log(-torch.log(torch.rand((requests, vocab), device=dev, generator=gen).clamp_(1e-9, 1 - 1e-7)))
                draws = {
                    "sequoia": torch.topk(dl[:, 0] / T + gum, k, dim=1).indices,
                    "specinfer": torch.multinomial(torch.softmax(dl[:, 0] / T, dim=1), k, replacement=True, generator=gen),
                    "top_k": torch.topk(dl[:, 0], k, dim=1).indices,
                }
                for name, kids in draws.items():
                    tok = torch.zeros((requests, n), dtype=torch.int32, device=dev)
                    tok[:, 1:] = kids.to(torch.int32)
                    _, plen, _ = B.seq_tree_verify_batch(par, tok, TL, None if name == "top_k" else DL, T, u, dev_status=status,
                                                         specinfer=name == "specinfer", target_sample=name == "top_k", stream=stream)
                    stream.synchronize()
                    rates[name].append(float((plen == 1).float().mean().item()))
            out["rejection_rate"][f"T={T}"] = rates
    if int(status.item()) != 0:
        raise RuntimeError(f"robustness dev_status = {int(status.item())}")
    out["note"] = "synthetic logits; outside the timed step"
    return out


def floors_leg(dev, stream) -> dict:
    """What the device gives to a kernel that only reads (GB/s over a buffer far larger than L2) and to a launch
    that does next to nothing (one warp, one dependent load from memory that is not in L2), both through this
    library's probe kernels, as CUDA graphs."""
    from paper_2402_12374_b200 import binding as B

    buf = torch.empty(1 << 30, dtype=torch.uint8, device=dev)
    buf.random_(0, 255)
    sink = torch.zeros(4096, dtype=torch.int64, device=dev)
    src = buf.view(torch.int32)
    dst = torch.zeros(1, dtype=torch.int32, device=dev)
    reps = 10
    with torch.cuda.stream(stream):
        B.seq_tree_probe_stream_read(buf, sink, stream)
        B.seq_tree_probe_dependent_load(src, dst, stream)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(reps):
                B.seq_tree_probe_stream_read(buf, sink, stream)
        n_small = 200
        g2 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g2, stream=stream):
            for i in range(n_small):  # addresses 4 MiB apart: every launch misses the L2 (the pass above evicted them)
                B.seq_tree_probe_dependent_load(src[i * (1 << 20):], dst, stream)
        out = {}
        for name, graph, per in (("read", g, reps), ("small", g2, n_small)):
            graph.replay()
            stream.synchronize()
            if name == "small":
                g.replay()  # evict
                stream.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            graph.replay()
            e1.record(stream)
            stream.synchronize()
            out[name] = e0.elapsed_time(e1) * 1e3 / per
    del buf
    return {"stream_read_gbs": (1 << 30) / (out["read"] * 1e-6) / 1e9, "stream_read_bytes": 1 << 30,
            "launch_with_one_dependent_load_us": out["small"],
            "note": "seq_tree_probe_stream_read over 1 GiB (10 passes in one graph) and seq_tree_probe_dependent_load "
                    "(200 launches in one graph, each on an address that is not in L2)"}


def run_workload(cfg, T, args, rank, local_rank, world, dev, stream, peaks, with_legs):
    """Everything measured on one workload; returns (result dict, state for the e2e / cpu legs)."""
    from paper_2402_12374_b200 import binding as B

    K, Wm = args.steps, max(3, args.warmup)
    n = cfg.n_tree
    attn_bytes = W.attention_algorithmic_bytes(cfg)
    na = n_sets(attn_bytes)
    logits_set_bytes = 2 * n * cfg.vocab * 4
    nv = 4 if logits_set_bytes < (1 << 28) else 3
    parent, attn_h, ver_h = build_requests(cfg, T, rank, na, 1, args.tree)

    status = torch.zeros(1, dtype=torch.int32, device=dev)
    parent_d = torch.from_numpy(parent).to(dev)
    mask = torch.empty((n, (n + 31) // 32), dtype=torch.int32, device=dev)
    depth = torch.empty(n, dtype=torch.int32, device=dev)
    fused_mask = (not args.separate_mask and args.kernel != B.KERNEL_CUDA_CORE and cfg.dtype in ("fp16", "bf16")
                  and 128 % (cfg.num_q_heads // cfg.num_kv_heads) == 0)
    attn_calls, ver_calls, workspace = [], [], None
    for ai in attn_h:
        call = B.AttentionCall(ai.q.to(dev), ai.k_cache.to(dev), ai.v_cache.to(dev), None if fused_mask else mask,
                               cfg.prefix_len, parent=parent_d, workspace=workspace, dev_status=status, kernel=args.kernel)
        workspace = call.workspace
        attn_calls.append(call)
    vi0 = ver_h[0]
    ver_sets = [(vi0.tokens.to(dev), vi0.target_logits.to(dev), vi0.draft_logits.to(dev), vi0.uniforms.to(dev))]
    ver_sets += device_verify_sets(cfg, parent, T, nv - 1, dev, rank_seed_base(rank))
    for tok, tl, dl, u in ver_sets:
        ver_calls.append(B.VerifyCall(parent_d, tok, tl, dl, T, u, dev_status=status))
    combine = args.kernel == B.KERNEL_CUDA_CORE and attn_calls[0].workspace_bytes_needed > 0
    launches_per_step = (0 if fused_mask else 1) + (2 if combine else 1) + 1

    def step(i, s):
        if not fused_mask:
            B.seq_tree_mask_from_parents(parent_d, mask_bits=mask, depth=depth, dev_status=status, stream=s)
        attn_calls[i % na].run(s)
        ver_calls[i % nv].run(s)

    flush = torch.empty(160 << 20, dtype=torch.uint8, device=dev)
    # Launches per graph of the per-kernel timings: every attention set four times, whatever K is.  On the 768-node
    # workload that is a burst of about 5 ms per replay, as the burst peak it is set against was measured (single GEMMs,
    # best of ten); a hundred such launches in a row run into the 1 kW power cap, and that figure is reported beside
    # it, against the sustained peak.
    Kb = 4 * na

    def graph_of(body, count):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(count):
                body(Wm + i)
        g.replay()  # untimed replay: uploads the graph
        stream.synchronize()
        return g

    with torch.cuda.stream(stream):
        for i in range(Wm):
            step(i, stream)
        stream.synchronize()
        g_step = graph_of(lambda i: step(i, stream), K)
        g_attn = graph_of(lambda i: attn_calls[i % na].run(stream), Kb)
        g_ver_warm = graph_of(lambda i: ver_calls[i % nv].run(stream), Kb)
        # verification with its logits out of the L2: a write larger than the L2 before every launch, and the same
        # graph without the launches to subtract
        Kc = 12
        g_ver_cold = graph_of(lambda i: (flush.fill_(i & 127), ver_calls[i % nv].run(stream)), Kc)
        g_flush = graph_of(lambda i: flush.fill_(i & 127), Kc)

        # The kernel alone, in bursts, first: set against the burst peak, it is taken as that peak was — from a GPU that
        # has not just run half a second of dense work under its power cap (two warm replays, then nine timed ones).
        timed_replays(g_attn, stream, 2, world, dev)
        ms_attn = timed_replays(g_attn, stream, 9, world, dev)
        with ClockSampler(local_rank) as clocks:
            ms_steps = timed_replays(g_step, stream, REPLAYS, world, dev)
            t_end = time.time() + 0.2  # keep the GPU under the same load a little longer: short regions still see clocks
            while time.time() < t_end:
                g_step.replay()
                stream.synchronize()
        # the same graph 30 times without a pause (a tensor-bound workload: > 100 ms of dense work under the power cap)
        sustained_reps = 30
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        stream.synchronize()
        ev0.record(stream)
        for _ in range(sustained_reps):
            g_attn.replay()
        ev1.record(stream)
        stream.synchronize()
        attn_sustained_us = ev0.elapsed_time(ev1) * 1e3 / (sustained_reps * Kb)
        ms_ver_warm = timed_replays(g_ver_warm, stream, 9, world, dev)
        ms_cold = timed_replays(g_ver_cold, stream, 9, world, dev)
        ms_flush = timed_replays(g_flush, stream, 9, world, dev)
    if int(status.item()) != 0:
        raise RuntimeError(f"{cfg.name}: dev_status = {int(status.item())} after the timed region")

    step_us = spread(ms_steps, K)
    attn_us = statistics.median(ms_attn) * 1e3 / Kb
    ver_warm_us = statistics.median(ms_ver_warm) * 1e3 / Kb
    ver_cold_us = (statistics.median(ms_cold) - statistics.median(ms_flush)) * 1e3 / Kc
    flops = W.attention_algorithmic_flops(cfg, parent)
    hbm_time = attn_bytes / (peaks["hbm_gbs"] * 1e9)
    tensor_time = flops / (peaks["bf16_tflops"] * 1e12)
    if hbm_time >= tensor_time:
        achieved = attn_bytes / (attn_us * 1e-6) / 1e9
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / peaks["hbm_gbs"], "frac_of_spec": achieved / SPEC_HBM_GBS, "spec_peak": SPEC_HBM_GBS}
    else:
        achieved = flops / (attn_us * 1e-6) / 1e12
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                    "frac": achieved / peaks["bf16_tflops"], "frac_of_spec": achieved / SPEC_BF16_TFLOPS,
                    "spec_peak": SPEC_BF16_TFLOPS}
        ach_s = flops / (attn_sustained_us * 1e-6) / 1e12
        roofline["sustained"] = {"us_per_launch": attn_sustained_us, "achieved": ach_s, "peak": peaks["bf16_tflops_sustained"],
                                 "frac": ach_s / peaks["bf16_tflops_sustained"], "launches": sustained_reps * Kb,
                                 "note": "the same launches in one unbroken run, against the sustained peak"}
    roofline.update({
        "traffic": ncu_traffic_bytes(cfg.name), "kernel": "seq_tree_attention", "us_per_launch": attn_us,
        "algorithmic_bytes": attn_bytes, "algorithmic_flops": flops, "peak_source": f"of {peaks['source']}",
        "hbm_gbs": attn_bytes / (attn_us * 1e-6) / 1e9,
        "timing": f"{Kb} launches of the kernel alone, back to back in one CUDA graph over {na} rotating input sets "
                  f"({na * attn_bytes >> 20} MiB, L2-cold), median of 9 replays",
    })
    # verification: the rows of the visited nodes are the algorithmic minimum (B_path); what the schedule moved on
    # top of that is speculative work
    has_child = np.zeros(n, dtype=bool)
    has_child[parent[1:][parent[1:] >= 0]] = True
    torch.cuda.synchronize()
    kids = W.children_lists(parent)
    row_bytes = lambda v: 4 * cfg.vocab * (2 if has_child[v] else 1)
    path_bytes, moved_bytes, visited = [], [], []
    for vc in ver_calls:
        plen = int(vc.path_len.item())
        nodes = vc.path[:plen].cpu().numpy().tolist()
        visited.append(plen)
        path_bytes.append(sum(row_bytes(v) for v in nodes))
        # what the walk really loads: the root's rows, and ahead of its test the rows of every child that is tested
        # (up to the accepted one, all of them where none is accepted)
        m = row_bytes(0)
        for i, v in enumerate(nodes):
            nxt = nodes[i + 1] if i + 1 < plen else None
            for ch in kids[v]:
                m += row_bytes(ch)
                if ch == nxt:
                    break
        moved_bytes.append(m)
    b_path = float(np.mean(path_bytes))
    moved = float(np.mean(moved_bytes))
    ver_gbs = moved / (ver_cold_us * 1e-6) / 1e9
    roofline_verify = {"bound": "hbm", "achieved": ver_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                       "frac": ver_gbs / peaks["hbm_gbs"], "frac_of_spec": ver_gbs / SPEC_HBM_GBS, "traffic": None,
                       "kernel": "seq_tree_verify", "us_per_launch": ver_cold_us, "us_per_launch_l2_warm": ver_warm_us,
                       "b_path_bytes": b_path, "bytes_moved": moved, "b_path_over_bytes_moved": b_path / moved,
                       "visited_nodes_mean": float(np.mean(visited)),
                       "timing": f"L2-cold: {Kc} launches in one graph, a 160 MiB write before each, minus the same graph "
                                 f"without the launches; L2-warm: {Kb} launches back to back over {nv} logit sets",
                       "note": "a dependent walk on one cluster of 16 CTAs: latency-bound, its HBM fraction says little; bytes moved "
                               "= the visited nodes' rows plus the rows of tested-and-rejected children, loaded ahead of their test"}
    res = {
        "us_per_step": step_us, "ms_per_step": step_us["median"] / 1e3,
        "attention_us": attn_us, "verify_us": ver_cold_us, "verify_us_l2_warm": ver_warm_us,
        "verify_us_in_step": step_us["median"] - attn_us,
        "roofline": roofline, "roofline_verify": roofline_verify, "clocks": clocks.summary(),
        "dtype": cfg.dtype, "gpu_launches": K * launches_per_step * (REPLAYS + 1),
        "config": dict(config_dict(cfg, T, args.tree),
                       l2=f"inputs rotate over {na} attention sets ({na * attn_bytes >> 20} MiB) and {nv} logit sets",
                       launch="CUDA graph of the K steps",
                       mask="from the parent array inside the attention kernel" if fused_mask else "separate launch"),
        "largest_share": "seq_tree_verify" if ver_cold_us > attn_us else "seq_tree_attention",
    }
    state = dict(parent=parent, attn_h=attn_h, ver_h=ver_h, fused_mask=fused_mask)
    if with_legs:
        legs = {"kv_commit": kv_commit_leg(cfg, parent, dev, stream, peaks)}
        if T > 0 and args.tree_search:
            legs["tree_search"] = tree_search_leg(cfg, T, dev, stream)
        legs["attention_batch"] = attention_batch_leg(cfg, parent, attn_h, dev, stream, peaks)
        ver_like = [_HostLike(*s) for s in ver_sets]
        legs["verify_batch"] = verify_batch_leg(cfg, parent, ver_like, T, dev, stream)
        if T > 0:
            legs["verify_bf16_logits"] = verify_bf16_leg(cfg, parent, ver_sets, T, dev, stream)
            legs["verify_greedy"] = verify_greedy_leg(cfg, parent, ver_sets, dev, stream)
            legs["top_p_filter"] = top_p_leg(cfg, ver_like, T, dev, stream, peaks)
            legs["draft_sample"] = draft_sample_leg(cfg, parent, ver_like, T, dev, stream, peaks)
        res["next_rows"] = legs
    del attn_calls, ver_calls, ver_sets, flush
    torch.cuda.empty_cache()
    return res, state


class _HostLike:
    """The fields of a logit set that the legs around the step read (tensors may live on either side)."""

    def __init__(self, tokens, target_logits, draft_logits, uniforms):
        self.tokens, self.target_logits, self.draft_logits, self.uniforms = tokens, target_logits, draft_logits, uniforms


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="all", choices=["all"] + sorted(W.CONFIGS),
                    help="all: the five workloads in one run, llama3-70b as the headline; or one of them alone")
    ap.add_argument("--temperature", type=float, default=None, help="default: the workload's own (0.6; 1.0 for llama2-13b)")
    ap.add_argument("--kernel", type=int, default=0, help="0 auto, 1 CUDA-core, 2 tensor-core attention")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-legs", action="store_true", help="skip the calls around the step (next_rows) and the floors")
    ap.add_argument("--tree", default="random", choices=["random", "dp"],
                    help="random: seeded random tree within the config's bounds; dp: Sequoia's dynamic program on the paper's acceptance vector")
    ap.add_argument("--tree-search", action="store_true",
                    help="also time the step on trees of growing size and run the Speedup(n, d) search on that t(n)")
    ap.add_argument("--robustness", action="store_true",
                    help="also sweep the three verifiers' rejection rate against the number of speculated children")
    ap.add_argument("--separate-mask", action="store_true",
                    help="build the ancestor mask with a launch of its own instead of inside the attention kernel")
    ap.add_argument("--ncu-traffic-csv", default=None,
                    help="no GPU work: parse this ncu --csv log (dram byte counters) into profiles/ for --workload")
    ap.add_argument("--ncu-command", default="", help="with --ncu-traffic-csv: the capture command, recorded beside the numbers")
    args = ap.parse_args()
    if args.ncu_traffic_csv:
        write_traffic_file(args.ncu_traffic_csv, HEADLINE if args.workload == "all" else args.workload, args.ncu_command)
        return
    names = ALL_WORKLOADS if args.workload == "all" else [args.workload]
    head_name = HEADLINE if args.workload == "all" else args.workload

    def temp_of(cfg):
        if args.temperature is not None:
            return args.temperature
        return 0.6 if 0.6 in cfg.temperatures else cfg.temperatures[-1]

    if args.impl == "reference":
        cfg = W.CONFIGS[head_name]
        run_reference(args, cfg, temp_of(cfg))
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
    peaks = measured_peaks()
    stream = torch.cuda.Stream(device=dev)

    per, head_state = {}, None
    for name in names:
        cfg = W.CONFIGS[name]
        res, state = run_workload(cfg, temp_of(cfg), args, rank, local_rank, world, dev, stream, peaks,
                                  with_legs=(name == head_name and not args.no_legs))
        per[name] = res
        if name == head_name:
            head_state = state
        else:
            del state
    cfg = W.CONFIGS[head_name]
    T = temp_of(cfg)
    head = per[head_name]

    # end to end from pinned host buffers through the public API, copies inside the timed region
    a0, v0 = head_state["attn_h"][0], head_state["ver_h"][0]
    host = B.HostStep(a0.q, a0.k_cache, a0.v_cache, torch.from_numpy(head_state["parent"]), cfg.prefix_len,
                      v0.tokens, v0.target_logits, v0.draft_logits, T, v0.uniforms, device=dev,
                      fused_mask=head_state["fused_mask"], kernel=args.kernel)
    Ke = max(3, min(args.steps, 10))

    def time_host_step(hs):
        with torch.cuda.stream(stream):
            for _ in range(3):
                hs.run(stream)
                stream.synchronize()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for _ in range(Ke):
                hs.run(stream)
                stream.synchronize()
            return 1e6 * (time.perf_counter() - t0) / Ke

    e2e_us = max_over_ranks(time_host_step(host), dev) / world
    # the same step with the verification's inputs on a second stream, and with the prefix of the cache resident
    e2e_variants = {}
    if not args.no_legs:
        for label, kw in (("two_streams", dict(two_streams=True)), ("resident_cache", dict(resident_cache=True)),
                          ("resident_cache_two_streams", dict(resident_cache=True, two_streams=True))):
            hs = B.HostStep(a0.q, a0.k_cache, a0.v_cache, torch.from_numpy(head_state["parent"]), cfg.prefix_len,
                            v0.tokens, v0.target_logits, v0.draft_logits, T, v0.uniforms, device=dev,
                            fused_mask=head_state["fused_mask"], kernel=args.kernel, **kw)
            e2e_variants[label] = {"value": max_over_ranks(time_host_step(hs), dev) / world, "unit": UNIT,
                                   "h2d_bytes_per_step": hs.h2d_bytes, "d2h_bytes_per_step": hs.d2h_bytes}
            del hs

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    K = args.steps
    value_us = head["us_per_step"]["median"] / world  # every rank verifies its own request per step (weak scaling)
    line = {
        "metric": METRIC, "value": value_us, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(3, args.warmup),
        "ms_per_step": head["ms_per_step"], "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": cfg.dtype, "data": "synthetic",
        "config": head["config"],
        "us_per_step_spread": head["us_per_step"],
        "clocks": head["clocks"],
        "e2e": {"value": e2e_us, "unit": UNIT, "h2d_bytes_per_step": host.h2d_bytes, "d2h_bytes_per_step": host.d2h_bytes,
                "steps": Ke, "variants": e2e_variants},
        "gpu_launches": sum(p["gpu_launches"] for p in per.values()),
        "roofline": head["roofline"],
        "roofline_verify": head["roofline_verify"],
        "breakdown_us": {"attention": head["attention_us"], "verify": head["verify_us"],
                         "verify_l2_warm": head["verify_us_l2_warm"], "verify_in_step": head["verify_us_in_step"],
                         "largest_share": head["largest_share"]},
        "per_workload": {k: {kk: vv for kk, vv in v.items() if kk != "next_rows"} for k, v in per.items()},
    }
    if "next_rows" in head:
        line["next_rows"] = head["next_rows"]
    if not args.no_legs:
        line["floors"] = floors_leg(dev, stream)
    if args.robustness:
        line.setdefault("next_rows", {})["robustness"] = robustness_leg(dev, stream)
    if not args.no_cpu_baseline:
        from oracle import oracle as O

        t, note = oracle_step_sample(cfg, head_state["parent"], a0, v0, T, budget_flops=2e11)  # the whole tree on every config
        line["cpu_baseline"] = {"value": 1e6 * t, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle", "sample": note}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
