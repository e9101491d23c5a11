#!/usr/bin/env python
"""Benchmark of BPT graph self-attention (forward + backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config NAME]

One step = one forward and one backward pass of the whole hot path over one batch of
seeded synthetic input.  The default workload is the character-level-LM-shaped layer
(batch 4, n = 8192, k = 64, left-only, 8 heads x 64, bf16).  Prints ONE JSON line.

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank processes
its own batch of the same shape (weak scaling); the only exchange is the all-reduce of
the relation-embedding gradient, which is shared by the whole batch.

`--impl reference` times the fp64 CPU oracle on the host cores on a bounded sample of
the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "BPT graph-attention fwd+bwd edges/sec"
UNIT = "edges/s"
GATHER_BYTES_PER_EDGE_HEAD = {  # algorithmic bytes of the gather model, per edge and head
    "fwd": lambda d, s: 2 * d * s,            # K row + V row
    "bwd_dst": lambda d, s: 2 * d * s,        # K row + V row again
    "bwd_src": lambda d, s: 2 * d * s + 8,    # Q row + dO row + (P, dS) or (lse, delta)
}
# Which part of the gather model each kernel carries: (passes, "token" | "span" | "all" destination rows).
KERNEL_MODEL = {
    "fwd_rows": (("fwd",), "all"), "bwd_dst": (("bwd_dst",), "all"), "bwd_src": (("bwd_src",), "all"),
    "fwd_tile": (("fwd",), "token"), "fwd_tc5": (("fwd",), "token"), "fwd_span": (("fwd",), "span"),
    "bwd_tile": (("bwd_dst", "bwd_src"), "token"), "bwd_span": (("bwd_dst", "bwd_src"), "span"),
    "bwd_q_tc5": (("bwd_dst",), "token"), "bwd_kv_tc5": (("bwd_src",), "token"),
}
# DRAM bytes (read + write) per (batch entry, head) pair of one launch, from ncu captures of the character-LM
# shape at batch 1 (n = 8192, k = 64, left-only, 8 heads; every pair is an independent problem, so traffic
# scales with pairs).  Each figure is tied to the source file of its kernel by a hash taken when the counters
# were read (re-taken after edits of the file that leave the measured kernel as it was, e.g. its helper kernels or
# comments); when the file has changed otherwise, the bench reports traffic = null instead of a stale number.
NCU_DRAM_BYTES_PER_PAIR = {
    # kernel: (bytes per pair, source file, sha256 of the file at capture time (first 16 hex digits))
    "fwd_tc5": (42.29e6 / 8, "attn_fwd_tc5.cu", "2f9c6b763080e59f"),
    "bwd_q_tc5": (60.69e6 / 8, "attn_bwd_q_tc5.cu", "d4456f5a3fecb677"),
    "bwd_kv_tc5": (113.88e6 / 8, "attn_bwd_kv_tc5.cu", "2342321c21ce8852"),
}
FLOPS_PER_EDGE_HEAD = {"fwd": 6, "bwd": 14}   # x d_head: q.k, q.r, P.v forward; s again, dP, dq, dk, dv, d_rel backward


def ncu_traffic_per_pair(kernel):
    """ncu DRAM bytes per pair for `kernel`, or None when unknown or taken from an older version of its source."""
    import hashlib
    ent = NCU_DRAM_BYTES_PER_PAIR.get(kernel)
    if ent is None:
        return None
    per_pair, fname, digest = ent
    path = os.path.join(ROOT, "paper_1911_04070_b200", "csrc", fname)
    try:
        now = hashlib.sha256(open(path, "rb").read()).hexdigest()[:16]
    except OSError:
        return None
    return per_pair if digest and now == digest else None


def load_peaks():
    """(HBM GB/s, sustained bf16 TFLOP/s, "measured" | "fallback")."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), float(p.get("bf16_tflops_sustained", 1400.0)), "measured"
    return 6650.0, 1400.0, "fallback"


def all_configs():
    from paper_1911_04070_b200 import synth
    c = dict(synth.CONFIGS)
    c.update(synth.sweep_configs())
    return c


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples during the timed region."""
    QUERY = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.QUERY,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self, t_begin=None, t_end=None):
        """Samples taken between the two host times (time.time()) when given and any fall inside, else all."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        import datetime
        rows = []
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 10:
                    continue
                try:
                    ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    rows.append((ts, float(f[2]), float(f[3]), f[6:10]))
                except ValueError:
                    continue
            os.unlink(self.path)
        except OSError:
            pass
        inside = [r for r in rows if t_begin is not None and t_begin - 0.02 <= r[0] <= t_end + 0.02]
        use = inside or rows
        if use:
            reasons = set()
            for r in use:
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            out.update(sm_mhz=statistics.median(r[1] for r in use), sm_max_mhz=max(r[2] for r in use), reasons=sorted(reasons),
                       samples=len(use), window="timed region" if inside else "warm-up and timed region")
        return out


def run_reference(args, cfg_name, cfg):
    """The fp64 oracle (plain C, OpenMP over batch x head) on the host cores.  Each step is a bounded
    sample of the workload: one batch entry and as many of its heads as keep the whole run to a
    couple of minutes (batch entries and heads are independent problems on the same graph)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import ctwin
    from paper_1911_04070_b200 import synth
    g = ctwin.CGraph(cfg["n"], cfg["k"], cfg["flags"])
    H = cfg["H"]
    x = synth.make_inputs(1, g.n_nodes, H, cfg["d"], g.n_rel, seed=cfg["seed"], std_qkv=cfg["std_qkv"], bf16=cfg["bf16"])
    scale = cfg["d"] ** -0.5

    def sliced(heads):
        return {a: np.ascontiguousarray(b if a == "rel_emb" else b[:, :, :heads], dtype=np.float64) for a, b in x.items()}

    def step(x64):
        ctwin.attn_fwd(g, x64["q"], x64["k"], x64["v"], x64["rel_emb"], scale)
        if cfg["backward"]:
            ctwin.attn_bwd(g, x64["q"], x64["k"], x64["v"], x64["rel_emb"], scale, x64["d_out"])

    one = sliced(1)
    t0 = time.perf_counter()
    step(one)
    t_head = time.perf_counter() - t0          # one head on one core
    cores = ctwin.threads()
    budget_s = 120.0
    per_step = budget_s / max(args.steps + args.warmup, 1)
    heads = int(max(1, min(H, (per_step / max(t_head, 1e-6)) * min(cores, H))))
    x64 = sliced(heads)
    for _ in range(args.warmup):
        step(x64)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step(x64)
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    value = g.n_edges * (heads / H) / dt       # an edge counts once all H heads of it are done
    sample = "per step: 1 of %d batch entries, %d of %d heads, full n (entries and heads are independent)" % (cfg["B"], heads, H)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg_name, "n": cfg["n"], "k": cfg["k"], "left_only": bool(cfg["flags"] & 1), "batch": 1,
                   "heads": heads, "d_head": cfg["d"], "pass": "fwd+bwd" if cfg["backward"] else "fwd"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": min(cores, heads), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def cpu_baseline(cfg):
    from oracle import ctwin
    from paper_1911_04070_b200 import synth
    g = ctwin.CGraph(cfg["n"], cfg["k"], cfg["flags"])
    Bs = min(cfg["B"], 2)
    x = synth.make_inputs(Bs, g.n_nodes, cfg["H"], cfg["d"], g.n_rel, seed=cfg["seed"], std_qkv=cfg["std_qkv"], bf16=cfg["bf16"])
    x64 = {a: np.ascontiguousarray(b, dtype=np.float64) for a, b in x.items()}
    scale = cfg["d"] ** -0.5
    t0 = time.perf_counter()
    ctwin.attn_fwd(g, x64["q"], x64["k"], x64["v"], x64["rel_emb"], scale)
    if cfg["backward"]:
        ctwin.attn_bwd(g, x64["q"], x64["k"], x64["v"], x64["rel_emb"], scale, x64["d_out"])
    dt = time.perf_counter() - t0
    return {"value": Bs * g.n_edges / dt, "unit": UNIT, "cores": ctwin.threads(), "kind": "oracle",
            "sample": "%d of %d batch entries, one pass, %.1f s" % (Bs, cfg["B"], dt)}


def run_ours(args, cfg_name, cfg):
    import torch
    import torch.distributed as dist
    from paper_1911_04070_b200 import binding, shard, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    B, H, d = cfg["B"], cfg["H"], cfg["d"]
    do_bwd = cfg["backward"]
    g = binding.bpt_build_graph(cfg["n"], cfg["k"], cfg["flags"], device=dev, with_transpose=do_bwd)
    E, N = g.n_edges, g.n_nodes
    # the graph build, timed on its own (second build: the first one pays the module load); not part of a step
    torch.cuda.synchronize()
    eb0, eb1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    eb0.record()
    binding.bpt_build_graph(cfg["n"], cfg["k"], cfg["flags"], device=dev, with_transpose=do_bwd)
    eb1.record()
    torch.cuda.synchronize()
    graph_build_ms = eb0.elapsed_time(eb1)
    dt_t = torch.bfloat16 if cfg["bf16"] else torch.float32
    esize = 2 if cfg["bf16"] else 4
    x = synth.make_inputs(B, N, H, d, g.n_rel, seed=cfg["seed"] + 1000 * rank, std_qkv=cfg["std_qkv"], bf16=cfg["bf16"], with_grad=do_bwd)
    host = {a: torch.from_numpy(b).to(dt_t).pin_memory() for a, b in x.items()}
    del x
    t = {a: b.to(dev, non_blocking=True) for a, b in host.items()}
    scale = d ** -0.5
    code = binding.BPT_BF16 if cfg["bf16"] else binding.BPT_F32
    ws_f = binding.bpt_attn_workspace_bytes(g, B, H, d, code, False)
    ws_b = binding.bpt_attn_workspace_bytes(g, B, H, d, code, True) if do_bwd else 0
    ws = torch.empty(max(ws_f, ws_b, 1), dtype=torch.uint8, device=dev)
    out = torch.empty_like(t["q"])
    lse = torch.empty((B, N, H), dtype=torch.float32, device=dev)
    dq, dk, dv = (torch.empty_like(t["q"]) for _ in range(3))
    d_rel = torch.empty((g.n_rel, d), dtype=torch.float32, device=dev)

    path = {"auto": binding.BPT_PATH_AUTO, "mma": binding.BPT_PATH_MMA, "tc5": binding.BPT_PATH_TC5}[args.path]

    def step():
        binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, out=out, lse=lse, workspace=ws, path=path)
        if do_bwd:
            binding.bpt_attn_bwd(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, out, lse, t["d_out"], workspace=ws,
                                 dq=dq, dk=dk, dv=dv, d_rel=d_rel, path=path)
            shard.allreduce_d_rel(d_rel)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        if world == 1:
            return ms
        v = torch.tensor([ms], dtype=torch.float64, device=dev)
        dist.all_reduce(v, op=dist.ReduceOp.MAX)
        return float(v.item())

    sampler = ClockSampler(local_rank)   # started before the warm-up: nvidia-smi takes a moment to deliver samples
    if rank == 0:
        sampler.start()
    for _ in range(args.warmup):
        step()
    barrier()
    t_load = time.time()
    while time.time() - t_load < 0.3:    # keep the GPU under the same load until the sampler is up (untimed)
        step()
    barrier()

    # ---- timed region: K steps, device-resident inputs ---------------------------------
    cap = min(args.steps * 16 + 8, 4000)
    # L2 (126 MB): a workload whose tensors exceed it evicts itself between steps; a smaller one gets a
    # 256 MB write between the timed steps, which are then timed one by one
    in_bytes = sum(v.numel() * v.element_size() for v in t.values()) + out.numel() * out.element_size()
    flush = in_bytes < 192 * 1024 * 1024
    scrub = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev) if flush else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_begin = time.time()
    if not flush:
        binding.bpt_trace_begin(cap)
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        barrier()
        ms_sum = e0.elapsed_time(e1)
        marks = binding.bpt_trace_end(cap)
    else:
        ms_sum, marks = 0.0, []
        for _ in range(args.steps):
            scrub.zero_()
            binding.bpt_trace_begin(16)
            e0.record()
            step()
            e1.record()
            torch.cuda.synchronize()
            ms_sum += e0.elapsed_time(e1)
            marks += binding.bpt_trace_end(16)
        barrier()
    t_end = time.time()
    device_status = binding.bpt_check(ws)   # a bounded device-side wait that ran out would make the timed results invalid
    if device_status:
        raise SystemExit("device-side failure report: %s" % binding.status_str(device_status))
    ms_total = max_over_ranks(ms_sum)
    clocks = sampler.stop(t_begin, t_end) if rank == 0 else None

    # ---- the same step recorded once into a CUDA graph and replayed (one GPU; reported beside the eager figure,
    # which stays the headline because only eager launches carry the per-kernel marks) ----
    ms_graph = None
    if world == 1:
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream())
        cg = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(cg, stream=side):
                step()
        torch.cuda.current_stream().wait_stream(side)
        for _ in range(args.warmup):
            cg.replay()
        torch.cuda.synchronize()
        if not flush:
            e0.record()
            for _ in range(args.steps):
                cg.replay()
            e1.record()
            torch.cuda.synchronize()
            ms_graph = e0.elapsed_time(e1) / args.steps
        else:
            acc = 0.0
            for _ in range(args.steps):
                scrub.zero_()
                e0.record()
                cg.replay()
                e1.record()
                torch.cuda.synchronize()
                acc += e0.elapsed_time(e1)
            ms_graph = acc / args.steps
        if binding.bpt_check(ws):
            raise SystemExit("device-side failure report after the graph replays")
    ms_step = ms_total / args.steps
    value = world * B * E / (ms_step * 1e-3)

    # ---- end to end: host buffers in, results back to the host, every step --------------
    # Every step copies its inputs from pinned host memory and its results back.  Two sets of device buffers and
    # three streams let the copies of the neighbouring steps run under the kernels of the current one; the
    # kernels of consecutive steps still run in order on one stream (they share the workspace).
    names_in = ["q", "k", "v", "rel_emb"] + (["d_out"] if do_bwd else [])
    t_in = [t, {a: torch.empty_like(b) for a, b in t.items()}]
    res_dev = [[out, lse] + ([dq, dk, dv, d_rel] if do_bwd else [])]
    res_dev.append([torch.empty_like(r) for r in res_dev[0]])
    res_host = [torch.empty(r.shape, dtype=r.dtype).pin_memory() for r in res_dev[0]]
    h2d = sum(host[a].numel() * host[a].element_size() for a in names_in)
    d2h = sum(r.numel() * r.element_size() for r in res_dev[0])
    s_comp = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    in_ready = [torch.cuda.Event() for _ in range(2)]
    comp_done = [torch.cuda.Event() for _ in range(2)]
    out_copied = [torch.cuda.Event() for _ in range(2)]

    def e2e_step(i):
        buf = i & 1
        ti, rd = t_in[buf], res_dev[buf]
        with torch.cuda.stream(s_in):
            if i >= 2:
                s_in.wait_event(comp_done[buf])        # the kernels that read this input set are done
            for a in names_in:
                ti[a].copy_(host[a], non_blocking=True)
            in_ready[buf].record(s_in)
        s_comp.wait_event(in_ready[buf])
        if i >= 2:
            s_comp.wait_event(out_copied[buf])         # this result set has been read out
        binding.bpt_attn_fwd(g, ti["q"], ti["k"], ti["v"], ti["rel_emb"], scale, out=rd[0], lse=rd[1], workspace=ws, path=path)
        if do_bwd:
            binding.bpt_attn_bwd(g, ti["q"], ti["k"], ti["v"], ti["rel_emb"], scale, rd[0], rd[1], ti["d_out"], workspace=ws,
                                 dq=rd[2], dk=rd[3], dv=rd[4], d_rel=rd[5], path=path)
            shard.allreduce_d_rel(rd[5])
        comp_done[buf].record(s_comp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(comp_done[buf])
            for r_d, r_h in zip(rd, res_host):
                r_h.copy_(r_d, non_blocking=True)
            out_copied[buf].record(s_out)

    e2e_steps = max(4, min(args.steps, 10))
    e2e_step(0)
    e2e_step(1)
    barrier()
    e0.record()
    for i in range(e2e_steps):
        e2e_step(i + 2)
    s_comp.wait_stream(s_out)
    s_comp.wait_stream(s_in)
    e1.record()
    barrier()
    ms_e2e = max_over_ranks(e0.elapsed_time(e1)) / e2e_steps

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- per-kernel shares and the roofline of the dominant kernel --------------------
    per = {}
    for name, ms in marks:
        per.setdefault(name, []).append(ms)
    total_ms = max(sum(m for _, m in marks), 1e-9)
    kernels = {name: {"launches": len(v), "avg_ms": sum(v) / len(v), "min_ms": min(v), "median_ms": statistics.median(v),
                      "max_ms": max(v), "share": sum(v) / total_ms} for name, v in per.items()}
    peak, tf_peak, peak_kind = load_peaks()
    E_span = cfg["n"] * (cfg["n"].bit_length() - 1)          # affiliated edges: one per token and level
    edges_of = {"all": E, "token": E - E_span, "span": E_span}
    modelled = [a for a in kernels if a in KERNEL_MODEL]
    dominant = max(modelled, key=lambda a: kernels[a]["avg_ms"] * kernels[a]["launches"]) if modelled else None
    roofline = None
    if dominant:
        passes, rows = KERNEL_MODEL[dominant]
        alg_bytes = sum(GATHER_BYTES_PER_EDGE_HEAD[a](d, esize) for a in passes) * B * H * edges_of[rows]
        achieved = alg_bytes / (kernels[dominant]["avg_ms"] * 1e-3) / 1e9
        per_pair = ncu_traffic_per_pair(dominant)
        roofline = {"bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak, "peak_kind": peak_kind + " copy bandwidth",
                    "unit": "GB/s", "frac": achieved / peak, "traffic": None if per_pair is None else per_pair * B * H,
                    "algorithmic_bytes": alg_bytes,
                    "model": "gather model: K/V (and, backward, Q/dO) rows fetched per edge and head with no on-chip reuse "
                             "credited; the tiled kernels stage each level's node range once per tile, so frac > 1 "
                             "measures that reuse, and `traffic` (ncu DRAM bytes) shows what HBM really moved"}
    # whole-step fraction of the gather-model roofline (the target figure of the benchmark definition)
    gathered = sum(GATHER_BYTES_PER_EDGE_HEAD[a](d, esize) for a in (["fwd", "bwd_dst", "bwd_src"] if do_bwd else ["fwd"])) * B * H * E
    step_roof_ms = gathered / (peak * 1e9) * 1e3
    # lower bound of a step: every input and output tensor crosses HBM once
    compulsory = ((4 + (5 if do_bwd else 0)) * B * N * H * d * esize + 4 * B * N * H * (2 if do_bwd else 1))
    compulsory_ms = compulsory / (peak * 1e9) * 1e3
    # true lower bound: the slower of the compulsory HBM traffic and the algorithmic FLOPs on the tensor cores
    flops_alg = (FLOPS_PER_EDGE_HEAD["fwd"] + (FLOPS_PER_EDGE_HEAD["bwd"] if do_bwd else 0)) * d * B * H * E
    flops_ms = flops_alg / (tf_peak * 1e12) * 1e3
    lower_bound_ms = max(compulsory_ms, flops_ms)
    if roofline:   # the same bound for the dominant kernel alone: its share of the algorithmic FLOPs, its own compulsory tensors
        passes, rows = KERNEL_MODEL[dominant]
        k_flops = sum({"fwd": 6, "bwd_dst": 8, "bwd_src": 6}[a] for a in passes) * d * B * H * edges_of[rows]
        k_tensors = {"fwd": 4, "bwd_dst": 6, "bwd_src": 6}   # node-major tensors the pass must read or write once
        k_bytes = sum(k_tensors[a] for a in passes) * B * N * H * d * esize
        k_lb = max(k_bytes / (peak * 1e9), k_flops / (tf_peak * 1e12)) * 1e3
        roofline.update(lower_bound_ms=k_lb, lower_bound_frac=k_lb / kernels[dominant]["avg_ms"],
                        flops_alg=k_flops, compulsory_bytes=k_bytes)

    # per-step series from the per-launch marks (launch order repeats every step)
    per_step = []
    if marks and len(marks) % args.steps == 0:
        n_per = len(marks) // args.steps
        per_step = [sum(m for _, m in marks[i * n_per:(i + 1) * n_per]) for i in range(args.steps)]
    # forward and backward separately: the forward's launches are the fwd_* kernels and the table kernel right before fwd_tc5
    fwd_ms = bwd_ms = None
    if per_step:
        f_sum = 0.0
        for i, (name, m) in enumerate(marks):
            nxt = marks[i + 1][0] if i + 1 < len(marks) else ""
            if name.startswith("fwd") or (name == "level_ranges" and nxt.startswith("fwd")):
                f_sum += m
        fwd_ms = f_sum / args.steps
        bwd_ms = sum(per_step) / args.steps - fwd_ms
    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if cfg["bf16"] else "f32", "data": "synthetic",
        "config": {"workload": cfg_name, "n": cfg["n"], "k": cfg["k"], "left_only": bool(cfg["flags"] & 1),
                   "batch_per_gpu": B, "heads": H, "d_head": d, "edges_per_sequence": E,
                   "pass": "fwd+bwd" if do_bwd else "fwd",
                   "l2": "flushed by a 256 MB write between timed steps" if flush else "inputs larger than L2", "parallelism": "batch shards x%d" % world,
                   "kernels": args.path},
        "edge_heads_per_s": value * H, "tokens_per_s": world * B * cfg["n"] / (ms_step * 1e-3),
        "hbm_roofline_frac_step": step_roof_ms / ms_step, "hbm_roofline_ms_step": step_roof_ms,
        "compulsory_hbm_ms_step": compulsory_ms, "compulsory_hbm_frac_step": compulsory_ms / ms_step,
        "flops_alg": flops_alg, "flops_ms_at_sustained_bf16_peak": flops_ms, "tensor_peak_tflops": tf_peak,
        "lower_bound_ms": lower_bound_ms, "lower_bound_frac": lower_bound_ms / ms_step,
        "clocks": clocks,
        "e2e": {"value": world * B * E / (ms_e2e * 1e-3), "unit": UNIT, "ms_per_step": ms_e2e,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "overlap": "copies of the neighbouring steps run under the kernels (three streams, two buffer sets)"},
        "gpu_launches": len(marks),
        "fwd_ms_per_step": fwd_ms, "bwd_ms_per_step": bwd_ms if do_bwd else None, "graph_build_call_ms": graph_build_ms,   # the whole binding call: device allocations of its arrays + 8 kernels (0.2 ms of kernels at the metric config)
        "cuda_graph": None if ms_graph is None else {"ms_per_step": ms_graph, "value": world * B * E / (ms_graph * 1e-3), "unit": UNIT,
                                                      "what": "the same step replayed from one CUDA graph, same L2 policy"},
        "step_ms_series": {"min": min(per_step), "median": statistics.median(per_step), "max": max(per_step),
                           "first": per_step[0], "last": per_step[-1]} if per_step else None,
        "kernels": kernels,
        "roofline": roofline,
    }
    if world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline(cfg)
    print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


def run_sweep(args):
    """Scaling sweep (n x k grid at 262144 tokens per batch): one JSON line per point with the measured
    step, the algorithmic FLOPs of the sparse attention and the dense full-attention FLOP / byte count
    at the same n.  Inputs are seeded normal draws made on the device (timing only)."""
    import torch
    from paper_1911_04070_b200 import binding, synth
    torch.cuda.set_device(0)
    peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))) if os.path.exists(os.path.join(ROOT, "MEASURED_PEAKS.json")) else {}
    tf_peak = float(peaks.get("bf16_tflops", 1590.0))
    for name, cfg in synth.sweep_configs().items():
        B, H, d, n = cfg["B"], cfg["H"], cfg["d"], cfg["n"]
        g = binding.bpt_build_graph(n, cfg["k"], cfg["flags"], device="cuda:0")
        gen = torch.Generator(device="cuda:0").manual_seed(cfg["seed"])
        shape = (B, g.n_nodes, H, d)
        q, k, v = ((torch.randn(shape, generator=gen, device="cuda:0") * cfg["std_qkv"]).bfloat16() for _ in range(3))
        r = (torch.randn((g.n_rel, d), generator=gen, device="cuda:0") * 0.02).bfloat16()
        d_out = torch.randn(shape, generator=gen, device="cuda:0").bfloat16()
        ws = torch.empty(max(binding.bpt_attn_workspace_bytes(g, B, H, d, binding.BPT_BF16, True),
                             binding.bpt_attn_workspace_bytes(g, B, H, d, binding.BPT_BF16, False), 1), dtype=torch.uint8, device="cuda:0")
        out = torch.empty_like(q); lse = torch.empty((B, g.n_nodes, H), dtype=torch.float32, device="cuda:0")
        dq, dk, dv = (torch.empty_like(q) for _ in range(3))
        d_rel = torch.empty((g.n_rel, d), dtype=torch.float32, device="cuda:0")

        def step():
            binding.bpt_attn_fwd(g, q, k, v, r, d ** -0.5, out=out, lse=lse, workspace=ws)
            binding.bpt_attn_bwd(g, q, k, v, r, d ** -0.5, out, lse, d_out, workspace=ws, dq=dq, dk=dk, dv=dv, d_rel=d_rel)

        for _ in range(3):
            step()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        steps = max(3, min(args.steps, 10))
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        E = g.n_edges
        bpt_flop = 20.0 * d * B * H * E                 # algorithmic: 6d forward + 14d backward per edge and head
        dense_flop = 14.0 * n * n * d * B * H           # full attention over the n tokens, forward + backward
        dense_bytes = 9.0 * B * n * H * d * 2 + 8.0 * B * n * H
        print(json.dumps({
            "workload": name, "n": n, "k": cfg["k"], "batch": B, "edges_per_sequence": E, "ms_per_step": ms,
            "edges_per_s": B * E / (ms * 1e-3), "tokens_per_s": B * n / (ms * 1e-3),
            "bpt_algorithmic_tflop": bpt_flop / 1e12, "bpt_achieved_tflops": bpt_flop / (ms * 1e-3) / 1e12,
            "dense_tflop": dense_flop / 1e12, "dense_compulsory_gb": dense_bytes / 1e9,
            "dense_ms_at_measured_bf16_peak": dense_flop / (tf_peak * 1e12) * 1e3,
            "dense_over_bpt_flop": dense_flop / bpt_flop,
            "speed_vs_dense_at_peak": dense_flop / (tf_peak * 1e12) * 1e3 / ms}), flush=True)
        del q, k, v, r, d_out, ws, out, lse, dq, dk, dv, d_rel, g
        torch.cuda.empty_cache()


def run_model(args):
    """Whole-model figure in the setting of the paper's Sec. 4.4 (6 layers, d = 512, d_ff = 2048, 8 heads,
    8192 tokens per batch, bf16): tokens/s of a forward pass (inference) and of a forward + backward pass
    through BPTEncoder, for a few sequence lengths and k.  One JSON line per point."""
    import torch
    from paper_1911_04070_b200 import layer
    torch.cuda.set_device(0)
    torch.manual_seed(0)
    for n in (512, 2048, 8192):
        for k in (4, 16, 64):
            B = 8192 // n
            enc = layer.BPTEncoder(n, k, 512, 8, 2048, 6, left_only=True, device="cuda:0").to("cuda:0", torch.bfloat16)
            x = torch.randn(B, n, 512, device="cuda:0", dtype=torch.bfloat16, requires_grad=True)

            def fwd():
                with torch.no_grad():
                    enc(x)

            def train():
                enc.zero_grad(set_to_none=True)
                enc(x).float().square().mean().backward()

            res = {}
            for name, fn in (("forward", fwd), ("forward_backward", train)):
                for _ in range(3):
                    fn()
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                steps = max(3, min(args.steps, 10))
                e0.record()
                for _ in range(steps):
                    fn()
                e1.record()
                torch.cuda.synchronize()
                res[name] = e0.elapsed_time(e1) / steps
            print(json.dumps({"workload": "6-layer BPT stack, d=512, d_ff=2048, 8 heads, left-only, 8192 tokens per batch, bf16",
                              "n": n, "k": k, "batch": B, "forward_ms": res["forward"], "forward_tokens_per_s": 8192 / (res["forward"] * 1e-3),
                              "forward_backward_ms": res["forward_backward"],
                              "forward_backward_tokens_per_s": 8192 / (res["forward_backward"] * 1e-3)}), flush=True)
            del enc, x
            torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg4_char_lm")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--path", default="auto", choices=["auto", "mma", "tc5"],
                    help="kernel family of the token rows: the library's choice by k, the warp-level (mma.sync) kernels, or the tensor-memory (tcgen05) kernels")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (profiling of a smaller case)")
    ap.add_argument("--sweep", action="store_true", help="run the n x k scaling sweep instead: one JSON line per point")
    ap.add_argument("--model", action="store_true", help="time a 6-layer BPT stack (Sec. 4.4 setting) instead: one JSON line per point")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    if args.sweep:
        return run_sweep(args)
    if args.model:
        return run_model(args)
    cfgs = all_configs()
    if args.config not in cfgs:
        raise SystemExit("unknown config %s; choose from %s" % (args.config, ", ".join(sorted(cfgs))))
    cfg = dict(cfgs[args.config])
    if args.batch > 0:
        cfg["B"] = args.batch
    if args.impl == "reference":
        run_reference(args, args.config, cfg)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # asked for N GPUs without a launcher: start one rank per GPU of this node and let them run this script
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
               "--master-addr", "127.0.0.1", "--master-port", str(29500 + os.getpid() % 2000), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd, env=dict(os.environ, NCCL_DEBUG=os.environ.get("NCCL_DEBUG", "INFO"))))
    else:
        if args.warmup < 3:
            args.warmup = 3
        run_ours(args, args.config, cfg)


if __name__ == "__main__":
    main()
