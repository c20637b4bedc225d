#!/usr/bin/env python
"""Benchmark of the draft-branch-attention hot path (forward + backward).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One step = one pass of the whole hot path over one synthetic batch: metadata
plan reuse, fused forward (through the partial-(O, LSE) + lse_merge zigzag
path for the long-context workload), backward preprocess, dQ, dK/dV, gradient
finalisation.  Prints ONE JSON line (rank 0).  `--impl reference` times the
fp64 CPU oracle on a bounded sample of the same workload instead.
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_07108_b200 import workloads as W  # noqa: E402

METRIC = "branch_attn_fwd_bwd_useful_tflops"
UNIT = "TFLOP/s"
DATASHEET_BF16_TFLOPS = 2250.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# name -> (config number, shrink, zigzag cp or 0, backward?)
WORKLOADS = {
    "config5_256k_zigzag": (5, 1, 8, True),
    "config5_256k_monolithic": (5, 1, 0, True),
    "config5_256k_zigzag_fwd": (5, 1, 8, False),
    "config5_256k_monolithic_fwd": (5, 1, 0, False),
    "config5_64k_zigzag": (5, 4, 8, True),
    "config4_tree_64k": (4, 1, 0, True),
    "config3_dflash_32k": (3, 1, 0, True),
    "config2_eagle3_8k": (2, 1, 0, False),
    # shape of the paper's packed variable-length operator benchmark (longest sequence 20,480 tokens)
    "varlen_ttt_72k": (6, 1, 0, True),
    # the same shape through the step-major calls: main rows, then depth 1, 2, 3 in turn
    "varlen_ttt_72k_stepwise": (6, 1, "stepwise", True),
    # config 5 through the K/V ring driver (shards copied into a local double buffer on a side stream)
    "config5_256k_ring": (5, 1, ("ring", 8), True),
}


# DRAM traffic of the dominant kernels comes from profiles/dram_traffic.json: one ncu capture
# per kernel on a small case (dram__bytes_read.sum + dram__bytes_write.sum of one launch),
# stored with the hash of the kernel's source files at capture time.  It is scaled to this
# workload's launches by the query rows a launch streams (Q, dO and the dQ accumulator rows
# are what the kernel moves); if the sources have changed since the capture, traffic is null.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.json")
CSRC = os.path.join(ROOT, "paper_2609_07108_b200", "csrc")


def source_hash(files):
    import hashlib
    h = hashlib.sha256()
    for f in sorted(files):
        with open(os.path.join(CSRC, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(kernel_name, rows_per_launch):
    """(bytes per launch scaled to `rows_per_launch`, description) or (None, reason)."""
    try:
        with open(TRAFFIC_FILE) as f:
            table = json.load(f)
    except (OSError, ValueError):
        return None, "no capture on file"
    e = table.get(kernel_name)
    if not e:
        return None, "no capture on file"
    if source_hash(e["source_files"]) != e["source_hash"]:
        return None, "kernel source changed since the capture"
    scaled = e["dram_bytes_per_launch"] * rows_per_launch / e["query_rows_per_launch"]
    return scaled, (f"ncu one launch on {e['case']} ({e['dram_bytes_per_launch'] / 1e6:.0f} MB for "
                    f"{e['query_rows_per_launch']} query rows) scaled by query rows; commit {e['commit']}")


def useful_flops(p, backward=True, branch_only=False):
    pairs = W.useful_pairs(p, with_main_queries=not branch_only)
    per_pair = 4 * p.head_dim * p.h_q
    return pairs * per_pair * (3.5 if backward else 1.0), pairs


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


# ----------------------------------------------------------------------------
# distributed plumbing (replicas only: no data-path collective)
# ----------------------------------------------------------------------------

def dist_setup(n_gpus, backend=None):
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world <= 1:
        return None, 0, 1
    backend = backend or ("nccl" if torch.cuda.is_available() else "gloo")
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    dist.init_process_group(backend=backend)
    return dist, dist.get_rank(), dist.get_world_size()


def max_over_ranks(dist, value, device="cpu"):
    """Slowest rank's time (the job finishes when the last replica does)."""
    import torch
    if dist is None:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(dist, flops_per_rank, local_ms, device="cpu"):
    """Whole-job throughput: every rank processed `flops_per_rank`; time = max."""
    world = 1 if dist is None else dist.get_world_size()
    ms = max_over_ranks(dist, local_ms, device)
    return world * flops_per_rank / (ms * 1e-3) / 1e12, ms


# ----------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------

class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "200", "-i", str(self.index)], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        res = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return res
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, reasons, mx, power = [], set(), None, []
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx = float(f[2]); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                  "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        if sm:
            res.update(sm_mhz=statistics.median(sm), sm_max_mhz=mx, reasons=sorted(reasons),
                       samples=len(sm), power_w_max=max(power))
        return res


# ----------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------

class Recorder:
    """Wraps the binding: counts kernel launches and brackets each library call
    with CUDA events on the launching stream so that per-kernel time inside the
    timed region can be summed afterwards."""

    def __init__(self, ba, plan_problem):
        import torch
        self.ba = ba
        self.torch = torch
        self.p = plan_problem
        self.events = []           # (kind, start, end)
        self.launches = 0
        self.enabled = False
        for name in ("PART_MAIN", "PART_BRANCH", "PART_ALL", "STAGE_ALL", "STAGE_ALL_FUSED", "STAGE_PREP", "STAGE_DQ",
                     "STAGE_DKDV", "STAGE_FUSED", "IMPL_TC"):
            setattr(self, name, getattr(ba, name))

    def _wrap(self, kind, n_launch, fn, *a, **k):
        if self.enabled:
            s = self.torch.cuda.Event(enable_timing=True)
            e = self.torch.cuda.Event(enable_timing=True)
            s.record()
            out = fn(*a, **k)
            e.record()
            self.events.append((kind, s, e))
            self.launches += n_launch
            return out
        return fn(*a, **k)

    def branch_attn_fwd(self, *a, **k):
        return self._wrap("fwd", 1, self.ba.branch_attn_fwd, *a, **k)

    def branch_attn_fwd_partial(self, *a, **k):
        return self._wrap("fwd", 1, self.ba.branch_attn_fwd_partial, *a, **k)

    def branch_attn_fwd_partial_merge(self, *a, **k):
        return self._wrap("fwd", 1, self.ba.branch_attn_fwd_partial_merge, *a, **k)

    def lse_merge(self, *a, **k):
        return self._wrap("lse_merge", 1, self.ba.lse_merge, *a, **k)

    def branch_attn_bwd(self, plan, q_main, *a, **k):
        # every stage of a backward call is bracketed separately: preprocess (one launch for the
        # main and the branch rows), dQ kernel, dK/dV kernel -- or the one fused kernel
        ba = self.ba
        k = dict(k)
        stages = k.pop("stages", ba.STAGE_ALL)
        acc = k.get("accumulate", False)
        fused_extra = 0 if acc else (2 if q_main is not None else 1)   # conversion of the fp32 dQ accumulators
        single = {ba.STAGE_PREP: ("bwd_prep", 1), ba.STAGE_DQ: ("bwd_dq", 1), ba.STAGE_DKDV: ("bwd_dkdv", 1),
                  ba.STAGE_FUSED: ("bwd_fused", 1 + fused_extra)}
        if stages in single:
            kind, n_l = single[stages]
            return self._wrap(kind, n_l, ba.branch_attn_bwd, plan, q_main, *a, stages=stages, **k)
        fused = stages == ba.STAGE_ALL_FUSED
        # gradients in the input dtype through the one-kernel backward: all stages share the larger workspace
        prep_kw = {"fused_scratch": True} if fused and not acc else {}
        out = self._wrap("bwd_prep", 1, ba.branch_attn_bwd, plan, q_main, *a, stages=ba.STAGE_PREP, **prep_kw, **k)
        k2 = dict(k)
        k2["grads"] = out
        if fused:   # one kernel for dQ, dK and dV
            return self._wrap("bwd_fused", 1 + fused_extra, ba.branch_attn_bwd, plan, q_main, *a,
                              stages=ba.STAGE_FUSED, **k2)
        self._wrap("bwd_dq", 1, ba.branch_attn_bwd, plan, q_main, *a, stages=ba.STAGE_DQ, **k2)
        return self._wrap("bwd_dkdv", 1, ba.branch_attn_bwd, plan, q_main, *a, stages=ba.STAGE_DKDV, **k2)

    def ba_finalize_grads(self, *a, **k):
        return self._wrap("finalize", 1, self.ba.ba_finalize_grads, *a, **k)

    def branch_attn_fwd_shard(self, *a, **k):
        return self._wrap("fwd", 1, self.ba.branch_attn_fwd_shard, *a, **k)

    def branch_attn_bwd_shard(self, *a, **k):
        ba = self.ba
        kind = {ba.STAGE_DQ: "bwd_dq", ba.STAGE_DKDV: "bwd_dkdv", ba.STAGE_FUSED: "bwd_fused"}[k["stages"]]
        return self._wrap(kind, 1, ba.branch_attn_bwd_shard, *a, **k)

    def branch_attn_fwd_depth(self, *a, **k):
        return self._wrap("fwd", 1, self.ba.branch_attn_fwd_depth, *a, **k)

    def branch_attn_bwd_depth(self, *a, **k):     # delta, the one-kernel backward, conversion of dQ
        return self._wrap("bwd_depth", 3, self.ba.branch_attn_bwd_depth, *a, **k)

    def totals(self):
        out = {}
        for kind, s, e in self.events:
            out.setdefault(kind, [0.0, 0])
            out[kind][0] += s.elapsed_time(e)
            out[kind][1] += 1
        return out


def make_device_inputs(p, torch, device, seed=0):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    dt = torch.bfloat16 if p.dtype == "bf16" else torch.float32

    def draw(shape, std):
        return (torch.randn(shape, generator=g, device=device, dtype=torch.float32) * std).to(dt)

    n, m = p.n_main, p.n_branch
    t = {"q_main": draw((n, p.h_q, p.head_dim), 0.5), "q_branch": draw((m, p.h_q, p.head_dim), 0.5),
         "k": draw((n + m, p.h_kv, p.head_dim), 0.5), "v": draw((n + m, p.h_kv, p.head_dim), 0.5),
         "d_o": draw((n + m, p.h_q, p.head_dim), 0.1)}
    return t


def run_fwd(rec, plan, t, cp):
    from paper_2609_07108_b200 import ring, zigzag
    mode = t.get("_mode", "zigzag" if cp else "mono")
    if mode == "stepwise":
        return stepwise_fwd(rec, plan, t)
    if mode == "ring":
        o, lse, _ = ring.forward(rec, plan, t["q_main"], t["q_branch"], t["k"], t["v"], cp, out=t.get("_o"),
                                 lse=t.get("_lse"), ws=t.get("_ws"), bufs=t["_bufs"], stats=t.get("_ring_stats"))
        return o, lse
    if cp:
        o, lse, _ = zigzag.forward(rec, plan, t["q_main"], t["q_branch"], t["k"], t["v"], cp,
                                   out=t.get("_o"), lse=t.get("_lse"), ws=t.get("_ws"))
        return o, lse
    return rec.branch_attn_fwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"], out=t.get("_o"), lse=t.get("_lse"))


def run_bwd(rec, plan, t, cp, o, lse, fused=False):
    from paper_2609_07108_b200 import ring, zigzag
    mode = t.get("_mode", "zigzag" if cp else "mono")
    if mode == "stepwise":
        return stepwise_bwd(rec, plan, t, o, lse, fused)
    if mode == "ring":
        return ring.backward(rec, plan, t["q_main"], t["q_branch"], t["k"], t["v"], o, lse, t["d_o"], cp,
                             fused=fused, ws=t.get("_ws"), bufs=t["_bufs"], stats=t.get("_ring_stats"))
    if cp:
        return zigzag.backward(rec, plan, t["q_main"], t["q_branch"], t["k"], t["v"], o, lse, t["d_o"], cp,
                               fused=fused, ws=t.get("_ws"))
    return rec.branch_attn_bwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"], o, lse, t["d_o"],
                               grads=t.get("_grads"), stages=rec.STAGE_ALL_FUSED if fused else rec.STAGE_ALL)


def run_step(rec, plan, t, cp, backward, fused=False):
    o, lse = run_fwd(rec, plan, t, cp)
    grads = run_bwd(rec, plan, t, cp, o, lse, fused=fused) if backward else None
    return o, lse, grads


# ---- the step-major form: the main rows through a branch-free plan, then one call per depth
# (a trainer produces the depth-d tokens only after depth d - 1), branch K / V stored depth-major

def stepwise_setup(ba, plan, p, t, torch, device):
    n, a, length = p.n_main, p.num_branches, int(p.branch_offsets[1])
    main_p = W.Problem(p.cu_seqlens, np.zeros(0, np.int32), np.zeros(1, np.int32), W.CHAIN, None, p.h_q, p.h_kv,
                       p.head_dim, dtype=p.dtype, name=p.name + "_main_rows")
    s = {"plan_main": ba.Plan(main_p, device=device, impl=plan.impl), "n": n, "a": a, "len": length}
    hq, hkv, d = p.h_q, p.h_kv, p.head_dim
    dt = plan.torch_dtype
    # the same random values, regrouped: queries / cotangents per depth, branch keys depth-major
    s["q_d"] = [t["q_branch"].reshape(a, length, hq, d)[:, j].contiguous() for j in range(length)]
    s["go_main"] = t["d_o"][:n].contiguous()
    s["go_d"] = [t["d_o"][n:].reshape(a, length, hq, d)[:, j].contiguous() for j in range(length)]

    def dm(x):
        return torch.cat([x[:n], x[n:].reshape(a, length, hkv, d).transpose(0, 1).reshape(a * length, hkv, d)], 0).contiguous()

    s["k"], s["v"] = dm(t["k"]), dm(t["v"])
    s["k_main"], s["v_main"] = s["k"][:n], s["v"][:n]
    s["o_main"] = torch.empty((n, hq, d), dtype=dt, device=device)
    s["lse_main"] = torch.empty((n, hq), dtype=torch.float32, device=device)
    s["o_d"] = [torch.empty((a, hq, d), dtype=dt, device=device) for _ in range(length)]
    s["lse_d"] = [torch.empty((a, hq), dtype=torch.float32, device=device) for _ in range(length)]
    s["dq_main32"] = torch.empty((n, hq, d), dtype=torch.float32, device=device)
    s["dq_main"] = torch.empty((n, hq, d), dtype=dt, device=device)
    s["dq_d"] = [torch.empty((a, hq, d), dtype=dt, device=device) for _ in range(length)]
    s["dk32"] = torch.empty((p.rows, hkv, d), dtype=torch.float32, device=device)
    s["dv32"] = torch.empty((p.rows, hkv, d), dtype=torch.float32, device=device)
    s["dk"] = torch.empty((p.rows, hkv, d), dtype=dt, device=device)
    s["dv"] = torch.empty((p.rows, hkv, d), dtype=dt, device=device)
    s["none"] = torch.empty((0, hq, d), dtype=torch.float32, device=device)
    return s


def stepwise_fwd(rec, plan, t):
    s = t["_sw"]
    rec.branch_attn_fwd(s["plan_main"], t["q_main"], None, s["k_main"], s["v_main"], out=s["o_main"], lse=s["lse_main"])
    for j in range(s["len"]):
        rec.branch_attn_fwd_depth(plan, j + 1, s["q_d"][j], s["k"], s["v"], out=s["o_d"][j], lse=s["lse_d"][j])
    return s["o_main"], s["lse_main"]


def stepwise_bwd(rec, plan, t, o, lse, fused):
    s = t["_sw"]
    n = s["n"]
    for x in (s["dq_main32"], s["dk32"], s["dv32"]):
        x.zero_()
    for j in reversed(range(s["len"])):            # deepest first, as backpropagation reaches them
        rec.branch_attn_bwd_depth(plan, j + 1, s["q_d"][j], s["k"], s["v"], s["o_d"][j], s["lse_d"][j], s["go_d"][j],
                                  s["dk32"], s["dv32"], dq=s["dq_d"][j])
    rec.branch_attn_bwd(s["plan_main"], t["q_main"], None, s["k_main"], s["v_main"], o, lse, s["go_main"],
                        accumulate=True, grads=(s["dq_main32"], s["none"], s["dk32"][:n], s["dv32"][:n]),
                        stages=rec.STAGE_ALL_FUSED if fused else rec.STAGE_ALL)
    rec.ba_finalize_grads(s["dq_main32"], dst=s["dq_main"])
    rec.ba_finalize_grads(s["dk32"], dst=s["dk"])
    rec.ba_finalize_grads(s["dv32"], dst=s["dv"])
    return s["dq_main"], s["dq_d"], s["dk"], s["dv"]


def use_fused_bwd(args, p, plan, ba):
    if plan.impl != ba.IMPL_TC or args.bwd == "split":
        return False
    return args.bwd == "fused" or p.n_main >= 131072


def run_ours(args):
    import torch
    from paper_2609_07108_b200 import binding as ba

    dist, rank, world = dist_setup(args.gpus)
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)

    name = args.workload
    if name == "auto":
        name = "config5_256k_zigzag"
    cfg, shrink, cp, backward = WORKLOADS[name]
    mode = "zigzag" if cp else "mono"
    if cp == "stepwise":
        mode, cp = "stepwise", 0
    elif isinstance(cp, tuple):
        mode, cp = cp
    p = W.CONFIGS[cfg](shrink) if cfg != 1 else W.config1()
    impl = {"auto": ba.IMPL_AUTO, "simt": ba.IMPL_SIMT, "tc": ba.IMPL_TC}[args.kernels]
    plan = ba.Plan(p, device=device, impl=impl)
    # metadata builder, timed on its own (it is reused by the forward, the backward and, in a
    # model, every layer): host wall clock around ba_plan_create incl. its stream synchronisations
    plan_times = []
    for _ in range(3):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        extra = ba.Plan(p, device=device, impl=impl)
        torch.cuda.synchronize()
        plan_times.append((time.perf_counter() - t0) * 1e3)
        extra.close()
    plan_ms = statistics.median(plan_times)
    branch_only = bool(args.branch_only)
    if branch_only and cp:
        raise SystemExit("--branch-only applies to the monolithic workloads")
    flops, pairs = useful_flops(p, backward, branch_only)
    t = make_device_inputs(p, torch, device)
    if branch_only:
        t["q_main"] = None   # draft-only form: main K/V are keys, only branch tokens are queries
    # outputs and (zigzag) the fp32 accumulators are allocated once, outside the steps
    t["_o"] = torch.empty((p.rows, p.h_q, p.head_dim), dtype=plan.torch_dtype, device=device)
    t["_lse"] = torch.empty((p.rows, p.h_q), dtype=torch.float32, device=device)
    t["_mode"] = mode
    if mode == "stepwise":
        t["_sw"] = stepwise_setup(ba, plan, p, t, torch, device)
    elif cp:
        from paper_2609_07108_b200 import ring, zigzag
        t["_ws"] = zigzag.Workspace(ba, plan, cp, backward=backward)
        if mode == "ring":
            t["_bufs"] = ring.RingBuffers(plan, cp)
    elif backward:
        t["_grads"] = (torch.empty((p.n_main, p.h_q, p.head_dim), dtype=plan.torch_dtype, device=device)
                       if not branch_only else None,
                       torch.empty((p.n_branch, p.h_q, p.head_dim), dtype=plan.torch_dtype, device=device),
                       torch.empty((p.rows, p.h_kv, p.head_dim), dtype=plan.torch_dtype, device=device),
                       torch.empty((p.rows, p.h_kv, p.head_dim), dtype=plan.torch_dtype, device=device))
    rec = Recorder(ba, p)
    in_bytes = sum(t[k].numel() * t[k].element_size() for k in ("q_main", "q_branch", "k", "v", "d_o")
                   if t[k] is not None)
    flush = None
    if in_bytes < 512 << 20:
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    fused = use_fused_bwd(args, p, plan, ba)
    for _ in range(args.warmup):
        run_step(rec, plan, t, cp, backward, fused=fused)
        if flush is not None:
            flush.fill_(1)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    rec.enabled = True
    step_ms = []
    if mode == "ring":
        from paper_2609_07108_b200 import ring
        t["_ring_stats"] = ring.new_stats()
    barrier()
    for _ in range(args.steps):
        if flush is not None:
            flush.fill_(1)
        s = torch.cuda.Event(enable_timing=True)
        e = torch.cuda.Event(enable_timing=True)
        s.record()
        last = run_step(rec, plan, t, cp, backward, fused=fused)
        e.record()
        step_ms.append((s, e))
    barrier()
    rec.enabled = False
    clocks = sampler.stop() if rank == 0 else {}
    local_ms = sum(s.elapsed_time(e) for s, e in step_ms)
    value, total_ms = aggregate_throughput(dist, flops * args.steps, local_ms, device)
    totals = rec.totals()
    launches = rec.launches
    ring_report = None
    if mode == "ring":
        # Eq. (cp-comm) volume, the copies' own device time, and the exposed part: this driver's step
        # against the same kernels run without any copy (the range-based zigzag driver)
        stats = t.pop("_ring_stats")
        t["_mode"] = "zigzag"
        s0 = torch.cuda.Event(enable_timing=True)
        e0 = torch.cuda.Event(enable_timing=True)
        s0.record()
        run_step(Recorder(ba, p), plan, t, cp, backward, fused=fused)
        e0.record()
        torch.cuda.synchronize()
        t["_mode"] = "ring"
        zz_ms = s0.elapsed_time(e0)
        ring_ms = local_ms / args.steps
        passes = (2 if backward else 1) * args.steps          # the backward replays the ring
        copy_total = ring.copy_ms(stats)
        n_copies = len(stats["copies"])
        ring_report = {
            "shard_bytes_per_rank_per_pass": ring.shard_bytes_per_rank(p, cp, 2),
            "copied_bytes_per_rank_per_pass": stats["copied_bytes"] // (cp * passes),
            "t_comm_ms_per_ring_step": round(copy_total / max(n_copies, 1), 4),
            "t_attn_ms_per_ring_step": round((ring_ms - 0.0) / ((2 if backward else 1) * cp * cp), 4),
            "step_ms_ring": round(ring_ms, 3), "step_ms_without_copies": round(zz_ms, 3),
            "exposed_ms_per_step": round(ring_ms - zz_ms, 3),
            "model": "Eq. cp-overlap: ring step time = max(t_comm, t_attn); exposed = max(0, t_comm - t_attn)",
            "transport": "device copies into a local double buffer on one GPU; unmeasured over NVLink"}

    # ---- CPU baseline (the oracle on a bounded sample of the same inputs) and the GPU's error
    # against it on those rows; before the end-to-end run, which overwrites inputs and outputs
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(p, seconds_target=15.0, backward=backward,
                           gpu=None if (branch_only or mode == "stepwise") else (t, last))

    # ---- end to end through the API with HOST buffers (pinned), copies timed
    e2e = None
    if not args.no_e2e and mode != "stepwise":
        e2e = run_e2e(torch, ba, plan, p, t, cp, backward, flops, dist, device, args)

    # ---- dominant kernel and its roofline
    peaks = load_peaks()
    roof = None
    if totals:
        kind = max(totals, key=lambda k: totals[k][0])
        ms, calls = totals[kind]
        # algorithmic flop of all launches of that kind over the timed steps
        # flop per visible pair and query head that the kernel itself executes, in
        # units of head_dim: forward 2 GEMMs (QK^T, PV); dQ kernel 3 (S, dP, dQ);
        # dK/dV kernel 4 (S^T and dP^T recomputed, dV, dK)
        share = {"fwd": 4.0, "bwd_dq": 6.0, "bwd_dkdv": 8.0, "bwd_fused": 10.0, "bwd_depth": 10.0}.get(kind)
        kernel_name = {"fwd": "tc_fwd_kernel", "bwd_dq": "tc_dq_kernel", "bwd_dkdv": "tc_dkdv_kernel",
                       "bwd_fused": "tc_bwd_fused_kernel", "bwd_depth": "tc_bwd_fused_kernel"}.get(kind, kind)
        if share is not None:
            kpairs = pairs
            if mode == "stepwise" and kind != "fwd":    # the per-depth calls cover the branch rows only
                lens = np.diff(p.cu_seqlens.astype(np.int64))
                main_pairs = int((lens * (lens + 1) // 2).sum())
                kpairs = pairs - main_pairs if kind == "bwd_depth" else main_pairs
            kflops = kpairs * p.head_dim * p.h_q * share * args.steps
            achieved = kflops / (ms * 1e-3) / 1e12
            long_step = total_ms / args.steps > 1000.0
            # query rows (row, head) one launch streams on average, for scaling the ncu traffic capture
            rows_per_launch = query_rows_streamed(p, cp, kind) * args.steps / max(calls, 1)
            traffic, traffic_src = ncu_traffic(kernel_name, rows_per_launch)
            if traffic is not None:
                traffic = round(traffic)
            peak = peaks["bf16_tflops_sustained" if long_step else "bf16_tflops"]
            roof = {"bound": "tensor", "kernel": kernel_name, "flop_per_pair_head": share * p.head_dim,
                    "achieved": round(achieved, 2), "peak": peak,
                    "unit": "TFLOP/s", "frac": round(achieved / peak, 4),
                    "traffic": traffic, "traffic_source": traffic_src,
                    "peak_source": f"{peaks['_source']} {'sustained' if long_step else 'burst'} bf16",
                    "launches": calls, "avg_launch_ms": round(ms / calls, 4),
                    "frac_of_burst": round(achieved / peaks["bf16_tflops"], 4),
                    "frac_of_datasheet": round(achieved / DATASHEET_BF16_TFLOPS, 4)}
        else:
            roof = {"bound": "hbm", "kernel": kind, "achieved": None, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": None, "traffic": None}


    if rank == 0:
        line = {
            "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(total_ms / args.steps, 3), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": p.dtype, "data": "synthetic",
            "config": {"workload": name, "n_main": p.n_main, "rows": p.rows, "h_q": p.h_q, "h_kv": p.h_kv,
                       "head_dim": p.head_dim, "mask": W.KIND_NAMES[p.kind], "pairs_per_head": pairs,
                       "path": (f"zigzag cp={cp}: partial fwd merged by Eq. lse-merge "
                                + ("in the kernel epilogue" if plan.impl == ba.IMPL_TC else "with lse_merge")
                                + ", partial bwd accumulate"
                                + (", K/V shards of the remote ring steps copied into a local double buffer "
                                   "on a side stream" if mode == "ring" else "")
                                if cp else "step-major: main rows, then one call per depth (depth-major branch K/V)"
                                if mode == "stepwise" else "monolithic fwd + bwd"),
                       "backward": backward,
                       "bwd_kernels": ("one fused kernel (dQ by fp32 atomic adds)" if fused
                                       else "dQ kernel + dK/dV kernel") if backward else None,
                       "queries": "branch tokens only" if branch_only else "main + branch",
                       "kernels": {ba.IMPL_SIMT: "simt", ba.IMPL_TC: "tcgen05"}[plan.impl],
                       "l2": "inputs larger than L2" if flush is None else "256 MiB flush between steps",
                       "parallelism": "replicas" if world > 1 else "single"},
            "frac_of_peak": {"burst": round(value / world / peaks["bf16_tflops"], 4),
                             "sustained": round(value / world / peaks["bf16_tflops_sustained"], 4),
                             "datasheet": round(value / world / DATASHEET_BF16_TFLOPS, 4),
                             "source": peaks["_source"]},
            "kernel_ms": {k: round(v[0] / args.steps, 3) for k, v in totals.items()},
            "plan_ms": round(plan_ms, 3),
            "gpu_launches": launches,
            "clocks": clocks,
            "e2e": e2e,
            "roofline": roof,
            "cpu_baseline": cpu,
        }
        if ring_report is not None:
            line["ring"] = ring_report
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_e2e(torch, ba, plan, p, t, cp, backward, flops, dist, device, args):
    """Same step, inputs in pinned host memory: H2D of Q/K/V/dO, the library
    calls, D2H of O/LSE and the gradients, all inside the timed region.  The copy
    of dO overlaps the forward, the copy of O and LSE overlaps the backward; on the
    zigzag workload the query rows also arrive, and dQ also leaves, chunk by chunk
    (`e2e_step_streamed`), so that only K, V and the first chunk are waited for
    before the first kernel and only dK, dV and the last chunk's dQ after the last."""
    import psutil
    names = tuple(k for k in ("q_main", "q_branch", "k", "v") + (("d_o",) if backward else ()) if t[k] is not None)
    h2d = sum(t[k].numel() * t[k].element_size() for k in names)
    out_shapes = [((p.rows, p.h_q, p.head_dim), plan.torch_dtype), ((p.rows, p.h_q), torch.float32)]
    if backward:
        if t["q_main"] is not None:
            out_shapes += [((p.n_main, p.h_q, p.head_dim), plan.torch_dtype)]
        out_shapes += [((p.n_branch, p.h_q, p.head_dim), plan.torch_dtype),
                       ((p.rows, p.h_kv, p.head_dim), plan.torch_dtype),
                       ((p.rows, p.h_kv, p.head_dim), plan.torch_dtype)]
    d2h = sum(int(np.prod(s)) * torch.empty(0, dtype=d).element_size() for s, d in out_shapes)
    world = 1 if dist is None else dist.get_world_size()
    # Full-size pinned host copies of every input and output when the host has room
    # for them on every rank; otherwise the same number of bytes moves through 1 GiB
    # pinned staging buffers (the inputs then repeat their first GiB).
    full = psutil.virtual_memory().available > 2 * world * (h2d + d2h)
    chunk = 1 << 30
    host_in, host_out = {}, []
    if full:
        for k in names:
            host_in[k] = torch.empty(t[k].shape, dtype=t[k].dtype, pin_memory=True)
            host_in[k].copy_(t[k])
        host_out = [torch.empty(s, dtype=d, pin_memory=True) for s, d in out_shapes]
    else:
        stage_in = torch.zeros(chunk, dtype=torch.uint8, pin_memory=True)
        stage_out = torch.empty(chunk, dtype=torch.uint8, pin_memory=True)
        first = t["k"].view(torch.uint8).reshape(-1)[:chunk]
        stage_in[:first.numel()].copy_(first)

    def h2d_copy(dst, key):
        if full:
            dst.copy_(host_in[key], non_blocking=True)
            return
        flat = dst.view(torch.uint8).reshape(-1)
        for off in range(0, flat.numel(), chunk):
            n_ = min(chunk, flat.numel() - off)
            flat[off:off + n_].copy_(stage_in[:n_], non_blocking=True)

    def d2h_copy(i, src):
        if full:
            host_out[i].copy_(src, non_blocking=True)
            return
        flat = src.view(torch.uint8).reshape(-1)
        for off in range(0, flat.numel(), chunk):
            n_ = min(chunk, flat.numel() - off)
            stage_out[:n_].copy_(flat[off:off + n_], non_blocking=True)

    rec = Recorder(ba, p)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    steps = max(1, min(args.steps, args.e2e_steps))
    # The cotangent is only needed by the backward and O / LSE are final after the
    # forward: their copies run on side streams behind the forward / the backward.
    main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()     # long-lived objects: made once, outside the steps
    fused = use_fused_bwd(args, p, plan, ba)
    s_ev = torch.cuda.Event(enable_timing=True)
    e_ev = torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    s_ev.record()
    streamed = bool(cp) and backward and full and t.get("_mode", "zigzag") == "zigzag"
    marks = []
    for _ in range(steps if streamed else 0):
        marks = e2e_step_streamed(torch, rec, plan, p, t, cp, fused, host_in, host_out, main, s_in, s_out)
    for _ in range(0 if streamed else steps):
        for k in names:
            if k != "d_o":
                h2d_copy(t[k], k)
        if backward:
            qkv_in = torch.cuda.Event()
            qkv_in.record(main)
            with torch.cuda.stream(s_in):
                s_in.wait_event(qkv_in)           # after Q, K, V: the link is theirs first
                h2d_copy(t["d_o"], "d_o")
                go_in = torch.cuda.Event()
                go_in.record(s_in)
        o, lse = run_fwd(rec, plan, t, cp)
        outs = [o, lse]
        if backward:
            fwd_done = torch.cuda.Event()
            fwd_done.record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(fwd_done)
                d2h_copy(0, o)
                d2h_copy(1, lse)
                o_out = torch.cuda.Event()
                o_out.record(s_out)
            main.wait_event(go_in)
            grads = run_bwd(rec, plan, t, cp, o, lse, fused=fused)
            for i, src in enumerate(x for x in grads[:4] if x is not None):
                d2h_copy(2 + i, src)
            main.wait_event(o_out)
        else:
            d2h_copy(0, o)
            d2h_copy(1, lse)
    e_ev.record()
    torch.cuda.synchronize()
    ms = s_ev.elapsed_time(e_ev)
    value, _ = aggregate_throughput(dist, flops * steps, ms, device)
    timeline = None
    if marks:   # last step: when its phases ended, in ms after the step's start
        timeline = {name: round(marks[0][1].elapsed_time(ev), 1) for name, ev in marks[1:]}
        timeline["step_start_in_timed_region"] = round(s_ev.elapsed_time(marks[0][1]), 1)
    return {"timeline_ms": timeline, "value": round(value, 3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "steps": steps, "ms_per_step": round(ms / steps, 3),
            "host_buffers": "pinned, full size" if full else "pinned 1 GiB staging (host memory too small for full copies)",
            "copies": ("streamed per query chunk: K, V, then the query rows in the order the chunks are used, dO behind "
                       "the forward; O / LSE and each chunk's dQ behind the backward, dK / dV at the end") if streamed
                      else "whole tensors: Q, K, V before the forward, dO behind it; O / LSE behind the backward, gradients after it"}


def e2e_step_streamed(torch, rec, plan, p, t, cp, fused, host_in, host_out, main, s_in, s_out):
    """One end-to-end step of the zigzag workload with the host copies streamed chunk by chunk:
    the forward of a query chunk starts as soon as K, V and that chunk's query rows are on the
    device, and a chunk's dQ leaves for the host as soon as its last backward block is done."""
    from paper_2609_07108_b200 import zigzag
    n = p.n_main
    bounds = zigzag.chunk_bounds(n, cp)
    anchors = np.asarray(p.anchor_idx, dtype=np.int64)
    ws = t["_ws"]

    class Hooks:
        q_events = {}

        @staticmethod
        def q_ready(qc):
            main.wait_event(Hooks.q_events[qc])

        @staticmethod
        def dq_done(qc, qm, tok):
            ev = torch.cuda.Event()
            ev.record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev)
                host_out[2][qm[0]:qm[1]].copy_(ws.outs[0][qm[0]:qm[1]], non_blocking=True)
                host_out[3][tok[0]:tok[1]].copy_(ws.outs[1][tok[0]:tok[1]], non_blocking=True)

    def mark(name, stream=main):
        ev = torch.cuda.Event(enable_timing=True)
        ev.record(stream)
        marks.append((name, ev))
        return ev

    marks = []
    start = mark("start")
    with torch.cuda.stream(s_in):
        s_in.wait_event(start)
        t["k"].copy_(host_in["k"], non_blocking=True)
        t["v"].copy_(host_in["v"], non_blocking=True)
        mark("k_v_on_device", s_in)
        for qc in zigzag.chunk_order(cp):
            q0, q1 = bounds[qc]
            b0 = int(np.searchsorted(anchors, q0, side="left"))
            b1 = int(np.searchsorted(anchors, q1, side="left"))
            t0, t1 = plan.token_range(b0, b1)
            t["q_main"][q0:q1].copy_(host_in["q_main"][q0:q1], non_blocking=True)
            t["q_branch"][t0:t1].copy_(host_in["q_branch"][t0:t1], non_blocking=True)
            ev = torch.cuda.Event()
            ev.record(s_in)
            Hooks.q_events[qc] = ev
        mark("queries_on_device", s_in)
        t["d_o"].copy_(host_in["d_o"], non_blocking=True)
        go_in = mark("cotangent_on_device", s_in)
    o, lse, _ = zigzag.forward(rec, plan, t["q_main"], t["q_branch"], t["k"], t["v"], cp, out=t.get("_o"),
                               lse=t.get("_lse"), ws=ws, hooks=Hooks)
    fwd_done = mark("forward_done")
    with torch.cuda.stream(s_out):
        s_out.wait_event(fwd_done)
        host_out[0].copy_(o, non_blocking=True)
        host_out[1].copy_(lse, non_blocking=True)
        mark("o_lse_on_host", s_out)
    main.wait_event(go_in)
    grads = zigzag.backward(rec, plan, t["q_main"], t["q_branch"], t["k"], t["v"], o, lse, t["d_o"], cp, fused=fused,
                            ws=ws, hooks=Hooks)
    done = mark("backward_done")
    with torch.cuda.stream(s_out):
        s_out.wait_event(done)
        mark("dq_on_host", s_out)
        host_out[4].copy_(grads[2], non_blocking=True)
        host_out[5].copy_(grads[3], non_blocking=True)
    main.wait_stream(s_out)
    mark("gradients_on_host")
    return marks


# ----------------------------------------------------------------------------
# CPU baseline = the oracle, as it stands, on a bounded sample
# ----------------------------------------------------------------------------

def query_rows_streamed(p, cp, kind):
    """Query rows one step's launches of `kind` stream in total (a row counts once per launch
    that walks it): every row once for a monolithic call, once per (q chunk, kv chunk) block of
    the emulated ring."""
    if not cp:
        return p.rows
    from paper_2609_07108_b200 import zigzag
    total = 0
    offs = p.branch_offsets.astype(np.int64)
    for b in zigzag.schedule(p, cp):
        total += (b.qm[1] - b.qm[0]) + int(offs[b.br[1]] - offs[b.br[0]])
    return total


def oracle_sample(p, n_rows, seed=0, gpu_inputs=None):
    """Rows sampled uniformly from the workload (main and branch rows), one KV
    group (h_q/h_kv query heads).  Returns the inputs and the sampled rows.  With
    `gpu_inputs` (the benchmark's device tensors) the values are those the GPU ran
    on, so that the oracle's results can be compared with the GPU's."""
    import copy
    rng = np.random.default_rng(seed)
    rows = np.sort(rng.choice(p.rows, size=min(n_rows, p.rows), replace=False)).astype(np.int64)
    p1 = copy.copy(p)
    p1.h_q, p1.h_kv = p.h_q // p.h_kv, 1
    d = p.head_dim
    if gpu_inputs is not None:
        import torch
        t = gpu_inputs
        n, g = p.n_main, p1.h_q
        dev = t["k"].device
        is_b = rows >= n
        q = np.empty((len(rows), g, d), dtype=np.float32)
        if (~is_b).any():
            q[~is_b] = t["q_main"][torch.from_numpy(rows[~is_b]).to(dev)][:, :g].float().cpu().numpy()
        if is_b.any():
            q[is_b] = t["q_branch"][torch.from_numpy(rows[is_b] - n).to(dev)][:, :g].float().cpu().numpy()
        k = t["k"][:, :1].float().cpu().numpy()
        v = t["v"][:, :1].float().cpu().numpy()
        go = t["d_o"][torch.from_numpy(rows).to(dev)][:, :g].float().cpu().numpy()
        return p1, rows, q, k, v, go
    q = W.round_to_bf16(rng.standard_normal((len(rows), p1.h_q, d), dtype=np.float32) * 0.5)
    k = W.round_to_bf16(rng.standard_normal((p.rows, 1, d), dtype=np.float32) * 0.5)
    v = W.round_to_bf16(rng.standard_normal((p.rows, 1, d), dtype=np.float32) * 0.5)
    go = W.round_to_bf16(rng.standard_normal((len(rows), p1.h_q, d), dtype=np.float32) * 0.1)
    return p1, rows, q, k, v, go


def sample_pairs(oracle, p1, rows):
    cu = p1.cu_seqlens.astype(np.int64)
    n = p1.n_main
    anchors = p1.anchor_idx.astype(np.int64)
    offs = p1.branch_offsets.astype(np.int64)
    loc = W.branch_local_counts(p1) if p1.n_branch and p1.n_branch <= 1 << 16 else None
    total = 0
    for r in rows:
        if r < n:
            s = np.searchsorted(cu, r, side="right") - 1
            total += r - cu[s] + 1
        else:
            tkn = r - n
            b = np.searchsorted(offs, tkn, side="right") - 1
            a = anchors[b]
            s = np.searchsorted(cu, a, side="right") - 1
            total += a - cu[s] + 1
            if loc is not None:
                total += loc[tkn]
            elif p1.kind == W.CHAIN:
                total += tkn - offs[b] + 1
            else:
                total += offs[b + 1] - offs[b]
    return int(total)


def time_oracle(p, n_rows, backward=True, gpu_inputs=None, keep=False):
    from oracle import oracle
    oracle.build()
    p1, rows, q, k, v, go = oracle_sample(p, n_rows, gpu_inputs=gpu_inputs)
    pairs = sample_pairs(oracle, p1, rows)
    t0 = time.perf_counter()
    res = {}
    if backward:
        res["dq"] = oracle.backward(p1, q, k, v, go, rows=rows)[0]       # runs the forward inside
    else:
        res["o"], res["lse"] = oracle.forward(p1, q, k, v, rows=rows)
    dt = time.perf_counter() - t0
    if keep and backward:                                                # untimed: O and LSE for the comparison
        res["o"], res["lse"] = oracle.forward(p1, q, k, v, rows=rows)
    fl = pairs * 4 * p.head_dim * p1.h_q * (3.5 if backward else 1.0)
    return fl / dt / 1e12, dt, len(rows), pairs, p1.h_q, (rows, res) if keep else None


def sized_rows(p, seconds_target, backward):
    """Sample size whose oracle run takes about `seconds_target` (found by doubling)."""
    n_rows, dt = 8, 0.0
    while n_rows < p.rows:
        _, dt, _, _, _, _ = time_oracle(p, n_rows, backward)
        if dt >= seconds_target / 4:
            break
        n_rows *= 4
    return int(max(8, min(p.rows, n_rows * seconds_target / max(dt, 1e-3))))


def gpu_vs_oracle(p, rows, res, gpu):
    """max abs and rel-RMS error of the GPU's O, LSE and dQ of the last timed step against the
    oracle on the CPU-baseline sample rows (first KV group)."""
    import torch
    t, last = gpu
    o, lse, grads = last
    g = p.h_q // p.h_kv
    n = p.n_main
    dev = o.device
    rows_t = torch.from_numpy(rows).to(dev)

    def metrics(got, want):
        err = got.astype(np.float64) - want
        den = float(np.sqrt(np.mean(want * want)))
        return {"max_abs": float(f"{np.abs(err).max():.3e}"),
                "rel_rms": float(f"{np.sqrt(np.mean(err * err)) / den:.3e}") if den > 0 else None}

    out = {"rows": int(len(rows)), "heads": g}
    out["O"] = metrics(o[rows_t][:, :g].float().cpu().numpy(), res["o"])
    out["LSE"] = metrics(lse[rows_t][:, :g].float().cpu().numpy(), res["lse"])
    if grads is not None and "dq" in res:
        is_b = rows >= n
        dq = np.empty((len(rows), g, p.head_dim), dtype=np.float32)
        if (~is_b).any():
            dq[~is_b] = grads[0][torch.from_numpy(rows[~is_b]).to(dev)][:, :g].float().cpu().numpy()
        if is_b.any():
            dq[is_b] = grads[1][torch.from_numpy(rows[is_b] - n).to(dev)][:, :g].float().cpu().numpy()
        out["dQ"] = metrics(dq, res["dq"])
    return out


def cpu_baseline(p, seconds_target=15.0, backward=True, gpu=None):
    cores = len(os.sched_getaffinity(0))
    n_rows = sized_rows(p, seconds_target, backward)
    val, dt, nr, pairs, hq, kept = time_oracle(p, n_rows, backward, gpu_inputs=gpu[0] if gpu else None,
                                               keep=gpu is not None)
    out = {"value": float(f"{val:.6g}"), "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": f"{nr} uniformly sampled query rows x {hq} query heads of one KV group, "
                     f"fwd{'+bwd' if backward else ''}, {pairs} visible pairs per head, {dt:.1f} s"}
    if kept is not None:
        out["gpu_vs_oracle"] = gpu_vs_oracle(p, kept[0], kept[1], gpu)
    return out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    name = "config5_256k_zigzag" if args.workload == "auto" else args.workload
    cfg, shrink, cp, backward = WORKLOADS[name]
    p = W.CONFIGS[cfg](shrink)
    cores = len(os.sched_getaffinity(0))
    n_rows = sized_rows(p, args.ref_seconds, backward)
    for _ in range(args.warmup):
        time_oracle(p, 8, backward)
    vals, secs = [], []
    for _ in range(args.steps):
        val, dt, nr, pairs, hq, _ = time_oracle(p, n_rows, backward)
        vals.append(val)
        secs.append(dt)
    value = sum(vals) / len(vals)
    sample = (f"{nr} uniformly sampled query rows x {hq} query heads of one KV group per step, "
              f"fwd{'+bwd' if backward else ''}, {pairs} visible pairs per head")
    line = {"impl": "reference", "metric": METRIC, "value": float(f"{value:.6g}"), "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(1e3 * sum(secs) / len(secs), 1), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": name, "n_main": p.n_main, "rows": p.rows, "h_q": p.h_q, "h_kv": p.h_kv,
                       "head_dim": p.head_dim, "mask": W.KIND_NAMES[p.kind]},
            "cpu_baseline": {"value": float(f"{value:.6g}"), "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": float(f"{value:.6g}"), "unit": UNIT, "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="auto", choices=["auto", *WORKLOADS])
    ap.add_argument("--kernels", default="auto", choices=["auto", "simt", "tc"])
    ap.add_argument("--bwd", default="auto", choices=["auto", "split", "fused"],
                    help="backward: dQ kernel + dK/dV kernel, or one kernel for all three (dQ summed with "
                         "atomic adds); auto = the one-kernel form from 131,072 tokens up (runs of seconds "
                         "at the power cap, decided by the work done), the two-kernel form below")
    ap.add_argument("--branch-only", action="store_true",
                    help="q_main = NULL: only the branch tokens are queries (monolithic workloads)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=1)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--ref-seconds", type=float, default=8.0)
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
