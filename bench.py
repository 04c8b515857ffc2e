#!/usr/bin/env python
"""Benchmark of the sharded weight update (one JSON line on stdout).

A step is one pass of the whole hot path over one model-shaped set of synthetic
tensors: the R replicas' gradients are reduced shard by shard, the optimizer
updates every 1/R slice of weights and slots, and the updated weights arrive in
the weight tensors.  `value` is updated (valid) parameters per second with
everything resident in HBM; `e2e` is the same step through the host-buffer
entry point with host<->device copies inside the timed region; `roofline` is
the dominant kernel's algorithmic bytes over its measured time against the
measured HBM copy bandwidth; `cpu_baseline` is the CPU oracle timed on this
box's host cores.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Without --workload the line is the largest single-GPU workload (decoder_1p5b:
1.56 G parameters, bf16 gradients, R = 4) and carries, under `configs`, one full
record for each of the other named workloads, under `transformer_r_sweep` the
Transformer set at R = 1 ... 1024 and alignments 8 and 32, and under
`next_workloads` the LARS, Adafactor, concatenated-layout and partial-sharding runs.

Whatever K is, the timed region lasts at least half a second: it covers
K x `inner_repeats` back-to-back steps and `ms_per_step` is their mean.

With N > 1 (launched by torch.distributed.run) every rank runs the same
workload on its own independently seeded tensor set: the update has no
data-path collective, so ranks only meet at the timing barriers.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "updated_params_per_sec"
UNIT = "params/s"
FALLBACK_HBM_GBS = 6650.0
HEADLINE = "decoder_1p5b"
MIN_TIMED_S = 0.5

# DRAM bytes per valid parameter (dram__bytes_read.sum + dram__bytes_write.sum of the update's launches
# ÷ parameters) from the ncu captures summarised under profiles/.  Workloads too large for a multi-pass
# capture were captured on a smaller copy (every dimension clipped, or a few layers at full size) and are
# scaled here by the parameter count: the kernels' traffic is proportional to the elements they process.
# Keyed by (workload, R, path): (bytes per parameter, which capture).
NCU_DRAM_BYTES_PER_PARAM = {
    ("resnet50", 8, "fused"): (47.06, "profiles/fused_update_kernel_resnet50_sgdm_R8.md (full size)"),
    ("decoder_1p5b", 4, "fused"): (33.73, "profiles/fused_update_kernel_decoder_bf16_R4.md (dimensions clipped to 1024)"),
    ("transformer", 8, "fused"): (55.70, "profiles/fused_update_kernel_transformer_adam.md (dimensions clipped to 1024)"),
    ("transformer", 1, "fused"): (27.46, "profiles/fused_update_kernel_transformer_adam.md (dimensions clipped to 1024)"),
    ("bert_large", 16, "fused"): (88.9, "profiles/lamb_one_kernel_bert_large_R16.md (six layers at full size: 88.2; the "
                                        "embeddings, a tenth of the parameters, captured by themselves: 96.0; weighted by "
                                        "parameters)"),
    ("resnet50_lars", 8, "fused"): (56.5, "profiles/fused_lars_kernels_resnet50_R8.md (full size, no cache flush between the launches)"),
    ("transformer_adafactor", 8, "fused"): (55.5, "profiles/fused_adafactor_kernels_transformer.md (dimensions clipped to 1024)"),
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="all",
                    choices=["all", "tiny", "resnet50", "transformer", "bert_large", "decoder_1p5b", "resnet50_lars",
                             "transformer_adafactor"],
                    help="all (default): headline decoder_1p5b plus one record per other workload and the sweeps")
    ap.add_argument("--R", type=int, default=0, help="override the workload's replica count")
    ap.add_argument("--opt", default="", choices=["", "sgdm", "adam", "lamb", "lars", "adafactor"],
                    help="override the workload's optimizer (profiling of small cases)")
    ap.add_argument("--grad-dtype", default="", choices=["", "f32", "bf16"], help="override the gradient dtype")
    ap.add_argument("--out-dtype", default="", choices=["", "f32", "bf16"], help="override the emitted weight dtype")
    ap.add_argument("--clip", type=int, default=0,
                    help="clip every tensor dimension to this size (a small copy of the workload for profiler captures)")
    ap.add_argument("--tensors", default="",
                    help="A:B - keep only tensors A..B-1 of the workload's list (a few layers at full size, for profiler captures)")
    ap.add_argument("--shards", type=int, default=0,
                    help="shard count of the plan when it differs from the replica count (partial sharding)")
    ap.add_argument("--layout", default="per_tensor", choices=["per_tensor", "concat"],
                    help="per_tensor: one piece of every tensor per shard; concat: the concatenation cut into R shards")
    ap.add_argument("--align", type=int, default=32)
    ap.add_argument("--tile", type=int, default=0, help="work-tile elements (0 = library default)")
    ap.add_argument("--path", default="both", choices=["both", "fused", "unfused"],
                    help="fused: one kernel reads the gradient tensors and writes the weight tensors; "
                         "unfused: pack, update, unpack as separate kernels; both: time both, headline = fused")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--min-timed-s", type=float, default=MIN_TIMED_S,
                    help="shortest timed region; steps are repeated back to back to reach it")
    ap.add_argument("--route", default="replicas", choices=["replicas", "nccl", "peer"],
                    help="replicas (default): every rank updates its own independent tensor set, no collective; "
                         "nccl: ONE model over the ranks, NCCL reduce-scatter / all-gather around the single-shard "
                         "kernels; peer: ONE model, one kernel per rank over symmetric-memory tensors")
    ap.add_argument("--three-launch", action="store_true",
                    help="LAMB as three launches (phase 1, combination, phase 2) instead of the one kernel")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-side-rows", action="store_true",
                    help="with --workload all: only the headline record, none of the other workloads or sweeps")
    return ap.parse_args()


def get_workload(name, R=0, opt="", grad_dtype="", out_dtype="", clip=0, tensors=""):
    from paper_2004_13336_b200 import workloads as W
    wl = W.WORKLOADS[name]()
    if R:
        wl.R = R
    if opt or grad_dtype or out_dtype:
        import torch
        dt = {"f32": torch.float32, "bf16": torch.bfloat16}
        if opt and opt != wl.opt:
            wl.opt = opt
            wl.hyper = dict(W.WORKLOADS[{"sgdm": "resnet50", "adam": "transformer", "lamb": "bert_large",
                                         "lars": "resnet50_lars", "adafactor": "transformer_adafactor"}[opt]]().hyper)
        if grad_dtype:
            wl.grad_dtype = dt[grad_dtype]
        if out_dtype:
            wl.out_dtype = dt[out_dtype]
        wl.name += "*"          # not one of the named workloads any more
    if clip:
        wl = W.scaled_down(wl, clip)
    if tensors:
        a, b = (int(x) for x in tensors.split(":"))
        wl.shapes = wl.shapes[a:b]
        wl.name += f"[{a}:{b}]"
    return wl


def workload_from_args(args):
    name = HEADLINE if args.workload == "all" else args.workload
    return get_workload(name, args.R, args.opt, args.grad_dtype, args.out_dtype, args.clip, args.tensors)


def measured_peak():
    """(GB/s, source): the measured device copy bandwidth of this machine, else the stated fallback."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def bytes_per_param(wl):
    """Bytes per valid parameter.

    `algorithmic`: what the method must move, every operand once (Section 2.2: read the gradient
    copies, the weight and the auxiliaries; write the weight and the auxiliaries): SGD-momentum
    g R + 16, Adam g R + 24 (+2 for a bf16 copy next to the fp32 master), LAMB g R + 24 (its phase 2
    re-reads are not algorithmic), LARS g R + 16, Adafactor g R + 8, with g = gradient element bytes.
    `update` / `fused`: what the separate-kernel update and the fused-formatting update move by design.
    `pack` / `unpack`: one formatting launch."""
    gb = 2 if str(wl.grad_dtype).endswith("bfloat16") else 4
    slots = {"sgdm": 1, "lars": 1, "adafactor": 0}.get(wl.opt, 2)
    out_b = 2 if str(wl.out_dtype).endswith("bfloat16") else 0
    alg = gb * wl.R + 4 * (1 + slots) * 2 + out_b
    upd = alg
    if wl.opt == "lamb":
        upd += 12          # two passes: phase 2 reads w, m', v' again
    if wl.opt == "lars":
        upd += 12          # phase 1 reads w and stores the summed gradient; phase 2 reads it back
    if wl.opt == "adafactor":
        upd += 16          # pass 1 stores the summed gradient, passes 2 and 3 read it back, pass 3 reads w again
    # fused formatting: same reads and state writes; fp32 weight tensors are the master copy themselves
    # (read and written in place, no sharded w), a bf16 weight list is the copy counted in `alg`
    fused = upd
    return {"algorithmic": alg, "update": upd, "fused": fused, "pack": 2 * gb, "unpack": 2 * (2 if out_b else 4)}


# ----------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.samples = []
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                pass

    def summary(self, t0, t1):
        def parse(window):
            sm, mx, reasons = [], [], set()
            for ts, line in list(self.samples):
                if not (window[0] <= ts <= window[1]):
                    continue
                p = [x.strip() for x in line.split(",")]
                if len(p) < 7:
                    continue
                try:
                    sm.append(float(p[0]))
                    mx.append(float(p[1]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[3:7]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            return sm, mx, reasons
        sm, mx, reasons = parse((t0, t1))
        window = "timed"
        if len(sm) < 3 and self.samples:
            sm, mx, reasons = parse((t0 - 1.0, t1 + 1.0))
            window = "timed +-1 s"
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "window": window}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "window": window}


# ----------------------------------------------------------------------------
# CPU oracle legs
# ----------------------------------------------------------------------------
def sample_stride(n_total, target):
    """Stride of the bounded tensor sample: about n_total / target, rounded up to a prime so that it does
    not fall in step with the period of a layer's tensor list (16 tensors per BERT layer)."""
    k = max(1, round(n_total / target))
    while k > 2 and any(k % d == 0 for d in range(2, int(k ** 0.5) + 1)):
        k += 1
    return k


def oracle_step_inputs(wl, stride, align):
    """Host copies of every `stride`-th tensor of the workload (the bounded sample), starting in the
    middle of the first stride so that the sample is not dominated by the embedding at index 0."""
    import torch
    from oracle import ws_oracle as O
    from paper_2004_13336_b200 import workloads as W
    idx = list(range(stride // 2 if stride < wl.T else 0, wl.T, stride))
    sub = W.Workload(**{**wl.__dict__})
    sub.shapes = [wl.shapes[i] for i in idx]
    w, m, v = W.make_state(sub, "cpu")
    g = W.make_grads(sub, "cpu")

    def np_(t):
        if t.dtype == torch.bfloat16:
            import numpy as np
            return t.view(torch.int16).numpy().view(np.uint16)
        return t.numpy()
    plan = O.Plan(sub.numels, sub.R, align)
    w, m, v = ([np_(x) for x in lst] for lst in (w, m, v))
    g = [[np_(x) for x in gk] for gk in g]
    pw, pm, pv = O.pack(plan, w), O.pack(plan, m), O.pack(plan, v)
    if sub.opt == "adafactor":      # no momentum; the second slot is the factored state
        pm, pv = None, W.make_factored_state(sub, O.factor_shapes(sub.shapes)[3], "cpu").numpy()
    return sub, plan, g, pw, pm, pv


def oracle_one_step(sub, plan, g, pw, pm, pv):
    """The whole path as the oracle states it: pack R gradient sets, sharded update, unpack."""
    from oracle import ws_oracle as O
    hs = O.make_hyper(sub.opt, sub.hyper)
    t0 = time.perf_counter()
    pg = [O.pack(plan, gk) for gk in g]
    out_dt = O.BF16 if str(sub.out_dtype).endswith("bfloat16") else None
    if sub.opt == "adafactor":
        gathered, _ = O.adafactor_sharded(hs, plan, sub.shapes, pg, pw, pv, out_dt)
    else:
        gathered, _, _ = O.sharded_update(hs, plan, pg, pw, pm, pv if sub.opt in ("adam", "lamb") else None, out_dt)
    O.unpack(plan, gathered if gathered is not None else pw)
    return time.perf_counter() - t0


def cpu_baseline(wl, align, target_params=0, min_seconds=10.0, max_steps=20):
    """The oracle's sharded route, as it stands, on this machine's host cores: once on one thread and once
    on all of them (the loops over independent (shard, tensor) pairs are split; results do not depend on
    the thread count).  `value` is the all-core rate."""
    from oracle import ws_oracle as O
    target_params = target_params or int(2e8 / (wl.R + 3))      # bounds the sample's host memory and set-up time
    stride = sample_stride(wl.N, target_params)
    sub, plan, g, pw, pm, pv = oracle_step_inputs(wl, stride, align)
    host_cores = len(os.sched_getaffinity(0))
    runs = {}
    for label, nthreads, secs in (("single_thread", 1, min_seconds * 0.6), ("all_cores", host_cores, min_seconds * 0.4)):
        prev = O.set_num_threads(nthreads)
        try:
            used = O.num_threads()
            oracle_one_step(sub, plan, g, pw, pm, pv)        # first touch
            dt, steps = 0.0, 0
            while steps < max_steps and (steps == 0 or dt < secs):
                dt += oracle_one_step(sub, plan, g, pw, pm, pv)
                steps += 1
        finally:
            O.set_num_threads(prev)
        runs[label] = {"value": sub.N * steps / dt, "unit": UNIT, "cores": used, "steps": steps, "seconds": round(dt, 2)}
    return {"value": runs["all_cores"]["value"], "unit": UNIT, "cores": runs["all_cores"]["cores"], "kind": "oracle",
            "sample": f"whole path (pack {sub.R} gradient sets, sharded update, unpack) over every {stride}-th tensor of "
                      f"{wl.name}: {sub.T} tensors, {sub.N} params, {runs['all_cores']['steps']} step(s) in "
                      f"{runs['all_cores']['seconds']} s on {runs['all_cores']['cores']} threads",
            "single_thread": runs["single_thread"], "host_cores": host_cores}


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on this machine's host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import ws_oracle as O
    O.build()
    wl = workload_from_args(args)
    stride = sample_stride(wl.N, 6_000_000)
    sub, plan, g, pw, pm, pv = oracle_step_inputs(wl, stride, args.align)
    cores = O.num_threads()
    for _ in range(max(1, args.warmup)):
        oracle_one_step(sub, plan, g, pw, pm, pv)
    t = 0.0
    for _ in range(args.steps):
        t += oracle_one_step(sub, plan, g, pw, pm, pv)
    val = sub.N * args.steps / t
    sample = (f"each step = whole path over every {stride}-th tensor of {wl.name} "
              f"({sub.T} tensors, {sub.N} params) on {cores} threads")
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": config_of(wl, args.align, args.layout, wl.R, extra={"sample": sample}),
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def config_of(wl, align, layout, shards, extra=None, path="fused"):
    steps = {"unfused": "pack R gradient sets + fused reduce/update of all shards + unpack weights (separate kernels)",
             "fused": "one kernel: gradients read from the R replicas' tensor lists (formatting fused in), reduce, "
                      "update of all shards, weights written to the weight tensors (fp32 weights: read from and "
                      "written to the tensors, which are the master copy)"}
    c = {"workload": f"{wl.name}: {wl.T} tensors, {wl.N} params, R={wl.R} replicas, {wl.opt}, "
                     f"grads {str(wl.grad_dtype).split('.')[-1]}, gathered {str(wl.out_dtype).split('.')[-1]}",
         "R": wl.R, "shards": shards or wl.R, "optimizer": wl.opt, "align_elems": align, "layout": layout,
         "step": steps[path],
         "l2": "inputs exceed L2 (no flush)" if wl.N * 4 * (wl.R + 3) > 256e6 else "flush between steps"}
    if extra:
        c.update(extra)
    return c


# ----------------------------------------------------------------------------
# multi-rank plumbing (one process per GPU; no data-path collective)
# ----------------------------------------------------------------------------
def rank_seed(base_seed: int, rank: int) -> int:
    """Each rank updates its own, independently seeded tensor set of the same workload."""
    return base_seed + 1000 * rank


def reduce_max(x: float, device) -> float:
    """Max over ranks of a per-rank time (the job is as slow as its slowest rank)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(n_params_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput: every rank updates n parameters per step (weak scaling)."""
    return world * n_params_per_rank / (ms_per_step * 1e-3)


def inner_repeats(est_ms_per_step: float, steps: int, min_timed_s: float) -> int:
    """Back-to-back repetitions of every counted step so that the timed region lasts at least
    `min_timed_s` whatever `steps` is."""
    if est_ms_per_step <= 0:
        return 1
    return max(1, min(20000, math.ceil(min_timed_s * 1e3 / (steps * est_ms_per_step))))


# ----------------------------------------------------------------------------
# GPU arm
# ----------------------------------------------------------------------------
def run_real_replicas(args):
    """--route nccl | peer: the ranks are the replicas of ONE model (shard count = number of ranks).
    Each step is the whole weight update of the model: with nccl, pack + reduce-scatter + update of the
    rank's shard + all-gather + unpack; with peer, one kernel per rank over symmetric-memory tensors
    between two stream-ordered barriers.  The work per step is fixed (N parameters), so scaling is strong."""
    import socket
    import torch
    import torch.distributed as dist
    from paper_2004_13336_b200 import build as ws_build
    from paper_2004_13336_b200 import workloads as W
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    else:
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1, device_id=dev)
    if rank == 0 and not ws_build.up_to_date():
        ws_build.build()
    dist.barrier()
    from paper_2004_13336_b200.collective import PeerShardedUpdate, ShardedUpdate
    wl = workload_from_args(args)
    wl.R = world
    w, m, v = W.make_state(wl, dev)                       # same seed on every rank: one model
    g = W.make_grads_one(wl, rank, dev)                   # this replica's own gradients
    kw = dict(out_dtype=wl.out_dtype, grad_dtype=wl.grad_dtype, align_elems=args.align, device=dev)
    if args.route == "nccl":
        su = ShardedUpdate(wl.shapes, wl.opt, wl.hyper, **kw)
        su.load_state(w, m, v)
        outs = [torch.empty(n, dtype=wl.out_dtype, device=dev) for n in wl.numels]
        step = lambda: su.step(g, outs)
        launches = {"sgdm": 3, "adam": 3, "lamb": 5, "lars": 5, "adafactor": 8}[wl.opt]   # ours: pack, update phases, unpack
    else:
        su = PeerShardedUpdate(wl.shapes, wl.opt, wl.hyper, **kw)
        su.load_state(w, m, v)
        for dst, src in zip(su.grads, g):
            dst.copy_(src)
        step = su.step
        launches = 1
    K, W_ = args.steps, max(3, args.warmup)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for _ in range(W_):
        step()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dist.barrier()
    torch.cuda.synchronize()
    t0 = time.time()
    e0.record()
    for _ in range(K):
        step()
    e1.record()
    dist.barrier()
    torch.cuda.synchronize()
    t1 = time.time()
    ms = reduce_max(e0.elapsed_time(e1), dev) / K
    sampler.stop()
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": wl.N / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W_,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": f"{wl.name}: one model of {wl.N} params over {world} replica(s), {wl.opt}",
                       "route": args.route, "inputs": "larger than L2" if wl.N * 12 > 256e6 else "fit in L2"},
            "roofline": None, "clocks": sampler.summary(t0, t1), "gpu_launches": K * launches}))
    dist.destroy_process_group()


class Ctx:
    """What every measurement of a process shares: ranks, device, the clock sampler."""

    def __init__(self, args):
        import torch
        import torch.distributed as dist
        self.args = args
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the sharded update has no CPU fallback")
        torch.cuda.set_device(self.local)
        self.dev = torch.device("cuda", self.local)
        if self.world > 1:
            dist.init_process_group("nccl", device_id=self.dev)
        from paper_2004_13336_b200 import build as ws_build
        if self.rank == 0 and not ws_build.up_to_date():
            ws_build.build()                      # one rank builds; the others wait at the barrier
        if self.world > 1:
            dist.barrier()
        from paper_2004_13336_b200 import binding as B
        B.lib()
        self.sampler = ClockSampler(self.local)
        if self.rank == 0:
            self.sampler.start()

    def barrier(self):
        import torch
        import torch.distributed as dist
        if self.world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def close(self):
        import torch.distributed as dist
        self.sampler.stop()
        if self.world > 1:
            dist.destroy_process_group()


def copy_floor(torch, dev, nbytes):
    """What a plain device-to-device copy that moves `nbytes` (half read, half written) achieves when it is
    timed like a short kernel here: back to back over rotating buffer pairs larger than L2 together, and
    alone on a drained GPU.  A launch of tens of microseconds cannot beat this by much: it is the ramp and
    tail of any grid, not the kernel's code, that separates it from the copy bandwidth of a long launch."""
    n = max(nbytes // 8, 1)
    pairs = max(1, min(8, int(512e6 // max(nbytes, 1)) + 1))
    try:
        bufs = [(torch.empty(n, dtype=torch.float32, device=dev), torch.empty(n, dtype=torch.float32, device=dev))
                for _ in range(pairs)]
    except RuntimeError:
        return None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for a, b in bufs:
        b.copy_(a)
    torch.cuda.synchronize()
    reps = max(2, min(40, int(4e-3 / (nbytes / 6.5e12)) // pairs + 1))
    e0.record()
    for _ in range(reps):
        for a, b in bufs:
            b.copy_(a)
    e1.record()
    torch.cuda.synchronize()
    b2b = e0.elapsed_time(e1) / (reps * pairs)
    iso = []
    for i in range(15):
        a, b = bufs[i % pairs]
        e0.record()
        b.copy_(a)
        e1.record()
        torch.cuda.synchronize()
        iso.append(e0.elapsed_time(e1))
    iso.sort()
    pk = measured_peak()[0]
    return {"what": "cudaMemcpyAsync device to device moving the same bytes, timed the same two ways",
            "bytes": nbytes, "ms_back_to_back": b2b, "frac_back_to_back": nbytes / (b2b * 1e-3) / 1e9 / pk,
            "ms_isolated_median": iso[len(iso) // 2],
            "frac_isolated": nbytes / (iso[len(iso) // 2] * 1e-3) / 1e9 / pk}


def measure(ctx, wl, align=32, layout="per_tensor", shards=0, tile=0, path="both", e2e=True, cpu=True,
            steps=20, warmup=5, e2e_steps=3, cpu_seconds=10.0):
    """One workload on this rank's GPU: the fused route (and the separate-kernel route), the roofline of
    the dominant kernel, the end-to-end step from host buffers and the CPU oracle beside it.  Returns the
    record (rank 0) or None."""
    import torch
    from paper_2004_13336_b200 import binding as B
    from paper_2004_13336_b200 import workloads as W
    args, dev, world, rank = ctx.args, ctx.dev, ctx.world, ctx.rank
    wl.seed = rank_seed(wl.seed, rank)        # every rank owns its own tensor set
    R, T, N = wl.R, wl.T, wl.N
    # partial sharding (Section 5.2): R gradient copies, but the update is sharded only `shards` ways
    shards = shards or R
    plan = B.Plan(wl.shapes, shards, align, tile, device=dev, layout=layout, one_launch=not args.three_launch)
    if shards != R:
        e2e = False               # the host-buffer entry point takes one gradient arena per shard
    gdt, odt = wl.grad_dtype, wl.out_dtype
    gb = 2 if gdt == torch.bfloat16 else 4
    wb = 2 if odt == torch.bfloat16 else 4
    numels = wl.numels
    A_el = plan.arena_elems
    total_mem = torch.cuda.get_device_properties(dev).total_memory
    run_unfused = path in ("both", "unfused")
    run_fused = path in ("both", "fused")
    need_unfused = R * (A_el + plan.G) * gb + 3 * plan.G * 4 + plan.G * wb + A_el * wb
    if R * A_el * gb + 3 * plan.G * 4 > 0.85 * total_mem:
        # not even the R gradient lists fit on one GPU (Transformer at R = 1024 needs 863 GB)
        return run_shard_window(ctx, wl, plan, align, layout, steps, warmup)
    unfused_skipped = None
    if run_unfused and need_unfused > 0.85 * total_mem:
        unfused_skipped = f"needs {need_unfused / 1e9:.0f} GB of device memory (tensor lists plus packed gradient buffers)"
        run_unfused = False
        run_fused = True
    if e2e and need_unfused > 0.85 * total_mem:
        e2e = False

    # ---- device-resident inputs: per replica one gradient arena, viewed tensor by tensor
    w, m, v = W.make_state(wl, dev)
    pw = torch.empty(plan.G, device=dev)
    pm, pv = torch.empty_like(pw), torch.empty_like(pw)
    for src, dst in ((w, pw), (m, pm), (v, pv)):
        B.ws_pack(plan, src, dst)
    if wl.opt in ("sgdm", "lars"):
        pv = None
    if wl.opt == "adafactor":
        pm, pv = None, W.make_factored_state(wl, plan.factored_elems, dev)
    w_arena = torch.zeros(A_el, dtype=odt, device=dev)
    w_views = B.PtrList(plan.arena_views(w_arena, numels))
    # fp32 weights: on the fused route the weight tensors are the master copy (no sharded w is passed)
    master = odt == torch.float32
    if master:
        for dst, src in zip(w_views, w):
            dst.copy_(src)
    del w, m, v
    g_arena = [torch.zeros(A_el, dtype=gdt, device=dev) for _ in range(R)]
    g_views = [B.PtrList(plan.arena_views(a, numels)) for a in g_arena]
    for k in range(R):
        gk = W.make_grads_one(wl, k, dev)
        for dst, src in zip(g_views[k], gk):
            dst.copy_(src)
        del gk
    ws = torch.empty(max(32, plan.workspace_bytes(wl.opt)), dtype=torch.uint8, device=dev)
    hy = B.make_hyper(wl.opt, wl.hyper)
    pg = gathered = None
    if run_unfused or e2e:
        pg = B.PtrList([torch.empty(plan.G, dtype=gdt, device=dev) for _ in range(R)])
        gathered = torch.empty(plan.G, dtype=odt, device=dev) if odt != torch.float32 else None
    gtab = wtab = gtab_u = None
    if run_unfused:
        gtab_u = B.TensorTable(plan, [gv.tensors for gv in g_views])
    if run_fused:
        gtab = B.TensorTable(plan, [gv.tensors for gv in g_views])
        wtab = B.TensorTable(plan, [w_views.tensors])
    flush = None
    if N * 4 * (R + 3) <= 256e6:
        flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)

    def step_unfused(ev=None):
        if flush is not None:
            flush.zero_()
        if ev:
            ev[0].record()
        B.ws_pack_sets(plan, gtab_u, pg)          # the R gradient lists in one launch
        if ev:
            ev[1].record()
        B.ws_shard_update(plan, -1, pg, pw, pm, pv, hy, gathered, ws)
        if ev:
            ev[2].record()
        B.ws_unpack(plan, gathered if gathered is not None else pw, w_views)
        if ev:
            ev[3].record()

    def step_fused(ev=None):
        if flush is not None:
            flush.zero_()
        if ev:
            ev[0].record()
        B.ws_fused_update(plan, -1, gtab, None if master else pw, pm, pv, hy, wtab, ws)
        if ev:
            ev[1].record()

    K = steps
    W_ = max(3, warmup)

    def time_path(step, nev):
        for _ in range(W_):
            step()
        # a first estimate fixes how often every counted step is repeated (same on every rank)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(nev)]
        ctx.barrier()
        est = []
        for _ in range(3):
            step(ev)
            torch.cuda.synchronize()
            est.append(ev[0].elapsed_time(ev[nev - 1]))
        inner = inner_repeats(reduce_max(min(est), dev), K, args.min_timed_s)
        n = K * inner
        if flush is None:
            # the timed region: n steps back to back between two events, nothing else on the stream
            e_start, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ctx.barrier()
            t0 = time.time()
            e_start.record()
            for i in range(n):
                step()
            e_end.record()
            ctx.barrier()
            t1 = time.time()
            total_ms = e_start.elapsed_time(e_end)
            # afterwards, a short pass with events around every kernel: the kernels' shares and each step's
            # own duration (an event between two launches keeps the second from starting under the first's tail)
            evs = [[torch.cuda.Event(enable_timing=True) for _ in range(nev)] for _ in range(min(n, 64))]
            for e in evs:
                step(e)
            torch.cuda.synchronize()
        else:
            # small inputs: the L2 is flushed in front of every step, so every step is timed by itself
            evs = [[torch.cuda.Event(enable_timing=True) for _ in range(nev)] for _ in range(n)]
            ctx.barrier()
            t0 = time.time()
            for i in range(n):
                step(evs[i])
            ctx.barrier()
            t1 = time.time()
            total_ms = sum(e[0].elapsed_time(e[nev - 1]) for e in evs)
        phase_ms = [sum(e[i].elapsed_time(e[i + 1]) for e in evs) / len(evs) for i in range(nev - 1)]
        if nev == 2 and flush is None:
            phase_ms = [total_ms / n]          # one update per step: its duration is the region's mean
        total_ms = reduce_max(total_ms, dev)
        per_step = sorted(e[0].elapsed_time(e[nev - 1]) for e in evs)      # each step's own launches
        stats = {"median": per_step[len(per_step) // 2], "min": per_step[0], "max": per_step[-1],
                 "mean_back_to_back": total_ms / n}
        return {"ms": total_ms / n, "phase_ms": phase_ms, "window": (t0, t1), "stats": stats, "inner": inner,
                "timed_s": total_ms * 1e-3}

    res = {}
    if run_fused:       # the headline route first: a long run of the other route leaves the GPU at its power cap
        res["fused"] = time_path(step_fused, 2)
    if run_unfused:
        res["unfused"] = time_path(step_unfused, 4)
    primary = "fused" if run_fused else "unfused"
    ms_per_step = res[primary]["ms"]
    value = job_value(N, world, ms_per_step)

    # ---- one replica's work: ws_shard_update for a single shard r (reads slice r of the R packed buffers)
    single = None
    if run_unfused and wl.opt in ("sgdm", "adam") and layout == "per_tensor" and shards == R:
        r_mid, S_ = R // 2, plan.S
        sl = slice(r_mid * S_, (r_mid + 1) * S_)
        valid = sum(min(max(sg.numel - r_mid * sg.piece, 0), sg.piece) for sg in plan.segments())
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        times = []
        for i in range(5 + 30):
            if flush is not None:
                flush.zero_()
            ev[0].record()
            B.ws_shard_update(plan, r_mid, pg, pw[sl], pm[sl], pv[sl] if pv is not None else None, hy, gathered, ws)
            ev[1].record()
            torch.cuda.synchronize()
            if i >= 5:
                times.append(ev[0].elapsed_time(ev[1]))
        times.sort()
        med = times[len(times) // 2]
        single = {"call": f"ws_shard_update(r={r_mid}) alone, one launch", "valid_params": valid,
                  "ms_median": med, "ms_min": times[0], "value": valid / (med * 1e-3), "unit": UNIT,
                  "achieved_gbs": valid * bytes_per_param(wl)["algorithmic"] / (med * 1e-3) / 1e9}
        single["frac"] = single["achieved_gbs"] / measured_peak()[0]
        # The isolated figure carries the idle-to-first-CTA latency of a launch on a drained GPU (an empty
        # kernel timed this way takes ~10 us).  Steady state: every shard's launch in turn, back to back, so
        # that each reads different memory (R launches together read the whole model: nothing comes from L2).
        if N * 4 * (R + 3) > 256e6:
            def one_of_each():
                for r_ in range(R):
                    s_ = slice(r_ * S_, (r_ + 1) * S_)
                    B.ws_shard_update(plan, r_, pg, pw[s_], pm[s_], pv[s_] if pv is not None else None, hy,
                                      gathered, ws)
            one_of_each()
            rounds = max(2, min(50, int(2000 / (med * 1e3 * R)) + 1))
            torch.cuda.synchronize()
            ev[0].record()
            for _ in range(rounds):
                one_of_each()
            ev[1].record()
            torch.cuda.synchronize()
            ss_ms = ev[0].elapsed_time(ev[1]) / (rounds * R)
            ss_bytes = N / R * bytes_per_param(wl)["algorithmic"]
            single["steady_state"] = {
                "what": f"the {R} shards' launches in turn, back to back, {rounds} rounds; mean per launch",
                "ms": ss_ms, "achieved_gbs": ss_bytes / (ss_ms * 1e-3) / 1e9,
                "frac": ss_bytes / (ss_ms * 1e-3) / 1e9 / measured_peak()[0]}
            single["copy_floor"] = copy_floor(torch, dev, int(ss_bytes))

    # ---- end to end through the host-buffer entry point
    e2e_rec = None
    if e2e:
        host_g = [torch.empty(A_el, dtype=gdt).pin_memory() for _ in range(R)]
        for k in range(R):
            host_g[k].copy_(g_arena[k])
        host_g = B.PtrList(host_g)
        host_w = torch.empty(A_el, dtype=odt).pin_memory()
        stage = torch.empty(A_el, dtype=gdt, device=dev)

        def e2e_step():
            B.ws_step_host(plan, host_g, stage, pg, pw, pm, pv, hy, w_arena, host_w, gathered, ws)
        for _ in range(2):
            e2e_step()
        ctx.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(e2e_steps):
            e2e_step()
        e1.record()
        ctx.barrier()
        e2e_ms = reduce_max(e0.elapsed_time(e1), dev)
        e2e_rec = {"value": world * N * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT,
                   "h2d_bytes_per_step": R * A_el * gb, "d2h_bytes_per_step": A_el * wb,
                   "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps,
                   "api": "ws_step_host (pinned host arenas)"}
        # The fused entry point also takes pinned host tensors as they are: the kernel then pulls the
        # gradients over PCIe itself and writes the weights back the same way (no staging copies).
        try:
            zg = B.TensorTable(plan, [plan.arena_views(a, numels) for a in host_g.tensors], device=dev)
            zw = B.TensorTable(plan, [plan.arena_views(host_w, numels)], device=dev)

            def zc_step():
                B.ws_fused_update(plan, -1, zg, pw, pm, pv, hy, zw, ws)
            zc_step()
            ctx.barrier()
            e0.record()
            for _ in range(e2e_steps):
                zc_step()
            e1.record()
            ctx.barrier()
            zc_ms = reduce_max(e0.elapsed_time(e1), dev)
            e2e_rec["zero_copy"] = {"value": world * N * e2e_steps / (zc_ms * 1e-3), "unit": UNIT,
                                    "ms_per_step": zc_ms / e2e_steps,
                                    "api": "ws_fused_update on pinned host tensors (kernel reads and writes host memory)"}
            del zg, zw
        except Exception as ex:
            e2e_rec["zero_copy"] = {"error": str(ex)[:200]}
        # Both are public calls that take host buffers; the headline is the faster one (the staged copies
        # run one direction of PCIe at a time, the kernel that reads and writes host memory uses both).
        zc = e2e_rec["zero_copy"]
        if "ms_per_step" in zc and zc["ms_per_step"] < e2e_rec["ms_per_step"]:
            staged = {k_: e2e_rec[k_] for k_ in ("value", "ms_per_step", "api")}
            e2e_rec.update({"value": zc["value"], "ms_per_step": zc["ms_per_step"], "api": zc["api"],
                            "staged_copies": staged})
            del e2e_rec["zero_copy"]
        del host_g, host_w, stage
    if rank != 0:
        return None

    # ---- per-kernel rates and the roofline of the dominant kernel
    peak, peak_src = measured_peak()
    bpp = bytes_per_param(wl)
    one_kernel = wl.opt == "lamb" and plan.sched_buf is not None and 8 <= R <= 32
    n_upd_launch = 1 if one_kernel else {"lamb": 3, "lars": 3, "adafactor": 6}.get(wl.opt, 1)
    chunks = -(-T // 1024)
    upd_name = ("two_phase_kernel (phase 1 and phase 2 of every tensor as work items of one kernel)" if one_kernel else
                "update_kernel" if n_upd_launch == 1 else
                "update_kernel pass 1 + af_moments_kernel + af_factors_kernel + pass 2 + af_finalize_clip_kernel + pass 3"
                if n_upd_launch == 6 else
                "update_kernel phase 1 + lamb_finalize_kernel + update_kernel phase 2")

    def kernel_rows(pth):
        ph = res[pth]["phase_ms"]
        if pth == "fused":
            rows = [{"kernel": upd_name + " (formatting fused in)", "launches_per_step": n_upd_launch,
                     "ms_per_step": ph[0], "algorithmic_bytes_per_step": N * bpp["algorithmic"],
                     "moved_bytes_per_step": N * bpp["fused"]}]
        else:
            rows = [{"kernel": "pack_sets_kernel (gradients, all R lists)", "launches_per_step": 1,
                     "ms_per_step": ph[0], "algorithmic_bytes_per_step": R * N * bpp["pack"],
                     "moved_bytes_per_step": R * N * bpp["pack"]},
                    {"kernel": upd_name, "launches_per_step": n_upd_launch, "ms_per_step": ph[1],
                     "algorithmic_bytes_per_step": N * bpp["algorithmic"], "moved_bytes_per_step": N * bpp["update"]},
                    {"kernel": "pack_kernel (unpack weights)", "launches_per_step": chunks,
                     "ms_per_step": ph[2], "algorithmic_bytes_per_step": N * bpp["unpack"],
                     "moved_bytes_per_step": N * bpp["unpack"]}]
        if pth == "unfused" and rows[2]["ms_per_step"] < 0.2:
            rows[2]["copy_floor"] = copy_floor(torch, dev, int(N * bpp["unpack"]))
        tot = sum(r_["ms_per_step"] for r_ in rows)
        for r_ in rows:
            r_["achieved_gbs"] = r_["algorithmic_bytes_per_step"] / (r_["ms_per_step"] * 1e-3) / 1e9
            r_["frac"] = r_["achieved_gbs"] / peak
            r_["moved_gbs"] = r_["moved_bytes_per_step"] / (r_["ms_per_step"] * 1e-3) / 1e9
            r_["share"] = r_["ms_per_step"] / tot
        return rows

    kernels = kernel_rows(primary)
    dom = max(kernels, key=lambda z: z["ms_per_step"])
    # the multi-launch optimizers' update is reported as one unit (its launches depend on one another)
    traffic_pp, traffic_src = NCU_DRAM_BYTES_PER_PARAM.get((wl.name, wl.R, primary), (None, None))
    if layout != "per_tensor" or shards != R or (wl.opt == "lamb" and not one_kernel):
        traffic_pp, traffic_src = None, None
    roofline = {"bound": "hbm", "kernel": dom["kernel"], "achieved": dom["achieved_gbs"], "peak": peak,
                "peak_source": f"{peak_src} copy bandwidth", "unit": "GB/s", "frac": dom["frac"],
                "algorithmic_bytes_per_launch": dom["algorithmic_bytes_per_step"],
                "algorithmic_bytes_per_param": bpp["algorithmic"],
                "moved_bytes_per_launch": dom["moved_bytes_per_step"],
                "launch": f"one step's update = {dom['launches_per_step']} dependent launch(es), timed together",
                "avg_launch_ms": dom["ms_per_step"],
                "traffic": traffic_pp * N if traffic_pp else None, "traffic_source": traffic_src,
                "frac_of_nominal_8TBs": dom["achieved_gbs"] / 8000.0}
    if wl.opt == "lamb":
        roofline["two_pass"] = {"bytes_per_param": bpp["algorithmic"] + 12,
                                "achieved": dom["achieved_gbs"] * (bpp["algorithmic"] + 12) / bpp["algorithmic"],
                                "frac": dom["frac"] * (bpp["algorithmic"] + 12) / bpp["algorithmic"]}
    pr = res[primary]
    rec = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": W_, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_of(wl, align, layout, shards, path=primary,
                            extra={"inner_repeats": pr["inner"], "timed_region_s": round(pr["timed_s"], 3),
                                   "timed_steps": K * pr["inner"]}),
        "roofline": roofline, "kernels": kernels, "clocks": ctx.sampler.summary(*pr["window"]),
        "gpu_launches": K * pr["inner"] * sum(kz["launches_per_step"] for kz in kernels),
        "step_ms": pr["stats"],
    }
    if "unfused" in res and primary != "unfused":
        rows = kernel_rows("unfused")
        ur = res["unfused"]
        rec["unfused_path"] = {
            "step": "ws_pack_sets (R gradient lists) + ws_shard_update(all shards) + ws_unpack as separate kernels",
            "value": world * N / (ur["ms"] * 1e-3), "unit": UNIT, "ms_per_step": ur["ms"],
            "kernels": rows, "gpu_launches": K * ur["inner"] * sum(kz["launches_per_step"] for kz in rows),
            "step_ms": ur["stats"], "clocks": ctx.sampler.summary(*ur["window"])}
        if single is not None:
            rec["unfused_path"]["single_shard"] = single
    if one_kernel:
        # the one-kernel route's waits are bounded; a wait that ran out leaves 1 in the workspace's status word
        off = plan.sync_status_offset()
        rec["config"]["one_kernel_wait_status"] = int(ws[off:off + 4].view(torch.int32).item())
        if rec["config"]["one_kernel_wait_status"] != 0:
            raise RuntimeError("one-kernel LAMB: a bounded wait ran out (status word set); the update is incomplete")
    if unfused_skipped:
        rec["unfused_path"] = {"skipped": unfused_skipped}
    if e2e_rec is not None:
        rec["e2e"] = e2e_rec
    if world == 1 and cpu:
        from oracle import ws_oracle as O
        O.build()
        rec["cpu_baseline"] = cpu_baseline(wl, align, min_seconds=cpu_seconds)
    return rec


def run_shard_window(ctx, wl, plan, align, layout, steps, warmup):
    """Replica counts whose gradients cannot exist on one GPU: time ws_shard_update shard by shard
    on a window of 16 shards, each fed from R S-element slices (what a reduce-scatter receive
    buffer holds), and extrapolate the whole-model step as R x the mean shard time."""
    import numpy as np
    import torch
    from paper_2004_13336_b200 import binding as B
    dev, world, rank = ctx.dev, ctx.world, ctx.rank
    R, N, S = wl.R, wl.N, plan.S
    rng = np.random.default_rng(wl.seed)
    window = sorted(set([0, 1, R // 2, R - 1] + [int(x) for x in rng.integers(2, R - 1, 12)]))
    gen = torch.Generator(device=dev).manual_seed(wl.seed)
    gsl = torch.empty(R, S, dtype=torch.float32, device=dev).normal_(0.0, wl.grad_std, generator=gen).to(wl.grad_dtype)
    gl = B.PtrList([gsl[k] for k in range(R)])
    w = torch.empty(S, device=dev).normal_(0.0, wl.w_std, generator=gen)
    m = torch.empty(S, device=dev).normal_(0.0, wl.m_std, generator=gen)
    v = torch.empty(S, device=dev).normal_(0.0, wl.v_std, generator=gen).abs_()
    hy = B.make_hyper(wl.opt, wl.hyper)
    K, W_ = max(20, steps), max(3, warmup)
    per_shard = []
    t0 = time.time()
    for r in window:
        for _ in range(W_):
            B.ws_shard_update(plan, r, gl, w, m, v if wl.opt != "sgdm" else None, hy, None, None, slice_mode=1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(K):
            B.ws_shard_update(plan, r, gl, w, m, v if wl.opt != "sgdm" else None, hy, None, None, slice_mode=1)
        e1.record()
        torch.cuda.synchronize()
        per_shard.append(e0.elapsed_time(e1) / K)
    t1 = time.time()
    mean_ms = reduce_max(float(np.mean(per_shard)), dev)
    if rank != 0:
        return None
    peak, peak_src = measured_peak()
    bpp = bytes_per_param(wl)["algorithmic"]
    gbs = (N / R) * bpp / (mean_ms * 1e-3) / 1e9
    return {
        "metric": METRIC, "value": job_value(N, world, R * mean_ms), "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": W_, "ms_per_step": R * mean_ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_of(wl, align, layout, R, path="unfused", extra={
            "window": f"extrapolated from {len(window)} of {R} shards: whole-model step = R x mean shard time; "
                      f"each shard call reads R slices of S={S} elements (slice mode 1)",
            "shard_ms_mean": mean_ms, "shard_ms_min": min(per_shard), "shard_ms_max": max(per_shard),
            "padding_pct": 100.0 * (R * S - N) / N}),
        "roofline": {"bound": "hbm", "kernel": "update_kernel (one shard)", "achieved": gbs, "peak": peak,
                     "peak_source": f"{peak_src} copy bandwidth", "unit": "GB/s", "frac": gbs / peak,
                     "algorithmic_bytes_per_launch": (N / R) * bpp, "avg_launch_ms": mean_ms, "traffic": None,
                     "frac_of_nominal_8TBs": gbs / 8000.0},
        "clocks": ctx.sampler.summary(t0, t1),
        "gpu_launches": K * len(window), "e2e": None,
    }


def short_row(rec):
    """The few figures of a sweep row."""
    if rec is None:
        return None
    rf = rec["roofline"]
    row = {"workload": rec["config"]["workload"], "R": rec["config"]["R"], "align_elems": rec["config"]["align_elems"],
           "layout": rec["config"]["layout"], "shards": rec["config"].get("shards", rec["config"]["R"]),
           "value": rec["value"], "unit": UNIT, "ms_per_step": rec["ms_per_step"],
           "timed_steps": rec["config"].get("timed_steps", rec["steps"]),
           "algorithmic_bytes_per_param": rf.get("algorithmic_bytes_per_param"),
           "achieved_gbs": rf["achieved"], "frac_of_measured_peak": rf["frac"],
           "frac_of_nominal_8TBs": rf["frac_of_nominal_8TBs"], "clocks": rec["clocks"]}
    for k in ("window", "padding_pct", "shard_ms_mean"):
        if k in rec["config"]:
            row[k] = rec["config"][k]
    if "two_pass" in rf:
        row["two_pass"] = rf["two_pass"]
    return row


def run_ours(args):
    import gc
    import torch
    if args.route != "replicas":
        return run_real_replicas(args)
    ctx = Ctx(args)

    def release():
        gc.collect()
        torch.cuda.empty_cache()

    def guarded(fn, what):
        try:
            return fn()
        except Exception as e:      # a failed side run must not lose the headline line
            release()
            return {"workload": what, "error": f"{type(e).__name__}: {str(e)[:200]}"}

    common = dict(steps=args.steps, warmup=args.warmup, e2e_steps=args.e2e_steps)
    head = measure(ctx, workload_from_args(args), align=args.align, layout=args.layout, shards=args.shards,
                   tile=args.tile, path=args.path, e2e=not args.no_e2e, cpu=not args.no_cpu_baseline, **common)
    release()
    side = (args.workload == "all" and ctx.world == 1 and not args.no_side_rows
            and not (args.R or args.opt or args.clip or args.tensors))
    if side:
        # one full record for each of the other named workloads
        head["configs"] = []
        for name in ("tiny", "resnet50", "transformer", "bert_large"):
            head["configs"].append(guarded(lambda: measure(
                ctx, get_workload(name), align=args.align, e2e=not args.no_e2e, cpu=not args.no_cpu_baseline,
                cpu_seconds=4.0, **common), name))
            release()
        # Transformer set over the replica counts of the tiny-shard study (Section 5.2), alignments 8 and 32
        sweep = []
        for R, A in ((1, 32), (2, 32), (8, 8), (32, 32), (128, 32), (128, 8), (1024, 32), (1024, 8)):
            sweep.append(guarded(lambda: short_row(measure(
                ctx, get_workload("transformer", R=R), align=A, path="fused", e2e=False, cpu=False, **common)),
                f"transformer R={R} A={A}"))
            release()
        for r_ in head["configs"]:          # the R = 8, A = 32 point is the full record above
            if isinstance(r_, dict) and r_.get("config", {}).get("workload", "").startswith("transformer"):
                sweep.insert(2, short_row(r_))
        head["transformer_r_sweep"] = sweep
        nxt = []
        for name, kw in (("resnet50_lars", {}), ("transformer_adafactor", {}),
                         ("bert_large", {"layout": "concat"}), ("decoder_1p5b", {"layout": "concat"}),
                         ("transformer", {"layout": "concat", "R": 1024}),
                         # partial sharding (Section 5.2): 8 gradient copies, the update sharded 2 ways
                         ("transformer", {"shards": 2, "R": 8})):
            R_ = kw.pop("R", 0)
            nxt.append(guarded(lambda: short_row(measure(
                ctx, get_workload(name, R=R_), align=args.align, path="fused", e2e=False, cpu=False, **kw, **common)),
                name))
            release()
        head["next_workloads"] = nxt
    if ctx.rank == 0:
        print(json.dumps(head))
    ctx.close()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
