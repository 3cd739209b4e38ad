#!/usr/bin/env python
"""Throughput of the SGNS step plus DASGD message application, in (centre, context) pairs per second.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A "step" is one pass of the whole hot path over one batch per replica: every replica trains its
mini-batch (gradient calculation, message build, local application, send) and then every replica
applies the messages that are due.  The default workload is the V = 1M, d = 300, W = 4 configuration.

One JSON line is printed by rank 0.  `value` is measured with the batches already in device memory;
`e2e` is the same metric through tensair_train_batch_host with the batches in pinned host memory and
every replica's loss copied back every step (tensair_read_loss_async) and read on the host one step later, behind an
event, so that the GPU does not wait for the host; the error word is read once per timed region.
`roofline` describes the kernel with the largest share of device time, timed with CUDA events inside the library in a separate pass.  `cpu_baseline`
is the CPU oracle timed on a bounded sample of the same workload on this host's cores.

`--impl reference` times the CPU oracle alone (the only "reference" there is: the paper ships no code).
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
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

from paper_2211_10280_b200 import synth  # noqa: E402

METRIC = "SGNS (center,context) pairs/sec on 1 B200; achieved HBM GB/s vs peak"
UNIT = "pairs/s"
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of a kernel relative to its algorithmic bytes, from
# the ncu captures summarised under profiles/ on a reduced case; the apply kernels are pure streams over the rows
# of their messages, so traffic grows in proportion to the algorithmic bytes of a launch.  Only valid for the
# source file the capture ran (checked by its SHA-256), null otherwise.
NCU_TRAFFIC = {"apply_step": {"traffic_per_algorithmic_byte": 1.026, "source": "paper_2211_10280_b200/csrc/apply.cu",
                              "sha256": "70cf5670dd3f12c83ff5bd2911bfa1de26036855059592189bafebb3ef2398b9",
                              "profile": "profiles/k_apply_step_small_case_V250k_W4.md"}}


def ncu_traffic(kernel: str, algorithmic_bytes: float):
    rec = NCU_TRAFFIC.get(kernel)
    if not rec:
        return None
    import hashlib

    src = ROOT / rec["source"]
    if not src.exists() or hashlib.sha256(src.read_bytes()).hexdigest() != rec["sha256"]:
        return None          # the kernel changed since the counters were taken
    return int(rec["traffic_per_algorithmic_byte"] * algorithmic_bytes)


def hbm_peak():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.rows = []
        self.proc = None
        self.gpu_id = gpu_id

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.gpu_id, f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self, t0: float, t1: float):
        rows = [r for t, r in self.rows if t0 <= t <= t1 and len(r) >= 8] or [r for _, r in self.rows if len(r) >= 8]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        sm = [float(r[0]) for r in rows if r[0].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[4 + i].lower() == "active" for r in rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": float(rows[0][1]), "samples": len(rows),
                "power_w_max": max(float(r[2]) for r in rows), "reasons": reasons}


def max_over_ranks(ms: float, dist, device) -> float:
    """The slowest rank's time: what a multi-rank run reports (works with nccl on GPUs and gloo on CPU)."""
    import torch

    x = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(x, op=dist.ReduceOp.MAX)
    return float(x.item())


MIN_TIMED_SECONDS = 2.0     # a K-step region is repeated until this much has been timed; the median region is reported
MAX_REPEATS = 40


def placement(wl: synth.Workload, world: int, sharded: bool) -> str:
    """How the workload's replicas are placed on the GPUs of the run this line stands for (the same words in both arms)."""
    if world == 1:
        return f"all {wl.W} replicas on one GPU"
    if sharded:
        return (f"{wl.W // world} of {wl.W} replicas per GPU, every message broadcast into every GPU's pool "
                f"on a communication stream")
    return f"{world} independent copies of the one-GPU job, no exchange between them"


def config_of(wl: synth.Workload, world: int, parallelism: str) -> dict:
    """The `config` object of the JSON line: the same keys and values, from the workload and the placement alone, in
    both arms."""
    stride = -(-wl.d // 8) * 8
    return {"workload": wl.name, "V": wl.V, "d": wl.d, "window": wl.window, "k": wl.k, "batch": wl.batch,
            "replicas": wl.W, "max_delay": wl.max_delay, "reduction": "mean" if wl.reduction else "sum",
            "max_grad_buffer": wl.max_grad_buffer,
            "routing": "hash of the centre word, one batch shared by the replicas" if wl.routed else "one substream per replica",
            "pairs_per_batch": wl.pairs_per_batch, "storage": "f32",
            "l2": "inputs larger than L2 (tables %.1f GB)" % (wl.W * 2 * wl.V * stride * 4 / 1e9),
            "parallelism": parallelism}


def repeats_for(ms_one_region: float, min_seconds: float = MIN_TIMED_SECONDS) -> int:
    """How many K-step regions to time so that at least min_seconds are covered."""
    if ms_one_region <= 0 or min_seconds <= 0:
        return 1
    return max(1, min(MAX_REPEATS, int(-(-min_seconds * 1e3 // ms_one_region))))


def pick_workload(name: str, override: str = "") -> synth.Workload:
    """A named workload, optionally with fields replaced (`--override V=250000,W=2`: reduced cases for profiling)."""
    if name not in synth.WORKLOADS:
        raise SystemExit(f"unknown workload {name!r}; one of {sorted(synth.WORKLOADS)}")
    wl = synth.WORKLOADS[name]
    if override:
        kw = {}
        for item in override.split(","):
            key, val = item.split("=")
            kw[key] = type(getattr(wl, key))(val)
        if "W" in kw:
            kw["stream_seeds"] = tuple(wl.stream_seeds[0] + i for i in range(kw["W"]))
        wl = synth.scaled(wl, name=f"{wl.name}[{override}]", **kw)
    return wl


def stream_batches(wl: synth.Workload) -> int:
    """Batches of the workload's stream kept for a run (the steps cycle through them): the whole stream up to 512,
    a whole number of drift epochs when the workload drifts."""
    nb = min(wl.batches, 512)
    if wl.drift_every and nb > wl.drift_every:
        nb -= nb % wl.drift_every
    return nb


def rank_streams(wl: synth.Workload, rank: int, batches: int):
    """Token batches [batches, W, B] of this rank and the unigram counts of its whole stream."""
    wl_r = synth.scaled(wl, stream_seeds=tuple(s + 1000 * rank for s in wl.stream_seeds))
    full = synth.all_streams(wl_r)                       # whole stream: its histogram feeds the sampler
    counts = synth.stream_counts(full, wl.V)
    reps = -(-batches // wl.batches)
    toks = np.stack([np.concatenate([s] * reps)[:batches] for s in full], axis=1)
    return np.ascontiguousarray(toks), counts


# ------------------------------------------------------------------------------------------------
def sharded_workload(wl: synth.Workload, world: int):
    """The workload as N processes run it: its W replicas spread evenly when N divides W (the one-GPU job, total work
    fixed: "strong"); otherwise one replica per GPU, W = N, the stream seeds continued (work per GPU fixed apart from
    the messages to apply, which grow with N: "weak")."""
    if wl.W % world == 0:
        return wl, wl.W // world, "strong"
    seeds = tuple(wl.stream_seeds[0] + i for i in range(world))
    return synth.scaled(wl, name=f"{wl.name}[W={world}]", W=world, stream_seeds=seeds), 1, "weak"


def run_sharded(args):
    """The paper's placement: the replicas spread over the ranks, one group per GPU, every message broadcast into
    every rank's pool over NCCL on a communication stream (paper_2211_10280_b200/exchange.py)."""
    import torch
    import torch.distributed as dist

    from paper_2211_10280_b200 import binding as B
    from paper_2211_10280_b200.exchange import ShardedReplicas

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the SGNS path has no CPU implementation")
    torch.cuda.set_device(local)
    if world > 1:
        os.environ.setdefault("NCCL_DEBUG", "INFO")      # the communicator log shows the ranks and the transport
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    wl = pick_workload(args.workload, args.override)
    if wl.routed or wl.max_grad_buffer != 1:
        raise SystemExit("the sharded placement needs an unrouted workload with maxGradBuffer 1")
    wl, Wl, scaling = sharded_workload(wl, world)
    B.tensair_tune("early_prepare", 2)                    # resident, complete batches (see run_ours)
    for item in filter(None, args.tune.split(",")):
        B.tensair_tune(item.split("=")[0], int(item.split("=")[1]))
    K, Wm = args.steps, max(args.warmup, 3)
    nb = stream_batches(wl)
    toks_all, counts = rank_streams(wl, 0, nb)                   # the one-process job's streams; this rank takes its replicas'
    toks_np = np.ascontiguousarray(toks_all[:, rank * Wl:(rank + 1) * Wl])
    ctx = B.Context(V=wl.V, d=wl.d, window=wl.window, k=wl.k, batch=wl.batch, W=Wl, lr=wl.lr, max_delay=wl.max_delay,
                    seed=wl.seed, counts=counts, device=local, reduction=wl.reduction, world_replicas=wl.W,
                    first_replica=rank * Wl)
    grp = ShardedReplicas(ctx, rank, world, Wl, dist if world > 1 else None, count_device="cuda")
    toks_dev = torch.from_numpy(toks_np).cuda()
    torch.cuda.synchronize()                              # the batches are complete before the first call names them
    toks_pin = torch.from_numpy(toks_np).pin_memory()
    losses_pin = torch.zeros(Wl, dtype=torch.float64).pin_memory()

    def step(t, host=False):
        b = t % nb
        if wl.drift_every and t and t % wl.drift_every == 0:
            ctx.tensair_update_sampler()
        for r in range(Wl):
            if host:
                ctx.tensair_train_batch_host(r, toks_pin[b, r], t)
                ctx.tensair_read_loss_async(losses_pin.data_ptr() + 8 * r)
            else:
                ctx.tensair_train_batch(r, toks_dev[b, r], t)
        grp.exchange(t)                                          # transfers start on the communication stream
        grp.apply(t)                                             # waits only for what is due here at step t
        if host and ctx.tensair_sync() != B.OK:      # the step's one synchronisation: the losses are in losses_pin now
            raise SystemExit("the device reported an error during the benchmark: " + ctx.tensair_last_error())

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(first, host):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        wall0 = time.time()
        ev0.record()
        for t in range(first, first + K):
            step(t, host=host)
        ev1.record()
        barrier()
        ms = ev0.elapsed_time(ev1)
        return (max_over_ranks(ms, dist, "cuda") if world > 1 else ms), wall0, time.time()

    def timed_regions(first, host):
        ms0, wall0, wall1 = timed(first, host)
        first += K
        regions = [ms0]
        reps = repeats_for(ms0, args.min_seconds)
        if world > 1:
            reps = int(max_over_ranks(float(reps), dist, "cuda"))
        for _ in range(reps - 1):
            ms, _, wall1 = timed(first, host)
            first += K
            regions.append(ms)
        return statistics.median(regions), regions, wall0, wall1, first

    uuid = str(torch.cuda.get_device_properties(local).uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    t = 0
    for _ in range(Wm):
        step(t)
        t += 1
    sampler.start()
    time.sleep(0.3)
    launches0, sent0 = ctx.tensair_kernel_launches(), grp.bytes_sent
    ms_dev, regions_dev, wall0, wall1, t = timed_regions(t, host=False)
    launches = (ctx.tensair_kernel_launches() - launches0) // len(regions_dev)
    sent = (grp.bytes_sent - sent0) / (len(regions_dev) * K)
    sampler.stop()
    for _ in range(Wm):
        step(t, host=True)
        t += 1
    ms_e2e, regions_e2e, _, _, t = timed_regions(t, host=True)
    if ctx.tensair_sync() != B.OK:
        raise SystemExit("the device reported an error during the benchmark: " + ctx.tensair_last_error())
    P = wl.pairs_per_batch
    out = {
        "metric": METRIC, "value": wl.W * P * K / (ms_dev * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms_dev / K, "higher_is_better": True, "scaling": scaling, "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": config_of(wl, world, placement(wl, world, True)),
        "timing": {"regions": len(regions_dev), "steps_per_region": K, "reported": "median region",
                   "ms_per_step_min": round(min(regions_dev) / K, 5), "ms_per_step_max": round(max(regions_dev) / K, 5),
                   "timed_seconds": round(sum(regions_dev) / 1e3, 3)},
        "e2e": {"value": wl.W * P * K / (ms_e2e * 1e-3), "unit": UNIT, "ms_per_step": ms_e2e / K, "regions": len(regions_e2e),
                "h2d_bytes_per_step": Wl * wl.batch * 4, "d2h_bytes_per_step": Wl * 8 + 4},
        "gpu_launches": int(launches),
        "exchange": {"bytes_sent_per_step_per_gpu": int(sent),
                     "transport": "NCCL broadcast per message on a communication stream" if world > 1 else "none (one rank)",
                     "received_bytes_waited_for_at_their_own_step": int(grp.bytes_waited_at_own_step),
                     "received_bytes_that_travelled_during_later_batches": int(grp.bytes_waited_later),
                     "hidden_share": round(grp.hidden_share(), 4)},
        "clocks": sampler.summary(wall0, wall1),
    }
    ctx.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2211_10280_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the SGNS path has no CPU implementation")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    wl = pick_workload(args.workload, args.override)
    # the batches are resident in device memory, complete, long before they are trained on: the library may sample and
    # sort a batch ahead of its turn on the stream
    B.tensair_tune("early_prepare", 2)
    for item in filter(None, args.tune.split(",")):
        B.tensair_tune(item.split("=")[0], int(item.split("=")[1]))
    K, Wm = args.steps, max(args.warmup, 3)
    Kp = min(K, 8)                                          # steps of the per-kernel timing pass
    nb = stream_batches(wl)                                 # batches held; step t trains batch t mod nb
    toks_np, counts = rank_streams(wl, rank, nb)
    P = wl.pairs_per_batch

    ctx = B.Context(V=wl.V, d=wl.d, window=wl.window, k=wl.k, batch=wl.batch, W=wl.W, lr=wl.lr,
                    max_delay=wl.max_delay, seed=wl.seed + rank, counts=counts, device=local, reduction=wl.reduction,
                    max_grad_buffer=wl.max_grad_buffer)
    toks_dev = torch.from_numpy(toks_np).cuda()
    torch.cuda.synchronize()                              # the batches are complete before the first call names them
    toks_pin = torch.from_numpy(toks_np).pin_memory()
    losses_pin = torch.zeros((2, wl.W), dtype=torch.float64).pin_memory()      # two steps' losses: one landing, one being read
    loss_events = [torch.cuda.Event(), torch.cuda.Event()]
    pending_loss = [None]
    step_losses = []
    n_rows = {}

    msg_ids = {}

    def step(t, host=False, info=False):
        if wl.drift_every and t and t % wl.drift_every == 0:
            ctx.tensair_update_sampler()                      # passive drift adaptation: the sampler follows the stream
        b = t % nb
        shared = toks_pin[b, 0].to("cuda", non_blocking=True) if (wl.routed and host) else None
        for i in range(wl.W):
            if wl.routed:       # one batch for all replicas, split by the hash of the centre word
                _, inf = ctx.tensair_train_batch_routed(i, shared if host else toks_dev[b, 0], t, want_loss=host,
                                                        want_info=host or info)
            elif host:
                # the loss of every replica travels back asynchronously; the step ends with one synchronisation
                _, inf = ctx.tensair_train_batch_host(i, toks_pin[b, i], t)
                ctx.tensair_read_loss_async(losses_pin.data_ptr() + 8 * (wl.W * (t & 1) + i))
            else:
                _, inf = ctx.tensair_train_batch(i, toks_dev[b, i], t, want_info=info)
            if inf is not None:
                n_rows[(i, t)] = (inf.n_rows, inf.n_in_rows)
            if info or args.log_applies:
                msg_ids[(i, t)] = ctx.tensair_read_message_ids(i, t)
        if args.apply_per_replica:
            for j in range(wl.W):
                ctx.tensair_apply_messages(j, t)
        else:
            ctx.tensair_apply_step(t)                         # all replicas' due messages in one pass
        if host and not wl.routed:
            # The losses of step t are read on the host while step t + 1 runs: an event marks the end of the step's
            # copies, and the host waits for the event of the step before, so the GPU never waits for the host.
            slot = t & 1
            loss_events[slot].record(ctx.stream)
            if pending_loss[0] is not None:
                loss_events[slot ^ 1].synchronize()
                step_losses.append(float(losses_pin[slot ^ 1].sum()))
            pending_loss[0] = slot

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(first, host):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        wall0 = time.time()
        ev0.record()
        for t in range(first, first + K):
            step(t, host=host)
        ev1.record()
        barrier()
        wall1 = time.time()
        if host and pending_loss[0] is not None:             # the last step's losses, and the error word
            step_losses.append(float(losses_pin[pending_loss[0]].sum()))
            pending_loss[0] = None
            if ctx.tensair_sync() != B.OK:
                raise SystemExit("the device reported an error during the benchmark: " + ctx.tensair_last_error())
        ms = ev0.elapsed_time(ev1)
        if world > 1:
            ms = max_over_ranks(ms, dist, "cuda")
        return ms, wall0, wall1

    def timed_regions(first, host):
        """K-step regions back to back until MIN_TIMED_SECONDS are covered: (median ms of a region, all of them,
        wall-clock bounds, the step after the last)."""
        ms0, wall0, wall1 = timed(first, host)
        first += K
        regions = [ms0]
        reps = repeats_for(ms0, args.min_seconds)
        if world > 1:                                        # every rank must time the same number of regions
            reps = int(max_over_ranks(float(reps), dist, "cuda"))
        for _ in range(reps - 1):
            ms, _, wall1 = timed(first, host)
            first += K
            regions.append(ms)
        return statistics.median(regions), regions, wall0, wall1, first

    uuid = str(torch.cuda.get_device_properties(local).uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    t = 0
    for _ in range(Wm):
        step(t)
        t += 1
    sampler.start()
    time.sleep(0.3)
    launches0 = ctx.tensair_kernel_launches()
    ms_dev, regions_dev, wall0, wall1, t = timed_regions(t, host=False)
    launches = (ctx.tensair_kernel_launches() - launches0) // len(regions_dev)
    sampler.stop()
    for _ in range(Wm):
        step(t, host=True)
        t += 1
    ms_e2e, regions_e2e, _, _, t = timed_regions(t, host=True)

    # per-kernel pass: CUDA events around every launch, on the library's stream
    for _ in range(wl.max_delay):                            # so that every message applied below has its ids on record
        step(t, info=True)
        t += 1
    ctx.tensair_profile(True)
    ctx.tensair_profile_read()
    first_prof = t
    for _ in range(Kp):
        step(t, info=True)
        t += 1
    prof = ctx.tensair_profile_read()
    ctx.tensair_profile(False)
    if ctx.tensair_sync() != B.OK:
        raise SystemExit("the device reported a bad token during the benchmark")

    rebuild = None
    if wl.drift_every:
        # the sampler's rebuild on its own: on the device (asynchronous) and, for comparison, on one host thread
        rebuild = {}
        for mode, knob in (("device_ms", 1), ("host_ms", 0)):
            B.tensair_tune("device_alias_build", knob)
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            ev0.record()
            ctx.tensair_update_sampler()
            ev1.record()
            torch.cuda.synchronize()
            rebuild[mode] = round(ev0.elapsed_time(ev1), 3)
        B.tensair_tune("device_alias_build", 1)

    pairs_per_step = P if wl.routed else wl.W * P
    value = world * pairs_per_step * K / (ms_dev * 1e-3)
    e2e_value = world * pairs_per_step * K / (ms_e2e * 1e-3)

    # algorithmic bytes (each distinct row moved once per pass), from the exact row counts
    row = 4 * wl.d
    msgs = [n_rows[(i, s)] for i in range(wl.W) for s in range(first_prof, first_prof + Kp)]
    U = float(np.mean([m[0] for m in msgs]))
    U_in = float(np.mean([m[1] for m in msgs]))
    U_out = U - U_in
    applied, groups = [], {}
    for j in range(wl.W):
        for origin, snd, due, at, _ in ctx.tensair_read_delivery_log(j).tolist():
            if first_prof <= at < first_prof + Kp and (snd, origin) in n_rows:
                ids_m = msg_ids.get((snd, origin))
                applied.append(ids_m.size if ids_m is not None else n_rows[(snd, origin)][0])
                groups.setdefault((j, at), []).append((snd, origin))
    U_applied = float(np.mean(applied)) if applied else U
    # one pass over the receiver's table for all messages due: every delta row read once, every row of the
    # union of their id sets read and written once
    fused_bytes = []
    for members in groups.values():
        if len(members) >= 2 and all(m in msg_ids and msg_ids[m] is not None for m in members):
            union = np.unique(np.concatenate([msg_ids[m] for m in members])).size
            fused_bytes.append(sum(msg_ids[m].size for m in members) * (row + 4) + union * 2 * row)
    algo = {
        "forward": (U_out + U_in) * row,                                   # every touched row gathered once
        "reduce_rows": U * (row + 4) + U_out * 2 * row,                   # message write + read/write of output rows
        "apply_message": U_applied * (row + 4 + 2 * row),                 # delta read + row read + row write
    }
    if fused_bytes:
        algo["apply_fused"] = float(np.mean(fused_bytes))
    # one pass for all receivers of a step: every delta row of the distinct messages read once, and per receiver
    # every row of the union of its messages' id sets read and written once
    per_step = {}
    for (j, at), members in groups.items():
        per_step.setdefault(at, {})[j] = members
    step_pass_bytes = []
    for at, per_j in sorted(per_step.items()):
        distinct = sorted({m for ms in per_j.values() for m in ms})
        if sum(len(ms) for ms in per_j.values()) < 2 or any(msg_ids.get(m) is None for m in distinct):
            continue
        delta_rows = sum(msg_ids[m].size for m in distinct)
        union_rows = sum(np.unique(np.concatenate([msg_ids[m] for m in ms])).size for ms in per_j.values())
        step_pass_bytes.append(delta_rows * (row + 4) + union_rows * 2 * row)
    if step_pass_bytes:
        algo["apply_step"] = float(np.mean(step_pass_bytes))
    if args.log_applies:
        # every apply launch of the run in call order, with the bytes it has to move (for matching ncu captures)
        calls = {}
        for j in range(wl.W):
            for origin, snd, due, at, _ in ctx.tensair_read_delivery_log(j).tolist():
                calls.setdefault(at, {}).setdefault(j, []).append((snd, origin))
        with open(args.log_applies, "w") as fh:
            for at, per_j in sorted(calls.items()):
                if any(msg_ids.get(m) is None for ms in per_j.values() for m in ms):
                    continue
                if args.apply_per_replica:
                    for j, members in sorted(per_j.items()):
                        ids = [msg_ids[m] for m in members]
                        union = np.unique(np.concatenate(ids)).size
                        fh.write(json.dumps({"step": at, "receiver": j, "messages": len(members), "kernel":
                                             "k_apply_step (one receiver)" if len(members) > 1 else "k_apply",
                                             "delta_rows": sum(x.size for x in ids), "union_rows": union,
                                             "algorithmic_bytes": sum(x.size for x in ids) * (row + 4) + union * 2 * row}) + "\n")
                else:
                    distinct = sorted({m for ms in per_j.values() for m in ms})
                    delta_rows = sum(msg_ids[m].size for m in distinct)
                    union_rows = sum(np.unique(np.concatenate([msg_ids[m] for m in ms])).size for ms in per_j.values())
                    fh.write(json.dumps({"step": at, "messages": len(distinct), "deliveries": sum(len(ms) for ms in per_j.values()),
                                         "kernel": "k_apply_step", "delta_rows": delta_rows, "union_rows": union_rows,
                                         "algorithmic_bytes": delta_rows * (row + 4) + union_rows * 2 * row}) + "\n")
    tot_ms = sum(v[1] for v in prof.values()) or 1.0
    kernels = {}
    for name, (cnt, ms) in prof.items():
        if not cnt:
            continue
        avg = ms / cnt
        rec = {"launches_per_step": cnt / Kp, "avg_ms": round(avg, 5), "share": round(ms / tot_ms, 4)}
        if name in algo:
            rec["algorithmic_bytes"] = int(algo[name])
            rec["gbs"] = round(algo[name] / (avg * 1e-3) / 1e9, 1)
        kernels[name] = rec
    dom = max((n for n in kernels if n in algo), key=lambda n: kernels[n]["share"])
    peak, peak_kind = hbm_peak()
    achieved = kernels[dom]["gbs"]
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "peak_source": f"of {peak_kind}",
                "unit": "GB/s", "frac": round(achieved / peak, 4),
                "traffic": ncu_traffic(dom, kernels[dom]["algorithmic_bytes"]),
                "algorithmic_bytes": kernels[dom]["algorithmic_bytes"],
                "avg_ms": kernels[dom]["avg_ms"], "share_of_device_time": kernels[dom]["share"]}
    own = U * row + U * (row + 4) + U * (row + 4 + 2 * row)
    # remote part: every message applied in the per-kernel pass, per-message model (delta read, row read, row write)
    # remote part, two models: what the launches really have to move (the one-pass apply reads a delta row once however
    # many receivers it is due for, and a table row once however many messages touch it), and the per-message model
    # (delta read, row read, row write for every delivery) that a message-by-message application would move
    per_message_model = len(applied) / Kp * U_applied * (row + 4 + 2 * row) if applied else 0.0
    if args.apply_per_replica:
        moved = (sum(fused_bytes) + sum(msg_ids[ms[0]].size * (3 * row + 4) for ms in groups.values()
                                        if len(ms) == 1 and msg_ids.get(ms[0]) is not None)) / Kp
    else:
        moved = sum(step_pass_bytes) / Kp
    remote_per_step = moved if moved else per_message_model
    step_bytes = wl.W * own + remote_per_step
    step_gbs = step_bytes / (ms_dev * 1e-3 / K) / 1e9
    model_gbs = (wl.W * own + per_message_model) / (ms_dev * 1e-3 / K) / 1e9

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms_dev / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": config_of(wl, world, placement(wl, world, False)),
        "timing": {"regions": len(regions_dev), "steps_per_region": K, "reported": "median region",
                   "ms_per_step_min": round(min(regions_dev) / K, 5), "ms_per_step_max": round(max(regions_dev) / K, 5),
                   "timed_seconds": round(sum(regions_dev) / 1e3, 3)},
        "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": ms_e2e / K, "regions": len(regions_e2e),
                "h2d_bytes_per_step": (1 if wl.routed else wl.W) * wl.batch * 4, "d2h_bytes_per_step": wl.W * (8 + 16 + 4) if wl.routed else wl.W * 8},
        "gpu_launches": int(launches),
        "clocks": sampler.summary(wall0, wall1),
        "roofline": roofline,
        "step_hbm": {"algorithmic_bytes_per_step": int(step_bytes), "gbs": round(step_gbs, 1),
                     "frac_of_peak": round(step_gbs / peak, 4), "rows_per_message": int(U),
                     "per_message_model_gbs": round(model_gbs, 1)},
        "kernels": kernels,
    }
    if rebuild:
        out["sampler_rebuild"] = dict(rebuild, every_batches=wl.drift_every)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(wl, toks_np, counts, steps=2)
    ctx.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))


# ------------------------------------------------------------------------------------------------
def make_oracle(wl, counts):
    from oracle import Oracle

    return Oracle(V=wl.V, d=wl.d, window=wl.window, k=wl.k, batch=wl.batch, W=wl.W, lr=wl.lr,
                  max_delay=wl.max_delay, seed=wl.seed, counts=counts, reduction=wl.reduction,
                  max_grad_buffer=wl.max_grad_buffer)


def cpu_baseline(wl, toks_np, counts, steps):
    """The oracle as it stands on a bounded sample: the first `steps` steps of all replicas."""
    import oracle

    o = make_oracle(wl, counts)
    t0 = time.time()
    for t in range(steps):
        for i in range(wl.W):
            rc, _, _ = o.train_batch(i, toks_np[t, i], t)
            assert rc == 0
        for j in range(wl.W):
            o.apply_messages(j, t)
    dt = time.time() - t0
    o.close()
    return {"value": wl.W * wl.pairs_per_batch * steps / dt, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": f"first {steps} steps of all {wl.W} replicas ({wl.W * steps} batches, {dt:.1f} s)"}


def run_reference(args):
    """The CPU oracle as the reference arm: every step trains one replica's batch (replicas in turn) and,
    once all replicas have trained a step, applies what is due - a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank != 0:
        return
    import oracle

    wl = pick_workload(args.workload, args.override)
    if world > 1 and not args.replicas_only:
        wl = sharded_workload(wl, world)[0]                 # the workload the N-rank arm runs
    K, Wm = args.steps, args.warmup
    total = Wm + K
    toks_np, counts = rank_streams(wl, 0, -(-total // wl.W) + 1)
    o = make_oracle(wl, counts)

    def step(s):
        t, i = divmod(s, wl.W)
        rc, _, _ = o.train_batch(i, toks_np[t, i], t)
        assert rc == 0
        if i == wl.W - 1:
            for j in range(wl.W):
                o.apply_messages(j, t)

    for s in range(Wm):
        step(s)
    t0 = time.time()
    for s in range(Wm, total):
        step(s)
    dt = time.time() - t0
    value = wl.pairs_per_batch * K / dt
    sample = f"{K} steps of one replica-batch each (replicas in turn, messages applied after every {wl.W}th)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": Wm, "ms_per_step": dt / K * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": config_of(wl, world, placement(wl, world, not args.replicas_only)),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_sweep(args):
    """The throughput sweep (V = 1M, one replica): one JSON line per (d, batch, k) point with pairs/s and
    the algorithmic HBM GB/s of the step (gather + message write + local application, each touched row once per pass)."""
    import torch

    from paper_2211_10280_b200 import binding as B

    peak, peak_kind = hbm_peak()
    steps = min(args.steps, 100)
    B.tensair_tune("early_prepare", 2)                    # resident, complete batches (see run_ours)
    for item in filter(None, args.tune.split(",")):
        B.tensair_tune(item.split("=")[0], int(item.split("=")[1]))
    for wl in synth.SWEEP:
        nb = steps + 6
        stream = synth.token_stream(wl, 0, nb)
        counts = synth.stream_counts([synth.token_stream(wl, 0, min(wl.batches, 100))], wl.V)
        ctx = B.Context(V=wl.V, d=wl.d, window=wl.window, k=wl.k, batch=wl.batch, W=1, lr=wl.lr, seed=wl.seed,
                        counts=counts, reduction=wl.reduction)
        toks = torch.from_numpy(stream).cuda()
        torch.cuda.synchronize()
        rows = []
        for t in range(3):
            _, info = ctx.tensair_train_batch(0, toks[t], t, want_info=True)
            rows.append(info.n_rows)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        ev0.record()
        for t in range(3, 3 + steps):
            ctx.tensair_train_batch(0, toks[t], t)
        ev1.record()
        torch.cuda.synchronize()
        ms = ev0.elapsed_time(ev1) / steps
        launches = ctx.tensair_kernel_launches()
        _, info = ctx.tensair_train_batch(0, toks[3 + steps], 3 + steps, want_info=True)
        launches = ctx.tensair_kernel_launches() - launches
        U = float(np.mean(rows + [info.n_rows]))
        row = 4 * wl.d
        own = U * row + U * (row + 4) + U * (row + 4 + 2 * row)
        # nominal model: every contribution's row fetched once by the gradient calculation and its centre row once by
        # the row sums (what the kernels request from L2; the distinct rows are what must come from DRAM)
        nominal = 2.0 * wl.pairs_per_batch * (wl.k + 1) * row + U * (row + 4) + U * 2 * row
        line = {"workload": wl.name, "d": wl.d, "batch": wl.batch, "k": wl.k, "pairs_per_batch": wl.pairs_per_batch,
                "rows_per_message": int(U), "ms_per_batch": round(ms, 4), "launches_per_batch": int(launches),
                "pairs_per_s": wl.pairs_per_batch / (ms * 1e-3), "algorithmic_gbs": round(own / (ms * 1e-3) / 1e9, 1),
                "frac_of_peak": round(own / (ms * 1e-3) / 1e9 / peak, 4), "peak": f"{peak} GB/s of {peak_kind}",
                "nominal_gbs": round(nominal / (ms * 1e-3) / 1e9, 1)}
        if not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(wl, stream[:, None, :], counts, steps=3)
        print(json.dumps(line), flush=True)
        ctx.close()
        del ctx, toks
        torch.cuda.empty_cache()


def launch_ranks(n: int, argv) -> int:
    """Runs this script as n ranks on one node under torch.distributed.run (rendezvous on 127.0.0.1, a free port)."""
    import socket

    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), str(Path(__file__).resolve()), *argv]
    return subprocess.call(cmd, env=env)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=synth.LARGE_DASGD.name)
    ap.add_argument("--override", default="", help="comma-separated field=value replacements of the workload")
    ap.add_argument("--tune", default="", help="comma-separated knob=value pairs passed to tensair_tune (sweeps)")
    ap.add_argument("--log-applies", default="", help="write one JSON line per apply call (bytes to move) to this file")
    ap.add_argument("--sweep", action="store_true", help="run the 32-point throughput sweep instead (one line per point)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--min-seconds", type=float, default=MIN_TIMED_SECONDS,
                    help="repeat the K-step timed region until this much has been timed (0: time it once; for captures under a profiler)")
    ap.add_argument("--apply-per-replica", action="store_true",
                    help="apply the due messages with one tensair_apply_messages call per replica instead of tensair_apply_step")
    ap.add_argument("--sharded", action="store_true",
                    help="the paper's placement: replicas spread over the ranks, messages exchanged (the default with --gpus > 1)")
    ap.add_argument("--replicas-only", action="store_true",
                    help="with --gpus > 1: N independent copies of the one-GPU job instead of the sharded placement")
    args = ap.parse_args()
    if args.gpus > 1 and "RANK" not in os.environ:
        # not started by a launcher: start the N ranks here, one per GPU, and hand on their exit status
        sys.exit(launch_ranks(args.gpus, sys.argv[1:]))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.sharded or (world > 1 and not args.replicas_only):
        run_sharded(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
