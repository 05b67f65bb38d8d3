#!/usr/bin/env python
"""Benchmark of the SAT epoch step on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload large]

A step is one steady-state SAT epoch over all partitions of the workload: layer-1 halo
pull, predictor (LSTM over the cached snapshots + graph convolution + skip) for every
cached layer, every layer forward (SpMM + transform), cache push, loss seed, every layer
backward, ring commit and the SGD step.  metric = edges/s = nnz(A + I) / epoch time.
Prints ONE JSON line on rank 0.

The default workload is the largest of the five configurations that fits one GPU
("large": 2.45 M nodes, 128 M entries of A + I, 32 partitions); the others are selectable.
--impl reference times the CPU oracle (as it stands) on the host cores instead, on a
bounded sample of the same workload per step.
With N > 1 every rank runs an independent replica of the workload (the path of this build
does not shard across GPUs; there is no collective on the data path); the value is the
aggregate over ranks, timed as the max over ranks.  Started as plain `python bench.py
--gpus N` it launches the N ranks itself (torch.distributed.run on 127.0.0.1).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per launch of the dominant kernel comes from the committed ncu
# summaries under profiles/: a line of the form
#     traffic_bytes_per_launch[<workload>/<family>] = <bytes>
# in any profiles/*.md is picked up; no such line for the workload that runs means "traffic": null in the JSON line.
def ncu_traffic(workload: str, family: str):
    import glob
    import re
    pat = re.compile(r"traffic_bytes_per_launch\[" + re.escape(workload) + "/" + re.escape(family) + r"\]\s*=\s*([0-9.eE+]+)")
    for path in sorted(glob.glob(os.path.join(ROOT, "profiles", "*.md"))):
        with open(path) as f:
            m = pat.search(f.read())
        if m:
            return float(m.group(1)), os.path.basename(path)
    return None, None


# predictor update period Delta-T of Algorithm 1 followed by the run (epochs between two parameter-version bumps)
PRED_PERIOD = 10
PRED_LR = 0.01

# The contractions run on the tensor cores in TF32 (two-term split: three TF32 MMAs per product term).  The box's
# measured tensor peak is a bf16 figure; TF32 is taken as measured bf16 x the nominal ratio 1.1 / 2.25 PFLOP/s.
TF32_OVER_BF16 = 1.1 / 2.25
TF32_MMAS_PER_TERM = 3


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm=float(p["hbm_gbs"]), bf16=float(p["bf16_tflops_sustained"]), source="measured")
    return dict(hbm=6650.0, bf16=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=[])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        for ln in self.lines:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    power_w_max=max(power) if power else None, samples=len(sm), reasons=sorted(reasons))


# ------------------------------------------------------------------------------------------
# CPU oracle leg (cpu_baseline of the default run, and the whole of --impl reference)
# ------------------------------------------------------------------------------------------
# one step of the CPU legs handles at most this many entries of A + I (a whole partition of the smaller workloads)
ORACLE_SAMPLE_ENTRIES = 1_200_000


class OracleSample:
    """The oracle on a bounded sample of the workload.  The unit of a sample is a `block`: a whole partition when a
    partition has at most ORACLE_SAMPLE_ENTRIES entries of A + I; otherwise every partition's contiguous id range is cut
    into `cut` equal ranges and the oracle runs one of them as a partition of that finer contiguous partitioning (all layers
    forward and backward plus the LSTM for the cached nodes the block reads: its out-of-block neighbours are its halo).
    The ring is full: tau snapshots of seeded non-negative embeddings, materialised only for the cache slots the
    sampled blocks read — the work does not depend on the values."""

    def __init__(self, wl, n_blocks: int):
        from oracle import sat_ref as orc
        from sat_synth import embedding_table, table_rows
        self.orc, self.wl = orc, wl
        per_part = wl.nnz / wl.M
        self.cut = 1 if wl.part_given is not None else max(1, int(np.ceil(per_part / ORACLE_SAMPLE_ENTRIES)))
        self.M = wl.M * self.cut
        part = wl.part_given if wl.part_given is not None else orc.contig_blocks(wl.n, self.M)
        # the sampled blocks: evenly spread over the id range
        n_blocks = min(n_blocks, self.M)
        self.blocks = [int(i * self.M // n_blocks) for i in range(n_blocks)]
        self.dtil, _ = orc.degrees(wl.rowptr)
        self.P = orc.build_partition(wl.rowptr, wl.col, part, self.M, only_parts=self.blocks)
        self.cache = orc.CacheRing(self.P.n_slots, wl.dims[1:-1], wl.tau)     # zero pages: nothing is touched yet
        need = [self.P.halo_slot[m] for m in self.blocks] + [self.P.slot[self.P.inner_gid[m][self.P.hrow_col[m]]] for m in self.blocks]
        slots = np.unique(np.concatenate(need)) if need else np.empty(0, dtype=np.int64)
        for li, buf in enumerate(self.cache.buf):
            table = embedding_table(wl.seed, wl.dims[1 + li])
            for s in range(buf.shape[0]):
                buf[s][slots] = table_rows(table, slots, 1 + s + 100 * li)
        self.cache.n_valid = wl.tau
        self.cores = orc.num_threads()

    def describe(self) -> str:
        wl = self.wl
        unit = (f"1 of {wl.M} partitions" if self.cut == 1 else
                f"1 of {self.M} contiguous id blocks (each of the {wl.M} partitions cut into {self.cut}; the block runs as a partition of that "
                f"finer partitioning, its out-of-block neighbours being its halo)")
        return (f"{unit} of the {wl.name} workload, all layers fwd+bwd+predictor incl. the LSTM for the cached nodes the block reads; "
                f"ring full (tau={wl.tau})")

    def run(self, blocks):
        wl = self.wl
        t0 = time.perf_counter()
        self.orc.run_epoch(self.P, self.dtil, self.cache, wl.X, wl.labels, wl.W, wl.b, wl.pred, wl.loss, keep=True, parts=blocks)
        dt = time.perf_counter() - t0
        edges = sum(int(self.P.loc_rowptr[m][-1]) for m in blocks)
        return edges, dt


def run_reference(args, wl):
    """--impl reference: the oracle, one block per step (rotating over the sampled blocks), W warm-up steps then K timed steps."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    smp = OracleSample(wl, args.warmup + args.steps)
    nb = len(smp.blocks)
    for i in range(args.warmup):
        smp.run([smp.blocks[i % nb]])
    edges, secs = 0, 0.0
    for i in range(args.steps):
        e, t = smp.run([smp.blocks[(args.warmup + i) % nb]])
        edges += e
        secs += t
    value = edges / secs
    sample = "per step: " + smp.describe()
    line = dict(impl="reference", metric="SAT epoch edges/s (fwd+bwd+predictor, P partitions)", value=value, unit="edges/s",
                n_gpus=0, steps=args.steps, warmup=args.warmup, ms_per_step=1e3 * secs / max(args.steps, 1), higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=workload_config(wl),
                cpu_baseline=dict(value=value, unit="edges/s", cores=smp.cores, kind="oracle", sample=sample),
                e2e=dict(value=value, unit="edges/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line), flush=True)


def workload_config(wl):
    return dict(workload=f"{wl.name}: {wl.n} nodes, nnz(A+I)={wl.nnz}, GCN {'-'.join(map(str, wl.dims))}, "
                         f"{wl.M} partitions ({'the blocks of the stochastic block model' if wl.part_given is not None else 'contiguous id blocks after BFS relabel'}), "
                         f"predictor history {wl.tau}, h={wl.pred[0]['h'] if wl.pred else 0}",
                nodes=wl.n, nnz=wl.nnz, partitions=wl.M, tau=wl.tau,
                predictor_update_period=f"{PRED_PERIOD} epochs (Algorithm 1's Delta-T): the predictor's parameter version is bumped every "
                                        f"{PRED_PERIOD}th epoch, which drops the cached LSTM input projections; the timed epochs contain "
                                        f"their share of such epochs",
                l2="working set per epoch (activations, saved aggregations, ring) far exceeds the 126 MB L2; no flush")


def max_over_ranks(values, dist, device):
    """Every rank contributes its own device-timed durations; all ranks get the maximum of each."""
    if dist is None:
        return [float(v) for v in values]
    import torch
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_value(total_ms, steps, units_per_rank_step, world):
    """(ms per step, units per second over all ranks): every rank processes its own replica of the workload (weak scaling)."""
    ms_per_step = total_ms / steps
    return ms_per_step, world * units_per_rank_step / (ms_per_step * 1e-3)


def side_workload(name: str, steps: int, peaks):
    """A short device-resident run of another configuration (ring filled, `steps` timed epochs with the per-family events
    on): epoch time, edges/s and the SpMM / whole-epoch fractions, for the side table of the JSON line."""
    import torch
    import paper_2308_13466_b200.binding as B
    from paper_2308_13466_b200.epoch import SatEpoch
    from sat_synth import make_workload
    wl = make_workload(name)
    dev = torch.device("cuda", torch.cuda.current_device())
    up = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    ep = SatEpoch(wl.rowptr, wl.col, wl.M, wl.dims, wl.tau, wl.loss, part_given=wl.part_given, device=dev.index)
    try:
        perm = np.concatenate([B.sat_part_lists(ep.ctx, m)["inner_gid"] for m in range(wl.M)])
        X = torch.zeros((wl.n, (wl.dims[0] + 3) & ~3), dtype=torch.float32, device=dev)[:, :wl.dims[0]]
        X.copy_(torch.from_numpy(wl.X))
        ep.set_inputs(X, up(wl.labels[perm]))
        W, b = [up(w) for w in wl.W], [up(x) for x in wl.b]
        preds = [B.make_pred_params(up(p["Wx"]), up(p["Uh"]), up(p["b"]), up(p["Wg"]), up(p["bg"]), int(p["h"]), 1) for p in wl.pred]
        for _ in range(wl.tau + 3):
            ep.step(W, b, preds, 0.01)
        stream = torch.cuda.current_stream(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            ep.step(W, b, preds, 0.01)
        e1.record(stream)
        stream.synchronize()
        ms = e0.elapsed_time(e1) / steps
        B.sat_profile_enable(ep.ctx, True)
        for _ in range(steps):
            ep.step(W, b, preds, 0.01)
        prof = B.sat_profile_read(ep.ctx)
        B.sat_profile_enable(ep.ctx, False)
        fam = {k: dict(ms_per_step=v["ms"] / steps, hbm_frac=v["bytes"] / (v["ms"] * 1e-3) / 1e9 / peaks["hbm"])
               for k, v in prof.items() if v["calls"] and v["ms"] > 0}
        alg = sum(v["bytes"] for v in prof.values()) / steps
        return dict(workload=workload_config(wl)["workload"], steps=steps, ms_per_step=ms, edges_per_s=wl.nnz / (ms * 1e-3),
                    epoch_hbm_frac=alg / (ms * 1e-3) / 1e9 / peaks["hbm"],
                    spmm_fwd=dict(ms_per_step=fam.get("spmm_fwd", {}).get("ms_per_step"), hbm_frac=fam.get("spmm_fwd", {}).get("hbm_frac"),
                                  gather_gbs=(prof["spmm_fwd"]["flops"] / 2.0 * 4.0 / (prof["spmm_fwd"]["ms"] * 1e-3) / 1e9) if prof.get("spmm_fwd", {}).get("ms") else None),
                    largest_families_ms={k: round(v["ms_per_step"], 3) for k, v in sorted(fam.items(), key=lambda kv: -kv[1]["ms_per_step"])[:5]},
                    halo_rows=int(ep.nb), boundary_fraction=ep.n_slots / wl.n)
    finally:
        ep.close()


# ------------------------------------------------------------------------------------------
def run_ours(args, wl):
    import torch
    import paper_2308_13466_b200.binding as B
    from paper_2308_13466_b200.epoch import SatEpoch

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU implementation")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def up(a):
        return torch.from_numpy(np.ascontiguousarray(a)).to(dev)

    def pad2d(a):
        full = torch.zeros((a.shape[0], (a.shape[1] + 3) & ~3), dtype=torch.float32, device=dev)
        v = full[:, :a.shape[1]]
        v.copy_(torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)))
        return v

    ep = SatEpoch(wl.rowptr, wl.col, wl.M, wl.dims, wl.tau, wl.loss, part_given=wl.part_given, device=local)
    perm = np.empty(wl.n, dtype=np.int64)
    off = 0
    for m in range(wl.M):
        lst = B.sat_part_lists(ep.ctx, m)["inner_gid"]
        perm[off:off + lst.shape[0]] = lst
        off += lst.shape[0]
    X_dev = pad2d(wl.X)
    labels_perm = np.ascontiguousarray(wl.labels[perm])
    ep.set_inputs(X_dev, up(labels_perm))
    W = [up(w) for w in wl.W]
    b = [up(x) for x in wl.b]
    preds = [B.make_pred_params(up(p["Wx"]), up(p["Uh"]), up(p["b"]), up(p["Wg"]), up(p["bg"]), int(p["h"]), 1) for p in wl.pred]
    lr = 0.01
    # Algorithm 1 fine-tunes the predictor every Delta-T epochs (the paper finds 5..15 best); between two updates its
    # parameters are fixed, which is what lets the library keep the LSTM input projections of the snapshots it has seen.
    # The run follows that schedule: every PRED_PERIOD-th epoch the parameter version is bumped as an update would do (same
    # values: the work does not depend on them), so the cached projections are dropped and the following tau epochs run
    # the older snapshots' steps from the raw ring.  The update's own kernels are timed separately (pred_update).
    epoch_no = [0]

    def sat_epoch(Wl, bl, rate):
        epoch_no[0] += 1
        for pp in preds:
            pp.version = 1 + epoch_no[0] // PRED_PERIOD
        ep.step(Wl, bl, preds, rate)

    # fill the ring with real embeddings (tau + 1 epochs), then W warm-up steps
    for _ in range(wl.tau + 1):
        sat_epoch(W, b, lr)
    # the clock sampler runs from the warm-up on: the GPU is busy back to back from here to the end of the timed region
    sampler = ClockSampler(local)
    sampler.start()
    for _ in range(max(args.warmup, 0)):
        sat_epoch(W, b, lr)
    stream = torch.cuda.current_stream(dev)

    # ---- profile pass (outside the headline): every kernel family bracketed by CUDA events for the per-family table.  Each
    #      bracket costs two event records on the stream, ~150 pairs per epoch, which slows an epoch by a few per cent ----
    B.sat_profile_select(ep.ctx, None)
    B.sat_profile_enable(ep.ctx, True)
    q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    q0.record(stream)
    for i in range(args.steps):
        sat_epoch(W, b, lr)
    q1.record(stream)
    stream.synchronize()
    ms_profiled = q0.elapsed_time(q1) / max(args.steps, 1)
    prof = B.sat_profile_read(ep.ctx)
    B.sat_profile_enable(ep.ctx, False)
    top_family = max(prof, key=lambda k: prof[k]["ms"])

    # ---- device-resident timing: the timed region carries the events of the dominant family only ----
    barrier()
    B.sat_profile_select(ep.ctx, [top_family])
    B.sat_profile_enable(ep.ctx, True)
    launches0 = B.sat_launch_count(ep.ctx)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    e0.record(stream)
    marks[0].record(stream)
    for i in range(args.steps):
        sat_epoch(W, b, lr)
        marks[i + 1].record(stream)
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    step_ms = [marks[i].elapsed_time(marks[i + 1]) for i in range(args.steps)]
    launches = B.sat_launch_count(ep.ctx) - launches0
    prof_top = B.sat_profile_read(ep.ctx)
    B.sat_profile_enable(ep.ctx, False)
    B.sat_profile_select(ep.ctx, None)
    loss = float(ep.loss_sum.item())
    # what the L2 -> SM path delivers on this GPU right now (64 MiB buffer resident in L2): contiguous stream, and random
    # rows of the hidden width with the SpMM's access shape
    l2_row = int(max(wl.dims[1:-1])) if wl.L > 1 else int(wl.dims[0])
    l2_row = min(1024, (l2_row + 3) & ~3)
    l2_stream_gbs, l2_gather_gbs = B.sat_profile_l2_rates(ep.ctx, l2_row)
    # how the forward aggregation walks the partitions at each of its widths (source blocks, work items, partial-sum rows)
    spmm_plan = {str(int(d)): dict(zip(("source_blocks", "work_items", "partial_rows"), B.sat_spmm_plan(ep.ctx, B.SAT_ALL_PARTS, int(d))))
                 for d in sorted(set(wl.dims[:-1]))}
    # for reference, outside the headline and without any profiling events: the same epochs (a) with a predictor that is
    # never updated (one version throughout: all tau - 1 older projections cached) and (b) with no version promise (nothing
    # kept between epochs: every epoch runs all steps from the raw ring, K = d + h in the recurrence)
    def side_epochs(version):
        for pp in preds:
            pp.version = version
        for _ in range(wl.tau + 1):
            ep.step(W, b, preds, lr)
        u0, u1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        u0.record(stream)
        for _ in range(args.steps):
            ep.step(W, b, preds, lr)
        u1.record(stream)
        stream.synchronize()
        return u0.elapsed_time(u1) / max(args.steps, 1)

    ms_cached = None if args.epochs_only else side_epochs(1 << 40)
    ms_uncached = None if args.epochs_only else side_epochs(0)
    for pp in preds:
        pp.version = 1 + epoch_no[0] // PRED_PERIOD

    # ---- end to end: host buffers in, host results out, every step ----
    hX = torch.from_numpy(np.ascontiguousarray(wl.X)).pin_memory()
    hlab = torch.from_numpy(labels_perm).pin_memory()
    hW = [torch.from_numpy(w.copy()).pin_memory() for w in wl.W]
    hb = [torch.from_numpy(x.copy()).pin_memory() for x in wl.b]
    # two sets of pinned result buffers: the host reads step i's results while step i + 1 is already queued
    h_loss = [torch.zeros(1, dtype=torch.float64).pin_memory() for _ in range(2)]
    h_gW = [[torch.zeros(w.shape, dtype=torch.float32).pin_memory() for w in wl.W] for _ in range(2)]
    lab_dev = ep.labels
    e2e_steps = max(3, min(args.steps, 50))   # the first step's input copy cannot overlap with anything: it is inside the timed region and amortises over the steps
    h2d = hX.numel() * 4 + hlab.numel() * hlab.element_size() + sum(w.numel() * 4 for w in hW) + sum(x.numel() * 4 for x in hb)
    d2h = 8 + sum(g.numel() * 4 for g in h_gW[0])

    # Pipelined like a training loop that streams its inputs: two sets of device input buffers; the inputs of step i + 1 are
    # copied from pinned host memory on a copy stream while step i computes; the step's results (loss, weight gradients)
    # are read back asynchronously into one of two pinned result sets; the host reads the results of step i while step i + 1 is
    # queued, and waits for a step before the buffers it used are overwritten.  Every step copies all
    # of its inputs and returns all of its results inside the timed region.
    copy_stream = torch.cuda.Stream(device=dev)
    X_dev2 = torch.zeros((X_dev.shape[0], (X_dev.shape[1] + 3) & ~3), dtype=torch.float32, device=dev)[:, :X_dev.shape[1]]  # padded rows like X_dev
    in_bufs = [(X_dev, lab_dev), (X_dev2, torch.empty_like(lab_dev))]
    w_bufs = [(W, b), ([torch.empty_like(t) for t in W], [torch.empty_like(t) for t in b])]
    ready = [torch.cuda.Event() for _ in range(2)]   # inputs of the step have landed
    done = [torch.cuda.Event() for _ in range(2)]    # the step that used the buffer set has finished
    for ev in done:
        ev.record(stream)

    def issue_copy(i):
        k = i & 1
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(done[k])
            in_bufs[k][0].copy_(hX, non_blocking=True)
            in_bufs[k][1].copy_(hlab, non_blocking=True)
            for d_, h_ in zip(w_bufs[k][0], hW):
                d_.copy_(h_, non_blocking=True)
            for d_, h_ in zip(w_bufs[k][1], hb):
                d_.copy_(h_, non_blocking=True)
            ready[k].record(copy_stream)

    seen = [0.0]

    def e2e_run(n):
        issue_copy(0)
        for i in range(n):
            k = i & 1
            if i + 1 < n:
                issue_copy(i + 1)
            stream.wait_event(ready[k])
            ep.set_inputs(*in_bufs[k])
            sat_epoch(w_bufs[k][0], w_bufs[k][1], None)
            h_loss[k].copy_(ep.loss_sum, non_blocking=True)
            for h_, d_ in zip(h_gW[k], ep.gW):
                h_.copy_(d_, non_blocking=True)
            done[k].record(stream)
            if i > 0:
                # the host takes delivery of the previous step's loss and gradients (a logging loop one step behind) while
                # this step runs: its launches are already queued, so the device does not wait for the host between steps
                done[k ^ 1].synchronize()
                seen[0] = float(h_loss[k ^ 1][0])
        stream.synchronize()
        seen[0] = float(h_loss[(n - 1) & 1][0])
        copy_stream.synchronize()

    e2e_run(2)
    barrier()
    t0 = time.perf_counter()
    e2e_run(e2e_steps)
    barrier()
    e2e_s = time.perf_counter() - t0
    e2e_loss = seen[0]
    clocks = sampler.stop()   # sampled from before the warm-up to the end of the end-to-end epochs: the GPU is under load throughout
    clocks["window"] = "warm-up + timed + end-to-end epochs"
    if not np.isfinite(e2e_loss) or not (0.5 * abs(loss) <= abs(e2e_loss) <= 2.0 * abs(loss)):
        raise RuntimeError(f"end-to-end path returned loss {e2e_loss}, device-resident path {loss}")

    # ---- predictor update of Algorithm 1 (not part of the epoch metric): one gradient step on the predictor objective per
    #      cached layer, between the pushes of an epoch and the commit ----
    pred_update = None
    if rank == 0 and wl.L > 1 and not args.epochs_only:
        ep.loss_sum.zero_()
        ep._forward_backward(B.SAT_ALL_PARTS, W, b, preds, 0, 0)
        first = ep.pred_update(preds, PRED_LR, max_steps=2, min_gain=0.0)      # warm-up (scratch allocation); reads the losses back
        B.sat_profile_enable(ep.ctx, True)
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_upd = 3
        l0 = B.sat_launch_count(ep.ctx)
        p0.record(stream)
        for _ in range(n_upd):
            ep.pred_update(preds, PRED_LR)
        p1.record(stream)
        stream.synchronize()
        upd_launches = (B.sat_launch_count(ep.ctx) - l0) // n_upd
        upd_fam = {k: v["ms"] / n_upd for k, v in B.sat_profile_read(ep.ctx).items() if v["calls"]}
        B.sat_profile_enable(ep.ctx, False)
        B.sat_cache_commit(ep.ctx)
        upd_ms = p0.elapsed_time(p1) / n_upd
        pred_update = dict(what="sat_pred_grad + SGD step on the five parameter arrays, for each of the cached layers "
                                "(forward with kept gates, loss against the pushed embeddings, back-propagation through time)",
                           ms=upd_ms, launches=int(upd_launches), period_epochs=PRED_PERIOD, ms_per_epoch_amortised=upd_ms / PRED_PERIOD,
                           loss_first_two_steps=[[float(x) for x in ls] for ls in first], kernel_families_ms=upd_fam)

    # ---- epochs with the gradient-side history (stale-gradient term of the Appendix's back-propagation; not part of the
    #      epoch metric) ----
    grad_history = None
    if rank == 0 and wl.L > 1 and args.extras:
        for _ in range(2):
            ep.step(W, b, preds, lr, grad_history=True)
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_gh = 5
        l0 = B.sat_launch_count(ep.ctx)
        g0.record(stream)
        for _ in range(n_gh):
            ep.step(W, b, preds, lr, grad_history=True)
        g1.record(stream)
        stream.synchronize()
        B.sat_profile_enable(ep.ctx, True)      # a second, bracketed pass for the per-family split
        for _ in range(n_gh):
            ep.step(W, b, preds, lr, grad_history=True)
        gh_fam = {k: v["ms"] / n_gh for k, v in B.sat_profile_read(ep.ctx).items() if v["calls"]}
        B.sat_profile_enable(ep.ctx, False)
        grad_history = dict(what="same epoch with SAT_BWD_GRAD_HISTORY on the layers >= 2: halo-row SpMM of D, per-partition adds "
                                 "into the history, gather + W^T contraction + add of the stale term on the boundary rows",
                            ms_per_epoch=g0.elapsed_time(g1) / n_gh, launches_per_epoch=int((B.sat_launch_count(ep.ctx) - l0) // n_gh),
                            history_bytes=int(sum(2 * ep.n_slots * ((d + 3) & ~3) * 4 for d in wl.dims[2:])),
                            kernel_families_ms=gh_fam)

    # ---- the same workload with graph-attention layers in place of the GCN layers (not part of the epoch metric; a first,
    #      untuned build of that backbone) ----
    gat = None
    if rank == 0 and wl.L > 1 and args.extras:
        grng = np.random.default_rng(5)
        gparams = []
        for l in range(wl.L):
            d_i, d_o = wl.dims[l], wl.dims[l + 1]
            gparams.append(dict(W=up((grng.standard_normal((d_i, d_o)) / np.sqrt(d_i)).astype(np.float32)),
                                a_src=up((grng.standard_normal(d_o) * 0.3).astype(np.float32)),
                                a_dst=up((grng.standard_normal(d_o) * 0.3).astype(np.float32)),
                                b=up(np.zeros(d_o, dtype=np.float32))))
        for _ in range(2):
            ep.step_gat(gparams, preds, lr)
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_ga = 5
        l0 = B.sat_launch_count(ep.ctx)
        a0.record(stream)
        for _ in range(n_ga):
            ep.step_gat(gparams, preds, lr)
        a1.record(stream)
        stream.synchronize()
        gat_ms = a0.elapsed_time(a1) / n_ga
        gat = dict(what="SAT epoch with single-head graph-attention layers (sat_gat_fwd / sat_gat_bwd) instead of GCN layers, same "
                        "pull / predict / push / loss / commit calls",
                   ms_per_epoch=gat_ms, edges_per_s=wl.nnz / (gat_ms * 1e-3), launches_per_epoch=int((B.sat_launch_count(ep.ctx) - l0) // n_ga),
                   loss=float(ep.loss_sum.item()))

    # ---- embedding codec on a ring snapshot (not part of the epoch metric; run last because it rewrites the snapshot) ----
    codec = None
    if rank == 0 and wl.L > 1 and args.extras:
        prec = 3
        B.sat_cache_requantise(ep.ctx, 1, 1, prec)          # warm-up (scratch allocation)
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record(stream)
        enc_bytes = B.sat_cache_requantise(ep.ctx, 1, 1, prec)
        c1.record(stream)
        stream.synchronize()
        raw = ep.n_slots * wl.dims[1] * 4
        codec_ms = c0.elapsed_time(c1)
        codec = dict(what="snapshot of cached layer 1 encoded and decoded in place (sat_cache_requantise: size pass, scan, "
                          "encode, decode)", precision=prec, raw_bytes=raw, encoded_bytes=int(enc_bytes), ratio=raw / max(enc_bytes, 1),
                     ms=codec_ms, gbs=(3 * raw + 2 * enc_bytes) / (codec_ms * 1e-3) / 1e9)

    # ---- max over ranks ----
    ms, e2e_s = max_over_ranks([ms, e2e_s], dist, dev)
    ms_per_step, value = whole_job_value(ms, args.steps, wl.nnz, world)
    e2e_value = world * wl.nnz * e2e_steps / e2e_s

    if rank == 0:
        peaks = measured_peaks()
        fam = top_family
        rec = prof_top[fam]     # measured inside the timed region
        per_launch_ms = rec["ms"] / max(rec["calls"], 1)
        traffic, traffic_src = ncu_traffic(wl.name if args.shrink == 1 else f"{wl.name}/{args.shrink}", fam)
        if fam.startswith("gemm") and fam != "gemm_side":   # gemm_side: K = h contractions with a streamed side operand (HBM-bound)
            tfl_alg = rec["flops"] / (rec["ms"] * 1e-3) / 1e12
            tfl = TF32_MMAS_PER_TERM * tfl_alg
            peak = peaks["bf16"] * TF32_OVER_BF16
            roofline = dict(kernel=fam, bound="tensor", achieved=tfl, peak=peak, unit="TFLOP/s", frac=tfl / peak,
                            achieved_2mnk=tfl_alg, frac_2mnk=tfl_alg / peak,
                            achieved_note="achieved / frac count the TF32 tensor flops issued = 3 x the method's 2mnk (two-term TF32 split, the "
                                          "price of the 1e-4 tolerance): the tensor pipe's utilisation; achieved_2mnk / frac_2mnk count the method's own flops",
                            peak_source=f"{peaks['source']} sustained bf16 {peaks['bf16']:.0f} TFLOP/s x nominal TF32/bf16 ratio {TF32_OVER_BF16:.3f}")
        else:
            gbs = rec["bytes"] / (rec["ms"] * 1e-3) / 1e9
            roofline = dict(kernel=fam, bound="hbm", achieved=gbs, peak=peaks["hbm"], unit="GB/s", frac=gbs / peaks["hbm"],
                            peak_source=f"{peaks['source']} HBM copy bandwidth")
        roofline.update(traffic=traffic, traffic_source=(f"profiles/{traffic_src}" if traffic_src else
                                                         "no ncu capture of this kernel on this workload is committed"),
                        launches=rec["calls"], ms_per_launch=per_launch_ms, share_of_step=rec["ms"] / ms)
        if fam.startswith("spmm") and rec["flops"] > 0:
            # the SpMM reads one neighbour row per entry: that stream comes mostly out of L2, not HBM; its rate is reported
            # beside the HBM figure (no roof is claimed for it)
            gather = rec["flops"] / 2.0 * 4.0 / (rec["ms"] * 1e-3) / 1e9
            roofline["l2_gather"] = dict(
                achieved=gather, unit="GB/s", reference=l2_gather_gbs, reference_stream=l2_stream_gbs, ratio=gather / l2_gather_gbs,
                what="neighbour-row bytes gathered per second (entries x row bytes / time) against the rate at which this GPU "
                     f"delivers random {l2_row}-float rows (reference) and a contiguous stream (reference_stream) out of an L2-resident "
                     "64 MiB buffer, both measured in this run (sat_profile_l2_rates); a ratio above 1 means rows served from L1 / shared memory")
        if fam == "spmm_fwd":
            roofline["walk"] = dict(by_width=spmm_plan,
                                    what="per input width of the forward aggregation: source blocks of the most finely cut partition "
                                         "(1 = rows walked once; > 1 = the partition is walked once per 64 MiB block of source rows and "
                                         "rows add one partial sum per block), work items and partial-sum rows per launch (sat_spmm_plan)")
        families = {k: dict(calls=v["calls"], ms_per_step=v["ms"] / args.steps,
                            gbs=(v["bytes"] / (v["ms"] * 1e-3) / 1e9) if v["ms"] > 0 else 0.0,
                            hbm_frac=(v["bytes"] / (v["ms"] * 1e-3) / 1e9 / peaks["hbm"]) if v["ms"] > 0 else 0.0,
                            tflops=(v["flops"] / (v["ms"] * 1e-3) / 1e12) if v["ms"] > 0 else 0.0)
                    for k, v in prof.items() if v["calls"]}
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            k = 4
            smp = OracleSample(wl, k)
            edges, secs = smp.run(list(smp.blocks))
            cpu = dict(value=edges / secs, unit="edges/s", cores=smp.cores, kind="oracle", seconds=secs,
                       sample=f"{len(smp.blocks)} x " + smp.describe() + f"; {edges} edges")
        # whole-epoch view: algorithmic bytes of every kernel family over the epoch time, against the HBM copy rate; the
        # SpMM families also as the gather rate they sustain (entries x row bytes / time)
        alg_bytes = sum(v["bytes"] for v in prof.values()) / args.steps
        epoch = dict(ms_median=float(np.median(step_ms)), ms_min=float(min(step_ms)), ms_max=float(max(step_ms)),
                     ms_with_events_on_every_family=ms_profiled,
                     ms_predictor_never_updated=ms_cached, ms_without_projection_cache=ms_uncached,
                     edge_passes_per_s=world * wl.nnz * 2 * wl.L / (ms_per_step * 1e-3),
                     algorithmic_bytes=alg_bytes, hbm_frac=alg_bytes / (ms_per_step * 1e-3) / 1e9 / peaks["hbm"],
                     spmm_gather_gbs={k: (prof[k]["flops"] / 2.0 * 4.0) / (prof[k]["ms"] * 1e-3) / 1e9
                                      for k in ("spmm_fwd", "spmm_bwd", "spmm_hrow") if prof.get(k, {}).get("ms", 0) > 0},
                     l2_stream_gbs=l2_stream_gbs, l2_random_row_gbs=l2_gather_gbs, l2_row_floats=l2_row)
        # the other configurations, briefly (device-resident epochs only; the headline above is the workload named in `config`)
        others = {}
        if world == 1 and args.others:
            ep.close()
            del X_dev, X_dev2, W, b, preds, in_bufs, w_bufs, hX
            torch.cuda.empty_cache()
            for name in [x for x in args.others.split(",") if x and x != wl.name]:
                try:
                    others[name] = side_workload(name, 5, peaks)
                except Exception as exc:      # a side table must not cost the headline line
                    others[name] = dict(error=f"{type(exc).__name__}: {exc}"[:300])
                torch.cuda.empty_cache()
        line = dict(metric="SAT epoch edges/s (fwd+bwd+predictor, P partitions)", value=value, unit="edges/s", n_gpus=world,
                    steps=args.steps, warmup=args.warmup, ms_per_step=ms_per_step, higher_is_better=True, scaling="weak",
                    vs_baseline=None, dtype="f32", data="synthetic", config=workload_config(wl),
                    e2e=dict(value=e2e_value, unit="edges/s", h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h, steps=e2e_steps,
                             loss=e2e_loss, pipelined="inputs of step i+1 copied on a second stream while step i computes; the host reads the results of step i while step i+1 is queued"),
                    gpu_launches=int(launches), clocks=clocks, roofline=roofline, cpu_baseline=cpu, epoch=epoch, pred_update=pred_update, grad_history=grad_history, gat=gat, codec=codec, kernel_families=families,
                    loss=loss, halo_rows=int(ep.nb), boundary_fraction=ep.n_slots / wl.n, other_workloads=others,
                    multi_gpu="replicas only" if world > 1 else None)
        print(json.dumps(line), flush=True)
    if ep.ctx is not None:
        ep.close()
    if dist is not None:
        dist.destroy_process_group()


def launch_ranks(n: int) -> int:
    """`python bench.py --gpus N` outside a launcher: start the N ranks on this node and hand back their exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large", choices=["tiny", "medium", "dense", "large", "multilabel", "odd"])
    ap.add_argument("--shrink", type=int, default=1)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--epochs-only", action="store_true",
                    help="skip the side measurements (predictor never updated / unversioned, predictor update)")
    ap.add_argument("--others", default="medium,multilabel,tiny",
                    help="comma-separated other configurations to run briefly for the side table of the line ('' = none; dense takes minutes to generate)")
    ap.add_argument("--extras", action="store_true",
                    help="also time the parts outside the epoch metric: gradient-side history, graph-attention backbone, embedding codec")
    args = ap.parse_args()
    if args.gpus < 1:
        ap.error("--gpus must be at least 1")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus > 1 and "RANK" not in os.environ:
        sys.exit(launch_ranks(args.gpus))
    if world != args.gpus:
        ap.error(f"--gpus {args.gpus} but the launcher started {world} rank(s)")
    from sat_synth import make_workload
    if args.impl == "reference" and int(os.environ.get("RANK", "0")) != 0:
        return
    wl = make_workload(args.workload, shrink=args.shrink)
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        if int(os.environ.get("LOCAL_RANK", "0")) == 0:
            from paper_2308_13466_b200.build import build
            build()
        run_ours(args, wl)


if __name__ == "__main__":
    main()
