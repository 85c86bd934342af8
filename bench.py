#!/usr/bin/env python
"""Benchmark of the BMU-search hot path (som_norms + som_bmu) on synthetic MeSH-shaped batches.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]

One step = one pass of the whole hot path over one batch: som_norms (norm pass) followed by
som_bmu (plan, fused search, combine/finalize).  Prints ONE JSON line on rank 0.

Without --config the graded map sizes are measured one after the other (64x64, 128x128, 512x512,
1024x1024): the line's own fields are those of the largest one (1024x1024, 125.8 GB codebook
resident in HBM, batches of 250 000 samples) and "per_config" carries one summary per size.
--config C measures that one configuration only.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_24067_b200 import synth  # noqa: E402

# Peak of the plain FP32 pipe that bounds the search: SMs x 128 lanes x max SM clock,
# one add per lane per clock (the search executes adds, no multiplies).
FP32_LANES_PER_SM = 128
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), float(d.get("sm_max_mhz", 1965.0)), "measured"
    return FALLBACK_HBM_GBS, 1965.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None
        self.t0 = self.t1 = None

    def begin(self):
        self.t0 = time.time()

    def end(self):
        self.t1 = time.time()

    def close(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.flush()
        rows = []
        import datetime
        for line in open(self.f.name):
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(parts[1]), float(parts[2]), parts[3], parts[4:9]))
            except Exception:
                continue
        os.unlink(self.f.name)
        inside = [r for r in rows if self.t0 is not None and self.t0 - 0.05 <= r[0] <= self.t1 + 0.05]
        use = inside if inside else rows
        if not use:
            return out
        out["samples"] = len(inside)
        out["sm_mhz"] = float(np.median([r[1] for r in use]))
        out["sm_max_mhz"] = float(use[0][2])
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = set()
        for r in use:
            for nm, val in zip(names, r[4][1:]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        out["reasons"] = sorted(reasons)
        return out


def _dist_env():
    ws = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    lr = int(os.environ.get("LOCAL_RANK", "0"))
    return ws, rank, lr


def replica_first_samples(rank: int, n_batches: int, batch: int):
    """First sample id of each batch of a rank: replicas draw disjoint parts of one sample stream."""
    return [(rank * n_batches + bi) * batch for bi in range(n_batches)]


def max_over_ranks(ms_local: float, dist, dev) -> float:
    """Timed region of the job = the slowest rank's (no-op without a process group)."""
    if dist is None:
        return float(ms_local)
    t = torch.tensor([ms_local], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_samples_per_s(world: int, batch: int, ms_per_step: float) -> float:
    """Whole-job throughput: every replica processed one batch per step."""
    return world * batch / (ms_per_step * 1e-3)


def _oracle_rate(w: synth.Workload, W_host_slab: np.ndarray, m_slab: int, indptr: np.ndarray,
                 indices: np.ndarray, target_s: float):
    """Time the CPU oracle on a bounded sample of the workload; returns (samples/s, description)."""
    from oracle import som_oracle as orc
    cores = orc.threads()
    nn = orc.norms(W_host_slab, w.V, m_slab)  # norm pass not timed (GPU arm reports it separately)
    n_probe = min(256, indptr.size - 1)
    t = time.perf_counter()
    orc.bmu(W_host_slab, w.V, m_slab, indptr[:n_probe + 1], indices, norms_=nn)
    dt = max(time.perf_counter() - t, 1e-6)
    n = int(max(n_probe, min(indptr.size - 1, n_probe * target_s / dt)))
    t = time.perf_counter()
    orc.bmu(W_host_slab, w.V, m_slab, indptr[:n + 1], indices, norms_=nn)
    dt = time.perf_counter() - t
    rate = n / dt * (m_slab / w.M)
    desc = "first %d samples of the batch x %d of %d neurons (rate scaled by the neuron fraction), %d threads" % (
        n, m_slab, w.M, cores)
    return rate, cores, desc, dt


def config_dict(w: synth.Workload, world: int, step: str, store_bytes: int = 4) -> dict:
    """The workload as both arms name it (nominal figures only, so that the two arms print the same)."""
    n_batches = max(1, min(4, w.N // w.batch))
    return {"workload": w.name, "V": w.V, "M": w.M, "batch": w.batch, "batches": n_batches,
            "mean_nnz": 1.0 + w.lam, "step": step, "replicas": world,
            "l2_policy": "inputs larger than L2 (codebook %.0f MB + CSR %.0f MB per step)" % (
                w.V * w.M * store_bytes / 1e6, w.batch * (1.0 + w.lam) * 4 / 1e6)
            if w.V * w.M * store_bytes > 126e6 else
            "inputs smaller than L2: steps rotate over %d distinct batches, no flush" % n_batches}


DEFAULT_STEP = "som_norms + som_bmu on one batch"


def run_reference(args, w: synth.Workload):
    """The CPU oracle as it stands, timed on host cores.  Every step is one bounded sample of the
    workload (the first samples of a batch against the first 4096 neurons of the configured
    codebook); `ms_per_step` is the measured time of such a step, `value` the rate it implies for
    the whole map (scaled by the neuron fraction)."""
    ws, rank, _ = _dist_env()
    if rank != 0:
        return
    m_slab = min(w.M, 4096)
    W_host = synth.codebook_slab(w.V, w.M, 0, m_slab, w.seed).numpy()
    n_gen = min(w.batch, 200_000)
    b = synth.sample_csr(n_gen, w.V, w.lam, w.seed)
    indptr, indices = b.indptr.numpy(), b.indices.numpy()
    per_step = max(0.5, min(10.0, 100.0 / max(1, args.steps + args.warmup)))
    rates, times, desc, cores = [], [], "", 1
    for i in range(args.warmup + args.steps):
        rate, cores, desc, dt = _oracle_rate(w, W_host, m_slab, indptr, indices, per_step)
        if i >= args.warmup:
            rates.append(rate)
            times.append(dt)
    value = float(np.mean(rates))
    line = {
        "impl": "reference", "metric": "bmu_samples_per_s", "value": value, "unit": "samples/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1000.0 * float(np.mean(times)),
        "ms_per_step_is": "measured time of one bounded oracle sample (cpu_baseline.sample), not of a whole batch",
        "ms_per_whole_batch_at_this_rate": 1000.0 * w.batch / value,
        "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(w, ws, DEFAULT_STEP),
        "cpu_baseline": {"value": value, "unit": "samples/s", "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "samples/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


class Ctx:
    """What every measured configuration shares: device, process group, peaks."""

    def __init__(self):
        self.ws, self.rank, self.lr = _dist_env()
        if not torch.cuda.is_available():
            raise SystemExit("bench.py: no CUDA device; the hot path has no CPU fallback")
        torch.cuda.set_device(self.lr)
        self.dev = torch.device("cuda", self.lr)
        self.dist = None
        if self.ws > 1:
            import torch.distributed as dist_mod
            self.dist = dist_mod
            self.dist.init_process_group("nccl", device_id=self.dev)
        from paper_2608_24067_b200 import som
        self.som = som
        self.hbm_gbs, self.sm_max_mhz, self.peak_src = _peaks()
        self.sm_count = torch.cuda.get_device_properties(self.dev).multi_processor_count
        self.add_peak = self.sm_count * FP32_LANES_PER_SM * self.sm_max_mhz * 1e6  # adds/s, derived
        # the same peak measured: independent FP32 add chains, nothing else (library microbenchmark)
        self.add_peak_measured = som.measure_fadd_peak(self.dev)
        # bytes per clock and SM along the paths an add's operand takes (shared memory, L2): what the search
        # kernel's time per sample is made of (library microbenchmark, about 40 ms)
        self.operand_paths = som.measure_operand_paths(self.dev)

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        torch.cuda.synchronize()

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()


def _committed_traffic(workload_name: str):
    """DRAM bytes per launch of the search kernel from the committed ncu summary of this workload
    (profiles/k_bmu_table_<workload>.md, a line `traffic_bytes_per_launch = ...`), or None."""
    tpath = os.path.join(ROOT, "profiles", "k_bmu_table_%s.md" % workload_name)
    if os.path.exists(tpath):
        for tl in open(tpath):
            if tl.startswith("traffic_bytes_per_launch"):
                return float(tl.split("=")[1])
    return None


def measure(ctx: Ctx, args, w: synth.Workload, steps: int, warmup: int, cpu_seconds: float) -> dict:
    """One configuration: device-resident throughput, end to end, two-stage leg, CPU baseline."""
    som, dev, dist, ws, rank = ctx.som, ctx.dev, ctx.dist, ctx.ws, ctx.rank
    hbm_gbs, add_peak = ctx.hbm_gbs, ctx.add_peak
    barrier = ctx.barrier

    # ---- inputs (synthetic, resident in HBM) -------------------------------------------------
    store_bytes = 2 if args.store == "f16" else 4
    W = torch.empty(w.V * w.M, dtype=torch.float16 if args.store == "f16" else torch.float32, device=dev)
    synth.fill_codebook(w.V, w.M, w.seed, out=W)
    n_batches = max(1, min(4, w.N // w.batch))
    batches = []
    for first in replica_first_samples(rank, n_batches, w.batch):  # each replica gets its own samples
        batches.append(synth.sample_csr(w.batch, w.V, w.lam, w.seed, zipf_s=w.zipf_s, device=dev,
                                        first_sample=first))
    nnz_mean = float(np.mean([b.nnz / b.n for b in batches]))
    h = som.Som(w.V, w.M, W)
    if args.variant is not None:
        h.set_option(0, args.variant)
    if args.hot_rows:
        h.set_option(1, args.hot_rows)
    if args.threads:
        h.set_option(2, args.threads)
    if args.lane_neurons:
        h.set_option(3, args.lane_neurons)
    if args.parts:
        h.set_option(4, args.parts)
    if args.update_mib:
        h.set_option(6, args.update_mib)
    if args.two_stage:
        h.set_option(7, 1)
    epoch_edge = int(round(w.M ** 0.5))
    if args.epoch and epoch_edge * epoch_edge != w.M:
        raise SystemExit("bench.py --epoch needs a square lattice")
    plans = [h.plan(b.indptr, b.indices) for b in batches] if (args.planned or args.epoch) else []
    sample_values = []
    if args.values:
        for bi, b in enumerate(batches):
            k = torch.arange(b.nnz, dtype=torch.int64, device=dev)
            sample_values.append(synth._u24_to_f32(synth.hash32(w.seed + 17, 5, k, bi), 0.25, 1.5))
    out_bmu = torch.empty(w.batch, dtype=torch.int32, device=dev)
    out_dist = torch.empty(w.batch, dtype=torch.float32, device=dev)

    def step(i):
        b = batches[i % n_batches]
        h.norms()
        if args.epoch:
            plans[i % n_batches].bmu(out_bmu, out_dist)
            h.update(epoch_edge, epoch_edge, b.indptr, b.indices, out_bmu,
                     args.radius if args.radius > 0 else max(1, epoch_edge // 4))
        elif args.planned:
            plans[i % n_batches].bmu(out_bmu, out_dist)
        elif args.values:
            h.bmu_values(b.indptr, b.indices, sample_values[i % n_batches])
        elif args.top2:
            h.bmu2(b.indptr, b.indices)
        else:
            h.bmu(b.indptr, b.indices, out_bmu, out_dist)

    # ---- device-resident timing -------------------------------------------------------------
    for i in range(warmup):
        step(i)
    barrier()
    sampler = ClockSampler(ctx.lr) if rank == 0 else None
    h.set_timing(True)
    l0 = h.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    if sampler:
        sampler.begin()
    e0.record()
    for i in range(steps):
        step(warmup + i)
    e1.record()
    barrier()
    if sampler:
        sampler.end()
    ms_total = e0.elapsed_time(e1)
    launches = h.launch_count() - l0
    phases = h.get_timing()
    h.set_timing(False)
    ms_total = max_over_ranks(ms_total, dist, dev)
    ms_per_step = ms_total / steps
    value = aggregate_samples_per_s(ws, w.batch, ms_per_step)

    # ---- end to end through the host entry point --------------------------------------------
    hb = [(b.indptr.cpu().pin_memory(), b.indices.cpu().pin_memory()) for b in batches]
    e2e_steps = max(1, min(steps, 5))

    # Streamed through som_bmu_host_async: every step uploads its batch and downloads both outputs;
    # the handle overlaps one step's copies with its neighbours' searches.  The timed region ends
    # after som_host_sync, when the last step's results are in host memory.
    h_outs = [(torch.empty(w.batch, dtype=torch.int32).pin_memory(),
               torch.empty(w.batch, dtype=torch.float32).pin_memory()) for _ in range(2)]

    def e2e_step(i):
        ip, ix = hb[i % n_batches]
        ob, od = h_outs[i % 2]
        h.norms()
        h.bmu_host_async(ip, ix, ob, od)

    for i in range(2):  # both staging buffers get allocated outside the timed region
        e2e_step(i)
    h.host_sync()
    barrier()
    e0.record()
    for i in range(e2e_steps):
        e2e_step(i + 2)
    h.host_sync()   # the last results are in host memory; only now is the closing event recorded
    e1.record()
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1) / e2e_steps, dist, dev)
    e2e_value = aggregate_samples_per_s(ws, w.batch, e2e_ms)
    h2d = int(np.mean([ip.numel() * 4 + ix.numel() * 4 for ip, ix in hb]))
    d2h = w.batch * 8
    # the blocking form of the same call: upload, search, download, wait; one step at a time
    ip0, ix0 = hb[0]
    h.norms()
    h.bmu_host(ip0, ix0, h_outs[0][0], h_outs[0][1])  # staging buffer allocated outside the timed region
    barrier()
    blk_steps = max(1, min(steps, 3))
    e0.record()
    for i in range(blk_steps):
        h.norms()
        h.bmu_host(hb[i % n_batches][0], hb[i % n_batches][1], h_outs[0][0], h_outs[0][1])
    e1.record()
    barrier()
    blocking_ms = max_over_ranks(e0.elapsed_time(e1) / blk_steps, dist, dev)

    clocks = sampler.close() if sampler else None

    # ---- the same step with the two-stage search (library option 7), reported beside the headline ----
    two_stage = None
    if (args.store == "f32" and w.M % 128 == 0 and not args.top2 and not args.two_stage and not args.values
            and not args.epoch and not args.no_two_stage_leg):
        free_b, _ = torch.cuda.mem_get_info()
        if free_b > w.V * w.M * 2 + (4 << 30):
            try:
                h2 = som.Som(w.V, w.M, W)
                if args.variant is not None:
                    h2.set_option(0, args.variant)
                h2.set_option(7, 1)

                def step2(i):
                    b = batches[i % n_batches]
                    h2.norms()
                    h2.bmu(b.indptr, b.indices, out_bmu, out_dist)

                for i in range(warmup):
                    step2(i)
                barrier()
                h2.set_timing(True)
                e0.record()
                for i in range(steps):
                    step2(warmup + i)
                e1.record()
                barrier()
                ms2 = max_over_ranks(e0.elapsed_time(e1) / steps, dist, dev)
                ph2 = h2.get_timing()
                adds2 = w.batch * nnz_mean * w.M
                two_stage = {"value": aggregate_samples_per_s(ws, w.batch, ms2), "unit": "samples/s",
                             "ms_per_step": ms2, "search_ms": ph2["search_ms"],
                             "frac": adds2 / (max(ph2["search_ms"], 1e-6) * 1e-3) / add_peak,
                             "uncertain_samples_last_call": h2.last_uncertain(),
                             "extra_device_bytes": w.V * w.M * 2,
                             "note": "first pass over an fp16 copy of the codebook, certified per sample; "
                                     "uncertain samples searched again with the fp32 weights"}
                h2.destroy()
            except som.SomError as exc:  # e.g. no memory for the copy
                two_stage = {"unavailable": str(exc)}
        else:
            two_stage = {"unavailable": "no device memory for the fp16 copy of the codebook (%.1f GB)"
                                        % (w.V * w.M * 2 / 1e9)}

    # ---- optional: the update phase of an epoch, timed on its own -----------------------------
    update = None
    edge = int(round(w.M ** 0.5))
    if args.with_update and edge * edge == w.M:
        b0 = batches[0]
        h.norms()
        bm, _ = h.bmu(b0.indptr, b0.indices)
        radius = args.radius if args.radius > 0 else max(1, edge // 4)
        h.update(edge, edge, b0.indptr, b0.indices, bm, radius)  # warm-up (allocates the workspace)
        barrier()
        u_steps = max(1, min(steps, 5))
        e0.record()
        for _ in range(u_steps):
            h.update(edge, edge, b0.indptr, b0.indices, bm, radius)
        e1.record()
        barrier()
        u_ms = max_over_ranks(e0.elapsed_time(e1) / u_steps, dist, dev)
        u_bytes = w.V * w.M * store_bytes + b0.nnz * 4 + (b0.n + 1) * 4 + b0.n * 4  # write W, read CSR + bmu
        update = {"ms": u_ms, "lattice": [edge, edge], "radius": radius, "algorithmic_bytes": u_bytes,
                  "hbm_frac": u_bytes / (u_ms * 1e-3) / (hbm_gbs * 1e9),
                  "share_of_epoch": u_ms / (u_ms + ms_per_step)}
        h.norms()

    line = None
    if rank == 0:
        # ---- roofline of the dominant kernel (the fused search) ---------------------------------
        adds = w.batch * nnz_mean * w.M  # nominal neuron-feature accumulations per launch
        search_s = max(phases["search_ms"], 1e-6) * 1e-3
        achieved = adds / search_s
        alg_bytes = (w.V * w.M * store_bytes + sum(b.nnz * 4 + (b.n + 1) * 4 for b in batches) / n_batches
                     + w.batch * 8)
        # DRAM bytes one launch of the search kernel really moves, from the committed ncu capture of
        # this workload's shipped kernel (None when there is none: the large maps are not captured
        # with full counter sets, their algorithmic bytes stand in and the key stays null)
        traffic = _committed_traffic(w.name) if args.store == "f32" else None
        t_alu = adds / add_peak
        t_hbm = (traffic if traffic is not None else alg_bytes) / (hbm_gbs * 1e9)
        roofline = {
            "bound": "alu" if t_alu >= t_hbm else "hbm", "kernel": "fused BMU search",
            "achieved": achieved / 1e12, "peak": add_peak / 1e12,
            "unit": "TFLOP/s", "frac": max(t_alu, t_hbm) / search_s, "traffic": traffic,
            # achieved and frac count the adds of the plain definition (every row of every sample against every
            # neuron) over the measured time; where the kernel prunes (bit-identical outputs) it executes only
            # part of them, so frac is the job done against the add pipe's peak, not the pipe's load, and can pass 1
            "frac_note": "algorithmic adds of the full product / time; the pruning kernel executes a fraction of them",
            "traffic_note": None if traffic is not None else "not measured at this size; hbm term uses the algorithmic bytes",
            "peak_source": "%d SMs x %d fp32 lanes x %.0f MHz (%s clock); adds only, no multiplies" % (
                ctx.sm_count, FP32_LANES_PER_SM, ctx.sm_max_mhz, ctx.peak_src),
            "peak_measured": ctx.add_peak_measured / 1e12,
            "frac_of_measured_peak": achieved / ctx.add_peak_measured if ctx.add_peak_measured > 0 else None,
            "alu_time_at_peak_ms": t_alu * 1e3, "hbm_time_at_peak_ms": t_hbm * 1e3,
            "search_ms": phases["search_ms"], "algorithmic_bytes": alg_bytes, "hbm_peak_gbs": hbm_gbs,
            "mean_nnz_measured": nnz_mean,
            "norms_ms": phases["norms_ms"],
            "norms_hbm_frac": (w.V * w.M * store_bytes / max(phases["norms_ms"], 1e-6) / 1e6) / hbm_gbs,
            "plan_ms": phases["plan_ms"], "finalize_ms": phases["finalize_ms"],
            "step_frac_of_alu_roofline": (adds / add_peak) / (ms_per_step * 1e-3),
            # operand delivery, the unit that really bounds the kernel: measured bytes per clock and SM from
            # shared memory (hot rows) and from L2 (tail rows), and the search's SM clocks per sample and 128 neurons
            "operand_paths_bytes_per_clk_per_sm": ctx.operand_paths,
            "sm_clk_per_sample_and_128_neurons": search_s * ctx.sm_max_mhz * 1e6 * ctx.sm_count / (w.batch * w.M / 128.0),
        }

        # ---- CPU baseline: the oracle on a bounded sample, rank 0, N=1 only ------------------
        cpu = None
        if ws == 1 and not args.no_cpu_baseline and cpu_seconds > 0:
            m_slab = min(w.M, 4096)
            Wh = W.view(w.V, w.M)[:, :m_slab].float().contiguous().cpu().numpy()
            b = batches[0]
            n_take = min(b.n, 100_000)
            ip = b.indptr[:n_take + 1].cpu().numpy()
            ix = b.indices[:int(b.indptr[n_take])].cpu().numpy()
            rate, cores, desc, _ = _oracle_rate(w, Wh, m_slab, ip, ix, cpu_seconds)
            cpu = {"value": rate, "unit": "samples/s", "cores": cores, "kind": "oracle", "sample": desc}

        step_name = ("som_norms + " + ("som_bmu_planned + som_update (a training-epoch step; plans built once, outside)"
                                       if args.epoch else
                                       "som_bmu_planned (plans built once, outside)" if args.planned else
                                       ("som_bmu_values" if args.values else ("som_bmu2" if args.top2 else "som_bmu")))
                     + " on one batch")
        line = {
            "metric": "bmu_samples_per_s", "value": value, "unit": "samples/s", "n_gpus": ws,
            "steps": steps, "warmup": warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if args.store == "f32" else "f32 accumulate, f16-stored codebook",
            "data": "synthetic",
            "config": config_dict(w, ws, step_name, store_bytes),
            "accumulations_per_s": ws * adds / (ms_per_step * 1e-3),
            "roofline": roofline,
            "cpu_baseline": cpu,
            "e2e": {"value": e2e_value, "unit": "samples/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_ms, "blocking_ms_per_step": blocking_ms,
                    "path": "som_norms + som_bmu_host_async / som_host_sync (binary samples, best unit) on the same "
                            "batches, copies overlapped with the neighbouring steps; blocking_ms_per_step is "
                            "som_norms + som_bmu_host, one step at a time"},
            "gpu_launches": int(launches),
            "clocks": clocks,
        }
        if update is not None:
            line["update"] = update
        if args.two_stage:
            line["two_stage"] = {"uncertain_samples_last_call": h.last_uncertain(), "batch": w.batch}
        elif two_stage is not None:
            line["two_stage"] = two_stage
    for p_ in plans:
        p_.destroy()
    h.destroy()
    del W, batches, hb, h_outs, out_bmu, out_dist, plans, sample_values
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    return line


def _summary(line: dict) -> dict:
    r = line["roofline"]
    return {"workload": line["config"]["workload"], "batch": line["config"]["batch"], "steps": line["steps"],
            "warmup": line["warmup"], "ms_per_step": line["ms_per_step"], "value": line["value"],
            "accumulations_per_s": line["accumulations_per_s"],
            "roofline": {"bound": r["bound"], "frac": r["frac"], "frac_of_measured_peak": r["frac_of_measured_peak"],
                         "achieved": r["achieved"], "traffic": r["traffic"],
                         "sm_clk_per_sample_and_128_neurons": r["sm_clk_per_sample_and_128_neurons"]},
            "search_ms": r["search_ms"], "norms_ms": r["norms_ms"], "norms_hbm_frac": r["norms_hbm_frac"],
            "plan_ms": r["plan_ms"], "finalize_ms": r["finalize_ms"],
            "e2e": {k: line["e2e"][k] for k in ("value", "ms_per_step", "blocking_ms_per_step",
                                                 "h2d_bytes_per_step", "d2h_bytes_per_step")},
            "two_stage": ({k: line["two_stage"].get(k) for k in ("value", "search_ms", "frac", "unavailable")
                           if k in line["two_stage"]} if line.get("two_stage") else None),
            "cpu_baseline": line["cpu_baseline"], "gpu_launches": line["gpu_launches"], "clocks": line["clocks"]}


def _cap_steps(w: synth.Workload, steps: int, warmup: int):
    """Steps and warm-ups of one size in the all-sizes run: the driver's counts, cut where the timed
    region of a size would pass about a minute (steps of the two largest maps take 0.3 to 0.6 s)."""
    est_ms = w.batch * (1.0 + w.lam) * w.M / 37.2e12 / 0.15 * 1e3 + w.V * w.M * 4 / 6.4e12 * 1e3
    cap = max(3, int(60_000.0 / max(est_ms, 1e-3)))
    return min(steps, cap), max(3, min(warmup, max(3, cap // 4)))


def run_ours(args, workloads):
    ctx = Ctx()
    lines = []
    for k, w in enumerate(workloads):
        last = k == len(workloads) - 1
        if len(workloads) > 1:
            steps, warmup = _cap_steps(w, args.steps, args.warmup)
        else:
            steps, warmup = args.steps, args.warmup
        lines.append(measure(ctx, args, w, steps, warmup, 12.0 if last else 5.0))
    if ctx.rank == 0:
        line = lines[-1]
        if len(lines) > 1:
            line["per_config"] = [_summary(x) for x in lines]
            line["steps_requested"] = args.steps
            line["warmup_requested"] = args.warmup
            if (line["steps"], line["warmup"]) != (args.steps, args.warmup):
                line["steps_note"] = ("steps / warm-ups of a size are cut where its timed region would pass "
                                      "about a minute; the counts used are in each per_config entry")
        print(json.dumps(line), flush=True)
    ctx.close()


def run_tc_probe(args):
    """Go / no-go microbenchmark of the densified hot-feature tile on tcgen05 (library call som_tc_probe):
    cycles per tile of 128 samples x 64 neurons for building the 0/1 tile, the MMAs and the drain, alone and
    pipelined, on every SM at once, with membership bits of the workload's H most frequent features."""
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device")
    from paper_2608_24067_b200 import som
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    w = synth.CONFIGS[2]
    n_tiles, repeats = 64, 40
    b = synth.sample_csr(n_tiles * 128, w.V, w.lam, w.seed, device="cpu")
    ip, ix = b.indptr.numpy().astype(np.int64), b.indices.numpy()
    row = np.repeat(np.arange(b.n), np.diff(ip))
    rng = np.random.default_rng(0)
    results = []
    modes = [(1, "build"), (2, "mma"), (4, "drain"), (6, "mma+drain"), (7, "build+mma+drain"),
             (15, "build+mma+drain+redistribute"), (16, "lds"), (18, "mma+lds")]
    for H in (32, 64, 128, 256):
        # the workload's ids are frequency ranks: the H most frequent features are ids 0 .. H-1
        sel = ix < H
        words = np.zeros((b.n, H // 32), np.uint32)
        np.bitwise_or.at(words, (row[sel], ix[sel] // 32), (np.uint32(1) << (ix[sel] % 32).astype(np.uint32)))
        inst = float(sel.sum()) / b.n
        rows = (rng.random((H, 64)) * 0.05).astype(np.float32)
        hnorm = (17.0 + rng.random(64)).astype(np.float32)
        member = ((words[:128, :, None] >> np.arange(32, dtype=np.uint32)[None, None, :]) & 1).reshape(128, H)
        want = hnorm.astype(np.float64)[None, :] - member.astype(np.float64) @ rows.astype(np.float64)
        d_rows, d_h = torch.from_numpy(rows).to(dev), torch.from_numpy(hnorm).to(dev)
        d_bits = torch.from_numpy(words.view(np.int32)).to(dev)
        for terms in (1, 2):
            entry = {"H": H, "terms": terms, "dense_instances_per_sample": inst, "cycles_per_tile": {}}
            for mode, name in modes:
                som.tc_probe(d_rows, d_h, d_bits, H, terms, n_tiles, mode, 2, sms)  # warm-up
                r = som.tc_probe(d_rows, d_h, d_bits, H, terms, n_tiles, mode, repeats, sms)
                torch.cuda.synchronize()
                if int(r["status"].item()) != 0:
                    raise SystemExit("tc probe: a bounded wait gave up (H=%d terms=%d mode=%d)" % (H, terms, mode))
                cyc = float(r["cycles"].double().mean().item()) / (n_tiles * repeats)
                entry["cycles_per_tile"][name] = cyc
                if mode == 7:
                    entry["max_abs_err_first_tile"] = float(np.abs(r["out"].cpu().numpy() - want).max())
                    entry["pairs_per_clk_per_sm"] = 128 * 64 / cyc
            results.append(entry)
    print(json.dumps({"tc_probe": results, "tile": "128 samples x 64 neurons", "blocks": sms,
                      "note": "cycles per tile, mean over blocks, every SM busy; membership of the 128x128 "
                              "workload's H most frequent features"}), flush=True)


def run_operand_probe():
    """Bytes per clock and SM along the paths an operand takes into a register (library microbenchmark), and
    what they make of a sample of the headline workload: clocks per sample and 128-neuron range if every hot
    row came at the shared-memory rate and every tail row at the L2 rate, one after the other."""
    from paper_2608_24067_b200 import som
    som.load_library()
    torch.cuda.set_device(0)
    p = som.measure_operand_paths()
    # rows per sample of the MeSH-shaped batches with the 368-row table (hot rows as issued, i.e. padded to the
    # warp's longest list, and prefix rebuilds; tail rows), by batch size and its number of mask features
    mix = {"250k samples, 9 mask features": (4.85, 3.92), "1M samples, 11": (4.60, 3.93), "4M samples, 13": (4.40, 3.93)}
    model = {}
    for name, (hot_rows, tail_rows) in mix.items():
        t_sh, t_l2 = 512.0 * hot_rows / p["shared"], 512.0 * tail_rows / p["l2_global"]
        model[name] = {"hot_rows": hot_rows, "tail_rows": tail_rows, "clk_shared": t_sh, "clk_l2": t_l2,
                       "clk_one_after_the_other": t_sh + t_l2, "clk_fully_overlapped": max(t_sh, t_l2),
                       "clk_at_the_probe's_two-stream_rate": 512.0 * (hot_rows + tail_rows) / p["shared_and_l2"]}
    print(json.dumps({"probe": "operand paths, 512-byte rows, eight lanes per row, one 512-thread block per SM",
                      "bytes_per_clk_per_sm": p, "model_clk_per_sample_and_128_neuron_range": model}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=None,
                    help="index into the five workloads; default: the four graded map sizes (1..4) one after "
                         "the other, headline = the largest (1024x1024)")
    ap.add_argument("--variant", type=int, default=None, help="search kernel variant (library option 0)")
    ap.add_argument("--hot-rows", type=int, default=0, help="row-table kernel: hot rows in shared memory")
    ap.add_argument("--threads", type=int, default=0, help="row-table kernel: block size (512 or 1024)")
    ap.add_argument("--lane-neurons", type=int, default=0, help="row-table kernel: neurons per lane (4 or 8)")
    ap.add_argument("--parts", type=int, default=0, help="row-table kernel: most sample parts per neuron range")
    ap.add_argument("--features", default="zipf", choices=["zipf", "uniform"],
                    help="feature popularity of the samples: the workload's Zipf law, or the stress variant "
                         "with features uniform over V (no sharing between samples)")
    ap.add_argument("--zipf-s", type=float, default=None,
                    help="override the Zipf exponent of the feature popularity (0 = uniform)")
    ap.add_argument("--store", default="f32", choices=["f32", "f16"],
                    help="codebook storage: fp32 (the configurations) or fp16 with fp32 accumulation")
    ap.add_argument("--with-update", action="store_true",
                    help="also time som_update (the batch update that follows the search in an epoch) "
                         "on a square lattice and report it under \"update\"")
    ap.add_argument("--update-mib", type=int, default=0, help="som_update: workspace budget in MiB (library option 6)")
    ap.add_argument("--two-stage", action="store_true",
                    help="fp32 storage: certified first pass over an fp16 copy, exact second pass (library option 7)")
    ap.add_argument("--no-two-stage-leg", action="store_true",
                    help="skip the extra measurement of the two-stage search that the default run reports beside the headline")
    ap.add_argument("--values", action="store_true",
                    help="time som_bmu_values (sparse real-valued samples: seeded values in [0.25, 1.75)) instead of som_bmu")
    ap.add_argument("--epoch", action="store_true",
                    help="time a whole training-epoch step on a square lattice: som_norms + som_bmu_planned + "
                         "som_update (radius = edge / 4); implies --planned")
    ap.add_argument("--planned", action="store_true",
                    help="epoch-loop mode: the batches' plans are built once (som_plan_create) outside the timed "
                         "region and every step runs som_norms + som_bmu_planned")
    ap.add_argument("--top2", action="store_true",
                    help="time som_bmu2 (best and second-best unit) instead of som_bmu")
    ap.add_argument("--radius", type=int, default=0, help="som_update: blur radius (default edge / 4)")
    ap.add_argument("--batch", type=int, default=0,
                    help="samples per batch instead of the configuration's (a sweep variant, named in the workload)")
    ap.add_argument("--V", type=int, default=0,
                    help="features instead of the configuration's 30 000 (a smaller variant of the same map for "
                         "profiler captures that must hold few GB; named in the workload)")
    ap.add_argument("--tc-probe", action="store_true",
                    help="run the tcgen05 microbenchmark of the densified hot-feature tile and print its numbers")
    ap.add_argument("--operand-probe", action="store_true",
                    help="run the microbenchmark of the operand paths (shared memory, L2 by global loads, both, "
                         "L2 by texture fetches: bytes per clock and SM) and print its numbers")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.tc_probe:
        run_tc_probe(args)
        return
    if args.operand_probe:
        run_operand_probe()
        return

    def variant_of(w):
        if args.features == "uniform":
            w = dataclasses.replace(w, name=w.name + "-uniform", zipf_s=0.0)
        if args.batch > 0:
            w = dataclasses.replace(w, name="%s-batch%d" % (w.name, args.batch), batch=args.batch,
                                    N=max(w.N, args.batch))
        if args.V > 0:
            w = dataclasses.replace(w, name="%s-V%d" % (w.name, args.V), V=args.V)
        if args.zipf_s is not None:
            w = dataclasses.replace(w, name="%s-zipf%g" % (w.name, args.zipf_s), zipf_s=args.zipf_s)
        if args.store == "f16":
            w = dataclasses.replace(w, name=w.name + "-f16")
        return w

    plain = not (args.epoch or args.planned or args.values or args.top2 or args.with_update or args.two_stage)
    if args.config is None:
        ids = [1, 2, 3, 4] if plain else [1]
    else:
        ids = [args.config]
    workloads = [variant_of(synth.CONFIGS[i]) for i in ids]
    if args.impl == "reference":
        run_reference(args, workloads[-1])
    else:
        run_ours(args, workloads)


if __name__ == "__main__":
    main()
