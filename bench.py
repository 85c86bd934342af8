#!/usr/bin/env python
"""Benchmark of the BMU-search hot path (som_norms + som_bmu) on synthetic MeSH-shaped batches.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]

One step = one pass of the whole hot path over one batch: som_norms (norm pass) followed by
som_bmu (plan, fused search, combine/finalize).  Prints ONE JSON line on rank 0.
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


def run_reference(args, w: synth.Workload):
    """The CPU oracle as it stands, timed on host cores, on bounded samples of the workload."""
    ws, rank, _ = _dist_env()
    if rank != 0:
        return
    m_slab = min(w.M, 4096)
    # the slab is the first m_slab neurons of the configured codebook
    W_host = synth.codebook_slab(w.V, w.M, 0, m_slab, w.seed).numpy()
    n_gen = min(w.batch, 200_000)
    b = synth.sample_csr(n_gen, w.V, w.lam, w.seed)
    indptr, indices = b.indptr.numpy(), b.indices.numpy()
    per_step = max(1.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    rates, desc, cores = [], "", 1
    for i in range(args.warmup + args.steps):
        rate, cores, desc, dt = _oracle_rate(w, W_host, m_slab, indptr, indices, per_step)
        if i >= args.warmup:
            rates.append(rate)
    value = float(np.mean(rates))
    line = {
        "impl": "reference", "metric": "bmu_samples_per_s", "value": value, "unit": "samples/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1000.0 * w.batch / value, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "V": w.V, "M": w.M, "batch": w.batch, "mean_nnz": 1 + w.lam},
        "cpu_baseline": {"value": value, "unit": "samples/s", "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "samples/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_ours(args, w: synth.Workload):
    ws, rank, lr = _dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the hot path has no CPU fallback")
    torch.cuda.set_device(lr)
    dev = torch.device("cuda", lr)
    dist = None
    if ws > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)
    from paper_2608_24067_b200 import som

    hbm_gbs, sm_max_mhz, peak_src = _peaks()
    sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
    add_peak = sm_count * FP32_LANES_PER_SM * sm_max_mhz * 1e6  # adds/s

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

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing -------------------------------------------------------------
    for i in range(args.warmup):
        step(i)
    barrier()
    sampler = ClockSampler(lr) if rank == 0 else None
    h.set_timing(True)
    l0 = h.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    if sampler:
        sampler.begin()
    e0.record()
    for i in range(args.steps):
        step(args.warmup + i)
    e1.record()
    barrier()
    if sampler:
        sampler.end()
    ms_total = e0.elapsed_time(e1)
    launches = h.launch_count() - l0
    phases = h.get_timing()
    h.set_timing(False)
    ms_total = max_over_ranks(ms_total, dist, dev)
    ms_per_step = ms_total / args.steps
    value = aggregate_samples_per_s(ws, w.batch, ms_per_step)

    # ---- end to end through the host entry point --------------------------------------------
    hb = [(b.indptr.cpu().pin_memory(), b.indices.cpu().pin_memory()) for b in batches]
    e2e_steps = max(1, min(args.steps, 5))

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

                for i in range(args.warmup):
                    step2(i)
                barrier()
                h2.set_timing(True)
                e0.record()
                for i in range(args.steps):
                    step2(args.warmup + i)
                e1.record()
                barrier()
                ms2 = max_over_ranks(e0.elapsed_time(e1) / args.steps, dist, dev)
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
        u_steps = max(1, min(args.steps, 5))
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

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (the fused search) -------------------------------------
    adds = w.batch * nnz_mean * w.M  # nominal neuron-feature accumulations per launch
    search_s = max(phases["search_ms"], 1e-6) * 1e-3
    achieved = adds / search_s
    alg_bytes = w.V * w.M * store_bytes + sum(b.nnz * 4 + (b.n + 1) * 4 for b in batches) / n_batches + w.batch * 8
    # DRAM bytes per launch of the search kernel from the committed ncu summary of this workload
    traffic = None
    tpath = os.path.join(ROOT, "profiles", "k_bmu_table_%s.md" % w.name)
    if os.path.exists(tpath) and args.store == "f32":  # the committed capture is of the fp32 path
        for tl in open(tpath):
            if tl.startswith("traffic_bytes_per_launch"):
                traffic = float(tl.split("=")[1])
    roofline = {
        "bound": "alu", "kernel": "fused BMU search", "achieved": achieved / 1e12, "peak": add_peak / 1e12,
        "unit": "TFLOP/s", "frac": achieved / add_peak, "traffic": traffic,
        "peak_source": "%d SMs x %d fp32 lanes x %.0f MHz (%s clock)" % (sm_count, FP32_LANES_PER_SM, sm_max_mhz, peak_src),
        "search_ms": phases["search_ms"], "algorithmic_bytes": alg_bytes,
        "hbm_time_at_peak_ms": alg_bytes / (hbm_gbs * 1e9) * 1e3, "hbm_peak_gbs": hbm_gbs,
        "norms_ms": phases["norms_ms"],
        "norms_hbm_frac": (w.V * w.M * store_bytes / max(phases["norms_ms"], 1e-6) / 1e6) / hbm_gbs,
        "plan_ms": phases["plan_ms"], "finalize_ms": phases["finalize_ms"],
        "step_frac_of_alu_roofline": (adds / add_peak) / (ms_per_step * 1e-3),
    }

    # ---- CPU baseline: the oracle on a bounded sample, rank 0, N=1 only ----------------------
    cpu = None
    if ws == 1 and not args.no_cpu_baseline:
        m_slab = min(w.M, 4096)
        Wh = W.view(w.V, w.M)[:, :m_slab].float().contiguous().cpu().numpy()
        b = batches[0]
        n_take = min(b.n, 100_000)
        ip = b.indptr[:n_take + 1].cpu().numpy()
        ix = b.indices[:int(b.indptr[n_take])].cpu().numpy()
        rate, cores, desc, _ = _oracle_rate(w, Wh, m_slab, ip, ix, 12.0)
        cpu = {"value": rate, "unit": "samples/s", "cores": cores, "kind": "oracle", "sample": desc}

    line = {
        "metric": "bmu_samples_per_s", "value": value, "unit": "samples/s", "n_gpus": ws,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" if args.store == "f32" else "f32 accumulate, f16-stored codebook",
        "data": "synthetic",
        "config": {"workload": w.name, "V": w.V, "M": w.M, "batch": w.batch, "mean_nnz": nnz_mean,
                   "step": "som_norms + %s on one batch" % ("som_bmu_planned + som_update (a training-epoch step; plans built once, outside)" if args.epoch else
                       "som_bmu_planned (plans built once, outside)" if args.planned else
                       ("som_bmu_values" if args.values else ("som_bmu2" if args.top2 else "som_bmu"))),
                   "replicas": ws,
                   "l2_policy": "inputs larger than L2 (codebook %.0f MB + CSR %.0f MB per step)" % (
                       w.V * w.M * store_bytes / 1e6, batches[0].nnz * 4 / 1e6) if w.V * w.M * store_bytes > 126e6 else
                   "inputs smaller than L2: steps rotate over %d distinct batches, no flush" % n_batches},
        "accumulations_per_s": ws * adds / (ms_per_step * 1e-3),
        "roofline": roofline,
        "cpu_baseline": cpu,
        "e2e": {"value": e2e_value, "unit": "samples/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms,
                "path": "som_norms + som_bmu_host_async / som_host_sync (binary samples, best unit) on the same batches"},
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    if update is not None:
        line["update"] = update
    if args.two_stage:
        line["two_stage"] = {"uncertain_samples_last_call": h.last_uncertain(), "batch": w.batch}
    elif two_stage is not None:
        line["two_stage"] = two_stage
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1, help="index into the five workloads (default 1: 64x64)")
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
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    w = synth.CONFIGS[args.config]
    if args.features == "uniform":
        w = dataclasses.replace(w, name=w.name + "-uniform", zipf_s=0.0)
    if args.batch > 0:
        w = dataclasses.replace(w, name="%s-batch%d" % (w.name, args.batch), batch=args.batch, N=max(w.N, args.batch))
    if args.zipf_s is not None:
        w = dataclasses.replace(w, name="%s-zipf%g" % (w.name, args.zipf_s), zipf_s=args.zipf_s)
    if args.store == "f16":
        w = dataclasses.replace(w, name=w.name + "-f16")
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
