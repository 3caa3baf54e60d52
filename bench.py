#!/usr/bin/env python
"""Throughput of the SFB minibatch step (samples/s) at the paper-scale MLR shape, with the update product's
roofline fraction, an end-to-end (host buffers) figure and the CPU oracle timed beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--precision bf16|fp32] [--workload mlr_large]
    python bench.py --impl reference ...      # times the fp64 CPU oracle on a bounded sample instead
    python bench.py --phase update ...        # adds a loop of the fused update alone (>= 2 s, back to back)
    torchrun ... bench.py --gpus N --shard rows   # W partitioned by rows over the N ranks (one exchange per step)

A step is one pass of the whole hot path over one minibatch of K = P*B synthetic samples: pack, forward
product, softmax-minus-onehot, gather, fused rank-K update of W.  Prints ONE JSON line on rank 0.
With N > 1 (torchrun) every rank runs an independent replica on its own minibatches: the path has no
cross-GPU exchange, so the aggregate is N replicas ("weak" scaling) and no collective is on the data path.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import sfb_inputs as I  # noqa: E402

METRIC = "sfb_step_samples_per_sec"
UNIT = "samples/s"


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ----------------------------------------------------------------------------------------------------------
# CPU oracle on a bounded sample of the workload
# ----------------------------------------------------------------------------------------------------------
def oracle_sample_setup(wl, budget_s):
    """A slab of the workload the oracle can step in about ``budget_s`` seconds: all K samples and the full
    feature dimension against the first J' rows of W (softmax over J' classes).  Cost is linear in rows, so
    samples/s for the full matrix is the slab's figure times J'/J."""
    from oracle import sfb_oracle as O  # the one place outside tests/ and smoke() that runs the oracle

    def make(rows):
        sub = I.scaled(wl, wl.name + f"_rows{rows}", rows=rows)
        W = I.initial_W(sub)
        inp = I.step_inputs(sub, 0)
        if sub.model == I.MLR:
            inp.labels = (inp.labels % rows).astype(np.int32)
        L = O.lipschitz_power_iteration(W) if sub.model == I.SC else None

        def step():
            return O.sfb_step(sub.model, W, inp.X, inp.Y, inp.labels, workers=sub.workers, eta=sub.eta,
                              margin=sub.dml_margin, lam=sub.sc_lambda, L=L, iters=sub.sc_iters,
                              prox=(sub.model == I.SC))
        return step

    probe_rows = int(min(wl.rows, 2048))
    probe = make(probe_rows)
    probe()
    t0 = time.perf_counter()
    probe()
    per_row = (time.perf_counter() - t0) / probe_rows             # seconds per row of W on this machine
    rows = int(max(probe_rows, min(wl.rows, budget_s / per_row)))
    return make(rows), rows


def host_mem_available_gb():
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable:"):
                return int(line.split()[1]) / 1e6
    except OSError:
        pass
    return 0.0


def time_oracle_mlr_full_forward(wl, W_host, sample_rows=8192):
    """Paper-scale MLR on the host cores with the oracle's own routines for shapes too large to hold W in fp64:
    the log-partition of all K samples over ALL rows of W (the whole forward product, visited block by block),
    then the update of a contiguous sample of rows from that log-partition, its time scaled to all rows.  The
    sampled-row routine forms the logits of its rows again, so the scaled figure is an upper bound on the time of
    a step that keeps them."""
    from oracle import sfb_oracle as O
    inp = I.step_inputs(wl, 0)
    t0 = time.perf_counter()
    lse = O.mlr_log_partition(W_host, inp.X)
    t_fwd = time.perf_counter() - t0
    n = int(min(sample_rows, wl.rows))
    ids = np.arange(n)
    t0 = time.perf_counter()
    O.mlr_updated_rows(W_host[:n], ids, inp.X, inp.labels, lse, wl.eta)
    t_upd = time.perf_counter() - t0
    full = t_fwd + t_upd * wl.rows / n
    sample = (f"oracle on the full problem: log-partition of all K={wl.K} samples over all {wl.rows} rows "
              f"({t_fwd:.1f} s), then the updated rows of a sample of {n} rows ({t_upd:.2f} s, scaled by "
              f"{wl.rows}/{n}; that routine recomputes its rows' logits)")
    return wl.K / full, t_fwd + t_upd, sample


def cores_used():
    try:
        from threadpoolctl import threadpool_info
        n = max((d.get("num_threads", 1) for d in threadpool_info()), default=1)
        return int(n)
    except Exception:
        return len(os.sched_getaffinity(0))


def time_oracle(wl, steps, warmup, budget_s):
    step, rows = oracle_sample_setup(wl, budget_s)
    for _ in range(warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = (time.perf_counter() - t0) / steps
    full = dt * wl.rows / rows                                    # cost is linear in the rows of W
    sample = (f"oracle sfb_step on rows [0,{rows}) of W ({rows}/{wl.rows} of the matrix), all K={wl.K} "
              f"samples, full feature dim; time scaled by {wl.rows}/{rows}")
    return wl.K / full, dt, sample


# ----------------------------------------------------------------------------------------------------------
def max_over_ranks(values, device, world):
    """Element-wise maximum over all ranks of a list of floats (the job is as slow as its slowest rank)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def aggregate_value(world, K, steps, total_ms):
    """Whole-job samples/s: every rank steps its own replica on K samples per step (no exchange between them)."""
    return world * K * steps / (total_ms * 1e-3)


def clocks_sampler(index):
    """Starts nvidia-smi sampling SM clock, power and throttle reasons every 20 ms (it needs a moment to start, so
    it is launched before the warm-up); clocks_summary keeps the samples that fall inside the timed region."""
    f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
    q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    try:
        p = subprocess.Popen(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits", "-lms", "20",
                              "-i", str(index)], stdout=f, stderr=subprocess.DEVNULL)
    except Exception:
        return None, f
    return p, f


def clocks_summary(p, f, t0, t1):
    """Median SM clock and the throttle reasons seen between wall-clock times t0 and t1."""
    import datetime
    out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
    if p is None:
        return out
    p.terminate()
    try:
        p.wait(timeout=5)
    except Exception:
        p.kill()
    f.flush()
    f.seek(0)
    sm, mx, pw, reasons = [], [], [], set()
    names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
    for line in f.read().splitlines():
        parts = [x.strip() for x in line.split(",")]
        if len(parts) < 8:
            continue
        try:
            ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
            if ts < t0 or ts > t1:
                continue
            sm.append(float(parts[1]))
            mx.append(float(parts[2]))
            pw.append(float(parts[3]))
        except ValueError:
            continue
        for nme, v in zip(names, parts[4:8]):
            if v.lower().startswith("active"):
                reasons.add(nme)
    f.close()
    os.unlink(f.name)
    if sm:
        out["sm_mhz"] = float(np.median(sm))
        out["sm_max_mhz"] = float(max(mx))
        out["power_w"] = float(np.median(pw))
        out["samples"] = len(sm)
    out["reasons"] = sorted(reasons)
    return out


# ----------------------------------------------------------------------------------------------------------
def run_reference(args, wl, rank):
    if rank != 0:
        return
    budget = 150.0 / max(1, args.steps + args.warmup)
    value, dt, sample = time_oracle(wl, args.steps, args.warmup, budget)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(wl, "f64"),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores_used(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# DRAM bytes per launch of the update kernel at the paper-scale MLR shape, from the one-pass ncu capture summarised in
# profiles/ncu_update_pair_kernel_mlr_large_dram.md (dram__bytes_read.sum + dram__bytes_write.sum of one launch of the
# full-size bench).  The bf16 copy of W is rewritten only where its rounding changed, so the traffic depends on the data
# and does not scale with the rows: the figure applies to this workload only.  "kernel_unchanged_since" names the
# commit of the kernel's sources (csrc/sfb_update.cu, csrc/sfb_ptx.cuh) the counters were taken at: when the kernel is edited
# this entry has to be re-captured
# or set to None.
NCU_UPDATE_TRAFFIC = {"rows": 325000, "cols": 10000, "K": 1024, "bytes": 15.29e9 + 13.85e9,
                      "kernel_unchanged_since": "d08beef"}


def ncu_traffic_per_launch(wl, prec):
    t = NCU_UPDATE_TRAFFIC
    if t["bytes"] is None or wl.model != I.MLR or wl.cols != t["cols"] or wl.K != t["K"] or wl.rows != t["rows"]             or prec != 0:
        return None
    return t["bytes"]


def workload_config(wl, dtype):
    return {"workload": wl.name, "family": ["mlr", "dml", "sc"][wl.model], "rows": wl.rows, "cols": wl.cols,
            "workers_P": wl.workers, "batch_B": wl.batch, "K": wl.K, "eta": wl.eta, "operands": dtype,
            "master_W": "f32", "l2": "inputs_larger_than_l2" if wl.rows * wl.cols * 4 > 2 * 126e6
            else "l2_flushed_between_steps"}


def precision_code(S, name):
    return {"bf16": S.PREC_BF16, "fp32": S.PREC_FP32, "tf32": S.PREC_TF32X3, "ffma": S.PREC_FP32_FFMA}[name]


def dtype_name(wl, name):
    """The arithmetic type of the products: bf16, f32 (FFMA) or tf32x3 (fp32 values as pairs of tf32 words)."""
    if name == "bf16":
        return "bf16"
    return "tf32x3" if runs_tf32(wl, name) else "f32"


def runs_tf32(wl, name):
    """Whether the fp32 mode runs this workload's products on the tensor cores (the library's own rule)."""
    if wl.model != I.MLR or name in ("bf16", "ffma"):
        return False
    return name == "tf32" or (wl.rows >= 2048 and wl.cols >= 512 and wl.K >= 128)


NOMINAL_BF16_TFLOPS = 2250.0        # dense bf16, vendor figure (context only)
NOMINAL_TF32_OVER_BF16 = 1100.0 / 2250.0   # nominal ratio of the dense tf32 and bf16 tensor rates
NOMINAL_HBM_GBS = 7700.0


def update_roofline(wl, prec_bf16, ms_u, peaks, clocks, sustained=True, tf32=False, copy_fraction=1.0):
    """Roofline entry of the fused update W += -eta U^T V (one launch per step).  Algorithmic bytes per launch: W read
    and written once in fp32 plus U and V read once (what the method has to move).  The bf16 copy of W that this design
    writes alongside (the operand of the next forward product) is real traffic of the kernel and is reported beside
    it, not counted as algorithmic."""
    K = wl.K
    esz = 2 if prec_bf16 else 4
    if prec_bf16 and wl.model != I.MLR:
        esz = 4                                                               # (hi, lo) pairs of bf16
    upd_flops = 2.0 * wl.rows * wl.cols * K
    upd_bytes = 8.0 * wl.rows * wl.cols + K * (wl.rows + wl.cols) * esz
    shadow_bytes = 2.0 * wl.rows * wl.cols * copy_fraction if (prec_bf16 and wl.model == I.MLR) else 0.0
    tf_peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    if prec_bf16:
        t_flop = upd_flops / (tf_peak * 1e12)
        t_mem = upd_bytes / (peaks["hbm_gbs"] * 1e9)
        if t_mem >= t_flop:
            roof = {"bound": "hbm", "achieved": upd_bytes / (ms_u * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s"}
        else:
            roof = {"bound": "tensor", "achieved": upd_flops / (ms_u * 1e-3) / 1e12, "peak": tf_peak,
                    "unit": "TFLOP/s"}
        roof["roof_ms"] = max(t_flop, t_mem) * 1e3
    elif tf32:
        # fp32 operands as tf32 pairs: three tf32 products per term.  Peak for that dtype = the measured bf16 figure
        # times the nominal tf32/bf16 ratio; "achieved" counts the three products the kernel executes.
        peak = tf_peak * NOMINAL_TF32_OVER_BF16
        roof = {"bound": "tensor", "achieved": 3.0 * upd_flops / (ms_u * 1e-3) / 1e12, "peak": peak, "unit": "TFLOP/s",
                "note": "tf32 peak = measured bf16 x nominal ratio 1.1/2.25; achieved = executed flops (3 products per term)"}
        roof["roof_ms"] = max(3.0 * upd_flops / (peak * 1e12), upd_bytes / (peaks["hbm_gbs"] * 1e9)) * 1e3
    else:
        # fp32 FMA pipe: SMs x 128 lanes x 2 flop x max SM clock
        peak = 148 * 128 * 2 * ((clocks or {}).get("sm_max_mhz") or 1965.0) * 1e6 / 1e12
        roof = {"bound": "alu", "achieved": upd_flops / (ms_u * 1e-3) / 1e12, "peak": peak, "unit": "TFLOP/s"}
        roof["roof_ms"] = upd_flops / (peak * 1e12) * 1e3
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = ncu_traffic_per_launch(wl, 0 if prec_bf16 else 1)
    roof["traffic_captured_at"] = NCU_UPDATE_TRAFFIC["kernel_unchanged_since"] if roof["traffic"] else None
    roof["kernel"] = "update_pair_kernel + label_rows_kernel (sfb_apply_update)" if prec_bf16 \
        else "update_pair_kernel<tf32 pairs> (sfb_apply_update)" if tf32 else "sgemm_kernel EPI_RMW (sfb_apply_update)"
    roof["ms"] = ms_u
    roof["peaks"] = "of " + peaks["source"] + (" (sustained tensor figure: timed inside a long step)" if sustained
                                               else " (burst tensor figure: timed alone)")
    roof["update_tflops"] = upd_flops / (ms_u * 1e-3) / 1e12
    roof["frac_of_measured_sustained"] = roof["update_tflops"] / peaks["bf16_tflops_sustained"]
    roof["frac_of_measured_burst"] = roof["update_tflops"] / peaks["bf16_tflops"]
    roof["frac_of_nominal_peak"] = max(roof["update_tflops"] / NOMINAL_BF16_TFLOPS,
                                       upd_bytes / (ms_u * 1e-3) / 1e9 / NOMINAL_HBM_GBS) if prec_bf16 else None
    roof["algorithmic_bytes"] = upd_bytes
    roof["algorithmic_flops"] = upd_flops
    roof["achieved_incl_bf16_copy_of_W"] = (upd_bytes + shadow_bytes) / (ms_u * 1e-3) / 1e9
    return roof


def forward_and_step_rooflines(wl, ms_f, ms_step, upd_roof_ms, peaks):
    """Rooflines of the factor phase (bf16 MLR: forward product + softmax finish) and of the whole step, against the
    measured sustained tensor figure and the measured copy bandwidth."""
    K = wl.K
    fl = 2.0 * wl.rows * wl.cols * K
    t_fwd = max(fl / (peaks["bf16_tflops_sustained"] * 1e12),
                (2.0 * wl.rows * wl.cols + 4.0 * K * wl.rows) / (peaks["hbm_gbs"] * 1e9))        # bf16 W in, logits out
    t_fin = (4.0 * K * wl.rows + 2.0 * K * wl.rows) / (peaks["hbm_gbs"] * 1e9)                    # logits in, bf16 U out
    fwd = {"bound": "tensor", "roof_ms": (t_fwd + t_fin) * 1e3, "ms": ms_f, "frac": (t_fwd + t_fin) * 1e3 / ms_f,
           "achieved": fl / (ms_f * 1e-3) / 1e12, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
           "kernel": "pack + forward_kernel + softmax finish (sfb_compute_factors)"}
    roof_ms = (t_fwd + t_fin) * 1e3 + upd_roof_ms
    step = {"roof_ms": roof_ms, "ms": ms_step, "frac": roof_ms / ms_step}
    return fwd, step


def draw_W(torch, wl, dev, seed, rows=None):
    """W ~ the workload's init distribution, drawn on the device (13 GB of host generation would dominate the run)."""
    rows = wl.rows if rows is None else rows
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    W = torch.empty((rows, wl.cols), dtype=torch.float32, device=dev)
    std = {"normal": wl.w_std, "dml": 1.0 / math.sqrt(wl.cols), "zeros": 0.0, "unit_columns": 1.0}[wl.w_init]
    for r0 in range(0, rows, 65536):
        blk = W[r0:r0 + 65536]
        if std == 0.0:
            blk.zero_()
        else:
            blk.normal_(0.0, std, generator=g)
    return W


# ----------------------------------------------------------------------------------------------------------
# W partitioned by rows over the ranks (strong scaling: one problem, N GPUs)
# ----------------------------------------------------------------------------------------------------------
def run_sharded(args, wl, rank, world, local):
    import torch
    import torch.distributed as dist
    import paper_1409_5705_b200 as S
    from paper_1409_5705_b200.sharded import exchange_model_bytes, row_shard_bounds, sharded_step

    if wl.model != I.MLR:
        raise SystemExit("--shard rows is built for the MLR workloads")
    if wl.K % world != 0:
        raise SystemExit(f"K = {wl.K} samples do not split over {world} ranks")
    if world > 1:
        # NCCL's own log (communicator set-up: ranks, transports) goes to a file, not into the JSON line's stream
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_FILE", os.path.join(tempfile.gettempdir(), "sfb_nccl.%h.%p.log"))
    S.build()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl")
    dev = torch.device("cuda", local)
    prec = precision_code(S, args.precision)
    peaks = load_peaks()
    r0, r1 = row_shard_bounds(wl.rows, world, rank)
    W = draw_W(torch, wl, dev, 1234 + rank, rows=r1 - r0)
    K, n = wl.K, wl.K // world
    nb = 4
    batches = [I.step_inputs(wl, t) for t in range(nb)]                 # every rank draws the step, keeps its workers
    dX = [torch.from_numpy(b.X[rank * n:(rank + 1) * n]).to(dev) for b in batches]
    dL = [torch.from_numpy(b.labels[rank * n:(rank + 1) * n]).to(dev) for b in batches]
    cfg = S.make_config(wl.model, r1 - r0, wl.cols, wl.workers, wl.batch, wl.eta, prec)
    ctx = S.Context(cfg, W)
    ctx.sfb_set_row_shard(r0, wl.rows)
    partials = torch.zeros((K, 4), dtype=torch.float32, device=dev)
    partials_all = torch.zeros((world, K, 4), dtype=torch.float32, device=dev)
    X_all = torch.zeros((K, wl.cols), dtype=torch.float32, device=dev)
    y_all = torch.zeros((K,), dtype=torch.int32, device=dev)
    d = dist if world > 1 else None

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler, sfile = clocks_sampler(local) if rank == 0 else (None, None)
    moved = None
    for i in range(args.warmup):
        moved = sharded_step(ctx, dX[i % nb], dL[i % nb], partials, partials_all, X_all, y_all, dist=d)
    launches0 = ctx.sfb_get_stats().kernel_launches
    barrier()
    wall0 = time.time()
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_start.record()
    for i in range(args.steps):
        sharded_step(ctx, dX[i % nb], dL[i % nb], partials, partials_all, X_all, y_all, dist=d)
    t_end.record()
    barrier()
    clocks = clocks_summary(sampler, sfile, wall0, time.time()) if rank == 0 else None
    total_ms = t_start.elapsed_time(t_end)
    st = ctx.sfb_get_stats()
    launches = st.kernel_launches - launches0
    status = ctx.sfb_get_status()
    ms_u = st.ms_update
    total_ms, ms_u = max_over_ranks([total_ms, ms_u], dev, world)
    if rank == 0:
        value = K * args.steps / (total_ms * 1e-3)                          # one problem: K samples per step in all
        shard = I.scaled(wl, wl.name, rows=r1 - r0)
        roof = update_roofline(shard, prec == S.PREC_BF16, ms_u, peaks, clocks, tf32=runs_tf32(shard, args.precision))
        roof["traffic"] = None
        roof["traffic_captured_at"] = None
        model = exchange_model_bytes(wl.workers, wl.batch, wl.rows, wl.cols, world)
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
                "scaling": "strong", "vs_baseline": None, "dtype": dtype_name(wl, args.precision),
                "data": "synthetic",
                "config": dict(workload_config(wl, dtype_name(wl, args.precision)),
                               parallelism=f"rows{world}", rows_per_rank=r1 - r0),
                "roofline": roof, "cpu_baseline": None, "e2e": None, "gpu_launches": int(launches), "clocks": clocks,
                "exchange": {"measured_bytes_received_per_rank": moved.total if moved else 0,
                             "samples": moved.samples if moved else 0, "partials": moved.partials if moved else 0,
                             "model_row_sharded_per_rank": model["row_sharded_per_rank"] if world > 1 else 0,
                             "paper_sfb_p2p_total": model["sfb_p2p"],
                             "paper_full_matrix_sync_total": model["full_matrix_sync"]},
                "status_word": status}
        print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="sfb", choices=["sfb", "reference"])
    ap.add_argument("--precision", default="bf16", choices=["bf16", "fp32", "tf32", "ffma"],
                    help="bf16 operands (default); fp32 = the 1e-5 mode (tensor cores with tf32 pairs at large MLR "
                         "shapes, FFMA otherwise); tf32 / ffma force either kernel family of that mode")
    ap.add_argument("--workload", default="mlr_large", choices=sorted(I.WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--rows", type=int, default=0,
                    help="run a slab of the workload with this many rows of W (small cases for profiler captures)")
    ap.add_argument("--phase", default="", choices=["", "update"],
                    help="update: after the timed steps, loop the fused update alone for --phase-seconds")
    ap.add_argument("--phase-seconds", type=float, default=2.0)
    ap.add_argument("--sparse-nnz", type=float, default=0.0,
                    help="MLR: samples in compressed-sparse-row form with about this many non-zeros each (tf-idf-like, "
                         "Zipf column popularity); the update then sums only the non-zeros of each column")
    ap.add_argument("--sparse-update", default="auto", choices=["auto", "sparse", "dense"],
                    help="with --sparse-nnz: which update the step takes (auto: the library's cost model)")
    ap.add_argument("--graph", action="store_true",
                    help="launch each step as one CUDA graph (captured once per rotating minibatch from the same library "
                         "calls): for the launch-bound small workloads; value and ms_per_step are then the replays'")
    ap.add_argument("--context-library-update", action="store_true",
                    help="MLR bf16: also time the library way to the same fused update (one cuBLAS GEMM through torch.addmm, "
                         "bf16 operands, fp32 W read and written with beta = 1), as context beside the roofline")
    ap.add_argument("--shard", default="", choices=["", "rows"],
                    help="rows: partition W by rows over the ranks instead of running replicas")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    wl = I.WORKLOADS[args.workload]
    if args.rows > 0:
        wl = I.scaled(wl, f"{wl.name}_rows{args.rows}", rows=args.rows)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, wl, rank)
        return
    if args.shard == "rows":
        run_sharded(args, wl, rank, world, local)
        return

    import torch
    import torch.distributed as dist
    import paper_1409_5705_b200 as S

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the SFB path has no CPU fallback")
    S.build()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl")
    dev = torch.device("cuda", local)
    prec = precision_code(S, args.precision)
    peaks = load_peaks()

    # ---- synthetic state: W drawn on the device; minibatches from the seeded input module (each rank its own
    # step indices)
    W = draw_W(torch, wl, dev, 1234 + rank)
    L = 0.0
    if wl.w_init == "unit_columns":
        W /= W.norm(dim=0, keepdim=True)
        L = float(torch.linalg.matrix_norm(W, 2) ** 2)
    # host copy of the initial W for the oracle timed beside the paper-scale run (taken before any step)
    W_host = None
    full_forward_oracle = (not args.no_cpu_baseline and world == 1 and wl.model == I.MLR
                           and wl.rows * wl.cols * 4 > 4e9 and host_mem_available_gb() > wl.rows * wl.cols * 4 / 1e9 + 16)
    if full_forward_oracle:
        W_host = W.cpu().numpy()
    nb = 4
    sparse = args.sparse_nnz > 0
    if sparse and wl.model != I.MLR:
        raise SystemExit("--sparse-nnz is for the MLR workloads")
    true_dict = I.sc_true_dictionary(wl) if wl.model == I.SC else None
    batches = [I.step_inputs(wl, rank * 1000 + t, true_dict) for t in range(nb)]
    nnz_max = 0
    if sparse:
        # the same labels, the features replaced by sparse ones; the dense arrays are not used
        sps = [I.sparse_samples(wl.seed, rank * 1000 + t, wl.K, wl.cols, args.sparse_nnz) for t in range(nb)]
        nnz_max = max(sp.nnz for sp in sps)
        hS = [(torch.from_numpy(sp.indptr).pin_memory(), torch.from_numpy(sp.indices).pin_memory(),
               torch.from_numpy(sp.values).pin_memory(), sp.nnz) for sp in sps]
        dS = [(a.to(dev), b.to(dev), c.to(dev), n) for a, b, c, n in hS]
        for b in batches:
            b.X = np.zeros((1, 4), dtype=np.float32)
    dX = [torch.from_numpy(b.X).to(dev) for b in batches]
    dY = [None if b.Y is None else torch.from_numpy(b.Y).to(dev) for b in batches]
    dL = [None if b.labels is None else torch.from_numpy(b.labels).to(dev) for b in batches]
    hX = [torch.from_numpy(b.X).pin_memory() for b in batches]
    hY = [None if b.Y is None else torch.from_numpy(b.Y).pin_memory() for b in batches]
    hL = [None if b.labels is None else torch.from_numpy(b.labels).pin_memory() for b in batches]

    cfg = S.make_config(wl.model, wl.rows, wl.cols, wl.workers, wl.batch, wl.eta, prec, dml_margin=wl.dml_margin,
                        sc_lambda=wl.sc_lambda, sc_ista_iters=wl.sc_iters, sc_lipschitz=L,
                        sc_prox=1 if wl.model == I.SC else 0, csr_nnz_max=nnz_max,
                        csr_update={"auto": 0, "sparse": 1, "dense": 2}[args.sparse_update])
    if args.graph:
        torch.cuda.set_stream(torch.cuda.Stream(dev))      # a step can only be captured on a stream of its own
    ctx = S.Context(cfg, W)
    flusher = None
    if wl.rows * wl.cols * 4 <= 2 * 126e6:
        flusher = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def factors_call(k):
        if sparse:
            ctx.sfb_compute_factors_csr(-1, dS[k][0], dS[k][1], dS[k][2], dS[k][3], dL[k])
        else:
            ctx.sfb_compute_factors(-1, dX[k], dY[k], dL[k])

    def phased_step(i, ev=None):
        k = i % nb
        if flusher is not None:
            flusher.zero_()
        if ev is not None:
            ev[0].record()
        factors_call(k)
        if ev is not None:
            ev[1].record()
        ctx.sfb_gather_factors()
        if ev is not None:
            ev[2].record()
        ctx.sfb_apply_update()
        if ev is not None:
            ev[3].record()

    # ---- device-resident timing
    sampler, sfile = clocks_sampler(local) if rank == 0 else (None, None)
    for i in range(args.warmup):
        phased_step(i)
    st0 = ctx.sfb_get_stats()
    launches0 = st0.kernel_launches
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    barrier()
    wall0 = time.time()
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_start.record()
    for i in range(args.steps):
        phased_step(i, evs[i])
    t_end.record()
    barrier()
    clocks = clocks_summary(sampler, sfile, wall0, time.time()) if rank == 0 else None
    total_ms = t_start.elapsed_time(t_end)
    ms_incl_flush = total_ms / args.steps
    if flusher is not None:
        # the L2 flush runs between the steps; the value counts the steps' own device intervals
        total_ms = sum(e[0].elapsed_time(e[3]) for e in evs)
    st1 = ctx.sfb_get_stats()
    launches = st1.kernel_launches - launches0
    copy_stats = {"row_pieces_per_step": (st1.copy_pieces - st0.copy_pieces) / args.steps,
                  "rewritten_per_step": (st1.copy_written - st0.copy_written) / args.steps,
                  "fraction_rewritten": (st1.copy_written - st0.copy_written) / max(1, st1.copy_pieces - st0.copy_pieces)} \
        if st1.copy_pieces > st0.copy_pieces else None
    status = ctx.sfb_get_status()
    ms_f = sum(e[0].elapsed_time(e[1]) for e in evs) / args.steps
    ms_g = sum(e[1].elapsed_time(e[2]) for e in evs) / args.steps
    ms_u = sum(e[2].elapsed_time(e[3]) for e in evs) / args.steps

    # ---- the same steps, each launched as one CUDA graph (captured from the same library calls on the context's stream)
    graph_info = None
    if args.graph:
        l0 = ctx.sfb_get_stats().kernel_launches
        graphs = []
        for k in range(nb):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=ctx.stream):
                factors_call(k)
                ctx.sfb_gather_factors()
                ctx.sfb_apply_update()
            graphs.append(g)
        per_step_launches = (ctx.sfb_get_stats().kernel_launches - l0) / nb
        for i in range(3):
            graphs[i % nb].replay()
        gev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
        barrier()
        for i in range(args.steps):
            if flusher is not None:
                flusher.zero_()
            gev[i][0].record()
            graphs[i % nb].replay()
            gev[i][1].record()
        barrier()
        g_ms = sum(e[0].elapsed_time(e[1]) for e in gev) if flusher is not None else gev[0][0].elapsed_time(gev[-1][1])
        graph_info = {"ms_per_step": g_ms / args.steps, "eager_ms_per_step": total_ms / args.steps,
                      "kernels_per_graph": per_step_launches, "graphs": nb}
        status |= ctx.sfb_get_status()
        total_ms = g_ms
        launches = int(per_step_launches * args.steps)

    # ---- the fused update alone, back to back (same factors applied again and again): separates the kernel from the
    # rest of the step; ms x median SM MHz is the clock-independent figure
    update_loop = None
    if args.phase == "update" and rank == 0:
        sampler2, sfile2 = clocks_sampler(local)
        for _ in range(3):
            ctx.sfb_replay_update()
        torch.cuda.synchronize()
        reps = max(10, int(args.phase_seconds * 1e3 / max(ms_u, 1e-3)))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        w0 = time.time()
        e0.record()
        for _ in range(reps):
            ctx.sfb_replay_update()
        e1.record()
        torch.cuda.synchronize()
        ck = clocks_summary(sampler2, sfile2, w0, time.time())
        ms_loop = e0.elapsed_time(e1) / reps
        update_loop = {"launches": reps, "ms": ms_loop, "seconds": ms_loop * reps * 1e-3, "clocks": ck,
                       "ms_x_sm_mhz": ms_loop * ck["sm_mhz"] if ck.get("sm_mhz") else None,
                       "roofline": update_roofline(wl, prec == S.PREC_BF16, ms_loop, peaks, ck,
                                                   tf32=runs_tf32(wl, args.precision))}

    # ---- end to end: host minibatch -> sfb_step_host -> loss back on the host, every step (sparse samples: the three
    # arrays and the labels copied from pinned memory, sfb_step_csr, the loss read back through sfb_get_stats)
    def host_step(i):
        k = i % nb
        if not sparse:
            return ctx.sfb_step_host(hX[k], hY[k], hL[k])[0]
        ip, ix, vl, n = hS[k]
        ctx.sfb_step_csr(ip.to(dev, non_blocking=True), ix.to(dev, non_blocking=True), vl.to(dev, non_blocking=True), n,
                         hL[k].to(dev, non_blocking=True))
        return ctx.sfb_get_stats().last_loss

    for i in range(3):
        host_step(i)
    barrier()
    e2e_steps = args.steps
    t0 = time.perf_counter()
    loss = 0.0
    for i in range(e2e_steps):
        loss = host_step(i)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0

    # ---- context, not a target: the same read-modify-write of W as one library GEMM (no bf16 copy of W, no fp32 label
    # entries); it runs last because it overwrites W with updates of the last step's factors
    library_update = None
    if args.context_library_update and rank == 0 and prec == S.PREC_BF16 and wl.model == I.MLR and not sparse:
        Uq, Vq, dt_, lo_, ldu_, ldv_ = ctx.sfb_get_factors()
        ws0 = ctx.workspace.data_ptr()
        UT = ctx.workspace[Uq - ws0:Uq - ws0 + wl.rows * ldu_ * 2].view(torch.bfloat16).view(wl.rows, ldu_)[:, :wl.K]
        VT = ctx.workspace[Vq - ws0:Vq - ws0 + wl.cols * ldv_ * 2].view(torch.bfloat16).view(wl.cols, ldv_)[:, :wl.K]
        def library_loop(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                torch.addmm(W, UT, VT.t(), out_dtype=torch.float32, beta=1.0, alpha=-wl.eta, out=W)
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / reps

        library_loop(3)
        time.sleep(1.0)                                  # let the clocks recover from the runs before
        ms_burst = library_loop(10)
        sampler3, sfile3 = clocks_sampler(local)
        w0 = time.time()
        reps = max(20, int(args.phase_seconds * 1e3 / ms_burst))
        ms_long = library_loop(reps)
        ck3 = clocks_summary(sampler3, sfile3, w0, time.time())
        library_update = {"call": "torch.addmm(W, U^T, V, out_dtype=float32, beta=1, alpha=-eta, out=W): one cuBLAS GEMM",
                          "ms_first_10_launches": ms_burst, "ms": ms_long, "launches": reps, "clocks": ck3,
                          "ms_x_sm_mhz": ms_long * ck3["sm_mhz"] if ck3.get("sm_mhz") else None,
                          "note": "context only: W read and written in fp32 like the update kernel, but no bf16 operand copy "
                                  "of W and no fp32 label rows; launches back to back for --phase-seconds"}

    total_ms, e2e_ms, ms_f, ms_g, ms_u = max_over_ranks([total_ms, e2e_s * 1e3, ms_f, ms_g, ms_u], dev, world)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    K = wl.K
    value = aggregate_value(world, K, args.steps, total_ms)
    e2e_value = aggregate_value(world, K, e2e_steps, e2e_ms)
    h2d = K * wl.in_dim * 4 + (K * wl.cols * 4 if wl.model == I.DML else 0) + (K * 4 if wl.model != I.SC else 0)
    if sparse:
        h2d = int(sum(8 * (K + 1) + 8 * n for _, _, _, n in hS) / nb) + K * 4

    # ---- roofline of the dominant kernel (the fused update), timed inside the long step: sustained tensor figure
    roof = update_roofline(wl, prec == S.PREC_BF16, ms_u, peaks, clocks, tf32=runs_tf32(wl, args.precision),
                           copy_fraction=min(1.0, copy_stats["rewritten_per_step"] / (wl.rows * math.ceil(wl.cols / 32)))
                           if copy_stats else 1.0)
    sparse_ran = sparse and st1.sparse_updates > st0.sparse_updates
    if sparse_ran:
        # the sparse update is one read-modify-write pass over W plus the factors: bound by HBM
        nnz = sum(n for _, _, _, n in hS) / nb
        usz = 2 if prec == S.PREC_BF16 else 4
        algo = 8.0 * wl.rows * wl.cols + usz * K * wl.rows + 8.0 * nnz
        peak = peaks["hbm_gbs"]
        roof = {"bound": "hbm", "achieved": algo / (ms_u * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                "frac": algo / (ms_u * 1e-3) / 1e9 / peak, "traffic": None, "peak_source": peaks["source"],
                "kernel": "sparse_update_kernel (+ label_rows_kernel in bf16 mode)", "ms": ms_u,
                "algorithmic_bytes": algo, "fma_per_entry_of_W": nnz / wl.cols,
                "note": "W read and written once in fp32, the factors u read once, 8 bytes per non-zero of v; "
                        "the operand copy of W is rewritten where its rounding changed (not counted)"}
    roof_fwd, roof_step = (None, None)
    if prec == S.PREC_BF16 and wl.model == I.MLR and not sparse:
        roof_fwd, roof_step = forward_and_step_rooflines(wl, ms_f, total_ms / args.steps, roof["roof_ms"], peaks)

    cpu = None
    if not args.no_cpu_baseline and world == 1:       # the oracle is timed beside the single-GPU run only
        if W_host is not None:
            v, dt, sample = time_oracle_mlr_full_forward(wl, W_host)
        else:
            v, dt, sample = time_oracle(wl, 1, 0, 15.0)
            sample += " (row-slab extrapolation: the host has no room for the full matrix, or the workload is small)" \
                if wl.rows * wl.cols * 4 > 4e9 else ""
        cpu = {"value": v, "unit": UNIT, "cores": cores_used(), "kind": "oracle", "sample": sample,
               "sample_seconds": dt}

    esz = 2 if prec == S.PREC_BF16 else 4
    if prec == S.PREC_BF16 and wl.model != I.MLR:
        esz = 4
    one_copy = K * (wl.rows + wl.cols) * esz
    cfg_line = workload_config(wl, dtype_name(wl, args.precision))
    if sparse:
        one_copy = K * wl.rows * esz + 8 * sum(n for _, _, _, n in hS) / nb
        cfg_line["features"] = (f"compressed sparse rows, about {args.sparse_nnz:g} non-zeros per sample "
                                f"(Poisson), Zipf(1) column popularity, log-normal values, unit-length samples")
        cfg_line["update"] = ("sparse" if sparse_ran else "dense") + f" ({args.sparse_update})"
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": dtype_name(wl, args.precision),
            "data": "synthetic", "config": cfg_line,
            "roofline": roof, "roofline_forward": roof_fwd, "roofline_step": roof_step, "cpu_baseline": cpu,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": 8,
                    "ms_per_step": e2e_ms / e2e_steps, "last_loss": loss},
            "gpu_launches": int(launches), "clocks": clocks,
            "phases_ms": {"factors": ms_f, "gather": ms_g, "update": ms_u},
            "bytes": {"sf_gather_one_copy": one_copy,
                      "sf_broadcast_p2p": (wl.workers - 1) * one_copy,
                      "dense_sync": wl.workers * wl.rows * wl.cols * 4,
                      "dense_over_sf": wl.workers * wl.rows * wl.cols * 4 / one_copy},
            "operand_copy": copy_stats, "status_word": status}
    if flusher is not None:
        line["ms_per_step_incl_l2_flush"] = ms_incl_flush
        line["config"]["l2"] = "l2_flushed_between_steps (the flush is outside the timed intervals)"
    if graph_info is not None:
        line["graph"] = graph_info
        line["config"]["launch"] = "one CUDA graph per step"

    if update_loop is not None:
        line["update_loop"] = update_loop
    if library_update is not None:
        line["library_update"] = library_update
    print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
