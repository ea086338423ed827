#!/usr/bin/env python
"""Benchmark of the SLIDE train step (libdslide) on synthetic data of the 670K-class shape.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl dslide|reference] [--config 670k]

A step is one pass of the whole hot path over one batch: hidden layer, hashing, bucket lookup and
union, active logits and softmax, sparse back-propagation, row-wise Adam, and the table rebuild
whenever the schedule (every 50 steps) places one inside the window.  Prints ONE JSON line.

  value      train samples/s with the batches already resident in HBM (CUDA events, max over ranks)
  e2e        the same through dslide_train_step_host_async: HOST (pinned) buffers, every step's host->device copy
             and the device->host read of its loss and status inside the timed region
  roofline   the dominant kernel: algorithmic bytes per launch / its mean launch duration (CUDA
             events around every launch of a second, separately timed pass) against the measured
             HBM copy bandwidth
  cpu_baseline  the CPU oracle, as it stands, timed on this machine's host cores on a bounded sample

With --gpus N > 1 (launched by torchrun) every rank runs an independent replica on its own batches:
the path has no exchange step, so no collective is on the data path.  --impl reference times the CPU
oracle alone (rank 0 only).
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2201_12667_b200 import workloads  # noqa: E402

METRIC = "train samples/s at 670K-class shape on 1 B200; achieved HBM GB/s vs peak"
REBUILD_PERIOD = 50
REF_BATCH = 32            # samples per step of the CPU-oracle arm (a bounded sample of the 256-sample batch)
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under profiles/, taken
# on early steps of this workload (more rows touched than in the timed window) and therefore kept as a ratio to
# the bytes that scale with the rows of the launch: update kernel 107.6 MB measured against 149.5 MB algorithmic;
# forward kernel 34.8 MB measured against 33.3 MB (the rows of W1 / W2 it gathers, tables, batch).
NCU_TRAFFIC_RATIO = {"adam": 107.6 / 149.5, "forward": 34.8 / 33.3}


def ncu_traffic(kernel, model):
    return NCU_TRAFFIC_RATIO[kernel] * model[kernel] if kernel in NCU_TRAFFIC_RATIO else None


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="dslide", choices=["dslide", "reference"])
    ap.add_argument("--config", default="670k", choices=sorted(workloads.CONFIGS))
    ap.add_argument("--batches", type=int, default=64, help="distinct pre-generated batches, cycled")
    ap.add_argument("--batch-size", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--rebuild-period", type=int, default=REBUILD_PERIOD)
    ap.add_argument("--budget", type=int, default=0, help="sampling budget per sample (Section 3.7); 0 = none, as in the headline")
    return ap.parse_args()


def hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def code_bits(c):
    return c["K"] if c["family"] == workloads.SIMHASH else c["K"] * int(np.log2(c["bin_size"]))


def byte_model(c, B, per_step, labels_per_step, gap):
    """Algorithmic bytes of one step: what the method itself must move, each distinct row once per use."""
    H, N, L = c["H"], c["N"], c["L"]
    nnz, sumA, U1, U2, fetched = (per_step[k] for k in ("nnz", "sum_active", "touched_w1", "touched_w2", "fetched"))
    csr = 8 * nnz + 4 * (B + 1)
    lab = 4 * labels_per_step + 4 * (B + 1)
    w1 = 6 * 4 * H * U1                      # read and write w, m, v of every distinct touched row
    w2 = 6 * 4 * (H + 1) * U2                # rows and their biases
    b1 = 3 * 2 * 4 * H
    tables = B * L * 8 + 4 * fetched         # two offsets per (sample, table) + the bucket slices
    act = 2 * (4 + 4) * sumA                 # active ids and one float each, written then read
    hid = 2 * 4 * B * H
    rebuild = (4 * H * N + 4 * N * L + 4 * L * (2 ** code_bits(c) + 1)) / gap if gap else 0.0
    total = csr + lab + w1 + w2 + b1 + tables + act + hid + rebuild
    # per kernel: the update kernel is booked the rows (read and write of w, m, v); the forward kernel, being a kernel
    # of its own, cannot be served those rows on chip, so its figure adds the rows it gathers (once each per use)
    # the "issued" figure: the step as two kernels -- the forward gather of the rows and the logit / error gathers are
    # added to the compulsory bytes
    issued = total + 4 * H * nnz + 2 * 4 * (H + 1) * sumA
    return dict(total=total, rebuild=rebuild, issued=issued,
                adam=w1 + w2 + b1 + act / 2 + hid / 2,
                forward=csr + lab + tables + act / 2 + hid / 2 + 4 * H * nnz + 4 * (H + 1) * sumA)


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device):
        self.device = device
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.device), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 7:
                    continue
                try:
                    sm.append(float(f[0])); mx.append(float(f[1]))
                except ValueError:
                    continue
                for n, v in zip(names, f[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


def dist_setup(ngpus):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return world, rank, local


def max_over_ranks(ms, world, device):
    """The slowest rank's time: every multi-GPU number is the maximum over the ranks."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def shard_seed(rank):
    """Every rank draws its own batches: replicas share no data and exchange nothing."""
    return 1000 * rank


# ------------------------------------------------------------------------------------------------
def run_reference(args):
    world, rank, _ = dist_setup(args.gpus)
    if rank != 0:
        return
    from oracle.oracle import Oracle
    c = workloads.config(args.config)
    B = min(REF_BATCH, args.batch_size or c["batch"])
    o = Oracle("float", D=c["D"], H=c["H"], N=c["N"], family=c["family"], K=c["K"], L=c["L"],
               bin_size=c["bin_size"], bucket_cap=c["bucket_cap"], lr=c["lr"], seed=0, init_std=0.01,
               rebuild_period0=args.rebuild_period, redraw=1)
    wl = workloads.Workload(c, seed=0)
    nb = min(args.batches, args.steps + args.warmup)
    batches = [wl.batch(i, batch_size=B) for i in range(nb)]
    for i in range(args.warmup):
        o.train_step(*batches[i % nb])
    t0 = time.perf_counter()
    for i in range(args.steps):
        o.train_step(*batches[(args.warmup + i) % nb])
    dt = time.perf_counter() - t0
    value = B * args.steps / dt
    sample = "%d of the %d samples of each batch per step, %d steps, scheduled rebuilds (every %d steps) included" % (
        B, c["batch"], args.steps, args.rebuild_period)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "samples/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(c, B, args, nb),
        "cpu_baseline": {"value": value, "unit": "samples/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "samples/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def workload_config(c, B, args, nb):
    return {"workload": "%s-class shape: D %d, H %d, N %d, %s K=%d L=%d cap %d, batch %d, ~%d nnz/row Zipf(1.1), "
                        "~%d labels/sample" % (c["name"], c["D"], c["H"], c["N"],
                                               "DWTA" if c["family"] == workloads.DWTA else "SimHash", c["K"], c["L"],
                                               c["bucket_cap"], B, c["mean_nnz"], c["mean_labels"]),
            "batch": B, "rebuild_every": args.rebuild_period, "distinct_batches": nb, "sampling_budget": args.budget,
            "l2": "inputs larger than L2: 1.3 GB of model state, a different batch (and so different rows) every step"}


def cpu_baseline(c, args, B):
    """The oracle, untuned, single-threaded, on a bounded sample: a few full-batch steps + one rebuild / period."""
    from oracle.oracle import Oracle
    o = Oracle("float", D=c["D"], H=c["H"], N=c["N"], family=c["family"], K=c["K"], L=c["L"],
               bin_size=c["bin_size"], bucket_cap=c["bucket_cap"], lr=c["lr"], seed=0, init_std=0.01, rebuild_period0=0)
    wl = workloads.Workload(c, seed=0)
    nsteps = 8
    batches = [wl.batch(i, batch_size=B) for i in range(nsteps + 2)]
    for b in batches[:2]:
        o.train_step(*b)
    t0 = time.perf_counter()
    for b in batches[2:]:
        o.train_step(*b)
    t_step = (time.perf_counter() - t0) / nsteps
    t0 = time.perf_counter()
    o.rebuild_tables()
    t_rebuild = time.perf_counter() - t0
    o.close()
    per = t_step + (t_rebuild / args.rebuild_period if args.rebuild_period else 0.0)
    return {"value": B / per, "unit": "samples/s", "cores": 1, "kind": "oracle",
            "sample": "%d full steps of batch %d (%.3f s each) + one table rebuild (%.2f s) amortised over %d steps"
                      % (nsteps, B, t_step, t_rebuild, args.rebuild_period)}


def run_dslide(args):
    import torch
    from paper_2201_12667_b200 import binding as ds

    world, rank, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the dslide arm")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    c = workloads.config(args.config)
    B = args.batch_size or c["batch"]
    K, W = args.steps, max(args.warmup, 3)

    cfg = ds.make_config(input_dim=c["D"], hidden_dim=c["H"], output_dim=c["N"], hash_family=c["family"], K=c["K"],
                         L=c["L"], dwta_bin_size=c["bin_size"], bucket_cap=c["bucket_cap"],
                         rebuild_period0=args.rebuild_period, rebuild_growth_lambda=0.0, redraw_hash_fns=1,
                         max_batch=B, max_labels=c["max_labels"], lr=c["lr"], init_std=0.01, seed=0, device=local,
                         sample_budget=args.budget, inputs_ready=1)
    ctx = ds.dslide_init(cfg)

    wl = workloads.Workload(c, seed=shard_seed(rank))
    nb = args.batches
    host = [wl.batch(i, batch_size=B) for i in range(nb)]
    labels_per_step = float(np.mean([len(b[4]) for b in host]))
    dev = [[torch.from_numpy(a).cuda() for a in b] for b in host]
    pinned = [[torch.from_numpy(a).pin_memory() for a in b] for b in host]
    loss = torch.zeros(1, device="cuda")

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def step(i):
        ds.dslide_train_step(ctx, B, *dev[i % nb], loss)

    for i in range(W):
        step(i)
    ds.dslide_sync(ctx)
    ds.dslide_cum_stats(ctx, reset=True)

    # ---- timed region: K steps, inputs resident in HBM ----
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = ds.dslide_kernel_launches(ctx)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for i in range(K):
        step(W + i)
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    launches = ds.dslide_kernel_launches(ctx) - launches0
    clocks = sampler.stop() if rank == 0 else None
    status = ds.dslide_sync(ctx, check=False)
    cum = ds.dslide_cum_stats(ctx, reset=True)
    ms = max_over_ranks(ms, world, "cuda")
    value = world * B * K / (ms * 1e-3)

    # ---- second pass of the same K steps with a CUDA event pair around every kernel launch: on a fresh model taken
    #      through the same warm-up, because the active sets grow as the model trains and a later window of steps
    #      touches more rows ----
    ds.dslide_destroy(ctx)
    ctx = ds.dslide_init(cfg)
    for i in range(W):
        step(i)
    ds.dslide_sync(ctx)
    ds.dslide_cum_stats(ctx, reset=True)
    ds.dslide_profile_begin(ctx)
    for i in range(K):
        step(W + i)
    prof = ds.dslide_profile_end(ctx)
    cum_prof = ds.dslide_cum_stats(ctx, reset=True)      # the per-kernel times go with the rows these steps touched

    # ---- end to end: host buffers in, loss out, every step ----
    e2e = None
    if not args.no_e2e:
        # the pipelined host-buffer entry point: every step copies its inputs from pinned host memory to the device
        # and its {status, loss} back; the loss of step i is handed out by call i + 1 (the last one by
        # dslide_host_result), so the device always has one step queued while the host packs the next
        # on a fresh model taken through the same warm-up, so that the timed steps are the same training steps as in
        # the device-resident pass (the active sets grow as the model trains, and later windows run slower)
        ds.dslide_destroy(ctx)
        ctx = ds.dslide_init(cfg)
        for i in range(W):
            ds.dslide_train_step_host_async(ctx, B, *pinned[i % nb])
        ds.dslide_host_result(ctx)
        barrier()
        e0.record()
        losses = 0
        for i in range(K):
            losses += ds.dslide_train_step_host_async(ctx, B, *pinned[(W + i) % nb]) is not None
        losses += ds.dslide_host_result(ctx) is not None
        e1.record()
        barrier()
        assert losses == K
        ms_e2e = e0.elapsed_time(e1)
        ms_e2e = max_over_ranks(ms_e2e, world, "cuda")
        h2d = float(np.mean([sum(a.numel() * a.element_size() for a in b) for b in pinned]))
        e2e = {"value": world * B * K / (ms_e2e * 1e-3), "unit": "samples/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": 8, "ms_per_step": ms_e2e / K,
               "api": "dslide_train_step_host_async + dslide_host_result (loss and status of every step read back)"}

    if rank == 0:
        per_step = {k: cum[k] / max(1, cum["steps"]) for k in ("nnz", "sum_active", "touched_w1", "touched_w2", "fetched")}
        model = byte_model(c, B, per_step, labels_per_step, args.rebuild_period)
        peak, peak_kind = hbm_peak()
        total_prof = sum(v[0] for v in prof.values()) or 1.0
        kernels = {}
        for name, (kms, cnt) in sorted(prof.items(), key=lambda kv: -kv[1][0]):
            kernels[name] = {"launches": cnt, "ms_total": kms, "us_per_launch": 1e3 * kms / cnt,
                             "share": kms / total_prof}
        dominant = max((n for n in prof if n in ("adam", "forward")), key=lambda n: prof[n][0])
        dur = prof[dominant][0] * 1e-3 / prof[dominant][1]
        per_step_prof = {k: cum_prof[k] / max(1, cum_prof["steps"]) for k in per_step}
        model_prof = byte_model(c, B, per_step_prof, labels_per_step, args.rebuild_period)
        achieved = model_prof[dominant] / dur / 1e9
        roofline = {"bound": "hbm", "kernel": "k_" + dominant, "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak, "traffic": ncu_traffic(dominant, model_prof),
                    "algorithmic_bytes_per_launch": model_prof[dominant], "us_per_launch": dur * 1e6,
                    "peak_source": "MEASURED_PEAKS.json hbm_gbs (of %s)" % peak_kind}
        step_gbs = model["total"] / (ms * 1e-3 / K) / 1e9
        rebuild_us = sum(1e3 * v[0] for n, v in prof.items() if n not in ("adam", "forward", "adam_dense")) / max(1, K)
        out = {
            "metric": METRIC, "value": value, "unit": "samples/s", "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": workload_config(c, B, args, nb),
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline,
            "step_roofline": {"algorithmic_bytes_per_step": model["total"], "achieved": step_gbs, "peak": peak,
                              "unit": "GB/s", "frac": step_gbs / peak, "frac_of_8TBps_nominal": step_gbs / 8000.0,
                              "issued_bytes_per_step": model["issued"],
                              "issued_gbs": model["issued"] / (ms * 1e-3 / K) / 1e9,
                              "us_per_step": 1e3 * ms / K, "rebuild_us_per_step_amortised": rebuild_us,
                              "us_per_step_without_rebuild": 1e3 * ms / K - rebuild_us},
            "kernels": kernels,
            "per_step": dict(per_step, labels=labels_per_step),
            "device_status": int(status),
        }
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline(c, args, B)
        print(json.dumps(out))
    ds.dslide_destroy(ctx)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_dslide(a)
