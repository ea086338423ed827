#!/usr/bin/env python
"""Benchmark of the SLIDE train step (libdslide) on synthetic data of the 670K-class shape.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl dslide|reference] [--config 670k] [--sweep]

A step is one pass of the whole hot path over one batch: hidden layer, hashing, bucket lookup and
union, active logits and softmax, sparse back-propagation, row-wise Adam, and its share of the
scheduled table rebuild (every 50 steps by default).  Prints ONE JSON line (--sweep: one per cell).

  value      train samples/s of the FULL step with the batches already resident in HBM: the median of
             --windows timed windows of K steps (CUDA events, max over ranks), every window on a fresh
             model taken through the same warm-up.  A window in which the schedule places exactly
             K / period rebuilds is reported as measured; otherwise the rebuilds inside it are taken out
             and one rebuild (timed with CUDA events in the same run) is added per `period` steps, so the
             figure never leaves the rebuild out and never books rebuild bytes without rebuild time.
  e2e        the same through dslide_train_step_host_async: HOST (pinned) buffers, every step's host->device
             copy and the device->host read of its loss and status inside the timed region
  roofline   the dominant kernel: algorithmic bytes per launch / its mean launch duration (CUDA
             events around every launch of a separately timed pass) against the measured HBM copy
             bandwidth; whole_step holds the same ratio for the full step
  cpu_baseline  the CPU oracle, as it stands, timed on this machine's host cores (one core, and all cores
             with its OpenMP build) on a bounded sample

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
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2201_12667_b200 import workloads  # noqa: E402

METRIC = "train samples/s at 670K-class shape on 1 B200; achieved HBM GB/s vs peak"
REBUILD_PERIOD = 50
REF_BATCH = 32            # samples per step of the CPU-oracle arm (a bounded sample of the 256-sample batch)
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under profiles/ (taken on
# early steps of this workload, where more rows are touched than in a later window), kept as a ratio to the
# algorithmic bytes of the captured launch, since the traffic follows the number of rows: update kernel 108.2 MB
# measured against 149.5 MB algorithmic; forward kernel 34.8 MB against 33.3 MB (the rows of W1 / W2 it gathers,
# tables, batch).  null for a kernel that has changed since its counters were taken.
NCU_TRAFFIC_RATIO = {"adam": 108.2 / 149.5, "forward": 34.8 / 33.3}
SWEEP_BATCHES = (64, 128, 256, 512, 1024, 2048)
# target active fraction of the 670,091 outputs -> (K, L, bucket cap, force_dense): the expected union is about
# L * min(cap, N / 8^K) ids before duplicates (DWTA, bins of eight: 8^K buckets per table)
SWEEP_FRACTIONS = (
    (0.0005, dict(K=6, L=130, bucket_cap=128)),       # 2.6 ids per bucket x 130 tables  ~ 335
    (0.002, dict(K=5, L=66, bucket_cap=128)),         # 20 per bucket x 66               ~ 1,350
    (0.01, dict(K=4, L=41, bucket_cap=256)),          # 164 per bucket x 41              ~ 6,700
    (0.05, dict(K=3, L=33, bucket_cap=1024)),         # 1,024 of 1,309 per bucket x 33   ~ 33,000
    (0.25, dict(K=2, L=18, bucket_cap=10470)),        # 10,470 per bucket x 18, a fifth of them duplicates ~ 165,000
    (1.0, dict(force_dense=1)),                       # the dense limit: every neuron active, no hashing
)


def ncu_traffic(kernel, model):
    return NCU_TRAFFIC_RATIO[kernel] * model[kernel] if kernel in NCU_TRAFFIC_RATIO else None


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="dslide", choices=["dslide", "reference"])
    ap.add_argument("--config", default="670k", choices=sorted(workloads.CONFIGS))
    ap.add_argument("--batches", type=int, default=64, help="distinct pre-generated batches, cycled")
    ap.add_argument("--batch-size", type=int, default=0)
    ap.add_argument("--windows", type=int, default=5, help="timed windows (each on a fresh model); the median is reported")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--rebuild-period", type=int, default=REBUILD_PERIOD)
    ap.add_argument("--rebuild-lambda", type=float, default=0.0, help="later gaps grow by exp(lambda * rebuilds)")
    ap.add_argument("--budget", type=int, default=0, help="sampling budget per sample (Section 3.7); 0 = none, as in the headline")
    ap.add_argument("--hidden-lsh", default="", help="K,L,cap: sample the hidden layer too (tables over the hidden neurons); default dense")
    ap.add_argument("--predict", type=int, default=0, metavar="K",
                    help="time top-K inference instead of training: over the retrieved neurons and over all neurons")
    ap.add_argument("--sweep", action="store_true",
                    help="batch 64..2048 x active fraction 0.05%%..100%% on the 670K shape: one JSON line per cell")
    ap.add_argument("--sweep-batches", default="", help="comma-separated subset of the sweep's batch sizes")
    ap.add_argument("--sweep-fractions", default="", help="comma-separated subset of the sweep's target fractions")
    return ap.parse_args(argv)


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
    """Algorithmic bytes of one step: what the method itself must move, each distinct row once per use.

    gap = steps per rebuild the step is charged for (0: no rebuild bytes)."""
    H, N, L = c["H"], c["N"], c["L"]
    nnz, sumA, U1, U2, fetched = (per_step[k] for k in ("nnz", "sum_active", "touched_w1", "touched_w2", "fetched"))
    csr = 8 * nnz + 4 * (B + 1)
    lab = 4 * labels_per_step + 4 * (B + 1)
    w1 = 6 * 4 * H * U1                      # read and write w, m, v of every distinct touched row
    w2 = 6 * 4 * (H + 1) * U2                # rows and their biases
    b1 = 3 * 2 * 4 * H
    dense = bool(c.get("force_dense"))
    tables = 0 if dense else B * L * 8 + 4 * fetched         # two offsets per (sample, table) + the bucket slices
    act = 2 * (4 + 4) * sumA                 # active ids and one float each, written then read
    hid = 2 * 4 * B * H
    rebuild = (4 * H * N + 4 * N * L + 4 * L * (2 ** code_bits(c) + 1)) / gap if (gap and not dense) else 0.0
    total = csr + lab + w1 + w2 + b1 + tables + act + hid + rebuild
    # per kernel: the update kernel is booked the rows (read and write of w, m, v); the forward kernel, being a kernel
    # of its own, cannot be served those rows on chip, so its figure adds the rows it gathers (once each per use).
    # the "issued" figure: the step as two kernels -- the forward gather of the rows and the logit / error gathers are
    # added to the compulsory bytes
    issued = total + 4 * H * nnz + 2 * 4 * (H + 1) * sumA
    return dict(total=total, rebuild=rebuild, issued=issued,
                adam=w1 + w2 + b1 + act / 2 + hid / 2,
                forward=csr + lab + tables + act / 2 + hid / 2 + 4 * H * nnz + 4 * (H + 1) * sumA)


def full_step_ms(window_ms, steps, rebuilds_in_window, rebuild_ms, period):
    """Milliseconds of one FULL step (its share of the scheduled rebuild included) from a timed window.

    A window that holds exactly steps / period rebuilds is taken as measured.  Otherwise the rebuilds that fell into
    the window are taken out at the separately measured cost of one rebuild, and one rebuild per `period` steps is
    added: the figure neither leaves the rebuild out nor counts it twice."""
    if not period:
        return window_ms / steps, "no rebuild scheduled"
    if rebuilds_in_window * period == steps:
        return window_ms / steps, "as measured: the window holds %d scheduled rebuilds in %d steps" % (rebuilds_in_window, steps)
    ms = (window_ms - rebuilds_in_window * rebuild_ms) / steps + rebuild_ms / period
    return ms, ("window of %d steps held %d rebuilds, not steps/period = %.2f: rebuilds inside the window taken out and "
                "one rebuild of %.3f ms (CUDA events, same run) added per %d steps"
                % (steps, rebuilds_in_window, steps / period, rebuild_ms, period))


class ClockSampler:
    """SM clock, power and throttle reasons for the whole run, time-stamped; summarised over the timed windows.

    Reads through NVML (read-only queries) from a thread; falls back to an nvidia-smi loop."""
    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20), ("sw_power_cap", 0x4))

    def __init__(self, device):
        self.device = device
        self.samples = []          # (time.time(), sm_mhz, max_mhz, power_w, reason bits)
        self.windows = []          # (t0, t1) of the timed regions
        self.thread = None
        self.stop_flag = False
        self.proc = None
        self.path = None
        self.stopped = False

    def _nvml_loop(self, handle, nv):
        mx = nv.nvmlDeviceGetMaxClockInfo(handle, nv.NVML_CLOCK_SM)
        reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or nv.nvmlDeviceGetCurrentClocksThrottleReasons
        while not self.stop_flag:
            try:
                sm = nv.nvmlDeviceGetClockInfo(handle, nv.NVML_CLOCK_SM)
                pw = nv.nvmlDeviceGetPowerUsage(handle) / 1000.0
                self.samples.append((time.time(), float(sm), float(mx), pw, int(reasons(handle))))
            except Exception:
                pass
            time.sleep(0.004)

    def start(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            uuid = None
            try:
                import torch
                uuid = str(torch.cuda.get_device_properties(self.device).uuid)
            except Exception:
                pass
            handle = None
            if uuid:
                for i in range(nv.nvmlDeviceGetCount()):
                    h = nv.nvmlDeviceGetHandleByIndex(i)
                    u = nv.nvmlDeviceGetUUID(h)
                    u = u.decode() if isinstance(u, bytes) else u
                    if uuid in u:
                        handle = h
            if handle is None:
                handle = nv.nvmlDeviceGetHandleByIndex(self.device)
            nv.nvmlDeviceGetClockInfo(handle, nv.NVML_CLOCK_SM)      # fails here rather than in the thread
            self.thread = threading.Thread(target=self._nvml_loop, args=(handle, nv), daemon=True)
            self.thread.start()
            return
        except Exception:
            self.thread = None
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            fields = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
                      "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
                      "clocks_event_reasons.sw_power_cap")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.device), "--query-gpu=" + fields,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def mark(self, t0, t1):
        self.windows.append((t0, t1))

    def _read_smi(self):
        import datetime
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 8:
                    continue
                try:
                    ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    bits = sum(b for (n, b), v in zip(self.REASONS, f[4:8]) if v.lower().startswith("active"))
                    self.samples.append((ts, float(f[1]), float(f[2]), float(f[3]), bits))
                except ValueError:
                    continue
            os.unlink(self.path)
        except Exception:
            pass

    def stop(self):
        if self.stopped:
            return
        self.stopped = True
        if self.thread is not None:
            self.stop_flag = True
            self.thread.join(timeout=2)
        if self.proc is not None:
            time.sleep(0.05)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
            self._read_smi()

    def summary(self):
        def stats(rows):
            if not rows:
                return {"sm_mhz": None, "sm_max_mhz": None, "power_w_max": None, "reasons": [], "samples": 0}
            bits = 0
            for r in rows:
                bits |= r[4]
            return {"sm_mhz": float(np.median([r[1] for r in rows])), "sm_max_mhz": float(max(r[2] for r in rows)),
                    "power_w_max": float(max(r[3] for r in rows)),
                    "reasons": sorted(n for n, b in self.REASONS if bits & b), "samples": len(rows)}
        rows = list(self.samples)
        inside = [r for r in rows if any(t0 <= r[0] <= t1 for t0, t1 in self.windows)]
        out = stats(inside)
        whole = stats(rows)
        if out["samples"] == 0:        # windows shorter than the sampling interval: the whole run stands in
            out = dict(whole, note="no sample fell inside a timed window: figures of the whole run")
        out["whole_run"] = whole
        out["source"] = "NVML queries from a thread, every 4 ms" if self.thread is not None else "nvidia-smi loop, every 20 ms"
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


def oracle_kwargs(c, **kw):
    d = dict(D=c["D"], H=c["H"], N=c["N"], family=c["family"], K=c["K"], L=c["L"], bin_size=c["bin_size"],
             bucket_cap=c["bucket_cap"], lr=c["lr"], seed=0, init_std=0.01, force_dense=int(bool(c.get("force_dense"))))
    d.update(c.get("hidden_lsh", {}))
    d.update(kw)
    return d


# ------------------------------------------------------------------------------------------------
def run_reference(args):
    world, rank, _ = dist_setup(args.gpus)
    if rank != 0:
        return
    from oracle.oracle import Oracle
    c = workloads.config(args.config)
    B = min(REF_BATCH, args.batch_size or c["batch"])
    o = Oracle("float", **oracle_kwargs(c, rebuild_period0=args.rebuild_period, rebuild_lambda=args.rebuild_lambda, redraw=1))
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
    what = "every neuron active (dense limit)" if c.get("force_dense") else "%s K=%d L=%d cap %d" % (
        "DWTA" if c["family"] == workloads.DWTA else "SimHash", c["K"], c["L"], c["bucket_cap"])
    return {"workload": "%s-class shape: D %d, H %d, N %d, %s, batch %d, ~%d nnz/row Zipf(1.1), "
                        "~%d labels/sample" % (c["name"], c["D"], c["H"], c["N"], what, B, c["mean_nnz"], c["mean_labels"]),
            "batch": B, "rebuild_every": args.rebuild_period, "rebuild_lambda": args.rebuild_lambda,
            "distinct_batches": nb, "sampling_budget": args.budget, "hidden_lsh": args.hidden_lsh or "dense hidden layer",
            "l2": "inputs larger than L2: the model state is far larger than L2 and every step reads a different batch "
                  "(different rows)"}


def cpu_baseline(c, args, B):
    """The oracle, untuned, on a bounded sample: a few full-batch steps + one rebuild / period, on one core and
    (its OpenMP build, same source, pinned bit-identical) on all the cores this process may use."""
    from oracle.oracle import Oracle
    out = None
    wl = workloads.Workload(c, seed=0)
    for real in ("float", "float_omp"):
        t_create = time.perf_counter()
        o = Oracle(real, **oracle_kwargs(c, rebuild_period0=0))
        t_create = time.perf_counter() - t_create
        threads = o.threads
        b0 = wl.batch(0, batch_size=B)
        t0 = time.perf_counter()
        o.train_step(*b0)
        t_first = time.perf_counter() - t0
        nsteps = int(max(2, min(8, 10.0 / max(t_first, 1e-3))))        # bounded: about 10 s of steps at most
        batches = [wl.batch(i + 1, batch_size=B) for i in range(nsteps)]
        t0 = time.perf_counter()
        for b in batches:
            o.train_step(*b)
        t_step = (time.perf_counter() - t0) / nsteps
        t_rebuild = 0.0
        if args.rebuild_period and not c.get("force_dense"):
            t0 = time.perf_counter()
            o.rebuild_tables()
            t_rebuild = time.perf_counter() - t0
        o.close()
        per = t_step + (t_rebuild / args.rebuild_period if args.rebuild_period else 0.0)
        rec = {"value": B / per, "unit": "samples/s", "cores": threads, "kind": "oracle",
               "sample": "%d full steps of batch %d (%.3f s each) + one table rebuild (%.2f s) amortised over %d steps"
                         % (nsteps, B, t_step, t_rebuild, args.rebuild_period)}
        if real == "float":
            out = rec
        else:
            out["all_cores"] = rec
        if t_create > 120.0:          # a shape whose model takes minutes to set up on the host: once is enough
            break
    return out


def hidden_lsh(args):
    if not args.hidden_lsh:
        return {}
    k, l, cap = (int(x) for x in args.hidden_lsh.split(","))
    return dict(hidden_K=k, hidden_L=l, hidden_cap=cap)


def make_ctx_config(ds, c, args, B, local):
    return ds.make_config(**hidden_lsh(args), input_dim=c["D"], hidden_dim=c["H"], output_dim=c["N"], hash_family=c["family"], K=c["K"],
                          L=c["L"], dwta_bin_size=c["bin_size"], bucket_cap=c["bucket_cap"],
                          rebuild_period0=args.rebuild_period, rebuild_growth_lambda=args.rebuild_lambda, redraw_hash_fns=1,
                          force_dense=int(bool(c.get("force_dense"))),
                          max_batch=B, max_labels=c["max_labels"], lr=c["lr"], init_std=0.01, seed=0, device=local,
                          sample_budget=args.budget, inputs_ready=1)


def measure(args, c, B, world, rank, local, windows, with_e2e, with_cpu, sampler):
    """All the timed passes for one workload; returns the JSON record (rank 0) or None."""
    import torch
    from paper_2201_12667_b200 import binding as ds
    if world > 1:
        import torch.distributed as dist

    K, W = args.steps, max(args.warmup, 3)
    cfg = make_ctx_config(ds, c, args, B, local)
    wl = workloads.Workload(c, seed=shard_seed(rank))
    nb = min(args.batches, K + W)
    host = [wl.batch(i, batch_size=B) for i in range(nb)]
    labels_per_step = float(np.mean([len(b[4]) for b in host]))
    dev = [[torch.from_numpy(a).cuda() for a in b] for b in host]
    loss = torch.zeros(1, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def rebuilds(ctx):
        return int(ds.dslide_get_tensor(ctx, "counters")[1])

    # ---- timed windows: K steps each, inputs resident in HBM, every window on a fresh model after the same warm-up
    #      (the active sets grow as the model trains: a later window of steps touches more rows) ----
    win_ms, win_rebuilds, launches, status, cum = [], [], 0, 0, None
    ctx = None
    for w in range(windows):
        if ctx is not None:
            ds.dslide_destroy(ctx)
        ctx = ds.dslide_init(cfg)
        for i in range(W):
            ds.dslide_train_step(ctx, B, *dev[i % nb], loss)
        ds.dslide_sync(ctx)
        ds.dslide_cum_stats(ctx, reset=True)
        r0 = rebuilds(ctx)
        launches0 = ds.dslide_kernel_launches(ctx)
        barrier()
        t0 = time.time()
        e0.record()
        for i in range(K):
            ds.dslide_train_step(ctx, B, *dev[(W + i) % nb], loss)
        e1.record()
        barrier()
        if sampler is not None:
            sampler.mark(t0, time.time())
        win_ms.append(max_over_ranks(e0.elapsed_time(e1), world, "cuda"))
        win_rebuilds.append(rebuilds(ctx) - r0)
        launches = ds.dslide_kernel_launches(ctx) - launches0
        status |= ds.dslide_sync(ctx, check=False)
        cum = ds.dslide_cum_stats(ctx, reset=True)

    # ---- one rebuild, timed by itself with CUDA events on the model the last window left (three of them, median) ----
    rebuild_ms = 0.0
    if args.rebuild_period and not c.get("force_dense"):
        ts = []
        for _ in range(3):
            barrier()
            e0.record()
            ds.dslide_rebuild_tables(ctx)
            e1.record()
            barrier()
            ts.append(e0.elapsed_time(e1))
        rebuild_ms = max_over_ranks(float(np.median(ts)), world, "cuda")
    med = int(np.argsort(win_ms)[len(win_ms) // 2])
    ms_step, how = full_step_ms(win_ms[med], K, win_rebuilds[med], rebuild_ms, args.rebuild_period)
    value = world * B / (ms_step * 1e-3)

    # ---- a pass of the same K steps with a CUDA event pair around every kernel launch, fresh model, same warm-up ----
    ds.dslide_destroy(ctx)
    ctx = ds.dslide_init(cfg)
    for i in range(W):
        ds.dslide_train_step(ctx, B, *dev[i % nb], loss)
    ds.dslide_sync(ctx)
    ds.dslide_cum_stats(ctx, reset=True)
    ds.dslide_profile_begin(ctx)
    for i in range(K):
        ds.dslide_train_step(ctx, B, *dev[(W + i) % nb], loss)
    prof = ds.dslide_profile_end(ctx)
    cum_prof = ds.dslide_cum_stats(ctx, reset=True)      # the per-kernel times go with the rows these steps touched

    # ---- end to end: host buffers in, loss out, every step ----
    e2e = None
    if with_e2e:
        # the pipelined host-buffer entry point: every step copies its inputs from pinned host memory to the device
        # and its {status, loss} back; the loss of step i is handed out by call i + 1 (the last one by
        # dslide_host_result), so the device always has one step queued while the host packs the next
        pinned = [[torch.from_numpy(a).pin_memory() for a in b] for b in host]
        ds.dslide_destroy(ctx)
        ctx = ds.dslide_init(cfg)
        for i in range(W):
            ds.dslide_train_step_host_async(ctx, B, *pinned[i % nb])
        ds.dslide_host_result(ctx)
        r0 = rebuilds(ctx)
        barrier()
        t0 = time.time()
        e0.record()
        losses = 0
        for i in range(K):
            losses += ds.dslide_train_step_host_async(ctx, B, *pinned[(W + i) % nb]) is not None
        losses += ds.dslide_host_result(ctx) is not None
        e1.record()
        barrier()
        if sampler is not None:
            sampler.mark(t0, time.time())
        assert losses == K
        ms_e2e = max_over_ranks(e0.elapsed_time(e1), world, "cuda")
        e2e_step, e2e_how = full_step_ms(ms_e2e, K, rebuilds(ctx) - r0, rebuild_ms, args.rebuild_period)
        h2d = float(np.mean([sum(a.numel() * a.element_size() for a in b) for b in pinned]))
        e2e = {"value": world * B / (e2e_step * 1e-3), "unit": "samples/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": 8, "ms_per_step": e2e_step, "rebuild_accounting": e2e_how,
               "api": "dslide_train_step_host_async + dslide_host_result (loss and status of every step read back)"}
    ds.dslide_destroy(ctx)

    if rank != 0:
        return None
    per_step = {k: cum[k] / max(1, cum["steps"]) for k in ("nnz", "sum_active", "touched_w1", "touched_w2", "fetched")}
    model = byte_model(c, B, per_step, labels_per_step, args.rebuild_period)
    peak, peak_kind = hbm_peak()
    total_prof = sum(v[0] for v in prof.values()) or 1.0
    kernels = {}
    for name, (kms, cnt) in sorted(prof.items(), key=lambda kv: -kv[1][0]):
        kernels[name] = {"launches": cnt, "ms_total": kms, "us_per_launch": 1e3 * kms / cnt, "share": kms / total_prof}
    step_kernels = [n for n in prof if n in ("adam", "forward", "adam_dense")]
    dominant = max(step_kernels, key=lambda n: prof[n][0])
    dur = prof[dominant][0] * 1e-3 / prof[dominant][1]
    per_step_prof = {k: cum_prof[k] / max(1, cum_prof["steps"]) for k in per_step}
    model_prof = byte_model(c, B, per_step_prof, labels_per_step, args.rebuild_period)
    booked = model_prof["adam" if dominant == "adam_dense" else dominant]
    achieved = booked / dur / 1e9
    step_gbs = model["total"] / (ms_step * 1e-3) / 1e9
    rebuild_us = 1e3 * rebuild_ms / args.rebuild_period if args.rebuild_period else 0.0
    roofline = {"bound": "hbm", "kernel": {"adam": "k_update", "adam_dense": "k_adam_dense", "forward": "k_forward"}[dominant], "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": ncu_traffic(dominant, model_prof),
                "algorithmic_bytes_per_launch": booked, "us_per_launch": dur * 1e6,
                "peak_source": "MEASURED_PEAKS.json hbm_gbs (of %s)" % peak_kind,
                "whole_step": {"algorithmic_bytes_per_step": model["total"], "achieved": step_gbs,
                               "frac": step_gbs / peak, "frac_of_8TBps_nominal": step_gbs / 8000.0,
                               "target": "0.50 of the HBM roofline for the full step",
                               "target_met": bool(step_gbs / peak >= 0.5)}}
    out = {
        "metric": METRIC, "value": value, "unit": "samples/s", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic", "config": workload_config(c, B, args, nb),
        "clocks": sampler.summary() if sampler is not None else None, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": roofline,
        "windows": {"ms": win_ms, "rebuilds_inside": win_rebuilds, "median_index": med,
                    "rebuild_ms": rebuild_ms, "rebuild_accounting": how},
        "step_roofline": {"algorithmic_bytes_per_step": model["total"], "rebuild_bytes_per_step": model["rebuild"],
                          "achieved": step_gbs, "peak": peak,
                          "unit": "GB/s", "frac": step_gbs / peak, "frac_of_8TBps_nominal": step_gbs / 8000.0,
                          "issued_bytes_per_step": model["issued"],
                          "issued_gbs": model["issued"] / (ms_step * 1e-3) / 1e9,
                          "us_per_step": 1e3 * ms_step, "rebuild_us_per_step_amortised": rebuild_us,
                          "us_per_step_without_rebuild": 1e3 * ms_step - rebuild_us},
        "kernels": kernels,
        "per_step": dict(per_step, labels=labels_per_step, active_fraction=per_step["sum_active"] / B / c["N"]),
        "device_status": int(status),
    }
    if with_cpu:
        out["cpu_baseline"] = cpu_baseline(c, args, B)
    return out


def run_dslide(args):
    import torch
    world, rank, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the dslide arm")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    sampler = None
    if rank == 0:
        sampler = ClockSampler(local)
        sampler.start()
    try:
        if args.sweep:
            run_sweep(args, world, rank, local)
        elif args.predict:
            out = run_predict(args, world, rank, local)
            if out is not None:
                sampler.stop()
                out["clocks"] = sampler.summary()
                print(json.dumps(out))
        else:
            c = workloads.config(args.config)
            c["hidden_lsh"] = hidden_lsh(args)
            B = args.batch_size or c["batch"]
            out = measure(args, c, B, world, rank, local, max(1, args.windows), not args.no_e2e,
                          world == 1 and not args.no_cpu_baseline, sampler)
            if out is not None:
                sampler.stop()
                out["clocks"] = sampler.summary()
                print(json.dumps(out))
    finally:
        if sampler is not None:
            sampler.stop()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_predict(args, world, rank, local):
    """Top-k inference on batches resident in HBM, CUDA events on the library's stream: over the neurons the tables
    retrieve (Algorithm 1's forward pass without labels) and over all neurons (Section 3.6: layer sparsity 1; on the
    tensor pipe when k <= 8).  Weights are the random initialisation: the work per batch does not depend on them."""
    import torch
    from paper_2201_12667_b200 import binding as ds
    c = workloads.config(args.config)
    B = args.batch_size or c["batch"]
    k, K, W = args.predict, args.steps, max(args.warmup, 3)
    ctx = ds.dslide_init(make_ctx_config(ds, c, args, B, local))
    wl = workloads.Workload(c, seed=shard_seed(rank))
    nb = min(args.batches, 16)
    dev = [[torch.from_numpy(a).cuda() for a in wl.batch(i, B)[:3]] for i in range(nb)]
    ids = torch.zeros(B * k, dtype=torch.int32, device="cuda")
    sc = torch.zeros(B * k, dtype=torch.float32, device="cuda")
    res = {}
    for name, dense in (("retrieved", 0), ("all_neurons", 1)):
        n = K if not dense else max(3, K // 10)
        for i in range(W):
            ds.dslide_predict_topk(ctx, B, *dev[i % nb], k, dense, ids, sc)
        ds.dslide_sync(ctx)
        barrier = (lambda: None) if world == 1 else torch.distributed.barrier
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()           # the context enqueues on torch's current stream
        for i in range(n):
            ds.dslide_predict_topk(ctx, B, *dev[(W + i) % nb], k, dense, ids, sc)
        e1.record()
        ds.dslide_sync(ctx)
        barrier()
        ms = max_over_ranks(e0.elapsed_time(e1), world, "cuda") / n
        res[name] = {"value": world * B / (ms * 1e-3), "unit": "samples/s", "us_per_batch": 1e3 * ms, "calls": n}
    status = ds.dslide_sync(ctx, check=False)
    ds.dslide_destroy(ctx)
    if rank != 0:
        return None
    peak, peak_kind = hbm_peak()
    w2_bytes = c["N"] * (c["H"] * 4 + 16)                       # every row of W2 and its record, read once per call
    d_us = res["all_neurons"]["us_per_batch"]
    groups = (B + 127) // 128
    res["all_neurons"]["roofline"] = {
        "bound": "hbm", "kernel": "k_dense_tc" if k <= 8 and c["H"] % 32 == 0 and c["H"] <= 256 else "k_predict_dense",
        "achieved": w2_bytes / (d_us * 1e-6) / 1e9, "peak": peak, "unit": "GB/s", "frac": w2_bytes / (d_us * 1e-6) / 1e9 / peak,
        "traffic": None, "algorithmic_bytes_per_call": w2_bytes, "peak_source": "MEASURED_PEAKS.json hbm_gbs (of %s)" % peak_kind,
        "tf32_tflops": 2.0 * groups * 128 * c["N"] * c["H"] / (d_us * 1e-6) / 1e12,
        "note": "whole call (hidden layer, threshold pass, filter pass, exact pass), not one kernel"}
    return {"metric": "top-%d inference samples/s at the %s shape on %d B200" % (k, args.config, world),
            "value": res["retrieved"]["value"], "unit": "samples/s", "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": res["retrieved"]["us_per_batch"] * 1e-3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": dict(workload_config(c, B, args, nb), predict_k=k), "retrieved": res["retrieved"],
            "all_neurons": res["all_neurons"], "device_status": int(status)}


def run_sweep(args, world, rank, local):
    """Batch size x target active fraction on the 670K shape (the large-batch claim of Section 3.4 and the dense limit
    of Section 3.6): one JSON line per cell, rebuild gaps growing by exp(0.1 * rebuilds) from 50 steps."""
    batches = [int(x) for x in args.sweep_batches.split(",") if x] or list(SWEEP_BATCHES)
    want = [float(x) for x in args.sweep_fractions.split(",") if x]
    for frac, over in SWEEP_FRACTIONS:
        if want and not any(abs(frac - w) < 1e-9 for w in want):
            continue
        for B in batches:
            c = workloads.config("670k", **over)
            a = argparse.Namespace(**vars(args))
            a.rebuild_lambda = 0.1
            a.steps, a.warmup, a.batches = min(args.steps, 20), min(max(args.warmup, 3), 5), 8
            out = measure(a, c, B, world, rank, local, 1, False, False, None)
            if out is not None:
                cell = {"sweep_cell": {"batch": B, "target_active_fraction": frac,
                                       "measured_active_fraction": out["per_step"]["active_fraction"], "K": c["K"], "L": c["L"],
                                       "bucket_cap": c["bucket_cap"], "force_dense": int(bool(c.get("force_dense")))}}
                cell.update({k: out[k] for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step",
                                                 "higher_is_better", "dtype", "data", "config", "roofline", "step_roofline",
                                                 "kernels", "per_step", "windows", "device_status")})
                print(json.dumps(cell), flush=True)


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_dslide(a)
