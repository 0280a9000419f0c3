"""Benchmark of the batch-size-test hot path on B200.

One step = one pass of the whole path over one batch of synthetic per-sample gradients:
  abs_test_stats (mean gradient, norm / inner-product / orthogonality variances)
  -> abs_next_batch (ceilings, max over workers, cap)
  -> local_adamw_step on the mean gradient with the model averaging fused in.
The headline value is the bytes of G the step consumes divided by the step time (GB/s);
rounds/s is its reciprocal.  Extra legs time the fused AdamW / SGD steps and the bf16
statistics on their own workloads.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-extra]
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOAD = dict(name="stats sweep centre: G fp32 [M=1, b=256, d=11.2M], sigma=1, eta=theta=nu=0.5",
                M=1, b=256, d=11_200_000, sigma=1.0, seed=2)
HP = dict(lr=3e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)
FALLBACK_HBM_GBS = 6650.0
LEG_PAUSE_S = 0.5
# DRAM bytes (read + write) of one abs_stats_tiled_kernel<float,16,keep,full> launch on the 1.024 GB case
# of profiles/stats_tiled_f32_b256_d1m.txt; traffic grows in proportion to the columns processed.
NCU_TRAFFIC_SMALL = dict(dram_bytes=1.024040e9 + 3.832e6, d=1_000_000)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 7:
                    continue
                try:
                    sm.append(float(parts[0]))
                    mx.append(float(parts[1]))
                except ValueError:
                    continue
                for name, val in zip(names, parts[3:7]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            sm.sort()
            out.update(sm_mhz=sm[len(sm) // 2], sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# --------------------------------------------------------------------------- CPU oracle legs
def oracle_step(G_np, x, m, v, b, t):
    """The whole step in the CPU oracle, as it stands."""
    import oracle.abs_oracle as orc
    s = orc.batch_test_stats(G_np)
    orc.next_batch([s], b, 1 << 20, "aug_ip", theta=0.5, nu=0.5)
    orc.next_batch([s], b, 1 << 20, "norm", eta=0.5)
    x, m, v = orc.adamw_step(x, m, v, s["gbar"][None, :], t=t, **HP)
    return orc.replica_average(x), m, v


def cpu_sample(divisor=4):
    import numpy as np
    from paper_2406_13936_b200 import inputs
    b, d = WORKLOAD["b"], WORKLOAD["d"] // divisor
    G = inputs.gaussian_rows(WORKLOAD["seed"], 1, b, d, WORKLOAD["sigma"], device="cpu")[0].numpy()
    x = np.zeros((1, d))
    return G, x, "first %d of %d columns (1/%d of the workload), all %d rows" % (d, WORKLOAD["d"], divisor, b)


def _limit_blas_threads():
    """One thread per process: the vector products of the oracle would otherwise be spread over all
    cores by the BLAS library and the stated core count would be wrong."""
    try:
        from threadpoolctl import threadpool_limits
        return threadpool_limits(limits=1)
    except Exception:
        return None


_POOL_SHM = None


def _pool_attach(name, shape):
    """Initialiser of an oracle worker process: attaches to the shared sample."""
    global _POOL_SHM
    import numpy as np
    from multiprocessing import shared_memory
    import oracle.abs_oracle  # noqa: F401  (imported before the clock starts)
    _limit_blas_threads()
    shm = shared_memory.SharedMemory(name=name)
    _POOL_SHM = (shm, np.ndarray(shape, dtype=np.float32, buffer=shm.buf))


def _pool_block(job):
    """The whole oracle step on one column block of the shared sample."""
    import numpy as np
    lo, hi, b = job
    if hi <= lo:
        return 0.0
    G = _POOL_SHM[1][:, lo:hi]
    x = np.zeros((1, hi - lo))
    t0 = time.perf_counter()
    oracle_step(G, x, np.zeros_like(x), np.zeros_like(x), b, 1)
    return time.perf_counter() - t0


def time_cpu_baseline():
    """The oracle as it stands on a quarter of the columns: on one core, and with one process per host
    core, each taking a block of the same columns (the processes are spawned, never forked)."""
    import multiprocessing as mp
    import numpy as np
    from multiprocessing import shared_memory
    G, x, what = cpu_sample()
    limit = _limit_blas_threads()
    t0 = time.perf_counter()
    oracle_step(G, x, np.zeros_like(x), np.zeros_like(x), WORKLOAD["b"], 1)
    dt = time.perf_counter() - t0
    del limit
    out = dict(value=G.nbytes / dt / 1e9, unit="GB/s", cores=1, kind="oracle", sample=what, seconds=round(dt, 3))
    cores = os.cpu_count() or 1
    try:
        cores = len(os.sched_getaffinity(0))
    except Exception:
        pass
    procs = min(cores, 64)
    shm = shared_memory.SharedMemory(create=True, size=G.nbytes)
    try:
        shared = np.ndarray(G.shape, dtype=np.float32, buffer=shm.buf)
        shared[:] = G
        d = G.shape[1]
        edges = [d * k // procs for k in range(procs + 1)]
        jobs = [(edges[k], edges[k + 1], WORKLOAD["b"]) for k in range(procs)]
        with mp.get_context("spawn").Pool(procs, initializer=_pool_attach, initargs=(shm.name, G.shape)) as pool:
            pool.map(_pool_block, [(0, 1, WORKLOAD["b"])] * procs)        # every process up and attached
            t0 = time.perf_counter()
            pool.map(_pool_block, jobs, chunksize=1)
            dt_all = time.perf_counter() - t0
        out["all_cores"] = dict(value=G.nbytes / dt_all / 1e9, unit="GB/s", cores=procs, host_cores=cores,
                                kind="oracle", sample=what + ", one column block per process",
                                seconds=round(dt_all, 3))
    except Exception as e:      # a box that cannot spawn processes still reports the single-core figure
        out["all_cores"] = dict(unavailable=str(e)[:200])
    finally:
        shm.close()
        shm.unlink()
    return out


def run_reference(args):
    """The oracle timed on the host cores on a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    G, x, what = cpu_sample(divisor=16)
    m, v = np.zeros_like(x), np.zeros_like(x)
    for t in range(args.warmup):
        oracle_step(G, x, m, v, WORKLOAD["b"], t + 1)
    t0 = time.perf_counter()
    for t in range(args.steps):
        oracle_step(G, x, m, v, WORKLOAD["b"], t + 1)
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    value = G.nbytes / dt / 1e9
    line = dict(impl="reference", metric="batch_test_step_GBps", value=value, unit="GB/s", n_gpus=args.gpus,
                steps=args.steps, warmup=args.warmup, ms_per_step=dt * 1e3, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=WORKLOAD["name"], sample=what),
                cpu_baseline=dict(value=value, unit="GB/s", cores=1, kind="oracle", sample=what),
                e2e=dict(value=value, unit="GB/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line))


def aggregate_over_ranks(seconds, units_per_rank, dist=None, device="cuda"):
    """Whole-job figures of a weak-scaling run: every rank processed `units_per_rank` in `seconds` of its
    own; returns (maximum of the ranks' times, all ranks' units divided by it).  dist=None: one rank."""
    world = 1
    if dist is not None:
        import torch
        world = dist.get_world_size()
        t = torch.tensor([seconds], dtype=torch.float64, device=device)
        dist.barrier()
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        seconds = float(t.item())
    return seconds, world * units_per_rank / seconds


# --------------------------------------------------------------------------- GPU legs
def time_steps(torch, fn, steps, warmup):
    """CUDA-event timing of `steps` calls of fn(i) after `warmup` untimed ones; returns seconds per call.
    Every leg starts from an idle GPU (a short pause): a leg measured right after a long one ran
    10-35 % slower here."""
    torch.cuda.synchronize()
    time.sleep(LEG_PAUSE_S)
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        fn(warmup + i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / 1e3 / steps


def extra_legs(torch, pkg, inputs, ctx, peak, steps, warmup):
    """The nine-cell statistics sweep, fused optimiser steps and bf16 statistics on their own workloads
    (not the headline)."""
    out = {}
    # The short statistics legs come first: run after the long optimiser legs they measured 10-35 %
    # lower (fp32 [1, 4, 124 M]: 4.5 instead of 7.0 TB/s), the long legs themselves do not care.
    # the worker-gradient estimator's shape: the rows are the batch gradients of 4 or 8 workers
    if torch.cuda.mem_get_info()[0] > 20e9:
        for rows, dt, name in ((4, torch.float32, "f32"), (8, torch.float32, "f32"), (4, torch.bfloat16, "bf16"),
                               (8, torch.bfloat16, "bf16")):
            G = inputs.gaussian_rows(2, 1, rows, 124_439_808, 1.0, device="cuda", dtype=dt)
            stats = ctx.new_stats(1)
            sec = time_steps(torch, lambda i: ctx.abs_test_stats(G, stats), 10, 3)
            gbs = G.numel() * G.element_size() / sec / 1e9
            out["stats_%s_rows%d" % (name, rows)] = dict(workload="G %s [1, %d, 124,439,808]" % (name, rows),
                                                         ms=sec * 1e3, GBps=gbs, frac_of_peak=gbs / peak)
            del G
            torch.cuda.empty_cache()
    # bf16 statistics with more rows per worker: the tcgen05 Gram kernel (32 < b <= 256)
    if torch.cuda.mem_get_info()[0] > 20e9:
        for bb, dd in ((64, 22_400_000), (128, 11_200_000), (256, 11_200_000)):
            G = inputs.gaussian_rows(2, 1, bb, dd, 1.0, device="cuda", dtype=torch.bfloat16)
            stats = ctx.new_stats(1)
            sec = time_steps(torch, lambda i: ctx.abs_test_stats(G, stats), 10, 3)
            gbs = G.numel() * 2 / sec / 1e9
            out["stats_bf16_b%d" % bb] = dict(workload="G bf16 [1, %d, %s]" % (bb, format(dd, ",")), ms=sec * 1e3,
                                              GBps=gbs, frac_of_peak=gbs / peak)
            del G
            torch.cuda.empty_cache()
    # the nine cells of the statistics sweep (behind the short legs above, before the long ones below)
    out["sweep"] = stats_sweep(torch, pkg, inputs, ctx, peak, steps, warmup)
    out["worst_cell"] = worst_cell(out["sweep"])
    # the sweep's other two noise levels on its centre cell: the same bytes are read whatever sigma is
    out["sweep_sigma"] = []
    for sigma in (0.1, 10.0):
        G = inputs.gaussian_rows(2, 1, 256, 11_200_000, sigma, device="cuda")
        stats = ctx.new_stats(1)
        sec = time_steps(torch, lambda i: ctx.abs_test_stats(G, stats), 10, 3)
        gbs = G.numel() * 4 / sec / 1e9
        out["sweep_sigma"].append(dict(b=256, d=11_200_000, sigma=sigma, ms=sec * 1e3, GBps=gbs, frac_of_peak=gbs / peak))
        del G
        torch.cuda.empty_cache()
    free = torch.cuda.mem_get_info()[0]
    # fused local AdamW + averaging: M=8 fp32 replicas of a GPT-2-small-sized model, H=16 steps per round
    M, d, H = 8, 124_439_808, 16
    if free > 40e9:
        X, m1, m2, grads = inputs.adamw_problem(4, M, d, pool=2, device="cuda")
        t = [0]

        def adamw(i, avg=False):
            t[0] += 1
            ctx.local_adamw_step(X, m1, m2, grads[i % 2], pkg.make_adamw_cfg(step=t[0], **HP), average_after=avg)

        sec = time_steps(torch, adamw, 8, 3)
        sec_avg = time_steps(torch, lambda i: adamw(i, True), 8, 3)
        gbs = 28.0 * M * d / sec / 1e9
        out["adamw_step"] = dict(workload="M=8 d=124,439,808 fp32, 28 B/element", ms=sec * 1e3, GBps=gbs,
                                 frac_of_peak=gbs / peak, ms_with_fused_average=sec_avg * 1e3,
                                 GBps_with_fused_average=28.0 * M * d / sec_avg / 1e9)
        round_s = (H - 1) * sec + sec_avg
        out["adamw_round"] = dict(workload="H=16 local AdamW steps, averaging fused into the last",
                                  rounds_per_s=1.0 / round_s, ms_per_round=round_s * 1e3)
        sec = time_steps(torch, lambda i: ctx.local_sgd_step(X, grads[i % 2], 1e-3), 8, 3)
        out["sgd_step"] = dict(workload="M=8 d=124,439,808 fp32, 12 B/element", ms=sec * 1e3,
                               GBps=12.0 * M * d / sec / 1e9, frac_of_peak=12.0 * M * d / sec / 1e9 / peak)
        sec = time_steps(torch, lambda i: ctx.local_shb_step(X, m1, grads[i % 2], 1e-3, 0.9, 1e-4), 8, 3)
        out["shb_step"] = dict(workload="M=8 d=124,439,808 fp32, 20 B/element", ms=sec * 1e3,
                               GBps=20.0 * M * d / sec / 1e9, frac_of_peak=20.0 * M * d / sec / 1e9 / peak)
        sec = time_steps(torch, lambda i: ctx.replica_average(X), 8, 3)
        out["replica_average"] = dict(workload="stand-alone, 8 B/element/replica", ms=sec * 1e3,
                                      GBps=8.0 * M * d / sec / 1e9, frac_of_peak=8.0 * M * d / sec / 1e9 / peak)
        del X, m1, m2, grads
        torch.cuda.empty_cache()
    # bf16 statistics: M=8 workers x 16 micro-batch gradients of a GPT-2-small-sized model
    free = torch.cuda.mem_get_info()[0]
    M, b = 8, 16
    if free > 45e9:
        G = inputs.student_t_rows(3, M, b, d, device="cuda")
        stats = ctx.new_stats(M)
        sec = time_steps(torch, lambda i: ctx.abs_test_stats(G, stats), 10, 3)
        gbs = G.numel() * 2 / sec / 1e9
        out["stats_bf16"] = dict(workload="G bf16 [8, 16, 124,439,808] Student-t rows", ms=sec * 1e3, GBps=gbs,
                                 frac_of_peak=gbs / peak)
        del G
        torch.cuda.empty_cache()
    # fp32 statistics at the large-batch end of the sweep (rows split over a thread-block cluster)
    if torch.cuda.mem_get_info()[0] > 60e9:
        G = inputs.gaussian_rows(2, 1, 1024, 11_200_000, 1.0, device="cuda")
        stats = ctx.new_stats(1)
        sec = time_steps(torch, lambda i: ctx.abs_test_stats(G, stats), 5, 3)
        gbs = G.numel() * 4 / sec / 1e9
        out["stats_f32_b1024"] = dict(workload="G fp32 [1, 1024, 11,200,000]", ms=sec * 1e3, GBps=gbs,
                                      frac_of_peak=gbs / peak)
        del G
        torch.cuda.empty_cache()
    out["rounds_logreg"] = end_to_end_rounds(torch, pkg, inputs, ctx, "logreg")
    try:
        out["rounds_logreg_fused"] = logreg_rounds_fused(torch, pkg, inputs, ctx)
    except pkg.AbsError as e:      # e.g. a tool that refuses cooperative cluster launches
        out["rounds_logreg_fused"] = dict(unavailable=str(e))
    try:
        out["rounds_logreg_fused_every_step"] = logreg_rounds_fused(torch, pkg, inputs, ctx, every_step=True)
    except pkg.AbsError as e:
        out["rounds_logreg_fused_every_step"] = dict(unavailable=str(e))
    out["rounds_mlp"] = end_to_end_rounds(torch, pkg, inputs, ctx, "mlp")
    out["rounds_mlp_fused_stats"] = end_to_end_rounds(torch, pkg, inputs, ctx, "mlp_fused")
    return out


def end_to_end_rounds(torch, pkg, inputs, ctx, which):
    """rounds/s of the two end-to-end configurations (producer + statistics + local SGD + averaging +
    batch-size update per round; the batch size is read back once per round to size the next one)."""
    if which == "logreg":
        n, d, M, H, lr, b, b_max, rounds = 65536, 256, 4, 8, 0.1, 16, 1024, 50
        A, y = inputs.logreg_dataset(1, n, d, device="cuda")
        cfg = pkg.make_test_cfg("norm", b_max, eta=0.5)
        X = torch.zeros((M, d), device="cuda")
        G = torch.empty((M, b_max, d), device="cuda")
    else:
        dims = (784, 1024, 1024, 10)
        n, M, H, lr, b, b_max, rounds = 1_048_576, 8, 4, 0.01, 32, 4096, 200
        inp, lab = inputs.gaussian_mixture(5, n, dim=dims[0], classes=dims[3], device="cuda")
        d = ctx.mlp_param_count(dims)
        X = inputs.mlp_init(6, dims, device="cuda").unsqueeze(0).repeat(M, 1).contiguous()
        cfg = pkg.make_test_cfg("aug_ip", b_max, theta=0.5, nu=0.5)
        stride = (d + 3) // 4 * 4
        scratch = ctx.mlp_scratch(M, b_max, dims)
        # "mlp": per-sample gradient rows are written out and read by abs_test_stats;
        # "mlp_fused": the statistics come from activations and deltas (abs_mlp_fused_stats)
        G = torch.empty((b_max, stride), device="cuda") if which == "mlp" else None
    idx = inputs.batch_indices(11, (rounds, H, M, b_max), n, device="cuda")
    Gb = torch.empty((M, d), device="cuda")
    stats = ctx.new_stats(M)
    b_dev = torch.tensor([b], dtype=torch.int64, device="cuda")
    def one_round(k, b):
        if which == "logreg":
            ctx.abs_logreg_round(A, y, idx[k], X, H, b, lr, cfg, G, Gb, stats, b_dev)
        else:
            ctx.abs_mlp_round(inp, lab, dims, idx[k], X, H, b, lr, cfg, scratch, G, stride, Gb, stats, b_dev)
        return int(b_dev.item())       # one 8-byte read-back per round

    # three untimed rounds (module loading, first-call queries), then the run starts over from x_0, b_0
    X0, b0 = X.clone(), b
    for k in range(3):
        b = one_round(k, b)
    X.copy_(X0)
    b = b0
    b_dev.fill_(b0)
    history = [b]
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for k in range(rounds):
        b = one_round(k, b)
        history.append(b)
    torch.cuda.synchronize()
    sec = time.perf_counter() - t0
    return dict(rounds=rounds, rounds_per_s=rounds / sec, seconds=sec, M=M, H=H, b_first=history[0],
                b_last=history[-1], rounds_until_cap=next((i for i, v in enumerate(history) if v >= b_max), None))


def logreg_rounds_fused(torch, pkg, inputs, ctx, every_step=False):
    """The logistic configuration with all 50 rounds in one cooperative launch (abs_logreg_rounds_fused:
    parameters in shared memory, batch size on the device, no per-sample gradient matrix), and with one
    launch per round; CUDA-event time of the launches, after one untimed run.  every_step: Algorithm 1's
    cadence (the test after every local step, one size per worker, sample counter on the device)."""
    n, d, M, H, lr, b0, b_max, rounds = 65536, 256, 4, 8, 0.1, 16, 1024, 50
    A, y = inputs.logreg_dataset(1, n, d, device="cuda")
    cfg = pkg.make_test_cfg("norm", b_max, eta=0.5)
    idx = inputs.batch_indices(11, (rounds, H, M, b_max), n, device="cuda")
    per = H if every_step else 1
    stats = ctx.new_stats(rounds * per * M)
    hist = torch.zeros((rounds + 1) if not every_step else (rounds * H * M), dtype=torch.int64, device="cuda")
    out = dict(rounds=rounds, M=M, H=H)
    ctl, opts = None, None
    for mode in ("one_launch", "launch_per_round"):
        best = None
        for rep in range(4):
            if every_step:     # fresh counters for every run
                ctl = ctx.new_round_ctl()
                opts = pkg.make_round_opts(test_every_step=True, per_worker=True, ctl=ctl)
            X = torch.zeros((M, d), device="cuda")
            b_dev = torch.full((M if every_step else 1,), b0, dtype=torch.int64, device="cuda")
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            if mode == "one_launch":
                if every_step:
                    ctx.abs_logreg_rounds_fused_opts(A, y, idx, X, H, lr, cfg, opts, stats, b_dev, b_hist=hist)
                else:
                    ctx.abs_logreg_rounds_fused(A, y, idx, X, H, lr, cfg, stats, b_dev, b_hist=hist)
            else:
                for k in range(rounds):
                    if every_step:
                        ctx.abs_logreg_rounds_fused_opts(A, y, idx[k:k + 1], X, H, lr, cfg, opts,
                                                         stats[k * per * M:(k + 1) * per * M], b_dev)
                    else:
                        ctx.abs_logreg_rounds_fused(A, y, idx[k:k + 1], X, H, lr, cfg, stats[k * M:(k + 1) * M], b_dev)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            if rep > 0:
                best = ms if best is None else min(best, ms)
        out[mode] = dict(rounds_per_s=rounds / (best * 1e-3), us_per_round=best * 1e3 / rounds)
    h = hist.tolist()
    if every_step:
        out.update(b_first=h[0], b_last=max(h), samples=int(ctl[0].item()))
    else:
        out.update(b_first=h[0], b_last=h[-1], rounds_until_cap=next((i for i, v in enumerate(h) if v >= b_max), None))
    return out


PROFILE_CASES = {
    # small cases of the same kernels for profiler captures: larger than L2, about 1 GB on the device
    "stats_f32_b256": dict(kind="stats", M=1, b=256, d=1_000_000, dtype="f32"),
    "stats_f32_b64": dict(kind="stats", M=1, b=64, d=4_000_000, dtype="f32"),
    "stats_f32_b1024": dict(kind="stats", M=1, b=1024, d=256_000, dtype="f32"),
    "stats_bf16_b16": dict(kind="stats", M=8, b=16, d=4_000_000, dtype="bf16"),
    "stats_bf16_b64": dict(kind="stats", M=1, b=64, d=8_000_000, dtype="bf16"),
    "stats_bf16_b128": dict(kind="stats", M=1, b=128, d=4_000_000, dtype="bf16"),
    "stats_bf16_b256": dict(kind="stats", M=1, b=256, d=2_000_000, dtype="bf16"),
    "adamw": dict(kind="adamw", M=8, d=8_000_000),
    "logreg_fused": dict(kind="logreg_fused"),          # the 50 rounds of the logistic configuration, fused
    "mlp_grads": dict(kind="mlp_grads", M=2, b=1024),   # forward/backward of the 784-1024-1024-10 MLP (tensor-core products)
    # full-size cases of the sweep, for timing only (not for multi-pass captures)
    "stats_f32_b64_d11m": dict(kind="stats", M=1, b=64, d=11_200_000, dtype="f32"),
    "stats_f32_b256_d11m": dict(kind="stats", M=1, b=256, d=11_200_000, dtype="f32"),
    "stats_f32_b1024_d11m": dict(kind="stats", M=1, b=1024, d=11_200_000, dtype="f32"),
    "stats_bf16_b16_d124m": dict(kind="stats", M=8, b=16, d=124_439_808, dtype="bf16"),
}


def run_profile_case(args):
    """A few launches of one kernel on a small case (for ncu); prints its CUDA-event time."""
    import torch
    import paper_2406_13936_b200 as pkg
    from paper_2406_13936_b200 import inputs
    if args.shape:
        M_, b_, d_, dt_ = args.shape.split(",")
        case = dict(kind="stats", M=int(M_), b=int(b_), d=int(d_), dtype=dt_)
        args.case = "shape:" + args.shape
    else:
        case = PROFILE_CASES[args.case]
    pkg.build.build()
    ctx = pkg.Context(0)
    for kv in args.tune:
        key, val = kv.split("=")
        ctx.set_tuning(key, int(val))
    peak, _ = measured_peak()
    if case["kind"] == "logreg_fused":
        print(json.dumps(dict(case=args.case, **logreg_rounds_fused(torch, pkg, inputs, ctx))))
        ctx.close()
        return
    if case["kind"] == "mlp_grads":
        dims, M, b, n = (784, 1024, 1024, 10), case["M"], case["b"], 65536
        inp, lab = inputs.gaussian_mixture(5, n, dim=dims[0], classes=dims[3], device="cuda")
        X = inputs.mlp_init(6, dims, device="cuda").unsqueeze(0).repeat(M, 1).contiguous()
        idx = inputs.batch_indices(11, (M, b), n, device="cuda")
        scratch = ctx.mlp_scratch(M, b, dims)
        Gb = torch.empty((M, ctx.mlp_param_count(dims)), device="cuda")
        sec = time_steps(torch, lambda i: ctx.abs_mlp_grads(inp, lab, dims, idx, X, b, Gb, scratch), args.steps,
                         args.warmup)
        flops = 3 * 2.0 * M * b * (dims[0] * dims[1] + dims[1] * dims[2] + dims[2] * dims[3])   # forward, two backward products
        print(json.dumps(dict(case=args.case, tune=args.tune, ms=sec * 1e3, TFLOPs=flops / sec / 1e12,
                              note="fp32-equivalent flops of the matrix products; each runs as 3 TF32 products")))
        ctx.close()
        return
    if case["kind"] == "stats":
        M, b, d = case["M"], case["b"], case["d"]
        if case["dtype"] == "f32":
            G = inputs.gaussian_rows(2, M, b, d, 1.0, device="cuda")
        else:
            G = inputs.gaussian_rows(2, M, b, d, 1.0, device="cuda", dtype=torch.bfloat16)
        stats = ctx.new_stats(M)
        nbytes = G.numel() * G.element_size()
        sec = time_steps(torch, lambda i: ctx.abs_test_stats(G, stats), args.steps, args.warmup)
    else:
        M, d = case["M"], case["d"]
        X, m1, m2, grads = inputs.adamw_problem(4, M, d, pool=1, device="cuda")
        nbytes = 28 * M * d
        sec = time_steps(torch, lambda i: ctx.local_adamw_step(X, m1, m2, grads[0],
                                                               pkg.make_adamw_cfg(step=i + 1, **HP)),
                         args.steps, args.warmup)
    print(json.dumps(dict(case=args.case, tune=args.tune, ms=sec * 1e3, GBps=nbytes / sec / 1e9,
                          frac_of_peak=nbytes / sec / 1e9 / peak, bytes=nbytes)))
    ctx.close()


def stats_sweep(torch, pkg, inputs, ctx, peak, steps, warmup):
    """The statistics sweep: b in {64, 256, 1024} x d in {1 M, 11.2 M, 25.6 M}, fp32, M = 1, each case
    abs_test_stats followed by abs_next_batch for the norm and the augmented inner-product test.
    The variance of the rows does not change what is read, so the sweep runs sigma = 1 only.
    Inputs under 1 GB rotate over 4 buffers so that L2 does not serve them.  Returns the nine cells."""
    cfgs = [pkg.make_test_cfg("norm", 1 << 20, eta=0.5), pkg.make_test_cfg("aug_ip", 1 << 20, theta=0.5, nu=0.5)]
    table = []
    for b in (64, 256, 1024):
        for d in (1_000_000, 11_200_000, 25_600_000):
            nbytes = 4 * b * d
            if nbytes + (8 << 30) > torch.cuda.mem_get_info()[0]:
                table.append(dict(b=b, d=d, GB=nbytes / 1e9, note="does not fit on this device"))
                continue
            copies = 4 if nbytes < (1 << 30) else 1
            Gs = [inputs.gaussian_rows(2 + k, 1, b, d, 1.0, device="cuda") for k in range(copies)]
            stats = ctx.new_stats(1)
            b_cur = torch.tensor([b], dtype=torch.int64, device="cuda")
            b_next = torch.zeros(1, dtype=torch.int64, device="cuda")

            def step(i):
                ctx.abs_test_stats(Gs[i % copies], stats)
                for cfg in cfgs:
                    ctx.abs_next_batch(stats, cfg, b_cur, b_next)

            n = steps if nbytes < (20 << 30) else max(5, steps // 4)
            sec = time_steps(torch, step, n, warmup)
            table.append(dict(b=b, d=d, GB=nbytes / 1e9, ms=sec * 1e3, GBps=nbytes / sec / 1e9,
                              frac_of_peak=nbytes / sec / 1e9 / peak, frac_of_nominal_8TBps=nbytes / sec / 8e12,
                              buffers=copies, steps=n, b_next=int(b_next.item())))
            del Gs
            torch.cuda.empty_cache()
    return table


def worst_cell(table):
    timed = [c for c in table if "GBps" in c]
    if not timed:
        return None
    w = min(timed, key=lambda c: c["frac_of_peak"])
    return dict(b=w["b"], d=w["d"], GBps=w["GBps"], frac=w["frac_of_peak"])


def run_sweep(args):
    """The statistics sweep alone; one JSON line."""
    import torch
    import paper_2406_13936_b200 as pkg
    from paper_2406_13936_b200 import inputs
    pkg.build.build()
    ctx = pkg.Context(0)
    for kv in args.tune:
        key, val = kv.split("=")
        ctx.set_tuning(key, int(val))
    peak, peak_kind = measured_peak()
    table = stats_sweep(torch, pkg, inputs, ctx, peak, args.steps, args.warmup)
    print(json.dumps(dict(sweep="stats fp32 M=1, abs_test_stats + 2 x abs_next_batch per step", steps=args.steps,
                          warmup=args.warmup, peak_GBps=peak, peak_kind=peak_kind, cases=table,
                          worst_cell=worst_cell(table))))
    ctx.close()


def run_ours(args):
    import torch
    import paper_2406_13936_b200 as pkg
    from paper_2406_13936_b200 import inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    pkg.build.build()
    ctx = pkg.Context(local)
    peak, peak_kind = measured_peak()

    M, b, d = WORKLOAD["M"], WORKLOAD["b"], WORKLOAD["d"]
    G = inputs.gaussian_rows(WORKLOAD["seed"] + rank, M, b, d, WORKLOAD["sigma"], device="cuda")
    X, m1, m2, _ = inputs.adamw_problem(4, M, d, pool=0, device="cuda")
    gbar = torch.empty((M, d), device="cuda")
    stats = ctx.new_stats(M)
    b_cur = torch.tensor([b], dtype=torch.int64, device="cuda")
    b_next = torch.zeros(1, dtype=torch.int64, device="cuda")
    T_out = torch.zeros(M, dtype=torch.int64, device="cuda")
    cfg = pkg.make_test_cfg("aug_ip", 1 << 20, theta=0.5, nu=0.5)
    cfg_norm = pkg.make_test_cfg("norm", 1 << 20, eta=0.5)
    g_bytes = G.numel() * G.element_size()
    n_ev = args.steps
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_ev)]

    def step(i, timed=-1):
        if timed >= 0:
            ev[timed][0].record()
        ctx.abs_test_stats(G, stats, gbar)
        if timed >= 0:
            ev[timed][1].record()
        ctx.abs_next_batch(stats, cfg, b_cur, b_next, T_out)       # augmented inner-product test
        ctx.abs_next_batch(stats, cfg_norm, b_cur, b_next, T_out)  # norm test
        ctx.local_adamw_step(X, m1, m2, gbar, pkg.make_adamw_cfg(step=i + 1, **HP), average_after=True)

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for i in range(args.steps):
        step(args.warmup + i, timed=i)
    t1.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    clocks = sampler.stop() if rank == 0 else None
    sec = t0.elapsed_time(t1) / 1e3
    stats_ms = sum(a.elapsed_time(z) for a, z in ev) / n_ev
    sec, value = aggregate_over_ranks(sec, g_bytes * args.steps / 1e9, dist)
    ms_per_step = sec / args.steps * 1e3
    launches_per_step = 2 + 2 + 1      # tiled statistics + finalise, two next-batch kernels, fused AdamW
    rec = pkg.stats_to_dicts(stats)[0]

    # end to end: G starts in pinned host memory, results are read back every step
    e2e = None
    if rank == 0 or world > 1:
        G_host = torch.empty((M, b, d), dtype=torch.float32, pin_memory=True)
        G_host.copy_(G)
        del G
        torch.cuda.empty_cache()

        def host_step(i):
            ctx.abs_test_stats_host(G_host, gbar_dev=gbar, stats_dev=stats)
            ctx.abs_next_batch(stats, cfg, b_cur, b_next, T_out)
            ctx.abs_next_batch(stats, cfg_norm, b_cur, b_next, T_out)
            ctx.local_adamw_step(X, m1, m2, gbar, pkg.make_adamw_cfg(step=i + 1, **HP), average_after=True)
            return b_next.item()

        host_step(0)
        torch.cuda.synchronize()
        n_e2e = 3
        w0 = time.perf_counter()
        for i in range(n_e2e):
            host_step(1 + i)
        torch.cuda.synchronize()
        e2e_sec = (time.perf_counter() - w0) / n_e2e
        e2e_sec, e2e_value = aggregate_over_ranks(e2e_sec, g_bytes / 1e9, dist)
        e2e = dict(value=e2e_value, unit="GB/s", h2d_bytes_per_step=g_bytes,
                   d2h_bytes_per_step=56 * M + 8, steps=n_e2e, ms_per_step=e2e_sec * 1e3)
        del G_host

    extra = None
    if rank == 0 and world == 1 and not args.no_extra:
        extra = extra_legs(torch, pkg, inputs, ctx, peak, args.steps, max(args.warmup, 3))
    cpu = time_cpu_baseline() if (rank == 0 and world == 1) else None

    if rank == 0:
        achieved = g_bytes / (stats_ms / 1e3) / 1e9
        line = dict(
            metric="batch_test_step_GBps", value=value, unit="GB/s", n_gpus=world, steps=args.steps,
            warmup=args.warmup, ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None,
            dtype="f32", data="synthetic",
            config=dict(workload=WORKLOAD["name"], M=M, b=b, d=d, bytes_per_step=g_bytes,
                        l2="inputs (11.5 GB) larger than L2, no flush needed",
                        step="abs_test_stats + abs_next_batch (aug. inner-product and norm) + local_adamw_step "
                             "with fused replica_average",
                        shard="one independent problem per GPU, no collective"),
            rounds_per_s=world * args.steps / sec,
            roofline=dict(bound="hbm", kernel="abs_stats_tiled_kernel<float,16,keep,full> (+ finalise)",
                          achieved=achieved, peak=peak, unit="GB/s", frac=achieved / peak, peak_kind=peak_kind,
                          frac_of_nominal_8TBps=achieved / 8000.0, ms=stats_ms,
                          traffic=NCU_TRAFFIC_SMALL["dram_bytes"] * d / NCU_TRAFFIC_SMALL["d"],
                          traffic_note="ncu DRAM read+write of the 1.024 GB case scaled by d; algorithmic bytes "
                                       "are config.bytes_per_step"),
            cpu_baseline=cpu, e2e=e2e, gpu_launches=launches_per_step * args.steps, clocks=clocks,
            result=dict(b_next=int(b_next.item()), var_norm=rec["var_norm"], gbar_sq=rec["gbar_sq"],
                        status=rec["status"]),
            extra=extra)
        print(json.dumps(line))
    ctx.close()
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extra", action="store_true")
    ap.add_argument("--case", default=None, choices=sorted(PROFILE_CASES),
                    help="run only a few launches of one kernel on a small case (for profiler captures)")
    ap.add_argument("--shape", default=None, help="M,b,d,f32|bf16: time abs_test_stats on that shape only")
    ap.add_argument("--sweep", action="store_true", help="time the nine fp32 (b, d) cases of the statistics sweep")
    ap.add_argument("--tune", action="append", default=[], help="key=value passed to abs_set_tuning (with --case)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    if args.sweep:
        run_sweep(args)
    elif args.case or args.shape:
        run_profile_case(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
