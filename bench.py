#!/usr/bin/env python
"""Benchmark of the parameter-server hot path on B200.

Workload: the largest configuration ("scale"): W = 128 logical workers, batch 128 each, stateless
server.  A step is one tick of the whole path: every worker pulls its snapshot, the grad step
writes 128 gradients into reserved queue slots, they are enqueued, and the server applies them
(the stateless server's step).  `value` is worker-samples/s with inputs resident in HBM; `e2e` is
the same tick through ps_tick_host with pinned host inputs copied in and losses copied out every
step.  The deferred replay of a 200-tick outage (25,600 gradients, 83 GB) is timed separately and
reported as GB/s under "replay".

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--precision bf16|fp32]
    python bench.py --case small [--workers 16] [--batch 64] [--ticks 3] [--down-ticks 50]
        a reduced run of the stateless workload for profiler captures (no JSON line, no timing claims)
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

W_WORKERS, BATCH = 128, 128
DOWN_TICKS = 200
LR = 0.01
DROP_SEED = 0x5EED
FLOP_PER_SAMPLE = 10_718_208            # 2 x (1,824,000 forward + 3,535,104 backward multiply-adds)
GRAD_BYTES = 813258 * 4                 # algorithmic bytes per queued gradient
N_BATCH_BUFFERS = 8
REPLAY_TRAFFIC_PER_GRADIENT = 2.654663e9 / 816
# dram bytes (read + written) per sample of the grad-step kernels, from one ncu capture of a reduced case
# (W=128, b=64: 8,192 samples; traffic grows in proportion to the samples, except for fc1_dw, whose 3.2 MB of output per
# worker do not depend on the batch: its figure holds at b = 64 only); None = not captured since the kernel changed
KERNEL_TRAFFIC_PER_SAMPLE = {"conv2_dw": 13406, "conv1_fwd": 7393, "conv2_bwd": 5515, "fc1_dw": 51641, "conv2_fwd": 10064,
                             "fc1_dx": 2452, "fc1_fwd": 6745, "fc2_fwd_bwd": 2061, "conv1_bwd": 12972}


# Algorithmic HBM bytes of the tensor-core path's grad-step kernels at (W, b): what each must read and write once
# (images fp32, p1 as 8 KB BF16 planes, decisions as bytes, p2 / a1 / da1 fp32, dp2 and dp1 BF16, the per-worker fc1
# weight gradient fp32; weights are small and stay in L2).
ALGORITHMIC_BYTES = {
    "conv1_fwd": lambda W, b: (3136 + 8192 + 3136) * W * b,
    "conv2_fwd": lambda W, b: (8192 + 6272 + 1568) * W * b,
    "fc1_fwd": lambda W, b: (6272 + 2048) * W * b,
    "fc2_fwd_bwd": lambda W, b: (2048 + 2048) * W * b,
    "fc1_dw": lambda W, b: (2048 + 6272) * W * b + 512 * 1568 * 4 * W,
    "fc1_dx": lambda W, b: (2048 + 3136) * W * b,
    "conv2_bwd": lambda W, b: (3136 + 1568 + 6272) * W * b,
    "conv2_dw": lambda W, b: (8192 + 3136 + 1568) * W * b,
    "conv1_bwd": lambda W, b: (3136 + 6272 + 3136) * W * b,
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                "sm_max_mhz": d.get("sm_max_mhz", 1965.0), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 1965.0,
            "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0=None, t1=None):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = [l for t, l in self.lines if (t0 is None or t >= t0) and (t1 is None or t <= t1 + 0.1)] or \
               [l for _, l in self.lines]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in rows:
            f = [v.strip() for v in l.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def cpu_baseline(budget_s=12.0):
    """The oracle, as it stands, on the host cores: the grad step of whole ticks of the workload, one group of
    `cores` workers at a time, until about budget_s seconds of CPU work have been timed."""
    from oracle import cnn
    from paper_2406_05546_b200 import synth
    cores = cnn.num_threads()
    theta = synth.init_params(1)
    px, py = synth.image_pool(8192, seed=0)
    done, t_used, tick = 0, 0.0, 0
    chunk = max(cores, 1)
    while t_used < budget_s:
        for w0 in range(0, W_WORKERS, chunk):
            n = min(chunk, W_WORKERS - w0)
            rows = synth.batch_rows(tick, W_WORKERS, BATCH, px.shape[0])[w0:w0 + n]
            x, y = px[rows], py[rows]
            t = time.perf_counter()
            cnn.workers_grad_step([theta] * n, list(range(w0, w0 + n)), x, y, DROP_SEED, tick, 0.25)
            t_used += time.perf_counter() - t
            done += n
            if t_used >= budget_s:
                break
        tick += 1
    # one worker on one thread (the OpenMP loop runs over workers, so a single worker uses a single core)
    rows = synth.batch_rows(0, W_WORKERS, BATCH, px.shape[0])[:1]
    n1, t1 = 0, 0.0
    while t1 < 3.0:
        t = time.perf_counter()
        cnn.workers_grad_step([theta], [0], px[rows], py[rows], DROP_SEED, n1, 0.25)
        t1 += time.perf_counter() - t
        n1 += 1
    # the oracle's replay (numpy, double sums, one thread) over a queue held in host memory
    from oracle import ps as ops
    Kq, Wq = 256, 16
    srv = ops.OraclePS(theta, external_store=True)
    srv.kill()
    for k in range(Kq // Wq):
        srv.enqueue(synth.random_gradients(Wq, seed=900 + k), range(Wq), [0] * Wq, k)
    srv.restore()
    t = time.perf_counter()
    srv.apply(ops.REPLAY, LR, 1.0 / (Kq // Wq))
    t_rep = time.perf_counter() - t
    return {"value": done * BATCH / t_used, "unit": "worker-samples/s", "cores": cores, "kind": "oracle",
            "sample": f"grad step of {done} workers (batch {BATCH}; the workload has {W_WORKERS} per tick), {t_used:.1f} s",
            "single_thread": {"value": n1 * BATCH / t1, "unit": "worker-samples/s", "cores": 1,
                              "sample": f"grad step of {n1} workers of batch {BATCH}, one at a time, {t1:.1f} s"},
            "replay": {"value": (Kq + 2) * GRAD_BYTES / t_rep / 1e9, "unit": "GB/s", "cores": 1,
                       "sample": f"oracle REPLAY of {Kq} gradients ({Kq * GRAD_BYTES / 1e9:.2f} GB) held in host memory, {t_rep:.1f} s"}}


def run_reference(args):
    """--impl reference: the CPU oracle on a bounded sample of the same workload, per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import cnn, ps as ops
    from paper_2406_05546_b200 import synth
    cores = cnn.num_threads()
    n = min(W_WORKERS, max(cores, 1))                # workers per step in the sample
    px, py = synth.image_pool(8192, seed=0)
    srv = ops.OraclePS(synth.init_params(1), external_store=True)
    times = []
    for step in range(args.warmup + args.steps):
        rows = synth.batch_rows(step, n, BATCH, px.shape[0])
        x, y = px[rows], py[rows]
        t = time.perf_counter()
        v, theta = srv.pull_snapshot(0)
        g, loss, am, _ = cnn.workers_grad_step([theta] * n, list(range(n)), x, y, DROP_SEED, step, 0.25)
        srv.enqueue(g.astype(np.float32), range(n), [v] * n, step)
        srv.apply(ops.REPLAY, LR)
        dt = time.perf_counter() - t
        if step >= args.warmup:
            times.append(dt)
    total = sum(times)
    value = n * BATCH * args.steps / total
    sample = f"{n} of the {W_WORKERS} workers per tick (batch {BATCH}): snapshot, grad step, enqueue, apply"
    print(json.dumps({
        "impl": "reference", "metric": "worker-samples/s", "value": value, "unit": "worker-samples/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "config 5 (scale): W=128 workers x batch 128, stateless server", "sample": sample},
        "cpu_baseline": {"value": value, "unit": "worker-samples/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "worker-samples/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_small_case(args):
    """--case small: a few ticks, an outage that buffers a few GB of gradients, and the catch-up replay, sized so
    that a profiler's multi-pass capture of one kernel ends by itself (the queue is larger than L2 but only a few
    GB).  Prints one summary line; nothing is timed."""
    import torch
    from paper_2406_05546_b200 import harness, ps, schedules, synth
    s = schedules.Schedule("small", W=args.workers, b=args.batch, mode=schedules.REPLAY,
                           ticks=2 * args.ticks + args.down_ticks, external_store=True,
                           kill_at=args.ticks, recover_at=args.ticks + args.down_ticks, recover_by="restore",
                           replay_scale=1.0 / max(1, args.down_ticks))
    px, py = synth.image_pool(8192, seed=0)
    srv = harness.make_server(s, synth.init_params(1), precision=ps.BF16 if args.precision == "bf16" else ps.FP32)
    log = harness.run(s, srv, px, py)
    torch.cuda.synchronize()
    st = srv.ps_stats()
    replay = log[s.recover_at]["apply"]
    theta = srv.ps_export_params()[0]
    assert np.isfinite(theta).all()
    print(f"small case: W={s.W} b={s.b}, {len(log)} ticks, replayed {replay['applied']} gradients "
          f"({replay['applied'] * ps.P * 4 / 1e9:.2f} GB), version {st['version']}, launches {st['kernel_launches']}")
    srv.close()


GRAD_KERNELS_EXCLUDED = ("sum_apply_direct", "sum_partial", "sum_finish", "async_apply", "copy_rows", "dropout_mask",
                         "sq_norm_partial", "clip_coef_finish", "eval_finish")      # server-side and auxiliary kernels


def measure_config(n, precision, pool_x, pool_y, ticks=10, warmup=3):
    """Configuration n at its stated size, inputs resident: per-kernel CUDA-event times over `ticks` ticks after
    `warmup` (each kernel timed alone).  Returns the grad step's time and the apply kernel's achieved bandwidth."""
    import torch
    from paper_2406_05546_b200 import harness, ps, schedules, synth
    s = schedules.config(n)
    srv = harness.make_server(s, synth.init_params(1), queue_slots=s.W,
                              precision=ps.BF16 if precision == "bf16" else ps.FP32)
    ids = list(range(s.W))
    n_pool = pool_x.shape[0]
    groups = set()
    for t in range(warmup + ticks):
        if t == warmup:
            srv.ps_profile(True)
        st = srv.ps_stats()
        lags = np.zeros(s.W, dtype=np.int32)
        if s.max_lag:
            lags = harness.clamp_lags(synth.lags(t, s.W, s.max_lag), st["version"], st["oldest_version"])
        rows = torch.from_numpy(synth.batch_rows(t, s.W, s.b, n_pool)).cuda()
        x, y = pool_x[rows].contiguous(), pool_y[rows].contiguous()
        snaps = [srv.ps_pull_snapshot(w, int(lags[w])) for w in range(s.W)]
        if t >= warmup:
            groups.add(len({sn.version for sn in snaps}))
        slots = srv.ps_queue_reserve(s.W)
        srv.workers_grad_step(snaps, ids, x, y, s.seed, t, slot_ids=slots)
        srv.ps_enqueue(ids, [sn.version for sn in snaps], t, slot_ids=slots)
        srv.ps_apply(s.mode, s.lr, 1.0, synth.arrival_order(t, s.W) if s.mode == schedules.ASYNC else None)
    prof = srv.ps_profile_read()
    srv.ps_profile(False)
    srv.close()
    per = {k: ms / cnt for k, (ms, cnt) in prof.items() if cnt}
    grad_ms = sum(v for k, v in per.items() if k not in GRAD_KERNELS_EXCLUDED)
    apply_k = "async_apply" if s.mode == schedules.ASYNC else "sum_apply_direct"
    mirror = 1 if s.chain_len > 1 else 0
    stored = min(s.ring_depth, s.W) if s.mode == schedules.ASYNC else 1
    apply_bytes = (s.W + 1 + stored + mirror) * GRAD_BYTES
    out = {"W": s.W, "b": s.b, "mode": ["sync", "async", "replay"][s.mode], "precision": precision,
           "grad_step_ms": grad_ms, "worker_samples_per_s": s.W * s.b / (grad_ms * 1e-3),
           "tflops": FLOP_PER_SAMPLE * s.W * s.b / (grad_ms * 1e-3) / 1e12,
           "distinct_snapshots": max(groups) if groups else 1,
           "apply_kernel": apply_k, "apply_ms": per.get(apply_k), "apply_bytes": apply_bytes,
           "apply_gb_per_s": apply_bytes / (per[apply_k] * 1e-3) / 1e9 if per.get(apply_k) else None,
           "ticks": ticks}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--precision", default="bf16", choices=["fp32", "bf16"],
                    help="arithmetic of the dense contractions of the grad step: fp32 = CUDA cores; bf16 = tensor "
                         "cores (BF16 operands in the convolution products, TF32 in the 512-unit layer)")
    ap.add_argument("--case", default="bench", choices=["bench", "small"],
                    help="small: a reduced run for profiler captures (see --workers/--batch/--ticks/--down-ticks)")
    ap.add_argument("--workers", type=int, default=16)
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--ticks", type=int, default=3)
    ap.add_argument("--down-ticks", type=int, default=50)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        return run_reference(args)
    if args.case == "small":
        return run_small_case(args)

    import torch
    from paper_2406_05546_b200 import ps, synth
    from paper_2406_05546_b200.ranks import Ranks

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    peaks = measured_peaks()
    # the CPU leg (OpenMP threads of the oracle) runs before the first GPU call
    cpu = None
    if rank == 0 and world == 1:
        cpu = cpu_baseline()
    torch.cuda.set_device(local)
    ranks = Ranks("nccl")
    barrier, max_over_ranks = ranks.barrier, ranks.max_over_ranks

    W, b = W_WORKERS, BATCH
    K_replay = DOWN_TICKS * W
    do_replay = True
    srv = ps.ParameterServer(synth.init_params(1), max_workers=W, max_batch=b, ring_depth=1,
                             queue_slots=(K_replay if do_replay else 0) + W, external_store=True, dropout_p=0.25,
                             precision=ps.BF16 if args.precision == "bf16" else ps.FP32)
    # synthetic stand-in for the 60,000-image training pool, resident in HBM; every rank its own rows
    px, py = synth.image_pool(synth.POOL_IMAGES, seed=0)
    pool_x, pool_y = torch.from_numpy(px).cuda(), torch.from_numpy(py).cuda()
    bufs = []
    for t in range(N_BATCH_BUFFERS):
        rows = torch.from_numpy(synth.batch_rows(ranks.batch_seed(t), W, b, px.shape[0])).cuda()
        bufs.append((pool_x[rows].contiguous(), pool_y[rows].contiguous()))
    loss_dev = torch.empty(W, dtype=torch.float32, device="cuda")
    am_dev = torch.empty((W, b), dtype=torch.int32, device="cuda")
    ids = list(range(W))
    tick_no = [0]

    def tick(apply=True):
        t = tick_no[0]
        x, y = bufs[t % N_BATCH_BUFFERS]
        snaps = [srv.ps_pull_snapshot(w) for w in range(W)]
        slots = srv.ps_queue_reserve(W)
        srv.workers_grad_step(snaps, ids, x, y, DROP_SEED, t, slot_ids=slots, loss_dev=loss_dev, argmax_dev=am_dev)
        srv.ps_enqueue(ids, [s.version for s in snaps], t, slot_ids=slots)
        if apply:
            srv.ps_apply(ps.REPLAY, LR)
        tick_no[0] += 1

    for _ in range(args.warmup):
        tick()
    # ---- timed region: K whole ticks, inputs resident, CUDA events on the library's stream
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    l0 = srv.ps_stats()["kernel_launches"]
    barrier()
    t_wall0 = time.time()
    ev0.record(srv.stream)
    for _ in range(args.steps):
        tick()
    ev1.record(srv.stream)
    barrier()
    t_wall1 = time.time()
    ms_total = max_over_ranks(ev0.elapsed_time(ev1))
    launches = srv.ps_stats()["kernel_launches"] - l0

    # ---- second pass with per-kernel events: which kernel dominates, and its roofline
    srv.ps_profile(True)
    for _ in range(args.steps):
        tick()
    prof = srv.ps_profile_read()
    srv.ps_profile(False)
    clocks = sampler.stop(t_wall0, time.time())

    # ---- end to end: pinned host inputs in, losses out, through ps_tick_host
    hx = [torch.from_numpy(px[synth.batch_rows(t, W, b, px.shape[0])]).pin_memory() for t in range(2)]
    hy = [torch.from_numpy(py[synth.batch_rows(t, W, b, px.shape[0])]).pin_memory() for t in range(2)]
    loss_host = torch.empty(W, dtype=torch.float32).pin_memory()
    e2e_steps = max(3, min(args.steps, 50))
    # Two ticks are kept in flight (ps_tick_host_submit / ps_tick_host_wait): the copy of the next tick's inputs runs
    # while the current tick computes.  Every timed step still copies its own inputs in and its losses out.
    loss_bufs = [loss_host, torch.empty(W, dtype=torch.float32).pin_memory()]
    for t in range(3):
        srv.ps_tick_host(hx[t % 2], hy[t % 2], DROP_SEED, 10_000 + t, ps.REPLAY, LR, loss_host=loss_host)
    barrier()
    t0 = time.perf_counter()
    srv.ps_tick_host_submit(hx[0], hy[0], DROP_SEED, 20_000, ps.REPLAY, LR, loss_host=loss_bufs[0])
    for t in range(1, e2e_steps):
        srv.ps_tick_host_submit(hx[t % 2], hy[t % 2], DROP_SEED, 20_000 + t, ps.REPLAY, LR, loss_host=loss_bufs[t % 2])
        srv.ps_tick_host_wait()
    srv.ps_tick_host_wait()
    barrier()
    e2e_ms = max_over_ranks((time.perf_counter() - t0) * 1e3)
    h2d = W * b * 784 * 4 + W * b * 4
    d2h = W * 4

    # ---- the summed step (every worker on the head, only the sum wanted) and the evaluation pass, same inputs
    gsum = torch.empty(ps.P_PAD, dtype=torch.float32, device="cuda")

    def summed_tick():
        t = tick_no[0]
        x, y = bufs[t % N_BATCH_BUFFERS]
        snaps = [srv.ps_pull_snapshot(w) for w in range(W)]
        srv.workers_grad_step_summed(snaps, ids, x, y, DROP_SEED, t, grad_sum_dev=gsum, loss_dev=loss_dev, argmax_dev=am_dev)
        srv.ps_apply_summed(gsum, W, LR)
        tick_no[0] += 1

    def timed(fn, n):
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(srv.stream)
        for _ in range(n):
            fn()
        e1.record(srv.stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1)) / n

    n_extra = max(3, min(args.steps, 50))
    summed_ms = timed(summed_tick, n_extra)
    srv.ps_profile(True)
    for _ in range(5):
        summed_tick()
    prof_s = srv.ps_profile_read()
    srv.ps_profile(False)
    summed = {"ms_per_tick": summed_ms, "worker_samples_per_s": W * b * world / (summed_ms * 1e-3), "ticks": n_extra,
              "kernels_ms": {k: ms / n for k, (ms, n) in prof_s.items() if n},
              "note": "pull + workers_grad_step_summed + ps_apply_summed: one summed gradient vector instead of W; "
                      "not the headline metric, which is the per-worker stale-weight step"}

    def eval_pass():
        x, y = bufs[0]
        srv.workers_eval([srv.ps_pull_snapshot(w) for w in range(W)], x, y)

    eval_ms = timed(eval_pass, n_extra)
    evaluation = {"ms_per_pass": eval_ms, "samples_per_s": W * b * world / (eval_ms * 1e-3), "samples": W * b}

    # ---- the other configurations at their stated sizes, and the FP32 path at this one (a few ticks each)
    configs, fp32_path = None, None
    if rank == 0:
        configs = {f"config{n}": measure_config(n, args.precision, pool_x, pool_y) for n in (1, 2, 3, 4)}
        if args.precision != "fp32":
            fp32_path = measure_config(5, "fp32", pool_x, pool_y)
            fp32_path["frac_of_fp32_pipe"] = fp32_path["tflops"] / (148 * 128 * 2 * peaks["sm_max_mhz"] / 1e6)
    barrier()

    # ---- deferred replay of a DOWN_TICKS outage (83 GB of buffered gradients)
    replay = None
    if do_replay:
        reps = []
        for rep in range(2):
            srv.ps_kill()
            for _ in range(DOWN_TICKS):
                tick(apply=False)
            srv.ps_restore()
            assert srv.ps_stats()["queue_len"] == K_replay
            r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier()
            r0.record(srv.stream)
            res = srv.ps_apply(ps.REPLAY, LR, scale=1.0 / DOWN_TICKS)
            r1.record(srv.stream)
            barrier()
            assert res["applied"] == K_replay
            reps.append(r0.elapsed_time(r1))
        ms = max_over_ranks(min(reps))
        bytes_alg = (K_replay + 2) * GRAD_BYTES
        gbs = bytes_alg / (ms * 1e-3) / 1e9
        replay = {"queue_gradients": K_replay, "bytes": bytes_alg, "ms": ms, "gb_per_s": gbs * world,
                  "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                               "frac": gbs / peaks["hbm_gbs"],
                               # dram bytes per queued gradient from the ncu capture of a reduced case
                               # (2.654663 GB over 816 gradients), scaled to this launch
                               "traffic": K_replay * REPLAY_TRAFFIC_PER_GRADIENT, "peak_source": peaks["source"]},
                  "all_ms": reps}
    # ---- the same replay with clipping by global norm: one pass that takes the norms, one that sums
    replay_clipped = None
    if do_replay:
        srv.ps_kill()
        for _ in range(DOWN_TICKS):
            tick(apply=False)
        srv.ps_restore()
        srv.ps_profile(True)
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        r0.record(srv.stream)
        res = srv.ps_apply_stale(ps.REPLAY, LR, scale=1.0 / DOWN_TICKS, clip_norm=1.0)
        r1.record(srv.stream)
        barrier()
        assert res["applied"] == K_replay
        ms = max_over_ranks(r0.elapsed_time(r1))
        prof_c = srv.ps_profile_read()
        srv.ps_profile(False)
        pass_bytes = K_replay * GRAD_BYTES
        replay_clipped = {"queue_gradients": K_replay, "ms": ms, "clip_norm": 1.0,
                          "norm_pass_ms": prof_c["sq_norm_partial"][0], "norm_pass_gb_per_s": pass_bytes / (prof_c["sq_norm_partial"][0] * 1e-3) / 1e9,
                          "sum_pass_ms": prof_c["sum_partial"][0], "sum_pass_gb_per_s": pass_bytes / (prof_c["sum_partial"][0] * 1e-3) / 1e9,
                          "frac_of_hbm_peak_per_pass": [pass_bytes / (prof_c["sq_norm_partial"][0] * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                                        pass_bytes / (prof_c["sum_partial"][0] * 1e-3) / 1e9 / peaks["hbm_gbs"]]}
    stats = srv.ps_stats()

    if rank == 0:
        value = ranks.whole_job_rate(W * b * args.steps, ms_total)
        total_prof = sum(ms for ms, _ in prof.values()) or 1.0
        kernels = {k: {"ms_per_launch": ms / n, "launches": n, "share": ms / total_prof}
                   for k, (ms, n) in prof.items() if n}
        top = max(kernels, key=lambda k: kernels[k]["share"])
        roof = kernel_roofline(top, kernels[top]["ms_per_launch"], W, b, peaks, args.precision)
        roof.pop("flops", None)
        per_sample = KERNEL_TRAFFIC_PER_SAMPLE.get(top) if args.precision != "fp32" else None
        if per_sample is not None:
            roof["traffic"] = per_sample * W * b
        grad_ms = sum(v["ms_per_launch"] for k, v in kernels.items() if k not in GRAD_KERNELS_EXCLUDED)
        tensor_flop = 2 * (3 * 903_168 + 3 * 802_816) * W * b
        # time the grad step would take if every product ran at the peak of the unit and type it uses
        # (convolution products BF16 tensor, 512-unit layer TF32 tensor, first convolution and output
        # layer FP32 FMA), the composite compute roofline of the step
        def composite_ms(sustained):
            roofs = {k: kernel_roofline(k, 1.0, W, b, peaks, args.precision, sustained) for k in kernels}
            return sum(r["flops"] / (r["peak"] * 1e12) * 1e3 for r in roofs.values() if r["bound"] != "hbm")
        sol_ms, sol_ms_sustained = composite_ms(False), composite_ms(True)
        # the same with every kernel bound by the larger of its compute time and the time the measured copy bandwidth
        # needs for its algorithmic bytes (tensor-core path; None on the FP32 path, whose buffers differ)
        def compute_or_hbm_ms():
            if args.precision == "fp32":
                return None, None
            per = {}
            for k in kernels:
                if k in GRAD_KERNELS_EXCLUDED or k not in ALGORITHMIC_BYTES:
                    continue
                r = kernel_roofline(k, 1.0, W, b, peaks, args.precision)
                t_c = r["flops"] / (r["peak"] * 1e12) * 1e3 if r["bound"] != "hbm" else 0.0
                t_m = ALGORITHMIC_BYTES[k](W, b) / (peaks["hbm_gbs"] * 1e9) * 1e3
                per[k] = max(t_c, t_m)
            return sum(per.values()), per
        bound_ms, bound_per_kernel = compute_or_hbm_ms()
        tflops = FLOP_PER_SAMPLE * W * b / (grad_ms * 1e-3) / 1e12
        grad_step = {"ms": grad_ms, "worker_samples_per_s": W * b / (grad_ms * 1e-3), "tflops": tflops,
                     "tensor_flop_share": tensor_flop / (FLOP_PER_SAMPLE * W * b),
                     "roofline_ms": sol_ms, "frac_of_composite_roofline": sol_ms / grad_ms,
                     "roofline_ms_sustained_peaks": sol_ms_sustained,
                     "frac_of_composite_roofline_sustained_peaks": sol_ms_sustained / grad_ms,
                     "frac_of_tf32_roofline": tflops / (peaks["bf16_tflops"] * (1.1 / 2.25)),
                     "roofline_ms_compute_or_hbm": bound_ms,
                     "frac_of_compute_or_hbm_roofline": bound_ms / grad_ms if bound_ms else None,
                     "per_kernel_frac_compute_or_hbm": {k: v / kernels[k]["ms_per_launch"] for k, v in bound_per_kernel.items()} if bound_per_kernel else None,
                     "per_kernel_frac": {k: kernel_roofline(k, v["ms_per_launch"], W, b, peaks, args.precision)["frac"]
                                         for k, v in kernels.items() if k not in GRAD_KERNELS_EXCLUDED and k not in ("conv_grad_reduce", "prep_w1")},
                     "note": "ms = sum of the per-kernel times measured one kernel at a time (in the timed region "
                             "independent branches of the backward pass overlap on side streams); roofline_ms = "
                             "sum over products of flop / peak of the unit and type each uses, with the measured "
                             "burst bf16 GEMM rate (kernels timed alone at the full SM clock); the _sustained_peaks "
                             "figures use the sustained rate instead; "
                             "frac_of_tf32_roofline = all flop / ms against the TF32 dense peak alone; "
                             "roofline_ms_compute_or_hbm = sum over kernels of max(flop / peak, algorithmic bytes / "
                             "measured copy bandwidth)"}
        # the whole grad step next to the dominant kernel
        roof["grad_step"] = {"ms": grad_ms, "roofline_ms": sol_ms, "frac": sol_ms / grad_ms, "bound": "composite compute",
                             "peaks": "burst"}
        out = {
            "metric": "worker-samples/s", "value": value, "unit": "worker-samples/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32" if args.precision == "fp32" else "bf16+tf32",
            "data": "synthetic",
            "config": {"workload": "config 5 (scale): W=128 workers x batch 128, stateless server, one tick = "
                                   "pull + grad step + enqueue + apply",
                       "W": W, "b": b, "l2": "inputs larger than L2: each tick writes 416 MB of gradients and "
                                             "cycles 8 distinct 51 MB input batches",
                       "replicas": "independent replica per GPU, no collective" if world > 1 else "single GPU"},
            "e2e": {"value": W * b * e2e_steps * world / (e2e_ms * 1e-3), "unit": "worker-samples/s",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "roofline": roof,
            "kernels": kernels,
            "grad_step": grad_step,
            "replay": replay,
            "replay_clipped": replay_clipped,
            "summed_step": summed,
            "evaluation": evaluation,
            "configs": configs,
            "fp32_path": fp32_path,
            "cpu_baseline": cpu,
            "final_version": stats["version"],
        }
        print(json.dumps(out))
    srv.close()
    ranks.close()


def kernel_roofline(name, ms_per_launch, W, b, peaks, precision, sustained=False):
    """Algorithmic work of one launch of the named kernel at (W, b) against the roofline that bounds it."""
    n = W * b
    sec = ms_per_launch * 1e-3
    sm_clock_ghz = peaks["sm_max_mhz"] / 1e3
    fp32_peak_tflops = 148 * 128 * 2 * sm_clock_ghz / 1e3        # 148 SMs x 128 FP32 lanes x FMA
    # Every kernel here is timed alone by CUDA events at the full SM clock, so the tensor peak that applies is the
    # measured BURST bf16 GEMM rate (the sustained one is what a seconds-long GEMM loop settles to under the power
    # cap); dense TF32 peak = that x the nominal tf32/bf16 ratio (1.1 / 2.25 PFLOP/s)
    bf16_peak_tflops = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    tf32_peak_tflops = bf16_peak_tflops * (1.1 / 2.25)
    which = "sustained" if sustained else "burst"
    flops = {
        "conv1_fwd": 2 * 112_896 * n, "conv2_fwd": 2 * 903_168 * n, "fc1_fwd": 2 * 802_816 * n,
        "fc1_dw": 2 * 802_816 * n, "fc1_dx": 2 * 802_816 * n,
        "conv2_bwd": 2 * (2 if precision == "fp32" else 1) * 903_168 * n, "conv2_dw": 2 * 903_168 * n,
        "conv1_bwd": 2 * 112_896 * n, "fc2_fwd_bwd": 2 * 3 * 5_120 * n,
    }
    tf32_kernels = {"fc1_fwd", "fc1_dw", "fc1_dx"}                               # tcgen05 kind::tf32
    bf16_kernels = {"conv2_fwd", "conv2_bwd", "conv2_dw", "conv1_bwd"}           # tcgen05 kind::f16 (conv1_bwd: mma.sync), BF16
    if name in flops:
        ach = flops[name] / sec / 1e12
        if precision != "fp32" and name in tf32_kernels:
            return {"kernel": name, "bound": "tensor", "achieved": ach, "peak": tf32_peak_tflops, "unit": "TFLOP/s",
                    "frac": ach / tf32_peak_tflops, "traffic": None, "flops": flops[name],
                    "peak_source": f"{peaks['source']} {which} bf16 GEMM x nominal tf32/bf16 ratio 1.1/2.25"}
        if precision != "fp32" and name in bf16_kernels:
            return {"kernel": name, "bound": "tensor", "achieved": ach, "peak": bf16_peak_tflops, "unit": "TFLOP/s",
                    "frac": ach / bf16_peak_tflops, "traffic": None, "flops": flops[name],
                    "peak_source": f"{peaks['source']} {which} bf16 GEMM"}
        return {"kernel": name, "bound": "alu", "achieved": ach, "peak": fp32_peak_tflops, "unit": "TFLOP/s",
                "frac": ach / fp32_peak_tflops, "traffic": None, "flops": flops[name],
                "peak_source": "148 SMs x 128 FP32 lanes x 2 x max SM clock"}
    bytes_ = {"sum_apply_direct": (W + 2) * GRAD_BYTES, "sum_partial": (W + 2) * GRAD_BYTES}.get(name, 0)
    ach = bytes_ / sec / 1e9
    return {"kernel": name, "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": ach / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["source"]}


if __name__ == "__main__":
    main()
