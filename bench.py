"""Throughput of Pipelined Backpropagation ticks (samples/s at batch 1).

One step is one STEADY-STATE tick: every stage's forward and backward on its
current samples plus the SC+LWP update of every stage.  Workload: the deep MLP
(16 FC stages of width 2048), whose weights and velocities (504 MB) exceed
the L2 cache, so every tick streams them from HBM.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

Before anything is timed the pipeline is FILLED: 2(S-1)+2 set-up ticks, after
which every stage runs its forward, its backward and its update in every tick
(a stage's first gradient arrives at tick 2(S-1)-s).  Then come the W warm-up
ticks and the K timed ticks.  A line whose implied memory bandwidth is beyond
what the device can deliver is refused (value null).

With N > 1 (under torch.distributed.run) each rank runs an independent replica
of the pipeline on its own GPU: the tick has no data-parallel form at update
size one, so the job scales by replicas and no collective is on the data path.
"""
import argparse
import hashlib
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

WORKLOAD = "mlp16x2048"
METRIC = "PB ticks/sec (samples/sec, batch 1)"
UNIT = "ticks/s"
HBM_HW_GBS = 7700.0            # HBM3e of one B200 in an HGX board, vendor figure
L2_BYTES = 126e6
# step sizes at which the diverging configurations stay bounded (same kernels, finite numbers)
STABLE_LR = {"mlp4": 0.001, "mlp16x2048": 1e-4, "resnet50": 5e-4, "resnet50_112": 5e-4}

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel,
# from the ncu captures summarised under profiles/; each entry names the source file of the
# kernel and that file's SHA-1 when the counters were taken, and is dropped (null) as soon as
# the file has changed since.
NCU_TRAFFIC = {
    "mlp16x2048": (957.0e6, "fc_kernels.cuh", "8e816cccda2aa74634cce0101eeca58fdb09f40e",
                   "profiles/fc_tick_kernel_mlp16x2048.md: 508.1 MB read + 448.8 MB written per launch (mean of two launches), "
                   "gpu__dram_throughput 67.2 % of the hardware peak"),
    "resnet50": (510.6e6, "conv_stage.cuh", "1b3325f6f592c6ed127aa778d10b1bff4146a2ca",
                 "profiles/tick_kernels_resnet50.md: update_kernel 285.5 MB read + 225.1 MB written per launch (mean of two "
                 "launches), gpu__dram_throughput 60.6 % of the hardware peak"),
}


def ncu_traffic(workload_name):
    ent = NCU_TRAFFIC.get(workload_name)
    if ent is None:
        return None, None
    nbytes, fname, sha, note = ent
    path = os.path.join(ROOT, "paper_2003_11666_b200", "csrc", fname)
    try:
        with open(path, "rb") as f:
            now = hashlib.sha1(f.read()).hexdigest()
    except OSError:
        return None, None
    if now != sha:
        return None, "kernel source changed since the counters were taken"
    return nbytes, note


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d.get("hbm_gbs", 6650.0), d.get("bf16_tflops_sustained", 1400.0), "measured"
    return 6650.0, 1400.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while timing."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(ms, world, device="cuda"):
    """Slowest rank's time: the job is done when the last replica is."""
    if world == 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(world, ticks_per_rank, ms):
    """Whole-job ticks/s: every replica ran `ticks_per_rank` ticks within `ms`."""
    return world * ticks_per_rank / (ms * 1e-3)


def replica_seed(base_seed, rank):
    """Replicas see different sample streams."""
    return base_seed + 1000 * rank


def fill_ticks(n_stages):
    """Set-up ticks before any timing: stage s gets its first gradient at tick
    2(S-1)-s, so after 2(S-1)+2 ticks every stage has forwarded, back-propagated
    and updated at least twice."""
    return 2 * (n_stages - 1) + 2


def tick_floor(work, peaks, bf16):
    """Least time one steady-state tick can take on this device, in microseconds, and
    what bounds it.  Memory: 16 B per parameter (one read and one write of w and v)
    plus every activation once (float32, or bfloat16 for tensor-core operands), at
    the L2 bandwidth when weights, velocities and activations together stay well
    inside the L2 cache, else at the HBM copy rate.  Arithmetic: three passes
    (forward, data gradient, weight gradient) of 2 flops per multiply-accumulate on
    the unit that runs them.  The floor is the largest of the three."""
    state = 8.0 * work["params"]
    act = work["act_elems"] * (2.0 if bf16 else 4.0)
    in_l2 = state + act < 0.6 * L2_BYTES
    bw = peaks["l2_gbs"] if in_l2 else peaks["hbm_gbs"]
    t_mem = (16.0 * work["params"] + act) / (bw * 1e9) * 1e6
    t_f32 = 6.0 * (work["macs_conv_f32"] + work["macs_fc"]) / (peaks["fp32_fma_tflops"] * 1e12) * 1e6
    t_tc = 6.0 * work["macs_conv_bf16"] / (peaks["bf16_tflops"] * 1e12) * 1e6
    parts = {"memory_us": t_mem, "fp32_fma_us": t_f32, "tensor_us": t_tc,
             "memory_level": "l2" if in_l2 else "hbm"}
    return max(t_mem, t_f32, t_tc), parts


def time_oracle(wl, budget_s=20.0, max_ticks=None):
    """Times the CPU checker as it stands on steady-state ticks of `wl`."""
    from oracle import PBOracle
    from pb_workloads import he_normal_weights, make_inputs
    S = wl.n_stages
    fill = 2 * (S - 1)
    o = PBOracle(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, wl.lr, wl.momentum, wl.flags & 7)
    o.set_weights(he_normal_weights(wl.seed, wl))
    cap = fill + (max_ticks if max_ticks else 64)
    x, y = make_inputs(wl.seed, cap, wl.sample_elems, wl.n_classes)
    with np.errstate(all="ignore"):
        for t in range(fill):
            o.tick(x[t], y[t])
        n, w0, c0 = 0, time.perf_counter(), time.process_time()
        while n < cap - fill and (n == 0 or time.perf_counter() - w0 < budget_s):
            o.tick(x[fill + n], y[fill + n])
            n += 1
        wall, cpu = time.perf_counter() - w0, time.process_time() - c0
    cores = max(1, int(round(cpu / wall)))
    return {"value": n / wall, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%d steady-state ticks (ticks %d..%d) of %s, numpy float64, %d host cores visible"
                      % (n, fill, fill + n - 1, wl.name, os.cpu_count())}, wall / n


def run_reference(args, rank):
    if rank != 0:
        return
    from pb_workloads import workload
    wl = workload(args.workload)
    base, s_per_tick = time_oracle(wl, budget_s=25.0, max_ticks=max(1, min(args.steps, 16)))
    line = {"impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * s_per_tick, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "stages": wl.n_stages, "note": "CPU checker on host cores"},
            "cpu_baseline": base,
            "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4096)
    ap.add_argument("--warmup", type=int, default=64)
    ap.add_argument("--impl", default="b200")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default=WORKLOAD,
                    help="mlp4 | mlp16x2048 (default, the headline) | vgg11 | resnet20 | resnet50")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2003_11666_b200 import build as pbuild
    if local_rank == 0:
        pbuild.build()
    import paper_2003_11666_b200 as pbm
    from pb_workloads import he_normal_weights, make_inputs, work_per_tick, workload

    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    wl = workload(args.workload)
    K, W = args.steps, max(args.warmup, 3)
    S = wl.n_stages
    F = fill_ticks(S)
    seed = replica_seed(wl.seed, rank)
    n_in = F + W + K
    x, y = make_inputs(seed, n_in, wl.sample_elems, wl.n_classes)
    stream = torch.cuda.current_stream()
    w_init = he_normal_weights(wl.seed, wl)
    xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    losses = torch.zeros(n_in, device="cuda")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def new_engine(lr):
        e = pbm.PB(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, lr, wl.momentum,
                   wl.flags, stream=stream.cuda_stream)
        e.set_weights(w_init)
        return e

    def timed_leg(e, with_clocks):
        """Fill (set-up), W warm-up ticks, then K timed ticks; returns (ms, clocks)."""
        e.run(xd[:F], yd[:F], F, losses[:F])
        e.run(xd[F:F + W], yd[F:F + W], W, losses[F:F + W])
        barrier()
        sampler = ClockSampler(local_rank)
        if with_clocks and rank == 0:
            sampler.start()
            time.sleep(0.3)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        e.run(xd[F + W:], yd[F + W:], K, losses[F + W:])
        e1.record(stream)
        barrier()
        ms_ = max_over_ranks(e0.elapsed_time(e1), world)
        return ms_, (sampler.stop() if with_clocks and rank == 0 else None)

    # ---- device-resident timing, literal hyper-parameters
    eng = new_engine(wl.lr)
    ms, clocks = timed_leg(eng, True)
    launches = eng.last_launch_count
    value = job_value(world, K, ms)
    finite_ticks = int(torch.isfinite(losses[F + W:]).sum().item())

    # ---- per-kernel durations (CUDA events on the engine's streams, separate pass, still steady state)
    eng.profile_enable(True)
    kp = min(K, 512)
    eng.run(xd[F:F + kp], yd[F:F + kp], kp, losses[F:F + kp])
    eng.sync()
    classes = {name: eng.profile_ms(c) for c, name in enumerate(("fc_phase0", "fc_phase1", "update", "conv_simt", "conv_tc_fprop",
                                                               "conv_post_fwd", "conv_post_bwd", "conv_tc_wgrad", "conv_tc_dgrad"))}
    eng.profile_enable(False)
    P = eng.num_params
    hbm_peak, bf16_peak, peak_kind = measured_peaks()
    peaks = {"hbm_gbs": hbm_peak, "hbm_source": peak_kind + " copy rate", "hbm_hw_gbs": HBM_HW_GBS,
             "bf16_tflops": bf16_peak,
             "l2_gbs": pbm.bench_l2_bandwidth(32 << 20, 200, stream.cuda_stream),
             "l2_source": "in-place sweep over 32 MiB, 200 passes, this run",
             "fp32_fma_tflops": pbm.bench_fp32_fma(8192, stream.cuda_stream),
             "fp32_fma_source": "16 FMA chains per thread, 8 blocks of 256 threads per SM, this run"}
    all_fc = all(int(L.op) in (0, 3, 7) for L in wl.layers)
    if all_fc:
        k_ms, k_n = classes["fc_phase0"]
        alg_bytes, kernel = eng.kernel_min_bytes(0), "fc_tick_kernel"
        if classes["fc_phase1"][1]:
            p_last = wl.layers[-2].c_in * wl.layers[-2].c_out + wl.layers[-2].c_out
            alg_bytes -= 16.0 * p_last
            kernel = "fc_tick_kernel(phase 0)"
    else:
        k_ms, k_n = classes["update"]
        alg_bytes, kernel = eng.kernel_min_bytes(2), "update_kernel"
    work = work_per_tick(wl)
    state_bytes = 8.0 * P
    in_l2 = state_bytes + 4.0 * work["act_elems"] < 0.6 * L2_BYTES
    k_peak = peaks["l2_gbs"] if in_l2 else hbm_peak
    traffic, traffic_note = ncu_traffic(args.workload)
    launch_s = k_ms / k_n * 1e-3
    achieved = alg_bytes / launch_s / 1e9
    floor_us, floor_parts = tick_floor(work, peaks, bool(wl.flags & 8))
    roofline = {"bound": "l2" if in_l2 else "hbm", "kernel": kernel, "achieved": achieved, "peak": k_peak,
                "unit": "GB/s", "frac": achieved / k_peak,
                "peak_source": ("L2 sweep of this run" if in_l2 else peak_kind + " copy rate (MEASURED_PEAKS.json)"),
                "frac_of_hw_peak": None if in_l2 else achieved / HBM_HW_GBS,
                "traffic": traffic, "traffic_note": traffic_note,
                "achieved_traffic": (traffic / launch_s / 1e9) if traffic else None,
                "algorithmic_bytes_per_launch": alg_bytes, "avg_launch_ms": k_ms / k_n, "launches_timed": k_n,
                "peaks": peaks,
                "tick_floor_us": floor_us, "tick_floor_parts": floor_parts,
                "tick_frac": floor_us / (1e3 * ms / K),
                "us_per_tick_by_class": {n: (1e3 * m / kp if c else 0.0) for n, (m, c) in classes.items()}}
    eng.destroy()

    # ---- the same workload at a bounded step size (finite numbers in every kernel)
    stable = None
    if args.workload in STABLE_LR:
        es = new_engine(STABLE_LR[args.workload])
        ms_s, clocks_s = timed_leg(es, True)
        stable = {"lr": STABLE_LR[args.workload], "ms_per_step": ms_s / K, "value": job_value(world, K, ms_s),
                  "finite_losses": int(torch.isfinite(losses[F + W:]).sum().item()), "of": K,
                  "sm_mhz": clocks_s["sm_mhz"] if clocks_s else None}
        es.destroy()

    # ---- end to end through the host-buffer entry point (pinned memory, copies timed)
    eng = new_engine(wl.lr)
    hx = torch.from_numpy(x).pin_memory()
    hy = torch.from_numpy(y).pin_memory()
    hl = torch.zeros(n_in).pin_memory()
    # set-up: fill the pipeline, then a warm-up call of the timed call's size, which also sizes
    # the library's staging buffer so that the timed call allocates nothing
    eng.run_host(hx[:F], hy[:F], F, hl[:F])
    eng.run_host(hx[F + W:], hy[F + W:], K, hl[F + W:])
    barrier()
    t0 = time.perf_counter()
    eng.run_host(hx[F + W:], hy[F + W:], K, hl[F + W:])
    torch.cuda.synchronize()
    e2e_ms = max_over_ranks((time.perf_counter() - t0) * 1e3, world)
    e2e = {"value": job_value(world, K, e2e_ms), "unit": UNIT,
           "h2d_bytes_per_step": wl.sample_elems * 4 + 4, "d2h_bytes_per_step": 4}
    eng.destroy()

    if rank == 0:
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            cpu, _ = time_oracle(wl, budget_s=15.0, max_ticks=8)
        # a tick cannot move its parameters faster than the memory system allows: refuse a
        # number that says otherwise (it would mean work was skipped in the timed region)
        rejected = None
        if state_bytes > L2_BYTES:
            implied = 16.0 * P / (ms / K * 1e-3) / 1e9 / world
            if implied > 1.2 * hbm_peak:
                rejected = "implied %.0f GB/s per GPU for 16 B/parameter exceeds 1.2 x the %.0f GB/s copy peak" % (implied, hbm_peak)
        line = {"metric": METRIC, "value": None if rejected else value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
                "fill_ticks": F, "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16" if wl.flags & 8 else "f32", "data": "synthetic",
                "config": {"workload": args.workload, "stages": S, "params": P, "batch": 1,
                           "parallelism": "replicas x%d" % world if world > 1 else "1 gpu",
                           "l2": ("weights+velocity %.0f MB stream from HBM every tick (> 126 MB L2), no flush needed" % (8e-6 * P))
                                 if state_bytes > L2_BYTES else
                                 ("weights+velocity %.1f MB stay in the L2 cache by design (steady state of the method); no flush" % (8e-6 * P)),
                           "steady_state": "timed ticks %d..%d, all %d stages forward, backward and update in each" % (F + W, F + W + K - 1, S),
                           "note": "literal hyper-parameters; losses finite on %d of %d timed ticks "
                                   "(the deep MLP and ResNet-50 runs diverge); stable_lr times the same "
                                   "kernels on finite numbers" % (finite_ticks, K)},
                "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
                "roofline": roofline, "stable_lr": stable, "cpu_baseline": cpu}
        if rejected:
            line["rejected"] = rejected
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
