"""Benchmark of the M-AVG round (Algorithm 1) on one B200 per rank.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl mavg|reference]

A step is one full round -- K_local SGD steps on all P learners, then the fused meta-update --
of the large MLP workload (3072-2048-2048-2048-10, bf16 GEMM operands, fp32 masters, P=32,
K_local=16, B=64: the largest configuration of the workload list that fits one GPU, and the one
whose kernels are bound by HBM) on seeded synthetic data.  Prints ONE JSON line (rank 0); the same
line carries, as extra keys, the CIFAR-shaped MLP (3072-512-512-10, P=8, K=8, B=128), the full
round at 25.6 M parameters with seeded pseudo-gradients (K = 1 and 64) and the meta-update sweep
at 11.2 M parameters.  With --gpus N > 1 every rank runs an independent replica of the same
workload on its own GPU (the method is simulated on one GPU; there is no exchange between GPUs),
and `value` is the sum over ranks.

--impl reference times the CPU oracle (oracle/) on the host cores on a bounded sample of the same
workload; it is a deliberately plain program and only a baseline.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "learner-samples/sec per MAVG round; meta-update HBM GB/s vs peak (1 B200)"
UNIT = "learner-samples/s"
WORKLOAD = "C4"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0,
                source="fallback")


class ClockSampler:
    """nvidia-smi clock/throttle samples taken while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-i", str(self.gpu), "-lms", "50"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f:
            t = [s.strip() for s in line.split(",")]
            if len(t) < 9:
                continue
            try:
                sm.append(float(t[1]))
                mx.append(float(t[2]))
            except ValueError:
                continue
            for name, val in zip(names, t[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        return out


def workload_inputs(name=None):
    from paper_2110_00625_b200 import workloads as W
    cfg = dict(W.CONFIGS[name or WORKLOAD])
    x, y = W.make_dataset(cfg)
    w1 = W.mlp_init(cfg["dims"])
    return cfg, x, y, w1


def workload_label(name, cfg):
    kind = {"C2": "CIFAR-shaped MLP", "C4": "large MLP"}.get(name, "MLP")
    return (f"{name} {kind} {'-'.join(map(str, cfg['dims']))}, P={cfg['P']}, K={cfg['K']}, "
            f"B={cfg['B']}, mu={cfg['mu']}, gamma={cfg['gamma']}, 50000 synthetic samples, labels "
            "from a random teacher")


def flop_per_sample(dims):
    # forward + weight gradient for every layer, data gradient for all but the first
    macs = sum(dims[l] * dims[l + 1] for l in range(len(dims) - 1))
    return 6 * macs - 2 * dims[0] * dims[1]


def cpu_oracle_rate(cfg, x, y, w1, k_sample, reps=1):
    """learner-samples/s of the oracle on a round cut down to k_sample local steps."""
    from oracle import oracle as O
    threads = min(cfg["P"], O.max_threads())
    o = O.Mavg(w1, P=cfg["P"], K=k_sample, gamma=cfg["gamma"], mu=cfg["mu"], zeta=cfg["zeta"],
               B=cfg["B"], seed=0x211000625, objective=O.OBJ_MLP, dims=cfg["dims"],
               bf16=bool(cfg["bf16"]), x=x, y=y, threads=threads)
    times = []
    for _ in range(reps):
        t0 = time.perf_counter()
        o.run_round()
        times.append(time.perf_counter() - t0)
    units = cfg["P"] * k_sample * cfg["B"]
    return units / statistics.median(times), threads, times


def bounded_oracle_sample(cfg, x, y, w1, budget_s):
    """Sizes a sample of the workload that the oracle finishes in about budget_s seconds: k_s of
    the K local steps on p_s of the P learners (+ their meta-update).  One (learner, step) is the
    smallest piece; it is timed first, on one thread."""
    from oracle import oracle as O
    _, _, t_cal = cpu_oracle_rate(dict(cfg, P=1), x, y, w1, 1, reps=1)
    t1 = max(t_cal[0], 1e-6)
    threads = min(cfg["P"], O.max_threads())
    waves = max(1, int(budget_s / t1))                     # pieces one thread can take in turn
    p_s = int(min(cfg["P"], threads * waves))              # whole waves of learners over the threads
    per_step = -(-p_s // threads)                          # waves one local step costs
    k_s = int(min(cfg["K"], max(1, waves // per_step)))
    return p_s, k_s, t1


def oracle_table():
    """The oracle timed on this host for every workload of the list (bounded samples where a full
    round would take minutes), with the threads it used.  Context figures for the results table."""
    from oracle import oracle as O
    from paper_2110_00625_b200 import workloads as W
    cores = O.max_threads()
    out = {"host_threads_available": cores}
    # C1: one full round, median of 3
    cfg, x, y, w1 = workload_inputs("C1")
    rate, th, times = cpu_oracle_rate(cfg, x, y, w1, cfg["K"], reps=3)
    out["C1"] = dict(learner_samples_per_s=rate, threads=th, seconds_per_round=statistics.median(times),
                     sample="full round")
    for name, budget in (("C2", 15.0), ("C4", 20.0)):
        cfg, x, y, w1 = workload_inputs(name)
        p_s, k_s, t1 = bounded_oracle_sample(cfg, x, y, w1, budget)
        rate, th, times = cpu_oracle_rate(dict(cfg, P=p_s), x, y, w1, k_s)
        out[name] = dict(learner_samples_per_s=rate, threads=th, seconds=times[0],
                         single_thread_seconds_per_learner_step=t1,
                         sample=f"{k_s} of {cfg['K']} local steps on {p_s} of {cfg['P']} learners + meta-update")
    # C3: the meta-update alone, n = 11.2 M, P = 16 (single thread: the oracle's loop over elements)
    n, P = W.CONFIGS["C3"]["n"], 16
    w1 = W.global_model(n)
    o = O.Mavg(w1, P=P, K=1, gamma=0.1, mu=0.9)
    o.replicas[:, :n] = w1[None, :] + np.float32(0.1)
    t0 = time.perf_counter(); o.meta_update(); t = time.perf_counter() - t0
    out["C3"] = dict(P=P, seconds_per_update=t, gbs=(8 * P + 16) * n / t / 1e9, threads=1,
                     sample="one meta-update at P = 16")
    # C5: one full round at K = 1 and K = 4 (local steps over the learners in parallel + meta-update)
    c5 = W.CONFIGS["C5"]
    w1 = W.global_model(c5["n"])
    for K in (1, 4):
        o = O.Mavg(w1, P=c5["P"], K=K, gamma=c5["gamma"], mu=0.9, seed=W.BASE_SEED,
                   objective=O.OBJ_PSEUDOGRAD, sigma=c5["sigma"], threads=min(c5["P"], cores))
        t0 = time.perf_counter(); o.run_round(); t = time.perf_counter() - t0
        out[f"C5_K{K}"] = dict(seconds_per_round=t, learner_steps_per_s=c5["P"] * K / t,
                               threads=min(c5["P"], cores), sample="one full round")
    print(json.dumps({"oracle_table": out}))
    return 0


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    name = args.workload if args.workload in ("C2", "C4") else WORKLOAD
    cfg, x, y, w1 = workload_inputs(name)
    # Bounded sample per step, sized from one calibration piece so that the whole run stays near
    # two minutes.
    total = args.warmup + args.steps
    p_s, k_s, t1 = bounded_oracle_sample(cfg, x, y, w1, 120.0 / max(total, 1))
    sub = dict(cfg, P=p_s)
    rate, threads, times = cpu_oracle_rate(sub, x, y, w1, k_s, reps=total)
    timed = times[args.warmup:]
    units = p_s * k_s * cfg["B"]
    value = units * len(timed) / sum(timed)
    sample = (f"each step = {k_s} of the {cfg['K']} local steps on {p_s} of the {cfg['P']} learners "
              f"(B={cfg['B']}) + their meta-update = {units} learner-samples")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(timed) / len(timed),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": workload_label(name, cfg) + " (bounded sample per step)",
                   "global_batch": cfg["P"] * cfg["B"]},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))
    return 0


# DRAM read + write bytes of ONE launch of the dominant kernel class, from the committed ncu
# captures (profiles/): None when no capture of the kernel as it stands exists.  The large MLP
# holds ~4.5 GB on the device at P = 32; its capture is taken with 8 learners (same layer shapes,
# kernels and tile plans) and scaled by 4, since every kernel's traffic is proportional to P.
NCU_TRAFFIC = {
    "C2": {"wgrad_sgd_gemm": None, "fwd_gemm": None, "dgrad_gemm": None},
    # profiles/step_kernels_c4_p8.md: sums over a middle step's launches of the class at P = 8,
    # times 4, divided by the launches of the class (4 weight-gradient, 1 forward, 3 dgrad)
    "C4": {"wgrad_sgd_gemm": 945.9e6, "fwd_gemm": 10.2e6, "dgrad_gemm": 198.2e6},
}


def algorithmic_bytes(cfg, tensor_path, deferred=False, momentum=False, fwd_run_tiles=(),
                      dense_layers=(), fwd_whole_rows=()):
    """Bytes that must cross HBM per ROUND for each kernel class (weights streamed once per
    product, activations in and out), and their total.  fwd_run_tiles[l-1], layers l = 1..m: in
    steps 1..K-1 the weight-gradient launch of layer l also forms the next step's forward product
    of that layer: its bf16 weights are not read by a forward kernel in steps 2..K (layer 1's copy
    is not even written); the layer's next input is read and its next activations are written by
    the weight-gradient launch, which also writes and reads back one fp32 partial sum [128, B]
    per learner, row tile and run of fwd_run_tiles[l-1] column tiles (not for the fwd_whole_rows[l-1]
    (learner, row tile) pairs that are taken as one run); the flops move with them.
    dense_layers: hidden layers whose first-step forward is one dense product over all learners'
    batch rows, reading the (shared) weights once instead of once per learner."""
    dims, P, K, B = cfg["dims"], cfg["P"], cfg["K"], cfg["B"]
    L = len(dims) - 1
    nW = [dims[l] * dims[l + 1] for l in range(L)]
    n = sum(nW) + sum(dims[1:])
    rows = P * B
    fwd_delta = wgrad_delta = flop_delta = 0
    for l in dense_layers:
        fwd_delta -= 2 * (P - 1) * nW[l - 1]
    for i, run in enumerate(fwd_run_tiles if K > 1 else ()):
        n_tiles = -(-dims[i] // 32)
        runs = -(-n_tiles // run)
        split_rows = P * -(-dims[i + 1] // 128) - (fwd_whole_rows[i] if i < len(fwd_whole_rows) else 0)
        partial = split_rows * runs * B * 128 * 4 if runs > 1 else 0
        moved = 2 * rows * dims[i] + 4 * rows * dims[i + 1]     # the layer's input read, A_l written twice
        fwd_delta -= (K - 1) * (2 * P * nW[i] + moved)
        wgrad_delta += (K - 1) * (moved + 2 * partial - (2 * P * nW[0] if i == 0 else 0))
        flop_delta += (K - 1) * 2 * rows * nW[i]
    per_round = {
        # replicas, w~, v read; v, w~ and (unless the copies are deferred) the replicas written
        "meta_update": dict(bytes=((4 if deferred else 8) * P + 16) * n, flops=0),
        # bf16 weights read once per learner and step; activations in and out
        "fwd_gemm": dict(bytes=K * (2 * P * sum(nW) + 2 * rows * (sum(dims[:-1]) + 2 * sum(dims[1:]))),
                         flops=K * 2 * rows * sum(nW)),
        "dgrad_gemm": dict(bytes=K * (2 * P * sum(nW[1:]) + 2 * rows * (sum(dims[2:]) + 3 * sum(dims[1:-1]))),
                           flops=K * 2 * rows * sum(nW[1:])),
        # fp32 master read + written, bf16 copy written; on the tensor-core path the first step
        # of a round reads the one copy of w~ instead of P masters
        # (learner momentum: the fp32 u tile read and written as well)
        "wgrad_sgd_gemm": dict(bytes=K * (P * (18 if momentum else 10) * sum(nW) + 2 * rows * sum(dims))
                               - (4 * (P - 1) * sum(nW) if tensor_path else 0),
                               flops=K * 2 * rows * sum(nW)),
    }
    per_round["fwd_gemm"]["bytes"] += fwd_delta
    per_round["fwd_gemm"]["flops"] -= flop_delta
    per_round["wgrad_sgd_gemm"]["bytes"] += wgrad_delta
    per_round["wgrad_sgd_gemm"]["flops"] += flop_delta
    return per_round


def kernel_rooflines(cfg, prof, steps, peaks, tensor_path, deferred=False, momentum=False,
                     fwd_run_tiles=(), dense_layers=(), fwd_whole_rows=()):
    """Per kernel class: algorithmic bytes or flops of all its launches / its summed device time."""
    per_round = algorithmic_bytes(cfg, tensor_path, deferred, momentum, fwd_run_tiles, dense_layers,
                                  fwd_whole_rows)
    out = {}
    for name, (ms, cnt) in prof.items():
        if cnt == 0 or ms <= 0:
            continue
        e = dict(ms_total=ms, launches=cnt, ms_per_launch=ms / cnt)
        if name in per_round:
            w = per_round[name]
            sec = ms * 1e-3
            e["gbs"] = w["bytes"] * steps / sec / 1e9
            e["frac_hbm"] = e["gbs"] / peaks["hbm_gbs"]
            if w["flops"]:
                e["tflops"] = w["flops"] * steps / sec / 1e12
                e["frac_tensor"] = e["tflops"] / peaks["bf16_tflops_sustained"]
            e["bytes_per_launch"] = w["bytes"] * steps / cnt
        out[name] = e
    return out


def meta_update_sweep(m, torch, peaks, reps=7, inner=10):
    """Meta-update alone at the ResNet-18-sized sweep: n = 11.2 M, P in {4, 16, 64}, mu in {0, 0.9}.
    Per repetition: fresh replicas ~ N(0, 0.01) around the current model (untimed), L2 flushed by a
    256 MiB memset, then `inner` meta-updates back to back inside one event pair (their time does
    not depend on the data; each of them streams more than the L2 holds); also one launch alone
    right after a flush (`cold_gbs`)."""
    n = 11_200_000
    res = []
    w1 = (0.05 * torch.randn(n, generator=torch.Generator().manual_seed(1))).numpy()
    for P in (4, 16, 64):
        for mu in (0.0, 0.9):
            g = m.Mavg(w1, P=P, K=1, local_lr=0.1, mu=mu, objective=m.OBJ_NONE)
            flush = torch.empty(256 << 20, dtype=torch.uint8, device=g.device)
            gen = torch.Generator(device=g.device).manual_seed(P)
            times, cold = [], []
            for u in range(2 + reps):
                g.replicas[:, :n] = g.w[None, :] + 0.1 * torch.randn((P, n), device=g.device,
                                                                     generator=gen)
                for count, sink in ((1, cold), (inner, times)):
                    flush.zero_()
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record()
                    for _ in range(count):
                        g.meta_update()
                    b.record()
                    b.synchronize()
                    if u >= 2:
                        sink.append(a.elapsed_time(b) / count)
            g.sync()
            by = ((8 * P + 16) - (4 if mu == 0.0 else 0)) * n
            ms = statistics.median(times)
            res.append(dict(P=P, mu=mu, n=n, ms=ms, gbs=by / ms / 1e6,
                            frac_measured=by / ms / 1e6 / peaks["hbm_gbs"],
                            frac_nominal_8tbs=by / ms / 1e6 / 8000.0,
                            cold_gbs=by / statistics.median(cold) / 1e6,
                            launches_per_timing=inner))
            g.close()
            del g, flush
            torch.cuda.empty_cache()
    return res


def reduce_max_over_ranks(values, device=None):
    """MAX over ranks of a list of floats (the slowest rank's times count); identity without a
    process group.  Works on any backend: the tensor lives on `device`."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_value(units_per_step, steps, total_ms, world):
    """Aggregate throughput of `world` independent replicas of the workload (replicas only: the
    method is simulated inside one GPU, there is nothing to exchange between GPUs)."""
    return world * units_per_step * steps / (total_ms * 1e-3)


def pseudograd_rounds(args, m, torch, peaks, Ks, steps):
    """Full round at the ResNet-50-sized vector (n = 25.6 M, P = 16) with seeded pseudo-gradients:
    per K the local pass, the meta-update and the whole round."""
    from paper_2110_00625_b200 import workloads as W
    cfg = W.CONFIGS["C5"]
    n, P = args.n or cfg["n"], cfg["P"]
    w1 = W.global_model(n)
    out = []
    for K in Ks:
        g = m.Mavg(w1, P=P, K=K, local_lr=cfg["gamma"], mu=0.9, seed=W.BASE_SEED,
                   objective=m.OBJ_PSEUDOGRAD, sigma=cfg["sigma"], defer_broadcast=not args.no_defer,
                   learner_momentum=args.beta)
        for _ in range(3):
            g.round()
        g.sync()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
        for a, b, c in ev:
            a.record(); g.local_steps(); b.record(); g.meta_update(); c.record()
        torch.cuda.synchronize()
        loc = statistics.median(a.elapsed_time(b) for a, b, c in ev)
        met = statistics.median(b.elapsed_time(c) for a, b, c in ev)
        # the local pass reads w~ once (every learner starts from it) and writes P learner models;
        # the meta-update reads them with w~ and v and writes w~, v and, unless deferred, P copies
        meta_b = ((8 if args.no_defer else 4) * P + 16) * n
        local_b = ((12 if args.beta else 4) * P + 4) * n
        var_rate = P * K * n / (loc * 1e-3)
        out.append(dict(K=K, local_ms=loc, meta_ms=met, round_ms=loc + met,
                        learner_steps_per_s=P * K / ((loc + met) * 1e-3),
                        local_gbs=local_b / loc / 1e6,
                        local_frac_hbm=local_b / loc / 1e6 / peaks["hbm_gbs"],
                        learner_momentum=args.beta,
                        variates_per_s=var_rate,
                        local_frac_alu=var_rate / PSEUDOGRAD_ALU_PEAK_VARIATES,
                        meta_gbs=meta_b / met / 1e6,
                        meta_frac_measured=meta_b / met / 1e6 / peaks["hbm_gbs"],
                        defer_broadcast=not args.no_defer))
        g.close()
        del g
        torch.cuda.empty_cache()
    return out


# Peak rate of the K-fused pseudo-gradient pass when instruction issue binds (variates/s): the
# kernel executes 29.5 instructions per variate (ncu: 4.717e8 warp instructions for 5.12e8
# variates at n = 2 M, P = 16, K = 16, profiles/pseudograd_k16.md; 64-bit SplitMix64 arithmetic on
# 32-bit ALUs), against an issue rate of 148 SMs x 4 schedulers x 1 warp instruction (32 lanes)
# per clock at the maximum SM clock of 1965 MHz.
PSEUDOGRAD_INSTR_PER_VARIATE = 29.5
PSEUDOGRAD_ALU_PEAK_VARIATES = 148 * 4 * 32 * 1.965e9 / PSEUDOGRAD_INSTR_PER_VARIATE


def run_pseudograd(args, m, torch, peaks, rank):
    from paper_2110_00625_b200 import workloads as W
    Ks = [int(k) for k in args.ks.split(",")] if args.ks else W.CONFIGS["C5"]["K"]
    out = pseudograd_rounds(args, m, torch, peaks, Ks, args.steps)
    if rank == 0:
        print(json.dumps({"workload": "C5 full round, n=25.6M fp32, P=16, seeded pseudo-gradients",
                          "steps": args.steps, "results": out}))
    return 0


def measure_mlp(name, args, m, torch, dist, peaks, world, rank, local, steps, with_cpu, with_e2e,
                with_clocks):
    """Times `steps` rounds of an MLP workload three ways: device-resident (one event pair per
    round, L2 flushed between rounds), end to end through mavg_round_host, and per kernel class.
    Returns the pieces of the JSON line."""
    cfg, x, y, w1 = workload_inputs(name)
    if args.learners:
        cfg["P"] = args.learners      # reduced-size captures under a profiler only

    # CPU baseline first (rank 0, single-GPU runs only), before the GPU is busy
    cpu = None
    if with_cpu:
        p_s, k_s, t1 = bounded_oracle_sample(cfg, x, y, w1, 20.0)
        rate, threads, times = cpu_oracle_rate(dict(cfg, P=p_s), x, y, w1, k_s)
        cpu = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": f"one round cut to {k_s} of {cfg['K']} local steps on {p_s} of "
                         f"{cfg['P']} learners + their meta-update ({p_s * k_s * cfg['B']} "
                         f"learner-samples, {times[0]:.1f} s)"}

    mode = args.gemm
    g = m.Mavg(w1, P=cfg["P"], K=cfg["K"], local_lr=cfg["gamma"], mu=cfg["mu"],
               block_lr=cfg["zeta"], B=cfg["B"], seed=0x211000625, objective=m.OBJ_MLP,
               dims=cfg["dims"], gemm_bf16=mode, x=x, y=y, x_bf16=True, device=f"cuda:{local}",
               defer_broadcast=not args.no_defer, learner_momentum=args.beta, l2_keep=args.l2_keep)
    g.set_schedule(args.schedule)
    units = cfg["P"] * cfg["K"] * cfg["B"]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=g.device)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        g.round()
    g.sync()

    # ---- timed region: device-resident inputs -------------------------------------------------
    sampler = ClockSampler(local) if with_clocks else None
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True),
           torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    l0 = g.launch_count()
    barrier()
    if sampler:
        sampler.start()
    t_wall0 = time.perf_counter()
    for a, mid, b in ev:
        if args.l2_keep:
            g.l2_release()                 # masters the library asked the L2 to keep: let go
        flush.zero_()                      # L2 flush, outside the step's event pair
        a.record()
        g.local_steps()
        mid.record()
        g.meta_update()
        b.record()
    barrier()
    t_wall = time.perf_counter() - t_wall0
    clocks = sampler.stop() if sampler else None
    launches = g.launch_count() - l0
    step_ms = [a.elapsed_time(b) for a, _, b in ev]
    meta_ms = [mid.elapsed_time(b) for _, mid, b in ev]
    total_ms = sum(step_ms)
    g.sync()

    # ---- end to end: model in host memory, copies inside the timed region ----------------------
    e2e_ms = 0.0
    if with_e2e:
        wh = torch.from_numpy(w1.copy()).pin_memory()
        vh = torch.zeros(g.n).pin_memory()
        for _ in range(2):
            g.round_host(wh, vh)
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps):
            g.round_host(wh, vh)
        b.record()
        barrier()
        e2e_ms = a.elapsed_time(b)

    # ---- per-kernel device times: the same steps again with an event pair around every launch ---
    g.set_profiling(True)
    g.get_profile(reset=True)
    psteps = min(steps, 20)
    for _ in range(psteps):
        if args.l2_keep:
            g.l2_release()
        flush.zero_()
        g.round()
    prof = g.get_profile(reset=True)
    g.set_profiling(False)
    plan = g.get_step_plan()
    fwd_run_tiles = tuple(plan["fwd_run_tiles"]) if args.schedule == 0 else ()
    dense_layers = tuple(plan["dense_first_step"]) if args.schedule == 0 else ()
    fwd_whole_rows = tuple(plan["fwd_whole_rows"]) if args.schedule == 0 else ()
    kern = kernel_rooflines(cfg, prof, psteps, peaks, mode == 1, deferred=not args.no_defer,
                            momentum=args.beta != 0.0, fwd_run_tiles=fwd_run_tiles,
                            dense_layers=dense_layers, fwd_whole_rows=fwd_whole_rows)
    n = g.n
    g.close()
    del g, flush
    torch.cuda.empty_cache()

    total_ms, e2e_ms = reduce_max_over_ranks([total_ms, e2e_ms], device=torch.device("cuda", local))

    # the roofline object describes the kernel class a local step spends most of its time in
    timed = {k: v for k, v in kern.items() if "gbs" in v and k != "meta_update"}
    dom = max(timed, key=lambda k: timed[k]["ms_total"]) if timed else None
    roof = None
    if dom:
        e = timed[dom]
        hbm_time = e["bytes_per_launch"] / (peaks["hbm_gbs"] * 1e9)
        tensor_time = (e.get("tflops", 0) and
                       e["tflops"] * 1e12 * e["ms_per_launch"] * 1e-3 /
                       (peaks["bf16_tflops_sustained"] * 1e12))
        if tensor_time and tensor_time > hbm_time:
            roof = {"bound": "tensor", "achieved": e["tflops"],
                    "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                    "frac": e["frac_tensor"], "traffic": None}
        else:
            roof = {"bound": "hbm", "achieved": e["gbs"], "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": e["frac_hbm"], "traffic": None}
        roof["kernel"] = dom
        roof["peak_source"] = peaks["source"]
        roof["bytes_per_launch"] = e["bytes_per_launch"]
        roof["ms_per_launch"] = e["ms_per_launch"]
        if mode == 1 and not args.learners and not args.beta:
            roof["traffic"] = NCU_TRAFFIC.get(name, {}).get(dom)
    # the whole round against the HBM roofline: every class's algorithmic bytes / the round's time
    per_round = algorithmic_bytes(cfg, mode == 1, deferred=not args.no_defer,
                                  momentum=args.beta != 0.0, fwd_run_tiles=fwd_run_tiles,
                                  dense_layers=dense_layers, fwd_whole_rows=fwd_whole_rows)
    round_bytes = sum(v["bytes"] for v in per_round.values())
    ms_round = total_ms / steps
    return dict(
        cfg=cfg, n=n, units=units, fwd_run_tiles=fwd_run_tiles, dense_layers=dense_layers,
        fwd_whole_rows=fwd_whole_rows, total_ms=total_ms, e2e_ms=e2e_ms, launches=launches,
        clocks=clocks, cpu=cpu, kern=kern, roof=roof, t_wall=t_wall, mode=mode,
        meta_in_round={"ms": statistics.median(meta_ms),
                       "gbs": per_round["meta_update"]["bytes"] / statistics.median(meta_ms) / 1e6},
        round_roofline={"bytes_per_round": round_bytes, "gbs": round_bytes / ms_round / 1e6,
                        "frac_hbm": round_bytes / ms_round / 1e6 / peaks["hbm_gbs"]},
        tflops_round=flop_per_sample(cfg["dims"]) * units * steps / (total_ms * 1e-3) / 1e12)


def run_mavg(args):
    import torch
    import torch.distributed as dist
    import paper_2110_00625_b200 as m

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = measured_peaks()
    if args.workload == "C5":
        return run_pseudograd(args, m, torch, peaks, rank)
    if args.sweep_only:
        print(json.dumps({"meta_update_sweep": meta_update_sweep(m, torch, peaks, reps=3)}))
        return 0

    single = rank == 0 and world == 1
    r = measure_mlp(args.workload, args, m, torch, dist, peaks, world, rank, local, args.steps,
                    with_cpu=single and not args.no_cpu_baseline, with_e2e=True, with_clocks=True)
    extras = {}
    if single and not args.no_extras:
        # the other workloads of the list, shorter, in the same process and on the same line
        other = "C2" if args.workload == "C4" else "C4"
        o = measure_mlp(other, args, m, torch, dist, peaks, world, rank, local,
                        steps=min(args.steps, 50), with_cpu=False, with_e2e=False, with_clocks=False)
        extras[other] = {
            "workload": workload_label(other, o["cfg"]), "ms_per_round": o["total_ms"] / min(args.steps, 50),
            "learner_samples_per_s": whole_job_value(o["units"], min(args.steps, 50), o["total_ms"], 1),
            "tflops_round": o["tflops_round"], "round_roofline": o["round_roofline"],
            "kernels": {k: {q: v[q] for q in ("ms_per_launch", "gbs", "frac_hbm", "tflops") if q in v}
                        for k, v in o["kern"].items()},
            "meta_update_in_round": o["meta_in_round"]}
        extras["C5"] = {"workload": "C5 full round, n=25.6M fp32, P=16, seeded pseudo-gradients, mu=0.9",
                        "results": pseudograd_rounds(args, m, torch, peaks, (1, 64), 20)}
    sweep = meta_update_sweep(m, torch, peaks) if single and not args.no_sweep else None

    if rank == 0:
        cfg, n, steps = r["cfg"], r["n"], args.steps
        clocks = r["clocks"]
        line = {
            "metric": METRIC, "value": whole_job_value(r["units"], steps, r["total_ms"], world),
            "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": args.warmup,
            "ms_per_step": r["total_ms"] / steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if r["mode"] else "f32", "data": "synthetic",
            "config": {"workload": workload_label(args.workload, cfg),
                       "global_batch": cfg["P"] * cfg["B"], "parallelism": "replicas only",
                       "gemm": {1: "tcgen05 tensor cores", 2: "CUDA cores, bf16-rounded operands",
                                0: "CUDA cores fp32"}[r["mode"]],
                       "defer_broadcast": not args.no_defer, "learner_momentum": args.beta,
                       "l2_keep": bool(args.l2_keep),
                       "schedule": {0: "CUDA graph of per-product launches",
                                    2: "CUDA graph of per-product launches, plain tensor-core tiles"}[args.schedule],
                       "forward_products": (f"layers 1..{len(r['fwd_run_tiles'])} inside their weight-gradient "
                                            "launch of the step before (steps 2..K; partial sums per "
                                            f"{list(r['fwd_run_tiles'])} column tiles, after {list(r['fwd_whole_rows'])} "
                                            "(learner, row tile) pairs taken whole)"
                                            if r["fwd_run_tiles"] else "launches of their own"),
                       "first_step_forward": (f"layers {list(r['dense_layers'])}: one dense product over the "
                                              "batch rows of all learners" if r["dense_layers"]
                                              else "per-learner tiles reading the one bf16 copy of the global model"),
                       "l2": "flushed between steps by a 256 MiB memset, outside the step's events",
                       "kernel_timing": "second pass over the same steps with one event pair per launch"},
            "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"],
                       "reasons": clocks["reasons"], "samples": clocks["samples"]},
            "e2e": {"value": whole_job_value(r["units"], steps, r["e2e_ms"], world), "unit": UNIT,
                    "h2d_bytes_per_step": 8 * n, "d2h_bytes_per_step": 8 * n + 4},
            "gpu_launches": r["launches"],
            "roofline": r["roof"],
            "cpu_baseline": r["cpu"],
            "wall_s_timed_region": r["t_wall"],
            "round_roofline": r["round_roofline"],
            "meta_update_in_round": r["meta_in_round"],
            "kernels": r["kern"],
            "meta_update_sweep": sweep,
            "tflops_round": r["tflops_round"],
            "other_workloads": extras or None,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="mavg", choices=["mavg", "reference"])
    ap.add_argument("--gemm", type=int, default=1, choices=[1, 2],
                    help="1: tensor cores (default); 2: CUDA cores with bf16-rounded operands")
    ap.add_argument("--workload", default=WORKLOAD, choices=["C2", "C4", "C5"],
                    help="C4 (large MLP) is the benchmark workload; C2 (CIFAR-shaped MLP) as the "
                         "main workload, or C5 (pseudo-gradient round at 25.6 M parameters) alone")
    ap.add_argument("--learners", type=int, default=0,
                    help="override P (for small profiler captures; not a benchmark setting)")
    ap.add_argument("--n", type=int, default=0,
                    help="override the vector length of --workload C5 (small profiler captures)")
    ap.add_argument("--ks", default="", help="comma-separated K values for --workload C5")
    ap.add_argument("--sweep-only", action="store_true",
                    help="run only the meta-update sweep (profiler captures)")
    ap.add_argument("--beta", type=float, default=0.0,
                    help="learner-level momentum (0 = Algorithm 1 as printed, the benchmark setting)")
    ap.add_argument("--schedule", type=int, default=0, choices=[0, 2],
                    help="0: the default CUDA graph; 2: the graph with every product as plain "
                         "tensor-core tiles (for comparison)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--oracle-table", action="store_true",
                    help="time the CPU oracle on every workload of the list (context figures)")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the other workloads that the default line carries as extra keys")
    ap.add_argument("--l2-keep", action="store_true",
                    help="ask the library to set L2 aside for the learners' masters (small models)")
    ap.add_argument("--no-defer", action="store_true",
                    help="write the P copies of w~ in the meta-update instead of folding them into "
                         "the next round's first local step")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "mavg":
        args.warmup = 3
    if args.oracle_table:
        return oracle_table()
    if args.impl == "reference":
        return run_reference(args)
    return run_mavg(args)


if __name__ == "__main__":
    sys.exit(main())
