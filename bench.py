#!/usr/bin/env python
"""Benchmark of the AET-SGD hot path: client-SGD samples per second.

One step = one pass of the whole path (schedule -> waves of local-SGD rounds ->
ordered aggregation) over one workload: `aet_reset` + `aet_run_rounds(R)`.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5] [--impl reference]

Prints one JSON line.  The default workload is cfg5 at 1,024 clients; the line also carries the
other configurations, device-timed for a few passes each, under `per_config`.  A pass of cfg5
takes under 2 ms, so a step repeats the pass (`config.passes_per_step`) until the timed region
is long enough for the clock sampler.  `value` is device-timed with the inputs resident in HBM;
`e2e` goes through the C ABI from pinned host buffers; `roofline` is the
local-SGD kernel against the measured HBM copy bandwidth; `cpu_baseline` is the
CPU checker timed on this machine.  With several GPUs every rank runs an independent
replica (own seed) and the job value is all samples over the slowest rank's time.
"""
from __future__ import annotations

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

import numpy as np  # noqa: E402

METRIC = "client_sgd_samples_per_sec"
UNIT = "samples/s"
CPU_LIMIT_S = 15.0      # CPU-baseline sample per run
REF_STEP_LIMIT_S = 2.5  # --impl reference: CPU work per step

DESCRIBE = {
    "cfg1": "cfg1: 4 clients, softmax regression 784->10 fp32, l2 1e-4, s_i=10i+10, 5 rounds",
    "cfg2": "cfg2: 16 clients, softmax regression 784->10 fp32, 60,000 samples Dirichlet(0.5), batch 1, "
            "s_i=20i+20, 30 rounds, 2 stragglers x10",
    "cfg3": "cfg3: 32 clients, MLP 784-128-10 fp32, batch 32, s_i=64i+64, 40 rounds",
    "cfg4": "cfg4: 64 clients, MLP 3072-256-128-10 bf16 operands / fp32 accumulate, batch 64, s_i=128i+128, 30 rounds",
    "cfg5": "cfg5: 1,024 clients, softmax regression 784->10 fp32, 1,024 samples/client, s_i=8i+8, 10 rounds",
    "cfg6": "cfg6 (the paper's own setting, Appendix Table 2): 5 nodes, softmax regression 784->10 fp32, "
            "s_i=10i from round 1, 110 rounds, eta_0=0.01 beta=0.01, d=1, uniform delays",
}
DESCRIBE["cfg7"] = ("cfg7: 16 clients, convolutional classifier of the LeNet shape (28x28x1 -> conv 6 -> conv 16 -> "
                    "120 -> 84 -> 10) fp32, batch 16, s_i=32i+32, 12 rounds")
DEFAULT_WORKLOAD = "cfg5"   # the configuration the HBM-roofline target of the regression kernel is quoted on
MIN_TIMED_S = 2.0           # short passes are repeated inside a step until the timed region is this long


# DRAM bytes (read + write) over algorithmic bytes of one launch of the round kernel, from the
# ncu captures summarised under profiles/ (traffic grows in proportion to the samples of a launch).
# Set an entry to None when its kernel changes after the counters were taken.
TRAFFIC_RATIO = {
    "cfg2": None,   # profiles/lr_block_kernel_cfg2.md predates the kernel's row addressing through the launch plan
    "cfg5": (48.44 / 51.94816, "profiles/lr_tc_kernel_cfg5_512clients.md"),
}


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def row_values(cfg):
    return cfg["dims"][0] * cfg["dims"][0] * cfg["dims"][1] if cfg["model"] == 2 else cfg["dims"][0]


def algorithmic_bytes(cfg, samples, n_tasks):
    """Bytes the local-SGD kernel must move: per sample one row and its label,
    per round-task the start model in and the update sum out."""
    from paper_2112_13935_b200 import workloads
    P = workloads.model_n_params(cfg)
    elem = 2 if cfg["precision"] == 1 else 4
    per_sample = elem * row_values(cfg) + 4
    return samples * per_sample + n_tasks * 8 * P


def algorithmic_flops(cfg, samples):
    """Contraction flops per sample: forward and weight-gradient products of every layer, input-gradient
    products of all but the first (dense layers: 2 flops per weight each; convolutions: per weight and
    output position)."""
    d = cfg["dims"]
    if cfg["model"] == 2:
        side, c_in, c1, c2, f1, f2, ncls = d
        s1 = side - 4
        p1 = s1 // 2
        s2 = p1 - 4
        flat = c2 * (s2 // 2) ** 2
        conv1 = c1 * c_in * 25 * s1 * s1
        conv2 = c2 * c1 * 25 * s2 * s2
        dense = [flat * f1, f1 * f2, f2 * ncls]
        macs = 2 * conv1 + 3 * conv2 + 3 * sum(dense)          # no input gradient for the first convolution
        return 2 * macs * samples
    per_sample = sum(4 * d[l] * d[l + 1] for l in range(len(d) - 1)) + \
        sum(2 * d[l] * d[l + 1] for l in range(1, len(d) - 1))
    return per_sample * samples


def fp32_fma_peak_tflops():
    """Plain fp32 FMA peak from the unit counts and the maximum SM clock:
    148 SMs x 128 fp32 lanes x 2 flops x clock (a register-only FMA loop measured 126 of the
    128 lanes per clock on this part)."""
    mhz = 1965.0
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            mhz = float(json.load(f).get("sm_max_mhz", mhz))
    except Exception:
        pass
    return 148 * 128 * 2 * mhz * 1e6 / 1e12, f"derived: 148 SMs x 128 fp32 lanes x 2 x {mhz:.0f} MHz"


def regression_flops(cfg, samples):
    """Softmax regression, batch 1: logits, model update and update sum are one FMA per
    parameter and sample each (the l2 term adds two more per weight)."""
    from paper_2112_13935_b200 import workloads
    P = workloads.n_params(cfg["dims"])
    per_sample = 2 * (3 + (2 if cfg["l2"] else 0)) * P
    return per_sample * samples


def measured_peak_tflops():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops_sustained"]), "measured, sustained bf16"
    except Exception:
        return 1400.0, "fallback, sustained bf16"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.path = index, None, None

    def __enter__(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None
        return self

    def __exit__(self, *exc):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        try:
            rows = [l.strip().split(", ") for l in open(self.path) if l.strip()]
            os.unlink(self.path)
        except Exception:
            return out
        sm = [float(r[1]) for r in rows if len(r) >= 9]
        if not sm:
            return out
        out["sm_mhz"] = float(np.median(sm))
        out["sm_max_mhz"] = float(rows[0][2])
        out["samples"] = len(sm)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for k, name in enumerate(names):
            if any(len(r) >= 9 and r[5 + k].strip().lower().startswith("active") for r in rows):
                out["reasons"].append(name)
        return out


def oracle_bounded(cfg, data, w0, limit_s):
    """The CPU checker as it stands on a bounded sample of the workload: its schedule (whole), then
    round-tasks in start order until the time limit is reached.  The rate returned is that of a whole
    pass at the sampled speed: all samples / (schedule time + task time scaled from the sampled
    round-tasks to all of them) - the schedule is computed once per pass whatever the sample, so
    dividing the sampled samples by the elapsed time would charge it to a fraction of the work."""
    from oracle import schedule, sim
    t0 = time.perf_counter()
    if cfg.get("topology"):
        events = schedule.simulate_ring(cfg, cfg["n_rounds"])[0]
    else:
        events, _, _ = schedule.simulate(cfg, cfg["n_rounds"])
    t_sched = time.perf_counter() - t0
    order = sorted(events, key=lambda e: (e["t_start"], e["client"]))
    all_samples = sum(e["samples"] for e in events)
    w = np.asarray(w0, dtype=np.float64)
    done_samples, done_tasks = 0, 0
    t1 = time.perf_counter()
    for e in order:
        sim.run_task(cfg, data[e["client"]], e["client"], e["round"], w)
        done_samples += e["samples"]
        done_tasks += 1
        if time.perf_counter() - t1 > limit_s:   # the limit bounds the sampled round-tasks; the schedule is always whole
            break
    t_tasks = time.perf_counter() - t1
    dt = time.perf_counter() - t0
    pass_s = t_sched + t_tasks * all_samples / max(1, done_samples)
    return all_samples / pass_s, done_samples, done_tasks, len(events), dt


def blas_threads(cfg):
    # batch-1 regression is matrix-vector work per sample: one thread does it all
    return 1 if cfg["model"] == 0 and cfg["batch"] == 1 else (os.cpu_count() or 1)


def config_block(cfg, samples, n_events):
    """The `config` object of the JSON line: names the workload, identical for both arms."""
    return {"workload": DESCRIBE[cfg["name"]] + (" [peer-to-peer ring]" if cfg.get("topology") else ""),
            "n_clients": cfg["n_clients"], "rounds": cfg["n_rounds"],
            "network_delay_mean": cfg["network_delay_mean"],
            "max_lag_d": "never wait" if cfg["max_lag_d"] == 0xFFFFFFFF else cfg["max_lag_d"],
            "samples_per_pass": samples, "events_per_pass": n_events}


def run_reference(args, cfg):
    """--impl reference: the CPU checker, timed per step on a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from threadpoolctl import threadpool_limits
    from paper_2112_13935_b200 import workloads
    data = workloads.make_client_data(cfg)
    w0 = workloads.make_start_model(cfg)
    cores = blas_threads(cfg)
    rates, sample = [], ""
    from oracle import schedule as _sched
    if cfg.get("topology"):
        _ev, _, _sum, _ = _sched.simulate_ring(cfg, cfg["n_rounds"])
    else:
        _ev, _sum, _ = _sched.simulate(cfg, cfg["n_rounds"])
    ref_samples, ref_events = _sum["samples_total"], len(_ev)
    with threadpool_limits(limits=cores):
        for step in range(args.warmup + args.steps):
            rate, n_s, n_t, n_e, dt = oracle_bounded(cfg, data, w0, REF_STEP_LIMIT_S)
            if step >= args.warmup:
                rates.append((rate, dt))
            sample = (f"per step: the schedule, then the first {n_t} of {n_e} round-tasks in start order ({n_s} samples); "
                      "value = all samples / (schedule time + task time scaled to all round-tasks)")
    value = float(np.mean([r for r, _ in rates]))   # whole-pass rate at the sampled speed, mean over the steps
    total_t = sum(t for _, t in rates)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": config_block(cfg, ref_samples, ref_events),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def measure_device(cfg, steps, warmup, passes_per_step=None, clock_index=None):
    """Device-timed passes of one workload with its inputs resident in HBM.
    Returns a dict with value (local, before any cross-rank reduction), roofline, stats."""
    import torch
    from paper_2112_13935_b200 import api, workloads
    stream = torch.cuda.current_stream()
    data = workloads.make_client_data(cfg)
    w0 = workloads.make_start_model(cfg)
    R = cfg["n_rounds"]
    dev = [(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()) for x, y in data]
    w0_dev = torch.from_numpy(w0).cuda()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")   # > L2 (126 MB)
    sess = api.Session(cfg, dev, w0_dev)
    plan_ms = None
    t_warm = []
    for _ in range(warmup):
        sess.reset()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        sess.run(R)
        b.record(stream)
        t_warm.append((a, b))
        if plan_ms is None:   # host time of the integer schedule + launch plan; later runs reuse the cached plan
            plan_ms = api.aet_get_stats(sess.h)["plan_ms"]
    torch.cuda.synchronize()
    events, summary = sess.log()
    samples = summary["samples_total"]
    stats = api.aet_get_stats(sess.h)
    launches_per_pass = sum(stats["launches"])
    if passes_per_step is None:
        pass_s = min(a.elapsed_time(b) for a, b in t_warm) / 1e3
        passes_per_step = max(1, int(np.ceil(MIN_TIMED_S / max(pass_s * steps, 1e-9))))
    n_pass = steps * passes_per_step

    # ---- timed region: every pass bracketed by events on the launching stream, L2 flushed before it ----
    from paper_2112_13935_b200 import dist
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(n_pass)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(n_pass)]
    dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(clock_index) if clock_index is not None else None
    if sampler:
        sampler.__enter__()
    for k in range(n_pass):
        flush.fill_(k & 0xFF)                      # evict L2 between timed passes
        sess.reset()
        starts[k].record(stream)
        sess.run(R)
        ends[k].record(stream)
    torch.cuda.synchronize()
    if sampler:
        sampler.__exit__()
    dist.barrier()
    seconds = sum(s.elapsed_time(e) for s, e in zip(starts, ends)) / 1e3

    # ---- per-kernel device time: a second set of passes with events around every launch ----
    api.aet_set_kernel_timing(sess.h, True)
    k_ms = [0.0, 0.0]
    k_pass = min(n_pass, 5)
    for k in range(k_pass):
        flush.fill_(k & 0xFF)
        sess.reset()
        sess.run(R)
        st = api.aet_get_stats(sess.h)
        k_ms[0] += st["kernel_ms"][0]
        k_ms[1] += st["kernel_ms"][1]
    api.aet_set_kernel_timing(sess.h, False)
    sess.close()
    del dev, flush

    n_sgd_launches = stats["launches"][0]
    n_tasks = cfg["n_clients"] * R
    alg_bytes = algorithmic_bytes(cfg, samples, n_tasks)
    sgd_ms = k_ms[0] / k_pass
    achieved = alg_bytes / (sgd_ms * 1e-3) / 1e9
    peak, peak_kind = measured_peak_gbs()
    ratio = TRAFFIC_RATIO.get(cfg["name"])
    traffic = ratio[0] * alg_bytes / n_sgd_launches if ratio and ratio[0] and not cfg.get("_cut") else None
    roof = {"bound": "hbm", "kernel": "local-SGD rounds", "achieved": achieved, "peak": peak,
            "unit": "GB/s", "frac": achieved / peak, "traffic": traffic,
            "traffic_source": ratio[1] if traffic else None, "peak_kind": peak_kind,
            "algorithmic_bytes_per_launch": alg_bytes / n_sgd_launches}
    if cfg["model"] >= 1:
        tf = algorithmic_flops(cfg, samples) / (sgd_ms * 1e-3) / 1e12
        if cfg["precision"] == 1:     # bf16 operands: the dense contraction runs on the tensor cores
            tpeak, tkind = measured_peak_tflops()
            bound = "tensor"
        else:                         # fp32 model: plain FMAs
            tpeak, tkind = fp32_fma_peak_tflops()
            bound = "alu"
        roof = {"bound": bound, "kernel": "local-SGD rounds (MLP)" if cfg["model"] == 1 else "local-SGD rounds (conv)", "achieved": tf, "peak": tpeak,
                "unit": "TFLOP/s", "frac": tf / tpeak, "traffic": None, "peak_kind": tkind,
                "hbm_gbs_algorithmic": achieved}
    else:
        # the batch-1 regression kernel sits on the FMA / HBM ridge: its fp32 FMA rate beside the HBM figure
        apeak, akind = fp32_fma_peak_tflops()
        atf = regression_flops(cfg, samples) / (sgd_ms * 1e-3) / 1e12
        roof.update(alu_tflops=atf, alu_peak=apeak, alu_frac=atf / apeak, alu_peak_kind=akind)
    roof.update(launches_per_step=n_sgd_launches, kernel_ms_per_step=sgd_ms,
                kernel_ms_mode="separate passes with events around every launch: no overlap between a kernel "
                               "and its neighbours, so the sum can exceed the pass it belongs to",
                aggregation_ms_per_step=k_ms[1] / k_pass, algorithmic_bytes_per_step=alg_bytes)
    return dict(samples=samples, seconds=seconds, n_pass=n_pass, passes_per_step=passes_per_step, roof=roof,
                launches_per_pass=launches_per_pass, events=n_tasks, waves=stats["waves"], plan_ms=plan_ms,
                clocks=sampler.summary() if sampler else None, data=data, w0=w0)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(DESCRIBE))
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--clients", type=int, default=0, help="override the workload's client count (cfg5 sweep)")
    ap.add_argument("--rounds", type=int, default=0, help="override the number of rounds (profiling on a smaller case)")
    ap.add_argument("--net-delay", type=float, default=None, help="override the mean network delay (time units)")
    ap.add_argument("--max-lag", type=int, default=None, help="override the checkpoint threshold d (-1 = never wait)")
    ap.add_argument("--topology", default=None, choices=["server", "ring"], help="override the topology of the workload")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--passes-per-step", type=int, default=0, help="0 = enough for a 2 s timed region")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="skip the device-timed passes of the other configurations")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "b200" else args.warmup

    from paper_2112_13935_b200 import workloads
    rank = int(os.environ.get("RANK", "0"))
    over = dict(n_clients=args.clients) if args.clients else {}
    if args.rounds:
        over["n_rounds"] = args.rounds
    if args.net_delay is not None:
        over["network_delay_mean"] = args.net_delay
    if args.max_lag is not None:
        over["max_lag_d"] = workloads.NEVER_WAIT if args.max_lag < 0 else args.max_lag
    if args.topology:
        over["topology"] = 1 if args.topology == "ring" else 0
    cfg = workloads.get_config(args.workload, seed=rank, **over)
    if args.rounds:
        cfg["_cut"] = True
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    from paper_2112_13935_b200 import api, dist
    rank, world, local = dist.init_from_env()
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local)

    m = measure_device(cfg, args.steps, args.warmup, args.passes_per_step or None, clock_index=local)
    data, w0, samples, R = m["data"], m["w0"], m["samples"], cfg["n_rounds"]
    value = dist.job_throughput(samples * m["n_pass"], m["seconds"])
    slowest = dist.max_over_ranks(m["seconds"])

    # ---- end to end through the C ABI from pinned host buffers ----
    pinned = [(torch.from_numpy(x).pin_memory(), torch.from_numpy(y).pin_memory()) for x, y in data]
    w0_pin = torch.from_numpy(w0).pin_memory()
    out_pin = torch.empty(w0.size, dtype=torch.float32).pin_memory()
    h2d = sum(x.numel() * 4 + y.numel() * 4 for x, y in pinned) + w0.size * 4
    d2h = w0.size * 4 + 32 * m["events"]          # the model, and per event the trigger and apply records the log call checks
    e2e_s = []
    for k in range(args.e2e_steps + 1 if args.e2e_steps > 0 else 0):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        h = api.aet_create(cfg)
        api.aet_prepare_rounds(h, R)                   # the schedule and the launch plan, under the copies below
        api.aet_set_global_model(h, w0_pin)
        for c, (x, y) in enumerate(pinned):
            api.aet_load_client_data(h, c, x, y)
        api.aet_run_rounds(h, R)
        api.aet_get_global_model(h, out_pin)
        ev, _ = api.aet_get_event_log(h, raw=True)     # the log with the library's cross-check of the device records
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        api.aet_destroy(h)
        if k > 0:                                      # first one warms allocator and caches
            e2e_s.append(dt)
    e2e_value = dist.job_throughput(samples * len(e2e_s), sum(e2e_s)) if e2e_s else None
    del pinned

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from threadpoolctl import threadpool_limits
        cores = blas_threads(cfg)
        with threadpool_limits(limits=cores):
            rate, n_s, n_t, n_e, dt = oracle_bounded(cfg, data, w0, CPU_LIMIT_S)
        cpu = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": (f"the schedule, then the first {n_t} of {n_e} round-tasks in start order ({n_s} samples, {dt:.1f} s); "
                          "value = all samples / (schedule time + task time scaled to all round-tasks)")}
    del data

    # ---- the other configurations, device-timed for a few passes each (no e2e, no CPU leg) ----
    per_config = []
    if rank == 0 and world == 1 and not args.no_per_config and not args.rounds and not args.clients:
        for name, steps, extra in (("cfg2", 10, {}), ("cfg3", 5, {}), ("cfg4", 3, {}), ("cfg6", 5, {}),
                                   ("cfg6", 5, dict(topology=1)), ("cfg7", 5, {})):
            if name == args.workload and not extra:
                continue
            c2 = workloads.get_config(name, seed=rank, **extra)
            r = measure_device(c2, steps, 3, passes_per_step=1)
            per_config.append({"workload": DESCRIBE[name] + (" [peer-to-peer ring]" if extra.get("topology") else ""), "value": r["samples"] * r["n_pass"] / r["seconds"],
                               "unit": UNIT, "ms_per_step": 1e3 * r["seconds"] / r["n_pass"], "steps": r["n_pass"],
                               "dtype": "bf16" if c2["precision"] == 1 else "f32",
                               "roofline": {k: r["roof"][k] for k in ("bound", "achieved", "peak", "unit", "frac",
                                                                      "peak_kind", "kernel_ms_per_step")}})

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * slowest / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if cfg["precision"] == 1 else "f32",
            "data": "synthetic",
            "config": dict(config_block(cfg, samples, m["events"]), l2="flushed before every timed pass (256 MB fill)",
                           passes_per_step=m["passes_per_step"]),
            "run": {"waves_per_pass": m["waves"], "ms_per_pass": 1e3 * slowest / m["n_pass"],
                    "multi_gpu": "independent replicas, one seed per rank"},
            "clocks": m["clocks"],
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": len(e2e_s), "note": "one pass per e2e step: create, schedule on a library thread under the copies, load from pinned host memory, run, model and event log back"},
            "gpu_launches": m["launches_per_pass"] * m["n_pass"],
            "roofline": m["roof"],
            "cpu_baseline": cpu,
            "per_config": per_config,
            "schedule_and_plan_ms_first_run": m["plan_ms"],
        }
        print(json.dumps(line))
    dist.shutdown()


if __name__ == "__main__":
    main()
