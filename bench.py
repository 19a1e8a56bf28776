#!/usr/bin/env python
"""Benchmark of the fused attention forward pass (BF16, head dim 128) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

A step is one pass of the whole forward path (one `attn_fwd` call) over one batch of synthetic
BF16 Q/K/V resident in HBM.  The default workload is the one the headline metric is quoted on:
non-causal multi-head attention, 16 heads, 32768 tokens as 2 sequences of 16384.  The metric is
TFLOP/s with 4*B*Hq*Sq*Sk*D FLOPs per call (halved when causal).

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank runs an independent
replica of the same workload -- attention rows never cross (batch, head), so nothing is
exchanged -- and the reported value is the sum over ranks divided by the slowest rank's time.

`--impl reference` times the CPU fp64 oracle instead (rank 0 only), on a bounded sample of the
same workload's rows per step.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from workloads import all_workloads, bf16_bits, make_workload_inputs  # noqa: E402

METRIC = "attn_fwd_bf16_d128_tflops"
UNIT = "TFLOP/s"
DEFAULT_WORKLOAD = "mha_noncausal_s16384"
FALLBACK_BF16_TFLOPS = 1590.0  # earlier measurement on this machine, used only without MEASURED_PEAKS.json
NOMINAL_BF16_TFLOPS = 2250.0
REFERENCE_ROWS_PER_STEP = 1024


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--op", default="fwd", choices=["fwd", "merge", "splitkv"],
                    help="fwd: the attention forward (default, the headline metric); merge: the LSE-weighted "
                         "merge of two partial results of the same shape (HBM-bound side kernel); splitkv: "
                         "one query row per sequence against a long key sequence (decoding shape), attn_fwd "
                         "against attn_fwd_splitkv for several numbers of key ranges (HBM-bound)")
    ap.add_argument("--sweep", action="store_true",
                    help="time every sequence-length sweep workload (10 warm-ups, then 10 repetitions of 30 launches: "
                         "mean and standard deviation) and print one JSON line with the per-workload TFLOP/s vector "
                         "and its geometric means; one GPU")
    ap.add_argument("--only", default="", help="--sweep: comma-separated workload-name prefixes to keep")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="target oracle time of the cpu_baseline leg")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--parity-rows", type=int, default=512,
                    help="rows of the timed launches' output that are compared with the CPU oracle when the "
                         "cpu_baseline leg does not run (that leg's rows are all compared); 0 skips the check")
    ap.add_argument("--sustained-seconds", type=float, default=2.0,
                    help="after the timed region, keep launching for this long and report the throughput of the "
                         "last third as `sustained` (the part is power-limited: a short timed region runs at a "
                         "higher clock than a long one); 0 skips it")
    ap.add_argument("--set", action="append", default=[], metavar="NAME=VALUE",
                    help="library option for this run (attn_set_option), e.g. --set kernel=2; repeatable; "
                         "recorded in config.options")
    return ap.parse_args()


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["bf16_tflops"]), float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "measured"
    return FALLBACK_BF16_TFLOPS, 1400.0, "fallback"


class ClockSampler:
    """Samples SM clock, power and clock-event reasons of one GPU through NVML from a thread, about
    every millisecond, with a host time stamp per sample; stop(t0, t1) keeps the samples taken
    inside the timed region only.  Falls back to an nvidia-smi child process (25 ms period, all its
    samples) when the NVML binding is not importable."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    REASON_BITS = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
                   "sw_power_cap": 0x4}

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.file = None
        self.thread = None
        self.samples = []  # (host time, sm MHz, power W, reasons mask)
        self.sm_max = None
        self._stop = False

    def _nvml_handle(self):
        import pynvml
        pynvml.nvmlInit()
        try:
            uuid = str(torch.cuda.get_device_properties(self.gpu_index).uuid)
            return pynvml, pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
        except Exception:
            return pynvml, pynvml.nvmlDeviceGetHandleByIndex(self.gpu_index)

    def _poll(self, pynvml, handle):
        while not self._stop:
            try:
                mhz = pynvml.nvmlDeviceGetClockInfo(handle, pynvml.NVML_CLOCK_SM)
                watts = pynvml.nvmlDeviceGetPowerUsage(handle) / 1000.0
                mask = pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(handle)
                self.samples.append((time.perf_counter(), float(mhz), watts, int(mask)))
            except Exception:
                pass
            time.sleep(0.001)

    def start(self):
        try:
            import threading
            pynvml, handle = self._nvml_handle()
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
            self.thread = threading.Thread(target=self._poll, args=(pynvml, handle), daemon=True)
            self.thread.start()
            return
        except Exception:
            self.thread = None
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "25"],
                stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self, t0=None, t1=None):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.thread is not None:
            self._stop = True
            self.thread.join(timeout=2)
            inside = [x for x in self.samples if (t0 is None or x[0] >= t0) and (t1 is None or x[0] <= t1)]
            if inside:
                mask = 0
                for x in inside:
                    mask |= x[3]
                out.update(sm_mhz=statistics.median(x[1] for x in inside), sm_max_mhz=self.sm_max,
                           reasons=sorted(n for n, bit in self.REASON_BITS.items() if mask & bit),
                           samples=len(inside), power_w_max=max(x[2] for x in inside),
                           sm_mhz_min=min(x[1] for x in inside), source="nvml, samples inside the timed region")
            return out
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, smax, power, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.file.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                smax.append(float(parts[2]))
                power.append(float(parts[3]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        try:
            os.unlink(self.file.name)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), reasons=sorted(reasons),
                       samples=len(sm), power_w_max=max(power), source="nvidia-smi, 25 ms period")
        return out


def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks of the default process group
    (identity when torch.distributed is not initialised).  Works with nccl and gloo."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def whole_job_tflops(flops_per_replica: float, world: int, ms_per_step: float) -> float:
    """Throughput of `world` independent replicas that all finish a step within `ms_per_step`."""
    return world * flops_per_replica / (ms_per_step * 1e-3) / 1e12


TOL_O, TOL_LSE = 2e-2, 1e-3  # max-norm bounds of the correctness check, as in the parity tests


def oracle_sample(w, q, k, v, n_rows, seed):
    """Runs the CPU oracle, as it stands, on `n_rows` seeded rows of the workload and times it.
    Returns (TFLOP/s, seconds, rows int32 [n, 3], O rows fp64 [n, D], LSE fp64 [n], threads)."""
    from oracle import attn_oracle as orc
    rng = np.random.default_rng(seed)  # uniform over (b, hq, i): unbiased under the causal mask
    rows = np.stack([rng.integers(w.B, size=n_rows), rng.integers(w.Hq, size=n_rows),
                     rng.integers(w.Sq, size=n_rows)], axis=1).astype(np.int32)
    qb, kb, vb = bf16_bits(q), bf16_bits(k), bf16_bits(v)
    t0 = time.perf_counter()
    o_ref, lse_ref = orc.attention_rows(qb, kb, vb, w.causal, w.scale, rows)
    dt = time.perf_counter() - t0
    # FLOPs of these rows under the metric's convention: 4 * Sk * D per (row), halved when causal
    flops = len(rows) * 4.0 * w.Sk * w.D * (0.5 if w.causal else 1.0)
    return flops / dt / 1e12, dt, rows, o_ref, lse_ref, orc.default_threads()


def oracle_sample_tflops(w, q, k, v, n_rows, seed):
    """Times the CPU oracle on `n_rows` seeded rows: (TFLOP/s, seconds, rows done, threads)."""
    rate, dt, rows, _, _, cores = oracle_sample(w, q, k, v, n_rows, seed)
    return rate, dt, len(rows), cores


def parity_of_rows(o_host, lse_host, rows, o_ref, lse_ref):
    """The correctness gate of the scoring function (the paper's Section 3.1: a candidate that fails
    the check scores 0): the given rows of the output the TIMED launches left behind against the
    oracle's.  o_host BF16 [B, Sq, Hq, D] and lse_host fp32 [B, Hq, Sq] are CPU tensors."""
    from workloads import bits_to_float64
    o64 = bits_to_float64(bf16_bits(o_host))[rows[:, 0], rows[:, 2], rows[:, 1]]
    l64 = lse_host.numpy().astype(np.float64)[rows[:, 0], rows[:, 1], rows[:, 2]]
    finite = bool(np.isfinite(o64).all() and np.isfinite(l64).all() and np.isfinite(lse_ref).all())
    d_o = float(np.abs(o64 - o_ref).max()) if finite else float("inf")
    d_l = float(np.abs(l64 - lse_ref).max()) if finite else float("inf")
    return {"rows": int(len(rows)), "max_dO": d_o, "max_dLSE": d_l, "tol_dO": TOL_O, "tol_dLSE": TOL_LSE,
            "ok": bool(finite and d_o <= TOL_O and d_l <= TOL_LSE)}


def block_pairs_per_sm(w, sm_count):
    """Pairs of 128 x 128 score blocks per SM under the metric's FLOP convention (8.39 MFLOP per
    block): what `clocks_per_block_pair` divides by.  The two GEMMs of a pair of blocks keep one SM's
    tensor pipe busy for 2048 clocks."""
    return w.flops / (4.0 * 128 * 128 * w.D) / sm_count / 2.0


def run_reference(args, w):
    """The oracle on host cores; each step is a bounded row sample of the workload."""
    rank, world, _ = dist_env()
    if rank != 0:
        return
    from oracle import attn_oracle as orc
    orc.build()
    q, k, v = make_workload_inputs(w)
    for i in range(args.warmup):
        oracle_sample_tflops(w, q, k, v, 64, seed=100 + i)
    times, rows_done = [], 0
    for i in range(args.steps):
        _, dt, n, cores = oracle_sample_tflops(w, q, k, v, REFERENCE_ROWS_PER_STEP, seed=1000 + i)
        times.append(dt)
        rows_done += n
    total = sum(times)
    flops = rows_done * 4.0 * w.Sk * w.D * (0.5 if w.causal else 1.0)
    value = flops / total / 1e12
    sample = f"{REFERENCE_ROWS_PER_STEP} seeded query rows (all keys) of {w.name} per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "Hq": w.Hq, "Hkv": w.Hkv, "Sq": w.Sq, "Sk": w.Sk, "D": w.D,
                   "causal": w.causal, "note": "CPU fp64 oracle on host cores, bounded row sample per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.default_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_ours(args, w):
    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    import paper_2603_24517_b200 as lib
    from paper_2603_24517_b200 import build as lib_build
    lib_build.build()
    lib.load_library()

    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    use_dist = world > 1
    if use_dist:
        import torch.distributed as dist
        dist.init_process_group(backend="nccl", device_id=dev)

    # every rank: an independent replica of the workload (same shapes, rank-specific seed)
    import dataclasses
    w_rank = dataclasses.replace(w, seed=w.seed + 10007 * rank)
    q_h, k_h, v_h = make_workload_inputs(w_rank)
    q, k, v = q_h.to(dev), k_h.to(dev), v_h.to(dev)
    o = torch.empty_like(q)
    lse = torch.empty((w.B, w.Hq, w.Sq), dtype=torch.float32, device=dev)
    scale = w.scale

    def barrier():
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        lib.attn_fwd(q, k, v, o, lse, w.causal, scale)
    barrier()

    # poison the outputs: whatever the timed launches do not write stays NaN for the correctness gate
    o.fill_(float("nan"))
    lse.fill_(float("nan"))
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.15)
    barrier()
    # K steps as up to 10 repetitions (the paper's Section 4.1 protocol: mean and deviation over
    # 10 runs) inside ONE timed region: an event after every repetition, no synchronisation between
    reps = max(1, min(10, args.steps))
    per_rep = [args.steps // reps + (1 if r < args.steps % reps else 0) for r in range(reps)]
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
    t_begin = time.perf_counter()
    ev[0].record()
    for r in range(reps):
        for _ in range(per_rep[r]):
            lib.attn_fwd(q, k, v, o, lse, w.causal, scale)
        ev[r + 1].record()
    barrier()
    t_end = time.perf_counter()
    ms_total = ev[0].elapsed_time(ev[reps])
    rep_ms = [ev[r].elapsed_time(ev[r + 1]) / per_rep[r] for r in range(reps)]
    clocks = sampler.stop(t_begin, t_end) if rank == 0 else None
    # NVML's clock reading lags a region of a fraction of a second; the kernel's own cycle counter
    # over its nanosecond timer gives the clock every timed launch really ran at
    in_kernel = lib.attn_launch_clocks(min(64, args.steps))
    mhz_median = statistics.median(in_kernel) if in_kernel else None
    if clocks is not None and in_kernel:
        clocks["sm_mhz_in_kernel_median"] = round(mhz_median, 1)
        clocks["sm_mhz_in_kernel_min"] = round(min(in_kernel), 1)
        clocks["sm_mhz_in_kernel_max"] = round(max(in_kernel), 1)
        clocks["sm_mhz_last_launch"] = round(in_kernel[0], 1)
        clocks["in_kernel_launches"] = len(in_kernel)
    st, code, detail = lib.attn_last_device_status()
    if st != 0:
        raise SystemExit(f"device status {st} code {code:#x} detail {detail}")
    # the output of the timed launches, for the correctness gate
    unwritten = bool(torch.isnan(o).any().item() or torch.isnan(lse).any().item())  # the whole output
    o_timed, lse_timed = (o.cpu(), lse.cpu()) if rank == 0 else (None, None)

    # sustained regime: the same launch repeated for a few seconds, the last third timed
    sustained = None
    ms_sustained = 0.0
    if args.sustained_seconds > 0:
        ms_guess = ms_total / args.steps
        n_sus = int(min(3000, max(30, args.sustained_seconds * 1e3 / ms_guess)))
        n_tail = max(10, n_sus // 3)
        for _ in range(n_sus - n_tail):
            lib.attn_fwd(q, k, v, o, lse, w.causal, scale)
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        for _ in range(n_tail):
            lib.attn_fwd(q, k, v, o, lse, w.causal, scale)
        s1.record()
        barrier()
        ms_sustained = s0.elapsed_time(s1) / n_tail
        sus_clocks = lib.attn_launch_clocks(min(64, n_tail))
        sustained = {"launches": n_sus, "timed_launches": n_tail,
                     "sm_mhz_in_kernel_median": round(statistics.median(sus_clocks), 1) if sus_clocks else None}

    # end to end through the host-buffer entry point: H2D of Q, K, V and D2H of O, LSE every step
    qp, kp, vp = q_h.pin_memory(), k_h.pin_memory(), v_h.pin_memory()
    op = torch.empty_like(q_h).pin_memory()
    lp = torch.empty((w.B, w.Hq, w.Sq), dtype=torch.float32).pin_memory()
    lib.attn_fwd_host(qp, kp, vp, op, lp, w.causal, scale, device=local)  # warm-up: allocates staging
    barrier()
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record()
    for _ in range(args.e2e_steps):
        lib.attn_fwd_host(qp, kp, vp, op, lp, w.causal, scale, device=local)
    e3.record()
    barrier()
    ms_e2e = e2.elapsed_time(e3)
    h2d = qp.numel() * 2 + kp.numel() * 2 + vp.numel() * 2
    d2h = op.numel() * 2 + lp.numel() * 4
    lib.attn_release_host_staging()

    ms_total, ms_e2e, ms_sustained = max_over_ranks([ms_total, ms_e2e, ms_sustained], device=dev)

    if rank == 0:
        ms_step = ms_total / args.steps
        value = whole_job_tflops(w.flops, world, ms_step)
        e2e_value = whole_job_tflops(w.flops, world, ms_e2e / args.e2e_steps)
        peak_burst, peak_sustained, peak_kind = measured_peaks()
        achieved = w.flops / (ms_step * 1e-3) / 1e12  # one GPU's kernel: one launch per step
        rep_tflops = [w.flops / (m * 1e-3) / 1e12 for m in rep_ms]   # rank 0's replica
        sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
        pairs = block_pairs_per_sm(w, sm_count)
        line = {
            "metric": METRIC, "value": value, "value_std": statistics.pstdev(rep_tflops) * world,
            "repetitions": {"n": reps, "launches_each": per_rep, "tflops": [round(x, 1) for x in rep_tflops],
                            "note": "events inside the one timed region; rank 0's replica"},
            "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "B": w.B, "Hq": w.Hq, "Hkv": w.Hkv, "Sq": w.Sq, "Sk": w.Sk,
                       "D": w.D, "causal": w.causal, "parallelism": f"replicas x{world}",
                       "l2": f"inputs+outputs {w.algorithmic_bytes / 2**20:.0f} MiB exceed the 126 MB L2; no flush",
                       "flops_per_step": w.flops, "options": args.options},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": args.e2e_steps},
            "gpu_launches": args.steps,
            "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak_burst, "unit": UNIT,
                         "frac": achieved / peak_burst, "peak_kind": f"{peak_kind} cuBLAS bf16 burst",
                         "frac_of_sustained": achieved / peak_sustained,
                         "frac_of_nominal_2250": achieved / NOMINAL_BF16_TFLOPS,
                         "traffic": TRAFFIC_BYTES.get(w.name), "algorithmic_bytes": w.algorithmic_bytes},
        }
        if mhz_median is not None:
            # time x clock: SM cycles per pair of 128 x 128 blocks per SM (2048 of them are tensor work);
            # unlike TFLOP/s this does not move with the clock the power limit allows
            line["clocks_per_block_pair"] = round(ms_step * 1e-3 * mhz_median * 1e6 / pairs, 1)
            line["roofline"]["tensor_clocks_per_block_pair"] = 2048
        if sustained is not None:
            sus_value = whole_job_tflops(w.flops, world, ms_sustained)
            sustained.update(value=sus_value, unit=UNIT, ms_per_step=ms_sustained,
                             frac_of_sustained_peak=sus_value / world / peak_sustained)
            if sustained["sm_mhz_in_kernel_median"]:
                sustained["clocks_per_block_pair"] = round(
                    ms_sustained * 1e-3 * sustained["sm_mhz_in_kernel_median"] * 1e6 / pairs, 1)
            line["sustained"] = sustained
        parity = None
        if not args.no_cpu_baseline and world == 1:
            from oracle import attn_oracle as orc
            orc.build()
            rate, dt, n, cores = oracle_sample_tflops(w, q_h, k_h, v_h, 256, seed=1)
            n_rows = int(max(256, min(200000, args.cpu_seconds * n / dt)))
            rate, dt, rows, o_ref, lse_ref, cores = oracle_sample(w, q_h, k_h, v_h, n_rows, seed=2)
            line["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": f"{len(rows)} seeded query rows (all keys) of {w.name}, {dt:.1f} s"}
            parity = parity_of_rows(o_timed, lse_timed, rows, o_ref, lse_ref)
        elif args.parity_rows > 0:
            from oracle import attn_oracle as orc
            orc.build()
            _, _, rows, o_ref, lse_ref, _ = oracle_sample(w_rank, q_h, k_h, v_h, args.parity_rows, seed=2)
            parity = parity_of_rows(o_timed, lse_timed, rows, o_ref, lse_ref)
        if parity is not None:
            parity["unwritten_elements"] = unwritten
            parity["ok"] = bool(parity["ok"] and not unwritten)
            line["parity"] = parity
            if not parity["ok"]:   # a wrong result has no throughput
                line["unchecked_value"] = line["value"]
                line["value"] = 0.0
                line["roofline"]["frac"] = 0.0
        print(json.dumps(line), flush=True)
    if use_dist:
        dist.destroy_process_group()


def run_merge(args, w):
    """attn_merge on two partial results shaped like the workload's O / LSE: GB/s against the
    measured HBM copy bandwidth.  One GPU."""
    import paper_2603_24517_b200 as lib
    from paper_2603_24517_b200 import build as lib_build
    lib_build.build()
    lib.load_library()
    dev = torch.device("cuda", 0)
    g = torch.Generator(device=dev)
    g.manual_seed(w.seed)
    shape = (w.B, w.Sq, w.Hq, w.D)
    o1 = torch.randn(shape, device=dev, generator=g).to(torch.bfloat16)
    o2 = torch.randn(shape, device=dev, generator=g).to(torch.bfloat16)
    l1 = torch.randn((w.B, w.Hq, w.Sq), device=dev, generator=g)
    l2 = torch.randn((w.B, w.Hq, w.Sq), device=dev, generator=g)
    o = torch.empty_like(o1)
    lse = torch.empty_like(l1)
    rows = w.B * w.Sq * w.Hq
    algorithmic = rows * (3 * w.D * 2 + 3 * 4)  # read O1, O2, LSE1, LSE2; write O, LSE
    for _ in range(max(3, args.warmup)):
        lib.attn_merge(o1, l1, o2, l2, o, lse)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        lib.attn_merge(o1, l1, o2, l2, o, lse)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    gbs = algorithmic / (ms * 1e-3) / 1e9
    peak = 6650.0
    kind = "fallback"
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            peak = float(json.load(f)["hbm_gbs"])
        kind = "measured"
    print(json.dumps({
        "metric": "attn_merge_gbs", "value": gbs, "unit": "GB/s", "n_gpus": 1, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True, "dtype": "f32",
        "data": "synthetic", "gpu_launches": args.steps,
        "config": {"workload": f"merge of two partial results shaped like {w.name}", "rows": rows,
                   "l2": f"{algorithmic / 2**20:.0f} MiB per launch exceed the 126 MB L2; no flush"},
        "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                     "peak_kind": f"{kind} copy bandwidth", "traffic": 381.4e6 if w.name == DEFAULT_WORKLOAD else None,
                     "algorithmic_bytes": algorithmic},
    }), flush=True)


def run_sweep(args):
    """The evaluation protocol of the paper's Section 4.1 on every sweep workload: TFLOP/s per
    configuration as mean and standard deviation over 10 repetitions, and the geometric mean per
    family -- the score vector of Section 3.1, correctness gate included: after its timed launches
    a workload's output is scanned for unwritten elements and `--parity-rows` seeded rows are
    compared with the CPU oracle; an entry that fails scores 0.  Each repetition also reports SM
    cycles per pair of 128 x 128 blocks per SM (time x the clock its launches ran at), which does
    not move with the power-limited clock the way TFLOP/s does."""
    import math
    import paper_2603_24517_b200 as lib
    from paper_2603_24517_b200 import build as lib_build
    lib_build.build()
    lib.load_library()
    if args.parity_rows > 0:
        from oracle import attn_oracle as orc
        orc.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
    reps, launches, warm = 10, 30, 10
    sampler = ClockSampler(0)
    sampler.start()
    entries = {}
    for name, w in all_workloads().items():
        if not ((name.startswith(("mha_", "gqa4_", "gqa8_")) and "_s" in name) or name == "long_causal_peaked"):
            continue
        if args.only and not any(name.startswith(pre) for pre in args.only.split(",")):
            continue
        q_h, k_h, v_h = make_workload_inputs(w)
        q, k, v = q_h.to(dev), k_h.to(dev), v_h.to(dev)
        o = torch.empty_like(q)
        lse = torch.empty((w.B, w.Hq, w.Sq), dtype=torch.float32, device=dev)
        for _ in range(warm):
            lib.attn_fwd(q, k, v, o, lse, w.causal, w.scale)
        o.fill_(float("nan"))
        lse.fill_(float("nan"))
        torch.cuda.synchronize()
        pairs = block_pairs_per_sm(w, sm_count)
        rates, cycles, mhzs = [], [], []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(launches):
                lib.attn_fwd(q, k, v, o, lse, w.causal, w.scale)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / launches
            rates.append(w.flops / (ms * 1e-3) / 1e12)
            mhz = statistics.median(lib.attn_launch_clocks(launches))
            mhzs.append(mhz)
            cycles.append(ms * 1e-3 * mhz * 1e6 / pairs)
        st, code, detail = lib.attn_last_device_status()
        if st != 0:
            raise SystemExit(f"{name}: device status {st} code {code:#x} detail {detail}")
        entry = {"tflops": statistics.mean(rates), "std": statistics.pstdev(rates),
                 "clocks_per_block_pair": statistics.mean(cycles), "clocks_std": statistics.pstdev(cycles),
                 "sm_mhz": statistics.mean(mhzs),
                 "B": w.B, "Hq": w.Hq, "Hkv": w.Hkv, "S": w.Sq, "causal": w.causal}
        if args.parity_rows > 0:
            unwritten = bool(torch.isnan(o).any().item() or torch.isnan(lse).any().item())
            _, _, rows, o_ref, lse_ref, _ = oracle_sample(w, q_h, k_h, v_h, args.parity_rows, seed=w.seed)
            par = parity_of_rows(o.cpu(), lse.cpu(), rows, o_ref, lse_ref)
            par["unwritten_elements"] = unwritten
            par["ok"] = bool(par["ok"] and not unwritten)
            entry["parity"] = par
            if not par["ok"]:
                entry["unchecked_tflops"] = entry["tflops"]
                entry["tflops"] = 0.0
        entries[name] = entry
        del q, k, v, o, lse
    clocks = sampler.stop()

    def geomean(prefix):
        xs = [e["tflops"] for n, e in entries.items() if n.startswith(prefix)]
        if not xs or min(xs) <= 0.0:
            return 0.0 if xs else None
        return math.exp(sum(math.log(x) for x in xs) / len(xs))

    # long_causal_peaked (one 65536-token sequence, scores four times as wide) is listed but belongs to no family
    families = ["mha_noncausal", "mha_causal", "gqa4_noncausal", "gqa4_causal", "gqa8_noncausal", "gqa8_causal"]
    print(json.dumps({
        "metric": METRIC + "_sweep", "unit": UNIT, "n_gpus": 1, "dtype": "bf16", "data": "synthetic",
        "protocol": {"warmup_launches": warm, "launches_per_repetition": launches, "repetitions": reps,
                     "parity_rows": args.parity_rows},
        "options": args.options,
        "geomean": {f: geomean(f) for f in families}, "workloads": entries, "clocks": clocks,
        "gpu_launches": len(entries) * (warm + reps * launches),
    }), flush=True)


def run_splitkv(args):
    """Decoding shape: B = 4 sequences, 32 query heads on 8 KV heads, ONE query row each, 32768 keys.
    The K/V tensors (537 MB) must be read once: the path is HBM-bound, and a single launch has only
    64 work items for 148 SMs.  Times attn_fwd and attn_fwd_splitkv; GB/s = K and V bytes / time."""
    import paper_2603_24517_b200 as lib
    from paper_2603_24517_b200 import build as lib_build
    lib_build.build()
    lib.load_library()
    dev = torch.device("cuda", 0)
    B, Hq, Hkv, Sq, Sk, D = 4, 32, 8, 1, 32768, 128
    g = torch.Generator(device=dev)
    g.manual_seed(4242)
    q = torch.randn((B, Sq, Hq, D), device=dev, generator=g).to(torch.bfloat16)
    k = torch.randn((B, Sk, Hkv, D), device=dev, generator=g).to(torch.bfloat16)
    v = torch.randn((B, Sk, Hkv, D), device=dev, generator=g).to(torch.bfloat16)
    o = torch.empty_like(q)
    lse = torch.empty((B, Hq, Sq), dtype=torch.float32, device=dev)
    scale = 1.0 / 128 ** 0.5
    kv_bytes = 2 * k.numel() * 2
    results = {}
    for n in (1, 2, 4, 8, 16, 32):
        ws = torch.empty(max(16, lib.attn_splitkv_workspace_bytes(B, Hq, Sq, D, n)), dtype=torch.uint8, device=dev)
        for _ in range(max(3, args.warmup)):
            lib.attn_fwd_splitkv(q, k, v, o, lse, False, scale, n, workspace=ws)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            lib.attn_fwd_splitkv(q, k, v, o, lse, False, scale, n, workspace=ws)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / args.steps
        results[n] = {"ms": ms, "gbs": kv_bytes / (ms * 1e-3) / 1e9}
    best = max(results, key=lambda n: results[n]["gbs"])
    # a chunk of a long context: 512 query rows against 65536 keys, 16 heads (tensor-bound, but only
    # 32 work items in one launch)
    Bc, Hc, Sqc, Skc = 1, 16, 512, 65536
    qc = torch.randn((Bc, Sqc, Hc, D), device=dev, generator=g).to(torch.bfloat16)
    kc = torch.randn((Bc, Skc, Hc, D), device=dev, generator=g).to(torch.bfloat16)
    vc = torch.randn((Bc, Skc, Hc, D), device=dev, generator=g).to(torch.bfloat16)
    oc = torch.empty_like(qc)
    lc = torch.empty((Bc, Hc, Sqc), dtype=torch.float32, device=dev)
    chunk_flops = 4.0 * Bc * Hc * Sqc * Skc * D
    chunk = {}
    for n in (1, 2, 4, 8):
        ws = torch.empty(max(16, lib.attn_splitkv_workspace_bytes(Bc, Hc, Sqc, D, n)), dtype=torch.uint8, device=dev)
        for _ in range(max(3, args.warmup)):
            lib.attn_fwd_splitkv(qc, kc, vc, oc, lc, False, scale, n, workspace=ws)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            lib.attn_fwd_splitkv(qc, kc, vc, oc, lc, False, scale, n, workspace=ws)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / args.steps
        chunk[n] = {"ms": ms, "tflops": chunk_flops / (ms * 1e-3) / 1e12}
    peak, kind = 6650.0, "fallback"
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            peak = float(json.load(f)["hbm_gbs"])
        kind = "measured"
    print(json.dumps({
        "metric": "attn_decode_kv_gbs", "value": results[best]["gbs"], "unit": "GB/s", "n_gpus": 1,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": results[best]["ms"],
        "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"decode B={B} Hq={Hq} Hkv={Hkv} Sq={Sq} Sk={Sk} D={D} non-causal", "best_n_splits": best,
                   "l2": f"K and V ({kv_bytes / 2**20:.0f} MiB) exceed the 126 MB L2; no flush"},
        "by_n_splits": results,
        "context_chunk": {"workload": f"B={Bc} H={Hc} Sq={Sqc} Sk={Skc} D={D} non-causal", "by_n_splits": chunk},
        "roofline": {"bound": "hbm", "achieved": results[best]["gbs"], "peak": peak, "unit": "GB/s",
                     "frac": results[best]["gbs"] / peak, "peak_kind": f"{kind} copy bandwidth", "traffic": None,
                     "algorithmic_bytes": kv_bytes},
    }), flush=True)


# dram__bytes_read.sum + dram__bytes_write.sum per launch of attn_fwd_kernel from the ncu capture
# summarised in profiles/attn_fwd_kernel_mha_noncausal_s16384_launches.md (403.3-404.5 MB read + 114.7-118.1 MB written, two launches).
TRAFFIC_BYTES: dict[str, float | None] = {"mha_noncausal_s16384": 521.3e6}


def apply_options(args):
    """Sets the library options given with --set (not for the reference arm, which loads no library)."""
    args.options = {}
    for item in args.set:
        name, _, value = item.partition("=")
        args.options[name] = int(value)
    if args.options and args.impl != "reference":
        import paper_2603_24517_b200 as lib
        for name, value in args.options.items():
            lib.attn_set_option(name, value)


def main():
    args = parse_args()
    apply_options(args)
    if args.sweep:
        run_sweep(args)
        return
    workloads = all_workloads()
    if args.workload not in workloads:
        raise SystemExit(f"unknown workload {args.workload}; choose from {sorted(workloads)}")
    w = workloads[args.workload]
    if args.op == "splitkv":
        run_splitkv(args)
    elif args.op == "merge":
        run_merge(args, w)
    elif args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
