#!/usr/bin/env python
"""Benchmark of the CLP decode-step attention (one step = one plt_decode_attn_run over the whole batch).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload I]

Prints ONE JSON line. Default workload: bf16 decode batch B=64, L=2, Hq=32, Hkv=8, d=128, N=4096, w=64
(the configuration the headline metric is quoted on). Without --workload, a one-GPU run then also times the other
three bf16 workloads and the E4M3-cache form of all four for --suite-steps steps each and reports them under
"workloads", each with its own clock record. Every timed region alternates between two copies of the inputs at
different addresses, so that no step can find the previous step's lines in L2.
Under torchrun (N > 1) every rank runs an
independent replica of the workload on its own GPU (no collective in the data path; weak scaling).
`--impl reference` times the fp64 CPU oracle on the host cores instead (rank 0 only).
Other legs: `--kv e4m3` stores the caches as E4M3 codes, `--prestep` times plt_decode_attn_step (pre-step kernel +
attention), `--ablation` adds the L loops as sequential single-loop calls, `--path` / `--loops` / `--hpc` / `--kw` /
`--stages` / `--cps` / `--rw` / `--ks` select the kernel path, an overridden L and launch variants.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

import numpy as np

METRIC = "clp_decode_attn_steps_per_s"
UNIT = "steps/s"
FALLBACK_HBM_GBS = 6650.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=None,
                    help="index into the five workloads; default: 1 (the headline) followed by the suite of the others")
    ap.add_argument("--suite-steps", type=int, default=300, help="timed steps per entry of the \"workloads\" list")
    ap.add_argument("--no-suite", action="store_true", help="headline workload only")
    ap.add_argument("--copies", type=int, default=2, choices=[1, 2],
                    help="copies of the inputs the timed steps alternate between (1: for profiler captures, which "
                         "save and restore device memory per pass and flush the caches themselves)")
    ap.add_argument("--hpc", type=int, default=0)
    ap.add_argument("--kw", type=int, default=0)
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--cps", type=int, default=0)
    ap.add_argument("--rw", type=int, default=0, help="warps that split the packed rows of a KV head (0 = automatic)")
    ap.add_argument("--ks", type=int, default=0, help="16-key slices per warp and tile (0 = automatic)")
    ap.add_argument("--loops", type=int, default=0, help="override the workload's number of loops L (for the traffic-vs-L sweep)")
    ap.add_argument("--path", type=int, default=0, help="kernel path: 0 automatic, 1 warp-level mma, 2 tcgen05")
    ap.add_argument("--kv", default="", choices=["", "e4m3"],
                    help="store the shared cache and the windows as E4M3 codes with per-KV-head scales (q and out stay bf16)")
    ap.add_argument("--prestep", action="store_true",
                    help="time plt_decode_attn_step: the pre-step kernel (cache append, window ring update, gate linear) "
                         "ahead of the attention, three launches per step")
    ap.add_argument("--ablation", action="store_true",
                    help="also time the same queries as L sequential single-loop calls, each scanning the shared cache "
                         "again (the vanilla loop order of Table 1), and report the ratio")
    ap.add_argument("--seq", action="store_true",
                    help="time the sequence-shaped attention (plt_seq_attn_run: prefill / training-forward) instead and "
                         "print its line: TFLOP/s over the key sets the definition names, against the measured bf16 peak")
    ap.add_argument("--seq-batch", type=int, default=4)
    ap.add_argument("--seq-len", type=int, default=5000)
    ap.add_argument("--seq-loops", type=int, default=2)
    ap.add_argument("--seq-steps", type=int, default=20)
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg")
    ap.add_argument("--cpu-seconds", type=float, default=20.0, help="CPU work budget of the oracle leg (core-seconds)")
    return ap.parse_args()


def workload_config(p, extra=None):
    from paper_2510_24824_b200.inputs import algorithmic_bytes
    by = algorithmic_bytes(p)
    cfg = {
        "workload": p.name, "B": p.B, "L": p.L, "Hq": p.Hq, "Hkv": p.Hkv, "d": p.d, "w": p.w,
        "seq_len_min": int(p.seq_lens.min()), "seq_len_max": int(p.seq_lens.max()),
        "sum_seq_len": int(p.seq_lens.sum()), "page_size": p.page_size,
        "algorithmic_bytes_per_step": by["total"],
        "l2": f"inputs {by['total'] / 1e6:.0f} MB per step exceed the 126 MB L2, and consecutive steps alternate between "
              "two copies of the inputs at different addresses; no flush",
    }
    if extra:
        cfg.update(extra)
    return cfg, by


def peak_hbm():
    f = ROOT / "MEASURED_PEAKS.json"
    if f.exists():
        try:
            return float(json.loads(f.read_text())["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback (6650 GB/s, earlier measurement on this pool)"


def recorded_traffic(name: str, kernel: str):
    """DRAM bytes per launch of the main kernel from the committed ncu capture of this workload and kernel, or None."""
    f = ROOT / "profiles" / "main_kernel_dram_traffic.json"
    if f.exists():
        try:
            entry = json.loads(f.read_text()).get(name, {})
            return entry.get("dram_bytes_per_launch") if entry.get("kernel") == kernel else None
        except Exception:
            return None
    return None


class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _poll(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake_slowdown",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._poll, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def replica_spec(index: int, rank: int, loops: int = 0, kv: str = "") -> dict:
    """Workload of one replica: every rank streams its own data (seed offset by rank), same shapes."""
    from paper_2510_24824_b200.inputs import workload
    spec = workload(index)
    spec["seed"] = spec["seed"] + 1000 * rank
    if loops > 0:
        spec["L"] = loops
        spec["name"] = f"{spec['name']}_L{loops}"
    if kv:
        spec["kv_dtype"] = kv
        spec["name"] = f"{spec['name']}_{kv}"
    return spec


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Slowest rank's time: all-reduce MAX over the default process group (identity for one rank)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_steps_per_s(world: int, ms_per_step: float) -> float:
    """Whole-job throughput of `world` independent replicas that each did one step per ms_per_step."""
    return world * 1e3 / ms_per_step


def physical_gpu_index(local_index: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


def time_oracle(p, cpu_seconds: float):
    """Times the fp64 oracle as it stands on a bounded sample of output rows. Returns (steps/s, dict)."""
    import oracle
    cores = oracle.threads()
    total_rows = p.B * p.L * p.Hq
    rng = np.random.default_rng(12345)
    all_rows = np.stack(np.meshgrid(np.arange(p.B), np.arange(p.L), np.arange(p.Hq), indexing="ij"), -1).reshape(-1, 3)
    probe = all_rows[rng.choice(total_rows, size=min(total_rows, 8 * cores), replace=False)]
    t0 = time.perf_counter()
    oracle.decode_attn_rows(p, probe)
    t_probe = time.perf_counter() - t0
    per_row = t_probe / len(probe)  # wall seconds per row with all cores busy
    n = int(min(total_rows, max(len(probe), cpu_seconds / cores / max(per_row, 1e-9))))
    rows = all_rows if n >= total_rows else all_rows[rng.choice(total_rows, size=n, replace=False)]
    # A workload the oracle finishes in well under the budget is repeated whole, so that the sample is
    # about cpu_seconds core-seconds of work either way.
    reps = 1
    if len(rows) == total_rows:
        reps = int(max(1, min(50, round(cpu_seconds / cores / max(per_row * total_rows, 1e-9)))))
    t0 = time.perf_counter()
    for _ in range(reps):
        oracle.decode_attn_rows(p, rows)
    t = time.perf_counter() - t0
    step_seconds = t / reps * total_rows / len(rows)
    sample = (f"{len(rows)} of {total_rows} output rows (b, loop, head) of the same workload, drawn uniformly"
              if len(rows) < total_rows else f"all {total_rows} output rows of the workload, {reps} full step(s)")
    return 1.0 / step_seconds, {"cores": cores, "kind": "oracle", "sample": sample, "sample_seconds": t}


def run_reference(args, rank: int):
    """The reference arm: the CPU oracle, as it stands, on this machine's host cores."""
    if rank != 0:
        return
    from paper_2510_24824_b200.inputs import make_problem, workload
    p = make_problem(workload(args.workload))
    cfg, by = workload_config(p)
    import oracle
    cores = oracle.threads()
    total_rows = p.B * p.L * p.Hq
    all_rows = np.stack(np.meshgrid(np.arange(p.B), np.arange(p.L), np.arange(p.Hq), indexing="ij"), -1).reshape(-1, 3)
    rng = np.random.default_rng(54321)
    # Size the per-step sample so that warm-up + timed steps end within about two minutes.
    probe = all_rows[rng.choice(total_rows, size=min(total_rows, 8 * cores), replace=False)]
    t0 = time.perf_counter()
    oracle.decode_attn_rows(p, probe)
    per_row = (time.perf_counter() - t0) / len(probe)
    budget = 120.0 / max(args.steps + args.warmup, 1)
    n = int(min(total_rows, max(cores, budget / max(per_row, 1e-9))))
    rows = all_rows if n >= total_rows else all_rows[rng.choice(total_rows, size=n, replace=False)]
    for _ in range(args.warmup):
        oracle.decode_attn_rows(p, rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.decode_attn_rows(p, rows)
    t = (time.perf_counter() - t0) / max(args.steps, 1)
    step_seconds = t * total_rows / len(rows)
    value = 1.0 / step_seconds
    sample = f"each step = {len(rows)} of {total_rows} output rows of the workload; time scaled to all rows"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_seconds * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": cfg,
        "loop_queries_per_s": value * p.B * p.L,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


class Replica:
    """One copy of a workload on the device with a handle of its own. A timed region alternates between two of them
    (same values, different addresses), so that a step never finds the lines of the step before it in L2."""

    def __init__(self, p, dev, local_rank, tuning, src=None):
        import torch
        from paper_2510_24824_b200.runner import DecodeAttn, DeviceProblem
        if src is None:
            self.dp = DeviceProblem(p, dev)
        else:                      # second copy: device-side clones of the first one's tensors
            self.dp = DeviceProblem.__new__(DeviceProblem)
            self.dp.problem, self.dp.device = p, dev
            for f in DeviceProblem.FIELDS:
                t = getattr(src.dp, f)
                setattr(self.dp, f, None if t is None else t.clone())
            self.dp.out = torch.empty_like(src.dp.out)
        self.op = DecodeAttn(p, device_index=local_rank, **tuning)
        self.args = self.dp.args()

    def close(self):
        self.op.close()


def time_steps(step_fns, steps, sampler, barrier):
    """K steps, alternating over step_fns, between two events on the current stream. Returns total milliseconds."""
    import torch
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    with sampler:
        ev0.record()
        for i in range(steps):
            step_fns[i & 1]()
        ev1.record()
        torch.cuda.synchronize()
    barrier()
    return ev0.elapsed_time(ev1)


def time_main_kernel(reps, step_fns, n_prof):
    """The same steps with an event pair around the main kernel of each (the library records them). Mean milliseconds."""
    import torch
    from paper_2510_24824_b200 import binding as B
    raw = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_prof)]
    for a, b in raw:
        a.record()  # materialise the underlying cudaEvent_t handles
        b.record()
    torch.cuda.synchronize()
    for i, (a, b) in enumerate(raw):
        B.plt_decode_attn_set_profile_events(reps[i & 1].op.handle, a.cuda_event, b.cuda_event)
        step_fns[i & 1]()
    torch.cuda.synchronize()
    for r in set(reps):
        B.plt_decode_attn_set_profile_events(r.op.handle, None, None)
    return float(np.mean([a.elapsed_time(b) for a, b in raw]))


def main_kernel_bytes(by):
    return by["shared_kv"] + by["window_kv"] + by["q_o"] // 2 + by["index"]


def peak_tflops():
    f = ROOT / "MEASURED_PEAKS.json"
    if f.exists():
        try:
            return float(json.loads(f.read_text())["bf16_tflops_sustained"]), "measured (MEASURED_PEAKS.json bf16_tflops_sustained)"
        except Exception:
            pass
    return 1400.0, "fallback (1.4 PFLOP/s sustained, earlier measurement on this pool)"


def seq_entry(batch, loops, n, dev, local_rank, steps, seed=0):
    """The sequence-shaped attention on the paper's serving shapes (prefill n, GQA 32/8, d = 128, w = 64): TFLOP/s."""
    import torch
    from paper_2510_24824_b200.inputs import make_seq_problem, seq_attn_flops
    from paper_2510_24824_b200.runner import SeqAttn
    p = make_seq_problem(B=batch, L=loops, T=n, Hq=32, Hkv=8, d=128, w=64, seed=seed, name=f"seq_B{batch}_L{loops}_n{n}")
    flops = seq_attn_flops(p)
    op = SeqAttn(p, dev, local_rank)
    for _ in range(3):
        op.run()
    torch.cuda.synchronize()
    assert op.check() == 0, "device status not clean after warm-up"
    sampler = ClockSampler(physical_gpu_index(local_rank))
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with sampler:
        ev0.record()
        for _ in range(steps):
            op.run()
        ev1.record()
        torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / steps
    peak, src = peak_tflops()
    tf = flops / (ms * 1e-3) / 1e12
    entry = {
        "workload": p.name, "B": batch, "L": loops, "n": n, "Hq": 32, "Hkv": 8, "d": 128, "w": 64, "steps": steps,
        "ms_per_call": ms, "algorithmic_flops_per_call": flops, "tflops": tf, "tokens_per_s": batch * n / (ms * 1e-3),
        "roofline": {"bound": "tensor", "kernel": "plt_seq_attn_kernel", "achieved": tf, "peak": peak, "unit": "TFLOP/s",
                     "frac": tf / peak, "peak_source": src,
                     "note": "flops of the two products over visible keys only (masked halves of diagonal tiles not counted)"},
        "inputs_bytes": int(sum(getattr(op, f).numel() * 2 for f in SeqAttn.FIELDS)),
        "clocks": sampler.summary(),
    }
    op.close()
    del op
    torch.cuda.empty_cache()
    return entry


def suite_entry(index, kv, dev, local_rank, steps, base=None):
    """One entry of the "workloads" list: a workload timed for `steps` steps with its own clock record."""
    import torch
    from paper_2510_24824_b200 import binding as B
    from paper_2510_24824_b200.inputs import algorithmic_bytes, make_problem, quantize_kv_e4m3, workload
    if base is None:
        base = make_problem(workload(index))
    p = quantize_kv_e4m3(base).with_(name=base.name + "_e4m3") if kv else base
    by = algorithmic_bytes(p)
    a = Replica(p, dev, local_rank, {})
    b = Replica(p, dev, local_rank, {}, src=a)
    reps = [a, b]
    stream = torch.cuda.current_stream().cuda_stream
    fns = [lambda r=r: B.plt_decode_attn_run(r.op.handle, r.args, stream) for r in reps]
    for i in range(10):
        fns[i & 1]()
    torch.cuda.synchronize()
    assert a.op.check(stream) == 0 and b.op.check(stream) == 0, "device status not clean after warm-up"
    sampler = ClockSampler(physical_gpu_index(local_rank))
    ms = time_steps(fns, steps, sampler, torch.cuda.synchronize) / steps
    main_ms = time_main_kernel(reps, fns, min(steps, 100))
    peak, _ = peak_hbm()
    gbs = by["total"] / (ms * 1e-3) / 1e9
    main_gbs = main_kernel_bytes(by) / (main_ms * 1e-3) / 1e9
    entry = {
        "workload": p.name, "kv": kv or "bf16", "steps": steps, "ms_per_step": ms, "steps_per_s": 1e3 / ms,
        "loop_queries_per_s": 1e3 / ms * p.B * p.L, "algorithmic_bytes_per_step": by["total"],
        "hbm_gbs_whole_step": gbs, "hbm_frac_of_8tbs": gbs / 8000.0, "hbm_frac_of_measured": gbs / peak,
        "main_kernel": {"avg_launch_ms": main_ms, "achieved_gbs": main_gbs, "frac_of_measured": main_gbs / peak},
        "launch": a.op.info, "clocks": sampler.summary(),
    }
    for r in reps:
        r.close()
    del a, b, reps
    torch.cuda.empty_cache()
    return entry, base


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    suite = args.workload is None and not args.no_suite and world == 1 and not (args.kv or args.loops or args.prestep)
    if args.workload is None:
        args.workload = 1
    if args.impl == "reference":
        run_reference(args, rank)
        return

    from paper_2510_24824_b200 import build as lib_build
    if not lib_build.LIB.exists():   # fresh checkout: the library is a build product (rank 0 compiles, the others wait)
        if local_rank == 0:
            lib_build.build()
        else:
            for _ in range(1800):
                if lib_build.LIB.exists():
                    break
                time.sleep(1.0)
    import torch
    import torch.distributed as dist
    from paper_2510_24824_b200 import binding as B
    from paper_2510_24824_b200.inputs import make_problem, workload
    from paper_2510_24824_b200.runner import DecodeAttn, DeviceProblem

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU implementation")
    B.load_library()  # fails loudly when the extension has not been built
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    if args.seq:
        if rank == 0:
            e = seq_entry(args.seq_batch, args.seq_loops, args.seq_len, dev, local_rank, args.seq_steps)
            line = {"metric": "plt_seq_attn_tflops", "value": e["tflops"], "unit": "TFLOP/s", "n_gpus": 1, "steps": args.seq_steps,
                    "warmup": 3, "ms_per_step": e["ms_per_call"], "higher_is_better": True, "scaling": "weak",
                    "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": {"workload": e["workload"]},
                    "gpu_launches": args.seq_steps, **e}
            print(json.dumps(line), flush=True)
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    p = make_problem(replica_spec(args.workload, rank, args.loops, args.kv))
    tuning = dict(heads_per_cta=args.hpc, key_slices=args.kw, stages=args.stages, ctas_per_sm=args.cps,
                  kernel_path=args.path, row_warps=args.rw, slices_per_warp=args.ks)
    reps = [Replica(p, dev, local_rank, tuning)]
    reps.append(Replica(p, dev, local_rank, tuning, src=reps[0]) if args.copies == 2 else reps[0])
    op, dp = reps[0].op, reps[0].dp
    stream = torch.cuda.current_stream().cuda_stream
    cfg, by = workload_config(p)
    if args.copies == 1:
        cfg["l2"] = f"inputs {by['total'] / 1e6:.0f} MB per step exceed the 126 MB L2; one copy of the inputs, no flush"

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    launches_per_step = int(op.info["kernels_per_run"])
    step_args = [None, None]
    if args.prestep:
        # Synthetic rows of this step: the same K/V rows and gate weights every step (the lengths do not advance, so
        # the same cache positions are rewritten: a timing stand-in for consecutive decode steps).
        from paper_2510_24824_b200.runner import to_torch
        from paper_2510_24824_b200.inputs import f32_to_bf16_bits
        rng = np.random.default_rng(1000 + rank)
        rows = [rng.standard_normal((p.B, p.L, p.Hkv, p.d)).astype(np.float32) for _ in range(2)]
        if p.dtype == "bf16":
            rows = [f32_to_bf16_bits(x) for x in rows]
        k_new, v_new = (to_torch(x, p.dtype, dev) for x in rows)
        w_gate = to_torch((rng.standard_normal((p.Hq, p.d)) / np.sqrt(p.d)).astype(np.float32), "", dev)
        b_gate = to_torch(rng.standard_normal(p.Hq).astype(np.float32), "", dev)
        step_args = [B.make_step_args(k_new, v_new, w_gate, b_gate, r.dp.gate_logits if p.L > 1 else None) for r in reps]
        launches_per_step += 1
        cfg["prestep"] = "plt_decode_attn_step: pre-step kernel + attention"

    def make_step(r, st):
        if args.prestep:
            return lambda: B.plt_decode_attn_step(r.op.handle, r.args, st, stream)
        return lambda: B.plt_decode_attn_run(r.op.handle, r.args, stream)

    step_fns = [make_step(r, st) for r, st in zip(reps, step_args)]

    for i in range(max(args.warmup, 3) + 1):
        step_fns[i & 1]()
    barrier()
    assert all(r.op.check(stream) == 0 for r in reps), "device status not clean after warm-up"

    # ---- timed region 1: K whole steps, device time between two events --------------------------------
    sampler = ClockSampler(physical_gpu_index(local_rank))
    ms_total = time_steps(step_fns, args.steps, sampler, barrier)

    # ---- timed region 2: the same steps with an event pair around the main kernel ---------------------
    n_prof = min(args.steps, 200)
    main_avg_ms = time_main_kernel(reps, step_fns, n_prof)

    # ---- ablation: the L loops one after the other, every loop scanning the shared cache again ---------------
    ablation = None
    if args.ablation and p.L > 1:
        ablation = run_ablation(args, p, reps, dev, local_rank, stream)

    # ---- end to end: host buffers through plt_decode_attn_run_host ------------------------------------
    e2e = None
    if not args.no_e2e:
        hp = DeviceProblem(p, device=None, pin=True)
        for _ in range(2):
            op.run_host(hp, stream)
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            op.run_host(hp, stream)  # synchronises the stream itself
        torch.cuda.synchronize()
        t_e2e = (time.perf_counter() - t0) / args.e2e_steps
        t_e2e = max_over_ranks(t_e2e, world, dev)
        e2e = {"value": job_steps_per_s(world, t_e2e * 1e3), "unit": UNIT, "h2d_bytes_per_step": hp.h2d_bytes(),
               "d2h_bytes_per_step": hp.d2h_bytes(), "steps": args.e2e_steps,
               "note": "plt_decode_attn_run_host with pinned host tensors; the whole KV cache crosses PCIe every step"}
        del hp

    ms_total = max_over_ranks(ms_total, world, dev)
    ms_per_step = ms_total / args.steps
    value = job_steps_per_s(world, ms_per_step)
    info = dict(op.info)
    kernel_path = info["kernel_path"]
    for r in set(reps):
        r.close()
    del reps, dp, op
    torch.cuda.empty_cache()

    if rank == 0:
        peak, peak_src = peak_hbm()
        main_bytes = main_kernel_bytes(by)
        achieved = main_bytes / (main_avg_ms * 1e-3) / 1e9
        kernel_name = {1: "plt_decode_main_" + p.dtype, 2: "plt_decode_main_umma" + ("_e4m3" if p.kv_dtype else "")}[kernel_path]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": p.dtype + ("+e4m3 cache" if p.kv_dtype else ""), "data": "synthetic", "config": cfg,
            "launch": info, "parallelism": f"replicas x{world} (no collective)",
            "loop_queries_per_s": value * p.B * p.L,
            "hbm_gbs_whole_step": by["total"] / (ms_per_step * 1e-3) / 1e9,
            "hbm_frac_of_8tbs": by["total"] / (ms_per_step * 1e-3) / 8e12,
            "clocks": sampler.summary(),
            "gpu_launches": launches_per_step * args.steps,
            "roofline": {
                "bound": "hbm", "kernel": kernel_name, "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src,
                "algorithmic_bytes_per_launch": main_bytes, "avg_launch_ms": main_avg_ms,
                "launches_timed": n_prof, "traffic": recorded_traffic(p.name, kernel_name),
            },
        }
        if e2e is not None:
            line["e2e"] = e2e
        if ablation is not None:
            ablation["ratio"] = ablation["sequential_single_loop_calls_ms"] / ms_per_step
            ablation["private_caches_ratio"] = ablation["private_caches_one_call_ms"] / ms_per_step
            line["ablation"] = ablation
        if suite:
            entries, base = [], None
            for index in (1, 2, 3, 4):
                base = p if index == args.workload else None
                if index != args.workload:
                    e, base = suite_entry(index, "", dev, local_rank, args.suite_steps)
                    entries.append(e)
                e, _ = suite_entry(index, "e4m3", dev, local_rank, args.suite_steps, base=base)
                entries.append(e)
                del base
            line["workloads"] = entries
            # the compute-bound sibling: sequence-shaped attention at the paper's prefill length
            line["seq_attn"] = [seq_entry(4, 2, 5000, dev, local_rank, 10), seq_entry(16, 3, 5000, dev, local_rank, 5)]
        if not args.no_cpu:
            v, cinfo = time_oracle(p, args.cpu_seconds)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, **cinfo}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_ablation(args, p, reps, dev, local_rank, stream):
    """The ablation rows of Table 1 at kernel level, beside the cross-loop-parallel step over one shared cache: the same
    loop-queries as L sequential single-loop calls, each scanning the shared cache again (loop order of the vanilla
    loop transformer), and as one cross-loop-parallel call over L private caches ("Loop+CLP" before KV sharing).
    Global attention only (no window, no gate): a lower bound for both."""
    import torch
    from paper_2510_24824_b200.runner import LoopOrderAblation
    abl = LoopOrderAblation(p, reps[0].dp, device_index=local_rank, kernel_path=args.path)
    n_abl = min(args.steps, 300)

    def timed(fn):
        for _ in range(5):
            fn(stream)
        torch.cuda.synchronize()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for _ in range(n_abl):
            fn(stream)
        a1.record()
        torch.cuda.synchronize()
        return a0.elapsed_time(a1) / n_abl

    seq_ms = timed(abl.run_sequential)
    priv_ms = timed(abl.run_private)
    assert abl.check(stream) == 0
    abl.close()
    return {"sequential_single_loop_calls_ms": seq_ms, "private_caches_one_call_ms": priv_ms, "calls_per_step": p.L,
            "steps_timed": n_abl,
            "note": "global attention only (no window, no gate): lower bounds of the sequential loop order (L launches, "
                    "L scans of the shared cache) and of cross-loop parallelism over L private caches (one launch, L "
                    "caches); ratios = these / ms_per_step of the step over one shared cache"}


if __name__ == "__main__":
    main()
