#!/usr/bin/env python
"""Benchmark of the TSP gated ring MLP on B200: TFLOP/s of the sharded gated-MLP path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

A step is one pass of the path (tsp_mlp_forward, or forward + backward for the `train`
workload) over one seeded synthetic batch, for all D ranks' token shards and all D weight
shards on one GPU.  With N > 1 (launched by torch.distributed.run) every GPU runs the same
single-GPU job on its own seeded batch: no collective is on the data path, so `scaling`
is "weak" and `value` is the sum over GPUs divided by the slowest GPU's time.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU fp64 oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2604_26294_b200 import inputs as inp  # noqa: E402

METRIC = "sharded gated-MLP TFLOP/s on 1 B200 and % of dense-BF16 tensor-core peak"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_BF16_TFLOPS = 1590.0

# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) comes from the ncu captures summarised under
# profiles/: profiles/dram_traffic.json maps "<kernel>|<workload>" to the bytes of one launch (or of all the launches one
# phase takes, where a long problem is cut up), and names the summary file and the commit of the kernels it was taken at.
def load_traffic():
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return {"entries": {}, "commit": None}
    with open(path) as f:
        return json.load(f)


def traffic_of(table, kernel, workload):
    e = table["entries"].get(f"{kernel}|{workload}")
    if e is None:
        return None, None
    return float(e["read"]) + float(e["write"]), f"{e['source']} @ {table.get('commit')}"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"burst": float(d["bf16_tflops"]), "sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"burst": FALLBACK_BF16_TFLOPS, "sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------------
# clock sampling during the timed region (read-only NVML queries)
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {
        0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
        0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
        0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting",
    }

    def __init__(self, device_index: int, period_s: float = 0.01):
        self.period = period_s
        self.samples = []
        self.reason_bits = 0
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch

            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self._nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                try:
                    self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"], "samples": 0}
        reasons = [name for bit, name in self.REASONS.items() if self.reason_bits & bit and name != "gpu_idle"]
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------------
def oracle_sample_seconds(host, rows):
    """Time the fp64 oracle (as it stands) on `rows` token rows of the workload; returns seconds."""
    from oracle import tsp_mlp_oracle as orc

    Xs = inp.bf16_bits_to_f64(host.X[rows])
    t0 = time.perf_counter()
    orc.gated_mlp_forward(Xs, host._Wg64, host._Wu64, host._Wd64)
    return time.perf_counter() - t0


def prepare_oracle_weights(host):
    host._Wg64 = inp.bf16_bits_to_f64(host.Wg)
    host._Wu64 = inp.bf16_bits_to_f64(host.Wu)
    host._Wd64 = inp.bf16_bits_to_f64(host.Wd)


def oracle_baseline(wl, host, target_s=12.0):
    """Forward oracle on a bounded row sample: calibrate on 64 rows, then size the sample for ~target_s."""
    prepare_oracle_weights(host)
    rows = inp.sample_rows(wl.S, wl.D)[:64]
    t = oracle_sample_seconds(host, rows)
    per_row = max(t / len(rows), 1e-9)
    n = int(min(wl.S, max(64, target_s / per_row)))
    n = max(64, (n // 64) * 64)
    rows = np.arange(n)
    t = oracle_sample_seconds(host, rows)
    flops = 6.0 * n * wl.H * wl.F
    cores = len(os.sched_getaffinity(0))
    return {"value": flops / t / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"fp64 numpy forward of the first {n} of {wl.S} token rows against the full weights "
                      f"({t:.2f} s; whole workload extrapolates to {t * wl.S / n:.1f} s)",
            "seconds": t}


def run_reference(args, wl):
    """--impl reference: the CPU oracle on the host cores, rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    host = inp.make_inputs(wl.S, wl.H, wl.F, seed=0)
    prepare_oracle_weights(host)
    # size one step to roughly (120 s / (steps + warmup)), at least 64 rows
    rows64 = np.arange(64)
    per_row = max(oracle_sample_seconds(host, rows64) / 64, 1e-9)
    budget = 120.0 / max(1, args.steps + args.warmup)
    n = int(min(wl.S, max(64, (budget / per_row) // 64 * 64)))
    rows = np.arange(n)
    for _ in range(args.warmup):
        oracle_sample_seconds(host, rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_sample_seconds(host, rows)
    dt = (time.perf_counter() - t0) / max(1, args.steps)
    tf = 6.0 * n * wl.H * wl.F / dt / 1e12
    cores = len(os.sched_getaffinity(0))
    line = {
        "impl": "reference", "metric": METRIC, "value": tf, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "S": wl.S, "H": wl.H, "F": wl.F, "D": wl.D,
                   "sample_rows_per_step": n},
        "cpu_baseline": {"value": tf, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"each step = fp64 numpy forward of the first {n} of {wl.S} token rows"},
        "e2e": {"value": tf, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# Further workloads in the same run (timing only): the other BASELINE configs and a power-limited loop.
# Their inputs have the recipe's distributions but are drawn on the device (seeded torch generator) to keep the run
# short; parity at these shapes is what tests/test_full_size_gpu.py checks, with the recipe's own bits.
# ------------------------------------------------------------------------------------------------
def _device_inputs(torch, S, H, F, D, train, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)

    def draw(shape, std):
        return (torch.randn(shape, generator=g, device="cuda", dtype=torch.float32) * std).to(torch.bfloat16)

    t = {"X": draw((S, H), 1.0), "Wg": draw((D, H, F // D), H ** -0.5), "Wu": draw((D, H, F // D), H ** -0.5),
         "Wd": draw((D, F // D, H), F ** -0.5)}
    if train:
        t["dY"] = draw((S, H), 1.0)
    return t


def time_workload(b, torch, name, wl, peaks, traffic, *, train=False, stored=False, steps=10, warmup=3, min_seconds=0.0,
                  local_rank=0):
    """CUDA-event timing of one workload through the C ABI; returns the sub-record for the bench line."""
    S, H, F, D = wl.S, wl.H, wl.F, wl.D
    t = _device_inputs(torch, S, H, F, D, train, seed=1234)
    Y = torch.empty(S, H, dtype=torch.bfloat16, device="cuda")
    plan = b.tsp_mlp_plan(H, F, D)
    ws = torch.empty(b.tsp_mlp_workspace_bytes(plan, S, b.TSP_WS_BACKWARD if train else b.TSP_WS_FORWARD),
                     dtype=torch.uint8, device="cuda")
    b.tsp_mlp_set_workspace(plan, ws)
    if train:
        dX = torch.empty(S, H, dtype=torch.bfloat16, device="cuda")
        dWg = torch.empty(D, H, F // D, dtype=torch.float32, device="cuda")
        dWu = torch.empty(D, H, F // D, dtype=torch.float32, device="cuda")
        dWd = torch.empty(D, F // D, H, dtype=torch.float32, device="cuda")
    if stored:
        saved = torch.empty(b.tsp_mlp_saved_bytes(plan, S), dtype=torch.uint8, device="cuda")

    def step():
        if stored:
            b.tsp_mlp_forward_save(plan, t["X"], t["Wg"], t["Wu"], t["Wd"], Y, saved, S, D)
            b.tsp_mlp_backward_saved(plan, t["X"], t["Wg"], t["Wu"], t["Wd"], t["dY"], saved, dX, dWg, dWu, dWd, S, D)
            return
        b.tsp_mlp_forward(plan, t["X"], t["Wg"], t["Wu"], t["Wd"], Y, S, D)
        if train:
            b.tsp_mlp_backward(plan, t["X"], t["Wg"], t["Wu"], t["Wd"], t["dY"], dX, dWg, dWu, dWd, S, D)

    for _ in range(max(3, warmup)):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if min_seconds > 0:      # size the loop from a short probe so that it runs for about min_seconds
        e0.record()
        for _ in range(5):
            step()
        e1.record()
        torch.cuda.synchronize()
        steps = max(steps, int(min_seconds * 1e3 / (e0.elapsed_time(e1) / 5)) + 1)
    calls = 2 if train else 1
    n_prof = min(4096, steps * calls)
    b.tsp_mlp_profile_begin(plan, n_prof)
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    sampler.stop()
    assert b.tsp_mlp_status(plan) == b.TSP_OK, f"device-side wait timed out ({name})"
    ms = e0.elapsed_time(e1) / steps
    per_call = [np.mean(np.asarray([b.tsp_mlp_profile_read(plan, i) for i in range(c, n_prof, calls)]), axis=0)
                for c in range(calls)]
    b.tsp_mlp_profile_end(plan)
    b.tsp_mlp_plan_destroy(plan)
    fwd_names = ["gate_up_store" if stored else "gate_up", "down"]
    bwd_names = ["dA_saved", "dX", "dW"] if stored else ["dA", "gate_up_backward", "dX", "dW"]
    shf = float(S) * H * F
    flops_of = {"gate_up": 4 * shf, "gate_up_store": 4 * shf, "down": 2 * shf, "dA": 2 * shf, "dA_saved": 2 * shf,
                "gate_up_backward": 4 * shf, "dX": 4 * shf, "dW": 6 * shf}
    kernels = {}
    for names, vals in zip((fwd_names, bwd_names), per_call):
        # a phase that was cut into several launches reports one interval per phase (events sit between phases)
        for n, v in zip(names, vals):
            tr, src = traffic_of(traffic, n, name)
            kernels[n] = {"ms": float(v), "tflops": flops_of[n] / (float(v) * 1e-3) / 1e12, "dram_bytes": tr,
                          "traffic_source": src}
    model_flops = wl.forward_flops() + (wl.backward_flops() if train else 0.0)
    hw_flops = model_flops + (4 * shf if train and not stored else 0.0)
    value = model_flops / (ms * 1e-3) / 1e12
    clocks = sampler.summary()
    return {"pass": ("forward+backward (stored activations)" if stored else "forward+backward (G, U recomputed)" if train
                     else "forward"), "S": S, "H": H, "F": F, "D": D, "steps": steps, "ms_per_step": ms, "tflops": value,
            "tflops_hardware": hw_flops / (ms * 1e-3) / 1e12,
            "frac_of_burst": value / peaks["burst"], "frac_of_sustained": value / peaks["sustained"],
            "frac_of_nominal": value / NOMINAL_BF16_TFLOPS, "kernels": kernels, "clocks": clocks,
            "ms_x_sm_mhz": (ms * clocks["sm_mhz"]) if clocks.get("sm_mhz") else None}


def extra_workloads(b, torch, peaks, traffic, local_rank):
    """The BASELINE configs beside the headline one, and the headline one over a power-limited loop."""
    out = {}
    plan_of = [("7b_long", dict(steps=6)), ("sweep_d1", dict(steps=10)), ("sweep_d16", dict(steps=10)),
               ("train", dict(train=True, steps=20)), ("train_stored", dict(train=True, stored=True, steps=20))]
    for name, kw in plan_of:
        wl = inp.WORKLOADS["train" if name == "train_stored" else name]
        try:
            out[name] = time_workload(b, torch, "train" if name == "train_stored" else name, wl, peaks, traffic,
                                      local_rank=local_rank, **kw)
        except Exception as e:   # noqa: BLE001 - a sub-run must not take the headline down with it
            out[name] = {"error": repr(e)}
        torch.cuda.empty_cache()
    sustained = None
    try:
        sustained = time_workload(b, torch, "7b_short", inp.WORKLOADS["7b_short"], peaks, traffic, min_seconds=3.0,
                                  local_rank=local_rank)
        sustained["note"] = ("the headline workload for at least 3 s: under the 1 kW cap the SM clock settles well below "
                             "its maximum; compare tflops with the measured sustained GEMM figure and ms x MHz with the "
                             "burst run")
    except Exception as e:   # noqa: BLE001
        sustained = {"error": repr(e)}
    return out, sustained


# ------------------------------------------------------------------------------------------------
# aggregation over ranks (N > 1: independent replicas, one per GPU)
# ------------------------------------------------------------------------------------------------
def max_over_ranks(value_ms: float, world: int, device="cpu") -> float:
    """Slowest rank's time: all-reduce(MAX) over the default process group (identity for world == 1)."""
    if world <= 1:
        return float(value_ms)
    import torch
    import torch.distributed as dist

    t = torch.tensor([value_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tflops(world: int, flops_per_rank_step: float, ms_per_step: float) -> float:
    """Aggregate over all replicas: every rank does `flops_per_rank_step` in the slowest rank's time."""
    return world * flops_per_rank_step / (ms_per_step * 1e-3) / 1e12


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------
def run_gpu(args, wl):
    import torch
    import torch.distributed as dist

    from paper_2604_26294_b200 import binding as b

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    # the library normally arrives built; if it is missing or older than its sources, rank 0 compiles it (nvcc, ~1 min)
    from paper_2604_26294_b200 import build as _build

    if local_rank == 0:
        _build.build_library()
    if world > 1:
        dist.barrier()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    train = wl.name == "train" or args.backward
    S, H, F, D = wl.S, wl.H, wl.F, wl.D
    host = inp.make_inputs(S, H, F, seed=rank, with_dy=train)

    def dev(bits):
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)

    Wg_h, Wu_h, Wd_h = inp.shard_columns(host.Wg, D), inp.shard_columns(host.Wu, D), inp.shard_rows(host.Wd, D)
    X, Wg, Wu, Wd = dev(host.X), dev(Wg_h), dev(Wu_h), dev(Wd_h)
    Y = torch.empty(S, H, dtype=torch.bfloat16, device="cuda")
    plan = b.tsp_mlp_plan(H, F, D)
    staged = args.mode == "staged"
    ws_bytes = max(b.tsp_mlp_workspace_bytes(plan, S, b.TSP_WS_BACKWARD if train else b.TSP_WS_FORWARD),
                   b.tsp_mlp_workspace_bytes_host(plan, S),
                   b.tsp_mlp_workspace_bytes_staged(plan, S) if staged else 0)
    copy_stream = torch.cuda.Stream() if staged else None
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    b.tsp_mlp_set_workspace(plan, ws)
    stored = train and args.stored_activations
    if stored:
        saved = torch.empty(b.tsp_mlp_saved_bytes(plan, S), dtype=torch.uint8, device="cuda")
    if train:
        dY = dev(host.dY)
        dX = torch.empty(S, H, dtype=torch.bfloat16, device="cuda")
        dWg = torch.empty(D, H, F // D, dtype=torch.float32, device="cuda")
        dWu = torch.empty(D, H, F // D, dtype=torch.float32, device="cuda")
        dWd = torch.empty(D, F // D, H, dtype=torch.float32, device="cuda")

    def step():
        if stored:
            b.tsp_mlp_forward_save(plan, X, Wg, Wu, Wd, Y, saved, S, D)
            b.tsp_mlp_backward_saved(plan, X, Wg, Wu, Wd, dY, saved, dX, dWg, dWu, dWd, S, D)
            return
        if staged:
            b.tsp_mlp_forward_staged(plan, X, Wg, Wu, Wd, Y, S, D, torch.cuda.current_stream(), copy_stream)
        else:
            b.tsp_mlp_forward(plan, X, Wg, Wu, Wd, Y, S, D)
        if train:
            b.tsp_mlp_backward(plan, X, Wg, Wu, Wd, dY, dX, dWg, dWu, dWd, S, D)

    model_flops = wl.forward_flops() + (wl.backward_flops() if train else 0.0)

    for _ in range(max(3, args.warmup)):
        step()
    barrier()
    assert b.tsp_mlp_status(plan) == b.TSP_OK, "device-side wait timed out during warm-up"
    # counted after a call has been made: the backward count depends on the shape-dependent path taken
    kernels_per_step = (2 * D if staged else b.tsp_mlp_kernels_per_call(plan, b.TSP_WS_FORWARD)) + (
        (3 if stored else b.tsp_mlp_kernels_per_call(plan, b.TSP_WS_BACKWARD)) if train else 0)

    # ---- timed region: K steps, inputs resident in HBM ----
    calls_per_step = 2 if train else 1
    REJECT = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"}
    remeasured = False
    for attempt in range(2):
        b.tsp_mlp_profile_begin(plan, min(4096, args.steps * calls_per_step))
        sampler = ClockSampler(local_rank)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        sampler.start()
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        barrier()
        sampler.stop()
        elapsed_ms = e0.elapsed_time(e1)
        assert b.tsp_mlp_status(plan) == b.TSP_OK, "device-side wait timed out"
        # per-kernel durations from the events the library recorded on the launch stream inside the timed region
        n_prof = min(4096, args.steps * calls_per_step)
        fwd_calls = [b.tsp_mlp_profile_read(plan, i) for i in range(0, n_prof, calls_per_step)]
        per_kernel = np.mean(np.asarray(fwd_calls), axis=0)
        step_sums = np.sum(np.asarray(fwd_calls), axis=1)   # kernel time of each forward call
        bwd_kernel = None
        if train:
            bwd_calls = [b.tsp_mlp_profile_read(plan, i) for i in range(1, n_prof, calls_per_step)]
            bwd_kernel = np.mean(np.asarray(bwd_calls), axis=0)
            step_sums = step_sums + np.sum(np.asarray(bwd_calls), axis=1)
        b.tsp_mlp_profile_end(plan)
        # a region that saw a hardware or thermal slowdown is thrown away and measured once more
        if attempt == 0 and REJECT & set(sampler.summary()["reasons"]):
            remeasured = True
            time.sleep(2.0)
            continue
        break

    elapsed_ms = max_over_ranks(elapsed_ms, world, "cuda")
    ms_per_step = elapsed_ms / args.steps
    value = whole_job_tflops(world, model_flops, ms_per_step)

    # ---- end to end: host buffers in pinned memory, H2D + forward + D2H every step ----
    e2e = None
    if not train and not args.no_e2e and not staged:
        hX = torch.from_numpy(host.X.view(np.int16)).pin_memory()
        hWg = torch.from_numpy(Wg_h.view(np.int16)).pin_memory()
        hWu = torch.from_numpy(Wu_h.view(np.int16)).pin_memory()
        hWd = torch.from_numpy(Wd_h.view(np.int16)).pin_memory()
        hY = torch.empty(S, H, dtype=torch.int16).pin_memory()
        n_e2e = max(2, min(args.steps, 8))
        for _ in range(2):
            b.tsp_mlp_forward_host(plan, hX, hWg, hWu, hWd, hY, S, D)
        barrier()
        e0.record()
        for _ in range(n_e2e):
            b.tsp_mlp_forward_host(plan, hX, hWg, hWu, hWd, hY, S, D)
            torch.cuda.current_stream().synchronize()  # the caller reads Y on the host
        e1.record()
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1), world, "cuda") / n_e2e
        h2d = hX.numel() * 2 + hWg.numel() * 2 + hWu.numel() * 2 + hWd.numel() * 2
        e2e = {"value": whole_job_tflops(world, model_flops, e2e_ms), "unit": UNIT,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(hY.numel() * 2),
               "ms_per_step": e2e_ms, "steps": n_e2e,
               "call": "tsp_mlp_forward_host (pinned host X, Wg, Wu, Wd -> host Y)"}
        # the host path must give the same bits as the device path
        same = bool((hY.cuda() == Y.view(torch.int16)).all())
        e2e["matches_device_path"] = same

    # context only (not a target, not the product path): torch eager = cuBLAS GEMMs + pointwise kernels, same shapes
    context = None
    if world == 1 and not train and not staged and not args.no_context:
        Wg_f = Wg.permute(1, 0, 2).reshape(H, F).contiguous()
        Wu_f = Wu.permute(1, 0, 2).reshape(H, F).contiguous()
        Wd_f = Wd.reshape(F, H)
        for _ in range(3):
            Yt = (torch.nn.functional.silu(X @ Wg_f) * (X @ Wu_f)) @ Wd_f
        torch.cuda.synchronize()
        n_ctx = max(3, min(args.steps, 20))
        e0.record()
        for _ in range(n_ctx):
            Yt = (torch.nn.functional.silu(X @ Wg_f) * (X @ Wu_f)) @ Wd_f
        e1.record()
        torch.cuda.synchronize()
        ctx_ms = e0.elapsed_time(e1) / n_ctx
        context = {"torch_eager_tflops": model_flops / (ctx_ms * 1e-3) / 1e12, "torch_eager_ms": ctx_ms,
                   "note": "library GEMMs + pointwise kernels on the same box and shapes; context, not a target",
                   "rel_diff_vs_this_library": float(((Y.float() - Yt.float()).norm() / Yt.float().norm()).item())}
        del Wg_f, Wu_f, Wd_f, Yt

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    traffic = load_traffic()
    if staged:
        # staged mode records one interval for the whole call; no per-kernel split
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "pass": "forward", "mode": "staged (ring copies on a side stream)",
                       "S": S, "H": H, "F": F, "D": D, "ring_copy_bytes_per_step": (D - 1) * 6 * H * F},
            "clocks": sampler.summary(), "gpu_launches": int(args.steps * kernels_per_step),
            "e2e": None, "roofline": None, "cpu_baseline": None,
        }
        print(json.dumps(line), flush=True)
        b.tsp_mlp_plan_destroy(plan)
        if world > 1:
            dist.destroy_process_group()
        return
    # dominant kernel: the gate|up GEMM with the SwiGLU epilogue (two thirds of the forward FLOPs)
    gate_up_ms = float(per_kernel[0])
    gate_up_flops = 4.0 * S * H * F
    achieved = gate_up_flops / (gate_up_ms * 1e-3) / 1e12
    pairs = (S // D) % 256 == 0 and os.environ.get("TSP_MLP_PAIR", "1") != "0"
    gate_up_name = ("pair_gemm_kernel<PairGateUpPolicyT<%d>>" % (2 if stored else 0)) if pairs else "gate_up_swiglu_kernel"
    down_name = "pair_{gemm,wide}_kernel<PairDownPolicy>" if pairs else "down_accumulate_kernel"
    roofline = {
        "bound": "tensor", "kernel": gate_up_name, "achieved": achieved, "peak": peaks["burst"],
        "unit": UNIT, "frac": achieved / peaks["burst"], "peak_source": f"of {peaks['source']} (burst bf16 GEMM)",
        "frac_of_sustained": achieved / peaks["sustained"], "frac_of_nominal": achieved / NOMINAL_BF16_TFLOPS,
        "flops_per_launch": gate_up_flops, "ms_per_launch": gate_up_ms,
        "traffic": traffic_of(traffic, "gate_up_store" if stored else "gate_up", wl.name)[0] if pairs else None,
        "traffic_source": traffic_of(traffic, "gate_up_store" if stored else "gate_up", wl.name)[1] if pairs else None,
        "algorithmic_bytes_per_launch": 2.0 * S * H + 4.0 * H * F + 2.0 * S * F,
        "kernels_ms": {gate_up_name: gate_up_ms, down_name: float(per_kernel[1])},
        "kernels_dram_bytes": {gate_up_name: traffic_of(traffic, "gate_up_store" if stored else "gate_up", wl.name)[0],
                               down_name: traffic_of(traffic, "down", wl.name)[0]} if pairs else None,
    }
    if bwd_kernel is not None:
        roofline["kernels_ms"].update({f"backward_kernel_{i}": float(v) for i, v in enumerate(bwd_kernel)})

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cpu = oracle_baseline(wl, host)

    # the other BASELINE configs and the power-limited loop ride along with the default run only
    workloads = sustained = None
    if world == 1 and wl.name == "7b_short" and not train and not args.no_extras:
        del X, Wg, Wu, Wd, Y, ws
        torch.cuda.empty_cache()
        workloads, sustained = extra_workloads(b, torch, peaks, traffic, local_rank)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "ms_per_step_kernels_median": float(np.median(step_sums)), "ms_per_step_kernels_min": float(np.min(step_sums)),
        "context": context,
        "config": {"workload": wl.name,
                   "pass": ("forward+backward (stored activations)" if stored else
                            "forward+backward (G, U recomputed)" if train else "forward"), "S": S, "H": H, "F": F,
                   "D": D, "tokens_per_rank": S // D, "shard_width": F // D, "model_flops_per_step": model_flops,
                   "l2": "inputs larger than L2 (X+W = %.0f MB, intermediate %.0f MB)" % (
                       (2 * S * H + 6 * H * F) / 1e6, 2 * S * F / 1e6),
                   "parallelism": "all D ranks' shards on one GPU; replicas across GPUs"},
        "pct_of_measured_bf16_peak": 100.0 * value / world / peaks["burst"],
        "pct_of_nominal_bf16_peak": 100.0 * value / world / NOMINAL_BF16_TFLOPS,
        "clocks": dict(sampler.summary(), remeasured=remeasured),
        "e2e": e2e,
        "gpu_launches": int(args.steps * kernels_per_step),
        "roofline": roofline,
        "cpu_baseline": cpu,
        "workloads": workloads,
        "sustained": sustained,
    }
    print(json.dumps(line), flush=True)
    b.tsp_mlp_plan_destroy(plan)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------
# Ring arm (opt-in, --mode ring): the D = N ranks are the N GPUs, every rank holds its own token shard and ONE
# weight shard, and the shards travel over NCCL send / receive (paper_2604_26294_b200/ring.py).  The work of the
# workload is divided over the ranks (strong scaling); at N = 1 it is the D = 1 problem through the step kernels.
# ------------------------------------------------------------------------------------------------
def run_ring(args, wl):
    import torch
    import torch.distributed as dist

    from paper_2604_26294_b200 import binding as b
    from paper_2604_26294_b200 import build as _build
    from paper_2604_26294_b200 import ring

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if local_rank == 0:
        _build.build_library()
    if world > 1:
        dist.barrier()
    train = wl.name == "train" or args.backward
    S, H, F, D = wl.S, wl.H, wl.F, world
    if S % D or F % D or (F // D) % (256 if train else 128):
        raise SystemExit(f"workload {wl.name} does not divide over {D} ranks")
    S_loc, F_d = S // D, F // D
    host = inp.make_inputs(S, H, F, seed=0, with_dy=train)      # the same problem on every rank; each keeps its shards

    def dev(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

    X_p = dev(host.X[rank * S_loc:(rank + 1) * S_loc])
    cols = slice(rank * F_d, (rank + 1) * F_d)
    shard = ring.pack_shard(dev(host.Wg[:, cols]), dev(host.Wu[:, cols]), dev(host.Wd[cols, :]))
    Y_p = torch.empty_like(X_p)
    mlp = ring.TspRingMlp(H, F, D, rank, S_loc, training=train)
    if train:
        dY_p = dev(host.dY[rank * S_loc:(rank + 1) * S_loc])
        dX_p = torch.empty_like(X_p)

    def step():
        mlp.forward(X_p, shard, Y_p)
        if train:
            mlp.backward(X_p, shard, dY_p, dX_p)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
    barrier()
    assert b.tsp_mlp_status(mlp.plan) == b.TSP_OK, "device-side wait timed out during warm-up"
    sampler = ClockSampler(local_rank)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    sampler.stop()
    assert b.tsp_mlp_status(mlp.plan) == b.TSP_OK, "device-side wait timed out"
    ms_per_step = max_over_ranks(e0.elapsed_time(e1), world, "cuda") / args.steps
    model_flops = wl.forward_flops() + (wl.backward_flops() if train else 0.0)   # of the whole job, all ranks together
    if rank == 0:
        line = {
            "metric": METRIC, "value": model_flops / (ms_per_step * 1e-3) / 1e12, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "pass": "forward+backward (G, U recomputed)" if train else "forward",
                       "mode": "ring (one rank per GPU, shards travel over NCCL send/receive)", "S": S, "H": H, "F": F,
                       "D": D, "tokens_per_rank": S_loc, "shard_width": F_d,
                       "ring_bytes_sent_per_rank_per_step": (D - 1) * 6 * H * F_d + (D * 12 * H * F_d if train and D > 1 else 0)},
            "clocks": sampler.summary(), "gpu_launches": int(args.steps * D * (6 if train else 2)),
            "e2e": None, "roofline": None, "cpu_baseline": None,
        }
        print(json.dumps(line), flush=True)
    mlp.close()
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------
# Attention-projection arm (workloads attn_*): the two dense steps of Algorithm 1, one kernel each.
# ------------------------------------------------------------------------------------------------
def run_attn(args, wl):
    import torch

    from paper_2604_26294_b200 import binding as b
    from paper_2604_26294_b200 import build as _build

    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        raise SystemExit("the attention-projection arm runs on one GPU")
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(0)
    _build.build_library()
    S, H, Hq, Hkv, D = wl.S, wl.H, wl.Hq, wl.Hkv, wl.D
    train = args.backward
    host = inp.make_attn_inputs(S, H, Hq, Hkv, seed=0, with_grads=train)

    def dev(bits):
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)

    X, Wq, Wk, Wv, A = dev(host.X), dev(host.Wq), dev(host.Wk), dev(host.Wv), dev(host.A)
    Wo = dev(inp.shard_out_columns(host.Wo, D))
    Q = torch.empty(S, Hq, dtype=torch.bfloat16, device="cuda")
    K = torch.empty(S, Hkv, dtype=torch.bfloat16, device="cuda")
    V = torch.empty(S, Hkv, dtype=torch.bfloat16, device="cuda")
    Y = torch.empty(S, H, dtype=torch.bfloat16, device="cuda")
    plan = b.tsp_attn_plan(H, Hq, Hkv, D)
    if train:
        dQ, dK, dV, dY = dev(host.dQ), dev(host.dK), dev(host.dV), dev(host.dY)
        dX, dA = torch.empty_like(X), torch.empty_like(A)
        dWq = torch.empty(Hq, H, dtype=torch.float32, device="cuda")
        dWk = torch.empty(Hkv, H, dtype=torch.float32, device="cuda")
        dWv = torch.empty(Hkv, H, dtype=torch.float32, device="cuda")
        dWo = torch.empty(D, H, Hq // D, dtype=torch.float32, device="cuda")

    def step():
        b.tsp_attn_qkv_forward(plan, X, Wq, Wk, Wv, Q, K, V, S, D)
        b.tsp_attn_out_forward(plan, A, Wo, Y, S, D)
        if train:
            b.tsp_attn_out_backward(plan, A, Wo, dY, dA, dWo, S, D)
            b.tsp_attn_qkv_backward(plan, X, Wq, Wk, Wv, dQ, dK, dV, dX, dWq, dWk, dWv, S, D)

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    assert b.tsp_attn_status(plan) == b.TSP_OK
    calls = 4 if train else 2
    n_prof = min(4096, calls * args.steps)
    b.tsp_attn_profile_begin(plan, n_prof)
    sampler = ClockSampler(0)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.start()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    sampler.stop()
    assert b.tsp_attn_status(plan) == b.TSP_OK, "device-side wait timed out"
    ms_per_step = e0.elapsed_time(e1) / args.steps
    qkv_ms = float(np.mean([b.tsp_attn_profile_read(plan, i)[0] for i in range(0, n_prof, calls)]))
    out_ms = float(np.mean([b.tsp_attn_profile_read(plan, i)[0] for i in range(1, n_prof, calls)]))
    kernels_ms = {"pair_gemm_kernel<PairQkvPolicy>": qkv_ms, "pair_gemm_kernel<PairOutPolicy>": out_ms}
    if train:
        ob = np.mean([b.tsp_attn_profile_read(plan, i) for i in range(2, n_prof, calls)], axis=0)
        qb = np.mean([b.tsp_attn_profile_read(plan, i) for i in range(3, n_prof, calls)], axis=0)
        kernels_ms.update({"pair_gemm_kernel<PairAttnDaPolicy>": float(ob[0]),
                           "pair_gemm_kernel<PairAttnDwPolicy> (dWo)": float(ob[1]),
                           "pair_gemm_kernel<PairAttnDxPolicy>": float(qb[0]),
                           "pair_gemm_kernel<PairAttnDwPolicy> (dWq, dWk, dWv)": float(qb[1])})
    b.tsp_attn_profile_end(plan)
    flops = (wl.qkv_flops() + wl.out_flops()) * (3.0 if train else 1.0)   # backward = twice the forward
    peaks = measured_peaks()
    achieved = wl.qkv_flops() / (qkv_ms * 1e-3) / 1e12
    # oracle timed on a bounded sample of rows (row-separable), host cores
    cpu = None
    if not args.no_cpu_baseline:
        from oracle import tsp_attn_proj_oracle as attn_orc   # the only use of the oracle in this arm

        f = [inp.bf16_bits_to_f64(a) for a in (host.X, host.Wq, host.Wk, host.Wv, host.A, host.Wo)]
        rows = np.arange(0, S, max(1, S // 256))[:256]
        t0 = time.perf_counter()
        reps = 0
        while time.perf_counter() - t0 < 10.0:
            attn_orc.qkv_rows(f[0], f[1], f[2], f[3], rows)
            attn_orc.output_rows(f[4], f[5], rows)
            reps += 1
        dt = (time.perf_counter() - t0) / reps
        cpu = {"value": (wl.qkv_flops() + wl.out_flops()) * len(rows) / S / dt / 1e12, "unit": UNIT, "cores": len(os.sched_getaffinity(0)),
               "kind": "oracle", "sample": f"forward on {len(rows)} of {S} token rows, fp64, {reps} repetitions"}
    line = {
        "metric": "TSP attention projection GEMMs (Q/K/V + output projection) TFLOP/s on 1 B200",
        "value": flops / (ms_per_step * 1e-3) / 1e12, "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl.name, "pass": "forward+backward" if train else "forward", "S": S, "H": H, "Hq": Hq, "Hkv": Hkv, "D": D, "model_flops_per_step": flops,
                   "l2": "inputs larger than L2 (X + weights + A = %.0f MB)" % (
                       (2 * S * H + 2 * H * (Hq + 2 * Hkv) + 2 * S * Hq + 2 * H * Hq) / 1e6)},
        "clocks": sampler.summary(), "gpu_launches": int((6 if train else 2) * args.steps), "e2e": None,
        "roofline": {"bound": "tensor", "kernel": "pair_gemm_kernel<PairQkvPolicy>", "achieved": achieved,
                     "peak": peaks["burst"], "unit": UNIT, "frac": achieved / peaks["burst"],
                     "peak_source": f"of {peaks['source']} (burst bf16 GEMM)",
                     # dram__bytes_read.sum + dram__bytes_write.sum of one launch, from the committed ncu capture
                     "traffic": traffic_of(load_traffic(), "attn_qkv", wl.name)[0],
                     "traffic_source": traffic_of(load_traffic(), "attn_qkv", wl.name)[1],
                     "algorithmic_bytes_per_launch": 2.0 * S * H + 2.0 * H * (Hq + 2 * Hkv) + 2.0 * S * (Hq + 2 * Hkv),
                     "kernels_ms": kernels_ms,
                     "out_projection_tflops": wl.out_flops() / (out_ms * 1e-3) / 1e12},
        "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    b.tsp_attn_plan_destroy(plan)


# ------------------------------------------------------------------------------------------------
# One rank's share of the ring (opt-in, --mode rank-steps): the tokens of ONE rank (S / D of the workload) and all D
# shards resident on this GPU, applied by the per-rank step entry points, g ring steps per launch pair.  No
# transfers: this is the compute side of what each GPU of a D-GPU ring does per forward (and backward) pass.
# ------------------------------------------------------------------------------------------------
def run_rank_steps(args, wl):
    import torch

    from paper_2604_26294_b200 import binding as b
    from paper_2604_26294_b200 import build as _build
    from paper_2604_26294_b200 import ring

    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        raise SystemExit("--mode rank-steps runs on one GPU")
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(0)
    _build.build_library()
    train = wl.name == "train" or args.backward
    S, H, F, D = wl.S, wl.H, wl.F, wl.D
    S_loc, F_d, g = S // D, F // D, max(1, min(args.steps_per_launch, D))
    host = inp.make_inputs(S_loc, H, F, seed=0, with_dy=train)      # rank 0's tokens, the whole layer's weights

    def dev(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

    X_p = dev(host.X)
    Wg, Wu, Wd = dev(inp.shard_columns(host.Wg, D)), dev(inp.shard_columns(host.Wu, D)), dev(inp.shard_rows(host.Wd, D))
    order = [ring.shard_at_step(0, t, D) for t in range(D)]
    packed = torch.stack([ring.pack_shard(Wg[k], Wu[k], Wd[k]) for k in order])      # row t = the shard met at step t
    Y_p = torch.empty_like(X_p)
    plan = b.tsp_mlp_plan(H, F, D)
    ws = torch.empty(max(b.tsp_mlp_workspace_bytes_ring(plan, S_loc, b.TSP_WS_BACKWARD),
                         b.tsp_mlp_workspace_bytes_ring_group(plan, S_loc, g),
                         b.tsp_mlp_workspace_bytes_ring_group_backward(plan, S_loc, g) if train else 0),
                     dtype=torch.uint8, device="cuda")
    b.tsp_mlp_set_workspace(plan, ws)
    if train:
        dY_p, dX_p = dev(host.dY), torch.empty_like(X_p)
        dW = torch.empty(D, 3 * H * F_d, dtype=torch.float32, device="cuda")

    def step():
        for t0 in range(0, D, g):
            a, u, d = ring.unpack_shard(packed[t0], H, F_d)
            b.tsp_mlp_ring_steps(plan, X_p, a, u, d, packed.shape[1], min(g, D - t0), Y_p, S_loc, t0, D)
        if train and g > 1:      # grouped backward: three kernels per group, the weight gradients shard by shard
            for t0 in range(0, D, g):
                n = min(g, D - t0)
                a, u, d = ring.unpack_shard(packed[t0], H, F_d)
                b.tsp_mlp_ring_steps_backward_dx(plan, X_p, a, u, d, packed.shape[1], n, dY_p, dX_p, S_loc, t0, D)
                for i in range(n):
                    ga, gu, gd = ring.unpack_shard(dW[t0 + i], H, F_d)
                    b.tsp_mlp_ring_steps_backward_dw(plan, X_p, dY_p, ga, gu, gd, S_loc, i, n, 0, D)
        elif train:
            for t in range(D):
                a, u, d = ring.unpack_shard(packed[t], H, F_d)
                ga, gu, gd = ring.unpack_shard(dW[t], H, F_d)
                b.tsp_mlp_ring_step_backward_dx(plan, X_p, a, u, d, dY_p, dX_p, S_loc, t, D)
                b.tsp_mlp_ring_step_backward_dw(plan, X_p, dY_p, ga, gu, gd, S_loc, 0, D)

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    assert b.tsp_mlp_status(plan) == b.TSP_OK
    run = step
    if args.graph:
        # one pass (all D ring steps) recorded once and replayed: the host's per-call work (argument marshalling,
        # tensor-map encoding, launch) leaves the timed region, what remains is the device side of the ring steps
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                step()
        torch.cuda.current_stream().wait_stream(side)
        run = graph.replay
        for _ in range(3):
            run()
        torch.cuda.synchronize()
    sampler = ClockSampler(0)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.start()
    e0.record()
    for _ in range(args.steps):
        run()
    e1.record()
    torch.cuda.synchronize()
    sampler.stop()
    assert b.tsp_mlp_status(plan) == b.TSP_OK, "device-side wait timed out"
    ms = e0.elapsed_time(e1) / args.steps
    flops = (6.0 + (12.0 if train else 0.0)) * S_loc * H * F
    launches = b.tsp_mlp_kernels_per_call(plan, b.TSP_WS_FORWARD) * ((D + g - 1) // g) + (
        (3 * ((D + g - 1) // g) + D if g > 1 else 4 * D) if train else 0)
    line = {
        "metric": METRIC, "value": flops / (ms * 1e-3) / 1e12, "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl.name, "pass": "forward+backward (G, U recomputed)" if train else "forward",
                   "mode": "rank-steps (one rank's tokens, all shards local, per-rank step entry points)",
                   "S_loc": S_loc, "H": H, "F": F, "D": D, "ring_steps_per_launch": g,
                   "launches": "replayed from a CUDA graph" if args.graph else "issued by the host every step",
                   "kernels_per_forward_call": b.tsp_mlp_kernels_per_call(plan, b.TSP_WS_FORWARD),
                   "us_per_ring_step": 1e3 * ms / D},
        "clocks": sampler.summary(), "gpu_launches": int(args.steps * launches), "e2e": None, "roofline": None,
        "cpu_baseline": None,
    }
    print(json.dumps(line), flush=True)
    b.tsp_mlp_plan_destroy(plan)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="7b_short", choices=sorted(inp.WORKLOADS) + sorted(inp.ATTN_WORKLOADS))
    ap.add_argument("--backward", action="store_true", help="time forward + backward (as the `train` workload does)")
    ap.add_argument("--stored-activations", action="store_true",
                    help="training step through tsp_mlp_forward_save / tsp_mlp_backward_saved (no recomputation)")
    ap.add_argument("--steps-per-launch", type=int, default=1,
                    help="--mode rank-steps: ring steps applied per group of launches (forward, and backward except dW)")
    ap.add_argument("--mode", default="direct", choices=["direct", "staged", "ring", "rank-steps"],
                    help="staged: Algorithm 2 step by step with the shard transfer emulated on a side stream; "
                         "ring: D = N ranks on N GPUs, the shards travel between the GPUs; "
                         "rank-steps: one rank's tokens against all D shards through the per-rank step calls")
    ap.add_argument("--graph", action="store_true",
                    help="--mode rank-steps: record one pass in a CUDA graph and time its replays (device side only)")
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-context", action="store_true", help="skip the torch-eager context measurement")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg (profiling runs)")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the further workloads and the sustained loop that ride along with the default run")
    args = ap.parse_args()
    if args.workload in inp.ATTN_WORKLOADS:
        if args.impl == "reference":
            raise SystemExit("the reference arm covers the gated-MLP workloads")
        return run_attn(args, inp.ATTN_WORKLOADS[args.workload])
    wl = inp.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
    elif args.mode == "ring":
        run_ring(args, wl)
    elif args.mode == "rank-steps":
        run_rank_steps(args, wl)
    else:
        run_gpu(args, wl)


if __name__ == "__main__":
    main()
