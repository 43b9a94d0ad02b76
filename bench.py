#!/usr/bin/env python
"""Benchmark of the dense hot path on B200: BF16 GEMM + MHA forward through the C ABI.

One *step* is one pass of the whole hot path over one batch of synthetic input:
one large GEMM (tile schedule, TMA loads, UMMA accumulate, K loop, epilogue) and one
D=128 causal attention forward on the long-sequence configuration (work schedule, Q/K/V
loads, S = QK^T, mask, online softmax, PV, finalize).  `value` is TFLOP/s over the step (conventional FLOP counts:
2MNK; 4*B*H*Nq*Nk*D, halved when causal), summed over all ranks.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl mlt|reference] [--all]

For N > 1 launch with torch.distributed.run: every rank runs the same workload on
its own GPU (independent problems, no data-path collective; weak scaling); NCCL is
used only for the barrier and the max-over-ranks time.

`--impl reference` times the CPU oracle (FP64, host threads) on a bounded sample of
the same workload; it is a deliberately slow checker, reported as a baseline.
`--all` adds per-configuration timings of every benchmark configuration under "configs".
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

from paper_2503_14985_b200 import inputs  # noqa: E402

METRIC = "TFLOP/s and % of B200 dense-BF16 peak for GEMM and MHA fwd (1 GPU)"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
GEMM_NAME = "gemm_8192x28672x4096"
MHA_NAME = "mha_b1h16n16384d128_causal"
WORKLOAD = f"{GEMM_NAME} + {MHA_NAME}"


# --------------------------------------------------------------------------
# distributed plumbing (rank / world from the environment; gloo-testable)
# --------------------------------------------------------------------------

def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def init_dist(backend: str):
    """Initialise torch.distributed from RANK/WORLD_SIZE/MASTER_* if WORLD_SIZE > 1; returns (rank, local, world)."""
    rank, local, world = dist_env()
    if world > 1:
        import torch.distributed as dist
        if not dist.is_initialized():
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29500")
            dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local, world


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def aggregate(ms_local: float, units_local: float, world: int, device=None):
    """Whole-job figures: (max time over ranks in ms, sum of units over ranks)."""
    if world == 1:
        return ms_local, units_local
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# --------------------------------------------------------------------------
# clocks (read-only NVML sampling during the timed region)
# --------------------------------------------------------------------------

class ClockSampler:
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
               0x80: "hw_power_brake_slowdown"}

    def __init__(self, index: int, period_s: float = 0.005):
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.power = [], set(), []
        self._stop = threading.Event()
        self._thread = None
        self.max_mhz = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
            # first calls into NVML can take tens of milliseconds: make them before the timed region starts
            pynvml.nvmlDeviceGetClockInfo(self._h, pynvml.NVML_CLOCK_SM)
            pynvml.nvmlDeviceGetCurrentClocksEventReasons(self._h)
            pynvml.nvmlDeviceGetPowerUsage(self._h)
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
                self.power.append(nv.nvmlDeviceGetPowerUsage(self._h) / 1000.0)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples),
                "power_w_max": max(self.power) if self.power else None}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"burst": float(d["bf16_tflops"]), "sustained": float(d["bf16_tflops_sustained"]),
                "hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return {"burst": 1590.0, "sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


# --------------------------------------------------------------------------
# the CPU oracle as a timed baseline (bounded sample of the same workload)
# --------------------------------------------------------------------------

def oracle_sample_step(data, gemm_rows: int, mha_rows: int):
    """One oracle 'step' on a sample of complete output rows; returns (seconds, flop, description)."""
    import oracle
    M, N, K = data["gemm_shape"]
    B, H, Nq, Nk, D, causal = data["mha_shape"]
    rows = np.linspace(0, M - 1, gemm_rows).astype(np.int64)
    qrows = np.unique(np.linspace(0, B * H * Nq - 1, mha_rows).astype(np.int64))
    t0 = time.perf_counter()
    oracle.gemm(data["A"], data["B"], M, N, K, rows=rows)
    oracle.mha_fwd(data["Q"], data["K"], data["V"], causal=bool(causal), scale=data["scale"], qrows=qrows)
    dt = time.perf_counter() - t0
    flop = 2.0 * len(rows) * N * K
    for r in qrows:
        i = int(r % Nq)
        visible = min(Nk, i + (Nk - Nq) + 1) if causal else Nk
        flop += 4.0 * visible * D
    what = f"{len(rows)} of {M} GEMM output rows + {len(qrows)} of {B * H * Nq} attention query rows (all columns)"
    return dt, flop, what


def make_host_data(gemm_name: str, mha_name: str):
    M, N, K, kind, seed = inputs.GEMM_CONFIGS[gemm_name]
    A, B = inputs.gemm_inputs(M, N, K, seed=seed, kind=kind)
    Bn, H, Nq, Nk, D, causal, mseed, outl = inputs.MHA_CONFIGS[mha_name]
    Q, Kk, V = inputs.mha_inputs(Bn, H, Nq, Nk, D, seed=mseed, outlier_percent=outl)
    return {"A": A, "B": B, "Q": Q, "K": Kk, "V": V, "gemm_shape": (M, N, K), "mha_shape": (Bn, H, Nq, Nk, D, causal),
            "scale": float(np.float32(1.0 / np.sqrt(D)))}


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return 0
    import oracle
    data = make_host_data(GEMM_NAME, MHA_NAME)
    cores = oracle.hardware_threads()
    gemm_rows, mha_rows = 64, 2048
    for _ in range(max(args.warmup, 1)):
        oracle_sample_step(data, 8, 64)
    t_total, f_total, what = 0.0, 0.0, ""
    for _ in range(args.steps):
        dt, flop, what = oracle_sample_step(data, gemm_rows, mha_rows)
        t_total += dt
        f_total += flop
    value = f_total / t_total / 1e12
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * t_total / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "note": "CPU oracle on a sample of complete output rows per step"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


# --------------------------------------------------------------------------
# the CUDA path
# --------------------------------------------------------------------------

def run_mlt(args):
    import torch
    import paper_2503_14985_b200 as mlt

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (sm_100a); there is no CPU fallback")
    rank, local, world = init_dist("nccl")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    mlt.load()

    data = make_host_data(GEMM_NAME, MHA_NAME)
    M, N, K = data["gemm_shape"]
    Bn, H, Nq, Nk, D, causal = data["mha_shape"]
    scale = data["scale"]
    gemm_flop = inputs.gemm_flops(M, N, K)
    mha_flop = inputs.mha_flops(Bn, H, Nq, Nk, D, causal)
    step_flop = gemm_flop + mha_flop

    def pinned(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).pin_memory()

    hA, hB, hQ, hK, hV = (pinned(data[k]) for k in ("A", "B", "Q", "K", "V"))
    dA, dB, dQ, dK, dV = (torch.empty_like(h, device=dev) for h in (hA, hB, hQ, hK, hV))
    dC = torch.empty((M, N), dtype=torch.int16, device=dev)
    dO = torch.empty_like(dQ)
    dL = torch.empty((Bn, H, Nq), dtype=torch.float32, device=dev)
    hC = torch.empty((M, N), dtype=torch.int16).pin_memory()
    hO = torch.empty(tuple(dQ.shape), dtype=torch.int16).pin_memory()
    hL = torch.empty((Bn, H, Nq), dtype=torch.float32).pin_memory()
    for d, h in ((dA, hA), (dB, hB), (dQ, hQ), (dK, hK), (dV, hV)):
        d.copy_(h)
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream

    def launch_gemm():
        rc = mlt.gemm_raw(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, K, N, N, sp)
        if rc:
            raise mlt.MltError(rc, "mlt_gemm")

    def launch_mha():
        rc = mlt.mha_fwd_raw(dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), dO.data_ptr(), dL.data_ptr(), Bn, H, Nq, Nk, D,
                             causal, scale, sp)
        if rc:
            raise mlt.MltError(rc, "mlt_mha_fwd")

    def step():
        launch_gemm()
        launch_mha()

    # ---- device-resident timing: W warm-up steps, then exactly K timed steps ----
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    K_steps = args.steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K_steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(world)
    torch.cuda.synchronize()
    with ClockSampler(local) as clocks:
        t_begin.record(stream)
        for i in range(K_steps):
            ev[i][0].record(stream)
            launch_gemm()
            ev[i][1].record(stream)
            launch_mha()
            ev[i][2].record(stream)
        t_end.record(stream)
        torch.cuda.synchronize()
    barrier(world)
    ms_total = t_begin.elapsed_time(t_end)
    gemm_ms = [e[0].elapsed_time(e[1]) for e in ev]
    mha_ms = [e[1].elapsed_time(e[2]) for e in ev]
    # the SM clock the last GEMM / attention launch of the timed region really ran at (cycle counter over ns timer
    # inside the kernels; NVML's figure does not show this part's power management)
    kernel_mhz = {"gemm": mlt.last_clock_mhz(0), "mha_fwd": mlt.last_clock_mhz(1)}
    rc, detail = mlt.last_device_error()
    if rc:
        raise mlt.MltError(rc, f"device status {detail}")

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region ----
    # Every step copies its inputs from pinned host memory and its results back.  Three streams and two sets of
    # device buffers let step i's upload, step i-1's kernels and step i-2's download overlap (PCIe is full duplex),
    # as a serving loop would run it; each step still moves all of its bytes inside the timed region.
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    sets = [{"in": (dA, dB, dQ, dK, dV), "out": (dC, dO, dL)}]
    sets.append({"in": tuple(torch.empty_like(t) for t in sets[0]["in"]), "out": tuple(torch.empty_like(t) for t in sets[0]["out"])})
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_comp = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]

    def e2e_pipeline(n_steps):
        for i in range(n_steps):
            b = i & 1
            (a_, b_, q_, k_, v_), (c_, o_, l_) = sets[b]["in"], sets[b]["out"]
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev_comp[b])  # the kernels of step i-2 have read this input set
                for d, h in ((a_, hA), (b_, hB), (q_, hQ), (k_, hK), (v_, hV)):
                    d.copy_(h, non_blocking=True)
                ev_in[b].record(s_in)
            stream.wait_event(ev_in[b])
            if i >= 2:
                stream.wait_event(ev_out[b])  # the results of step i-2 have left this output set
            rc = mlt.gemm_raw(a_.data_ptr(), b_.data_ptr(), c_.data_ptr(), M, N, K, K, N, N, sp)
            if rc:
                raise mlt.MltError(rc, "mlt_gemm")
            rc = mlt.mha_fwd_raw(q_.data_ptr(), k_.data_ptr(), v_.data_ptr(), o_.data_ptr(), l_.data_ptr(), Bn, H, Nq, Nk, D,
                                 causal, scale, sp)
            if rc:
                raise mlt.MltError(rc, "mlt_mha_fwd")
            ev_comp[b].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_comp[b])
                hC.copy_(c_, non_blocking=True)
                hO.copy_(o_, non_blocking=True)
                hL.copy_(l_, non_blocking=True)
                ev_out[b].record(s_out)
        stream.wait_stream(s_out)  # the timed region ends when the last result is on the host

    e2e_pipeline(max(2, min(args.warmup, 3)))
    torch.cuda.synchronize()
    e2e_steps = max(1, min(K_steps, 10))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(world)
    torch.cuda.synchronize()
    e0.record(stream)
    s_in.wait_event(e0)
    e2e_pipeline(e2e_steps)
    e1.record(stream)
    torch.cuda.synchronize()
    barrier(world)
    e2e_ms = e0.elapsed_time(e1)
    h2d = sum(h.numel() * h.element_size() for h in (hA, hB, hQ, hK, hV))
    d2h = sum(h.numel() * h.element_size() for h in (hC, hO, hL))

    ms_max, flop_all = aggregate(ms_total, step_flop * K_steps, world, dev)
    e2e_max, e2e_flop = aggregate(e2e_ms, step_flop * e2e_steps, world, dev)
    value = flop_all / (ms_max * 1e-3) / 1e12
    e2e_value = e2e_flop / (e2e_max * 1e-3) / 1e12

    # ---- every benchmark configuration on its own (single-GPU runs; rank 0 reports) ----
    per_config = None
    if args.all or (world == 1 and not args.no_configs):
        per_config = time_all_configs(mlt, torch, dev, stream, device_index=local)

    if rank != 0:
        return 0

    peaks = measured_peaks()
    gemm_avg_ms = float(np.mean(gemm_ms))
    mha_avg_ms = float(np.mean(mha_ms))
    achieved = gemm_flop / (gemm_avg_ms * 1e-3) / 1e12
    long_run = ms_total > 1000.0
    peak = peaks["sustained"] if long_run else peaks["burst"]
    roofline = {"bound": "tensor", "kernel": "gemm_bf16_pair_kernel<6, false>", "achieved": achieved, "peak": peak, "unit": UNIT,
                "frac": achieved / peak, "traffic": ncu_traffic_bytes(),
                "peak_source": f"{peaks['source']} cuBLAS bf16 {'sustained' if long_run else 'burst'}",
                "frac_of_nominal_2250": achieved / NOMINAL_BF16_TFLOPS,
                "achieved_hbm_gbs": 2.0 * (M * K + K * N + M * N) / (gemm_avg_ms * 1e-3) / 1e9}
    per_op = {"gemm": {"config": GEMM_NAME, "ms": gemm_avg_ms, "ms_min": float(np.min(gemm_ms)),
                       "tflops": achieved, "tflops_best": gemm_flop / (np.min(gemm_ms) * 1e-3) / 1e12,
                       "frac_of_2250": achieved / NOMINAL_BF16_TFLOPS},
              "mha_fwd": {"config": MHA_NAME, "ms": mha_avg_ms, "ms_min": float(np.min(mha_ms)),
                          "tflops": mha_flop / (mha_avg_ms * 1e-3) / 1e12,
                          "tflops_best": mha_flop / (np.min(mha_ms) * 1e-3) / 1e12,
                          "frac_of_2250": mha_flop / (mha_avg_ms * 1e-3) / 1e12 / NOMINAL_BF16_TFLOPS,
                          "timed": "inside the step, right after the GEMM (the GPU is under its power cap)"}}
    if per_config is not None:
        # the same kernels timed alone (pause, warm-up, L2 flushed between launches): see "configs"
        for op, name in (("gemm", GEMM_NAME), ("mha_fwd", MHA_NAME)):
            if name in per_config:
                c = per_config[name]
                per_op[op]["alone"] = {"ms_min": c["ms_min"], "ms_median": c["ms_median"], "tflops_best": c["tflops_best"],
                                       "tflops_median": c["tflops_median"],
                                       "frac_of_2250_best": c["tflops_best"] / NOMINAL_BF16_TFLOPS,
                                       "frac_of_2250_median": c["tflops_median"] / NOMINAL_BF16_TFLOPS}

    cpu_baseline = None
    if world == 1 or rank == 0:
        import oracle
        dt, flop, what = oracle_sample_step(data, 2048, 32768)
        cpu_baseline = {"value": flop / dt / 1e12, "unit": UNIT, "cores": oracle.hardware_threads(), "kind": "oracle",
                        "sample": what, "seconds": dt}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K_steps, "warmup": args.warmup,
            "ms_per_step": ms_max / K_steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "gemm": {"M": M, "N": N, "K": K}, "mha": {"B": Bn, "H": H, "Nq": Nq, "Nk": Nk,
                       "D": D, "causal": bool(causal)}, "l2": "inputs larger than L2 (302 MB GEMM operands; the GEMM's 772 MB stream evicts Q/K/V between steps)",
                       "flop_convention": "2MNK; 4*B*H*Nq*Nk*D halved when causal", "parallelism": f"replicas x{world}"},
            "clocks": {**clocks.summary(), "sm_mhz_in_kernel": kernel_mhz},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_max / e2e_steps, "steps": e2e_steps,
                    "overlap": "upload of step i, kernels of step i-1 and download of step i-2 on three streams, "
                               "two sets of device buffers"},
            "gpu_launches": 2 * K_steps, "roofline": roofline, "cpu_baseline": cpu_baseline, "per_op": per_op}
    if per_config is not None:
        line["configs"] = per_config
    print(json.dumps(line))
    return 0


def ncu_traffic_bytes():
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the GEMM kernel on the benchmark shape, taken from
    the rows of the committed ncu summary of that capture (None if the summary is not there)."""
    import re
    path = os.path.join(ROOT, "profiles", f"gemm_pair_{GEMM_NAME.split('_', 1)[1]}.md")
    try:
        text = open(path).read()
    except OSError:
        return None
    total = 0.0
    for key in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
        m = re.search(r"\|\s*" + re.escape(key) + r"\s*\|\s*([0-9.]+)\s*GB", text)
        if not m:
            return None
        total += float(m.group(1)) * 1e9
    return total


def time_all_configs(mlt, torch, dev, stream, iters: int = 20, only: str | None = None, warm: int = 3,
                     device_index: int = 0):
    """Min / median kernel time of every benchmark configuration alone (CUDA events, seeded inputs resident, a pause
    and warm-up launches first, L2 evicted between timed launches, NVML clocks sampled per configuration)."""
    out = {}
    sp = stream.cuda_stream

    def devbits(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev)

    flush = torch.empty(256 << 20, dtype=torch.int8, device=dev)

    def timeit(fn, flop, read_flush=False, kind=None):
        torch.cuda.synchronize()
        time.sleep(0.3)  # burst timing: let the power governor recover from the configuration before
        for _ in range(warm):
            fn()
        times = []
        sampler = ClockSampler(device_index, period_s=0.002)
        sampler.__enter__()
        for _ in range(iters):
            # evict L2 between timed launches: by writing a 256 MB buffer, or (for the HBM-bound decode kernel,
            # whose reads would otherwise have to push 126 MB of dirty lines out first) by reading it
            if read_flush:
                flush.view(torch.int32).sum()
            else:
                flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            torch.cuda.synchronize()
            times.append(a.elapsed_time(b))
        sampler.__exit__()
        ck = sampler.summary()
        tmin, tmed = float(np.min(times)), float(np.median(times))
        return {"ms_min": tmin, "ms_median": tmed, "tflops_best": flop / tmin / 1e9, "tflops_median": flop / tmed / 1e9,
                "frac_of_2250_best": flop / tmin / 1e9 / NOMINAL_BF16_TFLOPS, "launches": iters,
                "clocks": {"sm_mhz": ck["sm_mhz"], "samples": ck["samples"], "reasons": ck["reasons"],
                           # the clock the last timed launch really ran at (kernels that carry the probe)
                           "sm_mhz_in_kernel": mlt.last_clock_mhz({"gemm": 0, "mha_fwd": 1}[kind]) if kind else None}}

    for name, (M, N, K, kind, seed) in inputs.GEMM_CONFIGS.items():
        if only is not None and name != only:
            continue
        A, B = inputs.gemm_inputs(M, N, K, seed=seed, kind=kind)
        dA, dB = devbits(A), devbits(B)
        dC = torch.empty((M, N), dtype=torch.int16, device=dev)

        def fn():
            rc = mlt.gemm_raw(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, K, N, N, sp)
            assert rc == 0, rc
        out[name] = timeit(fn, inputs.gemm_flops(M, N, K), kind="gemm")
        del dA, dB, dC
    # the same shapes in the data types of Listing 2 (FP16 operands, FP32 result), plain and as C += A * B
    for base, (M, N, K, kind, seed) in inputs.GEMM_CONFIGS.items():
        names = {acc: base.replace("gemm_", "gemm_f16_acc_" if acc else "gemm_f16_") for acc in (0, 1)}
        if base == "gemm_512" or (only is not None and only not in names.values()):
            continue
        A, B, _ = inputs.gemm_f16_inputs(M, N, K, seed=seed, kind=kind, prior_c=False)
        dA, dB = devbits(A), devbits(B)
        dC = torch.zeros((M, N), dtype=torch.float32, device=dev)
        for acc, name in names.items():
            if only is not None and name != only:
                continue

            def fn():
                rc = mlt.gemm_f16_raw(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, K, N, N, acc, sp)
                assert rc == 0, rc
            out[name] = timeit(fn, inputs.gemm_flops(M, N, K), kind="gemm")
        del dA, dB, dC
    mha_cache = {}
    for name, (Bn, H, Nq, Nk, D, causal, seed, outl) in inputs.MHA_CONFIGS.items():
        if only is not None and name != only:
            continue
        key = (Bn, H, Nq, Nk, D, seed, outl)
        if key not in mha_cache:  # the causal and non-causal long-sequence configurations share their tensors
            mha_cache.clear()
            Q, Kk, V = inputs.mha_inputs(Bn, H, Nq, Nk, D, seed=seed, outlier_percent=outl)
            mha_cache[key] = (devbits(Q), devbits(Kk), devbits(V))
        dQ, dK, dV = mha_cache[key]
        dO = torch.empty_like(dQ)
        dL = torch.empty((Bn, H, Nq), dtype=torch.float32, device=dev)
        sc = float(np.float32(1.0 / np.sqrt(D)))

        def fn():
            rc = mlt.mha_fwd_raw(dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), dO.data_ptr(), dL.data_ptr(), Bn, H, Nq, Nk,
                                 D, causal, sc, sp)
            assert rc == 0, rc
        out[name] = timeit(fn, inputs.mha_flops(Bn, H, Nq, Nk, D, causal), kind="mha_fwd")
        del dO, dL
    mha_cache.clear()
    hbm_peak = measured_peaks()["hbm_gbs"]
    # memory-bound GEMM shapes (Sec. 4.1, next-token prediction): split-K through mlt_gemm_ex, reported in GB/s of
    # A, B and C each moved once
    for name, (M, N, K, kind, seed) in inputs.GEMM_DECODE_CONFIGS.items():
        if only is not None and name != only:
            continue
        A, B = inputs.gemm_inputs(M, N, K, seed=seed, kind=kind)
        dA, dB = devbits(A), devbits(B)
        dC = torch.empty((M, N), dtype=torch.int16, device=dev)
        ws = torch.empty(max(16, mlt.gemm_workspace_bytes(M, N, K)), dtype=torch.uint8, device=dev)

        def fn():
            rc = mlt.gemm_ex_raw(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, K, N, N, ws.data_ptr(), ws.numel(), sp)
            assert rc == 0, rc
        nbytes = 2.0 * (M * K + K * N + M * N)
        r = timeit(fn, inputs.gemm_flops(M, N, K), read_flush=True, kind="gemm")
        out[name] = {"ms_min": r["ms_min"], "ms_median": r["ms_median"], "gbs_best": nbytes / r["ms_min"] / 1e6,
                     "gbs_median": nbytes / r["ms_median"] / 1e6, "tflops_best": r["tflops_best"],
                     "frac_of_measured_hbm_best": nbytes / r["ms_min"] / 1e6 / hbm_peak, "launches": r["launches"],
                     "clocks": r["clocks"]}
        del dA, dB, dC, ws
    # paged-attention decode (Sec. 3.2 / 4.3): bound by HBM, reported in GB/s of visible K and V
    for name, (S, H, Hkv, D, bs, lo, hi, seed) in inputs.PAGED_CONFIGS.items():
        if only is not None and name != only:
            continue
        Q, Kc, Vc, table, lens = inputs.paged_inputs(S, H, Hkv, D, bs, seed=seed, min_len=lo, max_len=hi)
        dQ, dK, dV = devbits(Q), devbits(Kc), devbits(Vc)
        dT, dLn = torch.from_numpy(table).to(dev), torch.from_numpy(lens).to(dev)
        dO = torch.empty_like(dQ)
        dL = torch.empty((S, H), dtype=torch.float32, device=dev)
        ws = torch.empty(mlt.paged_attn_workspace_bytes(S, H, D), dtype=torch.uint8, device=dev)
        sc = float(np.float32(1.0 / np.sqrt(D)))

        def fn():
            rc = mlt.paged_attn_decode_raw(dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), dT.data_ptr(), dLn.data_ptr(),
                                           dO.data_ptr(), dL.data_ptr(), S, H, Hkv, D, bs, table.shape[1], Kc.shape[0],
                                           sc, ws.data_ptr(), ws.numel(), sp)
            assert rc == 0, rc
        nbytes = inputs.paged_bytes(lens, Hkv, D)
        r = timeit(fn, 4.0 * float(lens.sum()) * H * D, read_flush=True)
        out[name] = {"ms_min": r["ms_min"], "ms_median": r["ms_median"], "gbs_best": nbytes / r["ms_min"] / 1e6,
                     "gbs_median": nbytes / r["ms_median"] / 1e6, "kv_bytes": nbytes,
                     "frac_of_measured_hbm_best": nbytes / r["ms_min"] / 1e6 / hbm_peak, "launches": r["launches"],
                     "clocks": r["clocks"]}
        del dQ, dK, dV, dO, dL, ws
    return out


def run_sweeps(mlt, torch, dev, stream, iters: int = 20):
    """Paper-shaped sweeps (Sec. 4.1 / 4.2): compute-bound GEMM with m = 1k..16k on Llama-like (n, k), and the
    attention forward with 32k tokens in total, sequence length 1k..32k, hidden size 2048 as 32 heads of 64 or 16
    heads of 128.  Inputs come from the seeded generator, as in the parity tests of the same shapes."""
    sp = stream.cuda_stream
    flush = torch.empty(256 << 20, dtype=torch.int8, device=dev)
    rows = []

    def best_ms(fn):
        # burst timing: a pause first, because seconds of back-to-back load (the configurations before this one)
        # leave the GPU under its sustained power limit, where the same kernel runs 10-30 % slower on this pool
        torch.cuda.synchronize()
        time.sleep(0.3)
        for _ in range(3):
            fn()
        ts = []
        for _ in range(iters):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return float(np.min(ts))

    def devbits(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev)

    for (N, K) in ((4096, 4096), (14336, 4096), (4096, 14336), (8192, 8192)):
        scale = 1.0 / np.sqrt(K)
        Bm = devbits(inputs.matrix_bf16(K, N, seed=40, tensor_id=inputs.TENSOR_B, scale=scale))
        A_all = devbits(inputs.matrix_bf16(16384, K, seed=40, tensor_id=inputs.TENSOR_A, scale=scale))
        for M in (1024, 2048, 4096, 8192, 16384):
            A = A_all[:M]  # the first M rows of the same seeded matrix
            C = torch.empty(M, N, dtype=torch.int16, device=dev)

            def fn():
                rc = mlt.gemm_raw(A.data_ptr(), Bm.data_ptr(), C.data_ptr(), M, N, K, K, N, N, sp)
                assert rc == 0, rc
            ms = best_ms(fn)
            rows.append({"op": "gemm", "M": M, "N": N, "K": K, "ms": ms, "tflops": 2.0 * M * N * K / ms / 1e9})
            del A, C
        del Bm, A_all
    for D, H in ((64, 32), (128, 16)):
        for N in (1024, 2048, 4096, 8192, 16384, 32768):
            Bn = 32768 // N
            q, k, v = (devbits(t) for t in inputs.mha_inputs(Bn, H, N, N, D, seed=300 + N // 1024 + D))
            o = torch.empty_like(q)
            lse = torch.empty(Bn, H, N, dtype=torch.float32, device=dev)
            for causal in (0, 1):
                def fn():
                    rc = mlt.mha_fwd_raw(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(), Bn, H, N, N,
                                         D, causal, float(D ** -0.5), sp)
                    assert rc == 0, rc
                ms = best_ms(fn)
                rows.append({"op": "mha_fwd", "B": Bn, "H": H, "N": N, "D": D, "causal": causal, "ms": ms,
                             "tflops": inputs.mha_flops(Bn, H, N, N, D, causal) / ms / 1e9})
            del q, k, v, o, lse
    return rows


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["mlt", "reference"], default="mlt")
    ap.add_argument("--all", action="store_true", help="time every benchmark configuration on its own (the default on one GPU)")
    ap.add_argument("--no-configs", action="store_true", help="skip the per-configuration timings (\"configs\")")
    ap.add_argument("--sweep", action="store_true", help="paper-shaped GEMM and attention sweeps (one JSON line)")
    ap.add_argument("--only", default=None, help="time one named configuration alone (kernel launches only; for profiling)")
    args = ap.parse_args(argv)
    if args.sweep:
        import torch
        import paper_2503_14985_b200 as mlt
        torch.cuda.set_device(0)
        print(json.dumps({"sweep": run_sweeps(mlt, torch, torch.device("cuda", 0), torch.cuda.current_stream())}))
        return 0
    if args.only is not None:
        import torch
        import paper_2503_14985_b200 as mlt
        torch.cuda.set_device(0)
        res = time_all_configs(mlt, torch, torch.device("cuda", 0), torch.cuda.current_stream(), iters=args.steps,
                               only=args.only, warm=args.warmup)
        print(json.dumps({"only": args.only, **res.get(args.only, {"error": "unknown configuration"})}))
        return 0
    if args.warmup < 3 and args.impl == "mlt":
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)
    return run_mlt(args)


if __name__ == "__main__":
    sys.exit(main())
