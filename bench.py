#!/usr/bin/env python
"""Benchmark of the attention hot path on B200.

  python bench.py --gpus N --steps K --warmup W            # the CUDA library, one rank per GPU: under a launcher
                                                           # (RANK / WORLD_SIZE set) as one of its ranks, else
                                                           # bench.py starts the N ranks itself
  python bench.py --impl reference --steps K --warmup W    # the CPU oracle, as it stands
  python bench.py --workload ubench                        # the instruction-rate probes behind roofline.joint

A step is one pass of the hot path over the full-resolution self-attention workload: B=2, H=8,
Nq=Nk=4096, d=40, fp16, once on the plain N(0,1) inputs and once on the peaked (Q x 4) inputs --
two launches of the fused kernel.  Rank 0 prints ONE JSON line.  Multi-GPU runs are weak scaling:
every rank runs the same per-GPU work on its own inputs; attention has no exchange step, so there
is no data-path collective, only a barrier and a max over ranks of the device time.
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

from paper_2304_11267_b200 import distributed as D  # noqa: E402
from paper_2304_11267_b200 import workloads  # noqa: E402

METRIC = "attention TFLOP/s (4*B*H*Nq*Nk*d FLOPs per call), 4096-token self-attention"
UNIT = "TFLOP/s"
NOMINAL_FP16_TFLOPS = 2250.0
ROTATING_SETS = 8   # 8 x 42 MB of q/k/v/out for the two variants = 336 MB, above the 126 MB L2
# DRAM bytes per launch of the fused kernel on this workload: dram__bytes_read.sum + dram__bytes_write.sum of one
# ncu capture of the kernel instance named here (profiles/fused4s_c2_self_4096_d40.md): q, k, v read once (15.73 MB
# algorithmic) and next to nothing written during the launch -- the 5.2 MB of output are still in the 126 MB L2 when
# the kernel ends.  A constant from a capture: it moves only when the capture is redone.
FUSED_TRAFFIC = {"bytes_per_launch": 15801344, "kernel_instance": "fused4s_attention_kernel<2, 1, 1, 0>(Fused4Args)",
                 "capture": "profiles/fused4s_c2_self_4096_d40.md"}
# Of every 8 exponentials of the d = 40 kernel this many go to the FMA pipe (F4S_POLY_PER8 in fused4s_kernel.cuh), and
# FMA-pipe results per score element: scale, row sum, half a pack on the special-function path; 6 more on the
# polynomial path.
POLY_PER8 = 2
FMA_OPS_SFU_PATH, FMA_OPS_POLY_EXTRA = 3.0, 6.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "tflops": float(p["bf16_tflops"]),
                "tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "tflops": 1590.0, "tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, device_index: int):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.power = [], set(), []
        self.max_mhz = None
        self._stop_evt = threading.Event()
        self.nvml = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nvml = pynvml
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nvml = None

    def sample_once(self):
        if self.nvml is None:
            return
        n = self.nvml
        try:
            self.samples.append(int(n.nvmlDeviceGetClockInfo(self.h, n.NVML_CLOCK_SM)))
            get = getattr(n, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                getattr(n, "nvmlDeviceGetCurrentClocksThrottleReasons")
            mask = int(get(self.h))
            for bit, name in self.REASONS.items():
                if mask & bit:
                    self.reasons.add(name)
            self.power.append(n.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
        except Exception:
            pass

    def reset(self):
        self.samples, self.reasons, self.power = [], set(), []

    def run(self):
        while not self._stop_evt.is_set():
            self.sample_once()
            time.sleep(0.002)

    def stop(self):
        self._stop_evt.set()
        if self.ident is not None:
            self.join(timeout=2)
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples),
                "power_w_max": max(self.power) if self.power else None}


# ------------------------------------------------------------------------------------------ oracle arm

def oracle_sample_rows(call, every):
    return np.arange(0, call.B * call.H * call.Nq, every, dtype=np.int64)


def time_oracle(calls_inputs, every, keep=None):
    """Seconds the oracle needs for every `every`-th row of each call, and the FLOPs that covers.  `keep`, a list,
    receives (rows, result) per call."""
    import oracle
    t0 = time.perf_counter()
    flops = 0
    for call, (q, k, v) in calls_inputs:
        rows = oracle_sample_rows(call, every)
        ref, _, _ = oracle.forward(q, k, v, call.scale(), rows=rows)
        if keep is not None:
            keep.append((rows, ref))
        flops += 4 * len(rows) * call.Nk * call.d
    return time.perf_counter() - t0, flops


def cpu_baseline(calls_inputs, target_s=12.0):
    """The oracle as it stands on this machine's host cores, on a bounded sample (about 10-30 s of work).

    A calibration pass over every 16th row sizes the sample: either a thinned set of rows (slow box) or
    the whole step repeated (fast box), so that the timed part lands near `target_s` seconds.
    """
    import oracle
    dt16, _ = time_oracle(calls_inputs, 16)
    full = dt16 * 16
    every = 1
    while every < 16 and full / every > 2.0 * target_s:
        every *= 2
    dt, flops, passes = 0.0, 0, 0
    refs = []
    while passes == 0 or (every == 1 and dt < 0.85 * target_s and passes < 64):   # a fast box repeats the whole step
        keep = [] if passes == 0 else None
        t, f = time_oracle(calls_inputs, every, keep)
        if keep is not None:
            refs = keep
        dt += t
        flops += f
        passes += 1
    rows = sum(len(oracle_sample_rows(c, every)) for c, _ in calls_inputs)
    total = sum(c.B * c.H * c.Nq for c, _ in calls_inputs)
    return {"value": flops / dt / 1e12, "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle",
            "sample": "%d pass(es) over every %s row of both calls of the step (%d of %d rows per pass), %.1f s" % (
                passes, "" if every == 1 else "%d-th" % every, rows, total, dt),
            "seconds": dt}, refs


def parity_numbers(got, ref, v):
    """max |gpu - oracle| / max|V| and the relative L2 error of `got` (numpy, any float type) against oracle rows."""
    got = np.asarray(got, dtype=np.float64)
    err = np.abs(got - ref)
    return {"max_err_over_maxV": float(err.max() / np.abs(np.asarray(v, dtype=np.float64)).max()),
            "rel_l2": float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300)),
            "rows": int(ref.size // ref.shape[-1])}


def run_reference(args):
    rank, _, world = D.env_world()
    if rank != 0:
        return 0
    import oracle
    if world > 1:
        # a launcher of several ranks sets OMP_NUM_THREADS=1 for each; here rank 0 alone works, on all host cores, as
        # it does without a launcher
        oracle.set_threads(len(os.sched_getaffinity(0)))
    calls = workloads.config2()
    calls_inputs = [(c, workloads.make_inputs(c)) for c in calls]
    every = 32   # each step: every 32nd row of both variants, about a third of a second on 8 cores
    for _ in range(args.warmup):
        time_oracle(calls_inputs, every)
    t0 = time.perf_counter()
    flops = 0
    for _ in range(args.steps):
        _, f = time_oracle(calls_inputs, every)
        flops += f
    dt = time.perf_counter() - t0
    value = flops / dt / 1e12
    sample = "each step: every 32nd row of both variants (%d rows of %d)" % (
        sum(len(oracle_sample_rows(c, every)) for c in calls), sum(c.B * c.H * c.Nq for c in calls))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / max(args.steps, 1),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def workload_config():
    return {"workload": "c2: self-attention B=2 H=8 Nq=Nk=4096 d=40 fp16, scale 1/sqrt(40); each step = plain N(0,1) "
                        "call + peaked (Q x 4) call",
            "l2": "inputs larger than L2: rotating through %d input/output sets (336 MB)" % ROTATING_SETS,
            "per_gpu_units": "32 (batch, head) problems per step per GPU", "parallelism": "replicated per GPU, no collective"}


# ------------------------------------------------------------------------------------------ CUDA arm

def make_sets(calls, n_sets, device, rank):
    import torch
    sets = []
    for r in range(n_sets):
        entry = []
        for c in calls:
            shifted = workloads.Call(c.name, c.B, c.H, c.Nq, c.Nk, c.d, c.config_index,
                                     call_index=c.call_index + 1000 * r + 100000 * rank, peaked=c.peaked,
                                     padded_text=c.padded_text)
            q, k, v = workloads.make_inputs(shifted)
            tq, tk, tv = (torch.from_numpy(x).to(device) for x in (q, k, v))
            entry.append((c, tq, tk, tv, torch.empty_like(tq)))
        sets.append(entry)
    return sets


def run_ours(args):
    import torch
    from paper_2304_11267_b200 import binding as bd
    rank, local_rank, world = D.init_process_group("nccl")
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback (use --impl reference for the oracle)")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    stream = torch.cuda.current_stream().cuda_stream
    if args.workload == "ubench":
        if rank == 0:
            print(json.dumps({"workload": "ubench", "rates": instruction_rates(bd, stream)}))
        return 0
    if args.workload != "c2" and not args.kernel_loop_only:
        raise SystemExit("--workload other than c2 is a profiling aid: combine it with --kernel-loop-only")
    if args.workload == "groupnorm":
        sets, gamma, beta = groupnorm_sets(device, 16)
        for i in range(max(args.warmup, 3) + args.steps):
            groupnorm_call(bd, *sets[i % 16], gamma, beta, stream)
        torch.cuda.synchronize()
        print(json.dumps({"kernel_loop_only": True, "workload": "groupnorm", "launches": max(args.warmup, 3) + args.steps}))
        return 0
    if args.workload == "winograd":
        N, H, W, C, K = WG_SHAPE
        g = torch.Generator(device=device).manual_seed(11)
        w = (torch.randn(K, 3, 3, C, device=device, generator=g) / (9.0 * C) ** 0.5).to(torch.float16)
        layer = bd.WinogradConv3x3(w, None, stream)
        xs = [torch.randn(N, H, W, C, device=device, generator=g).to(torch.float16) for _ in range(4)]
        y = torch.empty(N, H, W, K, device=device, dtype=torch.float16)
        for i in range(max(args.warmup, 3) + args.steps):
            layer(xs[i % 4], out=y, stream=stream)
        torch.cuda.synchronize()
        print(json.dumps({"kernel_loop_only": True, "workload": "winograd", "launches": 3 * (max(args.warmup, 3) + args.steps)}))
        return 0
    if args.workload == "geglu":
        sets = geglu_sets(device, 4)
        for i in range(max(args.warmup, 3) + args.steps):
            x, o = sets[i % 4]
            rc = bd.sd_geglu_forward(x.data_ptr(), o.data_ptr(), GEGLU_ROWS, GEGLU_C, bd.F16, stream)
            if rc != bd.OK:
                raise bd.SdAttnError(rc, "sd_geglu_forward")
        torch.cuda.synchronize()
        print(json.dumps({"kernel_loop_only": True, "workload": "geglu", "launches": max(args.warmup, 3) + args.steps}))
        return 0
    mode = bd.MODE_TWOPASS if args.workload == "c1-twopass" else bd.MODE_AUTO
    att = bd.Attention(mode)
    calls = {"c2": workloads.config2, "c5-cross": lambda: [workloads.config5()[2]],
             "c3-cross": workloads.config3, "c4": workloads.config4,
             "c4-d80": lambda: [c for c in workloads.config4() if c.kind == "self" and c.d == 80][:1],
             "c1": workloads.config1, "c1-twopass": workloads.config1}[args.workload]()
    sets = make_sets(calls, ROTATING_SETS, device, rank)
    if mode == bd.MODE_TWOPASS:   # the comparator borrows its scratch from the caller
        need_ws = max(bd.sd_attn_workspace_bytes(mode, c.B, c.H, c.Nq, c.Nk, c.d, bd.F16) for c in calls)
        workspace = torch.empty(need_ws, dtype=torch.uint8, device=device)
        rc = bd.sd_attn_set_workspace(att.handle, workspace.data_ptr(), need_ws)
        if rc != bd.OK:
            raise bd.SdAttnError(rc, "sd_attn_set_workspace")
    flops_per_step = sum(c.flops for c in calls)
    launches_per_step = len(calls)

    def step(i):
        for c, tq, tk, tv, to in sets[i % ROTATING_SETS]:
            rc = bd.sd_attn_forward(att.handle, tq.data_ptr(), tk.data_ptr(), tv.data_ptr(), to.data_ptr(),
                                    c.B, c.H, c.Nq, c.Nk, c.d, float(c.scale()), bd.F16, stream)
            if rc != bd.OK:
                raise bd.SdAttnError(rc, "sd_attn_forward")

    # The instruction-rate probes of roofline.joint run first: some tens of milliseconds of full load, after which the
    # GPU's clocks have left their idle state, so that a run of few steps measures what a long one does (with
    # --steps 5 --warmup 3 straight from idle the same kernel measured 98 us per launch against 86).
    rates = None if args.kernel_loop_only else instruction_rates(bd, stream)
    # every rotating input set is used at least once before the timed region (a set's first use pays for its tensor
    # maps and its first walk through the TLBs, which a run of few steps would otherwise time)
    warmup_steps = max(args.warmup, 3) if args.kernel_loop_only else max(args.warmup, ROTATING_SETS)
    # Whatever takes host time (NVML start-up, the sampler's first queries, the status read-back) happens before or
    # under the warm-up: a GPU left idle for milliseconds between warm-up and timed region runs its next launches
    # slower (measured: 95 us per launch over ten launches after 50 ms of idling, 87 straight after a synchronisation).
    sampler = ClockSampler(local_rank)
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.start()
    step(0)
    att.check(stream)
    if args.workload == "c2":
        assert att.last_mode == bd.MODE_FUSED
    for i in range(warmup_steps):
        step(i)
    launches0 = att.launch_count
    D.barrier(world)
    torch.cuda.synchronize()
    sampler.reset()      # the clock record is that of the timed region only
    start.record()
    for i in range(args.steps):
        step(i)
    end.record()
    sampler.sample_once()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    D.barrier(world)
    gpu_launches = att.launch_count - launches0
    att.check(stream)
    ms_total = D.max_over_ranks(start.elapsed_time(end), world, device)
    ms_per_step = ms_total / args.steps
    value = world * flops_per_step / (ms_per_step * 1e-3) / 1e12

    # per-launch statistics: a second, shorter loop with an event behind every launch (the events keep a launch's
    # set-up from overlapping its predecessor's tail, so this loop is not the one `value` comes from)
    stat_steps = 0 if args.kernel_loop_only else max(3, min(args.steps, 50))
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(stat_steps * launches_per_step + 1)]
    if stat_steps:
        marks[0].record()
        n = 0
        for i in range(stat_steps):
            for c, tq, tk, tv, to in sets[i % ROTATING_SETS]:
                rc = bd.sd_attn_forward(att.handle, tq.data_ptr(), tk.data_ptr(), tv.data_ptr(), to.data_ptr(),
                                        c.B, c.H, c.Nq, c.Nk, c.d, float(c.scale()), bd.F16, stream)
                if rc != bd.OK:
                    raise bd.SdAttnError(rc, "sd_attn_forward")
                n += 1
                marks[n].record()
        torch.cuda.synchronize()
        per_launch_us = np.array([1e3 * marks[i].elapsed_time(marks[i + 1]) for i in range(n)])
        # what the timed buffers hold now is the output of the LAST launch on each set
        last_step_of_set0 = max(i for i in range(stat_steps) if i % ROTATING_SETS == 0)

    if args.kernel_loop_only:
        # profiling aid: just the warm-up and the timed loop, so that a profiler sees few launches
        if rank == 0:
            print(json.dumps({"kernel_loop_only": True, "workload": args.workload, "ms_per_step": ms_per_step,
                              "launches_per_step": gpu_launches / max(args.steps, 1),
                              "tflops": value, "gbs": world * sum(c.io_bytes() for c in calls) / (ms_per_step * 1e-3) / 1e9}))
        return 0

    # --- end to end through the C ABI with host buffers (pinned), copies inside the timed region
    c0 = calls[0]
    hsets = []
    for c, tq, tk, tv, to in sets[0]:
        hq, hk, hv = (t.cpu().pin_memory() for t in (tq, tk, tv))
        hsets.append((c, hq, hk, hv, torch.empty_like(hq).pin_memory()))
    need = bd.sd_attn_host_staging_bytes(c0.B, c0.H, c0.Nq, c0.Nk, c0.d, bd.F16)
    staging = torch.empty(need, dtype=torch.uint8, device=device)
    h2d = sum(hq.numel() * 2 + hk.numel() * 2 + hv.numel() * 2 for _, hq, hk, hv, _ in hsets)
    d2h = sum(ho.numel() * 2 for *_, ho in hsets)

    def e2e_step():
        for c, hq, hk, hv, ho in hsets:
            rc = bd.sd_attn_forward_host(att.handle, hq.data_ptr(), hk.data_ptr(), hv.data_ptr(), ho.data_ptr(),
                                         staging.data_ptr(), need, c.B, c.H, c.Nq, c.Nk, c.d, float(c.scale()),
                                         bd.F16, stream)
            if rc != bd.OK:
                raise bd.SdAttnError(rc, "sd_attn_forward_host")

    e2e_steps = max(3, min(args.steps, 30))
    # The copy path reaches its steady rate much later than the kernels do (measured: 540 us per call over the first
    # 40 calls after 20 warm-up calls, 460 us from then on), so this leg warms up for longer than --warmup asks.
    for _ in range(max(args.warmup, 60)):
        e2e_step()
    D.barrier(world)
    torch.cuda.synchronize()
    start.record()
    for _ in range(e2e_steps):
        e2e_step()
    end.record()
    torch.cuda.synchronize()
    D.barrier(world)
    e2e_ms = D.max_over_ranks(start.elapsed_time(end), world, device) / e2e_steps
    e2e = {"value": world * flops_per_step / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
           "api": "sd_attn_forward_host, pinned host buffers"}
    # the step's result as a user would read it: finite and inside the hull of V
    res = hsets[0][4]
    assert torch.isfinite(res.float()).all()

    if rank != 0:
        return 0

    peaks = measured_peaks()
    # the step's only kernel is the fused one, so its mean launch duration is the timed region / launches
    per_launch_s = ms_per_step * 1e-3 / launches_per_step
    achieved = calls[0].flops / per_launch_s / 1e12
    sms = torch.cuda.get_device_properties(device).multi_processor_count
    max_mhz = float(clocks.get("sm_max_mhz") or 1965)
    roofline = {"bound": "tensor", "kernel": "fused4s_attention_kernel", "achieved": achieved,
                "peak": peaks["tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["tflops"],
                "peak_source": "%s cuBLAS bf16 burst (fp16 peak = bf16 peak, nominal ratio 1.0)" % peaks["source"],
                "frac_of_nominal_2250": achieved / NOMINAL_FP16_TFLOPS,
                "traffic": FUSED_TRAFFIC["bytes_per_launch"], "traffic_source": FUSED_TRAFFIC,
                "algorithmic_bytes": calls[0].io_bytes(), "us_per_launch": per_launch_s * 1e6,
                "us_per_launch_stats": {"median": float(np.median(per_launch_us)), "min": float(per_launch_us.min()),
                                        "mean": float(per_launch_us.mean()), "launches": int(per_launch_us.size),
                                        "how": "an event behind every launch of a second loop (no overlap of a launch's "
                                               "set-up with its predecessor), rotating inputs larger than L2"},
                "joint": joint_roofline(calls[0], per_launch_s, rates, peaks, sms, max_mhz),
                "note": "one exponential per score element: at d=40 the special-function unit and the FMA pipe, not the "
                        "tensor pipe, bound the kernel; `joint` is the bound of all units together"}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup_steps, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f16", "data": "synthetic", "config": workload_config(),
            "clocks": clocks, "e2e": e2e, "gpu_launches": gpu_launches, "roofline": roofline,
            "pct_of_fp16_dense_peak": 100.0 * value / world / NOMINAL_FP16_TFLOPS}
    if world == 1:
        # the oracle on the very inputs that were timed (set 0), and the outputs the timed launches left there
        timed_outputs = [to.cpu().numpy() for *_, to in sets[0]]
        host_inputs = [(c, tuple(t.cpu().numpy() for t in (tq, tk, tv))) for c, tq, tk, tv, _ in sets[0]]
        line["extra"] = extras(att, bd, device, stream, peaks)
        line["cpu_baseline"], refs = cpu_baseline(host_inputs)
        line["parity"] = {"what": "outputs left in the timed buffers (input set 0) against the oracle's rows of the same inputs",
                          "tolerance": "max |err| <= 2e-3 max|V|",
                          "calls": [dict(name=c.name, **parity_numbers(out.reshape(-1, c.d)[rows], ref, v))
                                    for (c, (q, k, v)), out, (rows, ref) in zip(host_inputs, timed_outputs, refs)]}
        if any(p["max_err_over_maxV"] > 2e-3 for p in line["parity"]["calls"]):
            raise RuntimeError("the timed outputs do not match the oracle: %s" % line["parity"])
    print(json.dumps(line))
    return 0


def instruction_rates(bd, stream):
    """Results per clock per SM of the instructions the softmax sweep is made of, and of the sweep itself, measured
    now (sd_attn_ubench: a few hundred microseconds each), with the SM clock that was in effect."""
    out = {}
    for name, op in bd.UBENCH_OPS.items():
        rate, mhz = bd.sd_attn_ubench(op, 4096, stream)
        out[name] = {"per_clk_per_sm": rate, "sm_mhz": mhz}
    return out


def joint_roofline(call, per_launch_s, rates, peaks, sms, max_mhz):
    """Score elements per clock per SM against the bound of all units together.

    Per element: 4 d_pad tensor FLOPs; one exponential, a share x of them on the FMA pipe; 3 + 6x FMA-pipe results
    (scale, row sum, half a pack; six more on the polynomial path).  The bound is the slowest unit's pace at the
    measured rates: min(R_ex2 / (1 - x), R_fma / (3 + 6x), R_tensor / (4 d_pad)), with R_tensor the measured GEMM peak
    per clock per SM.  `softmax_sweep_poly` is what the sweep alone reaches with 16 warps per SM (no tensor memory, no
    hand-over): the practical ceiling of this instruction mix."""
    x = POLY_PER8 / 8.0
    dpad = (call.d + 15) // 16 * 16
    elements = call.B * call.H * call.Nq * call.Nk
    r_ex2 = rates["ex2"]["per_clk_per_sm"]
    r_fma = max(rates["fma"]["per_clk_per_sm"], rates["fma_x2"]["per_clk_per_sm"])
    eff_mhz = rates["softmax_sweep_poly"]["sm_mhz"]
    out = {"unit": "score elements/clk/SM", "poly_share": x,
           "rates_per_clk_per_sm": {k: v["per_clk_per_sm"] for k, v in rates.items()},
           "formula": "min(ex2/(1-x), fma/(3+6x), tensor_flop_per_clk/(4*dpad))"}
    for label, mhz in (("at_max_clock", max_mhz), ("at_effective_clock", eff_mhz)):
        r_tensor = peaks["tflops"] * 1e12 / (sms * mhz * 1e6)            # FLOP per clock per SM at that clock
        bound = min(r_ex2 / (1.0 - x), r_fma / (FMA_OPS_SFU_PATH + FMA_OPS_POLY_EXTRA * x), r_tensor / (4.0 * dpad))
        got = elements / (per_launch_s * sms * mhz * 1e6)
        out[label] = {"sm_mhz": mhz, "achieved": got, "bound": bound, "frac": got / bound,
                      "bound_units": {"sfu": r_ex2 / (1.0 - x), "fma": r_fma / (FMA_OPS_SFU_PATH + FMA_OPS_POLY_EXTRA * x),
                                      "tensor": r_tensor / (4.0 * dpad)},
                      "frac_of_sweep_alone": got / rates["softmax_sweep_poly"]["per_clk_per_sm"]}
    out["effective_clock_note"] = "clock64 against globaltimer inside the probe kernels, read-only"
    return out


def time_calls(att, bd, tensors, stream, iters, graph=False, dtype=None):
    """Mean microseconds for one pass over `tensors` (a list of calls), rotating nothing: small extras."""
    import torch
    dtype = bd.F16 if dtype is None else dtype

    def once():
        for c, tq, tk, tv, to in tensors:
            rc = bd.sd_attn_forward(att.handle, tq.data_ptr(), tk.data_ptr(), tv.data_ptr(), to.data_ptr(),
                                    c.B, c.H, c.Nq, c.Nk, c.d, float(c.scale()), dtype, stream)
            if rc != bd.OK:
                raise bd.SdAttnError(rc, "sd_attn_forward")
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        once()
    torch.cuda.synchronize()
    if graph:
        s = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(s):
            with torch.cuda.graph(g, stream=s):
                for c, tq, tk, tv, to in tensors:
                    bd.sd_attn_forward(att.handle, tq.data_ptr(), tk.data_ptr(), tv.data_ptr(), to.data_ptr(),
                                       c.B, c.H, c.Nq, c.Nk, c.d, float(c.scale()), dtype, s.cuda_stream)
        g.replay()
        torch.cuda.synchronize()
        start.record()
        for _ in range(iters):
            g.replay()
        end.record()
    else:
        start.record()
        for _ in range(iters):
            once()
        end.record()
    torch.cuda.synchronize()
    return 1e3 * start.elapsed_time(end) / iters


def time_calls_once(att, bd, t, stream):
    c, tq, tk, tv, to = t
    rc = bd.sd_attn_forward(att.handle, tq.data_ptr(), tk.data_ptr(), tv.data_ptr(), to.data_ptr(), c.B, c.H, c.Nq, c.Nk,
                            c.d, float(c.scale()), bd.F16, stream)
    if rc != bd.OK:
        raise bd.SdAttnError(rc, "sd_attn_forward")


def time_batch(att, bd, tensors, stream, iters):
    """Mean microseconds of one sd_attn_forward_batch call over `tensors`: plain, and replayed as a CUDA graph."""
    import torch
    probs = bd.make_problems([(tq.data_ptr(), tk.data_ptr(), tv.data_ptr(), to.data_ptr(), c.B, c.H, c.Nq, c.Nk, c.d,
                               float(c.scale())) for c, tq, tk, tv, to in tensors])

    def once(s):
        rc = bd.sd_attn_forward_batch(att.handle, probs, bd.F16, s)
        if rc != bd.OK:
            raise bd.SdAttnError(rc, "sd_attn_forward_batch")
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        once(stream)
    torch.cuda.synchronize()
    n0 = att.launch_count
    start.record()
    for _ in range(iters):
        once(stream)
    end.record()
    torch.cuda.synchronize()
    time_batch.launches_per_call = (att.launch_count - n0) // iters   # counted by the library, for the bench's note
    plain = 1e3 * start.elapsed_time(end) / iters
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            once(side.cuda_stream)
    g.replay()
    torch.cuda.synchronize()
    start.record()
    for _ in range(iters):
        g.replay()
    end.record()
    torch.cuda.synchronize()
    return plain, 1e3 * start.elapsed_time(end) / iters


def time_stats(fn, iters, sync):
    """{median, min, mean} microseconds of fn(i), an event behind every call (device time per call)."""
    import torch
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
    sync()
    marks[0].record()
    for i in range(iters):
        fn(i)
        marks[i + 1].record()
    sync()
    us = np.array([1e3 * marks[i].elapsed_time(marks[i + 1]) for i in range(iters)])
    return {"median": float(np.median(us)), "min": float(us.min()), "mean": float(us.mean()), "calls": iters}


def oracle_parity(call, host, out_tensor, rows=None):
    """Parity of a timed buffer: the oracle on the same inputs (all rows, or the sample `rows`) against what the
    library left in `out_tensor`."""
    import oracle
    q, k, v = host
    ref, _, _ = oracle.forward(q, k, v, call.scale(), rows=rows)
    got = out_tensor.cpu().numpy()
    got = got.reshape(-1, call.d)[rows] if rows is not None else got
    return parity_numbers(got, ref.reshape(got.shape), v)


def config_numbers(att, bd, device, stream, peaks):
    """The workloads beside the bench's own: c1 (single-pass and two-pass), the four c3 cross shapes (as CUDA graphs),
    c5 self-attention plain and peaked with the two-pass comparator beside it -- each timed (median / min / mean of
    per-call device times) and checked against the oracle on the buffers that were timed."""
    import torch
    out = {}

    def to_dev(call):
        host = workloads.make_inputs(call)
        tq, tk, tv = (torch.from_numpy(x).to(device) for x in host)
        return host, (call, tq, tk, tv, torch.empty_like(tq))

    def fwd(a, t, strm):
        c, tq, tk, tv, to = t
        rc = bd.sd_attn_forward(a.handle, tq.data_ptr(), tk.data_ptr(), tv.data_ptr(), to.data_ptr(), c.B, c.H, c.Nq, c.Nk,
                                c.d, float(c.scale()), bd.F16, strm)
        if rc != bd.OK:
            raise bd.SdAttnError(rc, "sd_attn_forward")

    # --- c1: the smallest instance, single-pass and the two-pass comparator of Sec. 3.2.1
    c1 = workloads.config1()[0]
    host, t = to_dev(c1)
    for _ in range(5):
        fwd(att, t, stream)
    entry = {"fused_us_back_to_back": time_calls(att, bd, [t], stream, 100),
             "fused_us": time_stats(lambda i: fwd(att, t, stream), 50, torch.cuda.synchronize),
             "note": "back_to_back: mean of a loop of launches, each one's set-up under its predecessor's tail; the "
                     "statistics: an event behind every call, so every call pays its whole launch"}
    att.check(stream)
    entry["fused_parity"] = oracle_parity(c1, host, t[4])
    tp = bd.Attention(bd.MODE_TWOPASS)
    need = bd.sd_attn_workspace_bytes(bd.MODE_TWOPASS, c1.B, c1.H, c1.Nq, c1.Nk, c1.d, bd.F16)
    ws = torch.empty(need, dtype=torch.uint8, device=device)
    bd.sd_attn_set_workspace(tp.handle, ws.data_ptr(), need)
    for _ in range(3):
        fwd(tp, t, stream)
    entry["twopass_us_back_to_back"] = time_calls(tp, bd, [t], stream, 40)
    entry["twopass_us"] = time_stats(lambda i: fwd(tp, t, stream), 20, torch.cuda.synchronize)
    tp.check(stream)
    entry["twopass_parity"] = oracle_parity(c1, host, t[4])
    entry["twopass_scratch_bytes"] = need
    entry["tflops_fused"] = c1.flops / (entry["fused_us_back_to_back"] * 1e-6) / 1e12
    out["c1_self_1024_d40"] = entry
    del ws

    # --- c3: the four cross-attention shapes, each as a CUDA graph of 8 back-to-back calls (microseconds per call)
    c3 = {}
    for c in workloads.config3():
        host, t = to_dev(c)
        fwd(att, t, stream)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for _ in range(8):
                fwd(att, t, side.cuda_stream)
        g.replay()
        st = time_stats(lambda i: g.replay(), 20, torch.cuda.synchronize)
        att.check(stream)
        c3[c.name] = {"us_per_call": {k: (v / 8 if k != "calls" else v * 8) for k, v in st.items()},
                      "achieved_gbs": c.io_bytes() / (st["median"] / 8 * 1e-6) / 1e9,
                      "parity": oracle_parity(c, host, t[4])}
    out["c3_cross_set"] = c3

    # --- c5: 9216 tokens, plain and peaked; the single-pass kernel and the two-pass comparator that materialises the
    # 9216 x 9216 score matrix (10.9 GB of binary32 scratch)
    c5 = {}
    g = np.random.default_rng(5)
    need = 0
    for c in workloads.config5()[:2]:
        need = max(need, bd.sd_attn_workspace_bytes(bd.MODE_TWOPASS, c.B, c.H, c.Nq, c.Nk, c.d, bd.F16))
    ws = torch.empty(need, dtype=torch.uint8, device=device)
    bd.sd_attn_set_workspace(tp.handle, ws.data_ptr(), need)
    for c in workloads.config5()[:2]:
        host, t = to_dev(c)
        other = (c, torch.randn_like(t[1]), torch.randn_like(t[2]), torch.randn_like(t[3]), torch.empty_like(t[4]))
        pair = [t, other]     # two sets of 94 MB each: rotating inputs larger than the L2
        rows = np.sort(g.choice(c.B * c.H * c.Nq, size=512, replace=False)).astype(np.int64)
        for i in range(3):
            fwd(att, pair[i % 2], stream)
        e = {"fused_us": time_stats(lambda i: fwd(att, pair[i % 2], stream), 8, torch.cuda.synchronize)}
        att.check(stream)
        e["fused_parity"] = oracle_parity(c, host, t[4], rows)
        e["tflops_fused"] = c.flops / (e["fused_us"]["median"] * 1e-6) / 1e12
        fwd(tp, t, stream)
        e["twopass_us"] = time_stats(lambda i: fwd(tp, t, stream), 3, torch.cuda.synchronize)
        tp.check(stream)
        e["twopass_parity"] = oracle_parity(c, host, t[4], rows)
        e["twopass_over_fused"] = e["twopass_us"]["median"] / e["fused_us"]["median"]
        c5[c.name] = e
        del pair, other, t
    c5["twopass_scratch_bytes"] = need
    c5["parity_rows"] = "512 seeded random rows of each call"
    out["c5_self_9216_d40"] = c5
    tp.close()
    del ws
    torch.cuda.empty_cache()
    return out


def extras(att, bd, device, stream, peaks):
    """Secondary numbers: the other workloads, the UNet-step attention set (32 calls), the memory-bound
    cross-attention, layouts and dtypes, and the three steps beside the attention path."""
    import torch
    out = config_numbers(att, bd, device, stream, peaks)
    calls = workloads.config4()
    tensors = []
    for c in calls:
        q, k, v = workloads.make_inputs(c)
        tq, tk, tv = (torch.from_numpy(x).to(device) for x in (q, k, v))
        tensors.append((c, tq, tk, tv, torch.empty_like(tq)))
    flops = sum(c.flops for c in calls)
    us = time_calls(att, bd, tensors, stream, 20)
    us_graph = time_calls(att, bd, tensors, stream, 20, graph=True)
    us_batch, us_batch_graph = time_batch(att, bd, tensors, stream, 20)
    out["unet_step_attention_set"] = {"calls": len(calls), "us_plain_launches": us, "us_cuda_graph": us_graph,
                                      "tflops_cuda_graph": flops / (us_graph * 1e-6) / 1e12,
                                      "us_batch_call": us_batch, "us_batch_call_cuda_graph": us_batch_graph,
                                      "tflops_batch_call_cuda_graph": flops / (us_batch_graph * 1e-6) / 1e12,
                                      "batch_launches": time_batch.launches_per_call,
                                      "batch_note": "the same 32 calls as independent problems of one "
                                                    "sd_attn_forward_batch call: one launch per shape "
                                                    "(batch_launches, counted by the library) over four streams",
                                      "note": "512x512, B=2, H=8: 16 self + 16 cross calls (L2-warm: 285 MB of tensors)"}
    # cross-attention at the large-latent size, rotating sets so that Q/O stream from HBM
    c = workloads.config5()[2]
    n_sets = 8     # 8 x 47.6 MB
    csets = []
    for r in range(n_sets):
        q, k, v = workloads.make_inputs(workloads.Call(c.name, c.B, c.H, c.Nq, c.Nk, c.d, c.config_index,
                                                       call_index=c.call_index + 10 * r, padded_text=True))
        tq, tk, tv = (torch.from_numpy(x).to(device) for x in (q, k, v))
        csets.append((c, tq, tk, tv, torch.empty_like(tq)))
    us_cross = time_calls(att, bd, csets, stream, 10) / n_sets
    gbs = c.io_bytes() / (us_cross * 1e-6) / 1e9
    cross_stats = time_stats(lambda i: time_calls_once(att, bd, csets[i % n_sets], stream), 24, torch.cuda.synchronize)
    att.check(stream)
    q0, k0, v0 = workloads.make_inputs(workloads.Call(c.name, c.B, c.H, c.Nq, c.Nk, c.d, c.config_index,
                                                      call_index=c.call_index, padded_text=True))
    rows = np.arange(0, c.B * c.H * c.Nq, 37, dtype=np.int64)
    out["cross_attention_9216x77_d40"] = {"us_per_call": us_cross, "us_per_call_with_an_event_behind_each": cross_stats,
                                          "achieved_gbs": gbs, "bound": "hbm",
                                          "peak_gbs": peaks["hbm_gbs"], "frac": gbs / peaks["hbm_gbs"],
                                          "frac_of_nominal_8000": gbs / 8000.0,
                                          "algorithmic_bytes": c.io_bytes(), "peak_source": peaks["source"],
                                          "parity": oracle_parity(c, (q0, k0, v0), csets[0][4], rows)}
    # four times the batch (B = 16): the same kernel with four times the items per CTA, so that ramp and pace show apart
    c4x = workloads.Call(c.name + "_4x_batch", 4 * c.B, c.H, c.Nq, c.Nk, c.d, c.config_index, call_index=c.call_index,
                         padded_text=True)
    bsets4 = []
    for r in range(2):     # 2 x 190 MB
        tq = torch.randn(c4x.B, c4x.H, c4x.Nq, c4x.d, device=device, dtype=torch.float16)
        tk = torch.randn(c4x.B, c4x.H, c4x.Nk, c4x.d, device=device, dtype=torch.float16)
        bsets4.append((c4x, tq, tk, torch.randn_like(tk), torch.empty_like(tq)))
    for i in range(3):
        time_calls_once(att, bd, bsets4[i % 2], stream)
    st4 = time_stats(lambda i: time_calls_once(att, bd, bsets4[i % 2], stream), 10, torch.cuda.synchronize)
    us4_b2b = time_calls(att, bd, bsets4, stream, 10) / 2    # back to back, as us_per_call above is measured
    att.check(stream)
    gbs4 = c4x.io_bytes() / (st4["median"] * 1e-6) / 1e9
    gbs4_b2b = c4x.io_bytes() / (us4_b2b * 1e-6) / 1e9
    out["cross_attention_9216x77_d40"]["at_4x_batch"] = {"us_per_call": st4, "achieved_gbs": gbs4,
                                                         "frac": gbs4 / peaks["hbm_gbs"], "bytes": c4x.io_bytes(),
                                                         "us_per_call_back_to_back": us4_b2b,
                                                         "achieved_gbs_back_to_back": gbs4_b2b,
                                                         "frac_back_to_back": gbs4_b2b / peaks["hbm_gbs"]}
    del bsets4
    # the same two measurements with the tensors read as token-major [B][N][H][d] (the head split and merge around
    # the attention as views): the same buffers, so the same bytes and the same sizes
    att_t = bd.Attention(layout=bd.LAYOUT_BNHD)
    us_graph_t = time_calls(att_t, bd, tensors, stream, 20, graph=True)
    us_cross_t = time_calls(att_t, bd, csets, stream, 10) / n_sets
    att_t.check(stream)
    att_t.close()
    out["token_major_layout"] = {"unet_step_attention_set_us_cuda_graph": us_graph_t,
                                 "cross_attention_9216x77_d40_us_per_call": us_cross_t,
                                 "note": "sd_attn_set_layout(SD_ATTN_LAYOUT_BNHD); compare with the two entries above"}
    # the bench's own shape with bfloat16 tensors: the same kernel with the other operand format
    c2 = workloads.config2()[0]
    bsets = []
    for r in range(8):     # 8 x 21 MB: larger than L2
        tq, tk, tv = (torch.randn(c2.B, c2.H, n, c2.d, device=device, dtype=torch.float32).to(torch.bfloat16)
                      for n in (c2.Nq, c2.Nk, c2.Nk))
        bsets.append((c2, tq, tk, tv, torch.empty_like(tq)))
    us_bf16 = time_calls(att, bd, bsets, stream, 5, dtype=bd.BF16) / len(bsets)
    att.check(stream)
    out["bf16_self_attention_4096_d40"] = {"us_per_call": us_bf16, "tflops": c2.flops / (us_bf16 * 1e-6) / 1e12,
                                           "note": "dtype SD_ATTN_BF16, rotating through 8 sets (168 MB)"}
    del bsets
    out["winograd_conv3x3_2x64x64x320_f16"] = winograd_numbers(bd, device, stream, peaks)
    out["geglu_8192x1280_f16"] = geglu_numbers(bd, device, stream, peaks)
    out["groupnorm_2x320x64x64_f16"] = groupnorm_numbers(bd, device, stream, peaks)
    return out


WG_SHAPE = (2, 64, 64, 320, 320)      # N, H, W, C, K: a 3x3 convolution of the UNet's 64 x 64 level at 512 x 512, batch 2


def winograd_numbers(bd, device, stream, peaks):
    """The Winograd 3x3 convolution (Sec. 3.3) on one UNet layer shape: microseconds per call (input transform, 36
    GEMMs, output transform), the rate in terms of the direct convolution's FLOPs, and the oracle on a sample."""
    import torch
    import oracle
    N, H, W, C, K = WG_SHAPE
    g = torch.Generator(device=device).manual_seed(11)
    w = (torch.randn(K, 3, 3, C, device=device, generator=g) / (9.0 * C) ** 0.5).to(torch.float16)
    b = (0.1 * torch.randn(K, device=device, generator=g)).to(torch.float16)
    layer = bd.WinogradConv3x3(w, b, stream)
    n_sets = 16       # 16 x (5.2 MB in + 5.2 MB out): with the 7.4 MB filter and 35 MB of scratch, more than the L2
    xs = [torch.randn(N, H, W, C, device=device, generator=g).to(torch.float16) for _ in range(n_sets)]
    ys = [torch.empty(N, H, W, K, device=device, dtype=torch.float16) for _ in range(n_sets)]
    for i in range(4):
        layer(xs[i], out=ys[i], stream=stream)
    torch.cuda.synchronize()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    iters = 48
    start.record()
    for i in range(iters):
        layer(xs[i % n_sets], out=ys[i % n_sets], stream=stream)
    end.record()
    torch.cuda.synchronize()
    rc, detail = bd.sd_winograd_query_status(stream)
    if rc != bd.OK:
        raise bd.SdAttnError(rc, "winograd device status %s" % detail)
    us = 1e3 * start.elapsed_time(end) / iters
    direct_flops = 2.0 * N * H * W * K * C * 9
    tiles = N * ((H + 3) // 4) * ((W + 3) // 4)
    gemm_flops = 2.0 * 36 * tiles * K * C
    io_bytes = 2.0 * (N * H * W * C + N * H * W * K + 36 * K * C)
    # the oracle, timed on the first rows of the first image (a few seconds of CPU work)
    hs, ws_ = 9, 64
    x0 = xs[0][:1, :hs + 1].cpu().numpy()
    t0 = time.perf_counter()
    ref = oracle.conv3x3_forward(x0, w.cpu().numpy(), b.cpu().numpy())[:, :hs]
    cpu_s = time.perf_counter() - t0
    got = ys[0][:1, :hs].cpu().numpy().astype("float64")
    rel = float(((got - ref) ** 2).sum() ** 0.5 / ((ref ** 2).sum() ** 0.5))
    # the same layer at 16 times the batch: enough tiles for many waves of GEMM CTAs (the rate of the kernels
    # themselves, where the UNet's own shape is a chain of three short kernels)
    NB = 16 * N
    xb = torch.randn(NB, H, W, C, device=device, generator=g).to(torch.float16)
    yb = torch.empty(NB, H, W, K, device=device, dtype=torch.float16)
    for _ in range(2):
        layer(xb, out=yb, stream=stream)
    torch.cuda.synchronize()
    start.record()
    for _ in range(5):
        layer(xb, out=yb, stream=stream)
    end.record()
    torch.cuda.synchronize()
    us_b = 1e3 * start.elapsed_time(end) / 5
    del xb, yb
    return {"us_per_call": us, "launches_per_call": 3,
            "at_16x_batch": {"us_per_call": us_b, "direct_conv_tflops_equivalent": 16 * direct_flops / (us_b * 1e-6) / 1e12,
                             "gemm_tflops": 16 * gemm_flops / (us_b * 1e-6) / 1e12},
            "direct_conv_tflops_equivalent": direct_flops / (us * 1e-6) / 1e12,
            "gemm_tflops": gemm_flops / (us * 1e-6) / 1e12,
            "bound": "hbm", "algorithmic_bytes": io_bytes, "achieved_gbs": io_bytes / (us * 1e-6) / 1e9,
            "peak_gbs": peaks["hbm_gbs"], "frac": io_bytes / (us * 1e-6) / 1e9 / peaks["hbm_gbs"],
            "peak_source": peaks["source"],
            "note": "x + y + transformed filter are the algorithmic bytes; V and M (35 MB) go through the L2",
            "rel_l2_vs_oracle_on_sample": rel,
            "cpu_oracle_gflops": 2.0 * 1 * (hs + 1) * ws_ * K * C * 9 / cpu_s / 1e9,
            "cpu_oracle_sample": "%d of %d rows of one image" % (hs + 1, H)}


GN_SHAPE, GN_GROUPS, GN_EPS = (2, 320, 64, 64), 32, 1e-5      # the 64 x 64 level of the UNet at 512 x 512, batch 2


def groupnorm_sets(device, n_sets, shape=GN_SHAPE):
    import torch
    g = torch.Generator(device="cpu").manual_seed(20230422)
    C = shape[1]
    gamma = (1.0 + 0.3 * torch.randn(C, generator=g)).to(torch.float16).to(device)
    beta = (0.2 * torch.randn(C, generator=g)).to(torch.float16).to(device)
    sets = []
    for _ in range(n_sets):
        x = (torch.randn(shape, generator=g, dtype=torch.float32) * 1.7 + 0.4).to(torch.float16).to(device)
        sets.append((x, torch.empty_like(x)))
    return sets, gamma, beta


def groupnorm_call(bd, x, o, gamma, beta, stream):
    N, C = x.shape[0], x.shape[1]
    rc = bd.sd_groupnorm_forward(x.data_ptr(), gamma.data_ptr(), beta.data_ptr(), o.data_ptr(), N, C,
                                 x.numel() // (N * C), GN_GROUPS, GN_EPS, bd.F16, stream)
    if rc != bd.OK:
        raise bd.SdAttnError(rc, "sd_groupnorm_forward")


def groupnorm_numbers(bd, device, stream, peaks):
    """The fused group normalisation (Eq. 1) at its largest UNet shape: HBM roofline, with the oracle timed beside it."""
    import torch
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(sets, gamma, beta, iters):
        for i in range(len(sets) + 3):
            groupnorm_call(bd, *sets[i % len(sets)], gamma, beta, stream)
        torch.cuda.synchronize()
        start.record()
        for i in range(iters):
            groupnorm_call(bd, *sets[i % len(sets)], gamma, beta, stream)
        end.record()
        torch.cuda.synchronize()
        return 1e3 * start.elapsed_time(end) / iters

    n_sets = 16                          # 16 x 10.5 MB: rotating inputs larger than the L2
    sets, gamma, beta = groupnorm_sets(device, n_sets)
    algo = 4 * sets[0][0].numel()        # 2 bytes read + 2 written per element
    us_eager = timed(sets, gamma, beta, 64)
    # a 10 MB call is shorter than the host's time to enqueue it: the device's time is that of a graph replay
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for x, o in sets:
            groupnorm_call(bd, x, o, gamma, beta, side.cuda_stream)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    start.record()
    for _ in range(10):
        graph.replay()
    end.record()
    torch.cuda.synchronize()
    us = 1e3 * start.elapsed_time(end) / (10 * n_sets)
    gbs = algo / (us * 1e-6) / 1e9
    import oracle
    xs = sets[0][0].cpu().numpy()
    ga, be = gamma.cpu().numpy(), beta.cpu().numpy()
    oracle.groupnorm_forward(xs[:1, :, :2], GN_GROUPS, GN_EPS, ga, be)
    t0 = time.perf_counter()
    oracle.groupnorm_forward(xs, GN_GROUPS, GN_EPS, ga, be)
    cpu_s = time.perf_counter() - t0
    del sets
    # sixteen times the batch: 1024 (sample, group) blocks instead of 64
    big, gamma, beta = groupnorm_sets(device, 2, shape=(32,) + GN_SHAPE[1:])
    us_big = timed(big, gamma, beta, 10)
    big_gbs = 16 * algo / (us_big * 1e-6) / 1e9
    return {"us_per_call": us, "us_per_call_eager": us_eager, "achieved_gbs": gbs, "bound": "hbm",
            "peak_gbs": peaks["hbm_gbs"], "frac": gbs / peaks["hbm_gbs"], "algorithmic_bytes": algo,
            "peak_source": peaks["source"],
            "l2": "rotating through 16 input/output sets (168 MB), timed as a CUDA graph of the 16 calls",
            "at_16x_batch": {"achieved_gbs": big_gbs, "frac": big_gbs / peaks["hbm_gbs"], "bytes": 16 * algo},
            "cpu_oracle_gbs": algo / cpu_s / 1e9, "cpu_oracle_sample": "the whole tensor"}


GEGLU_ROWS, GEGLU_C = 8192, 1280      # the feed-forward block of the 4096-token layers at 512 x 512, batch 2


def geglu_sets(device, n_sets):
    import torch
    g = torch.Generator(device="cpu").manual_seed(20230421)
    sets = []
    for _ in range(n_sets):
        x = (torch.randn((GEGLU_ROWS, 2 * GEGLU_C), generator=g, dtype=torch.float32) * 1.5).to(torch.float16).to(device)
        sets.append((x, torch.empty((GEGLU_ROWS, GEGLU_C), dtype=torch.float16, device=device)))
    return sets


def geglu_numbers(bd, device, stream, peaks):
    """The fused GEGLU step (Eq. 2) at its largest UNet shape: HBM roofline, with the oracle timed beside it."""
    import torch
    n_sets = 4                          # 4 x 63 MB: rotating inputs larger than the L2
    sets = geglu_sets(device, n_sets)
    algo = 6 * GEGLU_ROWS * GEGLU_C     # 4 bytes read + 2 written per output element
    def once(i):
        x, o = sets[i % n_sets]
        rc = bd.sd_geglu_forward(x.data_ptr(), o.data_ptr(), GEGLU_ROWS, GEGLU_C, bd.F16, stream)
        if rc != bd.OK:
            raise bd.SdAttnError(rc, "sd_geglu_forward")
    for i in range(8):
        once(i)
    torch.cuda.synchronize()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    iters = 40
    start.record()
    for i in range(iters):
        once(i)
    end.record()
    torch.cuda.synchronize()
    us = 1e3 * start.elapsed_time(end) / iters
    gbs = algo / (us * 1e-6) / 1e9
    # the oracle on a row sample of the same tensor
    import oracle
    xs = sets[0][0][:1024].cpu().numpy()
    oracle.geglu_forward(xs[:8])
    t0 = time.perf_counter()
    oracle.geglu_forward(xs)
    cpu_s = time.perf_counter() - t0
    # the same kernel on sixteen times the rows: the rate it settles at once launch and ramp no longer count
    big_rows = 16 * GEGLU_ROWS
    xb = torch.randn((big_rows, 2 * GEGLU_C), device=device, dtype=torch.float16)
    ob = torch.empty((big_rows, GEGLU_C), device=device, dtype=torch.float16)
    for _ in range(3):
        bd.sd_geglu_forward(xb.data_ptr(), ob.data_ptr(), big_rows, GEGLU_C, bd.F16, stream)
    torch.cuda.synchronize()
    start.record()
    for _ in range(10):
        bd.sd_geglu_forward(xb.data_ptr(), ob.data_ptr(), big_rows, GEGLU_C, bd.F16, stream)
    end.record()
    torch.cuda.synchronize()
    big_gbs = 16 * algo / (1e3 * start.elapsed_time(end) / 10 * 1e-6) / 1e9
    del xb, ob
    return {"us_per_call": us, "achieved_gbs": gbs, "bound": "hbm", "peak_gbs": peaks["hbm_gbs"],
            "frac": gbs / peaks["hbm_gbs"], "algorithmic_bytes": algo, "peak_source": peaks["source"],
            "l2": "rotating through 4 input/output sets (252 MB)",
            "at_16x_rows": {"achieved_gbs": big_gbs, "frac": big_gbs / peaks["hbm_gbs"], "bytes": 16 * algo},
            "cpu_oracle_gbs": 6 * xs.shape[0] * GEGLU_C / cpu_s / 1e9, "cpu_oracle_sample": "1024 of 8192 rows"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2", choices=["c2", "c5-cross", "c3-cross", "c4", "c4-d80", "c1", "c1-twopass", "geglu", "groupnorm", "winograd", "ubench"],
                    help="with --kernel-loop-only: which calls the loop runs (the bench line is always c2)")
    ap.add_argument("--kernel-loop-only", action="store_true",
                    help="run only the warm-up and the timed loop (for ncu captures)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if D.launched_by_a_launcher():
        world = int(os.environ["WORLD_SIZE"])
        if world != args.gpus:
            raise SystemExit("--gpus %d but the launcher started %d ranks" % (args.gpus, world))
        return run_ours(args)
    if args.gpus > 1:
        # no launcher: start the ranks here, one process per GPU (NCCL only for the barrier and the max of the times)
        import torch
        if torch.cuda.device_count() < args.gpus:
            raise SystemExit("--gpus %d but this node shows %d CUDA devices" % (args.gpus, torch.cuda.device_count()))
        os.environ.setdefault("NCCL_DEBUG", "INFO")     # the communicator lines go to stderr
        D.spawn_ranks(args.gpus, run_ours, (args,))
        return 0
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
