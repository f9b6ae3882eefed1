#!/usr/bin/env python
"""Benchmark of the ECO optimizer step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4] [--impl reference]

One "step" is one eco_step over every tensor of the workload's parameter set (the whole hot path:
dequantize, optimizer update, amax/scale, requantize with stochastic rounding, error injection, stores).
Prints ONE JSON line.  `value` = parameters updated per second with the state resident in HBM, timed
with CUDA events on the launching stream: blocks of exactly --steps steps, each bracketed by a barrier and
a synchronize, repeated until at least --min-seconds have been timed so that the GPU reaches the clock its
power cap allows; `value` is the MEDIAN block, the first block is reported beside it.  The default workload
is the largest of the benchmark sets that fits one GPU (c5, 15.5 B parameters); the other sets of a billion
parameters or more are timed after it and `roofline.min_frac_1b_plus` is the smallest of their fractions.
`e2e` = the same metric through eco_host_step with the state in pinned HOST memory (copies inside the
timed region).  With torchrun (N > 1) every rank steps its own
replica of the parameter set (no data-path collective exists in this method) and the time is the max
over ranks.  `--impl reference` times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "eco_optimizer_step_params_per_sec"
UNIT = "params/s"
FALLBACK_HBM_GBS = 6650.0
# the benchmark sets of a billion parameters or more, as configured
BIG_SETS = ("c3_gemma3_1b_fp8_tensor_adam_sr", "c4_smoe_2mat_fp8_block128_adam_sr", "c5_deepseek_moe16b_int4_group128_sgdm_sr")

PROFILE_SOURCES = ("eco_stream_kernels.cu", "eco_device.cuh", "eco_index.h")


def _kernel_sources_digest() -> str:
    """SHA-256 over the code (comments and white space stripped) of the sources the streaming kernels are built from:
    an ncu summary carries the digest of the sources it was captured on, and its counters are not quoted once they
    have changed."""
    import hashlib
    import re
    h = hashlib.sha256()
    for name in PROFILE_SOURCES:
        with open(os.path.join(ROOT, "paper_2601_22101_b200", "csrc", name), "r") as f:
            text = f.read()
        # the code only: comments and layout do not change a kernel (no string literal in these files holds "//")
        text = re.sub(r"//[^\n]*", "", text)
        h.update(" ".join(text.split()).encode())
    return h.hexdigest()


def _ncu_dram_bytes_per_param():
    """DRAM bytes per parameter (dram__bytes_read.sum + dram__bytes_write.sum over a launch, divided by its
    parameters) of every streaming-kernel instantiation that has a tracked ncu summary, read from the summaries at
    run time: {"<template arguments>": B/param}.  A summary whose source digest differs from the current sources is
    skipped (the kernel changed since the counters were taken)."""
    import glob
    import re
    out = {}
    digest = _kernel_sources_digest()
    for path in sorted(glob.glob(os.path.join(ROOT, "profiles", "eco_stream_kernel_*.md"))):
        text = open(path).read()
        m = re.search(r"kernel sources sha256: ([0-9a-f]{64})", text)
        if not m or m.group(1) != digest:
            continue
        for sec in text.split("\n## ")[1:]:
            name = sec.split("\n", 1)[0].strip()
            k = re.match(r"eco_stream_kernel<([0-9, ]+)>", name)
            v = re.search(r"derived: DRAM bytes per parameter \| ([0-9.]+) B", sec)
            if k and v:
                out.setdefault(k.group(1).replace(" ", ""), []).append(float(v.group(1)))
    return {k: sum(v) / len(v) for k, v in out.items()}


def _workload(name: str):
    from paper_2601_22101_b200 import workloads as wl
    return wl.BY_NAME[name]()


def _dominant_kernel(w):
    """(readable name, template arguments of its launches) of the kernel that moves most of a step's bytes: full-size
    sets are made of whole 128-element rows, which the persistent TMA-fed kernel takes.  Per-tensor scales are a
    pair of launches (amax pass, apply pass)."""
    from paper_2601_22101_b200 import workloads as wl
    fmt = {wl.FP8_E4M3: "fp8", wl.INT4: "int4", wl.FP8_E5M2: "e5m2"}[w.format]
    fi = {wl.FP8_E4M3: 0, wl.INT4: 1, wl.FP8_E5M2: 2}[w.format]
    opt = "adam" if w.optimizer == wl.ADAM else "sgdm"
    oi = 1 if w.optimizer == wl.ADAM else 0
    rnd = "sr" if w.rounding == wl.SR else "rtn"
    ri = 1 if w.rounding == wl.SR else 0
    mode = {wl.PER_BLOCK: "block" if w.block == 128 else "block32", wl.PER_TENSOR: "tensor_apply", wl.PER_ROW: "row"}[w.granularity]
    if w.granularity == wl.PER_TENSOR:
        args = [f"{fi},{oi},0,1,0", f"{fi},{oi},{ri},2,0"]
    else:
        mi = {"block": 0, "row": 3, "block32": 4}[mode]
        args = [f"{fi},{oi},{ri},{mi},0"]
    return f"eco_stream_kernel<{fmt},{opt},{rnd},{mode}>", args


def _two_pass_note(w, params, ms_per_step, peak):
    """Per-tensor scales need max|theta~| over a whole tensor before any element can be rounded, so a tensor
    larger than the on-chip memories is read twice: the kernels move 11 + 11 + 9 = 31 B/param (FP8 + Adam)
    where the method needs 20.  Reported beside the algorithmic figure so that both are visible."""
    from paper_2601_22101_b200 import workloads as wl
    if w.granularity != wl.PER_TENSOR:
        return {}
    code = 0.5 if w.format == wl.INT4 else 1.0
    moments = 4.0 * (2 if w.optimizer == wl.ADAM else 1)
    moved = 2 * (code + 2.0 + moments) + (code + moments)
    gbs = params * moved / (ms_per_step * 1e-3) / 1e9
    return {"two_pass_bytes_per_param": moved, "two_pass_achieved": gbs, "two_pass_frac": gbs / peak}


def _measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._ok = False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self._ok = True
        except Exception:
            self._ok = False

    def _loop(self):
        nv = self.nv
        names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
                 0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, n in names.items():
                    if r & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self._ok:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread:
            self._stop.set()
            self._thread.join()
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


def cpu_baseline(w, budget_s: float = 15.0):
    """The oracle as it stands, single thread, on a bounded sample of the workload."""
    import numpy as np
    from paper_2601_22101_b200 import workloads as wl
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from oracle_runner import OracleState
    # sample: the first tensors of the set up to ~4 M parameters, rows capped at 1024
    picked, total = [], 0
    for t in w.tensors:
        from dataclasses import replace
        t2 = replace(t, rows=min(t.rows, 1024))
        picked.append(t2)
        total += t2.numel
        if total >= 4_000_000:
            break
    from dataclasses import replace as _r
    ws = _r(w, tensors=picked)
    ora = OracleState(ws, threads=1)
    grads = [wl.gradient_bf16(ws, t, 1) for t in ws.tensors]
    ora.step(1, grads)                      # warm-up (page faults, library load)
    t0 = time.perf_counter()
    steps = 0
    while True:
        steps += 1
        ora.step(1 + steps, grads)
        el = time.perf_counter() - t0
        if el > budget_s or steps >= 50:
            break
    return {"value": ws.numel * steps / el, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{len(picked)} tensors of {w.name} (rows capped at 1024), {ws.numel} params x {steps} steps, "
                      f"{el:.1f} s single-threaded"}, ws.numel * steps, el


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = _workload(args.workload)
    import numpy as np
    from dataclasses import replace
    from paper_2601_22101_b200 import workloads as wl
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from oracle_runner import OracleState
    picked, total = [], 0
    for t in w.tensors:
        t2 = replace(t, rows=min(t.rows, 1024))
        picked.append(t2)
        total += t2.numel
        if total >= 4_000_000:
            break
    ws = replace(w, tensors=picked)
    ora = OracleState(ws, threads=1)
    grads = [wl.gradient_bf16(ws, t, 1) for t in ws.tensors]
    for s in range(args.warmup):
        ora.step(1 + s, grads)
    t0 = time.perf_counter()
    for s in range(args.steps):
        ora.step(1 + args.warmup + s, grads)
    el = time.perf_counter() - t0
    value = ws.numel * args.steps / el
    sample = (f"{len(picked)} tensors of {w.name} (rows capped at 1024), {ws.numel} params per step, "
              f"single-threaded CPU oracle")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": el / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "params": w.numel, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def run_e2e(w, device: int, steps: int, max_host_gb: float):
    """eco_host_step on pinned host buffers: every step copies codes/scales/grads/moments to the device, runs the
    kernels and copies codes/scales/moments back (all inside the timed region)."""
    import torch
    from dataclasses import replace
    from paper_2601_22101_b200 import eco, workloads as wl
    from paper_2601_22101_b200.state import config_of
    adam = w.optimizer == wl.ADAM
    per_param = (0.5 if w.format == wl.INT4 else 1.0) + 2 + (8 if adam else 4)
    picked, total = [], 0
    for t in w.tensors:
        if (total + t.numel) * per_param > max_host_gb * 2 ** 30 and picked:
            break
        picked.append(t)
        total += t.numel
    ws = replace(w, tensors=picked)
    sdt = {wl.SCALE_F32: torch.float32, wl.SCALE_BF16: torch.bfloat16, wl.SCALE_E8M0: torch.uint8}[w.scale_dtype]
    # the state lives in one pinned host buffer per kind (codes, scales, gradients, m, v), tensors back to back, as an
    # offloaded optimizer keeps it; eco_host_step then moves each kind of a chunk in one copy
    sb = wl.SCALE_BYTES[w.scale_dtype]
    n_code = sum(ws.code_bytes(t) for t in ws.tensors)
    n_scale = sum(ws.n_scales(t) for t in ws.tensors)
    flat_w = torch.empty(n_code, dtype=torch.uint8, pin_memory=True).random_(0, 120)
    flat_s = torch.empty(n_scale * sb, dtype=torch.uint8, pin_memory=True)
    flat_g = torch.empty(total, dtype=torch.bfloat16, pin_memory=True)
    flat_m = torch.zeros(total, dtype=torch.float32, pin_memory=True)
    flat_v = torch.zeros(total, dtype=torch.float32, pin_memory=True) if adam else None
    if w.scale_dtype == wl.SCALE_E8M0:
        flat_s.fill_(114)                               # 2^-13
    else:
        flat_s.view(sdt).fill_(1e-4)
    tensors = []
    ow = os_ = oe = 0
    for t in ws.tensors:
        cw = flat_w[ow: ow + ws.code_bytes(t)]
        cs = flat_s[os_: os_ + ws.n_scales(t) * sb].view(sdt)
        cg = flat_g[oe: oe + t.numel]
        cg.copy_(torch.randn(t.numel, dtype=torch.float32).mul_(w.grad_std).to(torch.bfloat16))
        cm = flat_m[oe: oe + t.numel]
        cv = flat_v[oe: oe + t.numel] if adam else None
        tensors.append(eco.Tensor(cw, cs, cg, cm, cv, t.rows, t.cols, t.tensor_id))
        ow += ws.code_bytes(t)
        os_ += ws.n_scales(t) * sb
        oe += t.numel
    cfg = config_of(ws)
    up = down = 0
    handle = eco.eco_host_create(cfg, tensors, device)
    n_in, n_out = eco.eco_host_copies(handle)
    eco.eco_host_step(handle, w.lr, w.beta1, w.beta2, w.eps, 1, w.step_seed)   # warm-up
    torch.cuda.synchronize(device)
    t0 = time.perf_counter()
    for s in range(steps):
        up, down = eco.eco_host_step(handle, w.lr, w.beta1, w.beta2, w.eps, 2 + s, w.step_seed)
    torch.cuda.synchronize(device)
    el = time.perf_counter() - t0
    eco.eco_host_destroy(handle)
    return {"value": ws.numel * steps / el, "unit": UNIT, "h2d_bytes_per_step": up, "d2h_bytes_per_step": down,
            "h2d_copies_per_step": n_in, "d2h_copies_per_step": n_out,
            "steps": steps, "params_per_step": ws.numel, "seconds": el,
            "sample": f"first {len(picked)} of {len(w.tensors)} tensors per GPU ({ws.numel / w.numel:.1%} of the parameters) "
                      f"held in pinned host memory"}


def time_dequantize(peak_gbs: float, reps: int = 20):
    """x^ = s * y of Sec. 3.1 (what the forward pass of quantized training reads every step): eco_dequantize on 256 Mi
    elements, codes and outputs much larger than L2, CUDA events around `reps` calls after 3 warm-up calls."""
    import torch
    from paper_2601_22101_b200 import eco
    rows, cols = 16384, 16384
    n = rows * cols
    out_rows = []
    st = torch.cuda.current_stream().cuda_stream
    for name, fmt, block, sdt, sd in (("fp8_e4m3_block128_f32_scales", eco.ECO_FORMAT_FP8_E4M3, 128, eco.ECO_SCALE_F32, torch.float32),
                                      ("int4_group128_bf16_scales", eco.ECO_FORMAT_INT4, 128, eco.ECO_SCALE_BF16, torch.bfloat16)):
        cfg = eco.Config(format=fmt, granularity=eco.ECO_SCALE_PER_BLOCK, block=block, scale_dtype=sdt)
        cb = n // 2 if fmt == eco.ECO_FORMAT_INT4 else n
        gen = torch.Generator(device="cuda").manual_seed(7)
        w = torch.randint(0, 120, (cb,), dtype=torch.uint8, device="cuda", generator=gen)
        s = torch.full((rows * (cols // block),), 1e-3, dtype=sd, device="cuda")
        out = torch.empty(n, dtype=torch.bfloat16, device="cuda")
        for _ in range(3):
            eco.eco_dequantize(cfg, w, s, rows, cols, out, stream=st)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            eco.eco_dequantize(cfg, w, s, rows, cols, out, stream=st)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        nbytes = cb + s.numel() * s.element_size() + 2 * n
        gbs = nbytes / ms / 1e6
        out_rows.append({"layout": name, "output": "bf16", "elements": n, "ms": ms, "achieved": gbs, "unit": "GB/s",
                         "frac": gbs / peak_gbs, "bytes": nbytes})
        del w, s, out
    torch.cuda.empty_cache()
    return out_rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c5", choices=["c3f", "c3fs", "c1", "c2", "c3", "c4", "c5", "c3r", "c5t", "c4g", "c4d", "c3s", "c3rs", "c4s", "c5s", "c4mx", "c4mxs", "c4ds"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--min-seconds", type=float, default=2.0, help="blocks of --steps steps are repeated until this much has been timed")
    ap.add_argument("--also", default="c3,c4,c4d,c2,c1", help="comma-separated workloads timed after the headline one and "
                    "reported under other_workloads (device-resident timing only)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-dequantize", action="store_true", help="skip the timing of eco_dequantize (1 GPU only)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--e2e-host-gb", type=float, default=24.0, help="pinned host memory the end-to-end leg may hold; the "
                    "leg runs on the first tensors of the set that fit and says which fraction that was")
    ap.add_argument("--option", action="append", default=[], help="name=value passed to eco_set_option")
    args = ap.parse_args()

    if args.impl == "reference":
        run_reference(args)       # every step is a bounded sample (about 4 M parameters, 0.15 s on one core)
        return

    import torch
    import torch.distributed as dist
    from paper_2601_22101_b200 import eco, workloads as wl
    from paper_2601_22101_b200.state import DeviceState

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the ECO step has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    for o in args.option:
        k, v = o.split("=")
        eco.eco_set_option(k, int(v))

    ncu_bpp = _ncu_dram_bytes_per_param()

    def time_workload(w_global, steps, warmup, min_seconds):
        """Device-resident timing of this rank's shard: blocks of `steps` eco_steps, each bracketed by a barrier and a
        synchronize and timed with CUDA events on the launching stream (max over ranks), repeated until min_seconds
        have been timed.  Returns a dict (rank 0) or None."""
        w_rank = wl.shard(wl.replicate(w_global, world), rank, world) if world > 1 else w_global
        st = DeviceState(w_rank, local)
        st.init_on_device(seed=1234 + rank)
        st.set_grads_on_device(seed=4321 + rank)
        st.create()
        launches_per_step = eco.eco_num_launches(st.handle)
        step_no = 0
        for _ in range(max(warmup, 3)):
            step_no += 1
            st.step(step_no, stream.cuda_stream)
        barrier()
        sampler = ClockSampler(local)
        sampler.start()
        blocks, total_ms = [], 0.0
        while True:
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record(stream)
            for _ in range(steps):
                step_no += 1
                st.step(step_no, stream.cuda_stream)
            ev1.record(stream)
            barrier()
            ms = ev0.elapsed_time(ev1)
            if world > 1:
                t = torch.tensor([ms], device="cuda", dtype=torch.float64)
                dist.all_reduce(t, op=dist.ReduceOp.MAX)
                ms = float(t.item())
            blocks.append(ms / steps)
            total_ms += ms
            if total_ms >= min_seconds * 1e3 or len(blocks) >= 200:     # same decision on every rank (ms is reduced)
                break
        clocks = sampler.stop()
        eco.eco_check(st.handle, stream.cuda_stream)
        state_bytes = st.device_bytes()
        st.destroy()
        del st
        torch.cuda.empty_cache()
        if rank != 0:
            return None
        ms_per_step = sorted(blocks)[len(blocks) // 2]
        peak, peak_src = _measured_peak()
        bpp = w_global.algorithmic_bytes_per_param()
        params_per_rank = w_rank.numel
        gbs = lambda ms: params_per_rank * bpp / (ms * 1e-3) / 1e9
        achieved = gbs(ms_per_step)
        kern, targs = _dominant_kernel(w_global)
        tr = sum(ncu_bpp[a] for a in targs) if all(a in ncu_bpp for a in targs) else None
        mhz = clocks.get("sm_mhz") if clocks else None
        return {
            "workload": w_global.name, "params_per_gpu": params_per_rank, "tensors_per_gpu": len(w_rank.tensors),
            "ms_per_step": ms_per_step, "value": params_per_rank * world / (ms_per_step * 1e-3),
            "blocks": len(blocks), "steps_per_block": steps, "timed_seconds": total_ms * 1e-3,
            "first_block": {"ms_per_step": blocks[0], "value": params_per_rank * world / (blocks[0] * 1e-3),
                            "frac": gbs(blocks[0]) / peak},
            "ms_per_step_x_sm_mhz": (ms_per_step * mhz if mhz else None),
            "launches_per_step": launches_per_step, "state_bytes_on_device": state_bytes, "clocks": clocks,
            "roofline": {"bound": "hbm", "kernel": kern, "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "peak_source": peak_src,
                         "frac_of_nominal_8000": achieved / 8000.0,
                         "algorithmic_bytes_per_param": bpp,
                         "traffic": (tr * params_per_rank if tr else None),
                         "traffic_source": ("ncu DRAM bytes per parameter of this kernel on the small capture case "
                                            "(profiles/), times the parameters of a full launch" if tr else
                                            "no ncu summary taken on the current kernel sources"),
                         **_two_pass_note(w_global, params_per_rank, ms_per_step, peak)},
        }

    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    w = _workload(args.workload)
    head = time_workload(w, args.steps, args.warmup, args.min_seconds)
    others = []
    for name in [n for n in args.also.split(",") if n and n != args.workload]:
        r = time_workload(_workload(name), args.steps, 3, args.min_seconds)
        if r is not None:
            others.append({k: r[k] for k in ("workload", "params_per_gpu", "ms_per_step", "value", "blocks", "first_block",
                                             "ms_per_step_x_sm_mhz", "launches_per_step", "clocks", "roofline")})

    if rank == 0:
        # the benchmark sets of a billion parameters or more, as configured (c3, c4, c5): the smallest fraction of the roofline
        big = [r for r in [head] + others if r["workload"] in BIG_SETS]
        roof = dict(head["roofline"])
        if big:
            worst = min(big, key=lambda r: r["roofline"]["frac"])
            roof["min_frac_1b_plus"] = worst["roofline"]["frac"]
            roof["min_frac_1b_plus_workload"] = worst["workload"]
            roof["fracs_1b_plus"] = {r["workload"]: r["roofline"]["frac"] for r in big}
        out = {
            "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": head["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "params_per_gpu": head["params_per_gpu"],
                       "tensors_per_gpu": head["tensors_per_gpu"],
                       "state_bytes_on_device": head["state_bytes_on_device"],
                       "timing": f"blocks of {args.steps} steps (barrier + synchronize on both sides, CUDA events on the "
                                 f"launching stream) repeated until {args.min_seconds} s were timed; value = median block",
                       "l2": "inputs much larger than the 126 MB L2, streamed once per step (no flush needed)",
                       "sharding": "whole tensors per rank, no data-path collective" if world > 1 else "single GPU"},
            "blocks": head["blocks"], "timed_seconds": head["timed_seconds"], "first_block": head["first_block"],
            "ms_per_step_x_sm_mhz": head["ms_per_step_x_sm_mhz"],
            "gpu_launches": head["launches_per_step"] * args.steps * head["blocks"],
            "clocks": head["clocks"],
            "roofline": roof,
            "other_workloads": others,
        }
    if rank == 0 and world == 1 and not args.no_dequantize:
        out["dequantize"] = time_dequantize(out["roofline"]["peak"])
    if not args.no_e2e:
        # every rank steps its own host-resident shard; the job's time is the slowest rank's
        barrier()
        e2e = run_e2e(w, local, args.e2e_steps, args.e2e_host_gb)
        if world > 1:
            t = torch.tensor([e2e["seconds"]], device="cuda", dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e2e["seconds"] = float(t.item())
            e2e["value"] = e2e["params_per_step"] * world * e2e["steps"] / e2e["seconds"]
        if rank == 0:
            out["e2e"] = e2e
    if rank == 0:
        if not args.no_cpu_baseline and world == 1:
            out["cpu_baseline"], _, _ = cpu_baseline(w)
        print(json.dumps(out))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
