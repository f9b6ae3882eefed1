"""Device-resident training state for a workload: quantized weights, scales, BF16
gradients and FP32 moments in a few large torch allocations, carved into
per-tensor views at 256-byte boundaries (the layout the kernels stream).

No arithmetic of the method lives here: the initial codes and scales come from
the library's own ``eco_quantize`` kernel.
"""
from __future__ import annotations

from typing import List, Optional

import numpy as np
import torch

from . import eco
from . import workloads as wl

_ALIGN = 256
_GUARD = 256          # bytes of guard before the first view, between views and after the last
_SENTINEL = 0xA5


def _carve(sizes_bytes: List[int]):
    """Offsets of the views inside one allocation: every view starts on a 256-byte boundary and is preceded and
    followed by at least _GUARD bytes that belong to no tensor (the guard areas, see DeviceState.check_guards)."""
    offs, total = [], _GUARD
    for b in sizes_bytes:
        offs.append(total)
        total += (b + _ALIGN - 1) // _ALIGN * _ALIGN + _GUARD
    return offs, total


def _guard_index(offs: List[int], sizes_bytes: List[int], total: int, device) -> torch.Tensor:
    """Byte positions of an allocation that lie in no view (int64 tensor on the device)."""
    starts = torch.tensor([0] + [o + b for o, b in zip(offs, sizes_bytes)], dtype=torch.int64)
    ends = torch.tensor(offs + [total], dtype=torch.int64)
    lens = ends - starts
    first = torch.repeat_interleave(starts, lens)
    within = torch.arange(int(lens.sum()), dtype=torch.int64) - torch.repeat_interleave(torch.cumsum(lens, 0) - lens, lens)
    return (first + within).to(device)


def config_of(w: wl.Workload, injection: int = eco.ECO_INJECT_ECO) -> eco.Config:
    return eco.Config(format=w.format, granularity=w.granularity, block=w.block, scale_dtype=w.scale_dtype,
                      optimizer=w.optimizer, rounding=w.rounding, injection=injection)


class DeviceState:
    """Buffers of every tensor of a workload on one CUDA device."""

    def __init__(self, w: wl.Workload, device: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("DeviceState needs a CUDA device (there is no CPU fallback)")
        self.workload = w
        self.device = device
        dev = torch.device("cuda", device)
        ts = w.tensors
        adam = w.optimizer == wl.ADAM
        sb = wl.SCALE_BYTES[w.scale_dtype]
        w_sizes, s_sizes = [w.code_bytes(t) for t in ts], [w.n_scales(t) * sb for t in ts]
        g_sizes, m_sizes = [t.numel * 2 for t in ts], [t.numel * 4 for t in ts]
        self._w_off, w_total = _carve(w_sizes)
        self._s_off, s_total = _carve(s_sizes)
        self._g_off, g_total = _carve(g_sizes)
        self._m_off, m_total = _carve(m_sizes)
        self.w_buf = torch.zeros(w_total, dtype=torch.uint8, device=dev)
        self.s_buf = torch.zeros(s_total, dtype=torch.uint8, device=dev)
        self.g_buf = torch.zeros(g_total, dtype=torch.uint8, device=dev)
        self.m_buf = torch.zeros(m_total, dtype=torch.uint8, device=dev)
        self.v_buf = torch.zeros(m_total, dtype=torch.uint8, device=dev) if adam else None
        # Guard areas: every byte of the five allocations that belongs to no tensor holds a sentinel.  A kernel that
        # stores past the end of a ragged tensor (or before its start) changes one, and check_guards() sees it.
        self._guards = []
        for buf, offs, sizes, total in ((self.w_buf, self._w_off, w_sizes, w_total), (self.s_buf, self._s_off, s_sizes, s_total),
                                        (self.g_buf, self._g_off, g_sizes, g_total), (self.m_buf, self._m_off, m_sizes, m_total),
                                        (self.v_buf, self._m_off, m_sizes, m_total)):
            if buf is None:
                continue
            idx = _guard_index(offs, sizes, total, dev)
            buf[idx] = _SENTINEL
            self._guards.append((buf, idx))
        self.tensors: List[eco.Tensor] = []
        sdt = {wl.SCALE_F32: torch.float32, wl.SCALE_BF16: torch.bfloat16, wl.SCALE_E8M0: torch.uint8}[w.scale_dtype]
        for i, t in enumerate(ts):
            cw = self.w_buf[self._w_off[i]: self._w_off[i] + w.code_bytes(t)]
            cs = self.s_buf[self._s_off[i]: self._s_off[i] + w.n_scales(t) * sb].view(sdt)
            cg = self.g_buf[self._g_off[i]: self._g_off[i] + t.numel * 2].view(torch.bfloat16)
            cm = self.m_buf[self._m_off[i]: self._m_off[i] + t.numel * 4].view(torch.float32)
            cv = self.v_buf[self._m_off[i]: self._m_off[i] + t.numel * 4].view(torch.float32) if adam else None
            self.tensors.append(eco.Tensor(cw, cs, cg, cm, cv, t.rows, t.cols, t.tensor_id))
        self.handle: Optional[int] = None

    # ---- initial state ----------------------------------------------------
    def quantize_from(self, i: int, x_f32: torch.Tensor) -> None:
        """theta_hat_0 = q_RTN(theta_0) for tensor i through the library's eco_quantize."""
        t = self.tensors[i]
        cfg = config_of(self.workload)
        cfg.rounding = eco.ECO_ROUND_NEAREST
        eco.eco_quantize(cfg, x_f32, t.rows, t.cols, t.w, t.scale, 0, 0, t.tensor_id, self.device,
                         torch.cuda.current_stream().cuda_stream)

    def init_from_host(self) -> None:
        """Seeded host weights (workloads.initial_weights) -> device -> eco_quantize."""
        for i, spec in enumerate(self.workload.tensors):
            x = torch.from_numpy(wl.initial_weights(self.workload, spec)).to(f"cuda:{self.device}")
            self.quantize_from(i, x)
        torch.cuda.synchronize(self.device)

    def init_on_device(self, seed: int = 1234) -> None:
        """Same distributions drawn by the device RNG (full-size timing runs)."""
        gen = torch.Generator(device=f"cuda:{self.device}")
        gen.manual_seed(seed)
        biggest = max(t.numel for t in self.workload.tensors)
        tmp = torch.empty(biggest, dtype=torch.float32, device=f"cuda:{self.device}")
        for i, spec in enumerate(self.workload.tensors):
            x = tmp[: spec.numel]
            x.normal_(0.0, self.workload.weight_std, generator=gen)
            self.quantize_from(i, x)
        torch.cuda.synchronize(self.device)
        del tmp

    # ---- gradients ----------------------------------------------------------
    def set_grads_from_host(self, step: int) -> None:
        for i, spec in enumerate(self.workload.tensors):
            g = wl.gradient_bf16(self.workload, spec, step)
            self.tensors[i].grad.view(torch.int16).copy_(torch.from_numpy(g.view(np.int16)), non_blocking=False)

    def set_grads_on_device(self, seed: int = 4321) -> None:
        gen = torch.Generator(device=f"cuda:{self.device}")
        gen.manual_seed(seed)
        for i, spec in enumerate(self.workload.tensors):
            if spec.zero_grad:
                self.tensors[i].grad.zero_()
            else:
                self.tensors[i].grad.normal_(0.0, self.workload.grad_std, generator=gen)
        torch.cuda.synchronize(self.device)

    # ---- stepping -------------------------------------------------------------
    def create(self, injection: int = eco.ECO_INJECT_ECO) -> int:
        self.handle = eco.eco_create(config_of(self.workload, injection), self.tensors, self.device)
        return self.handle

    def step(self, step: int, stream: Optional[int] = None, weight_decay: float = 0.0, grad_scale: float = 1.0) -> None:
        w = self.workload
        if stream is None:
            stream = torch.cuda.current_stream().cuda_stream
        if weight_decay != 0.0 or grad_scale != 1.0:
            eco.eco_step_ex(self.handle, w.lr, w.beta1, w.beta2, w.eps, step, w.step_seed, weight_decay, grad_scale, stream)
        else:
            eco.eco_step(self.handle, w.lr, w.beta1, w.beta2, w.eps, step, w.step_seed, stream)

    def destroy(self) -> None:
        if self.handle is not None:
            eco.eco_destroy(self.handle)
            self.handle = None

    def check_guards(self) -> None:
        """Raise if any byte outside the tensors' views was written since construction."""
        names = ("codes", "scales", "gradients", "m", "v")
        for name, (buf, idx) in zip(names, self._guards):
            got = buf[idx]
            if not bool((got == _SENTINEL).all()):
                bad = idx[got != _SENTINEL]
                raise AssertionError(f"guard bytes of the {name} allocation were overwritten: {bad.numel()} bytes, "
                                     f"first at offset {int(bad[0])}")

    def guard_bytes(self) -> int:
        return sum(int(idx.numel()) for _, idx in self._guards)

    def device_bytes(self) -> int:
        return sum(b.numel() for b in (self.w_buf, self.s_buf, self.g_buf, self.m_buf, self.v_buf) if b is not None)
