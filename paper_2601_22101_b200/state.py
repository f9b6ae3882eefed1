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


def _carve(sizes_bytes: List[int]):
    offs, total = [], 0
    for b in sizes_bytes:
        offs.append(total)
        total += (b + _ALIGN - 1) // _ALIGN * _ALIGN
    return offs, max(total, _ALIGN)


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
        self._w_off, w_total = _carve([w.code_bytes(t) for t in ts])
        self._s_off, s_total = _carve([w.n_scales(t) * sb for t in ts])
        self._g_off, g_total = _carve([t.numel * 2 for t in ts])
        self._m_off, m_total = _carve([t.numel * 4 for t in ts])
        self.w_buf = torch.zeros(w_total, dtype=torch.uint8, device=dev)
        self.s_buf = torch.zeros(s_total, dtype=torch.uint8, device=dev)
        self.g_buf = torch.zeros(g_total, dtype=torch.uint8, device=dev)
        self.m_buf = torch.zeros(m_total, dtype=torch.uint8, device=dev)
        self.v_buf = torch.zeros(m_total, dtype=torch.uint8, device=dev) if adam else None
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

    def device_bytes(self) -> int:
        return sum(b.numel() for b in (self.w_buf, self.s_buf, self.g_buf, self.m_buf, self.v_buf) if b is not None)
