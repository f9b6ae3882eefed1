"""Test helper: the oracle's side of a workload (numpy buffers + chained steps).
Imports only ``oracle`` and the seeded input generators."""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from typing import List, Optional

import numpy as np

import oracle
from paper_2601_22101_b200 import workloads as wl


def oracle_config(w: wl.Workload, injection: int = oracle.INJECT_ECO) -> oracle.Config:
    # the enumerations of the boundary and of the oracle agree by value
    return oracle.Config(format=w.format, granularity=w.granularity, block=w.block,
                         scale_dtype={wl.SCALE_F32: oracle.SCALE_NATIVE, wl.SCALE_BF16: oracle.SCALE_BF16,
                                      wl.SCALE_E8M0: oracle.SCALE_E8M0}[w.scale_dtype],
                         optimizer=w.optimizer, rounding=w.rounding, injection=injection,
                         grad_dtype=oracle.GRAD_BF16)


class OracleState:
    def __init__(self, w: wl.Workload, injection: int = oracle.INJECT_ECO, threads: int = 8,
                 weights: Optional[List[np.ndarray]] = None):
        self.workload = w
        self.cfg = oracle_config(w, injection)
        self.threads = threads
        init_cfg = oracle_config(w)
        init_cfg.rounding = oracle.RTN
        self.w, self.scale, self.m, self.v = [], [], [], []
        for i, t in enumerate(w.tensors):
            x = weights[i] if weights is not None else wl.initial_weights(w, t)
            cw, cs = oracle.quantize(init_cfg, x.reshape(t.rows, t.cols))
            self.w.append(cw)
            self.scale.append(cs)
            self.m.append(np.zeros(t.numel, np.float32))
            self.v.append(np.zeros(t.numel, np.float32) if w.optimizer == wl.ADAM else None)
        # the quantization error of the last step per tensor (read back by the exact injection of Appendix A)
        self.e = [np.zeros(t.numel, np.float32) for t in w.tensors]

    def step(self, step: int, grads: Optional[List[np.ndarray]] = None, weight_decay: float = 0.0,
             grad_scale: float = 1.0) -> None:
        w = self.workload

        def one(i):
            t = w.tensors[i]
            g = grads[i] if grads is not None else wl.gradient_bf16(w, t, step)
            if weight_decay == 0.0 and grad_scale == 1.0:
                ideal = self.cfg.injection == oracle.INJECT_IDEAL
                err = None if ideal else self.e[i]
                oracle.step(self.cfg, lr=float(np.float32(w.lr)), beta1=float(np.float32(w.beta1)),
                            beta2=float(np.float32(w.beta2)), eps=float(np.float32(w.eps)), step=step,
                            seed=w.step_seed, w=self.w[i], scale=self.scale[i], grad=g, m=self.m[i], v=self.v[i],
                            rows=t.rows, cols=t.cols, tensor_id=t.tensor_id, e_prev=self.e[i] if ideal else None, dbg_err=err)
                return
            oracle.step(self.cfg, lr=float(np.float32(w.lr)), beta1=float(np.float32(w.beta1)),
                        beta2=float(np.float32(w.beta2)), eps=float(np.float32(w.eps)), step=step,
                        seed=w.step_seed, w=self.w[i], scale=self.scale[i], grad=g, m=self.m[i], v=self.v[i],
                        rows=t.rows, cols=t.cols, tensor_id=t.tensor_id,
                        weight_decay=float(np.float32(weight_decay)), grad_scale=float(np.float32(grad_scale)))

        order = sorted(range(len(w.tensors)), key=lambda i: -w.tensors[i].numel)
        if self.threads > 1 and len(order) > 1:
            with ThreadPoolExecutor(self.threads) as ex:
                list(ex.map(one, order))
        else:
            for i in order:
                one(i)
