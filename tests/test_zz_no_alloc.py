"""eco_step_static: the per-tensor-scale step for callers that are not allowed to allocate device memory
(a framework that already owns the whole GPU through its own pool, a loop that cannot take the stall an
allocation causes, a host that bans allocation after start-up).  The entry point keeps its tables and
reduction slots in a fixed array inside the library image instead of the cudaMalloc'd tables of
eco_create, so its results must be the very bits eco_create + eco_step produce.  Checked here on two
calls in a row, because the second call finds the first call's leftovers in the shared array.

This file sorts last on purpose: a run that stops at the first failure has then already run everything else."""
import numpy as np
import pytest
import torch

from paper_2601_22101_b200 import eco, workloads as wl
from paper_2601_22101_b200.state import DeviceState, config_of

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-6, 1e-7      # the tolerance of the parity tests for the FP32 moments


def _workload(opt, fmt, shapes):
    ts = [wl.TensorSpec(f"t{i}", r, c, 900 + 3 * i) for i, (r, c) in enumerate(shapes)]
    return wl.Workload("no_alloc", fmt, wl.PER_TENSOR, 128, wl.SCALE_F32, opt, wl.SR, lr=1e-3, beta1=0.9, beta2=0.95,
                       eps=1e-8, weight_std=0.02, grad_std=1e-3, steps=2, step_seed=0x5EED, tensors=ts)


@pytest.mark.parametrize("opt,fmt", [(wl.ADAM, wl.FP8_E4M3), (wl.SGDM, wl.INT4)])
def test_static_entry_matches_context_entry_on_two_calls_in_a_row(opt, fmt):
    shapes = [(64, 1024), (3, 200), (1, 2), (33, 4224), (7, 130)]
    w = _workload(opt, fmt, shapes)
    ref = DeviceState(w)
    ref.init_from_host()
    ref.create()
    new = DeviceState(w)
    new.init_from_host()
    cfg = config_of(w)
    stream = torch.cuda.current_stream().cuda_stream
    try:
        for step in (1, 2):
            ref.set_grads_from_host(step)
            new.set_grads_from_host(step)
            ref.step(step)
            eco.eco_step_static(cfg, new.tensors, w.lr, w.beta1, w.beta2, w.eps, step, w.step_seed, 0, stream)
            torch.cuda.synchronize()
            for a, b in zip(ref.tensors, new.tensors):
                assert torch.equal(a.w, b.w), f"codes differ at step {step}"
                assert torch.equal(a.scale.view(torch.int32), b.scale.view(torch.int32)), f"scales differ at step {step}"
                np.testing.assert_allclose(b.m.cpu().numpy(), a.m.cpu().numpy(), rtol=RTOL, atol=ATOL)
                if a.v is not None:
                    np.testing.assert_allclose(b.v.cpu().numpy(), a.v.cpu().numpy(), rtol=RTOL, atol=ATOL)
    finally:
        ref.destroy()


def test_static_entry_rejects_what_does_not_fit():
    w = _workload(wl.ADAM, wl.FP8_E4M3, [(2, 128)])
    st = DeviceState(w)
    cfg = config_of(w)
    too_many = [eco.Tensor(t.w, t.scale, t.grad, t.m, t.v, t.rows, t.cols, i) for i, t in enumerate(st.tensors * 65)]
    with pytest.raises(eco.EcoError) as e:
        eco.eco_step_static(cfg, too_many, 1e-3, 0.9, 0.95, 1e-8, 1, 0)
    assert e.value.status == eco.ECO_ERR_INVALID_ARG and "at most 64 tensors" in str(e.value)
    t = st.tensors[0]
    huge = [eco.Tensor(t.w, t.scale, t.grad, t.m, t.v, 1 << 15, 1 << 13, 0)]      # 2^28 parameters: never launched
    with pytest.raises(eco.EcoError) as e:
        eco.eco_step_static(cfg, huge, 1e-3, 0.9, 0.95, 1e-8, 1, 0)
    assert e.value.status == eco.ECO_ERR_INVALID_ARG and "parameters per call" in str(e.value)
    block_cfg = config_of(wl.c2())
    with pytest.raises(eco.EcoError) as e:
        eco.eco_step_static(block_cfg, st.tensors, 1e-3, 0.9, 0.95, 1e-8, 1, 0)
    assert e.value.status == eco.ECO_ERR_UNSUPPORTED
