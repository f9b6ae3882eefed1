"""Thin Python binding of the C-ABI in ``include/eco.h``: argument marshalling only.

Every step of the ECO update runs in the CUDA kernels of ``libeco_b200.so``;
PyTorch is used for device memory and streams.  There is no CPU fallback: if
the shared library is missing or no CUDA device is present the calls raise.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libeco_b200.so")

# enum values of include/eco.h
ECO_OK = 0
ECO_ERR_INVALID_ARG, ECO_ERR_UNSUPPORTED, ECO_ERR_ALIGNMENT, ECO_ERR_CUDA, ECO_ERR_NOMEM, ECO_ERR_TIMEOUT = 1, 2, 3, 4, 5, 6
ECO_FORMAT_FP8_E4M3, ECO_FORMAT_INT4, ECO_FORMAT_FP8_E5M2 = 0, 1, 4
ECO_SCALE_PER_TENSOR, ECO_SCALE_PER_ROW, ECO_SCALE_PER_BLOCK = 0, 1, 2
ECO_SCALE_F32, ECO_SCALE_BF16, ECO_SCALE_E8M0 = 0, 1, 2
ECO_OPT_SGDM, ECO_OPT_ADAM = 0, 1
ECO_ROUND_NEAREST, ECO_ROUND_STOCHASTIC = 0, 1
ECO_INJECT_NONE, ECO_INJECT_ECO, ECO_INJECT_EXACT = 0, 1, 2

EXPORTED = ("eco_create", "eco_step", "eco_step_ex", "eco_step_begin", "eco_amax_buffer", "eco_step_end", "eco_step_host", "eco_host_create", "eco_host_step", "eco_host_copies", "eco_host_destroy",
            "eco_step_static", "eco_check", "eco_attach_error_buffers", "eco_selftest_wait", "eco_selftest_grid_wait", "eco_destroy", "eco_last_error", "eco_quantize", "eco_dequantize",
            "eco_set_option", "eco_num_launches", "eco_version")


class EcoError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"eco status {status}: {message}")
        self.status = status


class eco_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("format", "granularity", "block", "scale_dtype", "optimizer",
                                              "rounding", "injection", "reserved")]


class eco_hyper(ctypes.Structure):
    _fields_ = [("lr", ctypes.c_float), ("beta1", ctypes.c_float), ("beta2", ctypes.c_float), ("eps", ctypes.c_float),
                ("weight_decay", ctypes.c_float), ("grad_scale", ctypes.c_float),
                ("step", ctypes.c_uint64), ("seed", ctypes.c_uint64), ("reserved", ctypes.c_uint64)]


class eco_tensor(ctypes.Structure):
    _fields_ = [("w", ctypes.c_void_p), ("scale", ctypes.c_void_p), ("grad", ctypes.c_void_p),
                ("m", ctypes.c_void_p), ("v", ctypes.c_void_p),
                ("rows", ctypes.c_int64), ("cols", ctypes.c_int64),
                ("tensor_id", ctypes.c_uint32), ("row_offset", ctypes.c_uint32)]


_lib = None


def load_library() -> ctypes.CDLL:
    """Load ``libeco_b200.so`` (built in-tree by ``build.py``).  Fails loudly if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            # not built yet: compile it now if nvcc is available; there is no other implementation to fall back to
            try:
                from . import build as _build
                _build.build()
            except Exception as exc:
                raise ImportError(f"{_LIB_PATH} is missing and could not be built ({exc}): run "
                                  "`python -m paper_2601_22101_b200.build` (there is no CPU fallback)") from exc
        L = ctypes.CDLL(_LIB_PATH)
        vp, u64, u32, i64, f32 = ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int64, ctypes.c_float
        L.eco_create.restype = ctypes.c_int
        L.eco_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(eco_config), ctypes.POINTER(eco_tensor),
                                 ctypes.c_size_t, ctypes.c_int]
        L.eco_step.restype = ctypes.c_int
        L.eco_step.argtypes = [vp, f32, f32, f32, f32, u64, u64, vp]
        L.eco_step_ex.restype = ctypes.c_int
        L.eco_step_ex.argtypes = [vp, ctypes.POINTER(eco_hyper), vp]
        L.eco_step_begin.restype = ctypes.c_int
        L.eco_step_begin.argtypes = [vp, ctypes.POINTER(eco_hyper), vp]
        L.eco_amax_buffer.restype = ctypes.c_int
        L.eco_amax_buffer.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(ctypes.c_size_t)]
        L.eco_step_end.restype = ctypes.c_int
        L.eco_step_end.argtypes = [vp, vp]
        L.eco_step_host.restype = ctypes.c_int
        L.eco_step_host.argtypes = [ctypes.POINTER(eco_config), ctypes.POINTER(eco_tensor), ctypes.c_size_t,
                                    ctypes.c_int, f32, f32, f32, f32, u64, u64,
                                    ctypes.POINTER(u64), ctypes.POINTER(u64)]
        L.eco_host_create.restype = ctypes.c_int
        L.eco_host_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(eco_config), ctypes.POINTER(eco_tensor),
                                      ctypes.c_size_t, ctypes.c_int]
        L.eco_host_step.restype = ctypes.c_int
        L.eco_host_step.argtypes = [vp, f32, f32, f32, f32, u64, u64, ctypes.POINTER(u64), ctypes.POINTER(u64)]
        L.eco_host_copies.restype = ctypes.c_int
        L.eco_host_copies.argtypes = [vp, ctypes.POINTER(u64), ctypes.POINTER(u64)]
        L.eco_host_destroy.restype = ctypes.c_int
        L.eco_host_destroy.argtypes = [vp]
        L.eco_step_static.restype = ctypes.c_int
        L.eco_step_static.argtypes = [ctypes.POINTER(eco_config), ctypes.POINTER(eco_tensor), ctypes.c_size_t,
                                      ctypes.c_int, f32, f32, f32, f32, u64, u64, vp]
        L.eco_check.restype = ctypes.c_int
        L.eco_check.argtypes = [vp, vp]
        L.eco_attach_error_buffers.restype = ctypes.c_int
        L.eco_attach_error_buffers.argtypes = [vp, ctypes.POINTER(vp), ctypes.c_size_t]
        L.eco_selftest_wait.restype = ctypes.c_int
        L.eco_selftest_wait.argtypes = [vp, i64, vp]
        L.eco_selftest_grid_wait.restype = ctypes.c_int
        L.eco_selftest_grid_wait.argtypes = [vp, i64, vp]
        L.eco_destroy.restype = ctypes.c_int
        L.eco_destroy.argtypes = [vp]
        L.eco_last_error.restype = ctypes.c_char_p
        L.eco_last_error.argtypes = [vp]
        L.eco_quantize.restype = ctypes.c_int
        L.eco_quantize.argtypes = [ctypes.POINTER(eco_config), vp, i64, i64, vp, vp, u64, u64, u32, ctypes.c_int, vp]
        L.eco_dequantize.restype = ctypes.c_int
        L.eco_dequantize.argtypes = [ctypes.POINTER(eco_config), vp, vp, i64, i64, vp, ctypes.c_int, ctypes.c_int, vp]
        L.eco_set_option.restype = ctypes.c_int
        L.eco_set_option.argtypes = [ctypes.c_char_p, i64]
        L.eco_num_launches.restype = ctypes.c_int
        L.eco_num_launches.argtypes = [vp]
        L.eco_version.restype = ctypes.c_char_p
        _lib = L
    return _lib


@dataclass
class Config:
    format: int = ECO_FORMAT_FP8_E4M3
    granularity: int = ECO_SCALE_PER_BLOCK
    block: int = 128
    scale_dtype: int = ECO_SCALE_F32
    optimizer: int = ECO_OPT_ADAM
    rounding: int = ECO_ROUND_STOCHASTIC
    injection: int = ECO_INJECT_ECO

    def c(self) -> eco_config:
        return eco_config(self.format, self.granularity, self.block, self.scale_dtype, self.optimizer,
                          self.rounding, self.injection, 0)


@dataclass
class Tensor:
    """Device buffers of one parameter (torch CUDA tensors) or, for ``eco_step_host``, host
    buffers (torch CPU tensors or numpy arrays)."""
    w: object
    scale: object
    grad: object
    m: object
    v: Optional[object]
    rows: int
    cols: int
    tensor_id: int
    row_offset: int = 0


def _addr(x) -> Optional[int]:
    if x is None:
        return None
    if hasattr(x, "data_ptr"):
        assert x.is_contiguous(), "buffers must be contiguous"
        return x.data_ptr()
    return x.ctypes.data   # numpy


def _raise(status: int, handle=None):
    msg = load_library().eco_last_error(handle)
    raise EcoError(status, msg.decode() if msg else "")


def _tensor_array(tensors: Sequence[Tensor]):
    arr = (eco_tensor * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = eco_tensor(_addr(t.w), _addr(t.scale), _addr(t.grad), _addr(t.m), _addr(t.v),
                            t.rows, t.cols, t.tensor_id, t.row_offset)
    return arr


def eco_create(cfg: Config, tensors: Sequence[Tensor], device: int = 0) -> int:
    """Bind a tensor list; returns the context handle.  See ``eco_create`` in include/eco.h."""
    L = load_library()
    handle = ctypes.c_void_p()
    c = cfg.c()
    arr = _tensor_array(tensors)
    st = L.eco_create(ctypes.byref(handle), ctypes.byref(c), arr, len(tensors), device)
    if st != ECO_OK:
        _raise(st)
    return handle.value


def eco_step(handle: int, lr: float, beta1: float, beta2: float, eps: float, step: int, seed: int,
             stream: int = 0) -> None:
    """Enqueue one ECO step on ``stream`` (a raw cudaStream_t).  See ``eco_step`` in include/eco.h."""
    st = load_library().eco_step(handle, lr, beta1, beta2, eps, step, seed, stream)
    if st != ECO_OK:
        _raise(st, handle)


def eco_step_ex(handle: int, lr: float, beta1: float, beta2: float, eps: float, step: int, seed: int,
                weight_decay: float = 0.0, grad_scale: float = 1.0, stream: int = 0) -> None:
    """eco_step with decoupled weight decay and a factor on the gradient.  See ``eco_step_ex`` in include/eco.h."""
    h = eco_hyper(lr, beta1, beta2, eps, weight_decay, grad_scale, step, seed, 0)
    st = load_library().eco_step_ex(handle, ctypes.byref(h), stream)
    if st != ECO_OK:
        _raise(st, handle)


def eco_step_begin(handle: int, lr: float, beta1: float, beta2: float, eps: float, step: int, seed: int,
                   weight_decay: float = 0.0, grad_scale: float = 1.0, stream: int = 0) -> None:
    """Pass 1 of a per-tensor-scale step (max|theta~| per tensor).  See ``eco_step_begin`` in include/eco.h."""
    h = eco_hyper(lr, beta1, beta2, eps, weight_decay, grad_scale, step, seed, 0)
    st = load_library().eco_step_begin(handle, ctypes.byref(h), stream)
    if st != ECO_OK:
        _raise(st, handle)


class _DeviceWords:
    """A view of n 32-bit words of device memory that torch can wrap without copying."""

    def __init__(self, ptr: int, n: int):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": "<i4", "data": (ptr, False), "version": 2}


def eco_amax_tensor(handle: int, device: int = 0):
    """The context's amax vector as a torch int32 CUDA tensor aliasing the library's memory (bit patterns of
    non-negative floats: their integer order is their float order).  Reduce it with MAX across ranks in place
    between ``eco_step_begin`` and ``eco_step_end``."""
    import torch
    ptr, n = ctypes.c_void_p(), ctypes.c_size_t()
    st = load_library().eco_amax_buffer(handle, ctypes.byref(ptr), ctypes.byref(n))
    if st != ECO_OK:
        _raise(st, handle)
    return torch.as_tensor(_DeviceWords(ptr.value, n.value), device=torch.device("cuda", device))


def eco_step_end(handle: int, stream: int = 0) -> None:
    """Pass 2 of a per-tensor-scale step.  See ``eco_step_end`` in include/eco.h."""
    st = load_library().eco_step_end(handle, stream)
    if st != ECO_OK:
        _raise(st, handle)


def eco_step_sharded(handle: int, lr: float, beta1: float, beta2: float, eps: float, step: int, seed: int,
                     weight_decay: float = 0.0, grad_scale: float = 1.0, group=None, device: int = 0) -> None:
    """One per-tensor-scale step of a context that holds ROW SHARDS of tensors whose other rows live on other
    ranks of ``group`` (torch.distributed, NCCL): pass 1, one all-reduce(MAX) of the amax vector, pass 2.
    Argument marshalling and one collective only; runs on the current torch stream."""
    import torch
    import torch.distributed as dist
    stream = torch.cuda.current_stream(device).cuda_stream
    eco_step_begin(handle, lr, beta1, beta2, eps, step, seed, weight_decay, grad_scale, stream)
    dist.all_reduce(eco_amax_tensor(handle, device), op=dist.ReduceOp.MAX, group=group)
    eco_step_end(handle, stream)


def eco_step_host(cfg: Config, tensors: Sequence[Tensor], lr: float, beta1: float, beta2: float, eps: float,
                  step: int, seed: int, device: int = 0):
    """One step on state held in host memory; returns (h2d_bytes, d2h_bytes)."""
    L = load_library()
    c = cfg.c()
    arr = _tensor_array(tensors)
    up, down = ctypes.c_uint64(), ctypes.c_uint64()
    st = L.eco_step_host(ctypes.byref(c), arr, len(tensors), device, lr, beta1, beta2, eps, step, seed,
                         ctypes.byref(up), ctypes.byref(down))
    if st != ECO_OK:
        _raise(st)
    return up.value, down.value


def eco_host_create(cfg: Config, tensors: Sequence[Tensor], device: int = 0) -> int:
    """Bind a list of HOST buffers for repeated host-resident steps; returns the handle.  The buffers must
    stay alive until ``eco_host_destroy``.  See include/eco.h."""
    L = load_library()
    handle = ctypes.c_void_p()
    c = cfg.c()
    arr = _tensor_array(tensors)
    st = L.eco_host_create(ctypes.byref(handle), ctypes.byref(c), arr, len(tensors), device)
    if st != ECO_OK:
        _raise(st)
    return handle.value


def eco_host_step(handle: int, lr: float, beta1: float, beta2: float, eps: float, step: int, seed: int):
    """One step on the host-resident state bound by ``eco_host_create``; returns (h2d_bytes, d2h_bytes)."""
    up, down = ctypes.c_uint64(), ctypes.c_uint64()
    st = load_library().eco_host_step(handle, lr, beta1, beta2, eps, step, seed, ctypes.byref(up), ctypes.byref(down))
    if st != ECO_OK:
        _raise(st)
    return up.value, down.value


def eco_host_copies(handle: int):
    """(h2d, d2h) copies one eco_host_step issues.  See include/eco.h."""
    up, down = ctypes.c_uint64(0), ctypes.c_uint64(0)
    st = load_library().eco_host_copies(handle, ctypes.byref(up), ctypes.byref(down))
    if st != 0:
        raise EcoError(st, "eco_host_copies")
    return up.value, down.value


def eco_host_destroy(handle: int) -> None:
    load_library().eco_host_destroy(handle)


def eco_step_static(cfg: Config, tensors: Sequence[Tensor], lr: float, beta1: float, beta2: float, eps: float,
                    step: int, seed: int, device: int = 0, stream: int = 0) -> None:
    """One per-tensor-scale step with no context and no device allocation (the library's tables live in
    a fixed array inside the loaded image).  For callers that cannot call cudaMalloc; see
    ``eco_step_static`` in include/eco.h for the limits and the sharing rules."""
    c = cfg.c()
    arr = _tensor_array(tensors)
    st = load_library().eco_step_static(ctypes.byref(c), arr, len(tensors), device, lr, beta1, beta2, eps,
                                        step, seed, stream)
    if st != ECO_OK:
        _raise(st)


def eco_check(handle: int, stream: int = 0) -> None:
    """Synchronize ``stream`` and raise if a bounded device-side wait expired.  See include/eco.h."""
    st = load_library().eco_check(handle, stream)
    if st != ECO_OK:
        _raise(st, handle)


def eco_attach_error_buffers(handle: int, buffers) -> None:
    """Attach one FP32 error buffer per tensor (torch CUDA tensors).  See ``eco_attach_error_buffers`` in include/eco.h."""
    arr = (ctypes.c_void_p * len(buffers))(*[_addr(b) for b in buffers])
    st = load_library().eco_attach_error_buffers(handle, arr, len(buffers))
    if st != ECO_OK:
        _raise(st, handle)


def eco_selftest_wait(handle: int, limit_cycles: int = 2_000_000, stream: int = 0) -> int:
    """Run the bounded-wait self-test; returns the status (ECO_ERR_TIMEOUT when the mechanism works)."""
    return load_library().eco_selftest_wait(handle, limit_cycles, stream)


def eco_selftest_grid_wait(handle: int, limit_cycles: int = 2_000_000, stream: int = 0) -> int:
    """Run the self-test of the bounded grid barrier; returns the status (ECO_ERR_TIMEOUT when the mechanism works)."""
    return load_library().eco_selftest_grid_wait(handle, limit_cycles, stream)


def eco_destroy(handle: int) -> None:
    load_library().eco_destroy(handle)


def eco_quantize(cfg: Config, x, rows: int, cols: int, w, scale, seed: int = 0, step: int = 0,
                 tensor_id: int = 0, device: int = 0, stream: int = 0) -> None:
    """theta_hat_0 = q(x) on the device.  See ``eco_quantize`` in include/eco.h."""
    c = cfg.c()
    st = load_library().eco_quantize(ctypes.byref(c), _addr(x), rows, cols, _addr(w), _addr(scale),
                                     seed, step, tensor_id, device, stream)
    if st != ECO_OK:
        _raise(st)


def eco_dequantize(cfg: Config, w, scale, rows: int, cols: int, out, device: int = 0, stream: int = 0) -> None:
    """out = value(code) * scale; ``out`` is a float32 or bfloat16 torch CUDA tensor.  See include/eco.h."""
    import torch
    c = cfg.c()
    st = load_library().eco_dequantize(ctypes.byref(c), _addr(w), _addr(scale), rows, cols, _addr(out),
                                       1 if out.dtype == torch.bfloat16 else 0, device, stream)
    if st != ECO_OK:
        _raise(st)


def eco_set_option(name: str, value: int) -> None:
    st = load_library().eco_set_option(name.encode(), value)
    if st != ECO_OK:
        _raise(st)


def eco_num_launches(handle: int) -> int:
    return load_library().eco_num_launches(handle)


def eco_version() -> str:
    return load_library().eco_version().decode()
