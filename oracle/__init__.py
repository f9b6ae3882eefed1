"""ctypes binding of the ECO CPU oracle (``oracle/eco_oracle.cpp``).

TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this module; the CUDA library and its
Python binding never do.  The oracle states Algorithm 1-3 and the Sec. 3.1
quantizer of the paper in plain single-threaded C++; this file only compiles
it with g++ and marshals numpy arrays.
"""
from __future__ import annotations

import contextlib
import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "eco_oracle.cpp")
_LIB = os.path.join(_HERE, "libeco_oracle.so")

FP8_E4M3, INT4, IDENTITY, ADDITIVE_NOISE, FP8_E5M2 = 0, 1, 2, 3, 4
PER_TENSOR, PER_ROW, PER_BLOCK = 0, 1, 2
SCALE_NATIVE, SCALE_BF16, SCALE_E8M0 = 0, 1, 2
SGDM, ADAM = 0, 1
RTN, SR = 0, 1
INJECT_NONE, INJECT_ECO, INJECT_IDEAL = 0, 1, 2
GRAD_BF16, GRAD_NATIVE = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fused contraction, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fno-fast-math",
               "-Wall", "-Wextra", "-shared", "-fPIC", _SRC, "-o", _LIB]
        subprocess.run(cmd, check=True)
    return _LIB


class _Config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "format", "granularity", "block", "scale_dtype", "optimizer", "rounding",
        "injection", "grad_dtype")]


@dataclass
class Config:
    format: int = FP8_E4M3
    granularity: int = PER_BLOCK
    block: int = 128
    scale_dtype: int = SCALE_NATIVE
    optimizer: int = SGDM
    rounding: int = RTN
    injection: int = INJECT_ECO
    grad_dtype: int = GRAD_BF16

    def c(self) -> _Config:
        return _Config(self.format, self.granularity, self.block, self.scale_dtype,
                       self.optimizer, self.rounding, self.injection, self.grad_dtype)

    def n_scales(self, rows: int, cols: int) -> int:
        if self.granularity == PER_TENSOR:
            return 1
        if self.granularity == PER_ROW:
            return rows
        return rows * ((cols + self.block - 1) // self.block)

    def code_bytes(self, rows: int, cols: int) -> int:
        n = rows * cols
        return (n + 1) // 2 if self.format == INT4 else n


_lib = None


def _bind(path: str) -> ctypes.CDLL:
    L = ctypes.CDLL(path)
    L.eco_oracle_element_random_word.restype = ctypes.c_uint32
    L.eco_oracle_element_random_word.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint64]
    L.eco_oracle_code_value.restype = ctypes.c_double
    L.eco_oracle_code_value.argtypes = [ctypes.c_int, ctypes.c_int]
    L.eco_oracle_f32_to_bf16.restype = ctypes.c_uint16
    L.eco_oracle_f32_to_bf16.argtypes = [ctypes.c_float]
    vp, u64, u32, dbl = ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_double
    L.eco_oracle_philox4x32_10.argtypes = [vp, vp, vp]
    for sfx in ("f32", "f64"):
        getattr(L, f"eco_oracle_round_{sfx}").argtypes = [ctypes.c_int, ctypes.c_int, vp, vp, u64, vp]
        getattr(L, f"eco_oracle_quantize_{sfx}").argtypes = [vp, vp, u64, u64, vp, vp, u64, u64, u32, u64]
        getattr(L, f"eco_oracle_dequantize_{sfx}").argtypes = [vp, vp, vp, u64, u64, vp]
        getattr(L, f"eco_oracle_step_{sfx}").argtypes = [
            vp, dbl, dbl, dbl, dbl, u64, u64, vp, vp, vp, vp, vp, u64, u64, u32, vp, vp, vp, vp, u64]
        getattr(L, f"eco_oracle_step_ex_{sfx}").argtypes = [
            vp, dbl, dbl, dbl, dbl, dbl, dbl, u64, u64, vp, vp, vp, vp, vp, u64, u64, u32, u64]
    return L


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = _bind(build())
    return _lib


@contextlib.contextmanager
def use_library(path: str):
    """Route every call of this module to another build of the oracle for the length of the block.  The
    mutation tests use it: they compile a copy of eco_oracle.cpp with one mistake planted in it and check
    that the pins notice."""
    global _lib
    saved = lib()
    _lib = _bind(path)
    try:
        yield
    finally:
        _lib = saved


def _ptr(a):
    if a is None:
        return None
    assert isinstance(a, np.ndarray) and a.flags["C_CONTIGUOUS"], "need a C-contiguous numpy array"
    return a.ctypes.data_as(ctypes.c_void_p)


def _sfx(dtype) -> str:
    return {np.dtype(np.float32): "f32", np.dtype(np.float64): "f64"}[np.dtype(dtype)]


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.empty(4, dtype=np.uint32)
    lib().eco_oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def element_random_word(seed: int, step: int, tensor_id: int, i: int) -> int:
    return int(lib().eco_oracle_element_random_word(seed, step, tensor_id, i))


def code_value(fmt: int, code: int) -> float:
    return float(lib().eco_oracle_code_value(fmt, code))


def f32_to_bf16(x: float) -> int:
    return int(lib().eco_oracle_f32_to_bf16(float(x)))


def round_to_codes(fmt: int, rounding: int, y: np.ndarray, r: np.ndarray | None = None) -> np.ndarray:
    """Round already-scaled values ``y`` to codes; ``r`` are the random words (SR)."""
    y = np.ascontiguousarray(y)
    if r is not None:
        r = np.ascontiguousarray(r, dtype=np.uint32)
        assert r.size == y.size
    codes = np.empty(y.size, dtype=np.uint8)
    getattr(lib(), f"eco_oracle_round_{_sfx(y.dtype)}")(fmt, rounding, _ptr(y), _ptr(r), y.size, _ptr(codes))
    return codes


def scale_numpy_dtype(cfg: Config, real=np.float32):
    return {SCALE_BF16: np.uint16, SCALE_E8M0: np.uint8}.get(cfg.scale_dtype, real)


def quantize(cfg: Config, x: np.ndarray, seed: int = 0, step: int = 0, tensor_id: int = 0, index_base: int = 0):
    """theta_hat = q(x) for a [rows, cols] array; returns (codes, scales).  ``index_base``: position of
    x[0, 0] inside the full tensor when x is a slice of whole rows of it (random words are drawn per position)."""
    x = np.ascontiguousarray(x)
    rows, cols = x.shape
    w = np.zeros(cfg.code_bytes(rows, cols), dtype=np.uint8)
    s = np.zeros(cfg.n_scales(rows, cols), dtype=scale_numpy_dtype(cfg, x.dtype))
    c = cfg.c()
    rc = getattr(lib(), f"eco_oracle_quantize_{_sfx(x.dtype)}")(
        ctypes.byref(c), _ptr(x), rows, cols, _ptr(w), _ptr(s), seed, step, tensor_id, index_base)
    assert rc == 0
    return w, s


def dequantize(cfg: Config, w: np.ndarray, s: np.ndarray, rows: int, cols: int, real=np.float32) -> np.ndarray:
    x = np.empty((rows, cols), dtype=real)
    c = cfg.c()
    rc = getattr(lib(), f"eco_oracle_dequantize_{_sfx(real)}")(ctypes.byref(c), _ptr(w), _ptr(s), rows, cols, _ptr(x))
    assert rc == 0
    return x


def step(cfg: Config, *, lr: float, beta1: float, beta2: float = 0.0, eps: float = 0.0,
         step: int, seed: int = 0, w: np.ndarray, scale: np.ndarray | None, grad: np.ndarray,
         m: np.ndarray, v: np.ndarray | None = None, rows: int, cols: int, tensor_id: int = 0,
         noise: np.ndarray | None = None, e_prev: np.ndarray | None = None,
         dbg_theta_tilde: np.ndarray | None = None, dbg_err: np.ndarray | None = None,
         weight_decay: float = 0.0, grad_scale: float = 1.0, index_base: int = 0) -> None:
    """One Algorithm-1 step on one tensor, in place.  ``m.dtype`` selects binary32 or binary64.
    ``weight_decay`` (decoupled, AdamW style) and ``grad_scale`` (one factor on the gradient, e.g. the
    clipping factor) are the two additions of Sec. 4's training recipe to OPTIM_STEP.  ``index_base``: position of
    the buffers' first element inside the full tensor when they hold a slice of whole rows of it."""
    c = cfg.c()
    if weight_decay != 0.0 or grad_scale != 1.0:
        assert noise is None and e_prev is None and dbg_theta_tilde is None and dbg_err is None
        rc = getattr(lib(), f"eco_oracle_step_ex_{_sfx(m.dtype)}")(
            ctypes.byref(c), float(lr), float(beta1), float(beta2), float(eps), float(weight_decay), float(grad_scale),
            int(step), int(seed), _ptr(w), _ptr(scale), _ptr(grad), _ptr(m), _ptr(v), rows, cols, tensor_id, int(index_base))
        assert rc == 0
        return
    rc = getattr(lib(), f"eco_oracle_step_{_sfx(m.dtype)}")(
        ctypes.byref(c), float(lr), float(beta1), float(beta2), float(eps), int(step), int(seed),
        _ptr(w), _ptr(scale), _ptr(grad), _ptr(m), _ptr(v), rows, cols, tensor_id,
        _ptr(noise), _ptr(e_prev), _ptr(dbg_theta_tilde), _ptr(dbg_err), int(index_base))
    assert rc == 0
