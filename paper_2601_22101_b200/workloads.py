"""Seeded synthetic inputs for the ECO optimizer step: parameter-set shapes and
value generators.

This module holds none of the method's arithmetic (no quantizer, no optimizer
update): it only names the tensor shapes of the five benchmark parameter sets
and draws full-precision initial weights ~ N(0, std) and BF16 gradients
~ N(0, std) from numpy's counter-based Philox bit generator, keyed by
(data_seed, tensor_id, step, kind).  Both the CUDA path and the CPU oracle are
fed the bytes produced here.

The shapes stand in for the models the paper trains (Sec. 4: the 30M scaling
model, Gemma-3-1B, a sparse-MoE model, DeepSeek-MoE-16B); their datasets,
tokenizers and trained weights are not needed for an optimizer step.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Optional

import numpy as np

# Enumerations of the C-ABI (include/eco.h), by value.
FP8_E4M3, INT4, FP8_E5M2 = 0, 1, 4
PER_TENSOR, PER_ROW, PER_BLOCK = 0, 1, 2
SCALE_F32, SCALE_BF16, SCALE_E8M0 = 0, 1, 2
SCALE_BYTES = {SCALE_F32: 4, SCALE_BF16: 2, SCALE_E8M0: 1}
SGDM, ADAM = 0, 1
RTN, SR = 0, 1

_KIND_WEIGHT, _KIND_GRAD, _KIND_MASK = 1, 2, 3


@dataclass(frozen=True)
class TensorSpec:
    name: str
    rows: int
    cols: int
    tensor_id: int
    zero_grad: bool = False

    @property
    def numel(self) -> int:
        return self.rows * self.cols


@dataclass(frozen=True)
class Workload:
    name: str
    format: int
    granularity: int
    block: int
    scale_dtype: int
    optimizer: int
    rounding: int
    lr: float
    beta1: float
    beta2: float
    eps: float
    weight_std: float
    grad_std: float
    steps: int
    step_seed: int
    data_seed: int = 1234
    tensors: List[TensorSpec] = field(default_factory=list)

    @property
    def numel(self) -> int:
        return sum(t.numel for t in self.tensors)

    def n_scales(self, t: TensorSpec) -> int:
        if self.granularity == PER_TENSOR:
            return 1
        if self.granularity == PER_ROW:
            return t.rows
        return t.rows * ((t.cols + self.block - 1) // self.block)

    def code_bytes(self, t: TensorSpec) -> int:
        return (t.numel + 1) // 2 if self.format == INT4 else t.numel

    def state_bytes_per_param(self) -> float:
        """Bytes of persistent state per parameter (codes + moments), scales excluded."""
        w = 0.5 if self.format == INT4 else 1.0
        return w + 4.0 + (4.0 if self.optimizer == ADAM else 0.0)

    def algorithmic_bytes_per_param(self) -> float:
        """Bytes one step must move per parameter: read codes, grad, moments and
        old scale; write codes, moments and new scale."""
        w = 0.5 if self.format == INT4 else 1.0
        moments = 4.0 * (2 if self.optimizer == ADAM else 1)
        n_scale = sum(self.n_scales(t) for t in self.tensors)
        sb = float(SCALE_BYTES[self.scale_dtype]) * n_scale / max(self.numel, 1)
        return (w + 2.0 + moments + sb) + (w + moments + sb)


def _number(tensors):
    return [replace(t, tensor_id=i) for i, t in enumerate(tensors)]


def c1(rounding: int = SR) -> Workload:
    """One 1024x1024 linear weight, FP8 per-tensor scale, momentum SGD."""
    return Workload("c1_linear_1024_fp8_tensor_sgdm_" + ("sr" if rounding == SR else "rtn"),
                    FP8_E4M3, PER_TENSOR, 128, SCALE_F32, SGDM, rounding,
                    lr=1e-3, beta1=0.9, beta2=0.0, eps=0.0, weight_std=0.02, grad_std=1e-3,
                    steps=10, step_seed=0xEC0 + 0,
                    tensors=[TensorSpec("linear.weight", 1024, 1024, 0)])


def c2(layers: int = 6, vocab: int = 32000) -> Workload:
    """30M-class decoder (d=384, FFN 1536, vocab 32000), FP8 1x128 blocks, Adam, SR."""
    d, f = 384, 1536
    ts = []
    for l in range(layers):
        for n in ("q", "k", "v", "o"):
            ts.append(TensorSpec(f"layers.{l}.attn.{n}", d, d, 0))
        ts.append(TensorSpec(f"layers.{l}.ffn.up", f, d, 0))
        ts.append(TensorSpec(f"layers.{l}.ffn.down", d, f, 0))
    ts.append(TensorSpec("tok_embedding", vocab, d, 0))
    ts.append(TensorSpec("lm_head", vocab, d, 0))
    return Workload("c2_decoder30m_fp8_block128_adam_sr", FP8_E4M3, PER_BLOCK, 128, SCALE_F32, ADAM, SR,
                    lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_std=0.02, grad_std=1e-3,
                    steps=100, step_seed=0xEC0 + 1, tensors=_number(ts))


def c3(layers: int = 26, vocab: int = 262144) -> Workload:
    """Gemma-3-1B-shaped set (hidden 1152, 4 q / 1 kv heads of 256, gated FFN 6912), FP8 per-tensor, Adam, SR."""
    h, q, kv, f = 1152, 4 * 256, 1 * 256, 6912
    ts = []
    for l in range(layers):
        ts.append(TensorSpec(f"layers.{l}.attn.q", q, h, 0))
        ts.append(TensorSpec(f"layers.{l}.attn.k", kv, h, 0))
        ts.append(TensorSpec(f"layers.{l}.attn.v", kv, h, 0))
        ts.append(TensorSpec(f"layers.{l}.attn.o", h, q, 0))
        ts.append(TensorSpec(f"layers.{l}.ffn.gate", f, h, 0))
        ts.append(TensorSpec(f"layers.{l}.ffn.up", f, h, 0))
        ts.append(TensorSpec(f"layers.{l}.ffn.down", h, f, 0))
    if vocab:
        ts.append(TensorSpec("embedding", vocab, h, 0))
    return Workload("c3_gemma3_1b_fp8_tensor_adam_sr", FP8_E4M3, PER_TENSOR, 128, SCALE_F32, ADAM, SR,
                    lr=1e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_std=0.02, grad_std=1e-4,
                    steps=100, step_seed=0xEC0 + 2, tensors=_number(ts))


def c4(layers: int = 16, experts: int = 64, expert_mats: int = 2, data_seed: int = 1234) -> Workload:
    """Sparse-MoE expert set (d=1024, FFN 1024, 64 experts x 16 layers), FP8 1x128 blocks, Adam, SR.
    A seeded half of the (layer, expert) pairs receives an all-zero gradient.
    expert_mats = 2 gives 2,147,483,648 parameters (the set's "2.1B"); 3 adds the gate matrix."""
    d, f = 1024, 1024
    names = ("up", "down") if expert_mats == 2 else ("gate", "up", "down")
    n_pairs = layers * experts
    rng = np.random.Generator(np.random.Philox(np.random.SeedSequence([data_seed, 0, 0, _KIND_MASK])))
    zero = np.zeros(n_pairs, dtype=bool)
    zero[rng.permutation(n_pairs)[: n_pairs // 2]] = True
    ts = []
    for l in range(layers):
        for e in range(experts):
            for n in names:
                r, c = (d, f) if n == "down" else (f, d)
                ts.append(TensorSpec(f"layers.{l}.experts.{e}.{n}", r, c, 0, bool(zero[l * experts + e])))
    return Workload(f"c4_smoe_{expert_mats}mat_fp8_block128_adam_sr", FP8_E4M3, PER_BLOCK, 128, SCALE_F32, ADAM, SR,
                    lr=2e-5, beta1=0.9, beta2=0.95, eps=1e-8, weight_std=0.02, grad_std=1e-3,
                    steps=100, step_seed=0xEC0 + 3, data_seed=data_seed, tensors=_number(ts))


def c5(moe_layers: int = 27, experts: int = 66, dense_layers: int = 1) -> Workload:
    """DeepSeek-MoE-16B-shaped expert/FFN set (hidden 2048, 64 routed + 2 shared experts of 1408,
    first layer dense FFN 10944), INT4 with group-128 BF16 scales, momentum SGD, SR."""
    h, fe, fd = 2048, 1408, 10944
    ts = []
    for l in range(dense_layers):
        ts.append(TensorSpec(f"layers.{l}.mlp.gate", fd, h, 0))
        ts.append(TensorSpec(f"layers.{l}.mlp.up", fd, h, 0))
        ts.append(TensorSpec(f"layers.{l}.mlp.down", h, fd, 0))
    for l in range(dense_layers, dense_layers + moe_layers):
        for e in range(experts):
            ts.append(TensorSpec(f"layers.{l}.experts.{e}.gate", fe, h, 0))
            ts.append(TensorSpec(f"layers.{l}.experts.{e}.up", fe, h, 0))
            ts.append(TensorSpec(f"layers.{l}.experts.{e}.down", h, fe, 0))
    return Workload("c5_deepseek_moe16b_int4_group128_sgdm_sr", INT4, PER_BLOCK, 128, SCALE_BF16, SGDM, SR,
                    lr=2e-5, beta1=0.9, beta2=0.0, eps=0.0, weight_std=0.02, grad_std=1e-4,
                    steps=100, step_seed=0xEC0 + 4, tensors=_number(ts))


def shape_slice(w: Workload, max_rows: Optional[int] = None) -> Workload:
    """A shape-complete slice: one tensor of every distinct (rows, cols, zero_grad),
    optionally with rows capped (keeps cols, hence the block structure of a row)."""
    seen, ts = set(), []
    for t in w.tensors:
        key = (t.rows, t.cols, t.zero_grad)
        if key in seen:
            continue
        seen.add(key)
        rows = min(t.rows, max_rows) if max_rows else t.rows
        ts.append(replace(t, rows=rows))
    return replace(w, name=w.name + "_slice", tensors=ts)


def c3_small() -> Workload:
    """Two layers and a 32768-row embedding of the Gemma-3-1B-shaped set (profiling-sized: ~1 GB of state)."""
    w = c3(layers=2, vocab=32768)
    return replace(w, name=w.name + "_small")


def c3_no_embedding(layers: int = 26) -> Workload:
    """The layers of the Gemma-3-1B-shaped set without the embedding: every tensor is at most 88 MB of inputs, i.e. about
    as large as the L2 (the embedding is 3.3 GB)."""
    w = c3(layers=layers, vocab=0)
    return replace(w, name=w.name + f"_layers{layers}_only")


def c3_rowwise() -> Workload:
    """The Gemma-3-1B-shaped set with one FP8 scale per row: the granularity of the paper's own FP8 runs (Sec. 4.1)."""
    w = c3()
    return replace(w, name="c3_gemma3_1b_fp8_row_adam_sr", granularity=PER_ROW)


def c5_tensorwise_adam() -> Workload:
    """The DeepSeek-MoE-shaped expert set the way the paper fine-tuned it (Sec. 4.5): tensor-wise INT4, Adam."""
    w = c5()
    return replace(w, name="c5_deepseek_moe16b_int4_tensor_adam_sr", granularity=PER_TENSOR, scale_dtype=SCALE_F32,
                   optimizer=ADAM, beta2=0.95, eps=1e-8)


def c3_rowwise_small() -> Workload:
    """c3_small with one scale per row (profiling-sized)."""
    w = c3_small()
    return replace(w, name="c3_gemma3_1b_fp8_row_adam_sr_small", granularity=PER_ROW)


def c4_small() -> Workload:
    """One layer (64 experts) of the sparse-MoE set (profiling-sized: ~1.5 GB of state)."""
    w = c4(layers=1)
    return replace(w, name=w.name + "_small")


def c5_small() -> Workload:
    """The dense layer and one MoE layer of 16 experts of the DeepSeek-MoE-shaped set (~1.4 GB of state)."""
    w = c5(moe_layers=1, experts=16)
    return replace(w, name=w.name + "_small")


def shard(w: Workload, rank: int, world: int) -> Workload:
    """The tensors rank `rank` of `world` owns when a parameter set is split by whole tensors.

    Tensors never interact in the step (a scale block lies inside one tensor) and the random stream is
    keyed by (tensor_id, element index), so any split by whole tensors gives the same bits as the
    unsplit set with no communication.  Assignment: largest tensor first, each to the rank with the
    fewest parameters so far (ties to the lowest rank); deterministic, so every rank derives the same
    partition without talking to the others."""
    if not (0 <= rank < world):
        raise ValueError("rank must be in [0, world)")
    load = [0] * world
    mine = []
    order = sorted(range(len(w.tensors)), key=lambda i: (-w.tensors[i].numel, i))
    for i in order:
        r = min(range(world), key=lambda k: (load[k], k))
        load[r] += w.tensors[i].numel
        if r == rank:
            mine.append(i)
    mine.sort()
    return replace(w, name=f"{w.name}_shard{rank}of{world}", tensors=[w.tensors[i] for i in mine])


def replicate(w: Workload, copies: int) -> Workload:
    """`copies` parameter sets of the shape of `w` as one job (weak scaling: the job grows with the number
    of ranks); tensor ids stay unique so that every copy draws its own random stream."""
    n = len(w.tensors)
    ts = [replace(t, name=f"copy{c}.{t.name}", tensor_id=c * n + t.tensor_id) for c in range(copies) for t in w.tensors]
    return replace(w, name=f"{w.name}_x{copies}", tensors=ts)


def c4_dense() -> Workload:
    """The sparse-MoE set with EVERY expert receiving a gradient (no all-zero gradients): the dense-gradient rate of
    the FP8 1x128 Adam path at 2.1B parameters."""
    w = c4()
    return replace(w, name="c4_smoe_2mat_fp8_block128_adam_sr_all_routed", tensors=[replace(t, zero_grad=False) for t in w.tensors])


def c4_mx() -> Workload:
    """The all-routed sparse-MoE set in the microscaling layout: FP8-E4M3 codes, 1x32 blocks, one power-of-two
    exponent byte per block (20.03 B/param)."""
    w = c4_dense()
    return replace(w, name="c4_smoe_2mat_mxfp8_block32_e8m0_adam_sr_all_routed", block=32, scale_dtype=SCALE_E8M0)


def c4_mx_small() -> Workload:
    """c4_mx cut to the size of c4_small (profiling-sized)."""
    w = c4_small()
    return replace(w, name="c4_smoe_2mat_mxfp8_block32_e8m0_adam_sr_small", block=32, scale_dtype=SCALE_E8M0,
                   tensors=[replace(t, zero_grad=False) for t in w.tensors])


def c4_dense_small() -> Workload:
    """c4_dense cut to the size of c4_small (profiling-sized)."""
    w = c4_small()
    return replace(w, name="c4_smoe_2mat_fp8_block128_adam_sr_all_routed_small", tensors=[replace(t, zero_grad=False) for t in w.tensors])


BY_NAME = {"c3f": c3_no_embedding, "c3fs": lambda: c3_no_embedding(3), "c1": c1, "c2": c2, "c3": c3, "c4": c4, "c5": c5, "c3r": c3_rowwise, "c5t": c5_tensorwise_adam, "c4g": lambda: c4(expert_mats=3), "c4d": c4_dense,
           "c3s": c3_small, "c3rs": c3_rowwise_small, "c4s": c4_small, "c5s": c5_small,
           "c4mx": c4_mx, "c4mxs": c4_mx_small, "c4ds": c4_dense_small}


def _rng(w: Workload, t: TensorSpec, step: int, kind: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([w.data_seed, t.tensor_id, step, kind])))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round binary32 to bfloat16 bit patterns (nearest, ties to even); finite inputs."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    b = b + 0x7FFF + ((b >> 16) & 1)
    return (b >> 16).astype(np.uint16)


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(h, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def initial_weights(w: Workload, t: TensorSpec) -> np.ndarray:
    """Full-precision theta_0 ~ N(0, weight_std), float32 [rows, cols]."""
    x = _rng(w, t, 0, _KIND_WEIGHT).standard_normal((t.rows, t.cols), dtype=np.float32)
    x *= np.float32(w.weight_std)
    return x


def gradient_bf16(w: Workload, t: TensorSpec, step: int) -> np.ndarray:
    """BF16 bit patterns (uint16 [rows*cols]) of the gradient at a 1-based step."""
    if t.zero_grad:
        return np.zeros(t.numel, dtype=np.uint16)
    g = _rng(w, t, step, _KIND_GRAD).standard_normal(t.numel, dtype=np.float32)
    g *= np.float32(w.grad_std)
    return f32_to_bf16_bits(g)
