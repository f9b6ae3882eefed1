"""Noise floors of the three training regimes on a separable quadratic (Sec. 3.4 and Appendix C), run
through the CUDA library with its real FP8 quantizer.

Every coordinate is an independent 1-D problem f(x) = L/2 (x - x*)^2 with its own optimum x* ~ N(0, 0.02),
trained with momentum SGD from the optimum's quantized neighbourhood; the gradient is evaluated at the
QUANTIZED weights, as in quantized training.  Three regimes share the data:

  master   FP32 master weights kept by the caller, quantized for the "forward" each step (eco_quantize, SR)
  naive    no master weights, error dropped            (eco_step, injection off)
  eco      no master weights, error fed to the momentum (eco_step, the paper's method)
  exact    no master weights, stored error e_t, the exact injection of Appendix A (ECO_INJECT_EXACT)

Reported: the stationary mean of (theta_hat - x*)^2 over the coordinates.  Sec. 3.4 predicts that the
naive floor grows like 1/eta as the learning rate shrinks while the ECO floor stays bounded, and that the
master-weight floor is the quantization noise of the final weights.  (The appendix models the quantizer
as additive noise of fixed variance; FP8 noise is relative to each weight, so only the trends are compared,
not the closed forms.)

    python -m paper_2601_22101_b200.examples.quadratic_floors
"""
from __future__ import annotations

import torch

from .. import eco


_FP8_TENSOR = eco.Config(format=eco.ECO_FORMAT_FP8_E4M3, granularity=eco.ECO_SCALE_PER_TENSOR, scale_dtype=eco.ECO_SCALE_F32)


def _dequant(codes: torch.Tensor, scale: torch.Tensor) -> torch.Tensor:
    """The weights the "forward pass" sees: value(code) * scale, expanded by the library."""
    out = torch.empty(codes.numel(), dtype=torch.float32, device=codes.device)
    eco.eco_dequantize(_FP8_TENSOR, codes, scale, 1, codes.numel(), out, device=codes.device.index or 0,
                       stream=torch.cuda.current_stream(codes.device).cuda_stream)
    return out


def run(regime: str, lr: float, steps: int, n_rows: int = 256, cols: int = 1024, beta: float = 0.9,
        curvature: float = 1.0, seed: int = 0, burn_in: float = 0.5, device: int = 0, stochastic: bool = True,
        start_offset: float = 0.01) -> float:
    """Returns the mean of (theta_hat - x*)^2 over coordinates and over the last (1 - burn_in) of the steps."""
    assert regime in ("master", "naive", "eco", "exact")
    dev = torch.device("cuda", device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    n = n_rows * cols
    x_star = torch.empty(n, device=dev).normal_(0.0, 0.02, generator=gen)
    cfg = eco.Config(format=eco.ECO_FORMAT_FP8_E4M3, granularity=eco.ECO_SCALE_PER_TENSOR, scale_dtype=eco.ECO_SCALE_F32,
                     optimizer=eco.ECO_OPT_SGDM,
                     rounding=eco.ECO_ROUND_STOCHASTIC if stochastic else eco.ECO_ROUND_NEAREST,
                     injection={"eco": eco.ECO_INJECT_ECO, "exact": eco.ECO_INJECT_EXACT}.get(regime, eco.ECO_INJECT_NONE))
    codes = torch.zeros(n, dtype=torch.uint8, device=dev)
    scale = torch.zeros(1, dtype=torch.float32, device=dev)
    grad = torch.zeros(n, dtype=torch.bfloat16, device=dev)
    m = torch.zeros(n, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    # start away from the optimum; `theta` is the master copy (regime "master" only)
    theta = x_star + torch.empty(n, device=dev).normal_(0.0, start_offset, generator=gen)
    eco.eco_quantize(cfg, theta, n_rows, cols, codes, scale, seed=seed, step=0, tensor_id=0, device=device, stream=stream)
    handle = None
    if regime != "master":
        handle = eco.eco_create(cfg, [eco.Tensor(codes, scale, grad, m, None, n_rows, cols, 0)], device)
    err = torch.zeros(n, dtype=torch.float32, device=dev)
    if regime == "exact":
        # Appendix A initialises theta_hat_0 = q(theta_0), e_0 = theta_0 - theta_hat_0
        err.copy_(theta - _dequant(codes, scale))
    if regime in ("eco", "exact"):
        eco.eco_attach_error_buffers(handle, [err])
    acc, count = 0.0, 0
    try:
        for t in range(1, steps + 1):
            theta_hat = _dequant(codes, scale)
            g = curvature * (theta_hat - x_star)
            if t > burn_in * steps:
                acc += float((theta_hat - x_star).square().mean())
                count += 1
            if regime == "master":
                m.mul_(beta).add_(g, alpha=1.0 - beta)
                theta.add_(m, alpha=-lr)
                eco.eco_quantize(cfg, theta, n_rows, cols, codes, scale, seed=seed, step=t, tensor_id=0, device=device,
                                 stream=stream)
            else:
                grad.copy_(g)
                eco.eco_step(handle, lr, beta, 0.0, 0.0, t, seed, stream)
    finally:
        torch.cuda.synchronize(device)
        if handle is not None:
            eco.eco_destroy(handle)
    return acc / max(count, 1)


def error_similarity(lr: float, steps: int, n_rows: int = 256, cols: int = 1024, beta: float = 0.9, seed: int = 0,
                     device: int = 0):
    """The observation ECO rests on (Sec. 3.2, measured in Sec. 4.2 / Fig. 2): consecutive quantization errors are
    alike.  Runs the ECO regime with an attached error buffer and returns the means, over the second half of the run,
    of ||e_{t+1}|| / ||e_t|| and of the cosine between e_t and e_{t+1}."""
    dev = torch.device("cuda", device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    n = n_rows * cols
    x_star = torch.empty(n, device=dev).normal_(0.0, 0.02, generator=gen)
    theta = x_star + torch.empty(n, device=dev).normal_(0.0, 0.01, generator=gen)
    cfg = eco.Config(format=eco.ECO_FORMAT_FP8_E4M3, granularity=eco.ECO_SCALE_PER_TENSOR, scale_dtype=eco.ECO_SCALE_F32,
                     optimizer=eco.ECO_OPT_SGDM, rounding=eco.ECO_ROUND_NEAREST, injection=eco.ECO_INJECT_ECO)
    codes = torch.zeros(n, dtype=torch.uint8, device=dev)
    scale = torch.zeros(1, dtype=torch.float32, device=dev)
    grad = torch.zeros(n, dtype=torch.bfloat16, device=dev)
    m = torch.zeros(n, dtype=torch.float32, device=dev)
    err = torch.zeros(n, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    eco.eco_quantize(cfg, theta, n_rows, cols, codes, scale, seed=seed, step=0, tensor_id=0, device=device, stream=stream)
    handle = eco.eco_create(cfg, [eco.Tensor(codes, scale, grad, m, None, n_rows, cols, 0)], device)
    eco.eco_attach_error_buffers(handle, [err])
    ratios, cosines = [], []
    try:
        prev = None
        for t in range(1, steps + 1):
            grad.copy_(_dequant(codes, scale) - x_star)
            eco.eco_step(handle, lr, beta, 0.0, 0.0, t, seed, stream)
            cur = err.clone()
            if prev is not None and t > steps // 2:
                ratios.append(float(cur.norm() / prev.norm()))
                cosines.append(float(torch.dot(cur, prev) / (cur.norm() * prev.norm())))
            prev = cur
    finally:
        torch.cuda.synchronize(device)
        eco.eco_destroy(handle)
    return sum(ratios) / len(ratios), sum(cosines) / len(cosines)


def main() -> None:
    for stochastic in (False, True):
        print(f"rounding = {'stochastic' if stochastic else 'nearest'}   (mean (theta_hat - x*)^2; FP8, per-tensor scale, beta 0.9)")
        print(f"{'lr':>8} {'master':>12} {'naive':>12} {'eco':>12} {'exact':>12}")
        for lr, steps in ((0.3, 800), (0.1, 2000), (0.03, 6000), (0.01, 18000)):
            row = [run(r, lr, steps, stochastic=stochastic) for r in ("master", "naive", "eco", "exact")]
            print(f"{lr:8.3f} " + " ".join(f"{v:12.4e}" for v in row))
    print("consecutive errors in the ECO regime (round to nearest): mean ||e_t+1|| / ||e_t||, mean cosine(e_t, e_t+1)")
    for lr, steps in ((0.3, 800), (0.03, 6000)):
        r, c = error_similarity(lr, steps)
        print(f"{lr:8.3f} {r:12.4f} {c:12.4f}")


if __name__ == "__main__":
    main()
