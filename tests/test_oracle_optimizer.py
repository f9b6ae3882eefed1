"""Pins of the oracle's Algorithm 1-3 against what the paper and the mathematics fix:
identity quantizer -> plain SGDM / Adam (library optimizers), Lemma 3.5, the Adam
one-step identity, the error definition and its bounds, Appendix A (ideal injection
is master-weight SGDM), Appendix C (stationary second moments on a 1-D quadratic)."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import (ADAM, ADDITIVE_NOISE, FP8_E4M3, GRAD_BF16, GRAD_NATIVE, IDENTITY, INJECT_ECO, INJECT_IDEAL,
                    INJECT_NONE, INT4, PER_BLOCK, PER_ROW, PER_TENSOR, RTN, SCALE_BF16, SCALE_E8M0, SCALE_NATIVE, SGDM, SR)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split("=")
                out[k.strip()] = float(v)
    return out


# --------------------------------------------------------------------------- identity quantizer
@pytest.mark.parametrize("opt", [SGDM, ADAM])
def test_identity_quantizer_reduces_to_library_optimizer(opt):
    """With q = id the error is zero and nothing is injected (Algorithm 2/3, lines 2 and 5 with
    e = 0): the step is plain dampened SGDM (Eq. m_tilde, theta_tilde) / plain Adam."""
    rng = np.random.default_rng(10)
    n, lr, b1, b2, eps = 257, 3e-3, 0.9, 0.95, 1e-8
    cfg = oracle.Config(format=IDENTITY, optimizer=opt, grad_dtype=GRAD_NATIVE, injection=INJECT_ECO)
    theta0 = rng.standard_normal(n)
    w = theta0.copy()
    m, v = np.zeros(n), np.zeros(n)
    p = torch.tensor(theta0, dtype=torch.float64, requires_grad=True)
    if opt == SGDM:
        topt = torch.optim.SGD([p], lr=lr, momentum=b1, dampening=b1)
        topt.state[p]["momentum_buffer"] = torch.zeros_like(p)   # torch seeds its buffer with g otherwise
    else:
        topt = torch.optim.Adam([p], lr=lr, betas=(b1, b2), eps=eps)
    for t in range(1, 21):
        g = rng.standard_normal(n)
        err = np.full(n, np.nan)
        oracle.step(cfg, lr=lr, beta1=b1, beta2=b2, eps=eps, step=t, w=w, scale=None, grad=g, m=m,
                    v=v if opt == ADAM else None, rows=1, cols=n, dbg_err=err)
        assert (err == 0).all()
        p.grad = torch.tensor(g)
        topt.step()
        np.testing.assert_allclose(w, p.detach().numpy(), rtol=1e-12, atol=1e-14)
    if opt == SGDM:
        np.testing.assert_allclose(m, topt.state[p]["momentum_buffer"].numpy(), rtol=1e-12, atol=1e-15)
    else:
        np.testing.assert_allclose(m, topt.state[p]["exp_avg"].numpy(), rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(v, topt.state[p]["exp_avg_sq"].numpy(), rtol=1e-12, atol=1e-18)


def test_sgdm_closed_form_one_step():
    cfg = oracle.Config(format=IDENTITY, optimizer=SGDM, grad_dtype=GRAD_NATIVE)
    w, m, g = np.array([2.0]), np.array([0.5]), np.array([4.0])
    oracle.step(cfg, lr=0.25, beta1=0.75, step=1, w=w, scale=None, grad=g, m=m, rows=1, cols=1)
    assert m[0] == 0.75 * 0.5 + 0.25 * 4.0          # 1.375
    assert w[0] == 2.0 - 0.25 * 1.375


# --------------------------------------------------------------------------- Lemma 3.5
@pytest.mark.parametrize("fmt,gran,sdt,rnd", [
    (FP8_E4M3, PER_BLOCK, SCALE_NATIVE, SR), (FP8_E4M3, PER_TENSOR, SCALE_NATIVE, RTN),
    (FP8_E4M3, PER_ROW, SCALE_NATIVE, SR), (INT4, PER_BLOCK, SCALE_BF16, SR), (INT4, PER_TENSOR, SCALE_NATIVE, RTN),
    (FP8_E4M3, PER_BLOCK, SCALE_E8M0, SR), (INT4, PER_BLOCK, SCALE_E8M0, RTN)])
def test_lemma_3_5_virtual_sequence_telescopes(fmt, gran, sdt, rnd):
    """theta_t := theta^_t - (eta beta/(1-beta)) m^_t obeys theta_{t+1} = theta_t - eta g_t for ANY
    quantizer, so over T steps it moves by -eta sum g.  Pins the error definition, the sign and the
    size of alpha (Eq. alpha) and that the new scale is the one the codes are read with."""
    rng = np.random.default_rng(11)
    rows, cols, lr, beta = 6, 200, 2e-3, 0.9
    cfg = oracle.Config(format=fmt, granularity=gran, block=32 if sdt == SCALE_E8M0 else 128, scale_dtype=sdt,
                        optimizer=SGDM, rounding=rnd, grad_dtype=GRAD_NATIVE)
    theta0 = rng.standard_normal((rows, cols)) * 0.02
    w, s = oracle.quantize(cfg, theta0)
    m = rng.standard_normal(rows * cols) * 1e-3
    C = lr * beta / (1 - beta)
    virt = oracle.dequantize(cfg, w, s, rows, cols, np.float64).ravel() - C * m
    virt0, gsum = virt.copy(), np.zeros(rows * cols)
    for t in range(1, 41):
        g = rng.standard_normal(rows * cols) * 1e-2
        oracle.step(cfg, lr=lr, beta1=beta, step=t, seed=77, w=w, scale=s, grad=g, m=m, rows=rows, cols=cols,
                    tensor_id=3)
        new = oracle.dequantize(cfg, w, s, rows, cols, np.float64).ravel() - C * m
        np.testing.assert_allclose(new, virt - lr * g, rtol=0, atol=1e-13)
        virt, gsum = new, gsum + g
    np.testing.assert_allclose(virt, virt0 - lr * gsum, rtol=0, atol=1e-12)
    # the quantization really was lossy, so the identity is not vacuous
    err = np.zeros(rows * cols)
    oracle.step(cfg, lr=lr, beta1=beta, step=41, seed=77, w=w, scale=s, grad=g, m=m, rows=rows, cols=cols,
                tensor_id=3, dbg_err=err)
    assert np.abs(err).max() > 1e-5


def test_lemma_3_5_fails_for_a_wrong_alpha():
    """Self-check of the pin: with the injection switched off the identity must break."""
    rng = np.random.default_rng(12)
    n, lr, beta = 256, 2e-3, 0.9
    cfg = oracle.Config(format=FP8_E4M3, granularity=PER_BLOCK, optimizer=SGDM, rounding=RTN,
                        grad_dtype=GRAD_NATIVE, injection=INJECT_NONE)
    w, s = oracle.quantize(cfg, rng.standard_normal((1, n)) * 0.02)
    m = np.zeros(n)
    C = lr * beta / (1 - beta)
    virt = oracle.dequantize(cfg, w, s, 1, n, np.float64).ravel() - C * m
    g = rng.standard_normal(n) * 1e-2
    oracle.step(cfg, lr=lr, beta1=beta, step=1, w=w, scale=s, grad=g, m=m, rows=1, cols=n)
    new = oracle.dequantize(cfg, w, s, 1, n, np.float64).ravel() - C * m
    assert np.abs(new - (virt - lr * g)).max() > 1e-6


# --------------------------------------------------------------------------- Adam one-step identity
@pytest.mark.parametrize("fmt,gran", [(FP8_E4M3, PER_BLOCK), (FP8_E4M3, PER_TENSOR), (INT4, PER_BLOCK)])
def test_adam_one_step_identity(fmt, gran):
    """With eta_t = eta / ((1-b1^t) (sqrt(v/(1-b2^t)) + eps)) elementwise (Sec. 3.2, Adam), Algorithm 3
    gives  theta^' - (eta_t b1/(1-b1)) m^ = theta^ - (eta_t/(1-b1)) m~  for any quantizer: the Adam
    counterpart of Lemma 3.5 for a single step.  Pins the coefficient of Algorithm 3, line 5, and that v
    is returned without injection."""
    rng = np.random.default_rng(13)
    rows, cols, lr, b1, b2, eps = 4, 160, 1e-3, 0.9, 0.95, 1e-8
    cfg = oracle.Config(format=fmt, granularity=gran, optimizer=ADAM, rounding=SR, grad_dtype=GRAD_NATIVE)
    w, s = oracle.quantize(cfg, rng.standard_normal((rows, cols)) * 0.02)
    m = rng.standard_normal(rows * cols) * 1e-3
    v = rng.uniform(1e-7, 1e-5, rows * cols)
    for t in (1, 2, 7, 1000):
        g = rng.standard_normal(rows * cols) * 1e-3
        th_old = oracle.dequantize(cfg, w, s, rows, cols, np.float64).ravel()
        mt = b1 * m + (1 - b1) * g
        vt = b2 * v + (1 - b2) * g * g
        eta_t = lr / ((1 - b1 ** t) * (np.sqrt(vt / (1 - b2 ** t)) + eps))
        tht, err = np.zeros_like(m), np.zeros_like(m)
        oracle.step(cfg, lr=lr, beta1=b1, beta2=b2, eps=eps, step=t, seed=5, w=w, scale=s, grad=g, m=m, v=v,
                    rows=rows, cols=cols, dbg_theta_tilde=tht, dbg_err=err)
        th_new = oracle.dequantize(cfg, w, s, rows, cols, np.float64).ravel()
        np.testing.assert_allclose(v, vt, rtol=1e-14)
        np.testing.assert_allclose(tht, th_old - eta_t * mt, rtol=1e-12, atol=1e-16)        # plain Adam update
        np.testing.assert_allclose(err, tht - th_new, rtol=0, atol=1e-17)                    # line 2
        lhs = th_new - eta_t * b1 / (1 - b1) * m
        rhs = th_old - eta_t / (1 - b1) * mt
        np.testing.assert_allclose(lhs, rhs, rtol=0, atol=1e-13)
        assert np.abs(err).max() > 1e-6


# --------------------------------------------------------------------------- error definition and bounds
@pytest.mark.parametrize("fmt,rnd,sdt", [(FP8_E4M3, RTN, SCALE_NATIVE), (FP8_E4M3, SR, SCALE_NATIVE),
                                         (INT4, RTN, SCALE_BF16), (INT4, SR, SCALE_BF16)])
def test_error_is_before_minus_after_rounding_binary32(fmt, rnd, sdt):
    """e_{t+1} = theta~_{t+1} - theta^_{t+1} (Algorithm 2, line 2) in the binary32 instantiation: equal,
    bit for bit, to theta~ minus the dequantized stored result, and bounded by the grid gap."""
    rng = np.random.default_rng(14)
    rows, cols = 3, 320
    n = rows * cols
    cfg = oracle.Config(format=fmt, granularity=PER_BLOCK, scale_dtype=sdt, optimizer=SGDM, rounding=rnd,
                        grad_dtype=GRAD_BF16)
    from paper_2601_22101_b200.workloads import f32_to_bf16_bits
    w, s = oracle.quantize(cfg, (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32))
    m = np.zeros(n, np.float32)
    lr, beta = np.float32(1e-3), np.float32(0.9)
    for t in range(1, 6):
        g = f32_to_bf16_bits((rng.standard_normal(n) * 1e-3).astype(np.float32))
        tht, err = np.zeros(n, np.float32), np.zeros(n, np.float32)
        m_before = m.copy()
        oracle.step(cfg, lr=float(lr), beta1=float(beta), step=t, seed=9, w=w, scale=s, grad=g, m=m, rows=rows,
                    cols=cols, dbg_theta_tilde=tht, dbg_err=err)
        thq = oracle.dequantize(cfg, w, s, rows, cols, np.float32).ravel()
        assert (err == tht - thq).all()
        # gap of the grid around each element, in weight units
        sc = oracle.dequantize(cfg, np.full_like(w, 0x11 if fmt == INT4 else 0x38), s, rows, cols, np.float32).ravel()
        if fmt == INT4:
            gap = sc                                    # code 1 -> one integer step times the scale
        else:
            a = np.abs(thq / sc)                        # sc = 1.0 * scale
            gap = sc * np.maximum(2.0 ** (np.floor(np.log2(np.maximum(a, 2.0 ** -6))) - 3), 2.0 ** -9)
        bound = gap * (0.5 if rnd == RTN else 1.0) * (1 + 1e-3) + np.abs(tht) * 1e-2 * (sdt == SCALE_BF16)
        assert (np.abs(err) <= bound).all()
        # Algorithm 2, line 5 in the same arithmetic
        alpha = np.float32((1.0 / float(lr)) * (1.0 - 1.0 / float(beta)))
        mt = (m_before.astype(np.float64) * float(beta)
              + (np.float32(1.0 - float(beta)) * (g.astype(np.uint32) << 16).view(np.float32)).astype(np.float64))
        np.testing.assert_allclose(m, mt + float(alpha) * err.astype(np.float64), rtol=2e-6, atol=1e-9)


# --------------------------------------------------------------------------- Appendix A
@pytest.mark.parametrize("fmt,gran", [(FP8_E4M3, PER_BLOCK), (FP8_E4M3, PER_TENSOR), (INT4, PER_ROW)])
def test_ideal_injection_reproduces_master_weight_sgdm(fmt, gran):
    """Appendix A, Theorem (exact equivalence): storing e_t and injecting e_t/eta - e_{t+1}/(eta beta)
    gives the same quantized iterates as SGDM on full-precision master weights."""
    rng = np.random.default_rng(15)
    rows, cols, lr, beta = 5, 192, 5e-3, 0.9
    n = rows * cols
    cfg = oracle.Config(format=fmt, granularity=gran, optimizer=SGDM, rounding=RTN, grad_dtype=GRAD_NATIVE,
                        injection=INJECT_IDEAL)
    target = rng.standard_normal(n) * 0.02
    theta = rng.standard_normal((rows, cols)) * 0.02           # master weights
    m_mw = rng.standard_normal(n) * 1e-3
    w_mw, s_mw = oracle.quantize(cfg, theta)
    # initialisation of the injected method (Appendix A, Eq. init)
    w_im, s_im = oracle.quantize(cfg, theta)
    e_prev = theta.ravel() - oracle.dequantize(cfg, w_im, s_im, rows, cols, np.float64).ravel()
    m_im = m_mw - e_prev / (lr * beta)
    changed = 0
    for t in range(1, 61):
        g_mw = oracle.dequantize(cfg, w_mw, s_mw, rows, cols, np.float64).ravel() - target   # grad of 1/2|x - target|^2
        g_im = oracle.dequantize(cfg, w_im, s_im, rows, cols, np.float64).ravel() - target
        m_mw = beta * m_mw + (1 - beta) * g_mw
        theta = theta - lr * m_mw.reshape(rows, cols)
        w_new, s_mw = oracle.quantize(cfg, theta)
        changed += int((w_new != w_mw).sum())
        w_mw = w_new
        oracle.step(cfg, lr=lr, beta1=beta, step=t, w=w_im, scale=s_im, grad=g_im, m=m_im, rows=rows, cols=cols,
                    e_prev=e_prev)
        assert (w_im == w_mw).all(), t
        np.testing.assert_allclose(s_im, s_mw, rtol=1e-12)
    assert changed > n // 4          # the weights really moved across grid points


# --------------------------------------------------------------------------- Appendix C
def _stationary_second_moment(injection, L, lr, beta, sigma, chains=200000, steps=600, seed=16):
    rng = np.random.default_rng(seed)
    cfg = oracle.Config(format=ADDITIVE_NOISE, optimizer=SGDM, grad_dtype=GRAD_NATIVE, injection=injection)
    x = np.zeros(chains)
    m = np.zeros(chains)
    acc, cnt = 0.0, 0
    for t in range(1, steps + 1):
        g = L * x
        xi = rng.standard_normal(chains) * sigma
        oracle.step(cfg, lr=lr, beta1=beta, step=t, w=x, scale=None, grad=g, m=m, rows=1, cols=chains, noise=xi)
        if t > steps // 2:
            acc += float(np.mean(x * x))
            cnt += 1
    return acc / cnt


def test_appendix_c_stationary_second_moments():
    """1-D quadratic f = L/2 x^2 with q(x) = x + xi: stationary E[x^2] of the quantized iterate is
    2 s^2 / (2(1-b^2) - L eta (1-b)^2) for ECO and s^2 ((1-b^2) + 2 b L eta) / (L eta (2(1-b^2) - L eta (1-b)^2))
    for naive removal (Appendix C, closed forms of the ECO and naive regimes)."""
    gold = _golden("appendix_c_setting.txt")
    L, lr, beta, sigma = gold["L"], gold["eta"], gold["beta"], gold["sigma"]
    assert lr < 2 * (1 + beta) / ((1 - beta) * L)            # stability condition of Appendix C
    den = 2 * (1 - beta ** 2) - L * lr * (1 - beta) ** 2
    eco = 2 * sigma ** 2 / den
    naive = sigma ** 2 * ((1 - beta ** 2) + 2 * beta * L * lr) / (L * lr * den)
    got_eco = _stationary_second_moment(INJECT_ECO, L, lr, beta, sigma)
    got_naive = _stationary_second_moment(INJECT_NONE, L, lr, beta, sigma)
    assert abs(got_eco / eco - 1) < 0.02, (got_eco, eco)
    assert abs(got_naive / naive - 1) < 0.02, (got_naive, naive)
    assert abs(eco - gold["eco_expected"]) < 1e-3 and abs(naive - gold["naive_expected"]) < 1e-3
    # small-eta limits quoted in Sec. 3.4: ECO -> s^2/(1-b^2), naive ~ s^2/(2 L eta)
    small = 1e-2
    eco_small = _stationary_second_moment(INJECT_ECO, L, small, beta, sigma, chains=40000, steps=4000)
    assert abs(eco_small / (sigma ** 2 / (1 - beta ** 2)) - 1) < 0.05


def pin_master_weight_second_moments(chains=200000, steps=600, seed=17):
    """Appendix C, master-weight regime: full-precision x is kept, the gradient is taken at x^ = x + xi, and the
    update is plain SGDM on x (the oracle's step with the identity quantizer).  Stationary second moments against
    the closed forms u, v, w of that subsection and E[x^^2] = u + sigma^2."""
    gold = _golden("appendix_c_setting.txt")
    L, lr, beta, sigma = gold["L"], gold["eta"], gold["beta"], gold["sigma"]
    D = 2 * (1 + beta) - L * lr * (1 - beta)
    u = L * lr * sigma ** 2 * (1 + beta) / D
    v = L ** 2 * lr * sigma ** 2 * (beta - 1) / D
    w = 2 * L ** 2 * sigma ** 2 * (1 - beta) / D
    assert abs(u - gold["mw_u_expected"]) < 1e-6 and abs(v - gold["mw_v_expected"]) < 1e-6
    assert abs(w - gold["mw_w_expected"]) < 1e-6 and abs(u + sigma ** 2 - gold["mw_xhat2_expected"]) < 1e-6
    rng = np.random.default_rng(seed)
    cfg = oracle.Config(format=IDENTITY, optimizer=SGDM, grad_dtype=GRAD_NATIVE)
    x, m = np.zeros(chains), np.zeros(chains)
    acc = np.zeros(4)
    cnt = 0
    for t in range(1, steps + 1):
        xhat = x + rng.standard_normal(chains) * sigma
        oracle.step(cfg, lr=lr, beta1=beta, step=t, w=x, scale=None, grad=L * xhat, m=m, rows=1, cols=chains)
        if t > steps // 2:
            nxt = x + rng.standard_normal(chains) * sigma            # what the model would see now (not fed back)
            acc += [np.mean(x * x), np.mean(x * m), np.mean(m * m), np.mean(nxt * nxt)]
            cnt += 1
    gu, gv, gw, gx = acc / cnt
    assert abs(gu / u - 1) < 0.02, (gu, u)
    assert abs(gv / v - 1) < 0.05, (gv, v)
    assert abs(gw / w - 1) < 0.02, (gw, w)
    assert abs(gx / (u + sigma ** 2) - 1) < 0.01, (gx, u + sigma ** 2)


def test_appendix_c_master_weight_regime():
    pin_master_weight_second_moments()


def test_appendix_c_orders_the_three_regimes():
    """Sec. 3.4 at the golden setting: master weights sit at the quantization floor, ECO a constant factor above
    it, naive removal higher still -- as closed forms and as the ratios the paper draws from them."""
    gold = _golden("appendix_c_setting.txt")
    assert gold["mw_xhat2_expected"] < gold["eco_expected"] < gold["naive_expected"]
    beta, sigma = gold["beta"], gold["sigma"]
    assert abs(gold["eco_expected"] / (sigma ** 2 / (1 - beta ** 2)) - 1) < 0.01     # eta -> 0 limit already close


def test_memory_layout_matches_paper_count():
    """Sec. 4.4 (Discussion on Memory): 12 bytes per parameter with FP32 master weights, 9 without."""
    gold = _golden("paper_constants.txt")
    from paper_2601_22101_b200 import workloads as wl
    w = wl.c4(layers=1, experts=2)
    assert w.state_bytes_per_param() == gold["state_bytes_per_param_fp8_adam_no_master"] == 9
    assert w.state_bytes_per_param() + (4 - 1) == gold["state_bytes_per_param_fp32_master"] == 12


# --------------------------------------------------------------------------- Sec. 4 recipe: AdamW decay, clipping factor
def test_identity_quantizer_with_decay_and_clipping_matches_adamw():
    """Sec. 4.2 trains with AdamW (weight decay 0.1) and gradient clipping at norm 1.  With q = id the
    step must be the library's AdamW on the clipped gradient: theta (1 - eta lambda) - eta_t m_hat."""
    rng = np.random.default_rng(12)
    n, lr, b1, b2, eps, wd, clip = 193, 2e-3, 0.9, 0.95, 1e-8, 0.1, 1.0
    cfg = oracle.Config(format=IDENTITY, optimizer=ADAM, grad_dtype=GRAD_NATIVE)
    theta0 = rng.standard_normal(n)
    w, m, v = theta0.copy(), np.zeros(n), np.zeros(n)
    p = torch.tensor(theta0, dtype=torch.float64, requires_grad=True)
    topt = torch.optim.AdamW([p], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd)
    for t in range(1, 16):
        g = rng.standard_normal(n) * (3.0 if t % 2 else 0.01)          # clipped on odd steps, untouched on even ones
        p.grad = torch.tensor(g)
        total = float(torch.nn.utils.clip_grad_norm_([p], clip))
        factor = min(1.0, clip / (total + 1e-6))                        # the factor torch applies
        oracle.step(cfg, lr=lr, beta1=b1, beta2=b2, eps=eps, step=t, w=w, scale=None, grad=g, m=m, v=v,
                    rows=1, cols=n, weight_decay=wd, grad_scale=factor)
        topt.step()
        np.testing.assert_allclose(w, p.detach().numpy(), rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(m, topt.state[p]["exp_avg"].numpy(), rtol=1e-11, atol=1e-14)


def test_sgdm_decoupled_decay_closed_form():
    """One SGDM step with decay: theta~ = theta (1 - eta lambda) - eta (beta m + (1 - beta) c g)."""
    cfg = oracle.Config(format=IDENTITY, optimizer=SGDM, grad_dtype=GRAD_NATIVE)
    w, m, g = np.array([2.0, -1.0, 0.5]), np.array([0.1, 0.2, -0.3]), np.array([1.0, -2.0, 4.0])
    lr, b, wd, c = 0.05, 0.8, 0.3, 0.25
    expect_m = b * m + (1 - b) * (c * g)
    expect_w = w * (1 - lr * wd) - lr * expect_m
    oracle.step(cfg, lr=lr, beta1=b, step=1, w=w, scale=None, grad=g, m=m, rows=1, cols=3, weight_decay=wd, grad_scale=c)
    np.testing.assert_allclose(w, expect_w, rtol=1e-14)
    np.testing.assert_allclose(m, expect_m, rtol=1e-14)


def test_grad_scale_equals_prescaled_gradient_bit_for_bit():
    """A factor on the bf16 gradient is the same as handing in the binary32 product (quantized path, binary32)."""
    rng = np.random.default_rng(13)
    rows, cols, gs = 6, 256, 0.37
    x = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    qcfg = oracle.Config(format=FP8_E4M3, granularity=PER_BLOCK, optimizer=ADAM, rounding=SR)
    w0, s0 = oracle.quantize(oracle.Config(format=FP8_E4M3, granularity=PER_BLOCK), x)
    g32 = (rng.standard_normal(rows * cols) * 1e-3).astype(np.float32)
    gb = (g32.view(np.uint32) >> 16).astype(np.uint16)                  # bf16 patterns (truncation is fine here)
    gf = (gb.astype(np.uint32) << 16).view(np.float32)
    out = []
    for variant in range(2):
        w, s = w0.copy(), s0.copy()
        m, v = np.zeros(rows * cols, np.float32), np.zeros(rows * cols, np.float32)
        if variant == 0:
            oracle.step(qcfg, lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, step=1, seed=5, w=w, scale=s, grad=gb, m=m, v=v,
                        rows=rows, cols=cols, grad_scale=gs)
        else:
            ncfg = oracle.Config(format=FP8_E4M3, granularity=PER_BLOCK, optimizer=ADAM, rounding=SR, grad_dtype=GRAD_NATIVE)
            oracle.step(ncfg, lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, step=1, seed=5, w=w, scale=s,
                        grad=(gf * np.float32(gs)).astype(np.float32), m=m, v=v, rows=rows, cols=cols)
        out.append((w, s, m, v))
    for a, b in zip(out[0], out[1]):
        assert (a.view(np.uint8) == b.view(np.uint8)).all()
