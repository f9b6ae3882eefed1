"""Do the pins bite?  Each case plants ONE plausible mistake in a scratch copy of the oracle's source (a text
substitution, compiled to a library of its own in a temporary folder), routes the oracle module to that build
and requires the named pin to fail.  The committed oracle is never touched, and nothing here runs on a GPU.
"""
import os
import subprocess

import pytest

import oracle
import test_oracle_optimizer as pins_opt
import test_oracle_scale as pins_scale
from oracle import ADAM, FP8_E4M3, INT4, PER_BLOCK, PER_ROW, PER_TENSOR, SCALE_BF16, SCALE_NATIVE, SGDM, SR

SRC = os.path.join(os.path.dirname(os.path.abspath(oracle.__file__)), "eco_oracle.cpp")

# name, text in the oracle, replacement, pins that must notice
MUTATIONS = [
    ("scale and grid factor computed with rho / 2 (f32 scales)",
     "        s = amax / rho;\n        inv = rho / amax;",
     "        s = amax / (rho / R(2));\n        inv = (rho / R(2)) / amax;",
     [lambda: pins_scale.pin_quantize(FP8_E4M3, PER_BLOCK, 128, SCALE_NATIVE),
      lambda: pins_scale.pin_quantize(INT4, PER_TENSOR, 128, SCALE_NATIVE),
      lambda: pins_scale.pin_step(FP8_E4M3, PER_ROW, 128, SCALE_NATIVE, ADAM)]),
    ("grid factor alone with rho / 2",
     "        inv = rho / amax;",
     "        inv = (rho / R(2)) / amax;",
     [lambda: pins_scale.pin_quantize(FP8_E4M3, PER_TENSOR, 128, SCALE_NATIVE)]),
    ("stored scale alone with rho / 2",
     "        s = amax / rho;\n",
     "        s = amax / (rho / R(2));\n",
     [lambda: pins_scale.pin_quantize(FP8_E4M3, PER_BLOCK, 32, SCALE_NATIVE)]),
    ("bf16 scale computed with rho / 2",
     "f32_to_bf16_rne(static_cast<float>(amax / rho))",
     "f32_to_bf16_rne(static_cast<float>(amax / (rho / R(2))))",
     [lambda: pins_scale.pin_quantize(FP8_E4M3, PER_BLOCK, 128, SCALE_BF16),
      lambda: pins_scale.pin_step(INT4, PER_BLOCK, 128, SCALE_BF16, SGDM)]),
    ("rho of E4M3 taken as 480 (the non-FN flavour's largest value)",
     "format == FMT_FP8_E4M3 ? R(448)",
     "format == FMT_FP8_E4M3 ? R(480)",
     [lambda: pins_scale.pin_quantize(FP8_E4M3, PER_BLOCK, 128, SCALE_NATIVE)]),
    ("every scale block runs on to the end of its row",
     "    *len = (cols - c0 < static_cast<uint64_t>(cfg.block)) ? cols - c0 : cfg.block;",
     "    *len = cols - c0;",
     [lambda: pins_scale.pin_quantize(FP8_E4M3, PER_BLOCK, 128, SCALE_NATIVE)]),
    ("bias correction with t + 1",
     "const double t = static_cast<double>(h.step);",
     "const double t = static_cast<double>(h.step + 1);",
     [lambda: pins_opt.test_identity_quantizer_reduces_to_library_optimizer(ADAM),
      lambda: pins_opt.test_adam_one_step_identity(FP8_E4M3, PER_BLOCK)]),
    ("sign of alpha flipped",
     "s.alpha = R((1.0 / h.lr) * (1.0 - 1.0 / h.beta1));",
     "s.alpha = R((1.0 / h.lr) * (1.0 / h.beta1 - 1.0));",
     [lambda: pins_opt.test_lemma_3_5_virtual_sequence_telescopes(FP8_E4M3, PER_BLOCK, SCALE_NATIVE, SR)]),
    ("tentative weight taken with the OLD momentum",
     "tht = std::fma(sc.neg_lr, mt, th);",
     "tht = std::fma(sc.neg_lr, m[i], th);",
     [pins_opt.test_sgdm_closed_form_one_step, pins_opt.pin_master_weight_second_moments]),
    ("undampened momentum (no 1 - beta on the gradient)",
     "const R mt = std::fma(sc.beta1, m[i], sc.one_minus_beta1 * gi);",
     "const R mt = std::fma(sc.beta1, m[i], gi);",
     [lambda: pins_opt.pin_master_weight_second_moments(chains=50000, steps=400)]),
    ("position of a slice ignored by the random stream",
     "element_random_word(hyper.seed, hyper.step, tensor_id, hyper.index_base + i)",
     "element_random_word(hyper.seed, hyper.step, tensor_id, i)",
     [lambda: pins_scale.test_a_slice_of_rows_with_its_position_rounds_like_the_whole_tensor(FP8_E4M3, PER_BLOCK, 128)]),
    ("position added after the division by four",
     "const uint32_t ctr[4] = {static_cast<uint32_t>(i >> 2), tensor_id,",
     "const uint32_t ctr[4] = {static_cast<uint32_t>(static_cast<uint32_t>(i) >> 2), tensor_id,",
     [pins_scale.test_position_enters_the_counter_as_a_64_bit_sum]),
]


@pytest.mark.parametrize("name,old,new,pins", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_a_planted_mistake_is_caught(name, old, new, pins, tmp_path):
    text = open(SRC).read()
    assert text.count(old) == 1, f"the text to mutate must occur exactly once: {old!r}"
    src = tmp_path / "mutant.cpp"
    src.write_text(text.replace(old, new))
    lib = tmp_path / "libmutant.so"
    subprocess.run(["g++", "-O1", "-std=c++17", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
                    str(src), "-o", str(lib)], check=True)
    for pin in pins:
        pin()                                        # green on the committed oracle
        with oracle.use_library(str(lib)):
            with pytest.raises(AssertionError):
                pin()
