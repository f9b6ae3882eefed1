"""CPU-side checks of the boundary: the shared library builds, loads and exports every symbol the
header declares; host-side validation rejects bad arguments before any CUDA work."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2601_22101_b200 import build, eco
    build.build()
    return eco.load_library()


def _declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(eco_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol(lib):
    from paper_2601_22101_b200 import eco
    declared = _declared_symbols()
    assert declared == set(eco.EXPORTED)
    for name in declared:
        assert hasattr(lib, name), name
    assert re.fullmatch(r"\d+\.\d+\.\d+", eco.eco_version())


def test_struct_layouts_match_header(lib):
    from paper_2601_22101_b200 import eco
    assert ctypes.sizeof(eco.eco_config) == 32
    assert ctypes.sizeof(eco.eco_tensor) == 5 * 8 + 2 * 8 + 2 * 4


def test_validation_rejects_before_touching_cuda(lib):
    from paper_2601_22101_b200 import eco
    with pytest.raises(eco.EcoError) as e:
        eco.eco_create(eco.Config(format=7), [eco.Tensor(None, None, None, None, None, 1, 1, 0)])
    assert e.value.status == eco.ECO_ERR_UNSUPPORTED
    with pytest.raises(eco.EcoError) as e:
        eco.eco_create(eco.Config(block=64), [eco.Tensor(None, None, None, None, None, 1, 1, 0)])
    assert e.value.status == eco.ECO_ERR_UNSUPPORTED and "128" in str(e.value)
    with pytest.raises(eco.EcoError) as e:
        eco.eco_create(eco.Config(scale_dtype=3), [eco.Tensor(None, None, None, None, None, 1, 1, 0)])
    assert e.value.status == eco.ECO_ERR_UNSUPPORTED
    with pytest.raises(eco.EcoError) as e:
        eco.eco_create(eco.Config(), [])
    assert e.value.status == eco.ECO_ERR_INVALID_ARG
    # the configurations added beside the paper's own (E5M2, 1x32 blocks, power-of-two scales) pass the configuration
    # check: what is refused next is the empty tensor (rows = 0), an argument error
    for cfg in (eco.Config(format=eco.ECO_FORMAT_FP8_E5M2), eco.Config(block=32, scale_dtype=eco.ECO_SCALE_E8M0)):
        with pytest.raises(eco.EcoError) as e:
            eco.eco_create(cfg, [eco.Tensor(None, None, None, None, None, 0, 128, 0)])
        assert e.value.status == eco.ECO_ERR_INVALID_ARG and "rows" in str(e.value)
    with pytest.raises(eco.EcoError) as e:                    # more than 2^34 elements
        eco.eco_create(eco.Config(), [eco.Tensor(None, None, None, None, None, 1 << 20, 1 << 14, 0)])
    assert e.value.status == eco.ECO_ERR_INVALID_ARG and "2^34" in str(e.value)
    with pytest.raises(eco.EcoError) as e:                    # INT4 packs two codes per byte
        eco.eco_create(eco.Config(format=eco.ECO_FORMAT_INT4), [eco.Tensor(None, None, None, None, None, 4, 127, 0)])
    assert e.value.status == eco.ECO_ERR_INVALID_ARG
    with pytest.raises(eco.EcoError) as e:
        eco.eco_step(None, 1e-3, 0.9, 0.95, 1e-8, 1, 0)
    assert e.value.status == eco.ECO_ERR_INVALID_ARG
    with pytest.raises(eco.EcoError) as e:
        eco.eco_set_option("no_such_option", 1)
    assert e.value.status == eco.ECO_ERR_INVALID_ARG
    eco.eco_destroy(None)     # allowed


def test_no_cpu_fallback_without_a_device(lib):
    """Without a CUDA device the product path fails loudly instead of computing on the CPU."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    from paper_2601_22101_b200 import eco, workloads as wl
    from paper_2601_22101_b200.state import DeviceState
    with pytest.raises(RuntimeError):
        DeviceState(wl.c1())
    import numpy as np
    buf = np.zeros(64, np.uint8)
    with pytest.raises(eco.EcoError) as e:
        eco.eco_create(eco.Config(optimizer=eco.ECO_OPT_SGDM),
                       [eco.Tensor(buf, buf, buf, buf, None, 1, 16, 0)])
    assert e.value.status in (eco.ECO_ERR_CUDA, eco.ECO_ERR_ALIGNMENT, eco.ECO_ERR_INVALID_ARG)


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2601_22101_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert "import oracle" not in text and "from oracle" not in text and "eco_oracle" not in text, fn


def test_workload_shapes_match_the_stated_parameter_sets():
    from paper_2601_22101_b200 import workloads as wl
    assert wl.c1().numel == 1024 * 1024
    assert wl.c2().numel == 35_192_832 and len(wl.c2().tensors) == 38
    assert wl.c3().numel == 999_751_680 and len(wl.c3().tensors) == 183
    assert wl.c4().numel == 2_147_483_648 and len(wl.c4().tensors) == 2048
    assert wl.c4(expert_mats=3).numel == 3_221_225_472
    assert sum(t.zero_grad for t in wl.c4().tensors) == len(wl.c4().tensors) // 2
    assert wl.c5().numel == 15_482_880_000 and len(wl.c5().tensors) == 5349
    assert abs(wl.c2().algorithmic_bytes_per_param() - 20.0625) < 1e-9
    assert abs(wl.c1().algorithmic_bytes_per_param() - 12.0) < 1e-5
    assert abs(wl.c5().algorithmic_bytes_per_param() - (11 + 4 / 128)) < 1e-3
