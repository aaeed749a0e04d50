"""The C-ABI library loads without a GPU and exports every function that include/sradamw.h declares;
argument errors are reported before any device work."""

import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2502_20566_b200 import build
    build.build()
    from paper_2502_20566_b200 import binding
    return binding.lib()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "sradamw.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(?:sr_status|size_t|uint64_t|uint32_t|int|const char\*)\s+\*?\s*(\w+)\s*\(", text)
    return sorted(set(names))


def test_header_functions_are_exported(lib):
    from paper_2502_20566_b200 import binding
    declared = _declared_functions()
    assert len(declared) >= 12
    for name in declared:
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTS) == [d for d in declared if d in binding.EXPORTS]
    assert set(binding.EXPORTS) <= set(declared)


def test_abi_version_and_strings(lib):
    assert lib.sr_abi_version() == 1
    for s in range(5):
        assert len(lib.sr_status_string(s)) > 0


def test_hparams_struct_layout(lib):
    from paper_2502_20566_b200 import binding
    assert ctypes.sizeof(binding.HParams) == 48
    assert binding.HParams.grad_scale_dev.offset == 32 and binding.HParams.flags.offset == 40


def test_workspace_size_follows_the_tree(lib):
    f = lib.grad_sqnorm_workspace_bytes
    assert f(0) == 0 and f(1) == 0 and f(8192) == 0
    assert f(8193) == 2 * 8
    assert f(8192 * 8192) == 8192 * 8
    assert f(8192 * 8192 + 1) == (8193 + 2) * 8


def test_argument_errors_come_before_device_work(lib):
    from paper_2502_20566_b200 import binding as b
    hp = b.hparams(6e-4, 0.9, 0.95, 1e-8, 0.1)
    call = lambda hp_, step: lib.sr_adamw_step(None, None, 0, None, None, 0, ctypes.byref(hp_), 1, step, 0, 0, None)
    assert call(hp, 1) == b.SR_OK                              # n == 0: no-op
    assert call(hp, 0) == b.SR_ERR_INVALID_ARG                 # 1 - beta^0 = 0
    bad = b.hparams(6e-4, 1.0, 0.95, 1e-8, 0.1)
    assert call(bad, 1) == b.SR_ERR_INVALID_ARG
    bad = b.hparams(float("nan"), 0.9, 0.95, 1e-8, 0.1)
    assert call(bad, 1) == b.SR_ERR_INVALID_ARG
    bad = b.hparams(6e-4, 0.9, 0.95, 1e-8, 0.1, flags=16)
    assert call(bad, 1) == b.SR_ERR_INVALID_ARG
    bad = b.hparams(6e-4, 0.9, 0.95, 1e-8, 0.1)
    bad.struct_size = 44
    assert call(bad, 1) == b.SR_ERR_INVALID_ARG
    assert lib.sr_adamw_step(None, None, 0, None, None, 8, ctypes.byref(hp), 1, 1, 0, 0, None) == b.SR_ERR_INVALID_ARG
    assert lib.sr_downcast_f32_bf16(None, None, 0, 1, 0, 0, 0, None) == b.SR_OK
    assert lib.sr_downcast_f32_bf16(None, None, 5, 1, 0, 0, 0, None) == b.SR_ERR_INVALID_ARG
    assert lib.grad_sqnorm(None, 0, 10, None, None, 0, None) == b.SR_ERR_INVALID_ARG
    out = ctypes.c_double()
    assert lib.grad_sqnorm(ctypes.byref(out), 1, 10**6, ctypes.byref(out), None, 0, None) == b.SR_ERR_WORKSPACE


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2502_20566_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.lib()
