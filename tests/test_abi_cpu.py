"""CPU-side checks of the C-ABI library: it builds, loads, exports what the header declares,
and its host-only helpers behave.  No compute call is made (no GPU needed)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from ivit_inputs import ExpParams, Scale
from ivit_inputs.gen import dyadic

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2207_01405_b200 import build
    build.build()
    from paper_2207_01405_b200 import binding
    return binding.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ivit.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ivit_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2207_01405_b200 import binding
    names = declared_symbols()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/ivit.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_strerror_and_codes(lib):
    assert lib.ivit_strerror(0) == b"ok"
    msgs = {lib.ivit_strerror(-i) for i in range(1, 8)}
    assert len(msgs) == 7 and b"unknown error" not in msgs


def test_dyadic_from_double_host_helper(lib):
    from paper_2207_01405_b200 import binding
    rng = np.random.default_rng(0)
    for r in np.exp(rng.uniform(np.log(1e-6), np.log(0.9), 200)):
        m, s = binding.dyadic_from_double(float(r))
        assert (m, s) == dyadic(float(r))
        assert 2 ** 30 <= m < 2 ** 31 and abs(m / 2 ** s - r) <= r * 2.0 ** -31
    m, s = C.c_int32(), C.c_int32()
    assert lib.ivit_dyadic_from_double(-1.0, C.byref(m), C.byref(s)) == -1
    assert lib.ivit_dyadic_from_double(1e-30, C.byref(m), C.byref(s)) == -3
    assert lib.ivit_dyadic_from_double(1.5, C.byref(m), C.byref(s)) == -3      # ratios >= 1 are not representable


def test_validate_exp_params_bounds(lib):
    from paper_2207_01405_b200 import binding
    assert binding.validate_exp_params(ExpParams(11, 15), 197, False) == 0
    assert binding.validate_exp_params(ExpParams(23, 15), 577, False) == 0
    assert binding.validate_exp_params(ExpParams(33, 23), 1536, True) == 0
    assert binding.validate_exp_params(ExpParams(0, 15), 197, False) == -3          # I0 >= 1
    assert binding.validate_exp_params(ExpParams(11, 25), 197, False) == -3         # N <= 24
    assert binding.validate_exp_params(ExpParams(11, 15, M=40), 197, False) == -3   # M fixed at 45
    assert binding.validate_exp_params(ExpParams(1, 3), 10, False) == -3            # I0 * 2^N >= 2^14
    assert binding.validate_exp_params(ExpParams(600, 23), 64, False) == -3         # row sum must fit 32 bits
    assert binding.validate_exp_params(ExpParams(300, 23), 64, True) == -3          # 2 * I0 * 2^N < 2^32


def test_validate_scale(lib):
    from paper_2207_01405_b200 import binding
    good = Scale(np.array([2 ** 30, 2 ** 31 - 1], np.int32), np.array([31, 62], np.uint8))
    assert binding.validate_scale(good) == 0
    assert binding.validate_scale(Scale(np.array([0], np.int32), np.array([31], np.uint8))) == -3
    assert binding.validate_scale(Scale(np.array([5], np.int32), np.array([63], np.uint8))) == -3
    assert binding.validate_scale(Scale(np.array([5], np.int32), np.array([30], np.uint8))) == -3


def test_context_needs_a_gpu(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2207_01405_b200 import binding
    with pytest.raises(RuntimeError):
        binding.Context(0)
    h = C.c_void_p()
    assert lib.ivit_ctx_create(C.byref(h), 0, None) == -6     # no device: fails loudly, no CPU path
