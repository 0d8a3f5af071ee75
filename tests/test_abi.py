"""Host-only checks of the C-ABI boundary: the library loads, exports every symbol the header
declares, and rejects bad arguments before any launch (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2605_08565_b200 import build
    build.build()
    from paper_2605_08565_b200 import binding
    return binding.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "mxq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mxq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2605_08565_b200 import binding
    names = _declared_functions()
    assert len(names) >= 11
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_version_and_status_strings(lib):
    assert lib.mxq_version() >= 100
    for s in range(0, 8):
        assert lib.mxq_status_string(s)
    assert lib.mxq_status_string(0) == b"ok"
    assert lib.mxq_global_scale_from_amax(2688.0) == 1.0
    assert lib.mxq_global_scale_from_amax(0.0) == 1.0
    assert lib.mxq_tensor_mse_workspace_bytes(10) >= 8


def test_argument_errors_are_caught_on_the_host(lib):
    # fake, 16-byte aligned "device" addresses: validation must fail before anything is launched
    X, C, S, E = 0x10000, 0x20000, 0x30000, 0x40000
    q = lib.mxq_quantize_ex
    ok_args = dict(x=X, dtype=0, n=64, B=16, fmt=1, recipe=0, g=1.0, dg=0, codes=C, scales=S, sse=E, stream=0)

    def call(**kw):
        a = dict(ok_args)
        a.update(kw)
        return q(a["x"], a["dtype"], a["n"], a["B"], a["fmt"], a["recipe"], a["g"], a["dg"], a["codes"], a["scales"],
                 a["sse"], a["stream"])

    assert call(x=0) == 1 and call(codes=0) == 1 and call(scales=0) == 1
    assert call(dtype=2) == 2 and call(fmt=3) == 2 and call(fmt=-1) == 2 and call(recipe=6) == 2
    assert call(B=3) == 3 and call(B=128) == 3 and call(n=0) == 3 and call(n=60) == 3
    assert call(x=X + 4) == 4 and call(codes=C + 8) == 4 and call(sse=E + 4) == 4
    assert call(g=0.0) == 5 and call(g=-1.0) == 5 and call(g=float("inf")) == 5 and call(g=float("nan")) == 5
    assert lib.mxq_tensor_mse(E, 4, 64, 0x50000, 0, 0, 0) == 6
    assert lib.mxq_tensor_mse(E, 4, 64, 0x50000, 0x60000, 8, 0) == 6
    assert lib.mxq_tensor_mse(0, 4, 64, 0x50000, 0x60000, 8192, 0) == 1
    assert lib.mxq_tensor_amax(0, 0, 64, E, 0, 0) == 1
    assert lib.mxq_tensor_amax(X, 5, 64, E, 0, 0) == 2
    assert lib.mxq_dequantize(C, S, 64, 16, 1, 1.0, 0, 0, 0) == 1
    assert lib.mxq_dequantize(C, S, 64, 5, 1, 1.0, X, 0, 0) == 3
    assert lib.mxq_dequantize(C, S, 64, 16, 1, 0.0, X, 0, 0) == 5
    assert lib.mxq_dequantize_ex(C, S, 64, 16, 1, 0.0, 0, X, 0, 0) == 5
    assert lib.mxq_dequantize_ex(C, S, 64, 16, 1, 0.0, E + 2, X, 0, 0) == 4     # misaligned device scale
    assert lib.mxq_dequantize_ex(C, S, 64, 16, 1, 0.0, E, 0, 0, 0) == 1
    qm = lib.mxq_quantize_mse
    assert qm(X, 0, 64, 16, 1, 0, 1.0, 0, C, S, E, 0, 0x60000, 8192, 0) == 1           # no MSE output
    assert qm(X, 0, 64, 16, 1, 0, 1.0, 0, C, S, E, 0x50000, 0, 8192, 0) == 6           # no workspace
    assert qm(X, 0, 64, 16, 1, 0, 1.0, 0, C, S, E, 0x50000, 0x60000, 4096, 0) == 6     # workspace too small
    assert qm(X, 0, 60, 16, 1, 0, 1.0, 0, C, S, E, 0x50000, 0x60000, 8192, 0) == 3
    assert qm(X, 0, 64, 16, 1, 0, 1.0, 0, C, S, E, 0x50004, 0x60000, 8192, 0) == 4


def test_binding_refuses_cpu_tensors():
    import torch
    from paper_2605_08565_b200 import binding
    x = torch.zeros(64)
    with pytest.raises(binding.MxqError):
        binding.quantize(x, 16, binding.MXQ_SF_UE4M3, binding.MXQ_ABSMAX)
