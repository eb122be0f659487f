"""The C-ABI library loads, exports every function the header declares, and rejects bad arguments
on the host before touching the device (no compute happens in this file)."""
import ctypes
import os
import re

import pytest

from paper_2604_25925_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "sgbv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sgbv_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert set(binding.EXPORTS) <= set(names) and len(names) >= 7
    for n in names:
        assert getattr(lib, n) is not None


def test_status_strings(lib):
    for code in (0, -1, -2, -3, -4, -5, -6, -99):
        s = binding.status_string(code)
        assert isinstance(s, str) and s
    assert "TEMPERATURE" in binding.status_string(-3)


def test_workspace_bytes(lib):
    n = binding.workspace_bytes(8, 4, 4, 32000)
    assert n > 0 and n % 256 == 0
    assert binding.workspace_bytes(64, 8, 8, 151936) > n
    with pytest.raises(binding.SgbvError) as e:
        binding.workspace_bytes(0, 4, 4, 32000)
    assert e.value.code == -2
    for bad in ((1, 65, 1, 10), (1, 1, 65, 10), (1, 1, 1, (1 << 22) + 1), (1, 1, 0, 5)):
        with pytest.raises(binding.SgbvError):
            binding.workspace_bytes(*bad)
    with pytest.raises(binding.SgbvError):
        binding.workspace_bytes(1, 1, 1, 10, dtype=7)


def test_argument_errors_are_reported_before_any_launch(lib):
    buf = (ctypes.c_float * 64)()
    p = ctypes.addressof(buf)
    good = dict(zq=p, zp=p, tok=p, u=p, B=1, K=1, g=1, V=4, T=1.0, a=p, f=p, t=p)

    def call(**kw):
        a = dict(good, **kw)
        return lib.sgbv_verify(a["zq"], a["zp"], a["tok"], a["u"], a["B"], a["K"], a["g"], a["V"], a["T"],
                               a["a"], a["f"], a["t"], None)

    assert call(zq=None) == -1 and call(t=None) == -1 and call(u=None) == -1
    assert call(B=0) == -2 and call(K=65) == -2 and call(g=0) == -2 and call(V=0) == -2
    assert call(T=0.0) == -3 and call(T=-1.0) == -3 and call(T=float("nan")) == -3 and call(T=float("inf")) == -3
    assert call(zq=p + 2) == -4 and call(tok=p + 1) == -4
    # extended form: workspace too small / misaligned
    rc = lib.sgbv_verify_ex(p, p, 0, p, p, 1, 1, 1, 4, 1.0, p, p, p, p, 16, None, None, None, None)
    assert rc == -5
    rc = lib.sgbv_verify_ex(p, p, 3, p, p, 1, 1, 1, 4, 1.0, p, p, p, None, 0, None, None, None, None)
    assert rc == -2
    rc = lib.sgbv_verify_host(None, p, 0, p, p, 1, 1, 1, 4, 1.0, p, p, p, None, None)
    assert rc == -1
    rc = lib.sgbv_verify_host(p, p, 0, p, p, 1, 1, 1, 4, 0.0, p, p, p, None, None)
    assert rc == -3


def test_binding_refuses_host_tensors_on_the_device_entry_point(lib):
    import torch
    z = torch.zeros((1, 1, 2, 4))
    with pytest.raises(ValueError):
        binding.sgbv_verify(z, z[:, :, :1].contiguous(), torch.zeros((1, 1, 1), dtype=torch.int32),
                            torch.zeros((1, 2)), 1.0)
