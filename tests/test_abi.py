"""The C-ABI library loads, exports every declared symbol and validates arguments on the host
(no kernel is launched by anything in this file, so it runs without a GPU)."""
import ctypes
import os
import re

import pytest

import paper_2405_18425_b200 as vig
from paper_2405_18425_b200 import build as vig_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "vig_bigla.h")


@pytest.fixture(scope="module")
def lib():
    vig_build.build()
    return vig.load()


def _declared_symbols():
    text = re.sub(r"/\*.*?\*/", "", open(HEADER).read(), flags=re.S)
    return sorted(set(re.findall(r"\b(vig_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert {"vig_bigla_fwd", "vig_bigla_fwd_bf16", "vig_bigla_fwd_f32", "vig_gate_prep_bf16", "vig_gate_prep_f32",
            "vig_bigla_fwd_host", "vig_bigla_fwd_ws_bf16", "vig_bigla_workspace_bytes", "vig_status_string",
            "vig_last_device_status", "vig_kernel_launch_count"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in vig_bigla.h but not exported"


def test_status_strings(lib):
    seen = set()
    for code in range(0, -8, -1):
        s = vig.status_string(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 8
    assert vig.status_string(-99) == "unknown status"


A = 0x10000  # fake, 16-byte aligned, never dereferenced: validation fails before any CUDA call


@pytest.mark.parametrize("fn", ["vig_bigla_fwd", "vig_bigla_fwd_bf16", "vig_bigla_fwd_f32"])
def test_forward_argument_validation(lib, fn):
    f = getattr(lib, fn)
    before = vig.vig_kernel_launch_count()
    ok = [A, A, A, A, A, A, 2, 2, 8, 16, 32, None]
    for i in range(6):
        bad = list(ok)
        bad[i] = None
        assert f(*bad) == -1
        bad = list(ok)
        bad[i] = A + 8
        assert f(*bad) == -4
    for i, val in ((6, -1), (7, -1), (8, -1), (9, 0), (10, 0), (9, -16)):
        bad = list(ok)
        bad[i] = val
        assert f(*bad) == -2
    big = list(ok)
    big[9], big[10] = 512, 32
    assert f(*big) == -3
    big[9], big[10] = 16, 1024
    assert f(*big) == -3
    # empty problems are valid and launch nothing
    for i in (6, 7, 8):
        e = list(ok)
        e[i] = 0
        assert f(*e) == 0
    assert vig.vig_kernel_launch_count() == before


@pytest.mark.parametrize("fn", ["vig_gate_prep_bf16", "vig_gate_prep_f32"])
def test_gate_prep_argument_validation(lib, fn):
    f = getattr(lib, fn)
    before = vig.vig_kernel_launch_count()
    ok = [A, A, A, A, 2, 2, 8, 16, 16.0, None]
    for i in range(4):
        bad = list(ok)
        bad[i] = None
        assert f(*bad) == -1
        bad = list(ok)
        bad[i] = A + 4
        assert f(*bad) == -4
    for i, val in ((4, -1), (5, -2), (6, -3), (7, 0), (8, 0.0), (8, -1.0), (8, float("inf")), (8, float("nan"))):
        bad = list(ok)
        bad[i] = val
        assert f(*bad) == -2
    e = list(ok)
    e[6] = 0
    assert f(*e) == 0
    assert vig.vig_kernel_launch_count() == before


def test_host_entry_validation(lib):
    f = lib.vig_bigla_fwd_host
    ok = [A, A, A, A, A, A, 1, 1, 4, 16, 32, 16.0, 1, None]
    bad = list(ok); bad[3] = None
    assert f(*bad) == -1
    bad = list(ok); bad[11] = 0.0
    assert f(*bad) == -2
    bad = list(ok); bad[12] = 7
    assert f(*bad) == -3
    bad = list(ok); bad[9] = 1000
    assert f(*bad) == -3
    e = list(ok); e[6] = 0
    assert f(*e) == 0


def test_workspace_query_and_ws_validation(lib):
    assert vig.vig_bigla_workspace_bytes(0, 4, 196, 32, 64) == 0
    assert vig.vig_bigla_workspace_bytes(8, 4, 196, 32, 64, vig.VIG_DTYPE_F32) == 0
    assert vig.vig_bigla_workspace_bytes(64, 12, 196, 32, 64) == 0          # one block per unit: no scratch
    need = vig.vig_bigla_workspace_bytes(8, 4, 4096, 24, 48)
    assert need > 0 and need % 256 == 0
    f = lib.vig_bigla_fwd_ws_bf16
    args = [A, A, A, A, A, A, 8, 4, 4096, 24, 48]
    assert f(*args, None, 0, None) == -6
    assert f(*args, A, need - 1, None) == -6
    assert f(*args, A + 16, need, None) == -6                                 # not 256-byte aligned
    assert f(None, *args[1:], A, need, None) == -1


def test_binding_refuses_cpu_tensors(lib):
    import torch

    t = torch.zeros(1, 1, 4, 16)
    with pytest.raises(ValueError):
        vig.vig_bigla_fwd_f32(t, t, t, t, t, t)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2405_18425_b200 import binding

    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "libvig_bigla.so"))
    with pytest.raises(ImportError, match="no CPU or PyTorch fallback"):
        binding.load()
