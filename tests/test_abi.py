"""The C-ABI library loads and exports every symbol include/rr.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def librr():
    from paper_2402_12399_b200 import build
    return ctypes.CDLL(build.build())


def _declared():
    text = open(os.path.join(ROOT, "include", "rr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rr_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_expected_entry_points():
    names = _declared()
    for n in ("rr_route", "rr_route_workspace_bytes", "rr_moe_fwd", "rr_moe_bwd", "rr_moe_workspace_bytes",
              "rr_check", "rr_status_string", "rr_gate_fwd", "rr_gate_bwd", "rr_gate_workspace_bytes", "rr_aux_loss_fwd", "rr_aux_loss_bwd",
              "rr_aux_workspace_bytes", "rr_gate_route", "rr_gate_route_workspace_bytes", "rr_route_noalloc", "rr_route_loss",
              "rr_route_loss_workspace_bytes", "rr_test_set_wait_limit_ns"):
        assert n in names


def test_every_declared_symbol_is_exported(librr):
    for n in _declared():
        assert hasattr(librr, n), n


def test_host_side_argument_checks(librr):
    n = ctypes.c_size_t(0)
    f = librr.rr_route_workspace_bytes
    f.argtypes = [ctypes.c_int] * 5 + [ctypes.c_uint, ctypes.POINTER(ctypes.c_size_t)]
    assert f(65536, 64, 2, 2048, 8, 3, ctypes.byref(n)) == 0 and n.value > 0
    assert f(0, 4, 1, 4, 2, 3, ctypes.byref(n)) == 0           # empty input is accepted
    for bad in [(64, 8, 0, 8, 2, 0), (64, 8, 9, 8, 2, 0), (64, 8, 1, 8, 3, 0), (64, 8, 1, -1, 2, 0),
                (64, 8, 1, 8, 2, 8), (64, 8, 8, 8, 2, 2), (64, 512, 1, 8, 2, 0), (63, 8, 1, 8, 2, 0)]:
        assert f(*bad, ctypes.byref(n)) == 1, bad
    librr.rr_status_string.restype = ctypes.c_char_p
    assert librr.rr_status_string(0) == b"ok"
    assert b"wait" in librr.rr_status_string(6)
    g = librr.rr_aux_workspace_bytes
    g.argtypes = [ctypes.c_int] * 2 + [ctypes.POINTER(ctypes.c_size_t)]
    assert g(65536, 64, ctypes.byref(n)) == 0 and n.value >= 256 + 1024 + 64 * 4
    assert g(0, 8, ctypes.byref(n)) == 0 and g(8, 0, ctypes.byref(n)) == 1 and g(8, 257, ctypes.byref(n)) == 1
    # null pointers are refused before anything is launched
    assert librr.rr_route(None, 64, 8, 1, 8, 2, 0, None, None, ctypes.c_size_t(0), None) == 1


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    from paper_2402_12399_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(ImportError):
        binding.lib()


def test_backward_pass_is_refused_for_fp32_before_anything_runs(librr):
    """rr_moe_bwd exists for bf16 layers only: an fp32 shape gets RR_ERR_UNSUPPORTED from the argument
    checks (no pointer is touched, no kernel launched) and its workspace query reports zero bytes."""
    from paper_2402_12399_b200 import binding
    shape = binding._CShape(64, 8, 1, 8, 2, 64, 64, binding.F32, 3, 0, None)
    a, b, c = ctypes.c_size_t(1), ctypes.c_size_t(1), ctypes.c_size_t(1)
    f = librr.rr_moe_workspace_bytes
    f.argtypes = [ctypes.POINTER(binding._CShape)] + [ctypes.POINTER(ctypes.c_size_t)] * 3
    assert f(ctypes.byref(shape), ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)) == 0
    assert a.value > 0 and b.value == 0 and c.value == 0
    fake = ctypes.c_void_p(256)                      # aligned, never dereferenced
    tables = binding._CTables(*[256] * len(binding._TABLE_FIELDS))
    g = librr.rr_moe_bwd
    g.argtypes = [ctypes.POINTER(binding._CShape)] + [ctypes.c_void_p] * 6 + [ctypes.POINTER(binding._CTables)] + \
        [ctypes.c_void_p] * 7 + [ctypes.c_size_t, ctypes.c_void_p]
    rc = g(ctypes.byref(shape), fake, fake, fake, fake, fake, fake, ctypes.byref(tables), fake, fake, fake, fake, fake, fake,
           fake, ctypes.c_size_t(1 << 30), None)
    assert rc == 2
    shape.dtype = binding.BF16
    assert f(ctypes.byref(shape), ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)) == 0 and b.value > 0 and c.value > 0
