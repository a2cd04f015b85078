"""The C-ABI library builds, loads and exports every symbol the header declares; host-visible errors are
reported without a GPU (no compute call is made here)."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2511_13732_b200 import binding
from paper_2511_13732_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "pcg.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pcg_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = binding.load()
    names = _declared()
    assert set(binding.EXPORTS) <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in pcg.h but not exported"
    assert len(names) >= 10


def test_status_strings():
    lib = binding.load()
    seen = {lib.pcg_status_string(i).decode() for i in range(6)}
    assert len(seen) == 6 and "ok" in seen
    assert lib.pcg_status_string(99).decode() == "unknown status"


def _create(V, ptr, tok, deg, weights=None, hint=0):
    lib = binding.load()
    ptr, tok, deg = (np.ascontiguousarray(a, np.int32) for a in (ptr, tok, deg))
    w = None if weights is None else np.ascontiguousarray(weights, np.float32)
    csr = binding._Csr(V, len(ptr) - 1, len(tok), binding._np_ptr(ptr), binding._np_ptr(tok), binding._np_ptr(deg),
                       binding._np_ptr(w))
    h = ctypes.c_void_p()
    st = lib.pcg_groups_create(ctypes.byref(csr), hint, ctypes.byref(h))
    msg = lib.pcg_last_error().decode()
    if st == 0:
        lib.pcg_groups_destroy(h)
    return st, msg


def test_membership_validation_on_the_host():
    ok = W.groups_from_lists(5, [[0, 1], [1, 2, 3], [4], []])
    st, _ = _create(5, ok.group_ptr, ok.group_tok, ok.tok_degree)
    assert st in (0, 5)  # valid: PCG_OK with a GPU, PCG_ERR_CUDA (no device) without one
    bad = [
        ([0, 2, 5, 6, 6], [0, 1, 1, 2, 3, 7], [1, 2, 1, 1, 1], "outside"),  # token id out of range
        ([0, 2, 5, 6, 6], [1, 0, 1, 2, 3, 4], [1, 2, 1, 1, 1], "ascending"),  # unsorted group
        ([0, 2, 5, 6, 6], [0, 1, 1, 2, 3, 4], [1, 1, 1, 1, 1], "tok_degree"),  # wrong degree
        ([0, 2, 4, 5, 5], [0, 1, 1, 2, 4], [1, 2, 1, 0, 1], "tok_degree"),  # token 3 in no group
        ([0, 2, 1, 5, 5], [0, 1, 2, 3, 4], [1, 1, 1, 1, 1], "decreases"),  # pointer not monotone
        ([0, 9, 1, 5, 5], [0, 1, 2, 3, 4], [1, 1, 1, 1, 1], "decreases"),  # pointer beyond nnz before it decreases
        ([0, 1000, 3, 5, 5], [0, 1, 2, 3, 4], [1, 1, 1, 1, 1], "decreases"),
        ([0, -2, 3, 5, 5], [0, 1, 2, 3, 4], [1, 1, 1, 1, 1], "decreases"),  # negative pointer
        ([1, 2, 5, 6, 6], [0, 1, 1, 2, 3, 4], [1, 2, 1, 1, 1], "group_ptr[0]"),
    ]
    for ptr, tok, deg, word in bad:
        st, msg = _create(5, ptr, tok, deg)
        assert st == 2 and word in msg, (st, msg)
    # weights that do not sum to one over a token's groups
    st, msg = _create(5, ok.group_ptr, ok.group_tok, ok.tok_degree, weights=[1, 0.7, 0.7, 1, 1, 1])
    assert st == 2 and "sum" in msg


def test_argument_errors_before_any_launch():
    lib = binding.load()
    assert lib.pcg_groups_create(None, 0, None) == 1
    ok = W.groups_from_lists(3, [[0, 1, 2]])
    assert _create(3, ok.group_ptr, ok.group_tok, ok.tok_degree, hint=3)[0] == 1
    assert _create(0, [0, 0], [], [])[0] == 1
    assert lib.pcg_groups_info(None, None) == 1
    assert lib.pcg_group_probs(None, 0, 4, 1.0, None, None, None) == 1  # null handle
    assert lib.pcg_verify(None, None, 0, 1, 1, None, None, None, 1.0, None, None, None, None, None, 0, 0, None,
                          None) == 1
    assert lib.pcg_verify_host(None, None, 0, 1, 1, None, None, None, 1.0, None, None, None, None, None, 0, 0,
                               None) == 1
    lib.pcg_groups_destroy(None)  # allowed
    assert "null" in lib.pcg_last_error().decode()


def test_workspace_queries():
    lib = binding.load()
    a = lib.pcg_verify_workspace_bytes(256, 16, 65536, 16384, 1, 0)
    b = lib.pcg_verify_workspace_bytes(1, 4, 1024, 256, 0, 0)
    assert a >= 256 * 16 * 28 and b >= 256 and a % 256 == 0 and b % 256 == 0
    arena = lib.pcg_verify_host_arena_bytes(256, 16, 65536, 16384, 1, 0)
    assert arena >= 256 * 33 * 65536 * 2 + a
    g = lib.pcg_group_probs_workspace_bytes(65536, 16384)
    assert g >= 256 * (65536 + 16384) * 4 and g % 256 == 0 and lib.pcg_group_probs_workspace_bytes(0, 5) == 256
    assert lib.pcg_group_probs_ws(None, 0, 4, 1.0, None, None, None, 0, None) == 1  # null handle
    t = lib.pcg_verify_thinning_workspace_bytes(256, 16, 65536, 16384, 1)
    assert t >= 256 * 16 * 28 + 256 * 16384 * 4 and t % 256 == 0
    assert lib.pcg_verify_thinning(None, None, 0, 1, 1, None, None, None, None, 4, 1.0, None, None, None, None, None,
                                   None, 0, None, None) == 1  # null handle


def test_binding_has_no_fallback(monkeypatch):
    """If the shared library cannot be loaded the binding raises; it never computes anything itself."""
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding._build, "LIB", "/nonexistent/libpcg.so")
    monkeypatch.setattr(binding._build, "build", lambda *a, **k: (_ for _ in ()).throw(RuntimeError("no nvcc")))
    with pytest.raises((OSError, RuntimeError)):
        binding.load()
