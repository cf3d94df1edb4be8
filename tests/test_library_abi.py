"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
symbol include/gk.h declares, and rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import pytest

from paper_1911_08772_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "gk.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b([a-z_0-9]+)\s*\(", text)
    return sorted({n for n in names if n.startswith(("gk_", "topk_", "dgck_"))})


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert set(binding.EXPORTS) <= set(names)
    for n in ("gk_sparsify", "gk_sparsify_segmented", "topk_exact"):
        assert n in names
    for n in names:
        assert hasattr(lib, n), n


def test_version_and_error_text(lib):
    assert lib.gk_version() >= 1000
    assert binding.gk_strerror(0) == "ok"
    for code in range(-9, 0):
        assert "unknown" not in binding.gk_strerror(code)
    assert "unknown" in binding.gk_strerror(-99)


def test_workspace_bytes_is_modest_and_monotone(lib):
    small = binding.gk_workspace_bytes(1, 1)
    big = binding.gk_workspace_bytes(1 << 28, 1)
    seg = binding.gk_workspace_bytes(25_557_032, 161)
    assert 0 < small <= big
    assert big < 8 << 20          # status words: 8 B per 8192-element tile
    assert seg < 8 << 20
    assert binding.gk_workspace_bytes(0, 1) == 0


def test_argument_validation_happens_on_the_host(lib):
    a = 0x1000  # a fake, aligned, non-null address: validation must fail before any use
    st = None
    assert lib.gk_sparsify(None, a, 10, 1, a, a, a, st) == -1
    assert lib.gk_sparsify(a, a + 4096, 0, 1, a, a, a, st) == -2
    assert lib.gk_sparsify(a, a + 4096, 2 ** 31, 1, a, a, a, st) == -2
    assert lib.gk_sparsify(a, a + 4096, 10, 0, a, a, a, st) == -3
    assert lib.gk_sparsify(a, a + 4096, 10, 11, a, a, a, st) == -3
    assert lib.gk_sparsify(a + 4, a + 4096, 10, 1, a, a, a, st) == -4
    assert lib.gk_sparsify(a, a + 16, 10, 1, a, a, a, st) == -5     # g overlaps eps
    assert lib.topk_exact(None, 10, 1, a, a, st) == -1
    assert lib.topk_exact(a, 10, 11, a, a, st) == -3
    assert lib.topk_exact(a + 8, 10, 1, a, a, st) == -4
    assert lib.gk_sparsify_segmented(a, a + 4096, 10, None, a, 1, a, a, None, a, st) == -1
    assert lib.gk_sparsify_segmented(a, a + 4096, 10, a, a, 0, a, a, None, a, st) == -2
    assert lib.gk_sparsify_segmented(a, a + 4096, 10, a, a, 70000, a, a, None, a, st) == -2
    assert lib.topk_sparsify(a, a + 16, 10, 1, a, a, a, st) == -5
    import ctypes
    out = (ctypes.c_double * 3)()
    assert lib.gk_error_ratio(None, 10, a, a, st, out) == -1
    assert lib.gk_error_ratio(a, 10, a, a, st, None) == -1
    assert lib.gk_error_ratio(a, 0, a, a, st, out) == -2
    assert lib.gk_error_ratio(a + 4, 10, a, a, st, out) == -4
    assert lib.gk_set_capacity(-1) == -8
    assert lib.gk_set_capacity(0) == 0


def test_binding_refuses_cpu_tensors(lib):
    import torch
    t = torch.zeros(8)
    with pytest.raises(binding.GkError):
        binding.gk_sparsify(t, t.clone(), 1, torch.zeros(8, dtype=torch.int32), t.clone(),
                            torch.zeros(1, dtype=torch.int64))


def test_dgck_argument_validation_happens_on_the_host(lib):
    a = 0x1000
    st = None
    assert lib.dgck_select(None, 10, 1, a, 5, a, a, a, st) == -1
    assert lib.dgck_select(a, 10, 1, None, 5, a, a, a, st) == -1
    assert lib.dgck_select(a, 0, 1, a, 5, a, a, a, st) == -2
    assert lib.dgck_select(a, 10, 1, a, 0, a, a, a, st) == -2
    assert lib.dgck_select(a, 10, 11, a, 5, a, a, a, st) == -3
    assert lib.dgck_select(a + 4, 10, 1, a, 5, a, a, a, st) == -4
    assert lib.dgck_sparsify(a, a + 16, 10, 1, a, 5, a, a, a, st) == -5
    assert lib.dgck_sparsify(a, None, 10, 1, a, 5, a, a, a, st) == -1


def test_the_operator_and_the_setters_validate_on_the_host(lib):
    a = 0x1000
    assert lib.gk_select(None, 10, 1, a, a, a, None) == -1
    assert lib.gk_select(a, 0, 1, a, a, a, None) == -2
    assert lib.gk_select(a, 10, 11, a, a, a, None) == -3
    assert lib.gk_select(a + 4, 10, 1, a, a, a, None) == -4
    assert lib.gk_set_params(1, 0) == -2 and lib.gk_set_params(0, 5) == -2     # rounds outside 1 .. 4
    assert lib.gk_set_path(3) == -2 and lib.gk_set_path(-1) == -2
    assert lib.gk_debug_set(99, 0) == -2 and lib.gk_debug_set(-1, 0) == -2      # unknown keys
    assert lib.gk_debug_set(0, -2) == -2                                         # value out of range
