"""The C-ABI library builds, loads without a GPU, and exports what include/impact.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1912_00167_b200 import build, binding
    build.build()
    return binding.load_library()


def _declared():
    text = open(os.path.join(ROOT, "include", "impact.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(impact_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_1912_00167_b200 import binding
    names = _declared()
    assert len(names) >= 19
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_housekeeping_calls(lib):
    assert lib.impact_version() == 300
    assert lib.impact_status_string(0) == b"ok"
    assert b"full" in lib.impact_status_string(-5)
    assert b"empty" in lib.impact_status_string(-4)
    assert lib.impact_loss_workspace_bytes(0, 5) == 0
    assert lib.impact_loss_workspace_bytes(1024, 128) >= 1024 * 32


def test_struct_layout_matches_header():
    from paper_1912_00167_b200.binding import impact_coefficients
    assert ctypes.sizeof(impact_coefficients) == 48
    assert impact_coefficients.rho_tw.offset == 16 and impact_coefficients.objective.offset == 32
    assert impact_coefficients.global_steps.offset == 40


def test_host_side_validation_needs_no_gpu(lib):
    # null pointers and bad sizes are refused before any CUDA call
    from paper_1912_00167_b200.binding import impact_coefficients
    cf = impact_coefficients(0.5, 0.01, 0.0, 1.0, 1.0, 0, 0, 0, 0)
    st = lib.impact_loss_fwd_bwd(None, None, None, None, None, None, None, None, 1.0, 1.0, 0.2, ctypes.pointer(cf),
                                 4, 4, 4, 0, None, None, None, None, None, None, 0, None)
    assert st == -1
    fb = (ctypes.c_size_t * 1)(0)
    assert lib.impact_buffer_storage_bytes(4, 1, fb) == 0
    fb = (ctypes.c_size_t * 2)(100, 300)
    assert lib.impact_buffer_storage_bytes(4, 2, fb) == 4 * (256 + 512)
    h = ctypes.c_void_p()
    assert lib.impact_buffer_create(0, 1, 2, fb, 0, 0, None, ctypes.byref(h)) == -1
    assert lib.impact_buffer_create(2, 2, 2, fb, 0, 5, None, ctypes.byref(h)) == -1
    assert lib.impact_gather_rows(None, None, 1, 1, 4, None, None) == -1


def test_ring_bookkeeping_runs_on_caller_storage_without_a_gpu(lib, oracle):
    # with caller-provided storage and no copies requested, push/sample touch only host state
    fb = (ctypes.c_size_t * 1)(64)
    h = ctypes.c_void_p()
    fake_storage = ctypes.c_void_p(256 * 1024)  # never dereferenced: every field source below is NULL
    assert lib.impact_buffer_create(4, 2, 1, fb, 77, 0, fake_storage, ctypes.byref(h)) == 0
    ref = oracle.Ring(4, 2, 0, seed=77)
    src = (ctypes.c_void_p * 1)(None)
    slot, k = ctypes.c_int32(), ctypes.c_int32()
    for i in range(5):
        st = lib.impact_buffer_push(h, src, 0, ctypes.byref(slot), None)
        rst, rslot = ref.push()
        assert (st == -5) == (rst == ref.FULL)
        if st == 0:
            assert slot.value == rslot
    for i in range(9):
        st = lib.impact_buffer_sample(h, ctypes.byref(slot), ctypes.byref(k), None, None)
        rst, rslot, rk = ref.sample()
        assert (st == -4) == (rst == ref.EMPTY)
        if st == 0:
            assert (slot.value, k.value) == (rslot, rk)
    assert lib.impact_buffer_destroy(h) == 0
