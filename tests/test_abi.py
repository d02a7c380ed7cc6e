"""The C-ABI library loads and exports every symbol include/nb.h declares (no compute calls)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "nb.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    names = re.findall(r"\b(nb_[a-z_A-Z0-9]+)\s*\(", src)
    return sorted(set(names))


def test_header_declares_the_named_entry_points():
    names = _declared()
    for must in ("nb_create", "nb_accumulate", "nb_step", "nb_get_params", "nb_step_fused", "nb_destroy",
                 "nb_straggler_sample", "nb_get_device_mixing"):
        assert must in names


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2211_00889_b200.build import build_library
    path = build_library()
    lib = ctypes.CDLL(path)
    for name in _declared():
        assert hasattr(lib, name), name


def test_binding_covers_every_declared_symbol():
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding
    assert sorted(binding.EXPORTED) == _declared()


def test_argument_errors_are_reported_without_a_gpu():
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding as B
    h = ctypes.c_void_p()
    assert B.lib.nb_create(ctypes.byref(h), 0, 10, 1, 0.1, 0.9, B.NB_ALLREDUCE, None) == B.NB_ERR_ARG
    assert b"K" in B.lib.nb_last_error(None)
    assert B.lib.nb_create(ctypes.byref(h), 4, 0, 1, 0.1, 0.9, B.NB_ALLREDUCE, None) == B.NB_ERR_ARG
    assert B.lib.nb_create(ctypes.byref(h), 4, 8, 0, 0.1, 0.9, B.NB_ALLREDUCE, None) == B.NB_ERR_ARG
    assert B.lib.nb_create(ctypes.byref(h), 4, 8, 2, 0.1, 0.9, 9, None) == B.NB_ERR_ARG
    assert B.lib.nb_create(ctypes.byref(h), 65, 8, 2, 0.1, 0.9, B.NB_ALLREDUCE, None) == B.NB_ERR_UNSUPPORTED
    assert B.lib.nb_create(ctypes.byref(h), 4, 8, 2, 0.1, 0.9, B.NB_DPSGD, None) == B.NB_ERR_ARG   # needs a topology
    assert h.value is None
    assert B.lib.nb_destroy(None) == B.NB_OK
    assert B.lib.nb_step(None, None) == B.NB_ERR_ARG


def test_valid_create_fails_loudly_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        import pytest
        pytest.skip("a CUDA device is present")
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding as B
    h = ctypes.c_void_p()
    rc = B.lib.nb_create(ctypes.byref(h), 4, 1024, 4, 0.1, 0.9, B.NB_ALLREDUCE, None)
    assert rc in (B.NB_ERR_CUDA, B.NB_ERR_NOMEM) and h.value is None      # no CPU fallback exists
    assert B.lib.nb_last_error(None) != b""


def test_range_predicates_of_the_bounds_checked_build():
    """The kernels of a -DNB_DEBUG library guard every access with these predicates; fed an
    out-of-range span or index on the host they return the code the kernel would have recorded."""
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding as B
    lo, hi = 4096, 4096 + 1024
    assert B.lib.nb_debug_span_code(lo, 1024, lo, hi) == 0               # the whole array
    assert B.lib.nb_debug_span_code(hi - 16, 16, lo, hi) == 0            # its last vector
    assert B.lib.nb_debug_span_code(hi - 16, 0, lo, hi) == 0
    assert B.lib.nb_debug_span_code(hi - 12, 16, lo, hi) == 101          # runs 4 bytes past the end
    assert B.lib.nb_debug_span_code(lo - 4, 16, lo, hi) == 101           # starts before the array
    assert B.lib.nb_debug_span_code(hi + 64, 4, lo, hi) == 101           # entirely beyond it
    assert B.lib.nb_debug_span_code(lo, 2 ** 63, lo, hi) == 101          # a length that would wrap around
    assert B.lib.nb_debug_index_code(0, 16) == 0 and B.lib.nb_debug_index_code(15, 16) == 0
    assert B.lib.nb_debug_index_code(16, 16) == 106 and B.lib.nb_debug_index_code(-1, 16) == 106
    assert B.lib.nb_debug_build() == (1 if "debug" in os.path.basename(B.LIB_PATH) else 0)


def test_recommended_pitch():
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding as B
    f = B.lib.nb_recommended_pitch
    assert f(1, B.NB_BF16) == 1024 and f(1024, B.NB_BF16) == 1024 and f(1025, B.NB_BF16) == 2048
    assert f(512, B.NB_F32) == 512 and f(513, B.NB_F32) == 1024
    assert f(138_000_000, B.NB_BF16) == 138_000_384 and f(25_600_000, B.NB_BF16) == 25_600_000
    assert f(0, B.NB_F32) == 0 and f(8, 7) == 0
