"""Host-side checks that need no GPU: the shared library loads, exports every symbol the
header declares, and its argument validation answers before any device work."""
import ctypes
import os
import re

import paper_1801_04928_b200 as lf

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "leapfrog.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lf_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(lf.LIB_PATH)
    names = _declared_symbols()
    assert "lf_backward" in names and "lf_create" in names and len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(lf.EXPORTS)


def test_binding_has_the_same_names():
    for n in _declared_symbols():
        assert callable(getattr(lf, n)), n


def test_strerror_and_version():
    assert lf.lf_version() >= 100
    assert lf.lf_strerror(lf.LF_OK) == "ok"
    for code in range(-7, 0):
        assert lf.lf_strerror(code) != "unknown status"
    assert lf.lf_strerror(-99) == "unknown status"


def test_create_rejects_bad_sizes_before_touching_the_device():
    for args in [(0, 64, 1, 1), (4, 0, 1, 1), (4, 64, 0, 1), (4, 64, 1, 0), (4, 66, 1, 1),
                 (-1, 64, 1, 1)]:
        rc, h = lf.lf_create(*args)
        assert rc == lf.LF_EINVAL and not h.value


def test_create_widths_rejects_bad_sizes_before_touching_the_device():
    for widths, B, k in [([8, 6, 8], 1, 1), ([8, 0, 8], 1, 1), ([8], 1, 1), ([8, 8], 0, 1), ([8, 8], 1, 0),
                         ([8, -4, 8], 1, 1)]:
        rc, h = lf.lf_create_widths(widths, B, k)
        assert rc == lf.LF_EINVAL and not h.value
    # a NULL widths array or a NULL result pointer is LF_ENULL
    lib = ctypes.CDLL(lf.LIB_PATH)
    h = ctypes.c_void_p(None)
    assert lib.lf_create_widths(ctypes.byref(h), 2, None, 1, 1) == lf.LF_ENULL and not h.value
    assert lib.lf_create_widths(None, 2, (ctypes.c_int * 3)(8, 8, 8), 1, 1) == lf.LF_ENULL


def test_null_context_is_an_error_not_a_crash():
    assert lf.lf_sync(None) == lf.LF_ENULL
    assert lf.lf_destroy(None) == lf.LF_ENULL
    assert lf.lf_set_option(None, lf.LF_OPT_VARIANT, 1) == lf.LF_ENULL
    assert lf.lf_forward(None, 16, 16, 16, 16, 16) == lf.LF_ENULL
    assert lf.lf_backward(None, 16, 16, 16, 16, 16, 16, 16) == lf.LF_ENULL
    assert lf.lf_owner(None, 1) == -1
    assert lf.lf_grad_w(None, 16, 16, 16) == lf.LF_ENULL
    assert lf.lf_backward_sgd(None, 16, 16, 16, 16, 0.1, 16, 32, 16) == lf.LF_ENULL


def test_no_device_means_an_error_not_a_fallback():
    import torch
    if torch.cuda.is_available():
        return
    rc, h = lf.lf_create(4, 64, 1, 2)
    assert rc == lf.LF_ECUDA and not h.value
    rc, h = lf.lf_create_widths([64, 32, 16], 1, 2)
    assert rc == lf.LF_ECUDA and not h.value


def test_binding_checks_tensors_before_the_library_sees_them():
    # dtype, contiguity, side of the bus and size are checked while marshalling: the kernels trust the
    # context's sizes, so a buffer that is too small must never reach them
    import pytest
    import torch
    from paper_1801_04928_b200 import binding
    ok = torch.zeros(64, dtype=torch.float32)
    binding._check_tensor(ok, 64, "x", "test", on_device=False)
    binding._check_tensor(None, 64, "x", "test")
    binding._check_tensor(12345, 64, "x", "test")
    for bad, on_device in ((torch.zeros(64, dtype=torch.float64), False), (torch.zeros(63), False),
                           (torch.zeros(8, 16).t(), False), (ok, True)):
        with pytest.raises(lf.LeapfrogError) as e:
            binding._check_tensor(bad, 64, "x", "test", on_device=on_device)
        assert e.value.status == lf.LF_EINVAL
    # the static entry point checks before it calls into the library (no device is touched here)
    with pytest.raises(lf.LeapfrogError):
        lf.lf_delta_step_static(torch.zeros(16), torch.zeros(8), torch.zeros(8), torch.zeros(8), 8)
