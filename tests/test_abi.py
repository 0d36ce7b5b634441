"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2608_14376_b200 import build, corun

    build.build()
    return corun.lib()


def _declared():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in sorted(os.listdir(inc)):
        if not f.endswith(".h"):
            continue
        src = open(os.path.join(inc, f)).read()
        src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
        # declarations that exist only in a library built with -DCORUN_BUILD_DEBUG (kernel timelines)
        src = re.sub(r"#ifdef CORUN_BUILD_DEBUG.*?#endif", "", src, flags=re.S)
        names |= set(re.findall(r"\b(corun_[a-z_0-9]+)\s*\(", src))
    return sorted(names)


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert "corun_init" in names and "corun_prefill" in names and "corun_decode_step" in names \
        and "corun_release" in names
    for n in names:
        assert getattr(lib, n) is not None, n


def test_binding_lists_the_same_symbols():
    from paper_2608_14376_b200 import corun

    assert sorted(corun.EXPORTS) == _declared()


def test_argument_validation_needs_no_gpu(lib):
    from paper_2608_14376_b200 import corun

    h = C.c_void_p()
    assert lib.corun_init(None, None, 1, 16, 16, 0, None, C.byref(h)) == corun.EINVAL
    sh = corun.Shape(2, 250, 4, 2, 64, 768, 2048, 1e-6, 1e4, 0)     # hidden not a multiple of 64
    w = corun.Weights()
    assert lib.corun_init(C.byref(sh), C.byref(w), 1, 16, 16, 0, None, C.byref(h)) == corun.EINVAL
    assert lib.corun_decode_step(None, None, None, None) == corun.EINVAL
    assert lib.corun_release(None, 0) == corun.EINVAL
    assert lib.corun_prefill(None, 0, None, 0, 0, None, 0, None) == corun.EINVAL
    assert lib.corun_debug_gemm(None, 1, 64, None, 1, None, None) == corun.EINVAL
    lib.corun_destroy(None)


def test_misaligned_buffers_are_refused_before_any_launch(lib):
    """The raw-pointer entry points store their output 16 bytes at a time: a buffer that starts elsewhere must
    come back as EINVAL from the argument checks (no CUDA call, so this runs without a GPU)."""
    from paper_2608_14376_b200 import corun

    base = 0x7F0000001000                     # never dereferenced: the checks come first
    for fn in (lib.corun_debug_gemm, lib.corun_gemm_static):
        fn.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
        for off in (4, 8, 12):
            assert fn(base, 256, 64, base + 0x10000, 1, base + 0x20000 + off, None) == corun.EINVAL
        assert fn(base + 8, 256, 64, base + 0x10000, 1, base + 0x20000, None) == corun.EINVAL
        assert fn(base, 256, 64, base + 0x10002, 1, base + 0x20000, None) == corun.EINVAL
    lib.corun_moe_forward.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    assert lib.corun_moe_forward(base, base + 0x10000, base + 0x20004, None, None) == corun.EINVAL


def test_strerror_covers_every_status(lib):
    seen = set()
    for st in range(0, -9, -1):
        s = lib.corun_strerror(st)
        assert s and s != b"unknown status"
        seen.add(s)
    assert len(seen) == 9
    assert lib.corun_strerror(-99) == b"unknown status"


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2608_14376_b200 import corun

    monkeypatch.setattr(corun, "_lib", None)
    monkeypatch.setattr(corun, "LIB_PATH", "/nonexistent/libcorun.so")
    with pytest.raises(RuntimeError):
        corun.lib()
