"""CPU-side checks of the C ABI: the library loads, exports every function the header declares,
and rejects bad arguments on the host before touching the GPU."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "ciar.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ciar_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(ciar_lib):
    lib = ciar_lib.load()
    names = _declared_functions()
    assert {"ciar_quantify", "ciar_verify", "ciar_decode_step", "ciar_decode_init", "ciar_workspace_bytes",
            "ciar_status_string", "ciar_version", "ciar_launch_count"} <= set(names)
    for n in names:
        assert hasattr(lib, n), "libciar.so does not export %s" % n


def test_version_and_status_strings(ciar_lib):
    assert ciar_lib.version() == 100
    assert ciar_lib.status_string(0) == "ok"
    seen = {ciar_lib.status_string(s) for s in range(7)}
    assert len(seen) == 7 and "unknown status" not in seen
    assert ciar_lib.status_string(99) == "unknown status"


def test_workspace_bytes_monotone(ciar_lib):
    assert ciar_lib.workspace_bytes(-1, 8) == 0 and ciar_lib.workspace_bytes(8, 0) == 0
    a, b, c = (ciar_lib.workspace_bytes(r, 8) for r in (0, 2048, 65536))
    assert 0 < a < b < c
    assert c < 65536 * 32  # a few dozen bytes per row, never a copy of the logits


def test_host_validation_rejects_before_any_launch(ciar_lib):
    """No GPU is needed: each call returns an error code from the host-side checks."""
    lib = ciar_lib.load()
    c = ciar_lib
    before = c.launch_count()
    buf = (ctypes.c_char * 4096)()
    base = ctypes.addressof(buf)
    base += (-base) % 16
    good = c.LogitsDesc(4, 64, 64, 0, 64, c.F32)
    prm = c.IntervalParamsC(c.RADIUS_SCALAR, 0, None, 0.5, 10.0, 0.99, 1.01, c.POLICY_INTERVAL, 0.3, None)
    out = c.QuantifyOutC()
    q = lambda d, ptr, p, o: lib.ciar_quantify(ctypes.byref(d) if d else None, ptr, ctypes.byref(p) if p else None,
                                                 ctypes.byref(o) if o else None, None)
    assert q(None, base, prm, out) == 1
    assert q(good, None, prm, out) == 1
    assert q(good, base, None, out) == 1
    assert q(good, base, prm, None) == 1
    assert q(good, base + 4, prm, out) == 3  # misaligned base
    assert q(c.LogitsDesc(4, 66, 64, 0, 64, c.BF16), base, prm, out) == 3  # stride * 2 bytes not a multiple of 16
    assert q(c.LogitsDesc(4, 64, 64, 0, 64, 7), base, prm, out) == 2  # unknown dtype
    assert q(c.LogitsDesc(4, 64, 64, 60, 8, c.F32), base, prm, out) == 1  # slice past the row
    assert q(c.LogitsDesc(4, 64, 64, 0, 0, c.F32), base, prm, out) == 1
    assert q(c.LogitsDesc(-1, 64, 64, 0, 64, c.F32), base, prm, out) == 1
    assert q(c.LogitsDesc(4, 32, 64, 0, 64, c.F32), base, prm, out) == 1  # stride < vocab
    bad = c.IntervalParamsC(c.RADIUS_PER_ROW, 0, None, 0.5, 10.0, 0.99, 1.01, c.POLICY_INTERVAL, 0.3, None)
    assert q(good, base, bad, out) == 1  # per-row radius without a radius array
    bad = c.IntervalParamsC(c.RADIUS_SCALAR, 0, None, 0.5, 100.0, 0.99, 1.01, c.POLICY_INTERVAL, 0.3, None)
    assert q(good, base, bad, out) == 1  # r_max out of range
    bad = c.IntervalParamsC(c.RADIUS_SCALAR, 0, None, 0.5, 10.0, 0.99, 1.01, c.POLICY_RANDOM, 0.3, None)
    assert q(good, base, bad, out) == 1  # RANDOM policy without uniforms
    bad = c.IntervalParamsC(c.RADIUS_SCALAR, 0, None, 0.5, 10.0, 0.99, 1.01, 9, 0.3, None)
    assert q(good, base, bad, out) == 1
    assert q(c.LogitsDesc(0, 64, 64, 0, 64, c.F32), None, prm, out) == 0  # empty input: OK, nothing launched

    vout = c.VerifyOutC()
    def v(d, window, mode, flag, ws, ws_bytes, rm=None, se=None):
        vp = c.VerifyParamsC(window, mode)
        return lib.ciar_verify(ctypes.byref(d), base, base, base, flag, rm, se, base, base, ctypes.byref(vp),
                               ctypes.byref(vout), ws, ws_bytes, None)
    big = 1 << 20
    assert v(good, 3, c.VERIFY_ALL, None, base, big) == 1  # rows not a multiple of the window
    assert v(good, 0, c.VERIFY_ALL, None, base, big) == 1
    assert v(good, 65, c.VERIFY_ALL, None, base, big) == 1
    assert v(good, 4, 5, None, base, big) == 1  # unknown mode
    assert v(good, 4, c.VERIFY_ANCHORED, None, base, big) == 1  # flags required
    assert v(good, 4, c.VERIFY_ALL, None, None, big) == 1
    assert v(good, 4, c.VERIFY_ALL, None, base + 8, big) == 3
    assert v(good, 4, c.VERIFY_ALL, None, base, 8) == 4  # workspace too small
    assert v(good, 4, c.VERIFY_ALL, None, base, big, rm=base) == 1  # row_max without sum_exp

    vp = c.VerifyParamsC(4, c.VERIFY_ANCHORED)
    step = lambda s, d: lib.ciar_decode_step(ctypes.byref(s), ctypes.byref(d), base, base, base, base, base,
                                             ctypes.byref(prm), ctypes.byref(vp), base, big, None)
    assert step(c.DecodeStateC(3, 2, base, base, base), good) == 1  # pool rows != requests * seq_len
    assert step(c.DecodeStateC(2, 2, None, base, base), good) == 1
    assert lib.ciar_decode_init(ctypes.byref(c.DecodeStateC(2, 2, base, base, base)), 5, None) == 1  # pos0 > seq_len
    assert c.launch_count() == before  # nothing reached the GPU
