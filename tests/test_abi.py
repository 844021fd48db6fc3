"""CPU checks of the C ABI: the library builds, loads, exports every declared symbol, and
rejects bad arguments on the host before anything is launched (no GPU needed)."""
import ctypes
import re
from pathlib import Path

import pytest

from paper_2605_28396_b200 import api, build

ROOT = Path(__file__).resolve().parent.parent
HEADER = ROOT / "include" / "adwin.h"


@pytest.fixture(scope="module")
def L():
    build.build()
    return api.lib()


def declared_functions():
    text = HEADER.read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(adwin_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = declared_functions()
    assert {"adwin_opd_kl_fwd_bwd", "adwin_window_reduce", "adwin_probe_align"} <= set(names)
    for n in names:
        assert hasattr(L, n), f"{n} declared in adwin.h but not exported"
    assert set(api.EXPORTS) <= set(names)


def test_checked_flavour_builds_and_exports_the_same_symbols():
    lib = ctypes.CDLL(str(build.build(checked=True)))
    for n in declared_functions():
        assert hasattr(lib, n), f"{n} missing from the bounds-checked flavour"
    lib.adwin_version.restype = ctypes.c_int
    assert lib.adwin_version() == api.lib().adwin_version()


def test_lmhead_entry_point_rejects_bad_arguments_on_the_host(L):
    fake = ctypes.c_void_p(4096)   # never dereferenced: validation fails first
    status = ctypes.c_void_p(8192)

    def call(**over):
        a = dict(hs=fake, ws=fake, ht=fake, wt=fake, B=2, T=16, V=256, ds=64, dt=64, tok=fake,
                 win=fake, roll=None, scale=1.0, mode=0, flags=0, gh=None, ghd=0, gw=None, kl=fake,
                 c=fake, gsq=None, ls=None, lt=None, max_rows=0, ws_=fake, wsb=1 << 30, st=status)
        a.update(over)
        return L.adwin_opd_kl_lmhead_fwd_bwd(a["hs"], a["ws"], a["ht"], a["wt"], a["B"], a["T"],
                                             a["V"], a["ds"], a["dt"], a["tok"], a["win"],
                                             a["roll"], a["scale"], a["mode"], a["flags"], a["gh"],
                                             a["ghd"], a["gw"], a["kl"], a["c"], a["gsq"], a["ls"],
                                             a["lt"], a["max_rows"], a["ws_"], a["wsb"], a["st"],
                                             None)
    assert call(mode=7) == 4 and call(flags=4) == 4            # ADWIN_ERR_DTYPE
    assert call(V=0) == 2 and call(ds=0) == 2 and call(B=-1) == 2
    assert call(st=None) == 1 and call(kl=None) == 1 and call(ws=None) == 1
    assert call(V=260) == 8 and call(dt=68) == 8               # not multiples of 8
    assert call(hs=ctypes.c_void_p(4100)) == 3                 # misaligned
    assert call(wsb=1024) == 6 and call(ws_=None) == 6         # workspace
    assert call(B=0) == 0                                      # empty batch: nothing to do
    need = api.adwin_lmhead_workspace_bytes(2, 16, 256, 64, 64)
    assert need > 0 and need % 1024 == 0
    assert api.adwin_lmhead_workspace_bytes(16, 4096, 151936, 2048, 2560, 36000) < \
        api.adwin_lmhead_workspace_bytes(16, 4096, 151936, 2048, 2560, 0)


def test_version_and_status_strings(L):
    assert L.adwin_version() >= 1
    assert L.adwin_status_string(0) == b"ADWIN_OK"
    for code in range(1, 9):
        assert L.adwin_status_string(code).startswith(b"ADWIN_ERR_")


def test_workspace_bytes_is_positive_and_monotone(L):
    a = api.adwin_workspace_bytes(1, 1, 1)
    b = api.adwin_workspace_bytes(1024, 8192, 151936)
    assert a > 0 and b >= a and b % 256 == 0


def _call(L, **over):
    fake = ctypes.c_void_p(4096)   # never dereferenced: validation fails first
    a = dict(student=fake, teacher=fake, dtype=1, B=2, T=4, V=16, ld=16, tokens=fake, window=fake,
             rollout=None, scale=1.0, mode=0, flags=0, grad=None, gdtype=1, ldg=16, kl=fake,
             c=fake, gsq=None, ls=None, lt=None, ws=fake, wsb=1 << 20, status=fake, stream=None)
    a.update(over)
    return L.adwin_opd_kl_fwd_bwd(a["student"], a["teacher"], a["dtype"], a["B"], a["T"], a["V"],
                                  a["ld"], a["tokens"], a["window"], a["rollout"], a["scale"],
                                  a["mode"], a["flags"], a["grad"], a["gdtype"], a["ldg"], a["kl"],
                                  a["c"], a["gsq"], a["ls"], a["lt"], a["ws"], a["wsb"],
                                  a["status"], a["stream"])


def test_host_side_argument_validation(L):
    assert _call(L, dtype=7) == 4
    assert _call(L, mode=2) == 4
    assert _call(L, flags=1 << 10) == 4
    assert _call(L, flags=16) == 4
    assert _call(L, V=0) == 2
    assert _call(L, ld=8) == 2
    assert _call(L, B=-1) == 2
    assert _call(L, grad=ctypes.c_void_p(4096), ldg=8) == 2
    assert _call(L, student=None) == 1
    assert _call(L, kl=None) == 1
    assert _call(L, status=None) == 1
    assert _call(L, student=ctypes.c_void_p(4097)) == 3
    assert _call(L, ws=None) == 6
    assert _call(L, ws=ctypes.c_void_p(4096 + 64)) == 6
    assert _call(L, wsb=16) == 6
    assert _call(L, B=0) == 0            # empty batch: nothing to do, nothing launched


def test_reduce_and_align_validation(L):
    fake = ctypes.c_void_p(4096)
    assert L.adwin_window_reduce(fake, fake, None, fake, None, 2, 4, fake, None, None) == 1
    assert L.adwin_window_reduce(fake, fake, None, fake, None, -2, 4, fake, fake, None) == 2
    f64 = ctypes.c_double
    assert L.adwin_probe_align(fake, fake, fake, fake, None, 2, 4, None, 5, f64(0.0), fake, fake,
                               fake, fake, fake, None) == 2     # default list has 6 entries
    assert L.adwin_probe_align(fake, fake, fake, fake, None, 2, 4, fake, 65, f64(0.0), fake, fake,
                               fake, fake, fake, None) == 2
    assert L.adwin_probe_align(fake, fake, None, fake, None, 2, 4, None, 6, f64(0.0), fake, fake,
                               fake, fake, fake, None) == 1


def test_return_to_go_and_weighted_validation(L):
    fake = ctypes.c_void_p(4096)
    f64 = ctypes.c_double
    assert L.adwin_return_to_go(fake, fake, None, 2, 4, f64(0.5), 0, None, None) == 1
    assert L.adwin_return_to_go(fake, fake, None, 2, 4, f64(1.5), 0, fake, None) == 2
    assert L.adwin_return_to_go(fake, fake, None, 2, 4, f64(-0.1), 0, fake, None) == 2
    assert L.adwin_return_to_go(fake, fake, None, 2, 4, f64(float("nan")), 0, fake, None) == 2
    assert L.adwin_return_to_go(fake, fake, None, 2, 4, f64(0.5), 1, fake, None) == 4
    assert L.adwin_return_to_go(fake, fake, None, -1, 4, f64(0.5), 0, fake, None) == 2
    assert L.adwin_return_to_go(None, None, None, 0, 4, f64(0.5), 0, None, None) == 0
    args = [fake, fake, 1, 2, 4, 16, 16, fake, fake, None]
    tail = [1.0, 0, None, 1, 16, fake, fake, None, None, None, fake, 1 << 20, fake, None]
    assert L.adwin_opd_kl_fwd_bwd_weighted(*args, None, *tail) == 1       # no coefficients
    assert L.adwin_opd_kl_fwd_bwd_weighted(*args, ctypes.c_void_p(4098), *tail) == 3
    bad = list(tail)
    bad[1] = 1 << 10
    assert L.adwin_opd_kl_fwd_bwd_weighted(*args, fake, *bad) == 4        # unknown flag


def test_drift_validation(L):
    fake = ctypes.c_void_p(4096)
    assert L.adwin_teacher_drift(fake, 7, 2, 4, 16, 16, fake, None, fake, fake, fake, None) == 4
    assert L.adwin_teacher_drift(fake, 1, 2, 4, 16, 8, fake, None, fake, fake, fake, None) == 2
    assert L.adwin_teacher_drift(fake, 1, 2, 4, 16, 16, fake, None, None, fake, fake, None) == 1
    assert L.adwin_teacher_drift(fake, 1, 2, 4, 16, 16, fake, None, fake, fake, None, None) == 1
    assert L.adwin_teacher_drift(ctypes.c_void_p(4097), 1, 2, 4, 16, 16, fake, None, fake, fake,
                                 fake, None) == 3
    assert L.adwin_teacher_drift(None, 1, 0, 4, 16, 16, None, None, None, None, fake, None) == 0
    assert L.adwin_drift_curves(fake, fake, None, 2, 4, fake, 65, fake, fake, fake, fake, None) == 2
    assert L.adwin_drift_curves(fake, fake, None, 2, 4, None, 2, fake, fake, fake, fake, None) == 1
    assert L.adwin_drift_curves(fake, fake, None, 2, 4, fake, 2, None, fake, fake, fake, None) == 1
    assert L.adwin_drift_curves(None, None, None, 0, 4, None, 0, None, None, None, None, None) == 0


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(api, "_lib", None)
    monkeypatch.setattr(api, "LIB_PATH", tmp_path / "nope.so")
    with pytest.raises(FileNotFoundError):
        api.lib()
