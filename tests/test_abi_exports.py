"""The C-ABI library loads and exports what include/fff.h declares; host-side argument checks (no GPU work)."""
import ctypes as C
import os
import re

import pytest

from paper_2308_14711_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "fff.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fff_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = declared_symbols()
    assert "fff_create" in names and "fff_forward_infer" in names and "fff_destroy" in names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in fff.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_binding_tables_match_the_header_enums():
    """The binding's name tables carry the header's values (tuning switches, paths, activations)."""
    text = open(os.path.join(ROOT, "include", "fff.h")).read()
    enums = {k: int(v) for k, v in re.findall(r"\b(FFF_[A-Z0-9_]+)\s*=\s*(\d+)", text)}
    tune = {k[len("FFF_TUNE_"):].lower(): v for k, v in enums.items() if k.startswith("FFF_TUNE_") and k != "FFF_TUNE_COUNT"}
    assert binding.TUNING == tune
    assert enums["FFF_TUNE_COUNT"] == len(tune) == max(tune.values()) + 1
    for name, value in binding.ACTIVATIONS.items():
        assert enums["FFF_ACT_" + name.upper()] == value
    for name, value in binding.PATHS.items():
        assert enums["FFF_PATH_" + name.upper()] == value


def test_status_strings(lib):
    seen = {binding.status_string(s) for s in range(8)}
    assert len(seen) == 8 and "ok" in seen
    assert binding.status_string(99) == "unknown status"


def test_create_rejects_bad_arguments_on_the_host(lib):
    h = C.c_void_p(1234)
    fake = 0x1000   # never dereferenced: the checks below fail first
    args = dict(D=8, O=4, depth=2, l=2, act=0, dt=0)

    def create(out=None, nw=fake, w1=fake, w2=fake, **kw):
        a = dict(args, **kw)
        return lib.fff_create(C.byref(h) if out is None else out, a["D"], a["O"], a["depth"], a["l"], a["act"],
                              a["dt"], nw, None, w1, None, w2, None)
    assert create(out=C.POINTER(C.c_void_p)()) == 1
    for bad in (dict(D=0), dict(O=-1), dict(l=0), dict(depth=-1), dict(act=4), dict(act=-1), dict(dt=3)):
        assert create(**bad) == 1, bad
        assert h.value is None
    assert create(depth=21) == 2
    assert create(w1=None) == 1
    assert create(w2=None) == 1
    assert create(nw=None) == 1                 # depth > 0 needs node weights
    assert create(w1=fake + 4) == 1             # misaligned


def test_calls_reject_dead_handles(lib):
    assert lib.fff_destroy(None) == 6
    assert lib.fff_destroy(C.c_void_p(0xdead0)) == 6
    assert lib.fff_forward_infer(C.c_void_p(0xdead0), None, None, None, 1, None) == 6
    assert lib.fff_reserve(None, 10) == 6
    assert lib.fff_set_tuning(None, 0, 1) == 6
    assert lib.fff_capabilities(None) == -1
    assert lib.fff_get_last_status(None) == 6
    assert lib.fff_last_launch_count(None) == -1
