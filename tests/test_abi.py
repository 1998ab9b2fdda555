"""CPU-side checks of the C ABI: the library builds for sm_100a, loads, exports every
symbol that include/hx.h declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def hx():
    import __graft_entry__ as entry
    entry.build()
    import paper_2605_16637_b200 as mod
    return mod


def _declared():
    text = open(os.path.join(ROOT, "include", "hx.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hx_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(hx):
    lib = ctypes.CDLL(hx.lib_path())
    names = _declared()
    assert len(names) >= 15 and "hx_schedule_batch" in names and "hx_critical_path" in names
    for n in names:
        assert hasattr(lib, n), n


def test_binding_mirrors_the_header(hx):
    for n in _declared():
        assert hasattr(hx, n), "binding lacks " + n


def test_binding_constants_equal_the_header_macros(hx):
    text = open(os.path.join(ROOT, "include", "hx.h")).read()
    macros = {k: int(v, 0) for k, v in re.findall(r"#define\s+(HX_[A-Z_0-9]+)\s+(-?(?:0x[0-9A-Fa-f]+|\d+))\b", text)}
    assert macros["HX_FLAG_ONE_PASS"] == 8 and macros["HX_OK"] == 0
    checked = 0
    for name, value in macros.items():
        if hasattr(hx, name):
            assert getattr(hx, name) == value, name
            checked += 1
    assert checked >= 6                                          # the flags and score modes at least


def test_built_for_sm_100a():
    import importlib.util
    spec = importlib.util.spec_from_file_location("_b", os.path.join(ROOT, "paper_2605_16637_b200", "build.py"))
    b = importlib.util.module_from_spec(spec); spec.loader.exec_module(b)
    assert "arch=compute_100a,code=sm_100a" in b.NVCC_FLAGS and "-fmad=false" in b.NVCC_FLAGS
    assert len(b.sources()) >= 4


def _inst(P, D):
    a = np.zeros(P + D, dtype=[("type", "<u4"), ("role", "<u4"), ("load_s", "<f4"),
                               ("kv_cap_tokens", "<f4"), ("kv_free_tokens", "<f4")])
    a["role"][P:] = 1
    a["kv_cap_tokens"] = 1e6
    a["kv_free_tokens"] = 1e6
    return a


@pytest.mark.parametrize("mutate, fragment", [
    (lambda a: a.update(types=np.array([[0.0, 1.0]])), "rates"),
    (lambda a: a.update(types=np.array([[np.nan, 1.0]])), "rates"),
    (lambda a: a["inst"].__setitem__("type", 3), "type out of range"),
    (lambda a: a["inst"]["load_s"].__setitem__(0, -1.0), "load"),
    (lambda a: a["inst"]["role"].__setitem__(slice(None), [1, 0, 0, 1]), "prefill"),
    (lambda a: a.update(link=np.zeros((4, 4))), "bandwidth"),
    (lambda a: a.update(models=np.array([[1.0, -1.0, 1.0]])), "model"),
    (lambda a: a.update(inst=_inst(2, 0), link=np.full((2, 2), 100.0)), "pool"),
])
def test_create_rejects_bad_arguments_on_the_host(hx, mutate, fragment):
    args = dict(types=np.array([[990.0, 8.0]]), inst=_inst(2, 2), link=np.full((4, 4), 100.0),
                models=np.array([[1e10, 1e10, 1e5]]))
    mutate(args)
    with pytest.raises(hx.HxError) as e:
        hx.hx_cluster_create(args["types"], args["inst"], args["link"], args["models"])
    assert e.value.code == -1 and fragment in str(e.value)


def test_error_message_without_handle(hx):
    with pytest.raises(hx.HxError):
        hx.hx_cluster_create(np.array([[1.0, 1.0]]), _inst(1, 0)[:1], np.ones((1, 1)), np.array([[1.0, 1.0, 1.0]]))
    assert "prefill" in hx.hx_last_error(None) or "instance" in hx.hx_last_error(None)
