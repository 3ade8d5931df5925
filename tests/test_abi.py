"""The C-ABI library loads and exports every symbol include/evo.h declares (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

import paper_2202_05008_b200 as pk
from paper_2202_05008_b200 import build as B
from paper_2202_05008_b200.binding import EvoConfig, make_config, load_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build_library()
    return load_library()


def _declared_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(evo_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert {"evo_create", "evo_ask", "evo_rollout", "evo_tell", "evo_destroy"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_config_struct_size_matches_and_workspace_is_pure_host(lib):
    for name, w in pk.workloads.CONFIGS.items():
        cfg = make_config(w)
        n = C.c_size_t()
        assert lib.evo_workspace_bytes(C.byref(cfg), C.byref(n)) == 0, name
        ld = (w.param_dim + 31) // 32 * 32
        need = w.pop_size * ld * 4 * (1.5 if cfg.noise_mode == 0 else 1.0)
        assert n.value >= need
    # regenerated noise drops the eps matrix
    a, b = C.c_size_t(), C.c_size_t()
    w = pk.workloads.CFG4
    lib.evo_workspace_bytes(C.byref(make_config(w, noise_mode=0)), C.byref(a))
    lib.evo_workspace_bytes(C.byref(make_config(w, noise_mode=1)), C.byref(b))
    assert a.value - b.value >= (w.pop_size // 2) * w.param_dim * 4


def test_bad_configs_are_rejected(lib):
    n = C.c_size_t()
    w = pk.workloads.CFG1
    cfg = make_config(w); cfg.struct_size = 4
    assert lib.evo_workspace_bytes(C.byref(cfg), C.byref(n)) == 1
    for kw in (dict(pop_size=15), dict(pop_size=0), dict(param_dim=384), dict(sigma=0.0),
               dict(layer_sizes=(4, 16, 16, 1)), dict(episodes=0)):
        cfg = make_config(w.with_(**kw))
        assert lib.evo_workspace_bytes(C.byref(cfg), C.byref(n)) == 1, kw
    # the row pitch must fit 32 bits; the trace covers at most the horizon; the wait limit and the
    # debug bits are range-checked
    assert lib.evo_workspace_bytes(C.byref(make_config(pk.workloads.CFG5.with_(param_dim=(1 << 30) + 1))), C.byref(n)) == 1
    assert lib.evo_workspace_bytes(C.byref(make_config(pk.workloads.CFG5.with_(param_dim=0xFFFFFFF0))), C.byref(n)) == 1
    assert lib.evo_workspace_bytes(C.byref(make_config(w, trace_steps=w.horizon + 1)), C.byref(n)) == 1
    assert lib.evo_workspace_bytes(C.byref(make_config(w, trace_steps=w.horizon)), C.byref(n)) == 0
    assert lib.evo_workspace_bytes(C.byref(make_config(w, wait_cycles_log2=9)), C.byref(n)) == 1
    assert lib.evo_workspace_bytes(C.byref(make_config(w, wait_cycles_log2=41)), C.byref(n)) == 1
    assert lib.evo_workspace_bytes(C.byref(make_config(w, wait_cycles_log2=16, debug_flags=1)), C.byref(n)) == 0
    assert lib.evo_workspace_bytes(C.byref(make_config(w, debug_flags=2)), C.byref(n)) == 1
    assert lib.evo_workspace_bytes(None, C.byref(n)) == 1
    assert lib.evo_workspace_bytes(C.byref(make_config(w)), None) == 1
    # create without a workspace / with a misaligned one fails before any CUDA call
    h = C.c_void_p()
    assert lib.evo_create(C.byref(make_config(w)), None, 1 << 20, None, C.byref(h)) == 1
    assert lib.evo_create(C.byref(make_config(w)), 0x1001, 1 << 20, None, C.byref(h)) == 1
    assert lib.evo_ask(None, None, None) == 1 and lib.evo_tell(None, None) == 1
    assert lib.evo_status_string(5).decode().startswith("non-finite")
    assert lib.evo_version() == 10100                     # 1.1.0 as major*10000 + minor*100 + patch


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    import paper_2202_05008_b200.binding as bd
    monkeypatch.setattr(bd, "_lib", None)
    monkeypatch.setattr(bd, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(FileNotFoundError):
        bd.load_library()
