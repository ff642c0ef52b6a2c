"""The C-ABI library loads without a GPU and exports every function the headers under include/ declare;
host-only argument checks work (no compute is attempted here)."""
import ctypes as C
import os
import re

import pytest

from paper_2407_19947_b200 import build as stairs_build
from paper_2407_19947_b200 import stairs as st
from paper_2407_19947_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    stairs_build.build()
    return st.load_library()


def declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):          # the supported interface and the unstable inspection hooks
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(inc, fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(stairs_[a-z_]+)\s*\(", text))
    return sorted(names)


def test_every_declared_function_is_exported(lib):
    names = declared_functions()
    assert "stairs_validate" in names and "stairs_generate" in names and "stairs_init" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared under include/ but not exported"
    assert sorted(st.EXPORTS) == names


def make_cfg(shape, **kw):
    cfg = st.CConfig()
    cfg.struct_size = C.sizeof(st.CConfig)
    cfg.target = st.c_model(shape)
    cfg.max_requests, cfg.max_seq_len, cfg.k_max, cfg.kv_page_tokens = 2, 128, 4, 16
    for k, v in kw.items():
        setattr(cfg, k, v)
    return cfg


def test_workspace_size_grows_with_the_configuration(lib):
    shape = wl.workload(1).target
    a = lib.stairs_workspace_bytes(C.byref(make_cfg(shape)))
    b = lib.stairs_workspace_bytes(C.byref(make_cfg(shape, max_requests=4)))
    assert a > 0 and b > a and a % 256 == 0
    # KV pool of the target: layers * 2 * pages * page_tokens * Hkv*hd * 4 bytes must fit inside
    kv = shape.n_layers * 2 * (128 // 16) * 2 * 16 * shape.n_kv_heads * shape.head_dim * 4
    assert a > kv


@pytest.mark.parametrize("bad", [dict(kv_page_tokens=24), dict(k_max=64), dict(max_requests=0),
                                 dict(struct_size=8), dict(max_seq_len=100000)])
def test_bad_configurations_are_refused_with_a_message(lib, bad):
    cfg = make_cfg(wl.workload(1).target, **bad)
    assert lib.stairs_workspace_bytes(C.byref(cfg)) == 0
    assert len(lib.stairs_last_error(None)) > 0


def test_init_refuses_missing_workspace_before_touching_cuda(lib):
    cfg = make_cfg(wl.workload(1).target)
    w = st.CWeights()
    h = C.c_void_p()
    rc = lib.stairs_init(C.byref(cfg), C.byref(w), None, C.byref(h))
    assert rc == 1 and not h.value
    assert b"workspace" in lib.stairs_last_error(None)


def test_null_context_is_an_error_not_a_crash(lib):
    assert lib.stairs_sync(None) == 1
    assert lib.stairs_destroy(None) == 1
    assert lib.stairs_launch_count(None) == 0
