"""The C-ABI library loads without a GPU and exports everything include/wisv.h declares."""
import ctypes as C
import os
import re

import pytest

import paper_2604_17701_b200 as wisv
from paper_2604_17701_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return wisv.load_library()


def test_every_declared_symbol_is_exported(lib):
    names = wisv.exported_symbols()
    assert {"wisv_create", "wisv_verify", "wisv_verify_host", "wisv_destroy", "wisv_strerror",
            "wisv_version"} <= set(names)
    for n in names:
        assert getattr(lib, n) is not None


def test_version_and_error_strings(lib):
    header = open(os.path.join(ROOT, "include", "wisv.h")).read()
    assert lib.wisv_version() == int(re.search(r"#define WISV_VERSION (\d+)", header).group(1))
    codes = dict(re.findall(r"#define (WISV_E[A-Z]+)\s+(-\d+)", header))
    assert len(codes) >= 8
    seen = set()
    for name, v in codes.items():
        s = lib.wisv_strerror(int(v)).decode()
        assert s and s != "unknown error" and s not in seen
        seen.add(s)
    assert lib.wisv_strerror(-999).decode() == "unknown error"


def test_struct_layouts_match_the_header():
    # field order and types mirror include/wisv.h; sizes follow the C ABI on x86-64
    assert C.sizeof(binding._Config) == 13 * 4
    assert C.sizeof(binding._Weights) == 4 * 8 + 8
    assert C.sizeof(binding._Result) == 9 * 8
    assert binding._Batch.k_off.offset == 8 and binding._Batch.target_hidden.offset == 24
    assert binding._Batch.mode.offset == binding._Batch.uniforms.offset + 8
    header = open(os.path.join(ROOT, "include", "wisv.h")).read()
    for struct, cls in (("wisv_config", binding._Config), ("wisv_weights", binding._Weights),
                        ("wisv_batch", binding._Batch), ("wisv_result", binding._Result)):
        body = re.search(r"typedef struct \{([^}]*)\} %s;" % struct, header).group(1)
        body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
        fields = re.findall(r"\b([A-Za-z_0-9]+)\s*;", body)
        assert fields == [f[0] for f in cls._fields_], struct


def test_argument_errors_need_no_device(lib):
    h = C.c_void_p()
    assert lib.wisv_create(None, None, C.byref(h)) == -1
    assert h.value is None
    assert lib.wisv_destroy(None) == -1
    assert lib.wisv_verify(None, None, None, None) == -1
    assert lib.wisv_launch_count(None) == 0
    cfg = binding._Config(4096, 128256, 2048, 2, 1024, 7, 0, 0.5, 1, 9, 0, 0, 0)     # bad activation enum
    w = binding._Weights(16, 16, 16, 16, 0.0)
    assert lib.wisv_create(C.byref(cfg), C.byref(w), C.byref(h)) == -1
    cfg.act = 1
    cfg.H = 4097                                                               # H % 8 != 0
    assert lib.wisv_create(C.byref(cfg), C.byref(w), C.byref(h)) == -2
    cfg.H = 4096
    w.lm_head = 24                                                             # not 16-byte aligned
    assert lib.wisv_create(C.byref(cfg), C.byref(w), C.byref(h)) == -3
