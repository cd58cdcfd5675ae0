"""The C-ABI library loads and exports every symbol include/hf.h declares; host-side argument checks
that need no device."""
import ctypes as C
import os
import re

import pytest

from paper_2604_10103_b200 import binding as hf, build as hfbuild, inputs as gen

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    hfbuild.build()
    return hf.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "hf.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hf_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert sorted(hf.EXPORTS) == names
    for n in names:
        assert getattr(lib, n) is not None


def test_status_strings(lib):
    assert lib.hf_status_string(0) == b"HF_OK"
    assert [lib.hf_status_string(i).decode() for i in range(8)] == hf.STATUS_NAMES
    assert lib.hf_status_string(99) == b"HF_ERR_UNKNOWN"


def test_config_struct_matches_header():
    text = open(os.path.join(ROOT, "include", "hf.h")).read()
    body = re.search(r"typedef struct \{(.*?)\} hf_config;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for decl in body.split(";"):
        decl = decl.strip()
        if decl:
            ty, names = decl.split(None, 1)
            fields += [(n.strip(), ty) for n in names.split(",")]
    assert [(n, "float" if t is C.c_float else "int") for n, t in hf.hf_config._fields_] == fields


@pytest.mark.parametrize("bad", [
    dict(head_dim=96), dict(block=32), dict(window_frames=4), dict(window_frames=30), dict(topk=0, keep_permille=0),
    dict(keep_permille=1001), dict(batch=0), dict(layers=0), dict(tokens_per_frame=0),
])
def test_invalid_configs_are_rejected_before_any_device_call(lib, bad):
    w = gen.layer_832x480()
    cfg = hf.make_config(w)
    for k, v in bad.items():
        setattr(cfg, k, v)
    h = C.c_void_p()
    st = lib.hf_create(C.byref(cfg), 0, C.byref(h))
    assert st == 2 and not h.value, lib.hf_last_error()
    assert lib.hf_last_error() != b""


def test_null_arguments(lib):
    assert lib.hf_create(None, 0, None) == 1
    assert lib.hf_destroy(None) == 1
    assert lib.hf_kv_append(None, 0, None, None, None) == 1
    assert lib.hf_hybrid_forward(None, 0, None, None, None, None, None) == 1


def test_create_without_a_device_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(hf.HFError, match="HF_ERR_CUDA|HF_ERR_INVALID_ARG"):
        hf.Context(hf.make_config(gen.tiny()))
