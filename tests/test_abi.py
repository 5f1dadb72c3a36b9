"""The C boundary: the library loads, exports every symbol the header declares,
and fails loudly (never falls back) when there is no CUDA device.  No GPU."""
import ctypes
import os
import re

import pytest
import torch

import paper_2512_20687_b200 as ph
from paper_2512_20687_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return ph.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "photon.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(photon_[a-z_]+)\s*\(", text)))


def test_header_declares_the_expected_calls():
    names = declared_symbols()
    for want in ("photon_create", "photon_destroy", "photon_kv_append", "photon_coarse_attn",
                 "photon_flat_attn", "photon_converter", "photon_chunk_attn", "photon_chunk_causal_attn",
                 "photon_decode_step",
                 "photon_device_status", "photon_status_str"):
        assert want in names


def test_library_exports_every_declared_symbol(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), f"libphoton.so does not export {name}"


def test_binding_has_the_same_names():
    for name in declared_symbols():
        assert hasattr(ph, name), f"binding lacks {name}"


def test_struct_layouts_match_the_header():
    assert ctypes.sizeof(ph.photon_config) == 8 * 4
    # pointers are 8-byte aligned: 3 ptr + 3 int32 (+pad) + 4 ptr + 3 int32 (+pad)
    assert ctypes.sizeof(ph.photon_kv) == 24 + 16 + 32 + 16 + 8 + 16 and ph.photon_kv.page_table.offset == 88
    assert ph.photon_kv.max_len.offset == 32 and ph.photon_kv.k_shared.offset == 40
    assert ph.photon_step_args.scale_coarse.offset == 48 and ph.photon_step_args.x.offset == 56
    assert ctypes.sizeof(ph.photon_layer) == 6 * 8 + 4 * 4 and ph.photon_layer.F.offset == 52
    assert ctypes.sizeof(ph.photon_layer_scratch) == 9 * 8


def test_status_strings(lib):
    assert ph.photon_status_str(ph.PHOTON_OK) == "ok"
    assert "invalid" in ph.photon_status_str(ph.PHOTON_ERR_INVALID_ARG)
    assert ph.photon_status_str(99) == "unknown status"


def test_null_arguments_are_rejected_before_any_cuda_call(lib):
    assert lib.photon_create(None, None) == ph.PHOTON_ERR_INVALID_ARG
    assert lib.photon_destroy(None) == ph.PHOTON_ERR_INVALID_ARG
    assert lib.photon_decode_step(None, None, None) == ph.PHOTON_ERR_INVALID_ARG
    assert lib.photon_coarse_attn(None, None, None, None, None, 1.0, None) == ph.PHOTON_ERR_INVALID_ARG
    assert lib.photon_converter(None, None, None, 0, None, None, 1, None) == ph.PHOTON_ERR_INVALID_ARG
    bad = ph.photon_config(4, 3, 64, 256, 4, 4, 16, 0)          # Hq % Hkv != 0
    h = ctypes.c_void_p(0)
    assert lib.photon_create(ctypes.byref(h), ctypes.byref(bad)) == ph.PHOTON_ERR_INVALID_ARG
    bad = ph.photon_config(4, 2, 56, 256, 4, 4, 16, 0)          # head size the kernels are not built for
    assert lib.photon_create(ctypes.byref(h), ctypes.byref(bad)) == ph.PHOTON_ERR_UNSUPPORTED
    assert not h.value


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device behaviour")
def test_without_a_device_create_fails_loudly():
    with pytest.raises(ph.PhotonError) as e:
        ph.photon_create(4, 2, 64, 256, 4, 4, 16)
    assert e.value.code == ph.PHOTON_ERR_CUDA
    with pytest.raises(ValueError):
        ph.photon_converter(ctypes.c_void_p(1), torch.zeros(2, 2), None, 0, None, None)
