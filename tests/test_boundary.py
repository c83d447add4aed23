"""Host-side checks of the C-ABI library that need no GPU."""
import ctypes
import os
import re

import pytest

from paper_2411_00288_b200 import api, build as libbuild, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    libbuild.build()
    return api.lib()


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "ssconv.h")).read()
    declared = set(re.findall(r"\b(ssconv_[a-z_0-9]+)\s*\(", header))
    declared -= {"ssconv_status_t", "ssconv_desc_t"}
    assert declared == set(api.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_version_and_status_strings(lib):
    assert api.ssconv_version() >= 100
    assert api.ssconv_launch_count() >= 0  # host-only counter, callable without a GPU
    assert api.status_string(0) == "ok"
    assert "timed out" in api.status_string(api.ERR_TIMEOUT)


def test_out_shape_matches_layer_specs(lib):
    for cfg in (1, 2, 3, 4, 5):
        for spec in synth.config_layers(cfg):
            assert api.ssconv_out_shape(api.desc_from_spec(spec)) == (spec.H_out, spec.W_out)


def test_sizes_are_roughly_half_plus_metadata(lib):
    # 512 x 4608 (3x3, 512 channels): values C_out*K bytes, metadata C_out*K/8 bytes, no padding needed
    d = api.make_desc(1, 7, 7, 512, 512, 3, 3, 1, 1)
    s = api.ssconv_sizes(d)
    assert s.G == 512 * 4608 // 4
    assert s.w_comp_bytes == 512 * 4608
    assert s.meta_bytes == 512 * 4608 // 8
    # padded case: C_out 64 -> 128 rows, 9 k-blocks -> 10
    s = api.ssconv_sizes(api.make_desc(1, 14, 14, 64, 64, 3, 3, 1, 1))
    assert s.w_comp_bytes == 128 * 10 * 32 * 2 and s.meta_bytes == 5 * 2048


def test_host_detectable_errors_return_before_any_launch(lib):
    d = api.make_desc(1, 8, 8, 64, 64, 3, 3, 1, 1)
    p = ctypes.byref(d)
    h, w = ctypes.c_int32(), ctypes.c_int32()
    assert lib.ssconv_out_shape(None, ctypes.byref(h), ctypes.byref(w)) == 1
    bad = api.make_desc(1, 8, 8, 64, 64, 3, 3, 0, 1)  # stride 0
    assert lib.ssconv_out_shape(ctypes.byref(bad), ctypes.byref(h), ctypes.byref(w)) == 2
    empty = api.make_desc(1, 2, 2, 64, 64, 5, 5, 1, 0)  # filter larger than image
    assert lib.ssconv_out_shape(ctypes.byref(empty), ctypes.byref(h), ctypes.byref(w)) == 2
    # null tensors
    assert lib.ssconv_forward(p, None, None, None, None, None, None, 0, None, None) == 1
    assert lib.ssconv_forward_dense(p, None, None, None, None, None, 0, None, None) == 1
    assert lib.ssconv_compress(p, None, None, None, None, None) == 1
    assert lib.ssconv_select_mask(0, None, 4, None, None) == 1
    assert lib.ssconv_select_mask(7, None, 4, None, None) == 2
    assert lib.ssconv_select_mask(0, None, 0, None, None) == 0  # empty input is a no-op
    # unsupported shapes: channels not a multiple of 8
    odd = api.make_desc(1, 8, 8, 12, 64, 3, 3, 1, 1)
    assert lib.ssconv_forward(ctypes.byref(odd), 16, 16, 16, None, 16, None, 0, None, None) == 3
    assert lib.ssconv_compress(ctypes.byref(odd), 16, 16, 16, 16, None) == 3
    # misaligned pointer (never dereferenced: the check is on the address)
    nob = api.make_desc(1, 8, 8, 64, 64, 3, 3, 1, 1, bias=False)
    assert lib.ssconv_forward(ctypes.byref(nob), 8, 16, 16, None, 16, None, 0, None, None) == 4
    # bias flag set but no bias
    assert lib.ssconv_forward(p, 16, 16, 16, None, 16, None, 0, None, None) == 1
