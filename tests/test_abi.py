"""CPU checks of the C ABI: the library loads, exports every symbol the header
declares, and rejects bad arguments on the host before touching a device."""
import ctypes
import os
import re

import pytest

from paper_2609_37626_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def declared_symbols():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            names += re.findall(r"SPLASH_API\s+[\w\s\*]+?\b(splash_\w+)\s*\(", text)
    return names


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 10 and "splash_mla_decode" in names and "splash_kv_page_migrate" in names
    for n in names:
        assert hasattr(lib, n), n


def test_struct_layout_matches_header(lib):
    assert ctypes.sizeof(binding.MlaShape) == 88


def test_status_strings(lib):
    assert lib.splash_status_string(0) == b"ok"
    assert b"invalid" in lib.splash_status_string(-1)
    assert lib.splash_version() >= 100


def good_shape(**kw):
    s = binding.MlaShape(struct_size=ctypes.sizeof(binding.MlaShape), num_requests=2, num_heads=16, d_qk=576,
                         d_v=512, page_size=64, num_pool_pages=8, block_table_stride=4, kv_dtype=0,
                         softmax_scale=0.07, q_stride_request=16 * 576, q_stride_head=576,
                         out_stride_request=16 * 512, out_stride_head=512, lse_stride_request=16, flags=0, q_rows=0)
    for k, v in kw.items():
        setattr(s, k, v)
    return s


def call_decode(lib, shape, hb=0, he=16, ptr=0x1000, ws_bytes=1 << 20, q=None):
    p = ctypes.c_void_p(ptr)
    return lib.splash_mla_decode(ctypes.byref(shape), p if q is None else q, p, None, p, p, hb, he, None, None,
                                 p, p, p, ws_bytes, None)


def test_decode_rejects_bad_arguments_on_the_host(lib):
    assert call_decode(lib, good_shape(struct_size=4)) == binding.SPLASH_INVALID_ARG
    assert call_decode(lib, good_shape(d_qk=128)) == binding.SPLASH_UNSUPPORTED
    assert call_decode(lib, good_shape(page_size=16)) == binding.SPLASH_UNSUPPORTED
    assert call_decode(lib, good_shape(kv_dtype=7)) == binding.SPLASH_UNSUPPORTED
    assert call_decode(lib, good_shape(num_heads=256)) == binding.SPLASH_UNSUPPORTED
    assert call_decode(lib, good_shape(), hb=-1) == binding.SPLASH_INVALID_ARG
    assert call_decode(lib, good_shape(), hb=8, he=4) == binding.SPLASH_INVALID_ARG
    assert call_decode(lib, good_shape(), he=17) == binding.SPLASH_INVALID_ARG
    assert call_decode(lib, good_shape(q_stride_head=580)) == binding.SPLASH_INVALID_ARG
    assert call_decode(lib, good_shape(), q=ctypes.c_void_p(0)) == binding.SPLASH_INVALID_ARG
    assert call_decode(lib, good_shape(), ptr=0x1008) == binding.SPLASH_INVALID_ARG      # misaligned
    assert b"align" in lib.splash_last_error()
    # idle rank: no requests or an empty head slice is a successful no-op, nothing dereferenced
    assert call_decode(lib, good_shape(num_requests=0)) == binding.SPLASH_OK
    assert call_decode(lib, good_shape(), hb=4, he=4) == binding.SPLASH_OK
    assert lib.splash_last_launch_count() == 0


def test_merge_and_migrate_reject_bad_arguments(lib):
    p = ctypes.c_void_p(0x1000)
    assert lib.splash_lse_merge(2, 4, 510, p, p, p, p, None) == binding.SPLASH_INVALID_ARG
    assert lib.splash_lse_merge(2, 0, 512, p, p, p, p, None) == binding.SPLASH_OK
    assert lib.splash_lse_merge(2, 4, 512, p, p, None, p, None) == binding.SPLASH_INVALID_ARG
    assert lib.splash_lse_merge(2, 4, 512, p, p, p, p, None) == binding.SPLASH_INVALID_ARG   # out aliases parts
    assert lib.splash_kv_page_migrate(p, None, p, None, 73728, p, p, 0, 0, 0, 16, p, 8, p, 4096, None) == binding.SPLASH_OK
    assert lib.splash_kv_page_migrate(p, None, p, None, 100, p, p, 1, 0, 0, 16, p, 8, p, 4096, None) == binding.SPLASH_INVALID_ARG
    assert lib.splash_kv_page_migrate(p, p, p, None, 73728, p, p, 1, 0, 0, 16, p, 8, p, 4096, None) == binding.SPLASH_INVALID_ARG
    assert lib.splash_kv_page_migrate(p, None, p, None, 73728, p, p, 1, 0, 0, 1 << 20, p, 8, p, 64, None) == binding.SPLASH_INVALID_ARG
    assert lib.splash_kv_page_migrate_workspace_bytes(1000) >= 4000


def test_dop_layout_changes_reject_bad_arguments(lib):
    p, q = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x100000)
    # empty work is legal (a rank that owns no rows still takes part in the exchange)
    assert lib.splash_dop_pack_rows(p, 1024, 4096, 1024, p, 128, 512, 128, p, 0, 4, q, None) == binding.SPLASH_OK
    assert lib.splash_dop_swap_outer(p, 4, 0, 64, q, None) == binding.SPLASH_OK
    assert lib.splash_dop_unpack_rows(p, p, 0, 64, q, 64, None) == binding.SPLASH_OK
    # odd sizes, missing pointers, a head pitch shorter than the part, overlapping buffers
    assert lib.splash_dop_pack_rows(p, 1023, 4096, 1024, None, 0, 0, 0, p, 3, 4, q, None) == binding.SPLASH_INVALID_ARG
    assert lib.splash_dop_pack_rows(p, 1024, 4096, 1024, None, 128, 512, 128, p, 3, 4, q, None) == binding.SPLASH_INVALID_ARG
    assert lib.splash_dop_pack_rows(p, 1024, 4096, 512, None, 0, 0, 0, p, 3, 4, q, None) == binding.SPLASH_INVALID_ARG
    assert lib.splash_dop_pack_rows(p, 1024, 4096, 1024, None, 0, 0, 0, None, 3, 4, q, None) == binding.SPLASH_INVALID_ARG
    assert lib.splash_dop_swap_outer(p, 4, 4, 64, ctypes.c_void_p(0x1100), None) == binding.SPLASH_INVALID_ARG
    assert lib.splash_dop_swap_outer(p, 4, 4, 63, q, None) == binding.SPLASH_INVALID_ARG
    assert lib.splash_dop_unpack_rows(p, p, 3, 64, q, 32, None) == binding.SPLASH_INVALID_ARG
