"""The C-ABI library builds, loads without a GPU and exports every symbol include/hippo.h declares; argument
validation rejects bad calls before anything is launched.  CPU only."""
import ctypes
import os
import re

from paper_2601_08273_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "hippo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hippo_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    build.build_library()
    from paper_2601_08273_b200 import binding
    names = declared_functions()
    assert {"hippo_select_tokens", "hippo_gather_kv", "hippo_draft_attention", "hippo_verify_attention",
            "hippo_accept"} <= set(names)
    for n in names:
        assert hasattr(binding.lib, n), n
    assert binding.hippo_version() == 101
    assert binding.lib.hippo_status_string(-5).decode() == "device-side wait timed out"


def test_argument_validation_happens_before_any_launch():
    from paper_2601_08273_b200 import binding as hb
    lib = hb.lib
    assert lib.hippo_accept(0, 1, 10, None, None, None, None, None, 0, None, None, None, 0, None) == hb.HIPPO_ERR_INVALID_ARG
    assert lib.hippo_accept(1, 1, 10, None, None, None, None, None, 0, None, None, None, 0, None) == hb.HIPPO_ERR_INVALID_ARG
    assert b"null pointer" in lib.hippo_last_error()
    assert lib.hippo_accept(1, 1, 10, 256, 256, 256, 256, 256, 7, 256, 256, 256, 1 << 20, None) == hb.HIPPO_ERR_UNIMPLEMENTED   # unknown mode
    assert lib.hippo_accept(1, 1, 10, 256, 256, 256, 256, 256, 0, 256, 256, 256, 16, None) == hb.HIPPO_ERR_WORKSPACE_TOO_SMALL
    kv = hb.KVCacheStruct(ctypes.sizeof(hb.KVCacheStruct), hb.HIPPO_DTYPE_BF16, 2, 64, 10, 4, 1024, 2048, None)
    args = lambda **o: [o.get("B", 1), o.get("q_len", 1), o.get("hq", 14), 256, ctypes.byref(kv), 256, o.get("host_len"),
                        o.get("max_kv", 200), 0.0, 0, 256, None, o.get("ws", 256), o.get("ws_bytes", 1 << 30), None]
    assert lib.hippo_draft_attention(*args(hq=15)) == hb.HIPPO_ERR_INVALID_ARG          # 15 % 2 != 0
    assert lib.hippo_draft_attention(*args(max_kv=257)) == hb.HIPPO_ERR_INVALID_ARG      # > 4 pages
    assert lib.hippo_draft_attention(*args(ws_bytes=1000)) == hb.HIPPO_ERR_WORKSPACE_TOO_SMALL
    assert lib.hippo_draft_attention(*args(q_len=40)) == hb.HIPPO_ERR_UNSUPPORTED_SHAPE  # 40*7 packed rows
    assert lib.hippo_draft_attention(*args(B=3)) == hb.HIPPO_ERR_INVALID_ARG             # identity mapping needs 12 pages
    assert lib.hippo_draft_attention(*args(host_len=(ctypes.c_int32 * 1)(201))) == hb.HIPPO_ERR_INVALID_ARG   # host length > max_kv_len
    kv.struct_size = 8
    assert lib.hippo_verify_attention(*args()) == hb.HIPPO_ERR_INVALID_ARG
    n_visual = (ctypes.c_int32 * 1)(100)
    k = (ctypes.c_int32 * 1)(101)
    assert lib.hippo_select_tokens(1, n_visual, 14, 14, 5, 5, 64, 1, 256, 256, k, None, 7, 256, 256, 256, 1 << 30, None) == hb.HIPPO_ERR_INVALID_ARG
    k[0] = 10
    assert lib.hippo_select_tokens(1, n_visual, 14, 14, 6, 6, 64, 1, 256, 256, k, None, 7, 256, 256, 256, 1 << 30, None) == hb.HIPPO_ERR_UNSUPPORTED_SHAPE
    assert hb.hippo_select_workspace_bytes([100], 14, 14) >= 256 + 3 * 800
    assert hb.hippo_attention_workspace_bytes(1, 6, 28, 4, 128) > 42 * 130 * 4 * 4
    assert hb.hippo_accept_workspace_bytes(1, 5, 152064) > 0


def test_attention_mass_argument_validation():
    from paper_2601_08273_b200 import binding as hb
    lib = hb.lib
    kv = hb.KVCacheStruct(ctypes.sizeof(hb.KVCacheStruct), hb.HIPPO_DTYPE_BF16, 2, 128, 16, 8, 1024, 2048, None)
    nv = (ctypes.c_int32 * 2)(300, 200)
    need = lib.hippo_attention_mass_workspace_bytes(2, nv, 32, 8, 2, 128, hb.HIPPO_DTYPE_BF16)
    assert need > 256
    assert lib.hippo_attention_mass_workspace_bytes(2, nv, 32, 7, 2, 128, hb.HIPPO_DTYPE_BF16) == 0     # heads do not divide
    assert lib.hippo_attention_mass_workspace_bytes(65, nv, 32, 8, 2, 128, hb.HIPPO_DTYPE_BF16) == 0    # batch limit
    call = lambda **o: lib.hippo_attention_mass(o.get("B", 2), o.get("nv", nv), o.get("l_txt", 32), o.get("hq", 8), o.get("q", 256),
                                                ctypes.byref(kv), ctypes.c_float(o.get("scale", 0.0)), ctypes.c_float(o.get("w", 1.0)),
                                                o.get("mass", 256), o.get("ws", 256), o.get("ws_bytes", 1 << 30), None)
    assert call(q=None) == hb.HIPPO_ERR_INVALID_ARG
    assert call(hq=7) == hb.HIPPO_ERR_INVALID_ARG
    assert call(B=65) == hb.HIPPO_ERR_UNSUPPORTED_SHAPE
    assert call(ws_bytes=need - 1) == hb.HIPPO_ERR_WORKSPACE_TOO_SMALL
    assert call(ws=264) == hb.HIPPO_ERR_INVALID_ARG                      # workspace alignment
    assert call(scale=-1.0) == hb.HIPPO_ERR_INVALID_ARG
    assert call(q=264 + 2) == hb.HIPPO_ERR_INVALID_ARG                   # query alignment
    too_long = (ctypes.c_int32 * 2)(300, 8 * 64 + 1)
    assert call(nv=too_long) == hb.HIPPO_ERR_INVALID_ARG                 # longer than the cache's pages
    # identity page mapping needs batch * max_pages_per_seq <= n_pages: 2 * 8 = 16 fits, 3 sequences do not
    nv3 = (ctypes.c_int32 * 3)(10, 10, 10)
    assert call(B=3, nv=nv3) == hb.HIPPO_ERR_INVALID_ARG
    # nothing to score: accepted, nothing launched
    zero = (ctypes.c_int32 * 2)(0, 0)
    before = hb.hippo_launch_count()
    assert call(nv=zero) == hb.HIPPO_OK
    assert hb.hippo_launch_count() == before
