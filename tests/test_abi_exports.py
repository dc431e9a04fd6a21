"""The C-ABI library builds, loads on a machine without a GPU, and exports every
function that include/lorc.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "lorc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lorc_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = _declared()
    for must in ("lorc_load_factors", "lorc_append", "lorc_decode_attn", "lorc_create", "lorc_destroy"):
        assert must in names


def test_library_builds_loads_and_exports_every_declared_symbol():
    import paper_2410_03111_b200 as pkg
    path = pkg._build.build()
    lib = ctypes.CDLL(path)
    for name in _declared():
        assert hasattr(lib, name), f"{name} declared in lorc.h but not exported"
    b = pkg.load()
    assert sorted(b.EXPORTS) == _declared()


def test_struct_layouts_match_the_header():
    import paper_2410_03111_b200 as pkg
    b = pkg.load()
    assert ctypes.sizeof(b.lorc_model_desc) == 8 * 4 + 8
    assert ctypes.sizeof(b.lorc_cache) == 4 * 8 + 6 * 4 + 8
    assert b.lorc_cache.seq_stride.offset == 56


def test_null_arguments_are_rejected_without_a_gpu():
    import paper_2410_03111_b200 as pkg
    b = pkg.load()
    assert b._lib.lorc_create(None, None) == b.LORC_ERR_ARG
    assert b._lib.lorc_destroy(None) == b.LORC_ERR_ARG
    assert b._lib.lorc_workspace_bytes(None, 1, 1) == 0
    assert b._lib.lorc_last_error(None) == b"null context"
    desc = b.lorc_model_desc(1, 256, 4, 2, 96, 0, 128, 0, 10000.0)    # d_head 96 unsupported
    out = ctypes.c_void_p()
    assert b._lib.lorc_create(ctypes.byref(desc), ctypes.byref(out)) == b.LORC_ERR_UNSUPPORTED
    desc = b.lorc_model_desc(1, 256, 5, 2, 64, 0, 128, 0, 10000.0)    # 5 heads over 2 KV heads
    assert b._lib.lorc_create(ctypes.byref(desc), ctypes.byref(out)) == b.LORC_ERR_ARG
