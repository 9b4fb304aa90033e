"""The C-ABI library loads without a GPU, exports every symbol the header
declares, and rejects bad arguments on the host before touching CUDA."""
import ctypes as C
import os
import re

import pytest

from paper_2312_08538_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def b():
    build.build_library()
    from paper_2312_08538_b200 import binding
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "conef.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(conef_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(b):
    names = declared_functions()
    assert "conef_init" in names and "conef_step" in names and "conef_reduce_messages" in names \
        and "conef_decompress_error" in names
    for n in names:
        assert hasattr(b.lib, n), f"{n} is declared in include/conef.h but not exported"
    assert sorted(b.EXPORTS) == names


def test_workspace_query_validates_the_configuration(b):
    ok_q = dict(kind="randk", k_num=1, k_den=100, seed=1)
    ok_c = dict(kind="int8", block=256)
    assert b.conef_workspace_bytes([(256, 512, 1)], 2, ok_q, ok_c) > 256 * 512 * 2
    bad = [
        ([(0, 5, 1)], 2, ok_q, ok_c, b.ERR_INVALID_ARG),
        ([(4, 5, 1)], 0, ok_q, ok_c, b.ERR_INVALID_ARG),
        ([(4, 5, 1)], 65, ok_q, ok_c, b.ERR_UNSUPPORTED),
        ([(1 << 20, 1 << 13, 1)], 1, ok_q, ok_c, b.ERR_UNSUPPORTED),          # d >= 2^32
        ([(4, 5, 1)], 2, dict(kind="randk", k_num=2, k_den=1), ok_c, b.ERR_INVALID_ARG),
        ([(4, 5, 1)], 2, dict(kind="lowrank", rank=0), ok_c, b.ERR_INVALID_ARG),
        ([(4, 5, 1)], 2, dict(kind="lowrank", rank=9), ok_c, b.ERR_UNSUPPORTED),
        ([(4, 5, 1)], 2, ok_q, dict(kind="int8", block=100), b.ERR_INVALID_ARG),
        ([(4, 5, 1)], 2, ok_q, dict(kind="int4", block=32), b.ERR_INVALID_ARG),
        ([(4, 5, 1)], 2, ok_q, dict(kind="countsketch", cs_rows=4), b.ERR_INVALID_ARG),
        ([(4, 5, 1)], 2, ok_q, dict(kind="countsketch", cs_rows=9), b.ERR_INVALID_ARG),
        ([(64, 64, 1)], 2, ok_q, dict(kind="countsketch", cs_rows=3, cs_chunk=100), b.ERR_INVALID_ARG),    # not a multiple of 256
        ([(64, 64, 1)], 2, ok_q, dict(kind="countsketch", cs_rows=3, cs_chunk=-256), b.ERR_INVALID_ARG),
        ([(64, 64, 1)], 2, ok_q, dict(kind="countsketch", cs_rows=3, cs_col_div=100, cs_chunk=256), b.ERR_INVALID_ARG),  # < 4 cs_col_div
    ]
    for tensors, n, q, c, code in bad:
        with pytest.raises(b.ConEFError) as e:
            b.conef_workspace_bytes(tensors, n, q, c)
        assert e.value.code == code, (tensors, n, q, c)


def test_state_sizes_match_the_memory_saving_arithmetic(b):
    # int4 / blocks of 128 / fp16 scale: 0.5 + 2/128 bytes per element = 12.9 % of fp32
    tensors = [(1600, 6400, 1)]
    small = b.conef_workspace_bytes(tensors, 1, dict(kind="identity"), dict(kind="int4", block=128, scale_dtype="fp16"))
    dense = b.conef_workspace_bytes(tensors, 1, dict(kind="identity"), dict(kind="identity"))
    d = 1600 * 6400
    assert dense - small == pytest.approx(d * 4 - d * (0.5 + 2 / 128), abs=4096)


def test_init_rejects_bad_workspaces_on_the_host(b):
    t = b.make_tensors([(8, 8, 1)])
    q = b.make_q(dict(kind="randk", k_num=1, k_den=2, seed=1), None)
    c = b.make_c(dict(kind="int8", block=32))
    h = C.c_void_p()
    assert b.lib.conef_init(C.byref(h), t, 1, 1, C.byref(q), C.byref(c), 0.1, None, 1 << 20, None) == b.ERR_INVALID_ARG
    assert b.lib.conef_init(C.byref(h), t, 1, 1, C.byref(q), C.byref(c), 0.1, 256 * 1000, 16, None) == b.ERR_WORKSPACE_TOO_SMALL
    assert b.lib.conef_init(C.byref(h), t, 1, 1, C.byref(q), C.byref(c), 0.1, 256 * 1000 + 8, 1 << 20, None) == b.ERR_INVALID_ARG
    assert b.lib.conef_init(None, t, 1, 1, C.byref(q), C.byref(c), 0.1, 256 * 1000, 1 << 20, None) == b.ERR_INVALID_ARG
    assert h.value is None
    # null contexts are rejected everywhere
    assert b.lib.conef_step(None, 0, None, 0, None) == b.ERR_INVALID_ARG
    assert b.lib.conef_reduce_messages(None, 0, None, None) == b.ERR_INVALID_ARG
    assert b.lib.conef_decompress_error(None, 0, None, None) == b.ERR_INVALID_ARG
    assert b.lib.conef_message_elems(None, 0) == -1
    assert b.lib.conef_error_string(b.ERR_BAD_PHASE).decode().startswith("calls out of order")
