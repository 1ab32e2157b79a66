"""The shared library loads, exports every symbol the public header declares, and rejects bad
arguments on the host before touching the device (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def clv():
    from paper_2408_00264_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "clv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(clv_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(clv):
    names = declared_symbols()
    assert "clv_tree_attn" in names and "clv_kv_commit" in names and len(names) >= 11
    L = ctypes.CDLL(clv.LIB_PATH)
    for n in names:
        assert hasattr(L, n), n
    assert set(names) == set(clv.EXPORTS)


def test_version_and_status_strings(clv):
    assert clv.clv_version() >= 100
    assert clv.clv_status_string(0) == "ok"
    assert "tree" in clv.clv_status_string(clv.CLV_ERR_TREE)


def test_host_side_argument_checks(clv):
    L = clv.lib()
    ok = clv.make_shape(1, 16, 32, 32, 32000, 5)
    assert L.clv_tree_attn(None, *([None] * 6), 0, 1.0, *([None] * 4), 0, None) == clv.CLV_ERR_NULL
    for bad, code in [(clv.make_shape(0, 16, 32, 32), clv.CLV_ERR_SHAPE),
                      (clv.make_shape(1, 16, 30, 8), clv.CLV_ERR_SHAPE),
                      (clv.make_shape(1, 129, 32, 8), clv.CLV_ERR_UNSUPPORTED),
                      (clv.make_shape(1, 16, 32, 8, head_dim=64), clv.CLV_ERR_UNSUPPORTED)]:
        assert L.clv_accept_walk(clv._ref(bad), *([None] * 8)) == code
    assert L.clv_accept_walk(clv._ref(ok), *([None] * 8)) == clv.CLV_ERR_NULL
    # misaligned logits pointer / stride, too-small stride
    fake = ctypes.c_void_p(0x1000_0008)
    al = ctypes.c_void_p(0x1000_0000)
    assert L.clv_accept_argmax(clv._ref(ok), fake, 32000, al, None, 0, None) == clv.CLV_ERR_ALIGN
    assert L.clv_accept_argmax(clv._ref(ok), al, 32004, al, None, 0, None) == clv.CLV_ERR_ALIGN
    assert L.clv_accept_argmax(clv._ref(ok), al, 31992, al, None, 0, None) == clv.CLV_ERR_SHAPE
    # a split argmax needs a workspace
    assert L.clv_accept_argmax(clv._ref(ok), al, 32000, al, None, 0, None) == clv.CLV_ERR_WORKSPACE
    # paged cache with the wrong page size
    cache = clv.ClvKvCache(0x1000_0000, 0x2000_0000, 1, 0, 32, 10, 4, 0x3000_0000)
    args = [al] * 5
    assert L.clv_tree_attn(clv._ref(ok), clv._ref(cache), *args, 0, 1.0, al, None, al, None, 0,
                           None) == clv.CLV_ERR_UNSUPPORTED
    # commit refuses tree buffers that overlap the cache
    cache = clv.ClvKvCache(0x1000_0000, 0x2000_0000, 0, 4096, 64, 0, 0, None)
    inside = ctypes.c_void_p(0x1000_0000 + 4096)
    assert L.clv_kv_commit(clv._ref(ok), clv._ref(cache), inside, ctypes.c_void_p(0x4000_0000),
                           al, al, al, al, al, None) == clv.CLV_ERR_UNSUPPORTED


def test_workspace_size_is_monotone_and_covers_fixed_part(clv):
    s = clv.make_shape(4, 64, 32, 8, 128256, 7)
    small = clv.clv_workspace_bytes(s, None, 0)
    big = clv.clv_workspace_bytes(s, None, 4096)
    assert small >= 256 + 4 * 65536 and big >= small
    assert clv.clv_staging_bytes(s, 128256) > 4 * 64 * 128256 * 2


def test_host_step_checks_everything_before_it_enqueues_anything(clv):
    # clv_verify_step_host runs the argument checks of all three calls before its first copy, so
    # a mistake the host can see returns its code with nothing on the stream.  No device is needed
    # to see the codes: the pointers below are never dereferenced.
    L = clv.lib()
    s = clv.make_shape(2, 8, 4, 2, 1000, 5)
    cache = clv.ClvKvCache(0x1000_0000, 0x2000_0000, 0, 256, 64, 0, 0, None)
    host = ctypes.c_void_p(0x5000_0000)
    hin = clv.ClvHostInputs(*([0x5000_0000] * 6), 1000)
    hout = clv.ClvHostOutputs(*([0x6000_0000] * 6))
    staging = ctypes.c_void_p(0x7000_0000)
    need = clv.clv_staging_bytes(s, 1000)
    ws = ctypes.c_void_p(0x7800_0000)
    ws_need = clv.clv_workspace_bytes(s, None, 200)

    def call(hin=hin, staging_bytes=need, ws=ws, ws_bytes=ws_need):
        return L.clv_verify_step_host(clv._ref(s), clv._ref(cache), clv._ref(hin), clv._ref(hout), host, 200,
                                      1.0, staging, staging_bytes, ws, ws_bytes, None)
    bad_ld = clv.ClvHostInputs(*([0x5000_0000] * 6), 999)              # row stride below the vocabulary
    assert call(hin=bad_ld) == clv.CLV_ERR_SHAPE
    assert call(staging_bytes=need - 1) == clv.CLV_ERR_WORKSPACE
    assert call(ws=None, ws_bytes=0) == clv.CLV_ERR_WORKSPACE           # the attention's check
    assert call(ws_bytes=1024) == clv.CLV_ERR_WORKSPACE
