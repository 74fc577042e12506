"""Host-side checks of the C ABI that need no GPU: exports, status codes, table builder, ring state."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import sdvg_oracle as O
from paper_2604_17397_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return api.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "sdvg.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sdvg_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = declared_symbols()
    assert "sdvg_rope3d_qk" in names and "sdvg_block_attn_fwd" in names
    assert "sdvg_kv_commit" in names and "sdvg_route" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(api.SIGNATURES) == names


def test_status_strings(lib):
    assert lib.sdvg_status_string(0) == b"ok"
    seen = {lib.sdvg_status_string(i) for i in range(8)}
    assert len(seen) == 8
    assert lib.sdvg_status_string(99) == b"unknown status"


def test_pair_split_and_table_match_oracle_bits(lib):
    for d in (64, 128):
        assert api.sdvg_rope3d_pairs(d) == O.rope_axis_pairs(d)
    for d, tf, gh, gw in ((64, 6, 4, 8), (128, 48, 30, 52)):
        mine = api.sdvg_rope3d_table(d, tf, gh, gw).numpy()
        ref = O.rope_table(d, tf, gh, gw)
        assert mine.shape == ref.shape
        assert np.array_equal(mine.view(np.uint32), ref.view(np.uint32))
    assert lib.sdvg_rope3d_table_floats(63, 4, 4, 4) == 0
    assert lib.sdvg_rope3d_table_floats(64, 0, 4, 4) == 0


def _fake_cache(lib, slots=3, heads=2, T=64, D=64, k=0x10000, v=0x20000):
    h = C.c_void_p()
    st = lib.sdvg_cache_create(C.byref(h), k, v, slots, heads, T, D)
    return st, h


def test_cache_handle_validation_and_state(lib):
    assert lib.sdvg_cache_bytes(7, 40, 4680, 128) == 7 * 40 * 4680 * 128 * 2
    assert lib.sdvg_cache_bytes(7, 40, 4680, 96) == 0
    assert _fake_cache(lib, D=96)[0] == api.SDVG_ERR_BAD_SHAPE
    assert _fake_cache(lib, k=0x10010)[0] == api.SDVG_ERR_MISALIGNED
    assert _fake_cache(lib, k=0)[0] == api.SDVG_ERR_INVALID_ARG
    st, h = _fake_cache(lib)
    assert st == api.SDVG_OK
    nb, sb = C.c_int64(), C.c_int64()
    arr = (C.c_int64 * 3)()
    assert lib.sdvg_cache_state(h, C.byref(nb), arr, C.byref(sb)) == 0
    assert nb.value == 0 and list(arr) == [-1, -1, -1] and sb.value == -1
    # commits out of order / with bad flags are refused on the host before anything is launched
    assert lib.sdvg_kv_commit(h, 0x30000, 0x40000, 1, api.SDVG_FINAL, None, None) == api.SDVG_ERR_BAD_STATE
    assert lib.sdvg_kv_commit(h, 0x30000, 0x40000, 0, 3, None, None) == api.SDVG_ERR_INVALID_ARG
    assert lib.sdvg_kv_commit(h, 0x30008, 0x40000, 0, api.SDVG_FINAL, None, None) == api.SDVG_ERR_MISALIGNED
    assert lib.sdvg_kv_commit(h, None, 0x40000, 0, api.SDVG_FINAL, None, None) == api.SDVG_ERR_INVALID_ARG
    # attention: wrong block, unstaged self, tiny workspace
    ws = api.lib().sdvg_block_attn_workspace_bytes()
    assert ws >= 8
    f = lib.sdvg_block_attn_fwd
    assert f(0x50000, None, None, h, 0, 0x60000, None, 0.125, 0x70000, ws, None) == api.SDVG_ERR_BAD_STATE
    assert f(0x50000, 0x30000, 0x40000, h, 2, 0x60000, None, 0.125, 0x70000, ws, None) == api.SDVG_ERR_BAD_STATE
    assert f(0x50000, 0x30000, 0x40000, h, 0, 0x60000, None, 0.125, 0x70000, 4, None) == api.SDVG_ERR_INVALID_ARG
    assert f(0x50000, 0x30000, None, h, 0, 0x60000, None, 0.125, 0x70000, ws, None) == api.SDVG_ERR_INVALID_ARG
    assert f(0x50004, 0x30000, 0x40000, h, 0, 0x60000, None, 0.125, 0x70000, ws, None) == api.SDVG_ERR_MISALIGNED
    assert f(0x50000, 0x30000, 0x40000, h, 0, 0x60000, None, -1.0, 0x70000, ws, None) == api.SDVG_ERR_INVALID_ARG
    assert lib.sdvg_cache_destroy(h) == 0
    assert lib.sdvg_cache_destroy(None) == api.SDVG_ERR_INVALID_ARG


def test_rope_and_route_argument_checks(lib):
    r = lib.sdvg_rope3d_qk
    tab = 0x80000
    assert r(0x1000, 0x2000, 0x1000, 0x2000, 64, 2, 64, 2, 4, 8, 0, tab, 4, None) != api.SDVG_ERR_BAD_SHAPE
    assert r(0x1000, 0x2000, 0x1000, 0x2000, 63, 2, 64, 2, 4, 8, 0, tab, 4, None) == api.SDVG_ERR_BAD_SHAPE
    assert r(0x1000, 0x2000, 0x1000, 0x2000, 64, 2, 96, 2, 4, 8, 0, tab, 4, None) == api.SDVG_ERR_BAD_SHAPE
    assert r(0x1000, 0x2000, 0x1000, 0x2000, 64, 2, 64, 2, 4, 8, 3, tab, 4, None) == api.SDVG_ERR_BAD_STATE
    assert r(0x1000, 0x2000, 0x1000, 0x2000, 64, 2, 64, 2, 4, 8, -1, tab, 4, None) == api.SDVG_ERR_BAD_STATE
    assert r(0x1008, 0x2000, 0x1000, 0x2000, 64, 2, 64, 2, 4, 8, 0, tab, 4, None) == api.SDVG_ERR_MISALIGNED
    assert r(0x1000, 0x2000, None, 0x2000, 64, 2, 64, 2, 4, 8, 0, tab, 4, None) == api.SDVG_ERR_INVALID_ARG
    assert r(None, None, None, None, 64, 2, 64, 2, 4, 8, 0, tab, 4, None) == api.SDVG_ERR_INVALID_ARG
    assert r(0x1000, 0x2000, 0x1000, 0x2000, 64, 2, 64, 2, 4, 8, 0, None, 4, None) == api.SDVG_ERR_INVALID_ARG
    t = lib.sdvg_route
    assert t(0x1000, None, -1, 12, 0, -0.7, 0x2000, 0x3000, None, None) == api.SDVG_ERR_BAD_SHAPE
    assert t(0x1000, None, 4, 0, 0, -0.7, 0x2000, 0x3000, None, None) == api.SDVG_ERR_BAD_SHAPE
    assert t(0x1000, None, 0, 12, 0, -0.7, 0x2000, 0x3000, None, None) == api.SDVG_OK      # nothing to do
    assert t(None, None, 4, 12, 0, -0.7, 0x2000, 0x3000, None, None) == api.SDVG_ERR_INVALID_ARG
    assert t(0x1002, None, 4, 12, 0, -0.7, 0x2000, 0x3000, None, None) == api.SDVG_ERR_MISALIGNED


def test_e4m3_entry_points_validate_on_the_host(lib):
    assert lib.sdvg_cache_bytes_e4m3(7, 40, 4680, 128) == 7 * 40 * 4680 * 128
    assert lib.sdvg_cache_bytes_e4m3(7, 40, 4680, 64) == 0
    h8, h16 = C.c_void_p(), C.c_void_p()
    assert lib.sdvg_cache_create_e4m3(C.byref(h8), 0x10000, 0x20000, 3, 2, 64, 64) == api.SDVG_ERR_BAD_SHAPE
    assert lib.sdvg_cache_create_e4m3(C.byref(h8), 0x10010, 0x20000, 3, 2, 64, 128) == api.SDVG_ERR_MISALIGNED
    assert lib.sdvg_cache_create_e4m3(C.byref(h8), 0x10000, 0x20000, 3, 2, 64, 128) == api.SDVG_OK
    assert lib.sdvg_cache_create(C.byref(h16), 0x10000, 0x20000, 3, 2, 64, 128) == api.SDVG_OK
    sc = 0x90000
    commit8 = lib.sdvg_kv_commit_e4m3
    # the element types of ring and entry point must agree, either way round
    assert commit8(h16, 0x30000, 0x40000, sc, sc, 0, api.SDVG_FINAL, None, None) == api.SDVG_ERR_BAD_SHAPE
    assert lib.sdvg_kv_commit(h8, 0x30000, 0x40000, 0, api.SDVG_FINAL, None, None) == api.SDVG_ERR_BAD_SHAPE
    assert lib.sdvg_rope3d_qk_commit(h8, None, 0x30000, 0x40000, None, None, 1, 8, 8, 0, 0x80000, 4, 0, api.SDVG_FINAL,
                                     None, None) == api.SDVG_ERR_BAD_SHAPE
    assert commit8(h8, 0x30000, 0x40000, sc, sc, 1, api.SDVG_FINAL, None, None) == api.SDVG_ERR_BAD_STATE
    assert commit8(h8, 0x30000, 0x40000, sc, sc, 0, 3, None, None) == api.SDVG_ERR_INVALID_ARG
    assert commit8(h8, 0x30000, 0x40000, None, sc, 0, api.SDVG_FINAL, None, None) == api.SDVG_ERR_INVALID_ARG
    assert commit8(h8, 0x30008, 0x40000, sc, sc, 0, api.SDVG_FINAL, None, None) == api.SDVG_ERR_MISALIGNED
    assert commit8(h8, 0x30000, 0x40000, sc + 2, sc, 0, api.SDVG_FINAL, None, None) == api.SDVG_ERR_MISALIGNED
    fused8 = lib.sdvg_rope3d_qk_commit_e4m3
    tab = 0x80000
    assert fused8(h16, None, 0x30000, 0x40000, None, None, sc, sc, 1, 8, 8, 0, tab, 4, 0, api.SDVG_STAGE, None, None) == api.SDVG_ERR_BAD_SHAPE
    assert fused8(h8, 0x50000, 0x30000, 0x40000, None, sc, sc, sc, 1, 8, 8, 0, tab, 4, 0, api.SDVG_STAGE, None, None) == api.SDVG_ERR_INVALID_ARG
    assert fused8(h8, 0x50000, 0x30000, 0x40000, 0x60000, None, sc, sc, 1, 8, 8, 0, tab, 4, 0, api.SDVG_STAGE, None, None) == api.SDVG_ERR_INVALID_ARG
    assert fused8(h8, None, 0x30000, 0x40000, None, None, sc, sc, 1, 8, 7, 0, tab, 4, 0, api.SDVG_STAGE, None, None) == api.SDVG_ERR_BAD_SHAPE
    assert fused8(h8, None, 0x30000, 0x40000, None, None, sc, sc, 1, 8, 8, 4, tab, 4, 0, api.SDVG_STAGE, None, None) == api.SDVG_ERR_BAD_STATE
    assert fused8(h8, None, 0x30000, 0x40000, None, None, sc, sc, 1, 8, 8, 0, tab, 4, 2, api.SDVG_STAGE, None, None) == api.SDVG_ERR_BAD_STATE
    assert fused8(h8, None, 0x30008, 0x40000, None, None, sc, sc, 1, 8, 8, 0, tab, 4, 0, api.SDVG_STAGE, None, None) == api.SDVG_ERR_MISALIGNED
    ws = lib.sdvg_block_attn_workspace_bytes()
    f8, f16 = lib.sdvg_block_attn_fwd_e4m3, lib.sdvg_block_attn_fwd
    assert f8(0x50000, 0x30000, 0x40000, h16, 0, sc, sc, 0x60000, None, 0.125, 0x70000, ws, None) == api.SDVG_ERR_BAD_SHAPE
    assert f16(0x50000, 0x30000, 0x40000, h8, 0, 0x60000, None, 0.125, 0x70000, ws, None) == api.SDVG_ERR_BAD_SHAPE
    assert f8(0x50000, None, None, h8, 0, sc, sc, 0x60000, None, 0.125, 0x70000, ws, None) == api.SDVG_ERR_BAD_STATE
    assert f8(0x50000, 0x30000, 0x40000, h8, 1, sc, sc, 0x60000, None, 0.125, 0x70000, ws, None) == api.SDVG_ERR_BAD_STATE
    assert f8(0x50000, 0x30000, 0x40000, h8, 0, None, sc, 0x60000, None, 0.125, 0x70000, ws, None) == api.SDVG_ERR_INVALID_ARG
    assert f8(0x50000, 0x30000, 0x40000, h8, 0, sc, sc + 1, 0x60000, None, 0.125, 0x70000, ws, None) == api.SDVG_ERR_MISALIGNED
    assert f8(0x50000, 0x30000, 0x40000, h8, 0, sc, sc, 0x60000, None, 0.125, 0x70000, 4, None) == api.SDVG_ERR_INVALID_ARG
    q = lib.sdvg_quant_e4m3
    assert q(0x1000, sc, 0x2000, 16, 2, 96, None) == api.SDVG_ERR_BAD_SHAPE
    assert q(0x1000, sc, 0x2000, 0, 2, 128, None) == api.SDVG_ERR_BAD_SHAPE
    assert q(0x1000, None, 0x2000, 16, 2, 128, None) == api.SDVG_ERR_INVALID_ARG
    assert q(0x1008, sc, 0x2000, 16, 2, 128, None) == api.SDVG_ERR_MISALIGNED
    # ---- tile scales: one power-of-two scale per tile of 128 tokens and head
    assert lib.sdvg_cache_tile_scale_floats(7, 40, 4680) == 7 * 40 * 37
    assert lib.sdvg_cache_tile_scale_floats(7, 40, 128) == 7 * 40 and lib.sdvg_cache_tile_scale_floats(7, 40, 129) == 7 * 40 * 2
    assert lib.sdvg_cache_tile_scale_floats(0, 40, 4680) == 0
    commit_t, fused_t, attn_t = lib.sdvg_kv_commit_e4m3_tiled, lib.sdvg_rope3d_qk_commit_e4m3_tiled, lib.sdvg_block_attn_fwd_e4m3_tiled
    # no scale arrays attached yet
    assert commit_t(h8, 0x30000, 0x40000, 0, api.SDVG_FINAL, None, None) == api.SDVG_ERR_BAD_STATE
    assert attn_t(0x50000, sc, h8, 0, 0x60000, None, 0.125, 0x70000, ws, None) == api.SDVG_ERR_BAD_STATE
    assert lib.sdvg_cache_set_tile_scales(h16, sc, sc) == api.SDVG_ERR_BAD_SHAPE
    assert lib.sdvg_cache_set_tile_scales(h8, sc, None) == api.SDVG_ERR_INVALID_ARG
    assert lib.sdvg_cache_set_tile_scales(h8, sc + 2, sc) == api.SDVG_ERR_MISALIGNED
    assert lib.sdvg_cache_set_tile_scales(h8, sc, sc + 0x1000) == api.SDVG_OK
    assert commit_t(h16, 0x30000, 0x40000, 0, api.SDVG_FINAL, None, None) == api.SDVG_ERR_BAD_SHAPE
    assert commit_t(h8, 0x30000, 0x40000, 1, api.SDVG_FINAL, None, None) == api.SDVG_ERR_BAD_STATE
    assert commit_t(h8, 0x30000, None, 0, api.SDVG_FINAL, None, None) == api.SDVG_ERR_INVALID_ARG
    assert commit_t(h8, 0x30008, 0x40000, 0, api.SDVG_FINAL, None, None) == api.SDVG_ERR_MISALIGNED
    assert fused_t(h8, 0x50000, 0x30000, 0x40000, 0x60000, None, 1, 8, 8, 0, tab, 4, 0, api.SDVG_STAGE, None, None) == api.SDVG_ERR_INVALID_ARG
    assert fused_t(h8, 0x50000, 0x30000, 0x40000, None, sc, 1, 8, 8, 0, tab, 4, 0, api.SDVG_STAGE, None, None) == api.SDVG_ERR_INVALID_ARG
    assert fused_t(h8, None, 0x30000, 0x40000, None, None, 1, 8, 7, 0, tab, 4, 0, api.SDVG_STAGE, None, None) == api.SDVG_ERR_BAD_SHAPE
    assert fused_t(h8, None, 0x30000, 0x40000, None, None, 1, 8, 8, 0, tab, 4, 2, api.SDVG_STAGE, None, None) == api.SDVG_ERR_BAD_STATE
    assert fused_t(h16, None, 0x30000, 0x40000, None, None, 1, 8, 8, 0, tab, 4, 0, api.SDVG_STAGE, None, None) == api.SDVG_ERR_BAD_SHAPE
    assert attn_t(0x50000, sc, h8, 0, 0x60000, None, 0.125, 0x70000, ws, None) == api.SDVG_ERR_BAD_STATE     # block 0 not staged
    assert attn_t(0x50000, None, h8, 0, 0x60000, None, 0.125, 0x70000, ws, None) == api.SDVG_ERR_INVALID_ARG
    assert attn_t(0x50000, sc, h16, 0, 0x60000, None, 0.125, 0x70000, ws, None) == api.SDVG_ERR_BAD_SHAPE
    assert attn_t(0x50000, sc, h8, 0, 0x60000, None, 0.125, 0x70010, ws, None) == api.SDVG_ERR_MISALIGNED
    assert attn_t(0x50000, sc, h8, 0, 0x60000, None, -1.0, 0x70000, ws, None) == api.SDVG_ERR_INVALID_ARG
    qt = lib.sdvg_quant_e4m3_tiled
    assert qt(0x1000, 0x2000, sc, 16, 2, 64, None) == api.SDVG_ERR_BAD_SHAPE
    assert qt(0x1000, 0x2000, None, 16, 2, 128, None) == api.SDVG_ERR_INVALID_ARG
    assert qt(0x1000, 0x2008, sc, 16, 2, 128, None) == api.SDVG_ERR_MISALIGNED
    PP = C.c_void_p * 2
    two = PP(0x30000, 0x40000)
    steps_t = lib.sdvg_block_steps_e4m3_tiled
    assert steps_t(2, h8, two, two, two, two, None, two, 1, 8, 8, 0, tab, 4, 0, 0.125, 0x70000, ws, None) == api.SDVG_ERR_INVALID_ARG
    assert steps_t(0, h8, two, two, two, two, two, two, 1, 8, 8, 0, tab, 4, 0, 0.125, 0x70000, ws, None) == api.SDVG_ERR_BAD_SHAPE
    assert steps_t(2, h16, two, two, two, two, two, two, 1, 8, 8, 0, tab, 4, 0, 0.125, 0x70000, ws, None) == api.SDVG_ERR_BAD_SHAPE
    assert steps_t(2, h8, two, two, two, two, two, two, 1, 8, 8, 0, tab, 4, 1, 0.125, 0x70000, ws, None) == api.SDVG_ERR_BAD_STATE
    assert lib.sdvg_cache_destroy(h8) == 0 and lib.sdvg_cache_destroy(h16) == 0
