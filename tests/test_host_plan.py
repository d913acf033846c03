"""Host-side launch planning of the three products (no GPU): tile width, split-K plan, tile order.

The choices are cost models fitted to measurements; these tests pin their structural properties (every tile is
visited exactly once under every band height; a plan never asks for what the shape or the workspace cannot give)
and the decisions on the benchmark's shapes that the measurements settled.
"""
import ctypes

import pytest

from paper_2409_09099_b200 import binding as B, build

FWD, DW, DX = 0, 1, 2


@pytest.fixture(scope="module")
def lib():
    build.build()
    return B.load()


@pytest.mark.parametrize("m_tiles,n_tiles", [(1, 1), (5, 7), (64, 16), (43, 16), (3, 12)])
@pytest.mark.parametrize("group_m", [1, 2, 3, 8, 1000])
def test_tile_order_is_a_bijection(lib, m_tiles, n_tiles, group_m):
    seen = set()
    mt, nt = ctypes.c_int(), ctypes.c_int()
    prev_band = 0
    for tile in range(m_tiles * n_tiles):
        assert lib.sste_debug_tile_coords(tile, m_tiles, n_tiles, group_m, ctypes.byref(mt), ctypes.byref(nt)) == B.OK
        assert 0 <= mt.value < m_tiles and 0 <= nt.value < n_tiles
        seen.add((mt.value, nt.value))
        band = mt.value // min(group_m, m_tiles)
        assert band >= prev_band                      # bands are visited one after the other
        prev_band = band
    assert len(seen) == m_tiles * n_tiles
    assert lib.sste_debug_tile_coords(m_tiles * n_tiles, m_tiles, n_tiles, group_m, ctypes.byref(mt), ctypes.byref(nt)) == B.ERR_INVALID_ARG


def test_column_major_order_when_the_band_is_everything(lib):
    mt, nt = ctypes.c_int(), ctypes.c_int()
    for tile in range(35):
        lib.sste_debug_tile_coords(tile, 5, 7, 5, ctypes.byref(mt), ctypes.byref(nt))
        assert (mt.value, nt.value) == (tile % 5, tile // 5)


def test_plans_on_the_benchmark_shapes():
    # GPT-2-small fc1 (3072 x 768, 8192 tokens), bf16
    assert B.plan(FWD, B.BF16, 3072, 768, 8192)[0] in (192, 224)          # short K: two accumulators
    bn, splits, split_from, gm = B.plan(DW, B.BF16, 3072, 768, 8192)
    assert (bn, splits, split_from) == (256, 2, 0)                         # 36 tiles on 74 pairs: all split in two
    # GPT-2-large proj grad_X: 320 tiles of a short reduction, the second pass would cost more than it saves
    assert B.plan(DX, B.BF16, 1280, 1280, 16384)[1] == 1
    # 7B-shaped FP8 up projection: 256-wide tiles, banded order for the products whose A operand exceeds L2
    bn, _, _, gm = B.plan(FWD, B.E4M3, 11008, 4096, 16384)
    assert bn == 256 and gm == 43                                          # compressed W fits L2: plain order
    assert 4 <= B.plan(DX, B.E5M2, 11008, 4096, 16384)[3] <= 16            # 64 tile rows of dY: bands
    assert 4 <= B.plan(DW, B.E5M2, 11008, 4096, 16384)[3] <= 16


@pytest.mark.parametrize("product", [FWD, DW, DX])
@pytest.mark.parametrize("O,I,T", [(128, 128, 128), (768, 3072, 8192), (5120, 1280, 16384), (4096, 11008, 16384)])
def test_plan_is_feasible(product, O, I, T):
    for dt in (B.BF16, B.E4M3 if product == FWD else B.E5M2):
        bn, splits, split_from, gm = B.plan(product, dt, O, I, T)
        M, N, K = (T if product == DX else O), (T if product == FWD else I), (I if product == FWD else T if product == DW else O)
        m_tiles, n_tiles = -(-M // 256), -(-N // bn)
        assert bn in (128, 192, 224, 256) and 1 <= splits <= 4 and 1 <= gm <= m_tiles
        if splits == 1:
            assert split_from == m_tiles * n_tiles                       # nothing is split
        else:
            assert 0 <= split_from < m_tiles * n_tiles and split_from % 74 == 0     # whole waves first
            elt = 2 if dt == B.BF16 else 1
            bk = (256 if product != DX else 128) // elt
            assert (K // bk) % splits == 0 and K // bk // splits >= 8
        # without room for partial tiles nothing is split
        assert B.plan(product, dt, O, I, T, workspace_bytes=B.load().sste_workspace_bytes())[1] == 1


def test_plan_rejects_bad_arguments(lib):
    assert lib.sste_debug_plan(3, B.BF16, 128, 128, 128, 148, ctypes.c_size_t(0), None, None, None, None) == B.ERR_INVALID_ARG
    assert lib.sste_debug_plan(0, B.F32, 128, 128, 128, 148, ctypes.c_size_t(0), None, None, None, None) == B.ERR_INVALID_ARG
    assert lib.sste_debug_plan(0, B.BF16, 100, 128, 128, 148, ctypes.c_size_t(0), None, None, None, None) == B.ERR_SHAPE
    assert lib.sste_debug_plan(0, B.BF16, 128, 128, 128, 148, ctypes.c_size_t(0), None, None, None, None) == B.OK


def test_per_device_attribute_guard(lib):
    """The launches set a kernel's shared-memory opt-in once per device ordinal (and retry after a failure)."""
    assert lib.sste_debug_selftest_device_once() == B.OK
