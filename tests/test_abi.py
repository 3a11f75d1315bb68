"""CPU-side checks of the C ABI: the library loads, exports what the header
declares, validates arguments, and its plan matches the oracle bit for bit."""

import os
import re

import pytest

from oracle import prm_oracle as O
from paper_2608_20818_b200 import binding as B
from paper_2608_20818_b200 import build as build_mod
from paper_2608_20818_b200.workloads import workload

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()


def test_exports_match_header():
    hdr = open(os.path.join(ROOT, "include", "prm.h")).read()
    declared = set(re.findall(r"PRM_API\s+[\w\s\*]+?\b(prm_\w+)\s*\(", hdr))
    assert declared == set(B.EXPORTS)
    L = B.lib()
    for name in declared:
        assert hasattr(L, name), name


def test_option_constants_match_header():
    hdr = open(os.path.join(ROOT, "include", "prm.h")).read()
    for name, val in re.findall(r"#define\s+(PRM_(?:OPT|ERR)_\w+|PRM_OK)\s+(-?\d+)", hdr):
        assert getattr(B, name) == int(val), name


@pytest.mark.parametrize("cfg_id", [1, 2, 3, 4, 5])
def test_plan_matches_oracle(cfg_id):
    wl = workload(cfg_id)
    h = B.prm_create(wl.shapes, wl.K, wl.beta, wl.nesterov, wl.lr, wl.wd)
    g_ref, o_ref, gs = O.group_by_shape(wl.shapes)
    for t in range(0, 2 * wl.K + 1):
        refresh, n_groups, g, o = B.prm_plan(h, t, len(wl.shapes))
        assert refresh == O.is_refresh(t, wl.K)
        assert n_groups == len(gs) and g == g_ref and o == o_ref
    assert B.prm_workspace_bytes(h) > 0
    B.prm_destroy(h)


def test_plan_mixed_shapes_and_k1():
    shapes = [(2, 6), (2, 2), (8, 2), (2, 8), (2, 6), (8, 2), (2, 2)]
    h = B.prm_create(shapes, 1, 0.9, False, 1e-3, 0.0)
    refresh, n_groups, g, o = B.prm_plan(h, 7, len(shapes))
    assert refresh and n_groups == 4
    assert g == [0, 1, 2, 3, 0, 2, 1] and o == [0, 0, 0, 0, 1, 1, 1]
    B.prm_destroy(h)


def test_argument_errors():
    with pytest.raises(B.PrmError) as e:
        B.prm_create([(4, 4)], 0, 0.95, False, 1e-3, 0.0)
    assert e.value.code == B.PRM_ERR_ARG
    with pytest.raises(B.PrmError) as e:
        B.prm_create([(4, 0)], 2, 0.95, False, 1e-3, 0.0)
    assert e.value.code == B.PRM_ERR_SHAPE
    with pytest.raises(B.PrmError) as e:
        B.prm_create([], 2, 0.95, False, 1e-3, 0.0)
    assert e.value.code == B.PRM_ERR_ARG
    with pytest.raises(B.PrmError) as e:
        B.prm_create([(4, 4)], 2, 1.5, False, 1e-3, 0.0)
    assert e.value.code == B.PRM_ERR_ARG
    h = B.prm_create([(4, 4)], 2, 0.95, False, 1e-3, 0.0)
    with pytest.raises(B.PrmError) as e:
        B.prm_set_option(h, 999, 1.0)
    assert e.value.code == B.PRM_ERR_ARG
    with pytest.raises(B.PrmError) as e:
        B.prm_set_option(h, B.PRM_OPT_SCALE_MODE, 5)
    assert e.value.code == B.PRM_ERR_ARG
    # a step without a workspace is refused before any device work
    import ctypes
    arr = (ctypes.c_void_p * 1)(16)
    with pytest.raises(B.PrmError) as e:
        B.prm_step(h, arr, arr, arr, 0)
    assert e.value.code == B.PRM_ERR_WORKSPACE
    B.prm_destroy(h)


def test_workspace_scales_with_options():
    shapes = [(512, 1024)] * 4
    h = B.prm_create(shapes, 2, 0.95, False, 1e-3, 0.0)
    fast = B.prm_workspace_bytes(h)
    B.prm_set_option(h, B.PRM_OPT_CHECK_MODE, 1)
    check = B.prm_workspace_bytes(h)
    assert check > fast
    B.prm_set_option(h, B.PRM_OPT_NS_WORKSPACE_BYTES, 1)
    assert B.prm_workspace_bytes(h) < check
    B.prm_destroy(h)


def test_wide_kernel_option_values():
    h = B.prm_create([(8, 16)], 2, 0.95, False, 1e-3, 0.0)
    B.prm_set_option(h, B.PRM_OPT_WIDE_KERNEL, 1)
    B.prm_set_option(h, B.PRM_OPT_WIDE_KERNEL, 0)
    with pytest.raises(B.PrmError) as e:
        B.prm_set_option(h, B.PRM_OPT_WIDE_KERNEL, 2)
    assert e.value.code == B.PRM_ERR_ARG
    B.prm_destroy(h)


def test_split_input_option_changes_schedule_flop_and_workspace():
    """PRM_OPT_NS_SPLIT_INPUT: tensor-core groups from 1024 padded rows on take the Gram-space
    order, pay 4 r^2 c more flop and one more r x c matrix of workspace; smaller ones go to the
    fp32 path (printed recurrence)."""
    shapes = [(2048, 6144), (2048, 2048), (512, 1024), (32, 4096)]
    h = B.prm_create(shapes, 5, 0.95, True, 1e-3, 0.0)
    base = [B.prm_group_info(h, g) for g in range(4)]
    ws0 = B.prm_workspace_bytes(h)
    B.prm_set_option(h, B.PRM_OPT_NS_SPLIT_INPUT, 1)
    info = [B.prm_group_info(h, g) for g in range(4)]
    assert [g["gram_iters"] for g in base] == [3, 0, 0, 0]
    assert [g["gram_iters"] for g in info] == [3, 3, 0, 0]
    d = 2048.0
    assert info[0]["ns5_flop"] == base[0]["ns5_flop"] + 4 * d * d * 6144
    assert info[1]["ns5_flop"] == 9 * d ** 3 + 11 * d ** 3 + 4 * d ** 3       # Gram space, c = r: no shortcut for A_4
    assert info[2]["ns5_flop"] == base[2]["ns5_flop"] == 15 * 512.0 ** 2 * 1024 + 5 * 512.0 ** 3
    assert info[3]["ns5_flop"] == base[3]["ns5_flop"]
    assert B.prm_workspace_bytes(h) > ws0
    with pytest.raises(B.PrmError) as e:
        B.prm_set_option(h, B.PRM_OPT_NS_SPLIT_INPUT, 2)
    assert e.value.code == B.PRM_ERR_ARG
    B.prm_set_option(h, B.PRM_OPT_CHECK_MODE, 1)
    assert [B.prm_group_info(h, g)["gram_iters"] for g in range(4)] == [0] * 4
    B.prm_destroy(h)


def test_group_info_and_gram_span_option():
    shapes = [(2048, 6144), (2048, 2048), (8192, 2048), (2048, 6144), (256, 1024), (1024, 1280)]
    h = B.prm_create(shapes, 5, 0.95, True, 1e-3, 0.0)
    _, n_groups, group_of_mat, _ = B.prm_plan(h, 0, len(shapes))
    assert n_groups == 5 and group_of_mat == [0, 1, 2, 0, 3, 4]
    info = [B.prm_group_info(h, g) for g in range(n_groups)]
    assert [(g["rows"], g["cols"], g["count"]) for g in info] == [
        (2048, 6144, 2), (2048, 2048, 1), (8192, 2048, 1), (256, 1024, 1), (1024, 1280, 1)]
    # Gram-space iterations: >= 1024 oriented rows and c >= 1.5 r (padded to 256)
    assert [g["gram_iters"] for g in info] == [3, 0, 3, 0, 0]
    d = 2048.0
    assert [g["ns5_flop"] for g in info[:3]] == [8 * d * d * 6144 + 13 * d ** 3, 20 * d ** 3, 8 * d * d * 8192 + 13 * d ** 3]
    assert all(g["ns_batch"] == g["count"] for g in info)
    with_span = B.prm_workspace_bytes(h)
    B.prm_set_option(h, B.PRM_OPT_NS_GRAM_SPAN, 0)
    assert [B.prm_group_info(h, g)["gram_iters"] for g in range(n_groups)] == [0] * 5
    assert B.prm_workspace_bytes(h) < with_span
    B.prm_set_option(h, B.PRM_OPT_NS_GRAM_SPAN, 1)
    assert B.prm_group_info(h, 0)["ns5_flop"] == 9 * d * d * 6144 + 11 * d ** 3
    assert B.prm_workspace_bytes(h) == with_span
    B.prm_set_option(h, B.PRM_OPT_CHECK_MODE, 1)          # the check mode runs the printed recurrence
    assert [B.prm_group_info(h, g)["gram_iters"] for g in range(n_groups)] == [0] * 5
    with pytest.raises(B.PrmError) as e:
        B.prm_set_option(h, B.PRM_OPT_NS_GRAM_SPAN, 3)
    assert e.value.code == B.PRM_ERR_ARG
    with pytest.raises(B.PrmError) as e:
        B.prm_group_info(h, n_groups)
    assert e.value.code == B.PRM_ERR_ARG
    B.prm_destroy(h)
