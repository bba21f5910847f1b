"""Host logic and C-ABI surface (no GPU): the library loads, exports every symbol
the header declares, builds plans on the CPU, and rejects bad arguments."""
import ctypes
import os
import re
import numpy as np
import pytest

import paper_2512_18453_b200 as nv
from oracle import toom_cook as tc
from synth import POINT_SETS, point_set

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "nova.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(nova_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = nv.lib()
    declared = _declared_symbols()
    assert len(declared) >= 15
    for name in declared:
        assert hasattr(L, name), name
    assert set(nv.EXPORTED_SYMBOLS) <= set(declared)


@pytest.mark.parametrize("kind,m", sorted(POINT_SETS))
def test_plan_matrices_match_oracle_bit_for_bit(kind, m):
    pts = point_set(kind, m)
    plan = nv.Plan(m, pts)
    AT, G, BT = plan.matrices()
    oAT, oG, oBT = (tc.to_float(M) for M in tc.build_matrices(m, 3, pts))
    assert np.array_equal(AT, oAT) and np.array_equal(G, oG) and np.array_equal(BT, oBT)
    assert abs(plan.kappa() / tc.kappa2_V(pts) - 1) < 1e-9
    a16, g16, b16 = plan.device_tables()
    with np.errstate(over="ignore"):
        assert np.array_equal(a16, oAT.astype(np.float16).astype(np.float32))
        assert np.array_equal(g16, oG.astype(np.float16).astype(np.float32))
        assert np.array_equal(b16, oBT.astype(np.float16).astype(np.float32))
    a32, g32, b32 = nv.Plan(m, pts, nv.FP16_F32ACC, nv.COEF_FP32).device_tables()
    assert np.array_equal(b32, oBT.astype(np.float32))
    a32, _, _ = nv.Plan(m, pts, nv.FP32).device_tables()
    assert np.array_equal(a32, oAT.astype(np.float32))


def test_plan_accepts_unordered_and_asymmetric_points():
    pts = [(3, 7), (-2, 1), (0, 1), (5, 4), (-1, 3), (1, 0)]
    plan = nv.Plan(4, pts)
    AT, G, BT = plan.matrices()
    oAT, oG, oBT = (tc.to_float(M) for M in tc.build_matrices(4, 3, pts))
    assert np.array_equal(AT, oAT) and np.array_equal(G, oG) and np.array_equal(BT, oBT)


@pytest.mark.parametrize("pts,m,code", [
    ([(0, 1), (1, 1), (1, 1), (1, 0)], 2, -4),
    ([(0, 1), (2, 2), (1, 1), (1, 0)], 2, -4),            # 2/2 == 1/1
    ([(0, 1), (1, 1), (-1, 1), (2, 1)], 2, -2),
    ([(0, 1), (1, 0), (-1, 1), (1, 0)], 2, -3),
    ([(1, 0), (0, 1), (-1, 1), (1, 1)], 2, -3),           # infinity not last
    ([(0, 1), (1, 1), (-1, 1), (1, 0)], 4, -1),           # n != m + r - 1
    ([(0, 1), (1, 1), (-1, 1), (1, 0)], 3, -1),           # m not supported
    ([(0, 1), (1, -1), (-1, 1), (1, 0)], 2, -1),          # negative denominator
])
def test_plan_rejects_bad_point_sets(pts, m, code):
    with pytest.raises(nv.NovaError) as e:
        nv.Plan(m, pts)
    assert e.value.status == code


def test_plan_reports_rational_overflow_and_unsupported_r():
    big = 2 ** 62
    pts = [(big - 1, big - 3), (big - 5, big - 7), (big - 9, big - 11), (big - 15, big - 13),
           (big - 21, big - 17), (big - 25, big - 27), (big - 33, big - 31), (big - 35, big - 37),
           (big - 41, big - 39), (1, 0)]
    with pytest.raises(nv.NovaError) as e:
        nv.Plan(8, pts)
    assert e.value.status == -5
    with pytest.raises(nv.NovaError) as e:
        nv.Plan(4, point_set("std", 6), r=5)
    assert e.value.status == -7


def test_size_queries_and_argument_checks_without_a_device():
    plan = nv.Plan(6, point_set("nova", 6))
    assert plan.filter_transform_bytes(256, 256) == 64 * 256 * 256 * 2
    assert nv.Plan(6, point_set("nova", 6), nv.FP32).filter_transform_bytes(8, 8) == 64 * 8 * 8 * 4
    ws = plan.workspace_bytes(32, 56, 56, 256, 256)
    mn = plan.min_workspace_bytes(32, 56, 56, 256, 256)
    assert 0 < mn <= ws
    assert plan.workspace_bytes(1, 8, 8, 12, 8) == 0              # C % 8 != 0
    assert plan.launch_count(32, 56, 56, 256, 256, ws) % 3 == 0
    assert plan.launch_count(32, 56, 56, 256, 256, 1024) == -10
    L = nv.lib()
    assert L.nova_conv2d_fwd(plan._h, None, None, None, 1, 8, 8, 8, 8, None, 0, 0, None) == -1
    assert L.nova_filter_transform(plan._h, None, 8, 8, None, None) == -1
    assert L.nova_maxpool2x2(None, None, 1, 8, 8, 8, 1, None) == -1
    assert nv.status_string(-9) == "a bounded device-side wait expired"
