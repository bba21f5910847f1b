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
        nv.Plan(4, point_set("std", 6), r=4)
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


# ---------------------------------------------------------------- discovery helpers and rescaling
def test_snap_through_the_abi_equals_the_oracle():
    from fractions import Fraction
    rng = np.random.default_rng(11)
    xs = list(rng.uniform(-6, 6, size=300)) + [0.0, 0.25, 0.75, -0.75, 5.0, -5.0, 7.3, -100.0, 1e-12, 5 / 6, 7 / 6]
    for d_max in (1, 2, 6, 10, 20):
        for x in xs:
            want = tc.snap_to_rational(float(x), d_max)
            assert nv.snap_to_rational(x, d_max) == (want.numerator, want.denominator), (x, d_max)
    for bad in (0, 5000):
        with pytest.raises(nv.NovaError):
            nv.snap_to_rational(0.5, bad)
    with pytest.raises(nv.NovaError):
        nv.snap_to_rational(float("nan"), 10)


def test_plan_from_floats_recovers_the_discovered_sets():
    # continuous optima near the printed fractions snap onto them (Section "Snap-to-Rational")
    plan = nv.Plan.from_floats(4, [0.0004, 0.8329, -0.8338, 1.1671, -1.1660])
    want = nv.Plan(4, point_set("nova", 4))
    for a, b in zip(plan.matrices(), want.matrices()):
        assert np.array_equal(a, b)
    assert abs(plan.kappa() - 14.5) < 0.05
    with pytest.raises(nv.NovaError) as e:           # two points snapping to the same rational
        nv.Plan.from_floats(4, [0.0, 0.83, 0.834, 1.0, -1.0])
    assert e.value.status == -4


@pytest.mark.parametrize("kind,m", sorted(POINT_SETS))
def test_exact_matrices_and_per_matrix_conditioning_match_the_oracle(kind, m):
    pts = point_set(kind, m)
    plan = nv.Plan(m, pts)
    oAT, oG, oBT = tc.build_matrices(m, 3, pts)
    AT, G, BT = plan.matrices_rational()
    assert AT == oAT and G == oG and BT == oBT                    # exact, entry by entry
    kap, nrm = plan.kappa_matrices()
    for got, M in zip(kap, (oAT, oG, oBT)):
        assert abs(got / tc.kappa2(tc.to_float(M)) - 1) < 1e-9
    for got, M in zip(nrm, (oAT, oG, oBT)):
        assert abs(got / tc.norm2(tc.to_float(M)) - 1) < 1e-12


def test_verifier_accepts_valid_and_rejects_planted_mistakes():
    from fractions import Fraction
    AT, G, BT = tc.build_matrices(6, 3, point_set("nova", 6))
    assert nv.verify_decomposition(6, 3, AT, G, BT)
    bad = [row[:] for row in G]; bad[3][1] = -bad[3][1]
    assert not nv.verify_decomposition(6, 3, AT, bad, BT)
    bad = [row[:] for row in BT]; bad[2][4] += Fraction(1, 10 ** 9)
    assert not nv.verify_decomposition(6, 3, AT, G, bad)
    BTt = [[BT[j][i] for j in range(8)] for i in range(8)]         # transposed operand
    assert not nv.verify_decomposition(6, 3, AT, G, BTt)


def test_scaled_plan_matches_the_oracle_and_keeps_symmetry_only_for_paired_scales():
    # the even/odd fast path needs equal scales within a +- pair and unit columns of A^T at 0 and infinity
    from fractions import Fraction
    pts = point_set("nova", 6)
    sg = [Fraction(1, 4), Fraction(2), Fraction(2), Fraction(1, 4), Fraction(1, 4), Fraction(3), Fraction(3), Fraction(1, 2)]
    sb = [Fraction(4), Fraction(1, 2), Fraction(1, 2), Fraction(8), Fraction(8), Fraction(1), Fraction(1), Fraction(2)]
    plan = nv.Plan(6, pts, scale_G=sg, scale_B=sb)
    assert plan.matrices_rational() == tc.build_matrices(6, 3, pts, scale_G=sg, scale_B=sb)
    assert plan.frequency_order()[1] is True
    assert plan.kappa() == nv.Plan(6, pts).kappa()                 # rescaling does not touch kappa(V)
    sg[2] = Fraction(5)                                            # different scales within a +- pair
    plan = nv.Plan(6, pts, scale_G=sg, scale_B=sb)
    assert plan.matrices_rational() == tc.build_matrices(6, 3, pts, scale_G=sg, scale_B=sb)
    assert plan.frequency_order()[1] is False
    with pytest.raises(nv.NovaError):
        nv.Plan(6, pts, scale_G=[0] * 8)


# ---------------------------------------------------------------- plans for 5 x 5 filters
@pytest.mark.parametrize("m,key", [(2, ("std", 4)), (4, ("std", 6)), (4, ("nova", 6)), (6, ("std", 8)), (6, ("nova", 8))])
def test_r5_plans_are_exact(m, key):
    pts = point_set(*key)
    plan = nv.Plan(m, pts, r=5)
    assert plan.matrices_rational() == tc.build_matrices(m, 5, pts)
    AT, G, BT = plan.matrices()
    assert AT.shape == (m, m + 4) and G.shape == (m + 4, 5) and BT.shape == (m + 4, m + 4)
    oAT, oG, oBT = (tc.to_float(M) for M in tc.build_matrices(m, 5, pts))
    assert np.array_equal(AT, oAT) and np.array_equal(G, oG) and np.array_equal(BT, oBT)
    assert abs(plan.kappa() / tc.kappa2_V(pts) - 1) < 1e-9
    kap, _ = plan.kappa_matrices()
    for got, M in zip(kap, tc.build_matrices(m, 5, pts)):
        assert abs(got / tc.kappa2(tc.to_float(M)) - 1) < 1e-8
    # sizes follow n = m + 4
    assert plan.filter_transform_bytes(64, 64) == (m + 4) ** 2 * 64 * 64 * 2
    assert plan.workspace_bytes(1, 16, 16, 64, 64) > 0
    assert plan.int8_workspace_bytes(1, 16, 16, 64, 64) > 0
    assert plan.frequency_order() == (list(range(m + 4)), True)       # symmetric set already in internal order
    a16, g16, b16 = plan.device_tables()
    with np.errstate(over="ignore"):
        assert np.array_equal(g16, oG.astype(np.float16).astype(np.float32)) and g16.shape == (m + 4, 5)


def test_r5_rejects_what_it_cannot_build():
    with pytest.raises(nv.NovaError) as e:
        nv.Plan(8, point_set("std", 8) + [(5, 1), (-5, 1)], r=5)          # F(8,5) needs 12 points
    assert e.value.status in (-7, -3)
    with pytest.raises(nv.NovaError) as e:
        nv.Plan(4, point_set("std", 6), r=4)
    assert e.value.status == -7


def test_symmetric_search_through_the_abi_finds_the_discovered_sets():
    for m in (4, 6, 8):
        pts, k = nv.symmetric_search(m + 1, 6, 2)
        assert pts == point_set("nova", m)                       # Table 3, infinity last
        assert abs(k / tc.kappa2_V(point_set("nova", m)) - 1) < 1e-9
        plan = nv.Plan(m, pts)                                   # and the set builds a verified plan
        assert abs(plan.kappa() / k - 1) < 1e-9
    for n_finite, d in ((3, 6), (4, 5), (5, 8)):                 # same answer as the oracle's enumeration
        pts, k = nv.symmetric_search(n_finite, d, 2)
        opts, ok = tc.symmetric_search(n_finite, d)
        assert [(p.numerator, p.denominator) for p in opts] == pts[:-1] and abs(k / ok - 1) < 1e-9
    with pytest.raises(nv.NovaError) as e:                       # too many combinations to enumerate
        nv.symmetric_search(9, 30, 5)
    assert e.value.status == -7


def test_binding_constants_agree_with_the_header():
    # the flag, mode and error values of the binding are those include/nova.h declares (parsed from the
    # header's enums; catches a constant changed on one side only)
    text = open(os.path.join(os.path.dirname(__file__), "..", "include", "nova.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)

    def header_value(name):
        m = re.search(r"\b%s\s*=\s*([^,}\n]+)" % name, text)
        assert m, name
        return int(eval(m.group(1).strip(), {"__builtins__": {}}, {}))
    pairs = {"NOVA_RELU": nv.RELU, "NOVA_GEMM_SIMT": nv.GEMM_SIMT, "NOVA_GEMM_TCGEN05": nv.GEMM_TCGEN05,
             "NOVA_TRANSFORM_SIMT": nv.TRANSFORM_SIMT, "NOVA_PROFILE_WAITS": nv.PROFILE_WAITS,
             "NOVA_POOL2X2": nv.POOL2X2, "NOVA_FP32": nv.FP32, "NOVA_FP16_F32ACC": nv.FP16_F32ACC,
             "NOVA_COEF_ROUND_TO_MODE": nv.COEF_ROUND_TO_MODE, "NOVA_COEF_FP32": nv.COEF_FP32}
    for name, value in pairs.items():
        assert header_value(name) == value, name
    flags = [nv.RELU, nv.GEMM_SIMT, nv.GEMM_TCGEN05, nv.TRANSFORM_SIMT, nv.PROFILE_WAITS, nv.POOL2X2]
    assert len(set(flags)) == len(flags) and all(a & b == 0 for i, a in enumerate(flags) for b in flags[i + 1:])
    m = re.search(r"#define\s+NOVA_STATIC_SCRATCH_BYTES\s+\(\(size_t\)(\d+)\s*<<\s*(\d+)\)", text)
    assert m and (int(m.group(1)) << int(m.group(2))) == nv.STATIC_SCRATCH_BYTES
