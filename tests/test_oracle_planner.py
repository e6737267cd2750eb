"""The oracle's sizing law and calibration plan against the integers the paper prints and
against plans worked out by hand from its formulas."""
import math
import os

import numpy as np
import pytest

import oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                out.append(line.split())
    return out


def test_table_rect_law_bucket_counts():
    for n1, n2, n3, mb, mf in _rows("tab_rect_law_m.txt"):
        n1, n2, n3 = int(n1), int(n2), int(n3)
        assert O.m_start(n1, n2, n3, O.BF16) == int(mb), (n1, n2, n3)
        assert O.m_start(n1, n2, n3, O.FP16) == int(mf), (n1, n2, n3)


def test_other_printed_law_points():
    fn = {"m_num": lambda a, b, c, d: O.m_num(a, b, c, d, O.Params()),
          "m_max": lambda a, b, c, d: O.m_max(a, c),
          "m_start": lambda a, b, c, d: O.m_start(a, b, c, d)}
    for key, n1, n2, n3, dt, val in _rows("law_points.txt"):
        assert fn[key](int(n1), int(n2), int(n3), int(dt)) == int(val), (key, n1, n2, n3)


def test_sketch_memory_of_65536_cube_is_25_8_GiB():
    # "would need 25.8 GB for S, R and T" at m = 48010
    assert 3 * 48010 ** 2 * 4 / 2 ** 30 == pytest.approx(25.8, abs=0.05)


def test_m_comb_and_caps():
    assert O.m_comb(O.Params()) == 48                       # 3*2*8
    assert O.m_comb(O.Params(s_budget=1, delta_max=1)) == 6
    assert O.m_comb(O.Params(s_budget=400, delta_max=1)) == math.ceil(math.sqrt(2400))
    assert O.m_max(1024, 1024) == 256 and O.m_max(16, 16) == 16 and O.m_max(256, 256) == 64
    # m_mem: largest m with 4(3m^2 + 6 m n2) <= 2^31, checked by direct evaluation
    for n2 in (256, 4096, 11008, 16384, 65536):
        m = O.m_mem(n2)
        assert 4 * (3 * m * m + 6 * m * n2) <= 2 ** 31 < 4 * (3 * (m + 1) ** 2 + 6 * (m + 1) * n2)


def test_plan_worked_by_hand_bf16_4096_cube():
    """4096^3 BF16 at m=48 with sigma from Eq. (sigma), rms=1, rho_min=0.02:
    sigma = 0.19 * 2^-24 * 4096^1.5 * 0.5^0.07 / 48; B = 4096 sigma / 0.02 ~ 12.06;
    r_B = ceil(2.5 B) = 31 > 4; m_loc = 16 ceil(ceil(48*31/4)/16) = 384;
    B' = B*48/384 ~ 1.51; r = ceil(2.5 B') = 4."""
    sigma = 0.19 * 2.0 ** -24 * 4096 ** 1.5 * 0.5 ** 0.07 / 48
    m_loc, r, B = O.plan(4096, 4096, 4096, O.BF16, sigma, 1.0, 48)
    assert B == pytest.approx(12.06, abs=0.01)
    assert (m_loc, r) == (384, 4)
    # a non-positive estimate falls back to the same law value
    assert O.plan(4096, 4096, 4096, O.BF16, float("nan"), 1.0, 48)[:2] == (384, 4)
    assert O.plan(4096, 4096, 4096, O.BF16, sigma, 0.0, 48)[:2] == (384, 4)


def test_plan_branches():
    p = O.Params()
    # B <= 0.05: radius 0, bucket count kept
    assert O.plan(256, 256, 256, O.FP16, 0.05 * 0.02 / 256, 1.0, 48)[:2] == (48, 0)
    # 0.05 < B, small: radius max(2, ceil(2.5 B)) <= r*: bucket count kept
    assert O.plan(256, 256, 256, O.FP16, 0.5 * 0.02 / 256, 1.0, 48)[:2] == (48, 2)
    assert O.plan(256, 256, 256, O.FP16, 1.5 * 0.02 / 256, 1.0, 48)[:2] == (48, 4)
    # growth stopped by the population cap m_max = 64: radius grows instead, up to r_max
    m_loc, r, B = O.plan(256, 256, 256, O.FP16, 20 * 0.02 / 256, 1.0, 48)
    assert m_loc == 64 and r == min(16, math.ceil(2.5 * 20 * 48 / 64))
    m_loc, r, B = O.plan(256, 256, 256, O.FP16, 4 * 0.02 / 256, 1.0, 48)
    assert (m_loc, r) == (64, math.ceil(2.5 * 4 * 48 / 64))
    # m_loc never shrinks below the current count
    assert O.plan(256, 256, 256, O.FP16, 4 * 0.02 / 256, 1.0, 100)[0] == 100


def test_recalibrated_probe_bucket_count():
    # m' = max(m_comb, 16, min(ceil(m B1 / B*), m_max)), B1 = max(n1,n3) sigma / rms
    assert O.recalibrated_m(4096, 4096, 0.3 / 4096, 1.0, 100) == 100       # B1 = B*: unchanged
    assert O.recalibrated_m(4096, 4096, 0.6 / 4096, 1.0, 100) == 200
    assert O.recalibrated_m(4096, 4096, 1e-9, 1.0, 100) == 48              # floor m_comb
    assert O.recalibrated_m(4096, 4096, 1.0, 1.0, 100) == 1024             # cap m_max


def test_rms_estimate_stride_clip():
    C = np.full((512, 512), 2.0, dtype=np.float32)
    assert O.rms_c_estimate(C) == 2.0
    # stride = 512*512 // 65536 = 4: only flat indices 0,4,8,.. are seen
    C2 = C.copy()
    C2.ravel()[1::4] = 1e30
    assert O.rms_c_estimate(C2) == 2.0
    # a sampled outlier is clipped at 64 x median; non-finite samples are dropped
    C3 = C.copy()
    C3.ravel()[0] = 1e30
    C3.ravel()[4] = np.inf
    C3.ravel()[8] = np.nan
    n = 65536 - 2
    assert O.rms_c_estimate(C3) == pytest.approx(math.sqrt(((n - 1) * 4.0 + 128.0 ** 2) / n), rel=1e-12)
    # fewer than 65536 entries: stride 1
    g = np.random.default_rng(0)
    x = g.standard_normal((100, 100)).astype(np.float32)
    assert O.rms_c_estimate(x) == pytest.approx(float(np.sqrt(np.mean(x.astype(np.float64) ** 2))), rel=1e-12)


def test_law_sigma_matches_normalized_range_of_the_paper():
    # normalized sigma = c_f (n2/8192)^0.07: the envelope sits above the measured 0.162..0.219
    for n2, lo in ((1024, 0.162), (65536, 0.219)):
        norm = O.law_sigma(512, n2, 512, O.BF16, 1.0, 1.0) / (2.0 ** -24 * math.sqrt(512.0 * 512 * n2))
        assert norm == pytest.approx(0.19 * (n2 / 8192) ** 0.07, rel=1e-12)
        assert norm >= lo
    assert O.c_f(O.FP16) / O.c_f(O.BF16) == pytest.approx(1.76)
