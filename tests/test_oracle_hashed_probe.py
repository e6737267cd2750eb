"""Pins of the oracle's S only probe (Section "The Cheap S Only Probe", Eq. (S), Section "Thresholds").

The sketch is pinned by brute force on tiny inputs, by the exact image of a single fault on an
integer product, by the factored form (H1 A)(B H2^T) - H1 C H2^T, and by the one-bucket special
case; the rule by its closed form on a constructed sketch.
"""
import math

import numpy as np
import pytest

import oracle as o
from paper_2609_19758_b200 import workloads as wl


def _np(x):
    return x.double().numpy() if hasattr(x, "double") else np.asarray(x, dtype=np.float64)


def _ops(kind, n1, n2, n3, dtype, seed):
    A, B = wl.operands(kind, n1, n2, n3, dtype, seed)
    return _np(A), _np(B), wl.cpu_fp32_product(A, B).double().numpy()


def test_hashed_sum_sketch_brute_force():
    rng = np.random.default_rng(3)
    n1, n3, m = 13, 11, 4
    E = rng.standard_normal((n1, n3))
    h1, v1 = o.hash_round(99, 2, 0, n1, m)
    h2, v2 = o.hash_round(99, 2, 1, n3, m)
    S = o.hashed_sum_sketch(E, h1, v1, h2, v2, m)
    ref = [[0.0] * m for _ in range(m)]
    for i in range(n1):
        for j in range(n3):
            ref[int(h1[i])][int(h2[j])] += int(v1[i]) * int(v2[j]) * E[i, j]
    assert np.allclose(S, np.array(ref), rtol=0, atol=1e-13)
    # bucket sums partition the entries: the signed total is v1^T E v2
    assert abs(S.sum() - np.asarray(v1, float) @ E @ np.asarray(v2, float)) < 1e-12


def test_single_fault_lands_in_one_bucket_exactly():
    A, B, C = _ops("integer", 96, 64, 80, o.FP16, 5)
    res, S = o.probe_hashed(A, B, C, 11, 7, 8)
    assert not res.fired and np.all(S == 0.0)          # exact integer product: E = 0
    i, j, d = 37, 51, 3.0
    C2 = C.copy()
    C2[i, j] += d
    res2, S2 = o.probe_hashed(A, B, C2, 11, 7, 8)
    h1, v1 = o.hash_round(11, 7, 0, 96, 8)
    h2, v2 = o.hash_round(11, 7, 1, 80, 8)
    a, b = int(h1[i]), int(h2[j])
    expect = np.zeros((8, 8))
    expect[a, b] = -d * int(v1[i]) * int(v2[j])         # E = AB - C = -d at (i, j)
    assert np.array_equal(S2, expect)
    assert res2.fired and res2.argmax_col == a * 8 + b and res2.max_abs == d


def test_factored_form_matches_definition():
    A, B, C = _ops("gauss_scaled", 70, 48, 90, o.BF16, 8)
    m = 6
    _, S = o.probe_hashed(A, B, C, 5, 0, m)
    h1, v1 = o.hash_round(5, 0, 0, 70, m)
    h2, v2 = o.hash_round(5, 0, 1, 90, m)
    S2, _, _ = o.moment_sketches_compressed(A, B, C, h1, v1, h2, v2, m)
    scale = np.abs(_np(A)).sum() * np.abs(_np(B)).max()
    assert np.max(np.abs(S - S2)) <= 1e-13 * scale


def test_one_bucket_is_the_signed_total():
    A, B, C = _ops("uniform", 33, 20, 27, o.FP16, 2)
    C = C + 0.25
    res, S = o.probe_hashed(A, B, C, 4, 1, 1)
    _, v1 = o.hash_round(4, 1, 0, 33, 1)
    _, v2 = o.hash_round(4, 1, 1, 27, 1)
    E = _np(A) @ _np(B) - C
    assert S.shape == (1, 1)
    assert abs(S[0, 0] - np.asarray(v1, float) @ E @ np.asarray(v2, float)) < 1e-10


def test_rule_closed_form_and_population_cap():
    # constant-magnitude sketch: mean|S| = c, nothing clipped, sigma_hat = 1.2533 c
    m, c = 8, 2.0
    s = np.full(m * m, c)
    s[::2] *= -1.0
    tau = 1e9
    r = o.probe_verdict(s, tau, o.Params(), n_rows=4.0)
    assert math.isclose(r.sigma_hat, 1.2533 * c, rel_tol=1e-12)
    assert math.isclose(r.thr, 4.0 * math.sqrt(2.0 * math.log(m * m)) * 1.2533 * c, rel_tol=1e-12)
    assert not r.fired
    # the cap binds: thr = tau sqrt(population)
    r2 = o.probe_verdict(s, 0.5, o.Params(), n_rows=4.0)
    assert math.isclose(r2.thr, 1.0, rel_tol=1e-12) and r2.fired


def test_printed_rule_is_the_default_and_the_population_cap_is_opt_in():
    # Section "Thresholds": thr = min(tau, mu sqrt(2 ln m^2) sigma_hat).  A tiny inner dimension with large
    # entries of C makes the cap bind, so the two forms of the cap can be told apart.
    A, B, C = _ops("uniform", 64, 32, 48, o.FP16, 9)
    C = C + 3.0 * np.sign(np.random.default_rng(3).standard_normal(C.shape))       # noise far above tau
    tau = o.analytic_tau(_np(A), _np(B), 32)
    res, S = o.probe_hashed(A, B, C, 1, 0, 4)
    sig = 1.2533 * np.minimum(np.abs(S), 5.0 * np.abs(S).mean()).mean()
    assert 4.0 * math.sqrt(2.0 * math.log(16)) * sig > 10.0 * tau               # the noise term is not the minimum
    assert math.isclose(res.tau, tau, rel_tol=1e-12)
    assert math.isclose(res.thr, tau, rel_tol=1e-12) and res.fired
    res1, _ = o.probe_hashed(A, B, C, 1, 0, 4, o.Params(scale_cap=1))
    assert math.isclose(res1.thr, min(tau * math.sqrt(64 * 48 / 16.0), 4.0 * math.sqrt(2.0 * math.log(16)) * sig),
                        rel_tol=1e-12)
    assert res1.thr > res.thr


@pytest.mark.parametrize("bad", [np.inf, -np.inf, np.nan])
def test_nonfinite_entry_fires(bad):
    A, B, C = _ops("gauss_scaled", 40, 24, 36, o.BF16, 6)
    C[7, 9] = bad
    res, S = o.probe_hashed(A, B, C, 2, 3, 4)
    assert res.nonfinite and res.fired
    assert np.count_nonzero(~np.isfinite(S)) == 1


def test_detects_fault_above_floor_and_stays_clean_below():
    A, B, C = _ops("gauss_scaled", 256, 128, 256, o.BF16, 12)
    res, _ = o.probe_hashed(A, B, C, 3, 0, 16)
    assert not res.fired
    C[100, 17] += 20.0 * res.thr
    res2, _ = o.probe_hashed(A, B, C, 3, 0, 16)
    assert res2.fired


# ---------------------------------------------------------------- stateful probe
def test_state_accumulates_clean_noise_and_ors_the_verdicts():
    st = o.ProbeState()
    clean = o.ProbeResult(False, False, 3, 0.1, 0.25, 1.0, 2.0)
    dirty = o.ProbeResult(True, False, 5, 9.0, 0.75, 1.0, 2.0)
    for r in (clean, clean, dirty, clean, dirty):
        st.accumulate(r)
    assert (st.calls, st.clean_calls, st.fired_any, st.first_fired_call) == (5, 3, 1, 3)
    assert st.sigma_sum == 0.75 and st.sigma_bar() == 0.25          # dirty calls do not enter the average
    assert math.isnan(o.ProbeState().sigma_bar())


def test_recalibration_cadence():
    due = [c for c in range(1, 3100) if o.recalibration_due(c)]
    assert due == [16, 1024, 2048, 3072]


def test_recalibration_band_and_formula():
    # B1 = max(n1, n3) sigma / rms; m' = max(m_comb, 16, min(ceil(m B1 / B*), m_max)); B* = 0.3, m_comb = 48
    n = 4096
    assert o.recalibrate_probe(n, n, 0.3 / n, 1.0, 100) == (100, False)              # B1 = B*: m' = m
    assert o.recalibrate_probe(n, n, 0.3 * 1.25 / n, 1.0, 100) == (125, False)       # edge of the band: keep
    assert o.recalibrate_probe(n, n, 0.3 * 1.26 / n, 1.0, 100) == (126, True)        # outside: rebuild
    assert o.recalibrate_probe(n, n, 0.3 * 0.8 / n, 1.0, 100) == (80, False)         # m / 1.25 exactly: keep
    assert o.recalibrate_probe(n, n, 0.3 * 0.79 / n, 1.0, 100) == (79, True)
    assert o.recalibrate_probe(n, n, 1e-9, 1.0, 100) == (48, True)                   # floor m_comb
    assert o.recalibrate_probe(n, n, 1.0, 1.0, 100) == (1024, True)                  # cap m_max
    for bad in (float("nan"), 0.0, -1.0, float("inf")):
        assert o.recalibrate_probe(n, n, bad, 1.0, 100) == (100, False)
        assert o.recalibrate_probe(n, n, 1e-4, bad, 100) == (100, False)
