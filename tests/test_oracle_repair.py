"""Pins of the oracle's Algorithm 2 (scan, absolute repairs, apply, second probe) against exact
integer products, where the repaired matrix must equal the true product bit for bit."""
import numpy as np
import pytest

import oracle as O
from paper_2609_19758_b200 import workloads as W


def _int(n1, n2, n3, seed):
    A, B = W.operands("integer", n1, n2, n3, W.FP16, seed, lim=8)
    A, B = A.double().numpy(), B.double().numpy()
    return A, B, (A @ B).astype(np.float32)


def test_scan_finds_exactly_the_out_of_range_entries_in_row_major_order():
    C = np.zeros((5, 7), dtype=np.float32)
    C[3, 2] = np.nan
    C[0, 6] = np.inf
    C[4, 0] = -np.inf
    C[2, 2] = np.float32(O.FP32_MAX / 8)        # finite but beyond fp32max / 16
    C[1, 1] = np.float32(O.FP32_MAX / 32)       # large but in range
    assert O.scan_out_of_range(C, 64) == [(0, 6), (2, 2), (3, 2), (4, 0)]
    assert O.scan_out_of_range(C, 2) == [(0, 6), (2, 2)]


def test_clean_product_is_left_alone():
    A, B, C = _int(24, 9, 20, 1)
    out, F, rep = O.verify_repair(A, B, C, 3, O.FP16, O.Params(radius=1), m_b=4)
    assert rep["state"] == 0 and F == [] and np.array_equal(out, C)


def test_nonfinite_and_finite_faults_sharing_a_row_are_all_repaired():
    """An Inf and a NaN poison their bucket rows in a linear sketch; with the exact scan the
    finite faults next to them are still found, and C comes back equal to the true product."""
    A, B, C0 = _int(32, 8, 32, 7)
    C = C0.copy()
    C[5, 3] = np.nan
    C[5, 20] += 6.0           # same row as the NaN
    C[11, 9] = np.inf
    C[30, 9] -= 4.0           # same column as the Inf
    C[17, 17] = np.float32(-O.FP32_MAX / 4)
    C[2, 2] += 3.0
    out, F, rep = O.verify_repair(A, B, C, 2024, O.FP16, O.Params(radius=1, rounds=6), m_b=6)
    assert rep["first_probe"].fired and rep["first_probe"].nonfinite
    assert rep["n_absolute"] == 3 and rep["state"] == 1 and not rep["second_probe"].fired
    assert {(f.i, f.j) for f in F} == {(5, 3), (5, 20), (11, 9), (30, 9), (17, 17), (2, 2)}
    assert np.array_equal(out, C0)
    ab = {(f.i, f.j): f for f in F if f.round < 0}
    assert set(ab) == {(5, 3), (11, 9), (17, 17)}
    for (i, j), f in ab.items():
        assert f.delta == C0[i, j] and (f.bucket_a, f.bucket_b) == (-1, -1)
    fin = {(f.i, f.j): f.delta for f in F if f.round >= 0}
    assert fin == {(5, 20): -6.0, (30, 9): 4.0, (2, 2): -3.0}


def test_apply_corrections_modes():
    C = np.array([[1.0, 2.0], [3.0, np.nan]], dtype=np.float32)
    F = [O.Fault(0, 1, 0.5, 2.5, 2.0, 0, 0, 0), O.Fault(1, 1, 7.0, 7.0, float("nan"), -1, -1, -1)]
    out = O.apply_corrections(C, F)
    assert np.array_equal(out, np.array([[1.0, 2.5], [3.0, 7.0]], dtype=np.float32))
    assert np.isnan(C[1, 1])          # the input is not modified


def test_unrepairable_product_is_reported_for_recompute():
    """More faults in one row than the rounds can separate with 2 buckets and no search radius:
    whatever is left makes the second probe fire and the state says 'recompute'."""
    A, B, C0 = _int(16, 6, 16, 5)
    C = C0.copy()
    for j in range(0, 16, 2):
        C[3, j] += 2.0 + j
    out, F, rep = O.verify_repair(A, B, C, 1, O.FP16, O.Params(radius=0, rounds=1), m_b=2)
    assert rep["state"] in (1, 2)
    if rep["state"] == 2:
        assert rep["second_probe"].fired and not np.array_equal(out, C0)
    # never a wrong repair: every reported entry was corrupted, and repaired ones are exact
    for f in F:
        assert f.i == 3 and f.j % 2 == 0 and out[f.i, f.j] == C0[f.i, f.j]
