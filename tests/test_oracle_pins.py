"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests compares the oracle with itself: each checks a routine against brute
force on tiny integer inputs, a closed form, an invariant stated in the paper, or a value the
paper prints.
"""
import math
import os

import numpy as np
import pytest

import oracle as O
from paper_2609_19758_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _int_case(n1, n2, n3, seed, nfaults=0):
    A, B = W.operands("integer", n1, n2, n3, W.FP16, seed, lim=8)
    A, B = A.double().numpy(), B.double().numpy()
    C = A @ B
    g = np.random.default_rng(seed)
    faults = []
    for _ in range(nfaults):
        i, j, d = int(g.integers(n1)), int(g.integers(n3)), float(g.integers(1, 9) * (1 if g.integers(2) else -1))
        C[i, j] += d
        faults.append((i, j, d))
    return A, B, C, faults


# ---------------------------------------------------------------- Eq. (S): brute force
def _brute_sketches(A, B, C, h1, v1, h2, v2, m_b):
    """Triple loop over the definition: E_ij by a k loop, then bucket sums with 1-based weights."""
    n1, n2 = A.shape
    n3 = B.shape[1]
    p1 = 1
    while p1 < n1:
        p1 *= 2
    p3 = 1
    while p3 < n3:
        p3 *= 2
    S = np.zeros((m_b, m_b))
    R = np.zeros((m_b, m_b))
    T = np.zeros((m_b, m_b))
    for i in range(n1):
        for j in range(n3):
            e = 0.0
            for k in range(n2):
                e += A[i, k] * B[k, j]
            e -= C[i, j]
            sg = v1[i] * v2[j]
            S[h1[i], h2[j]] += sg * e
            R[h1[i], h2[j]] += sg * e * (i + 1) / p1
            T[h1[i], h2[j]] += sg * e * (j + 1) / p3
    return S, R, T


@pytest.mark.parametrize("n1,n2,n3,m_b,seed", [(7, 5, 9, 3, 1), (16, 12, 16, 4, 2), (13, 16, 6, 2, 3), (1, 3, 1, 1, 4)])
def test_sketch_definition_equals_brute_force_and_compressed_form(n1, n2, n3, m_b, seed):
    A, B, C, _ = _int_case(n1, n2, n3, seed, nfaults=3)
    h1, v1 = O.hash_round(99, 0, 0, n1, m_b)
    h2, v2 = O.hash_round(99, 0, 1, n3, m_b)
    E = O.error_matrix(A, B, C)
    S, R, T = O.moment_sketches(E, h1, v1, h2, v2, m_b)
    Sb, Rb, Tb = _brute_sketches(A, B, C, h1, v1, h2, v2, m_b)
    # integer data and dyadic weights: every sum is exact in FP64
    assert np.array_equal(S, Sb) and np.array_equal(R, Rb) and np.array_equal(T, Tb)
    Sc, Rc, Tc = O.moment_sketches_compressed(A, B, C, h1, v1, h2, v2, m_b)
    assert np.array_equal(S, Sc) and np.array_equal(R, Rc) and np.array_equal(T, Tc)


def test_probe_sketch_is_column_sum_of_E_and_needs_no_product():
    A, B, C, faults = _int_case(11, 7, 13, 5, nfaults=2)
    s = O.probe_sketch(O.error_matrix(A, B, C))
    # brute force: column sums of the injected changes (E = AB - C = -change)
    want = np.zeros(13)
    for (i, j, d) in faults:
        want[j] -= d
    assert np.array_equal(s, want)
    assert np.array_equal(O.probe_sketch_from_operands(A, B, C), want)


# ---------------------------------------------------------------- Eq. (recover)
@pytest.mark.parametrize("n1,n3,m_b", [(16, 16, 4), (13, 21, 3), (100, 37, 8)])
def test_single_fault_ratio_gives_exact_one_based_index(n1, n3, m_b):
    A, B, C, _ = _int_case(n1, 6, n3, 7)
    i0, j0, d = n1 - 3, 2, 5.0
    C[i0, j0] += d
    E = O.error_matrix(A, B, C)
    h1, v1 = O.hash_round(5, 1, 0, n1, m_b)
    h2, v2 = O.hash_round(5, 1, 1, n3, m_b)
    S, R, T = O.moment_sketches(E, h1, v1, h2, v2, m_b)
    a, b = h1[i0], h2[j0]
    p1 = 2 ** math.ceil(math.log2(n1))
    p3 = 2 ** math.ceil(math.log2(n3))
    assert p1 * R[a, b] / S[a, b] == i0 + 1
    assert p3 * T[a, b] / S[a, b] == j0 + 1
    assert abs(S[a, b]) == d
    # every other bucket is empty
    S[a, b] = 0
    assert not S.any()
    # and the full localizer returns exactly that entry with delta = -d
    F = O.localize(A, B, C, seed=5, m_b=m_b, dtype=W.FP16, params=O.Params(radius=0))
    assert [(f.i, f.j, f.delta) for f in F] == [(i0, j0, -d)]


def test_weights_are_one_based_scaled_by_power_of_two():
    w = O.index_weights(5)            # ceil(log2 5) = 3
    assert np.array_equal(w, np.array([1, 2, 3, 4, 5]) / 8.0)
    assert O.index_weights(8)[-1] == 1.0 and O.index_weights(9)[-1] == 9 / 16
    assert np.array_equal(O.index_weights(1), [1.0])
    # "no term of R is larger than the corresponding term of S"
    assert np.all(O.index_weights(4097) <= 1.0)


# ---------------------------------------------------------------- clean products
def test_clean_integer_product_is_clean():
    A, B, C, _ = _int_case(24, 9, 20, 11)
    E = O.error_matrix(A, B, C)
    assert not E.any()
    v = O.probe_verdict(O.probe_sketch(E), O.analytic_tau(A, B, 9), n_rows=24)
    assert not v.fired and not v.nonfinite and v.thr == 0.0
    assert O.localize(A, B, C, seed=3, m_b=4, dtype=W.FP16, params=O.Params(radius=2)) == []


def test_clean_fp32_product_reports_nothing_and_lemma1_scan():
    A, B = W.operands("uniform", 48, 64, 40, W.FP16, 21)
    C = W.cpu_fp32_product(A, B).numpy()
    A, B = A.double().numpy(), B.double().numpy()
    # Lemma 1: on a clean product no position at all passes validation
    for i in range(48):
        for j in range(40):
            ok, gamma, tau_ij = O.validate_entry(A, B, C, i, j)
            assert not ok
    st = {}
    F = O.localize(A, B, C, seed=8, m_b=4, dtype=W.FP16, params=O.Params(radius=3), stats=st)
    assert F == []
    v = O.probe_verdict(O.probe_sketch(O.error_matrix(A, B, C)), O.analytic_tau(A, B, 64), n_rows=48)
    assert not v.fired


def test_probe_flags_nonfinite_sketch():
    s = np.zeros(64)
    s[5] = np.nan
    v = O.probe_verdict(s, tau=1.0)
    assert v.fired and v.nonfinite
    s[5] = np.inf
    assert O.probe_verdict(s, tau=1.0).fired


def test_probe_threshold_formula_on_known_vector():
    # |s| all equal to x: mean|s| = x, no clipping, sigma_hat = 1.2533 x; N_b = 100
    s = np.full(100, 0.5) * np.where(np.arange(100) % 2, 1, -1)
    v = O.probe_verdict(s, tau=1e9)
    assert v.sigma_hat == pytest.approx(1.2533 * 0.5, rel=1e-12)
    assert v.thr == pytest.approx(4 * math.sqrt(2 * math.log(100)) * 1.2533 * 0.5, rel=1e-12)
    assert not v.fired          # 0.5 < thr
    assert O.probe_verdict(s, tau=0.4).fired and O.probe_verdict(s, tau=0.4).thr == 0.4
    # a sketch entry that sums n_rows entries of E: the analytic cap grows like sqrt(n_rows)
    assert O.probe_verdict(s, tau=0.1, n_rows=16).thr == pytest.approx(0.4) and O.probe_verdict(s, tau=0.1, n_rows=16).fired
    assert not O.probe_verdict(s, tau=0.2, n_rows=16).fired
    # one outlier is clipped at 5 mean|s| in the estimate
    s2 = np.ones(10)
    s2[0] = 91.0                      # mean|s| = 10, clip at 50
    assert O.sigma_clip(s2) == pytest.approx(1.2533 * (50 + 9) / 10, rel=1e-12)


def test_analytic_tau():
    A = np.array([[0.5, -3.0]])
    B = np.array([[2.0], [-0.25]])
    assert O.analytic_tau(A, B, 2) == 100 * 2 * 2.0 ** -23 * 3.0 * 2.0


# ---------------------------------------------------------------- noise estimators: Gaussian closed forms
def test_estimators_on_gaussian_noise():
    g = np.random.default_rng(0)
    sigma = 3.0
    x = g.standard_normal(400_000) * sigma
    # E|x| = sigma sqrt(2/pi) and clipping at 5 mean|x| ~ 4 sigma removes < 1e-4: clip-mean -> sigma
    assert O.sigma_clip(x) == pytest.approx(sigma, rel=5e-3)
    # signed MAD is the textbook consistent estimator
    assert O.sigma_mad(x, of_abs=0) == pytest.approx(sigma, rel=5e-3)
    # MAD of |x| as printed: median|x| = 0.6745 sigma and d with
    # Phi(0.6745+d) - Phi(0.6745-d) = 1/2 (x>0 branch), i.e. 1.4826 d = 0.592 sigma
    from scipy.stats import norm
    from scipy.optimize import brentq
    q = norm.ppf(0.75)
    # the half-normal |x|/sigma has CDF 2 Phi(t) - 1; P(| |x| - q | <= d) = 1/2
    f = lambda d: (2 * norm.cdf(q + d) - 1) - (2 * norm.cdf(max(q - d, 0.0)) - 1) - 0.5
    d = brentq(f, 1e-6, 3.0)
    assert 1.4826 * d == pytest.approx(0.592, abs=2e-3)
    assert O.sigma_mad(x, of_abs=1) == pytest.approx(1.4826 * d * sigma, rel=1e-2)
    # fraction of clean buckets above 2 sigma_MAD: 4.55 % for the signed form
    frac = np.mean(np.abs(x) > 2 * O.sigma_mad(x, of_abs=0))
    assert frac == pytest.approx(2 * (1 - norm.cdf(2.0)), abs=2e-3)
    # estimator constants are the Gaussian-consistent ones
    assert 1.2533 == pytest.approx(math.sqrt(math.pi / 2), abs=5e-5)
    assert 1.4826 == pytest.approx(1 / norm.ppf(0.75), abs=5e-5)


def test_lower_median():
    assert O.lower_median([4, 1, 3, 2]) == 2
    assert O.lower_median([5, 1, 3]) == 3
    assert O.lower_median([7]) == 7


# ---------------------------------------------------------------- hash rounds
def test_hash_rounds_uniform_independent_balanced():
    n, m_b = 40000, 64
    h, v = O.hash_round(1234567890123, 0, 0, n, m_b)
    assert h.min() >= 0 and h.max() < m_b and set(np.unique(v)) == {-1.0, 1.0}
    occ = np.bincount(h, minlength=m_b)
    chi2 = ((occ - n / m_b) ** 2 / (n / m_b)).sum()
    assert chi2 < 63 + 6 * math.sqrt(2 * 63)            # chi-square(63): mean 63, sd 11.2
    assert abs(v.sum()) < 5 * math.sqrt(n)               # sign balance
    # signs independent of buckets: per-bucket sign sums are small
    per = np.bincount(h, weights=v, minlength=m_b)
    assert np.all(np.abs(per) < 6 * np.sqrt(occ))
    # rounds and sides differ: agreement of two rounds' buckets ~ 1/m_b (Lemma 2's 1/m)
    for (r2, s2) in [(1, 0), (2, 0), (0, 1)]:
        h2, v2 = O.hash_round(1234567890123, r2, s2, n, m_b)
        agree = np.mean(h == h2)
        assert abs(agree - 1 / m_b) < 5 * math.sqrt((1 / m_b) / n)
        assert abs(np.mean(v == v2) - 0.5) < 5 * 0.5 / math.sqrt(n)
    # a different seed gives a different table
    h3, _ = O.hash_round(1234567890124, 0, 0, n, m_b)
    assert np.mean(h == h3) < 0.05


def test_pair_collision_rate_matches_lemma2():
    # two fixed rows collide with probability 1/m over the draw of the hash
    m_b, hits, trials = 16, 0, 4000
    for seed in range(trials):
        h, _ = O.hash_round(seed * 7919 + 13, 0, 0, 64, m_b)
        hits += int(h[3] == h[41])
    p = hits / trials
    assert abs(p - 1 / m_b) < 5 * math.sqrt((1 / m_b) * (1 - 1 / m_b) / trials)


def test_mix32_known_properties():
    # bijection on a sample (distinct inputs -> distinct outputs), zero is a fixed point of
    # multiply/xor-shift mixers, and avalanche: one input bit flips about half the output bits
    x = np.arange(1, 100000, dtype=np.uint64)
    y = O.mix32(x)
    assert len(np.unique(y)) == len(x)
    assert int(O.mix32(0)) == 0
    flips = O.mix32(x) ^ O.mix32(x ^ np.uint64(1 << 7))
    bits = np.array([bin(int(f)).count("1") for f in flips[:5000]])
    assert abs(bits.mean() - 16) < 0.5


# ---------------------------------------------------------------- selection / search order
def test_candidate_selection_order_and_cap():
    S = np.array([[0.0, 3.0, -3.0], [5.0, 1.0, np.nan], [np.inf, -2.0, 0.5]])
    idx = O.select_candidates(S, thr=0.9, K=64)
    # inf first, then 5, then the tie |3| by ascending flat index, then 2, then 1; NaN never
    assert list(idx) == [6, 3, 1, 2, 7, 4]
    assert list(O.select_candidates(S, thr=0.9, K=3)) == [6, 3, 1]
    U = O.decode_candidates(S, S, S, idx, 4, 4)
    assert [u[0] for u in U] == [3, 1, 2, 7, 4]           # the inf bucket is dropped from U


def test_search_offsets_order():
    offs = O.search_offsets(2)
    assert len(offs) == 25 and offs[0] == (0, 0)
    cheb = [max(abs(a), abs(b)) for a, b in offs]
    assert cheb == sorted(cheb)
    ring1 = offs[1:9]
    assert [abs(a) + abs(b) for a, b in ring1] == [1, 1, 1, 1, 2, 2, 2, 2]
    assert O.search_offsets(0) == [(0, 0)]
    assert O.cap_K(O.Params(s_budget=16)) == 128 and O.cap_K(O.Params()) == 64


# ---------------------------------------------------------------- multi-fault recovery with peeling
def test_colliding_faults_are_separated_by_later_rounds():
    n1, n2, n3, m_b = 32, 8, 32, 4
    A, B, C, _ = _int_case(n1, n2, n3, 17)
    # 6 faults, three of them in one row: with m_b = 4 some share a bucket in some round
    coords = [(5, 1), (5, 9), (5, 30), (17, 9), (28, 3), (2, 22)]
    for t, (i, j) in enumerate(coords):
        C[i, j] += 3.0 + t
    F = O.localize(A, B, C, seed=2024, m_b=m_b, dtype=W.FP16, params=O.Params(radius=1, rounds=6))
    got = {(f.i, f.j): f.delta for f in F}
    # zero false positives by construction, and every reported delta is exact
    for (i, j), d in got.items():
        assert (i, j) in coords and d == -(3.0 + coords.index((i, j)))
    assert len(got) >= 4


def test_recovery_over_rounds_bound_theorem2():
    """Thm 2: with m >= 3 c Delta and m^2 >= 3 c s, k rounds recover everything with
    probability >= 1 - s c^-k.  Monte Carlo on exact integer products (c=2, s=4, Delta=2)."""
    n1 = n3 = 64
    m_b, s, k = 12, 4, 3
    miss_trials = 0
    trials = 60
    for t in range(trials):
        A, B, C, _ = _int_case(n1, 4, n3, 100 + t)
        g = np.random.default_rng(t)
        coords = set()
        row = int(g.integers(n1))
        coords.add((row, int(g.integers(n3))))
        while len(coords) < 2:
            coords.add((row, int(g.integers(n3))))
        while len(coords) < s:
            coords.add((int(g.integers(n1)), int(g.integers(n3))))
        for (i, j) in coords:
            C[i, j] += float(g.integers(1, 6))
        F = O.localize(A, B, C, seed=t, m_b=m_b, dtype=W.FP16, params=O.Params(radius=0, rounds=k))
        assert {(f.i, f.j) for f in F} <= coords
        miss_trials += int(len(F) < s)
    assert miss_trials / trials <= s * 2.0 ** -k


# ---------------------------------------------------------------- peeling, pinned directly
def _fault_only_sketch(faults, h1, v1, h2, v2, m_b, n1, n3):
    """Sketches of an error matrix that is zero except E_ij = e at the listed (i, j, e):
    written out term by term, 1-based weights over the next power of two."""
    p1 = 1
    while p1 < n1:
        p1 *= 2
    p3 = 1
    while p3 < n3:
        p3 *= 2
    S = np.zeros((m_b, m_b))
    R = np.zeros((m_b, m_b))
    T = np.zeros((m_b, m_b))
    for (i, j, e) in faults:
        sg = v1[i] * v2[j]
        S[h1[i], h2[j]] += sg * e
        R[h1[i], h2[j]] += sg * e * (i + 1) / p1
        T[h1[i], h2[j]] += sg * e * (j + 1) / p3
    return S, R, T


@pytest.mark.parametrize("n1,n3,m_b,seed", [(24, 40, 3, 5), (64, 64, 8, 6), (17, 9, 2, 7)])
def test_peel_removes_exactly_what_a_confirmed_fault_put_into_the_sketches(n1, n3, m_b, seed):
    """Algorithm 1, peeling loop; Section "Peeling Across Hash Rounds".  On an exact integer product the
    sketches hold nothing but the faults, so peeling all of them must leave exact zeros in S, R and T, and
    peeling a subset must leave the sketches of the others (every value is a dyadic rational: exact)."""
    n2 = 6
    A, B, C, _ = _int_case(n1, n2, n3, seed)
    g = np.random.default_rng(seed)
    coords = set()
    row = int(g.integers(n1))
    while len(coords) < 3:                      # three in one row: some share a row bucket
        coords.add((row, int(g.integers(n3))))
    while len(coords) < 7:
        coords.add((int(g.integers(n1)), int(g.integers(n3))))
    written = []
    for t, (i, j) in enumerate(sorted(coords)):
        d = float((t + 1) * (1 if t % 2 else -1))
        C[i, j] += d
        written.append((i, j, d))
    E = O.error_matrix(A, B, C)
    for rnd in (0, 1):
        h1, v1 = O.hash_round(99, rnd, 0, n1, m_b)
        h2, v2 = O.hash_round(99, rnd, 1, n3, m_b)
        # the correction of a fault written as C_ij += d is delta = gamma - C_ij = -d
        F = [O.Fault(i, j, -d, 0.0, 0.0, 0, -1, -1) for (i, j, d) in written]
        S, R, T = O.moment_sketches(E, h1, v1, h2, v2, m_b)
        assert np.count_nonzero(S) > 0
        O.peel(S, R, T, F, h1, v1, h2, v2, n1, n3)
        assert not S.any() and not R.any() and not T.any()
        for keep in (1, 3, 6):
            S, R, T = O.moment_sketches(E, h1, v1, h2, v2, m_b)
            O.peel(S, R, T, F[keep:], h1, v1, h2, v2, n1, n3)
            Sx, Rx, Tx = _fault_only_sketch([(i, j, -d) for (i, j, d) in written[:keep]], h1, v1, h2, v2, m_b, n1, n3)
            assert np.array_equal(S, Sx) and np.array_equal(R, Rx) and np.array_equal(T, Tx)


# ---------------------------------------------------------------- normalisation of the noise constant
def test_noise_constant_normalisation_on_a_known_error_matrix():
    """Eq. (sigma) normalises the bucket noise as sigma m / (2^-24 sqrt(n1 n2 n3) rms(C)).  Feed the
    measurement an error matrix of i.i.d. N(0, s^2) entries and a constant C: a bucket that sums c entries
    is N(0, c s^2), the clipped mean of a Gaussian is its sigma (clipping at 5 mean|x| = 4 sigma removes
    1e-4), so c_hat has a closed form in s, the bucket populations and the constant."""
    n1, n2, n3, m0 = 3072, 8, 2048, 160
    s_e, c0 = 3.0e-4, 2.5
    g = np.random.default_rng(20)
    E = s_e * g.standard_normal((n1, n3))
    A = np.zeros((n1, n2))
    B = np.zeros((n2, n3))
    C = np.full((n1, n3), c0, dtype=np.float32)
    nz = O.measure_noise(A, B, C, seed=5, dtype=O.BF16, m0=m0, E=E)
    assert nz.m0 == m0 and nz.rms_c == c0
    h1, _ = O.hash_round(5, 0, 0, n1, m0)
    h2, _ = O.hash_round(5, 0, 1, n3, m0)
    pop = np.outer(np.bincount(h1, minlength=m0), np.bincount(h2, minlength=m0)).astype(float)
    sigma_expected = 1.2533 * math.sqrt(2.0 / math.pi) * s_e * np.sqrt(pop).mean()
    assert nz.sigma_clip == pytest.approx(sigma_expected, rel=1e-2)
    c_expected = sigma_expected * m0 / (2.0 ** -24 * math.sqrt(float(n1) * n2 * n3) * c0)
    assert nz.c_hat == pytest.approx(c_expected, rel=1e-2)
    # and against the plain population n1 n3 / m0^2 (the sqrt of a varying count loses under 2 %)
    plain = s_e * math.sqrt(n1 * n3) / (2.0 ** -24 * math.sqrt(float(n1) * n2 * n3) * c0)
    assert nz.c_hat == pytest.approx(plain, rel=3e-2)


# ---------------------------------------------------------------- the tolerance denominators
def test_abs_product_and_abs_sketch_brute_force():
    g = np.random.default_rng(8)
    n1, n2, n3, m_b = 9, 5, 11, 3
    A = g.integers(-4, 5, (n1, n2)).astype(float)
    B = g.integers(-4, 5, (n2, n3)).astype(float)
    h1, _ = O.hash_round(3, 0, 0, n1, m_b)
    h2, _ = O.hash_round(3, 0, 1, n3, m_b)
    ABS = O.abs_product(A, B)
    want = np.zeros((n1, n3))
    wantS = np.zeros((m_b, m_b))
    for i in range(n1):
        for j in range(n3):
            for k in range(n2):
                want[i, j] += abs(A[i, k]) * abs(B[k, j])
            wantS[h1[i], h2[j]] += want[i, j]
    assert np.array_equal(ABS, want)
    assert np.array_equal(O.abs_sketch(ABS, h1, h2, m_b), wantS)
    assert ABS.min() >= 0 and O.abs_sketch(ABS, h1, h2, m_b).sum() == want.sum()
